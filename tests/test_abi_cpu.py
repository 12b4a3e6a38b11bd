"""Host-side checks of the C interface: the library loads without a GPU, exports every declared
symbol, packs bit-identically to the oracle's own packer, and reports errors through status codes."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import paper_2310_19509_b200 as sbnn
from paper_2310_19509_b200 import build as sbnn_build
from oracle import reference as R
from sbnn_inputs import expand_mask, group_mask_balanced, group_mask_layer_global, tap_pattern_mask, dw_pattern_mask

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    sbnn_build.build()


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "sbnn.h")).read()
    names = sorted(set(re.findall(r"\b(sbnn_[a-z0-9_]+)\s*\(", hdr)))
    assert "sbnn_pack_weights" in names and "sbnn_conv1x1_gs" in names and "sbnn_mobilenet_v1_forward" in names
    L = sbnn.lib()
    for n in names:
        assert hasattr(L, n), f"{n} declared in sbnn.h but not exported"


def test_status_strings():
    assert sbnn.status_str(0) == "SBNN_OK"
    assert sbnn.status_str(4) == "SBNN_ERR_MASK_NOT_GROUP_UNIFORM"
    assert sbnn.status_str(99) == "SBNN_ERR_UNKNOWN"


@pytest.mark.parametrize("k,g,cin,cout,mode", [(1, 4, 64, 128, "bal"), (1, 8, 32, 64, "bal"), (3, 4, 16, 32, "bal"),
                                               (1, 1, 12, 5, "glob"), (1, 2, 20, 8, "glob"), (1, 16, 8, 32, "bal"),
                                               (3, 2, 8, 8, "glob")])
def test_pack_is_bit_identical_to_oracle_pack(k, g, cin, cout, mode):
    rng = np.random.default_rng(7)
    w = rng.standard_normal((cout, k, k, cin)).astype(np.float32)
    b = rng.standard_normal(cout).astype(np.float32)
    ng = cout // g
    um = group_mask_balanced(1, 3, ng, cin, 50) if mode == "bal" else group_mask_layer_global(1, 3, ng, cin, 60)
    m = expand_mask(um, g, k, k)
    p = sbnn.pack_weights(w, m, b, g)
    v = p.view()
    gp, idx, val = R.pack(w, m, g)
    assert v["nnz_units"] == len(idx) and v["ngroups"] == ng and v["G"] == g
    assert np.array_equal(v["group_ptr"], gp) and v["group_ptr"].dtype == np.int32
    assert np.array_equal(v["idx"], idx)
    assert v["val"].tobytes() == val.tobytes()
    assert v["bias"].tobytes() == b.tobytes()
    w2, m2 = p.unpack()
    assert np.array_equal(m2, m) and (w2.tobytes() == np.where(m != 0, w, np.float32(0)).tobytes())
    p.free()


@pytest.mark.parametrize("g,cin,cout,kept_taps", [(4, 16, 32, 4), (2, 8, 8, 4), (1, 6, 5, 6), (8, 8, 16, 1)])
def test_pattern_pack_is_bit_identical_to_oracle_pack(g, cin, cout, kept_taps):
    """3x3 kernels pruned tap by tap (one pattern per group and input channel): kept taps, zeros elsewhere, and the
    tap masks must equal the oracle's own packing; unpacking returns the mask exactly."""
    rng = np.random.default_rng(17)
    w = rng.standard_normal((cout, 3, 3, cin)).astype(np.float32)
    ng = cout // g
    um = group_mask_balanced(2, 3, ng, cin, 50)
    m = tap_pattern_mask(2, 19, um, g, kept_taps)
    assert m.reshape(ng, g, 9, cin).sum(axis=2).max() == kept_taps and m[:, 1, 1, :].sum() == um.sum() * g
    p = sbnn.pack_weights(w, m, None, g, tap_patterns=True)
    v = p.view()
    gp, idx, val, tm = R.pack_pattern(w, m, g)
    assert np.array_equal(v["group_ptr"], gp) and np.array_equal(v["idx"], idx)
    assert v["val"].tobytes() == val.tobytes()
    assert v["tap_mask"].dtype == np.uint16 and np.array_equal(v["tap_mask"], tm)
    assert all(bin(int(t)).count("1") == kept_taps and (int(t) >> 4) & 1 for t in tm)
    w2, m2 = p.unpack()
    assert np.array_equal(m2, m) and (w2.tobytes() == np.where(m != 0, w, np.float32(0)).tobytes())
    p.free()
    # the connectivity-only packer refuses such a mask, and a plain unit mask packs the same either way
    with pytest.raises(sbnn.SbnnError) as e:
        sbnn.pack_weights(w, m, None, g)
    assert e.value.code == 4
    if g > 1:
        bad = m.copy()
        c0 = int(np.flatnonzero(um[0])[0])
        bad[1, 0, 0, c0] ^= 1                      # one filter of the group deviates from the shared pattern
        with pytest.raises(sbnn.SbnnError) as e:
            sbnn.pack_weights(w, bad, None, g, tap_patterns=True)
        assert e.value.code == 4
    mu = expand_mask(um, g, 3, 3)
    a, b = sbnn.pack_weights(w, mu, None, g).view(), sbnn.pack_weights(w, mu, None, g, tap_patterns=True).view()
    assert a["val"].tobytes() == b["val"].tobytes() and np.array_equal(a["idx"], b["idx"]) and a["tap_mask"] is None
    assert np.all(b["tap_mask"] == 0x1FF)


@pytest.mark.parametrize("c,go,by_magnitude", [(64, 16, False), (24, 8, True), (12, 4, False), (160, 16, True)])
def test_dw_pattern_pack_is_bit_identical_to_oracle_pack(c, go, by_magnitude):
    """3:9 depthwise patterns: PatternInfo and the six surviving weights per channel equal the oracle's own packing."""
    rng = np.random.default_rng(23)
    w = rng.standard_normal((3, 3, c)).astype(np.float32)
    m = dw_pattern_mask(3, 5, c, go, w if by_magnitude else None)
    assert np.all(m.sum(axis=(0, 1)) == 6) and np.all(m[:, 1] == 1)
    if c // go >= 8 and not by_magnitude:
        assert len({tuple(m[:, :, b * go].reshape(-1)) for b in range(c // go)}) > 1      # blocks differ
    pat, w6 = sbnn.pack_dw_pattern(w, m, go)
    rpat, rw6 = R.pack_dw_pattern(w, m, go)
    assert np.array_equal(pat, rpat) and w6.tobytes() == rw6.tobytes()
    # what the compact form stands for: the masked dense weights
    dense = np.zeros_like(w)
    for b in range(c // go):
        for kh in range(3):
            side = 0 if (pat[b] >> kh) & 1 else 2
            dense[kh, side, b * go:(b + 1) * go] = w6[kh, 0, b * go:(b + 1) * go]
            dense[kh, 1, b * go:(b + 1) * go] = w6[kh, 1, b * go:(b + 1) * go]
    assert dense.tobytes() == np.where(m != 0, w, np.float32(0)).tobytes()
    # not a 3:9 pattern / not uniform inside a block / bad block size
    for bad in ("middle", "both", "deviate"):
        mb = m.copy()
        if bad == "middle":
            mb[1, 1, 0] = 0
        elif bad == "both":
            mb[0, 0, :go] = 1
            mb[0, 2, :go] = 1
        else:
            mb[2, 0, 1], mb[2, 2, 1] = mb[2, 2, 1], mb[2, 0, 1]
        with pytest.raises(sbnn.SbnnError) as e:
            sbnn.pack_dw_pattern(w, mb, go)
        assert e.value.code == 4
    with pytest.raises(sbnn.SbnnError) as e:
        sbnn.pack_dw_pattern(w, m, 5)
    assert e.value.code == 3


def test_pack_edge_cases():
    w = np.ones((8, 1, 1, 8), np.float32)
    # a group with no kept unit, a group with all units
    m = np.zeros((8, 1, 1, 8), np.uint8)
    m[4:8] = 1
    v = sbnn.pack_weights(w, m, None, 4).view()
    assert v["group_ptr"].tolist() == [0, 0, 8] and v["idx"].tolist() == list(range(8))
    assert not v["bias"].any()
    # a kept weight that is numerically zero stays stored
    w0 = w.copy()
    w0[4:8, 0, 0, 3] = 0.0
    v = sbnn.pack_weights(w0, m, None, 4).view()
    assert v["nnz_units"] == 8 and not v["val"][3].any()


def test_pack_errors():
    w = np.ones((8, 1, 1, 8), np.float32)
    m = np.ones((8, 1, 1, 8), np.uint8)
    bad = m.copy()
    bad[1, 0, 0, 3] = 0
    with pytest.raises(sbnn.SbnnError) as e:
        sbnn.pack_weights(w, bad, None, 4)
    assert e.value.name == "SBNN_ERR_MASK_NOT_GROUP_UNIFORM" and "group 0" in e.value.detail
    two = m.copy()
    two[0:4, 0, 0, 0] = 2
    with pytest.raises(sbnn.SbnnError) as e:
        sbnn.pack_weights(w, two, None, 4)
    assert e.value.name == "SBNN_ERR_MASK_NOT_GROUP_UNIFORM"
    m3 = np.ones((8, 3, 3, 8), np.uint8)
    m3[0:4, 1, 1, 2] = 0
    with pytest.raises(sbnn.SbnnError) as e:
        sbnn.pack_weights(np.ones((8, 3, 3, 8), np.float32), m3, None, 4)
    assert e.value.name == "SBNN_ERR_MASK_NOT_GROUP_UNIFORM"
    for g, name in [(3, "SBNN_ERR_GROUP"), (16, "SBNN_ERR_GROUP"), (0, "SBNN_ERR_GROUP")]:
        with pytest.raises(sbnn.SbnnError) as e:
            sbnn.pack_weights(w, m, None, g)
        assert e.value.name == name
    with pytest.raises(sbnn.SbnnError) as e:
        sbnn.pack_weights(np.ones((8, 2, 2, 8), np.float32), np.ones((8, 2, 2, 8), np.uint8), None, 4)
    assert e.value.name == "SBNN_ERR_SHAPE"
    L = sbnn.lib()
    h = C.c_void_p()
    assert L.sbnn_pack_weights(None, m.ctypes.data, None, 8, 1, 1, 8, 4, C.byref(h)) == 1
    assert L.sbnn_packed_free(None) == 0
    assert L.sbnn_packed_get(None, None) == 1


def test_compute_calls_validate_before_touching_a_device():
    """Argument errors are reported by status code; nothing is launched."""
    L = sbnn.lib()
    w = np.ones((8, 1, 1, 8), np.float32)
    m = np.ones((8, 1, 1, 8), np.uint8)
    p = sbnn.pack_weights(w, m, None, 4)
    assert L.sbnn_conv1x1_gs(p.handle, None, None, 1, 1, 1, 0, None) == 1            # NULL
    assert L.sbnn_conv1x1_gs(p.handle, 16, 32, -1, 1, 1, 0, None) == 2               # negative shape
    assert L.sbnn_conv1x1_gs(p.handle, 16, 36, 1, 1, 1, 0, None) == 5                # misaligned
    assert L.sbnn_conv1x1_gs(p.handle, 16, 32, 1, 1, 1, 64, None) == 6               # unknown flag
    assert L.sbnn_conv3x3_gs(p.handle, None, 32, 1, 1, 1, 0, None) != 0
    assert L.sbnn_dwconv3x3(16, None, 16, 32, 1, 4, 4, 6, 1, 0, None) == 6           # C % 4
    assert L.sbnn_dwconv3x3(16, None, 16, 32, 1, 4, 4, 8, 3, 0, None) == 2           # stride
    assert L.sbnn_conv3x3_dense(16, None, 16, 32, 1, 4, 4, 8, 32, 1, 0, None) == 6   # Cin > 4
    assert L.sbnn_avgpool(16, 32, 1, 0, 8, None) == 2
    assert L.sbnn_mobilenet_v1_create(None, None, None, None, None, None, 1, None) == 1
    a, b, c, d = C.c_int(), C.c_int(), C.c_int(), C.c_int()
    assert L.sbnn_mobilenet_v1_layer_shape(29, C.byref(a), C.byref(b), C.byref(c), C.byref(d)) == 2
    assert sbnn.mobilenet_v1_layer_shape(0) == (224, 3, 112, 32)
    assert sbnn.mobilenet_v1_layer_shape(26) == (7, 1024, 7, 1024)
    assert sbnn.mobilenet_v1_layer_shape(28) == (1, 1024, 1, 1000)
    assert b"" == L.sbnn_last_error()[:0]


def test_library_layer_table_matches_oracle_and_generator_tables():
    from sbnn_inputs import mobilenet_v1_shapes
    ot = R.mobilenet_v1_table()
    gt = mobilenet_v1_shapes()
    assert len(ot) == len(gt) == 29
    for i, ((kind, hin, ci, co, s), g) in enumerate(zip(ot, gt)):
        h_in, c_in, h_out, c_out = sbnn.mobilenet_v1_layer_shape(i)
        assert (h_in, c_in, c_out) == (hin, ci, co) == (g["hin"], g["cin"], g["cout"])
        assert g["kind"] == kind and g["stride"] == s
        if kind not in ("pool", "fc"):
            assert h_out == hin // s


def test_header_compiles_as_c99_and_the_binding_mirrors_the_view_struct(tmp_path):
    """include/sbnn.h is a C header: a C99 program that includes it, packs a layer, borrows the view, unpacks and
    frees through the C interface must compile with -Wall -Werror, link against libsbnn.so and run; the size and
    field offsets it prints for sbnn_packed_view must be those of the ctypes mirror in the binding."""
    import subprocess
    from paper_2310_19509_b200 import binding
    src = tmp_path / "use_sbnn.c"
    src.write_text(r'''
#include <stddef.h>
#include <stdio.h>
#include <string.h>
#include "sbnn.h"
int main(void) {
    float w[8 * 8];
    uint8_t m[8 * 8];
    float bias[8] = {0.5f, -1.0f, 0.25f, 2.0f, 0.0f, 1.0f, -2.0f, 3.0f};
    float w2[8 * 8];
    uint8_t m2[8 * 8];
    sbnn_packed* p = NULL;
    sbnn_packed_view v;
    sbnn_status st;
    int o, c, bad = 0;
    for (o = 0; o < 8; ++o)
        for (c = 0; c < 8; ++c) {
            w[o * 8 + c] = (float)(o * 8 + c + 1);
            m[o * 8 + c] = (uint8_t)(((o / 4) + c) % 2);       /* rows 0-3 share a mask, rows 4-7 the other */
        }
    st = sbnn_pack_weights(w, m, bias, 8, 1, 1, 8, 4, &p);
    if (st != SBNN_OK) { printf("pack: %s %s\n", sbnn_status_str(st), sbnn_last_error()); return 1; }
    if (sbnn_packed_get(p, &v) != SBNN_OK) return 2;
    if (v.Cout != 8 || v.Cin != 8 || v.G != 4 || v.ngroups != 2 || v.nnz_units != 8 || v.tap_mask != NULL) return 3;
    if (v.gi != 1 || v.block_idx != NULL) return 12;
    if (v.group_ptr[0] != 0 || v.group_ptr[1] != 4 || v.group_ptr[2] != 8) return 4;
    if (v.idx[0] != 1 || v.idx[3] != 7 || v.idx[4] != 0 || v.idx[7] != 6) return 5;
    if (v.val[0] != w[0 * 8 + 1] || v.val[1] != w[1 * 8 + 1] || v.bias[3] != 2.0f) return 6;
    if (sbnn_unpack_weights(p, w2, m2) != SBNN_OK) return 7;
    for (o = 0; o < 64; ++o) bad += (m2[o] != m[o]) || (w2[o] != (m[o] ? w[o] : 0.0f));
    if (bad) return 8;
    if (sbnn_pack_weights(w, m, bias, 8, 1, 1, 8, 3, &p) != SBNN_ERR_GROUP) return 9;
    if (strlen(sbnn_last_error()) == 0) return 10;
    if (sbnn_packed_free(p) != SBNN_OK) return 11;
    printf("%zu %zu %zu %zu %zu %zu %zu %zu %zu\n", sizeof(sbnn_packed_view), offsetof(sbnn_packed_view, nnz_units),
           offsetof(sbnn_packed_view, group_ptr), offsetof(sbnn_packed_view, idx), offsetof(sbnn_packed_view, val),
           offsetof(sbnn_packed_view, bias), offsetof(sbnn_packed_view, tap_mask), offsetof(sbnn_packed_view, gi),
           offsetof(sbnn_packed_view, block_idx));
    return 0;
}
''')
    exe = tmp_path / "use_sbnn"
    libdir = os.path.dirname(sbnn.lib_path())
    subprocess.run(["gcc", "-std=c99", "-pedantic", "-Wall", "-Wextra", "-Werror", "-I", os.path.join(ROOT, "include"),
                    str(src), "-o", str(exe), "-L", libdir, "-l:libsbnn.so", f"-Wl,-rpath,{libdir}"], check=True)
    out = subprocess.run([str(exe)], capture_output=True, text=True)
    assert out.returncode == 0, (out.returncode, out.stdout, out.stderr)
    got = [int(t) for t in out.stdout.split()]
    V = binding._View
    assert got == [C.sizeof(V), V.nnz_units.offset, V.group_ptr.offset, V.idx.offset, V.val.offset, V.bias.offset,
                   V.tap_mask.offset, V.gi.offset, V.block_idx.offset]


def test_weights_of_another_device_are_refused_without_a_launch():
    """A packed layer records the device it was uploaded to.  With the recorded device overwritten by the test hook,
    every compute entry point must return a status (never dereference the other device's pointers).  On a machine
    without a GPU the calls fail one check earlier; with one GPU the message names both devices."""
    L = sbnn.lib()
    w = np.ones((8, 1, 1, 8), np.float32)
    m = np.ones((8, 1, 1, 8), np.uint8)
    p = sbnn.pack_weights(w, m, None, 4)
    p3 = sbnn.pack_weights(np.ones((8, 3, 3, 8), np.float32), np.ones((8, 3, 3, 8), np.uint8), None, 4)
    was = [sbnn.debug_set_packed_device(q, 7) for q in (p, p3)]
    try:
        calls = [lambda: L.sbnn_conv1x1_gs(p.handle, 256, 512, 1, 2, 2, 0, None),
                 lambda: L.sbnn_conv1x1_gs_tuned(p.handle, 256, 512, 1, 2, 2, 0, 4, 1, 8, 64, None),
                 lambda: L.sbnn_conv1x1_gs_cm(p.handle, 256, 4, 512, 8, 4, 0, 0, 0, 0, 0, None),
                 lambda: L.sbnn_head_noalloc(p.handle, 256, 512, 1, 4, None),
                 lambda: L.sbnn_prepare(p.handle, 1, 2, 2, 0),
                 lambda: L.sbnn_conv3x3_gs(p3.handle, 256, 512, 1, 4, 4, 0, None),
                 lambda: L.sbnn_prepare(p3.handle, 1, 4, 4, 0)]
        for i, call in enumerate(calls):
            assert call() == 9, f"call {i}"                                           # SBNN_ERR_CUDA
            assert len(L.sbnn_last_error()) > 0
    finally:
        for q, d in zip((p, p3), was):
            sbnn.debug_set_packed_device(q, d)                                        # so that free() releases the real copies


# ---- packed-layer files (Section 3.5: the engine loads the converted model from its own sparse format) ----------

def _read_packed_file(path):
    """Independent reader of the documented file layout (include/sbnn.h), written from that description alone."""
    import struct
    raw = open(path, "rb").read()
    assert raw[:8] == b"SBNNPK\x01\x00"
    ver, cout, kh, kw, cin, g, has_taps, zero = struct.unpack_from("<8i", raw, 8)
    (nnz,) = struct.unpack_from("<q", raw, 40)
    off = 48
    ng = cout // g
    gp = np.frombuffer(raw, "<i4", ng + 1, off); off += 4 * (ng + 1)
    if zero == 4:
        blk = np.frombuffer(raw, "<i4", nnz // 4, off); off += 4 * (nnz // 4)
        idx = (blk[:, None] + np.arange(4)).reshape(-1).astype(np.int32)
    else:
        idx = np.frombuffer(raw, "<i4", nnz, off); off += 4 * nnz
    val = np.frombuffer(raw, "<f4", nnz * kh * kw * g, off).reshape(nnz, kh * kw, g); off += 4 * nnz * kh * kw * g
    bias = np.frombuffer(raw, "<f4", cout, off); off += 4 * cout
    taps = None
    if has_taps:
        taps = np.frombuffer(raw, "<u2", nnz, off); off += 2 * nnz
    (stored,) = struct.unpack_from("<Q", raw, off)
    assert off + 8 == len(raw)
    h = 1469598103934665603
    for byte in raw[:off]:
        h = ((h ^ byte) * 1099511628211) & 0xFFFFFFFFFFFFFFFF
    assert h == stored, "FNV-1a checksum of the file"
    return dict(ver=ver, cout=cout, kh=kh, kw=kw, cin=cin, g=g, zero=zero, gp=gp, idx=idx, val=val, bias=bias, taps=taps)


@pytest.mark.parametrize("k,g,cin,cout,patterns", [(1, 4, 24, 16, False), (3, 4, 12, 8, False), (3, 2, 10, 6, True),
                                                   (1, 8, 16, 8, False)])
def test_packed_layer_file_round_trip_and_layout(tmp_path, k, g, cin, cout, patterns):
    rng = np.random.default_rng(31)
    w = rng.standard_normal((cout, k, k, cin)).astype(np.float32)
    b = rng.standard_normal(cout).astype(np.float32)
    um = group_mask_layer_global(2, 3, cout // g, cin, 55)
    m = tap_pattern_mask(2, 19, um, g, 4) if patterns else expand_mask(um, g, k, k)
    p = sbnn.pack_weights(w, m, b, g, tap_patterns=patterns)
    path = str(tmp_path / "layer.sbnn")
    p.save(path)
    # (i) the bytes on disk, read by a reader of our own, are the oracle's packing of the same layer
    f = _read_packed_file(path)
    assert (f["ver"], f["cout"], f["kh"], f["kw"], f["cin"], f["g"]) == (1, cout, k, k, cin, g) and f["zero"] in (0, 4)
    if patterns:
        gp, idx, val, taps = R.pack_pattern(w, m, g)
        assert np.array_equal(f["taps"], taps)
    else:
        gp, idx, val = R.pack(w, m, g)
        assert f["taps"] is None
    assert np.array_equal(f["gp"], gp) and np.array_equal(f["idx"], idx)
    assert f["val"].tobytes() == np.asarray(val, np.float32).tobytes() and f["bias"].tobytes() == b.tobytes()
    # (ii) loading gives back an identical layer
    q = sbnn.load_packed(path)
    v0, v1 = p.view(), q.view()
    for key in v0:
        a0, a1 = v0[key], v1[key]
        if isinstance(a0, np.ndarray):
            assert a0.dtype == a1.dtype and a0.tobytes() == a1.tobytes(), key
        else:
            assert a0 == a1 or (a0 is None and a1 is None), key
    w2, m2 = q.unpack()
    assert np.array_equal(m2, m)
    p.free(); q.free()


def test_packed_layer_file_errors(tmp_path):
    rng = np.random.default_rng(32)
    w = rng.standard_normal((8, 1, 1, 12)).astype(np.float32)
    m = expand_mask(group_mask_balanced(3, 3, 2, 12, 50), 4, 1, 1)
    p = sbnn.pack_weights(w, m, None, 4)
    good = str(tmp_path / "good.sbnn")
    p.save(good)
    raw = open(good, "rb").read()
    p.free()

    def load(data, name):
        path = str(tmp_path / name)
        open(path, "wb").write(data)
        with pytest.raises(sbnn.SbnnError) as e:
            sbnn.load_packed(path)
        return e.value.name

    assert load(raw[:-3], "truncated") == "SBNN_ERR_IO"
    assert load(raw[:20], "short") == "SBNN_ERR_IO"
    assert load(raw + b"\0", "trailing") == "SBNN_ERR_IO"
    assert load(b"NOTSBNN!" + raw[8:], "magic") == "SBNN_ERR_IO"
    flipped = bytearray(raw); flipped[60] ^= 0x40
    assert load(bytes(flipped), "flipped") == "SBNN_ERR_IO"                     # checksum
    v2 = bytearray(raw); v2[8] = 2
    assert load(bytes(v2), "version") == "SBNN_ERR_UNSUPPORTED"
    with pytest.raises(sbnn.SbnnError) as e:
        sbnn.load_packed(str(tmp_path / "missing.sbnn"))
    assert e.value.name == "SBNN_ERR_IO"
    with pytest.raises(sbnn.SbnnError) as e:
        sbnn.pack_weights(w, m, None, 4).save(str(tmp_path / "no_such_dir" / "x.sbnn"))
    assert e.value.name == "SBNN_ERR_IO"

    # a file whose checksum is right but whose indices are not ascending is refused as inconsistent
    import struct
    bad = bytearray(raw[:-8])
    ng = 2
    off_idx = 48 + 4 * (ng + 1)
    i0, i1 = struct.unpack_from("<2i", bad, off_idx)
    struct.pack_into("<2i", bad, off_idx, i1, i0)
    h = 1469598103934665603
    for byte in bad:
        h = ((h ^ byte) * 1099511628211) & 0xFFFFFFFFFFFFFFFF
    assert load(bytes(bad) + struct.pack("<Q", h), "unsorted") == "SBNN_ERR_SHAPE"


def test_paper_style_4x4_blocks_are_recognised_and_stored_with_one_index_per_block(tmp_path):
    """Masks made of aligned runs of gi = 4 input channels (the paper's 4 x 4 blocks, Section 3.2): the view reports gi = 4
    and block_idx = the first channel of every run (Algorithm 1's SD), the file stores those instead of the per-channel
    indices (a quarter of them) and loads back to the same layer; any other mask reports gi = 1."""
    rng = np.random.default_rng(33)
    cin, cout, g = 32, 16, 4
    w = rng.standard_normal((cout, 1, 1, cin)).astype(np.float32)
    um = group_mask_balanced(4, 3, cout // g, cin, 50, 4)            # gi = 4
    assert np.all(um.reshape(cout // g, cin // 4, 4).all(axis=2) == um.reshape(cout // g, cin // 4, 4).any(axis=2))
    m = expand_mask(um, g, 1, 1)
    p = sbnn.pack_weights(w, m, None, g)
    v = p.view()
    gp, idx, val = R.pack(w, m, g)
    blocks = np.asarray(idx).reshape(-1, 4)
    assert np.array_equal(blocks, blocks[:, :1] + np.arange(4)) and np.all(blocks[:, 0] % 4 == 0)
    assert v["gi"] == 4 and np.array_equal(v["block_idx"], blocks[:, 0]) and np.array_equal(v["idx"], idx)
    path = str(tmp_path / "blocks.sbnn")
    p.save(path)
    raw = open(path, "rb").read()
    import struct
    hdr = struct.unpack_from("<8i", raw, 8)
    assert hdr[7] == 4
    nnz = len(idx)
    off = 48 + 4 * (cout // g + 1)
    assert np.array_equal(np.frombuffer(raw, "<i4", nnz // 4, off), blocks[:, 0])
    assert len(raw) == off + 4 * (nnz // 4) + 4 * nnz * g + 4 * cout + 8
    q = sbnn.load_packed(path)
    vq = q.view()
    assert vq["gi"] == 4 and np.array_equal(vq["idx"], idx) and vq["val"].tobytes() == v["val"].tobytes()
    assert np.array_equal(vq["block_idx"], v["block_idx"])
    p.free(); q.free()
    um1 = group_mask_balanced(4, 3, cout // g, cin, 50)               # single channels
    p1 = sbnn.pack_weights(w, expand_mask(um1, g, 1, 1), None, g)
    v1 = p1.view()
    assert v1["gi"] == 1 and v1["block_idx"] is None
    p1.save(path)
    assert struct.unpack_from("<8i", open(path, "rb").read(), 8)[7] == 0
    p1.free()


@pytest.mark.parametrize("ntiles,nchunks,nrow,ncta", [(16, 32, 16, 148), (16, 32, 19, 148), (3, 3, 1, 148), (1, 1, 1, 148),
                                                      (11, 32, 19, 132), (5, 7, 100, 4), (2, 40, 3, 7), (4, 9, 2, 1)])
def test_conv3x3_work_plan_covers_every_step_once_in_balanced_shares(ntiles, nchunks, nrow, ncta):
    """The persistent 3x3 kernel's plan (host arithmetic, through the C interface): the segments, read in CTA order,
    enumerate every (group tile, row tile, step) exactly once and in order; a CTA's weight differs from an equal share
    by less than one step; split tiles number their parts and own consecutive slots and one counter each."""
    rng = np.random.default_rng(ntiles * 1000 + nchunks)
    words = rng.integers(0, 60, size=(ntiles, nchunks)).astype(np.int64)
    words[rng.random(words.shape) < 0.1] = 0                       # steps in which the tile keeps nothing
    bp = np.zeros((ntiles, nchunks + 1), dtype=np.int32)
    bp[:, 1:] = np.cumsum(words, axis=1)
    bp += (np.arange(ntiles, dtype=np.int32) * 5000)[:, None]       # tiles follow one another in the stream
    cta_ptr, segs, nslots, ncounters = sbnn.debug_plan_conv3x3(bp, nrow, ncta)
    steps = ntiles * nrow * nchunks
    ncta_eff = min(ncta, steps)
    assert cta_ptr[0] == 0 and np.all(np.diff(cta_ptr) >= 0) and cta_ptr[-1] == len(segs)
    # coverage and order
    pos = 0                                                         # next step expected, in (by, bx, k) order
    for bx, by, k0, k1, part, nparts, slot, counter in segs:
        assert k1 > k0
        assert pos == (by * nrow + bx) * nchunks + k0
        assert (part == 0) == (k0 == 0)
        pos += k1 - k0
    assert pos == steps
    # parts, slots, counters
    by_tile = {}
    for i, sg in enumerate(segs):
        by_tile.setdefault((sg[1], sg[0]), []).append(sg)
    seen_slots, seen_counters = set(), set()
    for parts in by_tile.values():
        n = len(parts)
        assert [int(sg[4]) for sg in parts] == list(range(n)) and all(sg[5] == n for sg in parts)
        assert parts[-1][3] == nchunks
        if n > 1:
            assert len({int(sg[6]) for sg in parts}) == 1 and len({int(sg[7]) for sg in parts}) == 1
            slots = set(range(int(parts[0][6]), int(parts[0][6]) + n))
            assert not (slots & seen_slots) and int(parts[0][7]) not in seen_counters
            seen_slots |= slots
            seen_counters.add(int(parts[0][7]))
    assert seen_slots == set(range(nslots)) and seen_counters == set(range(ncounters))
    assert nslots <= 2 * ncta_eff
    # balance: weight of a step = its words + 6
    weight = words + 6
    total = int(weight.sum()) * nrow
    share = total / ncta_eff
    heaviest = int(weight.max())
    for c in range(ncta_eff):
        wc = sum(int(weight[sg[1], sg[2]:sg[3]].sum()) for sg in segs[cta_ptr[c]:cta_ptr[c + 1]])
        assert abs(wc - share) < heaviest + 1, (c, wc, share)
    # CTAs beyond the number of steps own nothing
    assert np.all(cta_ptr[ncta_eff:] == len(segs))


def test_conv3x3_work_plan_errors():
    bp = np.array([[0, 4, 2]], dtype=np.int32)                      # decreasing
    with pytest.raises(sbnn.SbnnError, match="SBNN_ERR_SHAPE"):
        sbnn.debug_plan_conv3x3(bp, 1, 4)
    with pytest.raises(sbnn.SbnnError, match="SBNN_ERR_SHAPE"):
        sbnn.debug_plan_conv3x3(np.array([[0, 4, 8]], dtype=np.int32), 0, 4)


def test_loading_a_pattern_layer_zeroes_the_weights_of_pruned_taps(tmp_path):
    """A file whose value block holds something at a pruned tap (written by another tool) loads with zeros there:
    the whole-kernel 3x3 loops multiply every stored tap, so the stored value of a pruned tap must be zero."""
    import struct
    rng = np.random.default_rng(41)
    g, cin, cout = 2, 10, 6
    w = rng.standard_normal((cout, 3, 3, cin)).astype(np.float32)
    um = group_mask_layer_global(2, 3, cout // g, cin, 40)
    m = tap_pattern_mask(2, 19, um, g, 4)
    p = sbnn.pack_weights(w, m, None, g, tap_patterns=True)
    path = str(tmp_path / "layer.sbnn")
    p.save(path)
    want = p.view()
    p.free()
    f = _read_packed_file(path)
    raw = bytearray(open(path, "rb").read())
    nnz = len(f["idx"])
    val_off = 48 + 4 * (cout // g + 1) + 4 * nnz
    poked = 0
    for u in range(nnz):
        for t in range(9):
            if not (int(f["taps"][u]) >> t) & 1:
                struct.pack_into("<f", raw, val_off + 4 * ((u * 9 + t) * g), 7.5)   # first filter of the group, pruned tap
                poked += 1
    assert poked > 0
    h = 1469598103934665603
    for byte in raw[:-8]:
        h = ((h ^ byte) * 1099511628211) & 0xFFFFFFFFFFFFFFFF
    struct.pack_into("<Q", raw, len(raw) - 8, h)
    bad = str(tmp_path / "poked.sbnn")
    open(bad, "wb").write(bytes(raw))
    q = sbnn.load_packed(bad)
    got = q.view()
    assert np.array_equal(got["val"], want["val"]) and np.array_equal(got["tap_mask"], want["tap_mask"])
    q.free()
