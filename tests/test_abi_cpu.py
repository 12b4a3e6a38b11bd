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
