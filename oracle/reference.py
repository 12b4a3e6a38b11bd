"""Python face of the CPU oracle.  TEST INFRASTRUCTURE ONLY (see sbnn_oracle.c).

* conv2d / dwconv3x3 / avgpool call the plain C loops (fp64 accumulation).
* pack / unpack are the oracle's own statement of the group-compressed weight
  format, written independently of the library's packer: per group of G output
  channels the ascending kept input-channel indices ("sparse info" of
  Algorithm 1) and a value block.
* mobilenet_v1_* hold the oracle's own copy of the MobileNet-v1 layer table,
  its multiply-accumulate counts (pinned to Table 3's FLOPs column) and the
  chained forward pass.

Every function here is pinned by tests/test_oracle_pins.py against brute force,
closed forms, a library routine and the paper's printed counts; nothing is
"parity unpinned" except mask *selection* quality, which is not computed here.
"""
from __future__ import annotations

import ctypes
import math

import numpy as np

from . import build as _build

_lib = None


def _L():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build.build())
        P, I, L = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64
        lib.oracle_conv2d.argtypes = [P, P, P, P, I, I, I, I, I, I, I, I, I, I, P, P]
        lib.oracle_dwconv3x3.argtypes = [P, P, P, I, I, I, I, I, I, P, P]
        lib.oracle_avgpool.argtypes = [P, I, I, I, P, P]
        lib.oracle_bf16_round.argtypes = [P, P, L]
        lib.oracle_num_threads.restype = I
        for f in (lib.oracle_conv2d, lib.oracle_dwconv3x3, lib.oracle_avgpool, lib.oracle_bf16_round):
            f.restype = None
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_L().oracle_num_threads())


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a, a.ctypes.data


def conv2d(x, w, mask, bias, stride=1, relu=True, bf16=False):
    """Convolution with W (.) M (Section 3.1).  x [N][H][W][Cin], w/mask [Cout][KH][KW][Cin].

    Returns (ref, S) as float64 arrays [N][Ho][Wo][Cout]; S = |b| + sum |w*m*x|.
    """
    x, xp = _f32(x)
    w, wp = _f32(w)
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    n, h, wd, cin = x.shape
    cout, kh, kw, cin2 = w.shape
    assert cin == cin2 and mask.shape == w.shape
    bp = None
    if bias is not None:
        bias, bp = _f32(bias)
    ho = (h + 2 * ((kh - 1) // 2) - kh) // stride + 1
    wo = (wd + 2 * ((kw - 1) // 2) - kw) // stride + 1
    ref = np.empty((n, ho, wo, cout), dtype=np.float64)
    s = np.empty_like(ref)
    _L().oracle_conv2d(xp, wp, mask.ctypes.data, bp, n, h, wd, cin, cout, kh, kw, stride,
                       int(relu), int(bf16), ref.ctypes.data, s.ctypes.data)
    return ref, s


def dwconv3x3(x, w, bias, stride=1, relu=True):
    """Dense depthwise 3x3, pad 1.  x [N][H][W][C], w [3][3][C]."""
    x, xp = _f32(x)
    w, wp = _f32(w)
    n, h, wd, c = x.shape
    assert w.shape == (3, 3, c)
    bp = None
    if bias is not None:
        bias, bp = _f32(bias)
    ho, wo = (h - 1) // stride + 1, (wd - 1) // stride + 1
    ref = np.empty((n, ho, wo, c), dtype=np.float64)
    s = np.empty_like(ref)
    _L().oracle_dwconv3x3(xp, wp, bp, n, h, wd, c, stride, int(relu), ref.ctypes.data, s.ctypes.data)
    return ref, s


def avgpool(x):
    """Global average over all positions.  x [N][H][W][C] -> (ref, S) [N][C]."""
    x, xp = _f32(x)
    n, h, wd, c = x.shape
    ref = np.empty((n, c), dtype=np.float64)
    s = np.empty_like(ref)
    _L().oracle_avgpool(xp, n, h * wd, c, ref.ctypes.data, s.ctypes.data)
    return ref, s


def bf16_round(a):
    a, ap = _f32(a)
    out = np.empty_like(a)
    _L().oracle_bf16_round(ap, out.ctypes.data, a.size)
    return out


# ---------------------------------------------------------------------------
# Group-compressed weight format (the oracle's own packer).
# ---------------------------------------------------------------------------

class MaskNotGroupUniform(ValueError):
    pass


def pack(w, mask, g):
    """Per group of g consecutive output channels: ascending kept input channels and their values.

    A unit (group, input channel) is kept iff its mask entries are 1; the mask
    must be constant over the g rows of a group and over the kernel taps
    (Eq. 2's block mask with gi = 1).  Returns (group_ptr int32 [ngroups+1],
    idx int32 [nnzU], val float32 [nnzU][KH*KW][g]).
    """
    w = np.asarray(w, dtype=np.float32)
    mask = np.asarray(mask, dtype=np.uint8)
    cout, kh, kw, cin = w.shape
    if cout % g:
        raise ValueError("Cout % G != 0")
    ngroups = cout // g
    group_ptr = [0]
    idx = []
    val = []
    for gi in range(ngroups):
        rows = mask[gi * g:(gi + 1) * g]          # [g][kh][kw][cin]
        first = rows[0, 0, 0]                     # [cin]
        if np.any(rows != first[None, None, None, :]) or np.any(first > 1):
            raise MaskNotGroupUniform(f"group {gi}")
        for c in range(cin):
            if first[c]:
                idx.append(c)
                # [kh*kw][g]: taps outer, the group's output channels inner
                val.append(w[gi * g:(gi + 1) * g, :, :, c].reshape(g, kh * kw).T)
        group_ptr.append(len(idx))
    val = np.array(val, dtype=np.float32).reshape(len(idx), kh * kw, g)
    return np.array(group_ptr, dtype=np.int32), np.array(idx, dtype=np.int32), val


def pack_pattern(w, mask, g):
    """Packing when the taps of a kernel are pruned individually (kernel patterns shared by the g filters of a
    group; Section 3.3's Conv3x3 pattern pruning).

    A unit (group, input channel) is kept iff any of its taps is; its pruned taps are stored as zeros.  Returns
    (group_ptr, idx, val, tap_mask) with tap_mask uint16 [nnzU], bit t set iff tap t = kh*KW + kw is kept.
    """
    w = np.asarray(w, dtype=np.float32)
    mask = np.asarray(mask, dtype=np.uint8)
    cout, kh, kw, cin = w.shape
    if cout % g:
        raise ValueError("Cout % G != 0")
    group_ptr, idx, val, tap_mask = [0], [], [], []
    for gi in range(cout // g):
        rows = mask[gi * g:(gi + 1) * g].reshape(g, kh * kw, cin)
        if np.any(rows != rows[0][None]) or np.any(rows > 1):
            raise MaskNotGroupUniform(f"group {gi}")
        wg = w[gi * g:(gi + 1) * g].reshape(g, kh * kw, cin)
        for c in range(cin):
            taps = rows[0, :, c]
            if not taps.any():
                continue
            idx.append(c)
            tap_mask.append(sum(1 << t for t in range(kh * kw) if taps[t]))
            val.append(np.where(taps[None, :] != 0, wg[:, :, c], np.float32(0)).T)   # [taps][g]
        group_ptr.append(len(idx))
    val = np.array(val, dtype=np.float32).reshape(len(idx), kh * kw, g)
    return (np.array(group_ptr, dtype=np.int32), np.array(idx, dtype=np.int32), val,
            np.array(tap_mask, dtype=np.uint16))


def pack_dw_pattern(w, mask, go):
    """Compact form of 3:9 pattern-pruned depthwise weights (Section 3.2, DwConv3x3; Algorithm 2's PatternInfo).

    w, mask: [3][3][C].  In every row the middle weight is kept and exactly one of the two side columns is
    pruned, identically for the `go` channels of a block.  Returns (pattern uint8 [C/go] with bit kh set iff the
    third column of row kh is pruned, w6 float32 [3][2][C] = per row the surviving side weight, then the middle).
    """
    w = np.asarray(w, dtype=np.float32)
    mask = np.asarray(mask, dtype=np.uint8)
    c = w.shape[2]
    if c % go:
        raise ValueError("C % go != 0")
    pattern = np.zeros(c // go, dtype=np.uint8)
    w6 = np.zeros((3, 2, c), dtype=np.float32)
    for blk in range(c // go):
        sl = slice(blk * go, (blk + 1) * go)
        for kh in range(3):
            rows = mask[kh, :, sl]                      # [kw][go]
            if np.any(rows != rows[:, :1]) or rows[1, 0] != 1 or int(rows[0, 0]) + int(rows[2, 0]) != 1:
                raise MaskNotGroupUniform(f"block {blk} row {kh}")
            third_pruned = rows[2, 0] == 0
            if third_pruned:
                pattern[blk] |= 1 << kh
            w6[kh, 0, sl] = w[kh, 0 if third_pruned else 2, sl]
            w6[kh, 1, sl] = w[kh, 1, sl]
    return pattern, w6


def unpack(group_ptr, idx, val, cout, kh, kw, cin, g):
    """Inverse of pack: returns (W (.) M, M)."""
    w = np.zeros((cout, kh, kw, cin), dtype=np.float32)
    m = np.zeros((cout, kh, kw, cin), dtype=np.uint8)
    for gi in range(cout // g):
        for u in range(group_ptr[gi], group_ptr[gi + 1]):
            c = idx[u]
            w[gi * g:(gi + 1) * g, :, :, c] = val[u].T.reshape(g, kh, kw)
            m[gi * g:(gi + 1) * g, :, :, c] = 1
    return w, m


# ---------------------------------------------------------------------------
# MobileNet-v1 (width 1.0, 224x224x3): layer table, MAC counts, chained forward.
# ---------------------------------------------------------------------------

def mobilenet_v1_table():
    """(kind, input side, Cin, Cout, stride) per layer; 3x3 stride-2 stem, 13 depthwise-separable
    blocks, 7x7 average pool and a 1000-way classifier."""
    t = [("conv0", 224, 3, 32, 2)]
    h = 112
    for ci, co, s in [(32, 64, 1), (64, 128, 2), (128, 128, 1), (128, 256, 2), (256, 256, 1), (256, 512, 2),
                      (512, 512, 1), (512, 512, 1), (512, 512, 1), (512, 512, 1), (512, 512, 1),
                      (512, 1024, 2), (1024, 1024, 1)]:
        t.append(("dw", h, ci, ci, s))
        h //= s
        t.append(("pw", h, ci, co, 1))
    t.append(("pool", 7, 1024, 1024, 1))
    t.append(("fc", 1, 1024, 1000, 1))
    return t


def mobilenet_v1_macs():
    """Dense multiply-accumulates per image, by layer kind."""
    out = {"conv0": 0, "dw": 0, "pw": 0, "fc": 0}
    for kind, hin, ci, co, s in mobilenet_v1_table():
        ho = hin // s
        if kind == "conv0":
            out[kind] += ho * ho * 27 * co
        elif kind == "dw":
            out[kind] += ho * ho * 9 * ci
        elif kind in ("pw", "fc"):
            out[kind] += ho * ho * ci * co
    return out


def mobilenet_v1_nonzero_macs(pointwise_sparsity: float) -> float:
    """MACs left when only the 13 pointwise layers are pruned to the given sparsity (Table 3's FLOPs column)."""
    m = mobilenet_v1_macs()
    return m["conv0"] + m["dw"] + m["fc"] + (1.0 - pointwise_sparsity) * m["pw"]


def mobilenet_v1_forward(x, layers, tol=1e-5):
    """Chained forward.  `layers` follows sbnn_inputs.mobilenet_v1_inputs.

    Every layer's fp64 result is rounded to fp32 before it feeds the next one.
    Returns a list with one dict per layer: "in" (fp32 input), "ref", "S"
    (fp64), and "E", a first-order bound on |approx - ref| for an
    implementation that is within tol*S on every layer:
    E_out = conv(|W~|, E_in) + tol*S (ReLU and pooling are 1-Lipschitz).
    """
    outs = []
    cur = np.ascontiguousarray(x, dtype=np.float32)
    err = np.zeros(cur.shape, dtype=np.float64)
    for L in layers:
        kind = L["kind"]
        rec = {"name": L["name"], "in": cur}
        e32 = err.astype(np.float32) * np.float32(1.0 + 2.0 ** -20)   # round the bound upward
        if kind == "conv0":
            ones = np.ones(L["w"].shape, dtype=np.uint8)
            ref, s = conv2d(cur, L["w"], ones, L["bias"], stride=L["stride"], relu=True)
            e, _ = conv2d(e32, np.abs(L["w"]), ones, None, stride=L["stride"], relu=False)
        elif kind == "dw":
            ref, s = dwconv3x3(cur, L["w"], L["bias"], stride=L["stride"], relu=True)
            e, _ = dwconv3x3(e32, np.abs(L["w"]), None, stride=L["stride"], relu=False)
        elif kind == "pw":
            ref, s = conv2d(cur, L["w"], L["mask"], L["bias"], relu=True)
            e, _ = conv2d(e32, np.abs(L["w"]), L["mask"], None, relu=False)
        elif kind == "pool":
            ref, s = avgpool(cur)
            e, _ = avgpool(e32)
            ref, s, e = (a.reshape(a.shape[0], 1, 1, a.shape[1]) for a in (ref, s, e))
        elif kind == "fc":
            ref, s = conv2d(cur, L["w"], L["mask"], L["bias"], relu=False)
            e, _ = conv2d(e32, np.abs(L["w"]), L["mask"], None, relu=False)
        else:
            raise ValueError(kind)
        err = e + tol * s + np.abs(ref) * 2.0 ** -24      # + the rounding of ref to fp32 below
        rec.update(ref=ref, S=s, E=err)
        outs.append(rec)
        cur = ref.astype(np.float32)
    return outs


def sample_outputs(x, w, mask, bias, positions, relu=True, bf16=False):
    """The definition evaluated one output at a time, for checks at sizes where the full loops take too long.

    positions: iterable of (n, y, x, o) output coordinates of a stride-1 convolution with zero padding
    (K-1)/2.  Returns (ref, S) as float64 arrays of len(positions), computed as
    b[o] + sum over taps and ALL input channels of w*m*x in fp64 (no zero skipping, as in conv2d).
    """
    x = np.asarray(x, dtype=np.float32)
    w = np.asarray(w, dtype=np.float32)
    mask = np.asarray(mask, dtype=np.uint8)
    n_, h, wd, cin = x.shape
    cout, kh, kw, _ = w.shape
    ph, pw = (kh - 1) // 2, (kw - 1) // 2
    ref = np.empty(len(positions), dtype=np.float64)
    s = np.empty(len(positions), dtype=np.float64)
    for i, (n, y, xx, o) in enumerate(positions):
        b = float(bias[o]) if bias is not None else 0.0
        acc, sa = b, abs(b)
        for dy in range(kh):
            iy = y + dy - ph
            if iy < 0 or iy >= h:
                continue
            for dx in range(kw):
                ix = xx + dx - pw
                if ix < 0 or ix >= wd:
                    continue
                wm = np.where(mask[o, dy, dx] != 0, w[o, dy, dx], np.float32(0))
                xv = x[n, iy, ix]
                if bf16:
                    wm, xv = bf16_round(wm), bf16_round(xv)
                p = wm.astype(np.float64) * xv.astype(np.float64)
                acc += float(p.sum())
                sa += float(np.abs(p).sum())
        ref[i] = max(acc, 0.0) if relu else acc
        s[i] = sa
    return ref, s
