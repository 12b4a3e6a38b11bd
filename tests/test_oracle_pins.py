"""Pins of the CPU oracle against things other than itself: brute force written differently,
closed forms, library routines (torch fp64 conv / matmul / bf16 cast) and counts the paper prints."""
import itertools
import os

import numpy as np
import pytest
import torch

from oracle import reference as R
from sbnn_inputs import dw_pattern_mask, expand_mask, group_mask_balanced, tap_pattern_mask

GOLD = os.path.join(os.path.dirname(__file__), "golden")
rng = np.random.default_rng(1234)


def _rand_layer(n, h, w, cin, cout, k, g, keep=0.5):
    x = rng.standard_normal((n, h, w, cin)).astype(np.float32)
    wt = rng.standard_normal((cout, k, k, cin)).astype(np.float32)
    b = rng.standard_normal(cout).astype(np.float32)
    um = rng.random((cout // g, cin)) < keep
    return x, wt, b, expand_mask(um, g, k, k), um


def _brute(x, wt, m, b, stride, relu):
    """im2col + naive GEMM in long double: a structurally different route to the same definition."""
    n, h, w, cin = x.shape
    cout, kh, kw, _ = wt.shape
    ph, pw = (kh - 1) // 2, (kw - 1) // 2
    xp = np.zeros((n, h + 2 * ph, w + 2 * pw, cin), dtype=np.longdouble)
    xp[:, ph:ph + h, pw:pw + w] = x
    ho, wo = (h + 2 * ph - kh) // stride + 1, (w + 2 * pw - kw) // stride + 1
    cols = np.zeros((n * ho * wo, kh * kw * cin), dtype=np.longdouble)
    r = 0
    for ni, oy, ox in itertools.product(range(n), range(ho), range(wo)):
        cols[r] = xp[ni, oy * stride:oy * stride + kh, ox * stride:ox * stride + kw].reshape(-1)
        r += 1
    wm = (wt.astype(np.longdouble) * m).reshape(cout, -1)
    out = np.zeros((cols.shape[0], cout), dtype=np.longdouble)
    for i in range(cols.shape[0]):
        for o in range(cout):
            acc = np.longdouble(b[o])
            for t in range(cols.shape[1]):
                acc += cols[i, t] * wm[o, t]
            out[i, o] = acc
    s = np.abs(cols) @ np.abs(wm).T + np.abs(b.astype(np.longdouble))
    if relu:
        out = np.maximum(out, 0)
    return out.reshape(n, ho, wo, cout), s.reshape(n, ho, wo, cout)


@pytest.mark.parametrize("k,stride,g", [(1, 1, 1), (1, 1, 4), (3, 1, 2), (3, 2, 4), (3, 1, 8)])
def test_p1_brute_force(k, stride, g):
    x, wt, b, m, _ = _rand_layer(2, 4, 5, 8, 8, k, g)
    ref, s = R.conv2d(x, wt, m, b, stride=stride, relu=True)
    bref, bs = _brute(x, wt, m, b, stride, True)
    assert ref.shape == bref.shape
    np.testing.assert_allclose(ref, bref.astype(np.float64), rtol=0, atol=1e-12)
    np.testing.assert_allclose(s, bs.astype(np.float64), rtol=1e-13, atol=1e-12)


def test_p2_all_ones_counts_kept_taps_in_bounds():
    n, h, w, cin, cout, g = 1, 5, 6, 8, 8, 4
    um = group_mask_balanced(3, 3, cout // g, cin, 50)
    m = expand_mask(um, g, 3, 3)
    x = np.ones((n, h, w, cin), np.float32)
    wt = np.ones((cout, 3, 3, cin), np.float32)
    b = np.full(cout, 0.5, np.float32)
    ref, s = R.conv2d(x, wt, m, b, relu=False)
    for oy, ox, o in itertools.product(range(h), range(w), range(cout)):
        taps = sum(1 for kh in range(3) for kw in range(3) if 0 <= oy + kh - 1 < h and 0 <= ox + kw - 1 < w)
        kept = int(um[o // g].sum())
        assert ref[0, oy, ox, o] == 0.5 + taps * kept
        assert s[0, oy, ox, o] == 0.5 + taps * kept


def test_p2_one_hot_weight_is_a_shift():
    """W[o][kh][kw][c] one-hot selects X[y+kh-1][x+kw-1][c] (cross-correlation, no kernel flip)."""
    x = rng.standard_normal((1, 6, 7, 4)).astype(np.float32)
    for kh, kw, c in [(0, 0, 1), (2, 1, 3), (1, 2, 0), (0, 2, 2)]:
        wt = np.zeros((4, 3, 3, 4), np.float32)
        wt[2, kh, kw, c] = 1.0
        ref, _ = R.conv2d(x, wt, np.ones_like(wt, dtype=np.uint8), None, relu=False)
        exp = np.zeros((6, 7))
        for y, xx in itertools.product(range(6), range(7)):
            iy, ix = y + kh - 1, xx + kw - 1
            if 0 <= iy < 6 and 0 <= ix < 7:
                exp[y, xx] = x[0, iy, ix, c]
        np.testing.assert_array_equal(ref[0, :, :, 2], exp)
        assert not ref[0, :, :, [0, 1, 3]].any()


def test_p2_zero_input_gives_relu_of_bias():
    x, wt, b, m, _ = _rand_layer(1, 3, 3, 8, 8, 3, 4)
    ref, s = R.conv2d(np.zeros_like(x), wt, m, b, relu=True)
    np.testing.assert_array_equal(ref, np.broadcast_to(np.maximum(b.astype(np.float64), 0), ref.shape))
    np.testing.assert_array_equal(s, np.broadcast_to(np.abs(b.astype(np.float64)), s.shape))


@pytest.mark.parametrize("k,stride", [(1, 1), (3, 1), (3, 2)])
def test_p3_matches_torch_conv2d(k, stride):
    x, wt, b, m, _ = _rand_layer(2, 9, 8, 12, 16, k, 4, keep=0.6)
    ref, s = R.conv2d(x, wt, m, b, stride=stride, relu=False)
    xt = torch.from_numpy(x).double().permute(0, 3, 1, 2)
    wm = torch.from_numpy(wt * m).double().permute(0, 3, 1, 2)
    y = torch.nn.functional.conv2d(xt, wm, torch.from_numpy(b).double(), stride=stride, padding=(k - 1) // 2)
    np.testing.assert_allclose(ref, y.permute(0, 2, 3, 1).numpy(), rtol=0, atol=1e-12)
    # dense special case (s = 0): full mask equals the plain convolution
    ref0, _ = R.conv2d(x, wt, np.ones_like(m), b, stride=stride, relu=False)
    y0 = torch.nn.functional.conv2d(xt, torch.from_numpy(wt).double().permute(0, 3, 1, 2),
                                    torch.from_numpy(b).double(), stride=stride, padding=(k - 1) // 2)
    np.testing.assert_allclose(ref0, y0.permute(0, 2, 3, 1).numpy(), rtol=0, atol=1e-12)


def test_p3_pointwise_is_a_matmul():
    x, wt, b, m, _ = _rand_layer(2, 5, 5, 16, 8, 1, 4)
    ref, s = R.conv2d(x, wt, m, b, relu=False)
    wm = (wt * m).reshape(8, 16).astype(np.float64)
    exp = x.reshape(-1, 16).astype(np.float64) @ wm.T + b
    np.testing.assert_allclose(ref.reshape(-1, 8), exp, rtol=0, atol=1e-12)
    exps = np.abs(x.reshape(-1, 16).astype(np.float64)) @ np.abs(wm).T + np.abs(b)
    np.testing.assert_allclose(s.reshape(-1, 8), exps, rtol=1e-13)


@pytest.mark.parametrize("stride", [1, 2])
def test_depthwise_matches_torch_and_diagonal_conv(stride):
    c = 8
    x = rng.standard_normal((2, 7, 6, c)).astype(np.float32)
    w = rng.standard_normal((3, 3, c)).astype(np.float32)
    b = rng.standard_normal(c).astype(np.float32)
    ref, s = R.dwconv3x3(x, w, b, stride=stride, relu=True)
    y = torch.nn.functional.conv2d(torch.from_numpy(x).double().permute(0, 3, 1, 2),
                                   torch.from_numpy(w).double().permute(2, 0, 1)[:, None],
                                   torch.from_numpy(b).double(), stride=stride, padding=1, groups=c)
    np.testing.assert_allclose(ref, torch.relu(y).permute(0, 2, 3, 1).numpy(), rtol=0, atol=1e-12)
    full = np.zeros((c, 3, 3, c), np.float32)
    for ch in range(c):
        full[ch, :, :, ch] = w[:, :, ch]
    ref2, s2 = R.conv2d(x, full, np.ones_like(full, dtype=np.uint8), b, stride=stride, relu=True)
    np.testing.assert_allclose(ref, ref2, rtol=0, atol=1e-13)
    np.testing.assert_allclose(s, s2, rtol=1e-13)


def test_avgpool_is_the_mean():
    x = rng.standard_normal((3, 7, 7, 16)).astype(np.float32)
    ref, s = R.avgpool(x)
    np.testing.assert_allclose(ref, x.astype(np.float64).mean(axis=(1, 2)), rtol=1e-14, atol=1e-15)
    np.testing.assert_allclose(s, np.abs(x.astype(np.float64)).mean(axis=(1, 2)), rtol=1e-14)


def test_p6_masked_equals_premasked_bit_for_bit():
    x, wt, b, m, _ = _rand_layer(1, 5, 5, 16, 16, 3, 4)
    a, sa = R.conv2d(x, wt, m, b)
    c, sc = R.conv2d(x, wt * m, np.ones_like(m), b)
    assert np.array_equal(a, c) and np.array_equal(sa, sc)


def test_p4_pack_round_trip_and_invariants():
    for k, g in [(1, 1), (1, 4), (3, 4), (1, 8), (3, 2)]:
        x, wt, b, m, um = _rand_layer(1, 2, 2, 24, 16, k, g)
        gp, idx, val = R.pack(wt, m, g)
        ng = 16 // g
        assert gp.dtype == np.int32 and idx.dtype == np.int32 and val.dtype == np.float32
        assert gp[0] == 0 and gp[-1] == um.sum() == len(idx) and np.all(np.diff(gp) >= 0)
        for gi in range(ng):
            seg = idx[gp[gi]:gp[gi + 1]]
            assert np.all(np.diff(seg) > 0) and np.array_equal(seg, np.nonzero(um[gi])[0])
        assert val.shape == (len(idx), k * k, g)
        # value block: taps outer, the group's g output channels inner
        u = int(gp[1]) - 1 if gp[1] > 0 else None
        if u is not None:
            c = idx[u]
            for t, r in itertools.product(range(k * k), range(g)):
                assert val[u, t, r] == wt[r, t // k, t % k, c]
        w2, m2 = R.unpack(gp, idx, val, 16, k, k, 24, g)
        assert np.array_equal(m2, m) and np.array_equal(w2, wt * m)


def test_p4_pack_rejects_non_uniform_mask():
    x, wt, b, m, um = _rand_layer(1, 2, 2, 8, 8, 1, 4, keep=1.0)
    m = m.copy()
    m[1, 0, 0, 3] = 0
    with pytest.raises(R.MaskNotGroupUniform):
        R.pack(wt, m, 4)
    m3 = np.ones((8, 3, 3, 8), np.uint8)
    m3[0:4, 1, 1, 2] = 0        # one tap removed for a whole group: not a whole-kernel mask
    with pytest.raises(R.MaskNotGroupUniform):
        R.pack(np.ones((8, 3, 3, 8), np.float32), m3, 4)


def test_p4_pattern_packers_reconstruct_the_masked_weights():
    """The two pattern formats, checked by writing the dense masked weights back out of them by hand (not through
    the oracle's own unpack): kernel patterns of a 3x3 layer, and the 3:9 patterns of depthwise weights; the
    convolution with the reconstructed weights is the masked convolution."""
    g, cin, cout = 4, 10, 8
    wt = rng.standard_normal((cout, 3, 3, cin)).astype(np.float32)
    um = rng.random((cout // g, cin)) < 0.6
    m = tap_pattern_mask(5, 19, um, g, 4)
    assert np.all(m.reshape(cout // g, g, 9, cin).sum(axis=2)[:, 0][um] == 4) and np.all(m[:, 1, 1].reshape(cout // g, g, cin)[:, 0] == um)
    gp, idx, val, tm = R.pack_pattern(wt, m, g)
    dense = np.zeros_like(wt)
    for gi in range(cout // g):
        for u in range(gp[gi], gp[gi + 1]):
            for t in range(9):
                kept = (int(tm[u]) >> t) & 1
                assert kept or not val[u, t].any()                      # pruned taps are stored as zeros
                dense[gi * g:(gi + 1) * g, t // 3, t % 3, idx[u]] = val[u, t]
                assert np.all(m[gi * g:(gi + 1) * g, t // 3, t % 3, idx[u]] == kept)
    assert np.array_equal(dense, wt * m) and gp[-1] == um.sum()
    x = rng.standard_normal((1, 4, 5, cin)).astype(np.float32)
    a, _ = R.conv2d(x, wt, m, None, relu=False)
    b, _ = R.conv2d(x, dense, np.ones_like(m), None, relu=False)
    assert np.array_equal(a, b)

    c, go = 32, 8
    wd = rng.standard_normal((3, 3, c)).astype(np.float32)
    md = dw_pattern_mask(5, 7, c, go, wd)
    pat, w6 = R.pack_dw_pattern(wd, md, go)
    dd = np.zeros_like(wd)
    for blk in range(c // go):
        sl = slice(blk * go, (blk + 1) * go)
        for kh in range(3):
            third_pruned = (int(pat[blk]) >> kh) & 1
            dd[kh, 0 if third_pruned else 2, sl] = w6[kh, 0, sl]
            dd[kh, 1, sl] = w6[kh, 1, sl]
            # the l1 rule: the kept side is the heavier one over the block
            l1 = np.abs(wd[kh, :, sl].astype(np.float64)).sum(axis=1)
            assert (l1[0] >= l1[2]) == bool(third_pruned)
    assert np.array_equal(dd, wd * md) and np.all(md.sum(axis=(0, 1)) == 6)
    with pytest.raises(R.MaskNotGroupUniform):
        bad = md.copy()
        bad[0, 0, 0] ^= 1
        R.pack_dw_pattern(wd, bad, go)


def test_p5_mobilenet_mac_counts_match_table3():
    rows = {}
    for line in open(os.path.join(GOLD, "mobilenet_v1_flops_table3.txt")):
        if line.startswith("#") or not line.strip():
            continue
        a, b = line.split()
        rows[a] = float(b)
    macs = R.mobilenet_v1_macs()
    assert sum(macs.values()) == 568_740_352
    share = rows.pop("conv3x3_share_percent")
    assert abs(100.0 * macs["conv0"] / sum(macs.values()) - share) < 0.005
    for sp, mflops in rows.items():
        ours = R.mobilenet_v1_nonzero_macs(float(sp)) / 1e6
        assert abs(ours - mflops) < 1.0, (sp, ours, mflops)     # the paper prints whole millions


def test_p7_bf16_rounding():
    vals = np.array([1.0, 1 + 2.0 ** -8, 1 + 2.0 ** -8 + 2.0 ** -20, 1 + 3 * 2.0 ** -8, -(1 + 2.0 ** -8), 0.0,
                     3.14159265], np.float32)
    exp = np.array([1.0, 1.0, 1 + 2.0 ** -7, 1 + 2.0 ** -6, -1.0, 0.0, 3.140625], np.float32)
    np.testing.assert_array_equal(R.bf16_round(vals), exp)
    a = rng.standard_normal(4096).astype(np.float32)
    np.testing.assert_array_equal(R.bf16_round(a), torch.from_numpy(a).bfloat16().float().numpy())
    x, wt, b, m, _ = _rand_layer(1, 3, 3, 16, 8, 1, 4)
    r1, s1 = R.conv2d(x, wt, m, b, bf16=True)
    r2, s2 = R.conv2d(R.bf16_round(x), R.bf16_round(wt * m), np.ones_like(m), b, bf16=False)
    assert np.array_equal(r1, r2) and np.array_equal(s1, s2)


def test_chain_error_bound_grows_and_layers_chain():
    """The chained oracle feeds each layer the fp32 rounding of the previous result."""
    from sbnn_inputs import mobilenet_v1_inputs
    x, layers = mobilenet_v1_inputs(1, 30, 4, seed=0)
    x = x[:, :32, :32]                          # small image: the table's shapes scale with H
    small = []
    h = 32
    for L in layers:
        if L["kind"] == "pool":
            break
        small.append(L)
    outs = R.mobilenet_v1_forward(x, small[:5])
    assert outs[1]["in"].dtype == np.float32
    np.testing.assert_array_equal(outs[1]["in"], outs[0]["ref"].astype(np.float32))
    assert np.all(outs[-1]["E"] >= 1e-5 * outs[-1]["S"])
    assert outs[-1]["ref"].shape == (1, 8, 8, 128)


def test_sample_outputs_agrees_with_the_full_loops():
    x, wt, b, m, _ = _rand_layer(2, 6, 5, 12, 8, 3, 4)
    ref, s = R.conv2d(x, wt, m, b, relu=True)
    pos = [(0, 0, 0, 0), (1, 5, 4, 7), (0, 3, 2, 5), (1, 0, 4, 2)]
    r2, s2 = R.sample_outputs(x, wt, m, b, pos, relu=True)
    for i, (n, y, xx, o) in enumerate(pos):
        assert abs(r2[i] - ref[n, y, xx, o]) < 1e-12 and abs(s2[i] - s[n, y, xx, o]) < 1e-12


# ---------------------------------------------------------------------------
# The chained MobileNet-v1 oracle (all 29 table entries) against an independent chain built here from
# torch's fp64 library convolution and mean, and its propagated bound E pinned from below and from above.
# ---------------------------------------------------------------------------

def _torch_layer(L, cur, tol_sign=None, tol=1e-5):
    """One layer of the network from library routines in fp64: NHWC in, (out, S) NHWC out.  Pointwise weights are
    multiplied by their mask; ReLU after every convolution but the classifier; the pool is a plain mean."""
    import torch.nn.functional as F
    kind = L["kind"]
    t = torch.from_numpy(np.ascontiguousarray(cur, dtype=np.float64)).permute(0, 3, 1, 2)
    if kind == "pool":
        out = t.mean(dim=(2, 3), keepdim=True)
        s = t.abs().mean(dim=(2, 3), keepdim=True)
        return out.permute(0, 2, 3, 1).numpy(), s.permute(0, 2, 3, 1).numpy()
    b = torch.from_numpy(L["bias"].astype(np.float64))
    if kind == "dw":
        w = torch.from_numpy(L["w"].astype(np.float64)).permute(2, 0, 1).unsqueeze(1)          # [C][1][3][3]
        conv = lambda a, ww, bb: F.conv2d(a, ww, bb, stride=L["stride"], padding=1, groups=a.shape[1])  # noqa: E731
    else:
        wm = L["w"].astype(np.float64)
        if "mask" in L:
            wm = wm * L["mask"]
        w = torch.from_numpy(wm).permute(0, 3, 1, 2)                                           # [Cout][Cin][KH][KW]
        pad = (w.shape[2] - 1) // 2
        conv = lambda a, ww, bb: F.conv2d(a, ww, bb, stride=L["stride"], padding=pad)          # noqa: E731
    out = conv(t, w, b)
    s = conv(t.abs(), w.abs(), b.abs())
    if kind != "fc":
        out = out.clamp_min(0)
    return out.permute(0, 2, 3, 1).numpy(), s.permute(0, 2, 3, 1).numpy()


def _small_network(seed, side=64, sparsity=50):
    """MobileNet-v1's 29 table entries on a side x side crop (the shapes scale with the image; 64 leaves a 2x2 map
    for the pool to average)."""
    from sbnn_inputs import mobilenet_v1_inputs
    x, layers = mobilenet_v1_inputs(1, sparsity, 4, seed=seed)
    return np.ascontiguousarray(x[:, :side, :side]), layers


def test_chain_every_layer_against_an_independent_fp64_chain():
    x, layers = _small_network(seed=3)
    outs = R.mobilenet_v1_forward(x, layers)
    assert [o["name"] for o in outs] == [L["name"] for L in layers] and len(outs) == 29
    # (i) layer by layer on the oracle's own fp32 inputs: value and S, tightly
    for L, rec in zip(layers, outs):
        ref, s = _torch_layer(L, rec["in"])
        assert rec["ref"].shape == ref.shape, L["name"]
        np.testing.assert_allclose(rec["ref"], ref, rtol=0, atol=1e-11 * float(np.max(s)), err_msg=L["name"])
        np.testing.assert_allclose(rec["S"], s, rtol=1e-12, atol=1e-300, err_msg=L["name"])
    # (ii) the chaining itself: each layer is fed the fp32 rounding of the previous result
    for prev, rec in zip(outs, outs[1:]):
        assert rec["in"].dtype == np.float32
        np.testing.assert_array_equal(rec["in"].reshape(-1), prev["ref"].astype(np.float32).reshape(-1))
    # (iii) a chain that never looks at the oracle's intermediates ends at the same logits (fp32 rounding between
    # layers may flip a last bit here and there, hence the looser comparison)
    cur = x
    for L in layers:
        cur = _torch_layer(L, cur)[0].astype(np.float32)
    assert cur.shape == (1, 1, 1, 1000) == outs[-1]["ref"].shape
    scale = float(np.max(np.abs(outs[-1]["ref"])))
    assert scale > 1e-3
    np.testing.assert_allclose(cur.astype(np.float64), outs[-1]["ref"], rtol=0, atol=2e-5 * scale)
    # the classifier has no ReLU (negative logits exist), the pool no ReLU either and it does average
    assert (outs[-1]["ref"] < 0).any()
    pool_in = outs[27]["in"].astype(np.float64)
    np.testing.assert_allclose(outs[27]["ref"].reshape(-1), pool_in.reshape(4, 1024).mean(axis=0), rtol=1e-13)


def _perturbed_chain(x, layers, tol, sign_of):
    """The independent fp64 chain with every layer's result moved by sign * tol * S (an implementation that uses
    its whole per-layer allowance).  No fp32 rounding between layers: E allows for that separately."""
    cur = x.astype(np.float64)
    for li, L in enumerate(layers):
        out, s = _torch_layer(L, cur)
        cur = out + sign_of(li, out.shape) * tol * s
    return cur


def test_chain_error_bound_is_pinned_from_both_sides():
    tol = 1e-5
    # (a) nonnegative weights, biases and image: every ReLU is active and nothing cancels, so a chain that errs by
    # +tol*S at every layer deviates by exactly the first-order bound; E must cover it and may not be much larger
    x, layers = _small_network(seed=4)
    pos = []
    for L in layers:
        L = dict(L)
        for k in ("w", "bias"):
            if k in L:
                L[k] = np.abs(L[k])
        pos.append(L)
    outs = R.mobilenet_v1_forward(x, pos, tol=tol)
    dev = _perturbed_chain(x, pos, tol, lambda li, shape: 1.0) - outs[-1]["ref"]
    e = outs[-1]["E"]
    assert np.all(dev > 0) and np.all(dev <= e)
    assert np.all(e <= 1.02 * dev), float(np.max(e / dev))       # slack: E also allows for rounding activations to fp32
    for rec in outs:                                             # and at every layer on the way
        assert np.all(rec["E"] >= tol * rec["S"])
    # (b) the network as generated (signed weights), errors of random sign and of one sign: inside E
    x, layers = _small_network(seed=5)
    outs = R.mobilenet_v1_forward(x, layers, tol=tol)
    r = np.random.default_rng(77)
    for sign_of in (lambda li, shape: 1.0, lambda li, shape: -1.0,
                    lambda li, shape: r.choice([-1.0, 1.0], size=shape)):
        dev = np.abs(_perturbed_chain(x, layers, tol, sign_of) - outs[-1]["ref"])
        assert np.all(dev <= outs[-1]["E"])
    # E scales with the per-layer tolerance (up to the fixed fp32-rounding allowance)
    outs10 = R.mobilenet_v1_forward(x, layers, tol=10 * tol)
    ratio = outs10[-1]["E"] / outs[-1]["E"]
    assert np.all(ratio > 9.0) and np.all(ratio <= 10.0 + 1e-9)
