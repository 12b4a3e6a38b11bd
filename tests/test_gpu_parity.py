"""GPU parity: every CUDA entry point against the CPU oracle on the same seeded inputs.

Tolerance (fp32 path): |gpu - ref| <= 1e-5 * S per output, S = |b| + sum |w*x| from the oracle.
Packed indices are compared bit for bit in test_abi_cpu.py.
"""
import numpy as np
import pytest
import torch

import paper_2310_19509_b200 as sbnn
from oracle import reference as R
from sbnn_inputs import workloads as WL
from sbnn_inputs import mobilenet_v1_inputs

pytestmark = pytest.mark.gpu
TOL = 1e-5


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def assert_within(y_gpu, ref, s, tol=TOL, what=""):
    y = y_gpu.astype(np.float64)
    assert y.shape == ref.shape, (y.shape, ref.shape)
    assert np.all(np.isfinite(y)), what
    ratio = np.abs(y - ref) / np.maximum(tol * s, 1e-300)
    bad = np.abs(y - ref) > tol * s
    assert not bad.any(), f"{what}: {bad.sum()} outputs outside tolerance, worst ratio {ratio[bad].max():.3g}"
    return float(np.max(np.where(s > 0, np.abs(y - ref) / np.maximum(tol * s, 1e-300), 0.0)))


GUARD = 256          # floats of NaN canary on either side of every output buffer


class Guarded:
    """An output buffer with GUARD floats of NaN before and after it: `t` is the tensor handed to the library
    (16-byte aligned, NaN-filled so unwritten outputs show), check() asserts that the canaries are untouched."""

    def __init__(self, shape):
        n = int(np.prod(shape))
        self.full = torch.full((n + 2 * GUARD,), float("nan"), device="cuda", dtype=torch.float32)
        self.t = self.full[GUARD:GUARD + n].view(*shape)
        self.n = n

    def check(self, what=""):
        assert bool(torch.isnan(self.full[:GUARD]).all()), f"{what}: wrote before the output buffer"
        assert bool(torch.isnan(self.full[GUARD + self.n:]).all()), f"{what}: wrote past the output buffer"

    def numpy(self, what=""):
        self.check(what)
        return self.t.cpu().numpy()


def run_1x1(d, flags=sbnn.SBNN_RELU, cfg=None):
    x = d["x"]
    n, h, w, cin = x.shape
    cout = d["w"].shape[0]
    p = sbnn.pack_weights(d["w"], d["mask"], d["bias"], d["g"])
    xd = dev(x)
    out = Guarded((n, h, w, cout))
    if cfg is None:
        sbnn.conv1x1_gs(p, xd, out.t, n, h, w, flags)
    else:
        sbnn.conv1x1_gs_tuned(p, xd, out.t, n, h, w, flags, *cfg)
    sbnn.get_async_status()
    y = out.numpy("1x1")
    p.free()
    return y


def test_config1_single_pointwise_layer():
    d = WL.config1()
    y = run_1x1(d)
    ref, s = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=True)
    worst = assert_within(y, ref, s, what="config 1")
    assert worst < 0.5       # fp32 accumulation error is far inside the bound on these inputs


CFGS = {1: [(8, 4, 8, 64)], 2: [(8, 2, 8, 64)],
        4: [(8, 1, 16, 64), (8, 2, 8, 64), (8, 2, 16, 32), (4, 1, 8, 64), (4, 2, 8, 64)],
        8: [(8, 1, 16, 32), (8, 1, 8, 64), (4, 1, 8, 64)], 16: [(4, 1, 8, 64)]}


@pytest.mark.parametrize("g", [1, 2, 4, 8, 16])
def test_every_kernel_instance_on_ragged_shapes(g):
    """Several pixel tiles with a ragged tail, several channel steps with a ragged tail, a ragged group tile."""
    for cfg in CFGS[g]:
        tm = 32 * cfg[0]
        d = WL.single_conv_inputs(1, 1, 2 * tm + 37, 148, 16 * 11, 1, g, 50, seed=3, mask_mode="layer_global")
        for relu in (True, False):
            y = run_1x1(d, sbnn.SBNN_RELU if relu else 0, cfg)
            ref, s = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=relu)
            assert_within(y, ref, s, what=f"G={g} cfg={cfg} relu={relu}")


@pytest.mark.parametrize("shape", [(1, 1, 1, 4, 4), (1, 7, 7, 12, 8), (2, 3, 5, 32, 64), (1, 1, 300, 8, 1000)])
def test_small_and_odd_shapes(shape):
    n, h, w, cin, cout = shape
    for sp in (0, 50, 100):
        d = WL.single_conv_inputs(n, h, w, cin, cout, 1, 4, sp, seed=5)
        y = run_1x1(d)
        ref, s = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=True)
        assert_within(y, ref, s, what=f"{shape} sp={sp}")


def test_group_without_kept_units_and_zero_bias_gives_exact_zero():
    d = WL.single_conv_inputs(1, 5, 5, 16, 16, 1, 4, 50, seed=2)
    d["mask"][4:8] = 0
    d["bias"][4:8] = 0.0
    y = run_1x1(d, 0)
    assert not y[..., 4:8].any()
    ref, s = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=False)
    assert_within(y, ref, s)


def test_paper_style_4x4_blocks_and_magnitude_masks():
    for mode, gi in (("balanced", 4), ("magnitude", 1)):
        d = WL.single_conv_inputs(1, 9, 13, 64, 64, 1, 4, 30, seed=9, mask_mode=mode, gi=gi)
        y = run_1x1(d)
        ref, s = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=True)
        assert_within(y, ref, s, what=mode)


def test_empty_batch_is_ok():
    d = WL.single_conv_inputs(1, 1, 1, 8, 8, 1, 4, 50)
    p = sbnn.pack_weights(d["w"], d["mask"], d["bias"], 4)
    x = torch.zeros(16, device="cuda")
    sbnn.conv1x1_gs(p, x, x, 0, 5, 5)


@pytest.mark.parametrize("stride", [1, 2])
@pytest.mark.parametrize("shape", [(2, 9, 11, 32), (1, 14, 14, 512), (1, 1, 1, 4), (1, 7, 7, 8)])
def test_depthwise(stride, shape):
    n, h, w, c = shape
    rng = np.random.default_rng(11)
    x = rng.random((n, h, w, c), dtype=np.float32)
    wt = rng.standard_normal((3, 3, c)).astype(np.float32)
    b = rng.standard_normal(c).astype(np.float32)
    ho, wo = (h - 1) // stride + 1, (w - 1) // stride + 1
    yd = torch.full((n, ho, wo, c), float("nan"), device="cuda")
    sbnn.dwconv3x3(dev(wt), dev(b), dev(x), yd, n, h, w, c, stride)
    sbnn.get_async_status()
    ref, s = R.dwconv3x3(x, wt, b, stride=stride, relu=True)
    assert_within(yd.cpu().numpy(), ref, s, what=f"dw {shape} s{stride}")


@pytest.mark.parametrize("stride,hw", [(1, (8, 8)), (1, (6, 8)), (1, (14, 14)), (1, (7, 14)), (1, (7, 7)), (1, (5, 6)),
                                       (2, (8, 16)), (2, (6, 8)), (2, (28, 28)), (2, (14, 14)), (2, (6, 6))])
@pytest.mark.parametrize("n,c", [(3, 5), (2, 37)])
def test_depthwise_channel_major_variants(stride, hw, n, c):
    """Every kernel behind the channel-major depthwise entry point (row blocks, the stride-2 row blocks, the one-row
    fallbacks, the 14 x 14 kernel, column strips, one output per thread), several images and channel counts that do
    not fill a CTA's channel slots, leading dimensions with padding."""
    h, w = hw
    rng = np.random.default_rng(41)
    x = rng.random((n, h, w, c), dtype=np.float32)
    wt = rng.standard_normal((3, 3, c)).astype(np.float32)
    b = rng.standard_normal(c).astype(np.float32)
    ho, wo = (h - 1) // stride + 1, (w - 1) // stride + 1
    ldx, ldy = (n * h * w + 3) // 4 * 4 + 4, (n * ho * wo + 3) // 4 * 4 + 8
    xt = torch.zeros((c, ldx), device="cuda")
    xt[:, :n * h * w] = dev(x).reshape(n * h * w, c).t()
    yt = torch.full((c, ldy), float("nan"), device="cuda")
    sbnn.dwconv3x3_cm(dev(wt), dev(b), xt, ldx, yt, ldy, n, h, w, c, stride)
    sbnn.get_async_status()
    y = yt[:, :n * ho * wo].t().reshape(n, ho, wo, c).cpu().numpy()
    ref, s = R.dwconv3x3(x, wt, b, stride=stride, relu=True)
    assert_within(y, ref, s, what=f"dw cm {hw} s{stride} n={n} c={c}")
    assert bool(torch.isnan(yt[:, n * ho * wo:]).all())          # nothing written past the last pixel


def test_depthwise_7x7_kernel_with_more_images_than_one_cta_takes():
    """The 7 x 7 kernel stages 64 images of two channels per CTA: 70 images give a full and a partial chunk, 5 channels
    an odd last pair."""
    rng = np.random.default_rng(42)
    n, c = 70, 5
    x = rng.random((n, 7, 7, c), dtype=np.float32)
    wt = rng.standard_normal((3, 3, c)).astype(np.float32)
    b = rng.standard_normal(c).astype(np.float32)
    ld = (n * 49 + 3) // 4 * 4 + 4
    xt = torch.zeros((c, ld), device="cuda")
    xt[:, :n * 49] = dev(x).reshape(n * 49, c).t()
    out = Guarded((c, ld))
    sbnn.dwconv3x3_cm(dev(wt), dev(b), xt, ld, out.t, ld, n, 7, 7, c, 1)
    sbnn.get_async_status()
    full = out.numpy("dw 7x7")
    assert np.all(np.isnan(full[:, n * 49:]))
    ref, s = R.dwconv3x3(x, wt, b, stride=1, relu=True)
    assert_within(full[:, :n * 49].T.reshape(n, 7, 7, c), ref, s, what="dw 7x7, 70 images")


@pytest.mark.parametrize("n,h,w,cin,cout,relu_dw", [(3, 20, 28, 32, 64, True), (2, 9, 112, 32, 64, True), (5, 8, 12, 72, 40, False),
                                                    (1, 56, 56, 128, 128, True), (2, 3, 4, 8, 8, True)])
def test_fused_depthwise_pointwise(n, h, w, cin, cout, relu_dw):
    """sbnn_dwconv3x3_conv1x1_gs_cm: depthwise 3x3 (stride 1) and group-sparse 1x1 in one kernel.  Several images (runs of
    256 pixels cross image borders, so every padding mask is exercised), the widest supported map, a ragged last pixel
    tile, several channel steps and group tiles, a channel count that is not a multiple of the step.  Oracle: depthwise
    in fp64, rounded to fp32 as a stored activation would be, then the masked dense 1x1; the bound adds what the
    depthwise layer's own tolerance and that rounding can contribute through |W~|."""
    rng = np.random.default_rng(51)
    x = rng.random((n, h, w, cin), dtype=np.float32)
    dw_w = (rng.standard_normal((3, 3, cin)) * 0.4).astype(np.float32)
    dw_b = (rng.standard_normal(cin) * 0.1).astype(np.float32)
    d = WL.single_conv_inputs(1, 1, 4, cin, cout, 1, 4, 50, seed=52, mask_mode="layer_global")
    m = n * h * w
    ldx, ldy = (m + 3) // 4 * 4 + 4, (m + 3) // 4 * 4
    xt = torch.full((cin, ldx), float("nan"), device="cuda")
    xt[:, :m] = dev(x).reshape(m, cin).t()
    out = Guarded((cout, ldy))
    p = sbnn.pack_weights(d["w"], d["mask"], d["bias"], 4)
    sbnn.dwconv3x3_conv1x1_gs_cm(p, dev(dw_w), dev(dw_b), xt, ldx, out.t, ldy, n, h, w,
                                 sbnn.SBNN_RELU if relu_dw else 0, sbnn.SBNN_RELU)
    sbnn.get_async_status()
    full = out.numpy("fused")
    assert np.all(np.isnan(full[:, m:]))
    y = full[:, :m].T.reshape(n, h, w, cout).astype(np.float64)
    mid, s_dw = R.dwconv3x3(x, dw_w, dw_b, stride=1, relu=relu_dw)
    mid32 = mid.astype(np.float32)
    ref, s_pw = R.conv2d(mid32, d["w"], d["mask"], d["bias"], relu=True)
    e_mid = (1e-5 * s_dw + np.abs(mid) * 2.0 ** -23).astype(np.float32)          # depthwise tolerance + one fp32 rounding
    prop, _ = R.conv2d(e_mid, np.abs(d["w"]), d["mask"], None, relu=False)
    bound = 1e-5 * s_pw + prop * (1 + 1e-6)
    err = np.abs(y - ref)
    assert np.all(np.isfinite(y))
    assert np.all(err <= bound), f"worst ratio {np.max(err / np.maximum(bound, 1e-300))}"
    # and the two-kernel route agrees within the same bound
    yt2 = torch.full((cin, ldy), float("nan"), device="cuda")
    sbnn.dwconv3x3_cm(dev(dw_w), dev(dw_b), xt, ldx, yt2, ldy, n, h, w, cin, 1, sbnn.SBNN_RELU if relu_dw else 0)
    out2 = Guarded((cout, ldy))
    sbnn.conv1x1_gs_cm(p, yt2, ldy, out2.t, ldy, m, sbnn.SBNN_RELU | sbnn.SBNN_OUT_CM)
    sbnn.get_async_status()
    y2 = out2.numpy("two kernels")[:, :m].T.reshape(n, h, w, cout).astype(np.float64)
    assert np.all(np.abs(y2 - ref) <= bound)
    p.free()


def test_fused_depthwise_pointwise_refuses_what_it_does_not_take():
    d = WL.single_conv_inputs(1, 1, 4, 16, 16, 1, 8, 50, seed=53)
    p = sbnn.pack_weights(d["w"], d["mask"], d["bias"], 8)
    xt = torch.zeros((16, 64), device="cuda")
    yt = torch.zeros((16, 64), device="cuda")
    w9, b = torch.zeros((3, 3, 16), device="cuda"), torch.zeros(16, device="cuda")
    with pytest.raises(sbnn.SbnnError) as e:
        sbnn.dwconv3x3_conv1x1_gs_cm(p, w9, b, xt, 64, yt, 64, 1, 8, 8)           # G = 8
    assert e.value.name == "SBNN_ERR_UNSUPPORTED"
    p.free()
    d = WL.single_conv_inputs(1, 1, 4, 16, 16, 1, 4, 50, seed=53)
    p = sbnn.pack_weights(d["w"], d["mask"], d["bias"], 4)
    with pytest.raises(sbnn.SbnnError) as e:
        sbnn.dwconv3x3_conv1x1_gs_cm(p, w9, b, xt, 64, yt, 64, 1, 9, 7)           # width not a multiple of 4
    assert e.value.name in ("SBNN_ERR_UNSUPPORTED", "SBNN_ERR_SHAPE")
    sbnn.get_async_status()
    p.free()


@pytest.mark.parametrize("stride", [1, 2])
@pytest.mark.parametrize("shape,go", [((2, 9, 11, 32), 16), ((1, 14, 14, 48), 8), ((1, 1, 1, 4), 4), ((3, 7, 7, 64), 16)])
def test_depthwise_3of9_patterns(stride, shape, go):
    """Depthwise 3x3 with 3:9 kernel patterns (compact weights + PatternInfo through the C interface) against the
    oracle's dense depthwise convolution on the masked weights."""
    from sbnn_inputs import dw_pattern_mask
    n, h, w, c = shape
    rng = np.random.default_rng(31)
    x = rng.random((n, h, w, c), dtype=np.float32)
    wt = rng.standard_normal((3, 3, c)).astype(np.float32)
    b = rng.standard_normal(c).astype(np.float32)
    m = dw_pattern_mask(7, 5, c, go)
    pat, w6 = sbnn.pack_dw_pattern(wt, m, go)
    ho, wo = (h - 1) // stride + 1, (w - 1) // stride + 1
    yd = torch.full((n, ho, wo, c), float("nan"), device="cuda")
    sbnn.dwconv3x3_pattern(dev(w6), torch.from_numpy(pat).cuda(), go, dev(b), dev(x), yd, n, h, w, c, stride)
    sbnn.get_async_status()
    ref, s = R.dwconv3x3(x, np.where(m != 0, wt, np.float32(0)), b, stride=stride, relu=True)
    assert_within(yd.cpu().numpy(), ref, s, what=f"dw 3:9 {shape} go={go} s{stride}")


@pytest.mark.parametrize("stride,shape", [(2, (2, 32, 32, 3, 32)), (1, (1, 9, 7, 3, 32)), (2, (1, 15, 17, 4, 8))])
def test_thin_dense_conv(stride, shape):
    n, h, w, cin, cout = shape
    rng = np.random.default_rng(12)
    x = rng.random((n, h, w, cin), dtype=np.float32)
    wt = rng.standard_normal((cout, 3, 3, cin)).astype(np.float32)
    b = rng.standard_normal(cout).astype(np.float32)
    ho, wo = (h - 1) // stride + 1, (w - 1) // stride + 1
    yd = torch.full((n, ho, wo, cout), float("nan"), device="cuda")
    sbnn.conv3x3_dense(dev(wt), dev(b), dev(x), yd, n, h, w, cin, cout, stride)
    sbnn.get_async_status()
    ref, s = R.conv2d(x, wt, np.ones_like(wt, dtype=np.uint8), b, stride=stride, relu=True)
    assert_within(yd.cpu().numpy(), ref, s, what=f"conv0 {shape}")


def test_avgpool():
    rng = np.random.default_rng(13)
    x = rng.standard_normal((3, 7, 7, 64)).astype(np.float32)
    yd = torch.full((3, 64), float("nan"), device="cuda")
    sbnn.avgpool(dev(x), yd, 3, 49, 64)
    ref, s = R.avgpool(x)
    assert_within(yd.cpu().numpy(), ref, s, what="avgpool")


def build_net(layers, max_batch):
    pw = [sbnn.pack_weights(L["w"], L["mask"], L["bias"], L["g"]) for L in layers if L["kind"] == "pw"]
    fcL = [L for L in layers if L["kind"] == "fc"][0]
    fc = sbnn.pack_weights(fcL["w"], fcL["mask"], fcL["bias"], fcL["g"])
    dw_w = [dev(L["w"]) for L in layers if L["kind"] == "dw"]
    dw_b = [dev(L["bias"]) for L in layers if L["kind"] == "dw"]
    c0 = layers[0]
    return sbnn.MobileNetV1(pw, fc, dw_w, dw_b, dev(c0["w"]), dev(c0["bias"]), max_batch)


@pytest.mark.parametrize("sparsity", [30])
def test_mobilenet_v1_batch1_layer_isolated_and_end_to_end(sparsity):
    x, layers = mobilenet_v1_inputs(1, sparsity, 4, seed=0)
    outs = R.mobilenet_v1_forward(x, layers)
    net = build_net(layers, 2)
    # (i) every layer alone, fed the oracle's fp32 input of that layer
    for li, rec in enumerate(outs):
        ref, s = rec["ref"], rec["S"]
        out = Guarded(ref.shape)
        net.run_layer(li, dev(rec["in"]), out.t, 1)
        sbnn.get_async_status()
        assert_within(out.numpy(f"layer {li}"), ref, s, what=f"layer {li} {rec['name']}")
    # (ii) the chain, against the propagated first-order bound
    lg = Guarded((1, 1000))
    logits = lg.t
    net.forward(dev(x), logits, 1)
    sbnn.get_async_status()
    y = lg.numpy("forward").astype(np.float64).reshape(outs[-1]["ref"].shape)
    err = np.abs(y - outs[-1]["ref"])
    assert np.all(err <= outs[-1]["E"]), f"worst ratio {np.max(err / outs[-1]['E'])}"
    # two copies of the image in one call give the same logits twice, bit for bit, and the single-image result
    # within the bound (the kernel picked for a layer, hence the order of its sums, depends on the pixel count)
    x2 = np.concatenate([x, x])
    l2 = torch.full((2, 1000), float("nan"), device="cuda")
    net.forward(dev(x2), l2, 2)
    sbnn.get_async_status()
    assert torch.equal(l2[0], l2[1])
    err2 = np.abs(l2[0].cpu().numpy().astype(np.float64).reshape(outs[-1]["ref"].shape) - outs[-1]["ref"])
    assert np.all(err2 <= outs[-1]["E"])
    net.free()


def test_forward_prefix_gives_the_intermediate_activations():
    """sbnn_mobilenet_v1_forward_prefix: the output of a middle pointwise layer, of the last depthwise layer and of the
    pool, each in the chain's channel-major layout, against the oracle's chained result within its propagated bound;
    the full prefix equals forward's logits bit for bit."""
    x, layers = mobilenet_v1_inputs(1, 30, 4, seed=0)
    outs = R.mobilenet_v1_forward(x, layers)
    net = build_net(layers, 1)
    xd = dev(x)
    for li in (6, 25, 27):
        ref, e = outs[li]["ref"], outs[li]["E"]
        n_, h_, w_, c_ = ref.shape
        ld = (n_ * h_ * w_ + 3) // 4 * 4
        out = Guarded((c_, ld))
        net.forward_prefix(xd, out.t, 1, li)
        sbnn.get_async_status()
        y = out.numpy(f"prefix {li}")[:, :n_ * h_ * w_].T.reshape(ref.shape).astype(np.float64)
        err = np.abs(y - ref)
        assert np.all(err <= e), f"layer {li}: worst ratio {np.max(err / np.maximum(e, 1e-300))}"
    lg, lp = Guarded((1, 1000)), Guarded((1, 1000))
    net.forward(xd, lg.t, 1)
    net.forward_prefix(xd, lp.t, 1, 28)
    sbnn.get_async_status()
    assert np.array_equal(lg.numpy("forward"), lp.numpy("prefix 28"))
    net.free()


def test_forward_graph_replay_matches_plain_launches():
    """forward records a CUDA graph on its second call with the same buffers and replays it afterwards: replays
    must give, bit for bit, what the plain first call gave, follow the current contents of the input buffer, and a
    different batch size on the same buffers must not reuse the recording."""
    x, layers = mobilenet_v1_inputs(2, 50, 4, seed=5)
    net = build_net(layers, 2)
    xd = dev(x)
    logits = torch.full((2, 1000), float("nan"), device="cuda")
    net.forward(xd, logits, 2)                       # plain
    sbnn.get_async_status()
    first = logits.clone()
    for _ in range(3):                               # recorded, then replayed twice
        logits.fill_(float("nan"))
        net.forward(xd, logits, 2)
        sbnn.get_async_status()
        assert torch.equal(logits, first)
    xd.copy_(xd.flip(0))                             # same buffer, other contents: the two images swapped
    net.forward(xd, logits, 2)
    sbnn.get_async_status()
    assert torch.equal(logits, first.flip(0))
    one = torch.full((2, 1000), float("nan"), device="cuda")
    for _ in range(3):                               # N = 1 on the same input buffer: its own recording
        net.forward(xd, one, 1)
        sbnn.get_async_status()
        assert bool(torch.isfinite(one[0]).all()) and bool(torch.isnan(one[1]).all())
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):                    # replay on another stream than the one it was first used on
        side.wait_stream(torch.cuda.current_stream())
        logits.fill_(float("nan"))
        net.forward(xd, logits, 2, stream=side)
        side.synchronize()
    assert torch.equal(logits, first.flip(0))
    net.free()


def test_forward_accepts_an_image_that_is_only_4_byte_aligned():
    """The first layer's fast kernel needs 16-byte aligned rows; an input at an odd float offset takes the generic
    first-layer kernel.  Both routes are compared with the oracle's chain (propagated bound), and the generic
    first-layer kernel alone with the oracle's first layer."""
    x, layers = mobilenet_v1_inputs(1, 50, 4, seed=6)
    outs = R.mobilenet_v1_forward(x, layers)
    ref, e = outs[-1]["ref"].reshape(1, 1000), outs[-1]["E"].reshape(1, 1000)
    net = build_net(layers, 1)
    flat = torch.zeros(x.size + 1, device="cuda")
    flat[1:] = dev(x).reshape(-1)
    for src in (dev(x), flat[1:]):                   # aligned (fast first-layer kernel), then at an odd float offset
        lg = Guarded((1, 1000))
        net.forward(src, lg.t, 1)
        sbnn.get_async_status()
        y = lg.numpy("forward").astype(np.float64)
        assert np.all(np.isfinite(y))
        assert np.all(np.abs(y - ref) <= e), f"worst ratio {np.max(np.abs(y - ref) / e)}"
    # layer 0 alone on the unaligned image, against the oracle's first layer
    out = Guarded(outs[0]["ref"].shape)
    net.run_layer(0, flat[1:], out.t, 1)
    sbnn.get_async_status()
    assert_within(out.numpy("conv0"), outs[0]["ref"], outs[0]["S"], what="first layer, 4-byte aligned image")
    net.free()


def run_3x3(d, flags=sbnn.SBNN_RELU):
    x = d["x"]
    n, h, w, cin = x.shape
    cout = d["w"].shape[0]
    p = sbnn.pack_weights(d["w"], d["mask"], d["bias"], d["g"])
    out = Guarded((n, h, w, cout))
    sbnn.conv3x3_gs(p, dev(x), out.t, n, h, w, flags)
    sbnn.get_async_status()
    y = out.numpy("3x3")
    p.free()
    return y


def test_config4_group_sparse_3x3_reduced_batch():
    """Config 4's layer (28x28, 256 -> 256, G=4, half of the kernels removed) on 3 images: the CTA tiles of
    56 image rows span image boundaries, with a ragged last tile."""
    d = WL.config4(n=3)
    y = run_3x3(d)
    ref, s = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=True)
    worst = assert_within(y, ref, s, what="config 4 (n=3)")
    assert worst < 0.5


@pytest.mark.parametrize("g", [1, 2, 4, 8, 16])
@pytest.mark.parametrize("hw", [(5, 5), (9, 13), (14, 14), (7, 32), (3, 57), (6, 100)])
def test_3x3_shapes_and_groups(g, hw):
    h, w = hw
    d = WL.single_conv_inputs(2, h, w, 20, 48, 3, g, 50, seed=4, w_sigma=0.1, mask_mode="layer_global")
    for relu in (True, False):
        y = run_3x3(d, sbnn.SBNN_RELU if relu else 0)
        ref, s = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=relu)
        assert_within(y, ref, s, what=f"3x3 G={g} {hw} relu={relu}")


@pytest.mark.parametrize("g,n,h,w,cin,cout", [(4, 40, 14, 28, 64, 64), (4, 9, 7, 28, 40, 96), (8, 12, 14, 28, 64, 128),
                                               (2, 30, 8, 56, 32, 24), (1, 20, 10, 28, 24, 40), (16, 6, 28, 28, 48, 64),
                                               (4, 200, 14, 28, 16, 32), (4, 20, 14, 28, 40, 72), (4, 3, 56, 56, 24, 120),
                                               (16, 20, 16, 8, 16, 32)])   # (8-wide map, 224 rows per CTA: one stage only)
def test_3x3_tiles_split_between_persistent_ctas(g, n, h, w, cin, cout):
    """The pipelined 3x3 kernel deals the channel steps of all tiles to one CTA per SM in equal shares.  Shapes with
    a few steps per CTA (every tile cut into several parts whose partial sums the last arrival adds), with about as
    many tiles as CTAs (tiles cut in two) and with many more tiles than CTAs (most tiles whole); even heights run two
    output rows per lane (G <= 4; both tile shapes of G = 4: 3 x 4 warps with 8-channel steps, 2 x 6 warps with 16-channel
    steps where the group count suits tiles of six), odd heights and wider groups one.  Every output against the oracle."""
    d = WL.single_conv_inputs(n, h, w, cin, cout, 3, g, 50, seed=21, w_sigma=0.05)
    for relu in (True, False):
        y = run_3x3(d, sbnn.SBNN_RELU if relu else 0)
        ref, s = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=relu)
        assert_within(y, ref, s, what=f"3x3 split tiles G={g} n={n} {h}x{w} {cin}->{cout} relu={relu}")


@pytest.mark.parametrize("g,n,h,w,cin,cout", [(4, 3, 28, 28, 256, 256), (4, 5, 14, 28, 40, 72), (8, 4, 7, 28, 32, 64),
                                               (2, 3, 8, 56, 24, 20), (16, 2, 6, 100, 20, 48), (1, 2, 10, 12, 8, 7),
                                               (4, 6, 14, 14, 64, 48), (8, 9, 7, 7, 32, 40), (4, 2, 5, 13, 12, 8), (16, 20, 16, 8, 16, 32)])
def test_3x3_channel_major_entry(g, n, h, w, cin, cout):
    """sbnn_conv3x3_gs_cm: activations given as channel-major planes (the layout the pipelined kernel stages from, no
    conversion pass), output pixel-major or, with SBNN_OUT_CM, channel-major with a padded leading dimension whose
    padding must stay untouched.  Every output against the oracle; both agree bit for bit with each other."""
    d = WL.single_conv_inputs(n, h, w, cin, cout, 3, g, 50, seed=31, w_sigma=0.05)
    p = sbnn.pack_weights(d["w"], d["mask"], d["bias"], g)
    m = n * h * w
    ld = (m + 3) // 4 * 4 + 8
    xt = torch.full((cin, ld), float("nan"), device="cuda")
    sbnn.to_channel_major(dev(d["x"]), xt, m, cin, ld)
    ref, s = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=True)
    ldy = (cout + 3) // 4 * 4
    y_pm = torch.full((m, ldy), float("nan"), device="cuda")
    sbnn.conv3x3_gs_cm(p, xt, ld, y_pm, ldy, n, h, w, sbnn.SBNN_RELU)
    sbnn.get_async_status()
    got = y_pm[:, :cout].cpu().numpy().reshape(n, h, w, cout)
    assert_within(got, ref, s, what=f"3x3 channel-major in, pixel-major out G={g}")
    assert torch.isnan(y_pm[:, cout:]).all()
    y_cm = torch.full((cout, ld), float("nan"), device="cuda")
    sbnn.conv3x3_gs_cm(p, xt, ld, y_cm, ld, n, h, w, sbnn.SBNN_RELU | sbnn.SBNN_OUT_CM)
    sbnn.get_async_status()
    assert torch.isnan(y_cm[:, m:]).all()
    assert torch.equal(y_cm[:, :m].t().contiguous(), y_pm[:, :cout].contiguous())
    p.free()


def test_bottleneck_block_chained_in_channel_major_layout():
    """1x1 (256 -> 64) -> 3x3 (64 -> 64) -> 1x1 (64 -> 256), all group-sparse (G = 4, 50 %), chained on the device in the
    channel-major layout with no conversion between the layers.  Each layer is checked against the oracle applied to
    the activations the previous GPU layer produced (so a layer's tolerance is its own, not a propagated one)."""
    n, h, w = 6, 28, 28
    m = n * h * w
    ld = (m + 3) // 4 * 4
    shapes = [(256, 64, 1), (64, 64, 3), (64, 256, 1)]
    layers = [WL.single_conv_inputs(n, h, w, ci, co, k, 4, 50, seed=40 + i, w_sigma=0.05, layer=i) for i, (ci, co, k) in enumerate(shapes)]
    packed = [sbnn.pack_weights(d["w"], d["mask"], d["bias"], 4) for d in layers]
    xt = torch.full((256, ld), float("nan"), device="cuda")
    sbnn.to_channel_major(dev(layers[0]["x"]), xt, m, 256, ld)
    acts = [xt] + [torch.full((co, ld), float("nan"), device="cuda") for _, co, _ in shapes]
    fl = sbnn.SBNN_RELU | sbnn.SBNN_OUT_CM
    sbnn.conv1x1_gs_cm(packed[0], acts[0], ld, acts[1], ld, m, fl)
    sbnn.conv3x3_gs_cm(packed[1], acts[1], ld, acts[2], ld, n, h, w, fl)
    sbnn.conv1x1_gs_cm(packed[2], acts[2], ld, acts[3], ld, m, fl)
    sbnn.get_async_status()
    host = [a[:, :m].t().contiguous().cpu().numpy() for a in acts]       # [m][C] each
    for i, (d, (ci, co, k)) in enumerate(zip(layers, shapes)):
        xin = host[i].reshape(n, h, w, ci)
        ref, s = R.conv2d(xin, d["w"], d["mask"], d["bias"], relu=True)
        assert_within(host[i + 1].reshape(n, h, w, co), ref, s, what=f"bottleneck layer {i} ({k}x{k}, {ci} -> {co})")
    for p in packed:
        p.free()


def test_3x3_channel_major_entry_refuses_what_it_cannot_run():
    d = WL.single_conv_inputs(1, 6, 6, 8, 8, 3, 4, 50, seed=32)
    p = sbnn.pack_weights(d["w"], d["mask"], d["bias"], 4)
    xt = torch.zeros((8, 40), device="cuda")
    y = torch.zeros((36, 8), device="cuda")
    with pytest.raises(sbnn.SbnnError, match="SBNN_ERR_SHAPE"):            # ldy < Cout
        sbnn.conv3x3_gs_cm(p, xt, 40, y, 4, 1, 6, 6, sbnn.SBNN_RELU)
    with pytest.raises(sbnn.SbnnError, match="SBNN_ERR_SHAPE"):            # ldx < M
        sbnn.conv3x3_gs_cm(p, xt, 32, y, 8, 1, 6, 6, sbnn.SBNN_RELU)
    wide_x, wide_y = torch.zeros((8, 240), device="cuda"), torch.zeros((240, 8), device="cuda")
    with pytest.raises(sbnn.SbnnError, match="SBNN_ERR_UNSUPPORTED"):      # rows of 240 pixels are wider than a staged plane row
        sbnn.conv3x3_gs_cm(p, wide_x, 240, wide_y, 8, 1, 1, 240, sbnn.SBNN_RELU)
    p.free()


@pytest.mark.parametrize("seed", list(range(24)))
def test_3x3_seeded_random_shapes(seed):
    """Shapes drawn from a seeded generator (widths 1-44 including odd ones, which the library pads to whole 16-byte
    rows; heights 1-20, odd and even; every group width; empty, sparse and dense masks; Cin a multiple of 4), through
    the pixel-major entry point and through the channel-major one.  Every output against the oracle."""
    rng = np.random.default_rng(1000 + seed)
    g = int(rng.choice([1, 2, 4, 8, 16]))
    n, h, w = int(rng.integers(1, 6)), int(rng.integers(1, 21)), int(rng.integers(1, 45))
    cin = 4 * int(rng.integers(1, 11))
    cout = g * int(rng.integers(1, 9))
    sp = int(rng.choice([0, 30, 50, 50, 80, 100]))
    relu = bool(rng.integers(0, 2))
    d = WL.single_conv_inputs(n, h, w, cin, cout, 3, g, sp, seed=100 + seed, w_sigma=0.1, mask_mode="layer_global")
    ref, s = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=relu)
    what = f"seed {seed}: {n}x{h}x{w}, {cin} -> {cout}, G={g}, {sp} % pruned, relu={relu}"
    y = run_3x3(d, sbnn.SBNN_RELU if relu else 0)
    assert_within(y, ref, s, what=what)
    if True:                                                    # every width: odd ones are padded into the scratch buffer
        p = sbnn.pack_weights(d["w"], d["mask"], d["bias"], g)
        m = n * h * w
        ld = (m + 3) // 4 * 4
        xt = torch.full((cin, ld), float("nan"), device="cuda")
        sbnn.to_channel_major(dev(d["x"]), xt, m, cin, ld)
        out = Guarded((cout, ld))
        sbnn.conv3x3_gs_cm(p, xt, ld, out.t, ld, n, h, w, (sbnn.SBNN_RELU if relu else 0) | sbnn.SBNN_OUT_CM)
        sbnn.get_async_status()
        full = out.numpy(what)
        assert np.all(np.isnan(full[:, m:]))
        assert_within(full[:, :m].T.reshape(n, h, w, cout), ref, s, what=what + " (channel-major)")
        p.free()


def test_3x3_same_result_on_every_run():
    """Split tiles are added in part order whichever part arrives last: two runs agree bit for bit."""
    d = WL.single_conv_inputs(40, 14, 28, 64, 64, 3, 4, 50, seed=22, w_sigma=0.05)
    y0 = run_3x3(d)
    for _ in range(3):
        assert np.array_equal(run_3x3(d), y0)


@pytest.mark.parametrize("g,kept_taps", [(4, 4), (2, 4), (8, 6), (8, 3), (16, 2), (1, 1)])
def test_3x3_kernel_patterns(g, kept_taps):
    """Kernels pruned tap by tap (centre + kept_taps - 1 others, one pattern per group and input channel, packed by
    sbnn_pack_weights_pattern) on top of 50 % removed kernels: same result as the oracle's masked dense convolution."""
    from sbnn_inputs import tap_pattern_mask, group_mask_balanced
    d = WL.single_conv_inputs(2, 9, 28, 24, 32, 3, g, 50, seed=14, w_sigma=0.1)
    um = group_mask_balanced(14, 3, 32 // g, 24, 50)
    m = tap_pattern_mask(14, 19, um, g, kept_taps)
    p = sbnn.pack_weights(d["w"], m, d["bias"], g, tap_patterns=True)
    n, h, w, _ = d["x"].shape
    yd = torch.full((n, h, w, 32), float("nan"), device="cuda")
    sbnn.conv3x3_gs(p, dev(d["x"]), yd, n, h, w, sbnn.SBNN_RELU)
    sbnn.get_async_status()
    ref, s = R.conv2d(d["x"], d["w"], m, d["bias"], relu=True)
    assert_within(yd.cpu().numpy(), ref, s, what=f"3x3 patterns G={g} taps={kept_taps}")
    p.free()


def test_3x3_kernel_patterns_on_config4_shape():
    """Config 4's layer (28 x 28, 256 -> 256, G = 4, half of the kernels removed) on 2 images with the 56 four-tap
    patterns on top: the tiled-copy kernel skips the pruned taps of every unit (several channel steps, two images in
    one CTA's rows) and must still match the oracle's masked dense convolution."""
    from sbnn_inputs import tap_pattern_mask
    d = WL.config4(n=2)
    m = tap_pattern_mask(0, 19, d["unit_mask"], 4, 4)
    p = sbnn.pack_weights(d["w"], m, d["bias"], 4, tap_patterns=True)
    n, h, w, _ = d["x"].shape
    out = Guarded((n, h, w, 256))
    sbnn.conv3x3_gs(p, dev(d["x"]), out.t, n, h, w, sbnn.SBNN_RELU)
    sbnn.get_async_status()
    ref, s = R.conv2d(d["x"], d["w"], m, d["bias"], relu=True)
    assert_within(out.numpy("3x3 patterns"), ref, s, what="3x3 four-tap patterns, config-4 shape")
    p.free()


def test_3x3_row_too_wide_for_the_tiled_copy():
    """A 252-pixel row needs a plane pitch above the copy engine's 256-element box limit: the cp.async variant runs."""
    d = WL.single_conv_inputs(1, 3, 252, 12, 16, 3, 4, 50, seed=15, w_sigma=0.1)
    y = run_3x3(d)
    ref, s = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=True)
    assert_within(y, ref, s, what="3x3 W=252")


def test_3x3_dense_and_empty_masks():
    for sp in (0, 100):
        d = WL.single_conv_inputs(1, 8, 8, 8, 8, 3, 4, sp, seed=6)
        y = run_3x3(d)
        ref, s = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=True)
        assert_within(y, ref, s, what=f"3x3 sp={sp}")


CM_CFGS = {1: [(8, 4, 8, 32)], 2: [(8, 2, 8, 32)],
           4: [(8, 1, 16, 32), (8, 2, 8, 32), (8, 2, 11, 32), (8, 2, 12, 32), (4, 1, 8, 32),
               (8, 1, 16, 64), (8, 2, 8, 64), (8, 2, 11, 64), (8, 2, 12, 64)],
           8: [(8, 1, 8, 32), (8, 1, 12, 32), (4, 1, 16, 32), (8, 1, 8, 64), (8, 1, 12, 64)], 16: [(4, 1, 8, 32)]}


def run_cm(d, flags, tile, out_cm):
    x = d["x"]
    n, h, w, cin = x.shape
    m = n * h * w
    cout = d["w"].shape[0]
    p = sbnn.pack_weights(d["w"], d["mask"], d["bias"], d["g"])
    ld = (m + 3) // 4 * 4
    xt = torch.full((cin, ld), float("nan"), device="cuda")
    sbnn.to_channel_major(dev(x), xt, m, cin, ld)
    if out_cm:
        out = Guarded((cout, ld))
        sbnn.conv1x1_gs_cm(p, xt, ld, out.t, ld, m, flags | sbnn.SBNN_OUT_CM, tile)
        sbnn.get_async_status()
        full = out.numpy("cm")
        assert np.all(np.isnan(full[:, m:]))                 # the row padding past the last pixel stays untouched
        y = full[:, :m].T.reshape(n, h, w, cout)
    else:
        out = Guarded((m, cout))
        sbnn.conv1x1_gs_cm(p, xt, ld, out.t, cout, m, flags, tile)
        sbnn.get_async_status()
        y = out.numpy("cm").reshape(n, h, w, cout)
    p.free()
    return y


def test_to_channel_major_is_a_transpose():
    x = torch.rand((1000 + 3, 70), device="cuda")
    ld = 1004
    xt = torch.zeros((70, ld), device="cuda")
    sbnn.to_channel_major(x, xt, 1003, 70, ld)
    assert torch.equal(xt[:, :1003], x.t())


@pytest.mark.parametrize("g", [1, 2, 4, 8, 16])
def test_channel_major_kernel_instances(g):
    """Every compiled instance of the bulk-copy pipeline kernel: several pixel tiles with a ragged tail that is
    not a multiple of 4, more channel steps than pipeline stages with a ragged last step, a ragged group tile."""
    for cfg in CM_CFGS[g]:
        tm = 32 * cfg[0]
        for sp in (50, 75):          # sparse layers take the staged pixel-major epilogue where the tile shape has one
            d = WL.single_conv_inputs(1, 1, 2 * tm + 37, 212, 16 * 11, 1, g, sp, seed=8, mask_mode="layer_global")
            for relu, out_cm in ((True, False), (False, True)):
                y = run_cm(d, sbnn.SBNN_RELU if relu else 0, cfg, out_cm)
                ref, s = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=relu)
                assert_within(y, ref, s, what=f"cm G={g} cfg={cfg} sp={sp} relu={relu} out_cm={out_cm}")


@pytest.mark.parametrize("g", [1, 2, 4, 8, 16])
@pytest.mark.parametrize("cin,sp", [(40, 50), (160, 50), (320, 40), (1024, 50)])
def test_few_pixel_kernel(g, cin, sp):
    """Launches with few pixels take the kernel that gives a CTA 32 pixels of one group and splits the group's list
    over 1, 2, 4 or 8 warps (by list length): ragged pixel count, variable list lengths (layer-global masks, empty
    quarters), both output layouts."""
    d = WL.single_conv_inputs(1, 3, 37, cin, 48, 1, g, sp, seed=21, mask_mode="layer_global")
    for relu, out_cm in ((True, False), (False, True)):
        y = run_cm(d, sbnn.SBNN_RELU if relu else 0, (0, 0, 0, 0), out_cm)
        ref, s = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=relu)
        assert_within(y, ref, s, what=f"few-pixel G={g} cin={cin} relu={relu} out_cm={out_cm}")


def test_channel_major_kernel_edge_cases():
    for sp in (0, 100):
        d = WL.single_conv_inputs(1, 3, 5, 40, 24, 1, 4, sp, seed=10)
        y = run_cm(d, sbnn.SBNN_RELU, (0, 0, 0, 0), False)
        ref, s = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=True)
        assert_within(y, ref, s, what=f"cm sp={sp}")


def test_layer_loaded_from_a_file_computes_bit_for_bit_what_the_packed_one_does(tmp_path):
    """sbnn_packed_save / sbnn_packed_load: the loaded layer has its own device copies and private layouts and must give
    the very bits the original gives (1x1 through the pipelined kernel, 3x3 with kernel patterns through the tap lists)."""
    from sbnn_inputs import tap_pattern_mask
    d = WL.single_conv_inputs(1, 40, 60, 160, 96, 1, 4, 50, seed=23)
    p = sbnn.pack_weights(d["w"], d["mask"], d["bias"], 4)
    p.save(str(tmp_path / "pw.sbnn"))
    q = sbnn.load_packed(str(tmp_path / "pw.sbnn"))
    xd = dev(d["x"])
    ya, yb = Guarded((1, 40, 60, 96)), Guarded((1, 40, 60, 96))
    sbnn.conv1x1_gs(p, xd, ya.t, 1, 40, 60, sbnn.SBNN_RELU)
    sbnn.conv1x1_gs(q, xd, yb.t, 1, 40, 60, sbnn.SBNN_RELU)
    sbnn.get_async_status()
    assert np.array_equal(ya.numpy("packed"), yb.numpy("loaded"))
    ref, s = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=True)
    assert_within(yb.numpy("loaded"), ref, s, what="loaded 1x1 layer")
    p.free(); q.free()
    d3 = WL.single_conv_inputs(2, 12, 28, 24, 32, 3, 4, 50, seed=24, w_sigma=0.1)
    m = tap_pattern_mask(24, 19, d3["unit_mask"], 4, 4)
    p3 = sbnn.pack_weights(d3["w"], m, d3["bias"], 4, tap_patterns=True)
    p3.save(str(tmp_path / "c3.sbnn"))
    q3 = sbnn.load_packed(str(tmp_path / "c3.sbnn"))
    x3 = dev(d3["x"])
    za, zb = Guarded((2, 12, 28, 32)), Guarded((2, 12, 28, 32))
    sbnn.conv3x3_gs(p3, x3, za.t, 2, 12, 28, sbnn.SBNN_RELU)
    sbnn.conv3x3_gs(q3, x3, zb.t, 2, 12, 28, sbnn.SBNN_RELU)
    sbnn.get_async_status()
    assert np.array_equal(za.numpy("packed 3x3"), zb.numpy("loaded 3x3"))
    ref3, s3 = R.conv2d(d3["x"], d3["w"], m, d3["bias"], relu=True)
    assert_within(zb.numpy("loaded 3x3"), ref3, s3, what="loaded 3x3 pattern layer")
    p3.free(); q3.free()


def test_wide_layer_through_the_nhwc_entry_point():
    """Config 5's layer shape at a reduced batch: the NHWC entry point routes it through the channel-major kernel."""
    for g, sp in ((4, 50), (8, 70)):
        d = WL.config5(g, sp, n=24)            # M = 4704 >= 4096
        y = run_1x1(d)
        ref, s = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=True)
        worst = assert_within(y, ref, s, what=f"config 5 G={g} s={sp} (n=24)")
        assert worst < 0.5


@pytest.mark.parametrize("g", [1, 2, 4, 8, 16])
def test_bf16_tensor_core_mode(g):
    """SBNN_BF16_TC against the oracle run on bf16-rounded operands (tight: products are exact in fp32,
    accumulation is fp32) and against the fp32 oracle with the stated bf16 tolerance 1e-2 * S
    (each operand is within 2^-9 relative after rounding, so 2 * 2^-9 * S plus accumulation)."""
    d = WL.single_conv_inputs(1, 3, 131, 212, 16 * 11, 1, g, 50, seed=12, mask_mode="layer_global")
    for relu in (True, False):
        flags = sbnn.SBNN_BF16_TC | (sbnn.SBNN_RELU if relu else 0)
        y = run_1x1(d, flags)
        ref16, s16 = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=relu, bf16=True)
        assert_within(y, ref16, s16, tol=1e-5, what=f"bf16 G={g} relu={relu} vs bf16 oracle")
        ref, s = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=relu)
        assert_within(y, ref, s, tol=1e-2, what=f"bf16 G={g} relu={relu} vs fp32 oracle")


@pytest.mark.parametrize("g,cin,cout,m", [(8, 136, 264, 300), (4, 64, 128, 1000), (4, 1024, 1024, 128 * 3 + 5),
                                          (16, 72, 48, 77), (4, 8, 4, 5), (8, 64, 512, 128 * 330 + 3)])
def test_bf16_dense_tensor_core_path(g, cin, cout, m):
    """SBNN_BF16_TC on shapes the tcgen05 kernel takes (Cin % 8 == 0): dense contraction over the masked weights.
    Ragged pixel, channel and output-channel tiles, all three output-tile widths (64, 128, 256), and a case with
    more tiles than two per SM, so that both accumulators and every pipeline stage are reused.  Against the
    oracle on bf16-rounded operands at 1e-5 * S, against the fp32 oracle at the stated 1e-2 * S; the gathered
    kernel (SBNN_BF16_GATHER) must agree with the same oracle."""
    d = WL.single_conv_inputs(1, 1, m, cin, cout, 1, g, 50, seed=21, mask_mode="layer_global")
    ref16, s16 = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=True, bf16=True)
    ref, s = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=True)
    y = run_1x1(d, sbnn.SBNN_BF16_TC | sbnn.SBNN_RELU)
    assert_within(y, ref16, s16, tol=1e-5, what=f"bf16 dense G={g} {cin}->{cout} M={m} vs bf16 oracle")
    assert_within(y, ref, s, tol=1e-2, what=f"bf16 dense G={g} {cin}->{cout} M={m} vs fp32 oracle")
    if m < 2000:
        yg = run_1x1(d, sbnn.SBNN_BF16_TC | sbnn.SBNN_BF16_GATHER | sbnn.SBNN_RELU)
        assert_within(yg, ref16, s16, tol=1e-5, what=f"bf16 gathered G={g} {cin}->{cout} M={m} vs bf16 oracle")


def test_bf16_dense_path_without_relu_and_fully_pruned_layer():
    for sp, relu in ((50, False), (100, True)):
        d = WL.single_conv_inputs(1, 3, 50, 96, 40, 1, 4, sp, seed=22)
        y = run_1x1(d, sbnn.SBNN_BF16_TC | (sbnn.SBNN_RELU if relu else 0))
        ref16, s16 = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=relu, bf16=True)
        assert_within(y, ref16, s16, tol=1e-5, what=f"bf16 dense sp={sp} relu={relu}")


@pytest.mark.parametrize("g,cout", [(4, 12), (2, 6), (1, 5), (1, 16), (2, 22)])
def test_bf16_mode_merged_groups_ragged_channel_count(g, cout):
    """Groups of fewer than 8 channels are merged into 8-column groups for the tensor cores; the last merged group
    may reach past Cout, and an odd Cout forces scalar stores."""
    d = WL.single_conv_inputs(1, 5, 37, 72, cout, 1, g, 50, seed=13, mask_mode="layer_global")
    y = run_1x1(d, sbnn.SBNN_BF16_TC | sbnn.SBNN_RELU)
    ref16, s16 = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=True, bf16=True)
    assert_within(y, ref16, s16, tol=1e-5, what=f"bf16 merged G={g} Cout={cout}")


def test_bf16_mode_on_config5_shape_reduced_batch():
    d = WL.config5(8, 50, n=6)
    y = run_1x1(d, sbnn.SBNN_BF16_TC | sbnn.SBNN_RELU)
    ref16, s16 = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=True, bf16=True)
    assert_within(y, ref16, s16, tol=1e-5, what="config 5 G=8 bf16")


def test_mobilenet_layer_on_channel_major_buffers():
    """run_layer_cm (what forward launches) against the oracle for one depthwise and one pointwise layer."""
    x, layers = mobilenet_v1_inputs(1, 50, 4, seed=1)
    outs = R.mobilenet_v1_forward(x, layers[:5])
    net = build_net(layers, 1)
    for li in (1, 2, 3, 4):
        rec = outs[li]
        hin, cin, hout, cout = sbnn.mobilenet_v1_layer_shape(li)
        xin = dev(np.ascontiguousarray(rec["in"].reshape(hin * hin, cin).T))      # [C][M]
        yd = torch.full((cout, hout * hout), float("nan"), device="cuda")
        net.run_layer_cm(li, xin, yd, 1)
        sbnn.get_async_status()
        y = yd.cpu().numpy().T.reshape(rec["ref"].shape)
        assert_within(y, rec["ref"], rec["S"], what=f"cm layer {li}")
    net.free()


def test_expired_wait_is_reported_and_the_context_stays_usable():
    """A bounded device-side wait that runs out sets the status word; nothing faults, later calls work."""
    sbnn.get_async_status()                                   # clean slate
    sbnn.selftest_wait_timeout()
    with pytest.raises(sbnn.SbnnError) as e:
        sbnn.get_async_status()
    assert e.value.name == "SBNN_ERR_TIMEOUT"
    sbnn.get_async_status()                                   # reported once, then clear
    d = WL.single_conv_inputs(1, 4, 4, 16, 16, 1, 4, 50, seed=3)
    y = run_1x1(d)
    ref, s = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=True)
    assert_within(y, ref, s, what="after an expired wait")


def test_device_side_check_of_a_packed_layer_reports_through_the_status_word():
    """sbnn_debug_check_packed: clean on a freshly packed layer; an index of the device copy pushed out of range, or out
    of order, is reported as SBNN_ERR_SHAPE by the next get_async_status (once), without a trap, and the context and the
    layer stay usable after the index is put back."""
    d = WL.single_conv_inputs(1, 4, 8, 40, 24, 1, 4, 50, seed=61)
    p = sbnn.pack_weights(d["w"], d["mask"], d["bias"], 4)
    sbnn.debug_check_packed(p)
    sbnn.get_async_status()
    for bad in (40, -1):
        prev = sbnn.debug_poke_device_index(p, 3, bad)
        sbnn.debug_check_packed(p)
        with pytest.raises(sbnn.SbnnError) as e:
            sbnn.get_async_status()
        assert e.value.name == "SBNN_ERR_SHAPE"
        sbnn.get_async_status()                                   # reported once
        sbnn.debug_poke_device_index(p, 3, prev)
    v = p.view()
    prev = sbnn.debug_poke_device_index(p, 1, int(v["idx"][0]))   # equal to its predecessor: not ascending
    sbnn.debug_check_packed(p)
    with pytest.raises(sbnn.SbnnError):
        sbnn.get_async_status()
    sbnn.debug_poke_device_index(p, 1, prev)
    sbnn.debug_check_packed(p)
    sbnn.get_async_status()
    y = run_1x1(d)
    ref, s = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=True)
    assert_within(y, ref, s, what="after the debug pokes")
    p.free()


def test_weights_of_another_device_are_refused_and_the_context_stays_usable():
    """With the recorded device of a packed layer overwritten (test hook), the compute calls return SBNN_ERR_CUDA
    naming both devices and launch nothing; with the number restored the same call works."""
    d = WL.single_conv_inputs(1, 4, 4, 16, 16, 1, 4, 50, seed=3)
    p = sbnn.pack_weights(d["w"], d["mask"], d["bias"], 4)
    x, out = dev(d["x"]), Guarded((1, 4, 4, 16))
    was = sbnn.debug_set_packed_device(p, 5)
    assert was == torch.cuda.current_device()
    for call in (lambda: sbnn.conv1x1_gs(p, x, out.t, 1, 4, 4), lambda: sbnn.head_noalloc(p, x, out.t, 1, 16),
                 lambda: sbnn.prepare(p, 1, 4, 4)):
        with pytest.raises(sbnn.SbnnError) as e:
            call()
        assert e.value.name == "SBNN_ERR_CUDA" and "device 5" in e.value.detail
    sbnn.get_async_status()
    assert bool(torch.isnan(out.t).all())                     # nothing ran
    sbnn.debug_set_packed_device(p, was)
    sbnn.conv1x1_gs(p, x, out.t, 1, 4, 4)
    sbnn.get_async_status()
    ref, s = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=True)
    assert_within(out.numpy(), ref, s)
    p.free()


def test_prepare_then_calls_only_enqueue_and_capture_refuses_to_grow_the_scratch():
    """sbnn_prepare builds the private layouts and sizes the per-device scratch for a shape; a larger NHWC call made
    while its stream is being captured is refused (the scratch cannot grow there) and leaves the capture intact; after
    preparing for that shape the same call is captured, and replaying the graph gives the oracle's result."""
    d = WL.single_conv_inputs(1, 1, 2600, 256, 64, 1, 4, 50, seed=17)           # Cin >= 128, M >= 2048: channel-major route
    n, h, w, cin = d["x"].shape
    p = sbnn.pack_weights(d["w"], d["mask"], d["bias"], 4)
    big = WL.single_conv_inputs(1, 1, 180000, 256, 64, 1, 4, 50, seed=17)       # same layer, 184 MB of scratch
    bx = dev(big["x"])
    bout = Guarded((1, 1, 180000, 64))
    side = torch.cuda.Stream()
    refused = None
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        try:
            sbnn.conv1x1_gs(p, bx, bout.t, 1, 1, 180000, stream=torch.cuda.current_stream())
        except sbnn.SbnnError as e:
            refused = e
    if refused is not None:          # (not refused only if an earlier test already grew the scratch this far)
        assert refused.name == "SBNN_ERR_UNSUPPORTED" and "sbnn_prepare" in refused.detail
    sbnn.prepare(p, 1, 1, 180000)
    g2 = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g2, stream=side):
        sbnn.conv1x1_gs(p, bx, bout.t, 1, 1, 180000, stream=torch.cuda.current_stream())
    g2.replay()
    torch.cuda.synchronize()
    sbnn.get_async_status()
    y = bout.numpy("captured call")
    pix = np.arange(0, 180000, 61)
    xs = np.ascontiguousarray(big["x"].reshape(-1, cin)[pix]).reshape(1, 1, len(pix), cin)
    ref, s = R.conv2d(xs, big["w"], big["mask"], big["bias"], relu=True)
    assert_within(y.reshape(-1, 64)[pix].reshape(ref.shape), ref, s, what="graph replay after sbnn_prepare")
    p.free()


def test_3x3_prepared_call_is_captured_and_replayed():
    """After sbnn_prepare for the shape (weight stream, work plan, scratch), a 3x3 call on a new width is recorded into a
    CUDA graph (conversion pass, clearing of the arrival counters, the persistent kernel) without allocating, and two
    replays give the oracle's result both times (the counters are cleared inside the graph)."""
    d = WL.single_conv_inputs(7, 12, 44, 24, 40, 3, 4, 50, seed=23, w_sigma=0.05)
    n, h, w, _ = d["x"].shape
    p = sbnn.pack_weights(d["w"], d["mask"], d["bias"], 4)
    sbnn.prepare(p, n, h, w)
    xd = dev(d["x"])
    out = Guarded((n, h, w, 40))
    side = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        sbnn.conv3x3_gs(p, xd, out.t, n, h, w, sbnn.SBNN_RELU, stream=torch.cuda.current_stream())
    ref, s = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=True)
    for _ in range(2):
        out.t.fill_(float("nan"))
        g.replay()
        torch.cuda.synchronize()
        sbnn.get_async_status()
        assert_within(out.numpy("captured 3x3"), ref, s, what="3x3 graph replay after sbnn_prepare")
    p.free()


def test_few_pixel_kernel_on_a_layer_without_kept_units():
    """Every unit pruned: the few-pixel kernel's look-ahead fetch has no unit to read; the output is act(bias)."""
    d = WL.single_conv_inputs(1, 3, 5, 40, 24, 1, 4, 100, seed=10)
    assert not d["mask"].any()
    for relu in (True, False):
        y = run_cm(d, sbnn.SBNN_RELU if relu else 0, (0, 0, 0, 0), True)
        want = np.maximum(d["bias"], 0) if relu else d["bias"]
        assert np.array_equal(y, np.broadcast_to(want, y.shape))
