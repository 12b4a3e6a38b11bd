"""Parity at the benchmark's full sizes, in the launch configurations the benchmark times.

The oracle's plain loops need a few seconds per billion multiply-adds, so at full size they run on a subset of the
pixels chosen to reach every tile of every launch: whole images at the start, the middle and the end of the batch plus
every 97th pixel of the batch (the kernels' pixel tiles are 128-256 pixels, so each tile is hit at least once, in all
its output channels), compared element by element; two cases are compared on ALL outputs.  NaN canaries surround
every output buffer.
"""
import numpy as np
import pytest
import torch

import paper_2310_19509_b200 as sbnn
from oracle import reference as R
from sbnn_inputs import workloads as WL
from sbnn_inputs import mobilenet_v1_inputs
from test_gpu_parity import Guarded, build_net, dev

pytestmark = pytest.mark.gpu
TOL = 1e-5


def check_pixels(y, d, pix, relu=True, bf16=False, tol=TOL, what=""):
    """1x1 layer: outputs of the pixels `pix` (indices into the flattened batch), all channels, against the oracle."""
    cin, cout = d["x"].shape[-1], d["w"].shape[0]
    xs = np.ascontiguousarray(d["x"].reshape(-1, cin)[pix]).reshape(1, 1, len(pix), cin)
    ref, s = R.conv2d(xs, d["w"], d["mask"], d["bias"], relu=relu, bf16=bf16)
    got = y.reshape(-1, cout)[pix].astype(np.float64).reshape(ref.shape)
    assert np.all(np.isfinite(got)), what
    bad = np.abs(got - ref) > tol * s
    assert not bad.any(), f"{what}: {bad.sum()} of {bad.size} compared outputs outside tolerance"
    return float(np.max(np.abs(got - ref) / np.maximum(tol * s, 1e-300)))


def config5_pixels(n, hw, everything):
    m = n * hw
    if everything:
        return np.arange(m)
    whole = np.concatenate([np.arange(i * hw, (i + 1) * hw) for i in (0, n // 2, n - 1)])
    return np.unique(np.concatenate([whole, np.arange(0, m, 97), [m - 1]]))


@pytest.mark.parametrize("g", [4, 8])
@pytest.mark.parametrize("sp", [0, 30, 50, 70, 90])
def test_config5_full_size(g, sp):
    d = WL.config5(g, sp)                       # batch 256: M = 50176, 1024 -> 1024
    n, h, w, cin = d["x"].shape
    p = sbnn.pack_weights(d["w"], d["mask"], d["bias"], g)
    xd = dev(d["x"])
    out = Guarded((n, h, w, 1024))
    sbnn.conv1x1_gs(p, xd, out.t, n, h, w, sbnn.SBNN_RELU)
    sbnn.get_async_status()
    y = out.numpy(f"config 5 G={g} s={sp}")
    assert np.all(np.isfinite(y))
    pix = config5_pixels(n, h * w, everything=(g, sp) in ((4, 50), (8, 90)))
    worst = check_pixels(y, d, pix, what=f"config 5 G={g} s={sp}")
    assert worst < 0.5
    p.free()


@pytest.mark.parametrize("g", [4, 8])
def test_config5_full_size_bf16_mode(g):
    """The bf16 tensor-core mode on config 5 at 50 %: against the oracle run on bf16-rounded operands (1e-5 * S) and
    against the fp32 oracle with the mode's stated tolerance (1e-2 * S)."""
    d = WL.config5(g, 50)
    n, h, w, cin = d["x"].shape
    p = sbnn.pack_weights(d["w"], d["mask"], d["bias"], g)
    out = Guarded((n, h, w, 1024))
    sbnn.conv1x1_gs(p, dev(d["x"]), out.t, n, h, w, sbnn.SBNN_RELU | sbnn.SBNN_BF16_TC)
    sbnn.get_async_status()
    y = out.numpy(f"config 5 bf16 G={g}")
    pix = config5_pixels(n, h * w, everything=False)
    check_pixels(y, d, pix, bf16=True, what=f"config 5 bf16 G={g} vs bf16 oracle")
    check_pixels(y, d, pix, tol=1e-2, what=f"config 5 bf16 G={g} vs fp32 oracle")
    p.free()


def test_config4_full_size_every_output():
    d = WL.config4()                            # batch 32, 28x28, 256 -> 256, 3x3
    n, h, w, cin = d["x"].shape
    p = sbnn.pack_weights(d["w"], d["mask"], d["bias"], 4)
    out = Guarded((n, h, w, 256))
    sbnn.conv3x3_gs(p, dev(d["x"]), out.t, n, h, w, sbnn.SBNN_RELU)
    sbnn.get_async_status()
    y = out.numpy("config 4").astype(np.float64)
    assert np.all(np.isfinite(y))
    ref, s = R.conv2d(d["x"], d["w"], d["mask"], d["bias"], relu=True)
    bad = np.abs(y - ref) > TOL * s
    assert not bad.any(), f"{bad.sum()} of {bad.size} outputs outside tolerance"
    assert float(np.max(np.abs(y - ref) / np.maximum(TOL * s, 1e-300))) < 0.5
    p.free()


@pytest.mark.parametrize("sparsity", [50, 70])
def test_mobilenet_batch64_matches_oracle_on_two_images_and_is_batch_invariant(sparsity):
    x, layers = mobilenet_v1_inputs(64, sparsity, 4, seed=0)
    net = build_net(layers, 64)
    lg = Guarded((64, 1000))
    logits = lg.t
    net.forward(dev(x), logits, 64)
    sbnn.get_async_status()
    y = lg.numpy("forward").astype(np.float64)
    assert np.all(np.isfinite(y))
    refs = {}
    for img in (0, 63):                         # the oracle's chain with its propagated error bound
        outs = R.mobilenet_v1_forward(x[img:img + 1], layers)
        ref, e = outs[-1]["ref"].reshape(-1), outs[-1]["E"].reshape(-1)
        refs[img] = (ref, e)
        assert np.all(np.abs(y[img] - ref) <= e), f"image {img}: worst ratio {np.max(np.abs(y[img] - ref) / e)}"
    # an image's logits do not depend on its position in the batch (bit for bit: same kernels, same order of sums)
    flipped = torch.full((64, 1000), float("nan"), device="cuda")
    net.forward(dev(np.ascontiguousarray(x[::-1])), flipped, 64)
    sbnn.get_async_status()
    assert torch.equal(flipped.flip(0), logits)
    # nor, within the oracle's bound, on the batch size (a batch of one runs the few-pixel kernels, which sum in
    # another order)
    one = torch.full((1, 1000), float("nan"), device="cuda")
    for img in (0, 63):
        net.forward(dev(x[img:img + 1]), one, 1)
        sbnn.get_async_status()
        ref, e = refs[img]
        assert np.all(np.abs(one[0].cpu().numpy().astype(np.float64) - ref) <= e)
    net.free()


def test_mobilenet_batch64_every_pointwise_layer_alone_at_full_size():
    """The 13 pointwise launches of the batch-64 step, each alone on the chain's channel-major buffers with random
    activations of its shape, every 97th pixel (all output channels) against the oracle."""
    x, layers = mobilenet_v1_inputs(1, 50, 4, seed=0)
    net = build_net(layers, 64)
    rng = np.random.default_rng(3)
    for li, L in enumerate(layers):
        if L["kind"] != "pw":
            continue
        hin, cin, hout, cout = sbnn.mobilenet_v1_layer_shape(li)
        m = 64 * hin * hin
        xt = torch.rand((cin, m), device="cuda")
        out = Guarded((cout, m))
        net.run_layer_cm(li, xt, out.t, 64)
        sbnn.get_async_status()
        pix = np.unique(np.concatenate([np.arange(0, m, 97), np.arange(m - 300, m)]))
        xs = np.ascontiguousarray(xt[:, torch.from_numpy(pix).cuda()].t().cpu().numpy()).reshape(1, 1, len(pix), cin)
        ref, s = R.conv2d(xs, L["w"], L["mask"], L["bias"], relu=True)
        got = out.t[:, torch.from_numpy(pix).cuda()].t().cpu().numpy().astype(np.float64).reshape(ref.shape)
        out.check(L["name"])
        bad = np.abs(got - ref) > TOL * s
        assert not bad.any(), f"{L['name']}: {bad.sum()} of {bad.size} outputs outside tolerance"
    net.free()


@pytest.mark.parametrize("batch,sparsity", [(64, 50), (64, 70), (1, 30)])
def test_mobilenet_chain_every_layer_within_its_own_tolerance(batch, sparsity):
    """The chain as forward launches it (programmatic dependent launches, the tile shapes of this batch size), layer by
    layer: the activations after layer l come from forward_prefix(l); for the first and the last image the oracle
    applies layer l to the GPU's own activations after layer l - 1 and the result must agree within that layer's
    tolerance 1e-5 * S.  Unlike the bound propagated through 29 layers, which grows by an order of magnitude per
    layer, this catches an error of a few ulps in any one launch, and a kernel that started before its predecessor's
    output was complete."""
    x, layers = mobilenet_v1_inputs(batch, sparsity, 4, seed=0)
    net = build_net(layers, batch)
    xd = dev(x)
    imgs = sorted({0, batch - 1})
    prev = {img: np.ascontiguousarray(x[img:img + 1]) for img in imgs}      # input of the next layer, as the GPU has it
    worst = 0.0
    for li, L in enumerate(layers):
        hin, cin, hout, cout = sbnn.mobilenet_v1_layer_shape(li)
        hw = hout * hout
        if L["kind"] == "fc":
            out = Guarded((batch, cout))
        else:
            ld = (batch * hw + 3) // 4 * 4
            out = Guarded((cout, ld))
        net.forward_prefix(xd, out.t, batch, li)
        sbnn.get_async_status()
        got_all = out.numpy(L["name"])
        for img in imgs:
            rec = R.mobilenet_v1_forward(prev[img], [L])[0]
            ref, s = rec["ref"], rec["S"]
            if L["kind"] == "fc":
                got = got_all[img].reshape(ref.shape)
            else:
                got = got_all[:, img * hw:(img + 1) * hw].T.reshape(ref.shape)
            assert np.all(np.isfinite(got)), f"{L['name']}, image {img}"
            err = np.abs(got.astype(np.float64) - ref)
            lim = TOL * s + np.abs(ref) * 2.0 ** -23                        # + the fp32 rounding of the stored result
            assert np.all(err <= lim), f"{L['name']}, image {img}: worst ratio {np.max(err / np.maximum(lim, 1e-300))}"
            worst = max(worst, float(np.max(err / np.maximum(lim, 1e-300))))
            prev[img] = np.ascontiguousarray(got, dtype=np.float32)
    assert worst < 1.0
    net.free()
