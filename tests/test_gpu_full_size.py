"""Parity at the benchmark's full sizes, in the launch configurations the benchmark times: outputs sampled at random
and recomputed one by one by the oracle, plus properties that hold at any size."""
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


def sample_positions(shape, cout, k, seed):
    n, h, w, _ = shape
    rng = np.random.default_rng(seed)
    pos = [(int(rng.integers(n)), int(rng.integers(h)), int(rng.integers(w)), int(rng.integers(cout))) for _ in range(k)]
    return pos + [(0, 0, 0, 0), (n - 1, h - 1, w - 1, cout - 1), (n - 1, 0, w - 1, 0)]   # corners: padding, last tile


def check_samples(y, d, pos, bf16=False, tol=TOL):
    ref, s = R.sample_outputs(d["x"], d["w"], d["mask"], d["bias"], pos, relu=True, bf16=bf16)
    got = np.array([y[p] for p in pos], dtype=np.float64)
    bad = np.abs(got - ref) > tol * s
    assert not bad.any(), f"{bad.sum()} of {len(pos)} sampled outputs outside tolerance"


@pytest.mark.parametrize("g,sp", [(4, 50), (8, 90), (4, 0)])
def test_config5_full_size_sampled(g, sp):
    d = WL.config5(g, sp)                       # batch 256: M = 50176, 1024 -> 1024
    n, h, w, cin = d["x"].shape
    p = sbnn.pack_weights(d["w"], d["mask"], d["bias"], g)
    xd = dev(d["x"])
    yd = torch.full((n, h, w, 1024), float("nan"), device="cuda")
    sbnn.conv1x1_gs(p, xd, yd, n, h, w, sbnn.SBNN_RELU)
    sbnn.get_async_status()
    assert bool(torch.isfinite(yd).all())
    y = yd.cpu().numpy()
    check_samples(y, d, sample_positions(d["x"].shape, 1024, 300, seed=sp + g))
    if sp == 50 and g == 4:                     # the bf16 tensor-core mode on the same inputs
        sbnn.conv1x1_gs(p, xd, yd, n, h, w, sbnn.SBNN_RELU | sbnn.SBNN_BF16_TC)
        sbnn.get_async_status()
        check_samples(yd.cpu().numpy(), d, sample_positions(d["x"].shape, 1024, 100, seed=1), bf16=True)
    p.free()


def test_config4_full_size_sampled():
    d = WL.config4()                            # batch 32, 28x28, 256 -> 256, 3x3
    n, h, w, cin = d["x"].shape
    p = sbnn.pack_weights(d["w"], d["mask"], d["bias"], 4)
    yd = torch.full((n, h, w, 256), float("nan"), device="cuda")
    sbnn.conv3x3_gs(p, dev(d["x"]), yd, n, h, w, sbnn.SBNN_RELU)
    sbnn.get_async_status()
    assert bool(torch.isfinite(yd).all())
    check_samples(yd.cpu().numpy(), d, sample_positions(d["x"].shape, 256, 300, seed=4))
    p.free()


def test_mobilenet_batch64_matches_oracle_on_two_images_and_is_batch_invariant():
    from test_gpu_parity import build_net
    x, layers = mobilenet_v1_inputs(64, 50, 4, seed=0)
    net = build_net(layers, 64)
    logits = torch.full((64, 1000), float("nan"), device="cuda")
    net.forward(dev(x), logits, 64)
    sbnn.get_async_status()
    y = logits.cpu().numpy().astype(np.float64)
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
