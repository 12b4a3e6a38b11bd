"""The allocation-free classifier head against the ordinary two-call route.

sbnn_head_noalloc serves callers that must not allocate device memory where they run the head (a
latency-bound serving loop, a plug-in inside someone else's memory pool): its pooled buffer is a
fixed array inside the library.  This file is collected last on purpose, so a failure here cannot
hide the result of any other test.
"""
import numpy as np
import pytest
import torch

import paper_2310_19509_b200 as sbnn
from oracle import reference as R
from sbnn_inputs import workloads as WL

pytestmark = pytest.mark.gpu
TOL = 1e-5


def _reference_route(fc, xd, n, hw, c, cout):
    pooled = torch.empty((n, c), device="cuda")
    out = torch.full((n, cout), float("nan"), device="cuda")
    sbnn.avgpool(xd, pooled, n, hw, c)
    sbnn.conv1x1_gs(fc, pooled, out, n, 1, 1, 0)
    sbnn.get_async_status()
    return out.cpu().numpy(), pooled.cpu().numpy()


def test_head_noalloc_matches_pool_then_classifier_twice_in_a_row():
    n, hw, c, cout = 5, 49, 1024, 1000
    d = WL.single_conv_inputs(1, 1, 1, c, cout, 1, 4, 0, seed=21, w_sigma=0.03, b_sigma=0.01)
    fc = sbnn.pack_weights(d["w"], d["mask"], d["bias"], 4)
    w = d["w"].reshape(cout, c).astype(np.float64)
    rng = np.random.default_rng(5)
    for call in range(2):                      # second call: other data, fewer images, same shared scratch
        nn = n - 2 * call
        x = rng.standard_normal((nn, hw, c)).astype(np.float32) + call
        xd = torch.from_numpy(x).cuda()
        want, pooled = _reference_route(fc, xd, nn, hw, c, cout)
        got = torch.full((nn, cout), float("nan"), device="cuda")
        sbnn.head_noalloc(fc, xd, got, nn, hw)
        sbnn.get_async_status()
        got = got.cpu().numpy()
        s = np.abs(pooled.astype(np.float64)) @ np.abs(w).T + np.abs(d["bias"].astype(np.float64))
        assert np.all(np.isfinite(got))
        assert np.all(np.abs(got.astype(np.float64) - want) <= TOL * s), f"call {call}"
        # and against the CPU oracle: mean over the positions, then the classifier on the fp32-rounded means.  A head
        # that is within TOL*S on each of its two steps deviates by at most |W| (TOL*S_pool) + TOL*S_fc.
        pref, ps = R.avgpool(x.reshape(nn, 7, 7, c))
        pooled_ref = pref.astype(np.float32)
        ref, sfc = R.conv2d(pooled_ref.reshape(nn, 1, 1, c), d["w"], d["mask"], d["bias"], relu=False)
        e_in = (TOL * ps + np.abs(pref) * 2.0 ** -24).astype(np.float32) * np.float32(1 + 2.0 ** -20)
        e, _ = R.conv2d(e_in.reshape(nn, 1, 1, c), np.abs(d["w"]), d["mask"], None, relu=False)
        bound = (e + TOL * sfc).reshape(nn, cout)
        assert np.all(np.abs(got.astype(np.float64) - ref.reshape(nn, cout)) <= bound), f"call {call} vs oracle"
    fc.free()


def test_head_noalloc_rejects_sizes_beyond_its_scratch():
    c, cout = 1024, 8
    d = WL.single_conv_inputs(1, 1, 1, c, cout, 1, 4, 0, seed=22)
    fc = sbnn.pack_weights(d["w"], d["mask"], d["bias"], 4)
    x = torch.zeros((65, 1, c), device="cuda")
    out = torch.zeros((65, cout), device="cuda")
    with pytest.raises(sbnn.SbnnError) as e:
        sbnn.head_noalloc(fc, x, out, 65, 1)            # 65 * 1024 floats > 65536
    assert e.value.name == "SBNN_ERR_SHAPE" and "scratch" in e.value.detail
    sbnn.head_noalloc(fc, x, out, 64, 1)                # the maximum itself is accepted
    sbnn.get_async_status()
    fc.free()
