"""Seeded input generators: determinism, value grids and the mask-count rules."""
import numpy as np
import pytest

import sbnn_inputs as SI
from sbnn_inputs import workloads as WL


def test_streams_are_counter_based_and_distinct():
    a = SI.u64_stream(0, 1, 100)
    b = SI.u64_stream(0, 1, 40, start=60)
    assert np.array_equal(a[60:], b)
    assert not np.array_equal(a, SI.u64_stream(0, 2, 100))
    assert not np.array_equal(a, SI.u64_stream(1, 1, 100))
    assert len(np.unique(a)) == 100


def test_uniform_grid_and_normal_moments():
    u = SI.uniform01(0, 0, 200000)
    assert u.dtype == np.float32 and u.min() >= 0 and u.max() < 1
    assert np.all(u * 2 ** 24 == np.floor(u * 2 ** 24))
    assert abs(u.mean() - 0.5) < 5e-3
    z = SI.normal(0, 1, 200001, 0.05)
    assert z.shape == (200001,) and abs(z.mean()) < 1e-3 and abs(z.std() - 0.05) < 1e-3


@pytest.mark.parametrize("ngroups,cin,pct", [(32, 64, 50), (16, 32, 30), (256, 1024, 70), (128, 1024, 90), (8, 32, 0)])
def test_balanced_mask_counts(ngroups, cin, pct):
    um = SI.group_mask_balanced(0, 3, ngroups, cin, pct)
    units = ngroups * cin
    removed = (pct * units + 50) // 100
    assert um.shape == (ngroups, cin) and um.sum() == units - removed
    per = cin - um.sum(axis=1)
    assert per.max() - per.min() <= 1 and np.all(np.diff(per) <= 0)
    if (pct * units) % 100 == 0:
        # whenever (1-s)*Cin*Cout is an integer the nonzero count equals it exactly
        g = 4
        assert SI.expand_mask(um, g, 1, 1).sum() * 100 == (100 - pct) * cin * ngroups * g


def test_paper_style_4x4_blocks_and_layer_global_mode():
    um = SI.group_mask_balanced(0, 3, 16, 64, 50, gi=4)
    blocks = um.reshape(16, 16, 4)
    assert np.all(blocks.all(axis=2) | (~blocks).all(axis=2)) and um.sum() == 16 * 32
    lg = SI.group_mask_layer_global(0, 3, 32, 64, 50)
    assert lg.sum() == 32 * 32 and len(set(lg.sum(axis=1))) > 1


def test_magnitude_mask_removes_smallest_units():
    w = SI.normal(0, 1, 16 * 32, 1.0).reshape(16, 1, 1, 32)
    um = SI.group_mask_magnitude(w, 4, 50)
    l1 = np.abs(w).reshape(4, 4, 32).sum(axis=1)
    assert um.sum() == 64 and l1[um].min() >= l1[~um].max()


def test_workload_shapes():
    c1 = WL.config1()
    assert c1["x"].shape == (1, 56, 56, 64) and c1["w"].shape == (128, 1, 1, 64)
    assert c1["unit_mask"].sum(axis=1).tolist() == [32] * 32
    shapes = SI.mobilenet_v1_shapes()
    assert len(shapes) == 29 and [s["name"] for s in shapes[-2:]] == ["pool", "fc"]
    assert [s["stride"] for s in shapes if s["kind"] == "dw"] == [1, 2, 1, 2, 1, 2, 1, 1, 1, 1, 1, 2, 1]
    x, layers = SI.mobilenet_v1_inputs(1, 30)
    kept = [int(L["mask"].sum()) // 4 for L in layers if L["kind"] == "pw"]
    assert kept == [358, 1434, 2867, 5734, 11469, 22938] + [45875] * 5 + [91750, 183501]
