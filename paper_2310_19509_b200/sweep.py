"""Timing of the single-layer configurations beside dense library baselines (cuDNN / cuBLAS through torch).

One JSON line per case: the group-sparse kernel's time, effective TFLOP/s on kept weights, fraction of the
roofline max(nonzero flops / FP32 peak, bytes / HBM bandwidth), and dense fp32 / TF32 times of the same shape.
Run as `python bench.py --sweep` or `python -m paper_2310_19509_b200.sweep [--tile P,GPW,NW,KC] [--only NAME]`.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

FP32_PEAK = 148 * 128 * 2 * 1.965e9


def _hbm():
    try:
        return float(json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))["hbm_gbs"]) * 1e9
    except Exception:
        return 6650e9


def _time(torch, fn, reps, flush):
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(3):
        fn()
    ts = []
    for _ in range(reps):
        if flush is not None:
            flush.add_(1.0)
        ev0.record()
        fn()
        ev1.record()
        ev1.synchronize()
        ts.append(ev0.elapsed_time(ev1) * 1e-3)
    return float(np.median(ts)), float(np.min(ts))


def dense_baselines(torch, x, cout, k, reps, flush):
    """cuDNN conv2d on channels-last tensors with TF32 off (like for like) and on (context); cuBLAS matmul for 1x1."""
    n, h, w, cin = x.shape
    xt = x.permute(0, 3, 1, 2)                                     # NCHW view of NHWC memory = channels_last
    wt = torch.randn(cout, cin, k, k, device="cuda").contiguous(memory_format=torch.channels_last)
    b = torch.randn(cout, device="cuda")
    out = {}
    for name, tf32 in (("cudnn_fp32", False), ("cudnn_tf32", True)):
        torch.backends.cudnn.allow_tf32 = tf32
        torch.backends.cuda.matmul.allow_tf32 = tf32
        f = lambda: torch.relu_(torch.nn.functional.conv2d(xt, wt, b, padding=(k - 1) // 2))  # noqa: E731
        out[name + "_us"] = _time(torch, f, reps, flush)[0] * 1e6
        if k == 1:
            x2, w2 = x.reshape(-1, cin), wt.reshape(cout, cin).t().contiguous()
            g = lambda: torch.relu_(torch.addmm(b, x2, w2))       # noqa: E731
            out[name.replace("cudnn", "cublas") + "_us"] = _time(torch, g, reps, flush)[0] * 1e6
    torch.backends.cudnn.allow_tf32 = False
    torch.backends.cuda.matmul.allow_tf32 = False
    return out


def run_case(torch, sbnn, name, d, k, reps, flush, tile=None, dense=True, flags=None, cm_tile=None):
    x = d["x"]
    n, h, w, cin = x.shape
    cout, g = d["w"].shape[0], d["g"]
    p = sbnn.pack_weights(d["w"], d["mask"], d["bias"], g)
    xd = torch.from_numpy(x).cuda()
    yd = torch.empty((n, h, w, cout), device="cuda")
    fl = sbnn.SBNN_RELU if flags is None else flags
    if k == 3:
        f = lambda: sbnn.conv3x3_gs(p, xd, yd, n, h, w, fl)                     # noqa: E731
    elif cm_tile is not None:
        m_, ld = n * h * w, (n * h * w + 3) // 4 * 4
        xt = torch.empty((cin, ld), device="cuda")

        def f():
            sbnn.to_channel_major(xd, xt, m_, cin, ld)
            sbnn.conv1x1_gs_cm(p, xt, ld, yd, cout, m_, fl, cm_tile)
    elif tile:
        f = lambda: sbnn.conv1x1_gs_tuned(p, xd, yd, n, h, w, fl, *tile)        # noqa: E731
    else:
        f = lambda: sbnn.conv1x1_gs(p, xd, yd, n, h, w, fl)                     # noqa: E731
    med, mn = _time(torch, f, reps, flush)
    sbnn.get_async_status()
    m = n * h * w
    units = int(d["unit_mask"].sum())
    flops = 2.0 * m * g * k * k * units
    byts = 4.0 * (m * (cin + cout) + units * (1 + g * k * k) + cout + cout // g + 1)
    roof = max(flops / FP32_PEAK, byts / _hbm())
    rec = {"case": name, "G": g, "sparsity_pct": d["sparsity_pct"], "M": m, "Cin": cin, "Cout": cout, "k": k,
           "us": med * 1e6, "us_min": mn * 1e6, "tflops_nonzero": flops / med / 1e12, "gbs": byts / med / 1e9,
           "roofline_us": roof * 1e6, "frac": roof / med, "bound": "alu" if flops / FP32_PEAK > byts / _hbm() else "hbm",
           "tile": cm_tile or tile}
    if dense:
        rec.update(dense_baselines(torch, xd, cout, k, reps, flush))
    p.free()
    return rec


def main(argv=None):
    import torch

    import paper_2310_19509_b200 as sbnn
    from sbnn_inputs import workloads as WL

    ap = argparse.ArgumentParser()
    ap.add_argument("--sweep", action="store_true")
    ap.add_argument("--tile", default=None, help="P,GPW,NW,KC for the 1x1 kernel")
    ap.add_argument("--cm-tile", default=None, help="P,GPW,NW,KC: transpose + channel-major kernel with this tile")
    ap.add_argument("--bf16", action="store_true", help="time the bf16 tensor-core mode instead of the fp32 kernel")
    ap.add_argument("--only", default=None)
    ap.add_argument("--layer", default=None, help="N,H,W,Cin,Cout,G,sparsity_pct: time that 1x1 layer as the MobileNet chain "
                                                  "runs it (channel-major in and out, tile shape chosen by the library)")
    ap.add_argument("--reps", type=int, default=10)
    ap.add_argument("--no-dense", action="store_true")
    ap.add_argument("--batch5", type=int, default=256)
    args, _ = ap.parse_known_args(argv)
    tile = tuple(int(t) for t in args.tile.split(",")) if args.tile else None
    cm_tile = tuple(int(t) for t in args.cm_tile.split(",")) if args.cm_tile else None
    flush = torch.zeros(64 * 1024 * 1024, device="cuda")
    if args.layer:
        n, h, w, cin, cout, g, sp = (int(v) for v in args.layer.split(","))
        d = WL.single_conv_inputs(1, 1, 64, cin, cout, 1, g, sp, 0, 0.05, 0.05)     # the weights; activations are random
        p = sbnn.pack_weights(d["w"], d["mask"], d["bias"], g)
        m = n * h * w
        ld = (m + 3) // 4 * 4
        xt, yt = torch.rand((cin, ld), device="cuda"), torch.empty((cout, ld), device="cuda")
        f = lambda: sbnn.conv1x1_gs_cm(p, xt, ld, yt, ld, m, sbnn.SBNN_RELU | sbnn.SBNN_OUT_CM, cm_tile or (0, 0, 0, 0))  # noqa: E731
        med, mn = _time(torch, f, args.reps, flush)
        sbnn.get_async_status()
        units = int(d["unit_mask"].sum())
        flops, byts = 2.0 * m * g * units, 4.0 * (m * (cin + cout) + units * (1 + g) + cout + cout // g + 1)
        roof = max(flops / FP32_PEAK, byts / _hbm())
        print(json.dumps({"case": f"layer {args.layer}", "M": m, "us": med * 1e6, "us_min": mn * 1e6, "roofline_us": roof * 1e6,
                          "frac": roof / med, "tile": cm_tile}), flush=True)
        p.free()
        return
    cases = [("config1", lambda: WL.config1(), 1)]
    for g in (4, 8):
        for sp in (0, 30, 50, 70, 90):
            cases.append((f"config5_G{g}_s{sp}", (lambda g=g, sp=sp: WL.config5(g, sp, n=args.batch5)), 1))
    cases.append(("config4", lambda: WL.config4(), 3))
    for name, mk, k in cases:
        if args.only and args.only not in name:
            continue
        try:
            fl = (sbnn.SBNN_RELU | sbnn.SBNN_BF16_TC) if (args.bf16 and k == 1) else None
            rec = run_case(torch, sbnn, name, mk(), k, args.reps, flush, tile if k == 1 else None, not args.no_dense,
                           flags=fl, cm_tile=cm_tile if k == 1 else None)
            rec["mode"] = "bf16_tc" if fl else "fp32"
        except sbnn.SbnnError as e:
            rec = {"case": name, "error": str(e)}
        print(json.dumps(rec), flush=True)


if __name__ == "__main__":
    main()
