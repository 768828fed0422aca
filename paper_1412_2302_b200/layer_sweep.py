#!/usr/bin/env python
"""Per-layer roofline sweep: every operation of the training step timed on its
own through the C ABI (alexnet_run_op), at AlexNet shapes.

    python -m paper_1412_2302_b200.layer_sweep [--batch 256] [--iters 20] [--burst 1] [--json out.json]

Tensor-core operations (convolution and FC forward, backward-data,
backward-weight) are reported in TFLOP/s of algorithmic work (2 x MACs of the
dense layer; padding of tiles or grids does not count) against the measured
bf16 peak; the other operations in GB/s of algorithmic bytes against the
measured HBM copy bandwidth.  Each timed run is preceded by a write of a buffer
larger than L2, so no operand is L2-resident from the run before; tensors hold
the values of a real training step.  An operation's time covers all the kernels
it launches (e.g. the split-K reduction after a weight-gradient GEMM).  With --burst N > 1 a timed run is N
back-to-back launches of the operation and the time is divided by N: the launches overlap their set-up and tails as
the kernels of a training step do (programmatic dependent launch), and operands stay in L2 from the launch before.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import numpy as np

MACS = {"CONV1": 105415200, "CONV2": 223948800, "CONV3": 149520384, "CONV4": 112140288, "CONV5": 74760192,
        "FC6": 37748736, "FC7": 16777216, "FC8": 4096000}
PARAMS = 60965224


def hbm_bytes(B):
    """Algorithmic bytes of the HBM-bound operations (bf16 activations, uint8 argmax)."""
    a1, a2, a5 = 96 * 55 * 55, 256 * 27 * 27, 256 * 13 * 13
    p1, p2, p5 = 96 * 27 * 27, 256 * 13 * 13, 256 * 6 * 6
    d = {
        "PREPROCESS": B * (154587 + 154587 * 4 + 2 * 155952),      # bytes gathered + mean read + bf16 written
        "LRN1_FWD": B * a1 * 4, "LRN2_FWD": B * a2 * 4,
        "LRN1_BWD": B * a1 * 6, "LRN2_BWD": B * a2 * 6,
        "POOL1_FWD": B * (a1 * 2 + p1 * 3), "POOL2_FWD": B * (a2 * 2 + p2 * 3), "POOL5_FWD": B * (a5 * 2 + p5 * 3),
        "POOL1_BWD": B * (a1 * 2 + p1 * 3), "POOL2_BWD": B * (a2 * 2 + p2 * 3), "POOL5_BWD": B * (a5 * 4 + p5 * 3),
        "SOFTMAX": B * 1000 * 6,
        "UPDATE": PARAMS * 22,                                      # r w,v,g; w w,v fp32 + bf16 copy
        "AVERAGE": PARAMS * (32 + 4),                               # r/w w,v of both replicas + both bf16 copies
        # the fused kernels the training step runs: a read, p + argmax written; a, dp, argmax read, da written
        "LRN1_POOL1_FWD": B * (a1 * 2 + p1 * 3), "LRN2_POOL2_FWD": B * (a2 * 2 + p2 * 3),
        "POOL1_LRN1_BWD": B * (a1 * 4 + p1 * 3), "POOL2_LRN2_BWD": B * (a2 * 4 + p2 * 3),
        "UPDATE_AVERAGE": PARAMS * 44,                              # r w,v,g of both replicas; w w,v and bf16 copy of both
        "SCALE_REFRESH": PARAMS * 6,                                # scale 1: r w, w bf16 copy
        # fc6 -> fc7 -> fc8 forward in one launch: the bf16 weights once, activations in and out, fc8's split partials
        "FC_CHAIN_FWD": 2 * (MACS["FC6"] + MACS["FC7"] + MACS["FC8"]) + B * (9216 + 2 * 4096 * 3) + B * 1000 * 4 * 16,
    }
    return d


def peaks():
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    p = os.path.join(root, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return d["bf16_tflops"], d["hbm_gbs"], "measured"
    return 1590.0, 6650.0, "fallback"


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--batch", type=int, default=256)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--burst", type=int, default=1)
    ap.add_argument("--json", default=None)
    ap.add_argument("--ops", default=None, help="comma-separated subset of operation names")
    args = ap.parse_args(argv)

    import torch
    from . import synth
    from .alexnet import FLAG_FC_CHAIN, OPS, AlexNet, AlexNetError

    B = args.batch
    seed = synth.BASE_SEED + 5
    net = AlexNet(batch=B, replicas=2, seed=seed, mean_image=synth.mean_image(seed), flags=FLAG_FC_CHAIN)
    w = synth.init_params(seed, variance_preserving=True)
    net.set_params(w, 0)
    net.set_params(w, 1)
    img = torch.from_numpy(synth.images(seed, 0, 0, B)).pin_memory()
    lab = torch.from_numpy(synth.labels(seed, 0, 0, B)).pin_memory()
    for r in (0, 1):                                   # real values in every tensor of both replicas
        net.load_batch_async(r, img, lab, 0)
        net.train_step(r)
    net.sync()
    cs = net.compute_stream
    flush = torch.empty(256 * 2**20, dtype=torch.uint8, device=net.device)
    tf_peak, hbm_peak, kind = peaks()
    hb = hbm_bytes(B)
    rows = []
    names = args.ops.split(",") if args.ops else OPS
    with torch.cuda.stream(cs):
        for name in names:
            try:
                for _ in range(3):
                    net.run_op(name)
            except AlexNetError:
                if name != "FC_CHAIN_FWD":
                    raise
                continue              # the one-launch FC forward exists at batch <= 128 only
            ts = []
            for _ in range(args.iters):
                flush.fill_(1)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(cs)
                net.run_op(name, iters=args.burst)
                e1.record(cs)
                ts.append((e0, e1))
            net.sync()
            ms = float(np.median([a.elapsed_time(b) for a, b in ts])) / args.burst
            layer = name.split("_")[0]
            if layer in MACS:
                tf = 2.0 * MACS[layer] * B / (ms * 1e-3) / 1e12
                rows.append({"op": name, "ms": ms, "tflops": tf, "frac": tf / tf_peak, "bound": "tensor"})
            else:
                gbs = hb[name] / (ms * 1e-3) / 1e9
                rows.append({"op": name, "ms": ms, "gbs": gbs, "frac": gbs / hbm_peak, "bound": "hbm"})
    # the evaluation pass (forward only, centre crop, top-1 / top-5 counts), batch resident on the device; the call
    # waits for its result, so this is wall-clock time per call
    import time
    dimg, dlab = img.to(net.device), lab.to(net.device)
    eval_ms = None
    if not args.ops:
        for _ in range(3):
            net.eval_batch(0, dimg, dlab)
        t0 = time.perf_counter()
        for _ in range(args.iters):
            net.eval_batch(0, dimg, dlab)
        eval_ms = (time.perf_counter() - t0) * 1e3 / args.iters
    net.close()
    print(f"# batch {B}, median of {args.iters} runs" + (f" of {args.burst} back-to-back launches" if args.burst > 1 else "")
          + f", L2 flushed before each; peaks ({kind}): "
          f"{tf_peak:.0f} TFLOP/s bf16 burst, {hbm_peak:.0f} GB/s HBM")
    print(f"{'operation':<20}{'ms':>9}{'TFLOP/s':>10}{'GB/s':>9}{'of peak':>9}")
    for r in rows:
        print(f"{r['op']:<20}{r['ms']:>9.4f}{r.get('tflops', float('nan')):>10.1f}{r.get('gbs', float('nan')):>9.0f}{r['frac']:>9.3f}")
    tot = sum(r["ms"] for r in rows)
    print(f"# sum of all operations: {tot:.3f} ms")
    if eval_ms is not None:
        print(f"# alexnet_eval_batch (forward + top-k, synchronous call): {eval_ms:.3f} ms per batch, {B / eval_ms * 1e3:.0f} images/s")
    if args.json:
        json.dump({"batch": B, "iters": args.iters, "peaks": {"bf16_tflops": tf_peak, "hbm_gbs": hbm_peak, "kind": kind},
                   "rows": rows}, open(args.json, "w"), indent=1)


if __name__ == "__main__":
    sys.exit(main())
