#!/usr/bin/env python
"""Per-role timeline of the convolution kernel, one launch at a time.

    python -m paper_1412_2302_b200.build --timeline        (once: the instrumented variant of the library)
    python -m paper_1412_2302_b200.timeline [--batch 128] [--ops CONV1_FWD,...]

Runs each operation through the C ABI (alexnet_run_op) on the instrumented library and prints, averaged over the CTAs
of the launch: when the CTAs started (spread), set-up, the issuer's main loop (cycles per instruction, and how much of
it was spent waiting for activations, weights or a free accumulator), and the time from the last instruction to the
last store.  `single` is one launch after a device synchronisation; `in a burst` is the third of three back-to-back
launches, whose set-up ran under the launch before (programmatic dependent launch), as inside a training step.
The timers cost a few per cent; the figures are for reading the structure of a launch, not for benchmarks.
"""
from __future__ import annotations

import argparse
import ctypes
import sys

import numpy as np

from . import build as _build

CONV_OPS = ["CONV1_FWD", "CONV2_FWD", "CONV3_FWD", "CONV4_FWD", "CONV5_FWD", "CONV2_BWD_DATA", "CONV3_BWD_DATA",
            "CONV4_BWD_DATA", "CONV5_BWD_DATA", "FC6_FWD", "FC7_FWD", "FC8_FWD"]


# fc_chain_kernel's slots, in the order the events happen
CHAIN_SLOTS = [(1, "set up"), (3, "fc6: first operands at the issuer"), (4, "fc6: last instruction committed"),
               (9, "fc6: accumulator at the epilogue"), (10, "fc6: the cluster's four partial tiles in shared memory"),
               (11, "fc6: reduced, stored and counted on the gate"), (15, "gate open: fc7's activations may be loaded"),
               (5, "fc7: first operands"), (6, "fc7: last instruction committed"), (12, "fc7: accumulator at the epilogue"),
               (13, "fc7: the cluster's partial tiles"), (14, "fc7: reduced, stored and counted on the gate"),
               (7, "fc8: first operands"), (8, "fc8: last instruction committed"), (2, "end")]


def read(lib, clear):
    buf = np.zeros((160, 16), np.int64)
    rc = lib.alexnet_timeline_read(ctypes.c_void_p(buf.ctypes.data), 1 if clear else 0)
    if rc != 0:
        raise RuntimeError("the loaded library has no timeline instrumentation (python -m paper_1412_2302_b200.build --timeline)")
    return buf


def summarise(name, buf, mhz):
    d = buf[buf[:, 0] > 0]
    iss = d[d[:, 7] > 0]
    us = lambda ns: ns / 1e3
    cyc_us = lambda c: c / mhz
    span = us(d[:, 2].max() - d[:, 0].min())
    out = {
        "op": name, "ctas": len(d), "span_us": span,
        "start_spread_us": us(d[:, 0].max() - d[:, 0].min()),
        "setup_us": us((d[:, 12] - d[:, 0]).mean()), "wait_for_predecessor_us": us((d[:, 1] - d[:, 12]).mean()),
        "body_us": us((d[:, 2] - d[:, 1]).mean()),
    }
    if len(iss):
        mma = iss[:, 7].mean()
        out.update({
            "issuer_ctas": len(iss), "before_loop_us": us((iss[:, 13] - iss[:, 1]).mean()), "loop_us": cyc_us(iss[:, 6].mean()),
            "instructions": mma, "cycles_per_instruction": iss[:, 6].mean() / mma,
            "cycles_per_instruction_outside_waits": (iss[:, 6] - iss[:, 3] - iss[:, 4] - iss[:, 5]).mean() / mma,
            "wait_share": {"activations": iss[:, 3].mean() / iss[:, 6].mean(), "weights": iss[:, 4].mean() / iss[:, 6].mean(),
                           "accumulator": iss[:, 5].mean() / iss[:, 6].mean()},
            "last_instruction_to_last_store_us": us((iss[:, 15] - iss[:, 14]).mean()),
            "last_instruction_to_exit_us": us((iss[:, 2] - iss[:, 14]).mean()),
        })
    return out


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--batch", type=int, default=128)
    ap.add_argument("--ops", default=None)
    ap.add_argument("--sm-mhz", type=float, default=1965.0, help="SM clock used to convert cycles to microseconds")
    args = ap.parse_args(argv)
    _build.LIB = _build.LIB_TIMELINE          # the binding loads this variant
    import torch
    from . import synth
    from .alexnet import FLAG_FC_CHAIN, AlexNet
    B = args.batch
    seed = synth.BASE_SEED + 5
    net = AlexNet(batch=B, replicas=1, seed=seed, mean_image=synth.mean_image(seed), flags=FLAG_FC_CHAIN if B <= 128 else 0)
    net.set_params(synth.init_params(seed, variance_preserving=True))
    img = torch.from_numpy(synth.images(seed, 0, 0, B)).pin_memory()
    lab = torch.from_numpy(synth.labels(seed, 0, 0, B)).pin_memory()
    net.load_batch_async(0, img, lab, 0)
    net.train_step(0)
    net.sync()
    print(f"# batch {B}; us from the global timer, cycles at {args.sm_mhz:.0f} MHz")
    print(f"{'operation':<26}{'span':>7}{'spread':>8}{'set-up':>8}{'loop':>8}{'cyc/mma':>9}{'busy':>7}{'wait A/W/acc %':>17}{'tail':>7}{'to exit':>9}")
    for op in (args.ops.split(",") if args.ops else CONV_OPS):
        for mode, n in (("single", 1), ("in a burst", 3)):
            net.run_op(op, iters=2)
            net.sync()
            read(net.lib, True)
            net.run_op(op, iters=n)
            net.sync()
            r = summarise(op, read(net.lib, True), args.sm_mhz)
            w = r.get("wait_share", {"activations": 0, "weights": 0, "accumulator": 0})
            print(f"{op + ' [' + mode + ']':<26}{r['span_us']:>7.1f}{r['start_spread_us']:>8.1f}{r['setup_us']:>8.2f}"
                  f"{r.get('loop_us', 0):>8.1f}{r.get('cycles_per_instruction', 0):>9.0f}{r.get('cycles_per_instruction_outside_waits', 0):>7.0f}"
                  f"{100 * w['activations']:>7.0f}/{100 * w['weights']:.0f}/{100 * w['accumulator']:.0f}"
                  f"{r.get('last_instruction_to_last_store_us', 0):>10.1f}{r.get('last_instruction_to_exit_us', 0):>9.1f}")
    # the one-launch FC forward (ALEXNET_FLAG_FC_CHAIN): where the time between its three weight streams goes
    if not args.ops and B <= 128:
        print("# FC_CHAIN_FWD: us since the first CTA started, mean / min / max over the 128 CTAs")
        for mode, n in (("single", 1), ("in a burst", 3)):
            net.run_op("FC_CHAIN_FWD", iters=2)
            net.sync()
            read(net.lib, True)
            net.run_op("FC_CHAIN_FWD", iters=n)
            net.sync()
            d = read(net.lib, True)
            d = d[d[:, 0] > 0]
            t0 = d[:, 0].min()
            print(f"  [{mode}] span {(d[:, 2].max() - t0) / 1e3:.1f} us")
            for k, what in CHAIN_SLOTS:
                v = (d[:, k] - t0) / 1e3
                print(f"    {what:<58}{v.mean():>8.2f}{v.min():>8.2f}{v.max():>8.2f}")
    net.close()


if __name__ == "__main__":
    sys.exit(main())
