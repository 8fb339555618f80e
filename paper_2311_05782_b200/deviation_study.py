"""Numeric-deviation study on the device (paper Section V-B, Table II and the ECDFs of the differences; Section VI-B,
the differences with each correction technique applied).

    python -m paper_2311_05782_b200.deviation_study [--trials N] [--json out.json]

For two synthetic activation/weight workloads (GELU activations x small-variance weights, K = 4096; ReLU activations x
He-scaled weights, K = 576), each in FP16, BF16 and TF32, it runs the paper's own trial -- a uniformly chosen output
element and term, 1, 2 or 4 adjacent flipped bits in the FP32 product, written back into the running sum that one HMMA
leaves (Eq. 1-2) -- under no check and under each of the three techniques with correction, and reduces the trial
records on the device (mpgemmfi_campaign_summary). Reported per cell: the share of trials whose sum did not change
("zero difference", Table II's metric) and where the non-zero deviations lie on a log2 scale (median, 80th percentile,
largest bin, count of infinite ones).

Everything runs through the library (mpgemmfi_campaign + mpgemmfi_campaign_summary); the CPU oracle is not involved.
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

WORKLOADS = {
    # name: (config whose operand distributions are used, M, N, K)
    "gelu_k4096": ("c3b", 2048, 1024, 4096),
    "relu_k576": ("c5", 16384, 64, 576),
}
FORMATS = {"fp16": 0, "bf16": 1, "tf32": 2}
TECHNIQUES = {"none": 0, "boundcheck": 1 | 16, "rangecheck_max": 2 | 16, "rangecheck_flip": 3 | 16}


def log2_quantile(hist: np.ndarray, q: float):
    """log2 of the lower edge of the exponent bin that holds quantile q of the non-zero deviations (None if none)."""
    total = int(hist.sum())
    if total == 0:
        return None
    c = np.cumsum(hist)
    e = int(np.searchsorted(c, q * total, side="left"))
    return e - 127 if e < 255 else float("inf")


def run_cell(mpg, synth, torch, workload: str, fmt: int, nbits: int, mode: int, trials: int, seed: int = 1,
             in_format: bool = False):
    """One cell of the study; returns the device summary (numpy record) and the derived figures.
    in_format: the product is held in the operand format when its bits are flipped (MPGEMMFI_TERM_IN_FORMAT; the
    masks then lie in that format's 16 or 19 bits) instead of in FP32."""
    cfg, M, N, K = WORKLOADS[workload]
    A, Bt = synth.make_operands(cfg, M, N, K, dtype=fmt)
    sites = synth.make_sites("term_op" if in_format else "term", fmt, M, N, K, trials,
                             synth.config_seed(cfg) + 100 * nbits + seed, nbits=nbits)
    if in_format:
        mode |= mpg.TERM_IN_FORMAT
    view = np.int32 if fmt == synth.DTYPE_TF32 else np.int16
    a = torch.from_numpy(A.view(view)).cuda()
    b = torch.from_numpy(Bt.view(view)).cuda()
    _, rec = mpg.campaign(fmt, a, b, sites, mode | mpg.TERM_HMMA_STEP)
    summ = mpg.campaign_summary(rec)
    hist = summ["dev_exponent_hist"].astype(np.int64)
    valid = int(summ["n_trials"]) - int(summ["n_invalid"])
    cell = {
        "trials": valid,
        "zero_diff_pct": 100.0 * int(summ["n_zero_diff"]) / max(valid, 1),
        "nonzero": int(hist.sum()),
        "log2_median": log2_quantile(hist, 0.5),
        "log2_p80": log2_quantile(hist, 0.8),
        "log2_max": (int(np.nonzero(hist)[0].max()) - 127) if hist.any() else None,
        "infinite": int(summ["n_nonfinite"]),
    }
    return summ, cell


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--trials", type=int, default=50000)
    ap.add_argument("--json", default=None)
    ap.add_argument("--product", default="fp32", choices=["fp32", "operand"],
                    help="format the product is held in when its bits are flipped (default: FP32, the library's default)")
    args = ap.parse_args()
    import torch

    import paper_2311_05782_b200 as mpg
    import synth
    if not torch.cuda.is_available():
        raise SystemExit("the study runs on a CUDA device (there is no CPU path)")
    mpg.load_library()
    results = {}
    for wname in WORKLOADS:
        for fname, fmt in FORMATS.items():
            for nbits in (1, 2, 4):
                for tname, mode in TECHNIQUES.items():
                    _, cell = run_cell(mpg, synth, torch, wname, fmt, nbits, mode, args.trials, in_format=args.product == "operand")
                    results[f"{wname}/{fname}/{nbits}bit/{tname}"] = cell
    print(f"{'cell':46s} {'zero-diff %':>11s} {'median':>7s} {'p80':>5s} {'max':>5s} {'inf':>6s}")
    for k, c in results.items():
        print(f"{k:46s} {c['zero_diff_pct']:11.2f} {str(c['log2_median']):>7s} {str(c['log2_p80']):>5s} "
              f"{str(c['log2_max']):>5s} {c['infinite']:6d}")
    if args.json:
        with open(args.json, "w") as f:
            json.dump({"trials_per_cell": args.trials, "product": args.product, "cells": results}, f, indent=1)


if __name__ == "__main__":
    main()
