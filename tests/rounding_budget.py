"""How far bf16 operands move the logits of a workload, and which rounding point moves them most.

    python -m tests.rounding_budget --workload llada8b [--layers 32] [--prompt 8] [--device cpu]

Runs the CPU oracle (and nothing else) on one root forward after a short prefill, once unrounded, once
with every contraction's operands rounded to bfloat16, and once per rounding source alone, all modes
through one pass over the weights.  Prints, per mode, the rms and the maximum of the logit difference
from the unrounded run, and the same for the confidences.  This is the per-source
error budget of bf16 operands; the GPU tests measure the same two totals (all sources, none) on their own inputs.
"""
from __future__ import annotations

import argparse
import time

import numpy as np

from oracle.ssd_oracle import ROUNDING_SOURCES, token_and_confidence
from paper_2510_04147_b200 import workloads as wl
from tests.helpers import LayerCachedWeights, lockstep_root_forward


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="llada8b")
    ap.add_argument("--layers", type=int, default=0, help="fewer layers of the same shape (0: all)")
    ap.add_argument("--prompt", type=int, default=8)
    ap.add_argument("--device", default="cpu", help="where the seeded generator draws the weights")
    args = ap.parse_args()
    w = wl.WORKLOADS[args.workload]
    if args.layers:
        w = w.replace(n_layers=args.layers)
    prompt = wl.make_prompts(w).numpy()[0, :args.prompt]
    ids = np.full(w.block_len, w.mask_id)
    modes = [None, "bf16"] + [(s,) for s in ROUNDING_SOURCES]
    t0 = time.time()
    res = lockstep_root_forward(w, LayerCachedWeights(w, args.device), prompt, ids, modes)
    base = res[None]["logits"]
    _, bconf = token_and_confidence(base, w.mask_id)
    print(f"{w.name}: {w.n_layers} layers, d {w.d_model}, vocab {w.vocab}, prompt {len(prompt)}, {w.block_len} rows; "
          f"logit std {base.std():.4f}; {time.time() - t0:.0f} s")
    print(f"{'rounded operands':<18} {'logit rms':>10} {'logit max':>10} {'rms/std':>9} {'conf rel max':>13} {'conf rel mean':>14}")
    for m in modes[1:]:
        d = res[m]["logits"] - base
        _, c = token_and_confidence(res[m]["logits"], w.mask_id)
        rel = np.abs(c / bconf - 1.0)
        name = "all (bf16 mode)" if m == "bf16" else m[0]
        print(f"{name:<18} {np.sqrt((d ** 2).mean()):>10.5f} {np.abs(d).max():>10.5f} "
              f"{np.sqrt((d ** 2).mean()) / base.std():>9.5f} {rel.max():>13.5f} {rel.mean():>14.5f}")
    # growth over the depth: distance of the bf16-mode residual stream from the unrounded one
    print("layer  |h_bf16 - h| / |h|  (residual stream entering the layer)")
    for l in range(0, w.n_layers + 1, max(1, w.n_layers // 8)):
        a, b = res["bf16"]["hidden"][l], res[None]["hidden"][l]
        print(f"{l:>5}  {np.sqrt(((a - b) ** 2).mean()) / np.sqrt((b ** 2).mean()):.5f}")


if __name__ == "__main__":
    main()
