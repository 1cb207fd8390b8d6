"""Glue used by the tests: turns a seeded workload into oracle inputs.

Holds no arithmetic of the method: it only converts tensors and builds configs.
"""
from __future__ import annotations

import numpy as np
import torch

from oracle.ssd_oracle import ModelConfig, Oracle, bf16_round
from paper_2510_04147_b200 import workloads as wl


def oracle_config(w: wl.Workload) -> ModelConfig:
    return ModelConfig(n_layers=w.n_layers, d_model=w.d_model, n_heads=w.n_heads, n_kv_heads=w.n_kv_heads,
                       head_dim=w.head_dim, d_ffn=w.d_ffn, vocab=w.vocab, mask_id=w.mask_id,
                       rope_theta=w.rope_theta, rms_eps=w.rms_eps)


def oracle_weights(w: wl.Workload, as_bf16: bool) -> dict:
    """All tensors of a (small) workload as fp64 numpy arrays.  ``as_bf16`` rounds the matrices
    to bfloat16 values first (what a bf16-only accelerator sees of fp32-drawn weights)."""
    out = {}
    for name, t in wl.iter_tensors(w, "cpu"):
        a = t.to(torch.float32).numpy().astype(np.float64)
        if as_bf16 and a.ndim == 2:
            a = bf16_round(a)
        out[name] = a
    return out


class LazyWeights:
    """The tensors of a LARGE workload one at a time, as the oracle asks for them (fp64, matrices rounded
    to bfloat16 values): nothing is kept, so a full-size model needs one tensor's worth of host memory.
    ``device`` is where the seeded generator runs (its output does not depend on it)."""

    def __init__(self, w: wl.Workload, device: str = "cpu"):
        self.w, self.device = w, device

    def __getitem__(self, name: str) -> np.ndarray:
        a = wl.make_tensor(self.w, name, self.device).to(torch.float32).cpu().numpy().astype(np.float64)
        return bf16_round(a) if a.ndim == 2 else a


class LayerCachedWeights:
    """Like LazyWeights, but keeps the most recently used tensors (one layer's worth), so that several
    oracles stepping through the same layer materialise each tensor once."""

    def __init__(self, w: wl.Workload, device: str = "cpu", keep: int = 12):
        self.w, self.device, self.keep = w, device, keep
        self.cache: dict = {}

    def __getitem__(self, name: str) -> np.ndarray:
        if name not in self.cache:
            while len(self.cache) >= self.keep:
                self.cache.pop(next(iter(self.cache)))
            a = wl.make_tensor(self.w, name, self.device).to(torch.float32).cpu().numpy().astype(np.float64)
            # weights drawn in bf16 already hold bf16 values: rounding them again changes nothing
            self.cache[name] = bf16_round(a) if (a.ndim == 2 and self.w.weight_dtype != "bf16") else a
        return self.cache[name]


def lockstep_root_forward(w: wl.Workload, weights, prompt: np.ndarray, ids: np.ndarray, modes):
    """Prefill of `prompt` and one forward of the rows `ids` [T] at positions len(prompt).., for several
    operand-rounding modes at once, stepping all of them through a layer before moving to the next (so a
    large model's tensors are drawn once).  Only calls the oracle's own ``layer``: per layer the prompt
    rows attend to themselves (the prefill), the block rows to the prompt's K/V plus themselves.
    Returns {mode: dict(hidden=[L+1] x [T,d], prefix_k=[L] x [P,Hkv,hd], prefix_v=..., logits=[T,V])}."""
    from oracle.ssd_oracle import rmsnorm
    cfg = oracle_config(w)
    P, T = len(prompt), len(ids)
    orcs = {m: Oracle(cfg, weights, m) for m in modes}
    emb = np.asarray(weights["embed"], dtype=np.float64)
    state = {m: dict(hp=emb[prompt].copy(), hb=emb[ids].copy(), hidden=[], prefix_k=[], prefix_v=[]) for m in modes}
    del emb
    empty = np.zeros((0, cfg.n_kv_heads, cfg.head_dim))
    pos_p, pos_b = np.arange(P), np.arange(P, P + T)
    for l in range(cfg.n_layers):
        for m, o in orcs.items():
            st = state[m]
            st["hidden"].append(st["hb"])
            (hp,), kp, vp = o.layer(l, [st["hp"]], [pos_p], empty, empty)
            (hb,), _, _ = o.layer(l, [st["hb"]], [pos_b], kp[0], vp[0])
            st["hp"], st["hb"] = hp, hb
            st["prefix_k"].append(kp[0])
            st["prefix_v"].append(vp[0])
    gf, wlm = np.asarray(weights["norm_final"], dtype=np.float64), np.asarray(weights["lm_head"], dtype=np.float64)
    for m, o in orcs.items():
        st = state[m]
        st["hidden"].append(st["hb"])
        st["logits"] = o.r["lm_in"](rmsnorm(st["hb"], gf, cfg.rms_eps)) @ wlm.T
        del st["hp"], st["hb"]
    return state


def make_oracle(w: wl.Workload, as_bf16: bool = False, operand_rounding=None) -> Oracle:
    return Oracle(oracle_config(w), oracle_weights(w, as_bf16), operand_rounding)


SMALL = wl.TINY.replace(name="small", d_model=64, n_heads=2, n_kv_heads=2, head_dim=32, d_ffn=96,
                        vocab=96, prompt_len=6, gen_len=12, block_len=6, seed=11)
SMALL_GQA = SMALL.replace(name="small_gqa", n_heads=4, n_kv_heads=2, head_dim=16, seed=12)
