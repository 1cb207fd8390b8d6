"""Seeded synthetic inputs: model shapes, weights and prompts.

This module is the ONLY code shared by the CPU oracle's tests and the CUDA
path's tests/bench.  It holds none of the method's arithmetic: it only names
the workloads (shapes, lengths) and draws their random numbers.

Every tensor is a pure function of (seed, tensor index, element index) through
a counter-based generator, so the same values can be produced on any torch
device (CPU for the oracle, CUDA for the library), for any single tensor, in
any order:

    u64  = splitmix64(element_index + key(seed, tensor_index))
    z    = QUANTILE[u64 >> 48]           # 65536 standard-normal quantiles
    w    = float32(z) * float32(std)     # one IEEE multiply -> device independent
    prompt id = (u64 >> 33) mod (vocab - 1)          # never the mask id (= vocab-1)

The quantile table is computed once on the CPU and copied to the device, so
both sides read the very same table.  The workloads stand in for the paper's
evaluation prompts (Section 4.1): only prompt length, generation length,
block length and model shape matter for the verification forward.
"""
from __future__ import annotations

import dataclasses
import functools
from typing import Dict, Iterator, List, Tuple

import torch

_MASK64 = (1 << 64) - 1


def _s64(c: int) -> int:
    """Two's-complement view of an unsigned 64-bit constant."""
    c &= _MASK64
    return c - (1 << 64) if c >= (1 << 63) else c


_GOLDEN = _s64(0x9E3779B97F4A7C15)
_MUL1 = _s64(0xBF58476D1CE4E5B9)
_MUL2 = _s64(0x94D049BB133111EB)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift on int64 (torch's >> is arithmetic)."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _key(seed: int, tensor_index: int) -> int:
    return _s64(((seed & 0xFFFFFFFF) << 32 | (tensor_index & 0xFFFFFFFF)) * 0x9E3779B97F4A7C15 + 0x632BE59BD9B4E019)


def hash_u64(seed: int, tensor_index: int, idx: torch.Tensor) -> torch.Tensor:
    """splitmix64 finaliser of (idx + key); int64 tensor holding the u64 bit pattern."""
    z = idx + _key(seed, tensor_index)
    z = z * _GOLDEN
    z = (z ^ _lsr(z, 30)) * _MUL1
    z = (z ^ _lsr(z, 27)) * _MUL2
    z = z ^ _lsr(z, 31)
    return z


def hash_u64_py(seed: int, tensor_index: int, i: int) -> int:
    """Pure-Python integer version of hash_u64 (used to pin the tensor version)."""
    z = (i + _key(seed, tensor_index)) & _MASK64
    z = (z * 0x9E3779B97F4A7C15) & _MASK64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK64
    z = z ^ (z >> 31)
    return z


@functools.lru_cache(maxsize=None)
def _quantiles_cpu() -> torch.Tensor:
    p = (torch.arange(65536, dtype=torch.float64) + 0.5) / 65536.0
    return torch.special.ndtri(p).to(torch.float32)


_QUANT_DEV: Dict[str, torch.Tensor] = {}


def _quantiles(device: torch.device) -> torch.Tensor:
    k = str(device)
    if k not in _QUANT_DEV:
        _QUANT_DEV[k] = _quantiles_cpu().to(device)
    return _QUANT_DEV[k]


def normal_tensor(seed: int, tensor_index: int, shape: Tuple[int, ...], std: float,
                  device="cpu", dtype=torch.float32, chunk: int = 1 << 24) -> torch.Tensor:
    """std * N(0,1) (65536-quantile approximation), element i = f(seed, tensor_index, i)."""
    device = torch.device(device)
    n = 1
    for s in shape:
        n *= int(s)
    out = torch.empty(n, dtype=dtype, device=device)
    table = _quantiles(device)
    stdt = torch.tensor(std, dtype=torch.float32, device=device)
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        idx = torch.arange(lo, hi, dtype=torch.int64, device=device)
        u = hash_u64(seed, tensor_index, idx)
        z = table[_lsr(u, 48)]
        out[lo:hi] = (z * stdt).to(dtype)
    return out.view(*shape)


def uniform_ids(seed: int, tensor_index: int, shape: Tuple[int, ...], n_values: int,
                device="cpu") -> torch.Tensor:
    """int32 ids uniform on [0, n_values)."""
    device = torch.device(device)
    n = 1
    for s in shape:
        n *= int(s)
    idx = torch.arange(n, dtype=torch.int64, device=device)
    u = hash_u64(seed, tensor_index, idx)
    return (_lsr(u, 33) % n_values).to(torch.int32).view(*shape)


@dataclasses.dataclass(frozen=True)
class Workload:
    """One synthetic configuration: model shape + decode lengths."""
    name: str
    n_layers: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rope_theta: float
    rms_eps: float
    weight_dtype: str          # "fp32" or "bf16": the precision the weights are DRAWN in
    seed: int
    prompt_len: int
    gen_len: int
    block_len: int
    batch: int
    init_std: float = 0.02
    lm_head_scale: float = 1.0  # >1 gives the labelled "peaked" variant (larger confidence gaps)

    @property
    def mask_id(self) -> int:
        return self.vocab - 1

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


TINY = Workload("tiny", n_layers=2, d_model=256, n_heads=4, n_kv_heads=4, head_dim=64, d_ffn=688,
                vocab=2048, rope_theta=10000.0, rms_eps=1e-5, weight_dtype="fp32", seed=0,
                prompt_len=32, gen_len=64, block_len=16, batch=1)
LLADA_8B = Workload("llada8b", n_layers=32, d_model=4096, n_heads=32, n_kv_heads=32, head_dim=128,
                    d_ffn=12288, vocab=126464, rope_theta=500000.0, rms_eps=1e-5, weight_dtype="bf16",
                    seed=1, prompt_len=512, gen_len=256, block_len=32, batch=1)
LLADA_8B_BATCH = LLADA_8B.replace(name="llada8b_batch", batch=8)
DREAM_7B = Workload("dream7b", n_layers=28, d_model=3584, n_heads=28, n_kv_heads=4, head_dim=128,
                    d_ffn=18944, vocab=152064, rope_theta=1000000.0, rms_eps=1e-6, weight_dtype="bf16",
                    seed=2, prompt_len=1024, gen_len=512, block_len=32, batch=1)
LLADA_8B_LONG = LLADA_8B.replace(name="llada8b_long", seed=3, prompt_len=4096, gen_len=1024,
                                 block_len=64, batch=4)

WORKLOADS = {w.name: w for w in (TINY, LLADA_8B, LLADA_8B_BATCH, DREAM_7B, LLADA_8B_LONG)}


def tensor_specs(w: Workload) -> List[Tuple[str, Tuple[int, ...], float]]:
    """(name, shape, std) of every random tensor, in the fixed drawing order.

    The position in this list is the tensor index fed to the generator.  Norm
    gains are not random (all ones) and are not listed.
    """
    q = w.n_heads * w.head_dim
    kv = w.n_kv_heads * w.head_dim
    s = w.init_std
    specs: List[Tuple[str, Tuple[int, ...], float]] = [("embed", (w.vocab, w.d_model), s)]
    for l in range(w.n_layers):
        p = f"layers.{l}."
        specs += [(p + "wq", (q, w.d_model), s), (p + "wk", (kv, w.d_model), s), (p + "wv", (kv, w.d_model), s),
                  (p + "wo", (w.d_model, q), s), (p + "w_gate", (w.d_ffn, w.d_model), s),
                  (p + "w_up", (w.d_ffn, w.d_model), s), (p + "w_down", (w.d_model, w.d_ffn), s)]
    specs.append(("lm_head", (w.vocab, w.d_model), s * w.lm_head_scale))
    return specs


def norm_names(w: Workload) -> List[str]:
    names = []
    for l in range(w.n_layers):
        names += [f"layers.{l}.norm_attn", f"layers.{l}.norm_ffn"]
    names.append("norm_final")
    return names


def make_tensor(w: Workload, name: str, device="cpu") -> torch.Tensor:
    """One weight tensor by name, in the workload's weight dtype (norm gains: ones, fp32)."""
    if name.endswith("norm_attn") or name.endswith("norm_ffn") or name == "norm_final":
        return torch.ones(w.d_model, dtype=torch.float32, device=device)
    for i, (n, shape, std) in enumerate(tensor_specs(w)):
        if n == name:
            dt = torch.bfloat16 if w.weight_dtype == "bf16" else torch.float32
            return normal_tensor(w.seed, i, shape, std, device=device, dtype=dt)
    raise KeyError(name)


def iter_tensors(w: Workload, device="cpu") -> Iterator[Tuple[str, torch.Tensor]]:
    """All weight tensors one at a time (a caller may free each before asking for the next)."""
    for name, _, _ in tensor_specs(w):
        yield name, make_tensor(w, name, device)
    for name in norm_names(w):
        yield name, make_tensor(w, name, device)


def make_prompts(w: Workload, device="cpu", batch: int | None = None, prompt_len: int | None = None) -> torch.Tensor:
    """[batch, prompt_len] int32 ids uniform on [0, vocab-1): never the mask id."""
    b = w.batch if batch is None else batch
    p = w.prompt_len if prompt_len is None else prompt_len
    return uniform_ids(w.seed + 1000, 0, (b, p), w.vocab - 1, device=device)
