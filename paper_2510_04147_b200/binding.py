"""ctypes binding of the C ABI in include/ssd.h: same names, argument marshalling only.

Every step of the path runs inside the shared library's CUDA kernels.  The library is looked for
in-tree (``libssd_b200.so`` next to this file, built by ``build.py``); if it is missing, or if no
CUDA device is present, calls fail loudly - there is no CPU path here.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence, Tuple

import numpy as np
import torch

from . import workloads as wl

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libssd_b200.so")

SSD_OK = 0
ERR_NAMES = {-1: "INVALID_ARG", -2: "SHAPE", -3: "OOM", -4: "CUDA", -5: "OVERFLOW", -6: "TIMEOUT", -7: "STATE",
             -8: "NONFINITE"}
DTYPE_BF16, DTYPE_F32 = 0, 1
MODE_STEPWISE, MODE_SSD = 0, 1
PROF_FAMILIES = ("gemm", "lmhead", "attn", "elemwise", "tree", "gemm_qkv", "gemm_o", "gemm_gu", "gemm_down")
PROF_TOP = PROF_FAMILIES[:5]          # the last four break "gemm" down by projection

EXPORTS = ["ssd_create", "ssd_destroy", "ssd_last_error", "ssd_load_weights", "ssd_prefill", "ssd_prefill_dev",
           "ssd_decode_block", "ssd_block_begin", "ssd_set_block_state", "ssd_get_block_state", "ssd_block_step",
           "ssd_set_next_block_state", "ssd_get_next_block_state", "ssd_read_forward_outputs", "ssd_refresh_cache", "ssd_refresh_count",
           "ssd_block_commit", "ssd_verify_forward", "ssd_read_cache", "ssd_write_cache", "ssd_verify_layers",
           "ssd_verify_forward_topk", "ssd_probe_acceptance_limit", "ssd_cache_length", "ssd_rewind", "ssd_gemm_bf16",
           "ssd_gemm_bf16_noalloc",
           "ssd_launch_count", "ssd_profile_enable", "ssd_profile_read", "ssd_set_option"]


class SsdConfig(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("d_ffn", C.c_int32), ("vocab", C.c_int32), ("mask_id", C.c_int32),
                ("rope_theta", C.c_float), ("rms_eps", C.c_float), ("max_batch", C.c_int32), ("max_seq", C.c_int32),
                ("block_len", C.c_int32), ("max_drafts", C.c_int32)]


class SsdError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"ssd error {code} ({ERR_NAMES.get(code, '?')}): {msg}")
        self.code = code


_lib = None


def load_library() -> C.CDLL:
    """dlopen the in-tree library and declare the prototypes.  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(f"{LIB_PATH} not found: build it with `python -m paper_2510_04147_b200.build` "
                                "(nvcc, sm_100a); there is no fallback implementation")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
    P = C.POINTER
    lib.ssd_create.argtypes = [P(SsdConfig), vp, P(vp)]
    lib.ssd_destroy.argtypes = [vp]
    lib.ssd_destroy.restype = None
    lib.ssd_last_error.argtypes = [vp]
    lib.ssd_last_error.restype = C.c_char_p
    lib.ssd_load_weights.argtypes = [vp, C.c_char_p, vp, i32, P(i64), i32]
    lib.ssd_prefill.argtypes = [vp, i32, i32, vp]
    lib.ssd_prefill_dev.argtypes = [vp, i32, i32, vp]
    lib.ssd_decode_block.argtypes = [vp, i32, i32, vp, vp, vp]
    lib.ssd_block_begin.argtypes = [vp, i32]
    lib.ssd_set_block_state.argtypes = [vp, vp, vp, vp, vp]
    lib.ssd_get_block_state.argtypes = [vp, vp, vp, vp, vp]
    lib.ssd_set_next_block_state.argtypes = [vp, vp, vp, vp, vp]
    lib.ssd_get_next_block_state.argtypes = [vp, vp, vp, vp, vp]
    lib.ssd_read_forward_outputs.argtypes = [vp, i32, vp, vp]
    lib.ssd_refresh_cache.argtypes = [vp]
    lib.ssd_refresh_count.argtypes = [vp]
    lib.ssd_refresh_count.restype = i64
    lib.ssd_block_step.argtypes = [vp, i32, vp, vp]
    lib.ssd_block_commit.argtypes = [vp]
    lib.ssd_verify_forward.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp]
    lib.ssd_read_cache.argtypes = [vp, i32, i32, i32, vp, vp]
    lib.ssd_write_cache.argtypes = [vp, i32, i32, i32, vp, vp]
    lib.ssd_verify_layers.argtypes = [vp, i32, i32, i32, i32, i32, vp, vp, vp, vp]
    lib.ssd_verify_forward_topk.argtypes = [vp, i32, i32, i32, vp, vp, i32, vp, vp]
    lib.ssd_probe_acceptance_limit.argtypes = [vp, i32, i32, i32, vp, vp, vp]
    lib.ssd_cache_length.argtypes = [vp]
    lib.ssd_rewind.argtypes = [vp, i32]
    lib.ssd_gemm_bf16.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32]
    lib.ssd_gemm_bf16_noalloc.argtypes = [vp, vp, vp, i32, i32, i32, i32, vp]
    lib.ssd_launch_count.argtypes = [vp]
    lib.ssd_launch_count.restype = i64
    lib.ssd_profile_enable.argtypes = [vp, i32]
    lib.ssd_profile_read.argtypes = [vp, vp, vp, vp]
    lib.ssd_set_option.argtypes = [vp, C.c_char_p, i32]
    for name in EXPORTS:
        fn = getattr(lib, name)
        if name not in ("ssd_destroy", "ssd_last_error", "ssd_launch_count", "ssd_refresh_count"):
            fn.restype = i32
    _lib = lib
    return lib


def gemm_bf16_noalloc(x: torch.Tensor, w: torch.Tensor, out: torch.Tensor, split_k: int = 1) -> int:
    """ssd_gemm_bf16_noalloc on caller-owned tensors (x [rows,k] bf16, w [n,k] bf16, out [rows,n] fp32, all on the
    current CUDA device).  Needs no context and allocates nothing; returns the C return code."""
    lib = load_library()
    assert x.is_cuda and w.is_cuda and out.is_cuda and x.dtype == w.dtype == torch.bfloat16 and out.dtype == torch.float32
    assert x.is_contiguous() and w.is_contiguous() and out.is_contiguous()
    assert x.shape[1] == w.shape[1] and out.shape == (x.shape[0], w.shape[0])
    return int(lib.ssd_gemm_bf16_noalloc(C.c_void_p(x.data_ptr()), C.c_void_p(w.data_ptr()), C.c_void_p(out.data_ptr()),
                                         x.shape[0], w.shape[0], x.shape[1], split_k,
                                         C.c_void_p(torch.cuda.current_stream().cuda_stream)))


def _np_ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def config_from_workload(w: wl.Workload, max_drafts: int, max_batch: Optional[int] = None,
                         max_seq: Optional[int] = None) -> SsdConfig:
    return SsdConfig(n_layers=w.n_layers, d_model=w.d_model, n_heads=w.n_heads, n_kv_heads=w.n_kv_heads,
                     head_dim=w.head_dim, d_ffn=w.d_ffn, vocab=w.vocab, mask_id=w.mask_id, rope_theta=w.rope_theta,
                     rms_eps=w.rms_eps, max_batch=max_batch or w.batch, max_seq=max_seq or (w.prompt_len + w.gen_len),
                     block_len=w.block_len, max_drafts=max_drafts)


class Ssd:
    """One library context.  Methods carry the C function names without the ``ssd_`` prefix."""

    def __init__(self, cfg: SsdConfig, stream: Optional[torch.cuda.Stream] = None):
        self.lib = load_library()
        self.cfg = cfg
        self._ctx = C.c_void_p()
        self.stream = stream
        handle = C.c_void_p(stream.cuda_stream if stream is not None else torch.cuda.current_stream().cuda_stream)
        rc = self.lib.ssd_create(C.byref(cfg), handle, C.byref(self._ctx))
        if rc != SSD_OK:
            raise SsdError(rc, self.lib.ssd_last_error(None).decode())

    # -- helpers
    def _check(self, rc: int):
        if rc != SSD_OK:
            raise SsdError(rc, self.lib.ssd_last_error(self._ctx).decode())

    def destroy(self):
        if self._ctx:
            self.lib.ssd_destroy(self._ctx)
            self._ctx = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    # -- C ABI, one method per entry point
    def load_weights(self, name: str, t: torch.Tensor):
        assert t.is_cuda and t.is_contiguous()
        dt = {torch.bfloat16: DTYPE_BF16, torch.float32: DTYPE_F32}[t.dtype]
        shape = (C.c_int64 * t.dim())(*t.shape)
        self._check(self.lib.ssd_load_weights(self._ctx, name.encode(), C.c_void_p(t.data_ptr()), dt, shape, t.dim()))

    def prefill(self, prompt_ids: np.ndarray):
        p = np.ascontiguousarray(prompt_ids, dtype=np.int32)
        assert p.ndim == 2
        self._check(self.lib.ssd_prefill(self._ctx, p.shape[0], p.shape[1], _np_ptr(p)))

    def prefill_dev(self, prompt_ids: torch.Tensor):
        assert prompt_ids.is_cuda and prompt_ids.dtype == torch.int32 and prompt_ids.is_contiguous()
        self._check(self.lib.ssd_prefill_dev(self._ctx, prompt_ids.shape[0], prompt_ids.shape[1],
                                             C.c_void_p(prompt_ids.data_ptr())))

    def decode_block(self, mode: int, block_tokens: int, batch: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
        tok = np.zeros((batch, block_tokens), np.int32)
        acc = np.zeros((batch, block_tokens), np.int32)
        nf = np.zeros(batch, np.int32)
        self._check(self.lib.ssd_decode_block(self._ctx, mode, block_tokens, _np_ptr(tok), _np_ptr(acc), _np_ptr(nf)))
        return tok, acc, nf

    def decode_block_into(self, mode: int, block_tokens: int, tok_ptr: int, acc_ptr: int, nf_ptr: int):
        """Same call with caller-owned host buffers given as addresses (e.g. pinned memory)."""
        self._check(self.lib.ssd_decode_block(self._ctx, mode, block_tokens, C.c_void_p(tok_ptr), C.c_void_p(acc_ptr),
                                              C.c_void_p(nf_ptr)))

    def prefill_ptr(self, batch: int, prompt_len: int, host_ptr: int):
        self._check(self.lib.ssd_prefill(self._ctx, batch, prompt_len, C.c_void_p(host_ptr)))

    def rewind(self, length: int):
        self._check(self.lib.ssd_rewind(self._ctx, length))

    def block_begin(self, block_tokens: int):
        self._check(self.lib.ssd_block_begin(self._ctx, block_tokens))

    def set_block_state(self, ids, masked, draft_tok=None, draft_conf=None):
        ids = np.ascontiguousarray(ids, dtype=np.int32)
        masked = np.ascontiguousarray(masked, dtype=np.uint8)
        dt = None if draft_tok is None else np.ascontiguousarray(draft_tok, dtype=np.int32)
        dc = None if draft_conf is None else np.ascontiguousarray(draft_conf, dtype=np.float32)
        self._check(self.lib.ssd_set_block_state(self._ctx, _np_ptr(ids), _np_ptr(masked), _np_ptr(dt), _np_ptr(dc)))

    def get_block_state(self, batch: int, block_tokens: int):
        ids = np.zeros((batch, block_tokens), np.int32)
        masked = np.zeros((batch, block_tokens), np.uint8)
        dt = np.zeros((batch, block_tokens), np.int32)
        dc = np.zeros((batch, block_tokens), np.float32)
        self._check(self.lib.ssd_get_block_state(self._ctx, _np_ptr(ids), _np_ptr(masked), _np_ptr(dt), _np_ptr(dc)))
        return ids, masked, dt, dc

    def set_next_block_state(self, ids, masked, draft_tok=None, draft_conf=None):
        ids = np.ascontiguousarray(ids, dtype=np.int32)
        masked = np.ascontiguousarray(masked, dtype=np.uint8)
        dt = None if draft_tok is None else np.ascontiguousarray(draft_tok, dtype=np.int32)
        dc = None if draft_conf is None else np.ascontiguousarray(draft_conf, dtype=np.float32)
        self._check(self.lib.ssd_set_next_block_state(self._ctx, _np_ptr(ids), _np_ptr(masked), _np_ptr(dt), _np_ptr(dc)))

    def get_next_block_state(self, batch: int, next_tokens: int):
        ids = np.zeros((batch, next_tokens), np.int32)
        masked = np.zeros((batch, next_tokens), np.uint8)
        dt = np.zeros((batch, next_tokens), np.int32)
        dc = np.zeros((batch, next_tokens), np.float32)
        self._check(self.lib.ssd_get_next_block_state(self._ctx, _np_ptr(ids), _np_ptr(masked), _np_ptr(dt), _np_ptr(dc)))
        return ids, masked, dt, dc

    def read_forward_outputs(self, n_rows: int):
        tok = np.zeros(n_rows, np.int32)
        conf = np.zeros(n_rows, np.float32)
        self._check(self.lib.ssd_read_forward_outputs(self._ctx, n_rows, _np_ptr(tok), _np_ptr(conf)))
        return tok, conf

    def refresh_cache(self):
        self._check(self.lib.ssd_refresh_cache(self._ctx))

    def refresh_count(self) -> int:
        return int(self.lib.ssd_refresh_count(self._ctx))

    def block_step(self, max_drafts: int, batch: int):
        acc = np.zeros(batch, np.int32)
        nn = np.zeros(batch, np.int32)
        self._check(self.lib.ssd_block_step(self._ctx, max_drafts, _np_ptr(acc), _np_ptr(nn)))
        return acc, nn

    def block_commit(self):
        self._check(self.lib.ssd_block_commit(self._ctx))

    def verify_forward(self, node_ids: np.ndarray, node_masked: np.ndarray, want_logits: bool = False):
        ids = np.ascontiguousarray(node_ids, dtype=np.int32)
        mk = np.ascontiguousarray(node_masked, dtype=np.uint8)
        assert ids.ndim == 3 and ids.shape == mk.shape
        b, n, t = ids.shape
        tok = np.zeros((b, n, t), np.int32)
        conf = np.zeros((b, n, t), np.float32)
        logits = np.zeros((b, n, t, self.cfg.vocab), np.float32) if want_logits else None
        self._check(self.lib.ssd_verify_forward(self._ctx, b, n, t, _np_ptr(ids), _np_ptr(mk), _np_ptr(tok),
                                                _np_ptr(conf), _np_ptr(logits)))
        return tok, conf, logits

    def verify_forward_topk(self, node_ids: np.ndarray, node_masked: np.ndarray, k: int):
        ids = np.ascontiguousarray(node_ids, dtype=np.int32)
        mk = np.ascontiguousarray(node_masked, dtype=np.uint8)
        assert ids.ndim == 3 and ids.shape == mk.shape
        b, n, t = ids.shape
        tok = np.zeros((b, n, t, k), np.int32)
        prob = np.zeros((b, n, t, k), np.float32)
        self._check(self.lib.ssd_verify_forward_topk(self._ctx, b, n, t, _np_ptr(ids), _np_ptr(mk), k, _np_ptr(tok),
                                                     _np_ptr(prob)))
        return tok, prob

    def probe_acceptance_limit(self, block_tokens: int, draft_len: int, k_max: int, batch: int):
        """Returns (tokens [batch, block_tokens], matched [k_max], steps)."""
        tok = np.zeros((batch, block_tokens), np.int32)
        matched = np.zeros(k_max, np.int64)
        steps = np.zeros(1, np.int64)
        self._check(self.lib.ssd_probe_acceptance_limit(self._ctx, block_tokens, draft_len, k_max, _np_ptr(tok),
                                                        _np_ptr(matched), _np_ptr(steps)))
        return tok, matched, int(steps[0])

    def read_cache(self, layer: int, seq: int, length: int):
        kv = self.cfg.n_kv_heads * self.cfg.head_dim
        k = np.zeros((length, self.cfg.n_kv_heads, self.cfg.head_dim), np.float32)
        v = np.zeros_like(k)
        assert k.size == length * kv
        self._check(self.lib.ssd_read_cache(self._ctx, layer, seq, length, _np_ptr(k), _np_ptr(v)))
        return k, v

    def write_cache(self, layer: int, seq: int, k: np.ndarray, v: np.ndarray):
        k = np.ascontiguousarray(k, dtype=np.float32)
        v = np.ascontiguousarray(v, dtype=np.float32)
        assert k.shape == v.shape and k.shape[1:] == (self.cfg.n_kv_heads, self.cfg.head_dim)
        self._check(self.lib.ssd_write_cache(self._ctx, layer, seq, k.shape[0], _np_ptr(k), _np_ptr(v)))

    def verify_layers(self, h_in: np.ndarray, batch: int, n_nodes: int, block_tokens: int, layer_begin: int,
                      layer_end: int, want_stats: bool = False):
        """Returns (h_out [batch*n_nodes*block_tokens, d], tok or None, conf or None)."""
        h = np.ascontiguousarray(h_in, dtype=np.float32).reshape(batch * n_nodes * block_tokens, self.cfg.d_model)
        out = np.zeros_like(h)
        tok = np.zeros((batch, n_nodes, block_tokens), np.int32) if want_stats else None
        conf = np.zeros((batch, n_nodes, block_tokens), np.float32) if want_stats else None
        self._check(self.lib.ssd_verify_layers(self._ctx, batch, n_nodes, block_tokens, layer_begin, layer_end,
                                               _np_ptr(h), _np_ptr(out), _np_ptr(tok), _np_ptr(conf)))
        return out, tok, conf

    def cache_length(self) -> int:
        rc = self.lib.ssd_cache_length(self._ctx)
        if rc < 0:
            self._check(rc)
        return rc

    def gemm_bf16(self, x: torch.Tensor, w: torch.Tensor, split_k: int = 1) -> torch.Tensor:
        assert x.is_cuda and w.is_cuda and x.dtype == w.dtype == torch.bfloat16
        assert x.is_contiguous() and w.is_contiguous() and x.shape[1] == w.shape[1]
        out = torch.empty((x.shape[0], w.shape[0]), dtype=torch.float32, device=x.device)
        self._check(self.lib.ssd_gemm_bf16(self._ctx, C.c_void_p(x.data_ptr()), C.c_void_p(w.data_ptr()),
                                           C.c_void_p(out.data_ptr()), x.shape[0], w.shape[0], x.shape[1], split_k))
        return out

    def launch_count(self) -> int:
        return int(self.lib.ssd_launch_count(self._ctx))

    def profile_enable(self, on):
        """False / 0: off; True / 1: CUDA events around every launch; 2: end-of-launch marks in the live stream."""
        self._check(self.lib.ssd_profile_enable(self._ctx, int(on)))

    def profile_read(self):
        n = len(PROF_FAMILIES)
        launches = (C.c_int64 * n)()
        ms = (C.c_double * n)()
        by = (C.c_double * n)()
        self._check(self.lib.ssd_profile_read(self._ctx, launches, ms, by))
        return {f: {"launches": int(launches[i]), "ms": float(ms[i]), "bytes": float(by[i])}
                for i, f in enumerate(PROF_FAMILIES)}

    def set_option(self, key: str, value: int):
        self._check(self.lib.ssd_set_option(self._ctx, key.encode(), value))

    # -- convenience built on the calls above (no arithmetic)
    def load_workload_weights(self, w: wl.Workload, device="cuda"):
        """Draw every tensor of the workload on the device, one at a time, and hand it to the library."""
        for name, t in wl.iter_tensors(w, device):
            self.load_weights(name, t.contiguous())
            del t

    def generate(self, mode: int, gen_len: int, block_len: int, batch: int, cross_block: bool = False):
        """All blocks of one generation after prefill.  Returns (tokens [batch, gen_len], accept counts
        per block, forwards per block).  ``cross_block``: candidates may run on into the next block (the
        option is set to the next block's length before every block, to 0 before the last)."""
        toks, accs, nfs = [], [], []
        done = 0
        while done < gen_len:
            t = min(block_len, gen_len - done)
            if cross_block:
                self.set_option("cross_block", min(block_len, gen_len - done - t))
            tok, acc, nf = self.decode_block(mode, t, batch)
            toks.append(tok)
            accs.append(acc)
            nfs.append(nf)
            done += t
        if cross_block:
            self.set_option("cross_block", 0)
        return np.concatenate(toks, axis=1), accs, nfs
