"""CPU oracle for Self Speculative Decoding (SSD) on a masked-diffusion LM.

TEST INFRASTRUCTURE.  Plain, slow, fp64 numpy.  Only the test-suite, the
smoke check and the benchmark's cpu-baseline leg may import this file; the
CUDA library shares no code with it and never calls it.

What is defined here, and from where:

* the model f_theta of Eq. 2 (a bidirectional transformer; the paper gives no
  architecture, the shapes and the pre-norm RMSNorm/RoPE/SwiGLU layout are the
  workload's) -> ``Oracle.forward_rows``;
* semi-autoregressive blocks, Eq. 3 -> ``block_ranges``;
* stepwise decoding (one token per forward, the highest-confidence masked
  position of the current block takes its argmax token; Fig. 2 and the
  baseline of Section 4.1) -> ``Oracle.decode_block_stepwise``;
* SSD: self-drafting (Eq. 4), greedy candidate selection (Section 3.2.2), the
  greedy verification chain of N+1 nodes (Section 3.2.3), batch verification
  (Eq. 5), parent-prediction-vs-child-draft traversal (Section 3.2.4) and the
  loop of Algorithm 1 -> ``select_candidates``, ``build_chain``,
  ``node_predictions``, ``accept_length``, ``Oracle.decode_block_ssd``;
* candidates that run on into the next block when the current one cannot fill the chain
  (Section 3.2.2), under the block order of Section 3.1 -> ``Oracle.verify_window``,
  ``Oracle.generate_spill``;
* the dual cache with a refresh interval of the paper's experimental set-up (Section 4.1) and
  the chain cap that keeps SSD identical to stepwise decoding under it ->
  ``Oracle.refresh_all``, ``Oracle.generate_dual_cache``;
* the acceptance-rate limit of self-drafting, Section 5.1 / Table 2 (how many stepwise
  tokens lie within the draft forward's top-k candidates) -> ``token_topk``,
  ``Oracle.acceptance_limit``;
* the mix-order tree of Section 5.2 (the chain plus one out-of-order branch per chain node
  that has a grandchild, 2N nodes) -> ``build_mix_order_tree``, ``accept_walk_mix_order``.

Readings where the paper is silent:
the forward of a block attends to the cached prefix plus the block itself; a
finished block enters the cache through one more forward over its final
tokens; confidence is the maximum softmax probability with the mask token
excluded; ties go to the lower token id / lower position; a draft "matches"
only if position AND token agree; the next drafts are the last valid node's
own predictions from the same forward.

Precision: everything is fp64.  ``operand_rounding`` optionally rounds the
operands of every contraction (matmul inputs, attention Q/K/V/P) to bfloat16,
which is the arithmetic type the accelerated path is specified to use (bf16
operands, wide accumulation); with ``None`` nothing is rounded.  A collection
of source names (``ROUNDING_SOURCES``) rounds only those operands, which is how
the share of each rounding point in the total bf16 noise is measured.

Pins: see tests/test_oracle_*.py.  The accept-count VALUES on random-init
models have no value printed in the paper to compare with: parity unpinned by
the paper for those (they are pinned by brute force against the stepwise
continuation instead).
"""
from __future__ import annotations

import dataclasses
from typing import Callable, Dict, List, Optional, Sequence, Tuple

import numpy as np


# --------------------------------------------------------------------------------------
# configuration and small helpers
# --------------------------------------------------------------------------------------
@dataclasses.dataclass(frozen=True)
class ModelConfig:
    n_layers: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    mask_id: int
    rope_theta: float
    rms_eps: float


def bf16_round(x: np.ndarray) -> np.ndarray:
    """Round to the nearest bfloat16 (ties to even); returns fp64 holding bf16 values."""
    f = np.ascontiguousarray(x, dtype=np.float32)
    b = f.view(np.uint32).astype(np.uint64)
    b = (b + 0x7FFF + ((b >> 16) & 1)) & 0xFFFF0000
    return b.astype(np.uint32).view(np.float32).astype(np.float64).reshape(np.shape(x))


# The operands a bf16 contraction rounds, by where they enter:
#   proj_in  normalised hidden state into the q/k/v and gate/up projections
#   qkv      rotated q and k, and v, into the two attention contractions
#   p        softmax probabilities into P.V
#   att      attention output into the output projection
#   act      SwiGLU activation into the down projection
#   lm_in    final-norm hidden state into the LM head
ROUNDING_SOURCES = ("proj_in", "qkv", "p", "att", "act", "lm_in")


def block_ranges(gen_len: int, block_len: int) -> List[Tuple[int, int]]:
    """Eq. 3: generation offsets [j*B, min((j+1)*B, L)) for j = 0 .. ceil(L/B)-1."""
    n_blocks = -(-gen_len // block_len)
    return [(j * block_len, min((j + 1) * block_len, gen_len)) for j in range(n_blocks)]


# --------------------------------------------------------------------------------------
# model primitives (each is its textbook definition)
# --------------------------------------------------------------------------------------
def rmsnorm(x: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    """x / sqrt(mean(x^2) + eps) * gain over the last axis."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * gain


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotary embedding, "rotate-half" pairing: feature i is paired with i + hd/2.

    x [T, H, hd], pos [T] absolute positions.  Pair (a, b) at frequency
    theta^(-2i/hd) is rotated by angle pos * frequency.
    """
    hd = x.shape[-1]
    half = hd // 2
    inv_freq = theta ** (-(np.arange(half, dtype=np.float64) * 2.0) / hd)
    ang = pos.astype(np.float64)[:, None] * inv_freq[None, :]
    c = np.cos(ang)[:, None, :]
    s = np.sin(ang)[:, None, :]
    a, b = x[..., :half], x[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, rnd: Callable[[np.ndarray], np.ndarray]) -> np.ndarray:
    """Bidirectional (unmasked) softmax attention with grouped KV heads.

    q [T, H, hd]; k, v [S, Hkv, hd]; query head h reads KV head h // (H/Hkv);
    scale 1/sqrt(hd).  ``rnd`` rounds the probability operand of P.V (the
    normaliser is the unrounded sum).  Returns [T, H*hd].
    """
    T, H, hd = q.shape
    group = H // k.shape[1]
    out = np.empty((T, H, hd), dtype=np.float64)
    for h in range(H):
        g = h // group
        s = (q[:, h, :] @ k[:, g, :].T) / np.sqrt(float(hd))
        p = np.exp(s - s.max(axis=-1, keepdims=True))
        out[:, h, :] = (rnd(p) @ v[:, g, :]) / p.sum(axis=-1, keepdims=True)
    return out.reshape(T, H * hd)


def token_and_confidence(logits: np.ndarray, mask_id: int) -> Tuple[np.ndarray, np.ndarray]:
    """Eq. 2 + Eq. 4 for rows of logits [T, V]: draft token = argmax of the softmax with
    the mask token excluded (lowest id on ties), confidence = that maximum probability."""
    l = np.array(logits, dtype=np.float64, copy=True)
    l[:, mask_id] = -np.inf
    tok = np.argmax(l, axis=-1)
    m = l.max(axis=-1, keepdims=True)
    conf = 1.0 / np.exp(l - m).sum(axis=-1)
    return tok.astype(np.int64), conf


def token_topk(logits: np.ndarray, mask_id: int, k: int) -> Tuple[np.ndarray, np.ndarray]:
    """The k most probable tokens per row of logits [T, V] (mask token excluded), most probable
    first, lower id first among equals, and their softmax probabilities."""
    l = np.array(logits, dtype=np.float64, copy=True)
    l[:, mask_id] = -np.inf
    order = np.argsort(-l, axis=-1, kind="stable")[:, :k]
    m = l.max(axis=-1, keepdims=True)
    z = np.exp(l - m).sum(axis=-1, keepdims=True)
    return order.astype(np.int64), np.exp(np.take_along_axis(l, order, axis=-1) - m) / z


def top2_gap(logits: np.ndarray, mask_id: int) -> np.ndarray:
    """Softmax probability of the best token minus that of the runner-up, per row."""
    l = np.array(logits, dtype=np.float64, copy=True)
    l[:, mask_id] = -np.inf
    m = l.max(axis=-1, keepdims=True)
    p = np.exp(l - m)
    z = p.sum(axis=-1)
    part = np.partition(p, -2, axis=-1)
    return (part[:, -1] - part[:, -2]) / z


# --------------------------------------------------------------------------------------
# SSD logic that does not touch the model (Section 3.2.2 - 3.2.4)
# --------------------------------------------------------------------------------------
def best_masked_position(conf: np.ndarray, masked: np.ndarray) -> int:
    """Highest-confidence masked position; the lower position wins ties."""
    best, best_c = -1, -1.0
    for p in range(len(conf)):
        if masked[p] and conf[p] > best_c:
            best, best_c = p, conf[p]
    return best


def select_candidates(draft_tok: np.ndarray, draft_conf: np.ndarray, masked: np.ndarray,
                      max_drafts: int, keep_one: bool = True) -> List[Tuple[int, int]]:
    """Greedy selection: the N = min(max_drafts, r-1) masked positions of the current block
    with the highest draft confidence, in descending confidence (lower position first on
    ties).  r-1 because every node of the chain must keep one masked position to predict;
    ``keep_one=False`` (the chain goes on into the next block, whose positions the last nodes
    predict) lets all r positions be candidates."""
    pos = [p for p in range(len(masked)) if masked[p]]
    n = max(0, min(max_drafts, len(pos) - (1 if keep_one else 0)))
    order = sorted(pos, key=lambda p: (-draft_conf[p], p))
    return [(p, int(draft_tok[p])) for p in order[:n]]


def build_chain(ids: np.ndarray, masked: np.ndarray, cand: Sequence[Tuple[int, int]], mask_id: int
                ) -> Tuple[np.ndarray, np.ndarray]:
    """Greedy verification chain: node i = current state with candidates 1..i written in
    (N+1 nodes for N candidates).  Returns node ids [N+1, B] and masked flags [N+1, B]."""
    n = len(cand) + 1
    node_ids = np.tile(np.where(masked, mask_id, ids), (n, 1)).astype(np.int64)
    node_masked = np.tile(masked.astype(bool), (n, 1))
    for i in range(1, n):
        for (p, t) in cand[:i]:
            node_ids[i, p] = t
            node_masked[i, p] = False
    return node_ids, node_masked


def node_predictions(tok: np.ndarray, conf: np.ndarray, node_masked: np.ndarray) -> List[Tuple[int, int]]:
    """Per node: the (position, token) that a stepwise step from that node's state would write."""
    out = []
    for i in range(node_masked.shape[0]):
        q = best_masked_position(conf[i], node_masked[i])
        out.append((q, int(tok[i, q])))
    return out


def accept_length(pred: Sequence[Tuple[int, int]], cand: Sequence[Tuple[int, int]]) -> int:
    """Walk the chain from the root: node i's prediction must equal (position and token) the
    draft that node i+1 assumed; stop at the first mismatch.  Returns a = index of the last
    valid node, so a+1 tokens are accepted."""
    a = 0
    while a < len(cand) and pred[a] == cand[a]:
        a += 1
    return a


def build_mix_order_tree(ids: np.ndarray, masked: np.ndarray, cand: Sequence[Tuple[int, int]], mask_id: int
                         ) -> Tuple[np.ndarray, np.ndarray]:
    """Greedy chain plus the mix-order branches of Section 5.2: every chain node that has a
    grandchild (node i, i <= N-2) gets one more child, its own state with candidate i+2
    written in INSTEAD of candidate i+1 - the state stepwise decoding reaches when it takes
    the two candidates in the other order.  Branch nodes get no children.  Node order: chain
    nodes 0..N, then the branch of chain node 0, 1, ..., N-2 (index N+1+i): 2N nodes for
    N >= 1 (6 / 8 / 10 for N = 3 / 4 / 5, Table 3)."""
    n_chain = len(cand) + 1
    chain_ids, chain_masked = build_chain(ids, masked, cand, mask_id)
    rows_ids, rows_masked = [chain_ids], [chain_masked]
    for i in range(n_chain - 2):
        p, t = cand[i + 1]
        bi, bm = chain_ids[i].copy(), chain_masked[i].copy()
        bi[p] = t
        bm[p] = False
        rows_ids.append(bi[None])
        rows_masked.append(bm[None])
    return np.concatenate(rows_ids), np.concatenate(rows_masked)


def accept_walk_mix_order(pred: Sequence[Tuple[int, int]], cand: Sequence[Tuple[int, int]]
                          ) -> Tuple[List[Tuple[int, int]], int]:
    """Traversal of the mix-order tree.  Along the chain as in ``accept_length``; where chain
    node a's prediction is not candidate a+1 but equals candidate a+2 (same tokens, other
    order), that candidate is accepted and the walk moves to node a's branch, whose own
    prediction is accepted too and ends the walk (branches have no children).  Returns the
    accepted (position, token) list in stepwise order and the index of the last valid node."""
    n = len(cand)
    a = 0
    while a < n and pred[a] == cand[a]:
        a += 1
    if a + 1 < n and pred[a] == cand[a + 1]:
        branch = n + 1 + a
        return list(cand[:a]) + [cand[a + 1], pred[branch]], branch
    return list(cand[:a]) + [pred[a]], a


# --------------------------------------------------------------------------------------
# the model and the decode loops
# --------------------------------------------------------------------------------------
class Cache:
    """Per-layer prefix K (post-RoPE) and V, each [S, Hkv, hd]."""

    def __init__(self, cfg: ModelConfig):
        self.k = [np.zeros((0, cfg.n_kv_heads, cfg.head_dim)) for _ in range(cfg.n_layers)]
        self.v = [np.zeros((0, cfg.n_kv_heads, cfg.head_dim)) for _ in range(cfg.n_layers)]

    @property
    def length(self) -> int:
        return self.k[0].shape[0]

    def append(self, new_k: List[np.ndarray], new_v: List[np.ndarray]) -> None:
        for l in range(len(self.k)):
            self.k[l] = np.concatenate([self.k[l], new_k[l]], axis=0)
            self.v[l] = np.concatenate([self.v[l], new_v[l]], axis=0)


@dataclasses.dataclass
class ForwardRecord:
    """Everything about one verification forward (for teacher-forced comparisons)."""
    block: int
    cache_len: int
    ids_before: np.ndarray          # [B] tokens (mask_id where masked)
    masked_before: np.ndarray       # [B] bool
    draft_tok: Optional[np.ndarray]  # [B] stale drafts used to build the chain (None: no drafts yet)
    draft_conf: Optional[np.ndarray]
    cand: List[Tuple[int, int]]
    node_ids: np.ndarray            # [n, B]
    node_masked: np.ndarray         # [n, B]
    tok: np.ndarray                 # [n, B] argmax token per row
    conf: np.ndarray                # [n, B] confidence per row
    gap: np.ndarray                 # [n, B] top-1 minus top-2 probability per row
    pred: List[Tuple[int, int]]
    accepted: int                   # a+1
    last_node: int = -1             # the node whose outputs became the next drafts (-1: not recorded)


class Oracle:
    """f_theta plus the two decode loops.

    ``weights`` maps names to arrays: embed [V,d], lm_head [V,d], norm_final [d] and per
    layer l ``layers.l.{wq,wk,wv,wo,w_gate,w_up,w_down,norm_attn,norm_ffn}`` with matmul
    weights stored [out_features, in_features].  It may be a dict or any object with
    ``__getitem__`` (so that large models can materialise one tensor at a time).
    """

    def __init__(self, cfg: ModelConfig, weights, operand_rounding=None):
        if operand_rounding is None:
            active = ()
        elif operand_rounding == "bf16":
            active = ROUNDING_SOURCES
        else:
            active = tuple(operand_rounding)
            assert all(src in ROUNDING_SOURCES for src in active), active
        self.cfg = cfg
        self.w = weights
        ident = lambda a: a
        self.r = {src: (bf16_round if src in active else ident) for src in ROUNDING_SOURCES}

    def _W(self, name: str) -> np.ndarray:
        return np.asarray(self.w[name], dtype=np.float64)

    # ---- one transformer layer over independent row groups --------------------------
    def layer(self, l: int, groups: List[np.ndarray], positions: List[np.ndarray],
              prefix_k: np.ndarray, prefix_v: np.ndarray) -> Tuple[List[np.ndarray], List[np.ndarray], List[np.ndarray]]:
        """Apply layer l to every group (a group = the rows of one node, [T, d]).  Each group
        attends to [prefix ; its own rows].  Returns (new hidden, post-RoPE K, V) per group."""
        c = self.cfg
        r = self.r
        p = f"layers.{l}."
        wq, wk, wv, wo = self._W(p + "wq"), self._W(p + "wk"), self._W(p + "wv"), self._W(p + "wo")
        wg, wu, wd = self._W(p + "w_gate"), self._W(p + "w_up"), self._W(p + "w_down")
        g1, g2 = self._W(p + "norm_attn"), self._W(p + "norm_ffn")
        outs, ks, vs = [], [], []
        for h, pos in zip(groups, positions):
            T = h.shape[0]
            u = r["proj_in"](rmsnorm(h, g1, c.rms_eps))
            q = rope((u @ wq.T).reshape(T, c.n_heads, c.head_dim), pos, c.rope_theta)
            k = rope((u @ wk.T).reshape(T, c.n_kv_heads, c.head_dim), pos, c.rope_theta)
            v = (u @ wv.T).reshape(T, c.n_kv_heads, c.head_dim)
            q, k, v = r["qkv"](q), r["qkv"](k), r["qkv"](v)
            keys = np.concatenate([prefix_k, k], axis=0)
            vals = np.concatenate([prefix_v, v], axis=0)
            att = r["att"](attention(q, keys, vals, r["p"]))
            h = h + att @ wo.T
            u = r["proj_in"](rmsnorm(h, g2, c.rms_eps))
            act = r["act"](silu(u @ wg.T) * (u @ wu.T))
            h = h + act @ wd.T
            outs.append(h)
            ks.append(k)
            vs.append(v)
        return outs, ks, vs

    def forward_rows(self, ids: np.ndarray, pos0: int, cache: Cache, want_logits: bool = True,
                     logit_rows: Optional[np.ndarray] = None, hidden_trace: Optional[list] = None):
        """f_theta on one or several nodes.  ids [n, T] (or [T]); all nodes sit at absolute
        positions pos0 .. pos0+T-1 and each attends to the cache plus its own T rows.
        Returns (logits [n, T, V] or None, K list per layer [n,T,Hkv,hd], V list).
        ``hidden_trace`` (a list) receives the residual stream [n, T, d] entering layer 0,
        1, ... and, last, the one leaving the final layer (for layer-by-layer comparisons)."""
        c = self.cfg
        ids = np.atleast_2d(np.asarray(ids))
        n, T = ids.shape
        emb = self._W("embed")
        groups = [emb[ids[i]].copy() for i in range(n)]
        pos = [np.arange(pos0, pos0 + T) for _ in range(n)]
        all_k, all_v = [], []
        for l in range(c.n_layers):
            if hidden_trace is not None:
                hidden_trace.append(np.stack(groups))
            groups, ks, vs = self.layer(l, groups, pos, cache.k[l], cache.v[l])
            all_k.append(np.stack(ks))
            all_v.append(np.stack(vs))
        if hidden_trace is not None:
            hidden_trace.append(np.stack(groups))
        logits = None
        if want_logits:
            gf, wlm = self._W("norm_final"), self._W("lm_head")
            logits = np.stack([self.r["lm_in"](rmsnorm(h, gf, c.rms_eps)) @ wlm.T for h in groups])
        return logits, all_k, all_v

    # ---- cache maintenance ----------------------------------------------------------
    def prefill(self, prompt: np.ndarray) -> Cache:
        """The prompt attends to the prompt only; its K/V become the prefix cache."""
        cache = Cache(self.cfg)
        _, ks, vs = self.forward_rows(prompt, 0, cache, want_logits=False)
        cache.append([k[0] for k in ks], [v[0] for v in vs])
        return cache

    def commit_block(self, ids: np.ndarray, cache: Cache) -> None:
        """One forward over the finished block appends its K/V to the prefix cache."""
        _, ks, vs = self.forward_rows(ids, cache.length, cache, want_logits=False)
        cache.append([k[0] for k in ks], [v[0] for v in vs])

    # ---- one verification forward ---------------------------------------------------
    def verify(self, node_ids: np.ndarray, node_masked: np.ndarray, cache: Cache):
        """Eq. 5: all nodes through the model at once; per row (token, confidence, gap)."""
        logits, _, _ = self.forward_rows(node_ids, cache.length, cache)
        n, T, V = logits.shape
        tok, conf = token_and_confidence(logits.reshape(n * T, V), self.cfg.mask_id)
        gap = top2_gap(logits.reshape(n * T, V), self.cfg.mask_id)
        return tok.reshape(n, T), conf.reshape(n, T), gap.reshape(n, T), logits

    # ---- decode loops ---------------------------------------------------------------
    def decode_block_stepwise(self, block_len: int, cache: Cache, block_index: int = 0,
                              trace: Optional[List[ForwardRecord]] = None):
        """One token per forward.  Returns (ids [B], accept counts = [1]*B)."""
        mid = self.cfg.mask_id
        ids = np.full(block_len, mid, dtype=np.int64)
        masked = np.ones(block_len, dtype=bool)
        counts = []
        while masked.any():
            node_ids, node_masked = build_chain(ids, masked, [], mid)
            tok, conf, gap, _ = self.verify(node_ids, node_masked, cache)
            pred = node_predictions(tok, conf, node_masked)
            if trace is not None:
                trace.append(ForwardRecord(block_index, cache.length, ids.copy(), masked.copy(), None, None, [],
                                           node_ids, node_masked, tok, conf, gap, pred, 1))
            q, t = pred[0]
            ids[q] = t
            masked[q] = False
            counts.append(1)
        return ids, counts

    def decode_block_ssd(self, block_len: int, cache: Cache, max_drafts: int, block_index: int = 0,
                         trace: Optional[List[ForwardRecord]] = None,
                         draft_override: Optional[Callable] = None, tree: str = "greedy"):
        """Algorithm 1 restricted to one block.  Returns (ids [B], accept counts per forward).

        ``tree`` is "greedy" (the chain of N+1 nodes, Section 3.2.3) or "mix_order" (the chain
        plus one out-of-order branch per chain node with a grandchild, Section 5.2).
        ``draft_override(ids, masked, draft_tok, draft_conf) -> (draft_tok, draft_conf)``
        lets a test replace the drafts (perfect or adversarial) to pin the accept logic
        independently of the model.
        """
        assert tree in ("greedy", "mix_order")
        mid = self.cfg.mask_id
        ids = np.full(block_len, mid, dtype=np.int64)
        masked = np.ones(block_len, dtype=bool)
        draft_tok: Optional[np.ndarray] = None
        draft_conf: Optional[np.ndarray] = None
        counts = []
        while masked.any():
            if draft_tok is None:
                cand: List[Tuple[int, int]] = []          # no drafts yet: root-only forward
            else:
                dt, dc = draft_tok, draft_conf
                if draft_override is not None:
                    dt, dc = draft_override(ids.copy(), masked.copy(), dt.copy(), dc.copy())
                cand = select_candidates(dt, dc, masked, max_drafts)
            if tree == "greedy":
                node_ids, node_masked = build_chain(ids, masked, cand, mid)
            else:
                node_ids, node_masked = build_mix_order_tree(ids, masked, cand, mid)
            tok, conf, gap, _ = self.verify(node_ids, node_masked, cache)
            pred = node_predictions(tok, conf, node_masked)
            if tree == "greedy":
                a = accept_length(pred, cand)
                accepted, last = list(cand[:a]) + [pred[a]], a
            else:
                accepted, last = accept_walk_mix_order(pred, cand)
            if trace is not None:
                trace.append(ForwardRecord(block_index, cache.length, ids.copy(), masked.copy(),
                                           None if draft_tok is None else draft_tok.copy(),
                                           None if draft_conf is None else draft_conf.copy(),
                                           list(cand), node_ids, node_masked, tok, conf, gap, pred,
                                           len(accepted), last))
            for (p, t) in accepted:
                ids[p] = t
                masked[p] = False
            # next drafts: the last valid node's own predictions on what is still masked
            draft_tok = np.where(masked, tok[last], 0).astype(np.int64)
            draft_conf = np.where(masked, conf[last], 0.0)
            counts.append(len(accepted))
        return ids, counts

    def generate(self, prompt: np.ndarray, gen_len: int, block_len: int, mode: str = "ssd",
                 max_drafts: int = 0, trace: Optional[List[ForwardRecord]] = None,
                 draft_override: Optional[Callable] = None, tree: str = "greedy"):
        """Semi-autoregressive generation of gen_len tokens after the prompt.
        Returns (tokens [gen_len], accept counts per block (list of lists), cache)."""
        cache = self.prefill(np.asarray(prompt))
        out, all_counts = [], []
        for j, (lo, hi) in enumerate(block_ranges(gen_len, block_len)):
            if mode == "stepwise":
                ids, counts = self.decode_block_stepwise(hi - lo, cache, j, trace)
            else:
                ids, counts = self.decode_block_ssd(hi - lo, cache, max_drafts, j, trace, draft_override, tree)
            self.commit_block(ids, cache)
            out.append(ids)
            all_counts.append(counts)
        return np.concatenate(out), all_counts, cache

    # ---- candidates from the next block (Section 3.2.2) -------------------------------
    def verify_window(self, node_ids: np.ndarray, node_masked: np.ndarray, T: int, cache: Cache):
        """Eq. 5 on nodes that span two consecutive blocks: rows [0, T) are the current block,
        rows [T, T+T2) the next one, at positions cache.length ...  The window is block-causal
        like the whole sequence: a row of the current block sees the prefix and its own block, a
        row of the next block sees the prefix, the node's current block and its own block - which
        is the current block's forward followed by the next block's forward with the current
        block's K/V appended to the prefix.  Returns (tok, conf, gap), each [n, T+T2]."""
        n, W = node_ids.shape
        S = cache.length
        toks, confs, gaps = [], [], []
        for i in range(n):
            la, ks, vs = self.forward_rows(node_ids[i, :T], S, cache)
            ext = Cache(self.cfg)
            ext.k = [np.concatenate([cache.k[l], ks[l][0]], axis=0) for l in range(self.cfg.n_layers)]
            ext.v = [np.concatenate([cache.v[l], vs[l][0]], axis=0) for l in range(self.cfg.n_layers)]
            lb, _, _ = self.forward_rows(node_ids[i, T:], S + T, ext)
            logits = np.concatenate([la[0], lb[0]], axis=0)
            t, c = token_and_confidence(logits, self.cfg.mask_id)
            toks.append(t)
            confs.append(c)
            gaps.append(top2_gap(logits, self.cfg.mask_id))
        return np.stack(toks), np.stack(confs), np.stack(gaps)

    def generate_spill(self, prompt: np.ndarray, gen_len: int, block_len: int, max_drafts: int,
                       trace: Optional[List[ForwardRecord]] = None):
        """SSD whose candidate list runs on into the next block (Section 3.2.2: positions of
        block j+1 are selected only when block j has fewer remaining positions than the draft
        length).  While the current block has more than max_drafts masked positions a forward
        is the single-block chain of ``decode_block_ssd``.  Otherwise the nodes span the window
        [current block | next block]: the candidates are ALL masked positions of the current
        block by draft confidence, then the most confident drafts of the next block up to
        max_drafts in total; a node whose current block is full predicts in the next block, so
        nothing of block j+1 is accepted before block j is complete (Section 3.1).  The next
        block keeps its accepted tokens and drafts when it becomes the current one.
        Returns (tokens [gen_len], accept counts per forward, forwards that used a window)."""
        mid = self.cfg.mask_id
        cache = self.prefill(np.asarray(prompt))
        ranges = block_ranges(gen_len, block_len)
        fresh = lambda T: dict(ids=np.full(T, mid, dtype=np.int64), masked=np.ones(T, dtype=bool), dt=None, dc=None)
        cur = fresh(ranges[0][1] - ranges[0][0])
        out, counts, windows = [], [], 0
        for j, (lo, hi) in enumerate(ranges):
            T = hi - lo
            nxt = fresh(ranges[j + 1][1] - ranges[j + 1][0]) if j + 1 < len(ranges) else None
            while cur["masked"].any():
                r = int(cur["masked"].sum())
                window = cur["dt"] is not None and nxt is not None and r <= max_drafts
                if not window:
                    cand = [] if cur["dt"] is None else select_candidates(cur["dt"], cur["dc"], cur["masked"], max_drafts)
                    node_ids, node_masked = build_chain(cur["ids"], cur["masked"], cand, mid)
                    tok, conf, gap, _ = self.verify(node_ids, node_masked, cache)
                    pred = node_predictions(tok, conf, node_masked)
                else:
                    windows += 1
                    T2 = len(nxt["ids"])
                    # every masked position of the current block, then the next block's (which keeps one to predict)
                    cand = select_candidates(cur["dt"], cur["dc"], cur["masked"], r, keep_one=False)
                    if nxt["dt"] is not None:
                        more = select_candidates(nxt["dt"], nxt["dc"], nxt["masked"], max_drafts - r)
                        cand = cand + [(T + p, t) for (p, t) in more]
                    ids2 = np.concatenate([cur["ids"], nxt["ids"]])
                    masked2 = np.concatenate([cur["masked"], nxt["masked"]])
                    node_ids, node_masked = build_chain(ids2, masked2, cand, mid)
                    tok, conf, gap = self.verify_window(node_ids, node_masked, T, cache)
                    # a node predicts in the current block while that has a masked position, else in the next
                    pred = []
                    for i in range(node_ids.shape[0]):
                        in_cur = node_masked[i, :T].any()
                        scope = np.zeros(T + T2, dtype=bool)
                        scope[:T] = in_cur
                        scope[T:] = not in_cur
                        q = best_masked_position(conf[i], node_masked[i] & scope)
                        pred.append((q, int(tok[i, q])))
                a = accept_length(pred, cand)
                accepted = list(cand[:a]) + [pred[a]]
                if trace is not None:
                    # a window forward records [current | next]; a next block without drafts shows tokens -1
                    ib, mb = cur["ids"].copy(), cur["masked"].copy()
                    db = None if cur["dt"] is None else cur["dt"].copy()
                    cb = None if cur["dc"] is None else cur["dc"].copy()
                    if window:
                        ib, mb = np.concatenate([ib, nxt["ids"]]), np.concatenate([mb, nxt["masked"]])
                        db = np.concatenate([db, nxt["dt"] if nxt["dt"] is not None else np.full(T2, -1)])
                        cb = np.concatenate([cb, nxt["dc"] if nxt["dc"] is not None else np.zeros(T2)])
                    trace.append(ForwardRecord(j, cache.length, ib, mb, db, cb, list(cand), node_ids, node_masked,
                                               tok, conf, gap, pred, len(accepted), a))
                for (p, t) in accepted:
                    blk, pp = (cur, p) if p < T else (nxt, p - T)
                    blk["ids"][pp] = t
                    blk["masked"][pp] = False
                cur["dt"] = np.where(cur["masked"], tok[a][:T], 0).astype(np.int64)
                cur["dc"] = np.where(cur["masked"], conf[a][:T], 0.0)
                if window:
                    nxt["dt"] = np.where(nxt["masked"], tok[a][T:], 0).astype(np.int64)
                    nxt["dc"] = np.where(nxt["masked"], conf[a][T:], 0.0)
                counts.append(len(accepted))
            self.commit_block(cur["ids"], cache)
            out.append(cur["ids"])
            cur = nxt
        return np.concatenate(out), counts, windows

    # ---- dual cache with a refresh interval (Section 4.1, implementation details) ------
    def refresh_all(self, tokens: np.ndarray) -> Cache:
        """K/V of EVERY position of the sequence [prompt | generation, MASK where undecoded] from one
        forward in which all positions see all positions (no block structure)."""
        cache = Cache(self.cfg)
        _, ks, vs = self.forward_rows(np.asarray(tokens), 0, cache, want_logits=False)
        cache.append([k[0] for k in ks], [v[0] for v in vs])
        return cache

    def generate_dual_cache(self, prompt: np.ndarray, gen_len: int, block_len: int, refresh: int,
                            max_drafts: int = 0, counts_out: Optional[list] = None):
        """Decoding under the dual cache of the paper's set-up (Section 4.1): the K/V of all positions
        OUTSIDE the current block - the prefix and the still masked suffix - are cached, a forward
        computes the current block's rows against them, and the cache is refreshed (``refresh_all``)
        at the start of every block and again whenever `refresh` tokens have been decoded since the
        last refresh.  Between refreshes the cached K/V are stale: this is an approximation of
        full-sequence decoding, so stepwise decoding is defined WITH the schedule.  max_drafts = 0 is
        that stepwise decoding; with max_drafts > 0 the verification chain is additionally capped so
        that a forward never accepts past the next refresh point (draft length <= refresh - decoded
        since the last refresh - 1), which keeps the tokens those of stepwise decoding under the same
        schedule.  Returns (tokens [gen_len], forwards, refreshes)."""
        mid = self.cfg.mask_id
        P = len(prompt)
        x = np.concatenate([np.asarray(prompt, dtype=np.int64), np.full(gen_len, mid, dtype=np.int64)])
        forwards = refreshes = 0
        for (lo, hi) in block_ranges(gen_len, block_len):
            S, T = P + lo, hi - lo
            ids = np.full(T, mid, dtype=np.int64)
            masked = np.ones(T, dtype=bool)
            dt = dc = None
            since = refresh                                     # a block starts with a refresh
            while masked.any():
                if since >= refresh:
                    full = self.refresh_all(x)
                    refreshes += 1
                    since = 0
                    outside = Cache(self.cfg)                   # everything but the current block's rows
                    outside.k = [np.concatenate([k[:S], k[S + T:]], axis=0) for k in full.k]
                    outside.v = [np.concatenate([v[:S], v[S + T:]], axis=0) for v in full.v]
                cap = min(max_drafts, refresh - since - 1)
                cand = [] if dt is None else select_candidates(dt, dc, masked, cap)
                node_ids, node_masked = build_chain(ids, masked, cand, mid)
                # (the cached keys carry their positions inside the rotated K, so they need not be a prefix)
                logits, _, _ = self.forward_rows(node_ids, S, outside)
                n, _, V = logits.shape
                tok, conf = token_and_confidence(logits.reshape(n * T, V), mid)
                tok, conf = tok.reshape(n, T), conf.reshape(n, T)
                pred = node_predictions(tok, conf, node_masked)
                a = accept_length(pred, cand)
                for (p, t) in list(cand[:a]) + [pred[a]]:
                    ids[p] = t
                    masked[p] = False
                x[S:S + T] = np.where(masked, mid, ids)
                dt = np.where(masked, tok[a], 0).astype(np.int64)
                dc = np.where(masked, conf[a], 0.0)
                since += a + 1
                forwards += 1
                if counts_out is not None:
                    counts_out.append(a + 1)
        return x[P:], forwards, refreshes

    # ---- acceptance-rate limit of self-drafting (Section 5.1, Table 2) ---------------
    def acceptance_limit_block(self, block_len: int, cache: Cache, draft_len: int, k_max: int):
        """Stepwise decoding of one block in rounds of draft_len + 1 steps.  The forward that opens a
        round is the draft: its k most probable tokens per masked position are recorded; every token
        the round then decodes (the first one comes from the draft forward itself and is not counted)
        is "matched at k" if it is among the draft's top k at its position - such a token could have
        been accepted without a forward of its own.  Returns (ids [B], matched [k_max] with
        matched[k-1] = tokens matched at k, steps = forwards stepwise decoding took)."""
        mid = self.cfg.mask_id
        ids = np.full(block_len, mid, dtype=np.int64)
        masked = np.ones(block_len, dtype=bool)
        matched = np.zeros(k_max, dtype=np.int64)
        steps, in_round, draft_top = 0, 0, None
        while masked.any():
            node_ids, node_masked = build_chain(ids, masked, [], mid)
            tok, conf, _, logits = self.verify(node_ids, node_masked, cache)
            q, t = node_predictions(tok, conf, node_masked)[0]
            if in_round == 0:
                draft_top, _ = token_topk(logits[0], mid, k_max)
            else:
                hit = np.nonzero(draft_top[q] == t)[0]
                if len(hit):
                    matched[int(hit[0]):] += 1          # matched at every k above the rank it was found at
            ids[q] = t
            masked[q] = False
            steps += 1
            in_round = (in_round + 1) % (draft_len + 1)
        return ids, matched, steps

    def acceptance_limit(self, prompt: np.ndarray, gen_len: int, block_len: int, draft_len: int, k_max: int):
        """Table 2's quantity for one generation: the fraction of stepwise forwards that drafts
        matched within their top k would save, for k = 1 .. k_max (bounded by N/(N+1)).  Returns
        (tokens [gen_len], reduction [k_max])."""
        cache = self.prefill(np.asarray(prompt))
        out, matched, steps = [], np.zeros(k_max, dtype=np.int64), 0
        for (lo, hi) in block_ranges(gen_len, block_len):
            ids, m, s = self.acceptance_limit_block(hi - lo, cache, draft_len, k_max)
            self.commit_block(ids, cache)
            out.append(ids)
            matched += m
            steps += s
        return np.concatenate(out), matched / float(steps)

    # ---- the uncached definition used to pin the cache semantics --------------------
    def uncached_block_causal(self, tokens: np.ndarray, segment_lengths: Sequence[int],
                              hidden_trace: Optional[list] = None):
        """Forward over the whole sequence with NO cache: position t attends to every
        position of its own segment and of all earlier segments (prompt = first segment).
        Returns (logits [T,V], K list [T,Hkv,hd], V list).  Written as a plain masked
        attention over the full sequence, independently of ``layer``'s cache handling.
        ``hidden_trace`` receives the residual stream [T, d] entering each layer, then the
        final one."""
        c = self.cfg
        T = len(tokens)
        seg = np.repeat(np.arange(len(segment_lengths)), segment_lengths)
        assert len(seg) == T
        allow = seg[None, :] <= seg[:, None]            # [query, key]
        pos = np.arange(T)
        h = self._W("embed")[np.asarray(tokens)].copy()
        r = self.r
        Ks, Vs = [], []
        for l in range(c.n_layers):
            if hidden_trace is not None:
                hidden_trace.append(h.copy())
            p = f"layers.{l}."
            u = r["proj_in"](rmsnorm(h, self._W(p + "norm_attn"), c.rms_eps))
            q = r["qkv"](rope((u @ self._W(p + "wq").T).reshape(T, c.n_heads, c.head_dim), pos, c.rope_theta))
            k = r["qkv"](rope((u @ self._W(p + "wk").T).reshape(T, c.n_kv_heads, c.head_dim), pos, c.rope_theta))
            v = r["qkv"]((u @ self._W(p + "wv").T).reshape(T, c.n_kv_heads, c.head_dim))
            group = c.n_heads // c.n_kv_heads
            att = np.empty((T, c.n_heads, c.head_dim))
            for hh in range(c.n_heads):
                s = (q[:, hh, :] @ k[:, hh // group, :].T) / np.sqrt(float(c.head_dim))
                s = np.where(allow, s, -np.inf)
                pr = np.exp(s - s.max(axis=-1, keepdims=True))
                att[:, hh, :] = (r["p"](pr) @ v[:, hh // group, :]) / pr.sum(axis=-1, keepdims=True)
            h = h + r["att"](att.reshape(T, -1)) @ self._W(p + "wo").T
            u = r["proj_in"](rmsnorm(h, self._W(p + "norm_ffn"), c.rms_eps))
            h = h + r["act"](silu(u @ self._W(p + "w_gate").T) * (u @ self._W(p + "w_up").T)) @ self._W(p + "w_down").T
            Ks.append(k)
            Vs.append(v)
        if hidden_trace is not None:
            hidden_trace.append(h.copy())
        logits = r["lm_in"](rmsnorm(h, self._W("norm_final"), c.rms_eps)) @ self._W("lm_head").T
        return logits, Ks, Vs
