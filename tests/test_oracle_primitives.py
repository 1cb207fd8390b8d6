"""Pins for the oracle's model arithmetic: every primitive against a library routine or a
closed form, and the whole forward against a composition of torch library calls."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import ssd_oracle as so
from tests.helpers import SMALL, SMALL_GQA, make_oracle, oracle_config, oracle_weights
from paper_2510_04147_b200 import workloads as wl

rng = np.random.default_rng(0)


def test_bf16_round_matches_torch():
    x = np.concatenate([rng.standard_normal(5000) * 10.0 ** rng.integers(-6, 6, 5000),
                        [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895313892515355e38]])
    got = so.bf16_round(x)
    ref = torch.tensor(x, dtype=torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(got, ref)
    # ties go to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert so.bf16_round(np.array([1.00390625]))[0] == 1.0
    assert so.bf16_round(np.array([1.01171875]))[0] == 1.015625


def test_rmsnorm_matches_torch():
    x = rng.standard_normal((7, 48))
    g = rng.standard_normal(48)
    ref = F.rms_norm(torch.tensor(x), (48,), torch.tensor(g), eps=1e-5).numpy()
    assert np.allclose(so.rmsnorm(x, g, 1e-5), ref, rtol=1e-12, atol=1e-12)
    # closed form: a constant row c has rms |c| -> output sign(c)*gain (eps -> 0)
    out = so.rmsnorm(np.full((1, 8), -3.0), np.arange(8.0), 0.0)
    assert np.allclose(out, -np.arange(8.0))


def test_silu_matches_torch_and_closed_form():
    x = rng.standard_normal(100) * 4
    assert np.allclose(so.silu(x), F.silu(torch.tensor(x)).numpy(), rtol=1e-12, atol=1e-14)
    assert so.silu(np.array([0.0]))[0] == 0.0
    assert np.isclose(so.silu(np.array([1.0]))[0], 1.0 / (1.0 + np.exp(-1.0)))


def test_rope_is_complex_rotation():
    T, H, hd, theta = 5, 3, 16, 10000.0
    x = rng.standard_normal((T, H, hd))
    pos = np.array([0, 1, 7, 100, 4095])
    got = so.rope(x, pos, theta)
    half = hd // 2
    z = x[..., :half] + 1j * x[..., half:]
    freq = theta ** (-np.arange(half) / half)
    zr = z * np.exp(1j * pos[:, None, None] * freq[None, None, :])
    assert np.allclose(got[..., :half], zr.real, atol=1e-12)
    assert np.allclose(got[..., half:], zr.imag, atol=1e-12)
    # position 0 is the identity; norms are preserved
    assert np.allclose(got[0], x[0])
    assert np.allclose(np.linalg.norm(got, axis=-1), np.linalg.norm(x, axis=-1))


def test_rope_scores_depend_on_relative_position_only():
    H, hd, theta = 2, 32, 500000.0
    q = rng.standard_normal((4, H, hd))
    k = rng.standard_normal((4, H, hd))
    pq, pk = np.array([3, 9, 20, 21]), np.array([0, 5, 17, 30])
    s0 = np.einsum("thd,shd->hts", so.rope(q, pq, theta), so.rope(k, pk, theta))
    s1 = np.einsum("thd,shd->hts", so.rope(q, pq + 777, theta), so.rope(k, pk + 777, theta))
    assert np.allclose(s0, s1, atol=1e-9)


@pytest.mark.parametrize("H,Hkv", [(4, 4), (6, 2)])
def test_attention_matches_torch_sdpa(H, Hkv):
    T, S, hd = 5, 11, 16
    q = rng.standard_normal((T, H, hd))
    k = rng.standard_normal((S, Hkv, hd))
    v = rng.standard_normal((S, Hkv, hd))
    got = so.attention(q, k, v, lambda a: a)
    tq = torch.tensor(q).permute(1, 0, 2)[None]
    tk = torch.tensor(k).permute(1, 0, 2)[None]
    tv = torch.tensor(v).permute(1, 0, 2)[None]
    ref = F.scaled_dot_product_attention(tq, tk, tv, enable_gqa=True)[0].permute(1, 0, 2).reshape(T, H * hd).numpy()
    assert np.allclose(got, ref, atol=1e-12)


def test_attention_single_key_returns_value():
    q = rng.standard_normal((3, 2, 8))
    k = rng.standard_normal((1, 2, 8))
    v = rng.standard_normal((1, 2, 8))
    out = so.attention(q, k, v, lambda a: a).reshape(3, 2, 8)
    assert np.allclose(out, np.broadcast_to(v, (3, 2, 8)))


def test_token_and_confidence():
    import scipy.special
    logits = rng.standard_normal((9, 40)) * 3
    mask_id = 39
    logits[2, mask_id] = 100.0                 # the mask token may never win
    logits[4, 7] = logits[4, 21] = 50.0        # tie -> lower id
    tok, conf = so.token_and_confidence(logits, mask_id)
    p = scipy.special.softmax(logits[:, :mask_id], axis=-1)
    assert np.array_equal(tok, p.argmax(-1))
    assert np.allclose(conf, p.max(-1), rtol=1e-12)
    assert tok[4] == 7 and tok[2] != mask_id
    gap = so.top2_gap(logits, mask_id)
    srt = np.sort(p, axis=-1)
    assert np.allclose(gap, srt[:, -1] - srt[:, -2], atol=1e-14)
    assert gap[4] == 0.0


def test_block_ranges_eq3():
    assert so.block_ranges(64, 16) == [(0, 16), (16, 32), (32, 48), (48, 64)]
    assert so.block_ranges(10, 4) == [(0, 4), (4, 8), (8, 10)]        # ragged tail via min()
    assert so.block_ranges(3, 8) == [(0, 3)]


# ---- the whole forward, rebuilt from torch library calls ---------------------------------
def _torch_forward(w: wl.Workload, W: dict, tokens, allow):
    """Full-sequence forward with an explicit attention mask, built from torch.nn.functional."""
    t = {k: torch.tensor(v) for k, v in W.items()}
    T = len(tokens)
    h = F.embedding(torch.tensor(tokens, dtype=torch.long), t["embed"])
    half = w.head_dim // 2
    freq = w.rope_theta ** (-torch.arange(half, dtype=torch.float64) / half)
    rot = torch.polar(torch.ones(T, half, dtype=torch.float64), torch.arange(T, dtype=torch.float64)[:, None] * freq)

    def rope(x):  # [T, H, hd]
        z = torch.complex(x[..., :half], x[..., half:]) * rot[:, None, :]
        return torch.cat([z.real, z.imag], dim=-1)

    for l in range(w.n_layers):
        p = f"layers.{l}."
        u = F.rms_norm(h, (w.d_model,), t[p + "norm_attn"], eps=w.rms_eps)
        q = rope(F.linear(u, t[p + "wq"]).view(T, w.n_heads, w.head_dim)).permute(1, 0, 2)[None]
        k = rope(F.linear(u, t[p + "wk"]).view(T, w.n_kv_heads, w.head_dim)).permute(1, 0, 2)[None]
        v = F.linear(u, t[p + "wv"]).view(T, w.n_kv_heads, w.head_dim).permute(1, 0, 2)[None]
        a = F.scaled_dot_product_attention(q, k, v, attn_mask=torch.tensor(allow), enable_gqa=True)
        h = h + F.linear(a[0].permute(1, 0, 2).reshape(T, -1), t[p + "wo"])
        u = F.rms_norm(h, (w.d_model,), t[p + "norm_ffn"], eps=w.rms_eps)
        h = h + F.linear(F.silu(F.linear(u, t[p + "w_gate"])) * F.linear(u, t[p + "w_up"]), t[p + "w_down"])
    return F.linear(F.rms_norm(h, (w.d_model,), t["norm_final"], eps=w.rms_eps), t["lm_head"]).numpy()


@pytest.mark.parametrize("w", [SMALL, SMALL_GQA], ids=lambda w: w.name)
def test_cached_forward_equals_torch_block_causal(w):
    """Prefill + two committed blocks + one verification forward of 3 nodes, against a single
    masked full-sequence forward assembled from torch library routines."""
    W = oracle_weights(w, as_bf16=False)
    o = so.Oracle(oracle_config(w), W)
    prompt = wl.make_prompts(w)[0].numpy()
    B = w.block_len
    blocks = [rng.integers(0, w.vocab - 1, B) for _ in range(2)]
    cache = o.prefill(prompt)
    for b in blocks:
        o.commit_block(b, cache)
    nodes = np.stack([np.where(rng.random(B) < 0.5, w.mask_id, rng.integers(0, w.vocab - 1, B)) for _ in range(3)])
    logits, _, _ = o.forward_rows(nodes, cache.length, cache)
    for i in range(3):
        seq = np.concatenate([prompt] + blocks + [nodes[i]])
        seg = np.repeat(np.arange(4), [len(prompt), B, B, B])
        allow = seg[None, :] <= seg[:, None]
        ref = _torch_forward(w, W, seq, allow)
        assert np.allclose(logits[i], ref[-B:], atol=1e-9), np.abs(logits[i] - ref[-B:]).max()


def test_cache_equals_uncached_recompute():
    """Cache semantics: K/V held in the cache and the logits of a cached forward equal those of
    an uncached block-causal forward over the truncated sequence."""
    w = SMALL
    o = make_oracle(w)
    prompt = wl.make_prompts(w)[0].numpy()
    B = w.block_len
    b0 = rng.integers(0, w.vocab - 1, B)
    b1 = np.where(rng.random(B) < 0.6, w.mask_id, rng.integers(0, w.vocab - 1, B))
    cache = o.prefill(prompt)
    o.commit_block(b0, cache)
    logits, ks, vs = o.forward_rows(b1, cache.length, cache)
    ref_logits, rK, rV = o.uncached_block_causal(np.concatenate([prompt, b0, b1]), [len(prompt), B, B])
    assert np.allclose(logits[0], ref_logits[-B:], atol=1e-5)
    for l in range(w.n_layers):
        assert np.allclose(cache.k[l], rK[l][:len(prompt) + B], atol=1e-5)
        assert np.allclose(cache.v[l], rV[l][:len(prompt) + B], atol=1e-5)
        assert np.allclose(ks[l][0], rK[l][-B:], atol=1e-5)


def test_later_blocks_are_invisible():
    """A block forward sees the prefix and itself only: logits do not change when tokens that
    would come after the block are appended to the uncached sequence as a later segment."""
    w = SMALL
    o = make_oracle(w)
    prompt = wl.make_prompts(w)[0].numpy()
    B = w.block_len
    b0 = rng.integers(0, w.vocab - 1, B)
    later = rng.integers(0, w.vocab - 1, B)
    l0, _, _ = o.uncached_block_causal(np.concatenate([prompt, b0]), [len(prompt), B])
    l1, _, _ = o.uncached_block_causal(np.concatenate([prompt, b0, later]), [len(prompt), B, B])
    assert np.allclose(l0, l1[:len(prompt) + B], atol=1e-12)


def test_operand_rounding_is_small_and_nonzero():
    w = SMALL
    W = oracle_weights(w, as_bf16=True)
    prompt = wl.make_prompts(w)[0].numpy()
    a = so.Oracle(oracle_config(w), W)
    b = so.Oracle(oracle_config(w), W, operand_rounding="bf16")
    la, _, _ = a.forward_rows(np.full(w.block_len, w.mask_id), len(prompt), a.prefill(prompt))
    lb, _, _ = b.forward_rows(np.full(w.block_len, w.mask_id), len(prompt), b.prefill(prompt))
    d = np.abs(la - lb).max()
    assert 0 < d < 2e-2


def test_rounding_sources_partition_the_bf16_mode():
    """Selective operand rounding only switches existing rounding points on and off: every source on is
    the "bf16" mode bit for bit, none on is the unrounded mode bit for bit, and a single source moves the
    logits by less than all of them together."""
    w = SMALL_GQA
    cfg, wts = oracle_config(w), oracle_weights(w, as_bf16=True)
    prompt = wl.make_prompts(w).numpy()[0]
    ids = np.array([[w.mask_id, 3, w.mask_id, 7, 9, w.mask_id]])

    def logits_of(mode):
        o = so.Oracle(cfg, wts, mode)
        return o.forward_rows(ids, len(prompt), o.prefill(prompt))[0]

    plain, full = logits_of(None), logits_of("bf16")
    assert np.array_equal(logits_of(()), plain)
    assert np.array_equal(logits_of(so.ROUNDING_SOURCES), full)
    total = np.abs(full - plain).max()
    assert total > 0
    for src in so.ROUNDING_SOURCES:
        one = np.abs(logits_of((src,)) - plain).max()
        assert 0 < one < 2 * total
    with pytest.raises(AssertionError):
        so.Oracle(cfg, wts, ("nonsense",))


def test_hidden_trace_is_the_residual_stream():
    """The recorded residual stream has one entry per layer boundary, starts at the embedding rows, ends
    at what the LM head normalises, and is the same through the cached and the uncached forward."""
    w = SMALL
    o = make_oracle(w)
    prompt = wl.make_prompts(w).numpy()[0]
    ids = np.array([5, w.mask_id, 8, w.mask_id, w.mask_id, 2])
    tr = []
    logits, _, _ = o.forward_rows(ids[None], len(prompt), o.prefill(prompt), hidden_trace=tr)
    assert len(tr) == w.n_layers + 1 and tr[0].shape == (1, len(ids), w.d_model)
    assert np.array_equal(tr[0][0], o._W("embed")[ids])
    assert np.allclose(so.rmsnorm(tr[-1][0], o._W("norm_final"), w.rms_eps) @ o._W("lm_head").T, logits[0],
                       rtol=1e-12, atol=1e-14)
    tr2 = []
    o.uncached_block_causal(np.concatenate([prompt, ids]), [len(prompt), len(ids)], hidden_trace=tr2)
    assert len(tr2) == w.n_layers + 1
    for a, b in zip(tr, tr2):
        assert np.allclose(a[0], b[len(prompt):], rtol=1e-9, atol=1e-12)


def test_lockstep_driver_equals_prefill_then_forward():
    """The layer-by-layer driver used for large models (several rounding modes through one pass over the
    weights) is the oracle's prefill followed by forward_rows, bit for bit."""
    from tests.helpers import lockstep_root_forward
    w = SMALL_GQA
    wts = oracle_weights(w, as_bf16=True)
    prompt = wl.make_prompts(w).numpy()[0]
    ids = np.array([w.mask_id, 3, w.mask_id, 7, 9, w.mask_id])
    got = lockstep_root_forward(w, wts, prompt, ids, (None, "bf16"))
    for mode in (None, "bf16"):
        o = so.Oracle(oracle_config(w), wts, mode)
        cache = o.prefill(prompt)
        tr = []
        logits, _, _ = o.forward_rows(ids[None], len(prompt), cache, hidden_trace=tr)
        assert np.array_equal(got[mode]["logits"], logits[0])
        for l in range(w.n_layers):
            assert np.array_equal(got[mode]["prefix_k"][l], cache.k[l])
            assert np.array_equal(got[mode]["prefix_v"][l], cache.v[l])
        for a, b in zip(got[mode]["hidden"], tr):
            assert np.array_equal(a, b[0])
