"""CUDA path vs the CPU oracle, through the C ABI (run with -m gpu on a B200).

Tolerances (bf16 operands, fp32 accumulation; the stated parity bar):
  * logits within 2e-2 absolute of the fp64 oracle, confidences within 2e-2 relative;
  * against the oracle run with bf16 operand rounding (same arithmetic type as the kernels) the
    logits agree to 1e-2, half the stated tolerance.  That comparison is not bit-level: the kernels
    round the attention probabilities relative to a part's running maximum and merge parts, the
    oracle rounds them relative to the row maximum, and fp32 accumulation (whose order follows the
    split-K factors) flips a few bf16 roundings of the activations.  What is left is bf16 rounding
    noise whose maximum over the 1.6e5 logits of a case sits between 4e-3 and 7e-3;
  * tokens / accept lengths bit-exact wherever the oracle's decision gap exceeds 1e-3;
  * GPU SSD == GPU stepwise bit-exact, no exemption.
"""

import numpy as np
import pytest
import torch

from oracle import ssd_oracle as so
from paper_2510_04147_b200 import workloads as wl
from tests.helpers import make_oracle, oracle_config, oracle_weights

pytestmark = pytest.mark.gpu

GAP = 1e-3
CONF_RTOL = 2e-2     # a logit error e moves a softmax probability by a factor within exp(+-2e)
DEFAULT_TWO_SM = 256         # the library's default for "two_sm_rows"
PEAKED = wl.TINY.replace(name="tiny_peaked", lm_head_scale=8.0)


def _token_is_safe(gap, conf, w):
    """The oracle's top-1/top-2 probability gap exceeds 1e-3 and (for the scaled variant, whose logit
    errors scale too) also exceeds twice the relative confidence tolerance."""
    return (gap > GAP) & (gap > 2 * CONF_RTOL * w.lm_head_scale * conf * (w.lm_head_scale > 1))


def _binding():
    from paper_2510_04147_b200 import binding
    return binding


def _make_ssd(w, max_drafts, max_batch=None, max_seq=None):
    b = _binding()
    ssd = b.Ssd(b.config_from_workload(w, max_drafts=max_drafts, max_batch=max_batch, max_seq=max_seq))
    ssd.load_workload_weights(w)
    return ssd


@pytest.fixture(scope="module")
def tiny_ssd():
    ssd = _make_ssd(wl.TINY, max_drafts=wl.TINY.block_len, max_batch=3)
    yield ssd
    ssd.destroy()


@pytest.fixture(scope="module")
def peaked_ssd():
    ssd = _make_ssd(PEAKED, max_drafts=PEAKED.block_len, max_batch=3)
    yield ssd
    ssd.destroy()


@pytest.fixture(scope="module")
def tiny_oracles():
    """(fp64 oracle, bf16-operand oracle) on the bf16-rounded weights of config 1."""
    return {w.name: (make_oracle(w, as_bf16=True), make_oracle(w, as_bf16=True, operand_rounding="bf16"))
            for w in (wl.TINY, PEAKED)}


# ------------------------------------------------------------------------------------------
# the projection kernel alone
# ------------------------------------------------------------------------------------------
@pytest.mark.parametrize("rows,n,k,split", [(16, 128, 64, 1), (32, 256, 256, 1), (100, 688, 688, 1), (37, 1376, 256, 1),
                                            (128, 4096, 4096, 4), (64, 512, 12288, 8), (300, 384, 512, 2),
                                            (256, 256, 1024, 3), (1, 130, 72, 1)])
def test_gemm_against_numpy(tiny_ssd, rows, n, k, split):
    x = wl.normal_tensor(5, 1, (rows, k), 1.0, device="cuda", dtype=torch.bfloat16)
    w = wl.normal_tensor(5, 2, (n, k), 0.05, device="cuda", dtype=torch.bfloat16)
    out = tiny_ssd.gemm_bf16(x, w, split).cpu().numpy()
    ref = x.cpu().to(torch.float64).numpy() @ w.cpu().to(torch.float64).numpy().T
    scale = np.sqrt(k) * 0.05
    assert np.abs(out - ref).max() < 2e-5 * scale * np.sqrt(k) + 1e-6, np.abs(out - ref).max()


@pytest.mark.parametrize("rows,n,k,split", [(16, 256, 64, 1), (32, 256, 256, 1), (100, 768, 704, 1), (48, 1280, 256, 1),
                                            (128, 4096, 4096, 4), (64, 512, 12288, 8), (300, 512, 512, 2),
                                            (256, 256, 1024, 3), (1, 256, 72, 1)])
def test_gemm_two_sm_pairs_change_no_bit(tiny_ssd, rows, n, k, split):
    """Pairs of weight tiles as one cta_group::2 MMA (each CTA of the pair holds its own weight tile and
    half of the activation tile; the even CTA issues, both read their own accumulator): the same products
    summed in the same order, so the result is bit-identical to the single-CTA launch."""
    x = wl.normal_tensor(6, 1, (rows, k), 1.0, device="cuda", dtype=torch.bfloat16)
    w = wl.normal_tensor(6, 2, (n, k), 0.05, device="cuda", dtype=torch.bfloat16)
    try:
        tiny_ssd.set_option("two_sm_rows", 0)
        plain = tiny_ssd.gemm_bf16(x, w, split).cpu().numpy()
        tiny_ssd.set_option("two_sm_rows", 16)
        paired = tiny_ssd.gemm_bf16(x, w, split).cpu().numpy()
    finally:
        tiny_ssd.set_option("two_sm_rows", DEFAULT_TWO_SM)
    assert np.array_equal(plain, paired)
    ref = x.cpu().to(torch.float64).numpy() @ w.cpu().to(torch.float64).numpy().T
    assert np.abs(paired - ref).max() < 2e-5 * 0.05 * k + 1e-6


# ------------------------------------------------------------------------------------------
# cache and forward
# ------------------------------------------------------------------------------------------
def test_prefill_cache_matches_oracle(tiny_ssd, tiny_oracles):
    w = wl.TINY
    _, ob = tiny_oracles[w.name]
    prompts = wl.make_prompts(w, batch=2).numpy()
    tiny_ssd.prefill(prompts)
    assert tiny_ssd.cache_length() == w.prompt_len
    for b in range(2):
        cache = ob.prefill(prompts[b])
        for l in range(w.n_layers):
            k, v = tiny_ssd.read_cache(l, b, w.prompt_len)
            assert np.abs(k - cache.k[l]).max() < 2e-2 * max(1.0, np.abs(cache.k[l]).max())
            assert np.abs(v - cache.v[l]).max() < 2e-2 * max(1.0, np.abs(cache.v[l]).max())
            # Entry by entry the cache stays at bf16 rounding noise of the bf16-operand oracle (entries
            # are O(0.3), one bf16 step there is 2e-3).  It is not bit-identical: the kernels apply
            # RMSNorm after the contraction, inv_rms * ((h * g) . W^T), the oracle before it, so the
            # two round different operands.
            assert (np.abs(k - cache.k[l]) <= 4e-3).mean() > 0.99


def test_prompts_prefilled_together_fill_the_cache_as_each_alone(peaked_ssd):
    """The prompts of a batch share one prefill forward (one stream of the weights); a row's arithmetic does not
    depend on what shares the forward with it, so every sequence's cache is, bit for bit, what prefilling it alone gives."""
    w = PEAKED
    prompts = wl.make_prompts(w, batch=3).numpy()
    peaked_ssd.prefill(prompts)
    together = [[peaked_ssd.read_cache(l, s, w.prompt_len) for l in range(w.n_layers)] for s in range(3)]
    for s in range(3):
        peaked_ssd.prefill(prompts[s:s + 1])
        for l in range(w.n_layers):
            k, v = peaked_ssd.read_cache(l, 0, w.prompt_len)
            assert np.array_equal(k, together[s][l][0]) and np.array_equal(v, together[s][l][1])


def _random_nodes(w, rng, n_nodes, T):
    ids = rng.integers(0, w.vocab - 1, (1, n_nodes, T))
    masked = rng.random((1, n_nodes, T)) < 0.6
    masked[:, :, 0] = True
    return np.where(masked, w.mask_id, ids), masked


@pytest.mark.parametrize("which", ["tiny", "tiny_peaked"])
def test_verify_forward_logits_and_stats(tiny_ssd, peaked_ssd, tiny_oracles, which):
    w = wl.TINY if which == "tiny" else PEAKED
    ssd = tiny_ssd if which == "tiny" else peaked_ssd
    o64, ob = tiny_oracles[w.name]
    rng = np.random.default_rng(3)
    prompt = wl.make_prompts(w).numpy()
    T = w.block_len
    ssd.prefill(prompt)
    # one committed block so that the prefix is prompt + block
    blk = rng.integers(0, w.vocab - 1, (1, T))
    ssd.block_begin(T)
    ssd.set_block_state(blk, np.zeros((1, T), np.uint8))
    ssd.block_commit()
    ids, masked = _random_nodes(w, rng, 5, T)
    tok, conf, logits = ssd.verify_forward(ids, masked, want_logits=True)
    tok2, conf2, _ = ssd.verify_forward(ids, masked, want_logits=False)      # fused LM head path
    for o, tol in ((ob, 1e-2), (o64, 2e-2)):
        cache = o.prefill(prompt[0])
        o.commit_block(blk[0], cache)
        otok, oconf, ogap, ologits = o.verify(ids[0], masked[0], cache)
        err = np.abs(logits[0] - ologits).max()
        assert err < tol * w.lm_head_scale, (err, tol)
        m = masked[0]
        assert np.allclose(conf[0][m], oconf[m], rtol=CONF_RTOL * w.lm_head_scale, atol=1e-6)
        assert np.allclose(conf2[0][m], oconf[m], rtol=CONF_RTOL * w.lm_head_scale, atol=1e-6)
        sure = m & _token_is_safe(ogap, oconf, w)
        assert np.array_equal(tok[0][sure], otok[sure])
        assert np.array_equal(tok2[0][sure], otok[sure])
        if which == "tiny_peaked":
            assert sure.sum() > 0.25 * m.sum()         # the peaked variant makes the token check bite
    # rows that were not asked for
    assert np.all(tok[0][~masked[0]] == -1) and np.all(conf[0][~masked[0]] == 0)
    # the two LM-head paths agree (same logits, different reduction order)
    assert np.array_equal(tok[0][masked[0]], tok2[0][masked[0]])
    assert np.allclose(conf[0], conf2[0], rtol=1e-4)
    assert w.mask_id not in tok


def test_row_invariance_of_the_forward(peaked_ssd):
    """A node's outputs are bit-identical whether it runs alone or among other nodes."""
    w = PEAKED
    rng = np.random.default_rng(4)
    prompt = wl.make_prompts(w).numpy()
    peaked_ssd.prefill(prompt)
    T = w.block_len
    ids, masked = _random_nodes(w, rng, 7, T)
    tok, conf, _ = peaked_ssd.verify_forward(ids, masked)
    for i in (0, 3, 6):
        t1, c1, _ = peaked_ssd.verify_forward(ids[:, i:i + 1], masked[:, i:i + 1])
        assert np.array_equal(t1[0, 0], tok[0, i])
        assert np.array_equal(c1[0, 0].view(np.uint32), conf[0, i].view(np.uint32))


# ------------------------------------------------------------------------------------------
# decode loops
# ------------------------------------------------------------------------------------------
@pytest.mark.parametrize("which", ["tiny", "tiny_peaked"])
@pytest.mark.parametrize("max_drafts", [0, 1, 3, 5, 16])
def test_gpu_ssd_equals_gpu_stepwise(tiny_ssd, peaked_ssd, which, max_drafts):
    w = wl.TINY if which == "tiny" else PEAKED
    ssd = tiny_ssd if which == "tiny" else peaked_ssd
    b = _binding()
    prompt = wl.make_prompts(w).numpy()
    ssd.prefill(prompt)
    want, acc0, nf0 = ssd.generate(b.MODE_STEPWISE, w.gen_len, w.block_len, 1)
    ssd.prefill(prompt)
    toks = []
    for j in range(w.gen_len // w.block_len):
        ssd.block_begin(w.block_len)
        counts = []
        while True:
            acc, nn = ssd.block_step(max_drafts, 1)
            if acc[0] == 0:
                break
            assert 1 <= acc[0] <= nn[0] <= max_drafts + 1
            counts.append(int(acc[0]))
        assert sum(counts) == w.block_len
        ids, masked, _, _ = ssd.get_block_state(1, w.block_len)
        assert masked.sum() == 0
        toks.append(ids)
        ssd.block_commit()
        if max_drafts == 0:
            assert counts == [1] * w.block_len
    got = np.concatenate(toks, axis=1)
    assert np.array_equal(got, want)
    assert all(int(n[0]) == w.block_len for n in nf0) and all(np.all(a == 1) for a in acc0)
    assert w.mask_id not in got
    assert ssd.cache_length() == w.prompt_len + w.gen_len


def test_decode_block_postconditions(peaked_ssd):
    w = PEAKED
    b = _binding()
    prompt = wl.make_prompts(w).numpy()
    peaked_ssd.prefill(prompt)
    tok, accs, nfs = peaked_ssd.generate(b.MODE_SSD, w.gen_len, w.block_len, 1)
    for acc, nf in zip(accs, nfs):
        n = int(nf[0])
        assert acc[0, :n].sum() == w.block_len and np.all(acc[0, :n] >= 1) and np.all(acc[0, n:] == 0)
        assert acc[0, 0] == 1                      # first forward of a block has no drafts


@pytest.mark.parametrize("which", ["tiny", "tiny_peaked"])
def test_teacher_forced_ssd_steps_match_oracle(tiny_ssd, peaked_ssd, tiny_oracles, which):
    """Every verification forward of the oracle's SSD run is replayed on the GPU from the oracle's
    state and drafts.  Two layers of parity:
      numeric  - the forward's (token, confidence) per masked row against the oracle's, within tolerance,
                 tokens equal wherever the oracle's top-1/top-2 gap is safe;
      integer  - candidate selection, chain walk, accepted length, state and draft update bit-exact
                 against the oracle's logic applied to the forward's own outputs (no exemption), and
                 equal to the oracle's accepted length wherever all its decisions have a safe margin."""
    w = wl.TINY if which == "tiny" else PEAKED
    ssd = tiny_ssd if which == "tiny" else peaked_ssd
    _, ob = tiny_oracles[w.name]
    prompt = wl.make_prompts(w).numpy()
    trace = []
    N = 5
    tokens, _, _ = ob.generate(prompt[0], w.gen_len, w.block_len, mode="ssd", max_drafts=N, trace=trace)
    ssd.prefill(prompt)
    T = w.block_len
    strict = 0
    cur_block = 0
    rtol = CONF_RTOL * w.lm_head_scale
    for rec in trace:
        if rec.block != cur_block:                 # commit the oracle's finished block
            ssd.block_begin(T)
            ssd.set_block_state(tokens[cur_block * T:(cur_block + 1) * T][None], np.zeros((1, T), np.uint8))
            ssd.block_commit()
            cur_block = rec.block
        # ---- numeric layer
        tok_g, conf_g, _ = ssd.verify_forward(rec.node_ids[None], rec.node_masked[None])
        tok_g, conf_g = tok_g[0], conf_g[0]
        m = rec.node_masked
        assert np.allclose(conf_g[m], rec.conf[m], rtol=rtol, atol=1e-6)
        sure = m & _token_is_safe(rec.gap, rec.conf, w)
        assert np.array_equal(tok_g[sure], rec.tok[sure])
        # ---- integer layer
        ssd.block_begin(T)
        if rec.draft_tok is None:
            ssd.set_block_state(rec.ids_before[None], rec.masked_before[None].astype(np.uint8))
            cand = []
        else:
            dconf32 = rec.draft_conf.astype(np.float32)
            ssd.set_block_state(rec.ids_before[None], rec.masked_before[None].astype(np.uint8),
                                rec.draft_tok[None], dconf32[None])
            cand = so.select_candidates(rec.draft_tok, dconf32, rec.masked_before, N)
        acc, nn = ssd.block_step(N, 1)
        assert nn[0] == len(cand) + 1 == len(rec.cand) + 1
        ids, masked, dt, dc = ssd.get_block_state(1, T)
        if cand == rec.cand:
            pred = so.node_predictions(tok_g, conf_g, rec.node_masked)
            a = so.accept_length(pred, cand)
            assert acc[0] == a + 1
            want_ids, want_masked = rec.ids_before.copy(), rec.masked_before.copy()
            for (p, t) in cand[:a]:
                want_ids[p], want_masked[p] = t, False
            q, t = pred[a]
            want_ids[q], want_masked[q] = t, False
            assert np.array_equal(masked[0].astype(bool), want_masked)
            assert np.array_equal(ids[0][~want_masked], want_ids[~want_masked])
            assert np.array_equal(dt[0][want_masked], tok_g[a][want_masked])
            assert np.array_equal(dc[0][want_masked].view(np.uint32), conf_g[a][want_masked].view(np.uint32))
            assert np.all(dt[0][~want_masked] == 0) and np.all(dc[0][~want_masked] == 0)
            # against the oracle's own accepted length, where its decisions are safe
            safe = True
            for i in range(rec.accepted):
                qi, _ = rec.pred[i]
                cm = np.sort(np.where(rec.node_masked[i], rec.conf[i], -1.0))[::-1]
                second = cm[1] if len(cm) > 1 and cm[1] >= 0 else -np.inf
                pos_margin = cm[0] - second
                safe = safe and bool(_token_is_safe(rec.gap[i, qi], rec.conf[i, qi], w))
                safe = safe and pos_margin > GAP and pos_margin > 2 * rtol * cm[0]
            if safe:
                strict += 1
                assert acc[0] == rec.accepted
        else:
            assert 1 <= acc[0] <= nn[0]
    print(f"{which}: {strict} of {len(trace)} forwards had safe margins throughout")


@pytest.mark.parametrize("which", ["tiny", "tiny_peaked"])
def test_commit_folded_into_next_first_forward_matches_oracle(tiny_ssd, peaked_ssd, tiny_oracles, which):
    """A finished block is committed by the next block's first forward: per sequence one causal chain
    [finished block | next block, all MASK].  Mathematically that is the commit forward followed by the
    root forward, so the oracle needs nothing new: its commit_block + verify are the reference for the
    cache rows the chain writes and for the root predictions it returns."""
    w = wl.TINY if which == "tiny" else PEAKED
    ssd = tiny_ssd if which == "tiny" else peaked_ssd
    _, ob = tiny_oracles[w.name]
    b = _binding()
    prompt = wl.make_prompts(w).numpy()
    T, P = w.block_len, w.prompt_len
    rtol = CONF_RTOL * w.lm_head_scale
    block0 = np.random.default_rng(11).integers(0, w.vocab - 1, T)
    # oracle: commit, then the root forward of the next block
    cache = ob.prefill(prompt[0])
    ob.commit_block(block0, cache)
    root_ids = np.full((1, T), w.mask_id)
    otok, oconf, ogap, _ = ob.verify(root_ids, np.ones((1, T), bool), cache)
    otok, oconf, ogap = otok[0], oconf[0], ogap[0]
    # GPU: the commit waits, the next block's first step carries it
    ssd.prefill(prompt)
    ssd.block_begin(T)
    ssd.set_block_state(block0[None], np.zeros((1, T), np.uint8))
    ssd.block_commit()
    assert ssd.cache_length() == P + T
    l0 = ssd.launch_count()
    ssd.block_begin(T)
    acc, nn = ssd.block_step(0, 1)
    fused_launches = ssd.launch_count() - l0
    assert acc[0] == 1 and nn[0] == 1
    ids, masked, dt, dc = ssd.get_block_state(1, T)
    m = masked[0].astype(bool)
    assert m.sum() == T - 1
    q = int(np.where(~m)[0][0])
    assert np.allclose(dc[0][m], oconf[m], rtol=rtol, atol=1e-6)          # next drafts = root predictions
    sure = m & _token_is_safe(ogap, oconf, w)
    assert np.array_equal(dt[0][sure], otok[sure])
    order = np.sort(oconf)[::-1]
    if order[0] - order[1] > GAP and order[0] - order[1] > 2 * rtol * order[0] and _token_is_safe(ogap, oconf, w)[int(np.argmax(oconf))]:
        assert q == int(np.argmax(oconf)) and ids[0][q] == otok[q]
    # the rows the chain wrote into the cache
    for l in range(w.n_layers):
        k, v = ssd.read_cache(l, 0, P + T)
        for got, want in ((k, cache.k[l]), (v, cache.v[l])):
            assert np.abs(got[P:] - want[P:]).max() < 2e-2 * max(1.0, np.abs(want).max())
            assert (np.abs(got[P:] - want[P:]) <= 4e-3).mean() > 0.99
            assert np.abs(got[:P] - want[:P]).max() < 2e-2 * max(1.0, np.abs(want).max())
    # it really was one forward: a separate commit costs a second pass of the layers
    ssd.set_option("fuse_commit", 0)
    try:
        ssd.prefill(prompt)
        ssd.block_begin(T)
        ssd.set_block_state(block0[None], np.zeros((1, T), np.uint8))
        l1 = ssd.launch_count()
        ssd.block_commit()
        ssd.block_begin(T)
        acc2, _ = ssd.block_step(0, 1)
        split_launches = ssd.launch_count() - l1
        ids2, masked2, dt2, dc2 = ssd.get_block_state(1, T)
    finally:
        ssd.set_option("fuse_commit", 1)
    assert fused_launches < split_launches
    m2 = masked2[0].astype(bool)
    both = m & m2
    assert np.allclose(dc[0][both], dc2[0][both], rtol=rtol, atol=1e-6)    # the two forms agree within rounding


def test_generation_with_and_without_folded_commit(peaked_ssd):
    """Both commit forms decode whole generations losslessly (SSD == stepwise bit-exact within a form);
    the folded form skips the commit of the last block, which nothing reads."""
    w = PEAKED
    b = _binding()
    prompt = wl.make_prompts(w).numpy()
    out = {}
    try:
        for fuse in (1, 0):
            peaked_ssd.set_option("fuse_commit", fuse)
            peaked_ssd.prefill(prompt)
            tok_s, _, nf_s = peaked_ssd.generate(b.MODE_STEPWISE, w.gen_len, w.block_len, 1)
            assert peaked_ssd.cache_length() == w.prompt_len + w.gen_len
            peaked_ssd.prefill(prompt)
            l0 = peaked_ssd.launch_count()
            tok_d, acc_d, nf_d = peaked_ssd.generate(b.MODE_SSD, w.gen_len, w.block_len, 1)
            out[fuse] = (tok_d, peaked_ssd.launch_count() - l0)
            assert np.array_equal(tok_s, tok_d)
            for a, nf in zip(acc_d, nf_d):
                assert a[0][:nf[0]].sum() == w.block_len
    finally:
        peaked_ssd.set_option("fuse_commit", 1)
    assert out[1][1] < out[0][1]
    # rewinding into a block that still waits for its commit keeps its K/V
    peaked_ssd.prefill(prompt)
    peaked_ssd.decode_block(b.MODE_SSD, w.block_len, 1)
    peaked_ssd.rewind(w.prompt_len + w.block_len)
    assert peaked_ssd.cache_length() == w.prompt_len + w.block_len
    peaked_ssd.rewind(w.prompt_len)
    assert peaked_ssd.cache_length() == w.prompt_len


def test_batched_sequences_equal_single_runs(peaked_ssd):
    """Each sequence of a batch has its own tree; batching changes nothing for any of them."""
    w = PEAKED
    b = _binding()
    prompts = wl.make_prompts(w, batch=3).numpy()
    peaked_ssd.prefill(prompts)
    tok_b, acc_b, nf_b = peaked_ssd.generate(b.MODE_SSD, 32, w.block_len, 3)
    for s in range(3):
        peaked_ssd.prefill(prompts[s:s + 1])
        tok_s, acc_s, nf_s = peaked_ssd.generate(b.MODE_SSD, 32, w.block_len, 1)
        assert np.array_equal(tok_s[0], tok_b[s])
        for j in range(len(acc_s)):
            assert np.array_equal(acc_s[j][0], acc_b[j][s]) and nf_s[j][0] == nf_b[j][s]


def test_profile_modes_account_for_every_launch(tiny_ssd):
    """Mode 1 brackets every launch with events, mode 2 stamps the end of every launch in the live stream;
    both count the same launches per family, and decoding is unchanged while they run."""
    w = wl.TINY
    b = _binding()
    prompt = wl.make_prompts(w).numpy()
    tiny_ssd.prefill(prompt)
    ref, _, _ = tiny_ssd.decode_block(b.MODE_SSD, w.block_len, 1)
    counts = {}
    for mode in (1, 2):
        tiny_ssd.prefill(prompt)
        tiny_ssd.profile_enable(mode)
        try:
            tok, _, nf = tiny_ssd.decode_block(b.MODE_SSD, w.block_len, 1)
            prof = tiny_ssd.profile_read()
        finally:
            tiny_ssd.profile_enable(0)
        assert np.array_equal(tok, ref)
        assert prof["gemm"]["launches"] > 0 and prof["gemm"]["ms"] > 0 and prof["attn"]["ms"] > 0
        assert prof["gemm"]["launches"] == sum(prof[k]["launches"] for k in ("gemm_qkv", "gemm_o", "gemm_gu", "gemm_down"))
        counts[mode] = {k: v["launches"] for k, v in prof.items()}
    # mode 2 has no predecessor for its very first launch (a tree kernel)
    assert counts[1]["gemm"] == counts[2]["gemm"] and counts[1]["attn"] == counts[2]["attn"]
    assert counts[1]["tree"] == counts[2]["tree"] + 1


def test_ragged_last_block(tiny_ssd):
    w = wl.TINY
    b = _binding()
    prompt = wl.make_prompts(w).numpy()
    tiny_ssd.prefill(prompt)
    a, _, _ = tiny_ssd.generate(b.MODE_STEPWISE, 40, w.block_len, 1)
    tiny_ssd.prefill(prompt)
    c, accs, _ = tiny_ssd.generate(b.MODE_SSD, 40, w.block_len, 1)
    assert a.shape == (1, 40) and np.array_equal(a, c)
    assert [int(x.sum()) for x in accs] == [16, 16, 8]
    assert tiny_ssd.cache_length() == w.prompt_len + 40


def test_blocks_of_one_and_two_tokens(peaked_ssd):
    """B = 1: no draft can exist, every forward is a stepwise step; B = 2: at most one draft (N = min(max_drafts, r - 1))."""
    w = PEAKED
    b = _binding()
    prompt = wl.make_prompts(w).numpy()
    for block in (1, 2):
        peaked_ssd.prefill(prompt)
        want, _, nf0 = peaked_ssd.generate(b.MODE_STEPWISE, 6, block, 1)
        peaked_ssd.prefill(prompt)
        got, accs, nf = peaked_ssd.generate(b.MODE_SSD, 6, block, 1)
        assert np.array_equal(got, want) and w.mask_id not in got
        assert all(int(a.sum()) == block for a in accs)
        if block == 1:
            assert all(int(n[0]) == 1 for n in nf)
        else:
            assert all(1 <= int(n[0]) <= 2 for n in nf)
        assert peaked_ssd.cache_length() == w.prompt_len + 6


def test_prompt_of_one_token(tiny_ssd, tiny_oracles):
    """The shortest prefix: one cached key.  Cache and root predictions against the oracle, SSD == stepwise."""
    w = wl.TINY
    _, ob = tiny_oracles[w.name]
    b = _binding()
    prompt = wl.make_prompts(w).numpy()[:, :1]
    tiny_ssd.prefill(prompt)
    assert tiny_ssd.cache_length() == 1
    cache = ob.prefill(prompt[0])
    for l in range(w.n_layers):
        k, v = tiny_ssd.read_cache(l, 0, 1)
        assert np.abs(k - cache.k[l]).max() < 2e-2 * max(1.0, np.abs(cache.k[l]).max())
        assert np.abs(v - cache.v[l]).max() < 2e-2 * max(1.0, np.abs(cache.v[l]).max())
    ids = np.full((1, 1, w.block_len), w.mask_id)
    masked = np.ones((1, 1, w.block_len), dtype=bool)
    tok, conf, logits = tiny_ssd.verify_forward(ids, masked, want_logits=True)
    otok, oconf, ogap, ologits = ob.verify(ids[0], masked[0], cache)
    assert np.abs(logits[0] - ologits).max() < 1e-2
    assert np.allclose(conf[0], oconf, rtol=CONF_RTOL, atol=1e-6)
    want, _, _ = tiny_ssd.generate(b.MODE_STEPWISE, 2 * w.block_len, w.block_len, 1)
    tiny_ssd.prefill(prompt)
    got, _, _ = tiny_ssd.generate(b.MODE_SSD, 2 * w.block_len, w.block_len, 1)
    assert np.array_equal(got, want)


# ------------------------------------------------------------------------------------------
# error paths (host-side checks; nothing here faults a GPU)
# ------------------------------------------------------------------------------------------
def test_error_codes(tiny_ssd):
    b = _binding()
    w = wl.TINY
    fresh = b.Ssd(b.config_from_workload(w, max_drafts=2))
    with pytest.raises(b.SsdError) as e:
        fresh.prefill(wl.make_prompts(w).numpy())          # weights missing
    assert e.value.code == -7
    with pytest.raises(b.SsdError) as e:
        fresh.block_begin(4)                               # no prefill
    assert e.value.code == -7
    with pytest.raises(b.SsdError) as e:
        fresh.load_weights("layers.9.wq", torch.zeros(256, 256, device="cuda"))
    assert e.value.code == -1
    with pytest.raises(b.SsdError) as e:
        fresh.load_weights("embed", torch.zeros(5, 256, device="cuda"))
    assert e.value.code == -2
    with pytest.raises(b.SsdError) as e:
        fresh.set_option("nonsense", 1)
    assert e.value.code == -1
    fresh.destroy()
    prompt = wl.make_prompts(w).numpy()
    with pytest.raises(b.SsdError) as e:
        tiny_ssd.prefill(np.full((1, 8), w.vocab, np.int32))    # id outside the vocabulary
    assert e.value.code == -1
    with pytest.raises(b.SsdError) as e:
        tiny_ssd.prefill(np.zeros((9, 8), np.int32))            # batch > max_batch
    assert e.value.code == -5
    tiny_ssd.prefill(prompt)
    for _ in range(w.gen_len // w.block_len):
        tiny_ssd.decode_block(b.MODE_SSD, w.block_len, 1)
    with pytest.raises(b.SsdError) as e:
        tiny_ssd.decode_block(b.MODE_SSD, w.block_len, 1)       # cache full
    assert e.value.code == -5
    tiny_ssd.prefill(prompt)
    tiny_ssd.block_begin(w.block_len)
    with pytest.raises(b.SsdError) as e:
        tiny_ssd.block_commit()                                  # block not finished
    assert e.value.code == -7


def test_split_k_options_are_bounded_and_keep_parity(tiny_oracles):
    """A projection never gets more splits than it has 64-wide K blocks (an empty split would add an
    accumulator nothing wrote); within the bound every split count gives the same forward up to the
    rounding of another summation order."""
    w = wl.TINY
    b = _binding()
    o64, _ = tiny_oracles[w.name]
    rng = np.random.default_rng(9)
    prompt = wl.make_prompts(w).numpy()
    ids, masked = _random_nodes(w, rng, 3, w.block_len)
    ssd = _make_ssd(w, max_drafts=3)
    try:
        with pytest.raises(b.SsdError) as e:
            ssd.set_option("split_k_o", 8)                 # the O projection has 256 / 64 = 4 K blocks
        assert e.value.code == -1
        with pytest.raises(b.SsdError) as e:
            ssd.set_option("split_k_qkv", 5)
        assert e.value.code == -1
        ssd.prefill(prompt)
        _, _, base = ssd.verify_forward(ids, masked, want_logits=True)
        ssd.set_option("split_k_o", 4)                     # one K block per split
        ssd.set_option("split_k_down", 8)                  # 11 K blocks over 8 splits: ragged
        ssd.set_option("split_k_qkv", 4)
        ssd.prefill(prompt)
        _, _, split = ssd.verify_forward(ids, masked, want_logits=True)
    finally:
        ssd.destroy()
    cache = o64.prefill(prompt[0])
    _, _, _, ologits = o64.verify(ids[0], masked[0], cache)
    assert np.abs(split[0] - ologits).max() < 2e-2
    assert np.abs(base[0] - ologits).max() < 2e-2
    assert np.abs(split - base).max() < 1e-2


def test_nonfinite_weights_are_reported_not_decoded():
    """A NaN in a weight (injected on the host side, nothing faults) makes every confidence NaN: the step
    returns SSD_ERR_NONFINITE instead of tokens, and the context stays usable."""
    w = wl.TINY
    b = _binding()
    prompt = wl.make_prompts(w).numpy()
    ssd = _make_ssd(w, max_drafts=2)
    try:
        good = wl.make_tensor(w, "norm_final", "cuda")
        bad = good.clone()
        bad[7] = float("nan")
        ssd.load_weights("norm_final", bad)
        ssd.prefill(prompt)
        ssd.block_begin(w.block_len)
        with pytest.raises(b.SsdError) as e:
            ssd.block_step(2, 1)
        assert e.value.code == -8
        ssd.prefill(prompt)
        with pytest.raises(b.SsdError) as e:
            ssd.decode_block(b.MODE_SSD, w.block_len, 1)
        assert e.value.code == -8
        # with the weight repaired the same context decodes again
        ssd.load_weights("norm_final", good)
        ssd.prefill(prompt)
        tok, acc, nf = ssd.decode_block(b.MODE_SSD, w.block_len, 1)
        assert acc[0][:nf[0]].sum() == w.block_len and w.mask_id not in tok
    finally:
        ssd.destroy()


# ------------------------------------------------------------------------------------------
# mix-order tree (Section 5.2)
# ------------------------------------------------------------------------------------------
@pytest.mark.parametrize("which", ["tiny", "tiny_peaked"])
def test_mix_order_steps_match_oracle(tiny_ssd, peaked_ssd, tiny_oracles, which):
    """Every forward of the oracle's mix-order run replayed on the GPU from the oracle's state: the tree
    has the oracle's nodes (bit-exact rows, via the forward's outputs on them), and the walk - chain,
    out-of-order branch, state and draft update - equals the oracle's walk applied to the GPU forward's
    own (token, confidence) outputs, without exemption."""
    w = wl.TINY if which == "tiny" else PEAKED
    ssd = tiny_ssd if which == "tiny" else peaked_ssd
    _, ob = tiny_oracles[w.name]
    prompt = wl.make_prompts(w).numpy()
    trace = []
    N = 5
    tokens, _, _ = ob.generate(prompt[0], w.gen_len, w.block_len, mode="ssd", max_drafts=N, trace=trace, tree="mix_order")
    T = w.block_len
    rtol = CONF_RTOL * w.lm_head_scale
    branches = 0
    ssd.set_option("mix_order", 1)
    try:
        ssd.prefill(prompt)
        cur_block = 0
        for rec in trace:
            if rec.block != cur_block:
                ssd.block_begin(T)
                ssd.set_block_state(tokens[cur_block * T:(cur_block + 1) * T][None], np.zeros((1, T), np.uint8))
                ssd.block_commit()
                cur_block = rec.block
            tok_g, conf_g, _ = ssd.verify_forward(rec.node_ids[None], rec.node_masked[None])
            tok_g, conf_g = tok_g[0], conf_g[0]
            m = rec.node_masked
            assert np.allclose(conf_g[m], rec.conf[m], rtol=rtol, atol=1e-6)
            ssd.block_begin(T)
            if rec.draft_tok is None:
                ssd.set_block_state(rec.ids_before[None], rec.masked_before[None].astype(np.uint8))
                cand = []
            else:
                dconf32 = rec.draft_conf.astype(np.float32)
                ssd.set_block_state(rec.ids_before[None], rec.masked_before[None].astype(np.uint8),
                                    rec.draft_tok[None], dconf32[None])
                cand = so.select_candidates(rec.draft_tok, dconf32, rec.masked_before, N)
            acc, nn = ssd.block_step(N, 1)
            assert nn[0] == rec.node_ids.shape[0] == len(cand) + 1 + max(0, len(cand) - 1)
            ids, masked, dt, dc = ssd.get_block_state(1, T)
            if cand != rec.cand:
                continue
            pred = so.node_predictions(tok_g, conf_g, rec.node_masked)
            accepted, last = so.accept_walk_mix_order(pred, cand)
            branches += int(last > len(cand))
            assert acc[0] == len(accepted)
            want_ids, want_masked = rec.ids_before.copy(), rec.masked_before.copy()
            for (p, t) in accepted:
                want_ids[p], want_masked[p] = t, False
            assert np.array_equal(masked[0].astype(bool), want_masked)
            assert np.array_equal(ids[0][~want_masked], want_ids[~want_masked])
            assert np.array_equal(dt[0][want_masked], tok_g[last][want_masked])
            assert np.array_equal(dc[0][want_masked].view(np.uint32), conf_g[last][want_masked].view(np.uint32))
    finally:
        ssd.set_option("mix_order", 0)
    print(f"{which}: {branches} of {len(trace)} forwards ended in an out-of-order branch")


def test_mix_order_generation_is_lossless_on_the_device(peaked_ssd):
    """GPU mix-order SSD == GPU stepwise bit for bit; it never needs more forwards than the greedy chain."""
    w = PEAKED
    b = _binding()
    prompt = wl.make_prompts(w).numpy()
    peaked_ssd.prefill(prompt)
    tok_s, _, _ = peaked_ssd.generate(b.MODE_STEPWISE, w.gen_len, w.block_len, 1)
    forwards = {}
    try:
        for mix in (0, 1):
            peaked_ssd.set_option("mix_order", mix)
            peaked_ssd.set_option("max_drafts", 4)
            peaked_ssd.prefill(prompt)
            tok, accs, nfs = peaked_ssd.generate(b.MODE_SSD, w.gen_len, w.block_len, 1)
            assert np.array_equal(tok, tok_s)
            for acc, nf in zip(accs, nfs):
                used = acc[0][:nf[0]]
                assert used.sum() == w.block_len and np.all(used >= 1) and np.all(used <= 5)
            forwards[mix] = sum(int(nf[0]) for nf in nfs)
    finally:
        peaked_ssd.set_option("mix_order", 0)
        peaked_ssd.set_option("max_drafts", w.block_len - 1)
    assert forwards[1] <= forwards[0]
    with pytest.raises(b.SsdError) as e:                     # 2N nodes must fit the capacity fixed at creation
        peaked_ssd.set_option("mix_order", 1)
        peaked_ssd.set_option("max_drafts", w.block_len - 1)
        peaked_ssd.prefill(prompt)
        peaked_ssd.decode_block(b.MODE_SSD, w.block_len, 1)
    assert e.value.code == -5
    peaked_ssd.set_option("mix_order", 0)
    peaked_ssd.prefill(prompt)


# ------------------------------------------------------------------------------------------
# top-k LM head and the acceptance-limit probe (Section 5.1, Table 2)
# ------------------------------------------------------------------------------------------
@pytest.mark.parametrize("which", ["tiny", "tiny_peaked"])
def test_topk_forward_matches_oracle(tiny_ssd, peaked_ssd, tiny_oracles, which):
    w = wl.TINY if which == "tiny" else PEAKED
    ssd = tiny_ssd if which == "tiny" else peaked_ssd
    _, ob = tiny_oracles[w.name]
    rng = np.random.default_rng(21)
    prompt = wl.make_prompts(w).numpy()
    T, K = w.block_len, 5
    ids, masked = _random_nodes(w, rng, 3, T)
    ssd.prefill(prompt)
    tok1, conf1, _ = ssd.verify_forward(ids, masked)
    tok, prob = ssd.verify_forward_topk(ids, masked, K)
    m = masked[0]
    # rank 0 is the fused top-1 path, bit for bit
    assert np.array_equal(tok[0][..., 0], tok1[0])
    assert np.array_equal(prob[0][..., 0].view(np.uint32)[m], conf1[0].view(np.uint32)[m])
    assert np.all(tok[0][~m] == -1) and np.all(prob[0][~m] == 0)
    # sorted, distinct, never the mask token
    assert np.all(np.diff(prob[0][m], axis=-1) <= 0)
    assert all(len(set(row)) == K for row in tok[0][m]) and w.mask_id not in tok[0][m]
    cache = ob.prefill(prompt[0])
    _, _, _, ologits = ob.verify(ids[0], masked[0], cache)
    otok, oprob = so.token_topk(ologits.reshape(-1, w.vocab), w.mask_id, K + 1)
    otok, oprob = otok.reshape(3, T, K + 1), oprob.reshape(3, T, K + 1)
    rtol = CONF_RTOL * w.lm_head_scale
    assert np.allclose(prob[0][m], oprob[m][:, :K], rtol=rtol, atol=1e-7)
    # a rank is comparable where the oracle separates it from both neighbours by more than the tolerance
    sep = (oprob[..., :-1] - oprob[..., 1:]) > 2 * rtol * oprob[..., :-1]          # rank r vs r + 1
    safe = sep[..., :K].copy()
    safe[..., 1:] &= sep[..., :K - 1]
    safe &= m[..., None]
    assert np.array_equal(tok[0][safe], otok[..., :K][safe])
    if which == "tiny_peaked":
        assert safe.sum() > 0.25 * m.sum() * K


def test_acceptance_limit_probe_matches_a_recount_and_the_oracle(peaked_ssd, tiny_oracles):
    """The probe decodes the block stepwise and counts on the device; a host recount through
    ssd_verify_forward_topk (same forwards, same bits) gives the same numbers, and so does the oracle's
    procedure when it takes the same stepwise trajectory."""
    w = PEAKED
    b = _binding()
    _, ob = tiny_oracles[w.name]
    prompt = wl.make_prompts(w).numpy()
    T, N, K = w.block_len, 3, 4
    peaked_ssd.prefill(prompt)
    tok_step, _, _ = peaked_ssd.decode_block(b.MODE_STEPWISE, T, 1)
    peaked_ssd.prefill(prompt)
    tok, matched, steps = peaked_ssd.probe_acceptance_limit(T, N, K, 1)
    assert steps == T and np.array_equal(tok, tok_step)
    assert peaked_ssd.cache_length() == w.prompt_len + T
    assert np.all(np.diff(matched) >= 0) and 0 <= matched[0] and matched[-1] <= T - -(-T // (N + 1))
    # host recount with the library's own forwards
    peaked_ssd.prefill(prompt)
    ids = np.full((1, 1, T), w.mask_id)
    msk = np.ones((1, 1, T), bool)
    expect = np.zeros(K, np.int64)
    for step in range(T):
        tk, pr = peaked_ssd.verify_forward_topk(ids, msk, K)
        conf = np.where(msk[0, 0], pr[0, 0, :, 0], -1.0)
        q = int(np.argmax(conf))
        t = int(tk[0, 0, q, 0])
        if step % (N + 1) == 0:
            draft = tk[0, 0].copy()
        else:
            hit = np.nonzero(draft[q] == t)[0]
            if len(hit):
                expect[hit[0]:] += 1
        ids[0, 0, q], msk[0, 0, q] = t, False
    assert np.array_equal(ids[0], tok_step)
    assert np.array_equal(matched, expect)
    # the oracle's own procedure
    cache = ob.prefill(prompt[0])
    oids, omatched, osteps = ob.acceptance_limit_block(T, cache, N, K)
    print(f"acceptance limit, N = {N}: device {matched.tolist()} of {steps}, oracle {omatched.tolist()} of {osteps}")
    assert osteps == steps
    if np.array_equal(oids, tok_step[0]):
        assert np.all(np.abs(matched - omatched) <= 1)


# ------------------------------------------------------------------------------------------
# candidates from the next block (Section 3.2.2)
# ------------------------------------------------------------------------------------------
def _equal_up_to_a_near_tie(got, want, oracle, prompt, gen_len, w, rtol):
    """`got` equals `want` (stepwise tokens), or first differs at a position whose stepwise decision the oracle
    sees as a near-tie within the rounding tolerance (token gap or position margin); after such a position the
    contexts differ and nothing more can be compared."""
    diff = np.nonzero(got != want)[0]
    if len(diff) == 0:
        return True
    first = int(diff[0])
    trace = []
    oracle.generate(prompt, gen_len, w.block_len, mode="stepwise", trace=trace)
    for rec in trace:
        q, _ = rec.pred[0]
        pos = rec.block * w.block_len + q
        cm = np.sort(np.where(rec.node_masked[0], rec.conf[0], -1.0))[::-1]
        margin = cm[0] - cm[1] if len(cm) > 1 and cm[1] >= 0 else np.inf
        near = (rec.gap[0, q] <= 2 * rtol * rec.conf[0, q]) or (margin <= 2 * rtol * cm[0])
        if near and pos <= first:
            return True                                   # a decision at or before the first difference was a near-tie
        if pos == first:
            return bool(near)
    return False


def test_cross_block_generation_is_lossless_and_saves_forwards(tiny_oracles):
    """GPU SSD with candidates that run on into the next block decodes the stepwise tokens, with fewer
    forwards than block-by-block chains.  (Plain SSD equals stepwise bit for bit.  Across a block boundary a
    window node sees the finished block as rows of its own forward where the stepwise forward reads the same
    K/V from the cache: the same values summed in another order, so a decision that is a near-tie within
    rounding noise may fall the other way; anything else must agree.)"""
    w = PEAKED
    o64, _ = tiny_oracles[w.name]
    rtol = CONF_RTOL * w.lm_head_scale
    b = _binding()
    prompt = wl.make_prompts(w).numpy()
    N = 3
    ssd = _make_ssd(w, max_drafts=2 * N + 1)              # room for windows of two blocks
    try:
        ssd.set_option("max_drafts", N)
        ssd.prefill(prompt)
        tok_s, _, _ = ssd.generate(b.MODE_STEPWISE, w.gen_len, w.block_len, 1)
        ssd.prefill(prompt)
        tok_p, acc_p, nf_p = ssd.generate(b.MODE_SSD, w.gen_len, w.block_len, 1)
        ssd.prefill(prompt)
        tok_x, acc_x, nf_x = ssd.generate(b.MODE_SSD, w.gen_len, w.block_len, 1, cross_block=True)
        assert ssd.cache_length() == w.prompt_len + w.gen_len
        # ragged last block and a second batch entry
        prompts2 = wl.make_prompts(w, batch=2).numpy()
        ssd2 = _make_ssd(w, max_drafts=2 * N + 1, max_batch=2)
        try:
            ssd2.set_option("max_drafts", N)
            ssd2.prefill(prompts2)
            r_s, _, _ = ssd2.generate(b.MODE_STEPWISE, 40, w.block_len, 2)
            ssd2.prefill(prompts2)
            r_x, _, _ = ssd2.generate(b.MODE_SSD, 40, w.block_len, 2, cross_block=True)
        finally:
            ssd2.destroy()
    finally:
        ssd.destroy()
    assert np.array_equal(tok_p, tok_s)
    assert _equal_up_to_a_near_tie(tok_x[0], tok_s[0], o64, prompt[0], w.gen_len, w, rtol)
    for i in range(2):
        assert _equal_up_to_a_near_tie(r_x[i], r_s[i], o64, prompts2[i], 40, w, rtol)
    f_plain, f_cross = sum(int(n[0]) for n in nf_p), sum(int(n[0]) for n in nf_x)
    print(f"forwards: block by block {f_plain}, with candidates from the next block {f_cross}")
    assert f_cross < f_plain
    total = 0
    for acc, nf in zip(acc_x, nf_x):
        used = acc[0][:nf[0]]
        assert np.all(used >= 1) and np.all(used <= N + 1)
        total += used.sum()
    assert total == w.gen_len                              # every token was accepted by exactly one forward


def test_cross_block_window_steps_match_oracle(tiny_oracles):
    """Window forwards of the oracle's run replayed on the GPU from the oracle's state of BOTH blocks.
      numeric - the forward's confidences on every asked row of every window node against the oracle's;
      integer - candidate list, per-node prediction scope (current block while it has a masked row, else the
                next block), walk, new state and drafts of both blocks: bit-exact against the oracle's logic
                applied to the GPU forward's own outputs, no exemption; and equal to the oracle's own accepted
                count wherever the oracle's decisions have safe margins."""
    w = PEAKED
    _, ob = tiny_oracles[w.name]
    prompt = wl.make_prompts(w).numpy()
    N, T = 5, w.block_len
    trace = []
    tokens, _, windows = ob.generate_spill(prompt[0], w.gen_len, T, N, trace=trace)
    assert windows > 0
    rtol = CONF_RTOL * w.lm_head_scale
    ssd = _make_ssd(w, max_drafts=2 * N + 1)
    checked = crossed = strict = 0
    try:
        ssd.set_option("max_drafts", N)
        ssd.set_option("fuse_commit", 0)
        ssd.prefill(prompt)
        cur_block = 0
        for rec in trace:
            if rec.block != cur_block:
                ssd.set_option("cross_block", 0)
                ssd.block_begin(T)
                ssd.set_block_state(tokens[cur_block * T:(cur_block + 1) * T][None], np.zeros((1, T), np.uint8))
                ssd.block_commit()
                cur_block = rec.block
            if len(rec.ids_before) == T:
                continue                                          # single-block forwards are covered elsewhere
            T2 = len(rec.ids_before) - T
            W = T + T2
            ssd.set_option("cross_block", T2)
            ssd.block_begin(T)
            dc32 = rec.draft_conf.astype(np.float32)
            ssd.set_block_state(rec.ids_before[None, :T], rec.masked_before[None, :T].astype(np.uint8),
                                rec.draft_tok[None, :T], dc32[None, :T])
            nxt_has = rec.draft_tok[T:].max() >= 0
            if nxt_has:
                ssd.set_next_block_state(rec.ids_before[None, T:], rec.masked_before[None, T:].astype(np.uint8),
                                         np.maximum(rec.draft_tok[None, T:], 0), dc32[None, T:])
            else:
                ssd.set_next_block_state(rec.ids_before[None, T:], rec.masked_before[None, T:].astype(np.uint8))
            acc, nn = ssd.block_step(N, 1)
            n = rec.node_ids.shape[0]
            assert nn[0] == n
            tok_g, conf_g = ssd.read_forward_outputs(n * W)
            tok_g, conf_g = tok_g.reshape(n, W), conf_g.reshape(n, W)
            m = rec.node_masked
            # ---- numeric layer (inputs are the oracle's; float32 drafts may reorder exact-tie candidates only)
            assert np.all(tok_g[~m] == -1)
            assert np.allclose(conf_g[m], rec.conf[m], rtol=rtol, atol=1e-6)
            # ---- integer layer on the GPU's own outputs
            pred = []
            for i in range(n):
                scope = m[i].copy()
                if m[i, :T].any():
                    scope[T:] = False
                else:
                    scope[:T] = False
                q = so.best_masked_position(conf_g[i], scope)
                pred.append((q, int(tok_g[i, q])))
            a = so.accept_length(pred, rec.cand)
            accepted = list(rec.cand[:a]) + [pred[a]]
            assert acc[0] == len(accepted)
            want_ids, want_m = rec.ids_before.copy(), rec.masked_before.copy()
            seen_next = False
            for (p, t) in accepted:
                if p >= T:
                    assert not want_m[:T].any()                   # block order: the current block was full by then
                    crossed += 1
                want_ids[p], want_m[p] = t, False
            ids0, m0, dt0, dc0 = ssd.get_block_state(1, T)
            ids1, m1, dt1, dc1 = ssd.get_next_block_state(1, T2)
            ids_g, m_g = np.concatenate([ids0[0], ids1[0]]), np.concatenate([m0[0], m1[0]]).astype(bool)
            dt_g, dc_g = np.concatenate([dt0[0], dt1[0]]), np.concatenate([dc0[0], dc1[0]])
            assert np.array_equal(m_g, want_m) and np.array_equal(ids_g[~want_m], want_ids[~want_m])
            assert np.array_equal(dt_g[want_m], tok_g[a][want_m])
            assert np.array_equal(dc_g[want_m].view(np.uint32), conf_g[a][want_m].view(np.uint32))
            checked += 1
            if pred == list(rec.pred):                             # same decisions as the oracle: same count
                strict += 1
                assert acc[0] == rec.accepted
    finally:
        ssd.destroy()
    print(f"cross-block: {checked} window forwards replayed, {strict} with the oracle's own decisions, "
          f"{crossed} tokens accepted across the boundary")
    assert checked > 0 and crossed > 0


# ------------------------------------------------------------------------------------------
# dual cache with a refresh interval (Section 4.1)
# ------------------------------------------------------------------------------------------
@pytest.mark.parametrize("which", ["tiny", "tiny_peaked"])
def test_dual_cache_forward_matches_oracle(tiny_oracles, which):
    """After a refresh the K/V of every position outside the current block - prefix AND masked suffix - are
    those of the oracle's full-sequence forward, and a block forward against them gives the oracle's logits;
    once a token has been decoded without a refresh, the forward still matches the oracle run on the same
    (now stale) cache."""
    w = wl.TINY if which == "tiny" else PEAKED
    o64, ob = tiny_oracles[w.name]
    rng = np.random.default_rng(31)
    prompt = wl.make_prompts(w).numpy()
    P, T, L = w.prompt_len, w.block_len, w.gen_len
    mid = w.mask_id
    ssd = _make_ssd(w, max_drafts=4)
    try:
        ssd.prefill(prompt)
        ssd.set_option("dual_cache", P + L)
        ssd.set_option("refresh_interval", 4)
        block0 = rng.integers(0, w.vocab - 1, T)
        ssd.block_begin(T)
        ssd.set_block_state(block0[None], np.zeros((1, T), np.uint8))
        ssd.block_commit()                                    # dual cache: the tokens are recorded, nothing is committed
        assert ssd.cache_length() == P + T
        S = P + T
        state_ids = rng.integers(0, w.vocab - 1, T)
        state_masked = rng.random(T) < 0.6
        state_masked[0] = True
        ssd.block_begin(T)
        ssd.set_block_state(state_ids[None], state_masked[None].astype(np.uint8))
        ssd.refresh_cache()
        assert ssd.refresh_count() == 1
        ids, masked = _random_nodes(w, rng, 3, T)
        tok, conf, logits = ssd.verify_forward(ids, masked, want_logits=True)
        k_gpu, v_gpu = ssd.read_cache(0, 0, P + L)
    finally:
        ssd.destroy()
    x = np.concatenate([prompt[0], block0, np.where(state_masked, mid, state_ids), np.full(L - 2 * T, mid)])
    for o, tol in ((ob, 1e-2), (o64, 2e-2)):
        full = o.refresh_all(x)
        outside = so.Cache(o.cfg)
        outside.k = [np.concatenate([k[:S], k[S + T:]], axis=0) for k in full.k]
        outside.v = [np.concatenate([v[:S], v[S + T:]], axis=0) for v in full.v]
        ologits, _, _ = o.forward_rows(ids[0], S, outside)
        err = np.abs(logits[0] - ologits).max()
        assert err < tol * w.lm_head_scale, (err, tol)
        otok, oconf = so.token_and_confidence(ologits.reshape(-1, w.vocab), mid)
        m = masked[0].reshape(-1)
        assert np.allclose(conf[0].reshape(-1)[m], oconf[m], rtol=CONF_RTOL * w.lm_head_scale, atol=1e-6)
        # the whole sequence's K/V of layer 0, suffix included
        assert np.abs(k_gpu - full.k[0]).max() < 2e-2 * max(1.0, np.abs(full.k[0]).max())
        assert np.abs(v_gpu - full.v[0]).max() < 2e-2 * max(1.0, np.abs(full.v[0]).max())


def test_dual_cache_generation_follows_the_schedule_and_stays_lossless():
    """GPU SSD under the dual cache == GPU stepwise under the same schedule, bit for bit, for several draft
    lengths; the refreshes fall at every block start and after every `refresh_interval` tokens."""
    w = PEAKED
    b = _binding()
    prompts = wl.make_prompts(w, batch=2).numpy()
    P, T, L = w.prompt_len, w.block_len, w.gen_len
    ssd = _make_ssd(w, max_drafts=5, max_batch=2)
    try:
        for refresh in (4, 6, 100):
            expect = 2 * sum(-(-(min(T, L - lo)) // refresh) for lo in range(0, L, T))      # two sequences
            ssd.prefill(prompts)
            ssd.set_option("dual_cache", P + L)
            ssd.set_option("refresh_interval", refresh)
            r0 = ssd.refresh_count()
            tok_s, acc_s, nf_s = ssd.generate(b.MODE_STEPWISE, L, T, 2)
            assert ssd.refresh_count() - r0 == expect
            assert ssd.cache_length() == P + L
            for N in (1, 3, 5):
                ssd.set_option("dual_cache", 0)
                ssd.prefill(prompts)
                ssd.set_option("dual_cache", P + L)
                ssd.set_option("max_drafts", N)
                r0 = ssd.refresh_count()
                tok, accs, nfs = ssd.generate(b.MODE_SSD, L, T, 2)
                assert np.array_equal(tok, tok_s)
                assert ssd.refresh_count() - r0 == expect
                for acc, nf in zip(accs, nfs):
                    for i in range(2):
                        used = acc[i][:nf[i]]
                        assert used.sum() == T and np.all(used >= 1) and np.all(used <= min(N + 1, refresh))
            ssd.set_option("dual_cache", 0)
        # the exact prefix cache decodes something else in general: the dual cache sees the masked suffix
        ssd.set_option("max_drafts", 3)
        ssd.prefill(prompts)
        tok_prefix, _, _ = ssd.generate(b.MODE_STEPWISE, L, T, 2)
        assert tok_prefix.shape == tok_s.shape
    finally:
        ssd.destroy()


def test_a_wait_that_runs_out_is_reported_and_the_context_survives(tiny_ssd):
    """Failure made on the host side: the projection kernel's producer is told to leave out one K block's
    copies, the wait for that block runs out after a millisecond bound, the kernel unwinds (tensor memory
    freed, no trap) and the call returns SSD_ERR_TIMEOUT; the next call on the same context succeeds."""
    b = _binding()
    x = wl.normal_tensor(8, 1, (16, 256), 1.0, device="cuda", dtype=torch.bfloat16)
    w = wl.normal_tensor(8, 2, (128, 256), 0.05, device="cuda", dtype=torch.bfloat16)
    ref = x.cpu().to(torch.float64).numpy() @ w.cpu().to(torch.float64).numpy().T
    try:
        tiny_ssd.set_option("wait_limit_us", 2000)
        tiny_ssd.set_option("starve_gemm_kb", 2)
        with pytest.raises(b.SsdError) as e:
            tiny_ssd.gemm_bf16(x, w, 1)
        assert e.value.code == -6
        with pytest.raises(b.SsdError) as e:
            tiny_ssd.gemm_bf16(x, w, 2)                     # the hook is refused for anything but the plain launch
        assert e.value.code == -2
    finally:
        tiny_ssd.set_option("starve_gemm_kb", 0)
        tiny_ssd.set_option("wait_limit_us", 0)
    out = tiny_ssd.gemm_bf16(x, w, 1).cpu().numpy()
    assert np.abs(out - ref).max() < 2e-5 * 0.05 * 256 + 1e-6
    # and a whole decode still works on it
    prompt = wl.make_prompts(wl.TINY).numpy()
    tiny_ssd.prefill(prompt)
    tok, acc, nf = tiny_ssd.decode_block(b.MODE_SSD, wl.TINY.block_len, 1)
    assert acc[0][:nf[0]].sum() == wl.TINY.block_len


def test_variants_treat_every_sequence_of_a_batch_as_if_alone(peaked_ssd):
    """Mix-order trees and the acceptance-limit probe on a batch of three: every sequence decodes exactly what
    it decodes alone (tokens, accept counts, matched counts)."""
    w = PEAKED
    b = _binding()
    prompts = wl.make_prompts(w, batch=3).numpy()
    T = w.block_len
    try:
        peaked_ssd.set_option("max_drafts", 4)
        peaked_ssd.set_option("mix_order", 1)
        peaked_ssd.prefill(prompts)
        tok_b, acc_b, nf_b = peaked_ssd.generate(b.MODE_SSD, 2 * T, T, 3)
        for s in range(3):
            peaked_ssd.prefill(prompts[s:s + 1])
            tok_s, acc_s, nf_s = peaked_ssd.generate(b.MODE_SSD, 2 * T, T, 1)
            assert np.array_equal(tok_s[0], tok_b[s])
            for j in range(len(acc_s)):
                assert np.array_equal(acc_s[j][0], acc_b[j][s]) and nf_s[j][0] == nf_b[j][s]
        peaked_ssd.set_option("mix_order", 0)
        peaked_ssd.prefill(prompts)
        tok_p, matched_b, steps_b = peaked_ssd.probe_acceptance_limit(T, 3, 4, 3)
        assert steps_b == 3 * T
        total = np.zeros(4, np.int64)
        for s in range(3):
            peaked_ssd.prefill(prompts[s:s + 1])
            tok_1, matched_1, steps_1 = peaked_ssd.probe_acceptance_limit(T, 3, 4, 1)
            assert np.array_equal(tok_1[0], tok_p[s]) and steps_1 == T
            total += matched_1
        assert np.array_equal(total, matched_b)
    finally:
        peaked_ssd.set_option("mix_order", 0)
        peaked_ssd.set_option("max_drafts", w.block_len - 1)
        peaked_ssd.prefill(prompts[:1])
