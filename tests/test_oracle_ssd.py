"""Pins for the oracle's decoding logic: what the paper fixes about SSD.

* output identical to stepwise decoding (abstract, Section 4.2, Conclusion);
* N+1 nodes for draft length N, between 1 and N+1 tokens per forward (Sections 3.2.3-3.2.4,
  Appendix A) and the node counts 4/5/6 printed in Table 3;
* the forward-pass reduction bound N/(N+1) printed in Table 2;
* a child is valid only if its parent's prediction equals the stepwise result, and a draft with
  the right tokens in another order fails (Section 5.1);
* block order (Section 3.1): nothing of block j+1 before block j is complete.
"""
import os

import numpy as np
import pytest

from oracle import ssd_oracle as so
from tests.helpers import SMALL, SMALL_GQA, make_oracle
from paper_2510_04147_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                a, b = line.split()
                rows.append((int(a), float(b)))
    return rows


# ---------------------------------------------------------------------------------------
# model-free pins: a scripted verifier replaces f_theta
# ---------------------------------------------------------------------------------------
class ScriptedOracle(so.Oracle):
    """verify() answers from a script instead of a transformer.

    ``rule(node_ids_row, node_masked_row) -> (tok[B], conf[B])`` plays the model for one node.
    """

    def __init__(self, vocab, rule):
        cfg = so.ModelConfig(0, 0, 0, 0, 0, 0, vocab, vocab - 1, 1.0, 0.0)
        super().__init__(cfg, {})
        self.rule = rule
        self.n_forwards = 0
        self.nodes_per_forward = []

    def verify(self, node_ids, node_masked, cache):
        self.n_forwards += 1
        self.nodes_per_forward.append(node_ids.shape[0])
        out = [self.rule(node_ids[i], node_masked[i]) for i in range(node_ids.shape[0])]
        tok = np.stack([o[0] for o in out])
        conf = np.stack([o[1] for o in out])
        return tok, conf, np.ones_like(conf), None


class NoCache:
    length = 0


def _context_free_rule(B):
    """Predictions depend on the position only: drafts never go stale."""
    tok = (np.arange(B) * 7 + 3) % 50
    conf = np.linspace(0.9, 0.1, B)
    return lambda ids, masked: (tok.copy(), conf.copy())


@pytest.mark.parametrize("N,pct", _golden("step_reduction_upper_bound.txt"))
def test_upper_bound_of_step_reduction(N, pct):
    """With drafts that are always right every forward after the first accepts N+1 tokens, so
    the reduction of forward passes tends to N/(N+1): 75.0 / 80.0 / 83.3 % (Table 2)."""
    B = 4000
    o = ScriptedOracle(64, _context_free_rule(B))
    ids, counts = o.decode_block_ssd(B, NoCache(), max_drafts=N)
    assert np.array_equal(ids, (np.arange(B) * 7 + 3) % 50)
    assert counts[0] == 1 and all(c == N + 1 for c in counts[1:-1]) and sum(counts) == B
    assert len(counts) == 1 + -(-(B - 1) // (N + 1))
    assert round(100.0 * (1 - len(counts) / B), 1) == pct
    assert abs((1 - len(counts) / B) - N / (N + 1)) < 1e-3


@pytest.mark.parametrize("N,nodes", _golden("greedy_verification_batch.txt"))
def test_chain_has_n_plus_one_nodes(N, nodes):
    B = 16
    o = ScriptedOracle(64, _context_free_rule(B))
    o.decode_block_ssd(B, NoCache(), max_drafts=N)
    # first forward is root-only; while at least N+1 positions are masked the chain has N+1 nodes
    assert o.nodes_per_forward[0] == 1
    assert o.nodes_per_forward[1] == int(nodes) == N + 1
    assert max(o.nodes_per_forward) == N + 1


def test_build_chain_contents():
    ids = np.array([5, 63, 63, 9, 63, 63])
    masked = np.array([0, 1, 1, 0, 1, 1], dtype=bool)
    cand = [(4, 11), (1, 12), (5, 13)]
    node_ids, node_masked = so.build_chain(ids, masked, cand, 63)
    assert node_ids.shape == (4, 6)
    assert node_ids.tolist() == [[5, 63, 63, 9, 63, 63], [5, 63, 63, 9, 11, 63],
                                 [5, 12, 63, 9, 11, 63], [5, 12, 63, 9, 11, 13]]
    assert node_masked.sum(axis=1).tolist() == [4, 3, 2, 1]
    assert node_masked[3].tolist() == [False, False, True, False, False, False]


def test_select_candidates_order_and_cap():
    tok = np.array([10, 11, 12, 13, 14, 15])
    conf = np.array([0.2, 0.9, 0.5, 0.9, 0.1, 0.7])
    masked = np.array([1, 1, 0, 1, 1, 1], dtype=bool)
    # descending confidence, lower position first on the 0.9 tie, unmasked position 2 never chosen
    assert so.select_candidates(tok, conf, masked, 10) == [(1, 11), (3, 13), (5, 15), (0, 10)]
    assert so.select_candidates(tok, conf, masked, 2) == [(1, 11), (3, 13)]
    assert so.select_candidates(tok, conf, masked, 0) == []
    one = np.array([0, 0, 0, 0, 1, 0], dtype=bool)
    assert so.select_candidates(tok, conf, one, 5) == []     # r = 1 -> plain stepwise step


def test_accept_length_walk():
    cand = [(4, 11), (1, 12), (5, 13)]
    assert so.accept_length([(4, 11), (1, 12), (5, 13), (2, 7)], cand) == 3
    assert so.accept_length([(4, 11), (1, 99), (5, 13), (2, 7)], cand) == 1     # wrong token
    assert so.accept_length([(4, 11), (5, 13), (1, 12), (2, 7)], cand) == 1     # right tokens, other order
    assert so.accept_length([(0, 11), (1, 12), (5, 13), (2, 7)], cand) == 0     # right token, wrong position
    assert so.accept_length([(3, 3)], []) == 0


def test_wrong_drafts_accept_exactly_one_and_keep_tokens():
    """Adversarial drafts (wrong token / swapped order) cost nothing but speed."""
    B = 24
    base = ScriptedOracle(64, _context_free_rule(B))
    want, _ = base.decode_block_stepwise(B, NoCache())

    def wrong_token(ids, masked, dt, dc):
        return (dt + 1) % 50, dc

    def swapped_order(ids, masked, dt, dc):
        return dt, 1.0 - dc         # same tokens, reversed priority

    for override in (wrong_token, swapped_order):
        o = ScriptedOracle(64, _context_free_rule(B))
        ids, counts = o.decode_block_ssd(B, NoCache(), max_drafts=4, draft_override=override)
        assert np.array_equal(ids, want)
        if override is wrong_token:
            assert counts == [1] * B
        else:
            # reversed priority: the first candidate is never the stepwise choice
            # (except when a single masked position is left)
            assert all(c == 1 for c in counts)


def test_context_dependent_script_matches_bruteforce():
    """A scripted model whose predictions change with the context (so drafts do go stale):
    accepted count per forward == 1 + longest common prefix of the draft chain with the true
    stepwise continuation from the same state, capped at N+1."""
    B, V = 14, 40
    table_rng = np.random.default_rng(5)
    tok_tab = table_rng.integers(0, V - 1, (B + 1, B))
    conf_tab = table_rng.random((B + 1, B))

    def rule(ids, masked):
        r = int(masked.sum())           # context = how many positions are still masked
        return tok_tab[r].copy(), conf_tab[r].copy()

    ref = ScriptedOracle(V, rule)
    want, _ = ref.decode_block_stepwise(B, NoCache())
    # stepwise order of (position, token)
    order = []
    ids = np.full(B, V - 1)
    masked = np.ones(B, dtype=bool)
    while masked.any():
        t, c = rule(ids, masked)
        q = so.best_masked_position(c, masked)
        order.append((q, int(t[q])))
        ids[q] = t[q]
        masked[q] = False
    for N in (1, 3, 5, B):
        trace = []
        o = ScriptedOracle(V, rule)
        got, counts = o.decode_block_ssd(B, NoCache(), max_drafts=N, trace=trace)
        assert np.array_equal(got, want)
        done = 0
        for rec in trace:
            cont = order[done:]
            lcp = 0
            while lcp < len(rec.cand) and rec.cand[lcp] == cont[lcp]:
                lcp += 1
            assert rec.accepted == lcp + 1
            assert 1 <= rec.accepted <= len(rec.cand) + 1 <= N + 1
            done += rec.accepted
        assert done == B


# ---------------------------------------------------------------------------------------
# pins that use the real model
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("w", [SMALL, SMALL_GQA], ids=lambda w: w.name)
@pytest.mark.parametrize("max_drafts", [0, 1, 3, 5, 64])
def test_ssd_equals_stepwise_small(w, max_drafts):
    o = make_oracle(w)
    prompt = wl.make_prompts(w)[0].numpy()
    want, c0, _ = o.generate(prompt, w.gen_len, w.block_len, mode="stepwise")
    got, c1, _ = o.generate(prompt, w.gen_len, w.block_len, mode="ssd", max_drafts=max_drafts)
    assert np.array_equal(got, want)
    for blk in c1:
        assert sum(blk) == w.block_len and all(1 <= c <= max_drafts + 1 for c in blk)
    if max_drafts == 0:
        assert c1 == c0            # no drafts -> exactly the stepwise forward count


def test_ssd_equals_stepwise_ragged_last_block():
    w = SMALL.replace(gen_len=10, block_len=4)
    o = make_oracle(w)
    prompt = wl.make_prompts(w)[0].numpy()
    want, _, cache0 = o.generate(prompt, w.gen_len, w.block_len, mode="stepwise")
    got, counts, cache1 = o.generate(prompt, w.gen_len, w.block_len, mode="ssd", max_drafts=3)
    assert np.array_equal(got, want) and len(got) == 10
    assert [sum(c) for c in counts] == [4, 4, 2]
    assert cache0.length == cache1.length == w.prompt_len + 10


@pytest.mark.parametrize("peaked", [1.0, 8.0])
def test_ssd_equals_stepwise_tiny_config(peaked):
    """Config 1 (tiny model, prompt 32, L 64, B 16), plain and the 'peaked' LM-head variant."""
    w = wl.TINY.replace(lm_head_scale=peaked)
    o = make_oracle(w)
    prompt = wl.make_prompts(w)[0].numpy()
    want, _, _ = o.generate(prompt, w.gen_len, w.block_len, mode="stepwise")
    trace = []
    got, counts, _ = o.generate(prompt, w.gen_len, w.block_len, mode="ssd", max_drafts=w.block_len, trace=trace)
    assert np.array_equal(got, want)
    assert all(sum(c) == w.block_len for c in counts)
    assert w.mask_id not in got
    # every record: accepted = 1 + LCP(draft chain, stepwise continuation from that state)
    o2 = make_oracle(w)
    for rec in trace[:12]:
        cache = _cache_at(o2, prompt, want, rec.block, w.block_len)
        ids, masked = rec.ids_before.copy(), rec.masked_before.copy()
        cont = []
        while masked.any() and len(cont) <= len(rec.cand):
            tok, conf, _, _ = o2.verify(*so.build_chain(ids, masked, [], w.mask_id), cache)
            q = so.best_masked_position(conf[0], masked)
            cont.append((q, int(tok[0, q])))
            ids[q] = tok[0, q]
            masked[q] = False
        lcp = 0
        while lcp < len(rec.cand) and lcp < len(cont) and rec.cand[lcp] == cont[lcp]:
            lcp += 1
        assert rec.accepted == lcp + 1


def _cache_at(o, prompt, tokens, block, B):
    cache = o.prefill(prompt)
    for j in range(block):
        o.commit_block(tokens[j * B:(j + 1) * B], cache)
    return cache


def test_block_length_one_is_stepwise():
    w = SMALL.replace(gen_len=5, block_len=1)
    o = make_oracle(w)
    prompt = wl.make_prompts(w)[0].numpy()
    a, ca, _ = o.generate(prompt, 5, 1, mode="stepwise")
    b, cb, _ = o.generate(prompt, 5, 1, mode="ssd", max_drafts=4)
    assert np.array_equal(a, b) and ca == cb == [[1]] * 5


def test_context_free_model_accepts_everything():
    """One layer with Wo = 0 and Wd = 0: a row's logits depend on its own token only, so a masked
    row always predicts the same thing, drafts never go stale and every verify accepts N+1."""
    w = SMALL.replace(n_layers=1, gen_len=12, block_len=12)
    from tests.helpers import oracle_config, oracle_weights
    W = oracle_weights(w, as_bf16=False)
    W["layers.0.wo"] = np.zeros_like(W["layers.0.wo"])
    W["layers.0.w_down"] = np.zeros_like(W["layers.0.w_down"])
    o = so.Oracle(oracle_config(w), W)
    prompt = wl.make_prompts(w)[0].numpy()
    # all masked rows are identical -> equal confidences -> lowest position first
    got, counts, _ = o.generate(prompt, 12, 12, mode="ssd", max_drafts=3)
    assert counts == [[1, 4, 4, 3]]
    assert len(set(got.tolist())) == 1


def test_block_order_constraint():
    """Nothing of block j+1 exists while block j is decoded: the trace of block j never touches
    positions beyond it, and the cache grows by exactly one block per commit."""
    w = SMALL
    o = make_oracle(w)
    prompt = wl.make_prompts(w)[0].numpy()
    trace = []
    o.generate(prompt, w.gen_len, w.block_len, mode="ssd", max_drafts=3, trace=trace)
    for rec in trace:
        assert rec.cache_len == w.prompt_len + rec.block * w.block_len
        assert rec.node_ids.shape[1] == w.block_len
        assert all(0 <= p < w.block_len for p, _ in rec.cand)


# ---------------------------------------------------------------------------------------
# mix-order tree (Section 5.2, Table 3)
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("N,nodes", _golden("mix_order_verification_batch.txt"))
def test_mix_order_tree_has_2n_nodes(N, nodes):
    B = 16
    o = ScriptedOracle(64, _context_free_rule(B))
    o.decode_block_ssd(B, NoCache(), max_drafts=N, tree="mix_order")
    assert o.nodes_per_forward[0] == 1
    assert o.nodes_per_forward[1] == int(nodes) == 2 * N
    assert max(o.nodes_per_forward) == 2 * N


def test_mix_order_tree_contents():
    ids = np.array([5, 63, 63, 9, 63, 63])
    masked = np.array([0, 1, 1, 0, 1, 1], dtype=bool)
    cand = [(4, 11), (1, 12), (5, 13)]
    node_ids, node_masked = so.build_mix_order_tree(ids, masked, cand, 63)
    chain_ids, chain_masked = so.build_chain(ids, masked, cand, 63)
    assert node_ids.shape == (6, 6)
    assert np.array_equal(node_ids[:4], chain_ids) and np.array_equal(node_masked[:4], chain_masked)
    # branch of node 0: candidate 2 alone; branch of node 1: candidates 1 and 3
    assert node_ids[4].tolist() == [5, 12, 63, 9, 63, 63]
    assert node_ids[5].tolist() == [5, 63, 63, 9, 11, 13]
    assert node_masked[4].tolist() == [False, False, True, False, True, True]
    assert node_masked[5].tolist() == [False, True, True, False, False, False]
    # fewer than two candidates: nothing to branch to
    assert so.build_mix_order_tree(ids, masked, cand[:1], 63)[0].shape == (2, 6)
    assert so.build_mix_order_tree(ids, masked, [], 63)[0].shape == (1, 6)


def test_mix_order_walk():
    cand = [(4, 11), (1, 12), (5, 13)]
    # node order: chain 0..3, branch of 0, branch of 1
    chain_ok = [(4, 11), (1, 12), (5, 13), (2, 7), (0, 0), (0, 0)]
    assert so.accept_walk_mix_order(chain_ok, cand) == ([(4, 11), (1, 12), (5, 13), (2, 7)], 3)
    swapped_at_root = [(1, 12), (0, 0), (0, 0), (0, 0), (4, 99), (0, 0)]
    assert so.accept_walk_mix_order(swapped_at_root, cand) == ([(1, 12), (4, 99)], 4)
    swapped_at_one = [(4, 11), (5, 13), (0, 0), (0, 0), (0, 0), (2, 8)]
    assert so.accept_walk_mix_order(swapped_at_one, cand) == ([(4, 11), (5, 13), (2, 8)], 5)
    # a skip of two, a wrong token at the other position, and the last chain node have no branch
    assert so.accept_walk_mix_order([(5, 13), (0, 0), (0, 0), (0, 0), (0, 0), (0, 0)], cand) == ([(5, 13)], 0)
    assert so.accept_walk_mix_order([(1, 99), (0, 0), (0, 0), (0, 0), (0, 0), (0, 0)], cand) == ([(1, 99)], 0)
    assert so.accept_walk_mix_order([(4, 11), (1, 12), (2, 7), (0, 0), (0, 0), (0, 0)], cand) == \
        ([(4, 11), (1, 12), (2, 7)], 2)
    assert so.accept_walk_mix_order([(3, 3)], []) == ([(3, 3)], 0)


def test_mix_order_recovers_the_swapped_order_case():
    """Section 5.2 / Fig. 4(b): drafts that hold the right tokens in another order cost the greedy chain
    everything but one token per forward; the mix-order branch accepts the swapped candidate and its
    own prediction."""
    B = 24
    base = ScriptedOracle(64, _context_free_rule(B))
    want, _ = base.decode_block_stepwise(B, NoCache())
    conf = np.linspace(0.9, 0.1, B)

    def swap_first_two(ids, masked, dt, dc):
        pos = [p for p in range(B) if masked[p]]
        order = sorted(pos, key=lambda p: -conf[p])
        dc = conf.copy()
        if len(order) >= 2:
            dc[order[0]], dc[order[1]] = conf[order[1]], conf[order[0]]
        return dt, dc

    g = ScriptedOracle(64, _context_free_rule(B))
    ids_g, counts_g = g.decode_block_ssd(B, NoCache(), max_drafts=4, draft_override=swap_first_two)
    m = ScriptedOracle(64, _context_free_rule(B))
    ids_m, counts_m = m.decode_block_ssd(B, NoCache(), max_drafts=4, draft_override=swap_first_two, tree="mix_order")
    assert np.array_equal(ids_g, want) and np.array_equal(ids_m, want)
    assert all(c == 1 for c in counts_g[:-1])
    assert all(c == 2 for c in counts_m[1:-3]) and len(counts_m) < len(counts_g)


def test_mix_order_matches_bruteforce_and_never_loses_to_greedy():
    """Context-dependent scripted model: the tokens a mix-order forward accepts are exactly the next
    stepwise steps from the same state, their number is the greedy count or one more, and the output
    is the stepwise output."""
    B, V = 14, 40
    table_rng = np.random.default_rng(7)
    # tokens mostly stable, confidences jitter with the context: the drafts usually hold the right
    # tokens, but their order goes stale - the out-of-order case of Fig. 4(a)
    tok_tab = np.tile(table_rng.integers(0, V - 1, B), (B + 1, 1))
    tok_tab[::4] = table_rng.integers(0, V - 1, (len(tok_tab[::4]), B))
    conf_tab = np.linspace(0.9, 0.2, B)[None, :] + 0.12 * table_rng.random((B + 1, B))

    def rule(ids, masked):
        r = int(masked.sum())
        return tok_tab[r].copy(), conf_tab[r].copy()

    ref = ScriptedOracle(V, rule)
    want, _ = ref.decode_block_stepwise(B, NoCache())
    order = []
    ids = np.full(B, V - 1)
    masked = np.ones(B, dtype=bool)
    while masked.any():
        t, c = rule(ids, masked)
        q = so.best_masked_position(c, masked)
        order.append((q, int(t[q])))
        ids[q] = t[q]
        masked[q] = False
    gained = 0
    for N in (2, 3, 5, B):
        trace = []
        o = ScriptedOracle(V, rule)
        got, counts = o.decode_block_ssd(B, NoCache(), max_drafts=N, trace=trace, tree="mix_order")
        assert np.array_equal(got, want)
        done = 0
        for rec in trace:
            n = len(rec.cand)
            accepted, last = so.accept_walk_mix_order(rec.pred, rec.cand)
            assert accepted == order[done:done + rec.accepted]            # exactly the stepwise continuation
            greedy = so.accept_length(rec.pred[:n + 1], rec.cand) + 1
            assert rec.accepted in (greedy, greedy + 1)
            assert rec.node_ids.shape[0] == n + 1 + max(0, n - 1)
            gained += rec.accepted - greedy
            done += rec.accepted
        assert done == B
    assert gained > 0                                                     # the branch is exercised


@pytest.mark.parametrize("w", [SMALL, SMALL_GQA], ids=lambda w: w.name)
@pytest.mark.parametrize("max_drafts", [1, 2, 3, 5, 64])
def test_mix_order_equals_stepwise_small(w, max_drafts):
    o = make_oracle(w)
    prompt = wl.make_prompts(w)[0].numpy()
    a, _, _ = o.generate(prompt, w.gen_len, w.block_len, mode="stepwise")
    b, counts, _ = o.generate(prompt, w.gen_len, w.block_len, mode="ssd", max_drafts=max_drafts, tree="mix_order")
    assert np.array_equal(a, b)
    assert all(sum(c) == w.block_len for c in counts)


# ---------------------------------------------------------------------------------------
# acceptance-rate limit of self-drafting (Section 5.1, Table 2)
# ---------------------------------------------------------------------------------------
def test_token_topk_matches_torch_and_top1():
    import torch
    rng = np.random.default_rng(3)
    logits = rng.standard_normal((9, 50))
    logits[2, 7] = logits[2, 11] = logits[2].max() + 1.0          # a tie: the lower id comes first
    mask_id = 49
    tok, prob = so.token_topk(logits, mask_id, 5)
    l = torch.tensor(logits)
    l[:, mask_id] = -float("inf")
    ref_p, ref_i = torch.topk(torch.softmax(l, -1), 5, dim=-1)
    assert np.allclose(prob, ref_p.numpy(), rtol=1e-12)
    assert tok[2, 0] == 7 and tok[2, 1] == 11
    rows = [r for r in range(9) if r != 2]
    assert np.array_equal(tok[rows], ref_i.numpy()[rows])
    t1, c1 = so.token_and_confidence(logits, mask_id)
    assert np.array_equal(tok[:, 0], t1) and np.allclose(prob[:, 0], c1, rtol=1e-12)
    assert mask_id not in tok


class ScriptedLogitsOracle(so.Oracle):
    """verify() answers logits from a script: rule(ids_row, masked_row) -> logits [B, V]."""

    def __init__(self, vocab, rule):
        super().__init__(so.ModelConfig(0, 0, 0, 0, 0, 0, vocab, vocab - 1, 1.0, 0.0), {})
        self.rule = rule

    def verify(self, node_ids, node_masked, cache):
        logits = np.stack([self.rule(node_ids[i], node_masked[i]) for i in range(node_ids.shape[0])])
        n, T, V = logits.shape
        tok, conf = so.token_and_confidence(logits.reshape(n * T, V), self.cfg.mask_id)
        return tok.reshape(n, T), conf.reshape(n, T), np.ones((n, T)), logits


@pytest.mark.parametrize("N,pct", _golden("step_reduction_upper_bound.txt"))
def test_acceptance_limit_reaches_the_printed_bound_when_drafts_never_go_stale(N, pct):
    """A model whose predictions do not depend on the context: every stepwise token is the draft's
    top-1, so the limit is the bound N/(N+1) of Table 2 already at k = 1."""
    B, V = 60 * (N + 1), 40
    rng = np.random.default_rng(N)
    fixed = rng.standard_normal((B, V)) * 3.0
    o = ScriptedLogitsOracle(V, lambda ids, masked: fixed)
    ids, matched, steps = o.acceptance_limit_block(B, NoCache(), N, 3)
    assert steps == B and np.all(matched == B - B // (N + 1))
    assert round(100.0 * matched[0] / steps, 1) == pct


def test_acceptance_limit_counts_match_bruteforce_and_grow_with_k():
    """Context-dependent scripted logits: the counts equal a direct recount from the stepwise trajectory,
    are non-decreasing in k, and k = vocabulary size matches everything (the bound)."""
    B, V, N = 18, 12, 2
    rng = np.random.default_rng(9)
    tabs = rng.standard_normal((B + 1, B, V)) * 2.0

    def rule(ids, masked):
        return tabs[int(masked.sum())]

    o = ScriptedLogitsOracle(V, rule)
    ids, matched, steps = o.acceptance_limit_block(B, NoCache(), N, V - 1)
    want, _ = o.decode_block_stepwise(B, NoCache())
    assert np.array_equal(ids, want) and steps == B
    # recount: replay stepwise, remember the ranking of every position at each round start
    cur = np.full(B, V - 1)
    msk = np.ones(B, dtype=bool)
    expect = np.zeros(V - 1, dtype=int)
    for step in range(B):
        logits = rule(cur, msk).copy()
        logits[:, V - 1] = -np.inf
        if step % (N + 1) == 0:
            rank_of = np.argsort(np.argsort(-logits, axis=-1, kind="stable"), axis=-1, kind="stable")
        conf = np.exp(logits - logits.max(-1, keepdims=True))
        conf = (conf / conf.sum(-1, keepdims=True)).max(-1)
        q = so.best_masked_position(conf, msk)
        t = int(np.argmax(logits[q]))
        if step % (N + 1) != 0:
            expect[rank_of[q, t]:] += 1
        cur[q], msk[q] = t, False
    assert np.array_equal(matched, expect)
    assert np.all(np.diff(matched) >= 0)
    assert matched[-1] == B - B // (N + 1)               # every token is within the top V-1
    assert 0 < matched[0] < matched[-1]                  # stale drafts: k = 1 misses some


def test_acceptance_limit_on_the_model_keeps_stepwise_tokens():
    w = SMALL
    o = make_oracle(w)
    prompt = wl.make_prompts(w)[0].numpy()
    want, _, _ = o.generate(prompt, w.gen_len, w.block_len, mode="stepwise")
    got, red = o.acceptance_limit(prompt, w.gen_len, w.block_len, 2, 4)
    assert np.array_equal(got, want)
    assert np.all(np.diff(red) >= 0) and np.all(red >= 0) and np.all(red <= 2.0 / 3.0 + 1e-12)


# ---------------------------------------------------------------------------------------
# candidates that run on into the next block (Section 3.2.2) under the block order of Section 3.1
# ---------------------------------------------------------------------------------------
class ScriptedWindowOracle(ScriptedOracle):
    """Scripted model over a window of two blocks: ``rule(ids_row, masked_row)`` sees the rows it is given
    (one block, or current + next block) and answers (tok, conf) for them.  prefill / commit do nothing."""

    def verify_window(self, node_ids, node_masked, T, cache):
        tok, conf, gap, _ = self.verify(node_ids, node_masked, cache)
        return tok, conf, gap

    def prefill(self, prompt):
        return NoCache()

    def commit_block(self, ids, cache):
        self.committed = getattr(self, "committed", []) + [np.array(ids)]


def _stepwise_order_two_level(rule_for_block, n_blocks, B):
    """Stepwise (position, token) order over several blocks: block by block, highest confidence first."""
    order = []
    for j in range(n_blocks):
        ids = np.full(B, 999)
        masked = np.ones(B, dtype=bool)
        while masked.any():
            t, c = rule_for_block(j, ids, masked)
            q = so.best_masked_position(c, masked)
            order.append((j, q, int(t[q])))
            ids[q] = t[q]
            masked[q] = False
    return order


@pytest.mark.parametrize("w", [SMALL, SMALL_GQA], ids=lambda w: w.name)
@pytest.mark.parametrize("max_drafts", [0, 1, 2, 3, 5, 64])
def test_spill_equals_stepwise_small(w, max_drafts):
    o = make_oracle(w)
    prompt = wl.make_prompts(w)[0].numpy()
    for gen_len in (w.gen_len, w.gen_len + 3):                     # whole blocks, and a ragged last block
        a, _, _ = o.generate(prompt, gen_len, w.block_len, mode="stepwise")
        b, counts, windows = o.generate_spill(prompt, gen_len, w.block_len, max_drafts)
        assert np.array_equal(a, b)
        assert sum(counts) == gen_len and all(1 <= c <= max_drafts + 1 for c in counts)
        if max_drafts == 0:
            assert windows == 0 and counts == [1] * gen_len


def test_spill_never_accepts_into_the_next_block_before_the_current_one_is_full():
    w = SMALL_GQA
    o = make_oracle(w)
    prompt = wl.make_prompts(w)[0].numpy()
    trace = []
    o.generate_spill(prompt, w.gen_len, w.block_len, 5, trace=trace)
    T = w.block_len
    crossed = 0
    for rec in trace:
        if len(rec.ids_before) == T:
            continue                                                # single-block forward
        a = rec.last_node
        accepted = list(rec.cand[:a]) + [rec.pred[a]]
        masked = rec.masked_before.copy()
        for (p, _) in accepted:
            if p >= T:
                assert not masked[:T].any()                         # the current block was complete by then
                crossed += 1
            masked[p] = False
        # candidates: the whole current block first, then the next block
        cur_part = [p for (p, _) in rec.cand if p < T]
        assert rec.cand[:len(cur_part)] == [c for c in rec.cand if c[0] < T]
        assert len(cur_part) == int(rec.masked_before[:T].sum())
    assert crossed > 0


def test_spill_accepts_the_stepwise_continuation_across_the_boundary():
    """Scripted model whose confidences drift with the context: every forward accepts exactly 1 + the longest
    common prefix of its candidate list with the true stepwise continuation (which finishes the current
    block before it enters the next), capped by the list."""
    B, V, n_blocks, N = 6, 50, 4, 4
    rng = np.random.default_rng(2)
    toks = rng.integers(0, V - 1, (n_blocks, B))
    base = rng.random((n_blocks, B))
    drift = 0.08 * rng.random((n_blocks, B + 1, B))

    def block_rule(j, ids, masked):
        return toks[j].copy(), base[j] + drift[j, int(masked.sum())]

    state = {"j": 0}

    def rule(ids, masked):
        if len(ids) == B:
            return block_rule(state["j"], ids, masked)
        t0, c0 = block_rule(state["j"], ids[:B], masked[:B])
        t1, c1 = block_rule(state["j"] + 1, ids[B:], masked[B:])
        return np.concatenate([t0, t1]), np.concatenate([c0, c1])

    order = _stepwise_order_two_level(block_rule, n_blocks, B)

    class Tracking(ScriptedWindowOracle):
        def commit_block(self, ids, cache):
            super().commit_block(ids, cache)
            state["j"] += 1

    o = Tracking(V, rule)
    trace = []
    got, counts, windows = o.generate_spill(np.zeros(1, int), n_blocks * B, B, N, trace=trace)
    assert np.array_equal(got, toks.reshape(-1)) and windows > 0
    done = 0
    for rec in trace:
        cont = [((jj - rec.block) * B + q, t) for (jj, q, t) in order[done:]]
        lcp = 0
        while lcp < len(rec.cand) and rec.cand[lcp] == cont[lcp]:
            lcp += 1
        assert rec.accepted == lcp + 1
        done += rec.accepted
    assert done == n_blocks * B
    # with drafts that are always right a window forward accepts its whole list plus one, and the generation
    # takes fewer forwards than block-by-block chains
    fixed = ScriptedWindowOracle(V, lambda ids, masked: (np.resize(toks[0], len(ids)), np.resize(np.linspace(0.9, 0.1, B), len(ids))))
    tr_f = []
    _, counts_f, _ = fixed.generate_spill(np.zeros(1, int), n_blocks * B, B, N - 1, trace=tr_f)
    assert counts_f[0] == 1 and sum(counts_f) == n_blocks * B
    assert all(rec.accepted == len(rec.cand) + 1 for rec in tr_f)
    plain = ScriptedOracle(V, lambda ids, masked: (toks[0].copy(), np.linspace(0.9, 0.1, B)))
    n_plain = sum(len(plain.decode_block_ssd(B, NoCache(), N - 1)[1]) for _ in range(n_blocks))
    assert len(counts_f) < n_plain


def test_spill_needs_fewer_forwards_on_the_tiny_peaked_model():
    w = wl.TINY.replace(name="tiny_peaked", lm_head_scale=8.0)
    o = make_oracle(w)
    prompt = wl.make_prompts(w)[0].numpy()
    a, counts, _ = o.generate(prompt, w.gen_len, w.block_len, mode="ssd", max_drafts=3)
    b, counts_spill, windows = o.generate_spill(prompt, w.gen_len, w.block_len, 3)
    assert np.array_equal(a, b)
    assert windows > 0 and len(counts_spill) < sum(len(c) for c in counts)


# ---------------------------------------------------------------------------------------
# dual cache with a refresh interval (Section 4.1, implementation details)
# ---------------------------------------------------------------------------------------
def _uncached_full_attention_stepwise(o, prompt, gen_len, block_len):
    """Textbook masked-diffusion stepwise decoding without any cache: every step runs the model over the WHOLE
    sequence [prompt | generation with MASK], all positions seeing all positions, and unmasks the most
    confident masked position of the current block."""
    mid = o.cfg.mask_id
    P = len(prompt)
    x = np.concatenate([prompt, np.full(gen_len, mid)])
    for (lo, hi) in so.block_ranges(gen_len, block_len):
        masked = np.zeros(P + gen_len, dtype=bool)
        masked[P + lo:P + hi] = True
        while masked.any():
            logits, _, _ = o.forward_rows(x[None], 0, so.Cache(o.cfg))
            tok, conf = so.token_and_confidence(logits[0], mid)
            q = so.best_masked_position(conf, masked)
            x[q] = tok[q]
            masked[q] = False
    return x[P:]


@pytest.mark.parametrize("w", [SMALL, SMALL_GQA], ids=lambda w: w.name)
def test_dual_cache_refreshed_every_token_is_uncached_decoding(w):
    """With a refresh before every forward nothing is ever stale: the dual cache is exact and reproduces
    full-sequence decoding without a cache."""
    o = make_oracle(w)
    prompt = wl.make_prompts(w)[0].numpy()
    want = _uncached_full_attention_stepwise(o, prompt, w.gen_len, w.block_len)
    got, forwards, refreshes = o.generate_dual_cache(prompt, w.gen_len, w.block_len, refresh=1)
    assert np.array_equal(got, want)
    assert forwards == refreshes == w.gen_len


@pytest.mark.parametrize("w", [SMALL, SMALL_GQA], ids=lambda w: w.name)
@pytest.mark.parametrize("refresh", [2, 3, 4, 100])
def test_ssd_under_the_dual_cache_equals_stepwise_under_the_same_schedule(w, refresh):
    o = make_oracle(w)
    prompt = wl.make_prompts(w)[0].numpy()
    want, f0, r0 = o.generate_dual_cache(prompt, w.gen_len, w.block_len, refresh, max_drafts=0)
    assert f0 == w.gen_len
    n_blocks = -(-w.gen_len // w.block_len)
    # a refresh at every block start and after every `refresh` tokens inside a block
    assert r0 == sum(-(-(hi - lo) // refresh) for (lo, hi) in so.block_ranges(w.gen_len, w.block_len))
    for N in (1, 2, 5):
        counts = []
        got, f, r = o.generate_dual_cache(prompt, w.gen_len, w.block_len, refresh, max_drafts=N, counts_out=counts)
        assert np.array_equal(got, want)
        assert r == r0 and f <= f0 and sum(counts) == w.gen_len
        assert all(1 <= c <= min(N + 1, refresh) for c in counts)
    if refresh == 100:
        assert r0 == n_blocks


def test_dual_cache_is_an_approximation_between_refreshes():
    """Stale K/V change the model's outputs: with a long interval the confidences seen by a forward differ from
    those of exact decoding, which is why stepwise decoding is defined together with its schedule."""
    w = SMALL
    o = make_oracle(w)
    prompt = wl.make_prompts(w)[0].numpy()
    mid = w.mask_id
    x = np.concatenate([prompt, np.full(w.gen_len, mid)])
    P, T = len(prompt), w.block_len
    full = o.refresh_all(x)
    x2 = x.copy()
    x2[P] = 5                                             # one token decoded since the refresh
    fresh = o.refresh_all(x2)
    ids = x2[P:P + T]

    def block_logits(cache):
        outside = so.Cache(o.cfg)
        outside.k = [np.concatenate([k[:P], k[P + T:]], axis=0) for k in cache.k]
        outside.v = [np.concatenate([v[:P], v[P + T:]], axis=0) for v in cache.v]
        return o.forward_rows(ids[None], P, outside)[0][0]

    stale, exact = block_logits(full), block_logits(fresh)
    whole, _, _ = o.forward_rows(x2[None], 0, so.Cache(o.cfg))
    assert np.allclose(exact, whole[0][P:P + T], rtol=1e-9, atol=1e-12)      # fresh cache == no cache
    assert np.abs(stale - exact).max() > 1e-6                                 # stale suffix K/V: not the same
