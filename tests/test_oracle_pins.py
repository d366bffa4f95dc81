"""Pins of the CPU oracle to things other than itself (no GPU needed).

Each test checks the oracle against what the paper or the mathematics fixes:
brute force over every prefix scored straight from eq. 9, exact rational
arithmetic on a hand-worked example, library routines, published known-answer
vectors, structural guarantees of Appendix A, and analytic acceptance
statistics.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import scipy.special

import oracle
import ubt_synth as synth
from helpers import (algorithm1_python, brute_force_tree, check_tree_invariants, layout_from_paths,
                     pair_logprobs, paths_of_tree)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ Philox
def test_philox_known_answers():
    with open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) as f:
        rows = [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        w = [int(x, 16) for x in r]
        got = oracle.philox4x32_10(w[0:4], w[4:6])
        assert [int(x) for x in got] == w[6:10]


def test_threshold_is_mulhi_of_first_two_words():
    rng = np.random.default_rng(1)
    for _ in range(50):
        seed = int(rng.integers(0, 2**63)); b = int(rng.integers(0, 1000)); n = int(rng.integers(0, 256))
        total = int(rng.integers(1, 2**58))
        x = oracle.philox4x32_10([n, b, 0, 0], [seed & 0xFFFFFFFF, seed >> 32])
        r = int(x[0]) | (int(x[1]) << 32)
        assert oracle.threshold(seed, b, n, total) == (r * total) >> 64      # Python big integers
        assert 0 <= oracle.threshold(seed, b, n, total) < total


# ------------------------------------------------------------------ step 1
def _rows_with_ties(rng, rows, V, dtype):
    x = rng.standard_normal((rows, V)).astype(np.float32) * 3
    x[0, :] = 1.25                                   # a constant row: every element ties
    x[1, ::7] = x[1].max()                           # many copies of the maximum
    x[2, 5] = 0.0; x[2, 9] = -0.0                    # +0 and -0 are equal
    x[2, x[2] > 0] *= -1                             # ... and they are the row maximum
    x[3] = np.round(x[3])                            # heavy quantisation
    return synth.f32_to_bf16_bits(x) if dtype == "bf16" else x


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("k", [1, 4, 13])
def test_topk_matches_full_stable_sort(dtype, k):
    rng = np.random.default_rng(7)
    x = _rows_with_ties(rng, 6, 997, dtype)
    ids, lp, lse = oracle.topk_logprob(x, k)
    xf = synth.as_f32(x, dtype).astype(np.float64)
    for r in range(x.shape[0]):
        # library: lexsort by (id asc) within (value desc); -0.0 == +0.0 numerically
        order = np.lexsort((np.arange(xf.shape[1]), -xf[r]))
        assert ids[r].tolist() == order[:k].tolist()
        np.testing.assert_allclose(lse[r], scipy.special.logsumexp(xf[r]), rtol=1e-13)
        np.testing.assert_allclose(lp[r], xf[r, order[:k]] - scipy.special.logsumexp(xf[r]), rtol=1e-12, atol=1e-12)


def test_lse_closed_form_integer_weights():
    # logits = ln(w) with integer w  =>  LSE = ln(sum w), lp = ln(w / sum w)
    w = np.array([[1, 10, 1, 5, 2, 1], [6, 1, 1, 1, 6, 5], [2, 2, 9, 1, 3, 3]], np.float64)
    x = np.log(w).astype(np.float32)
    ids, lp, lse = oracle.topk_logprob(x, 2)
    np.testing.assert_allclose(lse, np.log(20.0), rtol=1e-7)
    assert ids.tolist() == [[1, 3], [0, 4], [2, 4]]          # ties (6,6) and (3,3) -> lower id
    np.testing.assert_allclose(np.exp(lp), [[0.5, 0.25], [0.3, 0.3], [0.45, 0.15]], rtol=1e-6)


def test_logprobs_sum_to_one_over_vocabulary():
    rng = np.random.default_rng(3)
    x = (rng.standard_normal((3, 500)) * 4).astype(np.float32)
    _, lp, _ = oracle.topk_logprob(x, 500)
    np.testing.assert_allclose(np.exp(lp).sum(-1), 1.0, rtol=1e-12)


# ------------------------------------------------------------------ hand-worked example
def _example_e1():
    u = np.log(np.array([[1, 10, 1, 5, 2, 1], [6, 1, 1, 1, 6, 5], [2, 2, 9, 1, 3, 3]], np.float64)).astype(np.float32)
    big = np.log(np.array([[[1, 3], [2, 1]], [[1, 1], [2, 9]]], np.float64)).astype(np.float32)
    return u[None], big[None]


def _exact_rational_paths():
    """Path probabilities of example E1 in exact rationals (eq. 5, 9 with alpha = lambda = 1)."""
    q = [[Fraction(10, 20), Fraction(5, 20)], [Fraction(6, 20), Fraction(6, 20)], [Fraction(9, 20), Fraction(3, 20)]]
    toks = [[1, 3], [0, 4], [2, 4]]
    delta = [None, [[1, 3], [2, 1]], [[1, 1], [2, 9]]]
    out = {}
    def rec(path, prob):
        d = len(path)
        if d == 3:
            return
        ra = path[-1] if path else 0
        w = [q[d][rb] * (delta[d][ra][rb] if d > 0 else 1) for rb in range(2)]
        for rb in range(2):
            p = prob * w[rb] / sum(w)
            out[path + (rb,)] = p
            rec(path + (rb,), p)
    rec((), Fraction(1))
    return out, toks


def test_hand_worked_example_exact_rationals():
    u, big = _example_e1()
    probs, toks = _exact_rational_paths()
    # the five best prefixes, derived by hand: 2/3, 1/2, 1/3, 3/10, 2/9, then the cut at 1/5
    ranked = sorted(probs.items(), key=lambda e: (-e[1], len(e[0]), toks[len(e[0]) - 1][e[0][-1]]))
    assert [p for _, p in ranked[:6]] == [Fraction(2, 3), Fraction(1, 2), Fraction(1, 3), Fraction(3, 10),
                                          Fraction(2, 9), Fraction(1, 5)]
    tr = oracle.draft_tree(u, big, k=2, N=6)
    assert tr.n_nodes.tolist() == [6]
    assert tr.token_ids[0].tolist() == [-1, 1, 3, 4, 0, 4]
    assert tr.parents[0].tolist() == [-1, 0, 0, 1, 2, 3]
    assert tr.depths[0].tolist() == [0, 1, 1, 2, 2, 3]
    assert tr.cand_rank[0].tolist() == [-1, 0, 1, 1, 0, 1]
    assert tr.position_ids[0].tolist() == [0, 1, 1, 2, 2, 3]
    assert tr.mask[0, :, 0].tolist() == [0x01, 0x03, 0x05, 0x0B, 0x15, 0x2B]
    want = [1, Fraction(2, 3), Fraction(1, 3), Fraction(1, 2), Fraction(2, 9), Fraction(3, 10)]
    np.testing.assert_allclose(np.exp(tr.scores[0]), [float(x) for x in want], rtol=2e-7)
    # W = 1: the single greedy chain 1 -> 4 -> 4 with probabilities 2/3, 1/2, 3/10
    tr1 = oracle.draft_tree(u, big, k=2, N=6, W=1)
    assert tr1.n_nodes.tolist() == [4] and tr1.token_ids[0, :4].tolist() == [-1, 1, 4, 4]
    np.testing.assert_allclose(np.exp(tr1.scores[0, 1:4]), [2 / 3, 1 / 2, 3 / 10], rtol=2e-7)
    # W = 2 keeps the same five nodes as the unbounded search
    tr2 = oracle.draft_tree(u, big, k=2, N=6, W=2)
    assert tr2.token_ids.tolist() == tr.token_ids.tolist() and tr2.parents.tolist() == tr.parents.tolist()


def test_hand_worked_verify_example():
    u, big = _example_e1()
    tr = oracle.draft_tree(u, big, k=2, N=6)
    z = np.log(np.array([[1, 12, 1, 4, 1, 1], [2, 1, 1, 1, 14, 1], [5, 5, 4, 2, 2, 2], [1, 1, 10, 1, 5, 2],
                         [1, 1, 1, 1, 1, 15], [3, 3, 3, 3, 4, 4]], np.float64)).astype(np.float32)[None]
    v = oracle.verify(tr.token_ids, tr.parents, tr.n_nodes, 3, z, "greedy")
    assert v.node_pick[0].tolist() == [1, 4, 0, 2, 5, 4]          # node 2: the 5,5 tie -> token 0
    assert v.accepted_len.tolist() == [2] and v.bonus_token.tolist() == [2]
    assert v.accepted_nodes[0].tolist() == [0, 1, 3, -1] and v.out_tokens[0].tolist() == [1, 4, 2, -1]
    # sampling at T = 1: E[len] = .6 + .2 + .6*.7 + .2*.25 + .6*.7*.25 = 1.375, P(len) = .2 .33 .365 .105
    cdf = np.stack([oracle.row_cdf(z[0], n) for n in range(6)])
    seeds = np.arange(200_000, dtype=np.uint64)
    acc, bonus = oracle.walks_from_cdf(tr.token_ids[0], tr.parents[0], 6, cdf, 0, seeds)
    freq = np.bincount(acc, minlength=4) / len(seeds)
    np.testing.assert_allclose(freq, [0.2, 0.33, 0.365, 0.105], atol=4e-3)
    assert abs(acc.mean() - 1.375) < 0.01
    # the lazy walk and the all-rows walk agree, and agree with the CDF walk
    for s in range(20):
        a = oracle.verify(tr.token_ids, tr.parents, tr.n_nodes, 3, z, "sample", seed=s, all_nodes=True)
        bb = oracle.verify(tr.token_ids, tr.parents, tr.n_nodes, 3, z, "sample", seed=s, all_nodes=False)
        assert a.accepted_len[0] == bb.accepted_len[0] == acc[s] and a.bonus_token[0] == bb.bonus_token[0] == bonus[s]


# ------------------------------------------------------------------ steps 2-3
def _small_case(seed, L, k, V=50, B=2, bigram_std=1.0, quantise=False):
    rng = np.random.default_rng(seed)
    u = (rng.standard_normal((B, L, V)) * rng.uniform(0.5, 4, (B, L, 1))).astype(np.float32)
    big = (rng.standard_normal((B, L - 1, k, k)) * bigram_std).astype(np.float32)
    if quantise:                                      # force exact score ties
        u = np.round(u); big = np.round(big)
    return u, big


@pytest.mark.parametrize("seed,L,k,N", [(0, 4, 4, 16), (1, 3, 3, 8), (2, 5, 2, 20), (3, 4, 3, 200), (4, 2, 5, 31)])
def test_unbounded_width_equals_brute_force_over_all_prefixes(seed, L, k, N):
    u, big = _small_case(seed, L, k)
    ids, lp, _ = oracle.topk_logprob(u, k)
    tr = oracle.build_tree(ids, lp, big, N)
    for b in range(u.shape[0]):
        t = pair_logprobs(lp[b], big[b])
        np.testing.assert_allclose(tr.t[b, 0, 0], t[0, 0], rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(tr.t[b, 1:], t[1:], rtol=1e-12, atol=1e-12)
        want = layout_from_paths(brute_force_tree(ids[b], t, N), ids[b], N)
        assert tr.n_nodes[b] == want["n_nodes"]
        for name in ("token_ids", "parents", "depths", "cand_rank", "position_ids", "mask"):
            assert getattr(tr, name)[b].tolist() == want[name].tolist(), name
        np.testing.assert_allclose(tr.scores[b], want["scores"], rtol=1e-12, atol=1e-12)
        check_tree_invariants(tr, b, L, k, N)
    # any width >= N - 1 gives the same tree as the unbounded search
    trw = oracle.build_tree(ids, lp, big, N, W=max(N - 1, 1))
    assert trw.token_ids.tolist() == tr.token_ids.tolist() and trw.parents.tolist() == tr.parents.tolist()


@pytest.mark.parametrize("seed", [10, 11, 12])
def test_exact_ties_follow_the_total_order(seed):
    # rounded inputs with lambda = 0 make many scores EXACTLY equal (same sums in another order)
    u, big = _small_case(seed, 4, 3, quantise=True)
    ids, lp, _ = oracle.topk_logprob(u, 3)
    lam = np.zeros(4, np.float32)
    tr = oracle.build_tree(ids, lp, big, 12, lam=lam)
    for b in range(u.shape[0]):
        t = pair_logprobs(lp[b], big[b], lam=lam)
        want = layout_from_paths(brute_force_tree(ids[b], t, 12), ids[b], 12)
        assert tr.token_ids[b].tolist() == want["token_ids"].tolist()
        assert tr.parents[b].tolist() == want["parents"].tolist()


@pytest.mark.parametrize("W", [1, 2, 3, 5])
@pytest.mark.parametrize("zeta", [0.0, -0.3])
def test_finite_width_matches_second_statement_of_algorithm_1(W, zeta):
    u, big = _small_case(21, 5, 4, B=3)
    ids, lp, _ = oracle.topk_logprob(u, 4)
    N = 14
    tr = oracle.build_tree(ids, lp, big, N, W=W, zeta=zeta)
    for b in range(3):
        t = pair_logprobs(lp[b], big[b])
        want = layout_from_paths(algorithm1_python(ids[b], t, N, W, zeta), ids[b], N)
        assert tr.token_ids[b].tolist() == want["token_ids"].tolist()
        assert tr.parents[b].tolist() == want["parents"].tolist()
        np.testing.assert_allclose(tr.scores[b], want["scores"], rtol=1e-12, atol=1e-12)
        check_tree_invariants(tr, b, 5, 4, N, W=W)


def test_width_one_is_the_greedy_chain_on_combined_scores():
    # DFlash-2 style single chain (Section 2): r_d = argmax_r t[d, r_{d-1}, r]
    u, big = _small_case(5, 6, 4, B=3)
    ids, lp, _ = oracle.topk_logprob(u, 4)
    tr = oracle.build_tree(ids, lp, big, 10, W=1)
    for b in range(3):
        t = pair_logprobs(lp[b], big[b])
        prev, chain = 0, []
        for d in range(6):
            r = int(np.argmax(t[d, prev])); chain.append(int(ids[b, d, r])); prev = r
        assert tr.n_nodes[b] == 7
        assert tr.token_ids[b, 1:7].tolist() == chain
        assert tr.parents[b, :7].tolist() == [-1, 0, 1, 2, 3, 4, 5]


def test_lambda_zero_is_best_first_over_positionwise_logprobs():
    # DDTree special case (Section 2): score = sum_d of the renormalised unigram log-probabilities
    u, big = _small_case(6, 4, 3, B=2)
    ids, lp, _ = oracle.topk_logprob(u, 3)
    tr = oracle.build_tree(ids, lp, big, 9, lam=np.zeros(4, np.float32))
    for b in range(2):
        ren = lp[b] - scipy.special.logsumexp(lp[b], axis=1, keepdims=True)
        for i in range(1, int(tr.n_nodes[b])):
            path = paths_of_tree(tr.parents[b], tr.cand_rank[b], tr.n_nodes[b])[i - 1]
            np.testing.assert_allclose(tr.scores[b, i], sum(ren[d, r] for d, r in enumerate(path)), rtol=1e-12)


def test_single_candidate_gives_a_chain_and_prefers_ancestors():
    # k = 1: every normalised probability is 1, every score is exactly 0, all ties ->
    # ancestors first, so the tree is the chain of min(L, N-1) nodes
    u, _ = _small_case(7, 6, 1)
    big = np.zeros((2, 5, 1, 1), np.float32)
    for N, want in ((4, 4), (7, 7), (20, 7)):
        tr = oracle.draft_tree(u, big, 1, N)
        assert tr.n_nodes.tolist() == [want, want]
        assert tr.parents[0, :want].tolist() == list(range(-1, want - 1))
        assert np.all(tr.scores[0, :want] == 0.0)


def test_shift_invariance_of_the_tree():
    # adding a constant to a logits row, or to a row bigram[b,j,ra,:], is cancelled by eq. 9
    u, big = _small_case(8, 4, 4)
    base = oracle.draft_tree(u, big, 4, 16)
    u2 = u.copy(); u2[:, 1] += 3.0
    big2 = big.copy(); big2[:, 2, 1, :] -= 5.0
    other = oracle.draft_tree(u2, big2, 4, 16)
    assert other.token_ids.tolist() == base.token_ids.tolist()
    assert other.parents.tolist() == base.parents.tolist()
    np.testing.assert_allclose(other.scores, base.scores, rtol=1e-5, atol=1e-5)


def test_pair_logprobs_are_normalised_and_nonpositive():
    u, big = _small_case(9, 5, 6, bigram_std=2.0)
    tr = oracle.draft_tree(u, big, 6, 8)
    assert np.all(tr.t <= 0.0)
    np.testing.assert_allclose(np.exp(tr.t[:, 1:]).sum(-1), 1.0, rtol=1e-12)
    np.testing.assert_allclose(np.exp(tr.t[:, 0, 0]).sum(-1), 1.0, rtol=1e-12)


def test_options_alpha_lambda_anchor_offsets():
    u, big = _small_case(13, 3, 3, B=2)
    ids, lp, _ = oracle.topk_logprob(u, 3)
    rng = np.random.default_rng(0)
    alpha = rng.uniform(0.5, 2, 3).astype(np.float32); lam = rng.uniform(0.5, 2, 3).astype(np.float32)
    anchor = rng.standard_normal((2, 3)).astype(np.float32)
    tr = oracle.build_tree(ids, lp, big, 10, alpha=alpha, lam=lam, anchor_bigram=anchor,
                           anchor_tokens=np.array([11, 22]), pos_offset=np.array([100, 2000]))
    for b in range(2):
        t = pair_logprobs(lp[b], big[b], alpha, lam, anchor[b])
        want = layout_from_paths(brute_force_tree(ids[b], t, 10), ids[b], 10, [11, 22][b], [100, 2000][b])
        for name in ("token_ids", "parents", "position_ids"):
            assert getattr(tr, name)[b].tolist() == want[name].tolist(), name


def test_counts_and_invariants_on_the_tiny_config():
    cfg = synth.CONFIGS["c1"]
    di = synth.draft_inputs(cfg, seed=0)
    tr = oracle.draft_tree(di.unigram_logits, di.bigram_scores, cfg.k, cfg.N)
    check_tree_invariants(tr, 0, cfg.L, cfg.k, cfg.N)
    assert tr.n_nodes[0] == 16                                 # 340 prefixes >> 15 slots
    assert tr.mask.shape == (1, 16, 1)


def test_wide_budget_mask_has_256_bits_per_node():
    rng = np.random.default_rng(5)
    u = (rng.standard_normal((1, 8, 300)) * 1.5).astype(np.float32)
    big = (rng.standard_normal((1, 7, 6, 6)) * 2).astype(np.float32)
    tr = oracle.draft_tree(u, big, 6, 256)
    assert tr.mask.shape == (1, 256, 8) and tr.n_nodes[0] == 256
    check_tree_invariants(tr, 0, 8, 6, 256)
    # optimality certificate: no unselected child of a selected node beats the worst selected node
    sel = set(paths_of_tree(tr.parents[0], tr.cand_rank[0], 256)) | {()}
    worst = tr.scores[0, 1:256].min()
    score_of = {(): 0.0}
    for i, p in enumerate(paths_of_tree(tr.parents[0], tr.cand_rank[0], 256), start=1):
        score_of[p] = tr.scores[0, i]
    for p in sel:
        if len(p) == 8:
            continue
        for r in range(6):
            if p + (r,) not in sel:
                assert score_of[p] + tr.t[0, len(p), p[-1] if p else 0, r] <= worst


# ------------------------------------------------------------------ step 4
def test_greedy_pick_is_library_argmax_and_planted_path_is_found():
    cfg = synth.CONFIGS["c1"]
    for seed in range(6):
        di = synth.draft_inputs(cfg, seed)
        tr = oracle.draft_tree(di.unigram_logits, di.bigram_scores, cfg.k, cfg.N)
        z = synth.target_logits(cfg, seed)
        ends = synth.plant_path(z, cfg.dtype, tr.token_ids, tr.parents, tr.n_nodes, seed)
        v = oracle.verify(tr.token_ids, tr.parents, tr.n_nodes, cfg.L, z, "greedy")
        assert v.node_pick.tolist() == np.argmax(z, -1).tolist()         # np.argmax: first maximum
        assert v.accepted_len[0] == tr.depths[0, ends[0]]
        assert v.accepted_nodes[0, v.accepted_len[0]] == ends[0]
        assert 1 <= v.accepted_len[0] + 1 <= cfg.L + 1                   # tau in [1, gamma + 1]
        lazy = oracle.verify(tr.token_ids, tr.parents, tr.n_nodes, cfg.L, z, "greedy", all_nodes=False)
        assert lazy.accepted_len.tolist() == v.accepted_len.tolist()
        assert lazy.out_tokens.tolist() == v.out_tokens.tolist()


def test_walk_on_given_picks_hand_worked_and_consistent_with_verify():
    # (a) the hand-worked fixture
    par = np.array([[-1, 0, 0, 1, 1, 3]], np.int32)
    tok = np.array([[-1, 5, 7, 9, 2, 4]], np.int32)
    nn = np.array([6], np.int32)
    with open(os.path.join(GOLDEN, "walk_worked_example.txt")) as f:
        rows = [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 6
    for r in rows:
        picks = np.array([[int(x) for x in r[:6]]], np.int32)
        want_len, want_slots, want_tok = int(r[6]), [int(x) for x in r[7].split(",")], [int(x) for x in r[8].split(",")]
        v = oracle.verify_picks(tok, par, nn, 3, picks)
        assert v.accepted_len[0] == want_len
        assert v.accepted_nodes[0].tolist() == want_slots + [-1] * (4 - len(want_slots))
        assert v.out_tokens[0].tolist() == want_tok + [-1] * (4 - len(want_tok))
        assert v.bonus_token[0] == want_tok[-1]
    # a slot beyond n_nodes never matches, whatever it holds
    v = oracle.verify_picks(tok, par, np.array([3], np.int32), 3, np.array([[5, 9, 0, 4, 0, 8]], np.int32))
    assert v.accepted_len[0] == 1 and v.bonus_token[0] == 9
    # (b) on drafted trees: the walk on the picks of the full verification is that verification
    cfg = synth.CONFIGS["c1"]
    for seed in range(4):
        di = synth.draft_inputs(cfg, seed)
        tr = oracle.draft_tree(di.unigram_logits, di.bigram_scores, cfg.k, cfg.N)
        z = synth.target_logits(cfg, seed)
        synth.plant_path(z, cfg.dtype, tr.token_ids, tr.parents, tr.n_nodes, seed)
        for mode in ("greedy", "sample"):
            full = oracle.verify(tr.token_ids, tr.parents, tr.n_nodes, cfg.L, z, mode, seed=seed)
            w = oracle.verify_picks(tr.token_ids, tr.parents, tr.n_nodes, cfg.L, full.node_pick)
            for name in ("accepted_len", "accepted_nodes", "out_tokens", "bonus_token"):
                assert getattr(w, name).tolist() == getattr(full, name).tolist()


def test_weight_routine_against_double_exp():
    rng = np.random.default_rng(2)
    for T in (1.0, 0.7, 2.5):
        m = np.float32(rng.uniform(-20, 30))
        a, c = oracle.weight_consts(float(m), T)
        assert a == np.float32(np.float32(1.4426950408889634) * (np.float32(1) / np.float32(T)))
        z = (m - np.abs(rng.standard_normal(4000) * 6)).astype(np.float32)
        z[0] = m
        w = np.array([oracle.weight(float(x), a, c) for x in z], np.float64)
        exact = np.exp((z.astype(np.float64) - np.float64(m)) / T) * 2.0**40
        big = exact > 2.0**16
        np.testing.assert_allclose(w[big], exact[big], rtol=2e-5)         # c rounds once per row (common factor)
        large = exact > 2.0**24                                           # truncation below 6e-8 there
        ratio = w[large] / exact[large]
        assert ratio.max() / ratio.min() - 1 < 3e-6                       # per-element error: polynomial + fl32(a)
        assert np.all(np.abs(w - exact) <= exact * 2e-5 + 1.0)            # truncation loses < 1 unit
        assert oracle.weight(float(m) - 200.0, a, c) == 0


def test_sampling_distribution_matches_softmax_small_vocabulary():
    # losslessness: the first committed token is distributed as softmax(z_root / T)
    rng = np.random.default_rng(4)
    V = 12
    z = (rng.standard_normal((1, 1, V)) * 2).astype(np.float32)
    for T in (1.0, 0.5):
        cdf = oracle.row_cdf(z[0], 0, T)[None]
        seeds = np.arange(120_000, dtype=np.uint64)
        tok = np.zeros(1, np.int32) - 1; par = np.zeros(1, np.int32) - 1
        _, bonus = oracle.walks_from_cdf(tok, par, 1, cdf, 0, seeds)
        p = scipy.special.softmax(z[0, 0].astype(np.float64) / T)
        obs = np.bincount(bonus, minlength=V)
        chi2 = ((obs - p * len(seeds)) ** 2 / (p * len(seeds))).sum()
        assert chi2 < 40.0                                                # 11 dof: P(chi2 > 40) ~ 4e-5


def test_row_cdf_is_the_running_sum_of_weights():
    rng = np.random.default_rng(8)
    z = synth.f32_to_bf16_bits((rng.standard_normal((2, 3, 700)) * 3).astype(np.float32))
    pre = oracle.row_cdf(z.reshape(-1, 700), 4, 1.0)
    zf = synth.bf16_bits_to_f32(z.reshape(-1, 700)[4])
    a, c = oracle.weight_consts(float(zf.max()), 1.0)
    w = [oracle.weight(float(x), a, c) for x in zf]
    assert pre.tolist() == list(np.cumsum(np.array(w, dtype=object)))
    v = oracle.verify(np.full((2, 3), -1, np.int32), np.full((2, 3), -1, np.int32), np.ones(2, np.int32), 2, z,
                      "sample", seed=99)
    for b in range(2):
        for n in range(3):
            pre = oracle.row_cdf(z.reshape(-1, 700), b * 3 + n, 1.0)
            theta = oracle.threshold(99, b, n, int(pre[-1]))
            assert v.node_pick[b, n] == int(np.searchsorted(pre, theta, side="right"))


def test_analytic_acceptance_expectation_on_agreeing_targets():
    # E[accepted_len] = sum over non-root nodes of prod_{m on root->n} p_parent(m)(token(m))
    cfg = synth.CONFIGS["c1"].replace(V=64)
    di = synth.draft_inputs(cfg, 3)
    tr = oracle.draft_tree(di.unigram_logits, di.bigram_scores, cfg.k, cfg.N)
    z = synth.agree_targets(cfg, di.unigram_logits, tr.token_ids, tr.parents, tr.depths, tr.n_nodes, 3)
    p = scipy.special.softmax(z[0].astype(np.float64), axis=-1)
    reach = np.zeros(cfg.N); reach[0] = 1.0
    for i in range(1, int(tr.n_nodes[0])):
        reach[i] = reach[tr.parents[0, i]] * p[tr.parents[0, i], tr.token_ids[0, i]]
    expect = reach[1:].sum()
    cdf = np.stack([oracle.row_cdf(z[0], n) for n in range(cfg.N)])
    acc, _ = oracle.walks_from_cdf(tr.token_ids[0], tr.parents[0], int(tr.n_nodes[0]), cdf, 0,
                                   np.arange(100_000, dtype=np.uint64))
    assert expect > 0.3
    assert abs(acc.mean() - expect) < 0.01 * max(expect, 1.0) + 3 * acc.std() / math.sqrt(len(acc))
