"""Pins of the oracle's LM-head + candidate selection (Section 3.1.1, eq. 3: the unigram logits are the frozen
LM head applied to the proposer state) against things other than itself: a library matrix product in float64
with library sort / log-sum-exp, one-hot states (the logits are then a column of the weight table), integer
weights with a closed-form log-sum-exp, and the composition with the oracle's own selection on stored logits."""
import math

import numpy as np
import pytest
import scipy.special

import oracle
import ubt_synth as synth


def test_matches_a_library_product_sort_and_logsumexp():
    h, w = synth.lm_head_inputs(5, 96, 700, seed=3, scale=3.0)
    ids, lp, lse, logits = oracle.lm_head_topk(h, w, 6, want_logits=True)
    hf, wf = synth.bf16_bits_to_f32(h).astype(np.float64), synth.bf16_bits_to_f32(w).astype(np.float64)
    want = hf @ wf.T
    np.testing.assert_allclose(logits, want, rtol=0, atol=1e-12)
    for r in range(5):
        order = np.lexsort((np.arange(700), -want[r]))[:6]
        assert ids[r].tolist() == order.tolist()
        np.testing.assert_allclose(lse[r], scipy.special.logsumexp(want[r]), rtol=1e-13)
        np.testing.assert_allclose(lp[r], want[r, order] - scipy.special.logsumexp(want[r]), rtol=0, atol=1e-12)
        assert math.isclose(np.exp(logits[r] - lse[r]).sum(), 1.0, rel_tol=1e-12)


def test_one_hot_state_selects_a_column_of_the_table():
    rng = np.random.default_rng(1)
    V, d = 50, 16
    w = rng.integers(-8, 9, size=(V, d)).astype(np.float32)
    h = np.zeros((3, d), np.float32)
    cols = [0, 7, 15]
    for r, c in enumerate(cols):
        h[r, c] = 2.0                                  # fixes which operand is indexed by the token
    ids, lp, lse, logits = oracle.lm_head_topk(h, w, 4, want_logits=True)
    for r, c in enumerate(cols):
        assert logits[r].tolist() == (2.0 * w[:, c]).tolist()
        order = np.lexsort((np.arange(V), -2.0 * w[:, c].astype(np.float64)))[:4]
        assert ids[r].tolist() == order.tolist()       # ties (integer weights repeat) go to the lower id


def test_closed_form_row():
    # h = (1, 1), W[v] = (ln a_v, ln b_v)  =>  logit_v = ln(a_v b_v), LSE = ln sum a_v b_v
    a = np.array([1, 2, 3, 4, 5], np.float64); b = np.array([6, 1, 2, 2, 1], np.float64)
    w = np.stack([np.log(a), np.log(b)], axis=1).astype(np.float32)
    h = np.ones((1, 2), np.float32)
    ids, lp, lse, _ = oracle.lm_head_topk(h, w, 2)
    prod = np.exp(w.astype(np.float64).sum(axis=1))
    assert ids[0].tolist() == [3, 0]                   # 8 first; 6 (token 0) and 6 (token 2) tie -> token 0
    assert math.isclose(lse[0], math.log(prod.sum()), rel_tol=1e-12)
    assert math.isclose(math.exp(lp[0, 0]), prod[3] / prod.sum(), rel_tol=1e-12)


def test_composes_with_the_selection_on_stored_logits():
    h, w = synth.lm_head_inputs(4, 64, 300, seed=9, dtype="f32")
    ids, lp, lse, logits = oracle.lm_head_topk(h, w, 5, want_logits=True)
    # logits that are exactly representable in fp32 give the same selection through the stored-logits path
    q = np.round(logits * 64) / 64
    ids2, lp2, _ = oracle.topk_logprob(q.astype(np.float32), 5)
    for r in range(4):
        order = np.lexsort((np.arange(300), -q[r]))[:5]
        assert ids2[r].tolist() == order.tolist()
    assert ids.shape == (4, 5) and np.all(np.diff(lp, axis=1) <= 0)
