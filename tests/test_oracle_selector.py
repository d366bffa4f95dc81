"""Pins of the oracle's selector scores (Section 3.1.2, "Parallel Computation": Delta_i = Phi_{i-1} diag(P(h_i)) Psi_i^T).

The oracle sums g[r] * phi[a][r] * psi[b][r] in a plain loop; these tests check it against the matrix form of the
paper evaluated by a library contraction, and against cases whose value is known in closed form.
"""
import numpy as np
import pytest

import oracle
import ubt_synth as synth


def _tables(V, R, B, L, seed, dtype):
    phi, psi, gate = synth.selector_tables(V, R, B, L, seed, dtype)
    f = (lambda a: synth.bf16_bits_to_f32(a)) if dtype == "bf16" else (lambda a: a)
    return phi, psi, gate, f(phi).astype(np.float64), f(psi).astype(np.float64)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_matrix_form_of_the_paper_with_a_library_contraction(dtype):
    V, R, B, L, k = 300, 48, 3, 5, 6
    phi, psi, gate, phi64, psi64 = _tables(V, R, B, L, 1, dtype)
    rng = np.random.default_rng(2)
    cand = np.stack([np.stack([rng.choice(V, k, replace=False) for _ in range(L)]) for _ in range(B)]).astype(np.int32)
    anchor = rng.integers(0, V, B).astype(np.int32)
    big, anc = oracle.selector_scores(phi, psi, gate, cand, anchor)
    for b in range(B):
        for i in range(L):
            Psi = psi64[cand[b, i]]                                   # rows psi(b')^T, b' in C_i
            Phi = phi64[[anchor[b]]] if i == 0 else phi64[cand[b, i - 1]]
            delta = Phi @ np.diag(gate[b, i].astype(np.float64)) @ Psi.T
            got = anc[b][None, :] if i == 0 else big[b, i - 1]
            np.testing.assert_allclose(got, delta, rtol=1e-12, atol=1e-12)


def test_closed_forms():
    V, R, B, L, k = 40, 8, 2, 3, 4
    cand = np.tile(np.arange(k, dtype=np.int32), (B, L, 1)) + np.arange(L, dtype=np.int32)[None, :, None] * k
    anchor = np.array([7, 9], np.int32)
    # all-ones tables: every score is the sum of the gate of the successor position
    gate = np.arange(B * L * R, dtype=np.float32).reshape(B, L, R) / 16
    ones = np.ones((V, R), np.float32)
    big, anc = oracle.selector_scores(ones, ones, gate, cand, anchor)
    for b in range(B):
        assert np.all(anc[b] == gate[b, 0].astype(np.float64).sum())
        for j in range(L - 1):
            assert np.all(big[b, j] == gate[b, j + 1].astype(np.float64).sum())
    # one-hot gate at r0 picks one column: score = phi[a][r0] * psi[b][r0]; a transposed operand or a gate
    # taken from the predecessor position would give another value
    rng = np.random.default_rng(0)
    phi = rng.integers(-4, 5, (V, R)).astype(np.float32)
    psi = rng.integers(-4, 5, (V, R)).astype(np.float32)
    gate = np.zeros((B, L, R), np.float32)
    r0 = np.array([[1, 5, 2], [3, 0, 7]])
    for b in range(B):
        for i in range(L):
            gate[b, i, r0[b, i]] = 2.0
    big, anc = oracle.selector_scores(phi, psi, gate, cand, anchor)
    for b in range(B):
        np.testing.assert_array_equal(anc[b], 2.0 * phi[anchor[b], r0[b, 0]] * psi[cand[b, 0], r0[b, 0]])
        for j in range(L - 1):
            want = 2.0 * np.outer(phi[cand[b, j], r0[b, j + 1]], psi[cand[b, j + 1], r0[b, j + 1]])
            np.testing.assert_array_equal(big[b, j], want)
    # without an anchor only the L-1 inner transitions are produced
    big2, anc2 = oracle.selector_scores(phi, psi, gate, cand)
    assert anc2 is None and np.array_equal(big2, big)


def test_scores_feed_the_tree_like_given_bigram_scores():
    # the selector's output is exactly the bigram_scores / anchor_bigram input of the tree construction
    cfg = synth.CONFIGS["c1"]
    di = synth.draft_inputs(cfg, 4)
    ids, _, _ = oracle.topk_logprob(di.unigram_logits, cfg.k)
    phi, psi, gate = synth.selector_tables(cfg.V, 16, cfg.B, cfg.L, 4, "f32")
    anchor = np.array([3], np.int32)
    big, anc = oracle.selector_scores(phi, psi, gate, ids, anchor)
    t1 = oracle.draft_tree(di.unigram_logits, big.astype(np.float32), cfg.k, cfg.N,
                           anchor_bigram=anc.astype(np.float32), anchor_tokens=anchor)
    assert int(t1.n_nodes[0]) == cfg.N and t1.token_ids[0, 0] == 3
