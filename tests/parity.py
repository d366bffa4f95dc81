"""Comparison of the CUDA path with the oracle (used by the GPU tests, the smoke check and the bench)."""
from __future__ import annotations

from types import SimpleNamespace

import numpy as np

from helpers import check_tree_invariants, layout_from_paths, paths_of_tree

SCORE_TOL = 1e-5   # |gpu - oracle| <= SCORE_TOL * max(1, |oracle|): fp32 path scores against the fp64 oracle


def tree_to_numpy(tree) -> SimpleNamespace:
    """Host copy of a binding.Tree."""
    f = lambda t: t.detach().cpu().numpy()
    return SimpleNamespace(token_ids=f(tree.token_ids), parents=f(tree.parents), depths=f(tree.depths),
                           position_ids=f(tree.position_ids), cand_rank=f(tree.cand_rank),
                           scores=f(tree.scores).astype(np.float64), mask=f(tree.mask).view(np.uint32),
                           n_nodes=f(tree.n_nodes), cand_ids=f(tree.cand_ids),
                           cand_lp=f(tree.cand_logprob).astype(np.float64))


def close(a, b, tol=SCORE_TOL):
    a = np.asarray(a, np.float64); b = np.asarray(b, np.float64)
    both_inf = np.isinf(a) & np.isinf(b) & (np.sign(a) == np.sign(b))
    with np.errstate(invalid="ignore"):
        ok = np.abs(a - b) <= tol * np.maximum(1.0, np.abs(b))
    return bool(np.all(ok | both_inf))


def compare_draft(g, o, L, k, N, W=0, zeta=0.0, anchor_tokens=None, pos_offset=None, rows=None):
    """GPU tree ``g`` (tree_to_numpy) against oracle tree ``o``; returns the list of logged near-tie swaps.

    Candidates must match exactly (ids) and within SCORE_TOL (log-probs).  If the node sets agree every
    integer array must be bit-exact.  The only divergence allowed is, for an unbounded width, nodes of the
    symmetric difference whose oracle scores lie within SCORE_TOL of the oracle's cut-off score; then the GPU
    arrays must still be exactly the canonical layout of the GPU's own node set.
    """
    swaps = []
    B = len(g.n_nodes) if rows is None else len(rows)
    for bi in range(B):
        b = bi if rows is None else rows[bi]      # b indexes the GPU batch, bi the oracle sample
        assert g.cand_ids[b].tolist() == o.cand_ids[bi].tolist(), f"candidate ids differ in sequence {b}"
        assert close(g.cand_lp[b], o.cand_lp[bi]), f"candidate log-probs differ in sequence {b}"
        gv = SimpleNamespace(**{n: getattr(g, n)[b:b + 1] for n in
                                ("token_ids", "parents", "depths", "cand_rank", "scores", "mask", "n_nodes")})
        check_tree_invariants(gv, 0, L, k, N, W)
        gp = paths_of_tree(g.parents[b], g.cand_rank[b], g.n_nodes[b])
        op = paths_of_tree(o.parents[bi], o.cand_rank[bi], o.n_nodes[bi])
        if set(gp) == set(op):
            for name in ("token_ids", "parents", "depths", "cand_rank", "position_ids", "mask"):
                assert getattr(g, name)[b].tolist() == getattr(o, name)[bi].tolist(), (name, b)
            assert g.n_nodes[b] == o.n_nodes[bi]
            assert close(g.scores[b], o.scores[bi]), f"scores differ in sequence {b}"
            continue
        # node sets differ: only near-ties at the budget cut of an unbounded search are tolerated
        assert W == 0 or W >= N - 1, f"sequence {b}: node set differs under a finite width"
        assert len(gp) == len(op), f"sequence {b}: node count differs"
        t = o.t[bi]
        def oscore(p):
            s, prev = 0.0, 0
            for i, r in enumerate(p):
                s += t[i, prev if i else 0, r]; prev = r
            return s + zeta * len(p)
        cut = min(o.scores[bi, 1:o.n_nodes[bi]])
        for p in set(gp) ^ set(op):
            d = abs(oscore(p) - cut)
            assert d <= SCORE_TOL * max(1.0, abs(cut)), f"sequence {b}: node {p} differs by {d} from the cut-off"
            swaps.append((b, p, oscore(p) - cut))
        want = layout_from_paths([(p, oscore(p)) for p in gp], o.cand_ids[bi], N,
                                 -1 if anchor_tokens is None else int(anchor_tokens[b]),
                                 0 if pos_offset is None else int(pos_offset[b]))
        for name in ("token_ids", "parents", "depths", "cand_rank", "position_ids", "mask"):
            assert getattr(g, name)[b].tolist() == want[name].tolist(), (name, b, "after swap")
        assert close(g.scores[b], want["scores"])
    return swaps


def compare_verify(res, ov, node_pick=None, rows=None):
    """binding.VerifyResult against an oracle Verdict, bit-exact."""
    f = lambda t: t.detach().cpu().numpy()
    sel = slice(None) if rows is None else rows
    assert f(res.accepted_len)[sel].tolist() == ov.accepted_len.tolist(), "accepted_len"
    assert f(res.bonus_token)[sel].tolist() == ov.bonus_token.tolist(), "bonus_token"
    assert f(res.accepted_nodes)[sel].tolist() == ov.accepted_nodes.tolist(), "accepted_nodes"
    assert f(res.out_tokens)[sel].tolist() == ov.out_tokens.tolist(), "out_tokens"
    if node_pick is not None and ov.node_pick is not None:
        assert f(node_pick)[sel].tolist() == ov.node_pick.tolist(), "node_pick"
