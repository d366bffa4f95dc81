"""Test-side helpers that belong to neither the oracle nor the CUDA path."""
from __future__ import annotations

import itertools
import math

import numpy as np


def omega_key(score, depth, token, rank, path):
    """Sort key of the total order: score desc, depth asc, token asc, rank asc, path lex."""
    return (-score, depth, token, rank, tuple(path))


def pair_logprobs(cand_lp, bigram, alpha=None, lam=None, anchor=None):
    """t[i][ra][rb] from eq. 5 + eq. 9 for ONE sequence, in float64 numpy (independent of the oracle)."""
    L, k = cand_lp.shape
    t = np.zeros((L, k, k))
    for i in range(L):
        al = 1.0 if alpha is None else float(alpha[i])
        la = 1.0 if lam is None else float(lam[i])
        for ra in range(1 if i == 0 else k):
            if i == 0:
                delta = np.zeros(k) if anchor is None else np.asarray(anchor, np.float64)
            else:
                delta = np.asarray(bigram[i - 1, ra], np.float64)
            s = al * cand_lp[i] + la * delta
            t[i, ra] = s - (s.max() + math.log(np.exp(s - s.max()).sum()))
    return t


def brute_force_tree(cand_ids, t, N, zeta=0.0):
    """Exact global Top-(N-1) over EVERY prefix, each scored directly as the sum of eq. 9 terms."""
    L, k = cand_ids.shape
    allnodes = []
    for d in range(1, L + 1):
        for path in itertools.product(range(k), repeat=d):
            score = 0.0
            prev = 0
            for i, r in enumerate(path):
                score += t[i, prev if i > 0 else 0, r]
                prev = r
            score += zeta * d
            allnodes.append((omega_key(score, d, int(cand_ids[d - 1, path[-1]]), path[-1], path), path, score))
    allnodes.sort(key=lambda e: e[0])
    return [(p, s) for _, p, s in allnodes[: N - 1]]


def algorithm1_python(cand_ids, t, N, W, zeta=0.0):
    """Second, independent statement of Algorithm 1 (depth-wise Top_W, then Top_B) in Python."""
    L, k = cand_ids.shape
    frontier = [((), 0.0)]
    S = []
    for d in range(1, L + 1):
        E = []
        for path, sc in frontier:
            prev = path[-1] if path else 0
            for r in range(k):
                E.append((path + (r,), sc + t[d - 1, prev, r] + zeta))
        E.sort(key=lambda e: omega_key(e[1], d, int(cand_ids[d - 1, e[0][-1]]), e[0][-1], e[0]))
        frontier = E[:W] if W > 0 else E
        S.extend(frontier)
    S.sort(key=lambda e: omega_key(e[1], len(e[0]), int(cand_ids[len(e[0]) - 1, e[0][-1]]), e[0][-1], e[0]))
    return S[: N - 1]


def layout_from_paths(paths_scores, cand_ids, N, anchor_token=-1, pos_offset=0):
    """Canonical slot layout (root, then depth / parent slot / rank order) from a set of rank paths."""
    paths = sorted((p for p, _ in paths_scores), key=lambda p: (len(p), p))
    score_of = {p: s for p, s in paths_scores}
    slot = {(): 0}
    mw = (N + 31) // 32
    tok = np.full(N, -1, np.int32); par = np.full(N, -1, np.int32); dep = np.full(N, -1, np.int32)
    rk = np.full(N, -1, np.int32); pos = np.full(N, -1, np.int32); sc = np.full(N, -np.inf)
    mask = np.zeros((N, mw), np.uint32)
    tok[0] = anchor_token; dep[0] = 0; pos[0] = pos_offset; sc[0] = 0.0; mask[0, 0] = 1
    # lexicographic order of rank paths inside a depth == (parent slot, rank) order
    for i, p in enumerate(paths, start=1):
        slot[p] = i
        assert p[:-1] in slot, "selection is not prefix-closed"
        tok[i] = cand_ids[len(p) - 1, p[-1]]; par[i] = slot[p[:-1]]; dep[i] = len(p); rk[i] = p[-1]
        pos[i] = pos_offset + len(p); sc[i] = score_of[p]
        mask[i] = mask[par[i]]
        mask[i, i >> 5] |= np.uint32(1 << (i & 31))
    return dict(token_ids=tok, parents=par, depths=dep, cand_rank=rk, position_ids=pos, scores=sc,
                mask=mask, n_nodes=len(paths) + 1)


def paths_of_tree(parents, cand_rank, n_nodes):
    """Rank path of every non-root slot of one sequence's tree arrays."""
    out = []
    for i in range(1, int(n_nodes)):
        p = []
        j = i
        while j > 0:
            p.append(int(cand_rank[j]))
            j = int(parents[j])
        out.append(tuple(reversed(p)))
    return out


def check_tree_invariants(tr, b, L, k, N, W=0):
    """Structural guarantees of Appendix A on sequence b of a tree-like object."""
    n = int(tr.n_nodes[b])
    tok, par, dep, rk = tr.token_ids[b], tr.parents[b], tr.depths[b], tr.cand_rank[b]
    sc, mask = tr.scores[b], tr.mask[b]
    assert 1 <= n <= N
    assert par[0] == -1 and dep[0] == 0 and rk[0] == -1 and sc[0] == 0.0
    per_depth = {}
    for i in range(1, n):
        assert 0 <= par[i] < i                       # parents precede children
        assert dep[i] == dep[par[i]] + 1             # parent depth = child depth - 1
        assert 1 <= dep[i] <= L and 0 <= rk[i] < k
        assert sc[i] <= sc[par[i]]                   # prefix monotone (normalised probs <= 1, zeta <= 0)
        per_depth[int(dep[i])] = per_depth.get(int(dep[i]), 0) + 1
    for d, c in per_depth.items():
        assert c <= k ** d
        if W > 0:
            assert c <= W
    # siblings carry distinct tokens / ranks; slots ordered by (depth, parent, rank)
    keys = [(int(dep[i]), int(par[i]), int(rk[i])) for i in range(1, n)]
    assert keys == sorted(keys) and len(set(keys)) == len(keys)
    sib = {}
    for i in range(1, n):
        assert (int(par[i]), int(tok[i])) not in sib
        sib[(int(par[i]), int(tok[i]))] = i
    # mask = reflexive ancestor closure, recomputed by walking parents
    for i in range(N):
        bits = set()
        if i < n:
            j = i
            while j >= 0:
                bits.add(j)
                j = int(par[j])
        got = {w * 32 + bit for w in range(mask.shape[1]) for bit in range(32) if (int(mask[i, w]) >> bit) & 1}
        assert got == bits, (i, got, bits)
        if i < n:
            assert len(bits) == dep[i] + 1
    for i in range(n, N):
        assert tok[i] == -1 and par[i] == -1 and dep[i] == -1 and np.isneginf(sc[i])
