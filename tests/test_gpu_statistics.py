"""Acceptance statistics of the sampling verify at the full c5 shape (Sec. "Verification", rejection-free
walk with one target sample per visited node).

The accepted length of a sequence has the closed-form expectation
    E = sum over non-root nodes n of prod over the path root -> n of p_parent(m)(token(m)),
with p_s the temperature softmax of the target row of slot s.  The kernels draw 10^4 seeds x 128 sequences =
1.28 million walks, so that the standard error of the pooled mean is far below the bound; the mean must match the
mean of E, computed here in fp64 with library softmax, to 1 %.
"""
import math

import numpy as np
import pytest
import torch

import ubt_synth as synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_pooled_accept_length_matches_the_analytic_expectation_c5():
    import paper_2609_39972_b200 as u
    cfg = synth.CONFIGS["c5"]
    ud, bd, zd = synth.device_inputs(cfg, 21, DEV)
    tree = u.ubt_draft_tree(ud, bd, cfg.k, cfg.N)
    torch.cuda.synchronize()
    del ud, bd
    synth.boost_children_on_device(zd, tree.token_ids, tree.parents, tree.n_nodes, boost=12.0)
    tok = tree.token_ids.cpu().numpy(); par = tree.parents.cpu().numpy(); n = tree.n_nodes.cpu().numpy()

    expect = np.zeros(cfg.B)
    for b in range(cfg.B):
        p = torch.softmax(zd[b].double(), dim=-1)                      # [N, V], library softmax in fp64
        idx = np.arange(1, int(n[b]))
        edge = p[torch.as_tensor(par[b, idx], device=DEV).long(),
                 torch.as_tensor(tok[b, idx], device=DEV).long()].cpu().numpy()
        reach = np.zeros(cfg.N); reach[0] = 1.0
        for j, i in enumerate(idx):                                    # slots are ordered parent before child
            reach[i] = reach[par[b, i]] * edge[j]
        expect[b] = reach[1:].sum()
        del p
    seeds = 10_000                                                     # x 128 sequences = 1.28 million walks
    res = u.VerifyResult.empty(cfg.B, cfg.L, DEV)
    ws = u.workspace(u.ubt_verify_workspace_bytes(cfg.B, cfg.N, cfg.V, "sample"), DEV)
    tot = torch.zeros(cfg.B, dtype=torch.int64, device=DEV)
    tot2 = torch.zeros(cfg.B, dtype=torch.int64, device=DEV)
    for s in range(seeds):
        u.ubt_verify_tree(tree, zd, "sample", seed=1000 + s, temperature=1.0, result=res, ws=ws)
        a = res.accepted_len.long()
        tot += a
        tot2 += a * a
    torch.cuda.synchronize()
    tot, tot2 = tot.cpu().numpy().astype(np.float64), tot2.cpu().numpy().astype(np.float64)
    per = tot / seeds
    mean, want = per.mean(), expect.mean()
    var = tot2.sum() / (seeds * cfg.B) - mean ** 2
    sem = math.sqrt(var / (seeds * cfg.B))
    print(f"pooled accepted length {mean:.5f}, analytic {want:.5f}, standard error {sem:.5f}")
    assert want > 0.3                                                  # the case is not trivial
    assert abs(mean - want) < 0.01 * want
    # per-sequence: no sequence is off by more than 5 standard errors of its own mean
    per_sem = np.sqrt(np.maximum(tot2 / seeds - per ** 2, 0.0) / seeds) + 1e-9
    assert np.all(np.abs(per - expect) < 5 * per_sem + 0.002)
