"""Acceptance statistics of the sampling verify at the full c5 shape (Sec. "Verification", rejection-free
walk with one target sample per visited node).

The accepted length of a sequence has the closed-form expectation
    E = sum over non-root nodes n of prod over the path root -> n of p_parent(m)(token(m)),
with p_s the temperature softmax of the target row of slot s.  The kernels draw >= 10^4 walks (all sequences
x many seeds); their mean must match the mean of E, computed here in fp64 with library softmax, to 1 %.
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
    seeds = 80                                                         # 80 x 128 = 10240 walks
    acc = np.zeros((seeds, cfg.B))
    for s in range(seeds):
        res = u.ubt_verify_tree(tree, zd, "sample", seed=1000 + s, temperature=1.0)
        acc[s] = res.accepted_len.cpu().numpy()
    torch.cuda.synchronize()
    mean, want = acc.mean(), expect.mean()
    sem = acc.std() / math.sqrt(acc.size)
    print(f"pooled accepted length {mean:.4f}, analytic {want:.4f}, standard error {sem:.4f}")
    assert want > 0.3                                                  # the case is not trivial
    assert abs(mean - want) < 0.01 * max(want, 1.0) + 3 * sem
    # per-sequence: no sequence is off by more than 5 standard errors of its own mean
    per = acc.mean(axis=0)
    per_sem = acc.std(axis=0) / math.sqrt(seeds) + 1e-9
    assert np.all(np.abs(per - expect) < 5 * per_sem + 0.02)
