"""Stream order of the verify calls: calls enqueued one after the other on one stream, sharing one scratch
area and never synchronised in between, must each give the oracle's verdict.

The V-wide kernels are launched so that they become resident behind the kernel in front of them; what keeps a
call from overwriting scratch that the call in front still reads is (by default) a wait at the top of those
kernels and, for calls that opted into an early start, the point at which the walk kernel releases the kernel
behind it.  The shapes cut the logits so that some CTA's first row segment is only a few KB: its first key is
written microseconds after the kernel starts, which is when a missing order would show.
"""
import numpy as np
import pytest
import torch

import oracle
import ubt_synth as synth
from parity import compare_verify, tree_to_numpy

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
REPS = 200


def _case(cfg, seed):
    """A drafted tree, target logits with a planted path, and the oracle's verdicts (greedy and sampled)."""
    import paper_2609_39972_b200 as u
    di = synth.draft_inputs(cfg, seed)
    tree = u.ubt_draft_tree(synth.to_device(di.unigram_logits, cfg.dtype, DEV),
                            torch.from_numpy(di.bigram_scores).to(DEV), cfg.k, cfg.N)
    torch.cuda.synchronize()
    g = tree_to_numpy(tree)
    z = synth.target_logits(cfg, seed)
    synth.plant_path(z, cfg.dtype, g.token_ids, g.parents, g.n_nodes, seed)
    want = {m: oracle.verify(g.token_ids, g.parents, g.n_nodes, cfg.L, z, m, seed=7) for m in ("greedy", "sample")}
    return tree, synth.to_device(z, cfg.dtype, DEV), want


def _results(u, cfg, n):
    out = []
    for _ in range(n):
        r = u.VerifyResult.empty(cfg.B, cfg.L, DEV)
        for t in (r.accepted_len, r.bonus_token, r.accepted_nodes, r.out_tokens):
            t.fill_(-9)
        out.append(r)
    return out


# V = 32768 + 2048: with the minimum span of 32768 elements the second CTA starts 2048 elements (4 KB of bf16)
# before the end of row 0
SHAPE = dict(B=2, L=6, N=24, k=4, V=34816)


@pytest.mark.parametrize("mode", ["greedy", "sample"])
@pytest.mark.parametrize("early", [False, True])
def test_verify_calls_queued_on_one_stream_share_one_workspace(mode, early):
    import paper_2609_39972_b200 as u
    cfg = synth.CONFIGS["c2"].replace(**SHAPE)
    (ta, za, wa), (tb, zb, wb) = _case(cfg, 31), _case(cfg, 32)
    assert wa[mode].out_tokens.tolist() != wb[mode].out_tokens.tolist()
    ws = u.workspace(u.ubt_verify_workspace_bytes(cfg.B, cfg.N, cfg.V, mode), DEV)
    ra, rb = _results(u, cfg, REPS), _results(u, cfg, REPS)
    pa = [torch.full((cfg.B, cfg.N), -9, dtype=torch.int32, device=DEV) for _ in range(REPS)]
    torch.cuda.synchronize()
    for i in range(REPS):                      # A, B, A, B, ... with nothing in between
        u.ubt_verify_tree(ta, za, mode, seed=7, result=ra[i], ws=ws, node_pick=pa[i], early_start=early)
        u.ubt_verify_tree(tb, zb, mode, seed=7, result=rb[i], ws=ws, early_start=early)
    torch.cuda.synchronize()
    for i in range(REPS):
        compare_verify(ra[i], wa[mode], pa[i])
        compare_verify(rb[i], wb[mode])


def test_static_scratch_calls_queued_on_one_stream():
    import paper_2609_39972_b200 as u
    cfg = synth.CONFIGS["c2"].replace(**SHAPE)
    (ta, za, wa), (tb, zb, wb) = _case(cfg, 41), _case(cfg, 42)
    ra, rb = _results(u, cfg, REPS), _results(u, cfg, REPS)
    torch.cuda.synchronize()
    for i in range(REPS):
        u.ubt_verify_tree_static(ta, za, result=ra[i])
        u.ubt_verify_tree_static(tb, zb, result=rb[i])
    torch.cuda.synchronize()
    for i in range(REPS):
        compare_verify(ra[i], wa["greedy"])
        compare_verify(rb[i], wb["greedy"])


def test_draft_then_verify_chains_without_synchronisation():
    """draft(A) verify(A) draft(B) verify(B) ... on one stream with shared tree, workspaces and results per
    input: every verdict equals the oracle's, with and without the early start."""
    import paper_2609_39972_b200 as u
    cfg = synth.CONFIGS["c2"].replace(**SHAPE)
    cases = []
    for seed in (51, 52):
        di = synth.draft_inputs(cfg, seed)
        ud = synth.to_device(di.unigram_logits, cfg.dtype, DEV)
        bd = torch.from_numpy(di.bigram_scores).to(DEV)
        tree, zd, want = _case(cfg, seed)
        cases.append((ud, bd, zd, want["greedy"]))
    tree = u.Tree.empty(cfg.B, cfg.N, cfg.L, cfg.k, DEV)
    ws_d = u.workspace(u.ubt_draft_workspace_bytes(cfg.B, cfg.L, cfg.V, cfg.k, cfg.N), DEV)
    ws_v = u.workspace(u.ubt_verify_workspace_bytes(cfg.B, cfg.N, cfg.V, "greedy"), DEV)
    for early in (False, True):
        res = [_results(u, cfg, 50) for _ in cases]
        for i in range(50):
            for c, (ud, bd, zd, _) in enumerate(cases):
                u.ubt_draft_tree(ud, bd, cfg.k, cfg.N, tree=tree, ws=ws_d)
                u.ubt_verify_tree(tree, zd, "greedy", result=res[c][i], ws=ws_v, early_start=early)
        torch.cuda.synchronize()
        for c, (_, _, _, want) in enumerate(cases):
            for i in range(50):
                compare_verify(res[c][i], want)
