"""Non-finite logits: nothing traps, the sequences concerned are reported in the status words, and the other
sequences of the batch still match the oracle.  One case per kernel family (bulk-copy ring and plain loads;
top-k, greedy picks, sampled picks), plus the host-buffer forms' UBT_ERR_NONFINITE."""
import numpy as np
import pytest
import torch

import oracle
import ubt_synth as synth
from parity import compare_draft, compare_verify, tree_to_numpy

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
NAN, INF = float("nan"), float("inf")


def _cfg(V, dtype):
    return synth.CONFIGS["c2"].replace(B=3, L=5, N=20, k=4, V=V, dtype=dtype)


@pytest.mark.parametrize("V,dtype", [(40000, "bf16"), (4001, "bf16"), (8192, "f32"), (1001, "f32")])
def test_draft_reports_sequences_with_nan_or_inf(V, dtype):
    import paper_2609_39972_b200 as u
    cfg = _cfg(V, dtype)
    di = synth.draft_inputs(cfg, 3)
    ud = synth.to_device(di.unigram_logits, cfg.dtype, DEV)
    bd = torch.from_numpy(di.bigram_scores).to(DEV)
    ud[1, 2, V // 3] = NAN
    ud[2, 4, V - 1] = INF
    status = torch.full((cfg.B,), -5, dtype=torch.int32, device=DEV)
    tree = u.ubt_draft_tree(ud, bd, cfg.k, cfg.N, status=status)
    torch.cuda.synchronize()
    assert status.tolist() == [0, 1, 1]
    g = tree_to_numpy(tree)
    want = oracle.draft_tree(di.unigram_logits[:1], di.bigram_scores[:1], cfg.k, cfg.N)
    assert compare_draft(g, want, cfg.L, cfg.k, cfg.N, rows=[0]) == []
    # the flagged sequences still produced in-range arrays
    assert int(tree.n_nodes.min()) >= 1 and int(tree.n_nodes.max()) <= cfg.N
    clean = torch.full((cfg.B,), -5, dtype=torch.int32, device=DEV)
    u.ubt_draft_tree(synth.to_device(di.unigram_logits, cfg.dtype, DEV), bd, cfg.k, cfg.N, status=clean)
    assert clean.tolist() == [0, 0, 0]


@pytest.mark.parametrize("mode", ["greedy", "sample"])
@pytest.mark.parametrize("V,dtype", [(40000, "bf16"), (4001, "bf16"), (8192, "f32"), (1001, "f32")])
def test_verify_reports_sequences_with_nan_or_inf(V, dtype, mode):
    import paper_2609_39972_b200 as u
    cfg = _cfg(V, dtype)
    di = synth.draft_inputs(cfg, 4)
    tree = u.ubt_draft_tree(synth.to_device(di.unigram_logits, cfg.dtype, DEV),
                            torch.from_numpy(di.bigram_scores).to(DEV), cfg.k, cfg.N)
    torch.cuda.synchronize()
    g = tree_to_numpy(tree)
    z = synth.target_logits(cfg, 4)
    synth.plant_path(z, cfg.dtype, g.token_ids, g.parents, g.n_nodes, 4)
    zd = synth.to_device(z, cfg.dtype, DEV)
    zd[1, cfg.N - 1, 7] = NAN            # an unused slot's row counts too
    zd[2, 0, V // 2] = INF
    status = torch.full((cfg.B,), -5, dtype=torch.int32, device=DEV)
    res = u.ubt_verify_tree(tree, zd, mode, seed=9, status=status)
    torch.cuda.synchronize()
    assert status.tolist() == [0, 1, 1]
    want = oracle.verify(g.token_ids[:1], g.parents[:1], g.n_nodes[:1], cfg.L, z[:1], mode, seed=9)
    compare_verify(res, want, rows=slice(0, 1))
    acc = res.accepted_len.cpu().numpy()
    assert np.all(acc >= 0) and np.all(acc <= cfg.L)
    bonus = res.bonus_token.cpu().numpy()
    assert np.all(bonus >= 0) and np.all(bonus < V)


def test_build_tree_reports_non_finite_candidate_logprobs():
    import paper_2609_39972_b200 as u
    cfg = _cfg(4000, "bf16")
    di = synth.draft_inputs(cfg, 5)
    ud = synth.to_device(di.unigram_logits, cfg.dtype, DEV)
    bd = torch.from_numpy(di.bigram_scores).to(DEV)
    tree = u.Tree.empty(cfg.B, cfg.N, cfg.L, cfg.k, DEV)
    ws = u.workspace(u.ubt_draft_workspace_bytes(cfg.B * cfg.L, 1, cfg.V, cfg.k, 1), DEV)
    u.ubt_topk_logprob(ud, cfg.k, tree.cand_ids, tree.cand_logprob, ws)
    tree.cand_logprob[2, 1, 0] = NAN
    status = torch.full((cfg.B,), -5, dtype=torch.int32, device=DEV)
    u.ubt_build_tree(bd, tree, status=status)
    torch.cuda.synchronize()
    assert status.tolist() == [0, 0, 1]


def test_host_forms_return_nonfinite_when_asked_to_validate():
    import paper_2609_39972_b200 as u
    cfg = _cfg(8000, "bf16")
    di = synth.draft_inputs(cfg, 6)
    uh = synth.to_device(di.unigram_logits, cfg.dtype, "cpu").pin_memory()
    bh = torch.from_numpy(di.bigram_scores).pin_memory()
    tree_h = u.Tree.empty(cfg.B, cfg.N, cfg.L, cfg.k, DEV, pin=True)
    dbuf = u.workspace(u.ubt_draft_host_buffer_bytes(cfg.B, cfg.L, cfg.V, cfg.k, cfg.N, 1), DEV)
    st = torch.full((cfg.B,), -5, dtype=torch.int32).pin_memory()
    u.ubt_draft_tree_host(uh, bh, cfg.k, cfg.N, tree_h, dbuf, status=st, validate_finite=True)   # clean: no error
    assert st.tolist() == [0, 0, 0]
    uh[0, 0, 5] = NAN
    with pytest.raises(u.UbtError) as ei:
        u.ubt_draft_tree_host(uh, bh, cfg.k, cfg.N, tree_h, dbuf, status=st, validate_finite=True)
    assert ei.value.status == 6 and st.tolist() == [1, 0, 0]
    u.ubt_draft_tree_host(uh, bh, cfg.k, cfg.N, tree_h, dbuf, status=st)         # without validation: status only
    assert st.tolist() == [1, 0, 0]
    # verify: a clean tree, a target row with +inf
    uh[0, 0, 5] = 0.0
    u.ubt_draft_tree_host(uh, bh, cfg.k, cfg.N, tree_h, dbuf)
    zh = synth.to_device(synth.target_logits(cfg, 6), cfg.dtype, "cpu").pin_memory()
    res_h = u.VerifyResult.empty(cfg.B, cfg.L, DEV, pin=True)
    vbuf = u.workspace(u.ubt_verify_host_buffer_bytes(cfg.B, cfg.L, cfg.N, cfg.V, 1, "greedy"), DEV)
    u.ubt_verify_tree_host(tree_h, zh, res_h, vbuf, "greedy", status=st, validate_finite=True)
    assert st.tolist() == [0, 0, 0]
    zh[1, 3, 100] = INF
    with pytest.raises(u.UbtError) as ei:
        u.ubt_verify_tree_host(tree_h, zh, res_h, vbuf, "greedy", status=st, validate_finite=True)
    assert ei.value.status == 6 and st.tolist() == [0, 1, 0]
