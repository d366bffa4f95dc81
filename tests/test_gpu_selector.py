"""ubt_selector_scores (Section 3.1.2, "Parallel Computation") against the oracle, and the paper's data flow
top-k -> selector scores -> tree through the split entry points."""
import numpy as np
import pytest
import torch

import oracle
import ubt_synth as synth
from parity import compare_draft, tree_to_numpy

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _dev_table(a, dtype):
    return synth.to_device(a, dtype, DEV)


@pytest.mark.parametrize("dtype,V,R,B,L,k", [("f32", 3000, 64, 3, 5, 6), ("bf16", 3000, 64, 3, 5, 6),
                                             ("bf16", 5000, 256, 2, 4, 64), ("f32", 700, 1024, 2, 3, 8), ("bf16", 900, 1000, 2, 3, 64),
                                             ("bf16", 900, 8, 1, 1, 4), ("bf16", 2000, 128, 2, 3, 33),
                                             ("bf16", 2000, 192, 1, 2, 17)])
def test_scores_match_the_oracle(dtype, V, R, B, L, k):
    import paper_2609_39972_b200 as u
    phi, psi, gate = synth.selector_tables(V, R, B, L, 7, dtype)
    rng = np.random.default_rng(8)
    cand = np.stack([np.stack([rng.choice(V, k, replace=False) for _ in range(L)]) for _ in range(B)]).astype(np.int32)
    anchor = rng.integers(0, V, B).astype(np.int32)
    big, anc = oracle.selector_scores(phi, psi, gate, cand, anchor)
    gb, ga = u.ubt_selector_scores(_dev_table(phi, dtype), _dev_table(psi, dtype), torch.from_numpy(gate).to(DEV),
                                   torch.from_numpy(cand).to(DEV), torch.from_numpy(anchor).to(DEV))
    torch.cuda.synchronize()
    # fp32 products and sums against the double-precision sum: 1e-5 * max(1, |x|), the bar of all fp32 scores
    for got, want in ((gb.cpu().numpy(), big), (ga.cpu().numpy(), anc)):
        assert got.shape == want.shape
        assert np.all(np.abs(got - want) <= 1e-5 * np.maximum(1.0, np.abs(want)))
    # without an anchor only the inner transitions are written
    gb2, ga2 = u.ubt_selector_scores(_dev_table(phi, dtype), _dev_table(psi, dtype), torch.from_numpy(gate).to(DEV),
                                     torch.from_numpy(cand).to(DEV))
    torch.cuda.synchronize()
    assert ga2 is None and torch.equal(gb2, gb)


def test_paper_data_flow_topk_selector_tree():
    """Qwen3-sized vocabulary, selector rank 256, k = 64, W = 12, 64 non-root nodes, depth 15 (the paper's
    configuration): candidates from ubt_topk_logprob feed ubt_selector_scores, whose output feeds ubt_build_tree."""
    import paper_2609_39972_b200 as u
    cfg = synth.Config("p1", 4, 15, synth.V_QWEN3, 64, 65, "bf16", "pos_uniform:0.5,8", 1.0, 4.0, "greedy")
    R, W = 256, 12
    di = synth.draft_inputs(cfg, 2)
    phi, psi, gate = synth.selector_tables(cfg.V, R, cfg.B, cfg.L, 2, "bf16")
    anchor = np.arange(cfg.B, dtype=np.int32) * 1000 + 5
    ids, lp, _ = oracle.topk_logprob(di.unigram_logits, cfg.k)
    big, anc = oracle.selector_scores(phi, psi, gate, ids, anchor)
    otree = oracle.draft_tree(di.unigram_logits, big.astype(np.float32), cfg.k, cfg.N, W=W,
                              anchor_bigram=anc.astype(np.float32), anchor_tokens=anchor)

    ud = synth.to_device(di.unigram_logits, cfg.dtype, DEV)
    tree = u.Tree.empty(cfg.B, cfg.N, cfg.L, cfg.k, DEV)
    ws = u.workspace(u.ubt_draft_workspace_bytes(cfg.B, cfg.L, cfg.V, cfg.k, cfg.N), DEV)
    u.ubt_topk_logprob(ud, cfg.k, tree.cand_ids, tree.cand_logprob, ws)
    anchor_d = torch.from_numpy(anchor).to(DEV)
    gb, ga = u.ubt_selector_scores(_dev_table(phi, "bf16"), _dev_table(psi, "bf16"), torch.from_numpy(gate).to(DEV),
                                   tree.cand_ids, anchor_d)
    u.ubt_build_tree(gb, tree, search_width=W, anchor_bigram=ga, anchor_tokens=anchor_d)
    torch.cuda.synchronize()
    assert np.array_equal(tree.cand_ids.cpu().numpy(), ids)
    assert np.all(np.abs(gb.cpu().numpy() - big) <= 1e-5 * np.maximum(1.0, np.abs(big)))
    swaps = compare_draft(tree_to_numpy(tree), otree, cfg.L, cfg.k, cfg.N, W, 0.0, anchor, None)
    print("near-tie swaps:", swaps)
