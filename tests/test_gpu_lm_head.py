"""LM head fused with step a1 (tcgen05 GEMM with a log-sum-exp / top-k epilogue) against the oracle.

The kernel accumulates in fp32 in the tensor cores' order, the oracle in double, so two logits closer than the
accumulation error may come out in either order: the candidates must be a valid top-k of the oracle's logits
up to that tolerance, distinct, and their log-probabilities must match the oracle's values for those tokens.
"""
import numpy as np
import pytest
import torch

import oracle
import ubt_synth as synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
LOGIT_TOL = 1e-4      # |fp32 tensor-core sum - double sum| for sums of d <= 4096 products of unit scale
LP_TOL = 2e-4


def check_rows(ids_g, lp_g, o_ids, o_lp, o_lse, o_logits, k):
    swaps = 0
    for r in range(o_ids.shape[0]):
        g = ids_g[r].tolist()
        assert len(set(g)) == k and min(g) >= 0 and max(g) < o_logits.shape[1], (r, g)
        lg = o_logits[r, g]
        want = o_logits[r, o_ids[r]]
        tol = LOGIT_TOL * np.maximum(1.0, np.abs(want))
        assert np.all(np.abs(lg - want) <= tol), (r, g, o_ids[r].tolist())     # rank by rank the same value
        assert np.all(np.diff(lg) <= tol[1:]), (r, lg)                          # best first
        np.testing.assert_allclose(lp_g[r], lg - o_lse[r], rtol=0, atol=LP_TOL)
        swaps += int(g != o_ids[r].tolist())
    return swaps


# the last two have more work items than CTAs: a CTA comes back to a row block whose state it parked before
@pytest.mark.parametrize("rows,d,V,k", [(200, 128, 1000, 8), (300, 256, 5000, 16), (1, 64, 300, 4), (129, 512, 2049, 1),
                                        (300, 64, 51237, 5), (520, 64, 40000, 16)])
def test_small_shapes_every_row(rows, d, V, k):
    import paper_2609_39972_b200 as u
    h, w = synth.lm_head_inputs(rows, d, V, seed=rows + d, scale=3.0)
    ids_g, lp_g = u.ubt_lm_head_topk(synth.to_device(h, "bf16", DEV), synth.to_device(w, "bf16", DEV), k)
    torch.cuda.synchronize()
    assert u.ubt_debug_ring_timeouts() == 0
    o_ids, o_lp, o_lse, o_logits = oracle.lm_head_topk(h, w, k, want_logits=True)
    swaps = check_rows(ids_g.cpu().numpy(), lp_g.cpu().numpy().astype(np.float64), o_ids, o_lp, o_lse, o_logits, k)
    print(f"rows {rows} d {d} V {V} k {k}: near-tie swaps {swaps}")


def test_qwen3_shape_sampled_rows():
    """d = 4096, V = 151,936, 512 rows (the c3 batch): three rows against the oracle, every row against the
    unfused path (a library product in fp32 followed by ubt_topk_logprob on the stored logits)."""
    import paper_2609_39972_b200 as u
    rows, d, V, k = 512, 4096, 151936, 8
    hd, wd = synth.device_lm_head_inputs(rows, d, V, seed=5, device=DEV, scale=2.0)
    ids_g, lp_g = u.ubt_lm_head_topk(hd, wd, k)
    torch.cuda.synchronize()
    assert u.ubt_debug_ring_timeouts() == 0
    sample = [0, 131, 511]
    o_ids, o_lp, o_lse, o_logits = oracle.lm_head_topk(synth.to_host_bits(hd[sample]), synth.to_host_bits(wd), k,
                                                       want_logits=True)
    check_rows(ids_g[sample].cpu().numpy(), lp_g[sample].cpu().numpy().astype(np.float64), o_ids, o_lp, o_lse,
               o_logits, k)
    # every row: the same selection from logits stored by a library product (fp32), up to near-ties
    logits = (hd.float() @ wd.float().T).contiguous()
    ids_u = torch.empty((rows, k), dtype=torch.int32, device=DEV)
    lp_u = torch.empty((rows, k), dtype=torch.float32, device=DEV)
    ws = u.workspace(u.ubt_draft_workspace_bytes(rows, 1, V, k, 1), DEV)
    u.ubt_topk_logprob(logits, k, ids_u, lp_u, ws)
    torch.cuda.synchronize()
    same = (ids_u == ids_g).all(dim=1)
    assert float(same.float().mean()) > 0.98
    top = torch.gather(logits, 1, ids_g.long())
    ref = torch.gather(logits, 1, ids_u.long())
    assert float((top - ref).abs().max()) < 1e-3
    assert float((lp_g - (top - torch.logsumexp(logits.double(), dim=1, keepdim=True).float())).abs().max()) < 1e-3


def test_argument_checks():
    import paper_2609_39972_b200 as u
    h = torch.zeros((4, 96), dtype=torch.bfloat16, device=DEV)
    w = torch.zeros((100, 96), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(u.UbtError) as ei:
        u.ubt_lm_head_topk(h, w, 4, ws=u.workspace(1 << 20, DEV))       # d not a multiple of 64
    assert ei.value.status == 2
    h = torch.zeros((4, 128), dtype=torch.bfloat16, device=DEV)
    w = torch.zeros((100, 128), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(u.UbtError) as ei:
        u.ubt_lm_head_topk(h, w, 17, ws=u.workspace(1 << 20, DEV))      # beyond the fused epilogue's k
    assert ei.value.status == 2


@pytest.mark.parametrize("rows,d,V,k,cuts", [(200, 128, 5000, 8, [0, 1200, 2608, 5000]),
                                              (300, 256, 20011, 16, [0, 5003, 10006, 15009, 20011]),
                                              (64, 64, 4096, 1, [0, 2048, 4096])])
def test_head_split_along_the_vocabulary_matches_the_whole_head(rows, d, V, k, cuts):
    """The ranks of a tensor-parallel group, one after the other on this GPU: fused head on each slice of the head
    matrix, the partials laid out as an all-gather would, merge; against the oracle on the whole head and against
    the one-GPU fused call."""
    import paper_2609_39972_b200 as u
    h, w = synth.lm_head_inputs(rows, d, V, seed=rows + V, scale=3.0)
    hd, wd = synth.to_device(h, "bf16", DEV), synth.to_device(w, "bf16", DEV)
    shards = len(cuts) - 1
    nbytes = u.ubt_topk_shard_bytes(rows, k)
    gathered = torch.empty(shards * nbytes, dtype=torch.uint8, device=DEV)
    for r in range(shards):
        u.ubt_lm_head_topk_shard(hd, wd[cuts[r]:cuts[r + 1]].contiguous(), k, cuts[r],
                                 partial=gathered[r * nbytes:(r + 1) * nbytes])
    ids_g, lp_g = u.ubt_topk_merge_shards(gathered, shards, rows, k)
    torch.cuda.synchronize()
    assert u.ubt_debug_ring_timeouts() == 0
    o_ids, o_lp, o_lse, o_logits = oracle.lm_head_topk(h, w, k, want_logits=True)
    check_rows(ids_g.cpu().numpy(), lp_g.cpu().numpy().astype(np.float64), o_ids, o_lp, o_lse, o_logits, k)
    ids_1, lp_1 = u.ubt_lm_head_topk(hd, wd, k)
    torch.cuda.synchronize()
    assert float((ids_1 == ids_g).float().mean()) > 0.99          # the same up to near-ties
    assert float((lp_1 - lp_g).abs().max()) < 2e-4
