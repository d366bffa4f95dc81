"""The walk of step a4 on given per-slot picks (ubt_verify_tree_picks), and greedy verification straight from the
target's hidden states (LM head fused with the row arg max, then that walk), against the oracle (needs a B200)."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
import ubt_synth as synth
from parity import compare_verify, tree_to_numpy

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def drafted_tree(u, cfg, seed):
    di = synth.draft_inputs(cfg, seed)
    ud = synth.to_device(di.unigram_logits, cfg.dtype, DEV)
    bd = torch.from_numpy(di.bigram_scores).to(DEV)
    gtree = u.ubt_draft_tree(ud, bd, cfg.k, cfg.N)
    torch.cuda.synchronize()
    return gtree, tree_to_numpy(gtree)


def picks_that_walk(g, cfg, seed):
    """Per-slot picks: at half of the slots that have children the token of one of them, elsewhere any token."""
    rng = np.random.default_rng(seed)
    picks = rng.integers(0, cfg.V, (cfg.B, cfg.N)).astype(np.int32)
    for b in range(cfg.B):
        for n in range(int(g.n_nodes[b])):
            kids = [c for c in range(1, int(g.n_nodes[b])) if g.parents[b, c] == n]
            if kids and rng.random() < 0.7:
                picks[b, n] = g.token_ids[b, kids[int(rng.integers(0, len(kids)))]]
    return picks


@pytest.mark.parametrize("name,seed", [("c1", 0), ("c1", 1), ("c3", 2), ("c2", 3)])
def test_walk_on_given_picks_matches_oracle(name, seed):
    import paper_2609_39972_b200 as u
    cfg = synth.CONFIGS[name]
    gtree, g = drafted_tree(u, cfg, seed)
    picks = picks_that_walk(g, cfg, seed)
    ov = oracle.verify_picks(g.token_ids, g.parents, g.n_nodes, cfg.L, picks)
    assert ov.accepted_len.max() >= 1                      # the planted picks do walk
    status = torch.full((cfg.B,), -1, dtype=torch.int32, device=DEV)
    res = u.ubt_verify_tree_picks(gtree, torch.from_numpy(picks).to(DEV), status=status)
    torch.cuda.synchronize()
    compare_verify(res, ov)
    assert status.cpu().numpy().tolist() == [0] * cfg.B
    # the [B * N, 1] layout that the LM head call returns is the same memory
    res2 = u.ubt_verify_tree_picks(gtree, torch.from_numpy(picks).to(DEV).view(cfg.B * cfg.N, 1))
    torch.cuda.synchronize()
    compare_verify(res2, ov)


def test_negative_pick_is_reported_and_counts_as_token_zero():
    import paper_2609_39972_b200 as u
    cfg = synth.CONFIGS["c1"]
    gtree, g = drafted_tree(u, cfg, 5)
    picks = picks_that_walk(g, cfg, 5)
    picks[0, 0] = -1
    as_zero = picks.copy()
    as_zero[0, 0] = 0
    ov = oracle.verify_picks(g.token_ids, g.parents, g.n_nodes, cfg.L, as_zero)
    status = torch.zeros((cfg.B,), dtype=torch.int32, device=DEV)
    res = u.ubt_verify_tree_picks(gtree, torch.from_numpy(picks).to(DEV), status=status)
    torch.cuda.synchronize()
    compare_verify(res, ov)
    st = status.cpu().numpy()
    assert st[0] == 1 and not st[1:].any()          # UBT_STATUS_NONFINITE


def test_argument_checks():
    import paper_2609_39972_b200 as u
    from paper_2609_39972_b200 import binding
    cfg = synth.CONFIGS["c1"]
    gtree, _ = drafted_tree(u, cfg, 0)
    with pytest.raises(ValueError):
        u.ubt_verify_tree_picks(gtree, torch.zeros((cfg.B, cfg.N - 1), dtype=torch.int32, device=DEV))
    with pytest.raises(ValueError):
        u.ubt_verify_tree_picks(gtree, torch.zeros((cfg.B, cfg.N), dtype=torch.int64, device=DEV))
    res = binding.VerifyResult.empty(cfg.B, cfg.L, DEV)
    t, r = gtree.c_struct(), res.c_struct()
    rc = binding.load().ubt_verify_tree_picks(C.byref(t), None, 1, C.byref(r), None, None)
    assert rc == 1                                  # UBT_ERR_INVALID_ARG


@pytest.mark.parametrize("B,N,L,k,d,V,seed", [(4, 32, 6, 4, 128, 5000, 0), (2, 64, 8, 8, 256, 20011, 1)])
def test_greedy_verification_from_hidden_states(B, N, L, k, d, V, seed):
    """hidden state of a slot = the head's row of the token the target should pick there (its logit is that row's
    squared norm, far above the others'): the picks are known, the margin is wide, and the fused head must
    reproduce them and the oracle's walk."""
    import paper_2609_39972_b200 as u
    cfg = synth.CONFIGS["c1"].replace(name="h", B=B, L=L, V=V, k=k, N=N)
    gtree, g = drafted_tree(u, cfg, seed)
    want = picks_that_walk(g, cfg, seed + 100)
    _, w = synth.lm_head_inputs(1, d, V, seed=seed + 7, scale=8.0)
    w32 = synth.as_f32(w, "bf16")
    hidden = synth.f32_to_bf16_bits(w32[want.reshape(-1)] * 4.0)              # [B * N, d]
    o_ids, _, _, _ = oracle.lm_head_topk(hidden, w, 1)
    assert o_ids[:, 0].tolist() == want.reshape(-1).tolist()                 # the construction holds in double
    ov = oracle.verify_picks(g.token_ids, g.parents, g.n_nodes, L, o_ids.reshape(B, N))
    assert ov.accepted_len.max() >= 1
    res = u.verify_tree_from_hidden(gtree, synth.to_device(hidden, "bf16", DEV).view(B, N, d),
                                    synth.to_device(w, "bf16", DEV))
    torch.cuda.synchronize()
    assert u.ubt_debug_ring_timeouts() == 0
    compare_verify(res, ov, res.node_pick)


def test_greedy_verification_from_hidden_states_with_a_split_head():
    """The head cut into three vocabulary slices (ranks emulated one after the other): k = 1 partial per slice, merge,
    walk; the same verdict as the whole head."""
    import paper_2609_39972_b200 as u
    B, N, L, k, d, V = 3, 32, 6, 4, 128, 6000
    cfg = synth.CONFIGS["c1"].replace(name="h", B=B, L=L, V=V, k=k, N=N)
    gtree, g = drafted_tree(u, cfg, 3)
    want = picks_that_walk(g, cfg, 103)
    _, w = synth.lm_head_inputs(1, d, V, seed=10, scale=8.0)
    hidden = synth.f32_to_bf16_bits(synth.as_f32(w, "bf16")[want.reshape(-1)] * 4.0)
    ov = oracle.verify_picks(g.token_ids, g.parents, g.n_nodes, L, oracle.lm_head_topk(hidden, w, 1)[0].reshape(B, N))
    hd, wd = synth.to_device(hidden, "bf16", DEV), synth.to_device(w, "bf16", DEV)
    cuts, rows = [0, 1808, 4000, V], B * N
    nbytes = u.ubt_topk_shard_bytes(rows, 1)
    gathered = torch.empty(3 * nbytes, dtype=torch.uint8, device=DEV)
    for r in range(3):
        u.ubt_lm_head_topk_shard(hd, wd[cuts[r]:cuts[r + 1]].contiguous(), 1, cuts[r],
                                 partial=gathered[r * nbytes:(r + 1) * nbytes])
    picks, _ = u.ubt_topk_merge_shards(gathered, 3, rows, 1)
    res = u.ubt_verify_tree_picks(gtree, picks)
    torch.cuda.synchronize()
    compare_verify(res, ov, res.node_pick)
    one = u.verify_tree_from_hidden_vocab_parallel(gtree, hd.view(B, N, d), wd, 0)     # a group of one
    torch.cuda.synchronize()
    compare_verify(one, ov, one.node_pick)
