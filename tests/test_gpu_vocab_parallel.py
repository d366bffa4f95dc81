"""Step a1 with the vocabulary split over ranks (ubt_topk_shard, ubt_topk_merge_shards) against the oracle on the
whole rows.  The ranks are emulated one after the other on one GPU: each slice is copied into a dense tensor of
its own, its partial is computed, the partials are laid back to back in rank order (what an all-gather gives)
and merged.  Nothing waits on anything else, so no second GPU is needed for the arithmetic; the collective
itself is plain torch.distributed and is covered by the two-rank CPU test."""
import numpy as np
import pytest
import torch

import oracle
import shard_layout
import ubt_synth as synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _logits(rows, V, dtype, seed, quantise=False):
    rng = np.random.Generator(np.random.PCG64(seed))
    x = (rng.standard_normal((rows, V)) * rng.uniform(0.5, 6.0, size=(rows, 1))).astype(np.float32)
    if quantise:                       # a handful of distinct values: ties inside and across slices
        x = np.round(x * 2.0) / 2.0
    return synth.f32_to_bf16_bits(x) if dtype == "bf16" else x


def _cuts(V, shards, even, align):
    """Slice boundaries: equal widths, or ragged ones (multiples of `align`, the last slice takes the rest)."""
    if even:
        assert V % shards == 0
        return [V // shards * r for r in range(shards + 1)]
    w = V // shards
    cuts = [0]
    for r in range(1, shards):
        cuts.append(max(cuts[-1] + align, (w * r + (37 * r) % w // 3) // align * align))
    return cuts + [V]


@pytest.mark.parametrize("rows,V,k,shards,dtype,even,align,quantise", [
    (37, 8192, 8, 4, "bf16", True, 8, False),        # ring path in every slice
    (37, 8192, 8, 4, "bf16", False, 1, False),       # ragged widths: plain-load kernels
    (5, 151936, 16, 8, "bf16", True, 8, False),      # the Qwen3 vocabulary over eight ranks
    (64, 40000, 64, 8, "bf16", True, 8, False),      # k = 64: many long lists per row
    (19, 4096, 4, 2, "f32", True, 4, False),
    (23, 6000, 8, 3, "bf16", True, 8, True),         # ties across slices go to the lower token id
    (3, 1000, 8, 1, "f32", True, 4, False),          # one rank: the partial alone
])
def test_sharded_topk_equals_the_oracle_on_whole_rows(rows, V, k, shards, dtype, even, align, quantise):
    import paper_2609_39972_b200 as u
    x = _logits(rows, V, dtype, seed=rows * 1000 + shards, quantise=quantise)
    o_ids, o_lp, o_lse = oracle.topk_logprob(x, k)
    cuts = _cuts(V, shards, even, align)
    xd = synth.to_device(x, dtype, DEV)
    nbytes = u.ubt_topk_shard_bytes(rows, k)
    assert nbytes == shard_layout.offsets(rows, k)[4]
    gathered = torch.empty(shards * nbytes, dtype=torch.uint8, device=DEV)
    for r in range(shards):
        v0, v1 = cuts[r], cuts[r + 1]
        assert v1 - v0 >= k
        part = u.ubt_topk_shard(xd[:, v0:v1].contiguous(), k, v0)
        gathered[r * nbytes:(r + 1) * nbytes] = part[:nbytes]
        # the partial itself, against the oracle on the slice
        ms, val, idx, cnt = shard_layout.unpack(part.cpu().numpy(), rows, k)
        s_ids, s_lp, s_lse = oracle.topk_logprob(np.ascontiguousarray(x[:, v0:v1]), k)
        assert (cnt == k).all()
        np.testing.assert_array_equal(idx, s_ids + v0)
        np.testing.assert_allclose(ms[:, 0].astype(np.float64) + np.log(ms[:, 1].astype(np.float64)), s_lse,
                                   rtol=1e-5, atol=1e-5)
        np.testing.assert_allclose(val.astype(np.float64) - s_lse[:, None], s_lp, rtol=1e-5, atol=1e-5)
    ids, lp = u.ubt_topk_merge_shards(gathered, shards, rows, k)
    torch.cuda.synchronize()
    assert u.ubt_debug_ring_timeouts() == 0
    np.testing.assert_array_equal(ids.cpu().numpy(), o_ids)
    np.testing.assert_allclose(lp.cpu().numpy().astype(np.float64), o_lp, rtol=1e-5, atol=1e-5)
    # the same through the one-GPU entry point, and the host restatement of the merge
    ids1 = torch.empty((rows, k), dtype=torch.int32, device=DEV)
    lp1 = torch.empty((rows, k), dtype=torch.float32, device=DEV)
    u.ubt_topk_logprob(xd, k, ids1, lp1, u.workspace(u.ubt_draft_workspace_bytes(rows, 1, V, k, 1), DEV))
    torch.cuda.synchronize()
    assert torch.equal(ids1, ids)
    assert float((lp1 - lp).abs().max()) <= 1e-5 * max(1.0, float(lp.abs().max()))
    h_ids, h_lp = shard_layout.merge(gathered.cpu().numpy(), shards, rows, k)
    np.testing.assert_array_equal(h_ids, o_ids)
    np.testing.assert_allclose(h_lp, o_lp, rtol=1e-5, atol=1e-5)


def test_sharded_candidates_build_the_same_tree():
    """draft = sharded a1 + ubt_build_tree equals ubt_draft_tree on the whole rows (c2 shapes, four ranks)."""
    import paper_2609_39972_b200 as u
    cfg = synth.CONFIGS["c2"].replace(B=3)
    di = synth.draft_inputs(cfg, 77)
    ud = synth.to_device(di.unigram_logits, cfg.dtype, DEV)
    bd = torch.from_numpy(di.bigram_scores).to(DEV)
    whole = u.ubt_draft_tree(ud, bd, cfg.k, cfg.N)
    shards, rows = 4, cfg.B * cfg.L
    nbytes = u.ubt_topk_shard_bytes(rows, cfg.k)
    gathered = torch.empty(shards * nbytes, dtype=torch.uint8, device=DEV)
    w = cfg.V // shards
    for r in range(shards):
        gathered[r * nbytes:(r + 1) * nbytes] = u.ubt_topk_shard(ud[..., r * w:(r + 1) * w].contiguous(), cfg.k, r * w)[:nbytes]
    split = u.Tree.empty(cfg.B, cfg.N, cfg.L, cfg.k, DEV)
    u.ubt_topk_merge_shards(gathered, shards, rows, cfg.k, split.cand_ids, split.cand_logprob)
    u.ubt_build_tree(bd, split)
    torch.cuda.synchronize()
    for name in ("cand_ids", "token_ids", "parents", "depths", "position_ids", "cand_rank", "mask", "n_nodes"):
        assert torch.equal(getattr(whole, name), getattr(split, name)), name


def test_argument_checks():
    import paper_2609_39972_b200 as u
    x = torch.zeros((4, 64), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(u.UbtError):
        u.ubt_topk_shard(x, 128, 0)              # k > Vs
    with pytest.raises(u.UbtError):
        u.ubt_topk_shard(x, 8, -1)               # negative first column
    with pytest.raises(ValueError):
        u.ubt_topk_merge_shards(torch.zeros(16, dtype=torch.uint8, device=DEV), 2, 4, 8)


# ---- greedy verification with the target logits' vocabulary split over ranks
def _drafted(cfg, seed):
    import paper_2609_39972_b200 as u
    from parity import tree_to_numpy
    di = synth.draft_inputs(cfg, seed)
    tree = u.ubt_draft_tree(synth.to_device(di.unigram_logits, cfg.dtype, DEV),
                            torch.from_numpy(di.bigram_scores).to(DEV), cfg.k, cfg.N)
    torch.cuda.synchronize()
    return tree, tree_to_numpy(tree)


@pytest.mark.parametrize("V,shards,even", [(8192, 4, True), (8192, 3, False), (151936, 8, True)])
def test_sharded_greedy_verify_equals_the_oracle(V, shards, even):
    import paper_2609_39972_b200 as u
    from parity import compare_verify
    cfg = synth.CONFIGS["c2"].replace(B=3, L=6, N=24, k=4, V=V)
    tree, g = _drafted(cfg, 5)
    z = synth.target_logits(cfg, 5)
    synth.plant_path(z, cfg.dtype, g.token_ids, g.parents, g.n_nodes, 5)
    # a tie between two slices: the lower token id must win in every row of sequence 0
    zf = synth.as_f32(z, cfg.dtype)
    top = zf[0].max(axis=1) + 1.0
    for n in range(cfg.N):
        for col in (V - 3, 5):
            z[0, n, col] = synth.f32_to_bf16_bits(np.float32([top[n]]))[0]
    want = oracle.verify(g.token_ids, g.parents, g.n_nodes, cfg.L, z, "greedy")
    zd = synth.to_device(z, cfg.dtype, DEV)
    cuts = _cuts(V, shards, even, 1 if not even else 8)
    rows = cfg.B * cfg.N
    gathered = torch.empty(shards * rows, dtype=torch.int64, device=DEV)
    for r in range(shards):
        u.ubt_verify_keys_shard(zd[..., cuts[r]:cuts[r + 1]].contiguous(), cuts[r], gathered[r * rows:(r + 1) * rows])
    pick = torch.full((cfg.B, cfg.N), -9, dtype=torch.int32, device=DEV)
    status = torch.full((cfg.B,), -1, dtype=torch.int32, device=DEV)
    res = u.ubt_verify_tree_keys(tree, gathered, shards, node_pick=pick, status=status)
    torch.cuda.synchronize()
    compare_verify(res, want, pick)
    assert (pick[0] == 5).all()
    assert status.tolist() == [0] * cfg.B
    # and bit for bit what the one-GPU call gives
    one = u.ubt_verify_tree(tree, zd, "greedy")
    torch.cuda.synchronize()
    for name in ("accepted_len", "bonus_token", "accepted_nodes", "out_tokens"):
        assert torch.equal(getattr(one, name), getattr(res, name)), name


def test_sharded_greedy_verify_reports_a_nan_in_any_slice():
    import paper_2609_39972_b200 as u
    cfg = synth.CONFIGS["c2"].replace(B=2, L=6, N=24, k=4, V=8192)
    tree, g = _drafted(cfg, 9)
    z = synth.target_logits(cfg, 9)
    z[1, 3, 6000] = 0x7FC0                     # a bf16 NaN in the third slice of sequence 1
    zd = synth.to_device(z, cfg.dtype, DEV)
    shards, rows, w = 4, cfg.B * cfg.N, cfg.V // 4
    gathered = torch.empty(shards * rows, dtype=torch.int64, device=DEV)
    for r in range(shards):
        u.ubt_verify_keys_shard(zd[..., r * w:(r + 1) * w].contiguous(), r * w, gathered[r * rows:(r + 1) * rows])
    status = torch.zeros((cfg.B,), dtype=torch.int32, device=DEV)
    u.ubt_verify_tree_keys(tree, gathered, shards, status=status)
    torch.cuda.synchronize()
    assert status.tolist() == [0, 1]


def _sharded_sampling(u, tree, zd, cuts, seed, temperature, status=None):
    """The four steps of sampling verification over a vocabulary-parallel group, the ranks run one after the other
    on this GPU; the buffers that an all-gather would fill are written slice by slice."""
    shards = len(cuts) - 1
    B, N, _ = zd.shape
    rows = B * N
    shard = [zd[..., cuts[r]:cuts[r + 1]].contiguous() for r in range(shards)]
    g_keys = torch.empty(shards * rows, dtype=torch.int64, device=DEV)
    for r in range(shards):
        u.ubt_verify_keys_shard(shard[r], cuts[r], g_keys[r * rows:(r + 1) * rows])
    g_tot = torch.empty(shards * rows, dtype=torch.int64, device=DEV)
    ws = []
    for r in range(shards):
        _, w = u.ubt_sample_totals_shard(shard[r], g_keys, shards, temperature, totals=g_tot[r * rows:(r + 1) * rows])
        ws.append(w)
    g_picks = torch.empty(shards * rows, dtype=torch.int32, device=DEV)
    for r in range(shards):
        u.ubt_sample_picks_shard(shard[r], cuts[r], r, g_tot, shards, seed, ws[r], picks=g_picks[r * rows:(r + 1) * rows])
    res = u.ubt_verify_tree_picks(tree, g_picks, shards, status=status)
    torch.cuda.synchronize()
    return res, g_picks.view(shards, B, N)


@pytest.mark.parametrize("V,shards,even,dtype,temperature", [
    (8192, 4, True, "bf16", 1.0), (8192, 3, False, "bf16", 0.7), (4001, 2, False, "f32", 1.3),
    (151936, 8, True, "bf16", 1.0), (40000, 5, False, "f32", 1.0)])
def test_sharded_sampling_verify_equals_the_oracle(V, shards, even, dtype, temperature):
    import paper_2609_39972_b200 as u
    from parity import compare_verify
    cfg = synth.CONFIGS["c2"].replace(B=3, L=6, N=24, k=4, V=V, dtype=dtype, mode="sample")
    tree, g = _drafted(cfg, 11)
    z = synth.agree_targets(cfg, synth.draft_inputs(cfg, 11).unigram_logits, g.token_ids, g.parents, g.depths,
                            g.n_nodes, 11)
    zd = synth.to_device(z, cfg.dtype, DEV)
    cuts = _cuts(V, shards, even, 1 if not even else 8)
    walked = 0
    for seed in (0, 1, 12345678901234567):
        want = oracle.verify(g.token_ids, g.parents, g.n_nodes, cfg.L, z, "sample", seed=seed, temperature=temperature)
        status = torch.full((cfg.B,), -1, dtype=torch.int32, device=DEV)
        res, picks = _sharded_sampling(u, tree, zd, cuts, seed, temperature, status)
        compare_verify(res, want)
        assert status.tolist() == [0] * cfg.B
        # every slot has exactly one owner, and it holds the oracle's pick
        p = picks.cpu().numpy()
        assert ((p >= 0).sum(axis=0) == 1).all()
        assert (p.max(axis=0) == want.node_pick).all()
        walked += int(want.accepted_len.sum())
        # and bit for bit what the one-GPU call gives
        one = u.ubt_verify_tree(tree, zd, "sample", seed=seed, temperature=temperature)
        torch.cuda.synchronize()
        for name in ("accepted_len", "bonus_token", "accepted_nodes", "out_tokens"):
            assert torch.equal(getattr(one, name), getattr(res, name)), name
    assert walked > 0


def test_sharded_sampling_reports_a_nan_or_inf_in_any_slice():
    import paper_2609_39972_b200 as u
    from parity import compare_verify
    cfg = synth.CONFIGS["c2"].replace(B=3, L=6, N=24, k=4, V=8192, mode="sample")
    tree, g = _drafted(cfg, 9)
    z = synth.target_logits(cfg, 9)
    clean = z.copy()
    z[1, 3, 6000] = 0x7FC0                     # a bf16 NaN in the third slice of sequence 1
    z[2, 0, 100] = 0x7F80                      # +inf in the first slice of sequence 2
    zd = synth.to_device(z, cfg.dtype, DEV)
    status = torch.zeros((cfg.B,), dtype=torch.int32, device=DEV)
    res, picks = _sharded_sampling(u, tree, zd, [0, 2048, 4096, 6144, 8192], 3, 1.0, status)
    assert status.tolist() == [0, 1, 1]
    p = picks.cpu().numpy()
    assert (p[:, 1, 3] == -1).all() and (p[:, 2, 0] == -1).all()
    want = oracle.verify(g.token_ids[:1], g.parents[:1], g.n_nodes[:1], cfg.L, clean[:1], "sample", seed=3)
    compare_verify(res, want, rows=[0])


def test_sharded_sampling_argument_checks():
    import paper_2609_39972_b200 as u
    cfg = synth.CONFIGS["c2"].replace(B=1, L=4, N=8, k=4, V=4096)
    zd = synth.to_device(synth.target_logits(cfg, 1), cfg.dtype, DEV)
    keys = u.ubt_verify_keys_shard(zd, 0)
    small = torch.empty(16, dtype=torch.uint8, device=DEV)
    with pytest.raises(u.UbtError):
        u.ubt_sample_totals_shard(zd, keys, 1, ws=small)                       # workspace too small
    with pytest.raises(u.UbtError):
        u.ubt_sample_totals_shard(zd, keys, 1, temperature=0.0)
    totals, ws = u.ubt_sample_totals_shard(zd, keys, 1)
    with pytest.raises(u.UbtError):
        u.ubt_sample_picks_shard(zd, 0, 1, totals, 1, 0, ws)                   # rank outside the group
