"""CUDA path vs oracle through the C ABI, element by element on the same seeded inputs (needs a B200)."""
import numpy as np
import pytest
import torch

import oracle
import ubt_synth as synth
from parity import compare_draft, compare_verify, tree_to_numpy

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def ubt():
    import paper_2609_39972_b200 as u
    return u


def run_case(cfg, seed, targets="plant", W=0, zeta=0.0, use_opts=False, seeds_sample=(0,)):
    """Draft + verify one synthetic batch on the GPU and against the oracle; returns logged swaps."""
    u = ubt()
    di = synth.draft_inputs(cfg, seed)
    rng = np.random.default_rng(seed + 1000)
    kw_np = {}
    if use_opts:
        kw_np = dict(alpha=rng.uniform(0.5, 1.5, cfg.L).astype(np.float32),
                     lam=rng.uniform(0.5, 2.0, cfg.L).astype(np.float32),
                     anchor_bigram=rng.standard_normal((cfg.B, cfg.k)).astype(np.float32),
                     anchor_tokens=rng.integers(0, cfg.V, cfg.B).astype(np.int32),
                     pos_offset=rng.integers(0, 200000, cfg.B).astype(np.int32))
    otree = oracle.draft_tree(di.unigram_logits, di.bigram_scores, cfg.k, cfg.N, W=W, zeta=zeta, **kw_np)
    kw_t = {n: torch.from_numpy(v).to(DEV) for n, v in kw_np.items()}
    ud = synth.to_device(di.unigram_logits, cfg.dtype, DEV)
    bd = torch.from_numpy(di.bigram_scores).to(DEV)
    gtree = u.ubt_draft_tree(ud, bd, cfg.k, cfg.N, search_width=W, depth_bonus=zeta, **kw_t)
    torch.cuda.synchronize()
    g = tree_to_numpy(gtree)
    swaps = compare_draft(g, otree, cfg.L, cfg.k, cfg.N, W, zeta, kw_np.get("anchor_tokens"), kw_np.get("pos_offset"))
    # targets are built from the GPU's tree arrays (identical to the oracle's unless a swap was logged)
    if targets == "plant":
        z = synth.target_logits(cfg, seed)
        synth.plant_path(z, cfg.dtype, g.token_ids, g.parents, g.n_nodes, seed)
    elif targets == "agree":
        z = synth.agree_targets(cfg, di.unigram_logits, g.token_ids, g.parents, g.depths, g.n_nodes, seed)
    else:
        z = synth.target_logits(cfg, seed)
    zd = synth.to_device(z, cfg.dtype, DEV)
    pick = torch.empty((cfg.B, cfg.N), dtype=torch.int32, device=DEV)
    if cfg.mode == "greedy":
        res = u.ubt_verify_tree(gtree, zd, "greedy", node_pick=pick)
        torch.cuda.synchronize()
        ov = oracle.verify(g.token_ids, g.parents, g.n_nodes, cfg.L, z, "greedy")
        compare_verify(res, ov, pick)
        res2 = u.ubt_verify_tree(gtree, zd, "greedy")          # without node_pick
        torch.cuda.synchronize()
        compare_verify(res2, ov)
        _check_path_only(u, gtree, zd, "greedy", 0, ov, g, cfg)
    for s in (seeds_sample if cfg.mode == "sample" else ()):
        res = u.ubt_verify_tree(gtree, zd, "sample", seed=s, temperature=1.0, node_pick=pick)
        torch.cuda.synchronize()
        ov = oracle.verify(g.token_ids, g.parents, g.n_nodes, cfg.L, z, "sample", seed=s, temperature=1.0)
        compare_verify(res, ov, pick)
        _check_path_only(u, gtree, zd, "sample", s, ov, g, cfg)
    return swaps


def _check_path_only(u, gtree, zd, mode, seed, ov, g, cfg):
    """The path-only form of the verify call: the same verdict, picks reported at the visited slots only."""
    pick = torch.full((cfg.B, cfg.N), -7, dtype=torch.int32, device=DEV)
    res = u.ubt_verify_tree(gtree, zd, mode, seed=seed, temperature=1.0, node_pick=pick, path_only=True)
    torch.cuda.synchronize()
    compare_verify(res, ov)
    pk = pick.cpu().numpy()
    nodes = res.accepted_nodes.cpu().numpy()
    for b in range(cfg.B):
        visited = [int(n) for n in nodes[b] if n >= 0]
        for n in range(cfg.N):
            assert pk[b, n] == (ov.node_pick[b, n] if n in visited else -1), (b, n)


@pytest.mark.parametrize("seed", range(6))
def test_c1_tiny_fp32_exact(seed):
    assert run_case(synth.CONFIGS["c1"], seed) == []


@pytest.mark.parametrize("seed", range(3))
def test_c1_options_width_bonus(seed):
    cfg = synth.CONFIGS["c1"]
    run_case(cfg, seed, use_opts=True)
    run_case(cfg, seed, W=3, zeta=-0.25, use_opts=True)
    run_case(cfg, seed, W=1)


def test_c1_sampling_modes():
    cfg = synth.CONFIGS["c1"].replace(mode="sample")
    run_case(cfg, 0, targets="agree", seeds_sample=range(12))


def test_c2_single_stream():
    swaps = run_case(synth.CONFIGS["c2"], 0)
    print("c2 near-tie swaps:", swaps)


def test_c2_agree_targets():
    run_case(synth.CONFIGS["c2"], 1, targets="agree")


def test_c3_batched():
    swaps = run_case(synth.CONFIGS["c3"], 0, targets="plant")
    print("c3 near-tie swaps:", swaps)


def test_c4_reduced_batch_wide_tree():
    cfg = synth.CONFIGS["c4"].replace(B=4)
    swaps = run_case(cfg, 0, targets="plant")
    print("c4(B=4) near-tie swaps:", swaps)
    assert cfg.N == 256 and (cfg.N + 31) // 32 == 8          # 256 mask bits per node


def test_c5_reduced_batch_sampling():
    cfg = synth.CONFIGS["c5"].replace(B=3)
    run_case(cfg, 0, targets="agree", seeds_sample=(0, 7))


def test_paper_search_configuration_k64_w12():
    # the paper's academic setup (Appendix B): K = 64, W = 12, 64 non-root nodes, 15 future positions.
    # L = 8 keeps the whole pair table in shared memory, L = 15 goes through the on-demand row cache.
    for L in (8, 15):
        cfg = synth.Config("paper", 2, L, 4096, 64, 65, "bf16", "pos_uniform:0.5,4", 1.0, 0.0, "greedy")
        run_case(cfg, 0, W=12)
        run_case(cfg, 1, W=0)
        run_case(cfg, 2, W=12, zeta=-0.125, use_opts=True)
        run_case(cfg, 3, W=3)        # deep narrow tree: siblings at depth 11, where 6-bit rank fields of the
        run_case(cfg, 8, W=7)        # packed path key straddle its two 64-bit words
    # the largest shape of the interface: every limit at its maximum
    cfg = synth.Config("max", 1, 64, 4096, 64, 256, "bf16", "pos_uniform:0.5,4", 1.0, 0.0, "greedy")
    run_case(cfg, 3, W=0)
    run_case(cfg, 4, W=5)


@pytest.mark.parametrize("V,k,L,N,dtype", [
    (1000, 4, 4, 16, "bf16"),     # aligned bf16, tiny
    (1001, 4, 3, 9, "bf16"),      # V not a multiple of 8: scalar path
    (1003, 5, 3, 9, "f32"),       # V not a multiple of 4: scalar path
    (37, 8, 2, 5, "f32"),         # V smaller than a tile
    (64, 64, 2, 33, "f32"),       # k == V == 64
    (3000, 1, 5, 4, "bf16"),      # k = 1: a chain
    (2048, 3, 1, 4, "f32"),       # L = 1: no bigram tensor
    (500, 4, 4, 1, "f32"),        # N = 1: root only
    (70001, 16, 6, 200, "bf16"),  # several spans per row, ragged tail, scalar path
    (70000, 16, 6, 256, "bf16"),  # several spans per row, vector path
])
def test_edge_shapes(V, k, L, N, dtype):
    cfg = synth.Config("edge", 3, L, V, k, N, dtype, "pos_uniform:0.5,3", 1.0, 0.0, "greedy")
    run_case(cfg, 5, targets="plant")
    run_case(cfg.replace(mode="sample"), 5, targets="agree", seeds_sample=(3,))


@pytest.mark.parametrize("block", range(12))
def test_random_shapes_both_table_modes(block):
    """Shapes drawn over the whole range of the interface (k <= 64, L <= 64, N <= 256, any W), so that bit
    fields, table modes (resident / on-demand rows), slot counts and sub-warp group sizes meet in combinations
    no hand-picked case covers."""
    rng = np.random.default_rng(1000 + block)
    for _ in range(7):
        k = int(rng.choice([1, 2, 3, 5, 8, 13, 16, 24, 32, 33, 47, 64]))
        L = int(rng.choice([1, 2, 3, 7, 11, 16, 23, 32, 48, 64]))
        N = int(rng.choice([1, 2, 5, 16, 33, 64, 65, 100, 129, 256]))
        W = int(rng.choice([0, 0, 1, 2, 5, 12, 40]))
        V = max(int(rng.choice([64, 264, 999, 1001, 1000, 4096, 40000])), k + 3)   # odd V: plain-load kernels
        dtype = "bf16" if rng.random() < 0.5 else "f32"
        zeta = float(rng.choice([0.0, 0.0, -0.05]))
        cfg = synth.Config("rnd", int(rng.integers(1, 4)), L, V, k, N, dtype, "pos_uniform:0.5,4", 1.0, 0.0,
                           "greedy" if rng.random() < 0.7 else "sample")
        try:
            run_case(cfg, int(rng.integers(0, 1 << 20)), targets="agree" if rng.random() < 0.5 else "plant",
                     W=W, zeta=zeta, use_opts=bool(rng.random() < 0.5))
        except AssertionError as e:
            raise AssertionError(f"shape k={k} L={L} N={N} W={W} V={V} {dtype} zeta={zeta} {cfg.mode}: {e}") from e


@pytest.mark.parametrize("k,N,seed", [(8, 48, 0), (16, 96, 1), (6, 40, 2)])
def test_deep_chains_open_rows_beyond_the_positions_prepared_up_front(k, N, seed):
    """L = 28 positions with one dominant token per position: the tree is a few long chains, so the expansion
    appends nodes deeper than the positions whose rows the tree kernel prepares before it starts."""
    cfg = synth.CONFIGS["c2"].replace(name="deep", B=3, L=28, N=N, k=k, V=4096, scale="fixed:0.5", spike=12.0,
                                      bigram_std=0.3)
    di = synth.draft_inputs(cfg, seed)
    otree = oracle.draft_tree(di.unigram_logits, di.bigram_scores, cfg.k, cfg.N)
    assert int(otree.depths.max()) >= 20
    run_case(cfg, seed, targets="agree")
    run_case(cfg, seed, targets="plant", use_opts=True)


def test_rows_full_of_ties():
    # bf16 rows quantised to a handful of values, rows with +-0 at the top, a constant row
    u = ubt()
    rng = np.random.default_rng(0)
    V, k = 4096, 8
    x = np.round(rng.standard_normal((6, V)) * 2).astype(np.float32)
    x[1, :] = 0.75
    x[2] = -np.abs(x[2]); x[2, 100] = 0.0; x[2, 50] = -0.0
    x[3, ::3] = x[3].max()
    for dtype in ("bf16", "f32"):
        host = synth.f32_to_bf16_bits(x) if dtype == "bf16" else x
        ids, lp, _ = oracle.topk_logprob(host, k)
        d = synth.to_device(host, dtype, DEV)
        cid = torch.empty((6, k), dtype=torch.int32, device=DEV)
        clp = torch.empty((6, k), dtype=torch.float32, device=DEV)
        ws = u.workspace(u.ubt_draft_workspace_bytes(6, 1, V, k, 1), DEV)
        u.ubt_topk_logprob(d, k, cid, clp, ws)
        torch.cuda.synchronize()
        assert cid.cpu().numpy().tolist() == ids.tolist()
        np.testing.assert_allclose(clp.cpu().numpy(), lp, rtol=1e-5, atol=1e-5)
        # greedy picks on the same rows: lowest token among the maxima
        tree = u.Tree.empty(1, 6, 1, 1, DEV)
        for t in (tree.token_ids, tree.parents):
            t.fill_(-1)
        tree.n_nodes.fill_(1)
        pick = torch.empty((1, 6), dtype=torch.int32, device=DEV)
        u.ubt_verify_tree(tree, d.view(1, 6, V), "greedy", node_pick=pick)
        torch.cuda.synchronize()
        assert pick.cpu().numpy()[0].tolist() == np.argmax(synth.as_f32(host, dtype), -1).tolist()


def test_rows_whose_level_jumps_inside_one_warps_share():
    """Rows built against the streaming kernel's layout: a chunk of zeros, then a chunk in which only the
    elements that one warp reads are at 100 (so the CTA-wide bound rises to 100 without the other warps ever
    seeing a candidate), then a chunk of 95s, which are no candidates but lie far above those warps' exponent
    reference.  The sum of exponentials must survive that."""
    u = ubt()
    V, k, rows = 65536, 8, 512
    chunk, frag = 16384, 8
    e = np.arange(V)
    row = np.zeros(V, np.float32)
    in1 = (e >= chunk) & (e < 2 * chunk)
    row[in1 & (((e % chunk) // frag) % 256 < 32)] = 100.0
    row[(e >= 2 * chunk) & (e < 3 * chunk)] = 95.0
    rng = np.random.default_rng(3)
    x = np.tile(row, (rows, 1)) + rng.integers(0, 4, (rows, V)).astype(np.float32) * 0.25
    host = synth.f32_to_bf16_bits(x)
    ids, lp, _ = oracle.topk_logprob(host, k)
    d = synth.to_device(host, "bf16", DEV)
    cid = torch.empty((rows, k), dtype=torch.int32, device=DEV)
    clp = torch.empty((rows, k), dtype=torch.float32, device=DEV)
    ws = u.workspace(u.ubt_draft_workspace_bytes(rows, 1, V, k, 1), DEV)
    u.ubt_topk_logprob(d, k, cid, clp, ws)
    torch.cuda.synchronize()
    assert np.array_equal(cid.cpu().numpy(), ids)
    np.testing.assert_allclose(clp.cpu().numpy(), lp, rtol=1e-5, atol=1e-5)


@pytest.mark.parametrize("rows,V,k,dtype,kind", [
    (8, 98304, 64, "bf16", "levels"),      # every (thread, chunk) group holds the maximum: the group list overflows
    (3, 98304, 16, "bf16", "plateau"),     # 300 elements equal to the maximum: the candidate pool overflows
    (4, 300000, 16, "f32", "normal"),      # 37 chunks per row: the eight maxima slots of a thread wrap four times
    (2, 2200000, 8, "f32", "normal"),      # more than 256 chunks per row: beyond what a list entry can name
    (40, 30000, 64, "bf16", "normal"),     # k = 64: several groups per warp, short segments at the span borders
    (5, 16392, 16, "bf16", "normal"),      # a second chunk of one fragment
])
def test_topk_rows_that_leave_the_streaming_kernels_common_path(rows, V, k, dtype, kind):
    u = ubt()
    rng = np.random.default_rng(rows * 7 + k)
    if kind == "levels":
        x = rng.integers(0, 4, (rows, V)).astype(np.float32)
    elif kind == "plateau":
        x = rng.standard_normal((rows, V)).astype(np.float32)
        for r in range(rows):
            x[r, rng.choice(V, 300, replace=False)] = 9.0
    else:
        x = (rng.standard_normal((rows, V)) * 2.5).astype(np.float32)
    host = synth.f32_to_bf16_bits(x) if dtype == "bf16" else x
    ids, lp, _ = oracle.topk_logprob(host, k)
    d = synth.to_device(host, dtype, DEV)
    cid = torch.empty((rows, k), dtype=torch.int32, device=DEV)
    clp = torch.empty((rows, k), dtype=torch.float32, device=DEV)
    ws = u.workspace(u.ubt_draft_workspace_bytes(rows, 1, V, k, 1), DEV)
    u.ubt_topk_logprob(d, k, cid, clp, ws)
    torch.cuda.synchronize()
    assert np.array_equal(cid.cpu().numpy(), ids)
    np.testing.assert_allclose(clp.cpu().numpy(), lp, rtol=1e-5, atol=2e-5)


@pytest.mark.parametrize("rows,V,k,dtype", [
    (700, 16384, 16, "bf16"), (700, 16376, 7, "bf16"), (333, 32776, 33, "bf16"), (97, 49152, 64, "bf16"),
    (1200, 8200, 1, "bf16"), (450, 16388, 16, "f32"), (130, 40964, 64, "f32"), (64, 151936, 50, "bf16"),
    (9, 151936, 3, "f32")])
def test_topk_rows_cut_at_chunk_and_span_borders(rows, V, k, dtype):
    """Vocabularies one fragment off a multiple of the 32 KiB chunk, row counts that put the span borders (and
    with them very short row segments) at ever different columns."""
    u = ubt()
    rng = np.random.default_rng(rows + V + k)
    x = (rng.standard_normal((rows, V)) * rng.uniform(0.3, 6.0, (rows, 1))).astype(np.float32)
    host = synth.f32_to_bf16_bits(x) if dtype == "bf16" else x
    ids, lp, _ = oracle.topk_logprob(host, k)
    d = synth.to_device(host, dtype, DEV)
    cid = torch.empty((rows, k), dtype=torch.int32, device=DEV)
    clp = torch.empty((rows, k), dtype=torch.float32, device=DEV)
    ws = u.workspace(u.ubt_draft_workspace_bytes(rows, 1, V, k, 1), DEV)
    u.ubt_topk_logprob(d, k, cid, clp, ws)
    torch.cuda.synchronize()
    assert np.array_equal(cid.cpu().numpy(), ids)
    np.testing.assert_allclose(clp.cpu().numpy(), lp, rtol=1e-5, atol=2e-5)


def test_exact_score_ties_follow_total_order():
    # integer-valued inputs with lambda = 0: many node scores are exactly equal in fp32 and in double
    u = ubt()
    rng = np.random.default_rng(3)
    B, L, V, k, N = 4, 4, 64, 3, 12
    x = np.round(rng.standard_normal((B, L, V)) * 2).astype(np.float32)
    big = np.zeros((B, L - 1, k, k), np.float32)
    lam = np.zeros(L, np.float32)
    otree = oracle.draft_tree(x, big, k, N, lam=lam)
    gtree = u.ubt_draft_tree(torch.from_numpy(x).to(DEV), torch.from_numpy(big).to(DEV), k, N,
                             lam=torch.from_numpy(lam).to(DEV))
    torch.cuda.synchronize()
    compare_draft(tree_to_numpy(gtree), otree, L, k, N)


@pytest.mark.parametrize("L,V,k,N,W", [(4, 64, 4, 12, 0), (4, 64, 4, 12, 2), (4, 64, 4, 12, 5), (5, 128, 20, 40, 0),
                                       (5, 128, 20, 40, 4), (6, 128, 40, 60, 6), (15, 256, 64, 65, 12),
                                       (15, 256, 64, 65, 0), (6, 64, 8, 30, 3), (8, 128, 16, 100, 16)])
def test_duplicated_values_tie_exactly_in_every_form_of_the_expansion(L, V, k, N, W):
    """Every logit value occurs twice (tokens 2j and 2j + 1) and lambda = 0, so that the rows of a position do not
    depend on the predecessor: the two tokens of a pair tie inside every row, sibling nodes of a pair have equal
    scores, and so have their children of equal rank under either of them -- ties inside a row, across parents
    and across the final cut, all exact in double and in fp32 alike because the tied values come from identical
    operations.  Values that are not duplicates differ by O(1).  Every form of the expansion (threshold rounds,
    depth by depth, best-first on rows prepared on demand) and of the row ranking has to settle the ties by token
    and rank path as the oracle does."""
    u = ubt()
    rng = np.random.default_rng(30 + k + W)
    B = 3
    y = (rng.standard_normal((B, L, V // 2)) * 3).astype(np.float32)
    x = np.repeat(y, 2, axis=2)
    big = np.zeros((B, L - 1, k, k), np.float32)
    lam = np.zeros(L, np.float32)
    otree = oracle.draft_tree(x, big, k, N, lam=lam, W=W)
    gtree = u.ubt_draft_tree(torch.from_numpy(x).to(DEV), torch.from_numpy(big).to(DEV), k, N,
                             lam=torch.from_numpy(lam).to(DEV), search_width=W)
    torch.cuda.synchronize()
    compare_draft(tree_to_numpy(gtree), otree, L, k, N)


def test_split_entry_points_match_fused_call():
    u = ubt()
    cfg = synth.CONFIGS["c2"].replace(V=20000)
    di = synth.draft_inputs(cfg, 2)
    ud = synth.to_device(di.unigram_logits, cfg.dtype, DEV)
    bd = torch.from_numpy(di.bigram_scores).to(DEV)
    fused = u.ubt_draft_tree(ud, bd, cfg.k, cfg.N)
    split = u.Tree.empty(cfg.B, cfg.N, cfg.L, cfg.k, DEV)
    ws = u.workspace(u.ubt_draft_workspace_bytes(cfg.B, cfg.L, cfg.V, cfg.k, cfg.N), DEV)
    u.ubt_topk_logprob(ud, cfg.k, split.cand_ids, split.cand_logprob, ws)
    u.ubt_build_tree(bd, split)
    torch.cuda.synchronize()
    for name in ("token_ids", "parents", "depths", "position_ids", "cand_rank", "mask", "n_nodes", "cand_ids"):
        assert torch.equal(getattr(fused, name), getattr(split, name)), name
    assert torch.equal(fused.scores, split.scores)
    # the standalone mask builder reproduces mask and position ids from parents/depths
    off = torch.arange(cfg.B, dtype=torch.int32, device=DEV) * 1000 + 17
    want_mask = split.mask.clone()
    split.mask.zero_(); split.position_ids.zero_()
    u.ubt_build_mask(split, off)
    torch.cuda.synchronize()
    assert torch.equal(split.mask, want_mask)
    want_pos = torch.where(fused.depths >= 0, fused.depths + off[:, None], torch.full_like(fused.depths, -1))
    assert torch.equal(split.position_ids, want_pos)


def test_host_buffer_entry_points():
    u = ubt()
    cfg = synth.CONFIGS["c1"].replace(B=3, V=5000, dtype="bf16")
    di = synth.draft_inputs(cfg, 4)
    uh = synth.to_device(di.unigram_logits, cfg.dtype, "cpu").pin_memory()
    bh = torch.from_numpy(di.bigram_scores).pin_memory()
    tree_h = u.Tree.empty(cfg.B, cfg.N, cfg.L, cfg.k, DEV, pin=True)
    buf = u.workspace(u.ubt_draft_host_buffer_bytes(cfg.B, cfg.L, cfg.V, cfg.k, cfg.N, 1), DEV)
    u.ubt_draft_tree_host(uh, bh, cfg.k, cfg.N, tree_h, buf)
    otree = oracle.draft_tree(di.unigram_logits, di.bigram_scores, cfg.k, cfg.N)
    g = tree_to_numpy(tree_h)
    compare_draft(g, otree, cfg.L, cfg.k, cfg.N)
    z = synth.target_logits(cfg, 4)
    synth.plant_path(z, cfg.dtype, g.token_ids, g.parents, g.n_nodes, 4)
    zh = synth.to_device(z, cfg.dtype, "cpu").pin_memory()
    res = u.VerifyResult.empty(cfg.B, cfg.L, DEV, pin=True)
    pick = torch.empty((cfg.B, cfg.N), dtype=torch.int32).pin_memory()
    vbuf = u.workspace(u.ubt_verify_host_buffer_bytes(cfg.B, cfg.L, cfg.N, cfg.V, 1, "greedy"), DEV)
    u.ubt_verify_tree_host(tree_h, zh, res, vbuf, "greedy", node_pick=pick)
    compare_verify(res, oracle.verify(g.token_ids, g.parents, g.n_nodes, cfg.L, z, "greedy"), pick)


def test_repeat_calls_are_deterministic():
    u = ubt()
    cfg = synth.CONFIGS["c3"].replace(B=4)
    ud, bd, zd = synth.device_inputs(cfg, 3, DEV)
    a = u.ubt_draft_tree(ud, bd, cfg.k, cfg.N)
    ra = u.ubt_verify_tree(a, zd, "sample", seed=5)
    b = u.ubt_draft_tree(ud, bd, cfg.k, cfg.N)
    rb = u.ubt_verify_tree(b, zd, "sample", seed=5)
    torch.cuda.synchronize()
    for name in ("token_ids", "parents", "mask", "scores", "cand_logprob"):
        assert torch.equal(getattr(a, name), getattr(b, name)), name
    assert torch.equal(ra.accepted_len, rb.accepted_len) and torch.equal(ra.out_tokens, rb.out_tokens)
