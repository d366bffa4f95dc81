"""Full-size configurations in the launch configuration the benchmark times, every sequence checked.

Inputs of 0.8-5.6 GB are drawn on the device (seeded torch generator) and copied back bit for bit, so both sides
read the same bytes.  The oracle drafts every sequence and walks every tree (evaluating only the target rows a
walk visits); the picks at every slot are compared on eight sequences.
"""
import numpy as np
import pytest
import torch

import oracle
import ubt_synth as synth
from parity import compare_draft, compare_verify, tree_to_numpy

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _run_full(name, pick_rows, seeds=(0,)):
    """Every sequence of the full batch: the draft against the oracle, and the walk against the oracle's own lazy
    walk (which evaluates only the rows it visits).  ``pick_rows``: sequences whose picks at EVERY slot are
    compared as well."""
    import paper_2609_39972_b200 as u
    cfg = synth.CONFIGS[name]
    ud, bd, zd = synth.device_inputs(cfg, 11, DEV)
    gtree = u.ubt_draft_tree(ud, bd, cfg.k, cfg.N)
    torch.cuda.synchronize()
    g = tree_to_numpy(gtree)
    otree = oracle.draft_tree(synth.to_host_bits(ud), synth.to_host_bits(bd), cfg.k, cfg.N)
    del ud, bd
    swaps = compare_draft(g, otree, cfg.L, cfg.k, cfg.N)
    print(f"{name}: near-tie swaps over the whole batch: {swaps}")
    zh = synth.to_host_bits(zd)
    pick = torch.empty((cfg.B, cfg.N), dtype=torch.int32, device=DEV)
    rows = sorted(pick_rows)
    zr = zh[rows]
    for s in seeds:
        res = u.ubt_verify_tree(gtree, zd, cfg.mode, seed=s, node_pick=pick)
        torch.cuda.synchronize()
        # the oracle numbers sequences by their place in the arrays it is given: the whole batch keeps b true
        ov = oracle.verify(g.token_ids, g.parents, g.n_nodes, cfg.L, zh, cfg.mode, seed=s, all_nodes=False)
        compare_verify(res, ov)
        res_p = u.ubt_verify_tree(gtree, zd, cfg.mode, seed=s, path_only=True)     # visits the walk's rows only
        torch.cuda.synchronize()
        compare_verify(res_p, ov)
        if cfg.mode == "greedy":
            sub = lambda a: a[rows]
            ov8 = oracle.verify(sub(g.token_ids), sub(g.parents), sub(g.n_nodes), cfg.L, zr, "greedy")
        else:
            ov8 = _oracle_sample_rows(g, zr, rows, cfg, s)
        compare_verify(res, ov8, pick, rows=rows)
    # properties that hold at any size, on the whole batch
    n = g.n_nodes
    assert np.all(n >= 1) and np.all(n <= cfg.N)
    par = g.parents
    idx = np.arange(cfg.N)[None, :]
    assert np.all((par < idx) | (idx >= n[:, None]))
    acc = res.accepted_len.cpu().numpy()
    assert np.all(acc >= 0) and np.all(acc <= cfg.L)
    pk = pick.cpu().numpy()
    assert pk.min() >= 0 and pk.max() < cfg.V
    if cfg.mode == "greedy":
        # sampled rows of the full batch against a library argmax on the device copy
        rr = np.random.default_rng(0).integers(0, cfg.B * cfg.N, 64)
        flat = zd.view(cfg.B * cfg.N, cfg.V)
        for r in rr:
            assert int(torch.argmax(flat[r].float())) == pk.reshape(-1)[r] or \
                flat[r, pk.reshape(-1)[r]] == flat[r].max()


_CDF_CACHE = {}


def _oracle_sample_rows(g, zh, rows, cfg, seed):
    """Oracle sampling verdicts for sampled sequences, each under its TRUE batch index.

    The draw is keyed by (seed, b, n) and the oracle's whole-batch call numbers sequences by their
    position in the array it is given, so the sampled sequences go through its row-level primitives:
    row CDF, threshold of (seed, b, n), first token whose prefix sum exceeds it, then the walk.
    """
    acc, bonus, nodes, toks, picks = [], [], [], [], []
    for j, b in enumerate(rows):
        if (id(zh), j) not in _CDF_CACHE:
            _CDF_CACHE[(id(zh), j)] = np.stack([oracle.row_cdf(zh[j], n) for n in range(cfg.N)])
        cdf = _CDF_CACHE[(id(zh), j)]
        pk = np.array([int(np.searchsorted(cdf[n], oracle.threshold(seed, b, n, int(cdf[n, -1])), side="right"))
                       for n in range(cfg.N)], np.int32)
        a, bo = oracle.walks_from_cdf(g.token_ids[b], g.parents[b], int(g.n_nodes[b]), cdf, b,
                                      np.array([seed], np.uint64))
        cur, an, ot = 0, [0], []
        for _ in range(int(a[0])):
            x = pk[cur]
            cur = [c for c in range(1, int(g.n_nodes[b])) if g.parents[b, c] == cur and g.token_ids[b, c] == x][0]
            an.append(cur); ot.append(int(x))
        ot.append(int(bo[0]))
        pad = lambda v: v + [-1] * (cfg.L + 1 - len(v))
        acc.append(int(a[0])); bonus.append(int(bo[0])); nodes.append(pad(an)); toks.append(pad(ot)); picks.append(pk)
    return oracle.Verdict(np.array(acc, np.int32), np.array(nodes, np.int32), np.array(toks, np.int32),
                          np.array(bonus, np.int32), np.stack(picks))


def test_c3_full_batch():
    _run_full("c3", pick_rows=range(32))


def test_c4_full_batch():
    _run_full("c4", pick_rows=[0, 9, 17, 26, 35, 44, 53, 63])


def test_c5_full_batch():
    _run_full("c5", pick_rows=[0, 18, 36, 54, 72, 90, 108, 127], seeds=(0, 12345))
    _CDF_CACHE.clear()


def _same_tree(a, b):
    for name in ("token_ids", "parents", "depths", "position_ids", "cand_rank", "scores", "mask", "n_nodes",
                 "cand_ids", "cand_logprob"):
        assert torch.equal(getattr(a, name), getattr(b, name)), name


def _same_result(a, b):
    for name in ("accepted_len", "bonus_token", "accepted_nodes", "out_tokens"):
        assert torch.equal(getattr(a, name), getattr(b, name)), name


@pytest.mark.parametrize("early", [False, True])
@pytest.mark.parametrize("name", ["c3", "c5"])
def test_back_to_back_calls_equal_separated_calls(name, early):
    """Draft and verify enqueued with nothing between them; with ``early_start`` they run overlapped on the device
    (the verify call's V-wide kernel starts while the draft's kernels are still running).  Either way the outcome
    must be bit-identical to the same calls separated by a synchronisation, which the tests above check against
    the oracle."""
    import paper_2609_39972_b200 as u
    cfg = synth.CONFIGS[name].replace(B=32)
    ud, bd, zd = synth.device_inputs(cfg, 5, DEV)
    t_ref = u.ubt_draft_tree(ud, bd, cfg.k, cfg.N)
    torch.cuda.synchronize()
    r_ref = u.ubt_verify_tree(t_ref, zd, cfg.mode, seed=3)
    torch.cuda.synchronize()
    for _ in range(3):
        t = u.ubt_draft_tree(ud, bd, cfg.k, cfg.N)
        r = u.ubt_verify_tree(t, zd, cfg.mode, seed=3, early_start=early)
        torch.cuda.synchronize()
        _same_tree(t, t_ref)
        _same_result(r, r_ref)


def test_verify_scratch_that_reuses_a_draft_buffer_is_not_started_early():
    """Stream order allows a caller to hand the draft call's logits buffer to the verify call as scratch.  The
    library must then keep the verify kernel behind the draft even when an early start was asked for."""
    import paper_2609_39972_b200 as u
    cfg = synth.CONFIGS["c3"]
    ud, bd, zd = synth.device_inputs(cfg, 6, DEV)
    t_ref = u.ubt_draft_tree(ud, bd, cfg.k, cfg.N)
    torch.cuda.synchronize()
    r_ref = u.ubt_verify_tree(t_ref, zd, "greedy")
    torch.cuda.synchronize()
    need = u.ubt_verify_workspace_bytes(cfg.B, cfg.N, cfg.V, "greedy")
    for _ in range(3):
        scratch = ud.clone()
        ws = scratch.view(torch.uint8).reshape(-1)
        assert ws.numel() >= need
        t = u.ubt_draft_tree(scratch, bd, cfg.k, cfg.N)
        r = u.ubt_verify_tree(t, zd, "greedy", ws=ws, early_start=True)        # overwrites the draft's logits
        torch.cuda.synchronize()
        _same_tree(t, t_ref)
        _same_result(r, r_ref)
