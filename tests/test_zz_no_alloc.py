"""ubt_verify_tree_static: the greedy verification that takes no workspace and allocates nothing.

It exists for callers that cannot allocate device memory where they verify (a fully handed-out memory pool, a
plugin that only receives its buffers, a loop that must avoid cudaMalloc's implicit synchronisation).  Its
scratch is a fixed array inside libubt.so that every call reuses, so the test calls it twice in a row on
different inputs and compares each result, through the C ABI, with ubt_verify_tree on the same inputs and with
the CPU oracle's walk of the same tree.
Collected last on purpose: a run that stops at the first failure has then already run every other test.
"""
import ctypes as C

import pytest
import torch

import oracle
import ubt_synth as synth
from parity import compare_verify, tree_to_numpy

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _same(a, b):
    for name in ("accepted_len", "bonus_token", "accepted_nodes", "out_tokens"):
        assert torch.equal(getattr(a, name), getattr(b, name)), name


def test_static_scratch_entry_point_matches_workspace_entry_point_twice_in_a_row():
    import paper_2609_39972_b200 as u
    cfg = synth.CONFIGS["c3"].replace(B=5, V=40000)
    results = []
    for call, seed in enumerate((21, 22)):
        ud, bd, zd = synth.device_inputs(cfg, seed, DEV)
        tree = u.ubt_draft_tree(ud, bd, cfg.k, cfg.N)
        # make the walks non-trivial: the row of every slot gets its first child's token as the maximum
        par, tok = tree.parents.long(), tree.token_ids.long()
        for b in range(cfg.B):
            for c in range(int(tree.n_nodes[b]) - 1, 0, -1):
                zd[b, par[b, c], tok[b, c]] = 60.0 + (c % 3)
        want_pick = torch.empty((cfg.B, cfg.N), dtype=torch.int32, device=DEV)
        want = u.ubt_verify_tree(tree, zd, "greedy", node_pick=want_pick)
        got_pick = torch.full((cfg.B, cfg.N), -7, dtype=torch.int32, device=DEV)
        got = u.VerifyResult.empty(cfg.B, cfg.L, DEV)
        for t in (got.accepted_len, got.bonus_token, got.accepted_nodes, got.out_tokens):
            t.fill_(-7)
        u.ubt_verify_tree_static(tree, zd, node_pick=got_pick, result=got)
        torch.cuda.synchronize()
        _same(got, want)
        assert torch.equal(got_pick, want_pick)
        g = tree_to_numpy(tree)
        compare_verify(got, oracle.verify(g.token_ids, g.parents, g.n_nodes, cfg.L, synth.to_host_bits(zd), "greedy"),
                       got_pick)
        assert int(got.accepted_len.max()) >= 1
        results.append(got.out_tokens.clone())
    assert not torch.equal(results[0], results[1])          # the two calls really saw different inputs


def test_static_scratch_rejects_oversized_requests_before_launching():
    import paper_2609_39972_b200 as u
    from paper_2609_39972_b200 import binding
    lib = u.load()
    assert u.ubt_verify_static_capacity() == 65536
    # 40,000 rows need 80,000 keys: refused on the host with the dedicated status, pointers never touched
    tree = binding._Tree(200, 200, 4, 4, 7, *([0x1000] * 10))
    res = binding._VerifyResult(0x1000, 0x1000, 0x1000, 0x1000)
    rc = lib.ubt_verify_tree_static(C.byref(tree), C.c_void_p(0x1000), 1, 151936, None, C.byref(res), None)
    assert rc == 5 and "built-in scratch" in u.status_string(rc)
