"""Host-side logic of the multi-GPU benchmark path, run as two gloo ranks on CPU.

The hot path shards by sequence with no data-path collective (weak scaling): every rank runs the same step
on its own batch, and the only exchanges are the barrier around the timed region and the max-over-ranks of
the measured time.  These tests cover exactly that plumbing plus the reference arm under a two-rank launch.
"""
import json
import os
import socket
import subprocess
import sys

import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank: int, world: int, port: int, out_dir: str):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    import bench
    w, r, local = bench.dist_setup(world)
    assert (w, r, local) == (world, rank, rank)
    bench.barrier(w)
    # every rank times its own steps; the job's time is the slowest rank's
    mine = 10.0 + 2.5 * rank
    job = bench.max_over_ranks(mine, w, torch.device("cpu"))
    # whole-job throughput = units of all ranks / that time
    trees = 32 * 4 * w / (job * 1e-3)
    with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
        json.dump({"job_ms": job, "trees_per_s": trees}, f)
    bench.barrier(w)
    import torch.distributed as dist
    dist.destroy_process_group()


@pytest.mark.timeout(180)
def test_max_over_ranks_and_barrier_two_gloo_ranks(tmp_path):
    port = _free_port()
    mp.spawn(_rank_main, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    got = [json.load(open(tmp_path / f"rank{r}.json")) for r in range(2)]
    assert got[0] == got[1]
    assert got[0]["job_ms"] == 12.5
    assert got[0]["trees_per_s"] == pytest.approx(32 * 4 * 2 / 12.5e-3)


@pytest.mark.timeout(300)
def test_reference_arm_under_a_two_rank_launch_prints_one_line():
    port = _free_port()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.join(ROOT, "bench.py"),
           "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "3", "--workload", "c1"]
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="")
    p = subprocess.run(cmd, capture_output=True, text=True, cwd=ROOT, env=env, timeout=280)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [json.loads(l) for l in p.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    line = lines[0]
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert line["config"]["workload"] == "c1"


@pytest.mark.timeout(300)
def test_bare_command_with_gpus_2_starts_two_ranks_itself():
    """`python bench.py --gpus 2` outside any launcher must spawn the two ranks and report n_gpus = 2."""
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
           "--warmup", "3", "--workload", "c1"]
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_PORT")}
    env["CUDA_VISIBLE_DEVICES"] = ""
    p = subprocess.run(cmd, capture_output=True, text=True, cwd=ROOT, env=env, timeout=280)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [json.loads(l) for l in p.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1 and lines[0]["n_gpus"] == 2 and lines[0]["impl"] == "reference"


def test_default_invocation_measures_the_largest_configuration_first():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.WORKLOADS_DEFAULT[0] == "c4" and set(bench.WORKLOADS_DEFAULT) == {"c3", "c4", "c5"}


def test_ranks_draw_different_batches():
    """Weak scaling: rank r's input set s is seeded 1000 r + s, so no two ranks stream the same bytes."""
    sys.path.insert(0, ROOT)
    import bench
    seeds = {bench.input_seed(r, s) for r in range(8) for s in range(16)}
    assert len(seeds) == 8 * 16


# ---- vocabulary-parallel step a1: the all-gather of the ranks' partials (layout and rank order)
def _shard_rank_main(rank: int, world: int, port: int, out_dir: str):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, ROOT); sys.path.insert(0, os.path.join(ROOT, "tests"))
    import numpy as np
    import torch.distributed as dist
    import oracle
    import shard_layout
    import paper_2609_39972_b200 as u
    dist.init_process_group("gloo", rank=rank, world_size=world)
    rows, V, k = 9, 600, 5
    rng = np.random.Generator(np.random.PCG64(11))           # the same rows on every rank
    x = np.round(rng.standard_normal((rows, V)).astype(np.float32) * 4.0) / 4.0     # with ties across slices
    cuts = [0, 248, V]
    v0, v1 = cuts[rank], cuts[rank + 1]
    # this rank's partial from the oracle on its slice, packed as the header documents it
    ids, lp, lse = oracle.topk_logprob(np.ascontiguousarray(x[:, v0:v1]), k)
    val = np.take_along_axis(x[:, v0:v1], ids.astype(np.int64), axis=1)
    m = x[:, v0:v1].max(axis=1)
    s = np.exp(x[:, v0:v1].astype(np.float64) - m[:, None]).sum(axis=1)
    part = shard_layout.pack(np.stack([m, s], axis=1), val, ids + v0, np.full(rows, k, np.int32))
    assert part.size == u.ubt_topk_shard_bytes(rows, k)      # host-side query of the library
    gathered, shards = u.gather_shard_partials(torch.from_numpy(part))
    assert shards == world and gathered.numel() == world * part.size
    g_ids, g_lp = shard_layout.merge(gathered.numpy(), shards, rows, k)
    o_ids, o_lp, _ = oracle.topk_logprob(x, k)
    np.testing.assert_array_equal(g_ids, o_ids)
    np.testing.assert_allclose(g_lp, o_lp, rtol=1e-6, atol=1e-6)
    # ---- sampling a4 over the same split, on the host with the oracle's integer weights: maxima, totals and picks
    # travel through the same gather (8-, 8- and 4-byte entries per tree slot, rank order), and the picks are those
    # of whole rows
    B, N, seed, temp = 1, rows, 77, 0.9
    z = x.reshape(B, N, V)
    want = oracle.verify(np.full((B, N), -1, np.int32), np.full((B, N), -1, np.int32), np.ones(B, np.int32), 3, z,
                         "sample", seed=seed, temperature=temp).node_pick
    local_max = torch.from_numpy(x[:, v0:v1].max(axis=1).astype(np.float32))
    g_max, _ = u.gather_shard_partials(local_max)
    row_max = g_max.view(world, rows).max(dim=0).values.numpy()
    totals = np.zeros(rows, np.int64)
    cums = []
    for r_ in range(rows):
        a, c = oracle.weight_consts(float(row_max[r_]), temp)
        w = np.array([oracle.weight(float(zv), a, c) for zv in x[r_, v0:v1]], dtype=np.uint64)
        cums.append(np.cumsum(w))
        totals[r_] = int(cums[-1][-1])
    g_tot, _ = u.gather_shard_partials(torch.from_numpy(totals))
    g_tot = g_tot.view(world, rows).numpy().astype(np.uint64)
    picks = np.full(rows, -1, np.int32)
    for r_ in range(rows):
        total = int(g_tot[:, r_].sum())
        theta = oracle.threshold(seed, 0, r_, total)
        before = int(g_tot[:rank, r_].sum())
        if before <= theta < before + int(g_tot[rank, r_]):
            picks[r_] = v0 + int(np.searchsorted(cums[r_], np.uint64(theta - before), side="right"))
    g_picks, _ = u.gather_shard_partials(torch.from_numpy(picks))
    g_picks = g_picks.view(world, rows).numpy()
    assert ((g_picks >= 0).sum(axis=0) == 1).all()
    np.testing.assert_array_equal(g_picks.max(axis=0), want[0])
    with open(os.path.join(out_dir, f"shard{rank}.ok"), "w") as f:
        f.write("ok")
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.timeout(180)
def test_shard_partials_gathered_in_rank_order_two_gloo_ranks(tmp_path):
    port = _free_port()
    mp.spawn(_shard_rank_main, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    assert all((tmp_path / f"shard{r}.ok").exists() for r in range(2))
