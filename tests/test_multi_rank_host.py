"""World-size-2 checks of the multi-GPU host logic, on CPU with the gloo backend.

The path shards by columns: each rank simulates its own column range of one problem, draws the
same peers from the shared seed, and exchanges nothing per round.  No GPU is needed to check
that (i) the shard plan tiles the global vector with counter-aligned offsets, (ii) two column
shards evolved separately (here by the oracle) reproduce the unsharded run bit for bit, traces
included, (iii) the reductions bench.py performs across ranks (max of the elapsed time, sum of
the telemetry) behave, and (iv) the reference arm prints on rank 0 only."""
import json
import os
import subprocess
import sys

import numpy as np
import pytest
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import torch
    import bench
    from oracle import oracle
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    M, d, rounds, seed = 4, 1003, 7, 99
    plan = bench.shard_plan(d, world, rank)
    rng = np.random.default_rng(5)
    P = rng.random((M, M)) + 0.1
    np.fill_diagonal(P, 0.0)
    P /= P.sum(axis=1, keepdims=True)
    adj = (1 - np.eye(M)).astype(np.uint8)
    cols = plan["element_offset"] + np.arange(plan["d"], dtype=np.int64)
    sim = oracle.Sim(M, plan["global_d"], P, adj, alpha=0.05, rho=1.0, sigma=0.1, objective=1, seed=seed, cols=cols)
    sim.init(1.0, 1.0)
    sim.round(rounds)
    cons, loss = sim.telemetry()
    tel = torch.tensor(np.stack([cons, loss]))
    dist.all_reduce(tel, op=dist.ReduceOp.SUM)          # telemetry is additive over column shards
    elapsed = torch.tensor([10.0 + rank], dtype=torch.float64)
    dist.all_reduce(elapsed, op=dist.ReduceOp.MAX)      # timing is the max over ranks
    np.savez(os.path.join(out_dir, f"rank{rank}.npz"), x=sim.x(), trace=sim.trace(), tel=tel.numpy(),
             elapsed=elapsed.numpy(), offset=plan["element_offset"], global_d=plan["global_d"])
    dist.barrier()
    dist.destroy_process_group()


def test_column_shards_reproduce_the_unsharded_run(tmp_path):
    sys.path.insert(0, ROOT)
    import bench
    from oracle import oracle
    world, port = 2, 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    parts = [np.load(tmp_path / f"rank{r}.npz") for r in range(world)]
    M, d, rounds, seed = 4, 1003, 7, 99
    global_d = int(parts[0]["global_d"])
    assert [int(p["offset"]) for p in parts] == [0, 1004] and global_d == 2008
    for p in parts:
        assert int(p["offset"]) % 4 == 0 and float(p["elapsed"][0]) == 11.0
    rng = np.random.default_rng(5)
    P = rng.random((M, M)) + 0.1
    np.fill_diagonal(P, 0.0)
    P /= P.sum(axis=1, keepdims=True)
    adj = (1 - np.eye(M)).astype(np.uint8)
    cols = np.concatenate([int(p["offset"]) + np.arange(d, dtype=np.int64) for p in parts])
    whole = oracle.Sim(M, global_d, P, adj, alpha=0.05, rho=1.0, sigma=0.1, objective=1, seed=seed, cols=cols)
    whole.init(1.0, 1.0)
    whole.round(rounds)
    assert (np.concatenate([p["x"] for p in parts], axis=1) == whole.x()).all()
    assert (parts[0]["trace"] == parts[1]["trace"]).all() and (parts[0]["trace"] == whole.trace()).all()
    cons, loss = whole.telemetry()
    # loss is a plain sum over columns; so is the consensus distance (a sum of per-column variances)
    np.testing.assert_allclose(parts[0]["tel"][0], cons, rtol=1e-12)
    np.testing.assert_allclose(parts[0]["tel"][1], loss, rtol=1e-12)
    assert (parts[0]["tel"] == parts[1]["tel"]).all()


def test_shard_plan_tiles_the_global_vector():
    sys.path.insert(0, ROOT)
    import bench
    for d in (1, 3, 4, 1003, 11_173_962):
        for world in (1, 2, 4, 8):
            plans = [bench.shard_plan(d, world, r) for r in range(world)]
            d4 = (d + 3) // 4 * 4
            assert [p["element_offset"] for p in plans] == [r * d4 for r in range(world)]
            assert all(p["d"] == d and p["global_d"] == world * d4 for p in plans)


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, WORLD_SIZE="2", LOCAL_RANK="1", RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "3", "--warmup", "3", "--workload", "cfg1"], env=env, capture_output=True,
                         text=True, timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""
    env = dict(os.environ, WORLD_SIZE="2", LOCAL_RANK="0", RANK="0")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "3", "--warmup", "3", "--workload", "cfg1"], env=env, capture_output=True,
                         text=True, timeout=300)
    assert out.returncode == 0
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
