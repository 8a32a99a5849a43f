"""Multi-process paths on the CPU (gloo, world size 2).

The search does not shard in this build: `bench.py --gpus N` runs replicas.  What a sharded run would
need is the tiling sub-range of the objective (t_begin, t_end) plus one all-gather of k (key, idx)
pairs; that host-side logic is exercised here with the oracle standing in for the device search.
"""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import mmee_inputs as mi
import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _shard_worker(rank, world, port, out_path):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = mi.random_tiny_problem(5)
    obj = dict(cfg["searches"][0], objective=mi.OBJ_ENERGY, topk=8)
    T = oracle.make_problem(cfg["workload"], cfg["arch"], obj).T
    lo, hi = T * rank // world, T * (rank + 1) // world
    p = oracle.make_problem(cfg["workload"], cfg["arch"], dict(obj, t_begin=lo, t_end=hi))
    res = oracle.search(p, threads=1)
    mine = dict(pairs=[(r.e_key, r.idx) for r in res.topk], feasible=res.n_feasible, total=res.n_total)
    gathered = [None] * world
    dist.all_gather_object(gathered, mine)
    if rank == 0:
        merged = sorted(pair for g in gathered for pair in map(tuple, g["pairs"]))[:8]
        with open(out_path, "w") as f:
            json.dump(dict(merged=merged, feasible=sum(g["feasible"] for g in gathered),
                           total=sum(g["total"] for g in gathered)), f)
    dist.barrier()
    dist.destroy_process_group()


def test_tiling_ranges_shard_the_search_across_two_ranks(tmp_path):
    out = str(tmp_path / "merged.json")
    mp.spawn(_shard_worker, args=(2, 29517, out), nprocs=2, join=True)
    got = json.load(open(out))
    cfg = mi.random_tiny_problem(5)
    obj = dict(cfg["searches"][0], objective=mi.OBJ_ENERGY, topk=8)
    whole = oracle.search(oracle.make_problem(cfg["workload"], cfg["arch"], obj))
    assert [tuple(p) for p in got["merged"]] == [(r.e_key, r.idx) for r in whole.topk]
    assert got["feasible"] == whole.n_feasible and got["total"] == whole.n_total


def test_reference_arm_under_two_ranks_prints_one_line():
    """Launched the way the scaling run launches it: rank 0 alone measures and prints."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", "29519", os.path.join(ROOT, "bench.py"),
           "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0", "--workload", "tiny"]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["value"] > 0
    assert rec["e2e"]["h2d_bytes_per_step"] == 0 and rec["cpu_baseline"]["kind"] == "oracle"
