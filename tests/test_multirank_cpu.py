"""Host-side logic of the multi-rank bench path on CPU (gloo, world size 2): the reduction that turns
per-rank timings into the whole-job number, and the rank-0-only reference arm."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank r took (10 + 5 r) ms for (100 + r) units: the job took the slowest rank's time for all the units
    ms, units = bench.reduce_over_ranks(10.0 + 5.0 * rank, 100.0 + rank)
    dist.barrier()
    dist.destroy_process_group()
    out.put((rank, ms, units))


def test_reduce_over_ranks_gloo_world2():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got == [(0, 15.0, 201.0), (1, 15.0, 201.0)]


def test_reduce_over_ranks_is_identity_without_a_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_over_ranks(3.5, 7.0) == (3.5, 7.0)


def test_rank_seeds_and_gradient_rotation_are_disjoint():
    """Every rank draws its own inputs (seed offset 10000 per rank) and the shifted gradient views
    never repeat an alignment-breaking offset."""
    sys.path.insert(0, ROOT)
    import bench
    from paper_2010_08899_b200 import inputs
    a = inputs.dp_mixture(1 << 12, 501 + 10_000 * 0)
    b = inputs.dp_mixture(1 << 12, 501 + 10_000 * 1)
    assert not torch.equal(a, b)
    cfg = bench.WORKLOADS["small"]
    shifts = {4 * ((t // cfg["dp_bufs"]) % (cfg["dp_slack"] // 4)) for t in range(200)}
    assert all(s % 4 == 0 and s + cfg["dp_n"] <= cfg["dp_n"] + cfg["dp_slack"] for s in shifts)
    assert len(shifts) == 100


def test_reference_arm_runs_on_rank0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "1", "--workload", "small"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "1", "--workload", "small"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "GB/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert line["n_gpus"] == 2 and line["steps"] == 1
