"""The multi-process path of the benchmark on CPU (gloo, world size 2): ranks draw
disjoint seeded batches, exchange nothing but their measured times, and the job
throughput is all ranks' work over the slowest rank's time."""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), WORLD_SIZE=str(world),
                      RANK=str(rank), LOCAL_RANK=str(rank))
    sys.path.insert(0, ROOT)
    from paper_1603_05279_b200 import dist_util as du
    from paper_1603_05279_b200 import workloads as wl
    w, r = du.init("gloo")
    assert (w, r) == (world, rank)
    du.barrier()
    # each rank "measures" its own times; the reduction must return the slowest
    mine = [10.0 + rank, 20.0 - rank]
    slowest = du.max_over_ranks(mine)
    x = wl.make_input(wl.SINGLE[0], du.rank_seed(wl.layer_seed("single", 0), rank))
    q.put((rank, slowest, float(x.sum()), du.job_throughput(1000, 4, w, slowest[0])))
    du.barrier()
    du.finish()


def test_two_ranks_reduce_times_and_draw_disjoint_batches():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slowest, _, thr in got:
        assert slowest == [11.0, 20.0], (rank, slowest)
        assert abs(thr - 2 * 1000 * 4 / 11e-3) < 1e-6
    assert got[0][2] != got[1][2], "ranks must not share a batch"


def test_single_process_helpers_are_identities():
    sys.path.insert(0, ROOT)
    from paper_1603_05279_b200 import dist_util as du
    assert du.max_over_ranks([3.0, 4.5]) == [3.0, 4.5]
    assert du.rank_seed(1000, 0) == 1000 and du.rank_seed(1000, 3) == 301000
    assert du.job_throughput(10, 5, 1, 1000.0) == 50.0
    du.barrier()          # no process group: a no-op


def _bench(args, env_extra=None):
    env = dict(os.environ)
    env.update(env_extra or {})
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + args, env=env,
                          capture_output=True, text=True, timeout=600)


def test_reference_arm_prints_one_line_on_rank_zero_only():
    r = _bench(["--impl", "reference", "--workload", "single", "--steps", "2", "--warmup", "1"])
    assert r.returncode == 0, r.stderr
    lines = [l for l in r.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    j = json.loads(lines[0])
    assert j["impl"] == "reference" and j["gpu_launches"] == 0
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step",
                "higher_is_better", "scaling", "vs_baseline", "dtype", "data", "config",
                "cpu_baseline", "e2e"):
        assert key in j, key
    assert j["cpu_baseline"]["kind"] == "oracle" and j["cpu_baseline"]["cores"] >= 1
    assert j["e2e"]["value"] == j["value"] and j["e2e"]["h2d_bytes_per_step"] == 0
    assert j["value"] > 0 and np.isfinite(j["value"])
    # another rank of the same launch does no work and prints nothing
    r1 = _bench(["--impl", "reference", "--workload", "single", "--steps", "1"],
                {"RANK": "1", "WORLD_SIZE": "2", "LOCAL_RANK": "1"})
    assert r1.returncode == 0 and r1.stdout.strip() == ""


def test_bench_without_a_gpu_fails_loudly():
    import torch
    if torch.cuda.is_available():
        return
    r = _bench(["--steps", "1", "--workload", "single"])
    assert r.returncode != 0 and "CUDA" in (r.stderr + r.stdout)
