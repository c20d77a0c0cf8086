"""The N > 1 path of bench.py on CPU: two gloo ranks on 127.0.0.1.  The frame update has no exchange
step, so ranks are independent replicas; what they share is the timing rule (maximum over ranks), the
whole-job rate, distinct seeded sequences per rank, and that only rank 0 reports."""
import os
import socket
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    import argparse
    import bench
    from workloads import data
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local = [10.0 + 5.0 * rank, 20.0 - 3.0 * rank]            # rank 0: 10, 20; rank 1: 15, 17
    got = bench.max_over_ranks(local, dist, "cpu")
    args = argparse.Namespace(workload="c2", batch=2, frames=3)
    spec = bench.replica_spec(args, rank)
    x = data.make_inputs(spec)[0]
    t = torch.tensor([float(np.abs(x).sum())], dtype=torch.float64)
    sums = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
    dist.all_gather(sums, t)
    dist.barrier()
    out.put((rank, got, [float(v) for v in sums], bench.whole_job_frames_per_s(world, 32, got[0])))
    dist.destroy_process_group()


def test_two_gloo_ranks_time_as_the_slowest_and_roll_out_different_sequences():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, sums, rate in res:
        assert got == [15.0, 20.0]                             # maximum over ranks, element-wise
        assert sums[0] != sums[1]                              # each replica has its own seeded sequences
        assert rate == 2 * 32 / 15.0 * 1e3                     # whole-job frames/s: replicas add up


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0", "--workload", "c1"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0", "--workload", "c1"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0
    import json
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0


def test_gpus_flag_spawns_one_process_per_rank():
    # no WORLD_SIZE in the environment: bench.py starts the ranks itself, with the rendezvous variables set,
    # and only rank 0's line reaches stdout
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0", "--workload", "c1"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr
    import json
    lines = [l for l in r.stdout.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["config"]["parallelism"] == "replicas x2"


def test_spawned_ranks_get_distinct_rendezvous_variables(tmp_path):
    import bench
    probe = tmp_path / "probe.py"
    probe.write_text("import os, sys\n"
                     "open(sys.argv[1] + os.environ['RANK'], 'w').write(' '.join(os.environ[k] for k in "
                     "('RANK', 'LOCAL_RANK', 'WORLD_SIZE', 'MASTER_ADDR', 'MASTER_PORT')))\n")
    saved = bench.__file__
    try:
        bench.__file__ = str(probe)
        assert bench.spawn_ranks(3, [str(tmp_path / "rank")]) == 0
    finally:
        bench.__file__ = saved
    got = [open(tmp_path / ("rank%d" % r)).read().split() for r in range(3)]
    assert [g[0] for g in got] == ["0", "1", "2"] and [g[1] for g in got] == ["0", "1", "2"]
    assert all(g[2] == "3" and g[3] == "127.0.0.1" for g in got) and len({g[4] for g in got}) == 1
