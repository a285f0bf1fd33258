"""The benchmark's multi-rank bookkeeping on two CPU ranks (gloo): the operator has no
cross-(batch, head) term, so ranks run independent replicas and exchange one number, the slowest
rank's time; the whole-job rate is all ranks' units over that time.  Also: the reference arm
prints on rank 0 only."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    from paper_2507_01652_b200 import workloads

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        my_ms = 2.0 + rank          # rank 1 is the slow one
        ms = bench.max_over_ranks(my_ms, world, torch.device("cpu"))
        rate = bench.whole_job_rate(1000, world, ms)
        wl = workloads.WORKLOADS["config1"]
        q, _, _ = workloads.make_qkv(__import__("dataclasses").replace(wl, seed=bench.rank_seed(wl.seed, rank)))
        out.put((rank, ms, rate, float(q.double().sum())))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_sum_the_units():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    (r0, ms0, rate0, sum0), (r1, ms1, rate1, sum1) = res
    assert ms0 == ms1 == 3.0                      # max over ranks, seen by both
    assert rate0 == rate1 == 2 * 1000 / 3.0e-3     # whole-job units per second
    assert sum0 != sum1                            # each rank drew its own replica


def test_reference_arm_prints_on_rank_zero_only():
    def run(rank):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank))
        return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                               "--steps", "1", "--warmup", "1", "--prefill-workload", "config2"],
                              capture_output=True, text=True, env=env, timeout=600)
    r1 = run(1)
    assert r1.returncode == 0 and r1.stdout.strip() == ""
    r0 = run(0)
    assert r0.returncode == 0
    line = json.loads(r0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
