"""The N > 1 path of the benchmark on CPU: two gloo ranks.  The data path shards by rows with
no exchange between ranks; what the ranks do share is the timing reduction (slowest rank) and
the whole-job throughput built from it, and rank 0 alone reports."""
import json
import os
import subprocess
import sys

import numpy as np
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = bench.rank_workload("c3", rank, M=4, N=64)
    ms = [1.0, 2.5][rank]                                   # rank 1 is the slow one
    slowest = bench.max_over_ranks(ms, world, "cpu")
    value = bench.job_value(world, w.compulsory_bytes, slowest * 1e-3)
    out.put((rank, slowest, value, w.compulsory_bytes, float(np.asarray(w.inputs[0], dtype=np.float64).sum())))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_slowest_time_and_work_on_their_own_batches():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, s0, v0, b0, sum0), (r1, s1, v1, b1, sum1) = got
    assert (r0, r1) == (0, 1) and s0 == s1 == 2.5            # the maximum over ranks, on both
    assert b0 == b1 and v0 == v1 == 2 * b0 / 2.5e-3 / 1e9    # bytes of all ranks over the slowest time
    assert sum0 != sum1                                      # each rank drew its own batch


def test_reference_arm_reports_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "1"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "1"], env=env, capture_output=True, text=True, timeout=300)
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["n_gpus"] == 2


def test_gpus_flag_launches_the_ranks_itself():
    """`python bench.py --gpus 2` with no launcher around it starts two ranks (one per GPU) through
    torch.distributed.run; driven here on CPU with the reference arm, whose rank 0 reports and
    whose rank 1 leaves without work."""
    sys.path.insert(0, ROOT)
    import bench
    cmd = bench.torchrun_command(2, ["--gpus", "2", "--steps", "1"], 29999)
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node=2" in cmd and "--nnodes=1" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[cmd.index("--master-port") + 1] == "29999"
    assert cmd[-4:] == ["--gpus", "2", "--steps", "1"] and cmd[-5].endswith("bench.py")
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "1"], env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1                                   # rank 0 alone printed
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["cpu_baseline"]["cores"] >= 1
