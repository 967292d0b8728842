"""Host-side logic of bench.py's multi-rank mode, run as two gloo ranks on CPU: the ranks are independent replicas
(no data-path collective); the only exchanges are the barrier and the max-over-ranks of the device time."""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    import bench
    w, r, l = bench.dist_setup(world)
    assert (w, r, l) == (world, rank, rank)
    bench.barrier(w)
    slowest = bench.max_over_ranks(10.0 + 5.0 * rank, w, torch.device("cpu"))
    # whole-job value = replicas x per-replica work / slowest replica's time
    value = w * 1000.0 / slowest
    bench.barrier(w)
    out.put((rank, slowest, value))
    torch.distributed.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_slowest_time_and_aggregate():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [15.0, 15.0]
    assert all(abs(r[2] - 2 * 1000.0 / 15.0) < 1e-9 for r in res)


def test_reference_arm_prints_one_json_line_and_other_ranks_stay_silent():
    env = dict(os.environ, WORLD_SIZE="2", RANK="1")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                        "--steps", "1", "--warmup", "0"], capture_output=True, text=True, env=env, timeout=300)
    assert p.returncode == 0 and p.stdout.strip() == ""
    env = dict(os.environ, WORLD_SIZE="1", RANK="0")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                        "--steps", "1", "--warmup", "0"], capture_output=True, text=True, env=env, timeout=300)
    assert p.returncode == 0
    line = json.loads(p.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "TFLOP/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0


def test_ours_fails_loudly_without_a_gpu():
    if torch.cuda.is_available():
        pytest.skip("this check is for the CPU box")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "1"], capture_output=True, text=True,
                       timeout=300)
    assert p.returncode != 0 and "no CPU fallback" in p.stderr
