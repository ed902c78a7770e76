"""Host-side logic of bench.py that needs no GPU: the multi-rank reduction (gloo, two processes), the byte and
flop models, and the reference arm's JSON line."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402
from paper_2305_02299_b200 import inputs  # noqa: E402


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    seconds = 1.0 + 0.5 * rank                     # rank 1 is the slow one
    slowest = bench.max_over_ranks(seconds, dist, "cpu")
    value = bench.whole_job_value(2.0e9, world, slowest / 10)
    dist.barrier()
    if rank == 0:
        out.put((slowest, value))
    dist.destroy_process_group()


def test_two_rank_reduction_takes_the_slowest_rank_and_sums_the_work():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    slowest, value = q.get(timeout=120)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert slowest == 1.5
    assert abs(value - 2.0e9 * 2 / 0.15 / 1e9) < 1e-9
    assert bench.max_over_ranks(3.25, None, "cpu") == 3.25      # single process: nothing to reduce


def test_byte_and_flop_models_match_the_stated_figures():
    w = inputs.workloads()
    assert bench.algorithmic_flops(w["c2"], 3072) == 2 * 256 * 3072 * 77 == 121110528
    assert bench.algorithmic_bytes(w["c1"], 3072) == 3072 * 77 * 8 + 768 * 4 + 3072 * 4 + 3072 * 4 + 3072 * 4
    assert abs(bench.algorithmic_bytes(w["c4_s80_b1"], 4096) / 1e6 - 26.90) < 0.01
    assert abs(bench.algorithmic_bytes(w["c2"], 3072) / 1e6 - 5.849) < 0.001


def test_reference_arm_prints_one_json_line():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2", "--warmup", "1"],
                       capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr
    lines = [l for l in r.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "GFLOP/s" and d["value"] > 0 and d["gpu_launches"] == 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")             # other ranks of a torchrun launch do no work
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2", "--warmup", "1"],
                       capture_output=True, text=True, timeout=300, env=env)
    assert r.returncode == 0 and r.stdout.strip() == ""
