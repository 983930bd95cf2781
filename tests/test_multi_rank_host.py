"""Host logic of the multi-GPU run, on CPU with the gloo backend and two ranks.  The path shards by
batch with no exchange step (replicas only), so all there is between ranks is: the step time of the
job is the slowest rank's, the reported value is the sum over replicas, and only rank 0 prints."""
import json
import os
import socket
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
ms = bench.max_over_ranks(10.0 + 5.0 * rank, world)          # rank 1 is the slow one
val = bench.job_tflops(world, 1e12, ms)
dist.barrier()
dist.destroy_process_group()
print(json.dumps({{"rank": rank, "ms": ms, "value": val}}))
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _spawn(code_or_args, world=2, timeout=300):
    port = _free_port()
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable] + code_or_args, env=env, cwd=ROOT,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=timeout) for p in procs]
    return [(p.returncode, o, e) for p, (o, e) in zip(procs, outs)]


def test_two_ranks_agree_on_the_slowest_and_sum_the_work():
    pytest.importorskip("torch")
    res = _spawn(["-c", WORKER.format(root=ROOT)])
    for rc, out, err in res:
        assert rc == 0, err
    got = [json.loads(out.strip().splitlines()[-1]) for _, out, _ in res]
    for g in got:
        assert g["ms"] == 15.0                     # max over ranks, on every rank
        assert abs(g["value"] - 2 * 1e12 / 15e-3 / 1e12) < 1e-9


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1) == 3.5
    assert bench.job_tflops(1, 2e12, 1000.0) == 2.0


def test_reference_arm_runs_on_rank_zero_only():
    """Under a two-rank launch rank 0 times the oracle and prints one JSON line; rank 1 exits 0 silently."""
    res = _spawn([os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"],
                 timeout=900)
    (rc0, out0, err0), (rc1, out1, err1) = res
    assert rc0 == 0, err0
    assert rc1 == 0 and out1.strip() == "", (out1, err1)
    line = json.loads(out0.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0


def test_bench_starts_its_own_ranks_when_no_launcher_did():
    """`python bench.py --gpus 2` with no RANK / WORLD_SIZE in the environment starts two ranks itself;
    rank 0's line reports the number of ranks that really joined.  (--cpu-dry-run: gloo, no kernels.)"""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    proc = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--cpu-dry-run"], env=env,
                          cwd=ROOT, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True, timeout=300)
    assert proc.returncode == 0, proc.stderr
    line = json.loads(proc.stdout.strip().splitlines()[-1])
    assert line["n_gpus"] == 2 and line["cpu_dry_run"] is True
    assert line["ms_per_step"] == 11.0                 # the slower of the two ranks (10 + rank)


def test_bench_refuses_a_rank_count_it_does_not_have():
    """One process claiming --gpus 2 under a launcher that started only one rank must not print n_gpus 2."""
    env = dict(os.environ, RANK="0", LOCAL_RANK="0", WORLD_SIZE="1", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(_free_port()))
    proc = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--cpu-dry-run"], env=env,
                          cwd=ROOT, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True, timeout=300)
    assert proc.returncode != 0 and "n_gpus" not in proc.stdout
