"""The N > 1 path of bench.py on CPU: two gloo ranks on 127.0.0.1.  The path has no exchange step
(replicas only), so all that crosses ranks is the timing reduction: max over ranks, aggregate
throughput = ranks x units / slowest time; the reference arm runs on rank 0 alone."""
import importlib.util
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def load_bench():
    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(ROOT, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    bench = load_bench()
    mine = 10.0 + 5.0 * rank  # rank 1 is the slow one
    slowest = bench.max_over_ranks(mine, world, "cpu")
    out[rank] = (slowest, bench.aggregate_throughput(1000, 4, world, slowest))
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_aggregate_with_two_gloo_ranks():
    world, port = 2, free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(worker, args=(world, port, out), nprocs=world, join=True)
        assert out[0] == out[1] == (15.0, 2 * 1000 * 4 / 15e-3)


def test_single_rank_needs_no_process_group():
    bench = load_bench()
    assert bench.max_over_ranks(7.5, 1, "cpu") == 7.5
    assert bench.aggregate_throughput(10, 3, 1, 6.0) == 10 * 3 / 6e-3


def test_reference_arm_runs_on_rank0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", CUDA_VISIBLE_DEVICES="")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c1",
                        "--gpus", "2", "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True,
                       timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""  # other ranks exit 0 without work
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c1",
                        "--gpus", "2", "--steps", "1", "--warmup", "0", "--cpu-seconds", "0.5"], env=env,
                       capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and '"impl": "reference"' in r.stdout
