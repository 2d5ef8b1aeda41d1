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


# ------------------------------------------------------------------ column sharding (host logic)

def test_column_shards_tile_the_feature_axis():
    from paper_2207_12000_b200.shard import column_shard
    for F in (1, 3, 4, 16, 100, 128, 602, 1433):
        for world in (1, 2, 3, 4, 8):
            spans = [column_shard(F, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == F
            for (a, b), (c, d) in zip(spans, spans[1:]):
                assert b == c and a <= b and c <= d            # contiguous, in order, possibly empty at the end
            assert all(lo % 4 == 0 for lo, hi in spans if hi > lo)  # every non-empty slab starts on a 16-byte boundary
            widths = [hi - lo for lo, hi in spans if hi > lo]
            w = 4 * -(-F // (4 * world))
            assert all(x == w for x in widths[:-1]) and 0 < widths[-1] <= w   # equal slabs, a shorter last one


def shard_worker(rank, world, port, out):
    import numpy as np
    import gnnpre_inputs as gi
    import oracle as orc
    from paper_2207_12000_b200.shard import column_shard
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    g = gi.erdos_renyi(300, 1500, 5)
    X = gi.normal_matrix(300, 22, 6).numpy()
    K = 2
    lo, hi = column_shard(X.shape[1], world, rank)
    # the rank's slab alone (the oracle stands in for the device here: this test is about the partition)
    mine = orc.propagate(0, 0.0, g.rowptr.numpy(), g.colidx.numpy(), np.ascontiguousarray(X[:, lo:hi]), K)
    parts = [None] * world
    dist.all_gather_object(parts, (lo, hi, mine))  # the final placement; nothing crosses ranks before it
    if rank == 0:
        full = np.concatenate([p[2] for p in sorted(parts, key=lambda p: p[0])], axis=2)
        want = orc.propagate(0, 0.0, g.rowptr.numpy(), g.colidx.numpy(), X, K)
        out["equal"] = bool(np.array_equal(full, want))
    dist.barrier()
    dist.destroy_process_group()


def test_column_sharded_ranks_reproduce_the_unsharded_result():
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    world, port = 2, free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(shard_worker, args=(world, port, out), nprocs=world, join=True)
        assert out["equal"] is True
