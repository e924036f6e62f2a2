"""The N > 1 path of bench.py on CPU: two gloo ranks.

The hot path does not shard (every rank is an independent replica), so what more than one rank adds is host
logic only: weights of its own per replica, the slowest rank's time, the whole-job rate, and a reference arm
that only rank 0 runs.
"""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank: int, world: int, port: int, out_dir: str) -> None:
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import bench
    from paper_2409_17066_b200 import synth
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    try:
        assert bench.dist_env() == (rank, rank, world)
        # every replica draws weights of its own
        spec = synth.LayerSpec("r", 64, 96, v=8, k1=256)
        d = synth.make_layer(spec, 0, bench.replica_layer_ordinal(0, rank), 1)
        digest = torch.tensor([int(d["idx1"].astype(np.int64).sum())], dtype=torch.int64)
        seen = [torch.zeros(1, dtype=torch.int64) for _ in range(world)]
        dist.all_gather(seen, digest)
        assert len({int(t.item()) for t in seen}) == world
        # timing: the slowest rank counts, and the rate is over what all replicas processed
        ms = 2.0 + rank
        slowest = bench.max_over_ranks(ms, world, "cpu")
        assert slowest == 2.0 + (world - 1)
        assert bench.whole_job_gbps(1e9, world, slowest) == world * 1e9 / (slowest * 1e-3) / 1e9
        # the reference arm: the ranks other than 0 return at once, without work and without output
        if rank != 0:
            class Args:
                gpus, steps, warmup = world, 1, 0
            assert bench.run_reference(Args()) == 0
        dist.barrier()
        with open(os.path.join(out_dir, f"ok{rank}"), "w") as f:
            f.write("ok")
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_replicas_and_max_timing(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    assert sorted(os.listdir(tmp_path)) == ["ok0", "ok1"]


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1, "cpu") == 3.5
    assert bench.whole_job_gbps(2e9, 1, 1.0) == 2000.0


def test_bench_traffic_figures_expire_with_the_kernel_source():
    """bench.py scales DRAM traffic from an ncu capture only while the kernel's source file is byte for byte the
    one the capture was taken on; any other digest gives None (reported as null)."""
    import importlib
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    if root not in sys.path:
        sys.path.insert(0, root)
    bench = importlib.import_module("bench")
    table = bench.NCU_DRAM_BYTES_PER_ALGORITHMIC_BYTE
    assert bench.read_traffic("no_such_kernel", 1.0) is None
    for kernel, (ratio, source, digest) in table.items():
        assert os.path.exists(os.path.join(root, "paper_2409_17066_b200", "csrc", source)), source
        got = bench.read_traffic(kernel, 1000.0)
        assert got is None or got == ratio * 1000.0
    saved = dict(table)
    try:
        k = next(iter(table))
        table[k] = (table[k][0], table[k][1], "000000000000")
        assert bench.read_traffic(k, 1.0) is None
    finally:
        table.clear()
        table.update(saved)
