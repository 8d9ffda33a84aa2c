"""The N>1 path of bench.py shards requests over ranks with no data-path collective; what the ranks
share is host logic only (per-rank seeds, MAX over ranks of the timed region, whole-job throughput).
That logic is exercised here with two gloo ranks on CPU."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, results):
    sys.path.insert(0, ROOT)
    import bench
    import workloads as wl
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        seed = bench.rank_seed(2025, rank)
        cfg = wl.CONFIGS["qwen7b_ragged"]
        ctx = wl.context_lengths(cfg, seed)
        local_ms = 3.0 + rank              # rank 1 is the slow one
        total = bench.max_over_ranks(local_ms)
        results[rank] = (seed, ctx.tolist(), total, bench.job_throughput_gbs(10 ** 9, world, total))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_share_only_the_timing():
    world = 2
    port = _free_port()
    with mp.Manager() as mgr:
        results = mgr.dict()
        mp.spawn(_worker, args=(world, port, results), nprocs=world, join=True)
        r0, r1 = results[0], results[1]
    assert r0[0] != r1[0] and r0[1] != r1[1]            # own seeds, own ragged lengths
    assert r0[2] == r1[2] == 4.0                        # MAX over ranks
    assert abs(r0[3] - 2 * 10 ** 9 / 4e-3 / 1e9) < 1e-9  # all ranks' bytes over the slowest time


def test_single_process_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(1.25) == 1.25
    assert bench.rank_seed(7, 0) == 7


def _spawned(results):
    """What bench.py's own launcher hands every rank: the environment a torchrun rank would see."""
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    assert os.environ["MASTER_ADDR"] == "127.0.0.1" and int(os.environ["LOCAL_RANK"]) == rank
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        results[rank] = bench.max_over_ranks(10.0 * (rank + 1))
    finally:
        dist.destroy_process_group()


def test_bench_starts_its_own_ranks_without_a_launcher():
    sys.path.insert(0, ROOT)
    import bench
    with mp.Manager() as mgr:
        results = mgr.dict()
        bench.spawn_ranks(2, _spawned, (results,))
        assert dict(results) == {0: 20.0, 1: 20.0}


def test_both_arms_print_the_same_config():
    sys.path.insert(0, ROOT)
    import bench
    import workloads as wl
    cfg = wl.CONFIGS["qwen7b_ragged"]
    ctx = wl.context_lengths(cfg, 2025)
    a = bench.config_dict(cfg, ctx, 1)
    assert a == bench.config_dict(cfg, ctx, 1) and a["workload"] == "qwen7b_ragged" and "model" not in a
    assert a["kv_bytes_per_step"] == 4 * cfg.Hkv * cfg.D * int(ctx.sum())


def test_visible_keys_under_a_window_by_brute_force():
    """bench.py's algorithmic bytes under --sink/--window: the keys SOME row can see, counted one by one."""
    sys.path.insert(0, ROOT)
    import bench
    import workloads as wl
    saved = bench.MASK
    try:
        for gamma in (0, 3, 8):
            cfg = wl.VerifyConfig("w", B=3, Hq=8, Hkv=2, D=64, gamma=gamma, V=4096, ctx_lens=(300, 40, gamma + 1))
            for sink, window in ((0, 0), (4, 16), (0, 1), (50, 7), (4, 4092), (400, 3)):
                bench.MASK = (sink, window)
                want = 0
                for L in cfg.ctx_lens:
                    seen = set()
                    for i in range(cfg.R):
                        own = L - cfg.R + i
                        for j in range(own + 1):
                            if window <= 0 or j < sink or j > own - window:
                                seen.add(j)
                    want += len(seen)
                assert bench.visible_keys(cfg, cfg.ctx_lens) == want, (gamma, sink, window)
    finally:
        bench.MASK = saved
