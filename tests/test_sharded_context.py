"""Context sharding: the merge identity pinned against the attention definition, the shard bounds,
and the all-gather plumbing over two gloo ranks on CPU (partials computed by the oracle there)."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
import workloads as wl
from workloads import bf16_bits

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _shard_partial(qb, kb, vb, bounds, gamma, last):
    """One rank's partial by the oracle: its keys are rows [s, e) of every sequence's cache.  A shard
    without the rows' own keys is R one-row attentions (gamma = 0: the row sees every key)."""
    B, R, Hq, D = qb.shape
    Lloc = max(e - s for s, e in bounds)
    k = np.zeros((B, kb.shape[1], Lloc, D), np.uint16)
    v = np.zeros_like(k)
    lens = np.zeros(B, np.int32)
    for b, (s, e) in enumerate(bounds):
        k[b, :, :e - s] = kb[b, :, s:e]
        v[b, :, :e - s] = vb[b, :, s:e]
        lens[b] = e - s
    if last:
        return oracle.verify_attention(qb, k, v, lens, gamma)
    o = np.zeros((B, R, Hq, D)); l = np.zeros((B, R, Hq))
    for i in range(R):
        oi, li = oracle.verify_attention(np.ascontiguousarray(qb[:, i:i + 1]), k, v, lens, 0)
        o[:, i], l[:, i] = oi[:, 0], li[:, 0]
    return o, l


def _bounds(ctx, gamma, world):
    sys.path.insert(0, ROOT)
    from paper_2502_20330_b200.sharded import context_shard_bounds
    return context_shard_bounds(ctx, gamma, world)


@pytest.mark.parametrize("world", [2, 3, 5])
def test_merged_shards_equal_the_definition(world):
    cfg = wl.VerifyConfig("s", B=2, Hq=4, Hkv=2, D=64, gamma=2, V=4096, ctx_lens=(83, 40))
    q, k, v, ctx = wl.attention_inputs(cfg, seed=31)
    qb, kb, vb = bf16_bits(q), bf16_bits(k), bf16_bits(v)
    ref, ref_lse = oracle.verify_attention(qb, kb, vb, ctx.numpy(), cfg.gamma)
    bounds = _bounds(ctx.tolist(), cfg.gamma, world)
    parts = [_shard_partial(qb, kb, vb, bounds[r], cfg.gamma, r == world - 1) for r in range(world)]
    out, lse = oracle.merge_partials(np.stack([p[0] for p in parts]), np.stack([p[1] for p in parts]))
    np.testing.assert_allclose(out, ref, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, ref_lse, rtol=0, atol=1e-12)


def test_merge_ignores_empty_sets_and_is_a_convex_combination():
    rng = np.random.default_rng(0)
    o = rng.normal(size=(3, 5, 4))
    l = rng.normal(size=(3, 5))
    l[1] = -np.inf                                      # an empty shard
    out, lse = oracle.merge_partials(o, l)
    w = np.exp(l[[0, 2]] - np.logaddexp(l[0], l[2]))
    np.testing.assert_allclose(out, w[0][:, None] * o[0] + w[1][:, None] * o[2], atol=1e-14)
    np.testing.assert_allclose(lse, np.logaddexp(l[0], l[2]), atol=1e-14)
    out, lse = oracle.merge_partials(o, np.full((3, 5), -np.inf))
    assert (out == 0).all() and np.isneginf(lse).all()


def test_shard_bounds_partition_the_context():
    b = _bounds([1000, 37], 4, 4)
    for seq, L in enumerate([1000, 37]):
        runs = [b[r][seq] for r in range(4)]
        assert runs[0][0] == 0 and runs[-1][1] == L
        assert all(runs[r][1] == runs[r + 1][0] for r in range(3))
        assert all(e > s for s, e in runs)
        assert runs[-1][1] - runs[-1][0] >= 5           # the newest R keys stay on the last rank
    with pytest.raises(ValueError):
        _bounds([7], 4, 4)                              # 2 context keys cannot feed 4 ranks


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, results):
    sys.path.insert(0, ROOT)
    from paper_2502_20330_b200.sharded import context_shard_bounds, exchange_partials
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = wl.VerifyConfig("s", B=2, Hq=4, Hkv=2, D=64, gamma=3, V=4096, ctx_lens=(61, 29))
        q, k, v, ctx = wl.attention_inputs(cfg, seed=32)          # same seed: every rank draws the same request
        qb, kb, vb = bf16_bits(q), bf16_bits(k), bf16_bits(v)
        bounds = context_shard_bounds(ctx.tolist(), cfg.gamma, world)
        o, l = _shard_partial(qb, kb, vb, bounds[rank], cfg.gamma, rank == world - 1)
        o_parts, l_parts = exchange_partials(torch.from_numpy(o), torch.from_numpy(l))
        out, lse = oracle.merge_partials(o_parts.numpy(), l_parts.numpy())
        ref, ref_lse = oracle.verify_attention(qb, kb, vb, ctx.numpy(), cfg.gamma)
        results[rank] = (float(np.abs(out - ref).max()), float(np.abs(lse - ref_lse).max()), tuple(o_parts.shape))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_exchange_and_merge():
    world = 2
    port = _free_port()
    with mp.Manager() as mgr:
        results = mgr.dict()
        mp.spawn(_worker, args=(world, port, results), nprocs=world, join=True)
        r = [results[i] for i in range(world)]
    for err_o, err_l, shape in r:
        assert err_o < 1e-12 and err_l < 1e-12 and shape == (2, 2, 4, 4, 64)
