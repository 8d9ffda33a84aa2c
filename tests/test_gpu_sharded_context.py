"""Context-sharded verify attention on one GPU: the ranks' partials are computed one after another
(nothing waits on anything), stacked as the all-gather would leave them, and merged by the library."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle
from oracle import parity
import workloads as wl
from workloads import bf16_bits


def _partials(q, k, v, ctx, gamma, world):
    import paper_2502_20330_b200 as R
    from paper_2502_20330_b200.sharded import context_shard_bounds, local_partial
    bounds = context_shard_bounds(ctx.tolist(), gamma, world)
    B, Rr, Hq, D = q.shape
    o_parts, l_parts = [], []
    for r in range(world):
        Lloc = max(e - s for s, e in bounds[r])
        kl = torch.full((B, k.shape[1], Lloc, D), float("nan"), dtype=k.dtype, device=k.device)
        vl = torch.full_like(kl, float("nan"))
        lens = torch.zeros(B, dtype=torch.int32, device=k.device)
        for b, (s, e) in enumerate(bounds[r]):
            kl[b, :, :e - s] = k[b, :, s:e]
            vl[b, :, :e - s] = v[b, :, s:e]
            lens[b] = e - s
        ws = R.new_workspace(R.attention_workspace_bytes(B, Hq, k.shape[1], D, Lloc, gamma))
        o32, lse = local_partial(q, kl, vl, lens, gamma, ws, holds_newest=(r == world - 1))
        torch.cuda.synchronize()
        assert R.workspace_status(ws) == 0
        o_parts.append(o32)
        l_parts.append(lse)
    return torch.stack(o_parts), torch.stack(l_parts)


@pytest.mark.parametrize("world,lens,Hq,gamma", [
    (2, (3000, 517), 32, 8), (4, (4097, 1300), 32, 8), (8, (2048 + 37,), 32, 8),
    (2, (3000, 517), 64, 6),        # 56 grouped rows: the shard weights come from the two-group keys-on-M kernel
    (4, (5000, 1300), 64, 7),       # 64 grouped rows
    (2, (2500, 900), 64, 8),        # 72 grouped rows: rows on M
])
def test_sharded_context_against_oracle(world, lens, Hq, gamma):
    import paper_2502_20330_b200 as R
    cfg = wl.VerifyConfig("s", B=len(lens), Hq=Hq, Hkv=8, D=128, gamma=gamma, V=4096, ctx_lens=lens)
    q, k, v, ctx = wl.attention_inputs(cfg, seed=33, device="cuda")
    o_parts, l_parts = _partials(q, k, v, ctx, cfg.gamma, world)
    out = torch.empty_like(q)
    o32 = torch.empty(q.shape, dtype=torch.float32, device="cuda")
    lse = torch.empty(q.shape[:3], dtype=torch.float32, device="cuda")
    R.rapid_merge_partials(o_parts, l_parts, out=out, out_f32=o32, lse_out=lse)
    torch.cuda.synchronize()
    ref, ref_lse = oracle.verify_attention(bf16_bits(q), bf16_bits(k), bf16_bits(v), ctx.cpu().numpy(), cfg.gamma)
    rows = ~np.isnan(ref_lse)
    parity.check_attention(out.float().cpu().numpy(), ref, rows)
    parity.check_attention(o32.cpu().numpy(), ref, rows)
    assert np.abs(lse.cpu().numpy() - ref_lse).max() < 1e-4
    # the shard weights themselves: every rank's log-sum-exp against the oracle's over that rank's keys
    from paper_2502_20330_b200.sharded import context_shard_bounds
    bounds = context_shard_bounds(ctx.tolist(), cfg.gamma, world)
    r = 0                                                # a rank without the rows' own keys
    kb, vb = bf16_bits(k), bf16_bits(v)
    qb = bf16_bits(q)
    for b, (s0, e0) in enumerate(bounds[r]):
        for i in range(cfg.R):
            _, l_ref = oracle.verify_attention(np.ascontiguousarray(qb[b:b + 1, i:i + 1]),
                                               np.ascontiguousarray(kb[b:b + 1, :, s0:e0]),
                                               np.ascontiguousarray(vb[b:b + 1, :, s0:e0]),
                                               np.array([e0 - s0], np.int32), 0)
            assert np.abs(l_parts[r, b, i].cpu().numpy() - l_ref[0, 0]).max() < 1e-4


def test_sharded_call_on_a_side_stream(tmp_path):
    """sharded_verify_attention with a stream that is not the current one (a one-rank group on this GPU):
    allocations, the exchange and the kernels must all be ordered on that stream."""
    import torch.distributed as dist
    import paper_2502_20330_b200 as R
    from paper_2502_20330_b200.sharded import sharded_verify_attention
    cfg = wl.VerifyConfig("s", B=2, Hq=32, Hkv=8, D=128, gamma=8, V=4096, ctx_lens=(6000, 2100))
    q, k, v, ctx = wl.attention_inputs(cfg, seed=36, device="cuda")
    ref, ref_lse = oracle.verify_attention(bf16_bits(q), bf16_bits(k), bf16_bits(v), ctx.cpu().numpy(), cfg.gamma)
    own_group = not dist.is_initialized()
    if own_group:
        dist.init_process_group("nccl", init_method=f"file://{tmp_path}/rendezvous", rank=0, world_size=1,
                                device_id=torch.device("cuda", 0))
    try:
        ws = R.new_workspace(R.attention_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.D, k.shape[2], cfg.gamma))
        out = torch.zeros_like(q)
        torch.cuda.synchronize()
        side = torch.cuda.Stream()
        # keep the current stream busy, so that work wrongly put there would run late
        busy = torch.empty(1 << 28, device="cuda")
        for _ in range(20):
            busy.add_(1.0)
        sharded_verify_attention(q, k, v, ctx, cfg.gamma, out, ws, stream=side)
        side.synchronize()
        got = out.float().cpu().numpy()
        torch.cuda.synchronize()
        parity.check_attention(got, ref, ~np.isnan(ref_lse))
    finally:
        if own_group:
            dist.destroy_process_group()


def test_all_keys_visible_rows_are_one_row_decodes():
    """all_keys_visible: every row must equal the oracle's one-row attention over all keys."""
    import paper_2502_20330_b200 as R
    cfg = wl.VerifyConfig("s", B=2, Hq=28, Hkv=4, D=128, gamma=4, V=4096, ctx_lens=(700, 1))
    q, k, v, ctx = wl.attention_inputs(cfg, seed=34, device="cuda")
    ws = R.new_workspace(R.attention_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.D, k.shape[2], cfg.gamma))
    out = torch.empty_like(q)
    R.rapid_verify_attention(q, k, v, ctx, cfg.gamma, out, ws, R.AttnParams(all_keys_visible=True))
    torch.cuda.synchronize()
    assert R.workspace_status(ws) == 0                  # a one-key shard is a legal length here
    qb = bf16_bits(q)
    for i in range(cfg.R):
        ref, ref_lse = oracle.verify_attention(np.ascontiguousarray(qb[:, i:i + 1]), bf16_bits(k), bf16_bits(v),
                                               ctx.cpu().numpy(), 0)
        parity.check_attention(out[:, i:i + 1].float().cpu().numpy(), ref, ~np.isnan(ref_lse))


def test_merge_partials_against_the_oracle_merge():
    import paper_2502_20330_b200 as R
    g = torch.Generator(device="cuda").manual_seed(35)
    P, rows, D = 5, 1000, 128
    o = torch.randn(P, rows, D, generator=g, device="cuda")
    l = torch.randn(P, rows, generator=g, device="cuda") * 5
    l[2] = float("-inf")                                # an empty shard
    l[:, 7] = float("-inf")                             # a row with no keys anywhere
    o32 = torch.empty(rows, D, device="cuda")
    lse = torch.empty(rows, device="cuda")
    R.rapid_merge_partials(o, l, out_f32=o32, lse_out=lse)
    torch.cuda.synchronize()
    ref, ref_lse = oracle.merge_partials(o.cpu().numpy(), l.cpu().numpy())
    np.testing.assert_allclose(o32.cpu().numpy(), ref, rtol=0, atol=2e-5)
    fin = np.isfinite(ref_lse)
    np.testing.assert_allclose(lse.cpu().numpy()[fin], ref_lse[fin], rtol=0, atol=1e-5)
    assert np.isneginf(lse.cpu().numpy()[~fin]).all()
