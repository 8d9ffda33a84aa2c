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


@pytest.mark.parametrize("world,lens", [(2, (3000, 517)), (4, (4097, 1300)), (8, (2048 + 37,))])
def test_sharded_context_against_oracle(world, lens):
    import paper_2502_20330_b200 as R
    cfg = wl.VerifyConfig("s", B=len(lens), Hq=32, Hkv=8, D=128, gamma=8, V=4096, ctx_lens=lens)
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
    assert np.abs(lse.cpu().numpy() - ref_lse).max() < 1e-3


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
