"""KV append / step commit on the device against the oracle, and a few steps of Algorithm 1's outer
loop driven with synthetic logits: append -> verify attention -> accept -> commit."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle
from oracle import parity
import workloads as wl
from workloads import bf16_bits


def _bits(t):
    return bf16_bits(t)


def test_append_and_commit_match_the_oracle_bit_for_bit():
    import paper_2502_20330_b200 as R
    B, Hkv, Lmax, D, gamma = 4, 2, 300, 128, 3
    g = torch.Generator(device="cuda").manual_seed(3)
    k = torch.randn(B, Hkv, Lmax, D, generator=g, device="cuda").bfloat16()
    v = torch.randn(B, Hkv, Lmax, D, generator=g, device="cuda").bfloat16()
    kn = torch.randn(B, gamma + 1, Hkv, D, generator=g, device="cuda").bfloat16()
    vn = torch.randn(B, gamma + 1, Hkv, D, generator=g, device="cuda").bfloat16()
    ctx = torch.tensor([0, 100, 296, 298], dtype=torch.int32, device="cuda")   # the last has no room
    rk, rv, rctx, over = oracle.kv_append(_bits(k), _bits(v), _bits(kn), _bits(vn), ctx.cpu().numpy(), gamma)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    R.rapid_kv_append(kn, vn, k, v, ctx, gamma, status)
    torch.cuda.synchronize()
    assert (_bits(k) == rk).all() and (_bits(v) == rv).all()
    assert ctx.cpu().numpy().tolist() == rctx.tolist()
    assert over and int(status.item()) == 1
    alen = torch.tensor([0, 3, 1, 2], dtype=torch.int32, device="cuda")
    want = oracle.step_commit(ctx.cpu().numpy(), alen.cpu().numpy(), gamma)
    status.zero_()
    R.rapid_step_commit(ctx, alen, gamma, status)
    torch.cuda.synchronize()
    assert ctx.cpu().numpy().tolist() == want.tolist() and int(status.item()) == 0


def test_append_into_a_token_major_cache():
    import paper_2502_20330_b200 as R
    B, Hkv, Lmax, D, gamma = 2, 4, 64, 64, 1
    g = torch.Generator(device="cuda").manual_seed(4)
    base_k = torch.randn(B, Lmax, Hkv, D, generator=g, device="cuda").bfloat16()
    base_v = torch.randn(B, Lmax, Hkv, D, generator=g, device="cuda").bfloat16()
    k, v = base_k.permute(0, 2, 1, 3), base_v.permute(0, 2, 1, 3)          # [B,Hkv,Lmax,D] view, strided
    kn = torch.randn(B, 2, Hkv, D, generator=g, device="cuda").bfloat16()
    vn = torch.randn(B, 2, Hkv, D, generator=g, device="cuda").bfloat16()
    ctx = torch.tensor([5, 62], dtype=torch.int32, device="cuda")
    rk, rv, rctx, _ = oracle.kv_append(_bits(k), _bits(v), _bits(kn), _bits(vn), ctx.cpu().numpy(), gamma)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    R.rapid_kv_append(kn, vn, k, v, ctx, gamma, status)
    torch.cuda.synchronize()
    assert (_bits(k) == rk).all() and (_bits(v) == rv).all() and ctx.cpu().tolist() == rctx.tolist()


def test_several_steps_of_the_outer_loop():
    """Algorithm 1's while loop with synthetic K/V rows and logits: the device state (cache, lengths,
    emitted tokens) tracks an oracle-driven replica step by step."""
    import paper_2502_20330_b200 as R
    cfg = wl.VerifyConfig("loop", B=3, Hq=8, Hkv=2, D=128, gamma=4, V=4096, ctx_lens=(500, 130, 64), Lmax=700,
                          target_sigma=1.0)
    Rr = cfg.R
    q0, k, v, ctx = wl.attention_inputs(cfg, seed=50, device="cuda")
    ctx = ctx.clone()
    aws = R.new_workspace(R.attention_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.D, cfg.Lmax, cfg.gamma))
    cws = R.new_workspace(R.accept_workspace_bytes(cfg.B, cfg.gamma, cfg.V))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = torch.empty_like(q0)
    alen = torch.zeros(cfg.B, dtype=torch.int32, device="cuda"); ntok = torch.zeros_like(alen)
    ref_k, ref_v, ref_ctx = _bits(k).copy(), _bits(v).copy(), ctx.cpu().numpy().copy()
    seen = set()
    for step in range(6):
        g = torch.Generator(device="cuda").manual_seed(1000 + step)
        kn = torch.randn(cfg.B, Rr, cfg.Hkv, cfg.D, generator=g, device="cuda").bfloat16()
        vn = torch.randn(cfg.B, Rr, cfg.Hkv, cfg.D, generator=g, device="cuda").bfloat16()
        q = torch.randn(cfg.B, Rr, cfg.Hq, cfg.D, generator=g, device="cuda").bfloat16()
        z, d, tok, u = wl.accept_inputs(cfg, seed=60 + step, device="cuda")
        # device: one iteration of the loop, no host synchronisation in between
        R.rapid_kv_append(kn, vn, k, v, ctx, cfg.gamma, status)
        R.rapid_verify_step(q, k, v, ctx, cfg.gamma, out, aws, z, d, tok, u, 5.0, alen, ntok, cws)
        ctx_at_verify = ctx.clone()
        R.rapid_step_commit(ctx, alen, cfg.gamma, status)
        torch.cuda.synchronize()
        # oracle replica
        ref_k, ref_v, ref_ctx, over = oracle.kv_append(ref_k, ref_v, _bits(kn), _bits(vn), ref_ctx, cfg.gamma)
        assert not over and ctx_at_verify.cpu().numpy().tolist() == ref_ctx.tolist()
        ref_out, _ = oracle.verify_attention(_bits(q), ref_k, ref_v, ref_ctx, cfg.gamma)
        parity.check_attention(out.float().cpu().numpy(), ref_out)
        rep = parity.check_accept(z.cpu().numpy(), d.cpu().numpy(), tok.cpu().numpy(), u.cpu().numpy(), 5.0, 1.0,
                                  0.1, 0, alen.cpu().numpy(), ntok.cpu().numpy())
        assert rep["near_ties"] == []
        ref_ctx = oracle.step_commit(ref_ctx, alen.cpu().numpy(), cfg.gamma)
        assert ctx.cpu().numpy().tolist() == ref_ctx.tolist()
        assert (_bits(k) == ref_k).all() and (_bits(v) == ref_v).all()
        seen.update(alen.cpu().tolist())
    assert int(status.item()) == 0 and len(seen) >= 3
    assert R.workspace_status(aws) == 0 and R.workspace_status(cws) == 0


@pytest.mark.parametrize("token_major", [False, True])
def test_paged_append_matches_the_oracle_bit_for_bit(token_major):
    import paper_2502_20330_b200 as R
    B, Hkv, bs, D, gamma, mb = 4, 2, 64, 128, 3, 5
    nb = B * mb + 3
    g = torch.Generator(device="cuda").manual_seed(8)
    if token_major:
        kp = torch.randn(nb, bs, Hkv, D, generator=g, device="cuda").bfloat16().permute(0, 2, 1, 3)
        vp = torch.randn(nb, bs, Hkv, D, generator=g, device="cuda").bfloat16().permute(0, 2, 1, 3)
    else:
        kp = torch.randn(nb, Hkv, bs, D, generator=g, device="cuda").bfloat16()
        vp = torch.randn(nb, Hkv, bs, D, generator=g, device="cuda").bfloat16()
    kn = torch.randn(B, gamma + 1, Hkv, D, generator=g, device="cuda").bfloat16()
    vn = torch.randn(B, gamma + 1, Hkv, D, generator=g, device="cuda").bfloat16()
    table = torch.randperm(nb, generator=torch.Generator().manual_seed(9))[:B * mb].reshape(B, mb).to(torch.int32)
    table[1, 2] = -1                                   # sequence 1 crosses into a block nobody handed out
    table = table.cuda()
    ctx = torch.tensor([0, 126, 62, 318], dtype=torch.int32, device="cuda")   # the last has no room (cap 320)
    rk, rv, rctx, over, bad = oracle.kv_append_paged(_bits(kp), _bits(vp), table.cpu().numpy(), _bits(kn), _bits(vn),
                                                     ctx.cpu().numpy(), gamma)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    R.rapid_kv_append_paged(kn, vn, kp, vp, table, ctx, gamma, status)
    torch.cuda.synchronize()
    assert (_bits(kp) == rk).all() and (_bits(vp) == rv).all()
    assert ctx.cpu().numpy().tolist() == rctx.tolist()
    assert over and bad
    assert int(status.item()) == (R.STATUS_BAD_CTX_LEN | R.STATUS_BAD_BLOCK_TABLE)
