"""Parity of the paged-cache verify attention with the fp64 oracle, through the C ABI.

The oracle side sees only the pool and the block table the generator made: it writes the paged
cache out as a contiguous one (oracle.paged_gather) and applies the attention definition to that.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle
from oracle import parity
import workloads as wl
from workloads import bf16_bits


def _run_paged(q, kp, vp, table, ctx, gamma, num_ctas=0):
    import paper_2502_20330_b200 as R
    B, Rr, Hq, D = q.shape
    Hkv, bs = kp.shape[1], kp.shape[2]
    Lmax = table.shape[1] * bs
    ws = R.new_workspace(R.attention_workspace_bytes(B, Hq, Hkv, D, Lmax, gamma))
    out = torch.empty_like(q)
    lse = torch.empty(B, Rr, Hq, dtype=torch.float32, device=q.device)
    R.rapid_verify_attention_paged(q, kp, vp, table, ctx, gamma, out, ws,
                                   R.AttnParams(num_ctas=num_ctas, lse_out=lse))
    torch.cuda.synchronize()
    return out, lse, R.workspace_status(ws)


def _oracle_paged(q, kp, vp, table, ctx, gamma):
    c = ctx.cpu().numpy()
    t = table.cpu().numpy()
    kc = oracle.paged_gather(bf16_bits(kp), t, c)
    vc = oracle.paged_gather(bf16_bits(vp), t, c)
    return oracle.verify_attention(bf16_bits(q), kc, vc, c, gamma)


@pytest.mark.parametrize("Hq,Hkv,D,gamma,bs,lens,token_major", [
    (32, 8, 128, 8, 64, (2048 + 37,), False),        # one tile per block
    (32, 8, 128, 8, 256, (3000, 517, 1024), False),  # four tiles per block, ragged batch
    (28, 4, 128, 4, 128, (1500, 2300), True),        # [block, token, head, D] storage
    (8, 2, 64, 4, 512, (1000, 70), False),           # head_dim 64, a sequence inside one block
    (32, 8, 128, 0, 128, (777,), True),              # one-row decode
    (32, 8, 128, 2, 64, (5000, 900), False),         # 12 grouped rows: two softmax groups of 8 columns, 64-key blocks
    (32, 8, 128, 4, 256, (7000,), True),             # 20 rows: two groups of 16 columns
    (56, 8, 128, 8, 128, (4000, 2100), False),       # 63 rows: two groups of 32 columns
    (64, 8, 128, 8, 64, (3000, 1000), False),        # 72 rows: two groups of 40 columns, two boxes per tile
])
def test_paged_against_oracle(Hq, Hkv, D, gamma, bs, lens, token_major):
    cfg = wl.VerifyConfig("p", B=len(lens), Hq=Hq, Hkv=Hkv, D=D, gamma=gamma, V=4096, ctx_lens=lens)
    q, k, v, ctx = wl.attention_inputs(cfg, seed=21, device="cuda")
    kp, vp, table = wl.paged_layout(k, v, ctx, bs, seed=4, token_major=token_major)
    out, lse, status = _run_paged(q, kp, vp, table, ctx, gamma)
    assert status == 0
    ref, ref_lse = _oracle_paged(q, kp, vp, table, ctx, gamma)
    rows = ~np.isnan(ref_lse)
    parity.check_attention(out.float().cpu().numpy(), ref, rows)
    assert np.abs(lse.cpu().numpy()[rows] - ref_lse[rows]).max() < 1e-3
    assert not torch.isnan(out.float()).any()        # unused blocks and the blocks' tails hold NaN


def test_paged_equals_contiguous_bitwise():
    """Same keys in the same order: the paged call must reproduce the contiguous call bit for bit."""
    import paper_2502_20330_b200 as R
    cfg = wl.VerifyConfig("p", B=3, Hq=32, Hkv=8, D=128, gamma=8, V=4096, ctx_lens=(5000, 4097, 129))
    q, k, v, ctx = wl.attention_inputs(cfg, seed=22, device="cuda")
    kp, vp, table = wl.paged_layout(k, v, ctx, 256, seed=5)
    out_p, lse_p, status = _run_paged(q, kp, vp, table, ctx, cfg.gamma)
    assert status == 0
    ws = R.new_workspace(R.attention_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.D, k.shape[2], cfg.gamma))
    out_c = torch.empty_like(q)
    R.rapid_verify_attention(q, k, v, ctx, cfg.gamma, out_c, ws)
    torch.cuda.synchronize()
    assert torch.equal(out_p.view(torch.int16), out_c.view(torch.int16))


def test_bad_block_table_entry_is_reported_not_followed():
    import paper_2502_20330_b200 as R
    cfg = wl.VerifyConfig("p", B=1, Hq=8, Hkv=2, D=64, gamma=2, V=4096, ctx_lens=(1000,))
    q, k, v, ctx = wl.attention_inputs(cfg, seed=23, device="cuda")
    kp, vp, table = wl.paged_layout(k, v, ctx, 128, seed=6)
    table[0, 3] = kp.shape[0] + 5        # outside the pool
    out, lse, status = _run_paged(q, kp, vp, table, ctx, cfg.gamma)
    assert status & R.STATUS_BAD_BLOCK_TABLE
    assert torch.isfinite(out.float()).all()


def test_paged_argument_errors():
    import paper_2502_20330_b200 as R
    cfg = wl.VerifyConfig("p", B=1, Hq=8, Hkv=2, D=64, gamma=2, V=4096, ctx_lens=(300,))
    q, k, v, ctx = wl.attention_inputs(cfg, seed=24, device="cuda")
    ws = R.new_workspace(1 << 20)
    out = torch.empty_like(q)
    pool = torch.zeros(8, 2, 96, 64, dtype=torch.bfloat16, device="cuda")   # block size not a power of two
    table = torch.zeros(1, 4, dtype=torch.int32, device="cuda")
    with pytest.raises(R.RapidError) as e:
        R.rapid_verify_attention_paged(q, pool, pool, table, ctx, cfg.gamma, out, ws)
    assert e.value.code == 2
    pool = torch.zeros(8, 2, 32, 64, dtype=torch.bfloat16, device="cuda")   # smaller than a key tile
    with pytest.raises(R.RapidError) as e:
        R.rapid_verify_attention_paged(q, pool, pool, table, ctx, cfg.gamma, out, ws)
    assert e.value.code == 2
