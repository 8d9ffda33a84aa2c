"""Checks that stand in for a memory checker, and the status bits that only unusual inputs raise.

Guard bands: every output and scratch buffer of a call lives inside a larger allocation filled with
a sentinel; after the call the bytes around the buffer must be untouched.  Status bits: the empty
residual (defined fallback to p), and an on-chip wait that runs out (the kernel returns, says so,
and the next call on the same workspace is correct).
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle
from oracle import parity
import workloads as wl
from workloads import bf16_bits

BAND = 4096          # bytes of sentinel on either side
SENTINEL = 0xA5


class Banded:
    """A tensor carved out of the middle of a sentinel-filled byte buffer (256-byte aligned start)."""

    def __init__(self, shape, dtype, fill=None):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        self.nbytes = n
        self.raw = torch.full((BAND + n + BAND + 256,), SENTINEL, dtype=torch.uint8, device="cuda")
        off = (-self.raw.data_ptr() - BAND) % 256 + BAND
        self.off = off
        self.t = self.raw[off:off + n].view(dtype).view(shape)
        if fill is not None:
            self.t.copy_(fill)

    def intact(self):
        before = self.raw[:self.off]
        after = self.raw[self.off + self.nbytes:]
        return bool((before == SENTINEL).all().item()) and bool((after == SENTINEL).all().item())


def _banded_attention(cfg, seed, kernel=0, num_ctas=0, paged_block=0, plan=0, sink=0, window=0):
    import paper_2502_20330_b200 as R
    q, k, v, ctx = wl.attention_inputs(cfg, seed=seed, device="cuda", poison_padding=True)
    B, Rr, Hq, D = q.shape
    Hkv, Lmax = k.shape[1], k.shape[2]
    if paged_block:
        kp, vp, table = wl.paged_layout(k, v, ctx.cpu(), paged_block, seed=seed)
        Lmax = table.shape[1] * paged_block
    nbytes = R.attention_workspace_bytes(B, Hq, Hkv, D, Lmax, cfg.gamma)
    out = Banded(q.shape, torch.bfloat16)
    o32 = Banded(q.shape, torch.float32)
    lse = Banded(q.shape[:3], torch.float32)
    ws = Banded((nbytes,), torch.uint8)
    lens = Banded(ctx.shape, torch.int32, fill=ctx)
    R.workspace_init(ws.t)
    params = R.AttnParams(num_ctas=num_ctas, lse_out=lse.t, out_f32=o32.t, kernel=kernel, plan=plan,
                          sink_keys=sink, window_keys=window)
    if plan:
        R.rapid_attention_plan(lens.t, cfg.gamma, B, Hq, Hkv, D, Lmax, ws.t, params)
    if paged_block:
        R.rapid_verify_attention_paged(q, kp, vp, table, lens.t, cfg.gamma, out.t, ws.t, params)
    else:
        R.rapid_verify_attention(q, k, v, lens.t, cfg.gamma, out.t, ws.t, params)
    torch.cuda.synchronize()
    assert R.workspace_status(ws.t) == 0
    for name, b in (("out", out), ("out_f32", o32), ("lse", lse), ("workspace", ws), ("ctx_lens", lens)):
        assert b.intact(), f"bytes around {name} were written"
    assert torch.equal(lens.t, ctx)
    ref, ref_lse = oracle.verify_attention(bf16_bits(q), bf16_bits(k), bf16_bits(v), ctx.cpu().numpy(), cfg.gamma,
                                           sink=sink, window=window)
    parity.check_attention(out.t.float().cpu().numpy(), ref)


@pytest.mark.parametrize("kernel,num_ctas,paged_block,plan,sink,window", [
    (0, 0, 0, 0, 0, 0), (1, 0, 0, 0, 0, 0), (2, 0, 0, 0, 0, 0), (3, 0, 0, 0, 0, 0),
    (2, 512, 0, 1, 0, 0), (1, 512, 0, 1, 0, 0),      # the most CTAs the workspace is sized for
    (0, 0, 64, 0, 0, 0), (1, 0, 256, 2, 0, 0), (3, 0, 64, 2, 0, 0),
    (2, 0, 0, 0, 4, 300), (1, 7, 0, 0, 0, 129),
])
def test_attention_writes_nothing_outside_its_buffers(kernel, num_ctas, paged_block, plan, sink, window):
    """The ragged 7B-shaped batch (35 grouped rows) scaled down, on every kernel, split and cache layout."""
    cfg = wl.VerifyConfig("g", B=3, Hq=28, Hkv=4, D=128, gamma=4, V=4096, ctx_lens=(2900, 5, 1217), Lmax=3072)
    _banded_attention(cfg, 81, kernel, num_ctas, paged_block, plan, sink, window)


@pytest.mark.parametrize("Hq,Hkv,D,gamma", [(8, 2, 64, 4), (64, 8, 128, 8), (16, 1, 64, 7), (64, 8, 128, 7)])
def test_attention_guard_bands_other_row_counts(Hq, Hkv, D, gamma):
    """The tiny shape (20 rows, head_dim 64), 72 rows, the 128-row maximum, and 64 rows (two softmax groups)."""
    cfg = wl.VerifyConfig("g", B=2, Hq=Hq, Hkv=Hkv, D=D, gamma=gamma, V=4096, ctx_lens=(1500, 300), Lmax=1536)
    _banded_attention(cfg, 82)
    _banded_attention(cfg, 82, kernel=1, num_ctas=300)


def test_accept_and_bookkeeping_write_nothing_outside_their_buffers():
    import paper_2502_20330_b200 as R
    cfg = wl.VerifyConfig("g", B=5, Hq=8, Hkv=2, D=128, gamma=4, V=32000, ctx_lens=(300,) * 5, Lmax=384,
                          target_sigma=1.0)
    z, d, tok, u = wl.accept_inputs(cfg, seed=83, device="cuda")
    ws = Banded((R.accept_workspace_bytes(cfg.B, cfg.gamma, cfg.V),), torch.uint8)
    alen = Banded((cfg.B,), torch.int32)
    ntok = Banded((cfg.B,), torch.int32)
    ratios = Banded((cfg.B, cfg.gamma), torch.float32)
    R.workspace_init(ws.t)
    R.rapid_accept(z, d, tok, u, 5.0, alen.t, ntok.t, ws.t, R.AcceptParams(ratio_out=ratios.t))
    torch.cuda.synchronize()
    for name, b in (("workspace", ws), ("accept_len", alen), ("next_token", ntok), ("ratio_out", ratios)):
        assert b.intact(), f"bytes around {name} were written"
    parity.check_accept(z.cpu().numpy(), d.cpu().numpy(), tok.cpu().numpy(), u.cpu().numpy(), 5.0, 1.0, 0.1, 0,
                        alen.t.cpu().numpy(), ntok.t.cpu().numpy(), ratios.t.cpu().numpy())
    # draft sampling: token, log-probability, row statistics
    tokb, logq, stats = Banded((cfg.B,), torch.int32), Banded((cfg.B,), torch.float32), Banded((cfg.B, 2), torch.float32)
    ws2 = Banded((R.accept_workspace_bytes(cfg.B, 0, cfg.V),), torch.uint8)
    R.workspace_init(ws2.t)
    R.rapid_draft_sample(d[:, 0], u[:, 0].contiguous(), 1.0, tokb.t, logq.t, ws2.t, out_row_stats=stats.t)
    torch.cuda.synchronize()
    assert all(b.intact() for b in (tokb, logq, stats, ws2))
    # append + commit: the cache rows past the appended ones and the lengths' neighbours stay as they were
    q, k, v, ctx = wl.attention_inputs(cfg, seed=84, device="cuda")
    kc = Banded(k.shape, torch.bfloat16, fill=k)
    vc = Banded(v.shape, torch.bfloat16, fill=v)
    lens = Banded(ctx.shape, torch.int32, fill=ctx)
    status = Banded((1,), torch.int32, fill=torch.zeros(1, dtype=torch.int32, device="cuda"))
    g = torch.Generator(device="cuda").manual_seed(85)
    kn = torch.randn(cfg.B, cfg.R, cfg.Hkv, cfg.D, generator=g, device="cuda").to(torch.bfloat16)
    vn = torch.randn(cfg.B, cfg.R, cfg.Hkv, cfg.D, generator=g, device="cuda").to(torch.bfloat16)
    R.rapid_kv_append(kn, vn, kc.t, vc.t, lens.t, cfg.gamma, status.t)
    R.rapid_step_commit(lens.t, alen.t, cfg.gamma, status.t)
    torch.cuda.synchronize()
    assert all(b.intact() for b in (kc, vc, lens, status)) and int(status.t.item()) == 0
    assert torch.equal(kc.t[:, :, 300 + cfg.R:], k[:, :, 300 + cfg.R:]) and torch.equal(kc.t[:, :, :300], k[:, :, :300])
    assert torch.equal(kc.t[:, :, 300:300 + cfg.R].permute(0, 2, 1, 3), kn)


def test_sharded_merge_guard_bands():
    import paper_2502_20330_b200 as R
    g = torch.Generator(device="cuda").manual_seed(86)
    P, rows, D = 3, 333, 128
    o = torch.randn(P, rows, D, generator=g, device="cuda")
    l = torch.randn(P, rows, generator=g, device="cuda")
    out, o32, lse = Banded((rows, D), torch.bfloat16), Banded((rows, D), torch.float32), Banded((rows,), torch.float32)
    R.rapid_merge_partials(o, l, out=out.t, out_f32=o32.t, lse_out=lse.t)
    torch.cuda.synchronize()
    assert out.intact() and o32.intact() and lse.intact()
    ref, _ = oracle.merge_partials(o.cpu().numpy(), l.cpu().numpy())
    np.testing.assert_allclose(o32.t.cpu().numpy(), ref, rtol=0, atol=2e-5)


@pytest.mark.parametrize("Hq,gamma,lens,num_ctas,plan", [
    (32, 8, (3000, 777), 0, 0), (64, 8, (1500, 500), 0, 2), (32, 0, (2048,), 512, 1),
])
def test_fp8_attention_guard_bands(Hq, gamma, lens, num_ctas, plan):
    """The 8-bit-cache call inside sentinel bands, planned and unplanned, early copies included."""
    import paper_2502_20330_b200 as R
    cfg = wl.VerifyConfig("g8", B=len(lens), Hq=Hq, Hkv=8, D=128, gamma=gamma, V=4096, ctx_lens=lens)
    q, kc, vc, ks, vs, ctx = wl.attention_inputs_fp8(cfg, seed=91, device="cuda", poison_padding=True)
    Lmax = kc.shape[2]
    nbytes = R.attention_workspace_bytes(cfg.B, Hq, 8, 128, Lmax, gamma)
    out, o32 = Banded(q.shape, torch.bfloat16), Banded(q.shape, torch.float32)
    lse, ws = Banded(q.shape[:3], torch.float32), Banded((nbytes,), torch.uint8)
    lens_b = Banded(ctx.shape, torch.int32, fill=ctx)
    ksb, vsb = Banded(ks.shape, torch.float32, fill=ks), Banded(vs.shape, torch.float32, fill=vs)
    R.workspace_init(ws.t)
    params = R.AttnParams(num_ctas=num_ctas, lse_out=lse.t, out_f32=o32.t, plan=plan, kv_fp8=True,
                          kv_settled=plan == R.PLAN_SETTLED)
    if plan:
        R.rapid_attention_plan(lens_b.t, gamma, cfg.B, Hq, 8, 128, Lmax, ws.t, params)
        if plan == R.PLAN_SETTLED:
            torch.zeros(8, device="cuda").add_(1.0)
    R.rapid_verify_attention_fp8(q, kc, vc, ksb.t, vsb.t, lens_b.t, gamma, out.t, ws.t, params)
    torch.cuda.synchronize()
    assert R.workspace_status(ws.t) == 0
    for name, b in (("out", out), ("out_f32", o32), ("lse", lse), ("workspace", ws), ("ctx_lens", lens_b),
                    ("k_scale", ksb), ("v_scale", vsb)):
        assert b.intact(), f"bytes around {name} were written"
    ref, ref_lse = oracle.verify_attention_fp8(bf16_bits(q), kc.cpu().numpy(), vc.cpu().numpy(), ks.cpu().numpy(),
                                               vs.cpu().numpy(), ctx.cpu().numpy(), gamma)
    parity.check_attention(out.t.float().cpu().numpy(), ref, ~np.isnan(ref_lse))


# ---- RAPID_STATUS_RESIDUAL_FALLBACK ----------------------------------------------------------------------

def _accept(z, d, tok, u, eta, mode=0):
    import paper_2502_20330_b200 as R
    B, Rr, V = z.shape
    ws = R.new_workspace(R.accept_workspace_bytes(B, Rr - 1, V))
    alen = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    ntok = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    R.rapid_accept(z, d, tok, u, eta, alen, ntok, ws, R.AcceptParams(residual_mode=mode))
    torch.cuda.synchronize()
    return alen.cpu().numpy(), ntok.cpu().numpy(), R.workspace_status(ws)


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("hot", [1, 2, 8])
def test_empty_residual_falls_back_to_p_and_says_so(mode, hot):
    """Target and draft logits identical, all mass on `hot` tokens (the rest -inf): p = q = phat exactly
    (every sum is a power of two), so the ratio is exactly 1 and the residual is exactly empty.  An
    acceptance draw of 1.5 -- outside [0, 1), but the comparison u <= min(1, ratio) is defined for it --
    rejects the draft all the same, and Algorithm 1's residual step has nothing to draw from: the
    defined fallback draws from p and raises the status bit, in the oracle and on the device alike."""
    import paper_2502_20330_b200 as R
    B, gamma, V = 3, 2, 4096
    z = torch.full((B, gamma + 1, V), float("-inf"), device="cuda")
    z[:, :, 100:100 + hot] = 0.0
    d = z[:, :gamma].clone()
    tok = torch.full((B, gamma), 100, dtype=torch.int32, device="cuda")
    u = torch.tensor([[0.3, 1.5, 0.7],      # accepts position 0, is made to reject position 1: empty residual
                      [1.5, 0.2, 0.01],     # rejects position 0
                      [0.1, 0.2, 0.99]],    # accepts everything: bonus row, no fallback involved
                     dtype=torch.float32, device="cuda")
    ref = oracle.accept(z.cpu().numpy(), d.cpu().numpy(), tok.cpu().numpy(), u.cpu().numpy(), eta=5.0,
                        residual_mode=mode)
    assert ref["accept_len"].tolist() == [1, 0, 2]
    assert ref["flags"].tolist() == [oracle.FLAG_RESIDUAL_FALLBACK, oracle.FLAG_RESIDUAL_FALLBACK, 0]
    alen, ntok, status = _accept(z, d, tok, u, 5.0, mode)
    assert alen.tolist() == [1, 0, 2]
    assert status == R.STATUS_RESIDUAL_FALLBACK
    assert ntok.tolist() == ref["next_token"].tolist()          # p is (1/hot, ...) exactly: no boundary case
    # the same rows where Algorithm 1 never reaches the empty residual: no bit
    u2 = u.clone(); u2[0, 1] = 0.5; u2[1, 0] = 0.5
    alen, ntok, status = _accept(z, d, tok, u2, 5.0, mode)
    assert alen.tolist() == [2, 2, 2] and status == 0


def test_empty_residual_of_a_row_the_loop_never_reaches_raises_nothing():
    """Every row is evaluated speculatively; an empty residual behind the first rejection must stay silent."""
    cfg = wl.VerifyConfig("f", B=4, Hq=8, Hkv=2, D=64, gamma=3, V=4096, ctx_lens=(64,) * 4, target_sigma=1.0)
    z, d, tok, u = wl.accept_inputs(cfg, seed=87, device="cuda")
    z[:, 1:3] = float("-inf"); z[:, 1:3, 7] = 0.0        # positions 1 and 2: p = q = phat, empty residual
    d[:, 1:3] = z[:, 1:3]
    tok[:, 1:3] = 7
    u[:, 0] = 1.5                                        # position 0 (ordinary random logits) rejects
    ref = oracle.accept(z.cpu().numpy(), d.cpu().numpy(), tok.cpu().numpy(), u.cpu().numpy(), eta=0.5)
    assert ref["accept_len"].tolist() == [0] * 4 and ref["flags"].tolist() == [0] * 4
    alen, ntok, status = _accept(z, d, tok, u, 0.5)
    assert alen.tolist() == [0] * 4 and status == 0
    parity.check_accept(z.cpu().numpy(), d.cpu().numpy(), tok.cpu().numpy(), u.cpu().numpy(), 0.5, 1.0, 0.1, 0,
                        alen, ntok)


# ---- RAPID_STATUS_PIPELINE_TIMEOUT -----------------------------------------------------------------------

@pytest.mark.parametrize("limit", [1, 3000, 40000])
def test_a_wait_that_runs_out_after_early_copies_went_out(limit):
    """The same with a settled plan and kv_settled: the producer has copies in flight from before its
    stream-order wait when its first bounded wait gives up, and must see them land before the CTA ends."""
    import paper_2502_20330_b200 as R
    cfg = wl.VerifyConfig("to", B=2, Hq=32, Hkv=8, D=128, gamma=8, V=4096, ctx_lens=(40000, 30000))
    q, k, v, ctx = wl.attention_inputs(cfg, seed=89, device="cuda")
    Lmax = k.shape[2]
    ws = R.new_workspace(R.attention_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.D, Lmax, cfg.gamma))
    out = torch.empty_like(q)
    ref, _ = oracle.verify_attention(bf16_bits(q), bf16_bits(k), bf16_bits(v), ctx.cpu().numpy(), cfg.gamma)

    def call(lim):
        R.rapid_attention_plan(ctx, cfg.gamma, cfg.B, cfg.Hq, cfg.Hkv, cfg.D, Lmax, ws, R.AttnParams())
        torch.zeros(8, device="cuda").add_(1.0)
        R.rapid_verify_attention(q, k, v, ctx, cfg.gamma, out, ws,
                                 R.AttnParams(plan=R.PLAN_SETTLED, kv_settled=True, wait_cycle_limit=lim))
        torch.cuda.synchronize()
        return R.workspace_status(ws)

    status = call(limit)
    if limit == 1:
        assert status == R.STATUS_PIPELINE_TIMEOUT
    else:
        assert status in (0, R.STATUS_PIPELINE_TIMEOUT)
    R.workspace_init(ws)
    assert call(0) == 0
    parity.check_attention(out.float().cpu().numpy(), ref)


@pytest.mark.parametrize("limit", [1, 3000, 40000])
def test_a_wait_that_runs_out_over_the_fp8_cache(limit):
    import paper_2502_20330_b200 as R
    cfg = wl.VerifyConfig("to8", B=2, Hq=32, Hkv=8, D=128, gamma=8, V=4096, ctx_lens=(40000, 30000))
    q, kc, vc, ks, vs, ctx = wl.attention_inputs_fp8(cfg, seed=90, device="cuda")
    ws = R.new_workspace(R.attention_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.D, kc.shape[2], cfg.gamma))
    out = torch.empty_like(q)
    R.rapid_verify_attention_fp8(q, kc, vc, ks, vs, ctx, cfg.gamma, out, ws, R.AttnParams(wait_cycle_limit=limit))
    torch.cuda.synchronize()
    status = R.workspace_status(ws)
    if limit == 1:
        assert status == R.STATUS_PIPELINE_TIMEOUT
    else:
        assert status in (0, R.STATUS_PIPELINE_TIMEOUT)
    R.workspace_init(ws)
    R.rapid_verify_attention_fp8(q, kc, vc, ks, vs, ctx, cfg.gamma, out, ws)
    torch.cuda.synchronize()
    assert R.workspace_status(ws) == 0
    ref, ref_lse = oracle.verify_attention_fp8(bf16_bits(q), kc.cpu().numpy(), vc.cpu().numpy(), ks.cpu().numpy(),
                                               vs.cpu().numpy(), ctx.cpu().numpy(), cfg.gamma)
    parity.check_attention(out.float().cpu().numpy(), ref, ~np.isnan(ref_lse))


@pytest.mark.parametrize("kernel", [1, 2, 3])
@pytest.mark.parametrize("limit", [1, 3000, 40000])
def test_a_wait_that_runs_out_ends_the_kernel_and_is_reported(kernel, limit):
    """A healthy launch whose on-chip waits are given too little time (1 cycle: the first wait that is not
    already satisfied gives up; a few thousand cycles: some tile in mid-stream).  The kernel is the
    ordinary one, nothing is withheld from it: the waits simply give up early.  It must return, raise
    RAPID_STATUS_PIPELINE_TIMEOUT whenever a wait did run out, and leave the workspace usable."""
    import paper_2502_20330_b200 as R
    cfg = wl.VerifyConfig("to", B=2, Hq=32, Hkv=8, D=128, gamma=8, V=4096, ctx_lens=(40000, 30000))
    q, k, v, ctx = wl.attention_inputs(cfg, seed=88, device="cuda")
    ws = R.new_workspace(R.attention_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.D, k.shape[2], cfg.gamma))
    out = torch.empty_like(q)
    R.rapid_verify_attention(q, k, v, ctx, cfg.gamma, out, ws, R.AttnParams(kernel=kernel, wait_cycle_limit=limit))
    torch.cuda.synchronize()
    status = R.workspace_status(ws)
    ref, _ = oracle.verify_attention(bf16_bits(q), bf16_bits(k), bf16_bits(v), ctx.cpu().numpy(), cfg.gamma)
    if limit == 1:
        assert status == R.STATUS_PIPELINE_TIMEOUT
    else:
        assert status in (0, R.STATUS_PIPELINE_TIMEOUT)
        if status == 0:
            parity.check_attention(out.float().cpu().numpy(), ref)
    # the next ordinary call on the same workspace
    R.workspace_init(ws)
    out2 = torch.empty_like(q)
    R.rapid_verify_attention(q, k, v, ctx, cfg.gamma, out2, ws, R.AttnParams(kernel=kernel))
    torch.cuda.synchronize()
    assert R.workspace_status(ws) == 0
    parity.check_attention(out2.float().cpu().numpy(), ref)
