"""Verify attention over an FP8 E4M3 KV cache against the fp64 oracle over the same codes, through the C ABI."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle
from oracle import parity
import workloads as wl
from workloads import bf16_bits

# The log-sum-exp of the 8-bit path: the scores carry the rounding of q to two E4M3 parts (8 significant bits
# per element, about 2e-3 absolute on a score of unit-variance data), which a sum over many keys averages
# but a row that one key dominates shows in full.
LSE_TOL_FP8 = 5e-3


def _run(q, kc, vc, ks, vs, ctx, gamma, num_ctas=0, plan=0, scale=0.0):
    import paper_2502_20330_b200 as R
    B, Rr, Hq, D = q.shape
    Hkv, Lmax = kc.shape[1], kc.shape[2]
    ws = R.new_workspace(R.attention_workspace_bytes(B, Hq, Hkv, D, Lmax, gamma))
    out = torch.empty_like(q)
    lse = torch.empty(B, Rr, Hq, dtype=torch.float32, device=q.device)
    o32 = torch.empty(B, Rr, Hq, D, dtype=torch.float32, device=q.device)
    params = R.AttnParams(num_ctas=num_ctas, lse_out=lse, out_f32=o32, plan=plan, scale=scale, kv_fp8=True)
    if plan:
        R.rapid_attention_plan(ctx, gamma, B, Hq, Hkv, D, Lmax, ws, params)
        if plan == R.PLAN_SETTLED:
            torch.zeros(8, device=q.device).add_(1.0)
    R.rapid_verify_attention_fp8(q, kc, vc, ks, vs, ctx, gamma, out, ws, params)
    torch.cuda.synchronize()
    return out, lse, o32, R.workspace_status(ws)


def _compare(q, kc, vc, ks, vs, ctx, gamma, units=None, **kw):
    out, lse, o32, status = _run(q, kc, vc, ks, vs, ctx, gamma, **kw)
    assert status == 0
    ref, ref_lse = oracle.verify_attention_fp8(bf16_bits(q), kc.cpu().numpy(), vc.cpu().numpy(), ks.cpu().numpy(),
                                               vs.cpu().numpy(), ctx.cpu().numpy(), gamma, scale=kw.get("scale", 0.0),
                                               units=units)
    rows = ~np.isnan(ref_lse)
    rep = parity.check_attention(out.float().cpu().numpy(), ref, rows)
    parity.check_attention(o32.cpu().numpy(), ref, rows)
    rep["max_lse_err"] = float(np.abs(lse.cpu().numpy()[rows] - ref_lse[rows]).max())
    assert rep["max_lse_err"] < LSE_TOL_FP8, rep
    return rep, o32


@pytest.mark.parametrize("Hq,Hkv,gamma,lens", [
    (32, 8, 0, (777, 300)),          # one-row decode: 16 columns
    (8, 2, 4, (1000, 129)),          # 20 grouped rows: 32 columns
    (32, 8, 8, (2048 + 37, 700)),    # 36 rows: 48 columns
    (28, 4, 4, (3000, 5)),           # 35 rows, G = 7; a sequence of exactly R keys
    (64, 8, 6, (2900, 966)),         # 56 rows: 64 columns, two softmax groups
    (64, 8, 7, (1333, 444)),         # 64 rows
    (64, 8, 8, (1500, 500)),         # 72 rows: 96 columns, two groups
    (96, 8, 7, (4000, 1300)),        # 96 rows: the most
    (4, 4, 2, (70, 23)),             # G = 1, less than a tile
])
def test_shapes_against_oracle(Hq, Hkv, gamma, lens):
    cfg = wl.VerifyConfig("f8", B=len(lens), Hq=Hq, Hkv=Hkv, D=128, gamma=gamma, V=4096, ctx_lens=lens)
    q, kc, vc, ks, vs, ctx = wl.attention_inputs_fp8(cfg, seed=2, device="cuda", poison_padding=True)
    _, o32 = _compare(q, kc, vc, ks, vs, ctx, gamma)
    _, again = _compare(q, kc, vc, ks, vs, ctx, gamma, plan=2)
    assert torch.equal(o32, again)                         # bit-identical from run to run, planned or not
    _compare(q, kc, vc, ks, vs, ctx, gamma, num_ctas=3, plan=1)
    _compare(q, kc, vc, ks, vs, ctx, gamma, num_ctas=300)


def test_peaked_scores_move_the_references():
    """Queries four times larger and a few keys far above the rest, early and late in the context."""
    cfg = wl.VerifyConfig("f8", B=2, Hq=32, Hkv=8, D=128, gamma=8, V=4096, ctx_lens=(9000, 5000), q_scale=4.0)
    q, kc, vc, ks, vs, ctx = wl.attention_inputs_fp8(cfg, seed=5, device="cuda")
    _compare(q, kc, vc, ks, vs, ctx, cfg.gamma)
    ks2 = ks * 3.0                                         # every score three times larger still
    _compare(q, kc, vc, ks2, vs, ctx, cfg.gamma)
    _compare(q, kc, vc, ks, vs, ctx, cfg.gamma, scale=0.02)


def test_random_sweep():
    rng = np.random.default_rng(17)
    layouts = [(8, 2), (16, 2), (7, 7), (32, 8), (64, 8), (28, 4), (40, 4), (72, 8), (12, 12), (96, 8), (5, 1), (48, 8)]
    for trial in range(60):
        Hq, Hkv = layouts[int(rng.integers(len(layouts)))]
        G = Hq // Hkv
        gamma = int(rng.integers(0, min(11, 96 // G - 1) + 1))
        B = int(rng.integers(1, 4))
        Lmax = int(rng.integers(gamma + 1, 2600))
        lens = tuple(int(rng.integers(gamma + 1, Lmax + 1)) for _ in range(B))
        cfg = wl.VerifyConfig("f8s", B=B, Hq=Hq, Hkv=Hkv, D=128, gamma=gamma, V=4096, ctx_lens=lens, Lmax=Lmax,
                              q_scale=float(rng.choice([1.0, 1.0, 3.0])))
        q, kc, vc, ks, vs, ctx = wl.attention_inputs_fp8(cfg, seed=4000 + trial, device="cuda", poison_padding=True)
        num_ctas = int(rng.choice([0, 1, 2, 3, 5, 16, 37, 148, 300, 512]))
        _compare(q, kc, vc, ks, vs, ctx, gamma, num_ctas=num_ctas)


@pytest.mark.parametrize("name", ["llama8b_32k", "llama8b_128k", "llama70b_128k", "qwen7b_ragged", "drafter_8k"])
def test_full_size_workloads_every_row(name):
    cfg = wl.CONFIGS[name]
    q, kc, vc, ks, vs, ctx = wl.attention_inputs_fp8(cfg, seed=21, device="cuda", poison_padding=True)
    rep, _ = _compare(q, kc, vc, ks, vs, ctx, cfg.gamma)
    assert rep["rows"] == cfg.B * cfg.R * cfg.Hq
    _compare(q, kc, vc, ks, vs, ctx, cfg.gamma, plan=2)


def test_argument_errors():
    import paper_2502_20330_b200 as R
    cfg = wl.VerifyConfig("f8", B=1, Hq=8, Hkv=2, D=128, gamma=2, V=4096, ctx_lens=(128,))
    q, kc, vc, ks, vs, ctx = wl.attention_inputs_fp8(cfg, seed=9, device="cuda")
    ws = R.new_workspace(R.attention_workspace_bytes(1, 8, 2, 128, 128, 2))
    out = torch.empty_like(q)
    for bad in (dict(window_keys=5), dict(kernel=1), dict(kernel=3)):
        with pytest.raises(R.RapidError) as e:
            R.rapid_verify_attention_fp8(q, kc, vc, ks, vs, ctx, 2, out, ws, R.AttnParams(**bad))
        assert e.value.code == 2
    cfg64 = wl.VerifyConfig("f8", B=1, Hq=8, Hkv=2, D=64, gamma=2, V=4096, ctx_lens=(128,))
    q2 = torch.zeros(1, 3, 8, 64, dtype=torch.bfloat16, device="cuda")
    k2 = torch.zeros(1, 2, 128, 64, dtype=torch.uint8, device="cuda")
    ws2 = R.new_workspace(R.attention_workspace_bytes(1, 8, 2, 64, 128, 2))
    with pytest.raises(R.RapidError) as e:
        R.rapid_verify_attention_fp8(q2, k2, k2, ks, vs, ctx, 2, torch.empty_like(q2), ws2)
    assert e.value.code == 2


def test_a_plan_made_for_another_kernel_is_refused_not_followed():
    """72 grouped rows: a plan made for the rows-on-M kernel (64-key tiles, two partials per CTA).  The 8-bit call must not walk it: every CTA compares the plan's signature with its own call, does
    nothing on a mismatch, and the status word says why the output is empty."""
    import paper_2502_20330_b200 as R
    cfg = wl.VerifyConfig("f8", B=2, Hq=64, Hkv=8, D=128, gamma=8, V=4096, ctx_lens=(1500, 500))
    q, kc, vc, ks, vs, ctx = wl.attention_inputs_fp8(cfg, seed=2, device="cuda")
    ws = R.new_workspace(R.attention_workspace_bytes(2, 64, 8, 128, 1500, 8))
    R.rapid_attention_plan(ctx, 8, 2, 64, 8, 128, 1500, ws, R.AttnParams(kernel=R.ATTN_KERNEL_ROWS_ON_M))
    out = torch.full_like(q, 7.0)
    R.rapid_verify_attention_fp8(q, kc, vc, ks, vs, ctx, 8, out, ws, R.AttnParams(plan=R.PLAN_SETTLED))
    torch.cuda.synchronize()
    assert R.workspace_status(ws) & R.STATUS_STALE_PLAN
    assert (out == 0).all()
    # a workspace that never saw a plan at all
    ws2 = R.new_workspace(R.attention_workspace_bytes(2, 64, 8, 128, 1500, 8))
    ws2[256:].fill_(0x5A)
    R.rapid_verify_attention_fp8(q, kc, vc, ks, vs, ctx, 8, out, ws2, R.AttnParams(plan=R.PLAN_READY))
    q2, k2, v2, ctx2 = wl.attention_inputs(cfg, seed=2, device="cuda")
    R.rapid_verify_attention(q2, k2, v2, ctx2, 8, out, ws2, R.AttnParams(plan=R.PLAN_SETTLED, kernel=2))
    R.rapid_verify_attention(q2, k2, v2, ctx2, 8, out, ws2, R.AttnParams(plan=R.PLAN_SETTLED, kernel=R.ATTN_KERNEL_ROWS_ON_M))
    torch.cuda.synchronize()
    assert R.workspace_status(ws2) & R.STATUS_STALE_PLAN


def test_early_copies_of_the_settled_cache_change_nothing():
    """kv_settled over the 8-bit cache: two layers back to back, the second one's first tiles copied while
    the first one's merge still runs; the newest rows of each layer arrive right before its call."""
    import paper_2502_20330_b200 as R
    lens, gamma = (9000, 700), 8
    cfg = wl.VerifyConfig("f8", B=2, Hq=32, Hkv=8, D=128, gamma=gamma, V=4096, ctx_lens=lens)
    layers = [wl.attention_inputs_fp8(cfg, seed=70 + i, device="cuda") for i in range(2)]
    ctx, Lmax, Rr = layers[0][5], layers[0][1].shape[2], gamma + 1
    ws = R.new_workspace(R.attention_workspace_bytes(2, 32, 8, 128, Lmax, gamma))
    news = [[(kc[b, :, L - Rr:L].clone(), vc[b, :, L - Rr:L].clone()) for b, L in enumerate(lens)]
            for _, kc, vc, _, _, _ in layers]
    o32s = [torch.zeros(2, Rr, 32, 128, device="cuda") for _ in range(2)]
    outs = [torch.zeros_like(layers[0][0]) for _ in range(2)]

    def run(flag):
        for _, kc, vc, _, _, _ in layers:           # the newest rows are not there yet (NaN codes)
            for b, L in enumerate(lens):
                kc[b, :, L - Rr:L] = 0x7F
                vc[b, :, L - Rr:L] = 0x7F
        torch.cuda.synchronize()
        R.rapid_attention_plan(ctx, gamma, 2, 32, 8, 128, Lmax, ws, R.AttnParams(kv_fp8=True))
        for i, (q, kc, vc, ks, vs, _) in enumerate(layers):
            for b, L in enumerate(lens):
                kc[b, :, L - Rr:L] = news[i][b][0]
                vc[b, :, L - Rr:L] = news[i][b][1]
            R.rapid_verify_attention_fp8(q, kc, vc, ks, vs, ctx, gamma, outs[i], ws,
                                         R.AttnParams(plan=R.PLAN_SETTLED, kv_settled=flag, out_f32=o32s[i], kv_fp8=True))
        torch.cuda.synchronize()
        assert R.workspace_status(ws) == 0
        return [o.clone() for o in o32s]

    plain, early = run(False), run(True)
    for i, (q, kc, vc, ks, vs, _) in enumerate(layers):
        ref, ref_lse = oracle.verify_attention_fp8(bf16_bits(q), kc.cpu().numpy(), vc.cpu().numpy(), ks.cpu().numpy(),
                                                   vs.cpu().numpy(), ctx.cpu().numpy(), gamma)
        parity.check_attention(early[i].cpu().numpy(), ref, ~np.isnan(ref_lse))
        assert torch.equal(early[i], plain[i])
