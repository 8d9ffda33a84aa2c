"""Parity of the CUDA verify attention with the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle
from oracle import parity
import workloads as wl
from workloads import bf16_bits


# Absolute tolerance of the natural-log sum-exp, one figure for every kernel and shape.  When the
# caller takes this output, every kernel adds fp32 probabilities into fp32 row sums (the keys-on-M
# kernel then serves 49 to 64 grouped rows with two softmax groups, which have the registers for
# it).  What is left: each probability carries the relative error of ex2.approx (2 ulp, 2.4e-7)
# and of its fp32 argument (scores up to ~30 in log2 units, rounded to 24 bits: 2e-6), and the
# partial sums of at most 2^17 terms are added in a tree of depth ~17 over threads, CTAs and
# slots, each step rounding by 6e-8.  All of it is relative to the sum, so ln(sum) moves by at
# most a few 1e-6; the reference itself (m in base 2, times ln 2) rounds at |lse| * 6e-8 <= 1e-6.
LSE_TOL = 1e-4


def _run(q, k, v, ctx, gamma, num_ctas=0, scale=0.0, kernel=0, sink=0, window=0, plan=0, want_lse=True):
    import paper_2502_20330_b200 as R
    B, Rr, Hq, D = q.shape
    Hkv, Lmax = k.shape[1], k.shape[2]
    ws = R.new_workspace(R.attention_workspace_bytes(B, Hq, Hkv, D, Lmax, gamma))
    out = torch.empty_like(q)
    lse = torch.empty(B, Rr, Hq, dtype=torch.float32, device=q.device) if want_lse else None
    o32 = torch.empty(B, Rr, Hq, D, dtype=torch.float32, device=q.device)
    params = R.AttnParams(scale=scale, num_ctas=num_ctas, lse_out=lse, out_f32=o32, kernel=kernel,
                          sink_keys=sink, window_keys=window, plan=plan)
    if plan:
        R.rapid_attention_plan(ctx, gamma, B, Hq, Hkv, D, Lmax, ws, params)
        if plan == R.PLAN_SETTLED:      # some other kernel between the plan and the call
            torch.zeros(8, device=q.device).add_(1.0)
    R.rapid_verify_attention(q, k, v, ctx, gamma, out, ws, params)
    torch.cuda.synchronize()
    return out, lse, o32, R.workspace_status(ws)


def _oracle(q, k, v, ctx, gamma, scale=0.0, units=None, sink=0, window=0):
    return oracle.verify_attention(bf16_bits(q), bf16_bits(k), bf16_bits(v), ctx.cpu().numpy(), gamma,
                                   scale=scale, units=units, sink=sink, window=window)


def _compare(q, k, v, ctx, gamma, num_ctas=0, scale=0.0, units=None, kernel=0, sink=0, window=0, plan=0,
             want_lse=True):
    out, lse, o32, status = _run(q, k, v, ctx, gamma, num_ctas, scale, kernel, sink, window, plan, want_lse)
    assert status == 0
    ref, ref_lse = _oracle(q, k, v, ctx, gamma, scale, units, sink, window)
    rows = ~np.isnan(ref_lse)
    rep = parity.check_attention(out.float().cpu().numpy(), ref, rows)
    parity.check_attention(o32.cpu().numpy(), ref, rows)
    if want_lse:
        rep["max_lse_err"] = float(np.abs(lse.cpu().numpy()[rows] - ref_lse[rows]).max())
        assert rep["max_lse_err"] < LSE_TOL, rep
    return rep, out, o32


def test_tiny_config():
    cfg = wl.CONFIGS["tiny"]
    q, k, v, ctx = wl.attention_inputs(cfg, seed=1, device="cuda")
    rep, _, _ = _compare(q, k, v, ctx, cfg.gamma)
    assert rep["rows"] == cfg.B * cfg.R * cfg.Hq


@pytest.mark.parametrize("Hq,Hkv,D,gamma,L", [
    (32, 8, 128, 8, 2048 + 37),     # 36 grouped rows, ragged tail
    (64, 8, 128, 8, 1500),          # 72 grouped rows (five row blocks)
    (28, 4, 128, 4, 3000),          # 35 grouped rows, G = 7
    (32, 8, 128, 0, 777),           # one-row decode (drafter-side call)
    (8, 2, 64, 4, 1000),            # head_dim 64
    (16, 1, 64, 7, 513),            # 128 grouped rows: the maximum
    (4, 4, 128, 2, 70),             # G = 1
    (64, 8, 128, 6, 2900),          # 56 grouped rows: keys-on-M with packed probabilities, two K slots
    (64, 8, 128, 7, 1333),          # 64 grouped rows: the most the keys-on-M kernel takes
])
def test_shapes_against_oracle(Hq, Hkv, D, gamma, L):
    """The library's own choice of kernel, and the rows-on-M kernel forced (it serves every shape)."""
    cfg = wl.VerifyConfig("t", B=2, Hq=Hq, Hkv=Hkv, D=D, gamma=gamma, V=4096, ctx_lens=(L, max(gamma + 1, L // 3)))
    q, k, v, ctx = wl.attention_inputs(cfg, seed=2, device="cuda", poison_padding=True)
    _compare(q, k, v, ctx, gamma)
    _compare(q, k, v, ctx, gamma, kernel=1)
    # without the log-sum-exp output (49 to 64 rows then run one softmax group with bf16 row sums)
    _compare(q, k, v, ctx, gamma, want_lse=False)


@pytest.mark.parametrize("Hq,Hkv,gamma,L,num_ctas", [
    (64, 8, 8, 1500, 0),            # 72 grouped rows: two softmax groups of 40 columns
    (64, 8, 9, 2900, 5),            # 80 rows: no padding column
    (64, 8, 10, 1333, 1),           # 88 rows: two groups of 48 columns
    (64, 8, 11, 4000, 148),         # 96 rows: the most the keys-on-M kernel takes
    (72, 8, 8, 3000, 3),            # G = 9
    (40, 4, 8, 5000, 37),           # G = 10, CTAs that span units
])
def test_keys_on_m_two_softmax_groups(Hq, Hkv, gamma, L, num_ctas):
    """65 to 96 grouped rows on the keys-on-M kernel (on request: the library's own choice there is rows on M)."""
    cfg = wl.VerifyConfig("t", B=2, Hq=Hq, Hkv=Hkv, D=128, gamma=gamma, V=4096, ctx_lens=(L, max(gamma + 1, L // 3)))
    q, k, v, ctx = wl.attention_inputs(cfg, seed=2, device="cuda", poison_padding=True)
    _, _, o32 = _compare(q, k, v, ctx, gamma, num_ctas=num_ctas, kernel=2)
    _, _, again, _ = _run(q, k, v, ctx, gamma, num_ctas=num_ctas, kernel=2)
    assert torch.equal(o32, again)                     # bit-identical from run to run
    # scores far above the first tile's: the references move, in either group
    k2 = k.clone()
    k2[:, :, L // 2:L // 2 + 10] *= 6.0
    k2[:, :, L - 40:L - 35] *= 9.0
    _compare(q, k2, v, ctx, gamma, num_ctas=num_ctas, kernel=2)


@pytest.mark.parametrize("kernel", [1, 2])
@pytest.mark.parametrize("num_ctas", [1, 2, 7, 148, 509])
def test_split_invariance(num_ctas, kernel):
    """Any split of the KV length gives the oracle's answer, and fp32 results agree across splits."""
    cfg = wl.VerifyConfig("t", B=3, Hq=32, Hkv=8, D=128, gamma=8, V=4096, ctx_lens=(4100, 9, 1111), Lmax=4200)
    q, k, v, ctx = wl.attention_inputs(cfg, seed=3, device="cuda", poison_padding=True)
    _, _, o32 = _compare(q, k, v, ctx, cfg.gamma, num_ctas=num_ctas, kernel=kernel)
    _, _, base, _ = _run(q, k, v, ctx, cfg.gamma, num_ctas=1, kernel=kernel)
    # splits differ only through where the bf16 rounding of the probabilities falls
    rel = (o32 - base).norm(dim=-1) / base.norm(dim=-1)
    assert rel.max().item() < 5e-3


def test_minimum_context_equals_rows():
    """L_b = R: row i sees exactly i+1 keys; row 0 returns the first value row."""
    cfg = wl.VerifyConfig("t", B=2, Hq=8, Hkv=2, D=128, gamma=5, V=4096, ctx_lens=(6, 6), Lmax=64)
    q, k, v, ctx = wl.attention_inputs(cfg, seed=4, device="cuda", poison_padding=True)
    _, out, o32 = _compare(q, k, v, ctx, cfg.gamma)
    for h in range(8):
        assert torch.equal(out[:, 0, h], v[:, h // 4, 0])


def test_peaked_scores_and_planted_key():
    cfg = wl.VerifyConfig("t", B=1, Hq=32, Hkv=8, D=128, gamma=8, V=4096, ctx_lens=(5000,), q_scale=4.0)
    q, k, v, ctx = wl.attention_inputs(cfg, seed=5, device="cuda")
    k[0, :, 1234] = (q[0, 0, ::4] * 0.5)           # a key aligned with row 0 of each group's first head
    _compare(q, k, v, ctx, cfg.gamma)


def test_explicit_scale_and_strided_cache():
    cfg = wl.VerifyConfig("t", B=2, Hq=8, Hkv=2, D=128, gamma=3, V=4096, ctx_lens=(900, 640), Lmax=1024)
    q, k, v, ctx = wl.attention_inputs(cfg, seed=6, device="cuda")
    # token-major storage [B, L, Hkv, D] viewed as [B, Hkv, L, D]: non-dense strides
    ks = k.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    vs = v.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    assert not ks.is_contiguous()
    out, lse, o32, status = _run(q, ks, vs, ctx, cfg.gamma, scale=0.05)
    ref, _ = _oracle(q, k, v, ctx, cfg.gamma, scale=0.05)
    parity.check_attention(o32.cpu().numpy(), ref)


@pytest.mark.parametrize("kernel", [1, 2])
def test_run_to_run_bit_identity(kernel):
    cfg = wl.VerifyConfig("t", B=2, Hq=32, Hkv=8, D=128, gamma=8, V=4096, ctx_lens=(6000, 3000))
    q, k, v, ctx = wl.attention_inputs(cfg, seed=7, device="cuda")
    a = _run(q, k, v, ctx, cfg.gamma, kernel=kernel)
    b = _run(q, k, v, ctx, cfg.gamma, kernel=kernel)
    assert torch.equal(a[0], b[0]) and torch.equal(a[2], b[2]) and torch.equal(a[1], b[1])


def test_bad_context_length_sets_status_and_stays_defined():
    cfg = wl.VerifyConfig("t", B=2, Hq=8, Hkv=2, D=64, gamma=2, V=4096, ctx_lens=(200, 100), Lmax=256)
    q, k, v, ctx = wl.attention_inputs(cfg, seed=8, device="cuda")
    bad = ctx.clone(); bad[1] = 100000
    out, _, _, status = _run(q, k, v, bad, cfg.gamma)
    assert status & 1
    assert torch.isfinite(out.float()).all()


def test_argument_errors():
    import paper_2502_20330_b200 as R
    cfg = wl.VerifyConfig("t", B=1, Hq=8, Hkv=2, D=64, gamma=2, V=4096, ctx_lens=(128,))
    q, k, v, ctx = wl.attention_inputs(cfg, seed=9, device="cuda")
    out = torch.empty_like(q)
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(R.RapidError) as e:
        R.rapid_verify_attention(q, k, v, ctx, 2, out, small)
    assert e.value.code == 3
    ws = R.new_workspace(R.attention_workspace_bytes(1, 8, 2, 64, 128, 2))
    with pytest.raises(R.RapidError) as e:
        R.rapid_verify_attention(q, k, v, ctx, 2, out, ws, R.AttnParams(num_ctas=100000))
    assert e.value.code == 1
    with pytest.raises(R.RapidError) as e:                                # head_dim 64 has no keys-on-M kernel
        R.rapid_verify_attention(q, k, v, ctx, 2, out, ws, R.AttnParams(kernel=2))
    assert e.value.code == 2
    with pytest.raises(R.RapidError) as e:
        R.rapid_verify_attention(q, k, v, ctx, 2, out, ws, R.AttnParams(kernel=7))
    assert e.value.code == 1
    assert R.attention_workspace_bytes(1, 8, 2, 96, 128, 2) == 0          # unsupported head_dim
    assert R.attention_workspace_bytes(1, 64, 1, 128, 128, 8) == 0        # 576 grouped rows


def _check_every_row(q, k, v, ctx, gamma, variants):
    """Every row of a full-size workload against the oracle (one oracle pass, several device runs)."""
    ref, ref_lse = _oracle(q, k, v, ctx, gamma)
    for kw in variants:
        out, lse, o32, status = _run(q, k, v, ctx, gamma, **kw)
        assert status == 0
        rep = parity.check_attention(out.float().cpu().numpy(), ref)
        parity.check_attention(o32.cpu().numpy(), ref)
        assert rep["rows"] == ref_lse.size
        assert np.abs(lse.cpu().numpy() - ref_lse).max() < LSE_TOL


def test_llama8b_32k_every_row():
    """The 32K workload in the bench's launch configuration (the library's choice there is one cluster
    per KV head), and the two kernels with a merge launch."""
    cfg = wl.CONFIGS["llama8b_32k"]
    q, k, v, ctx = wl.attention_inputs(cfg, seed=10, device="cuda")
    _check_every_row(q, k, v, ctx, cfg.gamma, [dict(), dict(kernel=2), dict(kernel=1), dict(kernel=3),
                                               dict(plan=2), dict(kernel=2, plan=1)])


def test_llama8b_128k_and_70b_every_row():
    for name in ("llama8b_128k", "llama70b_128k"):
        cfg = wl.CONFIGS[name]
        q, k, v, ctx = wl.attention_inputs(cfg, seed=11, device="cuda")
        if name == "llama8b_128k":
            variants = [dict(), dict(plan=2), dict(kernel=1), dict(kernel=3)]
        else:
            variants = [dict(), dict(plan=2), dict(kernel=2)]   # kernel 2: two softmax groups at full size
        _check_every_row(q, k, v, ctx, cfg.gamma, variants)
        del q, k, v


def test_ragged_qwen_batch_every_row():
    cfg = wl.CONFIGS["qwen7b_ragged"]
    q, k, v, ctx = wl.attention_inputs(cfg, seed=12, device="cuda", poison_padding=True)
    _check_every_row(q, k, v, ctx, cfg.gamma, [dict(), dict(plan=2), dict(kernel=1, plan=1)])


def test_drafter_8k_every_row():
    """The drafter-side one-row decode over the retrieved context (gamma = 0)."""
    cfg = wl.CONFIGS["drafter_8k"]
    q, k, v, ctx = wl.attention_inputs(cfg, seed=13, device="cuda")
    _check_every_row(q, k, v, ctx, cfg.gamma, [dict(), dict(kernel=2), dict(kernel=3, plan=2), dict(kernel=1)])


def test_random_shapes_and_lengths():
    """Seeded sweep over head layouts, draft counts, ragged lengths and splits: every combination of
    odd/even first tiles, single and paired tiles, short units and CTAs that straddle several units."""
    rng = np.random.default_rng(123)
    layouts = [(8, 2, 128), (4, 4, 64), (12, 2, 64), (16, 2, 128), (7, 7, 128), (32, 8, 128), (64, 8, 128)]
    for trial in range(14):
        Hq, Hkv, D = layouts[trial % len(layouts)]
        G = Hq // Hkv
        gamma = int(rng.integers(0, max(1, min(9, 128 // G))))
        B = int(rng.integers(1, 5))
        Lmax = int(rng.integers(gamma + 1, 1500))
        lens = tuple(int(rng.integers(gamma + 1, Lmax + 1)) for _ in range(B))
        cfg = wl.VerifyConfig("fz", B=B, Hq=Hq, Hkv=Hkv, D=D, gamma=gamma, V=4096, ctx_lens=lens, Lmax=Lmax)
        q, k, v, ctx = wl.attention_inputs(cfg, seed=200 + trial, device="cuda", poison_padding=True)
        num_ctas = int(rng.choice([0, 1, 3, 5, 16, 37, 148, 300]))
        _compare(q, k, v, ctx, gamma, num_ctas=num_ctas)
        if D == 128 and G * (gamma + 1) <= 64:      # the automatic choice was keys-on-M: rows-on-M too
            _compare(q, k, v, ctx, gamma, num_ctas=num_ctas, kernel=1)


def test_keys_on_m_random_sweep():
    """Seeded sweep of the keys-on-M kernel over 1 to 96 grouped rows (every column count, one and two
    softmax groups, numbers of rows that are no multiple of 8), ragged batches with poisoned padding,
    splits from 1 to 512 CTAs, and, in a third of the cases, a few keys whose scores sit far above the
    rest, so that the softmax references move in the middle of a unit."""
    rng = np.random.default_rng(7)
    layouts = [(8, 2), (16, 2), (7, 7), (32, 8), (64, 8), (28, 4), (40, 4), (72, 8), (12, 12), (96, 8), (5, 1), (48, 8)]
    for trial in range(150):
        Hq, Hkv = layouts[int(rng.integers(len(layouts)))]
        G = Hq // Hkv
        gamma = int(rng.integers(0, min(11, 96 // G - 1) + 1))
        B = int(rng.integers(1, 4))
        Lmax = int(rng.integers(gamma + 1, 2600))
        lens = tuple(int(rng.integers(gamma + 1, Lmax + 1)) for _ in range(B))
        cfg = wl.VerifyConfig("sweep", B=B, Hq=Hq, Hkv=Hkv, D=128, gamma=gamma, V=4096, ctx_lens=lens, Lmax=Lmax)
        q, k, v, ctx = wl.attention_inputs(cfg, seed=1000 + trial, device="cuda", poison_padding=True)
        if rng.random() < 0.3:
            j = int(rng.integers(0, max(1, min(lens) - 1)))
            k[:, :, j:j + 3] *= float(rng.choice([4.0, 8.0]))
        num_ctas = int(rng.choice([0, 1, 2, 3, 5, 16, 37, 148, 300, 512]))
        _compare(q, k, v, ctx, gamma, num_ctas=num_ctas, kernel=2)


@pytest.mark.parametrize("B,Hq,Hkv,D,gamma,lo,hi,num_ctas", [
    (40, 16, 4, 128, 3, 600, 3000, 0),      # 160 short units: every CTA walks through several of them
    (24, 8, 8, 64, 1, 64, 900, 0),          # 192 units of 1..15 tiles, head_dim 64
    (3, 32, 8, 128, 8, 5000, 9000, 37),     # a caller-chosen split, a few dozen tiles per CTA
    (2, 8, 2, 128, 4, 9400, 9500, 0),       # tiles just above four per CTA: the padded split switches on
    (2, 8, 2, 128, 4, 9200, 9300, 0),       # ... and just below: the plain equal split
])
def test_many_units_per_cta(B, Hq, Hkv, D, gamma, lo, hi, num_ctas):
    """The work split charges every unit a few virtual tiles; ranges that begin or end inside that
    padding, hold several whole units, or hold nothing but padding must still cover every real tile
    exactly once and the merge must find every partial."""
    cfg = wl.VerifyConfig("mu", B=B, Hq=Hq, Hkv=Hkv, D=D, gamma=gamma, V=4096, ctx_range=(lo, hi), Lmax=hi)
    q, k, v, ctx = wl.attention_inputs(cfg, seed=300 + B, device="cuda", poison_padding=True)
    rng = np.random.default_rng(B)
    units = rng.choice(B * Hq * (gamma + 1), size=min(96, B * Hq * (gamma + 1)), replace=False).astype(np.int64)
    _compare(q, k, v, ctx, gamma, num_ctas=num_ctas, units=units)


# ---- one cluster per (sequence, KV head), merged on chip ----------------------------------------------------

def test_cluster_merge_random_sweep():
    """Seeded sweep of the cluster variant: every column count up to 96 rows, ragged batches with poisoned
    padding (units whose cluster has more CTAs than tiles), lengths below one tile, planted large scores.
    A shape whose clusters do not fit on the device together must be refused, not run."""
    import paper_2502_20330_b200 as R
    rng = np.random.default_rng(11)
    layouts = [(8, 2), (16, 2), (32, 8), (64, 8), (28, 4), (72, 8), (12, 12), (96, 8), (5, 1), (48, 8)]
    ran = 0
    for trial in range(70):
        Hq, Hkv = layouts[int(rng.integers(len(layouts)))]
        G = Hq // Hkv
        gamma = int(rng.integers(0, min(11, 96 // G - 1) + 1))
        B = int(rng.integers(1, 4))
        Lmax = int(rng.integers(gamma + 1, 6000))
        lens = tuple(int(rng.integers(gamma + 1, Lmax + 1)) for _ in range(B))
        cfg = wl.VerifyConfig("cl", B=B, Hq=Hq, Hkv=Hkv, D=128, gamma=gamma, V=4096, ctx_lens=lens, Lmax=Lmax)
        q, k, v, ctx = wl.attention_inputs(cfg, seed=3000 + trial, device="cuda", poison_padding=True)
        if rng.random() < 0.3:
            j = int(rng.integers(0, max(1, min(lens) - 1)))
            k[:, :, j:j + 3] *= float(rng.choice([4.0, 8.0]))
        try:
            _, _, o32 = _compare(q, k, v, ctx, gamma, kernel=3)
        except R.RapidError as e:
            assert e.code == 2 and "fit" in str(e)
            continue
        ran += 1
        if trial % 7 == 0:
            _, _, again, _ = _run(q, k, v, ctx, gamma, kernel=3)
            assert torch.equal(o32, again)             # bit-identical from run to run
            _compare(q, k, v, ctx, gamma, kernel=3, plan=1)
    assert ran >= 40


def test_cluster_merge_paged_and_no_lse():
    import paper_2502_20330_b200 as R
    cfg = wl.VerifyConfig("clp", B=1, Hq=32, Hkv=8, D=128, gamma=8, V=4096, ctx_lens=(5000,), Lmax=5120)
    q, k, v, ctx = wl.attention_inputs(cfg, seed=71, device="cuda", poison_padding=True)
    ref, _ = _oracle(q, k, v, ctx, cfg.gamma)
    for bs in (64, 256):
        kp, vp, table = wl.paged_layout(k, v, ctx.cpu(), bs, seed=5)
        ws = R.new_workspace(R.attention_workspace_bytes(1, 32, 8, 128, table.shape[1] * bs, cfg.gamma))
        out = torch.empty_like(q)
        R.rapid_verify_attention_paged(q, kp, vp, table, ctx, cfg.gamma, out, ws, R.AttnParams(kernel=3))
        torch.cuda.synchronize()
        assert R.workspace_status(ws) == 0
        parity.check_attention(out.float().cpu().numpy(), ref)


# ---- plans -------------------------------------------------------------------------------------------------

@pytest.mark.parametrize("kernel", [0, 1, 2])
@pytest.mark.parametrize("plan", [1, 2])
def test_planned_calls_match_unplanned_bit_for_bit(kernel, plan):
    cfg = wl.VerifyConfig("pl", B=3, Hq=32, Hkv=8, D=128, gamma=8, V=4096, ctx_lens=(4100, 9, 1111), Lmax=4200)
    q, k, v, ctx = wl.attention_inputs(cfg, seed=41, device="cuda", poison_padding=True)
    for num_ctas in (0, 5, 300):
        a = _run(q, k, v, ctx, cfg.gamma, num_ctas=num_ctas, kernel=kernel)
        b = _run(q, k, v, ctx, cfg.gamma, num_ctas=num_ctas, kernel=kernel, plan=plan)
        assert a[3] == 0 and b[3] == 0
        assert torch.equal(a[2], b[2]) and torch.equal(a[1], b[1])


def test_one_plan_serves_many_layers_and_a_stale_plan_is_flagged():
    import paper_2502_20330_b200 as R
    cfg = wl.VerifyConfig("pl", B=2, Hq=32, Hkv=8, D=128, gamma=8, V=4096, ctx_lens=(9000, 5000))
    B, Hq, Hkv, D, gamma = cfg.B, cfg.Hq, cfg.Hkv, cfg.D, cfg.gamma
    layers = [wl.attention_inputs(cfg, seed=50, device="cuda", layer=i) for i in range(3)]
    ctx = layers[0][3]
    ws = R.new_workspace(R.attention_workspace_bytes(B, Hq, Hkv, D, 9000, gamma))
    R.rapid_attention_plan(ctx, gamma, B, Hq, Hkv, D, 9000, ws)
    outs = []
    for i, (q, k, v, _) in enumerate(layers):
        out = torch.empty_like(q)
        R.rapid_verify_attention(q, k, v, ctx, gamma, out, ws, R.AttnParams(plan=1 if i == 0 else 2))
        outs.append(out)
    torch.cuda.synchronize()
    assert R.workspace_status(ws) == 0
    for (q, k, v, _), out in zip(layers, outs):
        ref, _ = _oracle(q, k, v, ctx, gamma)
        parity.check_attention(out.float().cpu().numpy(), ref)
    # the lengths move on (a step was committed) but the caller forgets to plan again
    ctx2 = ctx.clone(); ctx2[1] -= 3
    q, k, v, _ = layers[0]
    R.rapid_verify_attention(q, k, v, ctx2, gamma, torch.empty_like(q), ws, R.AttnParams(plan=2))
    torch.cuda.synchronize()
    assert R.workspace_status(ws) & R.STATUS_STALE_PLAN
    # ... and a plan made for another split
    R.workspace_init(ws)
    R.rapid_attention_plan(ctx, gamma, B, Hq, Hkv, D, 9000, ws, R.AttnParams(num_ctas=64))
    R.rapid_verify_attention(q, k, v, ctx, gamma, torch.empty_like(q), ws, R.AttnParams(plan=1))
    torch.cuda.synchronize()
    assert R.workspace_status(ws) & R.STATUS_STALE_PLAN


# ---- sink + window visibility ------------------------------------------------------------------------------

@pytest.mark.parametrize("Hq,Hkv,D,gamma,lens,sink,window", [
    (32, 8, 128, 8, (20000, 700), 4, 4092),        # the streaming drafter's budget over a long cache
    (32, 8, 128, 8, (5000, 4100), 4, 1000),
    (32, 8, 128, 8, (3000, 300), 0, 257),          # no sinks; the second sequence lies inside the window
    (64, 8, 128, 8, (6000, 2000), 130, 500),       # 72 rows (rows on M); sinks spill into a second tile
    (28, 4, 128, 4, (9000, 5), 7, 1),              # a window of one key: each row sees the sinks and itself
    (8, 2, 64, 4, (4096, 1000), 4, 600),           # head_dim 64
    (64, 8, 128, 6, (7000, 1500), 64, 128),        # 56 rows; sink and window on tile boundaries
])
def test_sink_and_window_mask(Hq, Hkv, D, gamma, lens, sink, window):
    cfg = wl.VerifyConfig("sw", B=len(lens), Hq=Hq, Hkv=Hkv, D=D, gamma=gamma, V=4096, ctx_lens=lens)
    q, k, v, ctx = wl.attention_inputs(cfg, seed=60, device="cuda", poison_padding=True)
    # Keys no row sees: their K may hold anything (a hidden score is never used), and so may the V of
    # the 128-key tiles that lie wholly in the hidden middle (those tiles are not read at all).  The V
    # rows of hidden keys that share a tile with visible ones are cache content like any other: finite.
    for b, L in enumerate(lens):
        lo, hi = sink, L - (gamma + 1) - window + 1
        if hi > lo:
            k[b, :, lo:hi] = float("nan")
            tlo, thi = (lo + 127) // 128 * 128, hi // 128 * 128
            if thi > tlo:
                v[b, :, tlo:thi] = float("nan")
    kernels = [0, 1] + ([2] if D == 128 and Hq // Hkv * (gamma + 1) <= 96 else [])
    for kernel in kernels:
        for num_ctas in (0, 3):
            _compare(q, k, v, ctx, gamma, num_ctas=num_ctas, kernel=kernel, sink=sink, window=window)
    _compare(q, k, v, ctx, gamma, sink=sink, window=window, plan=1)
    if D == 128 and Hq // Hkv * (gamma + 1) <= 96:
        _compare(q, k, v, ctx, gamma, kernel=3, sink=sink, window=window)


def test_window_over_a_128k_cache_reads_only_what_is_visible():
    """4 sinks + 4,092 recent keys over a 128K cache: parity on every row with the hidden keys poisoned."""
    cfg = wl.CONFIGS["llama8b_128k"]
    q, k, v, ctx = wl.attention_inputs(cfg, seed=61, device="cuda")
    L, R = 131072, cfg.R
    hi = L - R - 4092 + 1                      # the oldest key of row 0's window
    k[:, :, 4:hi] = float("nan"); v[:, :, 128:hi // 128 * 128] = float("nan")   # V: the tiles never read
    ref, ref_lse = _oracle(q, k, v, ctx, cfg.gamma, sink=4, window=4092)
    for kw in (dict(), dict(kernel=1), dict(kernel=3)):
        out, lse, o32, status = _run(q, k, v, ctx, cfg.gamma, sink=4, window=4092, **kw)
        assert status == 0
        parity.check_attention(out.float().cpu().numpy(), ref)
        assert np.abs(lse.cpu().numpy() - ref_lse).max() < LSE_TOL


def test_window_argument_errors():
    import paper_2502_20330_b200 as R
    cfg = wl.VerifyConfig("t", B=1, Hq=8, Hkv=2, D=128, gamma=2, V=4096, ctx_lens=(128,))
    q, k, v, ctx = wl.attention_inputs(cfg, seed=9, device="cuda")
    ws = R.new_workspace(R.attention_workspace_bytes(1, 8, 2, 128, 128, 2))
    for bad in (dict(sink_keys=4), dict(window_keys=-1), dict(sink_keys=-1, window_keys=5),
                dict(window_keys=5, all_keys_visible=True), dict(plan=7)):
        with pytest.raises(R.RapidError) as e:
            R.rapid_verify_attention(q, k, v, ctx, 2, torch.empty_like(q), ws, R.AttnParams(**bad))
        assert e.value.code == 1


@pytest.mark.parametrize("Hq,Hkv,gamma,lens,kernel,sink,window", [
    (32, 8, 8, (9000, 517), 0, 0, 0),       # keys on M; the short sequence has old tiles for few CTAs only
    (32, 8, 0, (8192,), 0, 0, 0),           # the drafter's one-row decode
    (32, 8, 8, (40000,), 3, 0, 0),          # one cluster per KV head
    (32, 8, 8, (30000, 4100), 0, 4, 1020),  # window variant: the early tiles are the sink tile and the window's
    (64, 8, 8, (5000, 300), 0, 0, 0),       # rows on M: the flag changes nothing there
])
def test_early_copies_of_the_settled_cache_change_nothing(Hq, Hkv, gamma, lens, kernel, sink, window):
    """kv_settled: two layers back to back on one stream, each layer's newest rows written by the kernels just
    ahead of its call (the older keys long before).  The second layer's first tiles are then copied while the
    first layer's merge still runs; results must equal the oracle and, bit for bit, the calls without the flag."""
    import paper_2502_20330_b200 as R
    cfg = wl.VerifyConfig("e", B=len(lens), Hq=Hq, Hkv=Hkv, D=128, gamma=gamma, V=4096, ctx_lens=lens)
    Rr = cfg.R
    layers = [wl.attention_inputs(cfg, seed=60 + i, device="cuda") for i in range(2)]
    ctx = layers[0][3]
    Lmax = layers[0][1].shape[2]
    news, caches = [], []
    for q, k, v, _ in layers:                       # take the newest rows out of the caches, poison their place
        kn = torch.stack([k[b, :, L - Rr:L].clone() for b, L in enumerate(lens)])
        vn = torch.stack([v[b, :, L - Rr:L].clone() for b, L in enumerate(lens)])
        kc, vc = k.clone(), v.clone()
        for b, L in enumerate(lens):
            kc[b, :, L - Rr:L] = float("nan")
            vc[b, :, L - Rr:L] = float("nan")
        news.append((kn, vn))
        caches.append((kc, vc))
    ws = R.new_workspace(R.attention_workspace_bytes(cfg.B, Hq, Hkv, 128, Lmax, gamma))
    outs = [torch.zeros_like(layers[0][0]) for _ in range(2)]
    o32s = [torch.zeros(cfg.B, Rr, Hq, 128, device="cuda") for _ in range(2)]
    torch.cuda.synchronize()

    def run(flag):
        base = R.AttnParams(kernel=kernel, sink_keys=sink, window_keys=window)
        R.rapid_attention_plan(ctx, gamma, cfg.B, Hq, Hkv, 128, Lmax, ws, base)
        for i, ((q, _, _, _), (kc, vc), (kn, vn)) in enumerate(zip(layers, caches, news)):
            for b, L in enumerate(lens):            # the layer's newest rows arrive right before its call
                kc[b, :, L - Rr:L] = kn[b]
                vc[b, :, L - Rr:L] = vn[b]
            R.rapid_verify_attention(q, kc, vc, ctx, gamma, outs[i], ws,
                                     R.AttnParams(kernel=kernel, sink_keys=sink, window_keys=window,
                                                  plan=R.PLAN_SETTLED, kv_settled=flag, out_f32=o32s[i]))
        torch.cuda.synchronize()
        assert R.workspace_status(ws) == 0
        return [o.clone() for o in o32s]

    plain = run(False)
    for (kc, vc) in caches:                         # poison the newest rows again for the second pass
        for b, L in enumerate(lens):
            kc[b, :, L - Rr:L] = float("nan")
            vc[b, :, L - Rr:L] = float("nan")
    torch.cuda.synchronize()
    early = run(True)
    for i, (q, k, v, _) in enumerate(layers):
        ref, ref_lse = _oracle(q, k, v, ctx, gamma, sink=sink, window=window)
        parity.check_attention(early[i].cpu().numpy(), ref, ~np.isnan(ref_lse))
        assert torch.equal(early[i], plain[i])


def test_describe_names_the_kernels_the_workloads_get():
    """rapid_attention_describe against the library's documented choices for the named workloads."""
    import paper_2502_20330_b200 as R
    want = {"llama8b_128k": (2, 2, 48), "llama8b_32k": (2, 2, 48), "llama70b_128k": (2, 2, 80),
            "qwen7b_ragged": (2, 1, 48), "drafter_8k": (2, 1, 16), "tiny": (1, 2, 64)}
    for name, (kernel, groups, cols) in want.items():
        cfg = wl.CONFIGS[name]
        Lmax = cfg.Lmax or max(cfg.ctx_lens)
        d = R.rapid_attention_describe(cfg.B, cfg.Hq, cfg.Hkv, cfg.D, Lmax, cfg.gamma)
        assert (d["kernel"], d["softmax_groups"], d["columns"]) == (kernel, groups, cols), (name, d)
        assert d["kernels_per_call"] == 2 and d["ctas"] > 0
    d = R.rapid_attention_describe(1, 64, 8, 128, 131072, 10)          # 88 grouped rows: rows on M
    assert d["kernel"] == 1
    d = R.rapid_attention_describe(1, 32, 8, 128, 8192, 0, R.AttnParams(kernel=R.ATTN_KERNEL_CLUSTER_MERGE))
    assert d["kernel"] == 3 and d["kernels_per_call"] == 1 and d["cluster_size"] >= 2
    d = R.rapid_attention_describe(1, 32, 8, 128, 131072, 8, R.AttnParams(kv_fp8=True))
    assert d["kernel"] == 2
