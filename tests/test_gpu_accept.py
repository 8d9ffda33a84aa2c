"""Parity of the CUDA accept/residual step with the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle
from oracle import parity
import workloads as wl


def _run(z, d, tok, u, eta, T=1.0, alpha=0.1, mode=0):
    import paper_2502_20330_b200 as R
    B, Rr, V = z.shape
    gamma = Rr - 1
    ws = R.new_workspace(R.accept_workspace_bytes(B, gamma, V))
    alen = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    ntok = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    ratios = torch.zeros(B, max(gamma, 1), dtype=torch.float32, device="cuda")
    R.rapid_accept(z, d, tok, u, eta, alen, ntok, ws,
                   R.AcceptParams(temperature=T, tail_alpha=alpha, residual_mode=mode, ratio_out=ratios))
    torch.cuda.synchronize()
    return alen.cpu().numpy(), ntok.cpu().numpy(), ratios.cpu().numpy()[:, :gamma], R.workspace_status(ws)


def _check(z, d, tok, u, eta, T=1.0, alpha=0.1, mode=0):
    alen, ntok, ratios, status = _run(z, d, tok, u, eta, T, alpha, mode)
    assert status == 0
    rep = parity.check_accept(z.cpu().numpy(), d.cpu().numpy(), tok.cpu().numpy(), u.cpu().numpy(), eta, T, alpha,
                              mode, alen, ntok, ratios)
    return rep, alen, ntok


def test_tiny_config():
    cfg = wl.CONFIGS["tiny"]
    z, d, tok, u = wl.accept_inputs(cfg, seed=1, device="cuda")
    _check(z, d, tok, u, cfg.eta)


@pytest.mark.parametrize("eta", [0.0, 0.5, 5.0, 20.0, 50.0])
@pytest.mark.parametrize("T", [1.0, 0.1])
@pytest.mark.parametrize("mode", [0, 1])
def test_parameter_grid(eta, T, mode):
    cfg = wl.VerifyConfig("t", B=16, Hq=8, Hkv=2, D=64, gamma=5, V=8196, ctx_lens=(64,) * 16, target_sigma=1.0,
                          temperature=T)
    z, d, tok, u = wl.accept_inputs(cfg, seed=int(eta * 10) + mode, device="cuda")
    rep, alen, _ = _check(z, d, tok, u, eta, T=T, alpha=0.1, mode=mode)
    assert len(rep["near_ties"]) <= 1


def test_tail_rule_off_and_on_differ_only_through_the_rule():
    cfg = wl.VerifyConfig("t", B=32, Hq=8, Hkv=2, D=64, gamma=4, V=4096, ctx_lens=(64,) * 32, target_sigma=1.0)
    z, d, tok, u = wl.accept_inputs(cfg, seed=3, device="cuda")
    for alpha in (0.0, 0.1, 0.5):
        _check(z, d, tok, u, 20.0, alpha=alpha)


def test_both_branches_and_every_stop_position_are_exercised():
    cfg = wl.VerifyConfig("t", B=64, Hq=8, Hkv=2, D=64, gamma=4, V=4096, ctx_lens=(64,) * 64, target_sigma=1.0)
    z, d, tok, u = wl.accept_inputs(cfg, seed=4, device="cuda")
    rep, alen, _ = _check(z, d, tok, u, 0.5)
    assert set(alen.tolist()) == set(range(cfg.gamma + 1))


def test_identical_logits_accept_everything():
    cfg = wl.VerifyConfig("t", B=8, Hq=8, Hkv=2, D=64, gamma=6, V=4096, ctx_lens=(64,) * 8)
    z, d, tok, u = wl.accept_inputs(cfg, seed=5, device="cuda")
    z[:, :cfg.gamma] = d
    u[:, :cfg.gamma] = 0.999
    rep, alen, _ = _check(z, d, tok, u, 20.0)
    assert (alen == cfg.gamma).all()


def test_eta_zero_matches_textbook_rule_on_device():
    cfg = wl.VerifyConfig("t", B=32, Hq=8, Hkv=2, D=64, gamma=4, V=4096, ctx_lens=(64,) * 32, target_sigma=1.0)
    z, d, tok, u = wl.accept_inputs(cfg, seed=6, device="cuda")
    a0, t0, r0, _ = _run(z, d, tok, u, 0.0, mode=0)
    a1, t1, r1, _ = _run(z, d, tok, u, 0.0, mode=1)
    np.testing.assert_array_equal(a0, a1)          # at eta = 0 both residual modes coincide
    np.testing.assert_array_equal(t0, t1)
    p = torch.softmax(z[:, :4].double(), -1); q = torch.softmax(d.double(), -1)
    ref = (p.gather(-1, tok.long()[..., None]) / q.gather(-1, tok.long()[..., None]))[..., 0].cpu().numpy()
    np.testing.assert_allclose(r0, ref, rtol=2e-4)


def test_adversarial_uniforms_at_the_ratio():
    """u placed a hair below / above the oracle's ratio: decisions still agree outside the 1e-5 band."""
    cfg = wl.VerifyConfig("t", B=16, Hq=8, Hkv=2, D=64, gamma=3, V=4096, ctx_lens=(64,) * 16, target_sigma=1.0)
    z, d, tok, u = wl.accept_inputs(cfg, seed=7, device="cuda")
    ref = oracle.accept(z.cpu().numpy(), d.cpu().numpy(), tok.cpu().numpy(), u.cpu().numpy(), eta=5.0)
    ratios = np.minimum(ref["ratios"], 1.0)
    for delta in (-3e-5, -1e-7, 1e-7, 3e-5):
        uu = u.clone()
        uu[:, :3] = torch.tensor(np.clip(ratios + delta, 0, 0.99999), dtype=torch.float32, device="cuda")
        rep, alen, _ = _check(z, d, tok, uu, 5.0)
        if abs(delta) > 1e-5:
            assert rep["near_ties"] == []


def test_gamma_zero_is_a_plain_sample_from_the_target():
    cfg = wl.VerifyConfig("t", B=4, Hq=8, Hkv=2, D=64, gamma=0, V=4096, ctx_lens=(64,) * 4)
    z, d, tok, u = wl.accept_inputs(cfg, seed=8, device="cuda")
    rep, alen, ntok = _check(z, d, tok, u, 3.0)
    assert (alen == 0).all()


def test_minus_infinity_logits_carry_no_mass():
    cfg = wl.VerifyConfig("t", B=4, Hq=8, Hkv=2, D=64, gamma=3, V=4096, ctx_lens=(64,) * 4, target_sigma=1.0)
    z, d, tok, u = wl.accept_inputs(cfg, seed=9, device="cuda")
    mask = torch.rand(4096, device="cuda") < 0.3
    mask[tok.long().flatten()] = False
    z[:, :, mask] = float("-inf"); d[:, :, mask] = float("-inf")
    rep, alen, ntok = _check(z, d, tok, u, 5.0)
    assert not mask[torch.tensor(ntok).long()].any()


def test_bad_draft_token_sets_status():
    cfg = wl.VerifyConfig("t", B=2, Hq=8, Hkv=2, D=64, gamma=2, V=4096, ctx_lens=(64,) * 2)
    z, d, tok, u = wl.accept_inputs(cfg, seed=10, device="cuda")
    tok[1, 0] = 999999
    alen, ntok, _, status = _run(z, d, tok, u, 0.5)
    assert status & 2
    assert ((ntok >= 0) & (ntok < 4096)).all() and ((alen >= 0) & (alen <= 2)).all()


def test_run_to_run_bit_identity_and_strided_rows():
    cfg = wl.VerifyConfig("t", B=4, Hq=8, Hkv=2, D=64, gamma=3, V=4096, ctx_lens=(64,) * 4, target_sigma=1.0)
    z, d, tok, u = wl.accept_inputs(cfg, seed=11, device="cuda")
    a = _run(z, d, tok, u, 5.0)
    b = _run(z, d, tok, u, 5.0)
    for x, y in zip(a[:3], b[:3]):
        np.testing.assert_array_equal(x, y)
    zp = torch.zeros(4, 4, 4096 + 64, device="cuda"); zp[..., :4096] = z
    dp = torch.zeros(4, 3, 4096 + 64, device="cuda"); dp[..., :4096] = d
    c = _run(zp[..., :4096], dp[..., :4096], tok, u, 5.0)
    for x, y in zip(a[:3], c[:3]):
        np.testing.assert_array_equal(x, y)


def test_argument_errors():
    import paper_2502_20330_b200 as R
    cfg = wl.VerifyConfig("t", B=1, Hq=8, Hkv=2, D=64, gamma=2, V=4096, ctx_lens=(64,))
    z, d, tok, u = wl.accept_inputs(cfg, seed=12, device="cuda")
    ws = R.new_workspace(R.accept_workspace_bytes(1, 2, 4096))
    o = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(R.RapidError) as e:
        R.rapid_accept(z, d, tok, u, 0.5, o, o.clone(), ws, R.AcceptParams(temperature=0.0))
    assert e.value.code == 1
    with pytest.raises(R.RapidError) as e:
        R.rapid_accept(z[..., :4094], d[..., :4094], tok, u, 0.5, o, o.clone(), ws)
    assert e.value.code == 2


@pytest.mark.parametrize("name", ["llama8b_32k", "qwen7b_ragged"])
def test_full_vocabulary_workloads(name):
    cfg = wl.CONFIGS[name]
    z, d, tok, u = wl.accept_inputs(cfg, seed=13, device="cuda")
    _check(z, d, tok, u, cfg.eta)
    _check(z, d, tok, u, 20.0, T=0.1)


@pytest.mark.parametrize("T", [1.0, 0.5])
def test_drafter_statistics_handed_to_the_accept_step(T):
    """Algorithm 1's drafting loop draws x'_j from q_j; rapid_draft_sample returns log q_j(x'_j) and the
    row's (max, log-sum-exp) from that pass.  Handed to the accept step they replace its own reductions
    over the draft rows: same accepted lengths, same tokens, ratios equal to rounding."""
    import paper_2502_20330_b200 as R
    cfg = wl.VerifyConfig("t", B=6, Hq=8, Hkv=2, D=64, gamma=5, V=32000, ctx_lens=(64,) * 6, target_sigma=1.0,
                          temperature=T)
    z, d, _, u = wl.accept_inputs(cfg, seed=14, device="cuda")
    B, gamma, V = cfg.B, cfg.gamma, cfg.V
    rows = d.reshape(B * gamma, V)
    g = torch.Generator(device="cuda").manual_seed(15)
    du = torch.rand(B * gamma, generator=g, device="cuda")
    tok = torch.zeros(B * gamma, dtype=torch.int32, device="cuda")
    logq = torch.zeros(B * gamma, device="cuda")
    stats = torch.zeros(B * gamma, 2, device="cuda")
    ws0 = R.new_workspace(R.accept_workspace_bytes(B * gamma, 0, V))
    R.rapid_draft_sample(rows, du, T, tok, logq, ws0, out_row_stats=stats)
    tok = tok.reshape(B, gamma)
    outs = []
    for params in (R.AcceptParams(temperature=T), R.AcceptParams(temperature=T, draft_row_stats=stats, draft_logq=logq),
                   R.AcceptParams(temperature=T, draft_row_stats=stats), R.AcceptParams(temperature=T, draft_logq=logq)):
        ws = R.new_workspace(R.accept_workspace_bytes(B, gamma, V))
        alen = torch.zeros(B, dtype=torch.int32, device="cuda"); ntok = torch.zeros_like(alen)
        params.ratio_out = torch.zeros(B, gamma, device="cuda")
        R.rapid_accept(z, d, tok, u, 5.0, alen, ntok, ws, params)
        torch.cuda.synchronize()
        assert R.workspace_status(ws) == 0
        outs.append((alen.cpu().numpy(), ntok.cpu().numpy(), params.ratio_out.cpu().numpy()))
        parity.check_accept(z.cpu().numpy(), d.cpu().numpy(), tok.cpu().numpy(), u.cpu().numpy(), 5.0, T, 0.1, 0,
                            outs[-1][0], outs[-1][1], outs[-1][2])
    for o in outs[1:]:
        np.testing.assert_array_equal(o[0], outs[0][0])
        np.testing.assert_array_equal(o[1], outs[0][1])
        np.testing.assert_allclose(o[2], outs[0][2], rtol=2e-5)
