"""Drafter-side fused sampling (x' ~ softmax(d/T), log q(x'), row statistics) against the oracle."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle
import workloads as wl

TIE_EPS = 1e-5


def _run(d, u, T):
    import paper_2502_20330_b200 as R
    B, V = d.shape
    ws = R.new_workspace(R.accept_workspace_bytes(B, 0, V))
    tok = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    logq = torch.zeros(B, dtype=torch.float32, device="cuda")
    stats = torch.zeros(B, 2, dtype=torch.float32, device="cuda")
    R.rapid_draft_sample(d, u, T, tok, logq, ws, out_row_stats=stats)
    torch.cuda.synchronize()
    assert R.workspace_status(ws) == 0
    return tok.cpu().numpy(), logq.cpu().numpy(), stats.cpu().numpy()


@pytest.mark.parametrize("B,V,T,sigma", [(1, 128256, 1.0, 2.0), (8, 152064, 0.7, 2.0), (33, 4096, 0.1, 1.0),
                                         (4, 196608, 1.0, 3.0), (16, 8196, 2.0, 2.0)])
def test_draft_sample_against_oracle(B, V, T, sigma):
    g = torch.Generator(device="cuda").manual_seed(41)
    d = torch.randn(B, V, generator=g, device="cuda") * sigma
    u = torch.rand(B, generator=g, device="cuda")
    tok, logq, stats = _run(d, u, T)
    dn, un = d.cpu().numpy(), u.cpu().numpy()
    ref_tok, ref_logq, ref_stats = oracle.draft_sample(dn, un, T)
    np.testing.assert_allclose(stats, ref_stats, rtol=0, atol=2e-4 * max(1.0, 1.0 / T))
    for b in range(B):
        x = dn[b].astype(np.float64) / T
        p = np.exp(x - ref_stats[b, 1])
        c = np.cumsum(p)
        t = int(tok[b])
        assert 0 <= t < V
        lo, hi = (c[t] - p[t]) / c[-1], c[t] / c[-1]
        assert lo - TIE_EPS <= float(un[b]) <= hi + TIE_EPS, f"row {b}: token {t} (oracle {ref_tok[b]})"
        assert abs(float(logq[b]) - float(np.log(p[t]))) < 1e-3
    assert (tok == ref_tok).mean() > 0.9


def test_draft_sample_strided_rows_and_reuse():
    """Rows taken from a wider buffer; two calls on one workspace give the same answer (the kernel's
    bookkeeping in the workspace header returns to its initial state)."""
    import paper_2502_20330_b200 as R
    g = torch.Generator(device="cuda").manual_seed(42)
    wide = torch.randn(6, 8192 + 64, generator=g, device="cuda") * 2
    d = wide[:, :8192]
    u = torch.rand(6, generator=g, device="cuda")
    ws = R.new_workspace(R.accept_workspace_bytes(6, 0, 8192))
    outs = []
    for _ in range(2):
        tok = torch.zeros(6, dtype=torch.int32, device="cuda")
        logq = torch.zeros(6, device="cuda")
        R.rapid_draft_sample(d, u, 1.0, tok, logq, ws)
        torch.cuda.synchronize()
        outs.append((tok.clone(), logq.clone()))
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
    ref_tok, _, _ = oracle.draft_sample(d.cpu().numpy(), u.cpu().numpy(), 1.0)
    assert (outs[0][0].cpu().numpy() == ref_tok).all()
