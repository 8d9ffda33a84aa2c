"""Comparison rules between a device result and the oracle -- TEST INFRASTRUCTURE ONLY.

Attention: max-abs <= 2e-2 (bf16 K/V, fp32 accumulation) AND per-row relative L2
error <= 1e-2 (flat softmax outputs at 128K are ~5e-3 in size, so an absolute bound
alone would accept an all-zero output).

Accept: accepted lengths must be equal, except where the acceptance draw lies within
1e-5 of the oracle's ratio (reported as a near tie).  The sampled token must be
consistent with the oracle's fp64 CDF: its weight is positive and the sampling uniform
lies within 1e-5 of its CDF interval (several tokens are correct when u*W falls within
rounding of a boundary).
"""
from __future__ import annotations

import numpy as np

from . import RESIDUAL_PAPER, accept as oracle_accept, rapid_distributions, residual_weights

ATTN_MAX_ABS = 2e-2
ATTN_ROW_REL_L2 = 1e-2
TIE_EPS = 1e-5


def check_attention(out_dev, out_ref, rows=None):
    """out_dev, out_ref: [B,R,Hq,D] arrays (device result as float64, oracle float64).
    rows: optional boolean mask [B,R,Hq] of rows the oracle computed.  Returns a report dict; raises on failure."""
    out_dev = np.asarray(out_dev, dtype=np.float64)
    out_ref = np.asarray(out_ref, dtype=np.float64)
    if rows is None:
        rows = np.ones(out_ref.shape[:3], dtype=bool)
    a = out_dev[rows]
    b = out_ref[rows]
    assert np.isfinite(a).all(), "device output has non-finite values"
    assert np.isfinite(b).all()
    max_abs = float(np.abs(a - b).max())
    rel = np.linalg.norm(a - b, axis=-1) / np.maximum(np.linalg.norm(b, axis=-1), 1e-30)
    report = dict(max_abs=max_abs, max_row_rel_l2=float(rel.max()), rows=int(rows.sum()))
    assert max_abs <= ATTN_MAX_ABS, report
    assert rel.max() <= ATTN_ROW_REL_L2, report
    return report


def check_accept(target_logits, draft_logits, draft_tokens, uniforms, eta, T, tail_alpha, mode,
                 dev_accept_len, dev_next_token, dev_ratios=None):
    """Compares a device accept result with the oracle under the near-tie rules. Returns a report."""
    z = np.asarray(target_logits, dtype=np.float32)
    B, R, V = z.shape
    gamma = R - 1
    d = np.asarray(draft_logits, dtype=np.float32).reshape(B, gamma, V)
    tok = np.asarray(draft_tokens, dtype=np.int32).reshape(B, gamma)
    u = np.asarray(uniforms, dtype=np.float32).reshape(B, R)
    ref = oracle_accept(z, d, tok, u, eta=eta, T=T, tail_alpha=tail_alpha, residual_mode=mode)
    near_ties, token_alternatives = [], []
    for b in range(B):
        n_dev, n_ref = int(dev_accept_len[b]), int(ref["accept_len"][b])
        assert 0 <= n_dev <= gamma
        if n_dev != n_ref:
            k = min(n_dev, n_ref)
            gap = abs(float(u[b, k]) - min(1.0, float(ref["ratios"][b, k])))
            assert gap < TIE_EPS, f"sequence {b}: accept_len {n_dev} vs oracle {n_ref}, |u-ratio|={gap}"
            near_ties.append((b, k, gap))
        # the device token is judged against the oracle's distribution of the row the DEVICE stopped at
        n = n_dev
        if n < gamma:
            p, q, phat, _ = rapid_distributions(z[b, n], d[b, n], T=T, eta=eta, tail_alpha=tail_alpha)
            w = residual_weights(p, q, phat, mode)
            if not (w.sum() > 0):
                w = p
        else:
            p, _, _, _ = rapid_distributions(z[b, gamma], z[b, gamma], T=T, eta=0.0, tail_alpha=0.0)
            w = p
        t = int(dev_next_token[b])
        assert 0 <= t < V and w[t] > 0, f"sequence {b}: token {t} has no residual mass"
        c = np.cumsum(w)
        W = c[-1]
        lo = (c[t] - w[t]) / W
        hi = c[t] / W
        uu = float(u[b, gamma])
        assert lo - TIE_EPS <= uu <= hi + TIE_EPS, f"sequence {b}: token {t}, u={uu} outside [{lo},{hi}]"
        if n_dev == n_ref and t != int(ref["next_token"][b]):
            token_alternatives.append((b, t, int(ref["next_token"][b])))
    rep = dict(near_ties=near_ties, token_alternatives=token_alternatives,
               accept_len_ref=ref["accept_len"].tolist())
    if dev_ratios is not None and gamma > 0:
        r_dev = np.asarray(dev_ratios, dtype=np.float64).reshape(B, gamma)
        r_ref = ref["ratios"]
        fin = np.isfinite(r_ref)
        err = np.abs(r_dev[fin] - r_ref[fin]) / np.maximum(np.abs(r_ref[fin]), 1e-30)
        rep["max_ratio_rel_err"] = float(err.max()) if err.size else 0.0
        assert rep["max_ratio_rel_err"] < 1e-3, rep
    return rep
