"""Pins for the accept/residual oracle.

Expected values come from the worked examples under tests/golden, from the
textbook speculative-sampling rules (eta = 0), from closed-form output laws
checked by Monte-Carlo, from a loop-level brute force and from the
distillation-gradient proposition -- never from the oracle itself.
"""
import json
import math
import os

import numpy as np
import pytest
from scipy.special import softmax
from scipy.stats import chi2

import oracle

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "hand_examples.json")))


def _num(x):
    return {"ln2": math.log(2.0), "ln3": math.log(3.0)}.get(x, x) if isinstance(x, str) else x


def _vec(xs):
    return np.array([_num(x) for x in xs], dtype=np.float64)


# ---------------------------------------------------------------- golden examples
@pytest.mark.parametrize("name", ["two_token", "four_token_tail"])
def test_hand_examples(name):
    ex = GOLD[name]
    z = _vec(ex["z"]).astype(np.float32); d = _vec(ex["d"]).astype(np.float32)
    p, q, phat, raw = oracle.rapid_distributions(z, d, T=ex["T"], eta=ex["eta"], tail_alpha=ex["tail_alpha"])
    np.testing.assert_allclose(p, ex["p"], atol=2e-6)
    np.testing.assert_allclose(q, ex["q"], atol=2e-6)
    np.testing.assert_allclose(phat, ex["phat"], atol=2e-6)
    if "phat_raw" in ex:
        np.testing.assert_allclose(raw, ex["phat_raw"], atol=2e-6)
    np.testing.assert_array_equal((raw < ex["tail_alpha"] * raw.max()).astype(int), ex["tail_mask"])
    np.testing.assert_allclose(phat / q, ex["ratio"], atol=5e-6)
    w = oracle.residual_weights(p, q, phat)
    np.testing.assert_allclose(w, ex["residual_unnormalised"], atol=2e-6)
    if "output_law" in ex:
        beta = np.minimum(q, phat).sum()
        np.testing.assert_allclose(np.minimum(q, phat) + (1 - beta) * w / w.sum(), ex["output_law"], atol=2e-6)
    # the full loop on this example, gamma = 1: every draft token, u just below / above the ratio
    V = z.size
    for x in range(V):
        ratio = min(1.0, ex["ratio"][x])
        for u0, want in ((max(ratio - 1e-4, 0.0), 1), (ratio + 1e-4, 0)):
            if u0 >= 1.0:
                continue
            zz = np.stack([z, z])[None]          # bonus row = z again
            res = oracle.accept(zz, d[None, None], np.array([[x]]), np.array([[u0, 0.5]]),
                                eta=ex["eta"], T=ex["T"], tail_alpha=ex["tail_alpha"])
            assert res["accept_len"][0] == want
            if want == 0:
                assert res["next_token"][0] == oracle.inverse_cdf(np.array(ex["residual_unnormalised"]), 0.5)
    if "residual_token" in ex:
        assert oracle.inverse_cdf(w, 0.999) == ex["residual_token"]


def test_closed_form_phat_two_tokens():
    z = np.array([math.log(2.0), 0.0], np.float32); d = np.array([0.0, math.log(3.0)], np.float32)
    _, _, phat, _ = oracle.rapid_distributions(z, d, T=1.0, eta=1.0, tail_alpha=0.0)
    assert abs(phat[0] - 2.0 / (2.0 + math.exp(5.0 / 6.0))) < 1e-7   # fp32 rounding of ln 2, ln 3


# ---------------------------------------------------------------- eta = 0: textbook speculative sampling
def _textbook_sd(z, d, tokens, u, T):
    """Section 2.1: accept r <= min(1, p/q); on rejection sample norm(max(p-q,0)); bonus from p."""
    gamma = d.shape[0]
    n = 0
    for k in range(gamma):
        p = softmax(z[k].astype(np.float64) / T); q = softmax(d[k].astype(np.float64) / T)
        if u[k] <= min(1.0, p[tokens[k]] / q[tokens[k]]):
            n += 1
            continue
        w = np.maximum(p - q, 0.0)
        break
    else:
        w = softmax(z[gamma].astype(np.float64) / T)
    c = np.cumsum(w)
    tok = int(np.searchsorted(c, u[gamma] * c[-1], side="right"))
    return n, tok


@pytest.mark.parametrize("T", [1.0, 0.1, 2.5])
@pytest.mark.parametrize("mode", [oracle.RESIDUAL_PAPER, oracle.RESIDUAL_PHAT])
@pytest.mark.parametrize("alpha", [0.0, 0.1])
def test_eta_zero_is_textbook_speculative_sampling(T, mode, alpha):
    rng = np.random.default_rng(5)
    B, gamma, V = 64, 4, 37
    d = rng.normal(0, 2, (B, gamma, V)).astype(np.float32)
    z = np.concatenate([d + rng.normal(0, 1.0, d.shape), rng.normal(0, 2, (B, 1, V))], 1).astype(np.float32)
    tokens = rng.integers(0, V, (B, gamma)).astype(np.int32)
    u = rng.random((B, gamma + 1)).astype(np.float32)
    res = oracle.accept(z, d, tokens, u, eta=0.0, T=T, tail_alpha=alpha, residual_mode=mode)
    lens = set()
    for b in range(B):
        n, tok = _textbook_sd(z[b], d[b], tokens[b], u[b], T)
        assert res["accept_len"][b] == n
        assert res["next_token"][b] == tok
        lens.add(n)
    assert len(lens) >= 3          # both branches and several stop positions were exercised


# ---------------------------------------------------------------- identical logits: everything accepted
@pytest.mark.parametrize("eta", [0.0, 0.5, 20.0])
def test_identical_logits_accept_everything(eta):
    rng = np.random.default_rng(6)
    B, gamma, V = 8, 5, 50
    d = rng.normal(0, 2, (B, gamma, V)).astype(np.float32)
    bonus = rng.normal(0, 2, (B, 1, V)).astype(np.float32)
    z = np.concatenate([d, bonus], 1)
    tokens = rng.integers(0, V, (B, gamma)).astype(np.int32)
    u = rng.random((B, gamma + 1)).astype(np.float32)
    u[:, 0] = np.nextafter(np.float32(1.0), np.float32(0.0))     # the largest uniform still accepts
    res = oracle.accept(z, d, tokens, u, eta=eta, T=0.7)
    assert (res["accept_len"] == gamma).all()
    np.testing.assert_allclose(res["ratios"], 1.0, rtol=1e-12)
    for b in range(B):
        c = np.cumsum(softmax(bonus[b, 0].astype(np.float64) / 0.7))
        assert res["next_token"][b] == int(np.searchsorted(c, u[b, gamma] * c[-1], side="right"))


# ---------------------------------------------------------------- Eq. (new_target) == softmax(zhat/T) of Eq. (delta)
@pytest.mark.parametrize("T,eta", [(1.0, 5.0), (0.1, 20.0), (2.0, 50.0)])
def test_two_forms_of_the_augmented_target_agree(T, eta):
    rng = np.random.default_rng(7)
    V = 200
    d = rng.normal(0, 2, V).astype(np.float32); z = (d + rng.normal(0, 1, V)).astype(np.float32)
    p, q, _, raw = oracle.rapid_distributions(z, d, T=T, eta=eta, tail_alpha=0.1)
    pp = softmax(z.astype(np.float64) / T); qq = softmax(d.astype(np.float64) / T)
    np.testing.assert_allclose(p, pp, rtol=1e-12)
    np.testing.assert_allclose(q, qq, rtol=1e-12)
    np.testing.assert_allclose(raw, softmax(z.astype(np.float64) / T + eta * (qq - pp)), rtol=1e-11)
    assert abs(raw.sum() - 1.0) < 1e-12


def test_tail_rule_mask_and_patch():
    rng = np.random.default_rng(8)
    V = 300
    d = rng.normal(0, 3, V).astype(np.float32); z = (d + rng.normal(0, 1, V)).astype(np.float32)
    p, q, phat, raw = oracle.rapid_distributions(z, d, T=1.0, eta=10.0, tail_alpha=0.1)
    mask = raw < 0.1 * raw.max()
    assert 0 < mask.sum() < V
    np.testing.assert_array_equal(phat[mask], p[mask])            # patched entries are p, bit for bit
    np.testing.assert_array_equal(phat[~mask], raw[~mask])
    _, _, off, raw2 = oracle.rapid_distributions(z, d, T=1.0, eta=10.0, tail_alpha=0.0)
    np.testing.assert_array_equal(off, raw2)


# ---------------------------------------------------------------- proposition: d/dz T^2 KL(q||p) = T (p - q)
def test_distillation_gradient_proposition():
    rng = np.random.default_rng(9)
    V, T = 12, 0.6
    z = rng.normal(0, 1, V).astype(np.float32); d = rng.normal(0, 1, V).astype(np.float32)
    p, q, _, _ = oracle.rapid_distributions(z, d, T=T, eta=0.0, tail_alpha=0.0)

    def loss(zv):
        pv, qv, _, _ = oracle.rapid_distributions(zv.astype(np.float32), d, T=T, eta=0.0, tail_alpha=0.0)
        return T * T * float(np.sum(qv * np.log(qv / pv)))

    # z is fp32 at the interface: use steps that are exact in fp32 around O(1) values
    h = 2.0 ** -9
    for i in range(V):
        zp = z.astype(np.float64).copy(); zm = zp.copy()
        zp[i] = np.float32(zp[i] + h); zm[i] = np.float32(zm[i] - h)
        g = (loss(zp) - loss(zm)) / (zp[i] - zm[i])
        assert abs(g - T * (p[i] - q[i])) < 2e-5


# ---------------------------------------------------------------- brute force over all accept / reject patterns
def _brute_accept(z, d, tokens, u, eta, T, alpha, mode):
    gamma, V = d.shape
    n = 0
    w = None
    for k in range(gamma):
        ez = [math.exp(float(z[k, v]) / T) for v in range(V)]; p = [e / sum(ez) for e in ez]
        ed = [math.exp(float(d[k, v]) / T) for v in range(V)]; q = [e / sum(ed) for e in ed]
        eh = [math.exp(float(z[k, v]) / T + eta * (q[v] - p[v])) for v in range(V)]
        raw = [e / sum(eh) for e in eh]
        ph = [p[v] if raw[v] < alpha * max(raw) else raw[v] for v in range(V)]
        x = int(tokens[k])
        if float(u[k]) <= min(1.0, ph[x] / q[x]):
            n += 1
            continue
        if mode == oracle.RESIDUAL_PAPER:
            w = [max(p[v] - ph[v], p[v] - q[v], 0.0) for v in range(V)]
        else:
            w = [max(ph[v] - q[v], 0.0) for v in range(V)]
        break
    if w is None:
        ez = [math.exp(float(z[gamma, v]) / T) for v in range(V)]; w = [e / sum(ez) for e in ez]
    tot = sum(w); c = 0.0; tok = None
    for v in range(V):
        c += w[v]
        if w[v] > 0 and c > float(u[gamma]) * tot:
            tok = v
            break
    return n, tok


@pytest.mark.parametrize("mode", [oracle.RESIDUAL_PAPER, oracle.RESIDUAL_PHAT])
def test_brute_force_all_patterns(mode):
    rng = np.random.default_rng(10)
    gamma, V, T, eta, alpha = 3, 9, 0.8, 6.0, 0.1
    d = rng.normal(0, 1.5, (gamma, V)).astype(np.float32)
    z = np.concatenate([d + rng.normal(0, 1.0, d.shape), rng.normal(0, 1.5, (1, V))]).astype(np.float32)
    tokens = np.argmax(d - z[:gamma], axis=1).astype(np.int32)     # draft favours them: ratio < 1
    full = oracle.accept(z[None], d[None], tokens[None], np.zeros((1, gamma + 1), np.float32), eta=eta, T=T,
                         tail_alpha=alpha, residual_mode=mode)
    ratios = np.minimum(full["ratios"][0], 1.0)
    seen = set()
    for pattern in range(2 ** gamma):
        for us in (0.03, 0.41, 0.77, 0.999):
            u = np.empty(gamma + 1, np.float32)
            for k in range(gamma):
                acc = (pattern >> k) & 1
                u[k] = 0.0 if acc else min(float(ratios[k]) + 0.05, 0.9999)
                if not acc and ratios[k] >= 0.9999:
                    u[k] = 0.0            # this position cannot be rejected
            u[gamma] = us
            res = oracle.accept(z[None], d[None], tokens[None], u[None], eta=eta, T=T, tail_alpha=alpha,
                                residual_mode=mode)
            n, tok = _brute_accept(z, d, tokens, u, eta, T, alpha, mode)
            assert res["accept_len"][0] == n and res["next_token"][0] == tok
            seen.add(n)
    assert seen == set(range(gamma + 1))


# ---------------------------------------------------------------- Monte-Carlo: the law of the emitted token
def _law_test(V, eta, alpha, mode, seed, trials=400_000, T=1.0):
    rng = np.random.default_rng(seed)
    d = rng.normal(0, 1.2, V).astype(np.float32); z = (d + rng.normal(0, 1.0, V)).astype(np.float32)
    p = softmax(z.astype(np.float64) / T); q = softmax(d.astype(np.float64) / T)
    raw = softmax(z.astype(np.float64) / T + eta * (q - p))
    ph = np.where(raw < alpha * raw.max(), p, raw)
    w = np.maximum(np.maximum(p - ph, p - q), 0) if mode == oracle.RESIDUAL_PAPER else np.maximum(ph - q, 0)
    beta = np.minimum(q, ph).sum()
    law = np.minimum(q, ph) + (1 - beta) * w / w.sum()
    assert abs(law.sum() - 1) < 1e-12
    tokens = rng.choice(V, size=trials, p=q).astype(np.int32)[:, None]
    u = rng.random((trials, 2)).astype(np.float32)
    zz = np.broadcast_to(np.stack([z, z])[None], (trials, 2, V))
    dd = np.broadcast_to(d[None, None], (trials, 1, V))
    res = oracle.accept(zz, dd, tokens, u, eta=eta, T=T, tail_alpha=alpha, residual_mode=mode)
    emitted = np.where(res["accept_len"] == 1, tokens[:, 0], res["next_token"])
    counts = np.bincount(emitted, minlength=V).astype(np.float64)
    keep = law * trials >= 5
    stat = ((counts[keep] - law[keep] * trials) ** 2 / (law[keep] * trials)).sum()
    pval = chi2.sf(stat, keep.sum() - 1)
    return law, p, ph, pval, res["accept_len"].mean(), beta


@pytest.mark.parametrize("V", [4, 8, 16])
def test_monte_carlo_eta_zero_gives_target_law(V):
    law, p, _, pval, acc, beta = _law_test(V, eta=0.0, alpha=0.1, mode=oracle.RESIDUAL_PAPER, seed=20 + V)
    np.testing.assert_allclose(law, p, atol=1e-12)       # textbook guarantee: the output follows p
    assert pval > 1e-3
    assert abs(acc - beta) < 4e-3                        # acceptance rate = sum min(p, q)


@pytest.mark.parametrize("V,eta", [(4, 2.0), (8, 5.0), (16, 20.0)])
def test_monte_carlo_augmented_target_law(V, eta):
    """With the clamp at 0 the emitted law is min(q,phat) + (1-beta) w/W (Appendix B's mixture)."""
    law, p, ph, pval, acc, beta = _law_test(V, eta=eta, alpha=0.1, mode=oracle.RESIDUAL_PAPER, seed=30 + V)
    assert pval > 1e-3
    assert abs(acc - beta) < 4e-3
    assert np.abs(law - p).max() > 1e-3                  # and it is NOT p once phat pulls above p


@pytest.mark.parametrize("V,eta", [(8, 5.0), (16, 20.0)])
def test_monte_carlo_phat_mode_gives_phat(V, eta):
    law, _, ph, pval, _, _ = _law_test(V, eta=eta, alpha=0.0, mode=oracle.RESIDUAL_PHAT, seed=40 + V)
    np.testing.assert_allclose(law, ph, atol=1e-12)      # standard sampling against phat
    assert pval > 1e-3


def test_wrong_law_is_detected_by_the_monte_carlo_check():
    """The chi-square has power: the eta>0 samples do not fit p."""
    V, eta, trials = 8, 5.0, 400_000
    rng = np.random.default_rng(38)
    d = rng.normal(0, 1.2, V).astype(np.float32); z = (d + rng.normal(0, 1.0, V)).astype(np.float32)
    p = softmax(z.astype(np.float64)); q = softmax(d.astype(np.float64))
    tokens = rng.choice(V, size=trials, p=q).astype(np.int32)[:, None]
    u = rng.random((trials, 2)).astype(np.float32)
    res = oracle.accept(np.broadcast_to(np.stack([z, z])[None], (trials, 2, V)),
                        np.broadcast_to(d[None, None], (trials, 1, V)), tokens, u, eta=eta)
    emitted = np.where(res["accept_len"] == 1, tokens[:, 0], res["next_token"])
    counts = np.bincount(emitted, minlength=V)
    stat = ((counts - p * trials) ** 2 / (p * trials)).sum()
    assert chi2.sf(stat, V - 1) < 1e-6


# ---------------------------------------------------------------- edge cases of the rule
def test_edge_cases():
    V = 6
    z = np.zeros((1, 2, V), np.float32); d = np.zeros((1, 1, V), np.float32)
    d[0, 0, 2] = 3.0                                    # q(2) large => ratio < 1 at token 2
    tok = np.array([[2]], np.int32)
    r = oracle.accept(z, d, tok, np.array([[0.0, 0.3]], np.float32), eta=0.0)
    assert r["accept_len"][0] == 1                      # u = 0 always accepts
    ratio = float(r["ratios"][0, 0])
    pq = softmax(z[0, 0].astype(np.float64))[2] / softmax(d[0, 0].astype(np.float64))[2]
    assert abs(ratio - pq) < 1e-14 and ratio < 1
    u_eq = np.float32(ratio)                            # r <= ratio: equality accepts (when fp32(ratio) <= ratio)
    r2 = oracle.accept(z, d, tok, np.array([[u_eq, 0.3]], np.float32), eta=0.0)
    assert r2["accept_len"][0] == int(float(u_eq) <= ratio)
    r3 = oracle.accept(z, d, tok, np.array([[np.nextafter(u_eq, np.float32(1)), 0.3]], np.float32), eta=0.0)
    r3b = oracle.accept(z, d, tok, np.array([[np.nextafter(np.nextafter(u_eq, np.float32(1)), np.float32(1)), 0.3]],
                                            np.float32), eta=0.0)
    assert r3b["accept_len"][0] == 0
    # rejected at token 2 with p uniform: residual puts no mass on token 2, equal mass elsewhere
    for uu, want in ((0.0, 0), (0.21, 1), (0.41, 3), (0.999, 5)):
        rr = oracle.accept(z, d, tok, np.array([[0.99, uu]], np.float32), eta=0.0)
        assert rr["accept_len"][0] == 0 and rr["next_token"][0] == want
    # gamma = 0: only the bonus draw from softmax(z_0)
    z0 = np.log(np.array([[[0.1, 0.2, 0.3, 0.4]]], np.float32))
    for uu, want in ((0.05, 0), (0.15, 1), (0.59, 2), (0.61, 3)):
        rr = oracle.accept(z0, np.zeros((1, 0, 4), np.float32), np.zeros((1, 0), np.int32),
                           np.array([[uu]], np.float32), eta=3.0)
        assert rr["accept_len"][0] == 0 and rr["next_token"][0] == want
    with pytest.raises(ValueError):
        oracle.accept(z, d, np.array([[V]], np.int32), np.zeros((1, 2), np.float32), eta=0.0)
    with pytest.raises(ValueError):
        oracle.accept(z, d, tok, np.zeros((1, 2), np.float32), eta=0.0, T=0.0)


def test_inverse_cdf_skips_zero_weights_and_handles_empty():
    w = np.array([0.0, 2.0, 0.0, 1.0, 1.0, 0.0])
    assert oracle.inverse_cdf(w, 0.0) == 1
    assert oracle.inverse_cdf(w, 0.4999) == 1
    assert oracle.inverse_cdf(w, 0.5) == 3
    assert oracle.inverse_cdf(w, 0.75) == 4
    assert oracle.inverse_cdf(w, 0.99999999) == 4
    assert oracle.inverse_cdf(np.zeros(4), 0.3) == -1


def test_draft_sample_on_a_known_distribution():
    """Logits = T * log of exact probabilities: the drawn token follows the printed CDF intervals and
    log q is the log of the printed probability, at any temperature."""
    probs = np.array([0.1, 0.2, 0.3, 0.4])
    for T in (1.0, 0.5, 2.0):
        logits = (T * np.log(probs)).astype(np.float32)[None, :].repeat(6, 0) + 3.0   # a shift changes nothing
        u = np.array([0.0, 0.05, 0.15, 0.45, 0.75, 0.999], dtype=np.float32)
        tok, logq, stats = oracle.draft_sample(logits, u, T)
        assert tok.tolist() == [0, 0, 1, 2, 3, 3]
        np.testing.assert_allclose(np.exp(logq), probs[tok], rtol=1e-6)
        np.testing.assert_allclose(stats[:, 0], (logits.astype(np.float64) / T).max(axis=1), rtol=0, atol=1e-12)
        np.testing.assert_allclose(stats[:, 1] - stats[:, 0], np.log((probs / probs.max()).sum()), atol=1e-6)


def test_draft_sample_is_the_gamma_zero_accept():
    """With no draft rows Algorithm 1's accept step only draws the bonus token from softmax(z/T):
    the same rule, so the two oracle routines must agree."""
    rng = np.random.default_rng(11)
    z = (rng.normal(size=(5, 1, 64)) * 3).astype(np.float32)
    u = rng.random(size=(5, 1)).astype(np.float32)
    ref = oracle.accept(z, np.zeros((5, 0, 64), np.float32), np.zeros((5, 0), np.int32), u, eta=0.0, T=0.7)
    tok, _, _ = oracle.draft_sample(z[:, 0], u[:, 0], 0.7)
    assert tok.tolist() == ref["next_token"].tolist()
