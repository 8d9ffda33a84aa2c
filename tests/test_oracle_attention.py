"""Pins for the attention oracle: brute force, closed forms and invariants.

None of these calls the oracle to produce its own expected value: expectations
come from a loop-level restatement without the max shift, from closed forms
(means, planted keys) or from invariances the definition implies.
"""
import numpy as np
import pytest
import torch

import oracle
from workloads import bf16_bits


def _bf16(x):
    return torch.tensor(np.asarray(x), dtype=torch.float32).to(torch.bfloat16)


def _rand(shape, seed, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(*shape, generator=g) * scale).to(torch.bfloat16)


def _brute(q, k, v, ctx, gamma, scale):
    """Three nested loops, exp() without any max shift (fine for small scores)."""
    q = q.double().numpy(); k = k.double().numpy(); v = v.double().numpy()
    B, R, Hq, D = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    out = np.zeros((B, R, Hq, D))
    lse = np.zeros((B, R, Hq))
    for b in range(B):
        L = int(ctx[b])
        for h in range(Hq):
            for i in range(R):
                num = np.zeros(D); den = 0.0
                for j in range(L - R + i + 1):
                    e = np.exp(scale * float(np.dot(q[b, i, h], k[b, h // G, j])))
                    num += e * v[b, h // G, j]
                    den += e
                out[b, i, h] = num / den
                lse[b, i, h] = np.log(den)
    return out, lse


@pytest.mark.parametrize("B,Hq,Hkv,D,Lmax,gamma,lens", [
    (1, 2, 1, 8, 16, 0, [16]),
    (2, 4, 2, 16, 40, 3, [40, 7]),
    (2, 6, 2, 4, 64, 2, [3, 64]),
])
def test_brute_force(B, Hq, Hkv, D, Lmax, gamma, lens):
    R = gamma + 1
    q = _rand((B, R, Hq, D), 1); k = _rand((B, Hkv, Lmax, D), 2); v = _rand((B, Hkv, Lmax, D), 3)
    ctx = np.array(lens, dtype=np.int32)
    scale = 1.0 / np.sqrt(D)
    out, lse = oracle.verify_attention(bf16_bits(q), bf16_bits(k), bf16_bits(v), ctx, gamma)
    ref, ref_lse = _brute(q, k, v, ctx, gamma, scale)
    np.testing.assert_allclose(out, ref, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(lse, ref_lse, rtol=1e-11, atol=1e-12)


def test_explicit_scale_is_used():
    q = _rand((1, 2, 2, 8), 4); k = _rand((1, 1, 12, 8), 5); v = _rand((1, 1, 12, 8), 6)
    ctx = np.array([12], dtype=np.int32)
    out, _ = oracle.verify_attention(bf16_bits(q), bf16_bits(k), bf16_bits(v), ctx, 1, scale=0.37)
    ref, _ = _brute(q, k, v, ctx, 1, 0.37)
    np.testing.assert_allclose(out, ref, rtol=1e-11)


def test_equal_keys_give_mean_of_visible_values():
    B, Hq, Hkv, D, L, gamma = 1, 4, 2, 8, 33, 3
    R = gamma + 1
    q = _rand((B, R, Hq, D), 7)
    krow = _rand((D,), 8)
    k = krow.expand(B, Hkv, L, D).contiguous()
    v = _rand((B, Hkv, L, D), 9)
    ctx = np.array([L], dtype=np.int32)
    out, lse = oracle.verify_attention(bf16_bits(q), bf16_bits(k), bf16_bits(v), ctx, gamma)
    vd = v.double().numpy()
    for i in range(R):
        n = L - R + i + 1
        for h in range(Hq):
            np.testing.assert_allclose(out[0, i, h], vd[0, h // 2, :n].mean(axis=0), rtol=1e-12)
            s = (q[0, i, h].double() @ krow.double()).item() / np.sqrt(D)
            assert abs(lse[0, i, h] - (s + np.log(n))) < 1e-12


def test_planted_key_dominates():
    B, Hq, Hkv, D, L, gamma = 1, 2, 1, 16, 50, 1
    q = torch.zeros(B, 2, Hq, D); q[..., 0] = 16.0
    k = torch.zeros(B, Hkv, L, D); k[0, 0, 17, 0] = 16.0   # score 256/4 = 64 above the rest
    v = _rand((B, Hkv, L, D), 10)
    ctx = np.array([L], dtype=np.int32)
    out, _ = oracle.verify_attention(bf16_bits(q.bfloat16()), bf16_bits(k.bfloat16()), bf16_bits(v),
                                     ctx, gamma)
    for i in range(2):
        for h in range(Hq):
            np.testing.assert_allclose(out[0, i, h], v[0, 0, 17].double().numpy(), atol=1e-20 + 1e-24,
                                       rtol=1e-6)


def test_permutation_of_shared_prefix_is_invisible():
    B, Hq, Hkv, D, L, gamma = 1, 4, 2, 8, 29, 2
    R = gamma + 1
    q = _rand((B, R, Hq, D), 11); k = _rand((B, Hkv, L, D), 12); v = _rand((B, Hkv, L, D), 13)
    ctx = np.array([L], dtype=np.int32)
    out, _ = oracle.verify_attention(bf16_bits(q), bf16_bits(k), bf16_bits(v), ctx, gamma)
    perm = torch.randperm(L - R + 1, generator=torch.Generator().manual_seed(0))
    k2 = k.clone(); v2 = v.clone()
    k2[:, :, :L - R + 1] = k[:, :, perm]; v2[:, :, :L - R + 1] = v[:, :, perm]
    out2, _ = oracle.verify_attention(bf16_bits(q), bf16_bits(k2), bf16_bits(v2), ctx, gamma)
    np.testing.assert_allclose(out, out2, rtol=1e-11, atol=1e-14)


def test_causal_mask_and_padding_are_never_read():
    """Row i must not depend on keys after L-R+i, nor on anything at or beyond L."""
    B, Hq, Hkv, D, Lmax, gamma = 2, 2, 1, 8, 24, 2
    R = gamma + 1
    q = _rand((B, R, Hq, D), 14); k = _rand((B, Hkv, Lmax, D), 15); v = _rand((B, Hkv, Lmax, D), 16)
    ctx = np.array([20, 11], dtype=np.int32)
    out, _ = oracle.verify_attention(bf16_bits(q), bf16_bits(k), bf16_bits(v), ctx, gamma)
    k2 = k.clone(); v2 = v.clone()
    for b in range(B):
        L = int(ctx[b])
        k2[b, :, L:] = float("nan"); v2[b, :, L:] = float("inf")
    out2, _ = oracle.verify_attention(bf16_bits(q), bf16_bits(k2), bf16_bits(v2), ctx, gamma)
    np.testing.assert_array_equal(out, out2)
    # change the key/value seen only by the last row: rows 0..R-2 stay, row R-1 moves
    k3 = k.clone(); v3 = v.clone()
    for b in range(B):
        L = int(ctx[b])
        k3[b, :, L - 1] += 1.0; v3[b, :, L - 1] += 1.0
    out3, _ = oracle.verify_attention(bf16_bits(q), bf16_bits(k3), bf16_bits(v3), ctx, gamma)
    np.testing.assert_array_equal(out[:, :R - 1], out3[:, :R - 1])
    assert np.abs(out[:, R - 1] - out3[:, R - 1]).max() > 1e-3
    # the first row sees exactly L-R+1 keys: with one visible key the output is that value row
    ctx1 = np.array([R, R], dtype=np.int32)
    out4, lse4 = oracle.verify_attention(bf16_bits(q), bf16_bits(k), bf16_bits(v), ctx1, gamma)
    np.testing.assert_allclose(out4[:, 0, 0], v[:, 0, 0].double().numpy(), rtol=1e-15)


def test_gqa_heads_share_their_kv_head():
    B, Hq, Hkv, D, L, gamma = 1, 6, 2, 8, 18, 1
    q = _rand((B, 2, Hq, D), 17)
    q[:, :, 1] = q[:, :, 0]; q[:, :, 2] = q[:, :, 0]      # group 0: same query on its 3 heads
    q[:, :, 4] = q[:, :, 0]                                # a head of group 1 with the same query
    k = _rand((B, Hkv, L, D), 18); v = _rand((B, Hkv, L, D), 19)
    ctx = np.array([L], dtype=np.int32)
    out, _ = oracle.verify_attention(bf16_bits(q), bf16_bits(k), bf16_bits(v), ctx, gamma)
    np.testing.assert_array_equal(out[:, :, 0], out[:, :, 1])
    np.testing.assert_array_equal(out[:, :, 0], out[:, :, 2])
    assert np.abs(out[:, :, 0] - out[:, :, 4]).max() > 1e-3   # other KV head, other answer


def test_matches_library_softmax_attention_at_medium_size():
    """torch's fp64 softmax/matmul on a several-thousand-key case with strides and a unit sample."""
    B, Hq, Hkv, D, Lmax, gamma = 2, 4, 2, 32, 3000, 3
    R = gamma + 1
    q = _rand((B, R, Hq, D), 20); k = _rand((B, Hkv, Lmax, D), 21); v = _rand((B, Hkv, Lmax, D), 22)
    ctx = np.array([2999, 1234], dtype=np.int32)
    units = np.array([0, 5, 17, 31], dtype=np.int64)
    out, lse = oracle.verify_attention(bf16_bits(q), bf16_bits(k), bf16_bits(v), ctx, gamma, units=units)
    seen = np.zeros((B, R, Hq), dtype=bool)
    for u in units:
        b, h, i = u // (Hq * R), (u // R) % Hq, u % R
        seen[b, i, h] = True
        n = int(ctx[b]) - R + i + 1
        s = (k[b, h // 2, :n].double() @ q[b, i, h].double()) / np.sqrt(D)
        ref = torch.softmax(s, 0) @ v[b, h // 2, :n].double()
        np.testing.assert_allclose(out[b, i, h], ref.numpy(), rtol=1e-10, atol=1e-14)
        assert abs(lse[b, i, h] - torch.logsumexp(s, 0).item()) < 1e-10
    assert np.isnan(out[~seen]).all()


def test_invalid_lengths_are_rejected():
    q = _rand((1, 3, 2, 8), 23); k = _rand((1, 1, 10, 8), 24)
    with pytest.raises(ValueError):
        oracle.verify_attention(bf16_bits(q), bf16_bits(k), bf16_bits(k), np.array([2], np.int32), 2)
    with pytest.raises(ValueError):
        oracle.verify_attention(bf16_bits(q), bf16_bits(k), bf16_bits(k), np.array([11], np.int32), 2)


# ---- sink + window visibility (Section 3.2: the streaming drafter's cache of 4,096 entries, 4 of them sinks) ----

def _brute_window(q, k, v, ctx, gamma, scale, sink, window):
    """Loops over an explicitly enumerated key set per row: the sinks, then the window."""
    q = q.double().numpy(); k = k.double().numpy(); v = v.double().numpy()
    B, R, Hq, D = q.shape
    G = Hq // k.shape[1]
    out = np.zeros((B, R, Hq, D)); lse = np.zeros((B, R, Hq))
    for b in range(B):
        L = int(ctx[b])
        for h in range(Hq):
            for i in range(R):
                own = L - R + i
                keys = sorted(set(range(min(sink, own + 1))) | set(range(max(0, own - window + 1), own + 1)))
                num = np.zeros(D); den = 0.0
                for j in keys:
                    e = np.exp(scale * float(np.dot(q[b, i, h], k[b, h // G, j])))
                    num += e * v[b, h // G, j]; den += e
                out[b, i, h] = num / den; lse[b, i, h] = np.log(den)
    return out, lse


@pytest.mark.parametrize("sink,window", [(0, 1), (0, 5), (4, 7), (3, 1), (10, 100), (2, 16)])
def test_window_brute_force(sink, window):
    B, Hq, Hkv, D, Lmax, gamma = 2, 4, 2, 8, 48, 3
    R = gamma + 1
    q = _rand((B, R, Hq, D), 31); k = _rand((B, Hkv, Lmax, D), 32); v = _rand((B, Hkv, Lmax, D), 33)
    ctx = np.array([48, 9], dtype=np.int32)
    out, lse = oracle.verify_attention(bf16_bits(q), bf16_bits(k), bf16_bits(v), ctx, gamma, sink=sink, window=window)
    ref, ref_lse = _brute_window(q, k, v, ctx, gamma, 1.0 / np.sqrt(D), sink, window)
    np.testing.assert_allclose(out, ref, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(lse, ref_lse, rtol=1e-11, atol=1e-12)


def test_window_that_covers_everything_is_the_plain_mask():
    B, Hq, Hkv, D, L, gamma = 1, 4, 2, 8, 37, 2
    q = _rand((B, gamma + 1, Hq, D), 34); k = _rand((B, Hkv, L, D), 35); v = _rand((B, Hkv, L, D), 36)
    ctx = np.array([L], dtype=np.int32)
    full, full_lse = oracle.verify_attention(bf16_bits(q), bf16_bits(k), bf16_bits(v), ctx, gamma)
    for sink, window in ((0, L), (0, 10 * L), (5, L), (L, 1)):     # the last: every key is a sink
        out, lse = oracle.verify_attention(bf16_bits(q), bf16_bits(k), bf16_bits(v), ctx, gamma, sink=sink, window=window)
        np.testing.assert_array_equal(out, full)
        np.testing.assert_array_equal(lse, full_lse)


def test_window_of_one_returns_the_rows_own_value_and_hidden_keys_are_never_read():
    B, Hq, Hkv, D, L, gamma = 1, 2, 1, 8, 30, 3
    R = gamma + 1
    q = _rand((B, R, Hq, D), 37); k = _rand((B, Hkv, L, D), 38); v = _rand((B, Hkv, L, D), 39)
    ctx = np.array([L], dtype=np.int32)
    out, lse = oracle.verify_attention(bf16_bits(q), bf16_bits(k), bf16_bits(v), ctx, gamma, sink=0, window=1)
    for i in range(R):
        own = L - R + i
        for h in range(Hq):
            np.testing.assert_allclose(out[0, i, h], v[0, 0, own].double().numpy(), rtol=1e-15)
            s = float(q[0, i, h].double() @ k[0, 0, own].double()) / np.sqrt(D)
            assert abs(lse[0, i, h] - s) < 1e-12
    # sinks 0..2 and a window of 4: keys 3 .. own-4 are hidden from row i and may hold anything
    sink, window = 3, 4
    base, _ = oracle.verify_attention(bf16_bits(q), bf16_bits(k), bf16_bits(v), ctx, gamma, sink=sink, window=window)
    k2 = k.clone(); v2 = v.clone()
    k2[:, :, sink:L - R - window + 1] = float("nan"); v2[:, :, sink:L - R - window + 1] = float("inf")
    again, _ = oracle.verify_attention(bf16_bits(q), bf16_bits(k2), bf16_bits(v2), ctx, gamma, sink=sink, window=window)
    np.testing.assert_array_equal(base, again)
    # the key just inside row 0's window is seen by row 0 only (row 1's window starts one key later)
    k3 = k.clone(); v3 = v.clone()
    edge = L - R - window + 1
    k3[:, :, edge] += 1.0; v3[:, :, edge] += 1.0
    moved, _ = oracle.verify_attention(bf16_bits(q), bf16_bits(k3), bf16_bits(v3), ctx, gamma, sink=sink, window=window)
    assert np.abs(moved[:, 0] - base[:, 0]).max() > 1e-3
    np.testing.assert_array_equal(moved[:, 1:], base[:, 1:])
    # a sink key is seen by every row
    k4 = k.clone(); k4[:, :, 1] += 1.0
    moved, _ = oracle.verify_attention(bf16_bits(q), bf16_bits(k4), bf16_bits(v), ctx, gamma, sink=sink, window=window)
    assert all(np.abs(moved[:, i] - base[:, i]).max() > 1e-4 for i in range(R))


# ---- FP8 E4M3 cache with per-(sequence, KV head) scales ----------------------------------------------------

def _codes(shape, seed):
    """Random E4M3 codes without the two NaN patterns."""
    g = torch.Generator().manual_seed(seed)
    c = torch.randint(0, 256, shape, generator=g, dtype=torch.int32)
    c[(c & 0x7F) == 0x7F] = 0x3A
    return c.to(torch.uint8)


def test_e4m3_decoding_of_every_code():
    """All 256 codes: against the library's own E4M3 type, and a few values known by heart from the format
    (bias 7, 3 mantissa bits, subnormals at exponent 0, no infinities, S.1111.111 = NaN, largest 448)."""
    lib = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).double().numpy()
    for code in range(256):
        v = oracle.e4m3_to_double(code)
        if np.isnan(lib[code]):
            assert np.isnan(v) and code in (0x7F, 0xFF)
        else:
            assert v == lib[code], hex(code)
    known = {0x00: 0.0, 0x01: 2.0 ** -9, 0x07: 7 * 2.0 ** -9, 0x08: 2.0 ** -6, 0x38: 1.0, 0x39: 1.125, 0x40: 2.0,
             0x7E: 448.0, 0x78: 256.0, 0xB8: -1.0, 0xFE: -448.0, 0x80: 0.0}
    for code, val in known.items():
        assert oracle.e4m3_to_double(code) == val
    assert np.copysign(1.0, oracle.e4m3_to_double(0x80)) == -1.0


def test_fp8_cache_equals_the_bf16_definition_on_values_both_can_hold():
    """Every E4M3 value times a power-of-two scale is a bf16 number: the bf16 oracle on those numbers must
    give the same bits."""
    B, Hq, Hkv, D, Lmax, gamma = 2, 4, 2, 16, 40, 3
    q = _rand((B, gamma + 1, Hq, D), 41)
    kc, vc = _codes((B, Hkv, Lmax, D), 42), _codes((B, Hkv, Lmax, D), 43)
    ks = torch.tensor([[0.5, 2.0], [0.125, 1.0]]); vs = torch.tensor([[4.0, 0.25], [1.0, 0.0625]])
    ctx = np.array([40, 9], dtype=np.int32)
    out8, lse8 = oracle.verify_attention_fp8(bf16_bits(q), kc.numpy(), vc.numpy(), ks.numpy(), vs.numpy(), ctx, gamma)
    k = (kc.view(torch.float8_e4m3fn).float() * ks[:, :, None, None]).to(torch.bfloat16)
    v = (vc.view(torch.float8_e4m3fn).float() * vs[:, :, None, None]).to(torch.bfloat16)
    assert torch.equal(k.float(), kc.view(torch.float8_e4m3fn).float() * ks[:, :, None, None])   # nothing was rounded
    out16, lse16 = oracle.verify_attention(bf16_bits(q), bf16_bits(k), bf16_bits(v), ctx, gamma)
    np.testing.assert_array_equal(out8, out16)
    np.testing.assert_array_equal(lse8, lse16)


def test_fp8_scales_act_as_the_definition_says():
    B, Hq, Hkv, D, Lmax, gamma = 1, 4, 2, 8, 30, 2
    q = _rand((B, gamma + 1, Hq, D), 44)
    kc, vc = _codes((B, Hkv, Lmax, D), 45), _codes((B, Hkv, Lmax, D), 46)
    ks = np.array([[0.37, 1.9]], np.float32); vs = np.array([[0.8, 3.1]], np.float32)
    ctx = np.array([30], dtype=np.int32)
    base, lse = oracle.verify_attention_fp8(bf16_bits(q), kc.numpy(), vc.numpy(), ks, vs, ctx, gamma)
    # the value scale multiplies the output of its own KV head's query heads, and nothing else
    vs2 = vs.copy(); vs2[0, 1] *= 4.0
    out, lse2 = oracle.verify_attention_fp8(bf16_bits(q), kc.numpy(), vc.numpy(), ks, vs2, ctx, gamma)
    np.testing.assert_allclose(out[:, :, 2:], 4.0 * base[:, :, 2:], rtol=1e-12)
    np.testing.assert_array_equal(out[:, :, :2], base[:, :, :2])
    np.testing.assert_array_equal(lse2, lse)
    # a key scale of 2 with the query halved (exact in bf16) leaves every score as it was
    ks2 = ks * 2.0
    out, lse3 = oracle.verify_attention_fp8(bf16_bits((q.float() * 0.5).to(torch.bfloat16)), kc.numpy(), vc.numpy(),
                                            ks2, vs, ctx, gamma)
    np.testing.assert_allclose(out, base, rtol=1e-12)
    np.testing.assert_allclose(lse3, lse, rtol=1e-12)
    # and it is the brute-force softmax of the decoded cache
    kd = kc.view(torch.float8_e4m3fn).double() * torch.tensor(ks, dtype=torch.float64)[:, :, None, None]
    vd = vc.view(torch.float8_e4m3fn).double() * torch.tensor(vs, dtype=torch.float64)[:, :, None, None]
    for i in range(gamma + 1):
        n = 30 - (gamma + 1) + i + 1
        for h in range(Hq):
            s = (kd[0, h // 2, :n] @ q[0, i, h].double()) / np.sqrt(D)
            ref = torch.softmax(s, 0) @ vd[0, h // 2, :n]
            np.testing.assert_allclose(base[0, i, h], ref.numpy(), rtol=1e-10, atol=1e-13)
