"""CPU oracle for the RAPID verify step -- TEST INFRASTRUCTURE ONLY.

A ctypes wrapper over ``rapid_oracle.c`` (plain fp64 C written from the paper:
Algorithm 1, Eq. (new_target), Eq. (delta), the tail rule of Section 2.4).
It shares nothing with the CUDA library and must not be imported by the
product package; only tests, the smoke check and the benchmark's CPU-baseline
leg may use it.

Arrays are numpy; bf16 tensors are passed as their raw bits (uint16).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rapid_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

RESIDUAL_PAPER = 0  # norm(max(p - phat, p - q, 0)): Algorithm 1, residual step
RESIDUAL_PHAT = 1   # norm(max(phat - q, 0)): Section 2.1's residual with phat as the target
FLAG_RESIDUAL_FALLBACK = 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP) if the shared object is missing or stale.

    ``RAPID_ORACLE_LIB`` may name another build of the same source; the tests
    use it to show that planted mistakes are caught by the pins.
    """
    override = os.environ.get("RAPID_ORACLE_LIB")
    if override:
        return override
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        subprocess.run(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"],
            check=True,
        )
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        c_i64 = ctypes.c_int64
        c_dbl = ctypes.c_double
        vp = ctypes.c_void_p
        lib.oracle_num_threads.restype = ctypes.c_int
        lib.oracle_verify_attention.restype = ctypes.c_int
        lib.oracle_verify_attention.argtypes = [
            vp, vp, vp, vp, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, c_i64,
            ctypes.c_int, c_i64, c_i64, c_i64, c_dbl, vp, c_i64, vp, vp,
        ]
        lib.oracle_verify_attention_window.restype = ctypes.c_int
        lib.oracle_verify_attention_window.argtypes = [
            vp, vp, vp, vp, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, c_i64,
            ctypes.c_int, c_i64, c_i64, c_i64, c_dbl, c_i64, c_i64, vp, c_i64, vp, vp,
        ]
        lib.oracle_e4m3_to_double.restype = c_dbl
        lib.oracle_e4m3_to_double.argtypes = [ctypes.c_uint8]
        lib.oracle_verify_attention_fp8.restype = ctypes.c_int
        lib.oracle_verify_attention_fp8.argtypes = [
            vp, vp, vp, vp, vp, vp, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, c_i64,
            ctypes.c_int, c_i64, c_i64, c_i64, c_dbl, vp, c_i64, vp, vp,
        ]
        lib.oracle_rapid_distributions.restype = None
        lib.oracle_rapid_distributions.argtypes = [vp, vp, c_i64, c_dbl, c_dbl, c_dbl, vp, vp, vp, vp]
        lib.oracle_residual_weights.restype = None
        lib.oracle_residual_weights.argtypes = [vp, vp, vp, c_i64, ctypes.c_int, vp]
        lib.oracle_inverse_cdf.restype = c_i64
        lib.oracle_inverse_cdf.argtypes = [vp, c_i64, c_dbl]
        lib.oracle_accept.restype = ctypes.c_int
        lib.oracle_accept.argtypes = [
            vp, vp, vp, vp, ctypes.c_int, ctypes.c_int, c_i64, c_dbl, c_dbl, c_dbl, ctypes.c_int,
            vp, vp, vp, vp,
        ]
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def verify_attention(q_bits, k_bits, v_bits, ctx_lens, gamma, scale=0.0, units=None,
                     kv_strides=None, sink=0, window=0):
    """Definition of verify attention.

    ``window > 0`` applies the sink + window visibility of the streaming drafter of Section 3.2
    (row i with own key lim sees key j iff j <= lim and (j < sink or j > lim - window)).

    q_bits [B,R,Hq,D] uint16 (bf16 bits); k_bits, v_bits [B,Hkv,Lmax,D] uint16
    (or flat arrays when ``kv_strides=(stride_b, stride_h, stride_l, Lmax, Hkv)``
    in elements is given); ctx_lens [B] int32.  Returns (out [B,R,Hq,D]
    float64, lse [B,R,Hq] float64).  ``units`` optionally lists the
    (b*Hq+h)*R+i units to compute; other rows are NaN.
    """
    lib = _load()
    q_bits = _c(q_bits, np.uint16)
    B, R, Hq, D = q_bits.shape
    assert R == gamma + 1
    if kv_strides is None:
        k_bits = _c(k_bits, np.uint16)
        v_bits = _c(v_bits, np.uint16)
        _, Hkv, Lmax, Dk = k_bits.shape
        assert Dk == D and v_bits.shape == k_bits.shape and k_bits.shape[0] == B
        sb, sh, sl = Hkv * Lmax * D, Lmax * D, D
    else:
        sb, sh, sl, Lmax, Hkv = kv_strides
        assert k_bits.dtype == np.uint16 and v_bits.dtype == np.uint16
        assert k_bits.flags.c_contiguous and v_bits.flags.c_contiguous
    ctx_lens = _c(ctx_lens, np.int32)
    out = np.full((B, R, Hq, D), np.nan, dtype=np.float64)
    lse = np.full((B, R, Hq), np.nan, dtype=np.float64)
    if units is not None:
        units = _c(units, np.int64)
        n_units = units.size
    else:
        n_units = 0
    if window > 0:
        rc = lib.oracle_verify_attention_window(
            _ptr(q_bits), _ptr(k_bits), _ptr(v_bits), _ptr(ctx_lens), B, Hq, Hkv, D, Lmax, gamma,
            sb, sh, sl, float(scale), int(sink), int(window), _ptr(units), n_units, _ptr(out), _ptr(lse))
    else:
        if sink:
            raise ValueError("sink keys need a window")
        rc = lib.oracle_verify_attention(
            _ptr(q_bits), _ptr(k_bits), _ptr(v_bits), _ptr(ctx_lens), B, Hq, Hkv, D, Lmax, gamma,
            sb, sh, sl, float(scale), _ptr(units), n_units, _ptr(out), _ptr(lse))
    if rc != 0:
        raise ValueError(f"oracle_verify_attention failed with {rc}")
    return out, lse


def e4m3_to_double(code: int) -> float:
    """Value of one FP8 E4M3 code (OCP 8-bit floating point: bias 7, no infinities, S.1111.111 = NaN)."""
    return float(_load().oracle_e4m3_to_double(int(code) & 0xFF))


def verify_attention_fp8(q_bits, k_codes, v_codes, k_scale, v_scale, ctx_lens, gamma, scale=0.0, units=None):
    """Verify attention over an FP8 E4M3 cache with one fp32 scale per (sequence, KV head) for K and for V:
    the attention definition applied to K = k_scale * decode(k_codes), V = v_scale * decode(v_codes), in fp64.
    q_bits [B,R,Hq,D] uint16 (bf16 bits); k_codes, v_codes [B,Hkv,Lmax,D] uint8; k_scale, v_scale [B,Hkv] float32.
    Returns (out [B,R,Hq,D] float64, lse [B,R,Hq] float64); ``units`` as in verify_attention."""
    lib = _load()
    q_bits = _c(q_bits, np.uint16)
    B, R, Hq, D = q_bits.shape
    assert R == gamma + 1
    k_codes = _c(k_codes, np.uint8)
    v_codes = _c(v_codes, np.uint8)
    _, Hkv, Lmax, Dk = k_codes.shape
    assert Dk == D and v_codes.shape == k_codes.shape and k_codes.shape[0] == B
    k_scale = _c(k_scale, np.float32).reshape(B, Hkv)
    v_scale = _c(v_scale, np.float32).reshape(B, Hkv)
    ctx_lens = _c(ctx_lens, np.int32)
    out = np.full((B, R, Hq, D), np.nan, dtype=np.float64)
    lse = np.full((B, R, Hq), np.nan, dtype=np.float64)
    n_units = 0
    if units is not None:
        units = _c(units, np.int64)
        n_units = units.size
    rc = lib.oracle_verify_attention_fp8(
        _ptr(q_bits), _ptr(k_codes), _ptr(v_codes), _ptr(k_scale), _ptr(v_scale), _ptr(ctx_lens), B, Hq, Hkv, D,
        Lmax, gamma, Hkv * Lmax * D, Lmax * D, D, float(scale), _ptr(units), n_units, _ptr(out), _ptr(lse))
    if rc != 0:
        raise ValueError(f"oracle_verify_attention_fp8 failed with {rc}")
    return out, lse


def rapid_distributions(z, d, T=1.0, eta=0.0, tail_alpha=0.1):
    """(p, q, phat_patched, phat_raw) for one draft position, all float64 [V]."""
    lib = _load()
    z = _c(z, np.float32)
    d = _c(d, np.float32)
    V = z.size
    assert d.size == V
    p = np.empty(V)
    q = np.empty(V)
    phat = np.empty(V)
    raw = np.empty(V)
    lib.oracle_rapid_distributions(_ptr(z), _ptr(d), V, float(T), float(eta), float(tail_alpha),
                                   _ptr(p), _ptr(q), _ptr(phat), _ptr(raw))
    return p, q, phat, raw


def residual_weights(p, q, phat, mode=RESIDUAL_PAPER):
    lib = _load()
    p = _c(p, np.float64)
    q = _c(q, np.float64)
    phat = _c(phat, np.float64)
    w = np.empty(p.size)
    lib.oracle_residual_weights(_ptr(p), _ptr(q), _ptr(phat), p.size, int(mode), _ptr(w))
    return w


def inverse_cdf(w, u) -> int:
    lib = _load()
    w = _c(w, np.float64)
    return int(lib.oracle_inverse_cdf(_ptr(w), w.size, float(u)))


def accept(target_logits, draft_logits, draft_tokens, uniforms, eta, T=1.0, tail_alpha=0.1,
           residual_mode=RESIDUAL_PAPER, want_ratios=True):
    """Algorithm 1's validation loop + residual draw.

    target_logits [B,gamma+1,V] f32, draft_logits [B,gamma,V] f32,
    draft_tokens [B,gamma] i32, uniforms [B,gamma+1] f32.
    Returns dict(accept_len [B] i32, next_token [B] i32, flags [B] i32,
    ratios [B,gamma] f64 or None).
    """
    lib = _load()
    z = _c(target_logits, np.float32)
    B, R, V = z.shape
    gamma = R - 1
    d = _c(draft_logits, np.float32).reshape(B, gamma, V)
    tok = _c(draft_tokens, np.int32).reshape(B, gamma)
    u = _c(uniforms, np.float32).reshape(B, R)
    accept_len = np.empty(B, dtype=np.int32)
    next_token = np.empty(B, dtype=np.int32)
    flags = np.empty(B, dtype=np.int32)
    ratios = np.full((B, gamma), np.nan) if want_ratios else None
    rc = lib.oracle_accept(_ptr(z), _ptr(d), _ptr(tok), _ptr(u), B, gamma, V, float(eta), float(T),
                           float(tail_alpha), int(residual_mode), _ptr(accept_len),
                           _ptr(next_token), _ptr(flags), _ptr(ratios))
    if rc != 0:
        raise ValueError(f"oracle_accept failed with {rc}")
    return dict(accept_len=accept_len, next_token=next_token, flags=flags, ratios=ratios)


def retrieval_select(chunk_emb, query_emb, k, threshold=0.3, n_chunks=None):
    """Section 2.3 / Section 3.1 ("RAG Setup"): cosine similarity of every chunk embedding with the
    query embedding; chunks scoring below the threshold are dropped, of the rest the k best are kept,
    best first (equal scores: lower index first).  fp64.  chunk_emb [B, N, Dm], query_emb [B, Dm].
    Returns (scores [B, N] (0 for a zero vector and past n_chunks[b]), list of B index lists)."""
    E = np.asarray(chunk_emb, dtype=np.float32).astype(np.float64)
    Q = np.asarray(query_emb, dtype=np.float32).astype(np.float64)
    B, N, _ = E.shape
    scores = np.zeros((B, N))
    chosen = []
    for b in range(B):
        n = N if n_chunks is None else int(n_chunks[b])
        qn = np.sqrt((Q[b] * Q[b]).sum())
        for i in range(n):
            den = np.sqrt((E[b, i] * E[b, i]).sum()) * qn
            scores[b, i] = (E[b, i] * Q[b]).sum() / den if den > 0 else 0.0
        order = sorted(range(n), key=lambda i: (-scores[b, i], i))
        chosen.append([i for i in order if scores[b, i] >= threshold][:k])
    return scores, chosen


def draft_sample(draft_logits, uniforms, T=1.0):
    """Algorithm 1, drafting loop: x' ~ q = softmax(d/T), drawn by the inverse-CDF rule with the given
    uniform.  fp64.  Returns (token [B] int32, log q(token) [B], row_stats [B,2] = (max d/T, log sum exp d/T))."""
    d = np.asarray(draft_logits, dtype=np.float32).astype(np.float64)
    B, V = d.shape
    tok = np.zeros(B, np.int32)
    logq = np.zeros(B)
    stats = np.zeros((B, 2))
    for b in range(B):
        x = d[b] / float(T)
        m = x.max()
        e = np.exp(x - m)
        S = e.sum()
        tok[b] = inverse_cdf(e / S, float(np.float32(uniforms[b])))
        stats[b] = (m, m + np.log(S))
        logq[b] = x[tok[b]] - stats[b, 1]
    return tok, logq, stats


def merge_partials(o_parts, lse_parts):
    """Attention over a union of disjoint key sets from the attentions over each set: with
    Z_p = sum_j exp(s_j) over set p (lse_p = log Z_p) and o_p = sum_j exp(s_j) v_j / Z_p,
    the result over the union is sum_p Z_p o_p / sum_p Z_p.  fp64; o_parts [P, ..., D], lse_parts [P, ...].
    A set without keys has lse = -inf and takes no part.  Returns (out [..., D], lse [...])."""
    o = np.asarray(o_parts, dtype=np.float64)
    l = np.asarray(lse_parts, dtype=np.float64)
    M = l.max(axis=0)
    safe = np.where(np.isfinite(M), M, 0.0)
    w = np.exp(l - safe)                      # exp(-inf) = 0 drops the empty sets
    den = w.sum(axis=0)
    num = (w[..., None] * np.where(w[..., None] > 0, o, 0.0)).sum(axis=0)
    with np.errstate(divide="ignore", invalid="ignore"):
        out = np.where(den[..., None] > 0, num / den[..., None], 0.0)
        lse = np.where(den > 0, safe + np.log(den), -np.inf)
    return out, lse


def paged_gather(pool, block_table, ctx_lens):
    """A paged cache written out as the contiguous cache it stands for (storage only; the paper's
    attention is defined on the logical sequence): pool [num_blocks, Hkv, block_size, D],
    block_table [B, max_blocks] -> cache [B, Hkv, max_blocks * block_size, D], where logical key j
    of sequence b is pool[block_table[b, j // block_size], :, j % block_size, :].  Only the
    ctx_lens[b] keys a sequence holds are looked up; the rest of its rows stay zero."""
    pool = np.asarray(pool)
    table = np.asarray(block_table)
    nb, Hkv, bs, D = pool.shape
    B, mb = table.shape
    out = np.zeros((B, Hkv, mb * bs, D), dtype=pool.dtype)
    for b in range(B):
        for j in range(int(ctx_lens[b])):
            blk = int(table[b, j // bs])
            if not 0 <= blk < nb:
                raise ValueError(f"block table entry {blk} of sequence {b} outside the pool")
            out[b, :, j, :] = pool[blk, :, j % bs, :]
    return out


def kv_append(k_cache, v_cache, k_new, v_new, ctx_lens, gamma):
    """Bookkeeping before a verify step (Algorithm 1: the last accepted token and the gamma drafts join
    the sequence the target scores): rows [L_b, L_b + R) of sequence b take k_new[b] / v_new[b]
    ([B, R, Hkv, D] -> cache [B, Hkv, Lmax, D]) and L_b grows by R = gamma + 1.  A sequence without
    room for R rows is left as it is.  Works on copies; returns (k_cache, v_cache, ctx_lens, overflowed)."""
    k_cache = np.array(k_cache, copy=True)
    v_cache = np.array(v_cache, copy=True)
    ctx = np.array(ctx_lens, dtype=np.int64, copy=True)
    R = gamma + 1
    Lmax = k_cache.shape[2]
    overflowed = False
    for b in range(k_cache.shape[0]):
        L = int(ctx[b])
        if L < 0 or L + R > Lmax:
            overflowed = True
            continue
        for i in range(R):
            for h in range(k_cache.shape[1]):
                k_cache[b, h, L + i, :] = k_new[b, i, h, :]
                v_cache[b, h, L + i, :] = v_new[b, i, h, :]
        ctx[b] = L + R
    return k_cache, v_cache, ctx.astype(np.int32), overflowed


def kv_append_paged(k_pool, v_pool, block_table, k_new, v_new, ctx_lens, gamma):
    """kv_append for a paged cache: the row for position j of sequence b goes to
    pool[block_table[b, j // block_size], :, j % block_size, :].  A sequence without room for R rows
    (capacity = max_blocks * block_size) is left as it is; a position whose table entry is not a
    block of the pool is skipped.  Works on copies; returns (k_pool, v_pool, ctx_lens, overflowed, bad_table)."""
    k_pool = np.array(k_pool, copy=True)
    v_pool = np.array(v_pool, copy=True)
    table = np.asarray(block_table)
    ctx = np.array(ctx_lens, dtype=np.int64, copy=True)
    R = gamma + 1
    nb, Hkv, bs, _ = k_pool.shape
    cap = table.shape[1] * bs
    overflowed = bad_table = False
    for b in range(table.shape[0]):
        L = int(ctx[b])
        if L < 0 or L + R > cap:
            overflowed = True
            continue
        for i in range(R):
            blk = int(table[b, (L + i) // bs])
            if not 0 <= blk < nb:
                bad_table = True
                continue
            for h in range(Hkv):
                k_pool[blk, h, (L + i) % bs, :] = k_new[b, i, h, :]
                v_pool[blk, h, (L + i) % bs, :] = v_new[b, i, h, :]
        ctx[b] = L + R
    return k_pool, v_pool, ctx.astype(np.int32), overflowed, bad_table


def step_commit(ctx_lens, accept_len, gamma):
    """Bookkeeping after a verify step (Algorithm 1: x_j <- x'_j for the accepted drafts, the others are
    discarded): the cache keeps the last accepted token and the accepted drafts, L_b -= gamma - n_b."""
    ctx = np.array(ctx_lens, dtype=np.int64, copy=True)
    for b in range(ctx.size):
        n = min(max(int(accept_len[b]), 0), gamma)
        ctx[b] -= gamma - n
    return ctx.astype(np.int32)
