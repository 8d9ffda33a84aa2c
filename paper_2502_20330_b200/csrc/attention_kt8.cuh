// Split-KV verify attention over an FP8 (E4M3) KV cache, keys on the M axis of the MMAs.
//
// Same decomposition, pipeline and partial format as the bf16 keys-on-M kernel (attention_kt.cuh: read
// that first); what differs is the arithmetic the 8-bit cache forces.  tcgen05.mma.kind::f8f6f4 takes
// both operands in 8 bits, so the two operands the cache does not supply are split in two E4M3 parts
// each, hi + lo on one scale, and every product is issued twice into the same accumulator:
//
//   S^T[128 keys x N] = K_tile Qhi^T + K_tile Qlo^T        Q rows scaled by a power of two per row so
//                                                           that |q| < 256; hi = E4M3(q), lo = E4M3(q - hi)
//   O^T[D x N]       += V_tile^T Phi^T + V_tile^T Plo^T     probabilities taken against a reference kept
//                                                           4..12 (log2) below the running maximum, so
//                                                           that 2^-9 <= p' <= 256 where it matters
// hi + lo carries 8 significant bits (what bf16 carries), and what falls below E4M3's subnormals is
// below 2^-17 of the row's largest entry.  The codes of K and V are exact; their fp32 scales (one per
// sequence and KV head each) multiply the scores' constant and the partial's O.
//
// A tile is 128 keys x 128 bytes = 16 KB for K and for V (one TMA box each), so a CTA streams twice
// the keys per byte: four K slots, six V slots.  Per (key, row) a softmax thread spends one FMA, one
// compare, one exponential, one add into the row sum, and the split: hi by integer rounding of the
// fp32 bits to 3 mantissa bits (the code falls out of the same bits), lo by the hardware conversion of
// the remainder, two columns at a time.
//
// Q is quantised in the kernel: at the start of a unit thread r of the first softmax group reads its
// grouped row of bf16 Q, finds the row's scale, and writes the row's hi and lo codes into the two
// K-major Q operands in shared memory (128-byte swizzle by hand), and the row's constant
// scale * log2(e) * k_scale / 2^s to shared memory.
#pragma once

#include <cuda_fp16.h>

namespace kt8 {

using kt::bar_softmax;
using kt::bar_softmax_or;
using kt::warp_max32;
using kt::warp_sum32;

// Barrier of all softmax threads (one group: its own barrier; two groups: a third one over both).
template <int SG>
__device__ __forceinline__ void bar_softmax_all() {
    if (SG == 1) asm volatile("bar.sync 1, 128;" ::: "memory");
    else asm volatile("bar.sync 3, 256;" ::: "memory");
}

constexpr int kKeys = 128;           // keys per tile
constexpr int kBlk = kKeys * 128;    // bytes of one tile: 128 keys x 128 E4M3 codes
constexpr int kNK = 4, kNV = 6;      // K and V slots
constexpr float kShift = 4.f;        // a new reference sits this far (log2) below the maximum it was taken from
constexpr float kJump = 8.f;         // a score this far above the reference (p' > 256) moves it
__host__ __device__ constexpr int threads(int SG) { return 128 * SG + 96; }
__host__ __device__ constexpr int smem_bytes(int NC) {
    // K ring + V ring + Q hi, lo (N rows of 128 bytes each) + P^T hi, lo (128 keys x 128 bytes each)
    return (kNK + kNV) * kBlk + 2 * (NC * 16) * 128 + 2 * kBlk + 1024;
}

// D[tmem] (+)= A[smem] * B[smem], both operands E4M3; issued by one thread.
__device__ __forceinline__ void umma_e4m3_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                             uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Instruction descriptor of kind::f8f6f4 with E4M3 A and B (format code 0) and fp32 accumulation:
// the bit fields of umma_idesc_bf16 with the two operand formats cleared.
__host__ __device__ constexpr uint32_t umma_idesc_e4m3(int M, int N, int a_mn_major, int b_mn_major) {
    return (1u << 4) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(N >> 3) << 17) |
           ((uint32_t)(M >> 4) << 24);
}
// Two fp32 -> two E4M3 codes (round to nearest even, saturating), `hi` in bits 8..15, `lo` in bits 0..7.
__device__ __forceinline__ uint32_t cvt_e4m3x2(float hi, float lo) {
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}
// Two E4M3 codes (bits 0..15) -> their values.
__device__ __forceinline__ float2 e4m3x2_to_float2(uint32_t codes) {
    uint32_t h2;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"((uint16_t)codes));
    return __half22float2(*reinterpret_cast<__half2*>(&h2));
}
// A non-negative value below 448 as hi + rest: hi keeps 3 mantissa bits (an E4M3 normal, or 0 below
// 2^-6); returns hi's E4M3 code and leaves the remainder in `rest`.
__device__ __forceinline__ uint32_t split_hi(float v, float& rest) {
    uint32_t h = (__float_as_uint(v) + 0x00080000u) & 0xFFF00000u;
    h = v >= 0.015625f ? h : 0u;
    rest = v - __uint_as_float(h);
    return h ? ((h >> 20) - 960u) & 0x7Fu : 0u;
}

template <int NC, int SG = 1>
__global__ void __launch_bounds__(threads(SG), 1)
verify_attn_splitkv_kt8_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                               const __grid_constant__ AttnArgs a) {
    constexpr int D = 128;
    constexpr int N = NC * 16;
    constexpr int NG = N / SG;  // columns per softmax group
    constexpr int WS = 4 * SG;  // softmax warps; the role warps follow
    static_assert(NG % 16 == 0 && NG <= 48, "a group's columns are whole 16-byte chunks of a P^T row, held as fp32");
    constexpr int NK = kNK, NV = kNV;
    constexpr uint32_t TMEM_COLS = 512;
    constexpr uint32_t COL_S = 0;    // S^T buffer b at COL_S + 128 b
    constexpr uint32_t COL_O = 256;  // O^T: N columns
    constexpr uint32_t OFF_K = 0, OFF_V = NK * kBlk, OFF_QH = (NK + NV) * kBlk, OFF_QL = OFF_QH + N * 128,
                       OFF_PH = OFF_QL + N * 128, OFF_PL = OFF_PH + kBlk;

    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t k_full[NK], k_empty[NK], v_full[NV], v_empty[NV];
    __shared__ uint64_t s_full[2], p_full[2];
    __shared__ uint64_t q_full;
    __shared__ uint64_t drain_bar[2];
    __shared__ uint32_t tmem_slot;
    __shared__ Walk s_walk;
    __shared__ int s_abort;
    __shared__ __align__(16) float sh_mref[128], sh_fac[128], sh_c[128], sh_w[4][128];

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    const int cta = blockIdx.x;

    if (tid == 0) {
        for (int s = 0; s < NK; ++s) {
            mbar_init(&k_full[s], 1);
            mbar_init(&k_empty[s], 1);
        }
        for (int s = 0; s < NV; ++s) {
            mbar_init(&v_full[s], 1);
            mbar_init(&v_empty[s], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&s_full[i], 1);
            mbar_init(&p_full[i], WS);
            mbar_init(&drain_bar[i], 1);
        }
        mbar_init(&q_full, 4);  // the four warps of the first softmax group
        fence_mbar_init();
        s_abort = 0;
        prefetch_tensormap(&tmK);
        prefetch_tensormap(&tmV);
    }
    if (warp == WS + 1) tmem_alloc(&tmem_slot, TMEM_COLS);  // the same warp frees it at the end
    // The rows of both Q operands past the grouped rows are never written: zero them once (scores 0).
    {
        const int pad_chunks = (N - a.GR) * 8;  // 16-byte chunks per operand
        for (int i = tid; i < 2 * pad_chunks; i += threads(SG)) {
            const int h = i >= pad_chunks, k16 = h ? i - pad_chunks : i;
            *reinterpret_cast<uint4*>(smem_gen + (h ? OFF_QL : OFF_QH) + a.GR * 128 + k16 * 16) = make_uint4(0, 0, 0, 0);
        }
        fence_proxy_async_smem();
    }
    Walk w;
    split_kernel_walk(a, cta, 1, w, &s_walk);
    if (cta == 0 && warp == WS && lane == 1) check_call_inputs(a, 1);
    const uint32_t tmem_base = tmem_slot;
    const WaitCtx wc = {&s_abort, a.wait_limit};

    if (warp == WS) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            int jj = 0, n_k = 0, n_v = 0;
            bool ok = true;
            while (w.remaining > 0 && ok) {
                const int seg = (int)min((long long)(w.ntiles - w.tile), w.remaining);
                for (int t = 0; t < seg && ok; ++t, ++jj) {
                    const int ks = jj % NK, vs = jj % NV;
                    const int key0 = (w.tile + t) * kKeys;
                    if (jj >= NK) ok = mbar_wait_bounded_relaxed(&k_empty[ks], ((jj / NK) - 1) & 1, wc);
                    if (!ok) break;
                    mbar_arrive_expect_tx(&k_full[ks], kBlk);
                    tma_load_4d(smem_gen + OFF_K + ks * kBlk, &tmK, &k_full[ks], 0, key0, w.kvh, w.b);
                    ++n_k;
                    if (jj >= NV) ok = mbar_wait_bounded_relaxed(&v_empty[vs], ((jj / NV) - 1) & 1, wc);
                    if (!ok) break;
                    mbar_arrive_expect_tx(&v_full[vs], kBlk);
                    tma_load_4d(smem_gen + OFF_V + vs * kBlk, &tmV, &v_full[vs], 0, key0, w.kvh, w.b);
                    ++n_v;
                }
                walk_advance(a, w, seg);
            }
            if (!ok) {  // leaving early: the copies already issued must land first
                for (int s = 0; s < NK && s < n_k; ++s)
                    mbar_wait_drain(&k_full[s], ((s + (n_k - 1 - s) / NK * NK) / NK) & 1);
                for (int s = 0; s < NV && s < n_v; ++s)
                    mbar_wait_drain(&v_full[s], ((s + (n_v - 1 - s) / NV * NV) / NV) & 1);
            }
        }
    } else if (warp == WS + 1) {
        // ---------------- QK^T issuer: S^T = K Qhi^T + K Qlo^T ----------------
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_e4m3(128, N, 0, 0);
            const uint64_t k_desc = umma_smem_desc(smem_base + OFF_K, 16, 1024);
            const uint64_t qh_desc = umma_smem_desc(smem_base + OFF_QH, 16, 1024);
            const uint64_t ql_desc = umma_smem_desc(smem_base + OFF_QL, 16, 1024);
            bool ok = true;
            int jj = 0, seg_idx = 0;
            while (w.remaining > 0 && ok) {
                const int seg = (int)min((long long)(w.ntiles - w.tile), w.remaining);
                // the unit's Q codes are in shared memory (written by the softmax threads, which have
                // read the previous unit out of tensor memory by then: all of its MMAs are complete)
                ok = mbar_wait_bounded(&q_full, seg_idx & 1, wc);
                for (int t = 0; t < seg && ok; ++t, ++jj) {
                    const int s = jj % NK, b = jj & 1;
                    ok = mbar_wait_bounded(&k_full[s], (jj / NK) & 1, wc);
                    if (ok && jj >= 2) ok = mbar_wait_bounded(&p_full[b], ((jj - 2) >> 1) & 1, wc);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t d = tmem_base + COL_S + 128u * b;
#pragma unroll
                    for (int kk = 0; kk < D / 32; ++kk) {  // 32 codes of the head dimension per MMA
                        const uint64_t ka = k_desc + (s * kBlk >> 4) + 2 * kk;
                        umma_e4m3_ss(d, ka, qh_desc + 2 * kk, idesc, kk > 0);
                        umma_e4m3_ss(d, ka, ql_desc + 2 * kk, idesc, 1u);
                    }
                    umma_commit(&s_full[b]);
                    umma_commit(&k_empty[s]);
                }
                walk_advance(a, w, seg);
                ++seg_idx;
            }
            if (!ok) {
                umma_commit(&drain_bar[0]);
                mbar_wait_drain(&drain_bar[0], 0);
            }
        }
    } else if (warp == WS + 2) {
        // ---------------- PV issuer: O^T += V^T Phi^T + V^T Plo^T ----------------
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_e4m3(D, N, 1, 1);
            // MN-major operands: one 128-byte row per key (128 codes along M resp. N), 8-key groups 1024 bytes apart
            const uint64_t v_desc = umma_smem_desc(smem_base + OFF_V, kBlk, 1024);
            const uint64_t ph_desc = umma_smem_desc(smem_base + OFF_PH, kBlk, 1024);
            const uint64_t pl_desc = umma_smem_desc(smem_base + OFF_PL, kBlk, 1024);
            const uint32_t d = tmem_base + COL_O;
            bool ok = true;
            int jj = 0;
            while (w.remaining > 0 && ok) {
                const int seg = (int)min((long long)(w.ntiles - w.tile), w.remaining);
                for (int t = 0; t < seg && ok; ++t, ++jj) {
                    const int s = jj % NV;
                    ok = mbar_wait_bounded(&p_full[jj & 1], (jj >> 1) & 1, wc);
                    if (ok) ok = mbar_wait_bounded(&v_full[s], (jj / NV) & 1, wc);
                    if (!ok) break;
                    tc_fence_after_sync();
#pragma unroll
                    for (int kk = 0; kk < kKeys / 32; ++kk) {  // 32 keys per MMA
                        const uint64_t va = v_desc + (s * kBlk >> 4) + kk * (4096 >> 4);
                        umma_e4m3_ss(d, va, ph_desc + kk * (4096 >> 4), idesc, (t > 0 || kk > 0) ? 1u : 0u);
                        umma_e4m3_ss(d, va, pl_desc + kk * (4096 >> 4), idesc, 1u);
                    }
                    umma_commit(&v_empty[s]);
                }
                walk_advance(a, w, seg);
            }
            if (!ok) {
                umma_commit(&drain_bar[1]);
                mbar_wait_drain(&drain_bar[1], 0);
            }
        }
    } else if (warp < WS) {
        // ---------------- softmax: thread t of group grp = key t of the tile = TMEM lane t ----------------
        const int grp = warp >> 2, wq = warp & 3;
        const int t = tid & 127;
        const int C0 = grp * NG;  // this group's first column
        const uint32_t lane_base = (uint32_t)(wq * 32) << 16;
        const uint32_t tO = tmem_base + lane_base + COL_O + C0;
        const int slot_stride = (int)slot_floats(a.GR, D);
        uint8_t* ph_gen = smem_gen + OFF_PH + t * 128;  // this key's rows of P^T hi and lo
        uint8_t* pl_gen = smem_gen + OFF_PL + t * 128;
        const int p_swz = t & 7;

        float lsum[NG];
        int jj = 0;
        bool ok = true;  // only records that a wait ran out: these warps run their loops to the end
        while (w.remaining > 0) {
            const int seg = (int)min((long long)(w.ntiles - w.tile), w.remaining);
            const int L = w.L;
            // ---- the unit's Q: row t of the first group, quantised to hi + lo codes on the row's own scale ----
            if (grp == 0) {
                if (t < a.GR) {
                    const int i = t / a.G, g = t % a.G;
                    const uint4* src = reinterpret_cast<const uint4*>(
                        a.q + (((size_t)w.b * a.R + i) * a.Hq + (size_t)w.kvh * a.G + g) * D);
                    uint4 raw[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) raw[j] = __ldg(src + j);
                    float amax = 0.f;
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const uint32_t u[4] = {raw[j].x, raw[j].y, raw[j].z, raw[j].w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            amax = fmaxf(amax, fabsf(__uint_as_float(u[e] << 16)));
                            amax = fmaxf(amax, fabsf(__uint_as_float(u[e] & 0xffff0000u)));
                        }
                    }
                    // 2^s with 128 <= amax * 2^s < 256 (s clamped to what fp32 holds; a zero row: 2^0)
                    int s2 = amax > 0.f ? 7 - ((int)((__float_as_uint(amax) >> 23) & 0xff) - 127) : 0;
                    s2 = s2 > 126 ? 126 : (s2 < -126 ? -126 : s2);
                    const float up = __uint_as_float((uint32_t)(s2 + 127) << 23), down = __uint_as_float((uint32_t)(127 - s2) << 23);
                    sh_c[t] = a.scale_log2 * __ldg(a.k_scale + (size_t)w.b * a.Hkv + w.kvh) * down;
                    uint8_t* qh = smem_gen + OFF_QH + t * 128;
                    uint8_t* ql = smem_gen + OFF_QL + t * 128;
#pragma unroll
                    for (int j2 = 0; j2 < 8; ++j2) {  // 16 codes = one 16-byte chunk = two loads of 8 bf16
                        uint32_t hw[4], lw[4];
#pragma unroll
                        for (int half = 0; half < 2; ++half) {
                            const uint4 r = raw[2 * j2 + half];
                            const uint32_t u[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
                            for (int e = 0; e < 4; e += 2) {
                                const float x0 = __uint_as_float(u[e] << 16) * up, x1 = __uint_as_float(u[e] & 0xffff0000u) * up;
                                const float x2 = __uint_as_float(u[e + 1] << 16) * up, x3 = __uint_as_float(u[e + 1] & 0xffff0000u) * up;
                                const uint32_t h01 = cvt_e4m3x2(x1, x0), h23 = cvt_e4m3x2(x3, x2);
                                const float2 d01 = e4m3x2_to_float2(h01), d23 = e4m3x2_to_float2(h23);
                                const uint32_t l01 = cvt_e4m3x2(x1 - d01.y, x0 - d01.x), l23 = cvt_e4m3x2(x3 - d23.y, x2 - d23.x);
                                hw[2 * half + (e >> 1)] = h01 | (h23 << 16);
                                lw[2 * half + (e >> 1)] = l01 | (l23 << 16);
                            }
                        }
                        const int off = ((j2 ^ (t & 7)) << 4);
                        *reinterpret_cast<uint4*>(qh + off) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
                        *reinterpret_cast<uint4*>(ql + off) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
                    }
                } else if (t < N) {
                    sh_c[t] = 0.f;
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(&q_full);
            }
            bar_softmax_all<SG>();  // sh_c is read by every softmax thread
#pragma unroll
            for (int i = 0; i < NG; ++i) lsum[i] = 0.f;

            for (int ti = 0; ti < seg; ++ti, ++jj) {
                const int b = jj & 1;
                const uint32_t tS = tmem_base + lane_base + COL_S + 128u * b + C0;
                const int key0 = (w.tile + ti) * kKeys;
                const int key = key0 + t;
                // the columns the causal stair hides from this key are a prefix [0, cmin)
                const int over_ctx = a.stair ? key - (L - a.R) : 0;
                const int cmin = key >= L ? N : (over_ctx > 0 ? over_ctx * a.G : 0);
                ok &= warp_wait_bounded(&s_full[b], (jj >> 1) & 1, wc);
                tc_fence_after_sync();

                float pv[NG];
                bool move = ti == 0;
                if (ti > 0) {
                    bool far = false;
#pragma unroll
                    for (int ch = 0; ch < NG / 16; ++ch) {
                        uint32_t sr[16];
                        tmem_ld_x16(tS + 16 * ch, sr);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < 16; e += 4) {
                            const int li = 16 * ch + e, col = C0 + li;
                            const float4 m = *reinterpret_cast<const float4*>(&sh_mref[col]);
                            const float4 cc = *reinterpret_cast<const float4*>(&sh_c[col]);
                            float x[4] = {fmaf(__uint_as_float(sr[e]), cc.x, -m.x), fmaf(__uint_as_float(sr[e + 1]), cc.y, -m.y),
                                          fmaf(__uint_as_float(sr[e + 2]), cc.z, -m.z), fmaf(__uint_as_float(sr[e + 3]), cc.w, -m.w)};
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                x[i] = col + i >= cmin ? x[i] : -INFINITY;
                                far |= x[i] > kJump;
                                pv[li + i] = fast_exp2(x[i]);
                            }
                        }
                    }
                    move = bar_softmax_or(grp, far);
                }
                if (jj >= 1) {  // PV of the previous tile is complete: P^T is free, O^T at rest
                    ok &= warp_wait_bounded(&v_empty[(jj - 1) % NV], ((jj - 1) / NV) & 1, wc);
                    tc_fence_after_sync();
                }
                if (move) {
                    // new reference = max(old, this tile's row maxima over the 128 keys - kShift)
#pragma unroll
                    for (int ch = 0; ch < NG / 16; ++ch) {
                        uint32_t sr[16];
                        tmem_ld_x16(tS + 16 * ch, sr);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < 16; ++e) {
                            const int col = C0 + 16 * ch + e;
                            const float v = (col >= cmin && col < a.GR) ? __uint_as_float(sr[e]) * sh_c[col] : -INFINITY;
                            const float wm = warp_max32(v);
                            if (lane == 0) sh_w[wq][col] = wm;
                        }
                    }
                    bar_softmax(grp);
                    if (t < NG) {
                        const int col = C0 + t;
                        const float old = ti == 0 ? -INFINITY : sh_mref[col];
                        const float tile_max = fmaxf(fmaxf(sh_w[0][col], sh_w[1][col]), fmaxf(sh_w[2][col], sh_w[3][col]));
                        const float nm = fmaxf(old, tile_max - kShift);  // -inf - 4 = -inf: a row that has seen no key yet
                        const bool pad = col >= a.GR;
                        sh_fac[col] = (pad || nm == old) ? 1.f : fast_exp2(old - nm);
                        sh_mref[col] = pad ? INFINITY : nm;
                    }
                    bar_softmax(grp);
                    if (ti > 0) {
#pragma unroll
                        for (int i = 0; i < NG; ++i) lsum[i] *= sh_fac[C0 + i];
#pragma unroll
                        for (int ch = 0; ch < NG / 16; ++ch) {
                            uint32_t orow[16];
                            tmem_ld_x16(tO + 16 * ch, orow);
                            tmem_wait_ld();
#pragma unroll
                            for (int e = 0; e < 16; ++e)
                                orow[e] = __float_as_uint(__uint_as_float(orow[e]) * sh_fac[C0 + 16 * ch + e]);
                            tmem_st_x16(tO + 16 * ch, orow);
                        }
                        tmem_wait_st();
                    }
#pragma unroll
                    for (int ch = 0; ch < NG / 16; ++ch) {
                        uint32_t sr[16];
                        tmem_ld_x16(tS + 16 * ch, sr);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < 16; ++e) {
                            const int li = 16 * ch + e, col = C0 + li;
                            const float m0 = sh_mref[col];
                            const float x0 = col >= cmin
                                                 ? fmaf(__uint_as_float(sr[e]), sh_c[col], m0 == -INFINITY ? 0.f : -m0)
                                                 : -INFINITY;
                            pv[li] = fast_exp2(x0);
                        }
                    }
                }
                // this key's rows of P^T: every probability as hi + lo codes, 16 columns per 16-byte chunk
#pragma unroll
                for (int c16 = 0; c16 < NG / 16; ++c16) {
                    uint32_t hw[4], lw[4];
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        float r0, r1, r2, r3;
                        const int o = 16 * c16 + 4 * q4;
                        const uint32_t h0 = split_hi(pv[o], r0), h1 = split_hi(pv[o + 1], r1), h2 = split_hi(pv[o + 2], r2),
                                       h3 = split_hi(pv[o + 3], r3);
                        hw[q4] = h0 | (h1 << 8) | (h2 << 16) | (h3 << 24);
                        lw[q4] = cvt_e4m3x2(r1, r0) | (cvt_e4m3x2(r3, r2) << 16);
                        lsum[o] += pv[o];
                        lsum[o + 1] += pv[o + 1];
                        lsum[o + 2] += pv[o + 2];
                        lsum[o + 3] += pv[o + 3];
                    }
                    const int g16 = C0 / 16 + c16;  // the chunk's place in the row
                    const int off = ((g16 ^ p_swz) << 4);
                    *reinterpret_cast<uint4*>(ph_gen + off) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
                    *reinterpret_cast<uint4*>(pl_gen + off) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
                }
                if (grp == 0 && key0 + kKeys > L) {
                    // V rows beyond the context may hold any codes (NaN among them): zero them so that 0 * row = 0
                    ok &= warp_wait_bounded(&v_full[jj % NV], (jj / NV) & 1, wc);
                    const int first_bad = max(L - key0, 0);
                    const int chunks = (kKeys - first_bad) * 8;
                    uint8_t* vgen = smem_gen + OFF_V + (jj % NV) * kBlk;
                    for (int chk = t; chk < chunks; chk += 128)
                        *reinterpret_cast<uint4*>(vgen + first_bad * 128 + chk * 16) = make_uint4(0, 0, 0, 0);
                }
                fence_proxy_async_smem();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&p_full[b]);
            }

            // ---- end of the unit: O^T out of tensor memory (times the V scale), row sums, partial ----
            ok &= warp_wait_bounded(&v_empty[(jj - 1) % NV], ((jj - 1) / NV) & 1, wc);
            tc_fence_after_sync();
            const int unit = w.b * a.Hkv + w.kvh;
            const float vs = __ldg(a.v_scale + unit);
            float* slot = a.partial + (size_t)(cta + unit) * slot_stride;
#pragma unroll
            for (int ch = 0; ch < NG / 16; ++ch) {
                uint32_t orow[16];
                tmem_ld_x16(tO + 16 * ch, orow);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                    const int col = C0 + 16 * ch + e;
                    if (col < a.GR && sh_mref[col] != -INFINITY) slot[(size_t)col * D + t] = __uint_as_float(orow[e]) * vs;
                }
            }
#pragma unroll
            for (int i = 0; i < NG; ++i) {
                const float ws = warp_sum32(lsum[i]);
                if (lane == 0) sh_w[wq][C0 + i] = ws;
            }
            bar_softmax(grp);
            if (t < NG && C0 + t < a.GR) {
                const int col = C0 + t;
                slot[a.GR * D + col] = sh_mref[col];
                slot[a.GR * D + a.GR + col] = ((sh_w[0][col] + sh_w[1][col]) + sh_w[2][col]) + sh_w[3][col];
            }
            bar_softmax_all<SG>();  // sh_w / sh_mref / sh_c are reused by the next unit
            walk_advance(a, w, seg);
        }
        (void)ok;
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == WS + 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
    if (tid == 0 && s_abort) atomicOr(a.status, RAPID_STATUS_PIPELINE_TIMEOUT);
}

}  // namespace kt8
