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

using kt::warp_max32;
using kt::warp_sum32;

// Named barriers: one per softmax group of 128 threads (ids 1 .. SG), one over all groups (id 15).
__device__ __forceinline__ void bar_softmax(int grp) {
    asm volatile("bar.sync %0, 128;" ::"r"(grp + 1) : "memory");
}
__device__ __forceinline__ bool bar_softmax_or(int grp, bool flag) {
    uint32_t res;
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.b32 q, %2, 0;\n\tbar.red.or.pred p, %1, 128, q;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(res)
                 : "r"(grp + 1), "r"((uint32_t)flag)
                 : "memory");
    return res != 0;
}
template <int SG>
__device__ __forceinline__ void bar_softmax_all() {
    asm volatile("bar.sync 15, %0;" ::"n"(128 * SG) : "memory");
}

constexpr int kKeys = 128;           // keys per tile
constexpr int kBlk = kKeys * 128;    // bytes of one tile: 128 keys x 128 E4M3 codes
constexpr int kNK = 4, kNV = 6;      // K and V slots
constexpr float kShift = 4.f;        // a new reference sits this far (log2) below the maximum it was taken from
constexpr float kJump = 8.f;         // a score this far above the reference (p' > 256) moves it
// Columns per softmax group.  (The kernel also runs with 8: six groups at 48 columns measured 75 us per
// 8B-128K layer against 68 us for three groups of 16 -- every group pays its own waits and barriers per
// tile, and the schedulers' issue slots, 47 % busy with three groups, are what runs out.)
__host__ __device__ constexpr int group_cols(int NC) { return 16; }
__host__ __device__ constexpr int threads(int NC) { return 128 * (NC * 16 / group_cols(NC)) + 96; }  // + three role warps
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
// Two values as hi + lo E4M3 pairs: hi = E4M3(v) by the hardware conversion, the remainders formed in
// packed half precision (v < 448 and its remainder need far fewer than half's 11 bits) and converted
// the same way.  v0's codes go to the low bytes of hi and lo.
__device__ __forceinline__ uint32_t split_e4m3x2(float v0, float v1, uint32_t& lo) {
    uint16_t h;
    uint32_t hf2, vf2, rf2;
    uint16_t l;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(h) : "f"(v1), "f"(v0));
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(hf2) : "h"(h));
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(vf2) : "f"(v1), "f"(v0));
    asm("sub.rn.f16x2 %0, %1, %2;" : "=r"(rf2) : "r"(vf2), "r"(hf2));
    asm("cvt.rn.satfinite.e4m3x2.f16x2 %0, %1;" : "=h"(l) : "r"(rf2));
    lo = l;
    return h;
}

__device__ __forceinline__ void split_e4m3x4(float v0, float v1, float v2, float v3, uint32_t& hi, uint32_t& lo) {
    uint32_t l01, l23;
    const uint32_t h01 = split_e4m3x2(v0, v1, l01), h23 = split_e4m3x2(v2, v3, l23);
    hi = h01 | (h23 << 16);
    lo = l01 | (l23 << 16);
}
// NC = N / 16 column chunks.  There are SG = N / NG softmax groups of 128 threads each (thread t of
// every group is key t of the tile): a group forms the probabilities of its own NG = 8 or 16 columns --
// half or all of a 16-byte chunk of the key's P^T hi row, and of its lo row -- and keeps those rows'
// references and sums.  What a tile costs is the time ONE warp takes over its 32 keys x NG columns
// (some 8 cycles per instruction: a latency chain, not an issue limit), and this cache delivers
// twice the keys per byte: narrow groups, several warps per scheduler, keep that chain short.
template <int NC>
__global__ void __launch_bounds__(threads(NC), 1)
verify_attn_splitkv_kt8_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                               const __grid_constant__ AttnArgs a) {
    constexpr int D = 128;
    constexpr int N = NC * 16;
    constexpr int NG = group_cols(NC);  // columns per softmax group
    constexpr int SG = N / NG;          // softmax groups
    constexpr int WS = 4 * SG;          // softmax warps; the role warps follow
    static_assert(SG <= 6, "named barriers 1..6 and 1024 threads at most");
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
        mbar_init(&q_full, WS);  // every softmax warp
        fence_mbar_init();
        s_abort = 0;
        prefetch_tensormap(&tmK);
        prefetch_tensormap(&tmV);
    }
    if (warp == WS + 1) tmem_alloc(&tmem_slot, TMEM_COLS);  // the same warp frees it at the end
    // The rows of both Q operands past the grouped rows are never written: zero them once (scores 0).
    {
        const int pad_chunks = (N - a.GR) * 8;  // 16-byte chunks per operand
        for (int i = tid; i < 2 * pad_chunks; i += threads(NC)) {
            const int h = i >= pad_chunks, k16 = h ? i - pad_chunks : i;
            *reinterpret_cast<uint4*>(smem_gen + (h ? OFF_QL : OFF_QH) + a.GR * 128 + k16 * 16) = make_uint4(0, 0, 0, 0);
        }
        fence_proxy_async_smem();
    }
    Walk w;
    // The walk, the stream-order wait and, between the two, the first tiles' copies where the caller
    // vouches for the older part of the cache (see the bf16 keys-on-M kernel).
    const bool settled = a.plan_mode == RAPID_PLAN_SETTLED;
    if (settled) load_walk(a, cta, 1, w);
    tc_fence_before_sync();
    __syncthreads();  // barriers initialised, tensor memory allocated
    tc_fence_after_sync();
    int pre_k = 0, pre_v = 0;  // tiles whose K / V copies were issued before the wait (producer lane only)
    if (a.kv_settled && warp == WS && lane == 0 && w.remaining > 0) {
        const int seg0 = (int)min((long long)(w.ntiles - w.tile), w.remaining);
        const int old_tiles = (w.L - a.R) >> 7;  // tiles 0 .. old_tiles-1 hold none of the newest R keys
        const int n_early = seg0 > 2 * NV ? NV : NK;  // a short walk: no V tiles ahead of the K tiles it needs next
        for (int t = 0; t < seg0 && t < n_early && w.tile + t < old_tiles; ++t) {
            const int key0 = (w.tile + t) * kKeys;
            if (t < NK) {
                mbar_arrive_expect_tx(&k_full[t], kBlk);
                tma_load_4d(smem_gen + OFF_K + t * kBlk, &tmK, &k_full[t], 0, key0, w.kvh, w.b);
                ++pre_k;
            }
            mbar_arrive_expect_tx(&v_full[t], kBlk);
            tma_load_4d(smem_gen + OFF_V + t * kBlk, &tmV, &v_full[t], 0, key0, w.kvh, w.b);
            ++pre_v;
        }
    }
    griddep_wait();               // inputs are read from here on
    griddep_launch_dependents();  // the merge blocks may take their seats (after the wait: see split_kernel_walk)
    if (!settled) {
        if (threadIdx.x == 0) {
            Walk t;
            load_walk(a, cta, 1, t);
            s_walk = t;
        }
        __syncthreads();
        w = s_walk;
    }
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
                    if (jj >= pre_k) {  // (the first pre_k tiles' K copies went out before the wait)
                        if (jj >= NK) ok = mbar_wait_bounded_relaxed(&k_empty[ks], ((jj / NK) - 1) & 1, wc);
                        if (!ok) break;
                        mbar_arrive_expect_tx(&k_full[ks], kBlk);
                        tma_load_4d(smem_gen + OFF_K + ks * kBlk, &tmK, &k_full[ks], 0, key0, w.kvh, w.b);
                    }
                    ++n_k;
                    if (jj >= pre_v) {
                        if (jj >= NV) ok = mbar_wait_bounded_relaxed(&v_empty[vs], ((jj / NV) - 1) & 1, wc);
                        if (!ok) break;
                        mbar_arrive_expect_tx(&v_full[vs], kBlk);
                        tma_load_4d(smem_gen + OFF_V + vs * kBlk, &tmV, &v_full[vs], 0, key0, w.kvh, w.b);
                    }
                    ++n_v;
                }
                walk_advance(a, w, seg);
            }
            if (!ok) {  // leaving early: the copies already issued must land first
                n_k = max(n_k, pre_k);
                n_v = max(n_v, pre_v);
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
            // ---- the unit's Q, quantised to hi + lo codes on every row's own scale ----
            // softmax thread st takes 16 consecutive elements (one 16-byte chunk of codes) of grouped row
            // st / 8: the eight threads of a row find its largest magnitude with three shuffles
            {
                const int st = grp * 128 + t;
                const int row = st >> 3, j2 = st & 7;
                const bool has = row < a.GR;
                uint4 r0 = make_uint4(0, 0, 0, 0), r1 = r0;
                if (has) {
                    const int i = row / a.G, g = row % a.G;
                    const uint4* src = reinterpret_cast<const uint4*>(
                        a.q + (((size_t)w.b * a.R + i) * a.Hq + (size_t)w.kvh * a.G + g) * D) + 2 * j2;
                    r0 = __ldg(src);
                    r1 = __ldg(src + 1);
                }
                const uint32_t u[8] = {r0.x, r0.y, r0.z, r0.w, r1.x, r1.y, r1.z, r1.w};
                float amax = 0.f;
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    amax = fmaxf(amax, fabsf(__uint_as_float(u[e] << 16)));
                    amax = fmaxf(amax, fabsf(__uint_as_float(u[e] & 0xffff0000u)));
                }
#pragma unroll
                for (int o = 1; o < 8; o <<= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
                // 2^s with 128 <= amax * 2^s < 256 (s clamped to what fp32 holds; a zero row: 2^0)
                int s2 = amax > 0.f ? 7 - ((int)((__float_as_uint(amax) >> 23) & 0xff) - 127) : 0;
                s2 = s2 > 126 ? 126 : (s2 < -126 ? -126 : s2);
                const float up = __uint_as_float((uint32_t)(s2 + 127) << 23), down = __uint_as_float((uint32_t)(127 - s2) << 23);
                if (has) {
                    if (j2 == 0) sh_c[row] = a.scale_log2 * __ldg(a.k_scale + (size_t)w.b * a.Hkv + w.kvh) * down;
                    uint32_t hw[4], lw[4];
#pragma unroll
                    for (int e = 0; e < 8; e += 2)
                        split_e4m3x4(__uint_as_float(u[e] << 16) * up, __uint_as_float(u[e] & 0xffff0000u) * up,
                                     __uint_as_float(u[e + 1] << 16) * up, __uint_as_float(u[e + 1] & 0xffff0000u) * up,
                                     hw[e >> 1], lw[e >> 1]);
                    const int off = row * 128 + ((j2 ^ (row & 7)) << 4);
                    *reinterpret_cast<uint4*>(smem_gen + OFF_QH + off) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
                    *reinterpret_cast<uint4*>(smem_gen + OFF_QL + off) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
                } else if (j2 == 0 && row < N) {
                    sh_c[row] = 0.f;
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
                    float xmax = -INFINITY;
                    uint32_t sr[NG];
                    tmem_ld_cols<NG>(tS, sr);
                    tmem_wait_ld();
                    // a tile every row sees whole (all of a long context but its end) takes the loop
                    // without any mask; the two loops are separate code so that the common one carries
                    // no predicate at all
                    if (key0 + kKeys <= L - a.stair) {
#pragma unroll
                        for (int e = 0; e < NG; e += 4) {
                            const float4 m = *reinterpret_cast<const float4*>(&sh_mref[C0 + e]);
                            const float4 cc = *reinterpret_cast<const float4*>(&sh_c[C0 + e]);
                            const float x0 = fmaf(__uint_as_float(sr[e]), cc.x, -m.x), x1 = fmaf(__uint_as_float(sr[e + 1]), cc.y, -m.y);
                            const float x2 = fmaf(__uint_as_float(sr[e + 2]), cc.z, -m.z), x3 = fmaf(__uint_as_float(sr[e + 3]), cc.w, -m.w);
                            xmax = fmaxf(fmaxf(xmax, x0), fmaxf(fmaxf(x1, x2), x3));
                            pv[e] = fast_exp2(x0);
                            pv[e + 1] = fast_exp2(x1);
                            pv[e + 2] = fast_exp2(x2);
                            pv[e + 3] = fast_exp2(x3);
                        }
                    } else {
#pragma unroll
                        for (int e = 0; e < NG; e += 4) {
                            const int col = C0 + e;
                            const float4 m = *reinterpret_cast<const float4*>(&sh_mref[col]);
                            const float4 cc = *reinterpret_cast<const float4*>(&sh_c[col]);
                            float x[4] = {fmaf(__uint_as_float(sr[e]), cc.x, -m.x), fmaf(__uint_as_float(sr[e + 1]), cc.y, -m.y),
                                          fmaf(__uint_as_float(sr[e + 2]), cc.z, -m.z), fmaf(__uint_as_float(sr[e + 3]), cc.w, -m.w)};
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                x[i] = col + i >= cmin ? x[i] : -INFINITY;
                                xmax = fmaxf(xmax, x[i]);
                                pv[e + i] = fast_exp2(x[i]);
                            }
                        }
                    }
                    move = bar_softmax_or(grp, xmax > kJump);
                }
                if (jj >= 1) {  // PV of the previous tile is complete: P^T is free, O^T at rest
                    ok &= warp_wait_bounded(&v_empty[(jj - 1) % NV], ((jj - 1) / NV) & 1, wc);
                    tc_fence_after_sync();
                }
                if (move) {
                    // new reference = max(old, this tile's row maxima over the 128 keys - kShift)
                    {
                        uint32_t sr[NG];
                        tmem_ld_cols<NG>(tS, sr);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < NG; ++e) {
                            const int col = C0 + e;
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
                        {
                            uint32_t orow[NG];
                            tmem_ld_cols<NG>(tO, orow);
                            tmem_wait_ld();
#pragma unroll
                            for (int e = 0; e < NG; ++e)
                                orow[e] = __float_as_uint(__uint_as_float(orow[e]) * sh_fac[C0 + e]);
                            tmem_st_cols<NG>(tO, orow);
                        }
                        tmem_wait_st();
                    }
                    {
                        uint32_t sr[NG];
                        tmem_ld_cols<NG>(tS, sr);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < NG; ++e) {
                            const int col = C0 + e;
                            const float m0 = sh_mref[col];
                            const float x0 = col >= cmin
                                                 ? fmaf(__uint_as_float(sr[e]), sh_c[col], m0 == -INFINITY ? 0.f : -m0)
                                                 : -INFINITY;
                            pv[e] = fast_exp2(x0);
                        }
                    }
                }
                // this key's rows of P^T: every probability as hi + lo codes; the group's NG columns are
                // all or half of one 16-byte chunk of either row
                {
                    uint32_t hw[NG / 4], lw[NG / 4];
#pragma unroll
                    for (int q4 = 0; q4 < NG / 4; ++q4) {
                        const int o = 4 * q4;
                        split_e4m3x4(pv[o], pv[o + 1], pv[o + 2], pv[o + 3], hw[q4], lw[q4]);
                        lsum[o] += pv[o];
                        lsum[o + 1] += pv[o + 1];
                        lsum[o + 2] += pv[o + 2];
                        lsum[o + 3] += pv[o + 3];
                    }
                    if constexpr (NG == 16) {
                        const int off = ((grp ^ p_swz) << 4);
                        *reinterpret_cast<uint4*>(ph_gen + off) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
                        *reinterpret_cast<uint4*>(pl_gen + off) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
                    } else {
                        const int off = (((grp >> 1) ^ p_swz) << 4) + ((grp & 1) << 3);
                        *reinterpret_cast<uint2*>(ph_gen + off) = make_uint2(hw[0], hw[1]);
                        *reinterpret_cast<uint2*>(pl_gen + off) = make_uint2(lw[0], lw[1]);
                    }
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
            {
                uint32_t orow[NG];
                tmem_ld_cols<NG>(tO, orow);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < NG; ++e) {
                    const int col = C0 + e;
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
