// Split-KV verify attention with the KEYS on the M axis of the MMAs (head_dim 128, up to 96 grouped rows).
//
//   S^T[128 keys x N] = K_tile[128 x D] Q^T        A = K tile (K-major), B = Q (N grouped rows, K-major)
//   O^T[D x N]       += V_tile^T[D x 128] P^T      A = V tile (MN-major), B = P^T (MN-major, written by the
//                                                   softmax threads into shared memory)
// N = grouped rows padded to a multiple of 16.  One softmax thread per KEY (TMEM lane = key), so all
// 128 softmax threads work whatever the number of grouped rows is, one exponential per (key, row)
// that exists, and the tensor-core work is proportional to N instead of to a 64- or 128-row tile.
//
// A tile is 128 keys (one TMA box of 128 rows per 64-column half).  K tiles and V tiles live in
// rings of their own (two K slots, four V slots; three V slots for more than 48 rows): a K slot is
// free once QK^T of its tile has completed, a V slot only after PV.  Work split, partial format (one partial per CTA and unit) and merge are shared with the
// rows-on-M kernel.  Roles (224 threads): warps 0-3 softmax (thread t = key t of the tile), warp 4
// TMA producer, warp 5 TMEM allocation + Q load + QK^T issue, warp 6 PV issue.  Beyond 64 grouped
// rows there are two softmax groups (warps 0-3 and 4-7, 352 threads, the role warps after them):
// each takes half of the columns for all 128 keys.
//
// Columns past the grouped rows (N is a multiple of 16) are made harmless once instead of being
// tested per element: their rows of Q are zeroed at set-up (scores 0) and their reference is +inf
// (probabilities 0).  A tile that every row sees whole -- all of a long context but its end -- takes
// a loop without the per-column mask.
//
// P^T in shared memory has the layout of a V tile half: one 128-byte row per key holding that key's
// probabilities for 64 grouped rows, 128-byte swizzle (16-byte chunk index XOR key & 7), 8-key groups
// 1024 bytes apart.  A softmax thread writes its row with one 16-byte store per 8 grouped rows.
//
// Softmax reference.  As in the rows-on-M kernel the probabilities are taken against a reference
// m_ref[row] that need not be the running maximum.  It lives in shared memory (every key thread
// needs every row's value).  It is set from the unit's first tile (a maximum over the 128 key
// threads: warp shuffles, then the four warps through shared memory) and moved, with a rescale of
// the O^T columns and of the sums, when a tile holds a score more than 16 (log2 units) above it.
// That is found in the one pass that forms the probabilities (a block-wide OR per tile); only then
// are they formed again against the new references.  The row sums are kept per thread (its keys'
// share of every row) and added up at the end of a unit in a fixed order.
//
// Pipeline: S^T is double-buffered in tensor memory, so QK^T(n+1) runs during softmax(n); P^T is
// single-buffered, so the P^T stores of tile n wait for PV(n-1), the arithmetic before them does not.
//
// Barriers: every parity wait is on a barrier whose next phase cannot complete before the waiter has
// passed the current one (per-buffer s_full / p_full, per-stage full / empty; empty doubles as
// "the PV of this tile has completed").
//
// Waits that run out.  Every mbarrier wait is bounded.  The single-thread roles (producer, MMA
// issuers) leave their loops when a wait fails, after seeing their own asynchronous work land (the
// producer its bulk copies, the issuers their MMAs).  The softmax warps do NOT leave early: the
// four warps of a group meet at named barriers, which have no time limit, so a warp that left
// while another had seen its wait succeed would strand it there.  They run their loops to the end
// instead; once the abort flag is up every wait returns at once, so that is quick, and what they
// write is in bounds and flagged invalid by RAPID_STATUS_PIPELINE_TIMEOUT.
//
// One cluster per unit (AttnArgs::cmerge).  For calls whose whole run is short (a decode over a
// few thousand keys) the merge kernel and its two kernel boundaries cost as much as the
// streaming.  There the CTAs of a thread-block cluster share one unit's tiles, leave their
// partial (O^T, references, sums) in their own shared memory, and after one cluster barrier CTA r
// combines the partials of the output rows r, r + cluster size, ... over distributed shared memory
// and writes them: one kernel per call.
#pragma once

namespace kt {

constexpr int kKeys = 128;                 // keys per tile
constexpr int kMaxNC = 4;                  // one softmax group serves up to 64 grouped rows
constexpr int kMaxNC2 = 6;                 // two softmax groups (half of the columns each) serve up to 96
__host__ __device__ constexpr int threads(int SG) { return 128 * SG + 96; }  // softmax warps + three role warps
constexpr int kThreads = threads(1);
constexpr int kBlk = kKeys * 128;          // bytes of one tile x 64-column half
constexpr float kJump = 16.f;              // a score this far (log2) above the reference moves it

// K and V tiles live in rings of their own: a K slot is free as soon as QK^T of its tile has
// completed, a V slot only after PV, so K gets by with two slots and V takes the rest (measured:
// 2 + 4 slots run 2 % faster than 3 + 3 on the 8B-128K layer; with more than 48 rows 2 + 3 fit).
__host__ __device__ constexpr int k_slots(int NC) { return 2; }
__host__ __device__ constexpr int v_slots(int NC) { return NC <= 3 ? 4 : 3; }
__host__ __device__ constexpr int p_blocks(int NC) { return (NC * 16 + 63) / 64; }  // 64-row blocks of P^T
__host__ __device__ constexpr int smem_bytes(int NC) {
    // K ring + V ring (two halves each) + Q (two halves) + P^T (128 keys x 128 bytes per 64 grouped rows)
    return 2 * (k_slots(NC) + v_slots(NC)) * kBlk + 2 * (NC * 16) * 128 + p_blocks(NC) * kBlk + 1024;
}

// Named barriers of one softmax group (128 threads): barrier 1 for group 0, barrier 2 for group 1.
__device__ __forceinline__ void bar_softmax(int grp) {
    if (grp == 0) asm volatile("bar.sync 1, 128;" ::: "memory");
    else asm volatile("bar.sync 2, 128;" ::: "memory");
}
#define RAPID_KT_BAR_OR(ID)                                                                              \
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.b32 q, %1, 0;\n\tbar.red.or.pred p, " #ID ", 128, q;\n\t" \
                 "selp.u32 %0, 1, 0, p;\n\t}"                                                            \
                 : "=r"(res)                                                                             \
                 : "r"((uint32_t)flag)                                                                   \
                 : "memory")
__device__ __forceinline__ bool bar_softmax_or(int grp, bool flag) {
    uint32_t res;
    if (grp == 0) RAPID_KT_BAR_OR(1);
    else RAPID_KT_BAR_OR(2);
    return res != 0;
}
#undef RAPID_KT_BAR_OR
// Cluster-wide barrier of all threads, release / acquire: what a CTA wrote to its shared memory
// before it is visible to its peers' distributed-shared-memory loads after it.
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_cta_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// A float of the shared memory of CTA `rank` of the cluster, at the same offset as `addr` here.
__device__ __forceinline__ float ld_dsmem_f32(uint32_t addr, int rank) {
    uint32_t raddr;
    float v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(raddr) : "r"(addr), "r"(rank));
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(raddr) : "memory");
    return v;
}
__device__ __forceinline__ float warp_max32(float v) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum32(float v) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// NC = N / 16 column chunks (N = grouped rows padded to 16).  SG = softmax groups of 128 threads:
// group g forms the probabilities of columns [g N/SG, (g+1) N/SG) for all 128 keys of a tile, keeps
// those rows' references and sums and rescales and reads out those columns of O^T; the groups meet
// only at the P^T barrier (PV starts when both have published) and at the end of a unit.
// WIN = the call has a sink + window mask (a kernel of its own, so that calls without one carry none
// of its code: the kernel's instruction footprint shows in every launch).
template <int NC, int SG = 1, bool WIN = false>
__global__ void __launch_bounds__(threads(SG), 1)
verify_attn_splitkv_kt_kernel(const __grid_constant__ CUtensorMap tmK,
                              const __grid_constant__ CUtensorMap tmV,
                              const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ AttnArgs a) {
    constexpr int D = 128;
    constexpr int N = NC * 16;
    constexpr int NG = N / SG;             // columns per softmax group
    constexpr int CH = NG % 16 == 0 ? 16 : 8;  // columns per tensor-memory load
    constexpr int WS = 4 * SG;             // softmax warps; the role warps follow
    static_assert(N % SG == 0 && NG % 8 == 0, "a group's columns are whole 16-byte chunks of a P^T row");
    constexpr int NK = k_slots(NC), NV = v_slots(NC);
    constexpr int TILE_TX = 2 * kBlk;  // one tile of K or of V: two 64-column halves
    constexpr uint32_t TMEM_COLS = 512;
    constexpr uint32_t COL_S = 0;    // S^T buffer b at COL_S + 128 b
    constexpr uint32_t COL_O = 256;  // O^T: N columns
    // shared-memory map (bytes from the 1024-aligned base)
    constexpr uint32_t OFF_K = 0, OFF_V = 2 * NK * kBlk, OFF_Q = 2 * (NK + NV) * kBlk, OFF_P = OFF_Q + 2 * N * 128;

    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t k_full[NK], k_empty[NK], v_full[NV], v_empty[NV];
    __shared__ uint64_t s_full[2], p_full[2];
    __shared__ uint64_t q_full, o_free;
    __shared__ uint64_t drain_bar[2];  // an MMA issuer that leaves early sees its MMAs complete here
    __shared__ uint32_t tmem_slot;
    __shared__ Walk s_walk;
    __shared__ int s_abort;
    __shared__ __align__(16) float sh_mref[128], sh_fac[128], sh_w[4][128];
    __shared__ float sh_lfin[128];  // cluster mode: the unit's row sums of this CTA

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
        mbar_init(&q_full, 1);
        mbar_init(&o_free, WS);
        fence_mbar_init();
        s_abort = 0;
        prefetch_tensormap(&tmK);
        prefetch_tensormap(&tmV);
        prefetch_tensormap(&tmQ);
    }
    if (warp == WS + 1) tmem_alloc(&tmem_slot, TMEM_COLS);  // the same warp frees it at the end
    // The Q rows past the grouped rows are never written by the Q loads: zero them once, so that
    // the scores of those columns are 0 whatever the shared memory held.
    {
        const int pad_chunks = (N - a.GR) * 8;  // 16-byte chunks per 64-column half
        for (int i = tid; i < 2 * pad_chunks; i += threads(SG)) {
            const int h = i >= pad_chunks, k16 = h ? i - pad_chunks : i;
            *reinterpret_cast<uint4*>(smem_gen + OFF_Q + h * (N * 128) + a.GR * 128 + k16 * 16) = make_uint4(0, 0, 0, 0);
        }
        fence_proxy_async_smem();
    }
    if (tid < 128) {  // a CTA of a cluster that gets no tile publishes "no partial"
        sh_mref[tid] = -INFINITY;
        sh_lfin[tid] = 0.f;
    }
    // The walk, the stream-order wait, and between the two, where the caller vouches for the older part
    // of the cache (kv_settled, which implies a settled plan), the first tiles' copies: they overlap
    // the work that precedes this kernel on the stream.  Only tiles wholly below the newest R keys
    // are taken early; everything else is read after the wait.
    Walk w;
    const bool settled = a.plan_mode == RAPID_PLAN_SETTLED;
    if (settled) load_walk(a, cta, 1, w);
    tc_fence_before_sync();
    __syncthreads();  // barriers initialised, tensor memory allocated
    tc_fence_after_sync();
    int pre_k = 0, pre_v = 0;  // tiles whose K / V copies were issued before the wait (producer lane only)
    if (a.kv_settled && warp == WS && lane == 0 && w.remaining > 0) {
        const int seg0 = (int)min((long long)(w.ntiles - w.tile), w.remaining);
        const int old_tiles = (w.L - a.R) >> 7;  // tiles 0 .. old_tiles-1 hold none of the newest R keys
        // a short walk takes only as many tiles early as there are K slots: more V tiles ahead would hold
        // up the K tiles it needs next (one-row decode at 8K: 12.7 against 13.3 us per layer)
        const int n_early = seg0 > 2 * NV ? NV : NK;
        for (int t = 0; t < seg0 && t < n_early; ++t) {
            const int tile = WIN ? real_tile(w, w.tile + t) : w.tile + t;
            if (tile >= old_tiles) break;
            if (t < NK) {
                mbar_arrive_expect_tx(&k_full[t], TILE_TX);
#pragma unroll
                for (int h = 0; h < 2; ++h)
                    tma_load_4d(smem_gen + OFF_K + (h * NK + t) * kBlk, &tmK, &k_full[t], h * 64, tile * kKeys, w.kvh, w.b);
                ++pre_k;
            }
            mbar_arrive_expect_tx(&v_full[t], TILE_TX);
#pragma unroll
            for (int h = 0; h < 2; ++h)
                tma_load_4d(smem_gen + OFF_V + (h * NV + t) * kBlk, &tmV, &v_full[t], h * 64, tile * kKeys, w.kvh, w.b);
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
    if (cta == 0 && warp == WS && lane == 1) check_call_inputs(a, 1);  // an idle lane of the producer warp
    const uint32_t tmem_base = tmem_slot;
    const WaitCtx wc = {&s_abort, a.wait_limit};
    const int unit_b = w.b, unit_kvh = w.kvh;  // cluster mode: the one unit this CTA works on

    if (warp == WS) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            int jj = 0, n_k = 0, n_v = 0;  // tiles met; K and V tiles whose copies were issued
            bool ok = true;
            while (w.remaining > 0 && ok) {
                const int seg = (int)min((long long)(w.ntiles - w.tile), w.remaining);
                for (int t = 0; t < seg && ok; ++t, ++jj) {
                    const int ks = jj % NK, vs = jj % NV;
                    const int tile = WIN ? real_tile(w, w.tile + t) : w.tile + t;
                    // a tile is one box of 128 keys, or, for a paged cache with 64-key blocks, two
                    // boxes of 64 keys from two physical blocks (parts = 2)
                    const int parts = a.kt_half_blocks ? 2 : 1;
                    int key0[2] = {tile * kKeys, 0}, outer[2] = {w.b, w.b};
                    if (a.block_table) {
                        for (int p = 0; p < parts; ++p) {
                            const int lb = a.kt_half_blocks ? 2 * tile + p : (tile >> a.tile_shift);
                            key0[p] = a.kt_half_blocks ? 0 : (tile & ((1 << a.tile_shift) - 1)) * kKeys;
                            if (a.kt_half_blocks && lb * 64 >= w.L) {
                                outer[p] = a.num_blocks;  // wholly past the context: zeros, no table entry is read
                                continue;
                            }
                            outer[p] = __ldg(a.block_table + (size_t)w.b * a.max_blocks + lb);
                            if ((unsigned)outer[p] >= (unsigned)a.num_blocks) {
                                atomicOr(a.status, RAPID_STATUS_BAD_BLOCK_TABLE);
                                outer[p] = a.num_blocks;  // outside the pool: the copy reads zeros
                            }
                        }
                    }
                    const uint32_t part_bytes = kBlk / parts;
                    if (jj >= pre_k) {  // (the first pre_k tiles' K copies went out before the wait)
                        if (jj >= NK) ok = mbar_wait_bounded_relaxed(&k_empty[ks], ((jj / NK) - 1) & 1, wc);
                        if (!ok) break;
                        mbar_arrive_expect_tx(&k_full[ks], TILE_TX);
                        for (int p = 0; p < parts; ++p)
#pragma unroll
                            for (int h = 0; h < 2; ++h)
                                tma_load_4d(smem_gen + OFF_K + (h * NK + ks) * kBlk + p * part_bytes, &tmK, &k_full[ks],
                                            h * 64, key0[p], w.kvh, outer[p]);
                    }
                    ++n_k;
                    if (jj >= pre_v) {
                        if (jj >= NV) ok = mbar_wait_bounded_relaxed(&v_empty[vs], ((jj / NV) - 1) & 1, wc);
                        if (!ok) break;
                        mbar_arrive_expect_tx(&v_full[vs], TILE_TX);
                        for (int p = 0; p < parts; ++p)
#pragma unroll
                            for (int h = 0; h < 2; ++h)
                                tma_load_4d(smem_gen + OFF_V + (h * NV + vs) * kBlk + p * part_bytes, &tmV, &v_full[vs],
                                            h * 64, key0[p], w.kvh, outer[p]);
                    }
                    ++n_v;
                }
                walk_advance(a, w, seg);
            }
            // leaving early: the copies already issued must have landed before the CTA gives up its
            // shared memory
            if (!ok) {
                n_k = max(n_k, pre_k);  // copies that went out before the wait count too
                n_v = max(n_v, pre_v);
                for (int s = 0; s < NK && s < n_k; ++s)
                    mbar_wait_drain(&k_full[s], ((s + (n_k - 1 - s) / NK * NK) / NK) & 1);
                for (int s = 0; s < NV && s < n_v; ++s)
                    mbar_wait_drain(&v_full[s], ((s + (n_v - 1 - s) / NV * NV) / NV) & 1);
            }
        }
    } else if (warp == WS + 1) {
        // ---------------- Q loader and QK^T issuer ----------------
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16(128, N, 0, 0);
            const uint64_t k_desc = umma_smem_desc(smem_base + OFF_K, 16, 1024);
            const uint64_t q_desc = umma_smem_desc(smem_base + OFF_Q, 16, 1024);
            bool ok = true;
            int jj = 0, seg_idx = 0;
            while (w.remaining > 0 && ok) {
                const int seg = (int)min((long long)(w.ntiles - w.tile), w.remaining);
                // the previous unit has been read out of tensor memory: every MMA of it is complete
                if (seg_idx > 0) ok = mbar_wait_bounded(&o_free, (seg_idx - 1) & 1, wc);
                if (!ok) break;
                mbar_arrive_expect_tx(&q_full, (uint32_t)a.GR * D * 2);
#pragma unroll
                for (int h = 0; h < 2; ++h)
                    tma_load_4d(smem_gen + OFF_Q + h * (N * 128), &tmQ, &q_full, h * 64, w.kvh * a.G, 0, w.b);
                ok = mbar_wait_bounded(&q_full, seg_idx & 1, wc);
                if (!ok) mbar_wait_drain(&q_full, seg_idx & 1);  // the Q copy is on its way: let it land
                for (int t = 0; t < seg && ok; ++t, ++jj) {
                    const int s = jj % NK, b = jj & 1;
                    ok = mbar_wait_bounded(&k_full[s], (jj / NK) & 1, wc);
                    // S^T buffer b is free once the probabilities of tile jj-2 have been published
                    if (ok && jj >= 2) ok = mbar_wait_bounded(&p_full[b], ((jj - 2) >> 1) & 1, wc);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t d = tmem_base + COL_S + 128u * b;
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        const uint32_t half = kk >> 2, ko16 = (kk & 3) * 2;
                        umma_bf16_ss(d, k_desc + ((half * NK + s) * kBlk >> 4) + ko16,
                                     q_desc + (half * (N * 128) >> 4) + ko16, idesc, kk > 0);
                    }
                    umma_commit(&s_full[b]);
                    umma_commit(&k_empty[s]);  // QK^T complete: the K slot is free
                }
                walk_advance(a, w, seg);
                ++seg_idx;
            }
            if (!ok) {  // leaving early: every MMA issued here must have completed before tensor memory is freed
                umma_commit(&drain_bar[0]);
                mbar_wait_drain(&drain_bar[0], 0);
            }
        }
    } else if (warp == WS + 2) {
        // ---------------- PV issuer ----------------
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16(D, N, 1, 1);
            // V tile as MN-major A: 64-column blocks NV*kBlk bytes apart, 8-key groups 1024 bytes apart
            const uint64_t v_desc = umma_smem_desc(smem_base + OFF_V, NV * kBlk, 1024);
            // P^T as MN-major B: one 128-byte row per key (64 grouped rows), 64-row blocks kBlk bytes apart
            const uint64_t p_desc = umma_smem_desc(smem_base + OFF_P, kBlk, 1024);
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
                    for (int kk = 0; kk < kKeys / 16; ++kk)
                        umma_bf16_ss(d, v_desc + (s * kBlk >> 4) + kk * (2048 >> 4), p_desc + kk * (2048 >> 4), idesc,
                                     (t > 0 || kk > 0) ? 1u : 0u);
                    umma_commit(&v_empty[s]);  // PV complete: the V slot and the P^T buffer are free
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
        constexpr int C0_STEP = NG;
        const int C0 = grp * C0_STEP;  // this group's first column
        const uint32_t lane_base = (uint32_t)(wq * 32) << 16;
        const uint32_t tO = tmem_base + lane_base + COL_O + C0;
        const float c = a.scale_log2;
        const int slot_stride = (int)slot_floats(a.GR, D);
        // this key's row of P^T (MN-major: 128 bytes = 64 grouped rows per key, 128-byte swizzle)
        uint8_t* p_gen = smem_gen + OFF_P + t * 128;
        const int p_swz = t & 7;

        float lsum[NG];  // this key slot's share of the sums of the group's rows
        int jj = 0;
        // `ok` only records that a wait ran out: these warps run their loops to the end whatever
        // happens (see "Waits that run out" above)
        bool ok = true;
        while (w.remaining > 0) {
            const int seg = (int)min((long long)(w.ntiles - w.tile), w.remaining);
            const int L = w.L;
#pragma unroll
            for (int i = 0; i < NG; ++i) lsum[i] = 0.f;

            for (int ti = 0; ti < seg; ++ti, ++jj) {
                const int b = jj & 1;
                const uint32_t tS = tmem_base + lane_base + COL_S + 128u * b + C0;
                const int key0 = (WIN ? real_tile(w, w.tile + ti) : w.tile + ti) * kKeys;  // the tile's first key
                const int key = key0 + t;
                // Row i sees keys <= L-R+i and rows are column i*G+g, so the columns the causal stair
                // hides from this key are a prefix [0, cmin) (no stair: every row sees every key
                // below L).  With a window the rows too new for this key are a suffix [cmax, N):
                // row i sees it iff key > L-R+i - window, unless it is a sink key.
                const int over_ctx = a.stair ? key - (L - a.R) : 0;
                const int cmin = key >= L ? N : (over_ctx > 0 ? over_ctx * a.G : 0);
                int cmax = N;
                if constexpr (WIN) {
                    if (key >= a.sink) {
                        const long long rows_in = (long long)key - (L - a.R) + a.window;
                        cmax = rows_in <= 0 ? 0 : (rows_in * a.G >= N ? N : (int)rows_in * a.G);
                    }
                }
                ok &= warp_wait_bounded(&s_full[b], (jj >> 1) & 1, wc);
                tc_fence_after_sync();

                // One pass over the scores: probabilities against the current references, kept in
                // registers until it is known that no visible score sits far above its reference.
                // (Kept as fp32 up to 48 columns; beyond that as packed bf16 pairs, to stay in registers.)
                constexpr bool kPacked = NG > 48;
                float pv[kPacked ? 2 : NG];
                uint32_t pq[kPacked ? NG / 2 : 1];
                // the same for every thread: no key of the tile is hidden from any row
                const bool tile_clear = key0 + kKeys <= L - a.stair &&
                                        (!WIN || key0 + kKeys <= a.sink || key0 > L - 1 - a.window);
                bool move = ti == 0;
                if (ti == 0 && tile_clear) {
                    // A unit's first tile, seen whole by every row: the scores of its first key serve as
                    // the references (any reference will do as long as no visible score sits far above
                    // it, which the pass below finds out).  That spares this tile the row maxima over its
                    // 128 keys, the longest stretch of code a CTA would otherwise run before its pipeline
                    // is full.
                    if (wq == 0) {
#pragma unroll
                        for (int ch = 0; ch < NG / CH; ++ch) {
                            uint32_t sr[CH];
                            tmem_ld_cols<CH>(tS + CH * ch, sr);
                            tmem_wait_ld();
                            if (lane == 0) {
#pragma unroll
                                for (int e = 0; e < CH; ++e) {
                                    const int col = C0 + CH * ch + e;
                                    sh_mref[col] = col < a.GR ? __uint_as_float(sr[e]) * c : INFINITY;
                                }
                            }
                        }
                    }
                    bar_softmax(grp);
                }
                if (ti > 0 || tile_clear) {
                    // MASKED = false for a tile every row sees whole (all of a long context but its end):
                    // no per-column predicate.  Columns past the grouped rows need none either: their
                    // scores are 0 (zero rows of Q) and their reference is +inf, so they come out as 0.
                    auto first_pass = [&](auto masked_tag) {
                        constexpr bool MASKED = decltype(masked_tag)::value;
                        bool far = false;
#pragma unroll
                        for (int ch = 0; ch < NG / CH; ++ch) {
                            uint32_t sr[CH];
                            tmem_ld_cols<CH>(tS + CH * ch, sr);
                            tmem_wait_ld();
#pragma unroll
                            for (int e = 0; e < CH; e += 4) {
                                const int li = CH * ch + e, col = C0 + li;
                                const float4 m = *reinterpret_cast<const float4*>(&sh_mref[col]);
                                float x[4] = {fmaf(__uint_as_float(sr[e]), c, -m.x), fmaf(__uint_as_float(sr[e + 1]), c, -m.y),
                                              fmaf(__uint_as_float(sr[e + 2]), c, -m.z),
                                              fmaf(__uint_as_float(sr[e + 3]), c, -m.w)};
#pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    if (MASKED) x[i] = (col + i >= cmin && (!WIN || col + i < cmax)) ? x[i] : -INFINITY;
                                    far |= x[i] > kJump;
                                    x[i] = fast_exp2(x[i]);
                                }
                                if (kPacked) {
                                    pq[li >> 1] = pack_bf16x2(x[0], x[1]);
                                    pq[(li >> 1) + 1] = pack_bf16x2(x[2], x[3]);
                                } else {
#pragma unroll
                                    for (int i = 0; i < 4; ++i) pv[kPacked ? 0 : li + i] = x[i];
                                }
                            }
                        }
                        return far;
                    };
                    move = tile_clear ? first_pass(std::false_type{}) : first_pass(std::true_type{});
                    move = bar_softmax_or(grp, move);
                }
                // PV of the previous tile must be complete: it reads P^T, and O^T may be rescaled now
                if (jj >= 1) {
                    ok &= warp_wait_bounded(&v_empty[(jj - 1) % NV], ((jj - 1) / NV) & 1, wc);
                    tc_fence_after_sync();
                }
                if (move) {
                    // new reference = max(old, this tile's row maxima over the 128 keys)
#pragma unroll
                    for (int ch = 0; ch < NG / CH; ++ch) {
                        uint32_t sr[CH];
                        tmem_ld_cols<CH>(tS + CH * ch, sr);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < CH; ++e) {
                            const int col = C0 + CH * ch + e;
                            const float v = (col >= cmin && (!WIN || col < cmax) && col < a.GR) ? __uint_as_float(sr[e]) * c : -INFINITY;
                            const float wm = warp_max32(v);
                            if (lane == 0) sh_w[wq][col] = wm;
                        }
                    }
                    bar_softmax(grp);
                    if (t < NG) {
                        const int col = C0 + t;
                        const float old = ti == 0 ? -INFINITY : sh_mref[col];
                        const float nm =
                            fmaxf(fmaxf(old, fmaxf(sh_w[0][col], sh_w[1][col])), fmaxf(sh_w[2][col], sh_w[3][col]));
                        const bool pad = col >= a.GR;  // a column past the grouped rows: reference +inf, probabilities 0
                        sh_fac[col] = (pad || nm == old) ? 1.f : fast_exp2(old - nm);  // old = -inf gives 0
                        sh_mref[col] = pad ? INFINITY : nm;
                    }
                    bar_softmax(grp);
                    if (ti > 0) {
#pragma unroll
                        for (int i = 0; i < NG; ++i) lsum[i] *= sh_fac[C0 + i];
                        // thread t is lane t of O^T (= output column d): rescale its group's row entries
#pragma unroll
                        for (int ch = 0; ch < NG / CH; ++ch) {
                            uint32_t orow[CH];
                            tmem_ld_cols<CH>(tO + CH * ch, orow);
                            tmem_wait_ld();
#pragma unroll
                            for (int e = 0; e < CH; ++e)
                                orow[e] = __float_as_uint(__uint_as_float(orow[e]) * sh_fac[C0 + CH * ch + e]);
                            tmem_st_cols<CH>(tO + CH * ch, orow);
                        }
                        tmem_wait_st();
                    }
                    // the probabilities again, against the new references
#pragma unroll
                    for (int ch = 0; ch < NG / CH; ++ch) {
                        uint32_t sr[CH];
                        tmem_ld_cols<CH>(tS + CH * ch, sr);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < CH; e += 2) {
                            const int li = CH * ch + e, col = C0 + li;
                            const float m0 = sh_mref[col], m1 = sh_mref[col + 1];
                            const float x0 = (col >= cmin && (!WIN || col < cmax)) ? fmaf(__uint_as_float(sr[e]), c, m0 == -INFINITY ? 0.f : -m0) : -INFINITY;
                            const float x1 = (col + 1 >= cmin && (!WIN || col + 1 < cmax)) ? fmaf(__uint_as_float(sr[e + 1]), c, m1 == -INFINITY ? 0.f : -m1) : -INFINITY;
                            const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
                            if (kPacked) {
                                pq[li >> 1] = pack_bf16x2(p0, p1);
                            } else {
                                pv[kPacked ? 0 : li] = p0;
                                pv[kPacked ? 1 : li + 1] = p1;
                            }
                        }
                    }
                }
                // this key's row of P^T: 16-byte chunks of 8 grouped rows each
#pragma unroll
                for (int c8 = 0; c8 < NG / 8; ++c8) {
                    const int g8 = C0 / 8 + c8;  // the chunk's place in the whole row
                    uint4 pk;
                    if (kPacked) {
                        pk = make_uint4(pq[4 * c8], pq[4 * c8 + 1], pq[4 * c8 + 2], pq[4 * c8 + 3]);
                        // the sums take the probabilities as the tensor cores will see them
                        const uint32_t u[4] = {pk.x, pk.y, pk.z, pk.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            lsum[8 * c8 + 2 * e] += __uint_as_float(u[e] << 16);
                            lsum[8 * c8 + 2 * e + 1] += __uint_as_float(u[e] & 0xffff0000u);
                        }
                    } else {
                        const int o = kPacked ? 0 : 8 * c8;
                        pk.x = pack_bf16x2(pv[o + 0], pv[o + 1]);
                        pk.y = pack_bf16x2(pv[kPacked ? 0 : o + 2], pv[kPacked ? 1 : o + 3]);
                        pk.z = pack_bf16x2(pv[kPacked ? 0 : o + 4], pv[kPacked ? 1 : o + 5]);
                        pk.w = pack_bf16x2(pv[kPacked ? 0 : o + 6], pv[kPacked ? 1 : o + 7]);
#pragma unroll
                        for (int e = 0; e < 8; ++e) lsum[8 * c8 + e] += pv[kPacked ? 0 : o + e];
                    }
                    *reinterpret_cast<uint4*>(p_gen + (g8 >> 3) * kBlk + (((g8 & 7) ^ p_swz) << 4)) = pk;
                }
                if (grp == 0 && key0 + kKeys > L) {
                    // V rows beyond the context may hold any bits: zero them so that 0 * row = 0
                    // (one group does it; PV waits for both groups' arrivals)
                    ok &= warp_wait_bounded(&v_full[jj % NV], (jj / NV) & 1, wc);  // the V tile has landed
                    const int first_bad = max(L - key0, 0);
                    const int chunks = (kKeys - first_bad) * 8;
                    for (int h = 0; h < 2; ++h) {
                        uint8_t* vgen = smem_gen + OFF_V + (h * NV + jj % NV) * kBlk;
                        for (int chk = t; chk < chunks; chk += 128)
                            *reinterpret_cast<uint4*>(vgen + first_bad * 128 + chk * 16) = make_uint4(0, 0, 0, 0);
                    }
                }
                fence_proxy_async_smem();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&p_full[b]);
            }
            // ---- end of the unit: O^T out of tensor memory, row sums added up, partial written ----
            ok &= warp_wait_bounded(&v_empty[(jj - 1) % NV], ((jj - 1) / NV) & 1, wc);
            tc_fence_after_sync();
            const int unit = w.b * a.Hkv + w.kvh;
            // the partial goes to the workspace, or, with one cluster per unit, to this CTA's own
            // shared memory (the K ring: every K tile has been consumed), [column][d] fp32
            float* slot = a.cmerge ? reinterpret_cast<float*>(smem_gen + OFF_K)
                                   : a.partial + (size_t)(cta + unit) * slot_stride;
#pragma unroll
            for (int ch = 0; ch < NG / CH; ++ch) {
                uint32_t orow[CH];
                tmem_ld_cols<CH>(tO + CH * ch, orow);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < CH; ++e) {
                    const int col = C0 + CH * ch + e;
                    if (col < a.GR && sh_mref[col] != -INFINITY) slot[(size_t)col * D + t] = __uint_as_float(orow[e]);
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
                const float l_fin = ((sh_w[0][col] + sh_w[1][col]) + sh_w[2][col]) + sh_w[3][col];
                if (a.cmerge) {
                    sh_lfin[col] = l_fin;
                } else {
                    slot[a.GR * D + col] = sh_mref[col];
                    slot[a.GR * D + a.GR + col] = l_fin;
                }
            }
            bar_softmax(grp);  // sh_w / sh_mref are reused by the next unit
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&o_free);
            walk_advance(a, w, seg);
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (a.cmerge) {
        // ---- one cluster per unit: combine the cluster's partials over distributed shared memory ----
        // CTA r of the cluster takes the output rows (columns) r, r + cmerge, ...; thread d the
        // output element d.  Fixed order over the ranks: results are bit-identical from run to run.
        cluster_sync_all();  // every CTA's partial is in its shared memory and visible
        const uint32_t rank = cluster_cta_rank();
        const uint32_t xo_addr = smem_base + OFF_K, m_addr = smem_u32(sh_mref), l_addr = smem_u32(sh_lfin);
        if (tid < D) {
            for (int col = (int)rank; col < a.GR; col += a.cmerge) {
                float M = -INFINITY;
                for (int p = 0; p < a.cmerge; ++p) M = fmaxf(M, ld_dsmem_f32(m_addr + 4u * col, p));
                float acc = 0.f, l = 0.f;
                for (int p = 0; p < a.cmerge; ++p) {
                    const float mp = ld_dsmem_f32(m_addr + 4u * col, p);
                    if (mp == -INFINITY) continue;  // that CTA saw no key of this row: its partial holds no O
                    const float wgt = exp2f(mp - M);
                    l += wgt * ld_dsmem_f32(l_addr + 4u * col, p);
                    acc += wgt * ld_dsmem_f32(xo_addr + 4u * (col * D + tid), p);
                }
                const float val = acc / l;
                const int i = col / a.G, g = col % a.G;
                const size_t row = ((size_t)unit_b * a.R + i) * a.Hq + (size_t)unit_kvh * a.G + g;
                a.out[row * D + tid] = __float2bfloat16_rn(val);
                if (a.out_f32) a.out_f32[row * D + tid] = val;
                if (a.lse_out && tid == 0) a.lse_out[row] = (M + log2f(l)) * 0.69314718055994530942f;
            }
        }
        cluster_sync_all();  // no CTA leaves while a peer may still read its shared memory
    }
    if (warp == WS + 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
    if (tid == 0 && s_abort) atomicOr(a.status, RAPID_STATUS_PIPELINE_TIMEOUT);
}

}  // namespace kt
