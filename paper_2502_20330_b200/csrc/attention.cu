// Verify attention (Algorithm 1, the target's single validation pass over the full context):
// split-KV kernel + log-sum-exp merge.
//
// Work decomposition.  A "unit" is one (sequence, KV head) pair; its K/V cache is cut into
// tiles of kTile keys.  All units' tiles form one flat list, cut into equal contiguous ranges,
// one per CTA, so every CTA streams the same number of bytes whatever the context lengths are.
// A CTA whose range crosses a unit boundary emits one partial result per unit it touches.
// The G*R grouped query rows of a KV head (G = Hq/Hkv heads times R = gamma+1 draft rows) ride
// together, so each K/V tile leaves HBM once.
//
// The split kernel (tcgen05 / tensor memory, described at its definition) writes fp32 partials
// (unnormalised O, softmax reference, sum) to the workspace, two per CTA and unit (one per
// softmax stream); the merge kernel combines them in a fixed order, so results are bit-identical
// from run to run.  The merge is launched as a programmatic dependent of the split kernel: its
// blocks are resident and have done their index arithmetic by the time the last partial lands.
#include <math.h>
#include <type_traits>

#include "common.cuh"
#include "tcgen05.cuh"

namespace rapid {

namespace {

constexpr int kTile = 64;  // keys per pipeline stage

constexpr int kStreams = 2;  // softmax streams per CTA = partials per CTA and unit
__host__ __device__ constexpr int stage_bytes(int D) { return 2 * kTile * D * 2; }
// floats per partial slot: GR rows of D, then GR maxima and GR sums; a multiple of 4 so that
// every row of every slot can be read with 16-byte loads
__host__ __device__ constexpr long long slot_floats(int GR, int D) {
    return ((long long)GR * (D + 2) + 3) / 4 * 4;
}

struct Walk;

struct AttnArgs {
    const __nv_bfloat16* q;
    const int32_t* ctx_lens;
    float* partial;   // [slots][GR*(D+2)] fp32
    int32_t* status;  // workspace status word
    int B, Hq, Hkv, G, R, GR;
    int Lmax;
    int num_ctas;
    float scale_log2;  // softmax scale * log2(e)
    // paged cache (block_table != nullptr): logical key tile t of sequence b lives in physical
    // block block_table[b * max_blocks + (t >> tile_shift)], at tile (t & tile_mask) inside it
    const int32_t* block_table;
    int max_blocks, num_blocks, tile_shift;
    // stair = R: row i sees keys <= L - R + i (the R newest keys are the rows' own, causal among
    // themselves); stair = 0: every row sees all L keys (a shard of the context without those rows).
    // Lmin = the shortest admissible length: R resp. 1.
    int stair, Lmin;
    // Work split.  Moving from one (sequence, KV head) unit to the next inside a CTA drains the
    // pipeline (the unit's O is read out, a new Q is loaded, the first scores have to come back),
    // which costs about as much as `pad` tiles of streaming.  The flat tile list the CTAs cut into
    // equal ranges therefore carries `pad` virtual tiles in front of every unit: a CTA whose range
    // spans a unit boundary gets that many fewer real tiles, and all CTAs finish together.
    int pad;
    int kt_half_blocks;  // keys-on-M kernel over a paged cache with 64-key blocks: two boxes per tile
    int tile_keys;  // keys per scheduling tile: what plan, walk and merge count in (64, or 128 for the keys-on-M kernel)
    int tile_log2;  // log2(tile_keys)
    // Sink + window visibility (window > 0): row i sees the keys below `sink` and the `window`
    // newest keys up to its own, (lim_i - window, lim_i].  Tiles no row sees are not streamed.
    int sink, window;
    // The plan attention_plan_kernel wrote for this geometry and these lengths: every CTA's walk and
    // every unit's range of partial slots.  plan_mode says how old it is: RAPID_PLAN_READY = made by
    // the kernel just before this call's, RAPID_PLAN_SETTLED = at least two kernels ago.  (A call
    // without a caller's plan launches the plan kernel itself and runs with RAPID_PLAN_READY.)
    int plan_mode;
    // kv_settled: tiles wholly below the newest R keys may be copied before the grid-dependency wait
    // (the caller vouches for them; needs a settled plan and a contiguous cache)
    int kv_settled;
    // merge_early: the 4-warp merge lets its dependents launch before its own wait (after a keys-on-M
    // split kernel; after the rows-on-M kernel it measured 2.5 us slower per layer of the smallest
    // workload and no faster on the largest, so there the order stays wait, then launch)
    int merge_early;
    int caller_plan;  // the caller supplied the plan: check it against the call's geometry and lengths
    const Walk* plan_walks;
    const int2* plan_units;  // (first CTA, number of slots) of every unit
    const int32_t* plan_ctx;  // the lengths the plan was made for
    const int32_t* plan_sig;  // the geometry the plan was made for (kPlanSigInts words)
    long long wait_limit;     // clock cycles an on-chip wait may take
    // One thread-block cluster per unit (cmerge = its size, 0 = off): the cluster's CTAs split the
    // unit's tiles, exchange their partials through distributed shared memory and write the
    // output rows themselves; no partial goes to the workspace and no merge kernel follows.
    int cmerge;
    // FP8 cache: one fp32 scale per (sequence, KV head) for the K codes and one for the V codes
    const float* k_scale;
    const float* v_scale;
    __nv_bfloat16* out;
    float* out_f32;
    float* lse_out;
};

// Where a CTA stands in its range of the flat tile list.  In sink + window mode a unit streams its
// tiles [0, ns) and [ns + gap, ...): the real tile behind index t is t + (t >= ns ? gap : 0).
struct __align__(16) Walk {
    int b, kvh, tile, ntiles, L;
    int ns, gap;
    int reserved;
    long long remaining;
    long long total;
};
static_assert(sizeof(Walk) == 48, "a walk is three 16-byte words of the plan");

constexpr int kPlanSigInts = 16;

__device__ __forceinline__ int clamp_len(int L, int R, int Lmax) {
    return L < R ? R : (L > Lmax ? Lmax : L);
}
__device__ __forceinline__ int tiles_of(const AttnArgs& a, int L) { return (L + a.tile_keys - 1) >> a.tile_log2; }

// The tiles a unit of L keys streams: all of them, or, with a window, the tiles that hold sink
// keys and the tiles from the oldest key of row 0's window on (the rows' windows end at their own
// keys, so row 0's reaches back furthest).
struct UnitGeom {
    int nt, ns, gap;
};
__device__ __forceinline__ UnitGeom unit_geom(const AttnArgs& a, int L) {
    UnitGeom g;
    const int full = tiles_of(a, L);
    g.nt = full;
    g.ns = full;
    g.gap = 0;
    if (a.window > 0) {
        const int w0 = L - a.R - a.window + 1;          // the oldest key row 0 sees through its window
        const int ns = tiles_of(a, a.sink);             // tiles that hold sink keys
        const int tw0 = w0 > 0 ? w0 >> a.tile_log2 : 0;  // the tile that key lives in
        if (tw0 > ns) {
            g.ns = ns;
            g.gap = tw0 - ns;
            g.nt = full - g.gap;
        }
    }
    return g;
}
__device__ __forceinline__ int unit_tiles(const AttnArgs& a, int b) {
    return unit_geom(a, clamp_len(a.ctx_lens[b], a.Lmin, a.Lmax)).nt;
}
__device__ __forceinline__ int real_tile(const Walk& w, int t) { return t + (t >= w.ns ? w.gap : 0); }

// The padding applies only when every CTA has a few tiles to stream.
__device__ __forceinline__ int unit_pad(const AttnArgs& a, long long T) {
    return T >= 4LL * a.num_ctas ? a.pad : 0;
}

// Real tiles among the first v tiles of the padded flat list (every unit: pad virtual, then nt real).
__device__ __forceinline__ long long real_tiles_before(const AttnArgs& a, int pad, long long v) {
    long long real = 0;
    for (int b = 0; b < a.B; ++b) {
        const int nt = unit_tiles(a, b);
        const long long ul = nt + pad, span = (long long)a.Hkv * ul;
        if (v >= span) {
            real += (long long)a.Hkv * nt;
            v -= span;
            continue;
        }
        const long long k = v / ul, rem = v - k * ul;
        long long part = rem - pad;
        part = part < 0 ? 0 : (part > nt ? nt : part);
        return real + k * nt + part;
    }
    return real;
}

__device__ __forceinline__ void walk_set_unit(const AttnArgs& a, Walk& w, int b) {
    w.L = clamp_len(a.ctx_lens[b], a.Lmin, a.Lmax);
    const UnitGeom g = unit_geom(a, w.L);
    w.ntiles = g.nt;
    w.ns = g.ns;
    w.gap = g.gap;
}

// Range of CTA c of n in the padded flat list: [c*Tv/n, (c+1)*Tv/n); its real tiles are what it works on.
// With one cluster per unit (cmerge): CTA c is rank c % cmerge of the cluster of unit c / cmerge and
// takes an equal share of that unit's tiles.
// (Only the plan kernel runs this.  The split kernels read what it wrote: the 64-bit divisions here
// are tens of kilobytes of code, and a split kernel that carries them no longer shares the SMs'
// instruction cache with the merge kernel, which costs every launch several microseconds.)
__device__ __forceinline__ void plan_cta(const AttnArgs& a, int cta, Walk& w) {
    w.b = 0;
    w.kvh = 0;
    w.tile = 0;
    w.L = 0;
    w.ntiles = 0;
    w.ns = 0;
    w.gap = 0;
    w.reserved = 0;
    w.remaining = 0;
    w.total = 0;
    if (a.cmerge) {
        const int unit = cta / a.cmerge, rank = cta % a.cmerge;
        w.b = unit / a.Hkv;
        w.kvh = unit % a.Hkv;
        walk_set_unit(a, w, w.b);
        const int t0 = (int)((long long)rank * w.ntiles / a.cmerge);
        const int t1 = (int)((long long)(rank + 1) * w.ntiles / a.cmerge);
        w.tile = t0;
        w.remaining = t1 - t0;
        w.total = w.ntiles;
        return;
    }
    long long T = 0;
    for (int b = 0; b < a.B; ++b) T += (long long)a.Hkv * unit_tiles(a, b);
    // with fewer tiles than CTAs only the first T CTAs work, one tile each: no CTA inside the
    // range of a unit is ever empty, which the merge relies on
    const long long nc = T < a.num_ctas ? T : a.num_ctas;
    const int pad = unit_pad(a, T);
    const long long Tv = T + (long long)pad * a.B * a.Hkv;
    long long t0 = 0, t1 = 0;
    if (cta < nc) {
        t0 = real_tiles_before(a, pad, (long long)cta * Tv / nc);
        t1 = real_tiles_before(a, pad, (long long)(cta + 1) * Tv / nc);
    }
    w.total = T;
    w.remaining = t1 - t0;
    if (w.remaining <= 0) return;
    long long t = t0;
    for (int b = 0; b < a.B; ++b) {
        const int nt = unit_tiles(a, b);
        const long long span = (long long)a.Hkv * nt;
        if (t < span) {
            w.b = b;
            w.kvh = (int)(t / nt);
            w.tile = (int)(t % nt);
            walk_set_unit(a, w, b);
            return;
        }
        t -= span;
    }
}

__device__ __forceinline__ void walk_advance(const AttnArgs& a, Walk& w, int seg) {
    w.remaining -= seg;
    w.tile += seg;
    if (w.tile >= w.ntiles) {
        w.tile = 0;
        if (++w.kvh == a.Hkv) {
            w.kvh = 0;
            ++w.b;
            if (w.b < a.B && w.remaining > 0) walk_set_unit(a, w, w.b);
        }
    }
}

// The partial slots of a unit: first CTA whose range holds one of its tiles, and how many slots
// (KS per CTA) the merge finds there.
__device__ __forceinline__ int2 unit_slot_range(const AttnArgs& a, int unit, int KS) {
    const int b = unit / a.Hkv, kvh = unit % a.Hkv;
    long long T = 0, t0 = 0;
    int nt_b = 0;
    for (int bb = 0; bb < a.B; ++bb) {
        const int nt = unit_tiles(a, bb);
        if (bb < b) t0 += (long long)a.Hkv * nt;
        if (bb == b) nt_b = nt;
        T += (long long)a.Hkv * nt;
    }
    t0 += (long long)kvh * nt_b;
    const long long units_before = (long long)b * a.Hkv + kvh;
    const long long nc = T < a.num_ctas ? T : a.num_ctas;
    // the unit's real tiles in the padded flat list the split kernel cut: [v0, v1)
    const int pad = unit_pad(a, T);
    const long long Tv = T + (long long)pad * a.B * a.Hkv;
    const long long v0 = t0 + (units_before + 1) * pad, v1 = v0 + nt_b;
    const int c_first = (int)(((v0 + 1) * nc - 1) / Tv);
    const int c_last = (int)((v1 * nc - 1) / Tv);
    return make_int2(c_first, (c_last - c_first + 1) * KS);
}

__device__ __forceinline__ void fill_plan_sig(const AttnArgs& a, int KS, int32_t (&sig)[kPlanSigInts]);

// True if the plan in the workspace was made for this call's geometry, kernel and split (the lengths
// it was made for are checked by CTA 0 alone: lengths that have moved on cannot send a kernel outside
// its buffers, a walk made for another geometry could).
__device__ __forceinline__ bool plan_matches(const AttnArgs& a, int KS) {
    int32_t want[kPlanSigInts];
    fill_plan_sig(a, KS, want);
    const uint4* src = reinterpret_cast<const uint4*>(a.plan_sig);
    bool same = true;
#pragma unroll
    for (int i = 0; i < kPlanSigInts / 4; ++i) {
        const uint4 x = __ldcg(src + i);
        same &= x.x == (uint32_t)want[4 * i] && x.y == (uint32_t)want[4 * i + 1] && x.z == (uint32_t)want[4 * i + 2] &&
                x.w == (uint32_t)want[4 * i + 3];
    }
    return same;
}

// A CTA's walk from the plan (three 16-byte loads); no work at all if the plan is not this call's.
__device__ __forceinline__ void load_walk(const AttnArgs& a, int cta, int KS, Walk& w) {
    const uint4* src = reinterpret_cast<const uint4*>(a.plan_walks + cta);
    uint4* dst = reinterpret_cast<uint4*>(&w);
    const uint4 x0 = __ldcg(src), x1 = __ldcg(src + 1), x2 = __ldcg(src + 2);
    const bool ok = plan_matches(a, KS);
    dst[0] = x0;
    dst[1] = x1;
    dst[2] = x2;
    if (!ok) {
        w.remaining = 0;
        w.b = 0;
        w.kvh = 0;
    }
}

__device__ __forceinline__ void fill_plan_sig(const AttnArgs& a, int KS, int32_t (&sig)[kPlanSigInts]) {
    const int32_t v[kPlanSigInts] = {a.B, a.Hkv, a.R, a.num_ctas, a.tile_keys, a.pad, a.stair, a.Lmin,
                                     a.Lmax, a.sink, a.window, a.cmerge, KS, 0x504c414e, 0, 0};
#pragma unroll
    for (int i = 0; i < kPlanSigInts; ++i) sig[i] = v[i];
}

// Checks of CTA 0 that only the device can make: every length inside [Lmin, Lmax], and, when a
// plan is used, that it was made for this geometry and for these lengths.
__device__ __noinline__ void check_call_inputs(const AttnArgs& a, int KS) {
    bool bad = false, stale = false;
    for (int b = 0; b < a.B; ++b) {
        const int L = a.ctx_lens[b];
        bad |= (L < a.Lmin) || (L > a.Lmax);
        if (a.caller_plan) stale |= __ldcg(a.plan_ctx + b) != L;
    }
    stale |= !plan_matches(a, KS);
    if (bad) atomicOr(a.status, RAPID_STATUS_BAD_CTX_LEN);
    if (stale) atomicOr(a.status, RAPID_STATUS_STALE_PLAN);
}

// Writes the plan of a call into its workspace: one block; thread c plans CTA c, thread u the
// slot range of unit u.
__global__ void __launch_bounds__(512) attention_plan_kernel(const __grid_constant__ AttnArgs a, int KS, Walk* walks, int2* units,
                                                             int32_t* ctx_copy, int32_t* sig_out) {
    griddep_wait();               // the lengths may come from the kernel just before this one
    griddep_launch_dependents();  // the split kernel may run its prologue; it reads the plan after its own wait
    const int n_ctas = a.cmerge ? a.B * a.Hkv * a.cmerge : a.num_ctas;
    for (int c = threadIdx.x; c < n_ctas; c += blockDim.x) {
        Walk w;
        plan_cta(a, c, w);
        walks[c] = w;
    }
    if (!a.cmerge)
        for (int u = threadIdx.x; u < a.B * a.Hkv; u += blockDim.x) units[u] = unit_slot_range(a, u, KS);
    for (int b = threadIdx.x; b < a.B; b += blockDim.x) ctx_copy[b] = a.ctx_lens[b];
    if (threadIdx.x == 0) {
        int32_t sig[kPlanSigInts];
        fill_plan_sig(a, KS, sig);
        for (int i = 0; i < kPlanSigInts; ++i) sig_out[i] = sig[i];
    }
}

// ---------------------------------------------------------------------------------------------
// Split-KV kernel on the 5th-generation tensor cores.
//
// Same work decomposition and partial format as above, but the two products run as tcgen05.mma
// with accumulators in tensor memory (TMEM):
//   S[128 x 128] = Q[128 x D] (K_n ; K_n+1)^T   two 64-key tiles per product: A = Q in shared
//                                                memory, B = the two K tiles, K-major, 128-byte swizzle
//   O[128 x D]  += P[128 x 64] V_tile            A = P in tensor memory, B = V tile, MN-major
// The grouped rows sit on the M axis (rows >= GR hold whatever memory holds; MMA rows are
// independent, so they only produce rows nobody reads).  A tcgen05.mma of 16 reduction steps
// costs about as much for 64 columns as for 128, and every commit costs its issuing thread
// about 200 cycles, so scores are produced for pairs of tiles: K tiles live in rings of their
// own (one per 64-column half) in which consecutive stages are adjacent, which lets one
// descriptor span the two tiles of a pair (pairs start at even tiles, stage counts are even).
//
// Tiles alternate between two independent softmax streams (even and odd tiles of the CTA).
// Each stream has its own half of the S buffer, O accumulator and running (reference, sum) and
// emits its own partial; the merge kernel sees two partials per CTA and unit.  Roles (352 threads):
//   warps 0-3  softmax of stream 0, warps 4-7 softmax of stream 1: a thread owns the TMEM lane
//              (= grouped row) 32*(warp%4)+lane: reads its S row, writes the bf16 probabilities
//              over the first half of the same columns, keeps the running sum, and writes the
//              partial at the end of a unit;
//   warp 8     TMA producer for K/V tiles;
//   warp 9     allocates tensor memory, loads Q by TMA and issues the QK^T MMAs;
//   warp 10    issues the PV MMAs; the commit of a tile's PV frees its K/V stage, and the same
//              barrier tells everyone else that the PV is complete.
//
// Softmax reference.  exp2(s*c - m_ref) is exact for any reference m_ref as long as nothing
// overflows, so the row maximum is not tracked tile by tile: the reference is the maximum of
// the stream's first tile and is moved (with a rescale of the O row and the sum) only when a
// tile's probabilities sum above 2^16.
//
// Barriers and phases.  Every mbarrier wait is a parity wait, which never returns if the
// barrier gets a whole phase ahead of the waiter.  Each barrier below is therefore one whose
// next phase cannot complete before all of its waiters have passed the current one:
//   full/empty[stage]   producer <-> MMA issuers (empty is also the "PV of this tile done" signal;
//                       with an even stage count a stage's next tile belongs to the same stream)
//   s_full[b]           scores of group g (b = g & 1) ready; the buffer's next group needs the PVs
//                       of this one, hence both streams past this wait
//   p_full[b][h]        probabilities of the tile in half h of buffer b published
//
// A wait whose outcome is the same for every lane of the warp (needed because the warp goes on
// to warp-collective TMEM instructions).
__device__ __forceinline__ bool warp_wait_bounded(uint64_t* bar, uint32_t parity, const WaitCtx& wc) {
    return __all_sync(0xffffffffu, mbar_wait_bounded(bar, parity, wc));
}

// Set-up of a split kernel after its input-free prologue: waits for the preceding kernel, lets the
// dependents launch and hands every thread the CTA's walk.  A settled plan (made at least two
// kernels earlier in the stream) was read before the wait, and nothing but the wait remains.
//
// Order matters here: in the plan kernel and in every split kernel launch_dependents comes after the
// wait.  A merge kernel therefore starts only once everything before its split kernel has completed,
// which is what allows it (a) to take the unit's slots from the plan before its own wait.  The merge
// kernels let their dependents go before their wait, so the next call's split kernel may start
// while this call's split kernel still runs; by then everything before THIS call's split kernel
// has completed, the plan kernel of the step included, which is what allows (b) a settled plan to be
// read before the wait, and (c) old K/V tiles to be copied there when the caller vouches for them.
__device__ __forceinline__ void split_kernel_walk(const AttnArgs& a, int cta, int KS, Walk& w, Walk* s_walk) {
    const bool settled = a.plan_mode == RAPID_PLAN_SETTLED;
    if (settled) load_walk(a, cta, KS, w);
    tc_fence_before_sync();
    __syncthreads();  // barriers initialised, tensor memory allocated
    tc_fence_after_sync();
    griddep_wait();               // inputs are read from here on
    griddep_launch_dependents();  // the merge blocks may take their seats
    if (!settled) {
        if (threadIdx.x == 0) {
            Walk t;
            load_walk(a, cta, KS, t);
            *s_walk = t;
        }
        __syncthreads();
        w = *s_walk;
    }
}

constexpr int kTcThreads = 352;
constexpr int kTcMaxStages = 8;
constexpr float kSumLimit = 65536.f;  // a tile sum at or above this moves the softmax reference

// K/V stages in the rings (even; with the 128-row Q tile they fill the 227 KB of shared memory)
__host__ __device__ constexpr int tc_stages(int D) { return D == 128 ? 6 : 8; }

struct TcLayout {
    int n_active;    // softmax warps per stream that own at least one grouped row
    uint32_t off_q;  // byte offset of the Q tile (after the K/V rings) from the 1024-aligned base
};

// Where tile n of a unit lives.  A unit's tiles n0 .. n0+seg-1 (CTA-wide indices) are grouped for
// the QK^T product: a leading single if n0 is odd, then pairs starting at even tiles, then a
// trailing single.  `group` counts groups CTA-wide (g0 = count before this unit).
struct TileSlot {
    int group;  // CTA-wide group index: S buffer = group & 1, barrier phase = (group >> 1) & 1
    int half;   // 0 or 1: which 64 columns of the buffer
};
__device__ __forceinline__ TileSlot tile_slot(int n, int n0, int g0) {
    const int lead = n0 & 1;
    TileSlot t;
    if (n == n0 && lead) {
        t.group = g0;
        t.half = 0;
    } else {
        const int m = n - n0 - lead;
        t.group = g0 + lead + (m >> 1);
        t.half = m & 1;
    }
    return t;
}
__device__ __forceinline__ int groups_in_unit(int n0, int seg) {
    const int lead = n0 & 1;
    return lead + (seg - lead + 1) / 2;
}

// MR = rows of the MMAs: 128, or 64 when the grouped rows fit (half the tensor-core work for the
// same issue cost: less power, higher clocks under the board's power cap).  With 64 rows the
// accumulator row r sits in TMEM lane 32*(r/16) + r%16: 16 lanes of each 32-lane quadrant.
template <int D, int MR>
__global__ void __launch_bounds__(kTcThreads, 1)
verify_attn_splitkv_tc_kernel(const __grid_constant__ CUtensorMap tmK,
                              const __grid_constant__ CUtensorMap tmV,
                              const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ AttnArgs a,
                              const TcLayout lay) {
    constexpr int BLK = kTile * 128;  // bytes of one 64-key x 64-column block
    constexpr int NHALF = D / 64;
    constexpr uint32_t TMEM_COLS = 512;
    constexpr uint32_t COL_S = 0;    // S buffer b at COL_S + 128 b; tile in half h at + 64 h; P over its first 32 columns
    constexpr uint32_t COL_O = 256;  // O of stream s at COL_O + 128 s

    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[kTcMaxStages];
    __shared__ uint64_t empty_bar[kTcMaxStages];
    __shared__ uint64_t s_full[2], p_full[2][2];
    __shared__ uint64_t q_full, o_free;
    __shared__ uint64_t drain_bar[2];  // an MMA issuer that leaves early sees its MMAs complete here
    __shared__ uint32_t tmem_slot;
    __shared__ Walk s_walk;
    __shared__ int s_abort;

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    const int cta = blockIdx.x;
    // The stage count is a compile-time constant: the roles below are single threads whose
    // index arithmetic (tile -> stage, phase) would otherwise be runtime divisions, and those
    // cost more than the MMAs they feed.
    constexpr int nstage = tc_stages(D);
    // shared-memory map: K rings (one per 64-column half), then V rings, then Q
    const uint32_t ring = (uint32_t)nstage * BLK;  // bytes of one ring
    const uint32_t off_k = 0, off_v = NHALF * ring;

    // Prologue that touches no input: it may overlap the tail of whatever kernel precedes this
    // one in the stream (the launch is a programmatic dependent).
    if (tid == 0) {
        for (int s = 0; s < nstage; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&s_full[i], 1);
            mbar_init(&p_full[i][0], lay.n_active);
            mbar_init(&p_full[i][1], lay.n_active);
            mbar_init(&drain_bar[i], 1);
        }
        mbar_init(&q_full, 1);
        mbar_init(&o_free, 2 * lay.n_active);
        fence_mbar_init();
        s_abort = 0;
        prefetch_tensormap(&tmK);
        prefetch_tensormap(&tmV);
        prefetch_tensormap(&tmQ);
    }
    if (warp == 9) tmem_alloc(&tmem_slot, TMEM_COLS);  // warp 9 also frees it at the end
    Walk w;
    split_kernel_walk(a, cta, kStreams, w, &s_walk);
    if (cta == 0 && warp == 8 && lane == 1) check_call_inputs(a, kStreams);  // an idle lane of the producer warp
    const uint32_t tmem_base = tmem_slot;
    const WaitCtx wc = {&s_abort, a.wait_limit};

    if (warp == 8) {
        // ---------------- TMA producer for K/V tiles ----------------
        if (lane == 0) {
            prefetch_tensormap(&tmK);
            prefetch_tensormap(&tmV);
            int n = 0;
            bool ok = true;
            while (w.remaining > 0 && ok) {
                const int seg = (int)min((long long)(w.ntiles - w.tile), w.remaining);
                for (int t = 0; t < seg && ok; ++t, ++n) {
                    const int s = n % nstage;
                    // coordinates of the tile: (key, outermost) = (logical position, sequence), or,
                    // paged, (position inside the block, physical block).  The table entry is
                    // fetched before the wait for a free stage, so the two overlap.
                    const int tile = real_tile(w, w.tile + t);
                    int key0 = tile * kTile, outer = w.b;
                    if (a.block_table) {
                        outer = __ldg(a.block_table + (size_t)w.b * a.max_blocks + (tile >> a.tile_shift));
                        key0 = (tile & ((1 << a.tile_shift) - 1)) * kTile;
                    }
                    if (n >= nstage)
                        ok = mbar_wait_bounded_relaxed(&empty_bar[s], ((n / nstage) - 1) & 1, wc);
                    if (!ok) break;
                    if (a.block_table && (unsigned)outer >= (unsigned)a.num_blocks) {
                        // the copy below reads zeros for a block outside the pool (the tensor map
                        // bounds every coordinate); say so in the status word
                        atomicOr(a.status, RAPID_STATUS_BAD_BLOCK_TABLE);
                        outer = a.num_blocks;
                    }
                    mbar_arrive_expect_tx(&full_bar[s], 2 * NHALF * BLK);
#pragma unroll
                    for (int h = 0; h < NHALF; ++h) {
                        tma_load_4d(smem_gen + off_k + h * ring + s * BLK, &tmK, &full_bar[s], h * 64,
                                    key0, w.kvh, outer);
                        tma_load_4d(smem_gen + off_v + h * ring + s * BLK, &tmV, &full_bar[s], h * 64,
                                    key0, w.kvh, outer);
                    }
                }
                walk_advance(a, w, seg);
            }
            // leaving early: the copies already issued must have landed before the CTA gives up its
            // shared memory
            if (!ok)
                for (int s = 0; s < nstage && s < n; ++s) {
                    const int u = s + (n - 1 - s) / nstage * nstage;  // the stage's latest tile
                    mbar_wait_drain(&full_bar[s], (u / nstage) & 1);
                }
        }
    } else if (warp == 9) {
        // ---------------- Q loader and QK^T issuer ----------------
        if (lane == 0) {
            prefetch_tensormap(&tmQ);
            const uint32_t idesc_1 = umma_idesc_bf16(MR, kTile, 0, 0);
            const uint32_t idesc_2 = umma_idesc_bf16(MR, 2 * kTile, 0, 0);
            // Descriptors are built once; per MMA only a small constant is added to the
            // start-address field (every address stays below 256 KB: the field never carries).
            const uint64_t k_desc = umma_smem_desc(smem_base + off_k, 16, 1024);
            const uint64_t q_desc = umma_smem_desc(smem_base + lay.off_q, 16, 1024);
            constexpr uint32_t QHALF16 = (128 * 128) >> 4;  // one 64-column half of Q: 128 rows of 128 bytes
            bool ok = true;
            int n = 0, g = 0, seg_idx = 0;
            int prev_first[2] = {-1, -1}, prev_cnt[2] = {0, 0};  // tiles of the last group in each S buffer
            while (w.remaining > 0 && ok) {
                const int seg = (int)min((long long)(w.ntiles - w.tile), w.remaining);
                // the previous unit's O rows have been read out, so all its MMAs have completed
                // and Q may be replaced
                if (seg_idx > 0) ok = mbar_wait_bounded(&o_free, (seg_idx - 1) & 1, wc);
                if (!ok) break;
                mbar_arrive_expect_tx(&q_full, (uint32_t)a.GR * D * 2);
#pragma unroll
                for (int h = 0; h < NHALF; ++h)
                    tma_load_4d(smem_gen + lay.off_q + h * (128 * 128), &tmQ, &q_full, h * 64,
                                w.kvh * a.G, 0, w.b);
                ok = mbar_wait_bounded(&q_full, seg_idx & 1, wc);
                if (!ok) mbar_wait_drain(&q_full, seg_idx & 1);  // the Q copy is on its way: let it land
                const int n_end = n + seg;
                while (n < n_end && ok) {
                    const int cnt = ((n & 1) || n + 1 >= n_end) ? 1 : 2;  // pairs start at even tiles
                    const int b = g & 1;
                    // the S buffer is free once the PVs of the group that used it last have completed
                    for (int i = 0; i < prev_cnt[b] && ok; ++i) {
                        const int pn = prev_first[b] + i;
                        ok = mbar_wait_bounded(&empty_bar[pn % nstage], (pn / nstage) & 1, wc);
                    }
                    for (int i = 0; i < cnt && ok; ++i)
                        ok = mbar_wait_bounded(&full_bar[(n + i) % nstage], ((n + i) / nstage) & 1, wc);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint64_t kd = k_desc + (uint64_t)((uint32_t)(n % nstage) * (BLK >> 4));
                    const uint32_t d = tmem_base + COL_S + 128u * b;
                    const uint32_t idesc = cnt == 2 ? idesc_2 : idesc_1;
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        const uint32_t half = kk >> 2, ko16 = (kk & 3) * 2;
                        umma_bf16_ss(d, q_desc + half * QHALF16 + ko16, kd + half * (ring >> 4) + ko16, idesc,
                                     kk > 0);
                    }
                    umma_commit(&s_full[b]);
                    prev_first[b] = n;
                    prev_cnt[b] = cnt;
                    n += cnt;
                    ++g;
                }
                walk_advance(a, w, seg);
                ++seg_idx;
            }
            if (!ok) {  // leaving early: every MMA issued here must have completed before tensor memory is freed
                umma_commit(&drain_bar[0]);
                mbar_wait_drain(&drain_bar[0], 0);
            }
        }
    } else if (warp == 10) {
        // ---------------- PV issuer ----------------
        if (lane == 0) {
            const uint32_t idesc_pv = umma_idesc_bf16(MR, D, 0, 1);
            // V tile as MN-major B: 64-column blocks `ring` bytes apart, 8-key groups 1024 bytes apart
            const uint64_t v_desc = umma_smem_desc(smem_base + off_v, ring, 1024);
            bool ok = true;
            int n = 0, g0 = 0;
            // p_full[b][0] completes one phase per group of buffer b, p_full[b][1] only for the
            // groups that are pairs: its phase is counted here
            int pairs_seen[2] = {0, 0};
            while (w.remaining > 0 && ok) {
                const int seg = (int)min((long long)(w.ntiles - w.tile), w.remaining);
                const int n0 = n;
                for (int t = 0; t < seg && ok; ++t, ++n) {
                    const TileSlot ts = tile_slot(n, n0, g0);
                    const int b = ts.group & 1;
                    // P(n) is published only after its stream has read the previous unit's O row
                    const int phase = ts.half ? pairs_seen[b]++ : (ts.group >> 1);
                    ok = mbar_wait_bounded(&p_full[b][ts.half], phase & 1, wc);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint64_t vd = v_desc + (uint64_t)((uint32_t)(n % nstage) * (BLK >> 4));
                    const uint32_t tP = tmem_base + COL_S + 128u * b + 64u * ts.half;
                    const uint32_t d = tmem_base + COL_O + 128u * (n & 1);
#pragma unroll
                    for (int kk = 0; kk < kTile / 16; ++kk)
                        umma_bf16_ts(d, tP + 8 * kk, vd + kk * (2048 >> 4), idesc_pv,
                                     (t >= 2 || kk > 0) ? 1u : 0u);
                    umma_commit(&empty_bar[n % nstage]);  // PV(n) complete: stage free, P/S columns free
                }
                g0 += groups_in_unit(n0, seg);
                walk_advance(a, w, seg);
            }
            if (!ok) {
                umma_commit(&drain_bar[1]);
                mbar_wait_drain(&drain_bar[1], 0);
            }
        }
    } else if ((warp & 3) < lay.n_active) {
        // ---------------- softmax warps: stream = warp / 4, grouped row = 32 (warp % 4) + lane ----------------
        const int stream = warp >> 2;
        const int quad = warp & 3;
        constexpr int RPQ = MR / 4;  // accumulator rows per 32-lane quadrant
        const int row = quad * RPQ + lane;
        const bool row_valid = lane < RPQ && row < a.GR;
        const int sidx = quad * 32 + lane;  // thread index within the stream's warps
        const int i_row = row_valid ? row / a.G : 0;
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        const uint32_t tO = tmem_base + lane_base + COL_O + 128u * stream;
        const float c = a.scale_log2;
        const int slot_stride = (int)slot_floats(a.GR, D);

        int n0 = 0, g0 = 0;  // CTA-wide tile / group index of the unit's first tile / group
        bool ok = true;
        while (w.remaining > 0 && ok) {
            const int seg = (int)min((long long)(w.ntiles - w.tile), w.remaining);
            const int L = w.L;
            const int lim = a.stair ? L - a.R + i_row : L - 1;
            const int all_see = a.stair ? L - a.R : L - 1;  // the last key every row sees
            // sink + window: keys in [sink, lo] are hidden from this row; lo_max is the newest key
            // that some row does not see any more
            const int lo = a.window > 0 ? lim - a.window : -1;
            const int lo_max = a.window > 0 ? L - 1 - a.window : -1;
            float m_ref = -INFINITY, l_run = 0.f;
            int last_n = -1;  // the stream's latest tile of this unit (CTA-wide index)

            for (int n = n0 + ((n0 ^ stream) & 1); n < n0 + seg && ok; n += 2) {
                const int key0 = real_tile(w, w.tile + (n - n0)) * kTile;
                const TileSlot ts = tile_slot(n, n0, g0);
                const uint32_t tS = tmem_base + lane_base + COL_S + 128u * (ts.group & 1) + 64u * ts.half;
                ok = warp_wait_bounded(&s_full[ts.group & 1], (ts.group >> 1) & 1, wc);
                if (!ok) break;
                tc_fence_after_sync();
                uint32_t sr[2][32];
                tmem_ld_x32(tS, sr[0]);
                tmem_ld_x32(tS + 32, sr[1]);
                tmem_wait_ld();

                // causal rows and the ragged end of the context, or the old edge of the windows: a key is
                // hidden from this row if it lies past lim or inside [hid0, lo]
                if (key0 + kTile - 1 > all_see || (key0 <= lo_max && key0 + kTile > a.sink)) {
                    const int hid0 = a.window > 0 ? a.sink : 0x7fffffff;
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int k = 0; k < 32; ++k) {
                            const int key = key0 + h * 32 + k;
                            if (key > lim || (key >= hid0 && key <= lo)) sr[h][k] = __float_as_uint(-INFINITY);
                        }
                }

                uint32_t pk[32];
                float sum = 0.f;
                auto exponentials = [&](float m_use) {
                    float s0 = 0.f, s1 = 0.f;
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int k = 0; k < 32; k += 2) {
                            const float p0 = fast_exp2(fmaf(__uint_as_float(sr[h][k]), c, -m_use));
                            const float p1 = fast_exp2(fmaf(__uint_as_float(sr[h][k + 1]), c, -m_use));
                            s0 += p0;
                            s1 += p1;
                            pk[h * 16 + (k >> 1)] = pack_bf16x2(p0, p1);
                        }
                    sum = s0 + s1;
                };
                const bool first = last_n < 0;
                bool redo = row_valid && m_ref == -INFINITY;
                if (!first) {
                    exponentials(m_ref == -INFINITY ? 0.f : m_ref);
                    redo = redo || (row_valid && !(sum < kSumLimit));
                }
                if (first || __any_sync(0xffffffffu, redo)) {
                    float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int k = 0; k < 32; ++k)
                            mx[k & 3] = fmaxf(mx[k & 3], __uint_as_float(sr[h][k]));
                    const float tile_max = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * c;
                    float factor = 1.f;
                    if (redo && tile_max > m_ref) {
                        factor = fast_exp2(m_ref - tile_max);  // 0 when there was no reference yet
                        l_run *= factor;
                        m_ref = tile_max;
                    }
                    if (!first) {
                        // O must be at rest (the stream's previous PV complete) while rows are rescaled
                        ok = warp_wait_bounded(&empty_bar[last_n % nstage], (last_n / nstage) & 1, wc);
                        if (!ok) break;
                        tc_fence_after_sync();
#pragma unroll
                        for (int c4 = 0; c4 < D / 32; ++c4) {
                            uint32_t orow[32];
                            tmem_ld_x32(tO + 32 * c4, orow);
                            tmem_wait_ld();
#pragma unroll
                            for (int k = 0; k < 32; ++k)
                                orow[k] = __float_as_uint(__uint_as_float(orow[k]) * factor);
                            tmem_st_x32(tO + 32 * c4, orow);
                        }
                        tmem_wait_st();
                    }
                    exponentials(m_ref == -INFINITY ? 0.f : m_ref);
                }
                l_run += sum;

                tmem_st_x32(tS, pk);  // P over the first half of the tile's own S columns
                if (key0 + kTile > L) {
                    // V rows beyond the context may hold any bits: zero them so that 0 * row = 0
                    const int first_bad = L - key0;
                    const int chunks = (kTile - first_bad) * 8;
                    for (int h = 0; h < NHALF; ++h) {
                        uint8_t* vgen = smem_gen + off_v + h * ring + (size_t)(n % nstage) * BLK;
                        for (int ch = sidx; ch < chunks; ch += lay.n_active * 32)
                            *reinterpret_cast<uint4*>(vgen + first_bad * 128 + ch * 16) = make_uint4(0, 0, 0, 0);
                    }
                    fence_proxy_async_smem();
                }
                tmem_wait_st();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&p_full[ts.group & 1][ts.half]);
                last_n = n;
            }
            if (!ok) break;

            // ---- end of the unit: read the O row out of tensor memory and emit the partial ----
            const int unit = w.b * a.Hkv + w.kvh;
            float* slot = a.partial + ((size_t)(cta + unit) * 2 + stream) * slot_stride;
            if (last_n >= 0) {
                ok = warp_wait_bounded(&empty_bar[last_n % nstage], (last_n / nstage) & 1, wc);
                if (!ok) break;
                tc_fence_after_sync();
#pragma unroll
                for (int c4 = 0; c4 < D / 32; ++c4) {
                    uint32_t orow[32];
                    tmem_ld_x32(tO + 32 * c4, orow);
                    tmem_wait_ld();
                    if (row_valid && m_ref != -INFINITY) {
#pragma unroll
                        for (int k = 0; k < 32; k += 4)
                            *reinterpret_cast<uint4*>(slot + (size_t)row * D + 32 * c4 + k) =
                                make_uint4(orow[k], orow[k + 1], orow[k + 2], orow[k + 3]);
                    }
                }
            }
            if (row_valid) {
                slot[a.GR * D + row] = m_ref;
                slot[a.GR * D + a.GR + row] = l_run;
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&o_free);
            g0 += groups_in_unit(n0, seg);
            n0 += seg;
            walk_advance(a, w, seg);
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 9) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
    if (tid == 0 && s_abort) atomicOr(a.status, RAPID_STATUS_PIPELINE_TIMEOUT);
}

#include "attention_kt.cuh"
#include "attention_kt8.cuh"

// Merge: out = sum_s 2^(m_s - M) O_s / sum_s 2^(m_s - M) l_s over the partials of a unit.
// One block of 4 warps per (grouped row, unit): warp w takes the slots j = w, w+4, ... (four
// loads in flight per lane), lanes span D; the four warp sums are added in warp order, so the
// result does not depend on timing.
template <int D>
__global__ void __launch_bounds__(128)
verify_attn_merge_kernel(const __grid_constant__ AttnArgs a, int KS, __nv_bfloat16* out, float* lse_out,
                         float* out_f32) {
    constexpr int VEC = D / 32;
    constexpr int UN = 10;
    __shared__ float sh_acc[4][D];
    __shared__ float sh_l[4];
    const int m = blockIdx.x;
    const int unit = blockIdx.y;
    const int b = unit / a.Hkv;
    const int kvh = unit % a.Hkv;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;

    // The unit's slots, from the plan.  It is read before the wait although an earlier kernel of the
    // stream wrote it: this kernel starts only after every CTA of the split kernel has passed its own
    // wait (it lets its dependents launch after it), and by then everything before the split kernel,
    // the plan kernel included, has completed.
    const int2 range = plan_matches(a, KS) ? __ldcg(a.plan_units + unit) : make_int2(0, 0);  // not this call's plan: nothing to merge
    const int c_first = range.x;
    const int nslots = range.y;
    const size_t slot_stride = (size_t)slot_floats(a.GR, D);
    const float* base = a.partial + (size_t)(c_first + unit) * KS * slot_stride;  // slots are consecutive

    // everything above depends on the call's inputs only; the partials need the split kernel
    // After a keys-on-M split kernel dependents may launch BEFORE this kernel's own wait: see
    // verify_attn_merge_rows_kernel for why that is safe for what the library's kernels do ahead of
    // their waits.
    if (a.merge_early) asm volatile("griddepcontrol.launch_dependents;");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (!a.merge_early) asm volatile("griddepcontrol.launch_dependents;");
    if (nslots <= 0) {  // the plan is not this call's (status says so): defined output, nothing read
        if (warp == 0) {
            const size_t row = ((size_t)b * a.R + m / a.G) * a.Hq + (size_t)kvh * a.G + m % a.G;
            for (int d = lane; d < D; d += 32) {
                out[row * D + d] = __float2bfloat16_rn(0.f);
                if (out_f32) out_f32[row * D + d] = 0.f;
            }
            if (lse_out && lane == 0) lse_out[row] = -INFINITY;
        }
        return;
    }

    // Warp w takes the slots j = w, w + 4, ...  The O rows of its first UN slots are requested at
    // once, together with every slot's running maximum: neither depends on the other, so the common
    // case (at most 4 * UN slots per unit) costs one round trip to the partials, not three.
    float ov[UN][VEC], ms[UN], lv[UN];
    auto fetch = [&](int j0) {
#pragma unroll
        for (int u = 0; u < UN; ++u) {
            const int j = min(j0 + 4 * u, nslots - 1);  // past the end: any valid slot, never used
            ms[u] = base[(size_t)j * slot_stride + a.GR * D + m];
            lv[u] = base[(size_t)j * slot_stride + a.GR * D + a.GR + m];  // garbage in an untouched slot: unused
            const float* slot = base + (size_t)j * slot_stride + (size_t)m * D + lane * VEC;
            if (VEC == 4) {
                const float4 t = *reinterpret_cast<const float4*>(slot);
                ov[u][0] = t.x; ov[u][1] = t.y; ov[u][2] = t.z; ov[u][VEC - 1] = t.w;
            } else {
                const float2 t = *reinterpret_cast<const float2*>(slot);
                ov[u][0] = t.x; ov[u][1] = t.y;
            }
        }
    };
    fetch(warp);
    float M = -INFINITY;
    for (int j = lane; j < nslots; j += 32) M = fmaxf(M, base[j * slot_stride + a.GR * D + m]);
#pragma unroll
    for (int o = 16; o; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));

    float acc[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) acc[e] = 0.f;
    float lsum = 0.f;
    for (int j0 = warp; j0 < nslots; j0 += 4 * UN) {
        if (j0 != warp) fetch(j0);
#pragma unroll
        for (int u = 0; u < UN; ++u) {
            const int j = j0 + 4 * u;
            if (j >= nslots || ms[u] == -INFINITY) continue;  // an untouched slot holds no O: its bits are never used
            const float wgt = exp2f(ms[u] - M);
            lsum += wgt * lv[u];
#pragma unroll
            for (int e = 0; e < VEC; ++e) acc[e] += wgt * ov[u][e];
        }
    }
#pragma unroll
    for (int e = 0; e < VEC; ++e) sh_acc[warp][lane * VEC + e] = acc[e];
    if (lane == 0) sh_l[warp] = lsum;
    __syncthreads();
    if (warp == 0) {
        const float l = ((sh_l[0] + sh_l[1]) + sh_l[2]) + sh_l[3];
        const int i = m / a.G;
        const int g = m % a.G;
        const size_t row = ((size_t)b * a.R + i) * a.Hq + (size_t)kvh * a.G + g;
#pragma unroll
        for (int e = 0; e < VEC; ++e) {
            const int d = lane * VEC + e;
            const float val = (((sh_acc[0][d] + sh_acc[1][d]) + sh_acc[2][d]) + sh_acc[3][d]) / l;
            out[row * D + d] = __float2bfloat16_rn(val);
            if (out_f32) out_f32[row * D + d] = val;
        }
        if (lse_out && lane == 0) lse_out[row] = (M + log2f(l)) * 0.69314718055994530942f;
    }
}

// The same merge as one WARP per (grouped row, unit), four rows to a block, for the keys-on-M kernel with
// one softmax group (one partial per CTA and unit: some twenty slots per unit when the SMs share eight
// units).  It uses no shared memory and few enough registers for a block to sit on an SM BESIDE a CTA of
// that split kernel: the merge blocks of a layer are resident while its split kernel runs and start
// the moment it completes, with every slot of a row requested at once.
//
// It lets its dependents launch BEFORE its own wait.  The kernel that follows it on the stream may
// therefore start while this layer's split kernel still runs (its CTAs take the SMs as this layer's
// CTAs leave them).  That is safe for what the library's kernels do ahead of their own waits: they
// read a settled plan (complete before this layer's split kernel passed its wait, or this kernel
// could not have been launched) and, where the caller vouches for it, old entries of a K/V cache
// (rapid_attn_params.kv_settled); everything else they read after their wait, which ends only when
// this kernel has completed.
template <int D>
__global__ void __launch_bounds__(128)
verify_attn_merge_rows_kernel(const __grid_constant__ AttnArgs a, __nv_bfloat16* out, float* lse_out,
                              float* out_f32) {
    constexpr int VEC = D / 32;
    constexpr int UN = 20;
    const int lane = threadIdx.x & 31;
    const int m = blockIdx.x * 4 + (threadIdx.x >> 5);
    const int unit = blockIdx.y;
    const int b = unit / a.Hkv;
    const int kvh = unit % a.Hkv;
    // the unit's slots, from the plan (read before the wait: see verify_attn_merge_kernel)
    const int2 range = plan_matches(a, 1) ? __ldcg(a.plan_units + unit) : make_int2(0, 0);
    const int c_first = range.x;
    const int nslots = range.y;
    const size_t slot_stride = (size_t)slot_floats(a.GR, D);
    const float* base = a.partial + (size_t)(c_first + unit) * slot_stride;  // slots are consecutive
    asm volatile("griddepcontrol.launch_dependents;");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (m >= a.GR) return;
    const size_t row = ((size_t)b * a.R + m / a.G) * a.Hq + (size_t)kvh * a.G + m % a.G;
    if (nslots <= 0) {  // the plan is not this call's (status says so): defined output, nothing read
        for (int d = lane; d < D; d += 32) {
            out[row * D + d] = __float2bfloat16_rn(0.f);
            if (out_f32) out_f32[row * D + d] = 0.f;
        }
        if (lse_out && lane == 0) lse_out[row] = -INFINITY;
        return;
    }
    // Slots are taken UN at a time (usually all at once): their O rows are requested first, lane u then
    // fetches the reference and the sum of slot u, and the weights go round by shuffle.
    float ov[UN][VEC];
    auto fetch = [&](int j0) {
#pragma unroll
        for (int u = 0; u < UN; ++u) {
            const int j = min(j0 + u, nslots - 1);  // past the end: any valid slot, never used
            const float* slot = base + (size_t)j * slot_stride + (size_t)m * D + lane * VEC;
            if (VEC == 4) {
                const float4 t = *reinterpret_cast<const float4*>(slot);
                ov[u][0] = t.x; ov[u][1] = t.y; ov[u][2] = t.z; ov[u][VEC - 1] = t.w;
            } else {
                const float2 t = *reinterpret_cast<const float2*>(slot);
                ov[u][0] = t.x; ov[u][1] = t.y;
            }
        }
    };
    fetch(0);
    // lane u's slot of the first round: its reference and its sum, requested together with the O rows
    // (the sum of an untouched slot is garbage and is never used: selected away, not multiplied)
    float mj = -INFINITY, lj = 0.f;
    if (lane < UN && lane < nslots) {
        mj = base[(size_t)lane * slot_stride + a.GR * D + m];
        lj = base[(size_t)lane * slot_stride + a.GR * D + a.GR + m];
    }
    float M = mj;
    for (int j = UN + lane; j < nslots; j += 32) M = fmaxf(M, base[j * slot_stride + a.GR * D + m]);  // rarely any
#pragma unroll
    for (int o = 16; o; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    float acc[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) acc[e] = 0.f;
    float lpart = 0.f;  // lane u: the sums of the slots u, u + UN, ...
    for (int j0 = 0; j0 < nslots; j0 += UN) {  // slots in their order: the result does not depend on timing
        if (j0) {
            fetch(j0);
            mj = -INFINITY;
            if (lane < UN && j0 + lane < nslots) {
                mj = base[(size_t)(j0 + lane) * slot_stride + a.GR * D + m];
                lj = base[(size_t)(j0 + lane) * slot_stride + a.GR * D + a.GR + m];
            }
        }
        float w = 0.f;
        if (mj != -INFINITY) {  // an untouched slot holds neither a sum nor an O row
            w = exp2f(mj - M);
            lpart += w * lj;
        }
#pragma unroll
        for (int u = 0; u < UN; ++u) {
            const float wu = __shfl_sync(0xffffffffu, w, u);
            if (wu == 0.f) continue;
#pragma unroll
            for (int e = 0; e < VEC; ++e) acc[e] += wu * ov[u][e];
        }
    }
    float lsum = lpart;  // a fixed tree over the lanes
#pragma unroll
    for (int o = 16; o; o >>= 1) lsum += __shfl_xor_sync(0xffffffffu, lsum, o);
#pragma unroll
    for (int e = 0; e < VEC; ++e) {
        const int d = lane * VEC + e;
        const float val = acc[e] / lsum;
        out[row * D + d] = __float2bfloat16_rn(val);
        if (out_f32) out_f32[row * D + d] = val;
    }
    if (lse_out && lane == 0) lse_out[row] = (M + log2f(lsum)) * 0.69314718055994530942f;
}

// Combines P partial attention results of the same rows over disjoint key sets (each normalised
// by its own sum, with the natural-log sum-exp of its scores) into the result over the union:
//   out = sum_p w_p o_p,  w_p = exp(lse_p - LSE),  LSE = log sum_p exp(lse_p).
// One warp per row; a partial with lse = -inf (no keys) takes no part.
__global__ void __launch_bounds__(128) merge_partials_kernel(const float* __restrict__ o_parts,
                                                             const float* __restrict__ lse_parts, int P,
                                                             long long rows, int D, __nv_bfloat16* out,
                                                             float* out_f32, float* lse_out) {
    const long long row = (long long)blockIdx.x * 4 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;");
    if (row >= rows) return;
    float M = -INFINITY;
    for (int p = 0; p < P; ++p) M = fmaxf(M, lse_parts[(size_t)p * rows + row]);
    float den = 0.f;
    for (int p = 0; p < P; ++p) {
        const float l = lse_parts[(size_t)p * rows + row];
        den += (l == -INFINITY) ? 0.f : __expf(l - M);
    }
    for (int d = lane; d < D; d += 32) {
        float acc = 0.f;
        for (int p = 0; p < P; ++p) {
            const float l = lse_parts[(size_t)p * rows + row];
            if (l != -INFINITY) acc += __expf(l - M) * o_parts[((size_t)p * rows + row) * D + d];
        }
        const float val = (M == -INFINITY) ? 0.f : acc / den;
        if (out) out[row * D + d] = __float2bfloat16_rn(val);
        if (out_f32) out_f32[row * D + d] = val;
    }
    if (lse_out && lane == 0) lse_out[row] = (M == -INFINITY) ? -INFINITY : M + logf(den);
}

// ---- host side ----------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) !=
                cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            return nullptr;
        fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// Tensor map of a cache [outer][Hkv][keys][D] with element strides sb / sh / sl: outer = sequences
// and keys = Lmax for a contiguous cache, outer = physical blocks and keys = block size for a paged one.
int make_kv_map(CUtensorMap* map, const void* base, const rapid_attn_shape& s, int64_t outer,
                int64_t keys, int64_t sb, int64_t sh, int64_t sl, int box_rows, bool fp8 = false) {
    EncodeTiledFn enc = get_encode_fn();
    if (!enc) {
        set_error("cuTensorMapEncodeTiled is not available from the CUDA driver");
        return RAPID_ERR_CUDA;
    }
    cuuint64_t dims[4] = {(cuuint64_t)s.D, (cuuint64_t)keys, (cuuint64_t)s.Hkv, (cuuint64_t)outer};
    // bf16: boxes of 64 columns (128 bytes); E4M3 codes: the whole 128-byte row of a key
    const cuuint64_t esz = fp8 ? 1 : 2;
    cuuint64_t strides[3] = {(cuuint64_t)sl * esz, (cuuint64_t)sh * esz, (cuuint64_t)sb * esz};
    cuuint32_t box[4] = {fp8 ? 128u : 64u, (cuuint32_t)box_rows, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(map, fp8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims,
                     strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_error("cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
        return RAPID_ERR_CUDA;
    }
    return RAPID_OK;
}

int make_q_map(CUtensorMap* map, const void* q, const rapid_attn_shape& s, int G, int R) {
    EncodeTiledFn enc = get_encode_fn();
    if (!enc) {
        set_error("cuTensorMapEncodeTiled is not available from the CUDA driver");
        return RAPID_ERR_CUDA;
    }
    // q [B, R, Hq, D]: a box of (64 columns, G heads, R rows) lands as G*R rows of 128 bytes,
    // row index i*G + g: the grouped-row order the kernels use
    cuuint64_t dims[4] = {(cuuint64_t)s.D, (cuuint64_t)s.Hq, (cuuint64_t)R, (cuuint64_t)s.B};
    cuuint64_t strides[3] = {(cuuint64_t)s.D * 2, (cuuint64_t)s.Hq * s.D * 2,
                             (cuuint64_t)R * s.Hq * s.D * 2};
    cuuint32_t box[4] = {64, (cuuint32_t)G, (cuuint32_t)R, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(q), dims, strides,
                     box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_error("cuTensorMapEncodeTiled (q) failed with CUresult %d", (int)r);
        return RAPID_ERR_CUDA;
    }
    return RAPID_OK;
}

constexpr int kMaxSmemOptin = 232448 - 1024;  // 227 KB per CTA on sm_100, less the static barriers
// Longest cache for which the library itself picks one cluster per KV head: the clusters leave some
// SMs without work, which a short run wins back by having no merge kernel.
constexpr int64_t kClusterMaxKeys = 65536;

template <int D, int MR>
int launch_split_tc(const CUtensorMap& tmK, const CUtensorMap& tmV, const CUtensorMap& tmQ,
                    const AttnArgs& a, cudaStream_t stream) {
    TcLayout lay;
    lay.n_active = (a.GR + MR / 4 - 1) / (MR / 4);
    const int qbytes = (D / 64) * 128 * 128;  // the MMAs read 128 rows of Q whatever GR is
    constexpr int nstage = tc_stages(D);  // even: pairs of tiles sit in adjacent stages, no wrap
    static_assert(nstage * stage_bytes(D) + (D / 64) * 128 * 128 + 1024 <= kMaxSmemOptin, "shared memory");
    static_assert(nstage <= kTcMaxStages && nstage % 2 == 0, "stage count");
    lay.off_q = (uint32_t)(nstage * stage_bytes(D));
    const int smem = nstage * stage_bytes(D) + qbytes + 1024;
    static bool configured[64] = {};
    int dev = 0;
    RAPID_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev >= 64 || !configured[dev]) {
        RAPID_CUDA_CHECK(cudaFuncSetAttribute(verify_attn_splitkv_tc_kernel<D, MR>,
                                              cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              kMaxSmemOptin));
        if (dev < 64) configured[dev] = true;
    }
    // programmatic dependent launch: the kernel's input-free prologue may overlap the tail of the
    // preceding kernel; it waits for that kernel's completion before it reads anything
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(a.num_ctas);
    cfg.blockDim = dim3(kTcThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    RAPID_CUDA_CHECK(cudaLaunchKernelEx(&cfg, verify_attn_splitkv_tc_kernel<D, MR>, tmK, tmV, tmQ, a, lay));
    return RAPID_OK;
}

int sm_count() {
    static int n = 0;
    if (!n) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) n = 0;
    }
    return n;
}

// Tiles of streaming a unit switch is charged with.  The switch itself takes about 7 us against
// 0.75 us per tile and SM at head_dim 128; swept on the 8B, 70B and ragged 7B shapes, the launch
// time falls until 8 and is flat from 8 to 12 (-4.3 % to -4.6 % against no padding).
int unit_switch_tiles(int D) { return D == 128 ? 10 : 12; }

bool attn_shape_ok(const rapid_attn_shape* s, int gamma) {
    if (!s) return false;
    if (s->B <= 0 || s->Hq <= 0 || s->Hkv <= 0 || s->Lmax <= 0 || gamma < 0) return false;
    if (s->Hq % s->Hkv != 0) return false;
    return true;
}

}  // namespace

// Largest cluster (16, 8, 4, 2) of this kernel of which `clusters_needed` fit on the device at once;
// 0 if none does.  Asked of the runtime once per device, kernel and size.
// Per-device attributes of a keys-on-M kernel: its dynamic shared memory, and clusters of 16 CTAs.
template <int NC, int SG, bool WIN>
cudaError_t kt_configure(int dev) {
    constexpr int smem = kt::smem_bytes(NC);
    static_assert(smem <= kMaxSmemOptin - 4096, "shared memory (dynamic + the kernel's static arrays)");
    static bool configured[64] = {};
    if (dev >= 0 && dev < 64 && configured[dev]) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(kt::verify_attn_splitkv_kt_kernel<NC, SG, WIN>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(kt::verify_attn_splitkv_kt_kernel<NC, SG, WIN>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) configured[dev] = true;
    return cudaSuccess;
}

// Clusters of `size` CTAs (16, 8, 4 or 2) of this kernel that can be resident on the device together;
// 0 if none.  Asked of the runtime once per device, kernel and size.
template <int NC, int SG, bool WIN = false>
int kt_resident_clusters(int size, int dev) {
    constexpr int smem = kt::smem_bytes(NC);
    static int resident[64][4] = {};  // by size 16, 8, 4, 2 (0 = not asked yet, -1 = none)
    const int i = size == 16 ? 0 : size == 8 ? 1 : size == 4 ? 2 : size == 2 ? 3 : -1;
    if (dev < 0 || dev >= 64 || i < 0) return 0;
    if (!resident[dev][i]) {
        int n = 0;
        if (kt_configure<NC, SG, WIN>(dev) == cudaSuccess) {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(size);
            cfg.blockDim = dim3(kt::threads(SG));
            cfg.dynamicSmemBytes = smem;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = size;
            attr[0].val.clusterDim.y = 1;
            attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            if (cudaOccupancyMaxActiveClusters(&n, kt::verify_attn_splitkv_kt_kernel<NC, SG, WIN>, &cfg) != cudaSuccess) n = 0;
        }
        cudaGetLastError();
        resident[dev][i] = n > 0 ? n : -1;
    }
    return resident[dev][i] > 0 ? resident[dev][i] : 0;
}

// Largest cluster of which `clusters_needed` fit on the device at once; 0 if none does.
template <int NC, int SG, bool WIN = false>
int kt_cluster_size_that_fits(int clusters_needed, int dev) {
    const int sizes[4] = {16, 8, 4, 2};
    for (int i = 0; i < 4; ++i)
        if (kt_resident_clusters<NC, SG, WIN>(sizes[i], dev) >= clusters_needed) return sizes[i];
    return 0;
}

template <int NC, int SG, bool WIN>
int launch_split_kt_w(const CUtensorMap& tmK, const CUtensorMap& tmV, const CUtensorMap& tmQ, AttnArgs& a,
                      cudaStream_t stream, bool want_cluster, bool need_cluster) {
    constexpr int smem = kt::smem_bytes(NC);
    int dev = 0;
    RAPID_CUDA_CHECK(cudaGetDevice(&dev));
    RAPID_CUDA_CHECK((kt_configure<NC, SG, WIN>(dev)));
    const int units = a.B * a.Hkv;
    a.cmerge = 0;
    if (want_cluster) {
        // (the kernel with and without the window mask take the same resources: one answer for both)
        const int cs = kt_cluster_size_that_fits<NC, SG>(units, dev);
        // on the library's own choice the clusters must also cover most of the machine
        if (cs && (need_cluster || units * cs * 4 >= sm_count() * 3)) a.cmerge = cs;
        if (!a.cmerge && need_cluster) {
            set_error("rapid_verify_attention: %d clusters (one per sequence and KV head) do not fit on the device "
                      "together", units);
            return RAPID_ERR_UNSUPPORTED;
        }
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(a.cmerge ? units * a.cmerge : a.num_ctas);
    cfg.blockDim = dim3(kt::threads(SG));
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (a.cmerge) {
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = a.cmerge;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        cfg.numAttrs = 2;
    }
    RAPID_CUDA_CHECK(cudaLaunchKernelEx(&cfg, kt::verify_attn_splitkv_kt_kernel<NC, SG, WIN>, tmK, tmV, tmQ,
                                        static_cast<const AttnArgs&>(a)));
    return RAPID_OK;
}

template <int NC, int SG = 1>
int launch_split_kt(const CUtensorMap& tmK, const CUtensorMap& tmV, const CUtensorMap& tmQ, AttnArgs& a,
                    cudaStream_t stream, bool want_cluster, bool need_cluster) {
    return a.window > 0 ? launch_split_kt_w<NC, SG, true>(tmK, tmV, tmQ, a, stream, want_cluster, need_cluster)
                        : launch_split_kt_w<NC, SG, false>(tmK, tmV, tmQ, a, stream, want_cluster, need_cluster);
}

// fp32_sums: the caller takes the log-sum-exp, so the row sums must add fp32 probabilities.  With
// 49 to 64 grouped rows one softmax group has no registers for that (it adds the bf16 values the
// tensor cores multiply); two groups of 32 columns each do.
int dispatch_split_kt(int NC, bool fp32_sums, bool two_groups, const CUtensorMap& tmK, const CUtensorMap& tmV,
                      const CUtensorMap& tmQ, AttnArgs& a, cudaStream_t stream, bool want_cluster, bool need_cluster) {
    switch (NC) {
        case 1:
            return two_groups ? launch_split_kt<1, 2>(tmK, tmV, tmQ, a, stream, want_cluster, need_cluster)
                              : launch_split_kt<1>(tmK, tmV, tmQ, a, stream, want_cluster, need_cluster);
        case 2:
            return two_groups ? launch_split_kt<2, 2>(tmK, tmV, tmQ, a, stream, want_cluster, need_cluster)
                              : launch_split_kt<2>(tmK, tmV, tmQ, a, stream, want_cluster, need_cluster);
        case 3:
            return two_groups ? launch_split_kt<3, 2>(tmK, tmV, tmQ, a, stream, want_cluster, need_cluster)
                              : launch_split_kt<3>(tmK, tmV, tmQ, a, stream, want_cluster, need_cluster);
        case 4:
            return (fp32_sums || two_groups) ? launch_split_kt<4, 2>(tmK, tmV, tmQ, a, stream, want_cluster, need_cluster)
                             : launch_split_kt<4>(tmK, tmV, tmQ, a, stream, want_cluster, need_cluster);
        // more than 64 grouped rows: two softmax groups, each with half of the columns
        case 5: return launch_split_kt<5, 2>(tmK, tmV, tmQ, a, stream, want_cluster, need_cluster);
        case 6: return launch_split_kt<6, 2>(tmK, tmV, tmQ, a, stream, want_cluster, need_cluster);
    }
    set_error("unsupported number of grouped rows");
    return RAPID_ERR_UNSUPPORTED;
}

int launch_merge_partials(const float* o_parts, const float* lse_parts, int P, int64_t rows, int D, void* out,
                          float* out_f32, float* lse_out, cudaStream_t stream) {
    if (!o_parts || !lse_parts || (!out && !out_f32) || P <= 0 || rows <= 0 || D <= 0) {
        set_error("rapid_merge_partials: NULL argument or non-positive size");
        return RAPID_ERR_INVALID_ARG;
    }
    const int64_t blocks = (rows + 3) / 4;
    if (blocks > 0x7fffffffLL) {
        set_error("rapid_merge_partials: too many rows");
        return RAPID_ERR_UNSUPPORTED;
    }
    RAPID_CUDA_CHECK(launch_dependent(merge_partials_kernel, dim3((unsigned)blocks), dim3(128), 0, stream, o_parts,
                                      lse_parts, P, (long long)rows, D, static_cast<__nv_bfloat16*>(out), out_f32,
                                      lse_out));
    count_launch(1);
    return RAPID_OK;
}

namespace {

// Where things live in an attention workspace (bytes from its start).
struct WsLayout {
    size_t sig, walks, units, ctx, partial, total;
};
WsLayout ws_layout(int B, int Hkv, int GR, int D) {
    WsLayout l;
    size_t off = kWorkspaceHeaderBytes;
    l.sig = off;
    off += align_up(kPlanSigInts * sizeof(int32_t), 256);
    l.walks = off;
    off += align_up((size_t)kMaxCtas * sizeof(Walk), 256);
    l.units = off;
    off += align_up((size_t)B * Hkv * sizeof(int2), 256);
    l.ctx = off;
    off += align_up((size_t)B * sizeof(int32_t), 256);
    l.partial = off;
    const int64_t slots = ((int64_t)kMaxCtas + (int64_t)B * Hkv) * kStreams;
    off += (size_t)slots * slot_floats(GR, D) * sizeof(float);
    l.total = off;
    return l;
}

// Everything the attention entry points share: validation, the choice of kernel, the arguments.
struct AttnCall {
    AttnArgs a;
    bool kt_path, kt_half_blocks, fp32_sums, want_cluster, need_cluster, few_slots, two_groups;
    int NC, KS, box_rows;
    int64_t sl, sh, sb, outer, keys;
};

int prepare_attention(const char* who, const int32_t* ctx_lens, int gamma, const rapid_attn_shape* shape,
                      const rapid_attn_params* params, void* workspace, size_t workspace_bytes,
                      const rapid_paged_kv* paged, const int32_t* block_table, AttnCall& c,
                      bool describe_only = false, bool fp8 = false) {
    if ((!ctx_lens && !describe_only) || !shape) {
        set_error("%s: NULL argument", who);
        return RAPID_ERR_INVALID_ARG;
    }
    if (!attn_shape_ok(shape, gamma)) {
        set_error("%s: invalid shape (B=%d Hq=%d Hkv=%d Lmax=%lld gamma=%d)", who, shape->B, shape->Hq, shape->Hkv,
                  (long long)shape->Lmax, gamma);
        return RAPID_ERR_INVALID_ARG;
    }
    if (params && params->kv_fp8) fp8 = true;  // planning for, or describing, a call over an 8-bit cache
    const rapid_attn_shape& s = *shape;
    const int R = gamma + 1;
    const int G = s.Hq / s.Hkv;
    const int GR = G * R;
    if (s.D != 64 && s.D != 128) {
        set_error("%s: head_dim %d is not supported (64 or 128)", who, s.D);
        return RAPID_ERR_UNSUPPORTED;
    }
    if (GR > 128) {
        set_error("%s: %d grouped rows per KV head exceed 128", who, GR);
        return RAPID_ERR_UNSUPPORTED;
    }
    const bool all_visible = params && params->all_keys_visible;
    if (s.Lmax < (all_visible ? 1 : R) || s.Lmax > 0x7fffffffLL - kTile) {
        set_error("%s: Lmax %lld out of range", who, (long long)s.Lmax);
        return RAPID_ERR_INVALID_ARG;
    }
    const int sink = params ? params->sink_keys : 0, window = params ? params->window_keys : 0;
    if (sink < 0 || window < 0 || (sink > 0 && window == 0) || (window > 0 && all_visible)) {
        set_error("%s: sink_keys and window_keys must not be negative, sink_keys needs a window, and a window "
                  "cannot be combined with all_keys_visible", who);
        return RAPID_ERR_INVALID_ARG;
    }
    c.outer = s.B;
    c.keys = s.Lmax;
    int tile_shift = 0;
    if (paged) {
        const int64_t bs = paged->block_size;
        if (bs < kTile || (bs & (bs - 1)) || paged->num_blocks <= 0 || paged->max_blocks_per_seq <= 0) {
            set_error("%s: block_size must be a power of two >= %d, num_blocks and max_blocks_per_seq positive", who,
                      kTile);
            return RAPID_ERR_UNSUPPORTED;
        }
        if (s.Lmax != (int64_t)paged->max_blocks_per_seq * bs) {
            set_error("%s: shape->Lmax must equal max_blocks_per_seq * block_size", who);
            return RAPID_ERR_INVALID_ARG;
        }
        while ((kTile << tile_shift) < bs) ++tile_shift;
        c.sl = paged->stride_l ? paged->stride_l : s.D;
        c.sh = paged->stride_h ? paged->stride_h : bs * c.sl;
        c.sb = paged->stride_block ? paged->stride_block : s.Hkv * c.sh;
        c.outer = paged->num_blocks;
        c.keys = bs;
    } else {
        c.sl = s.kv_stride_l ? s.kv_stride_l : s.D;
        c.sh = s.kv_stride_h ? s.kv_stride_h : s.Lmax * c.sl;
        c.sb = s.kv_stride_b ? s.kv_stride_b : s.Hkv * c.sh;
    }
    const int stride_unit = fp8 ? 16 : 8;  // 16 bytes either way
    if (c.sl < s.D || c.sl % stride_unit || c.sh % stride_unit || c.sb % stride_unit || c.sh <= 0 || c.sb <= 0) {
        set_error("%s: K/V strides must be positive multiples of %d elements", who, stride_unit);
        return RAPID_ERR_UNSUPPORTED;
    }
    if (fp8) {
        const int want8 = params ? params->kernel : RAPID_ATTN_KERNEL_AUTO;
        if (s.D != 128 || GR > 96 || sink || window || paged ||
            (want8 != RAPID_ATTN_KERNEL_AUTO && want8 != RAPID_ATTN_KERNEL_KEYS_ON_M)) {
            set_error("%s: the 8-bit cache needs head_dim 128, at most 96 grouped rows, a contiguous cache, no window "
                      "and the keys-on-M kernel", who);
            return RAPID_ERR_UNSUPPORTED;
        }
    }
    const WsLayout lay = ws_layout(s.B, s.Hkv, GR, s.D);
    if (!describe_only && (!workspace || workspace_bytes < lay.total || ((uintptr_t)workspace & 255))) {
        set_error("%s: workspace of %zu bytes needed (256-byte aligned), got %zu", who, lay.total, workspace_bytes);
        return RAPID_ERR_WORKSPACE;
    }
    int num_ctas = params && params->num_ctas ? params->num_ctas : sm_count();
    if (num_ctas <= 0 || num_ctas > kMaxCtas) {
        set_error("%s: num_ctas %d outside [1, %d]", who, num_ctas, kMaxCtas);
        return RAPID_ERR_INVALID_ARG;
    }
    const float scale = params && params->scale != 0.f ? params->scale : 1.0f / sqrtf((float)s.D);
    if (!(scale > 0.f) || !isfinite(scale)) {
        set_error("%s: scale must be positive and finite", who);
        return RAPID_ERR_INVALID_ARG;
    }
    if ((int64_t)s.B * s.Hkv > 65535) {
        set_error("%s: B*Hkv above 65535 is not supported", who);
        return RAPID_ERR_UNSUPPORTED;
    }
    const int plan_mode = params ? params->plan : RAPID_PLAN_NONE;
    if (plan_mode != RAPID_PLAN_NONE && plan_mode != RAPID_PLAN_READY && plan_mode != RAPID_PLAN_SETTLED) {
        set_error("%s: unknown plan mode %d", who, plan_mode);
        return RAPID_ERR_INVALID_ARG;
    }
    const long long wait_limit = params && params->wait_cycle_limit ? params->wait_cycle_limit : kWaitCycleLimit;
    if (wait_limit < 0) {
        set_error("%s: wait_cycle_limit must not be negative", who);
        return RAPID_ERR_INVALID_ARG;
    }

    // Which split kernel: keys on the MMA's M axis (a softmax thread per key, probabilities through
    // shared memory) when the grouped rows fit 64 columns -- faster and cheaper per byte there --,
    // rows on the M axis otherwise (more rows, head_dim 64).  From 65 to 80 rows the keys-on-M kernel
    // with two softmax groups is the choice as well (chains of eight 128K layers: 93.7 against 97.2 us
    // per layer at 72 rows, 94.1 against 97.9 at 80); at 88 and 96 rows it runs on request only (104.7
    // against 98.8, 109.4 against 101.5).  With one sequence, whose KV heads all have the same length, and a
    // cache of at most kClusterMaxKeys keys, the keys-on-M kernel runs as one cluster per KV head
    // and merges on chip; any call can ask for that (RAPID_ATTN_KERNEL_CLUSTER_MERGE).
    const int want = params ? params->kernel : RAPID_ATTN_KERNEL_AUTO;
    const bool kt_ok = s.D == 128 && (GR + 15) / 16 <= kt::kMaxNC2;
    if (want != RAPID_ATTN_KERNEL_AUTO && want != RAPID_ATTN_KERNEL_ROWS_ON_M && want != RAPID_ATTN_KERNEL_KEYS_ON_M &&
        want != RAPID_ATTN_KERNEL_CLUSTER_MERGE) {
        set_error("%s: unknown kernel choice %d", who, want);
        return RAPID_ERR_INVALID_ARG;
    }
    if ((want == RAPID_ATTN_KERNEL_KEYS_ON_M || want == RAPID_ATTN_KERNEL_CLUSTER_MERGE) && !kt_ok) {
        set_error("%s: the keys-on-M kernel needs head_dim 128 and at most %d grouped rows", who, 16 * kt::kMaxNC2);
        return RAPID_ERR_UNSUPPORTED;
    }
    const bool kt_auto = kt_ok && (GR + 15) / 16 <= kt::kMaxNC + 1;
    c.kt_path = want == RAPID_ATTN_KERNEL_KEYS_ON_M || want == RAPID_ATTN_KERNEL_CLUSTER_MERGE ||
                (want == RAPID_ATTN_KERNEL_AUTO && kt_auto);
    if (fp8) c.kt_path = true;
    c.need_cluster = !fp8 && want == RAPID_ATTN_KERNEL_CLUSTER_MERGE;
    c.want_cluster = !fp8 && (c.need_cluster ||
                     (want == RAPID_ATTN_KERNEL_AUTO && c.kt_path && s.B == 1 && s.Lmax <= kClusterMaxKeys &&
                      !(params && params->split_done_event)));
    if (c.need_cluster && (int64_t)s.B * s.Hkv * 2 > kMaxCtas) {
        set_error("%s: too many (sequence, KV head) units for one cluster each", who);
        return RAPID_ERR_UNSUPPORTED;
    }
    c.kt_half_blocks = c.kt_path && paged && paged->block_size == kTile;
    if (c.kt_path && paged && !c.kt_half_blocks) --tile_shift;  // blocks are counted in 128-key tiles
    c.box_rows = c.kt_path && !c.kt_half_blocks ? kt::kKeys : kTile;
    c.NC = (GR + 15) / 16;
    c.KS = c.kt_path ? 1 : kStreams;
    c.fp32_sums = params && params->lse_out;
    // Few partial slots per unit, or few rows: the warp-per-row merge whose blocks sit beside the split
    // kernel's CTAs pays (it needs the one-group kernel's registers).  Otherwise up to 64 grouped rows
    // run with two softmax groups of 8 to 32 columns: measured 30.2 against 32.0 us per 32K layer and
    // 83.8 against 84.5 per 128K layer of the 8-unit shape at 36 rows, 33.4 against 36.3 and 89.5 against
    // 91.1 at 63 rows, 14.5 against 16.1 per 8K layer at 20 rows, 12.6 against 13.0 at 12 rows (the
    // ragged batch of 32 units, with the other merge: 134.2 against 131.6, which is why it keeps one group).
    c.few_slots = GR <= 8 || num_ctas <= 8 * s.B * s.Hkv;
    c.two_groups = c.kt_path && !fp8 && c.NC <= 4 && !c.few_slots && !c.need_cluster;
    if (c.two_groups) c.want_cluster = false;

    AttnArgs& a = c.a;
    a = AttnArgs{};
    uint8_t* ws = static_cast<uint8_t*>(describe_only ? nullptr : workspace);
    a.ctx_lens = ctx_lens;
    a.partial = reinterpret_cast<float*>(ws + lay.partial);
    a.status = reinterpret_cast<int32_t*>(ws);
    a.B = s.B;
    a.Hq = s.Hq;
    a.Hkv = s.Hkv;
    a.G = G;
    a.R = R;
    a.GR = GR;
    a.Lmax = (int)s.Lmax;
    a.num_ctas = num_ctas;
    a.scale_log2 = scale * 1.4426950408889634f;
    a.block_table = paged ? block_table : nullptr;
    a.max_blocks = paged ? paged->max_blocks_per_seq : 0;
    a.num_blocks = paged ? paged->num_blocks : 0;
    a.tile_shift = tile_shift;
    a.kt_half_blocks = c.kt_half_blocks ? 1 : 0;
    a.tile_keys = c.kt_path ? kt::kKeys : kTile;
    a.tile_log2 = c.kt_path ? 7 : 6;
    a.pad = c.kt_path ? 5 : unit_switch_tiles(s.D);
    a.stair = all_visible ? 0 : R;
    a.Lmin = all_visible ? 1 : R;
    a.sink = window > 0 ? sink : 0;
    a.window = window;
    a.plan_mode = plan_mode;
    a.caller_plan = plan_mode != RAPID_PLAN_NONE;
    a.plan_sig = reinterpret_cast<const int32_t*>(ws + lay.sig);
    a.plan_walks = reinterpret_cast<const Walk*>(ws + lay.walks);
    a.plan_units = reinterpret_cast<const int2*>(ws + lay.units);
    a.plan_ctx = reinterpret_cast<const int32_t*>(ws + lay.ctx);
    a.wait_limit = wait_limit;
    a.kv_settled = params && params->kv_settled && plan_mode == RAPID_PLAN_SETTLED && !paged;
    a.merge_early = c.kt_path;
    a.cmerge = 0;
    return RAPID_OK;
}

}  // namespace

size_t attention_workspace_bytes(const rapid_attn_shape* s, int gamma) {
    if (!attn_shape_ok(s, gamma)) return 0;
    if (s->D != 64 && s->D != 128) return 0;
    const int64_t GR = (int64_t)(s->Hq / s->Hkv) * (gamma + 1);
    if (GR > 128) return 0;
    return ws_layout(s->B, s->Hkv, (int)GR, s->D).total;
}

// Clusters of `size` CTAs of the keys-on-M kernel that serves this call, resident together.
static int kt_max_clusters(const AttnCall& c, int size, int dev) {
    switch (c.NC) {
        case 1: return kt_resident_clusters<1, 1>(size, dev);
        case 2: return kt_resident_clusters<2, 1>(size, dev);
        case 3: return kt_resident_clusters<3, 1>(size, dev);
        case 4: return c.fp32_sums ? kt_resident_clusters<4, 2>(size, dev) : kt_resident_clusters<4, 1>(size, dev);
        case 5: return kt_resident_clusters<5, 2>(size, dev);
        case 6: return kt_resident_clusters<6, 2>(size, dev);
    }
    return 0;
}

// The cluster size a keys-on-M call of this geometry would run with (0 = no cluster).
static int cluster_size_for(const AttnCall& c) {
    if (!c.kt_path || !c.want_cluster) return 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    const int units = c.a.B * c.a.Hkv;
    int cs = 0;
    switch (c.NC) {
        case 1: cs = kt_cluster_size_that_fits<1, 1>(units, dev); break;
        case 2: cs = kt_cluster_size_that_fits<2, 1>(units, dev); break;
        case 3: cs = kt_cluster_size_that_fits<3, 1>(units, dev); break;
        case 4: cs = c.fp32_sums ? kt_cluster_size_that_fits<4, 2>(units, dev) : kt_cluster_size_that_fits<4, 1>(units, dev); break;
        case 5: cs = kt_cluster_size_that_fits<5, 2>(units, dev); break;
        case 6: cs = kt_cluster_size_that_fits<6, 2>(units, dev); break;
    }
    if (cs && !c.need_cluster && units * cs * 4 < sm_count() * 3) cs = 0;
    return cs;
}

int describe_attention(const rapid_attn_shape* shape, int gamma, const rapid_attn_params* params,
                       rapid_attn_launch_info* info) {
    if (!info) {
        set_error("rapid_attention_describe: NULL info");
        return RAPID_ERR_INVALID_ARG;
    }
    AttnCall c;
    int rc = prepare_attention("rapid_attention_describe", nullptr, gamma, shape, params, nullptr, 0, nullptr, nullptr,
                               c, true);
    if (rc != RAPID_OK) return rc;
    *info = rapid_attn_launch_info{};
    const int cs = cluster_size_for(c);
    const int units = c.a.B * c.a.Hkv;
    info->kernel = !c.kt_path ? RAPID_ATTN_KERNEL_ROWS_ON_M : (cs ? RAPID_ATTN_KERNEL_CLUSTER_MERGE : RAPID_ATTN_KERNEL_KEYS_ON_M);
    info->kernels_per_call = cs ? 1 : 2;
    info->ctas = cs ? units * cs : c.a.num_ctas;
    info->cluster_size = cs;
    info->softmax_groups = c.kt_path ? ((c.NC > 4 || (c.NC == 4 && c.fp32_sums) || c.two_groups) ? 2 : 1) : 2;
    info->columns = c.kt_path ? 16 * c.NC : (c.a.GR <= 64 ? 64 : 128);
    if (c.kt_path) {
        int dev = 0;
        if (cudaGetDevice(&dev) == cudaSuccess) {
            const int sizes[4] = {16, 8, 4, 2};
            for (int i = 0; i < 4; ++i) info->max_clusters[i] = kt_max_clusters(c, sizes[i], dev);
        }
    }
    if (c.need_cluster && !cs) {
        set_error("rapid_attention_describe: the clusters of this call do not fit on the device together");
        return RAPID_ERR_UNSUPPORTED;
    }
    return RAPID_OK;
}

static int launch_plan_kernel(const AttnCall& c, void* workspace, int D, cudaStream_t stream) {
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    const WsLayout lay = ws_layout(c.a.B, c.a.Hkv, c.a.GR, D);
    RAPID_CUDA_CHECK(launch_dependent(attention_plan_kernel, dim3(1), dim3(512), 0, stream, c.a, c.KS,
                                      reinterpret_cast<Walk*>(ws + lay.walks), reinterpret_cast<int2*>(ws + lay.units),
                                      reinterpret_cast<int32_t*>(ws + lay.ctx), reinterpret_cast<int32_t*>(ws + lay.sig)));
    count_launch(1);
    return RAPID_OK;
}

int launch_attention_plan(const int32_t* ctx_lens, int gamma, const rapid_attn_shape* shape,
                          const rapid_attn_params* params, void* workspace, size_t workspace_bytes,
                          cudaStream_t stream) {
    AttnCall c;
    rapid_attn_params p = params ? *params : rapid_attn_params{};
    p.plan = RAPID_PLAN_NONE;
    // a paged call plans like a contiguous one: the tiles are the same, only their addresses differ
    int rc = prepare_attention("rapid_attention_plan", ctx_lens, gamma, shape, &p, workspace, workspace_bytes, nullptr,
                               nullptr, c);
    if (rc != RAPID_OK) return rc;
    c.a.cmerge = cluster_size_for(c);
    if (c.need_cluster && !c.a.cmerge) {
        set_error("rapid_attention_plan: the clusters of this call do not fit on the device together");
        return RAPID_ERR_UNSUPPORTED;
    }
    return launch_plan_kernel(c, workspace, shape->D, stream);
}

template <int NC>
int launch_split_kt8(const CUtensorMap& tmK, const CUtensorMap& tmV, const AttnArgs& a, cudaStream_t stream) {
    constexpr int smem = kt8::smem_bytes(NC);
    static_assert(smem <= kMaxSmemOptin - 4096, "shared memory (dynamic + the kernel's static arrays)");
    static bool configured[64] = {};
    int dev = 0;
    RAPID_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        RAPID_CUDA_CHECK(cudaFuncSetAttribute(kt8::verify_attn_splitkv_kt8_kernel<NC>,
                                              cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    RAPID_CUDA_CHECK(launch_dependent(kt8::verify_attn_splitkv_kt8_kernel<NC>, dim3(a.num_ctas),
                                      dim3(kt8::threads(NC)), (size_t)smem, stream, tmK, tmV, a));
    return RAPID_OK;
}

int launch_verify_attention_fp8(const void* q, const void* k_cache, const void* v_cache, const float* k_scale,
                                const float* v_scale, const int32_t* ctx_lens, int gamma, void* out,
                                const rapid_attn_shape* shape, const rapid_attn_params* params, void* workspace,
                                size_t workspace_bytes, cudaStream_t stream) {
    if (!q || !k_cache || !v_cache || !k_scale || !v_scale || !ctx_lens || !out || !shape) {
        set_error("rapid_verify_attention_fp8: NULL argument");
        return RAPID_ERR_INVALID_ARG;
    }
    AttnCall c;
    int rc = prepare_attention("rapid_verify_attention_fp8", ctx_lens, gamma, shape, params, workspace, workspace_bytes,
                               nullptr, nullptr, c, false, true);
    if (rc != RAPID_OK) return rc;
    if (((uintptr_t)k_cache | (uintptr_t)v_cache | (uintptr_t)q | (uintptr_t)out) & 15) {
        set_error("rapid_verify_attention_fp8: q, k_cache, v_cache and out must be 16-byte aligned");
        return RAPID_ERR_UNSUPPORTED;
    }
    const rapid_attn_shape& s = *shape;
    AttnArgs& a = c.a;
    a.q = static_cast<const __nv_bfloat16*>(q);
    a.out = static_cast<__nv_bfloat16*>(out);
    a.lse_out = params ? params->lse_out : nullptr;
    a.out_f32 = params ? params->out_f32 : nullptr;
    a.k_scale = k_scale;
    a.v_scale = v_scale;
    CUtensorMap tmK, tmV;
    rc = make_kv_map(&tmK, k_cache, s, c.outer, c.keys, c.sb, c.sh, c.sl, kt8::kKeys, true);
    if (rc != RAPID_OK) return rc;
    rc = make_kv_map(&tmV, v_cache, s, c.outer, c.keys, c.sb, c.sh, c.sl, kt8::kKeys, true);
    if (rc != RAPID_OK) return rc;
    if (!a.caller_plan) {
        rc = launch_plan_kernel(c, workspace, s.D, stream);
        if (rc != RAPID_OK) return rc;
        a.plan_mode = RAPID_PLAN_READY;
    }
    switch (c.NC) {
        case 1: rc = launch_split_kt8<1>(tmK, tmV, a, stream); break;
        case 2: rc = launch_split_kt8<2>(tmK, tmV, a, stream); break;
        case 3: rc = launch_split_kt8<3>(tmK, tmV, a, stream); break;
        case 4: rc = launch_split_kt8<4>(tmK, tmV, a, stream); break;
        case 5: rc = launch_split_kt8<5>(tmK, tmV, a, stream); break;
        default: rc = launch_split_kt8<6>(tmK, tmV, a, stream); break;
    }
    if (rc != RAPID_OK) return rc;
    if (params && params->split_done_event)
        RAPID_CUDA_CHECK(cudaEventRecord(static_cast<cudaEvent_t>(params->split_done_event), stream));
    dim3 grid(a.GR, s.B * s.Hkv);
    RAPID_CUDA_CHECK(launch_dependent(verify_attn_merge_kernel<128>, grid, dim3(128), 0, stream, a, c.KS, a.out,
                                      a.lse_out, a.out_f32));
    count_launch(2);
    return RAPID_OK;
}

int launch_verify_attention(const void* q, const void* k_cache, const void* v_cache,
                            const int32_t* ctx_lens, int gamma, void* out,
                            const rapid_attn_shape* shape, const rapid_attn_params* params,
                            void* workspace, size_t workspace_bytes, cudaStream_t stream,
                            const rapid_paged_kv* paged, const int32_t* block_table) {
    if (!q || !k_cache || !v_cache || !ctx_lens || !out || !shape) {
        set_error("rapid_verify_attention: NULL argument");
        return RAPID_ERR_INVALID_ARG;
    }
    if (paged && !block_table) {
        set_error("rapid_verify_attention_paged: NULL block table");
        return RAPID_ERR_INVALID_ARG;
    }
    AttnCall c;
    int rc = prepare_attention("rapid_verify_attention", ctx_lens, gamma, shape, params, workspace, workspace_bytes,
                               paged, block_table, c);
    if (rc != RAPID_OK) return rc;
    if (((uintptr_t)k_cache | (uintptr_t)v_cache | (uintptr_t)q | (uintptr_t)out) & 15) {
        set_error("rapid_verify_attention: q, k_cache, v_cache and out must be 16-byte aligned");
        return RAPID_ERR_UNSUPPORTED;
    }
    const rapid_attn_shape& s = *shape;
    AttnArgs& a = c.a;
    a.q = static_cast<const __nv_bfloat16*>(q);
    a.out = static_cast<__nv_bfloat16*>(out);
    a.lse_out = params ? params->lse_out : nullptr;
    a.out_f32 = params ? params->out_f32 : nullptr;

    CUtensorMap tmK, tmV, tmQ;
    rc = make_kv_map(&tmK, k_cache, s, c.outer, c.keys, c.sb, c.sh, c.sl, c.box_rows);
    if (rc != RAPID_OK) return rc;
    rc = make_kv_map(&tmV, v_cache, s, c.outer, c.keys, c.sb, c.sh, c.sl, c.box_rows);
    if (rc != RAPID_OK) return rc;
    rc = make_q_map(&tmQ, q, s, a.G, a.R);
    if (rc != RAPID_OK) return rc;

    if (!a.caller_plan) {
        // no plan from the caller: make one now (a tiny kernel ahead of the split kernel, which reads
        // it after its grid-dependency wait)
        a.cmerge = cluster_size_for(c);
        rc = launch_plan_kernel(c, workspace, s.D, stream);
        if (rc != RAPID_OK) return rc;
        a.plan_mode = RAPID_PLAN_READY;
    }
    if (c.kt_path) {
        rc = dispatch_split_kt(c.NC, c.fp32_sums, c.two_groups, tmK, tmV, tmQ, a, stream, c.want_cluster, c.need_cluster);
    } else if (a.GR <= 64)
        rc = s.D == 128 ? launch_split_tc<128, 64>(tmK, tmV, tmQ, a, stream)
                        : launch_split_tc<64, 64>(tmK, tmV, tmQ, a, stream);
    else
        rc = s.D == 128 ? launch_split_tc<128, 128>(tmK, tmV, tmQ, a, stream)
                        : launch_split_tc<64, 128>(tmK, tmV, tmQ, a, stream);
    if (rc != RAPID_OK) return rc;
    if (a.cmerge) {  // merged on chip: one kernel
        count_launch(1);
        return RAPID_OK;
    }

    if (params && params->split_done_event)
        RAPID_CUDA_CHECK(cudaEventRecord(static_cast<cudaEvent_t>(params->split_done_event), stream));

    dim3 grid(a.GR, s.B * s.Hkv);
    // programmatic dependent launch: the merge blocks start while the split kernel still runs and
    // hold at their grid-dependency wait until its partials are complete and visible
    // Which merge: a warp per row (blocks that sit on an SM beside a CTA of the one-group keys-on-M kernel,
    // a quarter of the blocks) where a row has few slots or the call few rows; four warps per row
    // otherwise.  Measured per layer (split + merge, chains of layers): ragged batch of 8 132.5 against
    // 136.4 us, one-row decode at 8K 13.05 against 13.5, but 8 units of 36 rows 33.1 against 32.1 at
    // 32K and 86.9 against 86.3 at 128K.
    const bool one_group = c.kt_path && !c.two_groups && (c.NC <= 3 || (c.NC == 4 && !c.fp32_sums));
    const bool warp_per_row = one_group && c.few_slots;
    if (warp_per_row)
        RAPID_CUDA_CHECK(launch_dependent(verify_attn_merge_rows_kernel<128>, dim3((a.GR + 3) / 4, s.B * s.Hkv),
                                          dim3(128), 0, stream, a, a.out, a.lse_out, a.out_f32));
    else if (s.D == 128)
        RAPID_CUDA_CHECK(launch_dependent(verify_attn_merge_kernel<128>, grid, dim3(128), 0, stream, a, c.KS, a.out,
                                          a.lse_out, a.out_f32));
    else
        RAPID_CUDA_CHECK(launch_dependent(verify_attn_merge_kernel<64>, grid, dim3(128), 0, stream, a, c.KS, a.out,
                                          a.lse_out, a.out_f32));
    count_launch(2);
    return RAPID_OK;
}

}  // namespace rapid
