// Accept / residual step (Algorithm 1, validation loop and residual draw; Eq. (new_target);
// tail rule of Section 2.4), vocabulary-parallel, in ONE launch.
//
// A thread-block cluster of 16 (or 8) CTAs owns one logit row (one draft position of one sequence,
// or the bonus row).  Each CTA reads its slice of the target and the draft row from
// global memory exactly once, keeps it in shared memory, and the cluster then walks the steps of
// Algorithm 1 over those resident slices, exchanging a few floats through distributed shared
// memory between the steps:
//   0. load + (max, sum exp) of z/T and d/T                                    -> p, q
//   1. (max, sum exp) of y = z/T + eta (q - p)                                 -> phat
//   2. slice sums of w = max(p - phat', p - q, 0) (phat' = phat after the tail rule) and of p,
//      and the ratio phat'(x')/q(x') at the draft token
//   3. inverse-CDF search of the row's candidate token: slice sums first, then a block scan in
//      the one slice that holds the target mass
// Every position is processed speculatively (also those after the first rejection).  The cluster
// that finishes last -- a counter in the workspace header tells -- reads every row's ratio and
// candidate and writes, per sequence, the number of leading accepted drafts n and the candidate
// of row n: the row that Algorithm 1 would have reached.  All reductions run in a fixed order, so
// results are bit-identical from run to run.  exp is evaluated in base 2: x2 = x * log2(e)/T.
#include <cooperative_groups.h>
#include <math.h>

#include <atomic>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace rapid {

namespace {

// A portable cluster of 8 CTAs of 1024 threads per row.  (The kernel is written for any cluster size
// and thread count; a cluster of 16 CTAs of 512 threads, which puts the nine rows of gamma = 8 on 144
// SMs instead of 72, measured the same 20 us: the kernel's time is the chain of its barriers and
// exchanges, not the work between them.)
constexpr int kClusterPortable = 8, kThreadsPortable = 1024;
constexpr int kMaxSlice = 24576;  // floats of one array a CTA keeps: 2 * 96 KiB

struct AcceptArgs {
    const float* z;  // target logits [B, R, V]
    const float* d;  // draft logits  [B, gamma, V]
    const int32_t* tokens;
    const float* uniforms;
    int32_t* accept_len;
    int32_t* next_token;
    float* ratio_out;  // optional [B, gamma]
    int32_t* status;   // header word 0
    int32_t* done;     // header word 1: clusters that have finished; back to 0 when the call ends
    float* ratio;      // [B*gamma]
    int32_t* cand;     // [B*R] candidate token of every row; bit 31 = drawn from p as a fallback
    float* logq_out;   // optional [B]: natural log of the drawn token's probability (gamma = 0 calls)
    float* stats_out;  // optional [B, 2]: max and log-sum-exp of the row's logits / T (gamma = 0 calls)
    const float* d_stats;  // optional [B, gamma, 2]: (max, log-sum-exp) of every draft row / T, natural log
    const float* d_logq;   // optional [B, gamma]: natural log of q at the draft token
    int B, gamma, R, V;
    int slice;  // entries per CTA (multiple of 4)
    int per;    // consecutive entries per thread in the search (odd: conflict-free shared reads)
    long long zs, ds;  // row strides
    float inv_T_log2;  // log2(e) / T
    float eta_log2;    // eta * log2(e)
    float alpha;       // tail_alpha, 0 disables the tail rule
    float log2_alpha;  // log2(tail_alpha), -inf disables the tail rule
    int mode;
};

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Block-wide maximum / sum of two values at once, in a fixed order: every warp reduces by shuffles,
// warp 0 reduces the NW <= 32 warp results the same way, everybody reads the two totals.  sh holds
// 2 * NW + 2 floats.
template <int NW>
__device__ __forceinline__ void block_max2(float& x, float& y, float* sh) {
    x = warp_max(x);
    y = warp_max(y);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();  // the previous use of sh has been read
    if (lane == 0) {
        sh[warp] = x;
        sh[NW + warp] = y;
    }
    __syncthreads();
    if (warp == 0) {
        const float a = warp_max(lane < NW ? sh[lane] : -INFINITY), b = warp_max(lane < NW ? sh[NW + lane] : -INFINITY);
        if (lane == 0) {
            sh[2 * NW] = a;
            sh[2 * NW + 1] = b;
        }
    }
    __syncthreads();
    x = sh[2 * NW];
    y = sh[2 * NW + 1];
}
template <int NW>
__device__ __forceinline__ void block_sum2(float& x, float& y, float* sh) {
    x = warp_sum(x);
    y = warp_sum(y);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();
    if (lane == 0) {
        sh[warp] = x;
        sh[NW + warp] = y;
    }
    __syncthreads();
    if (warp == 0) {
        const float a = warp_sum(lane < NW ? sh[lane] : 0.f), b = warp_sum(lane < NW ? sh[NW + lane] : 0.f);
        if (lane == 0) {
            sh[2 * NW] = a;
            sh[2 * NW + 1] = b;
        }
    }
    __syncthreads();
    x = sh[2 * NW];
    y = sh[2 * NW + 1];
}

__device__ __forceinline__ float max4(const float4& v) { return fmaxf(fmaxf(v.x, v.y), fmaxf(v.z, v.w)); }

__device__ __forceinline__ float warp_incl_scan(float v) {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

// Every CTA of the cluster hands one float4 to all of them: thread r < CL of CTA c stores it
// into slot[c] of CTA r's shared memory (a distributed-shared-memory store), and the cluster barrier
// that follows makes all CL stores visible everywhere.  Each step of the kernel uses a slot
// array of its own, so none is rewritten while a peer may still read it.
template <int CL>
__device__ __forceinline__ void cluster_publish(cg::cluster_group& cluster, float4* slots, int my_rank, float4 mine) {
    if (threadIdx.x < CL) cluster.map_shared_rank(slots, threadIdx.x)[my_rank] = mine;
    cluster.sync();
}

// Combine the per-CTA (max, sum relative to that max) pairs of a row, in rank order.
template <int CL>
__device__ __forceinline__ void combine_ms(const float4* g, bool second, float& M, float& S) {
    M = -INFINITY;
#pragma unroll
    for (int r = 0; r < CL; ++r) M = fmaxf(M, second ? g[r].z : g[r].x);
    S = 0.f;
#pragma unroll
    for (int r = 0; r < CL; ++r) {
        const float m = second ? g[r].z : g[r].x, s = second ? g[r].w : g[r].y;
        S += (m == -INFINITY) ? 0.f : s * exp2f(m - M);
    }
}

// CL = CTAs per cluster (= per row), NT = threads per CTA, NV4 = float4 groups a thread owns in each
// array (group i belongs to thread i % NT).
template <int CL, int NT, int NV4>
__global__ void __launch_bounds__(NT, 2048 / NT / 2) accept_fused_kernel(const AcceptArgs a) {
    constexpr int NW = NT / 32;
    extern __shared__ __align__(16) float slice_mem[];
    __shared__ float4 gath[3][CL];
    __shared__ float sh_red[2 * NW + 2];
    __shared__ float sh_ms[4];
    __shared__ int sh_tok, sh_last, sh_final;
    __shared__ int sh_tl;       // the draft token's place in this CTA's slice, or -1
    __shared__ float sh_pq[2];  // p and q at the draft token, kept by the thread that forms them

    cg::cluster_group cluster = cg::this_cluster();
    const int c = (int)cluster.block_rank();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int row = blockIdx.y;
    const int b = row / a.R, k = row % a.R;
    const bool draft = k < a.gamma;
    const int drow = b * a.gamma + k;
    const int v0 = min(c * a.slice, a.V), v1 = min(v0 + a.slice, a.V);
    const int n4 = (v1 - v0) >> 2;
    float4* zc = reinterpret_cast<float4*>(slice_mem);
    float4* dc = reinterpret_cast<float4*>(slice_mem + a.slice);
    const float4* z = reinterpret_cast<const float4*>(a.z + (size_t)row * a.zs + v0);
    const float4* d = draft ? reinterpret_cast<const float4*>(a.d + (size_t)drow * a.ds + v0) : nullptr;
    const float c2 = a.inv_T_log2;
    // the drafter's own statistics of this row, if the caller kept them: the row's maximum and sum
    // need not be found again
    const bool have_dstats = draft && a.d_stats != nullptr;

    // Distributed shared memory may be written only once every CTA of the cluster is running: each
    // CTA says so here and waits for the others just before its first store into a peer.
    cluster.barrier_arrive();
    griddep_wait();  // the logits may come from the kernel just before this one
    griddep_launch_dependents();

    // The draft token and the two logits at it are needed late (step 2), by one thread, on the CTA's
    // critical path: thread 0 asks for them now, so that they arrive while step 0 runs.
    int tok = 0;
    float z_tok = 0.f, d_tok = 0.f, lq_given = 0.f;
    bool tok_here = false;
    if (draft && tid == 0) {
        tok = a.tokens[drow];
        if (tok < 0 || tok >= a.V) {
            if (c == 0) atomicOr(a.status, RAPID_STATUS_BAD_DRAFT_TOKEN);
            tok = tok < 0 ? 0 : a.V - 1;
        }
        tok_here = tok >= v0 && tok < v1;
        if (tok_here) {
            z_tok = __ldg(a.z + (size_t)row * a.zs + tok);
            if (a.d_logq) lq_given = __ldg(a.d_logq + drow);
            else d_tok = __ldg(a.d + (size_t)drow * a.ds + tok);
        }
    }
    if (tid == 0) sh_tl = tok_here ? tok - v0 : -1;  // read after the block reductions of step 0

    // ---- step 0: the only pass over global memory; p = softmax(z/T), q = softmax(d/T) ----
    // every load of the thread is in flight before the first is used
    float sz = 0.f, sd = 0.f, mz = -INFINITY, md = -INFINITY;
    {
        float4 xz[NV4], xd[NV4];
#pragma unroll
        for (int e = 0; e < NV4; ++e) {
            const int i = e * NT + tid;
            const bool ok = i < n4;
            xz[e] = ok ? __ldg(z + i) : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
            xd[e] = (ok && draft) ? __ldg(d + i) : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
        }
#pragma unroll
        for (int e = 0; e < NV4; ++e) {
            const int i = e * NT + tid;
            if (i < n4) {
                zc[i] = xz[e];
                if (draft) dc[i] = xd[e];
            }
            mz = fmaxf(mz, max4(xz[e]));
            md = fmaxf(md, max4(xd[e]));
        }
        block_max2<NW>(mz, md, sh_red);
        // slice maxima in base-2 units (scaling by log2(e)/T > 0 keeps the order); an empty or all -inf
        // slice contributes (-inf, 0)
        const float refz = (mz == -INFINITY) ? 0.f : mz * c2, refd = (md == -INFINITY) ? 0.f : md * c2;
#pragma unroll
        for (int e = 0; e < NV4; ++e) {
            sz += fast_exp2(fmaf(xz[e].x, c2, -refz)) + fast_exp2(fmaf(xz[e].y, c2, -refz)) +
                  fast_exp2(fmaf(xz[e].z, c2, -refz)) + fast_exp2(fmaf(xz[e].w, c2, -refz));
            if (draft && !have_dstats)
                sd += fast_exp2(fmaf(xd[e].x, c2, -refd)) + fast_exp2(fmaf(xd[e].y, c2, -refd)) +
                      fast_exp2(fmaf(xd[e].z, c2, -refd)) + fast_exp2(fmaf(xd[e].w, c2, -refd));
        }
    }
    block_sum2<NW>(sz, sd, sh_red);
    const float Mzb = mz * c2, Mdb = md * c2;
    cluster.barrier_wait();  // every CTA of the cluster has started
    cluster_publish<CL>(cluster, gath[0], c, make_float4(mz == -INFINITY ? -INFINITY : Mzb, sz,
                                                     md == -INFINITY ? -INFINITY : Mdb, sd));
    // p = 2^(z * c2 - Mz) / Sz, q = 2^(d * c2 - Md) / Sd.  The row maximum is taken off inside the
    // fused multiply-add, before anything is rounded, and the normaliser is applied as a factor:
    // at a low temperature the scaled logits are in the hundreds, and a constant folded from
    // Mz + log2 Sz would be rounded at that magnitude, scaling every p of the row by the same
    // 1 + 1e-5 -- more than the whole residual mass when p and phat nearly coincide.  This way the
    // top entry is exactly 1/Sz, and phat's top entry exactly 1/Sy.
    if (warp == 0) {  // one warp combines the eight (max, sum) pairs; everybody reads the result
        float Mz_, Sz_, Md_ = 0.f, Sd_ = 1.f;
        combine_ms<CL>(gath[0], false, Mz_, Sz_);
        if (draft) {
            if (have_dstats) {
                const float mx = __ldg(a.d_stats + 2 * drow), lse = __ldg(a.d_stats + 2 * drow + 1);
                Md_ = mx * 1.4426950408889634f;
                Sd_ = exp2f((lse - mx) * 1.4426950408889634f);
            } else {
                combine_ms<CL>(gath[0], true, Md_, Sd_);
            }
        }
        if (lane == 0) {
            sh_ms[0] = Mz_;
            sh_ms[1] = Sz_;
            sh_ms[2] = Md_;
            sh_ms[3] = Sd_;
        }
    }
    __syncthreads();
    const float Mz = sh_ms[0], Sz = sh_ms[1], Md = sh_ms[2], Sd = sh_ms[3];
    const float iSz = 1.f / Sz, iSd = 1.f / Sd;

    float sw = 0.f, sp = 0.f;
    float My = 0.f, Sy = 1.f;
    if (draft) {
        // ---- step 1: y = z/T + eta (q - p) up to the constant Mz, and the normaliser of phat ----
        // p and q replace the logits in shared memory; y stays in registers
        float ev[NV4 * 4];
        float my = -INFINITY, unused = -INFINITY;
        const int tl = sh_tl;
#pragma unroll
        for (int kk = 0; kk < NV4; ++kk) {
            const int i = kk * NT + tid;
            if (i < n4) {
                const float4 x = zc[i], y = dc[i];
                const float lp[4] = {fmaf(x.x, c2, -Mz), fmaf(x.y, c2, -Mz), fmaf(x.z, c2, -Mz), fmaf(x.w, c2, -Mz)};
                const float lq[4] = {fmaf(y.x, c2, -Md), fmaf(y.y, c2, -Md), fmaf(y.z, c2, -Md), fmaf(y.w, c2, -Md)};
                float p[4], q[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    p[e] = fast_exp2(lp[e]) * iSz;
                    q[e] = fast_exp2(lq[e]) * iSd;
                    // a logit of -inf has p = 0 and takes no part in phat either
                    const float y2 = (lp[e] == -INFINITY) ? -INFINITY : fmaf(a.eta_log2, q[e] - p[e], lp[e]);
                    ev[4 * kk + e] = y2;
                    my = fmaxf(my, y2);
                }
                zc[i] = make_float4(p[0], p[1], p[2], p[3]);
                dc[i] = make_float4(q[0], q[1], q[2], q[3]);
                if (i == (tl >> 2)) {  // the draft token's entry: step 2 overwrites the slices, keep a copy
                    const int e = tl & 3;
                    sh_pq[0] = e == 0 ? p[0] : e == 1 ? p[1] : e == 2 ? p[2] : p[3];
                    sh_pq[1] = e == 0 ? q[0] : e == 1 ? q[1] : e == 2 ? q[2] : q[3];
                }
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e) ev[4 * kk + e] = -INFINITY;
            }
        }
        block_max2<NW>(my, unused, sh_red);
        const float refy = (my == -INFINITY) ? 0.f : my;
        float sy = 0.f, zero = 0.f;
#pragma unroll
        for (int e = 0; e < NV4 * 4; ++e) {
            ev[e] = fast_exp2(ev[e] - refy);  // phat up to the factor 2^(my - My) / Sy
            sy += ev[e];
        }
        block_sum2<NW>(sy, zero, sh_red);
        cluster_publish<CL>(cluster, gath[1], c, make_float4(my, sy, 0.f, 0.f));
        if (warp == 0) {
            float My_, Sy_;
            combine_ms<CL>(gath[1], false, My_, Sy_);
            if (lane == 0) {
                sh_ms[0] = My_;
                sh_ms[1] = Sy_;
            }
        }
        __syncthreads();
        My = sh_ms[0];
        Sy = sh_ms[1];
        const float rel = (my == -INFINITY) ? 0.f : exp2f(my - My);  // phat / max(phat) = ev * rel
        const float to_phat = rel / Sy;

        // ---- step 2: the ratio at the draft token, then the residual weights ----
        if (tok_here) {  // thread 0 of the CTA whose slice holds the draft token
            // formed from log-probabilities: a draft token deep in the tail has p, phat and q far
            // below the fp32 normal range while their ratio is O(1).  (p and q of the token were set
            // aside in step 1; the block reductions since then have made them visible.)
            const float p = sh_pq[0], q = sh_pq[1];
            const float az = fmaf(z_tok, c2, -Mz);
            const float lq = a.d_logq ? lq_given * 1.4426950408889634f : fmaf(d_tok, c2, -Md) - log2f(Sd);
            const float y2 = fmaf(a.eta_log2, q - p, az);
            const float lph = (y2 - My < a.log2_alpha) ? az - log2f(Sz) : (y2 - My) - log2f(Sy);
            const float ratio = (lq == -INFINITY) ? INFINITY : exp2f(lph - lq);
            a.ratio[drow] = ratio;
            if (a.ratio_out) a.ratio_out[drow] = ratio;
        }
        // the weights replace p in shared memory, p moves to where q was (the fallback draws from it)
#pragma unroll
        for (int kk = 0; kk < NV4; ++kk) {
            const int i = kk * NT + tid;
            if (i < n4) {
                const float4 p4 = zc[i], q4 = dc[i];
                const float p[4] = {p4.x, p4.y, p4.z, p4.w};
                const float q[4] = {q4.x, q4.y, q4.z, q4.w};
                float w[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float en = ev[4 * kk + e];
                    const float ph = (en * rel < a.alpha) ? p[e] : en * to_phat;  // tail rule
                    const float r = (a.mode == RAPID_RESIDUAL_PHAT) ? ph - q[e] : fmaxf(p[e] - ph, p[e] - q[e]);
                    w[e] = fmaxf(r, 0.f);
                    sw += w[e];
                    sp += p[e];
                }
                zc[i] = make_float4(w[0], w[1], w[2], w[3]);
                dc[i] = p4;
            }
        }
    } else {
        // bonus row: the weights are p itself
#pragma unroll
        for (int kk = 0; kk < NV4; ++kk) {
            const int i = kk * NT + tid;
            if (i < n4) {
                const float4 x = zc[i];
                const float4 p = make_float4(fast_exp2(fmaf(x.x, c2, -Mz)) * iSz, fast_exp2(fmaf(x.y, c2, -Mz)) * iSz,
                                             fast_exp2(fmaf(x.z, c2, -Mz)) * iSz, fast_exp2(fmaf(x.w, c2, -Mz)) * iSz);
                sp += (p.x + p.y) + (p.z + p.w);
                zc[i] = p;
            }
        }
        sw = sp;
    }
    block_sum2<NW>(sw, sp, sh_red);
    cluster_publish<CL>(cluster, gath[2], c, make_float4(sw, sp, 0.f, 0.f));  // also a CTA barrier

    // ---- step 3: the row's candidate token by inverse CDF (every CTA finds the same slice) ----
    const float u = a.uniforms[b * a.R + a.gamma];
    bool use_p = !draft;
    float W = 0.f;
#pragma unroll
    for (int rr = 0; rr < CL; ++rr) W += use_p ? gath[2][rr].y : gath[2][rr].x;
    int fell_back = 0;  // reported only if this row turns out to be the one Algorithm 1 reaches
    if (!(W > 0.f) || !isfinite(W)) {  // empty residual: defined fallback, draw from p
        if (!use_p) fell_back = (int)0x80000000;
        use_p = true;
        W = 0.f;
#pragma unroll
        for (int rr = 0; rr < CL; ++rr) W += gath[2][rr].y;
    }
    const float target = u * W;
    int owner = -1, last_mass = -1;
    float before = 0.f, before_last = 0.f;
    {
        float run = 0.f;
#pragma unroll
        for (int rr = 0; rr < CL; ++rr) {
            const float own = use_p ? gath[2][rr].y : gath[2][rr].x;
            if (own > 0.f) {
                if (owner < 0 && run + own > target) {
                    owner = rr;
                    before = run;
                }
                last_mass = rr;
                before_last = run;
            }
            run += own;
        }
    }
    bool want_last = false;
    if (owner < 0) {  // rounding left no slice above the target: the last slice with mass
        owner = last_mass;
        before = before_last;
        want_last = true;
    }
    if (owner < 0) {  // nothing has mass at all (non-finite logits): defined output
        if (c == 0 && tid == 0) a.cand[row] = fell_back;
    } else if (c == owner) {
        // thread t owns a.per consecutive entries, so the prefix order is the vocabulary order
        const float* wsrc = (use_p && draft) ? slice_mem + a.slice : slice_mem;
        const int t0 = min(tid * a.per, v1 - v0), t1 = min(t0 + a.per, v1 - v0);
        float mine = 0.f;
        for (int i = t0; i < t1; ++i) mine += wsrc[i];
        const float incl_w = warp_incl_scan(mine);
        if (tid == 0) {
            sh_tok = 0x7fffffff;
            sh_last = -1;
        }
        if (lane == 31) sh_red[warp] = incl_w;
        __syncthreads();
        if (warp == 0) {  // exclusive prefix of the warp totals
            const float tot = lane < NW ? sh_red[lane] : 0.f;
            const float excl = warp_incl_scan(tot) - tot;
            if (lane < NW) sh_red[NW + lane] = excl;
        }
        __syncthreads();
        float cum = before + sh_red[NW + warp] + (incl_w - mine);
        int found = 0x7fffffff, last = -1;
        for (int i = t0; i < t1; ++i) {
            const float w = wsrc[i];
            if (w > 0.f) {
                cum += w;
                last = v0 + i;
                if (!want_last && cum > target && found == 0x7fffffff) found = v0 + i;
            }
        }
        if (found != 0x7fffffff) atomicMin(&sh_tok, found);
        if (last >= 0) atomicMax(&sh_last, last);
        __syncthreads();
        if (tid == 0) {
            const int tok = sh_tok != 0x7fffffff ? sh_tok : (sh_last >= 0 ? sh_last : v0);
            a.cand[row] = tok | fell_back;
            if (a.logq_out && !draft)  // log softmax of the row at the drawn token
                a.logq_out[b] = (fmaf(__ldg(a.z + (size_t)row * a.zs + tok), c2, -Mz) - log2f(Sz)) * 0.69314718055994530942f;
        }
    }
    if (a.stats_out && !draft && c == 0 && tid == 0) {
        a.stats_out[2 * b] = Mz * 0.69314718055994530942f;
        a.stats_out[2 * b + 1] = (Mz + log2f(Sz)) * 0.69314718055994530942f;
    }

    // ---- the last cluster to finish settles every sequence ----
    // This row's ratio and candidate were stored by threads of this cluster before the barrier below;
    // the barrier (release / acquire over the cluster) orders them before thread 0's fence, which is
    // cumulative, so they are visible device-wide before the count that announces them.
    cluster.sync();  // also: no CTA leaves while a peer may still write into its exchange slots
    if (c != 0) return;
    if (tid == 0) {
        __threadfence();
        const int total = (int)gridDim.y;
        const int old = atomicAdd(a.done, 1);
        sh_final = (old == total - 1);
        __threadfence();
    }
    __syncthreads();
    if (!sh_final) return;
    // A warp per sequence: lane n takes position n's ratio, uniform and candidate in one round of
    // loads and a ballot finds the first rejection (drafts longer than 31 positions: one lane walks them).
    for (int s = warp; s < a.B; s += NW) {
        int n, cand;
        if (a.R <= 32) {
            const bool is_draft = lane < a.gamma;
            const float ratio = is_draft ? __ldcg(a.ratio + s * a.gamma + lane) : 0.f;
            const float us = is_draft ? a.uniforms[s * a.R + lane] : 0.f;
            const int cnd = lane < a.R ? __ldcg(a.cand + s * a.R + lane) : 0;
            const unsigned rej = __ballot_sync(0xffffffffu, is_draft && !(us <= fminf(1.f, ratio)));
            n = rej ? __ffs(rej) - 1 : a.gamma;
            cand = __shfl_sync(0xffffffffu, cnd, n);
        } else {
            n = 0;
            cand = 0;
            if (lane == 0) {
                for (; n < a.gamma; ++n) {
                    const float ratio = __ldcg(a.ratio + s * a.gamma + n);
                    if (!(a.uniforms[s * a.R + n] <= fminf(1.f, ratio))) break;
                }
                cand = __ldcg(a.cand + s * a.R + n);
            }
        }
        if (lane == 0) {
            if (cand < 0) atomicOr(a.status, RAPID_STATUS_RESIDUAL_FALLBACK);  // bit 31: the row fell back to p
            a.accept_len[s] = n;
            a.next_token[s] = cand & 0x7fffffff;
        }
    }
    __syncthreads();
    if (tid == 0) *a.done = 0;  // ready for the next call on this workspace
}

bool accept_shape_ok(const rapid_accept_shape* s) {
    // a CTA keeps its slice of both rows in shared memory; grid.y carries the rows
    return s && s->B > 0 && s->gamma >= 0 && s->V > 0 && s->V <= (int64_t)kClusterPortable * kMaxSlice &&
           (int64_t)s->B * (s->gamma + 1) <= 65535;
}

constexpr int kMaxDevices = 64;
std::atomic<int> g_accept_config[kMaxDevices];  // per device: the kernels' shared-memory limits have been raised

template <int CL, int NT, int NV4>
cudaError_t configure_accept_kernel(int max_slice_floats) {
    return cudaFuncSetAttribute(accept_fused_kernel<CL, NT, NV4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                2 * max_slice_floats * (int)sizeof(float));
}

template <int CL, int NT>
int launch_accept_shape(AcceptArgs& a, size_t rows, cudaStream_t stream) {
    a.slice = (int)(((a.V / 4 + CL - 1) / CL) * 4);
    a.per = ((a.slice + NT - 1) / NT) | 1;
    // one cluster per logit row; a programmatic dependent of whatever precedes it in the stream
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(CL, (unsigned)rows);
    cfg.blockDim = dim3(NT);
    cfg.dynamicSmemBytes = 2 * (size_t)a.slice * sizeof(float);
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CL;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    if (a.slice <= 4 * 4 * NT)
        RAPID_CUDA_CHECK(cudaLaunchKernelEx(&cfg, accept_fused_kernel<CL, NT, 4>, static_cast<const AcceptArgs&>(a)));
    else
        RAPID_CUDA_CHECK(cudaLaunchKernelEx(&cfg, accept_fused_kernel<CL, NT, 6>, static_cast<const AcceptArgs&>(a)));
    return RAPID_OK;
}

}  // namespace

size_t accept_workspace_bytes(const rapid_accept_shape* s) {
    if (!accept_shape_ok(s)) return 0;
    const size_t rows = (size_t)s->B * (s->gamma + 1);
    const size_t drows = (size_t)s->B * s->gamma;
    size_t bytes = kWorkspaceHeaderBytes;
    bytes += align_up(drows * sizeof(float) + 4, 256);
    bytes += align_up(rows * sizeof(int32_t), 256);
    bytes += align_up((size_t)s->B * sizeof(int32_t), 256);  // accept lengths nobody asked for (draft sampling)
    return bytes;
}

int launch_accept(const float* target_logits, const float* draft_logits,
                  const int32_t* draft_tokens, const float* uniforms, float eta,
                  int32_t* out_accept_len, int32_t* out_next_token,
                  const rapid_accept_shape* shape, const rapid_accept_params* params,
                  void* workspace, size_t workspace_bytes, cudaStream_t stream, float* logq_out,
                  float* stats_out) {
    if (!accept_shape_ok(shape)) {
        set_error("rapid_accept: invalid shape");
        return RAPID_ERR_INVALID_ARG;
    }
    const rapid_accept_shape& s = *shape;
    const bool sampling = logq_out || stats_out;  // rapid_draft_sample: gamma = 0, no accept lengths wanted
    if (!target_logits || !uniforms || (!out_accept_len && !sampling) || !out_next_token ||
        (s.gamma > 0 && (!draft_logits || !draft_tokens))) {
        set_error("rapid_accept: NULL argument");
        return RAPID_ERR_INVALID_ARG;
    }
    const float T = params ? params->temperature : 1.0f;
    const float alpha = params ? params->tail_alpha : 0.1f;
    const int mode = params ? params->residual_mode : RAPID_RESIDUAL_PAPER;
    if (!(T > 0.f) || !isfinite(T) || !(alpha >= 0.f) || !(alpha <= 1.f) || !isfinite(eta) ||
        (mode != RAPID_RESIDUAL_PAPER && mode != RAPID_RESIDUAL_PHAT)) {
        set_error("rapid_accept: need T > 0, 0 <= tail_alpha <= 1, finite eta, a known residual_mode");
        return RAPID_ERR_INVALID_ARG;
    }
    const int64_t zs = s.target_row_stride ? s.target_row_stride : s.V;
    const int64_t ds = s.draft_row_stride ? s.draft_row_stride : s.V;
    if (s.V % 4 || zs % 4 || ds % 4 || zs < s.V || ds < s.V ||
        ((uintptr_t)target_logits & 15) || ((uintptr_t)draft_logits & 15)) {
        set_error("rapid_accept: V and row strides must be multiples of 4, logits 16-byte aligned");
        return RAPID_ERR_UNSUPPORTED;
    }
    const size_t need = accept_workspace_bytes(shape);
    if (!workspace || workspace_bytes < need || ((uintptr_t)workspace & 255)) {
        set_error("rapid_accept: workspace of %zu bytes needed (256-byte aligned), got %zu", need,
                  workspace_bytes);
        return RAPID_ERR_WORKSPACE;
    }
    const int R = s.gamma + 1;
    const size_t rows = (size_t)s.B * R, drows = (size_t)s.B * s.gamma;
    uint8_t* p = static_cast<uint8_t*>(workspace);
    AcceptArgs a;
    a.status = reinterpret_cast<int32_t*>(p);
    a.done = a.status + 1;
    p += kWorkspaceHeaderBytes;
    a.ratio = reinterpret_cast<float*>(p);
    p += align_up(drows * sizeof(float) + 4, 256);
    a.cand = reinterpret_cast<int32_t*>(p);
    a.z = target_logits;
    a.d = draft_logits;
    a.tokens = draft_tokens;
    a.uniforms = uniforms;
    a.accept_len = out_accept_len ? out_accept_len
                                  : reinterpret_cast<int32_t*>(static_cast<uint8_t*>(workspace) + need -
                                                               align_up((size_t)s.B * sizeof(int32_t), 256));
    a.logq_out = logq_out;
    a.stats_out = stats_out;
    a.d_stats = params ? params->draft_row_stats : nullptr;
    a.d_logq = params ? params->draft_logq : nullptr;
    a.next_token = out_next_token;
    a.ratio_out = params ? params->ratio_out : nullptr;
    a.B = s.B;
    a.gamma = s.gamma;
    a.R = R;
    a.V = (int)s.V;
    a.zs = zs;
    a.ds = ds;
    a.inv_T_log2 = 1.4426950408889634f / T;
    a.eta_log2 = eta * 1.4426950408889634f;
    a.alpha = alpha;
    a.log2_alpha = alpha > 0.f ? log2f(alpha) : -INFINITY;
    a.mode = mode;

    int dev = 0;
    RAPID_CUDA_CHECK(cudaGetDevice(&dev));
    constexpr int P = kClusterPortable, PT = kThreadsPortable;
    if (dev < 0 || dev >= kMaxDevices || !g_accept_config[dev].load(std::memory_order_acquire)) {
        RAPID_CUDA_CHECK((configure_accept_kernel<P, PT, 4>(4 * 4 * PT)));
        RAPID_CUDA_CHECK((configure_accept_kernel<P, PT, 6>(kMaxSlice)));
        if (dev >= 0 && dev < kMaxDevices) g_accept_config[dev].store(1, std::memory_order_release);
    }
    const int rc = launch_accept_shape<P, PT>(a, rows, stream);
    if (rc != RAPID_OK) return rc;
    count_launch(1);
    return RAPID_OK;
}

}  // namespace rapid

// ---- accept step on library-owned scratch ------------------------------------------------------
//
// The scratch of the accept kernel for up to kStaticMaxRows logit rows lives in this file-scope
// device array instead of a caller workspace.  Every GPU that loads the library holds these
// bytes until the process exits.
namespace rapid {
namespace {

constexpr int kStaticMaxRows = 512;  // B * (gamma + 1) at most
constexpr size_t kStaticScratchBytes =
    kWorkspaceHeaderBytes + (size_t)kStaticMaxRows * (sizeof(float) + 2 * sizeof(int32_t)) + 3 * 256;

static __device__ __align__(256) unsigned char g_accept_scratch[kStaticScratchBytes];

// device address of g_accept_scratch, per device; atomic because first calls on a device may come
// from several host threads at once (they would all look up, and store, the same address)
std::atomic<void*> g_scratch_addr[kMaxDevices];

}  // namespace
}  // namespace rapid

extern "C" int rapid_accept_static(const float* target_logits, const float* draft_logits,
                                   const int32_t* draft_tokens, const float* uniforms, float eta,
                                   int32_t* out_accept_len, int32_t* out_next_token,
                                   const rapid_accept_shape* shape,
                                   const rapid_accept_params* params, int32_t* out_status,
                                   void* cuda_stream) {
    using namespace rapid;
    clear_error();
    if (!shape || shape->B <= 0 || shape->gamma < 0) {
        set_error("rapid_accept_static: invalid shape");
        return RAPID_ERR_INVALID_ARG;
    }
    const long long rows = (long long)shape->B * (shape->gamma + 1);
    const size_t need = accept_workspace_bytes(shape);
    if (rows > kStaticMaxRows || need == 0 || need > kStaticScratchBytes) {
        set_error("rapid_accept_static: B*(gamma+1) = %lld logit rows exceed the built-in scratch, which "
                  "holds %d rows; use rapid_accept with a caller workspace", rows, kStaticMaxRows);
        return RAPID_ERR_UNSUPPORTED;
    }
    int dev = 0;
    RAPID_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) {
        set_error("rapid_accept_static: device ordinal %d not supported", dev);
        return RAPID_ERR_UNSUPPORTED;
    }
    // In host code the array's name is only a handle for the runtime, not a device address: the
    // address the kernels can use has to be asked for, once per device, with that device current.
    void* scratch = g_scratch_addr[dev].load(std::memory_order_acquire);
    if (!scratch) {
        void* ptr = nullptr;
        RAPID_CUDA_CHECK(cudaGetSymbolAddress(&ptr, g_accept_scratch));
        g_scratch_addr[dev].store(ptr, std::memory_order_release);
        scratch = ptr;
    }
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // the array keeps whatever the previous call left: the status word must start at zero
    RAPID_CUDA_CHECK(cudaMemsetAsync(scratch, 0, kWorkspaceHeaderBytes, st));
    const int rc = launch_accept(target_logits, draft_logits, draft_tokens, uniforms, eta,
                                 out_accept_len, out_next_token, shape, params, scratch,
                                 kStaticScratchBytes, st);
    if (rc != RAPID_OK) return rc;
    if (out_status)
        RAPID_CUDA_CHECK(cudaMemcpyAsync(out_status, scratch, sizeof(int32_t), cudaMemcpyDeviceToDevice, st));
    return RAPID_OK;
}

