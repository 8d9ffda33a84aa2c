// Accept / residual step (Algorithm 1, validation loop and residual draw; Eq. (new_target);
// tail rule of Section 2.4), vocabulary-parallel.
//
// Every logit row is cut into NCH chunks; a grid of (chunk, row) CTAs makes four short passes
// over rows that stay resident in L2 after the first one:
//   1. stats    : per-chunk (max, sum exp) of z/T and d/T                      -> p, q
//   2. shift    : per-chunk (max, sum exp) of y = z/T + eta (q - p)            -> phat
//   3. residual : per-chunk sums of w = max(p - phat', p - q, 0) (phat' = phat with the tail
//                 rule applied) and the ratio phat'(x')/q(x') at the draft token
//   4. select   : per sequence, the number of leading accepted drafts n, then an inverse-CDF
//                 search: chunk sums first, then a block scan inside the one chunk that holds
//                 the target mass
// Every position is processed speculatively (also those after the first rejection); pass 4
// picks the row that Algorithm 1 would have reached.  All reductions run in a fixed order, so
// results are bit-identical from run to run.  exp is evaluated in base 2: x2 = x * log2(e)/T.
#include <math.h>

#include "common.cuh"

namespace rapid {

namespace {

constexpr int kThreads = 256;
constexpr int kMaxChunks = 64;

struct AcceptArgs {
    const float* z;  // target logits [B, R, V]
    const float* d;  // draft logits  [B, gamma, V]
    const int32_t* tokens;
    const float* uniforms;
    int32_t* accept_len;
    int32_t* next_token;
    float* ratio_out;  // optional [B, gamma]
    int32_t* status;
    float4* stats;    // [B*R][NCH]  (max z2, sum z, max d2, sum d)
    float2* ystats;   // [B*gamma][NCH] (max y2, sum)
    float2* wsums;    // [B*R][NCH] (sum w, sum p)
    float* ratio;     // [B*gamma]
    int B, gamma, R, V, NCH, chunk;  // chunk = elements per chunk (multiple of 4)
    long long zs, ds;                // row strides
    float inv_T_log2;                // log2(e) / T
    float eta_log2;                  // eta * log2(e)
    float log2_alpha;                // log2(tail_alpha), -inf disables the tail rule
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

// Block-wide (max, rescaled sum) reduction of per-thread online-softmax states; fixed order.
__device__ __forceinline__ void block_reduce_ms(float& m, float& s, float* sh_m, float* sh_s) {
    const float wm = warp_max(m);
    s = (m == -INFINITY) ? 0.f : s * exp2f(m - wm);
    s = warp_sum(s);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();
    if (lane == 0) {
        sh_m[warp] = wm;
        sh_s[warp] = s;
    }
    __syncthreads();
    float M = -INFINITY;
#pragma unroll
    for (int i = 0; i < kThreads / 32; ++i) M = fmaxf(M, sh_m[i]);
    float S = 0.f;
#pragma unroll
    for (int i = 0; i < kThreads / 32; ++i)
        S += (sh_m[i] == -INFINITY) ? 0.f : sh_s[i] * exp2f(sh_m[i] - M);
    m = M;
    s = S;
}

__device__ __forceinline__ float block_reduce_sum(float v, float* sh) {
    v = warp_sum(v);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();
    if (lane == 0) sh[warp] = v;
    __syncthreads();
    float S = 0.f;
#pragma unroll
    for (int i = 0; i < kThreads / 32; ++i) S += sh[i];
    return S;
}

// Combine the per-chunk (max, sum) partials of a row.  Every warp does it for itself with its
// lanes spread over the chunks (at most kMaxChunks = 64, two per lane), in a fixed shuffle order.
__device__ __forceinline__ void combine_ms(const float* m, const float* s, int n, int stride,
                                           float& M, float& S) {
    const int lane = threadIdx.x & 31;
    const float m0 = lane < n ? m[lane * stride] : -INFINITY;
    const float m1 = lane + 32 < n ? m[(lane + 32) * stride] : -INFINITY;
    const float s0 = lane < n ? s[lane * stride] : 0.f;
    const float s1 = lane + 32 < n ? s[(lane + 32) * stride] : 0.f;
    M = warp_max(fmaxf(m0, m1));
    float part = (m0 == -INFINITY ? 0.f : s0 * exp2f(m0 - M)) + (m1 == -INFINITY ? 0.f : s1 * exp2f(m1 - M));
    S = warp_sum(part);
}

__device__ __forceinline__ void online_add(float& m, float& s, float x) {
    if (x > m) {
        s = s * exp2f(m - x) + 1.f;  // exp2f(-inf) = 0 covers the first element
        m = x;
    } else if (x != -INFINITY) {  // a logit of -inf carries no mass (and -inf - -inf is NaN)
        s += exp2f(x - m);
    }
}

// A thread's share of a chunk: up to kPerThread float4 groups, strided by the block, all loaded
// before any arithmetic so that the loads are in flight together.
constexpr int kPerThread = 3;
constexpr int kChunkMax = kThreads * 4 * kPerThread;  // 3072 entries

struct Frag {
    float4 x[kPerThread];
    bool ok[kPerThread];
};

__device__ __forceinline__ Frag load_frag(const float* row, int v0, int v1, float fill) {
    Frag f;
#pragma unroll
    for (int e = 0; e < kPerThread; ++e) {
        const int v = v0 + (e * kThreads + threadIdx.x) * 4;
        f.ok[e] = v < v1;
        f.x[e] = f.ok[e] ? __ldg(reinterpret_cast<const float4*>(row + v)) : make_float4(fill, fill, fill, fill);
    }
    return f;
}

// ---- pass 1 ----------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads) accept_stats_kernel(const AcceptArgs a) {
    __shared__ float sh_m[kThreads / 32], sh_s[kThreads / 32];
    const int c = blockIdx.x, row = blockIdx.y;
    const int b = row / a.R, k = row % a.R;
    const int v0 = c * a.chunk, v1 = min(v0 + a.chunk, a.V);
    const bool draft = k < a.gamma;
    griddep_wait();  // the logits may come from the kernel just before this one
    griddep_launch_dependents();
    const Frag fz = load_frag(a.z + (size_t)row * a.zs, v0, v1, -INFINITY);
    Frag fd;
    if (draft) fd = load_frag(a.d + (size_t)(b * a.gamma + k) * a.ds, v0, v1, -INFINITY);
    float mz = -INFINITY, sz = 0.f, md = -INFINITY, sd = 0.f;
#pragma unroll
    for (int e = 0; e < kPerThread; ++e) {
        online_add(mz, sz, fz.x[e].x * a.inv_T_log2);
        online_add(mz, sz, fz.x[e].y * a.inv_T_log2);
        online_add(mz, sz, fz.x[e].z * a.inv_T_log2);
        online_add(mz, sz, fz.x[e].w * a.inv_T_log2);
    }
    if (draft) {
#pragma unroll
        for (int e = 0; e < kPerThread; ++e) {
            online_add(md, sd, fd.x[e].x * a.inv_T_log2);
            online_add(md, sd, fd.x[e].y * a.inv_T_log2);
            online_add(md, sd, fd.x[e].z * a.inv_T_log2);
            online_add(md, sd, fd.x[e].w * a.inv_T_log2);
        }
    }
    block_reduce_ms(mz, sz, sh_m, sh_s);
    block_reduce_ms(md, sd, sh_m, sh_s);
    if (threadIdx.x == 0) a.stats[(size_t)row * a.NCH + c] = make_float4(mz, sz, md, sd);
}

struct RowStats {
    float Mz, inv_Sz, Md, inv_Sd;
};

__device__ __forceinline__ RowStats load_row_stats(const AcceptArgs& a, int row, bool has_draft) {
    const float* st = reinterpret_cast<const float*>(a.stats + (size_t)row * a.NCH);
    RowStats r;
    float S;
    combine_ms(st + 0, st + 1, a.NCH, 4, r.Mz, S);
    r.inv_Sz = 1.f / S;
    r.Md = 0.f;
    r.inv_Sd = 0.f;
    if (has_draft) {
        combine_ms(st + 2, st + 3, a.NCH, 4, r.Md, S);
        r.inv_Sd = 1.f / S;
    }
    return r;
}

// y in base-2 units: (z/T + eta (q - p)) * log2(e)
__device__ __forceinline__ float shifted_logit2(const AcceptArgs& a, const RowStats& r, float z,
                                                float d, float& p, float& q) {
    const float z2 = z * a.inv_T_log2;
    p = exp2f(z2 - r.Mz) * r.inv_Sz;
    q = exp2f(d * a.inv_T_log2 - r.Md) * r.inv_Sd;
    return fmaf(a.eta_log2, q - p, z2);
}

// ---- pass 2 ----------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads) accept_shift_stats_kernel(const AcceptArgs a) {
    __shared__ float sh_m[kThreads / 32], sh_s[kThreads / 32];
    const int c = blockIdx.x, drow = blockIdx.y;  // drow over B*gamma
    const int b = drow / a.gamma, k = drow % a.gamma;
    const int row = b * a.R + k;
    const int v0 = c * a.chunk, v1 = min(v0 + a.chunk, a.V);
    // the logits are inputs of the call (pass 1 has waited for their producer): load them while
    // pass 1 drains, then wait for its statistics
    griddep_launch_dependents();
    const Frag fz = load_frag(a.z + (size_t)row * a.zs, v0, v1, -INFINITY);
    const Frag fd = load_frag(a.d + (size_t)drow * a.ds, v0, v1, -INFINITY);
    griddep_wait();
    const RowStats r = load_row_stats(a, row, true);
    float my = -INFINITY, sy = 0.f;
#pragma unroll
    for (int e = 0; e < kPerThread; ++e) {
        if (!fz.ok[e]) continue;
        float p, q;
        online_add(my, sy, shifted_logit2(a, r, fz.x[e].x, fd.x[e].x, p, q));
        online_add(my, sy, shifted_logit2(a, r, fz.x[e].y, fd.x[e].y, p, q));
        online_add(my, sy, shifted_logit2(a, r, fz.x[e].z, fd.x[e].z, p, q));
        online_add(my, sy, shifted_logit2(a, r, fz.x[e].w, fd.x[e].w, p, q));
    }
    block_reduce_ms(my, sy, sh_m, sh_s);
    if (threadIdx.x == 0) a.ystats[(size_t)drow * a.NCH + c] = make_float2(my, sy);
}

// Residual weight of one vocabulary entry of a draft row; also returns phat' (tail rule applied).
__device__ __forceinline__ float residual_weight(const AcceptArgs& a, const RowStats& r, float My,
                                                 float inv_Sy, float z, float d, float& p,
                                                 float& q, float& ph) {
    const float y2 = shifted_logit2(a, r, z, d, p, q);
    const float rel = y2 - My;
    ph = (rel < a.log2_alpha) ? p : exp2f(rel) * inv_Sy;
    float w;
    if (a.mode == RAPID_RESIDUAL_PHAT)
        w = ph - q;
    else
        w = fmaxf(p - ph, p - q);
    return fmaxf(w, 0.f);
}

// ---- pass 3 ----------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads) accept_residual_kernel(const AcceptArgs a) {
    __shared__ float sh[kThreads / 32];
    const int c = blockIdx.x, row = blockIdx.y;
    const int b = row / a.R, k = row % a.R;
    const bool draft = k < a.gamma;
    const int v0 = c * a.chunk, v1 = min(v0 + a.chunk, a.V);
    const float* z = a.z + (size_t)row * a.zs;
    griddep_launch_dependents();
    const Frag fz = load_frag(z, v0, v1, -INFINITY);
    float sw = 0.f, sp = 0.f;
    if (draft) {
        const int drow = b * a.gamma + k;
        const Frag fd = load_frag(a.d + (size_t)drow * a.ds, v0, v1, -INFINITY);
        int tok = a.tokens[drow];
        griddep_wait();  // statistics of the earlier passes
        const RowStats r = load_row_stats(a, row, true);
        const float* ys = reinterpret_cast<const float*>(a.ystats + (size_t)drow * a.NCH);
        float My, Sy;
        combine_ms(ys, ys + 1, a.NCH, 2, My, Sy);
        const float inv_Sy = 1.f / Sy;
        if (tok < 0 || tok >= a.V) {
            if (c == 0 && threadIdx.x == 0) atomicOr(a.status, RAPID_STATUS_BAD_DRAFT_TOKEN);
            tok = tok < 0 ? 0 : a.V - 1;
        }
#pragma unroll
        for (int g = 0; g < kPerThread; ++g) {
            if (!fz.ok[g]) continue;
            const int v = v0 + (g * kThreads + threadIdx.x) * 4;
            const float xs[4] = {fz.x[g].x, fz.x[g].y, fz.x[g].z, fz.x[g].w};
            const float ys4[4] = {fd.x[g].x, fd.x[g].y, fd.x[g].z, fd.x[g].w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float p, q, ph;
                sw += residual_weight(a, r, My, inv_Sy, xs[e], ys4[e], p, q, ph);
                sp += p;
                if (v + e == tok) {
                    // the ratio is formed from log-probabilities: a draft token deep in the tail
                    // has p, phat and q far below the fp32 normal range while their ratio is O(1)
                    const float z2 = xs[e] * a.inv_T_log2;
                    const float lq = (ys4[e] * a.inv_T_log2 - r.Md) + log2f(r.inv_Sd);
                    const float y2 = fmaf(a.eta_log2, q - p, z2);
                    const float lph = (y2 - My < a.log2_alpha) ? (z2 - r.Mz) + log2f(r.inv_Sz)
                                                               : (y2 - My) + log2f(inv_Sy);
                    const float ratio = (lq == -INFINITY) ? INFINITY : exp2f(lph - lq);
                    a.ratio[drow] = ratio;
                    if (a.ratio_out) a.ratio_out[drow] = ratio;
                }
            }
        }
    } else {
        griddep_wait();
        const RowStats r = load_row_stats(a, row, false);
#pragma unroll
        for (int g = 0; g < kPerThread; ++g) {
            if (!fz.ok[g]) continue;
            sp += exp2f(fz.x[g].x * a.inv_T_log2 - r.Mz) * r.inv_Sz;
            sp += exp2f(fz.x[g].y * a.inv_T_log2 - r.Mz) * r.inv_Sz;
            sp += exp2f(fz.x[g].z * a.inv_T_log2 - r.Mz) * r.inv_Sz;
            sp += exp2f(fz.x[g].w * a.inv_T_log2 - r.Mz) * r.inv_Sz;
        }
        sw = sp;
    }
    sw = block_reduce_sum(sw, sh);
    sp = block_reduce_sum(sp, sh);
    if (threadIdx.x == 0) a.wsums[(size_t)row * a.NCH + c] = make_float2(sw, sp);
}

// ---- pass 4 ----------------------------------------------------------------------------------
// One CTA per sequence.  The chunk holding the target mass is found by a warp scan over the chunk
// sums; inside it thread t owns 12 consecutive entries, so the prefix order is the vocabulary order.
__device__ __forceinline__ float warp_incl_scan(float v) {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

__global__ void __launch_bounds__(kThreads) accept_select_kernel(const AcceptArgs a) {
    __shared__ float sh_warp[kThreads / 32];
    __shared__ int sh_tok;
    __shared__ int sh_last;
    const int b = blockIdx.x;
    const int tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5;
    griddep_wait();
    griddep_launch_dependents();

    // number of leading accepted drafts
    int n = 0;
    for (; n < a.gamma; ++n) {
        const float ratio = a.ratio[b * a.gamma + n];
        const float u = a.uniforms[b * a.R + n];
        if (!(u <= fminf(1.f, ratio))) break;
    }
    const int row = b * a.R + n;
    const bool draft = n < a.gamma;
    const float u = a.uniforms[b * a.R + a.gamma];
    const float2* ws = a.wsums + (size_t)row * a.NCH;

    // chunk sums: lane c holds chunks c and c + 32 (every warp computes the same thing)
    const float2 w0 = lane < a.NCH ? ws[lane] : make_float2(0.f, 0.f);
    const float2 w1 = lane + 32 < a.NCH ? ws[lane + 32] : make_float2(0.f, 0.f);
    bool use_p = !draft;
    float c0 = use_p ? w0.y : w0.x, c1 = use_p ? w1.y : w1.x;
    float i0 = warp_incl_scan(c0);
    float i1 = warp_incl_scan(c1) + __shfl_sync(0xffffffffu, i0, 31);
    float W = __shfl_sync(0xffffffffu, i1, 31);
    if (!(W > 0.f) || !isfinite(W)) {  // empty residual: defined fallback, draw from p
        if (!use_p && tid == 0) atomicOr(a.status, RAPID_STATUS_RESIDUAL_FALLBACK);
        use_p = true;
        c0 = w0.y;
        c1 = w1.y;
        i0 = warp_incl_scan(c0);
        i1 = warp_incl_scan(c1) + __shfl_sync(0xffffffffu, i0, 31);
        W = __shfl_sync(0xffffffffu, i1, 31);
    }
    const float target = u * W;
    const unsigned hit0 = __ballot_sync(0xffffffffu, c0 > 0.f && i0 > target);
    const unsigned hit1 = __ballot_sync(0xffffffffu, c1 > 0.f && i1 > target);
    const unsigned pos0 = __ballot_sync(0xffffffffu, c0 > 0.f);
    const unsigned pos1 = __ballot_sync(0xffffffffu, c1 > 0.f);
    int chunk = hit0 ? __ffs(hit0) - 1 : (hit1 ? 32 + __ffs(hit1) - 1 : -1);
    bool want_last = false;
    if (chunk < 0) {  // rounding left no chunk above the target: the last chunk with mass
        chunk = pos1 ? 63 - __clz(pos1) : (pos0 ? 31 - __clz(pos0) : -1);
        want_last = true;
    }
    if (chunk < 0) {  // nothing has mass at all (non-finite logits): defined output
        if (tid == 0) {
            a.accept_len[b] = n;
            a.next_token[b] = 0;
        }
        return;
    }
    // mass before the chosen chunk = its inclusive prefix minus its own sum
    const float incl = __shfl_sync(0xffffffffu, chunk < 32 ? i0 : i1, chunk & 31);
    const float own = __shfl_sync(0xffffffffu, chunk < 32 ? c0 : c1, chunk & 31);
    const float before = incl - own;

    const RowStats r = load_row_stats(a, row, draft);
    float My = 0.f, inv_Sy = 0.f;
    const float* z = a.z + (size_t)row * a.zs;
    const float* d = nullptr;
    if (draft) {
        const int drow = b * a.gamma + n;
        d = a.d + (size_t)drow * a.ds;
        const float* ys = reinterpret_cast<const float*>(a.ystats + (size_t)drow * a.NCH);
        float Sy;
        combine_ms(ys, ys + 1, a.NCH, 2, My, Sy);
        inv_Sy = 1.f / Sy;
    }
    const int v0 = chunk * a.chunk, v1 = min(v0 + a.chunk, a.V);
    constexpr int PER = 4 * kPerThread;  // consecutive entries per thread
    const int t0 = v0 + tid * PER;
    float wv[PER];
#pragma unroll
    for (int g = 0; g < kPerThread; ++g) {
        const int v = t0 + 4 * g;
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f), y = x;
        const bool ok = v < v1;
        if (ok) {
            x = __ldg(reinterpret_cast<const float4*>(z + v));
            if (draft) y = __ldg(reinterpret_cast<const float4*>(d + v));
        }
        const float xs[4] = {x.x, x.y, x.z, x.w};
        const float ys4[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            float w = 0.f;
            if (ok) {
                if (draft) {
                    float p, q, ph;
                    const float rw = residual_weight(a, r, My, inv_Sy, xs[e], ys4[e], p, q, ph);
                    w = use_p ? p : rw;
                } else {
                    w = exp2f(xs[e] * a.inv_T_log2 - r.Mz) * r.inv_Sz;
                }
            }
            wv[4 * g + e] = w;
        }
    }
    float mine = 0.f;
#pragma unroll
    for (int e = 0; e < PER; ++e) mine += wv[e];
    // block-wide exclusive prefix of the per-thread sums, in thread order
    const float incl_w = warp_incl_scan(mine);
    if (tid == 0) {
        sh_tok = 0x7fffffff;
        sh_last = -1;
    }
    if (lane == 31) sh_warp[warp] = incl_w;
    __syncthreads();
    float cum = before;
    for (int wdx = 0; wdx < warp; ++wdx) cum += sh_warp[wdx];
    cum += incl_w - mine;
    int found = 0x7fffffff, last = -1;
#pragma unroll
    for (int e = 0; e < PER; ++e) {
        if (wv[e] > 0.f) {
            cum += wv[e];
            last = t0 + e;
            if (!want_last && cum > target && found == 0x7fffffff) found = t0 + e;
        }
    }
    if (found != 0x7fffffff) atomicMin(&sh_tok, found);
    if (last >= 0) atomicMax(&sh_last, last);
    __syncthreads();
    if (tid == 0) {
        a.accept_len[b] = n;
        a.next_token[b] = sh_tok != 0x7fffffff ? sh_tok : (sh_last >= 0 ? sh_last : v0);
    }
}

bool accept_shape_ok(const rapid_accept_shape* s) {
    // a chunk holds at most kChunkMax entries and a row at most kMaxChunks chunks
    return s && s->B > 0 && s->gamma >= 0 && s->V > 0 && s->V <= (int64_t)kMaxChunks * kChunkMax &&
           (int64_t)s->B * (s->gamma + 1) <= 65535;
}

int pick_chunks(int64_t V) {
    // about 2K entries per chunk: two float4 loads per thread and array, all in flight at once
    int n = (int)((V + 2047) / 2048);
    return n < 1 ? 1 : (n > kMaxChunks ? kMaxChunks : n);
}

}  // namespace

size_t accept_workspace_bytes(const rapid_accept_shape* s) {
    if (!accept_shape_ok(s)) return 0;
    const size_t rows = (size_t)s->B * (s->gamma + 1);
    const size_t drows = (size_t)s->B * s->gamma;
    size_t bytes = kWorkspaceHeaderBytes;
    bytes += align_up(rows * kMaxChunks * sizeof(float4), 256);
    bytes += align_up(drows * kMaxChunks * sizeof(float2), 256);
    bytes += align_up(rows * kMaxChunks * sizeof(float2), 256);
    bytes += align_up(drows * sizeof(float) + 4, 256);
    return bytes;
}

int launch_accept(const float* target_logits, const float* draft_logits,
                  const int32_t* draft_tokens, const float* uniforms, float eta,
                  int32_t* out_accept_len, int32_t* out_next_token,
                  const rapid_accept_shape* shape, const rapid_accept_params* params,
                  void* workspace, size_t workspace_bytes, cudaStream_t stream) {
    if (!accept_shape_ok(shape)) {
        set_error("rapid_accept: invalid shape");
        return RAPID_ERR_INVALID_ARG;
    }
    const rapid_accept_shape& s = *shape;
    if (!target_logits || !uniforms || !out_accept_len || !out_next_token ||
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
    p += kWorkspaceHeaderBytes;
    a.stats = reinterpret_cast<float4*>(p);
    p += align_up(rows * kMaxChunks * sizeof(float4), 256);
    a.ystats = reinterpret_cast<float2*>(p);
    p += align_up(drows * kMaxChunks * sizeof(float2), 256);
    a.wsums = reinterpret_cast<float2*>(p);
    p += align_up(rows * kMaxChunks * sizeof(float2), 256);
    a.ratio = reinterpret_cast<float*>(p);
    a.z = target_logits;
    a.d = draft_logits;
    a.tokens = draft_tokens;
    a.uniforms = uniforms;
    a.accept_len = out_accept_len;
    a.next_token = out_next_token;
    a.ratio_out = params ? params->ratio_out : nullptr;
    a.B = s.B;
    a.gamma = s.gamma;
    a.R = R;
    a.V = (int)s.V;
    a.NCH = pick_chunks(s.V);
    a.chunk = (int)(((s.V / 4 + a.NCH - 1) / a.NCH) * 4);
    a.zs = zs;
    a.ds = ds;
    a.inv_T_log2 = 1.4426950408889634f / T;
    a.eta_log2 = eta * 1.4426950408889634f;
    a.log2_alpha = alpha > 0.f ? log2f(alpha) : -INFINITY;
    a.mode = mode;

    int launches = 0;
    // every pass is a programmatic dependent of the one before: it loads its logits while its
    // predecessor drains and waits for the predecessor's statistics only then
    RAPID_CUDA_CHECK(launch_dependent(accept_stats_kernel, dim3(a.NCH, (unsigned)rows), dim3(kThreads), 0, stream, a));
    ++launches;
    if (s.gamma > 0) {
        RAPID_CUDA_CHECK(launch_dependent(accept_shift_stats_kernel, dim3(a.NCH, (unsigned)drows), dim3(kThreads), 0,
                                          stream, a));
        ++launches;
    }
    RAPID_CUDA_CHECK(launch_dependent(accept_residual_kernel, dim3(a.NCH, (unsigned)rows), dim3(kThreads), 0, stream, a));
    RAPID_CUDA_CHECK(launch_dependent(accept_select_kernel, dim3(s.B), dim3(kThreads), 0, stream, a));
    launches += 2;
    count_launch(launches);
    return RAPID_OK;
}

}  // namespace rapid

// ---- accept step on library-owned scratch ------------------------------------------------------
//
// The scratch of the accept passes for up to kStaticMaxRows logit rows lives in this file-scope
// device array instead of a caller workspace.  Every GPU that loads the library holds these
// bytes until the process exits.
namespace rapid {
namespace {

constexpr int kStaticMaxRows = 512;  // B * (gamma + 1) at most
constexpr size_t kStaticScratchBytes =
    kWorkspaceHeaderBytes + (size_t)kStaticMaxRows * kMaxChunks * (sizeof(float4) + 2 * sizeof(float2)) +
    (size_t)kStaticMaxRows * sizeof(float) + 4 * 256;

static __device__ __align__(256) unsigned char g_accept_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices] = {};  // device address of g_accept_scratch, per device

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
    if (!g_scratch_addr[dev]) {
        void* ptr = nullptr;
        RAPID_CUDA_CHECK(cudaGetSymbolAddress(&ptr, g_accept_scratch));
        g_scratch_addr[dev] = ptr;
    }
    void* scratch = g_scratch_addr[dev];
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

