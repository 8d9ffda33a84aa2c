/*
 * CPU oracle for the RAPID verify step.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 statement of what the GPU library computes, written
 * from the paper.  It shares no code, header, table or constant with the CUDA
 * path and must never be linked into, imported by or called from the product.
 * Only the tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * Two parts:
 *   - verify attention: the target model scores all draft positions in one pass
 *     over the full context (Algorithm 1, the LogitsOf step; Section 2.1).  The
 *     paper prints no attention formula, so this is the textbook definition:
 *     masked softmax(scale * q k^T) v, causal among the draft rows.
 *   - accept / residual: Algorithm 1's validation loop with the
 *     retrieval-augmented target of Eq. (new_target) / Eq. (delta), the tail
 *     rule of Section 2.4 and the residual of Algorithm 1's last step.
 *
 * Every floating-point step is done in double.  bf16 inputs are widened
 * exactly (bf16 -> fp32 -> fp64 is lossless).  Loops are written in the order
 * the definitions state them; there is no tiling, fusion or reordering.
 * OpenMP only distributes independent (sequence, head, row) units over cores.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_RESIDUAL_PAPER 0 /* norm(max(p - phat, p - q, 0)), Algorithm 1 last step */
#define ORACLE_RESIDUAL_PHAT 1  /* norm(max(phat - q, 0)): Section 2.1's residual with phat as target */

#define ORACLE_FLAG_RESIDUAL_FALLBACK 1 /* W was 0 or non-finite: sampled from p instead */

static double bf16_bits_to_double(uint16_t h) {
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------------ */
/* Verify attention (definition).                                            */
/*                                                                           */
/* q   [B, R, Hq, D]      bf16 bits, R = gamma + 1, dense                    */
/* k,v [B, Hkv, Lmax, D]  bf16 bits, element strides (b, h, l) given, d = 1   */
/* Row i of sequence b is the query at absolute position L_b - R + i and     */
/* sees keys j <= L_b - R + i (bottom-right aligned causal mask).            */
/* out [B, R, Hq, D] fp64;  lse [B, R, Hq] fp64 (natural log), may be NULL.   */
/* Keys j > lim and j >= L_b are never read.                                 */
/* unit_list (may be NULL = all) names the (b, h, i) units to compute, each  */
/* as (b*Hq + h)*R + i; the other rows of out/lse are left untouched.  That  */
/* lets a caller check or time a sample of a workload too large to finish.   */
/* Returns 0, -1 on an invalid argument, -2 if memory ran out.               */
/* ------------------------------------------------------------------------ */
int oracle_verify_attention(const uint16_t* q, const uint16_t* k, const uint16_t* v,
                            const int32_t* ctx_lens, int B, int Hq, int Hkv, int D, int64_t Lmax,
                            int gamma, int64_t kv_stride_b, int64_t kv_stride_h,
                            int64_t kv_stride_l, double scale, const int64_t* unit_list,
                            int64_t n_units, double* out, double* lse) {
    const int R = gamma + 1;
    if (B < 0 || Hq <= 0 || Hkv <= 0 || D <= 0 || gamma < 0 || Hq % Hkv != 0) return -1;
    const int G = Hq / Hkv;
    for (int b = 0; b < B; ++b)
        if (ctx_lens[b] < R || (int64_t)ctx_lens[b] > Lmax) return -1;
    if (scale == 0.0) scale = 1.0 / sqrt((double)D);

    const int64_t all_units = (int64_t)B * Hq * R;
    if (!unit_list) n_units = all_units;
    for (int64_t t = 0; unit_list && t < n_units; ++t)
        if (unit_list[t] < 0 || unit_list[t] >= all_units) return -1;
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t t = 0; t < n_units; ++t) {
        const int64_t unit = unit_list ? unit_list[t] : t;
        const int b = (int)(unit / ((int64_t)Hq * R));
        const int h = (int)((unit / R) % Hq);
        const int i = (int)(unit % R);
        const int kvh = h / G;
        const int64_t L = ctx_lens[b];
        const int64_t lim = L - R + i; /* last visible key */
        const uint16_t* qrow = q + (((int64_t)b * R + i) * Hq + h) * D;
        const uint16_t* kbase = k + b * kv_stride_b + kvh * kv_stride_h;
        const uint16_t* vbase = v + b * kv_stride_b + kvh * kv_stride_h;
        double* s = (double*)malloc((size_t)(lim + 1) * sizeof(double));
        double* acc = (double*)calloc((size_t)D, sizeof(double));
        double* qd = (double*)malloc((size_t)D * sizeof(double));
        if (!s || !acc || !qd) {
#pragma omp atomic write
            failed = 1;
            free(s);
            free(acc);
            free(qd);
            continue;
        }
        for (int d = 0; d < D; ++d) qd[d] = bf16_bits_to_double(qrow[d]);
        /* scores */
        double m = -INFINITY;
        for (int64_t j = 0; j <= lim; ++j) {
            const uint16_t* krow = kbase + j * kv_stride_l;
            double dot = 0.0;
            for (int d = 0; d < D; ++d) dot += qd[d] * bf16_bits_to_double(krow[d]);
            s[j] = scale * dot;
            if (s[j] > m) m = s[j];
        }
        /* softmax weights and weighted sum of values */
        double denom = 0.0;
        for (int64_t j = 0; j <= lim; ++j) {
            const double e = exp(s[j] - m);
            denom += e;
            const uint16_t* vrow = vbase + j * kv_stride_l;
            for (int d = 0; d < D; ++d) acc[d] += e * bf16_bits_to_double(vrow[d]);
        }
        double* orow = out + (((int64_t)b * R + i) * Hq + h) * D;
        for (int d = 0; d < D; ++d) orow[d] = acc[d] / denom;
        if (lse) lse[((int64_t)b * R + i) * Hq + h] = m + log(denom);
        free(s);
        free(acc);
        free(qd);
    }
    return failed ? -2 : 0;
}

/* ------------------------------------------------------------------------ */
/* Verify attention under a sink + window mask.                              */
/*                                                                           */
/* Section 3.2 describes the streaming drafter the paper compares with       */
/* (MagicDec / StreamingLLM): a KV budget of 4,096 entries of which 4 are     */
/* "sink" tokens at the start of the sequence, the rest the most recent      */
/* ones.  Laid over a full cache that is a visibility rule: row i, whose own */
/* key is own = L_b - R + i, sees key j iff                                   */
/*     j <= own   and   ( j < sink   or   j > own - window ).                 */
/* Everything else is the definition above: masked softmax over the visible  */
/* keys, fp64.  Hidden keys are never read.  window >= 1 (a row always sees   */
/* its own key); sink >= 0.  Same layouts, unit_list and return codes as     */
/* oracle_verify_attention.                                                  */
/* ------------------------------------------------------------------------ */
int oracle_verify_attention_window(const uint16_t* q, const uint16_t* k, const uint16_t* v,
                                   const int32_t* ctx_lens, int B, int Hq, int Hkv, int D,
                                   int64_t Lmax, int gamma, int64_t kv_stride_b,
                                   int64_t kv_stride_h, int64_t kv_stride_l, double scale,
                                   int64_t sink, int64_t window, const int64_t* unit_list,
                                   int64_t n_units, double* out, double* lse) {
    const int R = gamma + 1;
    if (B < 0 || Hq <= 0 || Hkv <= 0 || D <= 0 || gamma < 0 || Hq % Hkv != 0) return -1;
    if (sink < 0 || window < 1) return -1;
    const int G = Hq / Hkv;
    for (int b = 0; b < B; ++b)
        if (ctx_lens[b] < R || (int64_t)ctx_lens[b] > Lmax) return -1;
    if (scale == 0.0) scale = 1.0 / sqrt((double)D);
    const int64_t all_units = (int64_t)B * Hq * R;
    if (!unit_list) n_units = all_units;
    for (int64_t t = 0; unit_list && t < n_units; ++t)
        if (unit_list[t] < 0 || unit_list[t] >= all_units) return -1;
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t t = 0; t < n_units; ++t) {
        const int64_t unit = unit_list ? unit_list[t] : t;
        const int b = (int)(unit / ((int64_t)Hq * R));
        const int h = (int)((unit / R) % Hq);
        const int i = (int)(unit % R);
        const int kv_head = h / G;
        const int64_t L = ctx_lens[b];
        const int64_t own = L - R + i; /* the row's own key */
        const uint16_t* qrow = q + (((int64_t)b * R + i) * Hq + h) * D;
        const uint16_t* kbase = k + b * kv_stride_b + kv_head * kv_stride_h;
        const uint16_t* vbase = v + b * kv_stride_b + kv_head * kv_stride_h;
        double* score = (double*)malloc((size_t)(own + 1) * sizeof(double));
        double* acc = (double*)calloc((size_t)D, sizeof(double));
        double* qd = (double*)malloc((size_t)D * sizeof(double));
        if (!score || !acc || !qd) {
#pragma omp atomic write
            failed = 1;
            free(score);
            free(acc);
            free(qd);
            continue;
        }
        for (int d = 0; d < D; ++d) qd[d] = bf16_bits_to_double(qrow[d]);
        double m = -INFINITY;
        for (int64_t j = 0; j <= own; ++j) {
            if (!(j < sink || j > own - window)) continue; /* hidden */
            const uint16_t* krow = kbase + j * kv_stride_l;
            double dot = 0.0;
            for (int d = 0; d < D; ++d) dot += qd[d] * bf16_bits_to_double(krow[d]);
            score[j] = scale * dot;
            if (score[j] > m) m = score[j];
        }
        double denom = 0.0;
        for (int64_t j = 0; j <= own; ++j) {
            if (!(j < sink || j > own - window)) continue;
            const double e = exp(score[j] - m);
            denom += e;
            const uint16_t* value_row = vbase + j * kv_stride_l;
            for (int d = 0; d < D; ++d) acc[d] += e * bf16_bits_to_double(value_row[d]);
        }
        double* orow = out + (((int64_t)b * R + i) * Hq + h) * D;
        for (int d = 0; d < D; ++d) orow[d] = acc[d] / denom;
        if (lse) lse[((int64_t)b * R + i) * Hq + h] = m + log(denom);
        free(score);
        free(acc);
        free(qd);
    }
    return failed ? -2 : 0;
}

/* ------------------------------------------------------------------------ */
/* Verify attention over an 8-bit KV cache.                                  */
/*                                                                           */
/* The paper's case for this path is that reading the long context's KV      */
/* cache is memory-bound (Introduction; Section 2.1), and it fixes no        */
/* storage precision.  Reading taken here: a cache stored as FP8 E4M3 codes  */
/* (1 sign, 4 exponent, 3 mantissa bits, bias 7, no infinities, S.1111.111   */
/* = NaN, exponent 0 = subnormals: the OCP 8-bit floating point format) with */
/* one fp32 scale per (sequence, KV head) for K and one for V:               */
/*     K[b,h,j,:] = k_scale[b,h] * decode(k_codes[b,h,j,:]),  V likewise.    */
/* The attention is the definition above applied to those K and V, in fp64;  */
/* q stays bf16.  Same masks, layouts (strides in elements = bytes),         */
/* unit_list and return codes as oracle_verify_attention.                    */
/* ------------------------------------------------------------------------ */
double oracle_e4m3_to_double(uint8_t code) {
    const int sign = code >> 7, e = (code >> 3) & 15, m = code & 7;
    double v;
    if (e == 15 && m == 7) return NAN;
    if (e == 0) v = ldexp((double)m, -9);          /* subnormal: m/8 * 2^-6 */
    else v = ldexp(1.0 + (double)m / 8.0, e - 7);  /* normal: 1.m * 2^(e-7) */
    return sign ? -v : v;
}

int oracle_verify_attention_fp8(const uint16_t* q, const uint8_t* k, const uint8_t* v,
                                const float* k_scale, const float* v_scale,
                                const int32_t* ctx_lens, int B, int Hq, int Hkv, int D, int64_t Lmax,
                                int gamma, int64_t kv_stride_b, int64_t kv_stride_h,
                                int64_t kv_stride_l, double scale, const int64_t* unit_list,
                                int64_t n_units, double* out, double* lse) {
    const int R = gamma + 1;
    if (B < 0 || Hq <= 0 || Hkv <= 0 || D <= 0 || gamma < 0 || Hq % Hkv != 0) return -1;
    const int G = Hq / Hkv;
    for (int b = 0; b < B; ++b)
        if (ctx_lens[b] < R || (int64_t)ctx_lens[b] > Lmax) return -1;
    if (scale == 0.0) scale = 1.0 / sqrt((double)D);
    const int64_t all_units = (int64_t)B * Hq * R;
    if (!unit_list) n_units = all_units;
    for (int64_t t = 0; unit_list && t < n_units; ++t)
        if (unit_list[t] < 0 || unit_list[t] >= all_units) return -1;
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t t = 0; t < n_units; ++t) {
        const int64_t unit = unit_list ? unit_list[t] : t;
        const int b = (int)(unit / ((int64_t)Hq * R));
        const int h = (int)((unit / R) % Hq);
        const int i = (int)(unit % R);
        const int head8 = h / G;
        const int64_t L = ctx_lens[b];
        const int64_t last = L - R + i; /* last visible key */
        const double ks = (double)k_scale[(int64_t)b * Hkv + head8];
        const double vs = (double)v_scale[(int64_t)b * Hkv + head8];
        const uint16_t* qrow = q + (((int64_t)b * R + i) * Hq + h) * D;
        const uint8_t* kbase = k + b * kv_stride_b + head8 * kv_stride_h;
        const uint8_t* vbase = v + b * kv_stride_b + head8 * kv_stride_h;
        double* sc = (double*)malloc((size_t)(last + 1) * sizeof(double));
        double* acc = (double*)calloc((size_t)D, sizeof(double));
        double* qd = (double*)malloc((size_t)D * sizeof(double));
        if (!sc || !acc || !qd) {
#pragma omp atomic write
            failed = 1;
            free(sc);
            free(acc);
            free(qd);
            continue;
        }
        for (int d = 0; d < D; ++d) qd[d] = bf16_bits_to_double(qrow[d]);
        double m = -INFINITY;
        for (int64_t j = 0; j <= last; ++j) {
            const uint8_t* kcodes = kbase + j * kv_stride_l;
            double dot = 0.0;
            for (int d = 0; d < D; ++d) dot += qd[d] * (ks * oracle_e4m3_to_double(kcodes[d]));
            sc[j] = scale * dot;
            if (sc[j] > m) m = sc[j];
        }
        double denom = 0.0;
        for (int64_t j = 0; j <= last; ++j) {
            const double e = exp(sc[j] - m);
            denom += e;
            const uint8_t* vcodes = vbase + j * kv_stride_l;
            for (int d = 0; d < D; ++d) acc[d] += e * (vs * oracle_e4m3_to_double(vcodes[d]));
        }
        double* orow = out + (((int64_t)b * R + i) * Hq + h) * D;
        for (int d = 0; d < D; ++d) orow[d] = acc[d] / denom;
        if (lse) lse[((int64_t)b * R + i) * Hq + h] = m + log(denom);
        free(sc);
        free(acc);
        free(qd);
    }
    return failed ? -2 : 0;
}

/* ------------------------------------------------------------------------ */
/* Accept / residual (Algorithm 1, validation loop and residual step).       */
/* ------------------------------------------------------------------------ */

/* softmax(x / T) over n entries, the usual max-subtracted evaluation. */
static void softmax_T(const double* x, int64_t n, double T, double* out) {
    double m = -INFINITY;
    for (int64_t j = 0; j < n; ++j)
        if (x[j] / T > m) m = x[j] / T;
    double sum = 0.0;
    for (int64_t j = 0; j < n; ++j) {
        out[j] = exp(x[j] / T - m);
        sum += out[j];
    }
    for (int64_t j = 0; j < n; ++j) out[j] /= sum;
}

/*
 * One draft position: p = softmax(z/T), q = softmax(d/T) (Algorithm 1),
 * zhat = z + eta*T*(q - p) (Eq. delta), phat = softmax(zhat/T), then the tail
 * rule of Section 2.4: entries of phat below tail_alpha * max(phat) take the
 * value of p.  The mask is decided on the un-patched phat and the patched
 * vector is NOT renormalised (the paper only says the entries are kept equal
 * to p).  tail_alpha = 0 disables the rule.  phat_raw (may be NULL) receives
 * the un-patched phat.
 */
void oracle_rapid_distributions(const float* z, const float* d, int64_t V, double T, double eta,
                                double tail_alpha, double* p, double* q, double* phat,
                                double* phat_raw) {
    double* zd = (double*)malloc((size_t)V * sizeof(double));
    double* dd = (double*)malloc((size_t)V * sizeof(double));
    double* zhat = (double*)malloc((size_t)V * sizeof(double));
    for (int64_t j = 0; j < V; ++j) {
        zd[j] = (double)z[j];
        dd[j] = (double)d[j];
    }
    softmax_T(zd, V, T, p);
    softmax_T(dd, V, T, q);
    for (int64_t j = 0; j < V; ++j) zhat[j] = zd[j] + eta * T * (q[j] - p[j]);
    softmax_T(zhat, V, T, phat);
    if (phat_raw) memcpy(phat_raw, phat, (size_t)V * sizeof(double));
    double mx = 0.0;
    for (int64_t j = 0; j < V; ++j)
        if (phat[j] > mx) mx = phat[j];
    const double thresh = tail_alpha * mx;
    for (int64_t j = 0; j < V; ++j)
        if (phat[j] < thresh) phat[j] = p[j]; /* mask uses the un-patched value: each entry is tested before it is overwritten */
    free(zd);
    free(dd);
    free(zhat);
}

/* Residual weights (un-normalised). */
void oracle_residual_weights(const double* p, const double* q, const double* phat, int64_t V,
                             int mode, double* w) {
    for (int64_t j = 0; j < V; ++j) {
        double r;
        if (mode == ORACLE_RESIDUAL_PHAT) {
            r = phat[j] - q[j];
        } else {
            const double a = p[j] - phat[j];
            const double b = p[j] - q[j];
            r = a > b ? a : b;
        }
        w[j] = r > 0.0 ? r : 0.0;
    }
}

/*
 * Inverse-CDF draw from un-normalised weights w with uniform u in [0,1):
 * the smallest v with w_v > 0 whose running sum exceeds u * W; if rounding
 * leaves none, the largest v with w_v > 0.  Returns -1 if W is 0 or not finite.
 */
int64_t oracle_inverse_cdf(const double* w, int64_t V, double u) {
    double W = 0.0;
    for (int64_t j = 0; j < V; ++j) W += w[j];
    if (!(W > 0.0) || !isfinite(W)) return -1;
    const double target = u * W;
    double c = 0.0;
    int64_t last = -1;
    for (int64_t j = 0; j < V; ++j) {
        if (w[j] > 0.0) {
            c += w[j];
            last = j;
            if (c > target) return j;
        }
    }
    return last;
}

/*
 * The validation loop for B sequences.
 *   target_logits [B, gamma+1, V] fp32, draft_logits [B, gamma, V] fp32,
 *   draft_tokens [B, gamma] int32, uniforms [B, gamma+1] fp32: entries
 *   0..gamma-1 are the acceptance draws r, entry gamma drives the one token
 *   sampled per step.
 * Outputs: accept_len [B]; next_token [B]; flags [B] (may be NULL);
 *   ratios [B, gamma] fp64 (may be NULL): phat(x')/q(x') for EVERY position
 *   (also those after the first rejection, for diagnostics; +inf if q(x')=0).
 * When all gamma drafts are accepted the extra token is drawn from
 * softmax(z_gamma / T), the (gamma+1)-th target row (the usual speculative
 * decoding convention; Algorithm 1 leaves this case implicit).
 * Returns 0, -1 on invalid arguments.
 */
int oracle_accept(const float* target_logits, const float* draft_logits,
                  const int32_t* draft_tokens, const float* uniforms, int B, int gamma, int64_t V,
                  double eta, double T, double tail_alpha, int residual_mode, int32_t* accept_len,
                  int32_t* next_token, int32_t* flags, double* ratios) {
    if (B < 0 || gamma < 0 || V <= 0 || !(T > 0.0) || tail_alpha < 0.0) return -1;
    if (residual_mode != ORACLE_RESIDUAL_PAPER && residual_mode != ORACLE_RESIDUAL_PHAT) return -1;
    for (int64_t t = 0; t < (int64_t)B * gamma; ++t)
        if (draft_tokens[t] < 0 || draft_tokens[t] >= V) return -1;
    const int R = gamma + 1;
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        double* p = (double*)malloc((size_t)V * sizeof(double));
        double* q = (double*)malloc((size_t)V * sizeof(double));
        double* phat = (double*)malloc((size_t)V * sizeof(double));
        double* w = (double*)malloc((size_t)V * sizeof(double));
        double* rej_p = (double*)malloc((size_t)V * sizeof(double));
        int n = 0;
        int rejected = 0;
        int flag = 0;
        for (int kpos = 0; kpos < gamma; ++kpos) {
            const float* z = target_logits + ((int64_t)b * R + kpos) * V;
            const float* d = draft_logits + ((int64_t)b * gamma + kpos) * V;
            if (rejected && !ratios) break;
            oracle_rapid_distributions(z, d, V, T, eta, tail_alpha, p, q, phat, NULL);
            const int32_t x = draft_tokens[(int64_t)b * gamma + kpos];
            const double ratio = q[x] > 0.0 ? phat[x] / q[x] : INFINITY;
            if (ratios) ratios[(int64_t)b * gamma + kpos] = ratio;
            if (rejected) continue;
            const double r = (double)uniforms[(int64_t)b * R + kpos];
            const double bound = ratio < 1.0 ? ratio : 1.0;
            if (r <= bound) {
                n += 1;
            } else {
                rejected = 1;
                oracle_residual_weights(p, q, phat, V, residual_mode, w);
                memcpy(rej_p, p, (size_t)V * sizeof(double));
            }
        }
        if (!rejected) {
            /* all drafts accepted: bonus token from the (gamma+1)-th target row */
            const float* z = target_logits + ((int64_t)b * R + gamma) * V;
            double* zd = (double*)malloc((size_t)V * sizeof(double));
            for (int64_t j = 0; j < V; ++j) zd[j] = (double)z[j];
            softmax_T(zd, V, T, w);
            memcpy(rej_p, w, (size_t)V * sizeof(double));
            free(zd);
        }
        const double u = (double)uniforms[(int64_t)b * R + gamma];
        int64_t tok = oracle_inverse_cdf(w, V, u);
        if (tok < 0) { /* empty residual: defined fallback, sample from p */
            flag |= ORACLE_FLAG_RESIDUAL_FALLBACK;
            tok = oracle_inverse_cdf(rej_p, V, u);
        }
        accept_len[b] = n;
        next_token[b] = (int32_t)tok;
        if (flags) flags[b] = flag;
        free(p);
        free(q);
        free(phat);
        free(w);
        free(rej_p);
    }
    return 0;
}
