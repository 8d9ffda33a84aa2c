/*
 * rapid.h -- C ABI of the RAPID verify-step library (NVIDIA B200, sm_100a).
 *
 * The library computes the target model's verification step of
 * retrieval-augmented speculative decoding (Algorithm 1 of the RAPID paper):
 *
 *   1. verify attention: the gamma+1 newest query rows of every sequence attend
 *      over that sequence's whole bf16 KV cache in one pass of the target over
 *      all gamma+1 positions (Algorithm 1, the LogitsOf step; Section 2.1),
 *      causally masked among themselves;
 *   2. accept / residual: the validation loop of Algorithm 1 with the
 *      retrieval-augmented target distribution of Eq. (new_target), the tail
 *      rule of Section 2.4 and the residual draw of Algorithm 1's last step.
 *
 * Conventions shared by every entry point
 *   - Pointers are DEVICE pointers owned by the caller unless a parameter is
 *     documented as host memory.  Structs are read on the host during the call.
 *   - Nothing is allocated and nothing is freed.  Scratch lives in a caller
 *     workspace whose size the *_workspace_bytes() functions give.  A workspace
 *     must be prepared once with rapid_workspace_init() before its first use
 *     and must not be shared by calls that can overlap on the GPU.
 *   - Calls are asynchronous on `cuda_stream` (a cudaStream_t passed as
 *     void*; NULL is the default stream).  There is no host synchronisation
 *     unless an entry point says so.  Work issued to the stream after a call
 *     sees its results, as after any kernel launch.  Among themselves the
 *     library's kernels are programmatic dependent launches (a kernel's
 *     prologue, and where the caller allows it the first copies of old cache
 *     tiles, overlap the kernel before it); a caller's own kernel launched
 *     with programmatic stream serialisation right after a call may likewise
 *     start while the call's kernels run and must pass its grid-dependency
 *     wait before it touches anything the call reads or writes.
 *   - Return value: RAPID_OK or one of the RAPID_ERR_* codes.  No exception
 *     crosses the boundary.  rapid_last_error() describes the last failure on
 *     the calling thread.
 *   - Problems only the device can see (a context length outside
 *     [gamma+1, Lmax], a draft token outside [0, V), an empty residual) set a
 *     bit of the sticky status word stored in the first 4 bytes of the
 *     workspace; the kernels never trap and always write defined outputs.
 */
#ifndef RAPID_H
#define RAPID_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define RAPID_VERSION 100

/* return codes */
#define RAPID_OK 0
#define RAPID_ERR_INVALID_ARG 1 /* NULL pointer, non-positive size, T <= 0, ...              */
#define RAPID_ERR_UNSUPPORTED 2 /* head_dim not 64/128, too many grouped rows, misalignment   */
#define RAPID_ERR_WORKSPACE 3   /* workspace missing or smaller than *_workspace_bytes()      */
#define RAPID_ERR_CUDA 4        /* a CUDA runtime / driver call failed (see rapid_last_error) */

/* bits of the device status word (first int32 of a workspace; sticky) */
#define RAPID_STATUS_BAD_CTX_LEN 1        /* ctx_lens[b] outside [gamma+1, Lmax]: clamped into range  */
#define RAPID_STATUS_BAD_DRAFT_TOKEN 2    /* draft token outside [0, V): clamped into range           */
#define RAPID_STATUS_RESIDUAL_FALLBACK 4  /* residual mass was 0 / not finite: token drawn from p    */
#define RAPID_STATUS_PIPELINE_TIMEOUT 8   /* an on-chip wait hit its time limit: outputs invalid      */
#define RAPID_STATUS_BAD_BLOCK_TABLE 16  /* a block-table entry outside [0, num_blocks): read as 0s  */
#define RAPID_STATUS_STALE_PLAN 32       /* the plan in the workspace was made for other lengths or another
                                            geometry than this call's: outputs invalid               */

/* residual_mode */
#define RAPID_RESIDUAL_PAPER 0 /* norm(max(p - phat, p - q, 0)): Algorithm 1, residual step               */
#define RAPID_RESIDUAL_PHAT 1  /* norm(max(phat - q, 0)): the residual of Section 2.1 with phat as target */

/*
 * Geometry of one attention call.
 *   q, out : [B, R, Hq, D] bf16, dense, R = gamma + 1.  Row i of sequence b is
 *            the query at absolute position ctx_lens[b] - R + i.
 *   k, v   : [B, Hkv, Lmax, D] bf16 with D contiguous; element strides between
 *            sequences / KV heads / tokens as given (0 = dense).  Strides must be
 *            multiples of 8 elements and the base pointers 16-byte aligned.
 *            Entries at token positions >= ctx_lens[b] are never used, whatever
 *            their bits.
 *   ctx_lens[b] counts the R newest tokens too (their K/V were appended by the
 *            caller) and must lie in [R, Lmax].
 *   Hq must be a multiple of Hkv; (Hq/Hkv) * R grouped rows per KV head may
 *   not exceed 128; D is 64 or 128.
 */
typedef struct rapid_attn_shape {
    int32_t B;
    int32_t Hq;
    int32_t Hkv;
    int32_t D;
    int64_t Lmax;
    int64_t kv_stride_b;
    int64_t kv_stride_h;
    int64_t kv_stride_l;
} rapid_attn_shape;

/* Which split kernel rapid_verify_attention uses (rapid_attn_params.kernel). */
#define RAPID_ATTN_KERNEL_AUTO 0      /* keys on M for head_dim 128 and <= 80 grouped rows, rows on M otherwise */
#define RAPID_ATTN_KERNEL_ROWS_ON_M 1 /* grouped rows on the MMA's M axis: any supported shape           */
#define RAPID_ATTN_KERNEL_KEYS_ON_M 2 /* keys on the M axis: head_dim 128, <= 96 grouped rows per KV head (two
                                         softmax groups beyond 64), any paged block size the call accepts;
                                         RAPID_ERR_UNSUPPORTED otherwise                                        */
#define RAPID_ATTN_KERNEL_CLUSTER_MERGE 3 /* the keys-on-M kernel as one thread-block cluster per (sequence,
                                         KV head): the cluster's CTAs share that unit's keys and merge their
                                         partial results on chip, so the call is ONE kernel.  Meant for short
                                         runs (a decode over a few thousand keys, a 32K layer) of sequences of
                                         similar lengths; RAPID_ERR_UNSUPPORTED if the clusters do not fit on
                                         the device together.  The library picks it by itself only where the
                                         clusters would fill three quarters of the SMs.                      */

/* rapid_attn_params.plan */
#define RAPID_PLAN_NONE 0    /* the call plans for itself: one more tiny kernel ahead of its own (default)    */
#define RAPID_PLAN_READY 1   /* the workspace holds a plan made by rapid_attention_plan for this call's
                                geometry and for the current ctx_lens                                      */
#define RAPID_PLAN_SETTLED 2 /* as RAPID_PLAN_READY, and at least one other kernel (or a synchronisation)
                                lies between rapid_attention_plan and this call in the stream: the plan is
                                then read while the preceding kernel still runs.  That kernel must be one
                                of this library's or an ordinary launch: a foreign kernel launched with
                                programmatic stream serialisation that lets its dependents go before the
                                plan kernel has completed does not settle anything                         */

/* Optional knobs and extra outputs of the attention call (NULL = defaults). */
typedef struct rapid_attn_params {
    float scale;      /* softmax scale; 0 = 1/sqrt(D)                                             */
    int32_t num_ctas; /* CTAs the KV length is split over; 0 = one per SM; at most 512            */
    float* lse_out;   /* device [B, R, Hq] fp32 natural-log sum-exp of the scaled scores, or NULL;
                         within 1e-4 of the exact value (the row sums then add fp32 probabilities
                         in every kernel)                                                         */
    float* out_f32;   /* device [B, R, Hq, D] fp32 output before bf16 rounding, or NULL           */
    void* split_done_event; /* a cudaEvent_t recorded on the stream between the split and the merge
                               kernel (lets a caller time the two separately), or NULL          */
    int32_t all_keys_visible; /* non-zero: no causal stair, every row sees all ctx_lens[b] keys, and
                                 ctx_lens[b] >= 1 suffices.  For a shard of the context that does not
                                 hold the rows' own keys (see rapid_merge_partials)                */
    int32_t kernel;           /* RAPID_ATTN_KERNEL_*: 0 lets the library choose                        */
    int32_t sink_keys;        /* with window_keys > 0: the first sink_keys keys stay visible to every row  */
    int32_t window_keys;      /* > 0: row i sees, besides the sink keys, only the window_keys newest keys up
                                 to and including its own, i.e. (lim_i - window_keys, lim_i] with
                                 lim_i = ctx_lens[b] - R + i.  The mask of a streaming drafter that keeps
                                 a few sink tokens and a recent window (Section 3.2, the MagicDec /
                                 StreamingLLM baseline: 4 sinks in a budget of 4,096) laid over a full
                                 cache; key tiles no row sees are not read.  0 = the plain causal mask  */
    int32_t plan;             /* RAPID_PLAN_*                                                           */
    int32_t kv_fp8;           /* non-zero in a call of rapid_attention_plan or rapid_attention_describe:
                                 the plan is for rapid_verify_attention_fp8 (which always runs the
                                 keys-on-M kernel); ignored elsewhere                                   */
    int64_t wait_cycle_limit; /* SM clock cycles an on-chip wait (for a tile, for the tensor cores) may take
                                 before the kernel gives up and sets RAPID_STATUS_PIPELINE_TIMEOUT;
                                 0 = the library's limit of about a second                              */
    int32_t kv_settled;       /* non-zero, together with plan = RAPID_PLAN_SETTLED and a contiguous cache: the
                                 caller states that every K/V entry OLDER than the R newest keys of each
                                 sequence (positions below ctx_lens[b] - R) was final before the work that
                                 precedes this call on the stream was issued.  The split kernel then starts
                                 copying its first such tiles while that preceding work still runs (before
                                 its own stream-order wait); the newest R rows, q and everything else are
                                 read after the wait as always.  True of a decode loop, where only the newest
                                 rows of a layer's cache are written inside a step.  0 = nothing is read
                                 early (default)                                                        */
} rapid_attn_params;

/*
 * Geometry of one accept call.
 *   target_logits : [B, gamma+1, V] fp32, row stride target_row_stride elements (0 = V)
 *   draft_logits  : [B, gamma,   V] fp32, row stride draft_row_stride elements (0 = V)
 *   V and both row strides are multiples of 4 and the bases 16-byte aligned;
 *   V <= 196,608 and B * (gamma+1) <= 65,535.
 */
typedef struct rapid_accept_shape {
    int32_t B;
    int32_t gamma;
    int64_t V;
    int64_t target_row_stride;
    int64_t draft_row_stride;
} rapid_accept_shape;

/* Parameters of the accept rule (NULL = T 1, tail_alpha 0.1, RAPID_RESIDUAL_PAPER, no extras). */
typedef struct rapid_accept_params {
    float temperature;     /* T > 0 of Algorithm 1; the same T scales target and draft logits   */
    float tail_alpha;      /* Section 2.4: entries of phat below tail_alpha * max(phat) keep p;
                              0 disables the rule                                              */
    int32_t residual_mode; /* RAPID_RESIDUAL_*                                                  */
    int32_t reserved;
    float* ratio_out;      /* device [B, gamma] fp32: phat(x')/q(x') of every position, or NULL */
    /* What the drafter already knows about its own rows (Algorithm 1, the drafting loop: x'_j is drawn
       from q_j, so q_j's normaliser and q_j(x'_j) existed once): rapid_draft_sample returns both, and a
       caller that kept them spares the accept step the reductions over the draft rows.  Either may be
       NULL; the values must belong to the same draft_logits and temperature.                          */
    const float* draft_row_stats; /* device [B, gamma, 2] fp32: (max_v d_v/T, log sum_v exp(d_v/T)), or NULL */
    const float* draft_logq;      /* device [B, gamma] fp32: natural log of q(x') at the draft token, or NULL */
} rapid_accept_params;

/* ---- workspaces ---------------------------------------------------------------------------- */

/* Bytes of scratch rapid_verify_attention() needs for this geometry (0 on invalid arguments). */
size_t rapid_attention_workspace_bytes(const rapid_attn_shape* shape, int gamma);

/* Bytes of scratch rapid_accept() needs (0 on invalid arguments). */
size_t rapid_accept_workspace_bytes(const rapid_accept_shape* shape);

/*
 * Prepares a workspace (device memory, 256-byte aligned): clears the status
 * word and the small bookkeeping header.  Asynchronous on the stream.  Call
 * once after allocating, and again whenever the status word should be cleared.
 */
int rapid_workspace_init(void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Copies the status word to *host_status.  Synchronises the stream. */
int rapid_workspace_status(const void* workspace, void* cuda_stream, int32_t* host_status);

/* ---- the verify step ------------------------------------------------------------------------- */

/*
 * Verify attention (Algorithm 1, the target's LogitsOf pass; Section 2.1).
 *
 * For every sequence b, query head h (KV head h / (Hq/Hkv)) and row i:
 *   out[b,i,h,:] = sum_j softmax_j(scale * q[b,i,h,:] . k[b,kvh,j,:]) * v[b,kvh,j,:]
 * over the keys 0 <= j <= ctx_lens[b] - R + i.  fp32 accumulation, bf16
 * probabilities in the second product, bf16 output.
 *
 * The KV length is split over the CTAs of one launch (each K/V tile is read
 * from HBM once per KV head, shared by all grouped rows) and the partial
 * results are merged by their log-sum-exp in a second launch.
 *
 *   q, k_cache, v_cache, out : device, see rapid_attn_shape
 *   ctx_lens : device int32 [B]
 *   gamma    : number of draft tokens (>= 0); gamma = 0 is a plain one-row decode
 *   params   : host, may be NULL
 *   workspace: device, >= rapid_attention_workspace_bytes(), initialised
 */
int rapid_verify_attention(const void* q, const void* k_cache, const void* v_cache,
                           const int32_t* ctx_lens, int gamma, void* out,
                           const rapid_attn_shape* shape, const rapid_attn_params* params,
                           void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * rapid_verify_attention over an 8-bit KV cache.  (The paper fixes no storage precision; its case for
 * this path is that reading the long context's KV cache is memory-bound -- Introduction, Section 2.1 --
 * and a cache of half the bytes is read in half the time.)
 *
 *   k_cache, v_cache : device [B, Hkv, Lmax, D] FP8 E4M3 codes (one byte each: 1 sign, 4 exponent,
 *                      3 mantissa bits, bias 7, no infinities), geometry and strides (in elements,
 *                      multiples of 16) of `shape`;  K = k_scale[b, kvh] * decode(code), V likewise
 *   k_scale, v_scale : device fp32 [B, Hkv], positive and finite
 *   q, out           : bf16 as in rapid_verify_attention
 * The result is the attention of rapid_verify_attention over those K and V.  Inside, q and the softmax
 * probabilities enter the 8-bit tensor-core products as the sum of two E4M3 numbers each (8 significant
 * bits, what bf16 carries), so the output meets the bf16 call's tolerances against the exact result
 * over the same codes; lse_out is within 5e-3.  head_dim 128, at most 96 grouped rows per KV head, a
 * contiguous cache, the plain causal mask; params->kernel 0 or RAPID_ATTN_KERNEL_KEYS_ON_M;
 * RAPID_ERR_UNSUPPORTED otherwise.  Workspace, plan, errors and status bits as in
 * rapid_verify_attention (a plan made by rapid_attention_plan for the same geometry serves both).
 */
int rapid_verify_attention_fp8(const void* q, const void* k_cache, const void* v_cache, const float* k_scale,
                               const float* v_scale, const int32_t* ctx_lens, int gamma, void* out,
                               const rapid_attn_shape* shape, const rapid_attn_params* params, void* workspace,
                               size_t workspace_bytes, void* cuda_stream);

/*
 * Works out once, on the device, what every attention call over the same lengths would otherwise
 * work out for itself: each CTA's share of the key tiles and each (sequence, KV head)'s range of
 * partial results.  (Not in the paper.  ctx_lens does not change between the layers of one verify
 * step, so the 32 or 80 attention calls of a step can share one plan; each then saves the
 * microsecond or two its own planning takes at the head of the kernel.)
 *
 * The plan is written into `workspace` (one tiny kernel on the stream) and is valid for calls
 * with the same B, Hq, Hkv, D, gamma, ctx_lens contents and the same params fields num_ctas,
 * kernel, all_keys_visible, sink_keys, window_keys, and the same presence of lse_out, that name
 * this workspace and set params->plan.  A call whose geometry or lengths differ from the plan's
 * sets RAPID_STATUS_STALE_PLAN (checked on the device by every call).  shape's strides and a
 * paged layout do not matter to the plan.
 */
int rapid_attention_plan(const int32_t* ctx_lens, int gamma, const rapid_attn_shape* shape,
                         const rapid_attn_params* params, void* workspace, size_t workspace_bytes,
                         void* cuda_stream);

/*
 * What rapid_verify_attention would launch for this geometry and these params on the current
 * device (nothing is launched; pointers inside params are only looked at for being NULL or not).
 */
typedef struct rapid_attn_launch_info {
    int32_t kernel;           /* RAPID_ATTN_KERNEL_ROWS_ON_M, _KEYS_ON_M or _CLUSTER_MERGE                 */
    int32_t kernels_per_call; /* 2 = split + merge, 1 = merged on chip                                   */
    int32_t ctas;             /* CTAs of the split kernel                                                */
    int32_t cluster_size;     /* CTAs per thread-block cluster; 0 = launched without clusters            */
    int32_t softmax_groups;   /* groups of four softmax warps per CTA                                    */
    int32_t columns;          /* grouped rows as the MMAs see them: padded to a multiple of 16 columns
                                 (keys on M) or to 64 / 128 rows (rows on M)                             */
    int32_t max_clusters[4];  /* keys-on-M kernel: clusters of 16, 8, 4, 2 CTAs that fit on the device
                                 together (0 where that does not apply)                                  */
} rapid_attn_launch_info;

int rapid_attention_describe(const rapid_attn_shape* shape, int gamma, const rapid_attn_params* params,
                             rapid_attn_launch_info* info);

/*
 * Combines P partial attention results of the same rows over disjoint sets of keys -- the context
 * of a sequence sharded over P GPUs, each of which ran rapid_verify_attention on its keys with
 * out_f32 and lse_out (all_keys_visible on every shard but the one that holds the R newest keys)
 * and gathered the others' results.  (Not in the paper, whose runs keep a sequence's cache on one
 * device or use the serving stack's own parallelism; the identity is the one the split kernels'
 * merge uses.)
 *   out[r,:] = sum_p exp(lse_parts[p,r] - LSE_r) * o_parts[p,r,:],  LSE_r = log sum_p exp(lse_parts[p,r])
 *   o_parts   : device fp32 [P, rows, D], each normalised by its own sum;  lse_parts : device fp32 [P, rows]
 *   out       : device bf16 [rows, D] or NULL;  out_f32 : device fp32 [rows, D] or NULL (one of the two at least)
 *   lse_out   : device fp32 [rows] or NULL
 * A partial with lse = -inf (a shard without keys) takes no part; a row with no keys anywhere is 0.
 */
int rapid_merge_partials(const float* o_parts, const float* lse_parts, int P, int64_t rows, int D, void* out,
                         float* out_f32, float* lse_out, void* cuda_stream);

/*
 * Geometry of a paged KV cache: a pool of fixed-size blocks shared by all
 * sequences, as serving engines keep it.  (The paper does not say how the
 * cache is stored; the computation is that of rapid_verify_attention.)
 *   k_pool / v_pool : [num_blocks, Hkv, block_size, D] bf16 with element
 *                     strides stride_block / stride_h / stride_l
 *                     (0 = dense: Hkv*block_size*D, block_size*D, D);
 *                     [num_blocks, block_size, Hkv, D] is the same pool with
 *                     stride_h = D and stride_l = Hkv*D
 *   block_table     : device int32 [B, max_blocks_per_seq]; logical keys
 *                     [i*block_size, (i+1)*block_size) of sequence b live in
 *                     physical block block_table[b, i].  Entries past the
 *                     blocks a sequence uses are never read.
 *   block_size      : a power of two, at least 64
 */
typedef struct rapid_paged_kv {
    int32_t block_size;
    int32_t num_blocks;
    int32_t max_blocks_per_seq;
    int32_t reserved;
    int64_t stride_block;
    int64_t stride_h;
    int64_t stride_l;
} rapid_paged_kv;

/*
 * rapid_verify_attention over a paged cache.  shape->Lmax must equal
 * max_blocks_per_seq * block_size (the logical capacity); shape's kv strides
 * are ignored.  A table entry outside [0, num_blocks) sets
 * RAPID_STATUS_BAD_BLOCK_TABLE and its keys and values read as zeros.  The
 * pools and the table are only read.  Everything else (arguments, results,
 * workspace, errors) is as in rapid_verify_attention.
 */
int rapid_verify_attention_paged(const void* q, const void* k_pool, const void* v_pool,
                                 const int32_t* block_table, const rapid_paged_kv* paged,
                                 const int32_t* ctx_lens, int gamma, void* out,
                                 const rapid_attn_shape* shape, const rapid_attn_params* params,
                                 void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Accept / residual (Algorithm 1, validation loop and residual step;
 * Eq. (new_target); Section 2.4).
 *
 * For each sequence b and position k = 0..gamma-1 with z = target_logits[b,k],
 * d = draft_logits[b,k], x' = draft_tokens[b,k]:
 *   p = softmax(z/T), q = softmax(d/T), phat = softmax(z/T + eta*(q - p)),
 *   phat_v := p_v wherever phat_v < tail_alpha * max(phat)   (not renormalised),
 *   position k is accepted iff uniforms[b,k] <= min(1, phat(x')/q(x')).
 * out_accept_len[b] = number of leading accepted positions n.
 * out_next_token[b] = inverse-CDF draw with uniforms[b,gamma] from
 *   norm(max(p - phat, p - q, 0)) of position n   if n < gamma  (or the
 *   RAPID_RESIDUAL_PHAT variant), else from softmax(target_logits[b,gamma]/T).
 * The draw returns the smallest token whose running sum of weights exceeds
 * uniforms[b,gamma] * total.
 *
 *   draft_tokens : device int32 [B, gamma];  uniforms : device fp32 [B, gamma+1] in [0,1)
 *   eta          : transfer strength of Eq. (new_target); 0 gives standard speculative sampling
 *   out_accept_len, out_next_token : device int32 [B]
 *   params : host, may be NULL;  workspace: device, >= rapid_accept_workspace_bytes(), initialised
 */
int rapid_accept(const float* target_logits, const float* draft_logits,
                 const int32_t* draft_tokens, const float* uniforms, float eta,
                 int32_t* out_accept_len, int32_t* out_next_token,
                 const rapid_accept_shape* shape, const rapid_accept_params* params,
                 void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Drafter-side sampling (Algorithm 1, the drafting loop: x'_j ~ q = softmax(d/T)), fused with what
 * the later accept step needs from the drafter: the drawn token's log-probability and the row's
 * softmax statistics, so that a caller can keep q(x') without another pass over the vocabulary.
 *   draft_logits : device fp32 [B, V], row stride row_stride elements (0 = V); V % 4 == 0, 16-byte aligned
 *   uniforms     : device fp32 [B] in [0,1); out_token[b] = the smallest token whose running sum of
 *                  softmax(d_b/T) exceeds uniforms[b]   (the inverse-CDF rule of rapid_accept)
 *   out_logq     : device fp32 [B], natural log of q(out_token[b])
 *   out_row_stats: device fp32 [B, 2] = (max_v d_v/T, log sum_v exp(d_v/T)), or NULL
 *   workspace    : device, >= rapid_accept_workspace_bytes() of {B, gamma = 0, V}, initialised
 * Same kernel, limits and error behaviour as rapid_accept with gamma = 0.
 */
int rapid_draft_sample(const float* draft_logits, const float* uniforms, float temperature, int32_t* out_token,
                       float* out_logq, float* out_row_stats, int32_t B, int64_t V, int64_t row_stride,
                       void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * rapid_accept without a caller workspace.  (The paper has no counterpart: this
 * entry point exists only for the sake of callers, not of the method.)
 *
 * Who it is for: code that is not allowed to obtain device memory at the moment
 * it needs an accept step -- a plugin running inside a serving process that
 * handed all device memory to its own pool at start-up, a decode loop that has
 * promised not to touch the allocator after warm-up because cudaMalloc and
 * cudaFree stall every stream of the device, or a component whose memory
 * budget is fixed by contract.  Such a caller still owns the logits, tokens,
 * uniforms and the two output arrays, but has nowhere to put the per-row
 * ratios and candidate tokens the accept kernel leaves for its epilogue.
 *
 * Here that scratch is a fixed array inside the library image (7,168 bytes,
 * resident on every GPU that loads the library until the process ends).  The
 * computation, the kernels and the results are those of rapid_accept.
 *
 * Limits and rules
 *   - B * (gamma+1) may not exceed 512 logit rows; larger shapes are rejected
 *     with RAPID_ERR_UNSUPPORTED and a message that says so.
 *   - The call allocates and frees nothing, on host or device.
 *   - The first call on each device looks up the array's device address (the
 *     device must be current).  Make that first call outside any stream
 *     capture; later calls only enqueue work on the stream.
 *   - All calls on a device share the one array, and it keeps what the last
 *     call wrote.  The status word is cleared at the start of every call, so
 *     status bits are per call here (not sticky).  Two calls whose GPU work can
 *     overlap (different streams, no dependency) race on the array and give
 *     undefined results; serialise them.
 *   - out_status: device int32 that receives this call's status word
 *     (RAPID_STATUS_* bits), or NULL.
 * Other arguments: exactly those of rapid_accept.
 */
int rapid_accept_static(const float* target_logits, const float* draft_logits,
                        const int32_t* draft_tokens, const float* uniforms, float eta,
                        int32_t* out_accept_len, int32_t* out_next_token,
                        const rapid_accept_shape* shape, const rapid_accept_params* params,
                        int32_t* out_status, void* cuda_stream);

/*
 * One verify step: rapid_verify_attention followed by rapid_accept on the same
 * stream, with no host synchronisation in between (Algorithm 1, one iteration
 * of the outer loop after drafting).  The projections and the LM head that turn
 * attention outputs into logits belong to the caller's model, so the logits are
 * inputs here.  Arguments are those of the two calls.  Because nothing in it
 * touches the host, the chain can be captured in a CUDA graph and replayed
 * (device pointers and shapes are frozen at capture; their contents are not).
 */
int rapid_verify_step(const void* q, const void* k_cache, const void* v_cache,
                      const int32_t* ctx_lens, int gamma, void* out,
                      const rapid_attn_shape* attn_shape, const rapid_attn_params* attn_params,
                      void* attn_workspace, size_t attn_workspace_bytes,
                      const float* target_logits, const float* draft_logits,
                      const int32_t* draft_tokens, const float* uniforms, float eta,
                      int32_t* out_accept_len, int32_t* out_next_token,
                      const rapid_accept_shape* accept_shape,
                      const rapid_accept_params* accept_params, void* accept_workspace,
                      size_t accept_workspace_bytes, void* cuda_stream);

/*
 * The same step (Algorithm 1, one verification) for callers whose tensors live
 * in HOST memory (pinned memory makes the copies asynchronous).  Every h_*
 * pointer is host memory; K/V must be dense.  Inputs are copied into
 * `device_arena` (device memory, at least rapid_verify_step_host_arena_bytes(),
 * 256-byte aligned; it also holds both workspaces and is initialised by the
 * call), the step runs, and out / accept_len / next_token are copied back.
 * The call returns after the stream has been synchronised, so the host outputs
 * are valid on return.  *h_status (may be NULL) receives the OR of both status
 * words.
 */
int rapid_verify_step_host(const void* h_q, const void* h_k_cache, const void* h_v_cache,
                           const int32_t* h_ctx_lens, int gamma, void* h_out,
                           const rapid_attn_shape* attn_shape, const rapid_attn_params* attn_params,
                           const float* h_target_logits, const float* h_draft_logits,
                           const int32_t* h_draft_tokens, const float* h_uniforms, float eta,
                           int32_t* h_accept_len, int32_t* h_next_token,
                           const rapid_accept_shape* accept_shape,
                           const rapid_accept_params* accept_params, void* device_arena,
                           size_t device_arena_bytes, int32_t* h_status, void* cuda_stream);

size_t rapid_verify_step_host_arena_bytes(const rapid_attn_shape* attn_shape, int gamma,
                                          const rapid_accept_shape* accept_shape);

/* ---- retrieval for the drafter's context --------------------------------------------------------- */

/*
 * Retrieval scoring (Section 2.3: chunks of the context are embedded and compared with the query by
 * cosine similarity; Section 3.1, "RAG Setup": top-k chunks, those below a similarity threshold of
 * 0.3 filtered out).  The embeddings come from the caller's encoder; this call does the scoring
 * and the selection for B independent requests.
 *   chunk_emb : device fp32 [B, Nmax, Dm] (16-byte aligned, Dm % 4 == 0);  query_emb : device fp32 [B, Dm]
 *   n_chunks  : device int32 [B], chunks request b really has (<= Nmax), or NULL = Nmax for all;
 *               a count outside [0, Nmax] is clamped and sets RAPID_STATUS_BAD_CTX_LEN
 *   scores_out: device fp32 [B, Nmax]: e.q / (|e| |q|), 0 for a zero vector and past n_chunks[b]
 *   sel_idx   : device int32 [B, k]: the chunks with score >= threshold, best first (equal scores:
 *               lower index first), at most k of them, padded with -1;  sel_count : device int32 [B]
 *   status_word : device int32 (for instance the first word of an initialised workspace)
 * Limits: Nmax <= 4096, (Dm + Nmax) * 4 bytes <= 200 KB; otherwise RAPID_ERR_UNSUPPORTED.
 */
int rapid_retrieval_select(const float* chunk_emb, const float* query_emb, const int32_t* n_chunks, int32_t B,
                           int32_t Nmax, int32_t Dm, float threshold, int32_t k, float* scores_out,
                           int32_t* sel_idx, int32_t* sel_count, int32_t* status_word, void* cuda_stream);

/*
 * Size of the drafter's retrieved context (Section 3.1, "RAG Setup": the retrieved text is bounded
 * by the larger of a fixed floor, 4,096 tokens, and 1/24 of the full context, in chunks of 512
 * tokens).  Host arithmetic only: returns floor(max(floor_tokens, context_tokens / divisor) /
 * chunk_tokens), the k to hand to rapid_retrieval_select, or -1 (with rapid_last_error set) when
 * context_tokens < 0 or one of the other three is not positive.
 */
int64_t rapid_retrieval_budget_chunks(int64_t context_tokens, int32_t chunk_tokens, int32_t floor_tokens,
                                      int32_t divisor);

/* ---- bookkeeping around the step --------------------------------------------------------------- */

/*
 * Appends the K/V rows of the R = gamma+1 newest tokens (the last accepted token and the gamma
 * drafts x'_i .. x'_{i+gamma-1} of Algorithm 1) to every sequence's cache and counts them in
 * ctx_lens, which is the state rapid_verify_attention expects.
 *   k_new, v_new : device [B, R, Hkv, D] bf16, dense
 *   k_cache, v_cache : device, geometry of `shape` (strides honoured)
 *   ctx_lens : device int32 [B]; on entry the number of cached tokens, on exit that number + R
 * A sequence whose cache cannot take R more rows (ctx_lens[b] + R > Lmax, or a negative length)
 * is left untouched and sets RAPID_STATUS_BAD_CTX_LEN in *status_word.
 *   status_word : device int32 (for instance the first word of an initialised workspace)
 */
int rapid_kv_append(const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                    int32_t* ctx_lens, int gamma, const rapid_attn_shape* shape,
                    int32_t* status_word, void* cuda_stream);

/*
 * rapid_kv_append into a paged cache (see rapid_paged_kv): position ctx_lens[b] + i of sequence b
 * is row (ctx_lens[b] + i) % block_size of physical block
 * block_table[b, (ctx_lens[b] + i) / block_size].  The table must already name a block for every
 * new position (handing out blocks is the caller's allocator's job); a position whose entry is
 * outside [0, num_blocks) is not written and sets RAPID_STATUS_BAD_BLOCK_TABLE.  The capacity of a
 * sequence is max_blocks_per_seq * block_size; block_size need not be a power of two here.
 *   k_new, v_new : device [B, R, Hkv, D] bf16, dense;  k_pool, v_pool, block_table : device
 */
int rapid_kv_append_paged(const void* k_new, const void* v_new, void* k_pool, void* v_pool,
                          const int32_t* block_table, const rapid_paged_kv* paged, int32_t* ctx_lens,
                          int gamma, int B, int Hkv, int D, int32_t* status_word, void* cuda_stream);

/*
 * Closes a verify step (Algorithm 1: accepted drafts become x_j, the rest is discarded): of the R
 * rows appended before the step the cache keeps the last accepted token and the accept_len[b]
 * accepted drafts,  ctx_lens[b] -= gamma - accept_len[b].  (The token sampled by the step is
 * appended, with the next drafts, by the next rapid_kv_append.)  accept_len outside [0, gamma]
 * is clamped and sets RAPID_STATUS_BAD_CTX_LEN in *status_word.
 *   ctx_lens : device int32 [B];  accept_len : device int32 [B] (rapid_accept's output)
 */
int rapid_step_commit(int32_t* ctx_lens, const int32_t* accept_len, int gamma, int B,
                      int32_t* status_word, void* cuda_stream);

/* ---- misc ------------------------------------------------------------------------------------ */

/* Description of the last error on this thread ("" if none).  Never NULL. */
const char* rapid_last_error(void);

/* RAPID_VERSION of the built library. */
int rapid_version(void);

/* Kernels launched by this library on the calling thread since the last reset (for accounting). */
int64_t rapid_kernel_launch_count(void);
void rapid_kernel_launch_count_reset(void);

#ifdef __cplusplus
}
#endif
#endif /* RAPID_H */
