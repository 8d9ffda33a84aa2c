// C ABI of the RAPID verify-step library: argument plumbing around the launchers.
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include "common.cuh"

namespace rapid {

namespace {
thread_local char g_error[512] = "";
thread_local int64_t g_launches = 0;
}  // namespace

void set_error(const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_error, sizeof g_error, fmt, ap);
    va_end(ap);
}
void clear_error() { g_error[0] = 0; }
void count_launch(int n) { g_launches += n; }

size_t attention_workspace_bytes(const rapid_attn_shape* s, int gamma);
size_t accept_workspace_bytes(const rapid_accept_shape* s);

namespace {

// One block per (sequence, new row, KV head): copies D bf16 of K and of V into the cache.
__global__ void kv_append_kernel(const uint4* __restrict__ k_new, const uint4* __restrict__ v_new,
                                 __nv_bfloat16* k_cache, __nv_bfloat16* v_cache,
                                 const int32_t* __restrict__ ctx_lens, int R, int Hkv, int D, long long Lmax,
                                 long long sb, long long sh, long long sl, int32_t* status) {
    const int b = blockIdx.z, i = blockIdx.y, h = blockIdx.x;
    const long long L = ctx_lens[b];
    if (L < 0 || L + R > Lmax) {
        if (i == 0 && h == 0 && threadIdx.x == 0) atomicOr(status, RAPID_STATUS_BAD_CTX_LEN);
        return;
    }
    const int chunks = D / 8;  // 16-byte chunks per row
    const size_t src = (((size_t)b * R + i) * Hkv + h) * chunks;
    const size_t dst = (size_t)b * sb + (size_t)h * sh + (size_t)(L + i) * sl;
    for (int c = threadIdx.x; c < chunks; c += blockDim.x) {
        reinterpret_cast<uint4*>(k_cache + dst)[c] = k_new[src + c];
        reinterpret_cast<uint4*>(v_cache + dst)[c] = v_new[src + c];
    }
}

// Runs after the copies (same stream): ctx_lens[b] += R where the rows fitted.
// The same append into a paged cache: position L + i of sequence b is row (L + i) % block_size of
// physical block block_table[b][(L + i) / block_size].
__global__ void kv_append_paged_kernel(const uint4* __restrict__ k_new, const uint4* __restrict__ v_new,
                                       __nv_bfloat16* k_pool, __nv_bfloat16* v_pool,
                                       const int32_t* __restrict__ block_table,
                                       const int32_t* __restrict__ ctx_lens, int R, int Hkv, int D,
                                       int block_size, int num_blocks, int max_blocks, long long sblk,
                                       long long sh, long long sl, int32_t* status) {
    const int b = blockIdx.z, i = blockIdx.y, h = blockIdx.x;
    const long long L = ctx_lens[b];
    const long long Lmax = (long long)max_blocks * block_size;
    if (L < 0 || L + R > Lmax) {
        if (i == 0 && h == 0 && threadIdx.x == 0) atomicOr(status, RAPID_STATUS_BAD_CTX_LEN);
        return;
    }
    const long long pos = L + i;
    const int blk = block_table[(size_t)b * max_blocks + pos / block_size];
    if (blk < 0 || blk >= num_blocks) {  // no block behind this position: the row is not written
        if (h == 0 && threadIdx.x == 0) atomicOr(status, RAPID_STATUS_BAD_BLOCK_TABLE);
        return;
    }
    const int chunks = D / 8;
    const size_t src = (((size_t)b * R + i) * Hkv + h) * chunks;
    const size_t dst = (size_t)blk * sblk + (size_t)h * sh + (size_t)(pos % block_size) * sl;
    for (int c = threadIdx.x; c < chunks; c += blockDim.x) {
        reinterpret_cast<uint4*>(k_pool + dst)[c] = k_new[src + c];
        reinterpret_cast<uint4*>(v_pool + dst)[c] = v_new[src + c];
    }
}

__global__ void kv_append_lens_kernel(int32_t* ctx_lens, int B, int R, long long Lmax) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const long long L = ctx_lens[b];
    if (L >= 0 && L + R <= Lmax) ctx_lens[b] = (int32_t)(L + R);
}

__global__ void step_commit_kernel(int32_t* ctx_lens, const int32_t* __restrict__ accept_len, int gamma, int B,
                                   int32_t* status) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    int n = accept_len[b];
    if (n < 0 || n > gamma) {
        atomicOr(status, RAPID_STATUS_BAD_CTX_LEN);
        n = n < 0 ? 0 : gamma;
    }
    ctx_lens[b] -= gamma - n;
}

}  // namespace

}  // namespace rapid

using namespace rapid;

extern "C" {

int rapid_kv_append(const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                    int32_t* ctx_lens, int gamma, const rapid_attn_shape* shape,
                    int32_t* status_word, void* cuda_stream) {
    clear_error();
    if (!k_new || !v_new || !k_cache || !v_cache || !ctx_lens || !shape || !status_word) {
        set_error("rapid_kv_append: NULL argument");
        return RAPID_ERR_INVALID_ARG;
    }
    const rapid_attn_shape& s = *shape;
    if (s.B <= 0 || s.Hkv <= 0 || s.Lmax <= 0 || gamma < 0 || s.B > 65535 || gamma + 1 > 65535) {
        set_error("rapid_kv_append: invalid shape");
        return RAPID_ERR_INVALID_ARG;
    }
    if (s.D <= 0 || s.D % 8) {
        set_error("rapid_kv_append: head_dim must be a positive multiple of 8");
        return RAPID_ERR_UNSUPPORTED;
    }
    const int64_t sl = s.kv_stride_l ? s.kv_stride_l : s.D;
    const int64_t sh = s.kv_stride_h ? s.kv_stride_h : s.Lmax * sl;
    const int64_t sb = s.kv_stride_b ? s.kv_stride_b : s.Hkv * sh;
    if (sl % 8 || sh % 8 || sb % 8 ||
        (((uintptr_t)k_new | (uintptr_t)v_new | (uintptr_t)k_cache | (uintptr_t)v_cache) & 15)) {
        set_error("rapid_kv_append: strides must be multiples of 8 elements and pointers 16-byte aligned");
        return RAPID_ERR_UNSUPPORTED;
    }
    const int R = gamma + 1;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    kv_append_kernel<<<dim3(s.Hkv, R, s.B), 32, 0, st>>>(
        static_cast<const uint4*>(k_new), static_cast<const uint4*>(v_new),
        static_cast<__nv_bfloat16*>(k_cache), static_cast<__nv_bfloat16*>(v_cache), ctx_lens, R, s.Hkv, s.D,
        (long long)s.Lmax, (long long)sb, (long long)sh, (long long)sl, status_word);
    kv_append_lens_kernel<<<(s.B + 127) / 128, 128, 0, st>>>(ctx_lens, s.B, R, (long long)s.Lmax);
    RAPID_CUDA_CHECK(cudaGetLastError());
    count_launch(2);
    return RAPID_OK;
}

int rapid_kv_append_paged(const void* k_new, const void* v_new, void* k_pool, void* v_pool,
                          const int32_t* block_table, const rapid_paged_kv* paged, int32_t* ctx_lens,
                          int gamma, int B, int Hkv, int D, int32_t* status_word, void* cuda_stream) {
    clear_error();
    if (!k_new || !v_new || !k_pool || !v_pool || !block_table || !paged || !ctx_lens || !status_word) {
        set_error("rapid_kv_append_paged: NULL argument");
        return RAPID_ERR_INVALID_ARG;
    }
    if (B <= 0 || Hkv <= 0 || gamma < 0 || B > 65535 || gamma + 1 > 65535 || paged->block_size <= 0 ||
        paged->num_blocks <= 0 || paged->max_blocks_per_seq <= 0) {
        set_error("rapid_kv_append_paged: invalid shape");
        return RAPID_ERR_INVALID_ARG;
    }
    if (D <= 0 || D % 8) {
        set_error("rapid_kv_append_paged: head_dim must be a positive multiple of 8");
        return RAPID_ERR_UNSUPPORTED;
    }
    const int64_t sl = paged->stride_l ? paged->stride_l : D;
    const int64_t sh = paged->stride_h ? paged->stride_h : (int64_t)paged->block_size * sl;
    const int64_t sblk = paged->stride_block ? paged->stride_block : Hkv * sh;
    if (sl % 8 || sh % 8 || sblk % 8 ||
        (((uintptr_t)k_new | (uintptr_t)v_new | (uintptr_t)k_pool | (uintptr_t)v_pool) & 15)) {
        set_error("rapid_kv_append_paged: strides must be multiples of 8 elements and pointers 16-byte aligned");
        return RAPID_ERR_UNSUPPORTED;
    }
    const int R = gamma + 1;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    kv_append_paged_kernel<<<dim3(Hkv, R, B), 32, 0, st>>>(
        static_cast<const uint4*>(k_new), static_cast<const uint4*>(v_new),
        static_cast<__nv_bfloat16*>(k_pool), static_cast<__nv_bfloat16*>(v_pool), block_table, ctx_lens, R,
        Hkv, D, paged->block_size, paged->num_blocks, paged->max_blocks_per_seq, (long long)sblk,
        (long long)sh, (long long)sl, status_word);
    kv_append_lens_kernel<<<(B + 127) / 128, 128, 0, st>>>(
        ctx_lens, B, R, (long long)paged->max_blocks_per_seq * paged->block_size);
    RAPID_CUDA_CHECK(cudaGetLastError());
    count_launch(2);
    return RAPID_OK;
}

int rapid_step_commit(int32_t* ctx_lens, const int32_t* accept_len, int gamma, int B,
                      int32_t* status_word, void* cuda_stream) {
    clear_error();
    if (!ctx_lens || !accept_len || !status_word || B <= 0 || gamma < 0) {
        set_error("rapid_step_commit: invalid argument");
        return RAPID_ERR_INVALID_ARG;
    }
    step_commit_kernel<<<(B + 127) / 128, 128, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        ctx_lens, accept_len, gamma, B, status_word);
    RAPID_CUDA_CHECK(cudaGetLastError());
    count_launch(1);
    return RAPID_OK;
}

size_t rapid_attention_workspace_bytes(const rapid_attn_shape* shape, int gamma) {
    return attention_workspace_bytes(shape, gamma);
}

size_t rapid_accept_workspace_bytes(const rapid_accept_shape* shape) {
    return accept_workspace_bytes(shape);
}

int rapid_workspace_init(void* workspace, size_t workspace_bytes, void* cuda_stream) {
    clear_error();
    if (!workspace || workspace_bytes < kWorkspaceHeaderBytes || ((uintptr_t)workspace & 255)) {
        set_error("rapid_workspace_init: need a 256-byte aligned workspace of at least %zu bytes",
                  kWorkspaceHeaderBytes);
        return RAPID_ERR_WORKSPACE;
    }
    RAPID_CUDA_CHECK(cudaMemsetAsync(workspace, 0, kWorkspaceHeaderBytes,
                                     static_cast<cudaStream_t>(cuda_stream)));
    return RAPID_OK;
}

int rapid_workspace_status(const void* workspace, void* cuda_stream, int32_t* host_status) {
    clear_error();
    if (!workspace || !host_status) {
        set_error("rapid_workspace_status: NULL argument");
        return RAPID_ERR_INVALID_ARG;
    }
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    RAPID_CUDA_CHECK(cudaMemcpyAsync(host_status, workspace, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    RAPID_CUDA_CHECK(cudaStreamSynchronize(st));
    return RAPID_OK;
}

int rapid_verify_attention(const void* q, const void* k_cache, const void* v_cache,
                           const int32_t* ctx_lens, int gamma, void* out,
                           const rapid_attn_shape* shape, const rapid_attn_params* params,
                           void* workspace, size_t workspace_bytes, void* cuda_stream) {
    clear_error();
    return launch_verify_attention(q, k_cache, v_cache, ctx_lens, gamma, out, shape, params,
                                   workspace, workspace_bytes,
                                   static_cast<cudaStream_t>(cuda_stream));
}

int rapid_verify_attention_fp8(const void* q, const void* k_cache, const void* v_cache, const float* k_scale,
                               const float* v_scale, const int32_t* ctx_lens, int gamma, void* out,
                               const rapid_attn_shape* shape, const rapid_attn_params* params, void* workspace,
                               size_t workspace_bytes, void* cuda_stream) {
    clear_error();
    return launch_verify_attention_fp8(q, k_cache, v_cache, k_scale, v_scale, ctx_lens, gamma, out, shape, params,
                                       workspace, workspace_bytes, static_cast<cudaStream_t>(cuda_stream));
}

int rapid_attention_plan(const int32_t* ctx_lens, int gamma, const rapid_attn_shape* shape,
                         const rapid_attn_params* params, void* workspace, size_t workspace_bytes,
                         void* cuda_stream) {
    clear_error();
    return launch_attention_plan(ctx_lens, gamma, shape, params, workspace, workspace_bytes,
                                 static_cast<cudaStream_t>(cuda_stream));
}

int rapid_attention_describe(const rapid_attn_shape* shape, int gamma, const rapid_attn_params* params,
                             rapid_attn_launch_info* info) {
    clear_error();
    return describe_attention(shape, gamma, params, info);
}

int rapid_verify_attention_paged(const void* q, const void* k_pool, const void* v_pool,
                                 const int32_t* block_table, const rapid_paged_kv* paged,
                                 const int32_t* ctx_lens, int gamma, void* out,
                                 const rapid_attn_shape* shape, const rapid_attn_params* params,
                                 void* workspace, size_t workspace_bytes, void* cuda_stream) {
    clear_error();
    if (!paged || !block_table) {
        set_error("rapid_verify_attention_paged: NULL paged geometry or block table");
        return RAPID_ERR_INVALID_ARG;
    }
    return launch_verify_attention(q, k_pool, v_pool, ctx_lens, gamma, out, shape, params, workspace,
                                   workspace_bytes, static_cast<cudaStream_t>(cuda_stream), paged,
                                   block_table);
}

int rapid_draft_sample(const float* draft_logits, const float* uniforms, float temperature, int32_t* out_token,
                       float* out_logq, float* out_row_stats, int32_t B, int64_t V, int64_t row_stride,
                       void* workspace, size_t workspace_bytes, void* cuda_stream) {
    clear_error();
    if (!out_logq) {
        set_error("rapid_draft_sample: out_logq is required");
        return RAPID_ERR_INVALID_ARG;
    }
    rapid_accept_shape shape = {B, 0, V, row_stride, 0};
    rapid_accept_params params = {temperature, 0.f, RAPID_RESIDUAL_PAPER, 0, nullptr, nullptr, nullptr};
    return launch_accept(draft_logits, nullptr, nullptr, uniforms, 0.f, nullptr, out_token, &shape, &params,
                         workspace, workspace_bytes, static_cast<cudaStream_t>(cuda_stream), out_logq,
                         out_row_stats);
}

int rapid_retrieval_select(const float* chunk_emb, const float* query_emb, const int32_t* n_chunks, int32_t B,
                           int32_t Nmax, int32_t Dm, float threshold, int32_t k, float* scores_out,
                           int32_t* sel_idx, int32_t* sel_count, int32_t* status_word, void* cuda_stream) {
    clear_error();
    return launch_retrieval_select(chunk_emb, query_emb, n_chunks, B, Nmax, Dm, threshold, k, scores_out, sel_idx,
                                   sel_count, status_word, static_cast<cudaStream_t>(cuda_stream));
}

int64_t rapid_retrieval_budget_chunks(int64_t context_tokens, int32_t chunk_tokens, int32_t floor_tokens,
                                      int32_t divisor) {
    clear_error();
    if (context_tokens < 0 || chunk_tokens <= 0 || floor_tokens <= 0 || divisor <= 0) {
        set_error("rapid_retrieval_budget_chunks: context_tokens >= 0 and positive chunk, floor and divisor wanted");
        return -1;
    }
    const int64_t share = context_tokens / divisor;
    return (share > floor_tokens ? share : (int64_t)floor_tokens) / chunk_tokens;
}

int rapid_merge_partials(const float* o_parts, const float* lse_parts, int P, int64_t rows, int D, void* out,
                         float* out_f32, float* lse_out, void* cuda_stream) {
    clear_error();
    return launch_merge_partials(o_parts, lse_parts, P, rows, D, out, out_f32, lse_out,
                                 static_cast<cudaStream_t>(cuda_stream));
}

int rapid_accept(const float* target_logits, const float* draft_logits,
                 const int32_t* draft_tokens, const float* uniforms, float eta,
                 int32_t* out_accept_len, int32_t* out_next_token,
                 const rapid_accept_shape* shape, const rapid_accept_params* params,
                 void* workspace, size_t workspace_bytes, void* cuda_stream) {
    clear_error();
    return launch_accept(target_logits, draft_logits, draft_tokens, uniforms, eta, out_accept_len,
                         out_next_token, shape, params, workspace, workspace_bytes,
                         static_cast<cudaStream_t>(cuda_stream));
}

int rapid_verify_step(const void* q, const void* k_cache, const void* v_cache,
                      const int32_t* ctx_lens, int gamma, void* out,
                      const rapid_attn_shape* attn_shape, const rapid_attn_params* attn_params,
                      void* attn_workspace, size_t attn_workspace_bytes,
                      const float* target_logits, const float* draft_logits,
                      const int32_t* draft_tokens, const float* uniforms, float eta,
                      int32_t* out_accept_len, int32_t* out_next_token,
                      const rapid_accept_shape* accept_shape,
                      const rapid_accept_params* accept_params, void* accept_workspace,
                      size_t accept_workspace_bytes, void* cuda_stream) {
    clear_error();
    if (accept_shape && attn_shape &&
        (accept_shape->gamma != gamma || accept_shape->B != attn_shape->B)) {
        set_error("rapid_verify_step: attention and accept shapes disagree on B or gamma");
        return RAPID_ERR_INVALID_ARG;
    }
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int rc = launch_verify_attention(q, k_cache, v_cache, ctx_lens, gamma, out, attn_shape,
                                     attn_params, attn_workspace, attn_workspace_bytes, st);
    if (rc != RAPID_OK) return rc;
    return launch_accept(target_logits, draft_logits, draft_tokens, uniforms, eta, out_accept_len,
                         out_next_token, accept_shape, accept_params, accept_workspace,
                         accept_workspace_bytes, st);
}

namespace {
struct HostArena {
    size_t q, k, v, ctx, out, z, d, tok, u, alen, ntok, attn_ws, acc_ws, total;
    size_t q_bytes, kv_bytes, ctx_bytes, z_bytes, d_bytes, tok_bytes, u_bytes, b_bytes;
    size_t attn_ws_bytes, acc_ws_bytes;
};

bool plan_host_arena(const rapid_attn_shape* as, int gamma, const rapid_accept_shape* cs,
                     HostArena& h) {
    if (!as || !cs || gamma < 0) return false;
    h.attn_ws_bytes = attention_workspace_bytes(as, gamma);
    h.acc_ws_bytes = accept_workspace_bytes(cs);
    if (!h.attn_ws_bytes || !h.acc_ws_bytes) return false;
    const size_t R = gamma + 1;
    h.q_bytes = (size_t)as->B * R * as->Hq * as->D * 2;
    h.kv_bytes = (size_t)as->B * as->Hkv * as->Lmax * as->D * 2;
    h.ctx_bytes = (size_t)as->B * 4;
    h.z_bytes = (size_t)cs->B * R * cs->V * 4;
    h.d_bytes = (size_t)cs->B * gamma * cs->V * 4;
    h.tok_bytes = (size_t)cs->B * gamma * 4;
    h.u_bytes = (size_t)cs->B * R * 4;
    h.b_bytes = (size_t)cs->B * 4;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t at = off;
        off += align_up(bytes ? bytes : 1, 256);
        return at;
    };
    h.q = take(h.q_bytes);
    h.k = take(h.kv_bytes);
    h.v = take(h.kv_bytes);
    h.ctx = take(h.ctx_bytes);
    h.out = take(h.q_bytes);
    h.z = take(h.z_bytes);
    h.d = take(h.d_bytes);
    h.tok = take(h.tok_bytes);
    h.u = take(h.u_bytes);
    h.alen = take(h.b_bytes);
    h.ntok = take(h.b_bytes);
    h.attn_ws = take(h.attn_ws_bytes);
    h.acc_ws = take(h.acc_ws_bytes);
    h.total = off;
    return true;
}
}  // namespace

size_t rapid_verify_step_host_arena_bytes(const rapid_attn_shape* attn_shape, int gamma,
                                          const rapid_accept_shape* accept_shape) {
    HostArena h;
    return plan_host_arena(attn_shape, gamma, accept_shape, h) ? h.total : 0;
}

int rapid_verify_step_host(const void* h_q, const void* h_k_cache, const void* h_v_cache,
                           const int32_t* h_ctx_lens, int gamma, void* h_out,
                           const rapid_attn_shape* attn_shape, const rapid_attn_params* attn_params,
                           const float* h_target_logits, const float* h_draft_logits,
                           const int32_t* h_draft_tokens, const float* h_uniforms, float eta,
                           int32_t* h_accept_len, int32_t* h_next_token,
                           const rapid_accept_shape* accept_shape,
                           const rapid_accept_params* accept_params, void* device_arena,
                           size_t device_arena_bytes, int32_t* h_status, void* cuda_stream) {
    clear_error();
    HostArena h;
    if (!plan_host_arena(attn_shape, gamma, accept_shape, h)) {
        set_error("rapid_verify_step_host: invalid shapes");
        return RAPID_ERR_INVALID_ARG;
    }
    if (!h_q || !h_k_cache || !h_v_cache || !h_ctx_lens || !h_out || !h_target_logits ||
        !h_uniforms || !h_accept_len || !h_next_token ||
        (gamma > 0 && (!h_draft_logits || !h_draft_tokens))) {
        set_error("rapid_verify_step_host: NULL argument");
        return RAPID_ERR_INVALID_ARG;
    }
    if (attn_shape->kv_stride_b || attn_shape->kv_stride_h || attn_shape->kv_stride_l ||
        accept_shape->target_row_stride || accept_shape->draft_row_stride) {
        set_error("rapid_verify_step_host: host tensors must be dense (all strides 0)");
        return RAPID_ERR_UNSUPPORTED;
    }
    if (accept_shape->gamma != gamma || accept_shape->B != attn_shape->B) {
        set_error("rapid_verify_step_host: attention and accept shapes disagree on B or gamma");
        return RAPID_ERR_INVALID_ARG;
    }
    if (!device_arena || device_arena_bytes < h.total || ((uintptr_t)device_arena & 255)) {
        set_error("rapid_verify_step_host: device arena of %zu bytes needed (256-byte aligned), got %zu",
                  h.total, device_arena_bytes);
        return RAPID_ERR_WORKSPACE;
    }
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint8_t* base = static_cast<uint8_t*>(device_arena);
    const cudaMemcpyKind H2D = cudaMemcpyHostToDevice, D2H = cudaMemcpyDeviceToHost;
    RAPID_CUDA_CHECK(cudaMemcpyAsync(base + h.q, h_q, h.q_bytes, H2D, st));
    RAPID_CUDA_CHECK(cudaMemcpyAsync(base + h.k, h_k_cache, h.kv_bytes, H2D, st));
    RAPID_CUDA_CHECK(cudaMemcpyAsync(base + h.v, h_v_cache, h.kv_bytes, H2D, st));
    RAPID_CUDA_CHECK(cudaMemcpyAsync(base + h.ctx, h_ctx_lens, h.ctx_bytes, H2D, st));
    RAPID_CUDA_CHECK(cudaMemcpyAsync(base + h.z, h_target_logits, h.z_bytes, H2D, st));
    if (gamma > 0) {
        RAPID_CUDA_CHECK(cudaMemcpyAsync(base + h.d, h_draft_logits, h.d_bytes, H2D, st));
        RAPID_CUDA_CHECK(cudaMemcpyAsync(base + h.tok, h_draft_tokens, h.tok_bytes, H2D, st));
    }
    RAPID_CUDA_CHECK(cudaMemcpyAsync(base + h.u, h_uniforms, h.u_bytes, H2D, st));
    RAPID_CUDA_CHECK(cudaMemsetAsync(base + h.attn_ws, 0, kWorkspaceHeaderBytes, st));
    RAPID_CUDA_CHECK(cudaMemsetAsync(base + h.acc_ws, 0, kWorkspaceHeaderBytes, st));
    int rc = launch_verify_attention(base + h.q, base + h.k, base + h.v,
                                     reinterpret_cast<const int32_t*>(base + h.ctx), gamma,
                                     base + h.out, attn_shape, attn_params, base + h.attn_ws,
                                     h.attn_ws_bytes, st);
    if (rc != RAPID_OK) return rc;
    rc = launch_accept(reinterpret_cast<const float*>(base + h.z),
                       reinterpret_cast<const float*>(base + h.d),
                       reinterpret_cast<const int32_t*>(base + h.tok),
                       reinterpret_cast<const float*>(base + h.u), eta,
                       reinterpret_cast<int32_t*>(base + h.alen),
                       reinterpret_cast<int32_t*>(base + h.ntok), accept_shape, accept_params,
                       base + h.acc_ws, h.acc_ws_bytes, st);
    if (rc != RAPID_OK) return rc;
    RAPID_CUDA_CHECK(cudaMemcpyAsync(h_out, base + h.out, h.q_bytes, D2H, st));
    RAPID_CUDA_CHECK(cudaMemcpyAsync(h_accept_len, base + h.alen, h.b_bytes, D2H, st));
    RAPID_CUDA_CHECK(cudaMemcpyAsync(h_next_token, base + h.ntok, h.b_bytes, D2H, st));
    int32_t st_words[2] = {0, 0};
    if (h_status) {
        RAPID_CUDA_CHECK(cudaMemcpyAsync(&st_words[0], base + h.attn_ws, 4, D2H, st));
        RAPID_CUDA_CHECK(cudaMemcpyAsync(&st_words[1], base + h.acc_ws, 4, D2H, st));
    }
    RAPID_CUDA_CHECK(cudaStreamSynchronize(st));
    if (h_status) *h_status = st_words[0] | st_words[1];
    return RAPID_OK;
}

const char* rapid_last_error(void) { return g_error; }
int rapid_version(void) { return RAPID_VERSION; }
int64_t rapid_kernel_launch_count(void) { return g_launches; }
void rapid_kernel_launch_count_reset(void) { g_launches = 0; }

}  // extern "C"
