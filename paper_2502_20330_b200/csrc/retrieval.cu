// Retrieval scoring for the RAG drafter's compressed context (Section 2.3; Section 3.1, "RAG
// Setup"): cosine similarity between a query embedding and the embeddings of the context's
// chunks, chunks below a similarity threshold dropped, the k most similar kept in order of
// similarity.  One CTA per request: a request has a few hundred chunks (128K tokens in 512-token
// chunks = 256) of ~1K dimensions, 1 MB in all, and runs once per request, not per token.
#include <math.h>

#include "common.cuh"

namespace rapid {

namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxChunksPerRequest = 4096;

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__global__ void __launch_bounds__(kThreads) retrieval_select_kernel(
    const float* __restrict__ chunk_emb, const float* __restrict__ query_emb,
    const int32_t* __restrict__ n_chunks, int Nmax, int Dm, float threshold, int k,
    float* __restrict__ scores_out, int32_t* __restrict__ sel_idx, int32_t* __restrict__ sel_count,
    int32_t* status) {
    extern __shared__ __align__(16) float sh[];  // [Dm] query, then [Nmax] scores
    float* qs = sh;
    float* sc = sh + Dm;
    __shared__ float sh_part[kWarps];
    __shared__ int sh_count;
    const int b = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    griddep_wait();
    griddep_launch_dependents();
    int n = n_chunks ? n_chunks[b] : Nmax;
    if (n < 0 || n > Nmax) {
        if (tid == 0) atomicOr(status, RAPID_STATUS_BAD_CTX_LEN);
        n = n < 0 ? 0 : Nmax;
    }
    const float* q = query_emb + (size_t)b * Dm;
    const float* E = chunk_emb + (size_t)b * Nmax * Dm;

    // the query and its norm
    float qq = 0.f;
    for (int d = tid; d < Dm; d += kThreads) {
        const float x = q[d];
        qs[d] = x;
        qq += x * x;
    }
    qq = warp_sum(qq);
    if (lane == 0) sh_part[warp] = qq;
    if (tid == 0) sh_count = 0;
    __syncthreads();
    qq = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) qq += sh_part[w];
    const float qnorm = sqrtf(qq);

    // one warp per chunk: dot product and norm in one pass over the embedding
    const int D4 = Dm >> 2;
    for (int i = warp; i < n; i += kWarps) {
        const float4* e = reinterpret_cast<const float4*>(E + (size_t)i * Dm);
        float dot = 0.f, ee = 0.f;
        for (int d = lane; d < D4; d += 32) {
            const float4 x = __ldg(e + d);
            const float4 y = reinterpret_cast<const float4*>(qs)[d];
            dot += x.x * y.x + x.y * y.y + x.z * y.z + x.w * y.w;
            ee += x.x * x.x + x.y * x.y + x.z * x.z + x.w * x.w;
        }
        dot = warp_sum(dot);
        ee = warp_sum(ee);
        if (lane == 0) {
            const float den = sqrtf(ee) * qnorm;
            const float s = den > 0.f ? dot / den : 0.f;  // a zero vector is similar to nothing
            sc[i] = s;
            scores_out[(size_t)b * Nmax + i] = s;
        }
    }
    for (int i = n + tid; i < Nmax; i += kThreads) scores_out[(size_t)b * Nmax + i] = 0.f;
    for (int j = tid; j < k; j += kThreads) sel_idx[(size_t)b * k + j] = -1;
    __syncthreads();

    // rank by counting: chunk i precedes chunk j if it scores higher, or the same with a lower
    // index.  Every chunk ahead of a chunk that passes the threshold passes it too, so the ranks
    // of the passing chunks are 0, 1, 2, ... and rank < k selects the k best of them.
    for (int i = tid; i < n; i += kThreads) {
        const float s = sc[i];
        if (!(s >= threshold)) continue;
        int rank = 0;
        for (int j = 0; j < n; ++j) {
            const float t = sc[j];
            rank += (t > s) || (t == s && j < i);
        }
        atomicAdd(&sh_count, 1);
        if (rank < k) sel_idx[(size_t)b * k + rank] = i;
    }
    __syncthreads();
    if (tid == 0) sel_count[b] = sh_count < k ? sh_count : k;
}

}  // namespace

int launch_retrieval_select(const float* chunk_emb, const float* query_emb, const int32_t* n_chunks, int B,
                            int Nmax, int Dm, float threshold, int k, float* scores_out, int32_t* sel_idx,
                            int32_t* sel_count, int32_t* status_word, cudaStream_t stream) {
    if (!chunk_emb || !query_emb || !scores_out || !sel_idx || !sel_count || !status_word) {
        set_error("rapid_retrieval_select: NULL argument");
        return RAPID_ERR_INVALID_ARG;
    }
    if (B <= 0 || Nmax <= 0 || Dm <= 0 || k <= 0 || !(threshold == threshold)) {
        set_error("rapid_retrieval_select: B, Nmax, Dm and k must be positive and the threshold a number");
        return RAPID_ERR_INVALID_ARG;
    }
    if (Nmax > kMaxChunksPerRequest || Dm % 4 || (size_t)(Dm + Nmax) * sizeof(float) > 200 * 1024 ||
        (((uintptr_t)chunk_emb | (uintptr_t)query_emb) & 15)) {
        set_error("rapid_retrieval_select: at most %d chunks per request, Dm a multiple of 4, Dm + Nmax floats "
                  "within 200 KB, embeddings 16-byte aligned", kMaxChunksPerRequest);
        return RAPID_ERR_UNSUPPORTED;
    }
    const size_t smem = (size_t)(Dm + Nmax) * sizeof(float);
    if (smem > 48 * 1024)
        RAPID_CUDA_CHECK(cudaFuncSetAttribute(retrieval_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)smem));
    RAPID_CUDA_CHECK(launch_dependent(retrieval_select_kernel, dim3(B), dim3(kThreads), smem, stream, chunk_emb,
                                      query_emb, n_chunks, Nmax, Dm, threshold, k, scores_out, sel_idx, sel_count,
                                      status_word));
    count_launch(1);
    return RAPID_OK;
}

}  // namespace rapid
