// Shared host/device helpers of the RAPID verify-step library: error plumbing,
// bounded mbarrier waits, TMA and tensor-core PTX wrappers for sm_100a.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "rapid.h"

namespace rapid {

// ---- host-side error plumbing -------------------------------------------------------------
void set_error(const char* fmt, ...);
void clear_error();
void count_launch(int n = 1);

#define RAPID_CUDA_CHECK(expr)                                                              \
    do {                                                                                    \
        cudaError_t err__ = (expr);                                                         \
        if (err__ != cudaSuccess) {                                                         \
            ::rapid::set_error("%s failed: %s (%s:%d)", #expr, cudaGetErrorString(err__),    \
                               __FILE__, __LINE__);                                         \
            return RAPID_ERR_CUDA;                                                          \
        }                                                                                   \
    } while (0)

constexpr size_t kWorkspaceHeaderBytes = 256;  // status word + bookkeeping, cleared by init
constexpr int kMaxCtas = 512;                  // upper bound on the KV split (sizes the workspace)

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

#if defined(__CUDACC__)
// Launch as a programmatic dependent of the preceding kernel in the stream: the kernel may start
// early and must call griddep_wait() before it reads anything an earlier kernel wrote.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                    cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

// internal launchers shared by the entry points (defined in attention.cu / accept.cu)
int launch_verify_attention(const void* q, const void* k_cache, const void* v_cache,
                            const int32_t* ctx_lens, int gamma, void* out,
                            const rapid_attn_shape* shape, const rapid_attn_params* params,
                            void* workspace, size_t workspace_bytes, cudaStream_t stream,
                            const rapid_paged_kv* paged = nullptr, const int32_t* block_table = nullptr);
int launch_verify_attention_fp8(const void* q, const void* k_cache, const void* v_cache, const float* k_scale,
                                const float* v_scale, const int32_t* ctx_lens, int gamma, void* out,
                                const rapid_attn_shape* shape, const rapid_attn_params* params, void* workspace,
                                size_t workspace_bytes, cudaStream_t stream);
int launch_attention_plan(const int32_t* ctx_lens, int gamma, const rapid_attn_shape* shape,
                          const rapid_attn_params* params, void* workspace, size_t workspace_bytes,
                          cudaStream_t stream);
int describe_attention(const rapid_attn_shape* shape, int gamma, const rapid_attn_params* params,
                       rapid_attn_launch_info* info);
int launch_retrieval_select(const float* chunk_emb, const float* query_emb, const int32_t* n_chunks, int B,
                            int Nmax, int Dm, float threshold, int k, float* scores_out, int32_t* sel_idx,
                            int32_t* sel_count, int32_t* status_word, cudaStream_t stream);
int launch_merge_partials(const float* o_parts, const float* lse_parts, int P, int64_t rows, int D, void* out,
                          float* out_f32, float* lse_out, cudaStream_t stream);
int launch_accept(const float* target_logits, const float* draft_logits,
                  const int32_t* draft_tokens, const float* uniforms, float eta,
                  int32_t* out_accept_len, int32_t* out_next_token,
                  const rapid_accept_shape* shape, const rapid_accept_params* params,
                  void* workspace, size_t workspace_bytes, cudaStream_t stream, float* logq_out = nullptr,
                  float* stats_out = nullptr);

// ---- device-side PTX wrappers ---------------------------------------------------------------
#if defined(__CUDACC__)

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}

__device__ __forceinline__ void fence_mbar_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void fence_proxy_async_smem() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
                 "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// The same test, but the hardware may park the thread until the phase completes or `ns` nanoseconds
// have passed: a waiting warp then costs its scheduler no issue slots.
__device__ __forceinline__ bool mbar_try_wait_parked(uint64_t* bar, uint32_t parity, uint32_t ns) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity), "r"(ns)
        : "memory");
    return ok != 0;
}

// Every wait on an mbarrier is bounded: after `limit` clock cycles (kWaitCycleLimit, about a
// second, unless the call names another figure) the waiter raises *abort (shared memory), which
// makes every later wait of the CTA return at once, and the kernel records
// RAPID_STATUS_PIPELINE_TIMEOUT.  Returns false on timeout / abort.
constexpr long long kWaitCycleLimit = 2000000000LL;

struct WaitCtx {
    volatile int* abort;  // the CTA's abort flag (shared memory)
    long long limit;      // clock cycles a wait may take
};

// Same wait for a role that is not on the critical path (the TMA producer runs several stages
// ahead): it sleeps between polls instead of spinning, which saves power for the clocks.
__device__ __forceinline__ bool mbar_wait_bounded_relaxed(uint64_t* bar, uint32_t parity, const WaitCtx& wc) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        __nanosleep(200);
        if (mbar_try_wait(bar, parity)) return true;
        if (*wc.abort) return false;
        if (clock64() - t0 > wc.limit) {
            *wc.abort = 1;
            return false;
        }
    }
}

__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, const WaitCtx& wc) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        if (mbar_try_wait_parked(bar, parity, 2000)) return true;
        if (*wc.abort) return false;
        if (clock64() - t0 > wc.limit) {
            *wc.abort = 1;
            return false;
        }
    }
}

// The wait of a role that is leaving after an abort and must see its own asynchronous work land
// first (a bulk copy it issued, the MMAs it committed): the abort flag does not end it, only the
// barrier or the library's own limit does.  Such work always completes, so this returns true
// unless the hardware has stopped.
static __device__ __noinline__ bool mbar_wait_drain(uint64_t* bar, uint32_t parity) {
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (clock64() - t0 > kWaitCycleLimit) return false;
        __nanosleep(100);
    }
    return true;
}

// 4-D tiled TMA load global -> shared, completion counted on an mbarrier (no multicast).
__device__ __forceinline__ void tma_load_4d(void* smem_dst, const CUtensorMap* map, uint64_t* bar,
                                            int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cta.global.tile.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%3, %4, %5, %6}], [%2];" ::"r"(smem_u32(smem_dst)),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2),
        "r"(c3)
        : "memory");
}

__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

// Programmatic dependent launch (kernels launched with cudaLaunchAttributeProgrammaticStreamSerialization):
// wait = the preceding kernel in the stream has completed and its writes are visible;
// launch_dependents = the next such kernel may start running its own prologue.
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;"); }

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

#endif  // __CUDACC__

}  // namespace rapid
