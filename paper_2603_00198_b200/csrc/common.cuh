// Shared host/device helpers for libstr (sm_100a).  Not part of the public ABI.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "str.h"

// Per-category device timing (optional): an event pair around each leaf entry point.
enum {
    STR_CAT_GEMM = 0, STR_CAT_SSD, STR_CAT_MAMBA_SCORE, STR_CAT_ATTN_SCORE, STR_CAT_TOPK, STR_CAT_COMPACT,
    STR_CAT_ATTN_FWD, STR_CAT_ELEMENTWISE, STR_CAT_COUNT
};
struct str_prof_span { int cat; cudaEvent_t beg, end; };

struct str_ctx {
    int device;
    int sm_count;
    int max_smem_optin;
    int *status_dev;          // device status word: 0 or the first STR_ERR_* a kernel recorded
    void *encode_tiled;       // cuTensorMapEncodeTiled entry point (driver), or nullptr
    long long launches;       // host-side count of kernels launched through this context
    long long tc_calls;       // entry-point calls that took a tensor-core (tcgen05) kernel
    long long fallback_calls; // entry-point calls that took the plain fp32-FMA kernel of the same entry point
    size_t smem_attr[8];      // dynamic shared memory already opted into on this device, per tensor-core kernel
    int gemm_pairs;           // CTA pairs the GEMM can keep resident (0 = not asked yet, -1 = pairs unavailable)
    cudaStream_t copy_stream; // host-buffer entry point: input chunks are copied on this stream while the caller's
    cudaEvent_t copy_ev[24];  // stream computes; [0] orders the copies after the caller's earlier work, [1..8] = input
                              // chunk landed, [9..16] = output row block computed, [17] = output copies done
    bool prof_on;             // record an event pair per leaf call
    std::vector<str_prof_span> prof_spans;
    std::vector<cudaEvent_t> prof_free;
};

struct StrProfScope {
    str_ctx *ctx; cudaStream_t st; cudaEvent_t end; bool on;
    StrProfScope(str_ctx *c, int cat, void *stream) : ctx(c), st((cudaStream_t)stream), end(nullptr), on(false) {
        if (!c || !c->prof_on) return;
        cudaEvent_t ev[2];
        for (int i = 0; i < 2; ++i) {
            if (!c->prof_free.empty()) { ev[i] = c->prof_free.back(); c->prof_free.pop_back(); }
            else if (cudaEventCreate(&ev[i]) != cudaSuccess) return;
        }
        cudaEventRecord(ev[0], st);
        c->prof_spans.push_back({cat, ev[0], ev[1]});
        end = ev[1];
        on = true;
    }
    ~StrProfScope() { if (on) cudaEventRecord(end, st); }
};

#define STR_CUDA_OK(call)                          \
    do {                                           \
        cudaError_t _e = (call);                   \
        if (_e != cudaSuccess) return STR_ERR_CUDA; \
    } while (0)

static inline int str_launch_ok(str_ctx *ctx, int n = 1) {
    ctx->launches += n;
    return cudaGetLastError() == cudaSuccess ? STR_OK : STR_ERR_CUDA;
}

// Opt a kernel into `bytes` of dynamic shared memory once per context (the attribute belongs to the device the
// context was created on, so it is tracked per context, not per process).
enum { STR_SMEM_GEMM = 0, STR_SMEM_SSD, STR_SMEM_ATTN_FWD, STR_SMEM_MAMBA_SCORE, STR_SMEM_ATTN_ROWSTATS, STR_SMEM_ATTN_COLSUM,
       STR_SMEM_MAMBA_DYN_SCORE, STR_SMEM_GEMM_PAIR };
template <typename F>
static inline int str_ensure_smem(str_ctx *ctx, int slot, F kernel, size_t bytes) {
    // The attribute belongs to the device's copy of the kernel, not to this context: every context raises it to
    // the same value (the device's opt-in maximum), so contexts that share a device never lower it for each other.
    if (bytes > (size_t)ctx->max_smem_optin) return STR_ERR_UNSUPPORTED_SHAPE;
    if (ctx->smem_attr[slot]) return STR_OK;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin) != cudaSuccess) return STR_ERR_CUDA;
    ctx->smem_attr[slot] = (size_t)ctx->max_smem_optin;
    return STR_OK;
}

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
static inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
static inline size_t dtype_size(int dtype) { return dtype == STR_BF16 ? 2 : 4; }

// ---- device: scalar load/store with widening to fp32 ----
__device__ __forceinline__ float ldf(const float *p) { return *p; }
__device__ __forceinline__ float ldf(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
__device__ __forceinline__ void stf(float *p, float v) { *p = v; }
__device__ __forceinline__ void stf(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float silu_f(float v) { return v / (1.0f + expf(-v)); }
// SiLU on the special-function unit (ex2 and rcp approximations); the one definition every bf16 kernel uses, so that
// a fused and an unfused route through the same arithmetic give the same bits.
__device__ __forceinline__ float silu_fast(float v) {
    float e, r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(-1.4426950408889634f * v));
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.0f + e));
    return v * r;
}
__device__ __forceinline__ float softplus_f(float v) { return v > 20.0f ? v : log1pf(expf(v)); }
