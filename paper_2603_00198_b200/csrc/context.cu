// Context management, error text, and the host-only retention-schedule helpers.
#include <math.h>
#include <new>

#include "common.cuh"

extern "C" int str_create(int device, str_ctx **out) {
    if (!out || device < 0) return STR_ERR_INVALID_ARG;
    int count = 0;
    STR_CUDA_OK(cudaGetDeviceCount(&count));
    if (device >= count) return STR_ERR_INVALID_ARG;
    STR_CUDA_OK(cudaSetDevice(device));
    str_ctx *c = new (std::nothrow) str_ctx();
    if (!c) return STR_ERR_CUDA;
    c->device = device;
    c->launches = 0;
    c->tc_calls = 0;
    c->fallback_calls = 0;
    c->prof_on = false;
    c->gemm_pairs = 0;
    for (size_t &v : c->smem_attr) v = 0;
    c->copy_stream = nullptr;
    for (cudaEvent_t &ev : c->copy_ev) ev = nullptr;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { delete c; return STR_ERR_CUDA; }
    c->sm_count = prop.multiProcessorCount;
    c->max_smem_optin = (int)prop.sharedMemPerBlockOptin;
    if (cudaMalloc(&c->status_dev, 256) != cudaSuccess) { delete c; return STR_ERR_CUDA; }
    if (cudaMemset(c->status_dev, 0, 256) != cudaSuccess) { cudaFree(c->status_dev); delete c; return STR_ERR_CUDA; }
    c->encode_tiled = nullptr;
    cudaDriverEntryPointQueryResult qres;
    void *fn = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
        c->encode_tiled = fn;
    (void)cudaGetLastError();
    if (!c->encode_tiled) {
        // Without the tensor-map encoder no tensor-core kernel can be launched.  Every call would quietly take the
        // fp32-FMA kernels, many times slower: refuse to create the context instead.
        cudaFree(c->status_dev);
        delete c;
        return STR_ERR_CUDA;
    }
    *out = c;
    return STR_OK;
}

extern "C" int str_destroy(str_ctx *ctx) {
    if (!ctx) return STR_ERR_INVALID_ARG;
    cudaFree(ctx->status_dev);
    for (auto &sp : ctx->prof_spans) { cudaEventDestroy(sp.beg); cudaEventDestroy(sp.end); }
    for (auto &ev : ctx->prof_free) cudaEventDestroy(ev);
    for (cudaEvent_t ev : ctx->copy_ev)
        if (ev) cudaEventDestroy(ev);
    if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
    delete ctx;
    return STR_OK;
}

extern "C" const char *str_strerror(int code) {
    switch (code) {
        case STR_OK: return "ok";
        case STR_ERR_INVALID_ARG: return "invalid argument";
        case STR_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
        case STR_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case STR_ERR_CUDA: return "CUDA error";
        case STR_ERR_TIMEOUT: return "device-side wait timed out";
        default: return "unknown error";
    }
}

extern "C" int str_check_status(str_ctx *ctx, void *stream) {
    if (!ctx) return STR_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    int host = 0;
    STR_CUDA_OK(cudaMemcpyAsync(&host, ctx->status_dev, sizeof(int), cudaMemcpyDeviceToHost, st));
    STR_CUDA_OK(cudaStreamSynchronize(st));
    if (host != 0) {
        STR_CUDA_OK(cudaMemsetAsync(ctx->status_dev, 0, sizeof(int), st));
        STR_CUDA_OK(cudaStreamSynchronize(st));
    }
    return host;
}

extern "C" int str_profile_enable(str_ctx *ctx, int on) {
    if (!ctx) return STR_ERR_INVALID_ARG;
    ctx->prof_on = on != 0;
    return STR_OK;
}

extern "C" int str_profile_collect(str_ctx *ctx, double *ms_by_category, long long *calls_by_category, int n) {
    if (!ctx || !ms_by_category || !calls_by_category || n < STR_CAT_COUNT) return STR_ERR_INVALID_ARG;
    for (int i = 0; i < n; ++i) { ms_by_category[i] = 0.0; calls_by_category[i] = 0; }
    for (auto &sp : ctx->prof_spans) {
        if (cudaEventSynchronize(sp.end) != cudaSuccess) return STR_ERR_CUDA;
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, sp.beg, sp.end) != cudaSuccess) return STR_ERR_CUDA;
        ms_by_category[sp.cat] += ms;
        calls_by_category[sp.cat] += 1;
        ctx->prof_free.push_back(sp.beg);
        ctx->prof_free.push_back(sp.end);
    }
    ctx->prof_spans.clear();
    return STR_OK;
}

extern "C" long long str_launch_count(const str_ctx *ctx) { return ctx ? ctx->launches : -1; }

extern "C" int str_path_counts(const str_ctx *ctx, long long *tensor_core_calls, long long *fallback_calls) {
    if (!ctx || !tensor_core_calls || !fallback_calls) return STR_ERR_INVALID_ARG;
    *tensor_core_calls = ctx->tc_calls;
    *fallback_calls = ctx->fallback_calls;
    return STR_OK;
}

// Section 3.2 / appendix schedules: alpha is a fraction of the original visual count.
extern "C" int str_schedule_keep_counts(const int *alpha_bp, int L, int n0, int min_keep, int *K_out) {
    if (!alpha_bp || !K_out || L < 0 || n0 < 0 || min_keep < 0) return STR_ERR_INVALID_ARG;
    long long n_cur = n0;
    for (int l = 0; l < L; ++l) {
        if (alpha_bp[l] < 0 || alpha_bp[l] > 10000) return STR_ERR_INVALID_ARG;
        long long k = ((long long)alpha_bp[l] * (long long)n0) / 10000;
        if (k < min_keep) k = min_keep;
        if (k > n_cur) k = n_cur;
        K_out[l] = (int)k;
        n_cur = k;
    }
    return STR_OK;
}

// Same with the layer kinds known: FFN layers only transform the rows they are given, so a cut that the schedule
// places on one is taken by the next Mamba / attention layer (the paper's all-layer schedules cut at those).
extern "C" int str_schedule_keep_counts_layers(const int *alpha_bp, const int *layer_kinds, int L, int n0, int min_keep,
                                               int *K_out) {
    if (!layer_kinds) return STR_ERR_INVALID_ARG;
    int rc = str_schedule_keep_counts(alpha_bp, L, n0, min_keep, K_out);
    if (rc != STR_OK) return rc;
    int n_cur = n0;
    for (int l = 0; l < L; ++l) {
        if (layer_kinds[l] != STR_LAYER_MAMBA && layer_kinds[l] != STR_LAYER_ATTN && layer_kinds[l] != STR_LAYER_FFN)
            return STR_ERR_INVALID_ARG;
        if (layer_kinds[l] != STR_LAYER_FFN && K_out[l] < n_cur) n_cur = K_out[l];
        K_out[l] = n_cur;
    }
    return STR_OK;
}

extern "C" int str_sigmoid_schedule_bp(int L, double k, double x0, double a_start, double a_end, int *alpha_bp_out) {
    if (!alpha_bp_out || L <= 0) return STR_ERR_INVALID_ARG;
    for (int l = 0; l < L; ++l) {
        double sg = 1.0 / (1.0 + exp(-k * (x0 - (double)l / (double)L)));
        double a = a_end + (a_start - a_end) * sg;
        long long bp = llround(a * 10000.0);
        if (bp < 0) bp = 0;
        if (bp > 10000) bp = 10000;
        alpha_bp_out[l] = (int)bp;
    }
    return STR_OK;
}
