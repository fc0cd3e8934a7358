// Diagnostics that sit beside the hot path: the density statistic of a score vector (how many tokens carry a
// given fraction of the importance mass) and a self-test of the bounded-wait / status-word mechanism.
#include "dispatch.cuh"
#include "tc_common.cuh"

namespace {

// ---- density statistic -------------------------------------------------------------------------
// Per row: the smallest k such that the k largest scores sum to at least `frac` of the row's total.  The dual of
// the top-K radix select: instead of a rank threshold the four 8-bit passes look for a MASS threshold.  Each
// pass histograms (count, fp64 sum) of the still-undecided scores by the next 8 key bits and walks the buckets
// from the top until the running mass would reach the target; after the last pass the threshold VALUE v is known
// exactly, and the answer is (#scores > v) + the number of copies of v still needed.
constexpr int DENS_THREADS = 1024;

__global__ void __launch_bounds__(DENS_THREADS, 1)
score_density_kernel(const float *__restrict__ scores, int n, double frac, int32_t *__restrict__ count_out) {
    __shared__ unsigned int h_cnt[256];
    __shared__ double h_sum[256];
    __shared__ double red[DENS_THREADS / 32];
    __shared__ unsigned int s_prefix, s_above_cnt, s_sel_cnt;
    __shared__ double s_above_sum, s_total;
    const float *row = scores + (size_t)blockIdx.x * n;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;

    double part = 0.0;
    for (int i = tid; i < n; i += DENS_THREADS) part += (double)row[i];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
    if (lane == 0) red[wid] = part;
    __syncthreads();
    if (tid == 0) {
        double t = 0.0;
        for (int w = 0; w < DENS_THREADS / 32; ++w) t += red[w];
        s_total = t;
        s_prefix = 0u; s_above_cnt = 0u; s_above_sum = 0.0; s_sel_cnt = 0u;
    }
    __syncthreads();
    const double total = s_total;
    if (!(total > 0.0)) {                         // an all-zero row carries no mass: zero tokens
        if (tid == 0) count_out[blockIdx.x] = 0;
        return;
    }
    const double target = frac * total;
    unsigned int mask = 0u;
#pragma unroll 1
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        if (tid < 256) { h_cnt[tid] = 0u; h_sum[tid] = 0.0; }
        __syncthreads();
        const unsigned int prefix = s_prefix;
        for (int i = tid; i < n; i += DENS_THREADS) {
            const float v = row[i];
            const unsigned int key = __float_as_uint(v);      // scores are >= 0: the bit pattern orders like the value
            if ((key & mask) == prefix) {
                const unsigned int b = (key >> shift) & 255u;
                atomicAdd(&h_cnt[b], 1u);
                atomicAdd(&h_sum[b], (double)v);
            }
        }
        __syncthreads();
        if (tid == 0) {
            double above = s_above_sum;
            unsigned int cnt = s_above_cnt;
            int b = 255;
            for (; b > 0; --b) {
                if (h_cnt[b] == 0u) continue;
                if (above + h_sum[b] >= target) break;
                above += h_sum[b];
                cnt += h_cnt[b];
            }
            s_above_sum = above;
            s_above_cnt = cnt;
            s_sel_cnt = h_cnt[b];
            s_prefix = prefix | ((unsigned int)b << shift);
        }
        mask |= 255u << shift;
        __syncthreads();
    }
    if (tid == 0) {
        const double v = (double)__uint_as_float(s_prefix);
        long long need = 0;
        if (v > 0.0) {
            need = (long long)ceil((target - s_above_sum) / v);
            if (need < 1) need = 1;
            if (need > (long long)s_sel_cnt) need = (long long)s_sel_cnt;
        }
        count_out[blockIdx.x] = (int32_t)((long long)s_above_cnt + need);
    }
}

// ---- bounded-wait self-test ----------------------------------------------------------------------
// One CTA waits on an mbarrier that nobody ever arrives at, with the probe limit given by the caller, gives up,
// records STR_ERR_TIMEOUT in the status word and returns: the same give-up path every pipelined kernel of the
// library has, exercised without any of their machinery (no TMA, no tensor memory).
__global__ void wait_timeout_selftest_kernel(unsigned int probe_limit, int *status) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        tc::mbar_init(&bar, 1);
        tc::fence_mbar_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned int probes = 0;
        bool done = false;
        while (!(done = tc::mbar_try_wait(&bar, 0)) && ++probes < probe_limit) { }
        if (!done) atomicCAS(status, 0, STR_ERR_TIMEOUT);
    }
}

}  // namespace

extern "C" int str_score_density(str_ctx *ctx, int Bz, int n_vis, const float *scores, float mass_fraction,
                                 int32_t *count_out, void *stream) {
    if (!ctx || Bz <= 0 || n_vis < 0 || !(mass_fraction > 0.f) || mass_fraction > 1.f) return STR_ERR_INVALID_ARG;
    if (!count_out || (n_vis > 0 && !scores)) return STR_ERR_INVALID_ARG;
    if (n_vis == 0) {
        STR_CUDA_OK(cudaMemsetAsync(count_out, 0, (size_t)Bz * sizeof(int32_t), (cudaStream_t)stream));
        return STR_OK;
    }
    score_density_kernel<<<Bz, DENS_THREADS, 0, (cudaStream_t)stream>>>(scores, n_vis, (double)mass_fraction, count_out);
    return str_launch_ok(ctx);
}

extern "C" int str_selftest_wait_timeout(str_ctx *ctx, unsigned int probe_limit, void *stream) {
    if (!ctx || probe_limit == 0 || probe_limit > (1u << 20)) return STR_ERR_INVALID_ARG;
    wait_timeout_selftest_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(probe_limit, ctx->status_dev);
    return str_launch_ok(ctx);
}
