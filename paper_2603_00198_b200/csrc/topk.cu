// str_topk_select: per-sequence radix select of the k largest fp32 scores, emitted in
// ascending index order (temporal order preserved; ties go to the lower index).
//
// Three paths: rows of up to 131072 scores are shared by a thread-block cluster that keeps the keys in
// registers (second part of this file); longer rows are split over many CTAs whose passes meet in a workspace
// (last part); without a workspace a long row takes one CTA that re-reads the scores every pass.  All: four 8-bit MSB-first passes over the order-preserving integer image
// of the scores narrow down the k-th largest key; per-warp private histograms with
// warp-aggregated increments keep shared-memory atomics uncontended even when every score
// shares its top byte.  A last ordered pass emits the survivors: each warp owns a contiguous
// index segment, so a single block-level exclusive scan of 32 warp counts orders the output.
#include <cooperative_groups.h>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace {

constexpr int TOPK_THREADS = 1024;
constexpr int TOPK_WARPS = TOPK_THREADS / 32;

__device__ __forceinline__ uint32_t score_key(float s) {
    const uint32_t u = __float_as_uint(s);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);   // larger float <=> larger key
}

__global__ void __launch_bounds__(TOPK_THREADS)
topk_select_kernel(int n, int k, const float *__restrict__ scores, int32_t *__restrict__ kept) {
    __shared__ uint32_t hist[TOPK_WARPS][256];
    __shared__ uint32_t total[256];
    __shared__ uint32_t sh_prefix, sh_need;
    __shared__ uint32_t warp_gt[TOPK_WARPS], warp_eq[TOPK_WARPS];

    const float *s = scores + (size_t)blockIdx.x * n;
    int32_t *out = kept + (size_t)blockIdx.x * k;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (k <= 0) return;

    uint32_t prefix = 0, mask = 0, need = (uint32_t)k;
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int i = tid; i < TOPK_WARPS * 256; i += TOPK_THREADS) (&hist[0][0])[i] = 0;
        __syncthreads();
        const int n_round = (n + 31) & ~31;
        for (int i = tid; i < n_round; i += TOPK_THREADS) {
            const bool in = i < n;
            const uint32_t key = in ? score_key(s[i]) : 0u;
            const bool live = in && ((key & mask) == prefix);
            const uint32_t bin = (key >> shift) & 255u;
            // warp-aggregated increment: lanes with the same bin elect one leader
            const uint32_t live_mask = __ballot_sync(0xffffffffu, live);
            if (live) {
                const uint32_t peers = __match_any_sync(live_mask, bin);
                if (lane == __ffs(peers) - 1) hist[warp][bin] += __popc(peers);
            }
            __syncwarp();
        }
        __syncthreads();
        if (tid < 256) {
            uint32_t t = 0;
#pragma unroll 8
            for (int w = 0; w < TOPK_WARPS; ++w) t += hist[w][tid];
            total[tid] = t;
        }
        __syncthreads();
        if (warp == 0) {
            // lane L owns bins 255-8L .. 248-8L (descending); find the bin holding the need-th largest
            uint32_t c[8], lane_sum = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) { c[j] = total[255 - 8 * lane - j]; lane_sum += c[j]; }
            uint32_t incl = lane_sum;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += v;
            }
            const uint32_t before = incl - lane_sum;
            if (before < need && need <= incl) {
                uint32_t run = before;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (run < need && need <= run + c[j]) {
                        sh_prefix = prefix | ((uint32_t)(255 - 8 * lane - j) << shift);
                        sh_need = need - run;
                    }
                    run += c[j];
                }
            }
        }
        __syncthreads();
        prefix = sh_prefix;
        need = sh_need;
        mask |= 255u << shift;
        __syncthreads();
    }
    // prefix = key of the k-th largest score; every key > prefix is kept, plus the first `need`
    // (in index order) of the keys == prefix.
    const int seg = (((n + TOPK_WARPS - 1) / TOPK_WARPS) + 31) & ~31;
    const int lo = warp * seg, hi = min(n, lo + seg);
    uint32_t gt = 0, eq = 0;
    for (int i = lo + lane; i < lo + seg; i += 32) {
        const bool in = i < hi;
        const uint32_t key = in ? score_key(s[i]) : 0u;
        gt += __popc(__ballot_sync(0xffffffffu, in && key > prefix));
        eq += __popc(__ballot_sync(0xffffffffu, in && key == prefix));
    }
    if (lane == 0) { warp_gt[warp] = gt; warp_eq[warp] = eq; }
    __syncthreads();
    uint32_t gt_before = 0, eq_before = 0;
    for (int w = 0; w < warp; ++w) { gt_before += warp_gt[w]; eq_before += warp_eq[w]; }
    const uint32_t lt_mask = (1u << lane) - 1u;
    for (int i = lo + lane; i < lo + seg; i += 32) {
        const bool in = i < hi;
        const uint32_t key = in ? score_key(s[i]) : 0u;
        const bool is_gt = in && key > prefix, is_eq = in && key == prefix;
        const uint32_t gt_b = __ballot_sync(0xffffffffu, is_gt);
        const uint32_t eq_b = __ballot_sync(0xffffffffu, is_eq);
        const uint32_t eq_rank = eq_before + __popc(eq_b & lt_mask);
        const bool take = is_gt || (is_eq && eq_rank < need);
        const uint32_t take_b = __ballot_sync(0xffffffffu, take);
        if (take) {
            const uint32_t pos = gt_before + min(eq_before, need) + __popc(take_b & lt_mask);
            out[pos] = i;
        }
        gt_before += __popc(gt_b);
        eq_before += __popc(eq_b);
    }
}


// ------------------------------------------------------------------------------------------
// Cluster version for rows of up to CL_MAX_N scores: a thread-block cluster of up to 8 CTAs shares one row.
// Every thread keeps a contiguous run of KPT keys in registers, so the scores are read from memory once.
// Per radix pass each CTA builds a 256-bin histogram of its live keys in shared memory; after one cluster
// barrier every CTA sums the histograms of the whole cluster through distributed shared memory and takes
// the same decision (histograms are double-buffered, so one barrier per pass is enough).  The ordered emit
// uses a block scan of per-thread (greater, equal) counts plus the totals of the lower-ranked CTAs.
constexpr int CL_THREADS = 1024, CL_MAX_CTAS = 8, CL_MAX_KPT = 16;
constexpr int CL_MAX_N = CL_THREADS * CL_MAX_CTAS * CL_MAX_KPT;      // 131072

template <int KPT>
__global__ void __launch_bounds__(CL_THREADS)
topk_cluster_kernel(int n, int k, const float *__restrict__ scores, int32_t *__restrict__ kept) {
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank(), ncta = (int)cluster.num_blocks();
    __shared__ uint32_t hist[2][256];
    __shared__ uint32_t total[256];
    __shared__ uint32_t sh_prefix, sh_need;
    __shared__ uint32_t warp_gt[32], warp_eq[32];
    __shared__ uint32_t cta_tot[2];

    const float *s = scores + (size_t)blockIdx.y * n;
    int32_t *out = kept + (size_t)blockIdx.y * k;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int per_cta = KPT * CL_THREADS;
    const int base = rank * per_cta + tid * KPT;                     // first index of this thread's run

    uint32_t key[KPT];
#pragma unroll
    for (int j = 0; j < KPT; ++j) key[j] = (base + j < n) ? score_key(__ldg(s + base + j)) : 0u;

    uint32_t prefix = 0, mask = 0, need = (uint32_t)k;
    int pass = 0;
    for (int shift = 24; shift >= 0; shift -= 8, ++pass) {
        uint32_t *h = hist[pass & 1];
        if (tid < 256) h[tid] = 0;
        __syncthreads();
#pragma unroll
        for (int j = 0; j < KPT; ++j) {
            const bool live = (base + j < n) && ((key[j] & mask) == prefix);
            const uint32_t bin = (key[j] >> shift) & 255u;
            const uint32_t live_mask = __ballot_sync(0xffffffffu, live);
            if (live) {       // warp-aggregated increment: lanes with the same bin elect one leader
                const uint32_t peers = __match_any_sync(live_mask, bin);
                if (lane == __ffs(peers) - 1) atomicAdd(&h[bin], (uint32_t)__popc(peers));
            }
            __syncwarp();
        }
        cluster.sync();
        if (tid < 256) {
            uint32_t t = 0;
            for (int r = 0; r < ncta; ++r) t += cluster.map_shared_rank(h, r)[tid];
            total[tid] = t;
        }
        __syncthreads();
        if (warp == 0) {
            // lane L owns bins 255-8L .. 248-8L (descending); find the bin holding the need-th largest
            uint32_t c[8], lane_sum = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) { c[j] = total[255 - 8 * lane - j]; lane_sum += c[j]; }
            uint32_t incl = lane_sum;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += v;
            }
            const uint32_t before = incl - lane_sum;
            if (before < need && need <= incl) {
                uint32_t run = before;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (run < need && need <= run + c[j]) {
                        sh_prefix = prefix | ((uint32_t)(255 - 8 * lane - j) << shift);
                        sh_need = need - run;
                    }
                    run += c[j];
                }
            }
        }
        __syncthreads();
        prefix = sh_prefix;
        need = sh_need;
        mask |= 255u << shift;
    }
    // prefix = key of the k-th largest score; keep every key > prefix plus the first `need` (in index order)
    // of the keys == prefix
    uint32_t gt = 0, eq = 0;
#pragma unroll
    for (int j = 0; j < KPT; ++j) {
        const bool in = base + j < n;
        gt += (in && key[j] > prefix) ? 1u : 0u;
        eq += (in && key[j] == prefix) ? 1u : 0u;
    }
    uint32_t gt_incl = gt, eq_incl = eq;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t a = __shfl_up_sync(0xffffffffu, gt_incl, o), b2 = __shfl_up_sync(0xffffffffu, eq_incl, o);
        if (lane >= o) { gt_incl += a; eq_incl += b2; }
    }
    if (lane == 31) { warp_gt[warp] = gt_incl; warp_eq[warp] = eq_incl; }
    __syncthreads();
    if (warp == 0) {
        uint32_t a = warp_gt[lane], b2 = warp_eq[lane], ai = a, bi = b2;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t x = __shfl_up_sync(0xffffffffu, ai, o), y = __shfl_up_sync(0xffffffffu, bi, o);
            if (lane >= o) { ai += x; bi += y; }
        }
        warp_gt[lane] = ai - a;                                      // exclusive prefix over warps
        warp_eq[lane] = bi - b2;
        if (lane == 31) { cta_tot[0] = ai; cta_tot[1] = bi; }
    }
    cluster.sync();
    uint32_t gt_before = warp_gt[warp] + (gt_incl - gt), eq_before = warp_eq[warp] + (eq_incl - eq);
    for (int r = 0; r < rank; ++r) {
        const uint32_t *t = cluster.map_shared_rank(cta_tot, r);
        gt_before += t[0];
        eq_before += t[1];
    }
#pragma unroll
    for (int j = 0; j < KPT; ++j) {
        const bool in = base + j < n;
        const bool is_gt = in && key[j] > prefix, is_eq = in && key[j] == prefix;
        if (is_gt || (is_eq && eq_before < need)) out[gt_before + min(eq_before, need)] = base + j;
        gt_before += is_gt ? 1u : 0u;
        eq_before += is_eq ? 1u : 0u;
    }
    cluster.sync();           // no CTA leaves while another may still read its shared memory
}

template <int KPT>
cudaError_t launch_cluster(int ncta, int Bz, int n, int k, const float *scores, int32_t *kept, cudaStream_t st) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ncta, Bz, 1);
    cfg.blockDim = dim3(CL_THREADS, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = ncta;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, topk_cluster_kernel<KPT>, n, k, scores, kept);
}

// ------------------------------------------------------------------------------------------
// Long rows (more than CL_MAX_N scores): the row is split over as many CTAs as it needs, GR_KEYS scores each, and
// the four radix passes become kernel launches that meet in a caller-provided workspace:
//   pass p:  grid_hist_kernel   every CTA histograms digit p of its keys that still match the prefix and adds its 256
//                               bins to the row's global histogram (integer atomics: the result is order-free);
//                               the prefix itself is recomputed by every CTA from the histograms of passes 0..p-1
//   then     grid_count_kernel  per CTA, how many keys lie above the threshold and how many equal it
//            grid_emit_kernel   every CTA sums the counts of the CTAs before it and emits its survivors in order
// Workspace per row: 4 x 256 histogram words | (gt, eq) per CTA.
constexpr int GR_KEYS = 16384;            // scores per CTA: 16 per thread

struct GridWs { uint32_t *hist; uint32_t *counts; };   // [Bz][4][256], [Bz][nblk][2]

// The threshold known after `passes` radix passes, recomputed by every CTA from the row's global histograms (a few
// hundred loads) instead of by a kernel of its own: warp 0 walks the passes, each time picking the bin that holds
// the need-th largest live key.  Result in sh[0] = prefix, sh[1] = need; the caller synchronises the block.
__device__ __forceinline__ void grid_resolve(const uint32_t *__restrict__ row_hist, int passes, int k, uint32_t *sh) {
    if (threadIdx.x >= 32) return;
    const int lane = threadIdx.x;
    uint32_t prefix = 0u, need = (uint32_t)k;
    for (int p = 0; p < passes; ++p) {
        const uint32_t *total = row_hist + p * 256;
        const int shift = 24 - 8 * p;
        // lane L owns bins 255-8L .. 248-8L (descending)
        uint32_t c[8], lane_sum = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) { c[j] = total[255 - 8 * lane - j]; lane_sum += c[j]; }
        uint32_t incl = lane_sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        const uint32_t before = incl - lane_sum;
        uint32_t np = 0u, nn = 0u;
        const bool mine = before < need && need <= incl;
        if (mine) {
            uint32_t run = before;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (run < need && need <= run + c[j]) {
                    np = prefix | ((uint32_t)(255 - 8 * lane - j) << shift);
                    nn = need - run;
                }
                run += c[j];
            }
        }
        const int src = __ffs(__ballot_sync(0xffffffffu, mine)) - 1;     // exactly one lane holds the bin
        prefix = __shfl_sync(0xffffffffu, np, src);
        need = __shfl_sync(0xffffffffu, nn, src);
    }
    if (lane == 0) { sh[0] = prefix; sh[1] = need; }
}

__global__ void __launch_bounds__(TOPK_THREADS)
grid_hist_kernel(int n, int k, int pass, const float *__restrict__ scores, GridWs ws) {
    __shared__ uint32_t hist[TOPK_WARPS][256];
    const int row = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __shared__ uint32_t sh_state[2];
    const float *s = scores + (size_t)row * n;
    grid_resolve(ws.hist + (size_t)row * 4 * 256, pass, k, sh_state);
    const int shift = 24 - 8 * pass;
    const uint32_t mask = pass == 0 ? 0u : 0xFFFFFFFFu << (32 - 8 * pass);
    for (int i = tid; i < TOPK_WARPS * 256; i += TOPK_THREADS) (&hist[0][0])[i] = 0;
    __syncthreads();
    const uint32_t prefix = sh_state[0];
    const int base = blockIdx.x * GR_KEYS;
    for (int i = base + tid; i < base + GR_KEYS; i += TOPK_THREADS) {      // GR_KEYS is a multiple of the block size
        const bool in = i < n;
        const uint32_t key = in ? score_key(__ldg(s + i)) : 0u;
        const bool live = in && ((key & mask) == prefix);
        const uint32_t bin = (key >> shift) & 255u;
        const uint32_t live_mask = __ballot_sync(0xffffffffu, live);
        if (live) {
            const uint32_t peers = __match_any_sync(live_mask, bin);
            if (lane == __ffs(peers) - 1) hist[warp][bin] += __popc(peers);
        }
        __syncwarp();
    }
    __syncthreads();
    if (tid < 256) {
        uint32_t t = 0;
#pragma unroll 8
        for (int w = 0; w < TOPK_WARPS; ++w) t += hist[w][tid];
        if (t) atomicAdd(ws.hist + ((size_t)row * 4 + pass) * 256 + tid, t);
    }
}

__global__ void __launch_bounds__(TOPK_THREADS)
grid_count_kernel(int n, int k, const float *__restrict__ scores, GridWs ws) {
    __shared__ uint32_t warp_gt[TOPK_WARPS], warp_eq[TOPK_WARPS], sh_state[2];
    const int row = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float *s = scores + (size_t)row * n;
    grid_resolve(ws.hist + (size_t)row * 4 * 256, 4, k, sh_state);
    __syncthreads();
    const uint32_t prefix = sh_state[0];
    const int base = blockIdx.x * GR_KEYS;
    uint32_t gt = 0, eq = 0;
    for (int i = base + tid; i < base + GR_KEYS; i += TOPK_THREADS) {
        const bool in = i < n;
        const uint32_t key = in ? score_key(__ldg(s + i)) : 0u;
        gt += __popc(__ballot_sync(0xffffffffu, in && key > prefix));
        eq += __popc(__ballot_sync(0xffffffffu, in && key == prefix));
    }
    if (lane == 0) { warp_gt[warp] = gt; warp_eq[warp] = eq; }
    __syncthreads();
    if (tid == 0) {
        uint32_t g = 0, e = 0;
        for (int w = 0; w < TOPK_WARPS; ++w) { g += warp_gt[w]; e += warp_eq[w]; }
        uint32_t *c = ws.counts + ((size_t)row * gridDim.x + blockIdx.x) * 2;
        c[0] = g; c[1] = e;
    }
}

__global__ void __launch_bounds__(TOPK_THREADS)
grid_emit_kernel(int n, int k, const float *__restrict__ scores, int32_t *__restrict__ kept, GridWs ws) {
    __shared__ uint32_t warp_gt[TOPK_WARPS], warp_eq[TOPK_WARPS], red_gt[TOPK_WARPS], red_eq[TOPK_WARPS], sh_state[2];
    const int row = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float *s = scores + (size_t)row * n;
    int32_t *out = kept + (size_t)row * k;
    grid_resolve(ws.hist + (size_t)row * 4 * 256, 4, k, sh_state);
    __syncthreads();
    const uint32_t prefix = sh_state[0], need = sh_state[1];
    // keys above / equal to the threshold in the CTAs before this one
    const uint32_t *cnt = ws.counts + (size_t)row * gridDim.x * 2;
    uint32_t g = 0, e = 0;
    for (int b = tid; b < (int)blockIdx.x; b += TOPK_THREADS) { g += cnt[2 * b]; e += cnt[2 * b + 1]; }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) { g += __shfl_xor_sync(0xffffffffu, g, o); e += __shfl_xor_sync(0xffffffffu, e, o); }
    if (lane == 0) { red_gt[warp] = g; red_eq[warp] = e; }
    // each warp owns a contiguous run of this CTA's keys
    constexpr int SEG = GR_KEYS / TOPK_WARPS;       // 512
    const int lo = blockIdx.x * GR_KEYS + warp * SEG;
    uint32_t gt = 0, eq = 0;
    for (int i = lo + lane; i < lo + SEG; i += 32) {
        const bool in = i < n;
        const uint32_t key = in ? score_key(__ldg(s + i)) : 0u;
        gt += __popc(__ballot_sync(0xffffffffu, in && key > prefix));
        eq += __popc(__ballot_sync(0xffffffffu, in && key == prefix));
    }
    if (lane == 0) { warp_gt[warp] = gt; warp_eq[warp] = eq; }
    __syncthreads();
    uint32_t gt_before = 0, eq_before = 0;
    for (int w = 0; w < TOPK_WARPS; ++w) { gt_before += red_gt[w]; eq_before += red_eq[w]; }
    for (int w = 0; w < warp; ++w) { gt_before += warp_gt[w]; eq_before += warp_eq[w]; }
    const uint32_t lt_mask = (1u << lane) - 1u;
    for (int i = lo + lane; i < lo + SEG; i += 32) {
        const bool in = i < n;
        const uint32_t key = in ? score_key(__ldg(s + i)) : 0u;
        const bool is_gt = in && key > prefix, is_eq = in && key == prefix;
        const uint32_t gt_b = __ballot_sync(0xffffffffu, is_gt);
        const uint32_t eq_b = __ballot_sync(0xffffffffu, is_eq);
        const uint32_t eq_rank = eq_before + __popc(eq_b & lt_mask);
        const bool take = is_gt || (is_eq && eq_rank < need);
        const uint32_t take_b = __ballot_sync(0xffffffffu, take);
        if (take) out[gt_before + min(eq_before, need) + __popc(take_b & lt_mask)] = i;
        gt_before += __popc(gt_b);
        eq_before += __popc(eq_b);
    }
}

size_t grid_ws_bytes(int Bz, int n) {
    const size_t nblk = (size_t)ceil_div(n, GR_KEYS);
    return align_up((size_t)Bz * 4 * 256 * 4, 256) + align_up((size_t)Bz * nblk * 2 * 4, 256);
}

}  // namespace

extern "C" size_t str_topk_select_workspace_size(int Bz, int n_vis, int k) {
    (void)k;
    if (Bz <= 0 || n_vis <= CL_MAX_N) return 0;
    return grid_ws_bytes(Bz, n_vis);
}

extern "C" int str_topk_select(str_ctx *ctx, int Bz, int n_vis, int k, const float *scores,
                               int32_t *kept_idx_out, void *workspace, size_t workspace_bytes, void *stream) {
    StrProfScope prof_scope(ctx, STR_CAT_TOPK, stream);
    if (!ctx || Bz <= 0 || n_vis < 0 || k < 0 || k > n_vis) return STR_ERR_INVALID_ARG;
    if (k == 0) return STR_OK;
    if (!scores || !kept_idx_out) return STR_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (n_vis <= CL_MAX_N) {
        // smallest cluster (power of two, at most 8 CTAs) and run length that cover the row
        int ncta = 1;
        while (ncta < CL_MAX_CTAS && ncta * CL_THREADS * 4 < n_vis) ncta *= 2;
        const int per_thread = ceil_div(n_vis, ncta * CL_THREADS);
        cudaError_t e;
        if (per_thread <= 1) e = launch_cluster<1>(ncta, Bz, n_vis, k, scores, kept_idx_out, st);
        else if (per_thread <= 2) e = launch_cluster<2>(ncta, Bz, n_vis, k, scores, kept_idx_out, st);
        else if (per_thread <= 4) e = launch_cluster<4>(ncta, Bz, n_vis, k, scores, kept_idx_out, st);
        else if (per_thread <= 8) e = launch_cluster<8>(ncta, Bz, n_vis, k, scores, kept_idx_out, st);
        else e = launch_cluster<16>(ncta, Bz, n_vis, k, scores, kept_idx_out, st);
        ctx->launches += 1;
        return e == cudaSuccess ? STR_OK : STR_ERR_CUDA;
    }
    if (workspace && workspace_bytes >= grid_ws_bytes(Bz, n_vis) && ((uintptr_t)workspace & 255) == 0) {
        const int nblk = ceil_div(n_vis, GR_KEYS);
        GridWs ws;
        ws.hist = (uint32_t *)workspace;
        ws.counts = (uint32_t *)((char *)workspace + align_up((size_t)Bz * 4 * 256 * 4, 256));
        STR_CUDA_OK(cudaMemsetAsync(ws.hist, 0, (size_t)Bz * 4 * 256 * 4, st));
        for (int pass = 0; pass < 4; ++pass)
            grid_hist_kernel<<<dim3(nblk, Bz), TOPK_THREADS, 0, st>>>(n_vis, k, pass, scores, ws);
        grid_count_kernel<<<dim3(nblk, Bz), TOPK_THREADS, 0, st>>>(n_vis, k, scores, ws);
        grid_emit_kernel<<<dim3(nblk, Bz), TOPK_THREADS, 0, st>>>(n_vis, k, scores, kept_idx_out, ws);
        return str_launch_ok(ctx, 6);
    }
    // no (or too small a) workspace: one CTA per row, every pass re-reads the row
    topk_select_kernel<<<Bz, TOPK_THREADS, 0, st>>>(n_vis, k, scores, kept_idx_out);
    return str_launch_ok(ctx);
}
