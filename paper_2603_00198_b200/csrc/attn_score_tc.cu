// Attention importance (Section 3.1 "Attention Layers") on tcgen05 tensor cores, bf16, head_dim 128:
//   s_i = 1/(M Hq) sum_{m,h} exp(z_mhi - max_i z_mhi) / sum_i' exp(z_mhi' - max_i z_mhi),  z = scale q_m^h . k_i^kv(h)
// with the softmax taken over the n_vis visual keys.  Two kernels:
//   1. row statistics: for every (head, text query) the maximum and the sum of exponentials over the
//      visual keys.  Queries are the M dimension of the product (one thread per query row keeps a
//      running maximum and sum, flash-attention style); the keys stream by as 256-wide N tiles.  The
//      key range is cut into segments so that the grid fills the machine; segments are merged in 2.
//   2. column sums: for every visual key the sum over heads and queries of the normalised weights.
//      Keys are the M dimension (one thread per key); persistent CTAs walk  head (outer) x their key
//      tiles (inner), so a head's text queries are fetched once per CTA; running sums in shared memory.
// Logits are handled in the log2 domain: zl = z * log2(e), weights = exp2(zl - maxl).
// Warps (both kernels): 0-7 CUDA-core part (warp w owns TMEM lanes 32 (w % 4).. and the column half w / 4 of
// the accumulator), 8 TMA producer, 9 MMA issuer.
// Every mbarrier wait is bounded; a give-up records STR_ERR_TIMEOUT and the CTA tears down.
#include <float.h>

#include "dispatch.cuh"
#include "tc_common.cuh"

namespace {

constexpr int HD = 128;
constexpr int TILE_16K = 16384;
constexpr int NUM_THREADS = 320;          // 8 CUDA-core warps (two per TMEM lane quadrant, half the columns each) + producer + MMA issuer
constexpr float NEG_BIG = -1.0e30f;

// ---------------------------------------------------------------------------------------------------
// Kernel 1: row statistics.  grid = (segments, Hq * m_tiles, Bz)
namespace rs {
constexpr int BN = 256;                                  // keys per step
constexpr int K_BYTES = BN * HD * 2;                     // 64 KB: two 64-column halves of 256 rows
constexpr int OFF_Q = 0, OFF_K = 2 * TILE_16K, STAGES = 2;
constexpr int OFF_BARS = OFF_K + STAGES * K_BYTES;
enum { B_Q = 0, B_FULL0, B_FULL1, B_EMPTY0, B_EMPTY1, B_ACCF0, B_ACCF1, B_ACCE0, B_ACCE1, B_COUNT };
constexpr size_t SMEM_BYTES = (size_t)OFF_BARS + B_COUNT * 8 + 32;
}  // namespace rs

__global__ void __launch_bounds__(NUM_THREADS, 1)
attn_rowstats_tc_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k, int Hq,
                        int Hkv, int n_vis, int n_text, int m_tiles, float scale_log2, float *__restrict__ ws_max,
                        float *__restrict__ ws_sum, int *status) {
    using namespace rs;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t *bars = (uint64_t *)(smem + OFF_BARS);
    uint32_t *tmem_slot = (uint32_t *)(bars + B_COUNT);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int seg = blockIdx.x, nseg = gridDim.x;
    const int h = blockIdx.y / m_tiles, mt = blockIdx.y % m_tiles, b = blockIdx.z;
    const int kv = h / (Hq / Hkv);
    const int ktiles = (n_vis + BN - 1) / BN;
    const int j_beg = (int)((long long)ktiles * seg / nseg), j_end = (int)((long long)ktiles * (seg + 1) / nseg);

    if ((tc::smem_u32(smem) & 1023u) != 0) {
        if (threadIdx.x == 0) atomicCAS(status, 0, STR_ERR_CUDA);
        return;
    }
    if (tc::cta_should_leave(status)) return;     // an earlier CTA failed: the whole CTA leaves at once
    if (threadIdx.x == 0) {
        tc::mbar_init(bars + B_Q, 1);
        for (int s = 0; s < 2; ++s) {
            tc::mbar_init(bars + B_FULL0 + s, 1); tc::mbar_init(bars + B_EMPTY0 + s, 1);
            tc::mbar_init(bars + B_ACCF0 + s, 1); tc::mbar_init(bars + B_ACCE0 + s, 8);
        }
        abort_flag[0] = 0; abort_flag[1] = 0;
        tc::fence_mbar_init();
        tc::prefetch_tmap(&tmap_q); tc::prefetch_tmap(&tmap_k);
    }
    if (warp == 9) { tc::tmem_alloc(tmem_slot, 512); tc::tmem_relinquish(); }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 8) {
        if (lane == 0) {
            bool ok = true;
            tc::mbar_arrive_expect_tx(bars + B_Q, 2 * TILE_16K);
            tc::tma_load_3d(smem + OFF_Q, &tmap_q, bars + B_Q, h * HD, n_vis + mt * 128, b);
            tc::tma_load_3d(smem + OFF_Q + TILE_16K, &tmap_q, bars + B_Q, h * HD + 64, n_vis + mt * 128, b);
            int it = 0;
            for (int j = j_beg; j < j_end; ++j, ++it) {
                const int s = it & 1;
                if (!tc::mbar_wait(bars + B_EMPTY0 + s, ((it >> 1) & 1) ^ 1, abort_flag)) { ok = false; break; }
                uint64_t *fb = bars + B_FULL0 + s;
                uint8_t *kt = smem + OFF_K + s * K_BYTES;
                tc::mbar_arrive_expect_tx(fb, K_BYTES);
                tc::tma_load_3d(kt, &tmap_k, fb, kv * HD, j * BN, b);
                tc::tma_load_3d(kt + K_BYTES / 2, &tmap_k, fb, kv * HD + 64, j * BN, b);
            }
            if (!ok) {
                atomicCAS(status, 0, STR_ERR_TIMEOUT);
                tc::mbar_wait(bars + B_Q, 0, abort_flag + 1);           // let copies already issued land
                for (int back = 1; back <= 2 && back <= it; ++back) {
                    const int q = it - back;
                    tc::mbar_wait(bars + B_FULL0 + (q & 1), (q >> 1) & 1, abort_flag + 1);
                }
            }
        }
    } else if (warp == 9) {
        const uint32_t idesc = tc::make_idesc_bf16(128, BN, 0, 0);
        const uint32_t sbase = tc::smem_u32(smem);
        bool ok = __all_sync(0xffffffffu, tc::mbar_wait(bars + B_Q, 0, abort_flag));
        int it = 0;
        for (int j = j_beg; j < j_end && ok; ++j, ++it) {
            const int s = it & 1;
            ok = __all_sync(0xffffffffu, tc::mbar_wait(bars + B_ACCE0 + s, ((it >> 1) & 1) ^ 1, abort_flag) &&
                                             tc::mbar_wait(bars + B_FULL0 + s, (it >> 1) & 1, abort_flag));
            if (!ok) break;
            tc::tc_fence_after();
            const uint32_t kt = sbase + OFF_K + (uint32_t)(s * K_BYTES);
            if (tc::elect_one()) {
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    tc::mma_ss(tmem + (uint32_t)s * BN, tc::desc_kmajor_sw128(sbase + OFF_Q + (ks >> 2) * TILE_16K, (ks & 3) * 16),
                               tc::desc_kmajor_sw128(kt + (ks >> 2) * (K_BYTES / 2), (ks & 3) * 16), idesc, ks != 0);
                tc::mma_commit(bars + B_EMPTY0 + s);
                tc::mma_commit(bars + B_ACCF0 + s);
            }
            __syncwarp();
        }
        if (!ok && lane == 0) atomicCAS(status, 0, STR_ERR_TIMEOUT);
    } else {
        const int quad = warp & 3, half = warp >> 2;                // TMEM lane quadrant, column half (128 keys of the 256)
        const int row = quad * 32 + lane, m = mt * 128 + row;       // text query index
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        float mx = NEG_BIG, sum = 0.f;                              // running maximum (log2 domain) and sum
        bool ok = true;
        int it = 0;
        for (int j = j_beg; j < j_end; ++j, ++it) {
            const int s = it & 1;
            if (!tc::mbar_wait(bars + B_ACCF0 + s, (it >> 1) & 1, abort_flag)) { ok = false; break; }
            tc::tc_fence_after();
            const int key0 = j * BN;
#pragma unroll 1
            for (int c = half * (BN / 2); c < (half + 1) * (BN / 2); c += 32) {
                if (key0 + c >= n_vis) break;                       // whole chunk beyond the visual keys
                uint32_t v[32];
                tc::tmem_ld32(tmem + lane_base + (uint32_t)(s * BN + c), v);
                tc::tmem_ld_wait();
                float z[32];
                float cmax = NEG_BIG;
                const bool ragged = key0 + c + 32 > n_vis;
#pragma unroll
                for (int e = 0; e < 32; ++e) {
                    z[e] = __uint_as_float(v[e]) * scale_log2;
                    if (ragged && key0 + c + e >= n_vis) z[e] = NEG_BIG;
                    cmax = fmaxf(cmax, z[e]);
                }
                const float nm = fmaxf(mx, cmax);
                sum *= tc::ex2(mx - nm);
                float a0 = 0.f, a1 = 0.f;
#pragma unroll
                for (int e = 0; e < 32; e += 2) { a0 += tc::ex2(z[e] - nm); a1 += tc::ex2(z[e + 1] - nm); }
                sum += a0 + a1;
                mx = nm;
            }
            tc::tc_fence_before();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(bars + B_ACCE0 + s);
        }
        if (ok) {
            if (m < n_text) {
                // the two column halves are stored as two segments of their own
                const size_t o = (((size_t)b * Hq + h) * (2 * nseg) + 2 * seg + half) * n_text + m;
                ws_max[o] = mx;
                ws_sum[o] = sum;
            }
        } else if (lane == 0) {
            atomicCAS(status, 0, STR_ERR_TIMEOUT);
        }
    }
    tc::tc_fence_before();
    __syncthreads();
    if (warp == 9) { tc::tc_fence_after(); tc::tmem_dealloc(tmem, 512); }
}

// ---------------------------------------------------------------------------------------------------
// Between the two: merge the key segments into one (max, 1/sum) per (sequence, head, text query).
__global__ void __launch_bounds__(256)
attn_merge_stats_kernel(int rows, int n_text, int nseg, const float *__restrict__ ws_max, const float *__restrict__ ws_sum,
                        float *__restrict__ mg_max, float *__restrict__ mg_inv) {
    const int r = blockIdx.x * blockDim.x + threadIdx.x;          // r = (b * Hq + h) * n_text + m
    if (r >= rows) return;
    const int bh = r / n_text, m = r - bh * n_text;
    const size_t o = (size_t)bh * nseg * n_text + m;
    float M_ = NEG_BIG;
    for (int sg = 0; sg < nseg; ++sg) M_ = fmaxf(M_, ws_max[o + (size_t)sg * n_text]);
    float S_ = 0.f;
    for (int sg = 0; sg < nseg; ++sg) S_ += ws_sum[o + (size_t)sg * n_text] * tc::ex2(ws_max[o + (size_t)sg * n_text] - M_);
    mg_max[r] = M_;
    mg_inv[r] = 1.0f / S_;
}

// ---------------------------------------------------------------------------------------------------
// Kernel 2: column sums.  grid = (CTAs per sequence, Bz); CTA x owns key tiles x, x + gridDim.x, ...
namespace cs {
constexpr int TI = 128;
constexpr int K_TILE = 32768;                // 128 keys x 128 bf16, two 64-column halves
constexpr int MAX_STAGES = 4, MAX_ITEMS = 8, MAX_TEXT = 256;
enum { B_FULL0 = 0, B_EMPTY0 = MAX_STAGES, B_QF0 = 2 * MAX_STAGES, B_QE0 = B_QF0 + 2, B_ACCF0 = B_QE0 + 2, B_ACCE0 = B_ACCF0 + 2,
       B_PAIR0 = B_ACCE0 + 2, B_COUNT = B_PAIR0 + 4 };
}  // namespace cs

__global__ void __launch_bounds__(NUM_THREADS, 1)
attn_colsum_tc_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_q, int Hq, int Hkv,
                      int n_vis, int n_text, int n_pad, int stages, float scale_log2,
                      const float *__restrict__ mg_max, const float *__restrict__ mg_inv, float *__restrict__ scores,
                      int *status) {
    using namespace cs;
    extern __shared__ __align__(1024) uint8_t smem[];
    const int q_bytes = n_pad * 256;                         // text tile: n_pad rows x 128 bf16
    uint8_t *q_smem = smem + stages * K_TILE;
    float *totals = (float *)(q_smem + 2 * q_bytes);          // [column half][MAX_ITEMS][128] running sums of this CTA's tiles
    float *stats = totals + 2 * MAX_ITEMS * TI;               // [8 warps][max | 1/sum][MAX_TEXT / 2], one private copy per warp
    uint64_t *bars = (uint64_t *)(stats + 8 * MAX_TEXT);
    uint32_t *tmem_slot = (uint32_t *)(bars + B_COUNT);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = blockIdx.y;
    const int tiles = (n_vis + TI - 1) / TI;
    const int my_tiles = (tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    const int qpk = Hq / Hkv;
    const uint32_t acc_cols = n_pad <= 128 ? 128u : 256u;

    if ((tc::smem_u32(smem) & 1023u) != 0) {
        if (threadIdx.x == 0) atomicCAS(status, 0, STR_ERR_CUDA);
        return;
    }
    if (tc::cta_should_leave(status)) return;     // an earlier CTA failed: the whole CTA leaves at once
    if (threadIdx.x == 0) {
        for (int s = 0; s < MAX_STAGES; ++s) { tc::mbar_init(bars + B_FULL0 + s, 1); tc::mbar_init(bars + B_EMPTY0 + s, 1); }
        for (int s = 0; s < 2; ++s) {
            tc::mbar_init(bars + B_QF0 + s, 1); tc::mbar_init(bars + B_QE0 + s, 1);
            tc::mbar_init(bars + B_ACCF0 + s, 1); tc::mbar_init(bars + B_ACCE0 + s, 8);
        }
        for (int w = 0; w < 4; ++w) tc::mbar_init(bars + B_PAIR0 + w, 1);
        abort_flag[0] = 0; abort_flag[1] = 0;
        tc::fence_mbar_init();
        tc::prefetch_tmap(&tmap_k); tc::prefetch_tmap(&tmap_q);
    }
    if (warp == 9) { tc::tmem_alloc(tmem_slot, 2 * acc_cols); tc::tmem_relinquish(); }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    // All roles walk the same sequence: rounds of up to MAX_ITEMS tiles; inside a round, head h (outer) and
    // tile k (inner).  `it` counts (head, tile) steps and `cg` counts (round, head) steps across the kernel.
    if (warp == 8) {
        if (lane == 0) {
            bool ok = true;
            int it = 0, cg = 0, q_issued = 0;
            for (int r0 = 0; r0 < my_tiles && ok; r0 += MAX_ITEMS) {
                const int kr = min(MAX_ITEMS, my_tiles - r0);
                for (int h = 0; h < Hq && ok; ++h, ++cg) {
                    const int qs = cg & 1, kv = h / qpk;
                    if (!tc::mbar_wait(bars + B_QE0 + qs, ((cg >> 1) & 1) ^ 1, abort_flag)) { ok = false; break; }
                    tc::mbar_arrive_expect_tx(bars + B_QF0 + qs, (uint32_t)q_bytes);
                    tc::tma_load_3d(q_smem + qs * q_bytes, &tmap_q, bars + B_QF0 + qs, h * HD, n_vis, b);
                    tc::tma_load_3d(q_smem + qs * q_bytes + n_pad * 128, &tmap_q, bars + B_QF0 + qs, h * HD + 64, n_vis, b);
                    ++q_issued;
                    for (int k = 0; k < kr; ++k, ++it) {
                        const int s = it % stages;
                        if (!tc::mbar_wait(bars + B_EMPTY0 + s, ((it / stages) & 1) ^ 1, abort_flag)) { ok = false; break; }
                        const int i0 = ((int)blockIdx.x + (r0 + k) * (int)gridDim.x) * TI;
                        uint64_t *fb = bars + B_FULL0 + s;
                        tc::mbar_arrive_expect_tx(fb, K_TILE);
                        tc::tma_load_3d(smem + s * K_TILE, &tmap_k, fb, kv * HD, i0, b);
                        tc::tma_load_3d(smem + s * K_TILE + K_TILE / 2, &tmap_k, fb, kv * HD + 64, i0, b);
                    }
                }
            }
            if (!ok) {
                atomicCAS(status, 0, STR_ERR_TIMEOUT);
                for (int back = 1; back <= stages && back <= it; ++back) {        // let copies already issued land
                    const int j = it - back;
                    tc::mbar_wait(bars + B_FULL0 + j % stages, (j / stages) & 1, abort_flag + 1);
                }
                for (int back = 1; back <= 2 && back <= q_issued; ++back) {
                    const int j = q_issued - back;
                    tc::mbar_wait(bars + B_QF0 + (j & 1), (j >> 1) & 1, abort_flag + 1);
                }
            }
        }
    } else if (warp == 9) {
        const uint32_t idesc = tc::make_idesc_bf16(TI, n_pad, 0, 0);
        const uint32_t sbase = tc::smem_u32(smem), qbase = tc::smem_u32(q_smem);
        bool ok = true;
        int it = 0, cg = 0;
        for (int r0 = 0; r0 < my_tiles && ok; r0 += MAX_ITEMS) {
            const int kr = min(MAX_ITEMS, my_tiles - r0);
            for (int h = 0; h < Hq && ok; ++h, ++cg) {
                const int qs = cg & 1;
                ok = __all_sync(0xffffffffu, tc::mbar_wait(bars + B_QF0 + qs, (cg >> 1) & 1, abort_flag));
                const uint32_t qt = qbase + (uint32_t)(qs * q_bytes);
                for (int k = 0; k < kr && ok; ++k, ++it) {
                    const int s = it & 1, sl = it % stages;           // accumulator buffer, operand slot
                    ok = __all_sync(0xffffffffu, tc::mbar_wait(bars + B_ACCE0 + s, ((it >> 1) & 1) ^ 1, abort_flag) &&
                                                     tc::mbar_wait(bars + B_FULL0 + sl, (it / stages) & 1, abort_flag));
                    if (!ok) break;
                    tc::tc_fence_after();
                    const uint32_t kt = sbase + (uint32_t)(sl * K_TILE);
                    if (tc::elect_one()) {
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks)
                            tc::mma_ss(tmem + (uint32_t)s * acc_cols, tc::desc_kmajor_sw128(kt + (ks >> 2) * (K_TILE / 2), (ks & 3) * 16),
                                       tc::desc_kmajor_sw128(qt + (uint32_t)((ks >> 2) * n_pad * 128), (ks & 3) * 16), idesc, ks != 0);
                        tc::mma_commit(bars + B_EMPTY0 + sl);
                        tc::mma_commit(bars + B_ACCF0 + s);
                        if (k == kr - 1) tc::mma_commit(bars + B_QE0 + qs);     // last product that reads this Q buffer
                    }
                    __syncwarp();
                }
            }
        }
        if (!ok && lane == 0) atomicCAS(status, 0, STR_ERR_TIMEOUT);
    } else {
        const int quad = warp & 3, half = warp >> 2;                  // TMEM lane quadrant, column half
        const int row = quad * 32 + lane;
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        const int c_mid = ((n_pad / 2 + 15) / 16) * 16;                // both halves are multiples of 16 columns
        const int c_beg = half ? c_mid : 0, c_end = half ? n_pad : c_mid;
        float *tot = totals + half * MAX_ITEMS * TI;
        // (max, 1/sum) of the text queries of this warp's column half: a private copy per warp in shared memory
        // (no warp waits for another here), the next head's values fetched into registers a head ahead
        float *st_mx = stats + warp * MAX_TEXT, *st_inv = st_mx + MAX_TEXT / 2;
        bool ok = true;
        int it = 0, cg = 0, round = 0;
        for (int r0 = 0; r0 < my_tiles && ok; r0 += MAX_ITEMS, ++round) {
            const int kr = min(MAX_ITEMS, my_tiles - r0);
            for (int k = 0; k < kr; ++k) tot[k * TI + row] = 0.f;         // each thread only touches its own entries
            float nmx[MAX_TEXT / 64], ninv[MAX_TEXT / 64];
            auto fetch_stats = [&](int h) {
#pragma unroll
                for (int u = 0; u < MAX_TEXT / 64; ++u) {
                    const int m = c_beg + lane + 32 * u;
                    const bool in = m < n_text && m < c_end;               // padded rows contribute exp2(0 - 0) * 0
                    const size_t o = ((size_t)b * Hq + h) * n_text + m;
                    nmx[u] = in ? __ldg(mg_max + o) : 0.f;
                    ninv[u] = in ? __ldg(mg_inv + o) : 0.f;
                }
            };
            fetch_stats(0);
            for (int h = 0; h < Hq && ok; ++h, ++cg) {
                __syncwarp();
#pragma unroll
                for (int u = 0; u < MAX_TEXT / 64; ++u) { st_mx[lane + 32 * u] = nmx[u]; st_inv[lane + 32 * u] = ninv[u]; }
                __syncwarp();
                if (h + 1 < Hq) fetch_stats(h + 1);
#pragma unroll 1
                for (int k = 0; k < kr; ++k, ++it) {
                    const int s = it & 1;
                    if (!tc::mbar_wait(bars + B_ACCF0 + s, (it >> 1) & 1, abort_flag)) { ok = false; break; }
                    tc::tc_fence_after();
                    float a0 = 0.f, a1 = 0.f;
#pragma unroll 1
                    for (int c = c_beg; c < c_end; c += 32) {
                        uint32_t v[32];
                        tc::tmem_ld32(tmem + lane_base + (uint32_t)s * acc_cols + (uint32_t)c, v);
                        tc::tmem_ld_wait();
                        const int lim = (c + 32 <= c_end) ? 32 : 16;
#pragma unroll
                        for (int e = 0; e < 32; e += 4) {
                            if (e < lim) {
                                const float4 mx4 = *(const float4 *)(st_mx + (c - c_beg) + e), in4 = *(const float4 *)(st_inv + (c - c_beg) + e);
                                a0 = fmaf(tc::ex2(fmaf(__uint_as_float(v[e]), scale_log2, -mx4.x)), in4.x, a0);
                                a1 = fmaf(tc::ex2(fmaf(__uint_as_float(v[e + 1]), scale_log2, -mx4.y)), in4.y, a1);
                                a0 = fmaf(tc::ex2(fmaf(__uint_as_float(v[e + 2]), scale_log2, -mx4.z)), in4.z, a0);
                                a1 = fmaf(tc::ex2(fmaf(__uint_as_float(v[e + 3]), scale_log2, -mx4.w)), in4.w, a1);
                            }
                        }
                    }
                    tc::tc_fence_before();
                    __syncwarp();
                    if (lane == 0) tc::mbar_arrive(bars + B_ACCE0 + s);
                    tot[k * TI + row] += a0 + a1;
                }
            }
            // the upper-half warp hands its sums to its lower-half partner (bounded wait), which writes the scores
            if (half == 1) {
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(bars + B_PAIR0 + quad);       // release: the sums above are visible
            } else if (ok) {
                ok = tc::mbar_wait(bars + B_PAIR0 + quad, round & 1, abort_flag);
                if (ok) {
                    const float *hi = totals + MAX_ITEMS * TI;
                    for (int k = 0; k < kr; ++k) {
                        const int i = ((int)blockIdx.x + (r0 + k) * (int)gridDim.x) * TI + row;
                        if (i < n_vis) scores[(size_t)b * n_vis + i] = (tot[k * TI + row] + hi[k * TI + row]) / ((float)n_text * (float)Hq);
                    }
                }
            }
        }
        if (!ok && lane == 0) atomicCAS(status, 0, STR_ERR_TIMEOUT);
    }
    tc::tc_fence_before();
    __syncthreads();
    if (warp == 9) { tc::tc_fence_after(); tc::tmem_dealloc(tmem, 2 * acc_cols); }
}

}  // namespace

// Number of key segments of kernel 1: enough CTAs to fill the machine, never more than STR_ATTN_SCORE_MAX_SEGMENTS.
static int attn_score_segments(const str_ctx *ctx, const str_attn_score_shape *s, int n_vis, int n_text) {
    const int m_tiles = (n_text + 127) / 128;
    const int ktiles = (n_vis + rs::BN - 1) / rs::BN;
    int seg = ctx->sm_count / (s->Bz * s->Hq * m_tiles);          // a single wave of CTAs
    if (2 * seg > STR_ATTN_SCORE_MAX_SEGMENTS) seg = STR_ATTN_SCORE_MAX_SEGMENTS / 2;    // each segment stores two column halves
    if (seg > ktiles) seg = ktiles;
    return seg < 1 ? 1 : seg;
}

bool str_attn_importance_tc_supported(const str_attn_score_shape *s, int n_vis, int n_text, const void *q, const void *k) {
    if (s->dtype != STR_BF16 || s->d != HD || n_text < 1 || n_text > cs::MAX_TEXT || n_vis < 1) return false;
    return (((uintptr_t)q | (uintptr_t)k) & 15) == 0;
}

int str_attn_importance_tc(str_ctx *ctx, const str_attn_score_shape *s, int n_vis, int n_text, const void *q, const void *k,
                           float scale, float *scores, float *workspace, bool causal_row, cudaStream_t st) {
    const int n_pad = (n_text + 15) / 16 * 16, m_tiles = (n_text + 127) / 128;
    const int nseg = attn_score_segments(ctx, s, n_vis, n_text);
    const size_t rows = (size_t)s->Bz * s->Hq * n_text;
    const int nstore = 2 * nseg;                                  // stored segments: two column halves per key segment
    float *ws_max = workspace, *ws_sum = ws_max + rows * nstore, *mg_max = ws_sum + rows * nstore, *mg_inv = mg_max + rows;
    const float scale_log2 = scale * 1.4426950408889634f;
    CUtensorMap tq128, tk256, tk128, tqpad;
    int rc = str_make_tmap_3d_bf16_sw128(ctx, &tq128, q, (uint64_t)s->Hq * HD, (uint64_t)s->T, (uint64_t)s->Bz, 128);
    if (rc == STR_OK) rc = str_make_tmap_3d_bf16_sw128(ctx, &tk256, k, (uint64_t)s->Hkv * HD, (uint64_t)s->T, (uint64_t)s->Bz, rs::BN);
    if (rc == STR_OK) rc = str_make_tmap_3d_bf16_sw128(ctx, &tk128, k, (uint64_t)s->Hkv * HD, (uint64_t)s->T, (uint64_t)s->Bz, cs::TI);
    if (rc == STR_OK) rc = str_make_tmap_3d_bf16_sw128(ctx, &tqpad, q, (uint64_t)s->Hq * HD, (uint64_t)s->T, (uint64_t)s->Bz, (uint32_t)n_pad);
    if (rc != STR_OK) return rc;
    const size_t fixed2 = 2 * (size_t)n_pad * 256 + 2 * (size_t)cs::MAX_ITEMS * cs::TI * 4 + 8 * cs::MAX_TEXT * 4 + cs::B_COUNT * 8 + 32;
    int stages = cs::MAX_STAGES;
    while (stages > 2 && fixed2 + (size_t)stages * cs::K_TILE > (size_t)ctx->max_smem_optin) --stages;
    const size_t smem2 = fixed2 + (size_t)stages * cs::K_TILE;
    if (smem2 > (size_t)ctx->max_smem_optin || rs::SMEM_BYTES > (size_t)ctx->max_smem_optin) return STR_ERR_UNSUPPORTED_SHAPE;
    rc = str_ensure_smem(ctx, STR_SMEM_ATTN_ROWSTATS, attn_rowstats_tc_kernel, rs::SMEM_BYTES);
    if (rc == STR_OK) rc = str_ensure_smem(ctx, STR_SMEM_ATTN_COLSUM, attn_colsum_tc_kernel, smem2);
    if (rc != STR_OK) return rc;
    dim3 g1(nseg, s->Hq * m_tiles, s->Bz);
    attn_rowstats_tc_kernel<<<g1, NUM_THREADS, rs::SMEM_BYTES, st>>>(tq128, tk256, s->Hq, s->Hkv, n_vis, n_text, m_tiles, scale_log2,
                                                                      ws_max, ws_sum, ctx->status_dev);
    attn_merge_stats_kernel<<<(unsigned)((rows + 255) / 256), 256, 0, st>>>((int)rows, n_text, nstore, ws_max, ws_sum, mg_max, mg_inv);
    rc = str_launch_ok(ctx, 2);
    if (rc == STR_OK && causal_row)
        rc = str_attn_text_keys_stats(ctx, s, n_vis, n_text, q, k, scale, true, mg_max, mg_inv, st);
    if (rc != STR_OK) return rc;
    const int tiles = ceil_div(n_vis, cs::TI);
    const int per_seq = ceil_div(ctx->sm_count, s->Bz);
    dim3 g2(tiles < per_seq ? tiles : per_seq, s->Bz);
    attn_colsum_tc_kernel<<<g2, NUM_THREADS, smem2, st>>>(tk128, tqpad, s->Hq, s->Hkv, n_vis, n_text, n_pad, stages, scale_log2,
                                                         mg_max, mg_inv, scores, ctx->status_dev);
    return str_launch_ok(ctx);
}
