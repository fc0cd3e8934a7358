// bf16 GEMM on the 5th-generation tensor cores: out[M,N] = a[M,K] * w[N,K]^T (+ residual).
//
// Two persistent, warp-specialised kernels with the same roles and the same epilogue function.  gemm_tc_pair_kernel
// (further down) runs one 256 x 256 tile per cluster of two CTAs and is the one used above 128 rows; gemm_tc_kernel
// runs one 128 x 256 tile per CTA:
//   warp 0     TMA producer: streams 128x64 A tiles and 256x64 W tiles (128-byte swizzle) through a
//              4-stage shared-memory ring guarded by full/empty mbarriers.
//   warp 1     MMA issuer: one thread issues tcgen05.mma (M=128, N=256, K=16) into one of two
//              256-column fp32 accumulators in tensor memory; tcgen05.commit frees smem stages and
//              publishes finished accumulators.
//   warps 2-5  epilogue: tcgen05.ld the accumulator (each warp its own 32-lane quadrant), add the
//              residual, narrow to bf16, 16-byte stores.  Runs concurrently with the next tile's
//              main loop thanks to the double-buffered accumulator.
//   warps 6-9  second epilogue group, used by the fused pre-scan epilogue only (it does several times the
//              work per element and would otherwise outlast the main loop): warps w and w + 4 share a
//              lane quadrant and take 128 of the tile's 256 columns each.
// Tiles are walked in bands of 8 column tiles so that a band of W stays in L2 while A streams.
// The epilogue can fuse the RMSNorm that surrounds the projections of a pre-norm block: it scales the accumulator
// row by 1/rms of the A row (from partial sums of squares left by the kernel that wrote A), and it leaves the
// partial sums of squares of its own output rows, one per 256-column tile, for the next projection.  For a Mamba
// in-projection it can run the block's pre-scan step (conv, SiLU, split, softplus) instead of storing the projection.
// Every mbarrier wait is bounded; on give-up the kernel records STR_ERR_TIMEOUT and tears down.
#include <stdlib.h>

#include "dispatch.cuh"
#include "tc_common.cuh"

namespace {

constexpr int BM = 128, BN = 256, BK = 64, STAGES = 4, UMMA_K = 16;
constexpr int A_BYTES = BM * BK * 2, W_BYTES = BN * BK * 2, STAGE_BYTES = A_BYTES + W_BYTES;
constexpr int NUM_THREADS = 320;            // 10 warps
constexpr int BAND = 8;                     // column tiles per L2 band
constexpr size_t SMEM_BYTES = 1024 /*align slack*/ + (size_t)STAGES * STAGE_BYTES + 256;

struct TileCoord { int m, n; };
__device__ __forceinline__ TileCoord tile_coord(int t, int tiles_m, int tiles_n) {
    const int per_band = BAND * tiles_m;
    const int band = t / per_band, r = t % per_band;
    const int n0 = band * BAND;
    const int width = min(BAND, tiles_n - n0);
    return {r / width, n0 + r % width};
}

// Fused pre-scan epilogue (StrConvEpilogue): 32 columns (first column `col`, a multiple of 32, so all in one of the
// segments z | x | B | C | dt) of an in-projection row.  The whole warp calls this together, because the conv reads
// the three lanes below through shuffles.  `raw_dst` is where the unfused GEMM would store the 32 values.  One
// tensor-memory load per 32 columns and everything of those columns unrolled: measured, the same work cut into
// 8-column steps with their own tensor-memory loads (rolled or software-pipelined) slowed the main loop three times
// as much.
__device__ __forceinline__ float bf16_half(uint32_t word, int e) {
    return e ? __uint_as_float(word & 0xFFFF0000u) : __uint_as_float(word << 16);
}
__device__ __forceinline__ void prescan_columns(const uint32_t (&v)[32], float scale, int lane, bool row_ok, int t_in, int grow,
                                                int col, __nv_bfloat16 *__restrict__ raw_dst, const StrConvEpilogue &cv) {
    const int seg = col - cv.zoff, conv_dim = cv.d_inner + 2 * cv.gn;
    uint32_t rw[16];                                             // the projection as the unfused GEMM stores it
#pragma unroll
    for (int q = 0; q < 16; ++q) rw[q] = tc::pack_bf16x2(__uint_as_float(v[2 * q]) * scale, __uint_as_float(v[2 * q + 1]) * scale);
    if (seg < 0) {                                               // gate columns: stored as they are
        if (row_ok) {
#pragma unroll
            for (int g = 0; g < 4; ++g)
                *reinterpret_cast<uint4 *>(raw_dst + g * 8) = make_uint4(rw[4 * g], rw[4 * g + 1], rw[4 * g + 2], rw[4 * g + 3]);
        }
        return;
    }
    if (seg >= conv_dim) {                                       // dt columns: softplus(dt + bias), fp32
        const int h0 = seg - conv_dim, valid = min(32, cv.H - h0);
        float *dst = cv.dt_out + (size_t)grow * cv.H + h0;
#pragma unroll
        for (int g = 0; g < 8; ++g) {
            if (g * 4 < valid && row_ok) {
                float o[4];
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    o[j] = softplus_f(bf16_half(rw[2 * g + (j >> 1)], j & 1) + __ldg(cv.dt_bias + h0 + g * 4 + j));
                *reinterpret_cast<float4 *>(dst + g * 4) = make_float4(o[0], o[1], o[2], o[3]);
            }
        }
        return;
    }
    __nv_bfloat16 *dst;
    if (seg < cv.d_inner) dst = cv.x_out + (size_t)grow * cv.d_inner + seg;
    else if (seg < cv.d_inner + cv.gn) dst = cv.B_out + (size_t)grow * cv.gn + (seg - cv.d_inner);
    else dst = cv.C_out + (size_t)grow * cv.gn + (seg - cv.d_inner - cv.gn);
    const bool keep_raw = row_ok && (lane < 3 || lane >= 29);     // rows the edge-row kernel reads keep the projection
    const bool own = row_ok && lane >= 3;                        // rows whose three predecessors are in this warp
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        if (keep_raw) *reinterpret_cast<uint4 *>(raw_dst + g * 8) = make_uint4(rw[4 * g], rw[4 * g + 1], rw[4 * g + 2], rw[4 * g + 3]);
        float o[8];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            // the three earlier rows' values of this channel pair, as packed bf16 words from the lanes below; zero
            // where the sequence starts (no earlier tokens)
            const uint32_t cur = rw[4 * g + q];
            uint32_t w1 = __shfl_up_sync(0xffffffffu, cur, 1), w2 = __shfl_up_sync(0xffffffffu, cur, 2),
                     w3 = __shfl_up_sync(0xffffffffu, cur, 3);
            if (t_in < 1) w1 = 0u;
            if (t_in < 2) w2 = 0u;
            if (t_in < 3) w3 = 0u;
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int ch = seg + g * 8 + 2 * q + e;
                const float4 w = __ldg(reinterpret_cast<const float4 *>(cv.conv_w) + ch);
                float acc = __ldg(cv.conv_b + ch);
                acc = fmaf(w.x, bf16_half(w3, e), acc);
                acc = fmaf(w.y, bf16_half(w2, e), acc);
                acc = fmaf(w.z, bf16_half(w1, e), acc);
                acc = fmaf(w.w, bf16_half(cur, e), acc);
                o[2 * q + e] = silu_fast(acc);
            }
        }
        if (own) {
            uint4 ov;
            ov.x = tc::pack_bf16x2(o[0], o[1]);
            ov.y = tc::pack_bf16x2(o[2], o[3]);
            ov.z = tc::pack_bf16x2(o[4], o[5]);
            ov.w = tc::pack_bf16x2(o[6], o[7]);
            *reinterpret_cast<uint4 *>(dst + g * 8) = ov;
        }
    }
}

// Epilogue of one accumulator row: this thread owns tensor-memory lane `taddr`'s lane field = output row `row`, columns
// [256 tile_n, 256 tile_n + 256).  Fused RMSNorm of the A rows: 1/rms from the partial sums of squares the producer
// of A left behind, summed in index order (deterministic), applied to the accumulator row; then the residual, the
// narrowing to bf16, 16-byte stores, and the partial sum of squares of the stored values in column order.
__device__ __forceinline__ void store_rows(uint32_t taddr, int row, int tile_n, int tiles_n, int M, int N,
                                           const __nv_bfloat16 *__restrict__ residual, __nv_bfloat16 *__restrict__ out,
                                           const StrRowNorm &rn, const StrConvEpilogue &cv, int c_begin, int c_end) {
    const int col0 = tile_n * BN;
    const int lane = threadIdx.x & 31;
    const int grow = cv.row_base + row;                      // row among all sequences' rows
    const int t_in = cv.T ? grow % cv.T : 0;                 // position in its sequence
    float scale = 1.0f;
    if (rn.ss_in && row < M) {
        float t = 0.f;
        for (int j = 0; j < rn.nt_in; ++j) t += __ldg(rn.ss_in + (size_t)row * rn.nt_in + j);
        scale = rsqrtf(t * rn.inv_dim + rn.eps);
    }
    float ss = 0.f;                              // sum of squares of this row's stored outputs in this tile
#pragma unroll 1
    for (int c = c_begin; c < c_end; c += 32) {
        uint32_t v[32];
        tc::tmem_ld32(taddr + c, v);
        tc::tmem_ld_wait();
        if (cv.T != 0) {
            // fused pre-scan step; the whole warp stays together (the conv reads the lanes below)
            if (col0 + c < N)
                prescan_columns(v, scale, lane, row < M, t_in, grow, col0 + c, out + (size_t)row * N + col0 + c, cv);
            continue;
        }
        if (row < M && col0 + c < N) {
            const size_t off = (size_t)row * N + col0 + c;
            const int valid = min(32, N - (col0 + c));       // multiple of 8 (N % 8 == 0)
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                if (g * 8 < valid) {
                    float f[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) f[j] = __uint_as_float(v[g * 8 + j]) * scale;
                    if (residual) {
                        const uint4 r = *reinterpret_cast<const uint4 *>(residual + off + g * 8);
                        const uint32_t rw[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            f[2 * j] += __uint_as_float(rw[j] << 16);
                            f[2 * j + 1] += __uint_as_float(rw[j] & 0xFFFF0000u);
                        }
                    }
                    uint4 o;
                    o.x = tc::pack_bf16x2(f[0], f[1]);
                    o.y = tc::pack_bf16x2(f[2], f[3]);
                    o.z = tc::pack_bf16x2(f[4], f[5]);
                    o.w = tc::pack_bf16x2(f[6], f[7]);
                    *reinterpret_cast<uint4 *>(out + off + g * 8) = o;
                    if (rn.ss_out) {
                        const uint32_t ow[4] = {o.x, o.y, o.z, o.w};
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const float lo = __uint_as_float(ow[j] << 16), hi = __uint_as_float(ow[j] & 0xFFFF0000u);
                            ss = fmaf(lo, lo, ss);
                            ss = fmaf(hi, hi, ss);
                        }
                    }
                }
            }
        }
    }
    if (rn.ss_out && row < M) rn.ss_out[(size_t)row * tiles_n + tile_n] = ss;
}

__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w, int M, int N,
               int K, const __nv_bfloat16 *__restrict__ residual, __nv_bfloat16 *__restrict__ out, StrRowNorm rn, StrConvEpilogue cv,
               int *status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t *bars = (uint64_t *)(smem + (size_t)STAGES * STAGE_BYTES);
    uint64_t *full = bars, *empty = bars + STAGES, *acc_full = bars + 2 * STAGES, *acc_empty = bars + 2 * STAGES + 2;
    uint32_t *tmem_slot = (uint32_t *)(bars + 2 * STAGES + 4);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tiles_m = (M + BM - 1) / BM, tiles_n = (N + BN - 1) / BN, tiles = tiles_m * tiles_n;
    const int k_blocks = (K + BK - 1) / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { tc::mbar_init(full + s, 1); tc::mbar_init(empty + s, 1); }
        for (int a = 0; a < 2; ++a) { tc::mbar_init(acc_full + a, 1); tc::mbar_init(acc_empty + a, cv.T ? 8 : 4); }
        abort_flag[0] = 0;
        abort_flag[1] = 0;
        tc::fence_mbar_init();
        tc::prefetch_tmap(&tmap_a);
        tc::prefetch_tmap(&tmap_w);
    }
    if (warp == 1) { tc::tmem_alloc(tmem_slot, 512); tc::tmem_relinquish(); }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            int it = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < tiles && ok; t += gridDim.x) {
                const TileCoord tc_ = tile_coord(t, tiles_m, tiles_n);
                for (int kb = 0; kb < k_blocks; ++kb, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1;
                    if (!tc::mbar_wait(empty + s, ph ^ 1, abort_flag)) { ok = false; break; }
                    tc::mbar_arrive_expect_tx(full + s, STAGE_BYTES);
                    uint8_t *sa = smem + (size_t)s * STAGE_BYTES;
                    tc::tma_load_2d(sa, &tmap_a, full + s, kb * BK, tc_.m * BM);
                    tc::tma_load_2d(sa + A_BYTES, &tmap_w, full + s, kb * BK, tc_.n * BN);
                }
            }
            if (!ok) {
                atomicCAS(status, 0, STR_ERR_TIMEOUT);
                // let copies already issued land before the CTA's shared memory goes away
                for (int back = 1; back <= STAGES && back <= it; ++back) {
                    const int j = it - back;
                    tc::mbar_wait(full + j % STAGES, (j / STAGES) & 1, abort_flag + 1);
                }
            }
        }
    } else if (warp == 1) {
        // one elected thread for the whole loop; each 64-column stage is one block of four tcgen05.mma
        if (tc::elect_one()) {
            const uint32_t idesc = tc::make_idesc_bf16(BM, BN, 0, 0);
            int it = 0, local = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < tiles && ok; t += gridDim.x, ++local) {
                const int acc = local & 1;
                const uint32_t aph = (local >> 1) & 1;
                if (!tc::mbar_wait(acc_empty + acc, aph ^ 1, abort_flag)) { ok = false; break; }
                tc::tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)acc * BN;
                for (int kb = 0; kb < k_blocks; ++kb, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1;
                    if (!tc::mbar_wait(full + s, ph, abort_flag)) { ok = false; break; }
                    tc::tc_fence_after();
                    const uint32_t sa = tc::smem_u32(smem + (size_t)s * STAGE_BYTES);
                    static_assert(BK / UMMA_K == 4, "one stage is four K-slices");
                    tc::mma4_ss<tc::StepKMajor64, tc::StepKMajor64>(d_tmem, tc::desc_kmajor_sw128(sa, 0),
                                                                    tc::desc_kmajor_sw128(sa + A_BYTES, 0), idesc, kb != 0);
                    tc::mma_commit(empty + s);
                }
                if (ok) tc::mma_commit(acc_full + acc);
            }
            if (!ok) atomicCAS(status, 0, STR_ERR_TIMEOUT);
        }
        __syncwarp();
    } else if (warp < 6 || cv.T != 0) {
        const int quad = warp & 3;                       // TMEM lane quadrant this warp may read
        // the fused pre-scan epilogue splits the tile's columns between the two warps of a quadrant
        const int c_begin = cv.T ? (warp < 6 ? 0 : BN / 2) : 0, c_end = cv.T ? c_begin + BN / 2 : BN;
        int local = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < tiles && ok; t += gridDim.x, ++local) {
            const TileCoord tc_ = tile_coord(t, tiles_m, tiles_n);
            const int acc = local & 1;
            const uint32_t aph = (local >> 1) & 1;
            if (!tc::mbar_wait(acc_full + acc, aph, abort_flag)) { ok = false; break; }
            tc::tc_fence_after();
            store_rows(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)acc * BN, tc_.m * BM + quad * 32 + lane,
                       tc_.n, tiles_n, M, N, residual, out, rn, cv, c_begin, c_end);
            tc::tc_fence_before();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(acc_empty + acc);
        }
        if (!ok && lane == 0) atomicCAS(status, 0, STR_ERR_TIMEOUT);
    }
    tc::tc_fence_before();
    __syncthreads();
    if (warp == 1) { tc::tc_fence_after(); tc::tmem_dealloc(tmem_base, 512); }
}

// ---- the same GEMM on CTA pairs ------------------------------------------------------------------
// A cluster of two CTAs on neighbouring SMs owns a 256 x 256 output tile and runs it as ONE tcgen05.mma of M = 256
// per K-slice (cta_group::2), issued by CTA 0.  CTA r stages rows [128 r, 128 r + 128) of the A tile and rows
// [128 r, 128 r + 128) of the W tile, so an SM moves 8 KB of operands per K-slice through its shared memory instead
// of 12 KB, and holds rows [128 r, 128 r + 128) of the accumulator in its own tensor memory; its four epilogue warps
// store them exactly as the lone-CTA kernel does (same arithmetic in the same order: the outputs are bit-identical).
// Barriers: each CTA has its own `empty` ring (CTA 0's commit arrives on both) and `acc_full` pair (likewise); the
// `full` ring and the `acc_empty` pair that count are CTA 0's: both producers' copies complete their bytes there,
// and both CTAs' epilogue warps arrive there.
constexpr int P_BM = 256, P_STAGES = 7;
constexpr int P_A_BYTES = 128 * BK * 2, P_W_BYTES = 128 * BK * 2, P_STAGE_BYTES = P_A_BYTES + P_W_BYTES;
constexpr size_t P_SMEM_BYTES = 1024 /*align slack*/ + (size_t)P_STAGES * P_STAGE_BYTES + 256;

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
gemm_tc_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w, int M, int N,
                    int K, const __nv_bfloat16 *__restrict__ residual, __nv_bfloat16 *__restrict__ out, StrRowNorm rn,
                    StrConvEpilogue cv, int *status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t *bars = (uint64_t *)(smem + (size_t)P_STAGES * P_STAGE_BYTES);
    uint64_t *full = bars, *empty = bars + P_STAGES, *acc_full = bars + 2 * P_STAGES, *acc_empty = bars + 2 * P_STAGES + 2;
    uint32_t *tmem_slot = (uint32_t *)(bars + 2 * P_STAGES + 4);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = tc::cluster_cta_rank();
    const int pair = blockIdx.x >> 1, pairs = gridDim.x >> 1;
    const int tiles_m = (M + P_BM - 1) / P_BM, tiles_n = (N + BN - 1) / BN, tiles = tiles_m * tiles_n;
    const int k_blocks = (K + BK - 1) / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < P_STAGES; ++s) { tc::mbar_init(full + s, 1); tc::mbar_init(empty + s, 1); }
        for (int a = 0; a < 2; ++a) { tc::mbar_init(acc_full + a, 1); tc::mbar_init(acc_empty + a, cv.T ? 16 : 8); }
        abort_flag[0] = 0;
        tc::fence_mbar_init();
        tc::prefetch_tmap(&tmap_a);
        tc::prefetch_tmap(&tmap_w);
    }
    __syncthreads();
    tc::cluster_sync_all();                  // both CTAs' barriers exist before anything can signal them
    if (warp == 1) { tc::tmem_alloc_pair(tmem_slot, 512); tc::tmem_relinquish_pair(); }
    tc::tc_fence_before();
    __syncthreads();
    tc::cluster_sync_all();                  // both halves of the accumulator are allocated before the first MMA
    tc::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            int it = 0;
            bool ok = true;
            for (int t = pair; t < tiles && ok; t += pairs) {
                const TileCoord tc_ = tile_coord(t, tiles_m, tiles_n);
                for (int kb = 0; kb < k_blocks; ++kb, ++it) {
                    const int s = it % P_STAGES;
                    const uint32_t ph = (it / P_STAGES) & 1;
                    if (!tc::mbar_wait(empty + s, ph ^ 1, abort_flag)) { ok = false; break; }
                    if (rank == 0) tc::mbar_arrive_expect_tx(full + s, 2 * P_STAGE_BYTES);
                    const uint32_t full_cta0 = tc::map_to_cta(full + s, 0);
                    uint8_t *sa = smem + (size_t)s * P_STAGE_BYTES;
                    tc::tma_load_2d_pair(sa, &tmap_a, full_cta0, kb * BK, tc_.m * P_BM + (int)rank * 128);
                    tc::tma_load_2d_pair(sa + P_A_BYTES, &tmap_w, full_cta0, kb * BK, tc_.n * BN + (int)rank * 128);
                }
            }
            // every commit aimed at this CTA's ring has arrived before the CTA may leave
            for (int back = 0; back < P_STAGES && ok; ++back, ++it)
                if (!tc::mbar_wait(empty + it % P_STAGES, ((it / P_STAGES) & 1) ^ 1, abort_flag)) ok = false;
            if (!ok) {
                atomicCAS(status, 0, STR_ERR_TIMEOUT);
                for (int i = 0; i < 2000; ++i) __nanosleep(1000);    // copies already issued land before the CTA leaves
            }
        }
    } else if (warp == 1) {
        if (rank == 0 && tc::elect_one()) {
            const uint32_t idesc = tc::make_idesc_bf16(P_BM, BN, 0, 0);
            int it = 0, local = 0;
            bool ok = true;
            for (int t = pair; t < tiles && ok; t += pairs, ++local) {
                const int acc = local & 1;
                const uint32_t aph = (local >> 1) & 1;
                if (!tc::mbar_wait(acc_empty + acc, aph ^ 1, abort_flag)) { ok = false; break; }
                tc::tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)acc * BN;
                for (int kb = 0; kb < k_blocks; ++kb, ++it) {
                    const int s = it % P_STAGES;
                    const uint32_t ph = (it / P_STAGES) & 1;
                    if (!tc::mbar_wait(full + s, ph, abort_flag)) { ok = false; break; }
                    tc::tc_fence_after();
                    const uint32_t sa = tc::smem_u32(smem + (size_t)s * P_STAGE_BYTES);
                    tc::mma4_ss_pair<tc::StepKMajor64, tc::StepKMajor64>(d_tmem, tc::desc_kmajor_sw128(sa, 0),
                                                                         tc::desc_kmajor_sw128(sa + P_A_BYTES, 0), idesc, kb != 0);
                    tc::mma_commit_pair(empty + s, 3);
                }
                if (ok) tc::mma_commit_pair(acc_full + acc, 3);
            }
            if (!ok) atomicCAS(status, 0, STR_ERR_TIMEOUT);
        }
        __syncwarp();
    } else if (warp < 6 || cv.T != 0) {
        const int quad = warp & 3;                       // TMEM lane quadrant this warp may read
        // the fused pre-scan epilogue splits the tile's columns between the two warps of a quadrant
        const int c_begin = cv.T ? (warp < 6 ? 0 : BN / 2) : 0, c_end = cv.T ? c_begin + BN / 2 : BN;
        int local = 0;
        bool ok = true;
        for (int t = pair; t < tiles && ok; t += pairs, ++local) {
            const TileCoord tc_ = tile_coord(t, tiles_m, tiles_n);
            const int acc = local & 1;
            const uint32_t aph = (local >> 1) & 1;
            if (!tc::mbar_wait(acc_full + acc, aph, abort_flag)) { ok = false; break; }
            tc::tc_fence_after();
            store_rows(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)acc * BN,
                       tc_.m * P_BM + (int)rank * 128 + quad * 32 + lane, tc_.n, tiles_n, M, N, residual, out, rn, cv, c_begin, c_end);
            tc::tc_fence_before();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive_cluster(tc::map_to_cta(acc_empty + acc, 0));
        }
        if (!ok && lane == 0) atomicCAS(status, 0, STR_ERR_TIMEOUT);
    }
    tc::tc_fence_before();
    __syncthreads();
    tc::cluster_sync_all();                  // neither CTA leaves, or frees tensor memory, while the other still works
    if (warp == 1) { tc::tc_fence_after(); tc::tmem_dealloc_pair(tmem_base, 512); }
}

}  // namespace

bool str_gemm_tc_supported(int dtype, int M, int N, int K, const void *a, const void *w, const void *residual,
                           const void *out) {
    if (dtype != STR_BF16 || M < 1 || N % 8 != 0 || K % 8 != 0 || K < 8) return false;
    const uintptr_t al = (uintptr_t)a | (uintptr_t)w | (uintptr_t)residual | (uintptr_t)out;
    return (al & 15) == 0;
}

// How many CTA pairs the device runs at once (one per SM pair that a cluster of two can occupy), found once per
// context; 0 when clusters of two cannot be launched or STR_GEMM_PAIR=0 asks for the lone-CTA kernel (A/B runs).
static int str_gemm_pairs(str_ctx *ctx) {
    if (ctx->gemm_pairs != 0) return ctx->gemm_pairs > 0 ? ctx->gemm_pairs : 0;
    ctx->gemm_pairs = -1;
    const char *e = getenv("STR_GEMM_PAIR");
    if (e && e[0] == '0') return 0;
    if (str_ensure_smem(ctx, STR_SMEM_GEMM_PAIR, gemm_tc_pair_kernel, P_SMEM_BYTES) != STR_OK) return 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * ctx->sm_count);
    cfg.blockDim = dim3(NUM_THREADS);
    cfg.dynamicSmemBytes = P_SMEM_BYTES;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&clusters, gemm_tc_pair_kernel, &cfg) != cudaSuccess || clusters < 1) {
        (void)cudaGetLastError();
        return 0;
    }
    ctx->gemm_pairs = clusters;
    return clusters;
}

bool str_gemm_conv_supported(int dtype, int M, int N, int K, const void *a, const void *w, const void *out,
                             const StrConvEpilogue &cv) {
    if (!str_gemm_tc_supported(dtype, M, N, K, a, w, nullptr, out)) return false;
    if (cv.T <= 0 || cv.row_base % 32 != 0 || cv.zoff % 32 != 0 || cv.d_inner % 32 != 0 || cv.gn % 32 != 0 || cv.H % 8 != 0)
        return false;
    if (N != cv.zoff + cv.d_inner + 2 * cv.gn + cv.H) return false;
    const uintptr_t al = (uintptr_t)cv.conv_w | (uintptr_t)cv.x_out | (uintptr_t)cv.B_out | (uintptr_t)cv.C_out | (uintptr_t)cv.dt_out;
    return (al & 15) == 0 && cv.conv_w && cv.conv_b && cv.dt_bias && cv.x_out && cv.B_out && cv.C_out && cv.dt_out;
}

int str_gemm_tc(str_ctx *ctx, int M, int N, int K, const void *a, const void *w, const void *residual, void *out,
                const StrRowNorm &rn, const StrConvEpilogue &cv, cudaStream_t st) {
    if (cv.T != 0 && (residual || rn.ss_out)) return STR_ERR_INVALID_ARG;
    // CTA pairs whenever the problem has more than one row tile and the device can co-schedule clusters of two
    const bool paired = M > BM && str_gemm_pairs(ctx) > 0;
    CUtensorMap ta, tw;
    int rc = str_make_tmap_2d_bf16(ctx, &ta, a, (uint64_t)M, (uint64_t)K, (uint64_t)K, BM, BK, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc != STR_OK) return rc;
    rc = str_make_tmap_2d_bf16(ctx, &tw, w, (uint64_t)N, (uint64_t)K, (uint64_t)K, paired ? 128 : BN, BK, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc != STR_OK) return rc;
    if (paired) {
        const int tiles = ceil_div(M, P_BM) * ceil_div(N, BN);
        const int pairs = tiles < ctx->gemm_pairs ? tiles : ctx->gemm_pairs;
        gemm_tc_pair_kernel<<<2 * pairs, NUM_THREADS, P_SMEM_BYTES, st>>>(ta, tw, M, N, K, (const __nv_bfloat16 *)residual,
                                                                         (__nv_bfloat16 *)out, rn, cv, ctx->status_dev);
        return str_launch_ok(ctx);
    }
    rc = str_ensure_smem(ctx, STR_SMEM_GEMM, gemm_tc_kernel, SMEM_BYTES);
    if (rc != STR_OK) return rc;
    const int tiles = ceil_div(M, BM) * ceil_div(N, BN);
    const int grid = tiles < ctx->sm_count ? tiles : ctx->sm_count;
    gemm_tc_kernel<<<grid, NUM_THREADS, SMEM_BYTES, st>>>(ta, tw, M, N, K, (const __nv_bfloat16 *)residual,
                                                         (__nv_bfloat16 *)out, rn, cv, ctx->status_dev);
    return str_launch_ok(ctx);
}
