// Causal GQA softmax attention forward on tcgen05 tensor cores (bf16 in/out, fp32 accumulate,
// head_dim 128).  One CTA owns 256 consecutive query rows of one head: two 128-row query tiles
// that take turns on the tensor pipe, so that the softmax of one overlaps the matrix products of
// the other.
//
// Per key tile j (128 keys) and query tile i:
//   S_i  = Q_i K_j^T                 128x128, both operands K-major in shared memory (TMA, 128-byte swizzle)
//   P_i  = exp2(c S_i - c m_i)       one thread per query row; running row maximum m_i and row sum l_i
//                                    in fp32; P_i is written as bf16 over the first 64 columns of S_i in
//                                    tensor memory and is the A operand of the next product
//   O_i += P_i V_j                   128x128, A from tensor memory, V as MN-major shared-memory operand
//   out  = O_i / l_i
// The accumulator O_i is rescaled only when a row maximum grows by more than 2^8: until then the
// stale maximum stays in use, which changes nothing in exact arithmetic (the same factor divides out
// through l_i) and keeps P_i <= 2^8.
// Tensor memory (512 columns): S_0 | S_1 | O_0 | O_1, 128 columns each.
// Warps: 0-3 softmax of tile 0, 4-7 softmax of tile 1 (warp w may touch TMEM lanes 32 (w % 4)...),
// 8 TMA producer (Q once, then a 2-slot ring for K and one for V), 9 MMA issuer.
// Query rows may be a gathered subset of the sequence (a layer that has already selected its survivors only needs
// their outputs): row r then carries its index t_r in the key sequence (ascending), attends to keys <= t_r, and a
// query tile walks the key tiles up to the one holding its last row's index.  Everything that decides a row's
// arithmetic (its mask, when its running maximum is raised) depends on that row alone, so a row's output does not
// depend on which other rows share its tile: gathered and ungathered calls give bit-identical rows.
// Every mbarrier wait is bounded; a give-up records STR_ERR_TIMEOUT and the CTA tears down.
#include "dispatch.cuh"
#include "tc_common.cuh"

namespace {

constexpr int BQ = 128, BKV = 128, HD = 128;
constexpr int TILE_16K = 16384;                    // 128 rows x 64 bf16
constexpr int OFF_Q = 0;                           // [tile i][half] 4 x 16 KB
constexpr int OFF_K = 4 * TILE_16K;                // [slot][half]
constexpr int OFF_V = 8 * TILE_16K;                // [slot][half]
constexpr int OFF_MISC = 12 * TILE_16K;
enum { B_Q = 0, B_KF0, B_KF1, B_KE0, B_KE1, B_VF0, B_VF1, B_VE0, B_VE1, B_SF0, B_SF1, B_PF0, B_PF1, B_OF0, B_OF1, B_COUNT };
constexpr size_t SMEM_BYTES = (size_t)OFF_MISC + B_COUNT * 8 + 32;
constexpr int NUM_THREADS = 320;
constexpr uint32_t TM_S = 0, TM_O = 256;
constexpr float MASKED = -1.0e30f;
constexpr float RESCALE_THRESHOLD = 8.0f;          // in log2 units

__global__ void __launch_bounds__(NUM_THREADS, 1)
attn_fwd_tc_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                   const __grid_constant__ CUtensorMap tmap_v, int Tq, int Tk, int Hq, int Hkv, float scale_log2,
                   const int32_t *__restrict__ row_pos, __nv_bfloat16 *__restrict__ out, int *status) {
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t *bars = (uint64_t *)(smem + OFF_MISC);
    uint32_t *tmem_slot = (uint32_t *)(bars + B_COUNT);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int pair = (int)gridDim.x - 1 - (int)blockIdx.x;        // longest rows first
    const int h = blockIdx.y, b = blockIdx.z, kv = h / (Hq / Hkv);
    const int r0 = pair * 2 * BQ;
    // index in the key sequence of query row r of this sequence (rows beyond the end take the last row's)
    const int32_t *rp = row_pos ? row_pos + (size_t)b * Tq : nullptr;
    auto key_index = [&](int r) -> int { r = min(r, Tq - 1); return rp ? min(max(__ldg(rp + r), 0), Tk - 1) : r; };
    const int n0 = key_index(r0 + BQ - 1) / BKV + 1;                                  // key tiles of query tile 0
    const int n1 = (r0 + BQ < Tq) ? max(n0, key_index(r0 + 2 * BQ - 1) / BKV + 1) : n0;  // key tiles of query tile 1

    if ((tc::smem_u32(smem) & 1023u) != 0) {
        if (threadIdx.x == 0) atomicCAS(status, 0, STR_ERR_CUDA);
        return;
    }
    // once any CTA has recorded an error the rest of the grid leaves at once
    if (tc::cta_should_leave(status)) return;     // an earlier CTA failed: the whole CTA leaves at once
    if (threadIdx.x == 0) {
        tc::mbar_init(bars + B_Q, 1);
        for (int s = 0; s < 2; ++s) {
            tc::mbar_init(bars + B_KF0 + s, 1); tc::mbar_init(bars + B_KE0 + s, 1);
            tc::mbar_init(bars + B_VF0 + s, 1); tc::mbar_init(bars + B_VE0 + s, 1);
            tc::mbar_init(bars + B_SF0 + s, 1); tc::mbar_init(bars + B_PF0 + s, 4);
            tc::mbar_init(bars + B_OF0 + s, 1);
        }
        abort_flag[0] = 0; abort_flag[1] = 0;
        tc::fence_mbar_init();
        tc::prefetch_tmap(&tmap_q); tc::prefetch_tmap(&tmap_k); tc::prefetch_tmap(&tmap_v);
    }
    if (warp == 9) { tc::tmem_alloc(tmem_slot, 512); tc::tmem_relinquish(); }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 8) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            bool ok = true;
            tc::mbar_arrive_expect_tx(bars + B_Q, 4 * TILE_16K);
            for (int i = 0; i < 2; ++i)
                for (int hf = 0; hf < 2; ++hf)
                    tc::tma_load_3d(smem + OFF_Q + (i * 2 + hf) * TILE_16K, &tmap_q, bars + B_Q, h * HD + hf * 64,
                                    r0 + i * BQ, b);
            int issued_k = 0, issued_v = 0;
            for (int j = 0; j < n1; ++j) {
                const int s = j & 1;
                const uint32_t ph = ((j >> 1) & 1) ^ 1;
                if (!tc::mbar_wait(bars + B_KE0 + s, ph, abort_flag)) { ok = false; break; }
                tc::mbar_arrive_expect_tx(bars + B_KF0 + s, 2 * TILE_16K);
                for (int hf = 0; hf < 2; ++hf)
                    tc::tma_load_3d(smem + OFF_K + (s * 2 + hf) * TILE_16K, &tmap_k, bars + B_KF0 + s, kv * HD + hf * 64,
                                    j * BKV, b);
                ++issued_k;
                if (!tc::mbar_wait(bars + B_VE0 + s, ph, abort_flag)) { ok = false; break; }
                tc::mbar_arrive_expect_tx(bars + B_VF0 + s, 2 * TILE_16K);
                for (int hf = 0; hf < 2; ++hf)
                    tc::tma_load_3d(smem + OFF_V + (s * 2 + hf) * TILE_16K, &tmap_v, bars + B_VF0 + s, kv * HD + hf * 64,
                                    j * BKV, b);
                ++issued_v;
            }
            if (!ok) {
                atomicCAS(status, 0, STR_ERR_TIMEOUT);
                // let copies already issued land before the CTA's shared memory goes away
                tc::mbar_wait(bars + B_Q, 0, abort_flag + 1);
                for (int back = 1; back <= 2 && back <= issued_k; ++back) {
                    const int j = issued_k - back;
                    tc::mbar_wait(bars + B_KF0 + (j & 1), (j >> 1) & 1, abort_flag + 1);
                }
                for (int back = 1; back <= 2 && back <= issued_v; ++back) {
                    const int j = issued_v - back;
                    tc::mbar_wait(bars + B_VF0 + (j & 1), (j >> 1) & 1, abort_flag + 1);
                }
            }
        }
    } else if (warp == 9) {
        // ------------------------------------------------------------------ MMA issuer
        // One elected thread runs the loop and issues each product as one block of eight tcgen05.mma (see
        // tc_common.cuh: issued statement by statement the products lose the issue slot to the softmax warps).
        if (tc::elect_one()) {
            const uint32_t id_s = tc::make_idesc_bf16(BQ, BKV, 0, 0);     // Q (K-major) x K (K-major)
            const uint32_t id_o = tc::make_idesc_bf16(BQ, HD, 0, 1);      // P (tensor memory) x V (MN-major)
            const uint32_t sbase = tc::smem_u32(smem);
            auto issue_s = [&](int i, int slot) {
                const uint32_t qa = sbase + OFF_Q + (uint32_t)i * 2 * TILE_16K;
                const uint32_t ka = sbase + OFF_K + (uint32_t)slot * 2 * TILE_16K;
                tc::mma8_ss<tc::StepKMajor2x64, tc::StepKMajor2x64>(tmem + TM_S + (uint32_t)i * 128, tc::desc_kmajor_sw128(qa, 0),
                                                                    tc::desc_kmajor_sw128(ka, 0), id_s, false);
                tc::mma_commit(bars + B_SF0 + i);
            };
            auto issue_pv = [&](int i, int slot, bool first) {
                const uint32_t va = sbase + OFF_V + (uint32_t)slot * 2 * TILE_16K;
                tc::mma8_ts<tc::StepTmem8, tc::StepMNMajor>(tmem + TM_O + (uint32_t)i * 128, tmem + TM_S + (uint32_t)i * 128,
                                                            tc::make_smem_desc(va, TILE_16K, 1024, tc::SWZ_128B), id_o, !first);
            };
            bool ok = tc::mbar_wait(bars + B_Q, 0, abort_flag) && tc::mbar_wait(bars + B_KF0, 0, abort_flag);
            if (ok) {
                tc::tc_fence_after();
                issue_s(0, 0);
                issue_s(1, 0);
                tc::mma_commit(bars + B_KE0);
            }
            for (int j = 0; j < n1 && ok; ++j) {
                const int s = j & 1, ns = (j + 1) & 1;
                if (j < n0) {
                    if (!tc::mbar_wait(bars + B_PF0, j & 1, abort_flag)) { ok = false; break; }
                }
                if (!tc::mbar_wait(bars + B_VF0 + s, (j >> 1) & 1, abort_flag)) { ok = false; break; }
                tc::tc_fence_after();
                if (j < n0) {
                    issue_pv(0, s, j == 0);
                    if (j == n0 - 1) tc::mma_commit(bars + B_OF0);
                }
                if (j + 1 < n1) {
                    if (!tc::mbar_wait(bars + B_KF0 + ns, ((j + 1) >> 1) & 1, abort_flag)) { ok = false; break; }
                    tc::tc_fence_after();
                    if (j + 1 < n0) issue_s(0, ns);
                }
                if (!tc::mbar_wait(bars + B_PF1, j & 1, abort_flag)) { ok = false; break; }
                tc::tc_fence_after();
                issue_pv(1, s, j == 0);
                tc::mma_commit(bars + B_VE0 + s);
                if (j + 1 < n1) {
                    issue_s(1, ns);
                    tc::mma_commit(bars + B_KE0 + ns);
                } else {
                    tc::mma_commit(bars + B_OF1);
                }
            }
            if (!ok) atomicCAS(status, 0, STR_ERR_TIMEOUT);
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ softmax warps
        const int i = warp >> 2, quad = warp & 3;
        const int row = quad * 32 + lane;                       // row inside the query tile
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        const uint32_t tS = tmem + lane_base + TM_S + (uint32_t)i * 128;
        const uint32_t tO = tmem + lane_base + TM_O + (uint32_t)i * 128;
        const int ni = i == 0 ? n0 : n1;
        const int t_row = key_index(r0 + i * BQ + row);         // this row attends to keys 0 .. t_row
        float m = MASKED, l = 0.f;
        bool ok = true;
        for (int j = 0; j < ni; ++j) {
            if (!tc::mbar_wait(bars + B_SF0 + i, j & 1, abort_flag)) { ok = false; break; }
            tc::tc_fence_after();
            uint32_t v[4][32];
#pragma unroll
            for (int c = 0; c < 4; ++c) tc::tmem_ld32(tS + c * 32, v[c]);
            tc::tmem_ld_wait();
            if (__any_sync(0xffffffffu, j * BKV + BKV - 1 > t_row)) {      // some row of this warp ends inside (or before) this tile
                const int lim = t_row - j * BKV;                            // keys of this tile beyond lim are masked
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        if (c * 32 + e > lim) v[c][e] = __float_as_uint(MASKED);
            }
            float tmax = MASKED;
#pragma unroll
            for (int c = 0; c < 4; ++c)
#pragma unroll
                for (int e = 0; e < 32; ++e) tmax = fmaxf(tmax, __uint_as_float(v[c][e]));
            const float m_new = fmaxf(m, tmax);
            // a row raises its maximum only when it has grown by more than the threshold: a decision of the row alone
            const bool grow = (m_new - m) * scale_log2 > RESCALE_THRESHOLD;
            if (j == 0) {
                m = m_new;
            } else if (__any_sync(0xffffffffu, grow)) {
                // S_j complete implies the previous P V product of this tile is complete: O is stable.  The whole warp
                // runs the (warp-collective) accumulator update; rows that keep their maximum multiply by exactly 1.
                const float f = grow ? tc::ex2((m - m_new) * scale_log2) : 1.0f;
                if (grow) { l *= f; m = m_new; }
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    uint32_t o[32];
                    tc::tmem_ld32(tO + c * 32, o);
                    tc::tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * f);
                    tc::tmem_st32(tO + c * 32, o);
                }
                tc::tmem_st_wait();
            }
            const float mc = m * scale_log2;
            float sum = 0.f;
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t pk[32];
#pragma unroll
                for (int e = 0; e < 32; ++e) {
                    const int cc = 2 * c + (e >> 4), ee = (2 * e) & 31;
                    const float p0 = tc::ex2(fmaf(__uint_as_float(v[cc][ee]), scale_log2, -mc));
                    const float p1 = tc::ex2(fmaf(__uint_as_float(v[cc][ee + 1]), scale_log2, -mc));
                    sum += p0 + p1;
                    pk[e] = tc::pack_bf16x2(p0, p1);
                }
                tc::tmem_st32(tS + c * 32, pk);
            }
            l += sum;
            tc::tmem_st_wait();
            tc::tc_fence_before();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(bars + B_PF0 + i);
        }
        if (ok) ok = tc::mbar_wait(bars + B_OF0 + i, 0, abort_flag);
        if (ok) {
            tc::tc_fence_after();
            const int t = r0 + i * BQ + row;
            const float inv = 1.0f / l;
            __nv_bfloat16 *dst = out + (((size_t)b * Tq + t) * Hq + h) * HD;
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                uint32_t o[32];
                tc::tmem_ld32(tO + c * 32, o);
                tc::tmem_ld_wait();
                if (t < Tq) {
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        uint4 w;
                        w.x = tc::pack_bf16x2(__uint_as_float(o[8 * g]) * inv, __uint_as_float(o[8 * g + 1]) * inv);
                        w.y = tc::pack_bf16x2(__uint_as_float(o[8 * g + 2]) * inv, __uint_as_float(o[8 * g + 3]) * inv);
                        w.z = tc::pack_bf16x2(__uint_as_float(o[8 * g + 4]) * inv, __uint_as_float(o[8 * g + 5]) * inv);
                        w.w = tc::pack_bf16x2(__uint_as_float(o[8 * g + 6]) * inv, __uint_as_float(o[8 * g + 7]) * inv);
                        *reinterpret_cast<uint4 *>(dst + c * 32 + g * 8) = w;
                    }
                }
            }
        } else if (lane == 0) {
            atomicCAS(status, 0, STR_ERR_TIMEOUT);
        }
    }
    tc::tc_fence_before();
    __syncthreads();
    if (warp == 9) { tc::tc_fence_after(); tc::tmem_dealloc(tmem, 512); }
}

}  // namespace

bool str_attn_prefill_tc_supported(const str_attn_shape *s, const void *q, const void *k, const void *v, const void *o) {
    if (s->dtype != STR_BF16 || s->d != HD || s->T < 1) return false;
    return (((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)o) & 15) == 0;
}

int str_attn_prefill_tc(str_ctx *ctx, const str_attn_shape *s, int n_rows, const void *q, const int32_t *row_pos, const void *k,
                        const void *v, float scale, void *o, cudaStream_t st) {
    if (SMEM_BYTES > (size_t)ctx->max_smem_optin) return STR_ERR_UNSUPPORTED_SHAPE;
    CUtensorMap tq, tk, tv;
    int rc = str_make_tmap_3d_bf16_sw128(ctx, &tq, q, (uint64_t)s->Hq * HD, (uint64_t)n_rows, (uint64_t)s->Bz, BQ);
    if (rc == STR_OK) rc = str_make_tmap_3d_bf16_sw128(ctx, &tk, k, (uint64_t)s->Hkv * HD, (uint64_t)s->T, (uint64_t)s->Bz, BKV);
    if (rc == STR_OK) rc = str_make_tmap_3d_bf16_sw128(ctx, &tv, v, (uint64_t)s->Hkv * HD, (uint64_t)s->T, (uint64_t)s->Bz, BKV);
    if (rc != STR_OK) return rc;
    rc = str_ensure_smem(ctx, STR_SMEM_ATTN_FWD, attn_fwd_tc_kernel, SMEM_BYTES);
    if (rc != STR_OK) return rc;
    dim3 grid(ceil_div(n_rows, 2 * BQ), s->Hq, s->Bz);
    attn_fwd_tc_kernel<<<grid, NUM_THREADS, SMEM_BYTES, st>>>(tq, tk, tv, n_rows, s->T, s->Hq, s->Hkv,
                                                             scale * 1.4426950408889634f, row_pos, (__nv_bfloat16 *)o,
                                                             ctx->status_dev);
    return str_launch_ok(ctx);
}
