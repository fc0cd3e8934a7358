// Mamba-2 SSD chunked scan on tcgen05 tensor cores (bf16 in, fp32 accumulate), head dim p = 64,
// state dim n = 128.  One CTA per (sequence, head) walks the sequence in chunks of 128 tokens and
// carries the running state in registers, so chunk states never travel through global memory.
//
// Per chunk c, with l_t the in-chunk inclusive cumulative log-decay (l_t = sum_{u<=t} dt_u A_h <= 0):
//   CB      = C B^T                                  [128 x 128]   tcgen05, K-major operands
//   W[t,j]  = CB[t,j] exp(l_t - l_j) dt_j 1[j<=t]    fp32 on CUDA cores -> bf16, written back over CB in
//                                                    tensor memory: the A operand of the next product
//   Y_intra = W X                                    [128 x 64]    tcgen05, A from tensor memory, X MN-major
//   Y_inter = C S_prev^T                             [128 x 64]    tcgen05, bf16 copy of the state
//   y_t     = Y_intra[t] + exp(l_t) Y_inter[t]                     fp32 epilogue -> bf16 -> global
//   dS^T    = B^T Xs,  Xs_j = exp(l_end - l_j) dt_j x_j  [128 x 64] tcgen05, both operands MN-major
//   S^T    <- exp(l_end) S^T + dS^T                                fp32 registers (the master state)
// Every decay factor is formed from a difference of cumulative sums that is <= 0.  Off the
// diagonal 32x32 blocks exp(l_t - l_j) is split into three factors, each <= 1 (row part, block-pair
// scalar, column part); the diagonal blocks take one exponential per element.
//
// The chunk loop is software-pipelined across warp roles that only meet at mbarriers; the only
// serial chains from chunk to chunk are  dS_c -> state update -> Y_inter_{c+1}  and
// dS_c -> Xs_{c+1} -> dS_{c+1}  (single Xs buffer):
//   warps 0-3, 14, 15  W_c from CB_c in 16-column pieces of a 32-row quadrant (one thread per token row)
//   warps 4-7          state update (one thread per state row n, 64 fp32 registers of state);
//                      lane 0 of warp 4 is the TMA producer (B,C ring of 2, X ring of 3, 128-byte swizzle): seeing
//                      dS_c complete is what frees the slots of chunk c+2, so there are no slot-release barriers
//   warps 8-11         Xs_{c+1}, then the epilogue of chunk c (one thread per token row)
//   warp 12            the decay vectors of each chunk (cumulative sum, exponentials) into a ring of 4; depends on
//                      dt only and runs up to three chunks ahead of its readers
//   warp 13            MMA issuer (one elected thread); iteration c issues  CB_c, Y_intra_{c-1}, Y_inter_c, dS_c
// Loops are kept rolled where registers allow: the instruction footprint of all roles together has to
// stay inside the instruction cache, or every role slows down together.
// Tensor memory: CB/W 2 x 128 columns | Y_inter 2 x 64 | Y_intra 64 | dS 64.  W's K-slice ks (keys
// 16 ks .. 16 ks + 15) sits in columns [16 ks, 16 ks + 8) of the CB buffer it was computed from, so a
// thread only overwrites accumulator columns that it has read itself.
// All mbarrier waits are bounded; a give-up records STR_ERR_TIMEOUT and tears the CTA down.
#include "dispatch.cuh"
#include "tc_common.cuh"

namespace {

constexpr int Q = 128, P = 64, NS = 128;
constexpr int TILE_16K = 16384;
constexpr int X_SLOTS = 3, DEC_DEPTH = 4, DEC_FLOATS = 800;
constexpr int OFF_X = 0;                                  // 3 x 16 KB
constexpr int OFF_B = OFF_X + X_SLOTS * TILE_16K;         // 2 x 32 KB
constexpr int OFF_C = OFF_B + 4 * TILE_16K;               // 2 x 32 KB
constexpr int OFF_XS = OFF_C + 4 * TILE_16K;              // 16 KB
constexpr int OFF_SB = OFF_XS + TILE_16K;                 // 16 KB
constexpr int OFF_DEC = OFF_SB + TILE_16K;                // 4 x 3200 B
constexpr int OFF_BARS = OFF_DEC + DEC_DEPTH * DEC_FLOATS * 4;
// decay vectors of one chunk (floats): log2-domain cumulative decay l_j, log2(dt_j) - l_j, column / state / row factors
constexpr int D_LS = 0, D_NLC = 128, D_COLF = 256, D_XW = 384, D_ROWF = 512, D_EROW = 640, D_BLK = 768, D_EEND = 784;
enum {
    B_XF = 0, B_BCF = 3, B_DECF = 5, B_DECE = 9, B_CBF = 13, B_WF = 15, B_XSF = 17, B_DSF, B_DSE,
    B_SF, B_YF, B_YE, B_COUNT
};
constexpr size_t SMEM_BYTES = (size_t)OFF_BARS + B_COUNT * 8 + 32;
constexpr int NUM_WARPS = 16, NUM_THREADS = NUM_WARPS * 32;
constexpr int W_WARPS = 6;
constexpr int DEC_READERS = W_WARPS + 4 + 4;              // warps that read a chunk's decay vectors
constexpr uint32_t TM_CB = 0, TM_YO = 256, TM_YI = 384, TM_DS = 448;
constexpr float LOG2E = 1.4426950408889634f;

__device__ __forceinline__ void warp_arrive(uint64_t *bar, int lane) {
    __syncwarp();
    if (lane == 0) tc::mbar_arrive(bar);
}

// Descriptor arithmetic: the 14-bit start-address field holds (shared address >> 4); every operand of
// this kernel lies below 256 KB, so adding a byte offset >> 4 to the descriptor never carries out of it.
__device__ __forceinline__ uint64_t desc_add(uint64_t d, uint32_t bytes) { return d + (uint64_t)(bytes >> 4); }
// Xs_c = exp(l_end - l_j) dt_j x_j (same swizzled layout as the X tile): 128 threads, eight 16-byte units each.
// The row factor is narrowed to bf16 and applied with packed bf16 multiplies (one instruction per two elements).
__device__ __forceinline__ void scale_x(const uint8_t *x_tile, uint8_t *xs_tile, const float *dec_xw, int tid_g) {
    const uint4 *src = (const uint4 *)x_tile;
    uint4 *dst = (uint4 *)xs_tile;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int u = tid_g + 128 * i;
        const __nv_bfloat162 sc = __float2bfloat162_rn(dec_xw[u >> 3]);
        uint4 v = src[u];
        __nv_bfloat162 *pv = reinterpret_cast<__nv_bfloat162 *>(&v);
#pragma unroll
        for (int j = 0; j < 4; ++j) pv[j] = __hmul2(pv[j], sc);
        dst[u] = v;
    }
}

// One 16-column piece of W = CB o decay for this thread's token row: fp32 CB values in, eight packed bf16 pairs out.
// Diagonal 32x32 block: one exponential per element, exp2(l_t + (log2 dt_j - l_j)), masked above the diagonal.
__device__ __forceinline__ void w_piece_diag(const uint32_t (&v)[16], uint32_t (&packed)[8], const float *dec, int col0, int row, float l_t) {
    const float2 lt2 = make_float2(l_t, l_t);
#pragma unroll
    for (int i4 = 0; i4 < 4; ++i4) {
        const float4 nl = *(const float4 *)(dec + D_NLC + col0 + 4 * i4);
        const int j0 = col0 + 4 * i4;
        const float2 a01 = __fadd2_rn(lt2, make_float2(nl.x, nl.y)), a23 = __fadd2_rn(lt2, make_float2(nl.z, nl.w));
        const float f0 = (j0 <= row) ? tc::ex2(a01.x) : 0.f;
        const float f1 = (j0 + 1 <= row) ? tc::ex2(a01.y) : 0.f;
        const float f2 = (j0 + 2 <= row) ? tc::ex2(a23.x) : 0.f;
        const float f3 = (j0 + 3 <= row) ? tc::ex2(a23.y) : 0.f;
        const float2 r01 = __fmul2_rn(make_float2(__uint_as_float(v[4 * i4]), __uint_as_float(v[4 * i4 + 1])), make_float2(f0, f1));
        const float2 r23 = __fmul2_rn(make_float2(__uint_as_float(v[4 * i4 + 2]), __uint_as_float(v[4 * i4 + 3])), make_float2(f2, f3));
        packed[2 * i4] = tc::pack_bf16x2(r01.x, r01.y);
        packed[2 * i4 + 1] = tc::pack_bf16x2(r23.x, r23.y);
    }
}
// Block below the diagonal: exp(l_t - l_j) dt_j = f (row part times block-pair scalar) * column part, each <= 1.
__device__ __forceinline__ void w_piece_below(const uint32_t (&v)[16], uint32_t (&packed)[8], const float *dec, int col0, float f) {
    const float2 ff = make_float2(f, f);
#pragma unroll
    for (int i4 = 0; i4 < 4; ++i4) {
        const float4 cf = *(const float4 *)(dec + D_COLF + col0 + 4 * i4);
        const float2 r01 = __fmul2_rn(make_float2(__uint_as_float(v[4 * i4]), __uint_as_float(v[4 * i4 + 1])), __fmul2_rn(ff, make_float2(cf.x, cf.y)));
        const float2 r23 = __fmul2_rn(make_float2(__uint_as_float(v[4 * i4 + 2]), __uint_as_float(v[4 * i4 + 3])), __fmul2_rn(ff, make_float2(cf.z, cf.w)));
        packed[2 * i4] = tc::pack_bf16x2(r01.x, r01.y);
        packed[2 * i4 + 1] = tc::pack_bf16x2(r23.x, r23.y);
    }
}

__global__ void __launch_bounds__(NUM_THREADS, 1)
ssd_tc_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_b,
              const __grid_constant__ CUtensorMap tmap_c, int Tlen, int H, int G, const float *__restrict__ dt,
              const float *__restrict__ A, __nv_bfloat16 *__restrict__ y, float *__restrict__ final_state, int *status) {
    extern __shared__ __align__(1024) uint8_t smem[];
    float *decs = (float *)(smem + OFF_DEC);
    uint64_t *bars = (uint64_t *)(smem + OFF_BARS);
    uint32_t *tmem_slot = (uint32_t *)(bars + B_COUNT);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);

    // Role numbers (the `warp` used below) are decoupled from hardware warp numbers: when several warps of a
    // scheduler are ready it favours the lower-numbered one, so the MMA issuer and the decay warp, which need
    // few issue slots but need them promptly, take hardware warps 0 and 1 and the instruction-heavy W roles
    // the highest numbers.  Roles that touch tensor memory keep role % 4 == hardware warp % 4 (lane quadrant).
    const int hw_warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int warp = hw_warp < 2 ? 13 - hw_warp : hw_warp < 4 ? hw_warp + 12 : hw_warp < 12 ? hw_warp : hw_warp - 12;
    const int h = blockIdx.x, b = blockIdx.y, g = h / (H / G);
    const int nchunks = (Tlen + Q - 1) / Q;

    if ((tc::smem_u32(smem) & 1023u) != 0) {          // swizzled tiles need a 1024-byte aligned base
        if (threadIdx.x == 0) atomicCAS(status, 0, STR_ERR_CUDA);
        return;
    }
    if (tc::cta_should_leave(status)) return;     // an earlier CTA failed: the whole CTA leaves at once
    if (threadIdx.x == 0) {
        for (int i = 0; i < X_SLOTS; ++i) tc::mbar_init(bars + B_XF + i, 1);
        for (int i = 0; i < 2; ++i) {
            tc::mbar_init(bars + B_BCF + i, 1);
            tc::mbar_init(bars + B_CBF + i, 1); tc::mbar_init(bars + B_WF + i, W_WARPS);
        }
        for (int i = 0; i < DEC_DEPTH; ++i) { tc::mbar_init(bars + B_DECF + i, 1); tc::mbar_init(bars + B_DECE + i, DEC_READERS); }
        tc::mbar_init(bars + B_XSF, 4); tc::mbar_init(bars + B_DSF, 1); tc::mbar_init(bars + B_DSE, 4);
        tc::mbar_init(bars + B_SF, 4); tc::mbar_init(bars + B_YF, 1); tc::mbar_init(bars + B_YE, 4);
        abort_flag[0] = 0; abort_flag[1] = 0;
        tc::fence_mbar_init();
        tc::prefetch_tmap(&tmap_x); tc::prefetch_tmap(&tmap_b); tc::prefetch_tmap(&tmap_c);
    }
    if (warp == 13) { tc::tmem_alloc(tmem_slot, 512); tc::tmem_relinquish(); }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 12) {
        // ------------------------------------------------------------------ decay vectors
        const float Ah2 = A[h] * LOG2E;
        const float *dtb = dt + (size_t)b * Tlen * H + h;
        bool ok = true;
        float dv[4], dn[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) dn[i] = (4 * lane + i < Tlen) ? __ldg(dtb + (size_t)(4 * lane + i) * H) : 0.f;
#pragma unroll 1
        for (int c = 0; c < nchunks; ++c) {
            const int d = c & (DEC_DEPTH - 1);
#pragma unroll
            for (int i = 0; i < 4; ++i) {             // this chunk's dt was fetched one iteration ago
                dv[i] = dn[i];
                const int t = (c + 1) * Q + 4 * lane + i;
                dn[i] = t < Tlen ? __ldg(dtb + (size_t)t * H) : 0.f;
            }
            if (!tc::mbar_wait(bars + B_DECE + d, ((c >> 2) & 1) ^ 1, abort_flag)) { ok = false; break; }
            float l[4];
            l[0] = dv[0] * Ah2;
#pragma unroll
            for (int i = 1; i < 4; ++i) l[i] = fmaf(dv[i], Ah2, l[i - 1]);
            float incl = l[3];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const float v = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += v;
            }
            const float excl = incl - l[3];
            const float l_start = __shfl_sync(0xffffffffu, excl, lane & ~7);     // start of this 32-token block
            const float l_endb = __shfl_sync(0xffffffffu, incl, lane | 7);       // end of this 32-token block
            const float l_end = __shfl_sync(0xffffffffu, incl, 31);
            // blk[bt][bj] = exp(l_start(bt) - l_endblock(bj)), bj < bt; lanes 0..15 hold (bt, bj) = (lane/4, lane%4)
            const float bs = __shfl_sync(0xffffffffu, excl, ((lane >> 2) & 3) * 8);
            const float be = __shfl_sync(0xffffffffu, incl, (lane & 3) * 8 + 7);
            float *dec = decs + d * DEC_FLOATS;
            float o_ls[4], o_nlc[4], o_colf[4], o_xw[4], o_rowf[4], o_erow[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float li = excl + l[i];
                o_ls[i] = li;
                o_nlc[i] = tc::lg2(dv[i]) - li;          // exp2(l_t + nlc_j) = exp(l_t - l_j) dt_j; a padded token (dt = 0) gives -inf
                o_colf[i] = tc::ex2(l_endb - li) * dv[i];
                o_xw[i] = tc::ex2(l_end - li) * dv[i];
                o_rowf[i] = tc::ex2(li - l_start);
                o_erow[i] = tc::ex2(li);
            }
            *(float4 *)(dec + D_LS + 4 * lane) = make_float4(o_ls[0], o_ls[1], o_ls[2], o_ls[3]);
            *(float4 *)(dec + D_NLC + 4 * lane) = make_float4(o_nlc[0], o_nlc[1], o_nlc[2], o_nlc[3]);
            *(float4 *)(dec + D_COLF + 4 * lane) = make_float4(o_colf[0], o_colf[1], o_colf[2], o_colf[3]);
            *(float4 *)(dec + D_XW + 4 * lane) = make_float4(o_xw[0], o_xw[1], o_xw[2], o_xw[3]);
            *(float4 *)(dec + D_ROWF + 4 * lane) = make_float4(o_rowf[0], o_rowf[1], o_rowf[2], o_rowf[3]);
            *(float4 *)(dec + D_EROW + 4 * lane) = make_float4(o_erow[0], o_erow[1], o_erow[2], o_erow[3]);
            if (lane < 16) dec[D_BLK + lane] = ((lane & 3) < (lane >> 2)) ? tc::ex2(bs - be) : 0.f;
            if (lane == 0) dec[D_EEND] = tc::ex2(l_end);
            warp_arrive(bars + B_DECF + d, lane);
        }
        if (!ok && lane == 0) atomicCAS(status, 0, STR_ERR_TIMEOUT);
    } else if (warp == 13) {
        // ------------------------------------------------------------------ MMA issuer
        // One elected thread runs the whole loop (the region is entered once, so the compiler knows it to be
        // single-threaded) and issues every product as one straight-line block of eight tcgen05.mma: issued any
        // other way the products cost two to five times the tensor pipe's own time as soon as the arithmetic
        // warps of this scheduler are busy.  Product order per iteration: CB_c, Y_intra_{c-1}, Y_inter_c, dS_c.
        if (tc::elect_one()) {
            const uint32_t id_cb = tc::make_idesc_bf16(128, 128, 0, 0);   // C (K-major) x B (K-major)
            const uint32_t id_kn = tc::make_idesc_bf16(128, 64, 0, 1);    // K-major / tensor-memory A x MN-major B
            const uint32_t id_nn = tc::make_idesc_bf16(128, 64, 1, 1);    // MN-major A x MN-major B
            const uint32_t sbase = tc::smem_u32(smem);
            const uint64_t dk_c0 = tc::desc_kmajor_sw128(sbase + OFF_C, 0), dk_b0 = tc::desc_kmajor_sw128(sbase + OFF_B, 0);
            const uint64_t dm_b0 = tc::make_smem_desc(sbase + OFF_B, TILE_16K, 1024, tc::SWZ_128B);
            const uint64_t dm_xs = tc::make_smem_desc(sbase + OFF_XS, TILE_16K, 1024, tc::SWZ_128B);
            const uint64_t dm_sb = tc::make_smem_desc(sbase + OFF_SB, TILE_16K, 1024, tc::SWZ_128B);
            const uint64_t dm_x0 = tc::make_smem_desc(sbase + OFF_X, TILE_16K, 1024, tc::SWZ_128B);
            bool ok = true;
#pragma unroll 1
            for (int c = 0; c <= nchunks && ok; ++c) {
                const int s = c & 1;
                const uint64_t dk_c = desc_add(dk_c0, (uint32_t)s * 2 * TILE_16K), dk_b = desc_add(dk_b0, (uint32_t)s * 2 * TILE_16K);
                if (c < nchunks) {
                    ok = tc::mbar_wait(bars + B_BCF + s, (c >> 1) & 1, abort_flag);
                    if (!ok) break;
                    tc::tc_fence_after();
                    tc::mma8_ss<tc::StepKMajor2x64, tc::StepKMajor2x64>(tmem + TM_CB + (uint32_t)s * 128, dk_c, dk_b, id_cb, false);   // CB_c = C B^T
                    tc::mma_commit(bars + B_CBF + s);
                }
                if (c >= 1) {
                    const int cp = c - 1, sp = cp & 1;
                    // the epilogue has read the Y accumulators of chunk c-2; W_{c-1} is in tensor memory
                    ok = (c < 2 || tc::mbar_wait(bars + B_YE, (c - 2) & 1, abort_flag)) &&
                         tc::mbar_wait(bars + B_WF + sp, (cp >> 1) & 1, abort_flag);
                    if (!ok) break;
                    tc::tc_fence_after();
                    // Y_intra_{c-1} = W X; K-slice ks of W sits in columns [16 ks, 16 ks + 8)
                    tc::mma8_ts<tc::StepTmem16, tc::StepMNMajor>(tmem + TM_YI, tmem + TM_CB + (uint32_t)sp * 128,
                                                                     desc_add(dm_x0, (uint32_t)(cp % X_SLOTS) * TILE_16K), id_kn, false);
                    tc::mma_commit(bars + B_YF);
                }
                if (c < nchunks) {
                    if (c > 0) {
                        ok = tc::mbar_wait(bars + B_SF, (c - 1) & 1, abort_flag);
                        if (!ok) break;
                        tc::tc_fence_after();
                        // Y_inter_c = C S_{c-1}^T
                        tc::mma8_ss<tc::StepKMajor2x64, tc::StepMNMajor>(tmem + TM_YO + (uint32_t)s * 64, dk_c, dm_sb, id_kn, false);
                    }
                    ok = tc::mbar_wait(bars + B_XSF, c & 1, abort_flag) && (c == 0 || tc::mbar_wait(bars + B_DSE, (c - 1) & 1, abort_flag));
                    if (!ok) break;
                    tc::tc_fence_after();
                    // dS_c^T = B^T Xs
                    tc::mma8_ss<tc::StepMNMajor, tc::StepMNMajor>(tmem + TM_DS, desc_add(dm_b0, (uint32_t)s * 2 * TILE_16K), dm_xs, id_nn, false);
                    tc::mma_commit(bars + B_DSF);
                }
            }
            if (!ok) atomicCAS(status, 0, STR_ERR_TIMEOUT);
        }
        __syncwarp();
    } else if (warp < 4 || warp >= 14) {
        // ------------------------------------------------------------------ W_c = CB_c o decay
        // Work is dealt out in 16-column pieces of a 32-row quadrant (a warp can only reach the tensor-memory lanes
        // of its own quadrant); the later row quadrants have more pieces below the diagonal and get two warps:
        //   quadrant 0: columns 0-31        quadrant 1: 0-63        quadrant 2: 0-63 | 64-95        quadrant 3: 0-79 | 80-127
        // plus zeros for the pieces above the diagonal.  The bf16 result of piece [16k, 16k+16) goes to the 32-bit
        // columns [16k, 16k+8) of the same accumulator buffer, i.e. into columns the same thread has just read, so
        // pieces need no ordering among themselves.
        const int quad = warp & 3, half = warp >= 14 ? 1 : 0;
        const int row = quad * 32 + lane;
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        const int first = half ? (quad == 2 ? 64 : 80) : 0;
        const int n_real = half ? (quad == 2 ? 2 : 3) : (quad == 0 ? 2 : quad == 1 ? 4 : quad + 2);
        const int zero_first = half ? 96 : (quad == 0 ? 32 : 64);
        const int n_zero = half ? (quad == 2 ? 2 : 0) : (quad == 0 ? 6 : quad == 1 ? 4 : 0);
        bool ok = true;
#pragma unroll 1
        for (int c = 0; c < nchunks; ++c) {
            const int d = c & (DEC_DEPTH - 1), s = c & 1;
            const float *dec = decs + d * DEC_FLOATS;
            if (!tc::mbar_wait(bars + B_DECF + d, (c >> 2) & 1, abort_flag)) { ok = false; break; }
            const float l_t = dec[D_LS + row], rf = dec[D_ROWF + row];
            if (!tc::mbar_wait(bars + B_CBF + s, (c >> 1) & 1, abort_flag)) { ok = false; break; }
            tc::tc_fence_after();
            const uint32_t tW = tmem + lane_base + TM_CB + (uint32_t)(s * 128);
            // every piece is fetched before any is worked on: a tensor-memory load takes a few hundred clocks to
            // return while the tensor pipe is busy
            uint32_t v[5][16];
#pragma unroll
            for (int k = 0; k < 5; ++k)
                if (k < n_real) tc::tmem_ld16(tW + (uint32_t)(first + 16 * k), v[k]);
            tc::tmem_ld_wait();
#pragma unroll
            for (int k = 0; k < 5; ++k) {
                if (k < n_real) {
                    const int col0 = first + 16 * k, bj = col0 >> 5;
                    uint32_t packed[8];
                    if (bj == quad) w_piece_diag(v[k], packed, dec, col0, row, l_t);
                    else w_piece_below(v[k], packed, dec, col0, rf * dec[D_BLK + quad * 4 + bj]);
                    tc::tmem_st8(tW + (uint32_t)col0, packed);
                }
            }
            if (n_zero > 0) {
                uint32_t zero[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) zero[i] = 0u;
#pragma unroll 1
                for (int k = 0; k < n_zero; ++k) tc::tmem_st8(tW + (uint32_t)(zero_first + 16 * k), zero);
            }
            tc::tmem_st_wait();
            tc::tc_fence_before();
            warp_arrive(bars + B_WF + s, lane);
            if (lane == 0) tc::mbar_arrive(bars + B_DECE + d);
        }
        if (!ok && lane == 0) atomicCAS(status, 0, STR_ERR_TIMEOUT);
    } else if (warp < 8) {
        // ------------------------------------------------------------------ state update
        const int quad = warp & 3, row = quad * 32 + lane;        // row = state index n
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        float S[64];
#pragma unroll
        for (int i = 0; i < 64; ++i) S[i] = 0.f;
        bool ok = true;
        // Lane 0 of the first state warp is the TMA producer.  The operands of chunk c+2 go into the slots of chunk
        // c (B, C: ring of 2) and chunk c-1 (X: ring of 3) once dS_c is seen complete: the tensor pipe runs in
        // order, so CB_c, Y_inter_c, Y_intra_{c-1} and dS_{c-1} (issued after all of Xs_{c-1} was written, i.e.
        // after every read of X_{c-1}) are complete too.  No slot-release barriers are needed.
        const bool loader = warp == 4 && lane == 0;
        int n_loaded = 0;
        auto load_chunk = [&](int c) {
            const int t0 = c * Q, s = c & 1, sx = c % X_SLOTS;
            uint64_t *fb = bars + B_BCF + s;
            tc::mbar_arrive_expect_tx(fb, 4 * TILE_16K);
            tc::tma_load_3d(smem + OFF_B + (s * 2) * TILE_16K, &tmap_b, fb, g * NS, t0, b);
            tc::tma_load_3d(smem + OFF_B + (s * 2 + 1) * TILE_16K, &tmap_b, fb, g * NS + 64, t0, b);
            tc::tma_load_3d(smem + OFF_C + (s * 2) * TILE_16K, &tmap_c, fb, g * NS, t0, b);
            tc::tma_load_3d(smem + OFF_C + (s * 2 + 1) * TILE_16K, &tmap_c, fb, g * NS + 64, t0, b);
            tc::mbar_arrive_expect_tx(bars + B_XF + sx, TILE_16K);
            tc::tma_load_3d(smem + OFF_X + sx * TILE_16K, &tmap_x, bars + B_XF + sx, h * P, t0, b);
            ++n_loaded;
        };
        if (loader) {
            load_chunk(0);
            if (nchunks > 1) load_chunk(1);
        }
#pragma unroll 1
        for (int c = 0; c < nchunks && ok; ++c) {
            const int d = c & (DEC_DEPTH - 1);
            if (!tc::mbar_wait(bars + B_DECF + d, (c >> 2) & 1, abort_flag)) { ok = false; break; }
            const float eend = decs[d * DEC_FLOATS + D_EEND];
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(bars + B_DECE + d);
            if (!tc::mbar_wait(bars + B_DSF, c & 1, abort_flag)) { ok = false; break; }
            tc::tc_fence_after();
            uint8_t *srow = smem + OFF_SB + (row >> 3) * 1024 + (row & 7) * 128;
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                uint32_t v[32];
                tc::tmem_ld32(tmem + lane_base + TM_DS + (uint32_t)(hf * 32), v);
                tc::tmem_ld_wait();
                if (hf == 1) {                        // both halves of dS_c are in registers: the accumulator is free
                    tc::tc_fence_before();
                    warp_arrive(bars + B_DSE, lane);
                }
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    const float2 r = __ffma2_rn(make_float2(eend, eend), make_float2(S[hf * 32 + i], S[hf * 32 + i + 1]),
                                                make_float2(__uint_as_float(v[i]), __uint_as_float(v[i + 1])));
                    S[hf * 32 + i] = r.x;
                    S[hf * 32 + i + 1] = r.y;
                }
                // bf16 copy of S^T for the next chunk's Y_inter (dS_c complete implies Y_inter_c complete, so
                // the previous copy is no longer being read)
#pragma unroll
                for (int ci = 0; ci < 4; ++ci) {
                    const int q4 = hf * 4 + ci;
                    *(uint4 *)(srow + ((q4 ^ (row & 7)) << 4)) =
                        make_uint4(tc::pack_bf16x2(S[8 * q4], S[8 * q4 + 1]), tc::pack_bf16x2(S[8 * q4 + 2], S[8 * q4 + 3]),
                                   tc::pack_bf16x2(S[8 * q4 + 4], S[8 * q4 + 5]), tc::pack_bf16x2(S[8 * q4 + 6], S[8 * q4 + 7]));
                }
            }
            tc::fence_proxy_async();
            warp_arrive(bars + B_SF, lane);
            if (loader && c + 2 < nchunks) load_chunk(c + 2);
        }
        if (!ok && lane == 0) atomicCAS(status, 0, STR_ERR_TIMEOUT);
        if (!ok && loader) {                          // let copies already issued land before the CTA goes away
            for (int back = 1; back <= 2 && back <= n_loaded; ++back) {
                const int j = n_loaded - back;
                tc::mbar_wait(bars + B_BCF + (j & 1), (j >> 1) & 1, abort_flag + 1);
                tc::mbar_wait(bars + B_XF + j % X_SLOTS, (j / X_SLOTS) & 1, abort_flag + 1);
            }
        }
        if (ok && final_state) {
            float *fs = final_state + ((size_t)b * H + h) * P * NS;
#pragma unroll
            for (int i = 0; i < 64; ++i) fs[(size_t)i * NS + row] = S[i];
        }
    } else if (warp < 12) {
        // ------------------------------------------------------------------ Xs_{c+1}, then y of chunk c
        const int quad = warp & 3, row = quad * 32 + lane;
        const int tid_g = threadIdx.x - 256;
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        __nv_bfloat16 *yb = y + ((size_t)b * Tlen * H + h) * P;
        bool ok = true;
#pragma unroll 1
        for (int c = 0; c <= nchunks; ++c) {
            if (c < nchunks) {
                // Xs_c = exp(l_end - l_j) dt_j x_j, same swizzled layout as the X tile
                const int d = c & (DEC_DEPTH - 1), sx = c % X_SLOTS;
                const float *dec = decs + d * DEC_FLOATS;
                if (!tc::mbar_wait(bars + B_DECF + d, (c >> 2) & 1, abort_flag)) { ok = false; break; }
                if (!tc::mbar_wait(bars + B_XF + sx, (c / X_SLOTS) & 1, abort_flag)) { ok = false; break; }
                if (c > 0 && !tc::mbar_wait(bars + B_DSF, (c - 1) & 1, abort_flag)) { ok = false; break; }   // Xs buffer free
                scale_x(smem + OFF_X + sx * TILE_16K, smem + OFF_XS, dec + D_XW, tid_g);
                tc::fence_proxy_async();
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(bars + B_XSF);
            }
            if (c >= 1) {
                const int cp = c - 1, d = cp & (DEC_DEPTH - 1), t0 = cp * Q;
                const float er = decs[d * DEC_FLOATS + D_EROW + row];      // DECF of chunk cp was seen one iteration ago
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(bars + B_DECE + d);
                if (!tc::mbar_wait(bars + B_YF, cp & 1, abort_flag)) { ok = false; break; }
                tc::tc_fence_after();
                uint4 *dst = (uint4 *)(yb + (size_t)(t0 + row) * H * P);
                const bool valid = t0 + row < Tlen;
                uint32_t ya[32], yb2[32], yo[32];
                tc::tmem_ld32(tmem + lane_base + TM_YI, ya);
                if (cp > 0) tc::tmem_ld32(tmem + lane_base + TM_YO + (uint32_t)((cp & 1) * 64), yo);
                tc::tmem_ld_wait();
                if (cp > 0) {
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        const float2 r = __ffma2_rn(make_float2(er, er), make_float2(__uint_as_float(yo[i]), __uint_as_float(yo[i + 1])),
                                                    make_float2(__uint_as_float(ya[i]), __uint_as_float(ya[i + 1])));
                        ya[i] = __float_as_uint(r.x);
                        ya[i + 1] = __float_as_uint(r.y);
                    }
                }
                // second half in flight while the first is narrowed and stored
                tc::tmem_ld32(tmem + lane_base + TM_YI + 32, yb2);
                if (cp > 0) tc::tmem_ld32(tmem + lane_base + TM_YO + (uint32_t)((cp & 1) * 64 + 32), yo);
                if (valid) {
#pragma unroll
                    for (int ci = 0; ci < 4; ++ci)
                        dst[ci] = make_uint4(tc::pack_bf16x2(__uint_as_float(ya[8 * ci]), __uint_as_float(ya[8 * ci + 1])),
                                             tc::pack_bf16x2(__uint_as_float(ya[8 * ci + 2]), __uint_as_float(ya[8 * ci + 3])),
                                             tc::pack_bf16x2(__uint_as_float(ya[8 * ci + 4]), __uint_as_float(ya[8 * ci + 5])),
                                             tc::pack_bf16x2(__uint_as_float(ya[8 * ci + 6]), __uint_as_float(ya[8 * ci + 7])));
                }
                tc::tmem_ld_wait();
                tc::tc_fence_before();               // both accumulators are in registers
                warp_arrive(bars + B_YE, lane);
                if (cp > 0) {
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        const float2 r = __ffma2_rn(make_float2(er, er), make_float2(__uint_as_float(yo[i]), __uint_as_float(yo[i + 1])),
                                                    make_float2(__uint_as_float(yb2[i]), __uint_as_float(yb2[i + 1])));
                        yb2[i] = __float_as_uint(r.x);
                        yb2[i + 1] = __float_as_uint(r.y);
                    }
                }
                if (valid) {
#pragma unroll
                    for (int ci = 0; ci < 4; ++ci)
                        dst[4 + ci] = make_uint4(tc::pack_bf16x2(__uint_as_float(yb2[8 * ci]), __uint_as_float(yb2[8 * ci + 1])),
                                                 tc::pack_bf16x2(__uint_as_float(yb2[8 * ci + 2]), __uint_as_float(yb2[8 * ci + 3])),
                                                 tc::pack_bf16x2(__uint_as_float(yb2[8 * ci + 4]), __uint_as_float(yb2[8 * ci + 5])),
                                                 tc::pack_bf16x2(__uint_as_float(yb2[8 * ci + 6]), __uint_as_float(yb2[8 * ci + 7])));
                }
            }
        }
        if (!ok && lane == 0) atomicCAS(status, 0, STR_ERR_TIMEOUT);
    }
    tc::tc_fence_before();
    __syncthreads();
    if (warp == 13) { tc::tc_fence_after(); tc::tmem_dealloc(tmem, 512); }
}

}  // namespace

bool str_ssd_tc_supported(const str_ssd_shape *s, const void *x, const void *B, const void *C, const void *y,
                          const float *D, const float *init_state) {
    if (s->dtype != STR_BF16 || s->p != P || s->n != NS || D || init_state || s->T < 1) return false;
    return (((uintptr_t)x | (uintptr_t)B | (uintptr_t)C | (uintptr_t)y) & 15) == 0;
}

int str_ssd_tc(str_ctx *ctx, const str_ssd_shape *s, const void *x, const float *dt, const float *A, const void *B,
               const void *C, void *y, float *final_state, cudaStream_t st) {
    if (SMEM_BYTES > (size_t)ctx->max_smem_optin) return STR_ERR_UNSUPPORTED_SHAPE;
    CUtensorMap tx, tb, tcm;
    int rc = str_make_tmap_3d_bf16_sw128(ctx, &tx, x, (uint64_t)s->H * P, (uint64_t)s->T, (uint64_t)s->Bz, Q);
    if (rc == STR_OK) rc = str_make_tmap_3d_bf16_sw128(ctx, &tb, B, (uint64_t)s->G * NS, (uint64_t)s->T, (uint64_t)s->Bz, Q);
    if (rc == STR_OK) rc = str_make_tmap_3d_bf16_sw128(ctx, &tcm, C, (uint64_t)s->G * NS, (uint64_t)s->T, (uint64_t)s->Bz, Q);
    if (rc != STR_OK) return rc;
    rc = str_ensure_smem(ctx, STR_SMEM_SSD, ssd_tc_kernel, SMEM_BYTES);
    if (rc != STR_OK) return rc;
    dim3 grid(s->H, s->Bz);
    ssd_tc_kernel<<<grid, NUM_THREADS, SMEM_BYTES, st>>>(tx, tb, tcm, s->T, s->H, s->G, dt, A, (__nv_bfloat16 *)y,
                                                        final_state, ctx->status_dev);
    return str_launch_ok(ctx);
}
