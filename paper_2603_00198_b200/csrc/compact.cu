// str_compact: stable, coalesced, 16-byte-vectorised gather of the retained rows
// (hidden states, positions, index map).  Pure HBM traffic: each retained row is read once
// and written once.
#include "common.cuh"

namespace {

// One flat index space over the 16-byte vectors of the output.  Vector v belongs to output row
// v / row_vec; its source row is kept_idx[...] for the first k rows of a sequence and the text
// row for the rest.  Four independent vectors per thread keep enough loads in flight.
__global__ void __launch_bounds__(256)
compact_kernel(int Bz, int T_in, int n_vis, int n_text, int k, int row_vec,
               const uint4 *__restrict__ hidden, const int32_t *__restrict__ positions,
               const int32_t *__restrict__ idx_map, const int32_t *__restrict__ kept,
               uint4 *__restrict__ hidden_out, int32_t *__restrict__ positions_out,
               int32_t *__restrict__ idx_map_out) {
    const int T_out = k + n_text;
    const long long rows = (long long)Bz * T_out;
    const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long nthreads = (long long)gridDim.x * blockDim.x;

    if (positions_out) {
        for (long long r = tid; r < rows; r += nthreads) {
            const int b = (int)(r / T_out), j = (int)(r % T_out);
            const int src = j < k ? kept[(long long)b * k + j] : n_vis + (j - k);
            positions_out[r] = positions[(long long)b * T_in + src];
            idx_map_out[r] = idx_map[(long long)b * T_in + src];
        }
    }

    const long long total = rows * row_vec;
    for (long long v0 = tid; v0 < total; v0 += 4 * nthreads) {
        uint4 val[4];
        long long dst[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const long long v = v0 + u * nthreads;
            dst[u] = -1;
            if (v < total) {
                const long long r = v / row_vec;
                const int c = (int)(v % row_vec);
                const int b = (int)(r / T_out), j = (int)(r % T_out);
                const int src = j < k ? __ldg(kept + (long long)b * k + j) : n_vis + (j - k);
                val[u] = __ldg(hidden + ((long long)b * T_in + src) * row_vec + c);
                dst[u] = v;
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (dst[u] >= 0) hidden_out[dst[u]] = val[u];
    }
}

}  // namespace

extern "C" int str_compact(str_ctx *ctx, int Bz, int T_in, int n_vis, int n_text, int k, int D, int dtype,
                           const void *hidden, const int32_t *positions, const int32_t *idx_map,
                           const int32_t *kept_idx, void *hidden_out, int32_t *positions_out,
                           int32_t *idx_map_out, void *stream) {
    StrProfScope prof_scope(ctx, STR_CAT_COMPACT, stream);
    if (!ctx || Bz <= 0 || n_vis < 0 || n_text < 0 || k < 0 || k > n_vis || D <= 0 ||
        T_in != n_vis + n_text || (dtype != STR_F32 && dtype != STR_BF16))
        return STR_ERR_INVALID_ARG;
    const bool have_pos = positions || idx_map || positions_out || idx_map_out;
    if (have_pos && !(positions && idx_map && positions_out && idx_map_out)) return STR_ERR_INVALID_ARG;
    if (k + n_text == 0) return STR_OK;
    if (!hidden || !hidden_out || (k > 0 && !kept_idx)) return STR_ERR_INVALID_ARG;
    const size_t row_bytes = (size_t)D * dtype_size(dtype);
    if (row_bytes % 16 != 0) return STR_ERR_UNSUPPORTED_SHAPE;
    if (((uintptr_t)hidden | (uintptr_t)hidden_out) & 15) return STR_ERR_INVALID_ARG;
    const int row_vec = (int)(row_bytes / 16);
    const long long total = (long long)Bz * (k + n_text) * row_vec;
    long long want = (total + 256LL * 4 - 1) / (256LL * 4);
    const long long cap = (long long)ctx->sm_count * 8;
    int grid = (int)(want < cap ? (want < 1 ? 1 : want) : cap);
    compact_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>(
        Bz, T_in, n_vis, n_text, k, row_vec, (const uint4 *)hidden, positions, idx_map, kept_idx,
        (uint4 *)hidden_out, positions_out, idx_map_out);
    return str_launch_ok(ctx);
}
