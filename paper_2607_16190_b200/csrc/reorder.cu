// Video-aware block reorder and its inverse (Sec. 3.1, 3-D tile reading): pure data movement,
// HBM-bound.  One CTA moves one block (Bs rows) of a chunk of heads with 16-byte vectors.
// For a fixed token the heads are adjacent in the caller's layout, so consecutive threads
// walk (head, vector) and the token side of every copy is one contiguous run of
// heads*d*2 bytes; the tiled side is a 2*d-byte row per (head, row).
#include "common.cuh"

namespace fvattn {

constexpr int kReorderThreads = 256;
constexpr int kHeadChunk = 8;

template <bool kInverse>
__global__ void __launch_bounds__(kReorderThreads)
reorder_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, GridDims m, int H, int vec_per_row,
               int64_t sb, int64_t sn, int64_t sh /* strides of the token layout in 16-byte vectors */) {
    const int blk = blockIdx.x;
    const int h0 = blockIdx.y * kHeadChunk;
    const int hc = min(kHeadChunk, H - h0);
    const int b = blockIdx.z;
    const int per_row = hc * vec_per_row;
    const int items = m.bs * per_row;
    const int64_t tiled_row_vecs = vec_per_row;
    for (int it = threadIdx.x; it < items; it += kReorderThreads) {
        int o = it / per_row;
        int rem = it - o * per_row;
        int hl = rem / vec_per_row;
        int v = rem - hl * vec_per_row;
        int64_t token;
        bool valid = row_to_token(m, blk, o, &token);
        int h = h0 + hl;
        int64_t tiled = (((int64_t)b * H + h) * m.n_pad + (int64_t)blk * m.bs + o) * tiled_row_vecs + v;
        int64_t tok = b * sb + token * sn + h * sh + v;
        if (!kInverse) {
            uint4 val = make_uint4(0u, 0u, 0u, 0u);
            if (valid) val = __ldg(src + tok);
            dst[tiled] = val;
        } else {
            if (valid) dst[tok] = __ldg(src + tiled);
        }
    }
}

static fvattn_status_t launch_any(bool inverse, const void* src, void* dst, const fvattn_tok_layout_t& lay,
                                  const GridDims& m, cudaStream_t s) {
    int vec_per_row = lay.d / 8;
    dim3 grid((unsigned)m.nb, (unsigned)((lay.H + kHeadChunk - 1) / kHeadChunk), (unsigned)lay.B);
    if (inverse)
        reorder_kernel<true><<<grid, kReorderThreads, 0, s>>>((const uint4*)src, (uint4*)dst, m, lay.H, vec_per_row,
                                                              lay.stride_b / 8, lay.stride_n / 8, lay.stride_h / 8);
    else
        reorder_kernel<false><<<grid, kReorderThreads, 0, s>>>((const uint4*)src, (uint4*)dst, m, lay.H, vec_per_row,
                                                               lay.stride_b / 8, lay.stride_n / 8, lay.stride_h / 8);
    return launch_status();
}

fvattn_status_t launch_reorder(const void* src, const fvattn_tok_layout_t& lay, const GridDims& m, void* dst_r,
                               cudaStream_t s) {
    return launch_any(false, src, dst_r, lay, m, s);
}

fvattn_status_t launch_inverse_reorder(const void* src_r, const GridDims& m, void* dst,
                                       const fvattn_tok_layout_t& lay, cudaStream_t s) {
    return launch_any(true, src_r, dst, lay, m, s);
}

} // namespace fvattn
