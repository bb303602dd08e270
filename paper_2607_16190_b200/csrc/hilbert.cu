// Hilbert-curve block organisation (Sec. 3.1: tokens are reordered along a Hilbert curve so that
// spatially adjacent tokens fall into nearby blocks).  Host code: the curve position of every cell
// of the (T, Y, X) grid is its index on the 3-D Hilbert curve of the enclosing power-of-two cube
// (coordinates -> index by the transpose method: undo the excess rotations bit plane by bit plane,
// Gray-encode, interleave), and the grid's tokens are ranked by that index.  Blocks are Bs
// consecutive tokens along the curve; only the last block can have padding rows.
#include <algorithm>
#include <vector>

#include "common.cuh"

namespace {

// Index of cell (c0, c1, c2) on the Hilbert curve of a cube with `bits` bits per axis.
uint64_t hilbert_index(uint32_t c0, uint32_t c1, uint32_t c2, int bits) {
    uint32_t x[3] = {c0, c1, c2};
    const uint32_t top = 1u << (bits - 1);
    for (uint32_t q = top; q > 1; q >>= 1) {          // undo the rotations, high plane to low
        const uint32_t p = q - 1;
        for (int i = 0; i < 3; ++i) {
            if (x[i] & q) {
                x[0] ^= p;
            } else {
                const uint32_t t = (x[0] ^ x[i]) & p;
                x[0] ^= t;
                x[i] ^= t;
            }
        }
    }
    for (int i = 1; i < 3; ++i) x[i] ^= x[i - 1];     // Gray encode
    uint32_t t = 0;
    for (uint32_t q = top; q > 1; q >>= 1)
        if (x[2] & q) t ^= q - 1;
    for (int i = 0; i < 3; ++i) x[i] ^= t;
    uint64_t h = 0;                                   // interleave: axis 0 holds the most significant bit
    for (int b = bits - 1; b >= 0; --b)
        for (int i = 0; i < 3; ++i) h = (h << 1) | ((x[i] >> b) & 1u);
    return h;
}

} // namespace

extern "C" fvattn_status_t fvattn_hilbert_row_tokens(int32_t T, int32_t Y, int32_t X, int32_t block_tokens,
                                                     int32_t* row_token, int64_t n_rows) {
    if (!row_token || T <= 0 || Y <= 0 || X <= 0 || block_tokens <= 0) return FVATTN_ERR_INVALID_ARG;
    const int64_t n = (int64_t)T * Y * X;
    if (n > 0x7fffffffLL) return FVATTN_ERR_UNSUPPORTED_SHAPE;
    const int64_t need = (n + block_tokens - 1) / block_tokens * block_tokens;
    if (n_rows != need) return FVATTN_ERR_INVALID_ARG;
    int bits = 1;
    while ((1 << bits) < std::max(T, std::max(Y, X))) ++bits;
    std::vector<std::pair<uint64_t, int32_t>> keyed((size_t)n);
    for (int32_t t = 0; t < T; ++t)
        for (int32_t y = 0; y < Y; ++y)
            for (int32_t x = 0; x < X; ++x) {
                const int64_t tok = ((int64_t)t * Y + y) * X + x;
                keyed[(size_t)tok] = {hilbert_index((uint32_t)t, (uint32_t)y, (uint32_t)x, bits), (int32_t)tok};
            }
    std::sort(keyed.begin(), keyed.end());
    for (int64_t r = 0; r < n; ++r) row_token[r] = keyed[(size_t)r].second;
    for (int64_t r = n; r < n_rows; ++r) row_token[r] = -1;
    return FVATTN_OK;
}
