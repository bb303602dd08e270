// FP8 (E4M3) quantisation of the tiled V tensor, one scale per (batch, head): the paper's kernel
// quantises V before the block-sparse attention (Sec. 3.4) without stating a format; this is the
// per-head symmetric reading.  Two HBM-bound passes: the head's largest magnitude, then
// code = nearest-even E4M3 of V / scale with scale = max|V| / 448 (all in fp32, saturating).
#include <cuda_fp8.h>

#include "common.cuh"

namespace fvattn {

constexpr int kQuantThreads = 256;
constexpr int kQuantVecsPerCta = 4096;   // 16-byte vectors (8 bf16 each) per CTA = 64 KB of V

__global__ void __launch_bounds__(kQuantThreads)
v_absmax_kernel(const uint4* __restrict__ v_r, int64_t vecs_per_head, unsigned int* __restrict__ amax_bits) {
    const int64_t bh = blockIdx.y;
    const uint4* v = v_r + bh * vecs_per_head;
    const int64_t v0 = (int64_t)blockIdx.x * kQuantVecsPerCta;
    const int64_t v1 = min(v0 + kQuantVecsPerCta, vecs_per_head);
    float m = 0.f;
    for (int64_t i = v0 + threadIdx.x; i < v1; i += kQuantThreads) {
        const uint4 raw = __ldg(v + i);
        const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 f = __bfloat1622float2(h2[e]);
            m = fmaxf(m, fmaxf(fabsf(f.x), fabsf(f.y)));
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    // non-negative floats order like their bit patterns
    if ((threadIdx.x & 31) == 0 && m > 0.f) atomicMax(amax_bits + bh, __float_as_uint(m));
}

__global__ void __launch_bounds__(kQuantThreads)
v_quantize_kernel(const uint4* __restrict__ v_r, int64_t vecs_per_head, const unsigned int* __restrict__ amax_bits,
                  uint2* __restrict__ v8, float* __restrict__ v_scale) {
    const int64_t bh = blockIdx.y;
    const float amax = __uint_as_float(amax_bits[bh]);
    const float sc = amax > 0.f ? __fdiv_rn(amax, 448.0f) : 1.0f;
    if (blockIdx.x == 0 && threadIdx.x == 0) v_scale[bh] = sc;
    const uint4* v = v_r + bh * vecs_per_head;
    uint2* out = v8 + bh * vecs_per_head;
    const int64_t v0 = (int64_t)blockIdx.x * kQuantVecsPerCta;
    const int64_t v1 = min(v0 + kQuantVecsPerCta, vecs_per_head);
    for (int64_t i = v0 + threadIdx.x; i < v1; i += kQuantThreads) {
        const uint4 raw = __ldg(v + i);
        const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
        unsigned short q[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 f = __bfloat1622float2(h2[e]);
            q[e] = __nv_cvt_float2_to_fp8x2(make_float2(__fdiv_rn(f.x, sc), __fdiv_rn(f.y, sc)), __NV_SATFINITE, __NV_E4M3);
        }
        out[i] = make_uint2((uint32_t)q[0] | ((uint32_t)q[1] << 16), (uint32_t)q[2] | ((uint32_t)q[3] << 16));
    }
}

fvattn_status_t launch_quantize_v(const void* v_r, int64_t BH, int64_t elems_per_head, void* v8, float* v_scale,
                                  unsigned int* amax_bits, cudaStream_t s) {
    const int64_t vecs = elems_per_head / 8;
    const unsigned ctas = (unsigned)((vecs + kQuantVecsPerCta - 1) / kQuantVecsPerCta);
    FVATTN_CUDA_OK(cudaMemsetAsync(amax_bits, 0, sizeof(unsigned int) * (size_t)BH, s));
    v_absmax_kernel<<<dim3(ctas, (unsigned)BH), kQuantThreads, 0, s>>>((const uint4*)v_r, vecs, amax_bits);
    if (launch_status() != FVATTN_OK) return FVATTN_ERR_CUDA;
    v_quantize_kernel<<<dim3(ctas, (unsigned)BH), kQuantThreads, 0, s>>>((const uint4*)v_r, vecs, amax_bits, (uint2*)v8,
                                                                          v_scale);
    return launch_status();
}

} // namespace fvattn
