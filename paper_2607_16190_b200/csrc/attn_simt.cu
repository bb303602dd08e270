// Block-sparse attention on CUDA cores (Sec. 2.1: only the retained (query block, key block)
// pairs are evaluated).  This is the plain kernel for the block/head sizes the tensor-core
// kernel does not cover (Bs or d = 64) and an on-GPU cross-check for it.  One CTA per
// (head, query block) tile, taken from the heaviest-first order; per retained key block:
// S = Q K^T in fp32, online softmax (running max / sum per row), O = O * corr + P V.
#include "common.cuh"

namespace fvattn {

constexpr int kSimtThreads = 256;

template <int BS, int D>
struct SimtSmem {
    static constexpr int LD = D + 2;   // bf16 elements per staged row (odd number of words: no bank conflicts)
    static constexpr int LS = BS + 1;  // floats per score row
    static constexpr size_t bytes = sizeof(__nv_bfloat16) * 3 * BS * LD + sizeof(float) * (BS * LS + 3 * BS) +
                                    sizeof(int) * BS;
};

template <int BS, int D>
__device__ __forceinline__ void stage_tile(__nv_bfloat16* dst, const __nv_bfloat16* src) {
    // src: BS rows of D contiguous bf16 (16-byte aligned); dst rows are LD apart (4-byte aligned)
    constexpr int LD = SimtSmem<BS, D>::LD;
    constexpr int VPR = D / 8;
    for (int it = threadIdx.x; it < BS * VPR; it += kSimtThreads) {
        int r = it / VPR, v = it - r * VPR;
        uint4 raw = __ldg(reinterpret_cast<const uint4*>(src) + it);
        uint32_t* d32 = reinterpret_cast<uint32_t*>(dst + r * LD + v * 8);
        d32[0] = raw.x; d32[1] = raw.y; d32[2] = raw.z; d32[3] = raw.w;
    }
}

template <int BS, int D>
__global__ void __launch_bounds__(kSimtThreads)
attn_simt_kernel(const __nv_bfloat16* __restrict__ q_r, const __nv_bfloat16* __restrict__ k_r,
                 const __nv_bfloat16* __restrict__ v_r, const uint16_t* __restrict__ idx,
                 const int32_t* __restrict__ counts, GridDims m, float sm_scale, __nv_bfloat16* __restrict__ o_r,
                 const uint32_t* __restrict__ order, void* workspace) {
    using L = SimtSmem<BS, D>;
    constexpr int LD = L::LD, LS = L::LS;
    constexpr int RB = BS / 16;   // S rows / O rows per thread
    constexpr int CB = BS / 16;   // S columns per thread
    constexpr int DB = D / 16;    // O columns per thread
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __nv_bfloat16* Qs = reinterpret_cast<__nv_bfloat16*>(smem_raw);
    __nv_bfloat16* Ks = Qs + BS * LD;
    __nv_bfloat16* Vs = Ks + BS * LD;
    float* Ss = reinterpret_cast<float*>(Vs + BS * LD);
    float* row_m = Ss + BS * LS;
    float* row_l = row_m + BS;
    float* row_corr = row_l + BS;
    int* kvalid = reinterpret_cast<int*>(row_corr + BS);

    const uint32_t tile = order[blockIdx.x];
    const int64_t bh = tile / (uint32_t)m.nb;
    const int i = (int)(tile % (uint32_t)m.nb);
    const int tid = threadIdx.x;
    const int tx = tid % 16, ty = tid / 16;
    const int c = min(max(counts[tile], 0), m.nb);
    const uint16_t* irow = idx + (int64_t)tile * m.nb;
    const int64_t head_base = bh * m.n_pad * D;

    stage_tile<BS, D>(Qs, q_r + head_base + (int64_t)i * BS * D);
    if (tid < BS) {
        row_m[tid] = -INFINITY;
        row_l[tid] = 0.f;
    }
    float o[RB][DB];
#pragma unroll
    for (int a = 0; a < RB; ++a)
#pragma unroll
        for (int b = 0; b < DB; ++b) o[a][b] = 0.f;
    __syncthreads();

    for (int t = 0; t < c; ++t) {
        const int kb = irow[t];
        if (kb >= m.nb) {   // uniform across the CTA: everyone reads the same entry
            if (tid == 0) report_error(workspace, FVATTN_ERR_DEVICE_BOUNDS, tile);
            break;
        }
        stage_tile<BS, D>(Ks, k_r + head_base + (int64_t)kb * BS * D);
        stage_tile<BS, D>(Vs, v_r + head_base + (int64_t)kb * BS * D);
        if (tid < BS) {
            int64_t token;
            kvalid[tid] = row_to_token(m, kb, tid, &token) ? 1 : 0;
        }
        __syncthreads();

        // S = sm_scale * Q K^T ; thread owns rows ty + 16a, columns tx + 16b
        float acc[RB][CB];
#pragma unroll
        for (int a = 0; a < RB; ++a)
#pragma unroll
            for (int b = 0; b < CB; ++b) acc[a][b] = 0.f;
        for (int c2 = 0; c2 < D; c2 += 2) {
            float2 qv[RB], kv[CB];
#pragma unroll
            for (int a = 0; a < RB; ++a)
                qv[a] = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(Qs + (ty + 16 * a) * LD + c2));
#pragma unroll
            for (int b = 0; b < CB; ++b)
                kv[b] = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(Ks + (tx + 16 * b) * LD + c2));
#pragma unroll
            for (int a = 0; a < RB; ++a)
#pragma unroll
                for (int b = 0; b < CB; ++b) acc[a][b] = fmaf(qv[a].y, kv[b].y, fmaf(qv[a].x, kv[b].x, acc[a][b]));
        }
#pragma unroll
        for (int a = 0; a < RB; ++a)
#pragma unroll
            for (int b = 0; b < CB; ++b)
                Ss[(ty + 16 * a) * LS + tx + 16 * b] = kvalid[tx + 16 * b] ? sm_scale * acc[a][b] : -INFINITY;
        __syncthreads();

        // online softmax, one thread per query row
        if (tid < BS) {
            float* srow = Ss + tid * LS;
            float mo = row_m[tid], mn = mo;
            for (int j = 0; j < BS; ++j) mn = fmaxf(mn, srow[j]);
            float sum = 0.f;
            if (mn == -INFINITY) {
                for (int j = 0; j < BS; ++j) srow[j] = 0.f;
                row_corr[tid] = 1.f;
            } else {
                for (int j = 0; j < BS; ++j) {
                    float pj = expf(srow[j] - mn);
                    srow[j] = pj;
                    sum += pj;
                }
                float corr = (mo == -INFINITY) ? 0.f : expf(mo - mn);
                row_corr[tid] = corr;
                row_l[tid] = row_l[tid] * corr + sum;
                row_m[tid] = mn;
            }
        }
        __syncthreads();

        // O = O * corr + P V ; thread owns rows ty + 16a, columns tx + 16b of d
#pragma unroll
        for (int a = 0; a < RB; ++a) {
            float corr = row_corr[ty + 16 * a];
#pragma unroll
            for (int b = 0; b < DB; ++b) o[a][b] *= corr;
        }
        for (int j = 0; j < BS; ++j) {
            float pv[RB], vv[DB];
#pragma unroll
            for (int a = 0; a < RB; ++a) pv[a] = Ss[(ty + 16 * a) * LS + j];
#pragma unroll
            for (int b = 0; b < DB; ++b) vv[b] = __bfloat162float(Vs[j * LD + tx + 16 * b]);
#pragma unroll
            for (int a = 0; a < RB; ++a)
#pragma unroll
                for (int b = 0; b < DB; ++b) o[a][b] = fmaf(pv[a], vv[b], o[a][b]);
        }
        __syncthreads();
    }

    // normalise and store; padding query rows and rows with no valid key give 0
#pragma unroll
    for (int a = 0; a < RB; ++a) {
        int r = ty + 16 * a;
        int64_t token;
        bool qvalid = row_to_token(m, i, r, &token);
        float l = row_l[r];
        float inv = (qvalid && l > 0.f) ? 1.f / l : 0.f;
        __nv_bfloat16* orow = o_r + head_base + ((int64_t)i * BS + r) * D;
#pragma unroll
        for (int b = 0; b < DB; ++b) orow[tx + 16 * b] = __float2bfloat16(o[a][b] * inv);
    }
}

template <int BS, int D>
static fvattn_status_t launch_one(const void* q_r, const void* k_r, const void* v_r, const uint16_t* idx,
                                  const int32_t* counts, int64_t BH, const GridDims& m, float sm_scale, void* o_r,
                                  const uint32_t* order, void* workspace, cudaStream_t s) {
    auto kern = attn_simt_kernel<BS, D>;
    size_t smem = SimtSmem<BS, D>::bytes;
    FVATTN_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    kern<<<(unsigned)(BH * m.nb), kSimtThreads, smem, s>>>(
        (const __nv_bfloat16*)q_r, (const __nv_bfloat16*)k_r, (const __nv_bfloat16*)v_r, idx, counts, m, sm_scale,
        (__nv_bfloat16*)o_r, order, workspace);
    return launch_status();
}

fvattn_status_t launch_attn_simt(const void* q_r, const void* k_r, const void* v_r, const uint16_t* idx,
                                 const int32_t* counts, int64_t BH, int d, const GridDims& m, float sm_scale,
                                 void* o_r, const uint32_t* order, void* workspace, cudaStream_t s) {
#define FVATTN_SIMT_CASE(BS_, D_) \
    if (m.bs == BS_ && d == D_)   \
        return launch_one<BS_, D_>(q_r, k_r, v_r, idx, counts, BH, m, sm_scale, o_r, order, workspace, s);
    FVATTN_SIMT_CASE(64, 64)
    FVATTN_SIMT_CASE(64, 128)
    FVATTN_SIMT_CASE(128, 64)
    FVATTN_SIMT_CASE(128, 128)
#undef FVATTN_SIMT_CASE
    return FVATTN_ERR_UNSUPPORTED_SHAPE;
}

} // namespace fvattn
