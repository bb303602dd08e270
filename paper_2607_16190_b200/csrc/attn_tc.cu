// Block-sparse attention on the sm_100a tensor cores (Sec. 2.1: only the retained
// (query block, key block) pairs are evaluated), Bs = d = 128, bf16 in, fp32 accumulate.
//
// Persistent CTAs pop (head, query-block) tiles from an atomic queue in heaviest-first order.
// Per tile: Q (128 x 128) is TMA-loaded once; for every retained key block the K and V tiles
// are TMA-loaded by index (each is one contiguous 128 x 128 tile of the head-major layout),
// S = Q K^T and O += P V run as tcgen05 MMAs with the accumulators in tensor memory, and the
// online softmax (running max and sum per query row, fp32, base-2 exponentials) runs one
// thread per query row on the S tile read back from tensor memory.  P is written back to
// tensor memory as bf16 and fed to the second MMA as its A operand.  Padded keys of edge
// blocks are masked to -inf; padded query rows are written as zero.
//
// Shared-memory tiles use the 128-byte swizzle: a 128 x 128 bf16 tile is two TMA boxes of
// 128 rows x 64 columns (16 KB each).  Q and K are K-major MMA operands; V (keys x d, d
// contiguous) is the MN-major B operand of the second MMA.
//
// Every wait on an mbarrier is bounded; when one runs out the CTA records
// FVATTN_ERR_DEVICE_TIMEOUT in the workspace, stops taking tiles, frees its tensor memory
// and returns.
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace fvattn {

using namespace ptx;

namespace tc {
constexpr int BS = 128;
constexpr int D = 128;
constexpr int kThreads = 128;
constexpr uint32_t kHalfBytes = 128 * 64 * 2;      // one TMA box: 128 rows x 64 bf16
constexpr uint32_t kTileBytes = 2 * kHalfBytes;    // 128 x 128 bf16
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColS = 0;      // S accumulator, 128 fp32 columns
constexpr uint32_t kColO = 128;    // O accumulator, 128 fp32 columns
constexpr uint32_t kColP = 256;    // P operand, 128 bf16 = 64 columns
constexpr float kLog2e = 1.4426950408889634f;

struct __align__(1024) Smem {
    unsigned char q[kTileBytes];
    unsigned char k[kTileBytes];
    unsigned char v[kTileBytes];
    unsigned char pad_to_one_cta_per_sm[24 * 1024];   // > half of the SM's shared memory in total
    unsigned long long bar_q, bar_kv, bar_s, bar_o;
    uint32_t tmem_base;
    uint32_t kmask[4];
    int tile;
    int abort_flag;
};
} // namespace tc

__global__ void __launch_bounds__(tc::kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
               const __grid_constant__ CUtensorMap map_v, const uint16_t* __restrict__ idx,
               const int32_t* __restrict__ counts, GridDims m, float sm_scale, __nv_bfloat16* __restrict__ o_r,
               const uint32_t* __restrict__ order, int n_tiles, void* workspace) {
    using namespace tc;
    extern __shared__ unsigned char smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    WsHeader* hdr = reinterpret_cast<WsHeader*>(workspace);

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const uint32_t bar_q = smem_u32(&sm.bar_q), bar_kv = smem_u32(&sm.bar_kv), bar_s = smem_u32(&sm.bar_s),
                   bar_o = smem_u32(&sm.bar_o);
    const uint32_t sq = smem_u32(sm.q), sk = smem_u32(sm.k), sv = smem_u32(sm.v);

    if (tid == 0) {
        mbar_init(bar_q, 1);
        mbar_init(bar_kv, 1);
        mbar_init(bar_s, 1);
        mbar_init(bar_o, 1);
        sm.abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&map_q);
        prefetch_tensormap(&map_k);
        prefetch_tensormap(&map_v);
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&sm.tmem_base), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;
    const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);   // this warp's 32 lanes

    constexpr uint32_t idesc_qk = make_idesc_bf16(128, 128, false);
    constexpr uint32_t idesc_pv = make_idesc_bf16(128, 128, true);
    const float sl2 = sm_scale * kLog2e;
    uint32_t ph_q = 0, ph_kv = 0, ph_s = 0, ph_o = 0;
    volatile int* abort_flag = &sm.abort_flag;
    bool alive = true;

    while (alive) {
        if (tid == 0) sm.tile = (int)atomicAdd(&hdr->tile_counter, 1u);
        tc_fence_before();
        __syncthreads();   // also: every thread is done with the previous tile's TMEM and smem
        tc_fence_after();
        const int slot = sm.tile;
        __syncthreads();   // everyone holds its copy before thread 0 may overwrite it
        if (slot >= n_tiles) break;
        const uint32_t tile = order[slot];
        const int64_t bh = tile / (uint32_t)m.nb;
        const int i = (int)(tile % (uint32_t)m.nb);
        const int c = min(max(counts[tile], 0), m.nb);
        const uint16_t* irow = idx + (int64_t)tile * m.nb;
        const int64_t head_row0 = bh * m.n_pad;

        if (tid == 0 && c > 0) {
            mbar_expect_tx(bar_q, kTileBytes);
            tma_load_2d(sq, &map_q, 0, (int)(head_row0 + (int64_t)i * BS), bar_q);
            tma_load_2d(sq + kHalfBytes, &map_q, 64, (int)(head_row0 + (int64_t)i * BS), bar_q);
        }
        float m_run = -INFINITY, l_run = 0.f;

        for (int t = 0; t < c; ++t) {
            const int kb = irow[t];
            if (kb >= m.nb) {   // same value in every thread
                if (tid == 0) report_error(workspace, FVATTN_ERR_DEVICE_BOUNDS, tile);
                if (t == 0 && tid == 0) (void)mbar_wait(bar_q, ph_q, abort_flag);   // drain the Q copy in flight
                if (t == 0) { ph_q ^= 1; l_run = 0.f; }
                break;
            }
            const bool edge = block_valid_tokens(m, kb) != BS;
            if (edge) {
                int64_t token;
                unsigned int bal = __ballot_sync(0xffffffffu, row_to_token(m, kb, tid, &token));
                if (lane == 0) sm.kmask[warp] = bal;
            }
            bool ok = true;
            if (tid == 0) {
                mbar_expect_tx(bar_kv, 2 * kTileBytes);
                const int krow = (int)(head_row0 + (int64_t)kb * BS);
                tma_load_2d(sk, &map_k, 0, krow, bar_kv);
                tma_load_2d(sk + kHalfBytes, &map_k, 64, krow, bar_kv);
                tma_load_2d(sv, &map_v, 0, krow, bar_kv);
                tma_load_2d(sv + kHalfBytes, &map_v, 64, krow, bar_kv);
                if (t == 0) ok = mbar_wait(bar_q, ph_q, abort_flag);
                ok = ok && mbar_wait(bar_kv, ph_kv, abort_flag);
                if (ok) {
                    tc_fence_after();
                    // S = Q K^T : 8 steps of K = 16 over d = 128; both operands K-major
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks) {
                        uint32_t off = (uint32_t)(ks >> 2) * kHalfBytes + (uint32_t)(ks & 3) * 32u;
                        umma_ss(tmem + kColS, make_smem_desc_sw128(sq + off, 16, 1024),
                                make_smem_desc_sw128(sk + off, 16, 1024), idesc_qk, ks > 0 ? 1u : 0u);
                    }
                    umma_commit(bar_s);
                } else {
                    *abort_flag = 1;
                }
            }
            if (t == 0) ph_q ^= 1;
            ph_kv ^= 1;
            ok = mbar_wait(bar_s, ph_s, abort_flag);
            ph_s ^= 1;
            if (!__syncthreads_and(ok ? 1 : 0)) { alive = false; break; }
            tc_fence_after();

            // ---- online softmax on row `tid` of S -------------------------------------------
            uint32_t r[32];
            float mx = m_run;
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
                tmem_ld32(lane_addr + kColS + ch * 32, r);
                tmem_wait_ld();
                const uint32_t km = edge ? sm.kmask[ch] : 0xffffffffu;
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    if ((km >> j) & 1u) mx = fmaxf(mx, __uint_as_float(r[j]));
            }
            // mx == -inf only if no valid key so far: exponent offset 0 keeps everything finite
            const float moff = (mx == -INFINITY) ? 0.f : mx * sl2;
            float sum = 0.f;
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
                tmem_ld32(lane_addr + kColS + ch * 32, r);
                tmem_wait_ld();
                const uint32_t km = edge ? sm.kmask[ch] : 0xffffffffu;
                uint32_t packed[16];
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                    float p0 = ((km >> j) & 1u) ? exp2f(fmaf(__uint_as_float(r[j]), sl2, -moff)) : 0.f;
                    float p1 = ((km >> (j + 1)) & 1u) ? exp2f(fmaf(__uint_as_float(r[j + 1]), sl2, -moff)) : 0.f;
                    __nv_bfloat162 b2 = __floats2bfloat162_rn(p0, p1);   // .x (low half) = even column
                    // the row sum uses the rounded values that the second MMA will see
                    float2 back = __bfloat1622float2(b2);
                    sum += back.x + back.y;
                    packed[j >> 1] = *reinterpret_cast<uint32_t*>(&b2);
                }
                tmem_st16(lane_addr + kColP + ch * 16, packed);
            }
            const float corr = (m_run == -INFINITY) ? 0.f : exp2f(m_run * sl2 - moff);
            l_run = l_run * corr + sum;
            m_run = mx;
            if (t > 0 && __any_sync(0xffffffffu, corr != 1.f)) {   // rescale the running O
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    tmem_ld32(lane_addr + kColO + ch * 32, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * corr);
                    tmem_st32(lane_addr + kColO + ch * 32, r);
                }
            }
            tmem_wait_st();
            tc_fence_before();
            __syncthreads();

            // ---- O (+)= P V : 8 steps of K = 16 keys; A = P from tensor memory, B = V MN-major ---
            if (tid == 0) {
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < BS / 16; ++ks)
                    umma_ts(tmem + kColO, tmem + kColP + ks * 8,
                            make_smem_desc_sw128(sv + (uint32_t)ks * 2048u, kHalfBytes, 1024), idesc_pv,
                            (t > 0 || ks > 0) ? 1u : 0u);
                umma_commit(bar_o);
            }
            ok = mbar_wait(bar_o, ph_o, abort_flag);
            ph_o ^= 1;
            if (!__syncthreads_and(ok ? 1 : 0)) { alive = false; break; }
            tc_fence_after();
        }
        if (!alive) break;

        // ---- epilogue: O / l -> bf16 -> global; padded query rows and empty rows give 0 --------
        {
            int64_t token;
            const bool qvalid = row_to_token(m, i, tid, &token);
            const float inv = (qvalid && l_run > 0.f) ? 1.f / l_run : 0.f;
            uint4* orow = reinterpret_cast<uint4*>(o_r + (head_row0 + (int64_t)i * BS + tid) * D);
            uint32_t r[32];
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
                if (l_run > 0.f || c > 0) {   // c is CTA-uniform: the load below is warp-uniform
                    tmem_ld32(lane_addr + kColO + ch * 32, r);
                    tmem_wait_ld();
                }
                uint32_t outw[16];
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                    float a = inv != 0.f ? __uint_as_float(r[j]) * inv : 0.f;
                    float b = inv != 0.f ? __uint_as_float(r[j + 1]) * inv : 0.f;
                    __nv_bfloat162 b2 = __floats2bfloat162_rn(a, b);
                    outw[j >> 1] = *reinterpret_cast<uint32_t*>(&b2);
                }
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4)
                    orow[ch * 4 + q4] = make_uint4(outw[q4 * 4], outw[q4 * 4 + 1], outw[q4 * 4 + 2], outw[q4 * 4 + 3]);
            }
        }
    }

    if (!alive && tid == 0) report_error(workspace, FVATTN_ERR_DEVICE_TIMEOUT, blockIdx.x);
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

// ---- host side ------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        else
            (void)cudaGetLastError();
    }
    return fn;
}

// [rows, 128] bf16 row-major tensor, box = 128 rows x 64 columns, 128-byte swizzle.
static bool make_tile_map(CUtensorMap* map, const void* base, uint64_t rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)tc::D, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)tc::D * 2};
    cuuint32_t box[2] = {64, 128};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

fvattn_status_t launch_attn_tc(const void* q_r, const void* k_r, const void* v_r, const uint16_t* idx,
                               const int32_t* counts, int64_t BH, const GridDims& m, float sm_scale, void* o_r,
                               const uint32_t* order, void* workspace, cudaStream_t s) {
    const uint64_t rows = (uint64_t)BH * (uint64_t)m.n_pad;
    if (rows > 0x7fffffffull) return FVATTN_ERR_UNSUPPORTED_SHAPE;   // TMA coordinates are 32-bit
    CUtensorMap mq, mk, mv;
    if (!make_tile_map(&mq, q_r, rows) || !make_tile_map(&mk, k_r, rows) || !make_tile_map(&mv, v_r, rows))
        return FVATTN_ERR_CUDA;
    int dev = 0, sms = 0;
    FVATTN_CUDA_OK(cudaGetDevice(&dev));
    FVATTN_CUDA_OK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const size_t smem = sizeof(tc::Smem) + 1024;
    FVATTN_CUDA_OK(cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const int n_tiles = (int)(BH * m.nb);
    const int grid = n_tiles < sms ? n_tiles : sms;
    attn_tc_kernel<<<grid, tc::kThreads, smem, s>>>(mq, mk, mv, idx, counts, m, sm_scale, (__nv_bfloat16*)o_r, order,
                                                   n_tiles, workspace);
    return launch_status();
}

} // namespace fvattn
