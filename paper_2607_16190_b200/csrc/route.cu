// Top-p block routing with a Top-k floor (Sec. 2.1, Sec. 3.1, Eq. 1).
//
//   pool_kernel    block means of Q and K over valid rows            HBM-bound: reads Q, K once
//   score_kernel   s = sm_scale * qbar kbar^T per head, fp32 FFMA    small fp32 GEMM, L2-resident
//   select_kernel  per (head, query block): softmax, sort by (score desc, index asc),
//                  prefix-sum mass cut at p, floor, bit mask + counts + compact index list
//   head_load_kernel  L_h = mean_i counts (Eq. 1)
//
// All arithmetic that decides the mask is fp32 with fp32 accumulation in a fixed order
// (no tensor cores, no fast-math), so the mask is reproducible run to run and differs from
// an fp64 evaluation only on rows whose cumulative mass sits within rounding of p.
#include "common.cuh"

namespace fvattn {

// ------------------------------------------------------------------------------------ pool
constexpr int kPoolThreads = 256;

template <int D>
__global__ void __launch_bounds__(kPoolThreads)
pool_kernel(const uint4* __restrict__ q_r, const uint4* __restrict__ k_r, float* __restrict__ qbar,
            float* __restrict__ kbar, GridDims m) {
    constexpr int VPR = D / 8;                // 16-byte vectors per row
    constexpr int RG = kPoolThreads / VPR;    // rows in flight per pass
    __shared__ float partial[RG][D];

    const int blk = blockIdx.x;
    const int64_t bh = blockIdx.y;
    const uint4* x = (blockIdx.z == 0 ? q_r : k_r) + (bh * m.n_pad + (int64_t)blk * m.bs) * VPR;
    float* out = (blockIdx.z == 0 ? qbar : kbar) + (bh * m.nb + blk) * D;

    const int v = threadIdx.x % VPR;
    const int rg = threadIdx.x / VPR;
    const bool full = block_valid_tokens(m, blk) == m.bs;   // no padding rows in this block
    // issue every load of this thread before the first add: 8 x 16 B in flight per thread
    constexpr int kPasses = 8;
    uint4 raw[kPasses];
#pragma unroll
    for (int it = 0; it < kPasses; ++it) {
        const int o = rg + it * RG;
        int64_t token;
        const bool take = o < m.bs && (full || row_to_token(m, blk, o, &token));   // padding rows take no part
        raw[it] = take ? __ldg(x + (int64_t)o * VPR + v) : make_uint4(0u, 0u, 0u, 0u);
    }
    float acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.f;
#pragma unroll
    for (int it = 0; it < kPasses; ++it) {
        const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&raw[it]);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            float2 f = __bfloat1622float2(h2[e]);
            acc[2 * e] += f.x;
            acc[2 * e + 1] += f.y;
        }
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) partial[rg][v * 8 + e] = acc[e];
    __syncthreads();
    if (threadIdx.x < D) {
        float s = 0.f;
#pragma unroll
        for (int g = 0; g < RG; ++g) s += partial[g][threadIdx.x];
        out[threadIdx.x] = s / (float)block_valid_tokens(m, blk);
    }
}

// ----------------------------------------------------------------------------------- scores
constexpr int kScoreTile = 64;
constexpr int kScoreK = 32;

__global__ void __launch_bounds__(256)
score_kernel(const float* __restrict__ qbar, const float* __restrict__ kbar, float* __restrict__ scores, int nb,
             int d, int score_stride, float sm_scale) {
    __shared__ __align__(16) float As[kScoreK][kScoreTile + 4];
    __shared__ __align__(16) float Bs[kScoreK][kScoreTile + 4];
    const int64_t bh = blockIdx.z;
    const int i0 = blockIdx.y * kScoreTile, j0 = blockIdx.x * kScoreTile;
    const float* A = qbar + bh * (int64_t)nb * d;
    const float* Bm = kbar + bh * (int64_t)nb * d;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    float acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;

    for (int k0 = 0; k0 < d; k0 += kScoreK) {
        // 64 rows x 32 k per operand; thread -> (row = t / 8 + 32 * r, 4 consecutive k)
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            int row = threadIdx.x / 8 + 32 * r;
            int kk = (threadIdx.x % 8) * 4;
            float4 va = make_float4(0.f, 0.f, 0.f, 0.f), vb = va;
            if (i0 + row < nb) va = *reinterpret_cast<const float4*>(A + (int64_t)(i0 + row) * d + k0 + kk);
            if (j0 + row < nb) vb = *reinterpret_cast<const float4*>(Bm + (int64_t)(j0 + row) * d + k0 + kk);
            As[kk + 0][row] = va.x; As[kk + 1][row] = va.y; As[kk + 2][row] = va.z; As[kk + 3][row] = va.w;
            Bs[kk + 0][row] = vb.x; Bs[kk + 1][row] = vb.y; Bs[kk + 2][row] = vb.z; Bs[kk + 3][row] = vb.w;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < kScoreK; ++kk) {
            float4 a4 = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
            float4 b4 = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
            float av[4] = {a4.x, a4.y, a4.z, a4.w};
            float bv[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(av[a], bv[b], acc[a][b]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        int i = i0 + ty * 4 + a;
        if (i >= nb) continue;
        float* out = scores + (bh * nb + i) * (int64_t)score_stride;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            int j = j0 + tx * 4 + b;
            if (j < nb) out[j] = sm_scale * acc[a][b];
        }
    }
}

// ----------------------------------------------------------------------------------- select
constexpr int kSelThreads = 256;

__device__ __forceinline__ unsigned long long make_key(float s, int j) {
    unsigned int u = __float_as_uint(s);
    u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);   // increasing in s
    return ((unsigned long long)(~u) << 32) | (unsigned int)j;   // ascending key = score desc, index asc
}

__device__ __forceinline__ float block_max(float v, float* red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = red[0];
    for (int w = 1; w < kSelThreads / 32; ++w) r = fmaxf(r, red[w]);
    __syncthreads();
    return r;
}

__device__ __forceinline__ float block_sum(float v, float* red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = red[0];
    for (int w = 1; w < kSelThreads / 32; ++w) r += red[w];
    __syncthreads();
    return r;
}

// dynamic smem: keys u64[n2] | prob f32[n2] | sorted prob f32[n2] | bits u32[n2/32] | wpre u32[n2/32]
__global__ void __launch_bounds__(kSelThreads)
select_kernel(const float* __restrict__ scores, int nb, int n2, int score_stride, float p, int k_floor,
              uint32_t* __restrict__ mask_bits, int32_t* __restrict__ counts, uint16_t* __restrict__ idx) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    unsigned long long* keys = reinterpret_cast<unsigned long long*>(smem_raw);
    float* prob = reinterpret_cast<float*>(keys + n2);
    float* sp = prob + n2;
    uint32_t* bits = reinterpret_cast<uint32_t*>(sp + n2);
    const int nwords_pad = max(n2 / 32, 1);
    uint32_t* wpre = bits + nwords_pad;
    __shared__ float red[kSelThreads / 32];
    __shared__ float scan_tot[kSelThreads];
    __shared__ int cut;

    const int64_t row = blockIdx.x;
    const float* srow = scores + row * score_stride;
    const int tid = threadIdx.x;

    // softmax over the row
    float mx = -INFINITY;
    for (int j = tid; j < nb; j += kSelThreads) {
        float s = srow[j] + 0.0f;   // -0 -> +0 so equal scores have equal keys
        prob[j] = s;
        mx = fmaxf(mx, s);
    }
    mx = block_max(mx, red);
    float z = 0.f;
    for (int j = tid; j < nb; j += kSelThreads) {
        float s = prob[j];
        keys[j] = make_key(s, j);
        float e = expf(s - mx);
        prob[j] = e;
        z += e;
    }
    for (int j = nb + tid; j < n2; j += kSelThreads) keys[j] = ~0ull;
    z = block_sum(z, red);
    for (int j = tid; j < nb; j += kSelThreads) prob[j] = prob[j] / z;
    if (tid == 0) cut = nb;
    for (int w = tid; w < nwords_pad; w += kSelThreads) bits[w] = 0u;
    __syncthreads();

    // bitonic sort, ascending keys
    for (int k = 2; k <= n2; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int t = tid; t < (n2 >> 1); t += kSelThreads) {
                int a = ((t & ~(j - 1)) << 1) | (t & (j - 1));
                int b = a | j;
                bool up = (a & k) == 0;
                unsigned long long ka = keys[a], kb = keys[b];
                if ((ka > kb) == up) {
                    keys[a] = kb;
                    keys[b] = ka;
                }
            }
            __syncthreads();
        }
    }

    // cumulative mass in sorted order; c_p = first m (1-based) with cum >= p
    for (int m_ = tid; m_ < n2; m_ += kSelThreads)
        sp[m_] = (m_ < nb) ? prob[(unsigned int)(keys[m_] & 0xffffffffull)] : 0.f;
    __syncthreads();
    const int chunk = (n2 + kSelThreads - 1) / kSelThreads;
    const int beg = tid * chunk, end = min(beg + chunk, n2);
    float local = 0.f;
    for (int m_ = beg; m_ < end; ++m_) local += sp[m_];
    scan_tot[tid] = local;
    __syncthreads();
    if (tid < 32) {   // exclusive scan of the 256 thread totals by one warp, 8 per lane
        float v[8], run = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) { v[e] = scan_tot[tid * 8 + e]; run += v[e]; }
        float inc = run;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            float n = __shfl_up_sync(0xffffffffu, inc, o);
            if (tid >= o) inc += n;
        }
        float base = inc - run;
#pragma unroll
        for (int e = 0; e < 8; ++e) { scan_tot[tid * 8 + e] = base; base += v[e]; }
    }
    __syncthreads();
    if (p < 1.0f) {
        float cum = scan_tot[tid];
        for (int m_ = beg; m_ < end && m_ < nb; ++m_) {
            cum += sp[m_];
            if (cum >= p) { atomicMin(&cut, m_ + 1); break; }
        }
    }
    __syncthreads();
    const int c = max(cut, min(k_floor, nb));

    // materialise: bit mask, ascending index list, count
    for (int m_ = tid; m_ < c; m_ += kSelThreads) {
        unsigned int j = (unsigned int)(keys[m_] & 0xffffffffull);
        atomicOr(&bits[j >> 5], 1u << (j & 31));
    }
    __syncthreads();
    const int nwords = (nb + 31) / 32;
    if (tid < 32) {
        unsigned int carry = 0;
        for (int w0 = 0; w0 < nwords; w0 += 32) {
            int w = w0 + tid;
            unsigned int pc = (w < nwords) ? __popc(bits[w]) : 0u;
            unsigned int inc = pc;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                unsigned int n = __shfl_up_sync(0xffffffffu, inc, o);
                if (tid >= o) inc += n;
            }
            if (w < nwords) wpre[w] = carry + inc - pc;
            carry += __shfl_sync(0xffffffffu, inc, 31);
        }
    }
    __syncthreads();
    uint32_t* mrow = mask_bits + row * nwords;
    for (int w = tid; w < nwords; w += kSelThreads) mrow[w] = bits[w];
    uint16_t* irow = idx + row * nb;
    for (int j = tid; j < nb; j += kSelThreads) {
        unsigned int word = bits[j >> 5];
        if (word & (1u << (j & 31))) irow[wpre[j >> 5] + __popc(word & ((1u << (j & 31)) - 1u))] = (uint16_t)j;
    }
    if (tid == 0) counts[row] = c;
}

// One warp per (head, query block) row, nb <= 1024: the row lives in registers (E = ceil(nb/32)
// entries per lane, block j = lane + 32 e).  Instead of sorting, the warp bisects on the 32-bit
// order-preserving image of the score: the smallest threshold t such that the blocks with
// key <= t hold mass >= p and number at least max(1, min(k_floor, nb)) is the key of the last
// kept block, so {key <= t} is exactly the prefix the descending sort would have kept.  Blocks
// whose score equals the threshold's are admitted in index order one at a time (the tie rule).
// The ballot of the keep flags over entry e is the mask word for blocks 32e..32e+31, and its
// prefix pop-counts give the ascending compact index list.
constexpr int kSelWarpsPerCta = 8;

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ int warp_sum(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

template <int E>
__global__ void __launch_bounds__(kSelWarpsPerCta * 32)
select_warp_kernel(const float* __restrict__ scores, int nb, int64_t n_rows, int score_stride, float p, int k_floor,
                   uint32_t* __restrict__ mask_bits, int32_t* __restrict__ counts, uint16_t* __restrict__ idx) {
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * kSelWarpsPerCta + (threadIdx.x >> 5);
    if (row >= n_rows) return;
    const float* srow = scores + row * score_stride;

    float prob[E];
    uint32_t key[E];
    float mx = -INFINITY;
#pragma unroll
    for (int e = 0; e < E; ++e) {
        const int j = lane + 32 * e;
        const float sc = (j < nb) ? srow[j] + 0.0f : -INFINITY;   // -0 -> +0: equal scores, equal keys
        prob[e] = sc;
        mx = fmaxf(mx, sc);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float z = 0.f;
#pragma unroll
    for (int e = 0; e < E; ++e) {
        const int j = lane + 32 * e;
        uint32_t u = __float_as_uint(prob[e]);
        u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
        key[e] = (j < nb) ? ~u : 0xffffffffu;                   // ascending key = descending score
        const float ex = (j < nb) ? expf(prob[e] - mx) : 0.f;
        prob[e] = ex;
        z += ex;
    }
    z = warp_sum(z);
#pragma unroll
    for (int e = 0; e < E; ++e) prob[e] = prob[e] / z;

    const int need_cnt = max(1, min(k_floor, nb));
    uint32_t thr = 0xffffffffu;          // p >= 1 keeps everything
    int r_ties = 1 << 30;                // how many blocks with key == thr are kept (index order)
    if (p < 1.0f) {
        uint32_t lo = 0u, hi = 0xffffffffu;
#pragma unroll 1
        while (lo < hi) {
            const uint32_t mid = lo + ((hi - lo) >> 1);
            float mass = 0.f;
            int cnt = 0;
#pragma unroll
            for (int e = 0; e < E; ++e) {
                const bool in = key[e] <= mid;
                mass += in ? prob[e] : 0.f;
                cnt += in ? 1 : 0;
            }
            mass = warp_sum(mass);
            cnt = warp_sum(cnt);
            if (mass >= p && cnt >= need_cnt) hi = mid; else lo = mid + 1;
        }
        thr = hi;
        // blocks tied with the threshold score: admit them one by one, lowest index first
        float mass_lt = 0.f, p_tie = 0.f;
        int cnt_lt = 0, n_tie = 0;
#pragma unroll
        for (int e = 0; e < E; ++e) {
            const bool lt = key[e] < thr, eq = key[e] == thr && (lane + 32 * e) < nb;
            mass_lt += lt ? prob[e] : 0.f;
            cnt_lt += lt ? 1 : 0;
            n_tie += eq ? 1 : 0;
            p_tie = eq ? prob[e] : p_tie;
        }
        mass_lt = warp_sum(mass_lt);
        cnt_lt = warp_sum(cnt_lt);
        n_tie = warp_sum(n_tie);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) p_tie = fmaxf(p_tie, __shfl_xor_sync(0xffffffffu, p_tie, o));
        if (n_tie > 1) {
            float cum = mass_lt;
            int r = 0;
            while (r < n_tie) {
                cum += p_tie;
                ++r;
                if (cum >= p && cnt_lt + r >= need_cnt) break;
            }
            r_ties = r;
        }
    }

    // materialise
    uint32_t* mrow = mask_bits + row * ((nb + 31) / 32);
    uint16_t* irow = idx + row * nb;
    int base = 0, ties_seen = 0;
#pragma unroll
    for (int e = 0; e < E; ++e) {
        const int j = lane + 32 * e;
        const bool eq = key[e] == thr && j < nb;
        const uint32_t eq_ballot = __ballot_sync(0xffffffffu, eq);
        const int tie_rank = ties_seen + __popc(eq_ballot & ((1u << lane) - 1u));
        ties_seen += __popc(eq_ballot);
        const bool keep = j < nb && (key[e] < thr || (eq && tie_rank < r_ties));
        const uint32_t word = __ballot_sync(0xffffffffu, keep);
        if (32 * e < nb) {
            if (lane == 0) mrow[e] = word;
            if (keep) irow[base + __popc(word & ((1u << lane) - 1u))] = (uint16_t)j;
        }
        base += __popc(word);
    }
    if (lane == 0) counts[row] = base;
}

template <int E>
static fvattn_status_t launch_select_warp(const float* scores, int nb, int64_t n_rows, int score_stride, float p,
                                          int k_floor, uint32_t* mask_bits, int32_t* counts, uint16_t* idx,
                                          cudaStream_t s) {
    const unsigned ctas = (unsigned)((n_rows + kSelWarpsPerCta - 1) / kSelWarpsPerCta);
    select_warp_kernel<E><<<ctas, kSelWarpsPerCta * 32, 0, s>>>(scores, nb, n_rows, score_stride, p, k_floor,
                                                                  mask_bits, counts, idx);
    return launch_status();
}

__global__ void __launch_bounds__(256)
head_load_kernel(const int32_t* __restrict__ counts, int nb, float* __restrict__ head_load) {
    __shared__ unsigned int red[8];
    const int64_t bh = blockIdx.x;
    unsigned int s = 0;
    for (int i = threadIdx.x; i < nb; i += 256) s += (unsigned int)counts[bh * nb + i];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned int t = 0;
        for (int w = 0; w < 8; ++w) t += red[w];
        head_load[bh] = (float)t / (float)nb;   // Eq. 1
    }
}

// ------------------------------------------------------------------------------------ launch
fvattn_status_t launch_route(const void* q_r, const void* k_r, int64_t BH, int d, const GridDims& m, float p,
                             int k_floor, float sm_scale, uint32_t* mask_bits, int32_t* counts, uint16_t* idx,
                             float* head_load, void* workspace, cudaStream_t s) {
    RouteWs w = route_ws(BH, m.nb, d);
    char* ws = static_cast<char*>(workspace);
    float* qbar = reinterpret_cast<float*>(ws + w.qbar);
    float* kbar = reinterpret_cast<float*>(ws + w.kbar);
    float* scores = reinterpret_cast<float*>(ws + w.scores);

    dim3 pgrid((unsigned)m.nb, (unsigned)BH, 2);
    if (d == 128)
        pool_kernel<128><<<pgrid, kPoolThreads, 0, s>>>((const uint4*)q_r, (const uint4*)k_r, qbar, kbar, m);
    else
        pool_kernel<64><<<pgrid, kPoolThreads, 0, s>>>((const uint4*)q_r, (const uint4*)k_r, qbar, kbar, m);
    if (launch_status() != FVATTN_OK) return FVATTN_ERR_CUDA;

    unsigned tiles = (unsigned)((m.nb + kScoreTile - 1) / kScoreTile);
    score_kernel<<<dim3(tiles, tiles, (unsigned)BH), 256, 0, s>>>(qbar, kbar, scores, m.nb, d, w.score_stride,
                                                                   sm_scale);
    if (launch_status() != FVATTN_OK) return FVATTN_ERR_CUDA;

    if (m.nb <= 1024) {
        const int e = (m.nb + 31) / 32;
        const int64_t n_rows = BH * m.nb;
        fvattn_status_t st;
#define FVATTN_SEL_CASE(E_) \
    if (e <= E_) st = launch_select_warp<E_>(scores, m.nb, n_rows, w.score_stride, p, k_floor, mask_bits, counts, idx, s); else
        FVATTN_SEL_CASE(1) FVATTN_SEL_CASE(4) FVATTN_SEL_CASE(8) FVATTN_SEL_CASE(12) FVATTN_SEL_CASE(16)
        FVATTN_SEL_CASE(20) FVATTN_SEL_CASE(24) FVATTN_SEL_CASE(28)
        st = launch_select_warp<32>(scores, m.nb, n_rows, w.score_stride, p, k_floor, mask_bits, counts, idx, s);
#undef FVATTN_SEL_CASE
        if (st != FVATTN_OK) return st;
    } else {
        int n2 = 2048;
        while (n2 < m.nb) n2 <<= 1;
        size_t smem = (size_t)n2 * (8 + 4 + 4) + 2 * sizeof(uint32_t) * (size_t)(n2 / 32);
        FVATTN_CUDA_OK(cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        select_kernel<<<(unsigned)(BH * m.nb), kSelThreads, smem, s>>>(scores, m.nb, n2, w.score_stride, p, k_floor,
                                                                      mask_bits, counts, idx);
        if (launch_status() != FVATTN_OK) return FVATTN_ERR_CUDA;
    }

    if (head_load) {
        head_load_kernel<<<(unsigned)BH, 256, 0, s>>>(counts, m.nb, head_load);
        if (launch_status() != FVATTN_OK) return FVATTN_ERR_CUDA;
    }
    return FVATTN_OK;
}

} // namespace fvattn
