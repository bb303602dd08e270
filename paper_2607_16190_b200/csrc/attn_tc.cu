// Block-sparse attention on the sm_100a tensor cores (Sec. 2.1: only the retained
// (query block, key block) pairs are evaluated), Bs = d = 128, bf16 in, fp32 accumulate.
//
// One persistent CTA per SM, 12 warps, warp-specialised:
//   warp 0        producer: pops (head, query-block) tiles from the heaviest-first queue, TMA-loads
//                 Q once per tile and the retained K tiles by index into a 3-deep ring
//   warp 2        second producer: the retained V tiles into their own 3-deep ring
//   warps 1, 3    MMA issuers (one thread each), one per stream: S = Q K^T and O += P V as tcgen05
//                 MMAs with the accumulators in tensor memory
//   warps 4-7     softmax of the even retained blocks  (stream 0)
//   warps 8-11    softmax of the odd retained blocks   (stream 1)
// The retained blocks of a tile alternate between two independent streams, each with its own O
// accumulator (128 columns) and two S/P slots of 64 columns in tensor memory (all 512 columns) and
// its own running max and sum; the two partial results are merged once per tile
// (O = (O0 w0 + O1 w1) / (l0 w0 + l1 w1)).  A block is pipelined as two half-blocks of 64 keys:
// with two S slots per stream the QK MMA of a stream's next half-block is finished while its
// softmax warps are still on the current one, and the online-softmax recurrence simply runs per
// half-block.  One thread owns one query row: it reads 64 S values from tensor memory, keeps a
// running max with lazy rescaling (O is only rescaled when the max grows by more than 2^8, after
// the PV MMA in flight on it has completed), writes P back as bf16 over its S slot, and the PV
// thread feeds P from tensor memory as the A operand of the second MMA.  Padded keys of edge
// blocks are masked to -inf from a per-block validity table; padded query rows give zero.
//
// Shared-memory tiles use the 128-byte swizzle: a 128 x 128 bf16 tile is two TMA boxes of
// 128 rows x 64 columns (16 KB each).  Q and K are K-major MMA operands; V (keys x d, d
// contiguous) is the MN-major B operand of the second MMA.  No TMA multicast is used.
//
// Every wait is a bounded mbarrier wait; when one runs out the CTA records
// FVATTN_ERR_DEVICE_TIMEOUT in the workspace, every role leaves its loop, tensor memory is
// freed and the kernel returns.
#include <cuda_fp8.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace fvattn {

using namespace ptx;

namespace tc {
constexpr int BS = 128;
constexpr int D = 128;
constexpr int kThreads = 384;
constexpr int KS = 3;                               // K ring depth
constexpr int VS = 3;                               // V ring depth
constexpr int TS = 2;                               // tile-info ring depth
constexpr uint32_t kHalfBytes = 128 * 64 * 2;       // one TMA box: 128 rows x 64 bf16
constexpr uint32_t kTileBytes = 2 * kHalfBytes;     // 128 x 128 bf16
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColS = 0;                       // S / P of stream a, half-block slot h at kColS + 128 a + 64 h
constexpr uint32_t kColO = 256;                     // O of stream a at kColO + 128 a
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kRescaleThreshold = 8.0f;           // log2 units

struct __align__(1024) Smem {
    unsigned char q[kTileBytes];
    unsigned char k[KS][kTileBytes];
    unsigned char v[VS][kTileBytes];
    float ml[2][2][BS];                             // [stream][m, l][row]
    unsigned long long q_full, q_empty, k_full[KS], k_empty[KS], v_full[VS], v_empty[VS];
    unsigned long long s_full[2][2], p_full[2][2], pv_done[2][2], o_full, o_free, ml_ready, ml_done, tile_full[TS], tile_empty[TS];
    int tile_id[TS];
    int tile_cnt[TS];
    uint32_t tmem_base;
    int abort_flag;
};
static_assert(sizeof(Smem) <= 232448, "shared memory budget");

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
// (x, y) <- (x, y) * a + b, one packed fp32x2 instruction
__device__ __forceinline__ void fma2(float& x, float& y, float a, float b) {
    unsigned long long v, va, vb;
    asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "f"(x), "f"(y));
    asm("mov.b64 %0, {%1, %1};" : "=l"(va) : "f"(a));
    asm("mov.b64 %0, {%1, %1};" : "=l"(vb) : "f"(b));
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(v) : "l"(v), "l"(va), "l"(vb));
    asm("mov.b64 {%0, %1}, %2;" : "=f"(x), "=f"(y) : "l"(v));
}
// acc + (bf16 in the low / high half of a packed pair), fp32 result
__device__ __forceinline__ void add_bf16_pair(float& acc_lo, float& acc_hi, uint32_t packed) {
    unsigned short lo, hi;
    asm("mov.b32 {%0, %1}, %2;" : "=h"(lo), "=h"(hi) : "r"(packed));
    asm("add.rn.f32.bf16 %0, %1, %0;" : "+f"(acc_lo) : "h"(lo));
    asm("add.rn.f32.bf16 %0, %1, %0;" : "+f"(acc_hi) : "h"(hi));
}
template <int N>
__device__ __forceinline__ void setmaxnreg_inc() {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
}
template <int N>
__device__ __forceinline__ void setmaxnreg_dec() {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}
} // namespace tc

// Validity of the 128 key rows of every block (bit o of word o >> 5), for masking padded keys.
__global__ void __launch_bounds__(128)
key_mask_kernel(GridDims m, uint32_t* __restrict__ kmask) {
    int64_t token;
    unsigned int bal = __ballot_sync(0xffffffffu, threadIdx.x < m.bs && row_to_token(m, blockIdx.x, threadIdx.x, &token));
    if ((threadIdx.x & 31) == 0) kmask[blockIdx.x * 4 + (threadIdx.x >> 5)] = bal;
}

// kV8: V is FP8 E4M3 with one scale per (batch, head) (written by fvattn_quantize_v); P is then handed
// to the second MMA as E4M3 too (kind::f8f6f4, K = 32 per instruction), and the output is multiplied by
// the head's scale.  Everything else is identical to the bf16 path.
template <bool kV8>
__global__ void __launch_bounds__(tc::kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
               const __grid_constant__ CUtensorMap map_v, const uint16_t* __restrict__ idx,
               const int32_t* __restrict__ counts, GridDims m, float sm_scale, __nv_bfloat16* __restrict__ o_r,
               const uint32_t* __restrict__ order, const uint4* __restrict__ kmask, int has_pad, int n_tiles,
               void* workspace, const float* __restrict__ v_scale) {
    using namespace tc;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>(smem_raw);
    WsHeader* hdr = reinterpret_cast<WsHeader*>(workspace);

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    volatile int* abort_flag = &sm.abort_flag;

    if ((smem_u32(smem_raw) & 1023u) != 0u) {   // the swizzled tiles need a 1024-byte aligned base
        if (tid == 0) report_error(workspace, FVATTN_ERR_CUDA, 0x1024u);
        return;
    }
    if (tid == 0) {
        mbar_init(smem_u32(&sm.q_full), 1);
        mbar_init(smem_u32(&sm.q_empty), 2);
        for (int s = 0; s < KS; ++s) { mbar_init(smem_u32(&sm.k_full[s]), 1); mbar_init(smem_u32(&sm.k_empty[s]), 1); }
        for (int s = 0; s < VS; ++s) { mbar_init(smem_u32(&sm.v_full[s]), 1); mbar_init(smem_u32(&sm.v_empty[s]), 1); }
        for (int a = 0; a < 2; ++a)
            for (int h = 0; h < 2; ++h) {
                mbar_init(smem_u32(&sm.s_full[a][h]), 1);
                mbar_init(smem_u32(&sm.p_full[a][h]), 4);
                mbar_init(smem_u32(&sm.pv_done[a][h]), 1);
            }
        mbar_init(smem_u32(&sm.o_full), 2);
        mbar_init(smem_u32(&sm.o_free), 8);
        mbar_init(smem_u32(&sm.ml_ready), 8);
        mbar_init(smem_u32(&sm.ml_done), 8);
        for (int s = 0; s < TS; ++s) { mbar_init(smem_u32(&sm.tile_full[s]), 1); mbar_init(smem_u32(&sm.tile_empty[s]), 11); }
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
    const float sl2 = sm_scale * kLog2e;
    bool failed = false;

    if (warp < 4) {
        setmaxnreg_dec<40>();
        if (warp == 0) {
            // ======================= Q / K producer and tile queue ======================================
            uint32_t n = 0, kn = 0, qn = 0;
            bool ok = true;
            while (ok) {
                const uint32_t slot = n % TS;
                int tile = -1, c = 0;
                if (lane == 0) {
                    ok = mbar_wait(smem_u32(&sm.tile_empty[slot]), ((n / TS) & 1u) ^ 1u, abort_flag);
                    if (ok) {
                        const unsigned int q = atomicAdd(&hdr->tile_counter, 1u);
                        if (q < (unsigned int)n_tiles) {
                            tile = (int)order[q];
                            c = min(max(counts[tile], 0), m.nb);
                        }
                        sm.tile_id[slot] = tile;
                        sm.tile_cnt[slot] = c;
                        mbar_arrive(smem_u32(&sm.tile_full[slot]));
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                tile = __shfl_sync(0xffffffffu, tile, 0);
                c = __shfl_sync(0xffffffffu, c, 0);
                ++n;
                if (!ok || tile < 0) break;
                if (c == 0) continue;
                const int64_t bh = (uint32_t)tile / (uint32_t)m.nb;
                const int i = (int)((uint32_t)tile % (uint32_t)m.nb);
                const int64_t head_row0 = bh * m.n_pad;
                const uint16_t* irow = idx + (int64_t)tile * m.nb;
                if (lane == 0) {
                    ok = mbar_wait(smem_u32(&sm.q_empty), (qn & 1u) ^ 1u, abort_flag);
                    if (ok) {
                        const uint32_t bar = smem_u32(&sm.q_full);
                        mbar_expect_tx(bar, kTileBytes);
                        tma_load_2d(smem_u32(sm.q), &map_q, 0, (int)(head_row0 + (int64_t)i * BS), bar);
                        tma_load_2d(smem_u32(sm.q) + kHalfBytes, &map_q, 64, (int)(head_row0 + (int64_t)i * BS), bar);
                    }
                }
                ++qn;
                for (int t0 = 0; t0 < c && ok; t0 += 32) {
                    const int mine = (t0 + lane < c) ? (int)irow[t0 + lane] : 0;
                    const int lim = min(32, c - t0);
                    for (int tt = 0; tt < lim; ++tt) {
                        int kb = __shfl_sync(0xffffffffu, mine, tt);
                        if (lane == 0 && ok) {
                            if (kb >= m.nb) {
                                report_error(workspace, FVATTN_ERR_DEVICE_BOUNDS, (unsigned int)tile);
                                kb = 0;   // keep the pipeline consistent; the tile's result is undefined
                            }
                            const int krow = (int)(head_row0 + (int64_t)kb * BS);
                            const uint32_t ks = kn % KS;
                            ok = mbar_wait(smem_u32(&sm.k_empty[ks]), ((kn / KS) & 1u) ^ 1u, abort_flag);
                            if (ok) {
                                const uint32_t bar = smem_u32(&sm.k_full[ks]);
                                mbar_expect_tx(bar, kTileBytes);
                                tma_load_2d(smem_u32(sm.k[ks]), &map_k, 0, krow, bar);
                                tma_load_2d(smem_u32(sm.k[ks]) + kHalfBytes, &map_k, 64, krow, bar);
                            }
                        }
                        ++kn;
                    }
                    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                }
            }
            failed = !ok;
        } else if (warp == 2) {
            // ======================= V producer ========================================================
            // A second producer warp, so that a K tile is fetched the moment its ring slot frees (after
            // the QK MMA) instead of queueing behind the wait for a V slot (freed only after the PV MMA).
            uint32_t n = 0, vn = 0;
            bool ok = true;
            while (ok) {
                const uint32_t slot = n % TS;
                int tile = -1, c = 0;
                if (lane == 0) {
                    ok = mbar_wait(smem_u32(&sm.tile_full[slot]), (n / TS) & 1u, abort_flag);
                    if (ok) {
                        tile = sm.tile_id[slot];
                        c = sm.tile_cnt[slot];
                        mbar_arrive(smem_u32(&sm.tile_empty[slot]));
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                tile = __shfl_sync(0xffffffffu, tile, 0);
                c = __shfl_sync(0xffffffffu, c, 0);
                ++n;
                if (!ok || tile < 0) break;
                const int64_t head_row0 = (int64_t)((uint32_t)tile / (uint32_t)m.nb) * m.n_pad;
                const uint16_t* irow = idx + (int64_t)tile * m.nb;
                for (int t0 = 0; t0 < c && ok; t0 += 32) {
                    const int mine = (t0 + lane < c) ? (int)irow[t0 + lane] : 0;
                    const int lim = min(32, c - t0);
                    for (int tt = 0; tt < lim; ++tt) {
                        int kb = __shfl_sync(0xffffffffu, mine, tt);
                        if (lane == 0 && ok) {
                            if (kb >= m.nb) kb = 0;   // reported by the K producer
                            const int krow = (int)(head_row0 + (int64_t)kb * BS);
                            const uint32_t vs = vn % VS;
                            ok = mbar_wait(smem_u32(&sm.v_empty[vs]), ((vn / VS) & 1u) ^ 1u, abort_flag);
                            if (ok) {
                                const uint32_t bar = smem_u32(&sm.v_full[vs]);
                                if constexpr (kV8) {      // 128 keys x 128 one-byte columns: a single 16 KB box
                                    mbar_expect_tx(bar, kHalfBytes);
                                    tma_load_2d(smem_u32(sm.v[vs]), &map_v, 0, krow, bar);
                                } else {
                                    mbar_expect_tx(bar, kTileBytes);
                                    tma_load_2d(smem_u32(sm.v[vs]), &map_v, 0, krow, bar);
                                    tma_load_2d(smem_u32(sm.v[vs]) + kHalfBytes, &map_v, 64, krow, bar);
                                }
                            }
                        }
                        ++vn;
                    }
                    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                }
            }
            failed = !ok;
        } else if ((warp == 1 || warp == 3) && lane == 0) {
            // ======================= MMA issuers: one thread for S = Q K^T, one for O += P V =============
            // Two threads on two schedulers halve the serial time per block that a single issuer spends on
            // barrier polls, commits and MMA instructions.  The only ordering the two need between them is
            // that a QK MMA must not overwrite an S/P slot before the PV MMA of the slot's previous
            // occupant has read P: the QK thread waits for that PV's completion (pv_done, a commit by the
            // PV thread).
            constexpr uint32_t idesc_qk = make_idesc_bf16(128, 128, false);
            constexpr uint32_t idesc_pv = make_idesc_bf16(128, 128, true);
            // descriptor words that never change: high word (stride 1024 B, version, 128-byte swizzle);
            // low word = (address >> 4) | (leading offset >> 4) << 16, advanced by adding (bytes >> 4)
            const uint32_t desc_hi = (uint32_t)(make_smem_desc_sw128(0, 16, 1024) >> 32);
            const uint32_t q_lo = (uint32_t)make_smem_desc_sw128(smem_u32(sm.q), 16, 1024);
            const uint32_t k_lo0 = (uint32_t)make_smem_desc_sw128(smem_u32(sm.k[0]), 16, 1024);
            const uint32_t v_lo0 = (uint32_t)make_smem_desc_sw128(smem_u32(sm.v[0]), kHalfBytes, 1024);
            // A retained block (128 keys) is pipelined as two half-blocks of 64 keys, and each stream owns two
            // S/P slots (one per half): the QK MMA of a stream's next half-block is finished while its softmax
            // warps are still on the current one, so in steady state they do not wait for the tensor pipe.
            constexpr uint32_t idesc_qk64 = make_idesc_bf16(128, 64, false);
            // One issuer thread per stream (warp 1: stream 0, warp 3: stream 1).  Inside a stream the order
            // PV(v), QK(v + 2) is program order, so the QK MMA that refills an S/P slot needs no barrier
            // against the PV MMA that read it, and the stream's next half-block is on the tensor pipe as
            // soon as the current P has been consumed; the two streams never wait on each other.
            const int a = warp == 3 ? 1 : 0;
            uint32_t n = 0, ring0 = 0, qn = 0, pcnt = 0;   // ring0: ring position of the tile's block 0; pcnt: half-blocks PV'd
            bool ok = true;
            const uint32_t tOa = tmem + kColO + 128u * a;

            auto issue_qk = [&](int v) {                    // half-block v of this stream in the current tile
                const int u = v >> 1, half = v & 1;
                const uint32_t ring = ring0 + (uint32_t)(2 * u + a), st = ring % KS;
                if (half == 0) ok = ok && mbar_wait(smem_u32(&sm.k_full[st]), (ring / KS) & 1u, abort_flag);
                if (!ok) return;
                tc_fence_after();
                const uint32_t tSa = tmem + kColS + 128u * a + 64u * half;
                const uint32_t kh = k_lo0 + st * (kTileBytes >> 4) + (uint32_t)half * (8192u >> 4);   // key rows 64 half ..
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t off16 = ((uint32_t)(ks >> 2) * kHalfBytes + (uint32_t)(ks & 3) * 32u) >> 4;
                    umma_ss(tSa, ((uint64_t)desc_hi << 32) | (q_lo + off16), ((uint64_t)desc_hi << 32) | (kh + off16), idesc_qk64,
                            ks > 0 ? 1u : 0u);
                }
                if (half == 1) umma_commit(smem_u32(&sm.k_empty[st]));
                umma_commit(smem_u32(&sm.s_full[a][half]));
            };

            while (ok) {
                const uint32_t slot = n % TS;
                ok = mbar_wait(smem_u32(&sm.tile_full[slot]), (n / TS) & 1u, abort_flag);
                if (!ok) break;
                const int tile = sm.tile_id[slot];
                const int c = sm.tile_cnt[slot];
                mbar_arrive(smem_u32(&sm.tile_empty[slot]));
                ++n;
                if (tile < 0) break;
                if (c == 0) continue;
                const int n_a = (c - a + 1) >> 1, nv = 2 * n_a;
                // Q loaded also means that the previous tile's q_empty phase is complete
                ok = mbar_wait(smem_u32(&sm.q_full), qn & 1u, abort_flag);
                if (ok && n_a == 0) {
                    // c == 1 and this is stream 1: arrive in this tile's phases only
                    ok = mbar_wait(smem_u32(&sm.o_free), (qn & 1u) ^ 1u, abort_flag);
                    if (ok) { mbar_arrive(smem_u32(&sm.q_empty)); mbar_arrive(smem_u32(&sm.o_full)); }
                }
                if (ok && nv > 0) {
                    issue_qk(0);
                    issue_qk(1);
                    if (ok && nv == 2) umma_commit(smem_u32(&sm.q_empty));     // this stream's last QK of the tile
                }
                for (int v = 0; v < nv && ok; ++v) {
                    const int u = v >> 1, half = v & 1;
                    const uint32_t ring = ring0 + (uint32_t)(2 * u + a), st = ring % VS;
                    ok = mbar_wait(smem_u32(&sm.p_full[a][half]), (pcnt >> 1) & 1u, abort_flag);
                    if (half == 0) {
                        ok = ok && mbar_wait(smem_u32(&sm.v_full[st]), (ring / VS) & 1u, abort_flag);
                        if (ok && v == 0) ok = mbar_wait(smem_u32(&sm.o_free), (qn & 1u) ^ 1u, abort_flag);
                    }
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t tPb = tmem + kColS + 128u * a + 64u * half;
                    const uint32_t first = v == 0 ? 0u : 1u;                   // overwrite O on a stream's first half-block
                    if constexpr (kV8) {
                        // 2 steps of 32 keys: P is 4 E4M3 per tensor-memory column, V rows are 128 B apart
                        constexpr uint32_t idesc_pv8 = make_idesc_e4m3(128, 128);
                        const uint32_t vlo8 = (uint32_t)make_smem_desc_sw128(smem_u32(sm.v[st]), 16, 1024);
#pragma unroll
                        for (int ks = 0; ks < 2; ++ks)
                            umma_ts_f8(tOa, tPb + ks * 8,
                                       ((uint64_t)desc_hi << 32) | (vlo8 + (uint32_t)half * (8192u >> 4) + (uint32_t)ks * (4096u >> 4)),
                                       idesc_pv8, ks > 0 ? 1u : first);
                    } else {
                        const uint32_t vlo = v_lo0 + st * (kTileBytes >> 4);
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks)
                            umma_ts(tOa, tPb + ks * 8,
                                    ((uint64_t)desc_hi << 32) | (vlo + (uint32_t)half * (8192u >> 4) + (uint32_t)ks * (2048u >> 4)),
                                    idesc_pv, ks > 0 ? 1u : first);
                    }
                    umma_commit(smem_u32(&sm.pv_done[a][half]));             // for the softmax warps' rare rescale of O
                    if (half == 1) umma_commit(smem_u32(&sm.v_empty[st]));
                    ++pcnt;
                    if (v + 2 < nv) {
                        issue_qk(v + 2);                                       // refills the slot PV(v) has just read
                        if (ok && v + 3 == nv) umma_commit(smem_u32(&sm.q_empty));   // that was the stream's last QK of the tile
                    }
                }
                if (ok && nv > 0) umma_commit(smem_u32(&sm.o_full));          // this stream's PVs (hence its QKs) are done
                ring0 += (uint32_t)c;
                ++qn;
            }
            failed = !ok;
        }
    } else {
        // ======================= softmax warpgroups ==================================================
        setmaxnreg_inc<232>();
        const int a = (warp - 4) >> 2;            // stream
        const int row = tid - 128 - 128 * a;      // query row of the tile = TMEM lane
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tS = tmem + lane_base + kColS + 128u * a;
        const uint32_t tO = tmem + lane_base + kColO + 128u * a;
        uint32_t n = 0, sn = 0, tile_seq = 0;
        bool ok = true;

        while (ok) {
            const uint32_t slot = n % TS;
            ok = mbar_wait(smem_u32(&sm.tile_full[slot]), (n / TS) & 1u, abort_flag);
            if (!ok) break;
            const int tile = sm.tile_id[slot];
            const int c = sm.tile_cnt[slot];
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sm.tile_empty[slot]));
            ++n;
            if (tile < 0) break;
            const int64_t bh = (uint32_t)tile / (uint32_t)m.nb;
            const int i = (int)((uint32_t)tile % (uint32_t)m.nb);
            const uint16_t* irow = idx + (int64_t)tile * m.nb;
            // this thread stores columns [64 a, 64 a + 64) of output row `row`
            uint4* orow = reinterpret_cast<uint4*>(o_r + ((bh * m.n_pad + (int64_t)i * BS + row) * D + 64 * a));
            if (c == 0) {
#pragma unroll
                for (int q4 = 0; q4 < 8; ++q4) orow[q4] = make_uint4(0u, 0u, 0u, 0u);
                continue;
            }
            const int n_a = (c - a + 1) >> 1;     // blocks t = a, a + 2, ... of this stream
            float m_run = -INFINITY, l_run = 0.f;

            for (int v = 0; v < 2 * n_a && ok; ++v) {            // half-blocks of 64 keys of this stream
                const int u = v >> 1, half = v & 1;
                uint32_t kw0 = 0xffffffffu, kw1 = 0xffffffffu;    // validity of this half-block's 64 keys
                if (has_pad) {
                    const int kb = min((int)irow[2 * u + a], m.nb - 1);
                    const uint2 kv = __ldg(reinterpret_cast<const uint2*>(kmask + kb) + half);
                    kw0 = kv.x;
                    kw1 = kv.y;
                }
                ok = mbar_wait(smem_u32(&sm.s_full[a][half]), (sn >> 1) & 1u, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t tSh = tS + 64u * half;
                uint32_t s[64];
                tmem_ld32(tSh, *reinterpret_cast<uint32_t(*)[32]>(&s[0]));
                tmem_ld32(tSh + 32, *reinterpret_cast<uint32_t(*)[32]>(&s[32]));
                tmem_wait_ld();
                if ((kw0 & kw1) != 0xffffffffu) {                 // edge block: padded keys -> -inf
#pragma unroll
                    for (int j = 0; j < 64; ++j)
                        if (!(((j < 32 ? kw0 : kw1) >> (j & 31)) & 1u)) s[j] = 0xff800000u;
                }
                float mx0 = __uint_as_float(s[0]), mx1 = __uint_as_float(s[1]), mx2 = __uint_as_float(s[2]),
                      mx3 = __uint_as_float(s[3]);
#pragma unroll
                for (int j = 4; j < 64; j += 8) {
                    mx0 = max3(mx0, __uint_as_float(s[j]), __uint_as_float(s[j + 1]));
                    mx1 = max3(mx1, __uint_as_float(s[j + 2]), __uint_as_float(s[j + 3]));
                    if (j + 4 < 64) {
                        mx2 = max3(mx2, __uint_as_float(s[j + 4]), __uint_as_float(s[j + 5]));
                        mx3 = max3(mx3, __uint_as_float(s[j + 6]), __uint_as_float(s[j + 7]));
                    }
                }
                const float m_new = fmaxf(m_run, fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)));
                // lazy rescale: keep the old reference max unless the new one is more than 2^8 above it
                const bool need = (m_new - m_run) * sl2 > kRescaleThreshold;   // also true for m_run = -inf
                if (__any_sync(0xffffffffu, need)) {
                    float corr = 1.f;
                    if (need) {
                        corr = (m_run == -INFINITY) ? 0.f : ex2((m_run - m_new) * sl2);
                        m_run = m_new;
                    }
                    l_run *= corr;
                    if (v > 0) {
                        // O still receives the previous half-block's P V: wait for that MMA before touching it
                        ok = mbar_wait(smem_u32(&sm.pv_done[a][half ^ 1]), ((sn - 1u) >> 1) & 1u, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                        uint32_t r[32];
#pragma unroll
                        for (int ch = 0; ch < 4; ++ch) {
                            tmem_ld32(tO + ch * 32, r);
                            tmem_wait_ld();
#pragma unroll
                            for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * corr);
                            tmem_st32(tO + ch * 32, r);
                        }
                    }
                }
                const float moff = (m_run == -INFINITY) ? 0.f : m_run * sl2;   // -inf only if no valid key yet
                float sum0 = 0.f, sum1 = 0.f, sum2 = 0.f, sum3 = 0.f;
                if constexpr (kV8) {
                    uint32_t pk8[16];                              // 4 E4M3 weights per column, lowest key in the lowest byte
#pragma unroll
                    for (int j = 0; j < 64; j += 4) {
                        float e0 = __uint_as_float(s[j]), e1 = __uint_as_float(s[j + 1]), e2 = __uint_as_float(s[j + 2]),
                              e3 = __uint_as_float(s[j + 3]);
                        fma2(e0, e1, sl2, -moff);
                        fma2(e2, e3, sl2, -moff);
                        const float p0 = ex2(e0), p1 = ex2(e1), p2 = ex2(e2), p3 = ex2(e3);
                        const uint32_t lo = __nv_cvt_float2_to_fp8x2(make_float2(p0, p1), __NV_SATFINITE, __NV_E4M3);
                        const uint32_t hi = __nv_cvt_float2_to_fp8x2(make_float2(p2, p3), __NV_SATFINITE, __NV_E4M3);
                        pk8[j >> 2] = lo | (hi << 16);
                        sum0 += p0; sum1 += p1; sum2 += p2; sum3 += p3;
                    }
                    l_run += (sum0 + sum1) + (sum2 + sum3);
                    tmem_st16(tSh, pk8);
                } else {
                    uint32_t pk[32];
#pragma unroll
                    for (int j = 0; j < 64; j += 4) {
                        float e0 = __uint_as_float(s[j]), e1 = __uint_as_float(s[j + 1]), e2 = __uint_as_float(s[j + 2]),
                              e3 = __uint_as_float(s[j + 3]);
                        fma2(e0, e1, sl2, -moff);
                        fma2(e2, e3, sl2, -moff);
                        __nv_bfloat162 lo = __floats2bfloat162_rn(ex2(e0), ex2(e1));   // .x (low half) = even column
                        __nv_bfloat162 hi = __floats2bfloat162_rn(ex2(e2), ex2(e3));
                        const uint32_t wlo = *reinterpret_cast<uint32_t*>(&lo), whi = *reinterpret_cast<uint32_t*>(&hi);
                        pk[j >> 1] = wlo;
                        pk[(j >> 1) + 1] = whi;
                        // the row sum takes the bf16-rounded weights the second MMA sees, so numerator and
                        // denominator stay consistent (an exact weighted average of V)
                        add_bf16_pair(sum0, sum1, wlo);
                        add_bf16_pair(sum2, sum3, whi);
                    }
                    l_run += (sum0 + sum1) + (sum2 + sum3);
                    tmem_st32(tSh, pk);                           // P over the first 32 columns of this S slot
                }
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sm.p_full[a][half]));
                ++sn;
            }
            if (!ok) break;

            // ---- merge the two streams and store ----------------------------------------------------
            sm.ml[a][0][row] = m_run;
            sm.ml[a][1][row] = l_run;
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sm.ml_ready));
            ok = mbar_wait(smem_u32(&sm.ml_ready), tile_seq & 1u, abort_flag);
            ok = ok && mbar_wait(smem_u32(&sm.o_full), tile_seq & 1u, abort_flag);
            if (!ok) break;
            tc_fence_after();
            const float m0 = sm.ml[0][0][row], l0 = sm.ml[0][1][row];
            const float m1 = sm.ml[1][0][row], l1 = sm.ml[1][1][row];
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sm.ml_done));
            const bool has1 = c >= 2;                       // stream 1 saw at least one block
            const float mm = has1 ? fmaxf(m0, m1) : m0;
            const float w0 = (m0 == -INFINITY) ? 0.f : ex2((m0 - mm) * sl2);
            const float w1 = (!has1 || m1 == -INFINITY) ? 0.f : ex2((m1 - mm) * sl2);
            const float lsum = l0 * w0 + l1 * w1;
            int64_t token;
            const bool qvalid = !has_pad || row_to_token(m, i, row, &token);
            const float inv = (qvalid && lsum > 0.f) ? 1.f / lsum : 0.f;
            const float vs_h = kV8 ? v_scale[bh] : 1.f;
            const float f0 = w0 * inv * vs_h, f1 = w1 * inv * vs_h;
            const uint32_t tO0 = tmem + lane_base + kColO + 64u * a;
            const uint32_t tO1 = tO0 + 128u;
#pragma unroll
            for (int ch = 0; ch < 2; ++ch) {
                uint32_t r0[32], r1[32];
                tmem_ld32(tO0 + ch * 32, r0);
                if (has1) tmem_ld32(tO1 + ch * 32, r1);
                tmem_wait_ld();
                uint32_t outw[16];
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                    float x = f0 != 0.f ? __uint_as_float(r0[j]) * f0 : 0.f;
                    float y = f0 != 0.f ? __uint_as_float(r0[j + 1]) * f0 : 0.f;
                    if (has1 && f1 != 0.f) {
                        x = fmaf(__uint_as_float(r1[j]), f1, x);
                        y = fmaf(__uint_as_float(r1[j + 1]), f1, y);
                    }
                    __nv_bfloat162 b2 = __floats2bfloat162_rn(x, y);
                    outw[j >> 1] = *reinterpret_cast<uint32_t*>(&b2);
                }
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4)
                    orow[ch * 4 + q4] = make_uint4(outw[q4 * 4], outw[q4 * 4 + 1], outw[q4 * 4 + 2], outw[q4 * 4 + 3]);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sm.o_free));
            // nobody may overwrite ml for the next tile before every row of this one has been read
            ok = mbar_wait(smem_u32(&sm.ml_done), tile_seq & 1u, abort_flag);
            ++tile_seq;
        }
        failed = !ok;
    }

    if (failed) {
        *abort_flag = 1;
        report_error(workspace, FVATTN_ERR_DEVICE_TIMEOUT, blockIdx.x);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
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

// [rows, 128] one-byte (E4M3) row-major tensor, box = 128 rows x 128 columns (128 B), 128-byte swizzle.
static bool make_tile_map_u8(CUtensorMap* map, const void* base, uint64_t rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)tc::D, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)tc::D};
    cuuint32_t box[2] = {128, 128};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// v_scale == NULL: v_r is bf16.  Otherwise v_r holds E4M3 codes and v_scale one fp32 scale per (batch, head).
fvattn_status_t launch_attn_tc(const void* q_r, const void* k_r, const void* v_r, const uint16_t* idx,
                               const int32_t* counts, int64_t BH, const GridDims& m, float sm_scale, void* o_r,
                               const uint32_t* order, void* workspace, const float* v_scale, cudaStream_t s) {
    const uint64_t rows = (uint64_t)BH * (uint64_t)m.n_pad;
    if (rows > 0x7fffffffull) return FVATTN_ERR_UNSUPPORTED_SHAPE;   // TMA coordinates are 32-bit
    CUtensorMap mq, mk, mv;
    if (!make_tile_map(&mq, q_r, rows) || !make_tile_map(&mk, k_r, rows)) return FVATTN_ERR_CUDA;
    if (!(v_scale ? make_tile_map_u8(&mv, v_r, rows) : make_tile_map(&mv, v_r, rows))) return FVATTN_ERR_CUDA;
    int dev = 0, sms = 0;
    FVATTN_CUDA_OK(cudaGetDevice(&dev));
    FVATTN_CUDA_OK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    uint32_t* kmask = reinterpret_cast<uint32_t*>(static_cast<char*>(workspace) + attn_ws(BH, m.nb).kmask);
    const int has_pad = m.n_pad != m.n ? 1 : 0;
    if (has_pad) {
        key_mask_kernel<<<(unsigned)m.nb, 128, 0, s>>>(m, kmask);
        if (launch_status() != FVATTN_OK) return FVATTN_ERR_CUDA;
    }
    const size_t smem = sizeof(tc::Smem);
    const int n_tiles = (int)(BH * m.nb);
    const int grid = n_tiles < sms ? n_tiles : sms;
    if (v_scale) {
        FVATTN_CUDA_OK(cudaFuncSetAttribute(attn_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        attn_tc_kernel<true><<<grid, tc::kThreads, smem, s>>>(mq, mk, mv, idx, counts, m, sm_scale, (__nv_bfloat16*)o_r,
                                                             order, reinterpret_cast<const uint4*>(kmask), has_pad,
                                                             n_tiles, workspace, v_scale);
    } else {
        FVATTN_CUDA_OK(cudaFuncSetAttribute(attn_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        attn_tc_kernel<false><<<grid, tc::kThreads, smem, s>>>(mq, mk, mv, idx, counts, m, sm_scale, (__nv_bfloat16*)o_r,
                                                              order, reinterpret_cast<const uint4*>(kmask), has_pad,
                                                              n_tiles, workspace, nullptr);
    }
    return launch_status();
}

} // namespace fvattn
