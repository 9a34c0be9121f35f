// Split-m multi-query decode kernel (Section 3: logits = einsum(bhk,bmk->bhm), softmax over m,
// o = einsum(bhm,bmv->bhv)) for sm_100a.
//
// One CTA owns one split of one sequence's memory axis.  A producer warp streams that split's
// K and V rows HBM -> shared memory with TMA (cp.async.bulk.tensor, 128-byte swizzle) through
// a ring of stages guarded by full/empty mbarriers; every K/V byte is fetched from HBM once
// and is then used for ALL h heads, which is the whole point of the multi-query layout
// (h flops per byte instead of 1).  At h flops per byte the CUDA cores cannot keep up with
// HBM, so the two contractions run on the tensor cores with the heads as the M rows:
//     S[h x rows]   = Q[h x k] * K_tile^T          (bf16 mma, fp32 accumulate)
//     O[h x v]     += P[h x rows] * V_tile         (P = exp2(S - max), split into bf16 hi + lo
//                                                  parts so that the weights keep ~16 bits)
// Each consumer warp takes whole 32-row tiles round-robin and keeps its own online-softmax
// state (running max, running sum, fp32 accumulators) in registers; warps are merged through
// shared memory at the end and the CTA writes its partial (or the final o for a single split).
//
// Rows at or beyond lens[b] are never used: their logits are replaced by -inf by index and
// their V fragments are zeroed by index (a NaN times a zero weight would still be a NaN).
#pragma once
#include <cuda.h>

#include "combine.cuh"
#include "common.cuh"

namespace mqa {

constexpr int kTileRows = 32;                          // cache rows per pipeline stage
constexpr int kBoxCols = 64;                           // 64 bf16 = 128 bytes = one swizzle span
constexpr int kBoxBytes = kTileRows * kBoxCols * 2;    // 4 KiB
constexpr int kStageBytes = 4 * kBoxBytes;             // K lo, K hi, V lo, V hi = 16 KiB
constexpr int kRowWarps = 4;                           // consumer warps that share the tiles
constexpr long long kWaitLimitCycles = 2000000000ll;    // every mbarrier wait gives up after ~1 s of SM clock ...
constexpr uint32_t kWaitRounds = 1u << 24;             // ... or after this many polling rounds

template <int M_TILES>
struct MmaCfg {
    static constexpr int kConsumerWarps = M_TILES * kRowWarps;
    static constexpr int kThreads = (kConsumerWarps + 1) * 32;
    // Ring depth.  It must be a multiple of kRowWarps: tile i lives in stage i % kStages and belongs
    // to row-warp i % kRowWarps, so with this rule every use of a stage is waited on by the same warp.
    // A parity wait can only tell the current phase from the one before it; a warp that skipped a use
    // of a stage could mistake an old phase for the one it needs.
    static constexpr int kStages = (M_TILES == 1) ? 4 : 12;
    static_assert(kStages % kRowWarps == 0, "a stage must always be consumed by the same warp");
    static constexpr int kSmemBytes = kStages * kStageBytes + 1024 /* alignment slack */ + 256 /* barriers */;
    static constexpr int kMinBlocks = (M_TILES == 1) ? 2 : 1;
};

// ---- PTX wrappers ------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done != 0;
}
// Bounded wait: false if the phase has not completed about one second after the first miss.
// The limit is checked twice in a row so that a single odd clock reading cannot end a wait.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t round = 0; round < kWaitRounds; ++round) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (clock64() - t0 > kWaitLimitCycles && clock64() - t0 > kWaitLimitCycles) return false;
    }
    return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// {hi16: bf16(x_hi), lo16: bf16(x_lo)}, round to nearest even
__device__ __forceinline__ uint32_t pack_bf16(float x_lo, float x_hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(x_hi), "f"(x_lo));
    return r;
}

// Byte offset of (row, 16-byte chunk 0..15 along the 128 columns) inside one K or V tile as
// TMA lays it out: two 64-column boxes, each 128-byte-swizzled (chunk index XOR row mod 8).
__device__ __forceinline__ uint32_t tile_offset(int row, int chunk) {
    return (uint32_t)((chunk >> 3) * kBoxBytes + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}

template <int M_TILES>
__global__ void __launch_bounds__(MmaCfg<M_TILES>::kThreads, MmaCfg<M_TILES>::kMinBlocks)
mqa_decode_split_mma_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                            const uint32_t* __restrict__ q, const int32_t* __restrict__ lens,
                            float* __restrict__ o, float2* __restrict__ part_ml, float* __restrict__ part_acc,
                            int32_t* __restrict__ status, int h, int m_max, int chunk_rows, int n_splits) {
    using Cfg = MmaCfg<M_TILES>;
    constexpr int kStages = Cfg::kStages;
    const int seq = blockIdx.x / n_splits;
    const int split = blockIdx.x % n_splits;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    const int L = clamp_len(lens[seq], m_max, threadIdx.x == 0 ? status : nullptr);
    const int r0 = split * chunk_rows;
    const int r1 = min(L, r0 + chunk_rows);
    if (r0 >= L) {                                         // nothing valid in this split (uniform)
        if (n_splits == 1)                                 // L == 0: the empty prefix gives zeros
            for (int i = threadIdx.x; i < h * kHeadDim; i += Cfg::kThreads) o[(size_t)seq * h * kHeadDim + i] = 0.f;
        return;
    }
    const int n_tiles = (r1 - r0 + kTileRows - 1) / kTileRows;

    extern __shared__ uint8_t smem_raw[];
    // 1 KiB alignment in the shared window: the 128-byte swizzle repeats every 8 rows x 128 bytes
    uint8_t* stages = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);
    uint64_t* bars = reinterpret_cast<uint64_t*>(stages + kStages * kStageBytes);   // full[kStages], empty[kStages]
    const uint32_t stages_s = smem_addr(stages);
    const uint32_t full_s = smem_addr(bars), empty_s = full_s + kStages * 8;
    __shared__ int timed_out, issued;   // a wait ran out; tiles whose copies were started

    if (threadIdx.x == 0) {
        timed_out = 0;
        issued = 0;
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full_s + s * 8, 1);                  // the producer's arrive + the TMA bytes
            mbar_init(empty_s + s * 8, M_TILES);           // one arrive per warp that read the tile
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    if (warp == Cfg::kConsumerWarps) {
        // ------------------------------------------------------------------ producer warp
        if (lane == 0) {
            const int row_base = seq * m_max + r0;         // row coordinate in the [b*m_max, 128] view
            bool ok = true;
            for (int i = 0; i < n_tiles && ok; ++i) {
                const int s = i % kStages;
                if (i >= kStages) ok = mbar_wait(empty_s + s * 8, ((i / kStages) - 1) & 1);
                if (!ok) break;
                const uint32_t bar = full_s + s * 8;
                const uint32_t dst = stages_s + s * kStageBytes;
                mbar_expect_tx(bar, kStageBytes);
                const int y = row_base + i * kTileRows;
                tma_load_2d(dst, &map_k, 0, y, bar);
                tma_load_2d(dst + kBoxBytes, &map_k, kBoxCols, y, bar);
                tma_load_2d(dst + 2 * kBoxBytes, &map_v, 0, y, bar);
                tma_load_2d(dst + 3 * kBoxBytes, &map_v, kBoxCols, y, bar);
                issued = i + 1;
            }
            if (!ok) atomicExch(&timed_out, 1);
        }
    }

    // Per-thread state of a consumer warp (declared for all warps; the producer leaves it unused).
    const int cw = warp;                                   // consumer warp index
    const int mt = cw % M_TILES;                           // which 16-head tile this warp serves
    const int rw = cw / M_TILES;                           // which tiles (round-robin over kRowWarps)
    const int g = lane >> 2, t4 = lane & 3;
    float acc[16][4];
    float m_run[2] = {-INFINITY, -INFINITY};               // heads mt*16+g and mt*16+g+8
    float l_run[2] = {0.f, 0.f};                           // this thread's share of the row sums

    if (warp < Cfg::kConsumerWarps) {
        // --------------------------------------------------------------- consumer warps
#pragma unroll
        for (int i = 0; i < 16; ++i) { acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f; }

        // Q fragments (A operand, 16 heads x 128), straight from global memory; heads >= h are zero.
        uint32_t qa[8][4];
        {
            const int head0 = mt * 16 + g, head1 = head0 + 8;
            const uint32_t* q0 = q + ((size_t)seq * h + head0) * (kHeadDim / 2);
            const uint32_t* q1 = q + ((size_t)seq * h + head1) * (kHeadDim / 2);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                const int w0 = ks * 8 + t4;                // 32-bit word index: columns ks*16 + t4*2 + {0,1}
                qa[ks][0] = head0 < h ? q0[w0] : 0u;
                qa[ks][1] = head1 < h ? q1[w0] : 0u;
                qa[ks][2] = head0 < h ? q0[w0 + 4] : 0u;   // columns + 8
                qa[ks][3] = head1 < h ? q1[w0 + 4] : 0u;
            }
        }
        // ldmatrix lane roles (matrix = lane / 8, row within the matrix = lane % 8)
        const int lm = lane >> 3, lr = lane & 7;

        bool ok = true;
        for (int i = rw; i < n_tiles; i += kRowWarps) {
            const int s = i % kStages;
            ok = mbar_wait(full_s + s * 8, (i / kStages) & 1);
            if (!ok) break;
            const uint32_t k_s = stages_s + s * kStageBytes;
            const uint32_t v_s = k_s + 2 * kBoxBytes;
            const int row0 = r0 + i * kTileRows;           // first cache row of this tile
            const bool ragged = row0 + kTileRows > r1;

            // S = Q K^T for 32 rows: 4 n-tiles of 8 rows
            float sc[4][4];
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
#pragma unroll
                for (int np = 0; np < 2; ++np) {           // n-tile pairs (0,1) and (2,3)
                    uint32_t b0, b1, b2, b3;
                    const int row = (np * 2 + (lm >> 1)) * 8 + lr;
                    ldmatrix_x4(k_s + tile_offset(row, ks * 2 + (lm & 1)), b0, b1, b2, b3);
                    mma_bf16(sc[np * 2], qa[ks], b0, b1);
                    mma_bf16(sc[np * 2 + 1], qa[ks], b2, b3);
                }
            }
            // scale to log2 units, mask by index, row maxima
            float top[2] = {-INFINITY, -INFINITY};
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int row = row0 + nt * 8 + t4 * 2 + (j & 1);
                    const float x = sc[nt][j] * kLog2e;
                    sc[nt][j] = (!ragged || row < r1) ? x : -INFINITY;      // select, never multiply
                    top[j >> 1] = fmaxf(top[j >> 1], sc[nt][j]);
                }
            }
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                top[r] = fmaxf(top[r], __shfl_xor_sync(0xffffffffu, top[r], 1));
                top[r] = fmaxf(top[r], __shfl_xor_sync(0xffffffffu, top[r], 2));
            }
            float rescale[2];
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                const float m_new = fmaxf(m_run[r], top[r]);    // the tile's first row is valid: finite
                rescale[r] = fast_exp2(m_run[r] - m_new);       // 0 on this warp's first tile
                m_run[r] = m_new;
                l_run[r] *= rescale[r];
            }
#pragma unroll
            for (int vt = 0; vt < 16; ++vt) {
                acc[vt][0] *= rescale[0]; acc[vt][1] *= rescale[0];
                acc[vt][2] *= rescale[1]; acc[vt][3] *= rescale[1];
            }
            // P = exp2(S - max) as bf16 hi + lo A-fragments for the two 16-row k-steps
            uint32_t p_hi[2][4], p_lo[2][4];
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
                float p[4], ph[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    p[j] = fast_exp2(sc[nt][j] - m_run[j >> 1]);   // exactly 1 at the maximum, 0 when masked
                    l_run[j >> 1] += p[j];
                }
                const uint32_t hi01 = pack_bf16(p[0], p[1]), hi23 = pack_bf16(p[2], p[3]);
                ph[0] = bf16_lo(hi01); ph[1] = bf16_hi(hi01); ph[2] = bf16_lo(hi23); ph[3] = bf16_hi(hi23);
                const uint32_t lo01 = pack_bf16(p[0] - ph[0], p[1] - ph[1]);
                const uint32_t lo23 = pack_bf16(p[2] - ph[2], p[3] - ph[3]);
                const int kk = nt >> 1, hf = (nt & 1) * 2;          // A regs: {g,k}, {g+8,k}, {g,k+8}, {g+8,k+8}
                p_hi[kk][hf] = hi01; p_hi[kk][hf + 1] = hi23;
                p_lo[kk][hf] = lo01; p_lo[kk][hf + 1] = lo23;
            }
            // O += P V : 2 k-steps of 16 rows x 16 n-tiles of 8 columns
#pragma unroll
            for (int kk = 0; kk < 2; ++kk) {
                uint32_t keep_lo = 0xffffffffu, keep_hi = 0xffffffffu;   // per-register row masks (ragged tile)
                if (ragged) {
                    const int ra = row0 + kk * 16 + t4 * 2;              // rows held by b0/b1: ra, ra+1; b2/b3: +8
                    keep_lo = (ra < r1 ? 0x0000ffffu : 0u) | (ra + 1 < r1 ? 0xffff0000u : 0u);
                    keep_hi = (ra + 8 < r1 ? 0x0000ffffu : 0u) | (ra + 9 < r1 ? 0xffff0000u : 0u);
                }
#pragma unroll
                for (int vp = 0; vp < 8; ++vp) {                         // pairs of 8-column n-tiles
                    uint32_t b0, b1, b2, b3;
                    const int row = kk * 16 + (lm & 1) * 8 + lr;
                    ldmatrix_x4_trans(v_s + tile_offset(row, vp * 2 + (lm >> 1)), b0, b1, b2, b3);
                    if (ragged) { b0 &= keep_lo; b1 &= keep_hi; b2 &= keep_lo; b3 &= keep_hi; }
                    mma_bf16(acc[vp * 2], p_hi[kk], b0, b1);
                    mma_bf16(acc[vp * 2], p_lo[kk], b0, b1);
                    mma_bf16(acc[vp * 2 + 1], p_hi[kk], b2, b3);
                    mma_bf16(acc[vp * 2 + 1], p_lo[kk], b2, b3);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_s + s * 8);                 // this warp is done with the stage
        }
        if (!ok) atomicExch(&timed_out, 1);
    }

    __syncthreads();   // every tile has landed and been consumed (or a wait ran out)
    if (timed_out) {
        // A wait ran out.  Before this CTA's shared memory is released, make sure (again with a
        // bound) that the last copy started into each stage has landed; then flag the status
        // word and leave without writing results.
        if (threadIdx.x == 0) {
            for (int s = 0; s < kStages && s < issued; ++s) {
                const int last_use = (issued - 1 - s) / kStages;
                mbar_wait(full_s + s * 8, last_use & 1);
            }
            if (status) atomicOr(status, kStatusPipelineTimeout);
        }
        __syncthreads();
        return;
    }

    // ---- merge the kRowWarps warps of each head tile through shared memory (stages are free now)
    float* sm_acc = reinterpret_cast<float*>(stages);                   // [consumer warp][16][128]
    float2* sm_ml = reinterpret_cast<float2*>(stages + Cfg::kConsumerWarps * 16 * kHeadDim * 4);  // [cw][16]
    if (warp < Cfg::kConsumerWarps) {
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
            l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
        }
        float* mine = sm_acc + (size_t)cw * 16 * kHeadDim;
#pragma unroll
        for (int vt = 0; vt < 16; ++vt) {
            *reinterpret_cast<float2*>(mine + g * kHeadDim + vt * 8 + t4 * 2) = make_float2(acc[vt][0], acc[vt][1]);
            *reinterpret_cast<float2*>(mine + (g + 8) * kHeadDim + vt * 8 + t4 * 2) = make_float2(acc[vt][2], acc[vt][3]);
        }
        if (t4 == 0) {
            sm_ml[cw * 16 + g] = make_float2(m_run[0], l_run[0]);
            sm_ml[cw * 16 + g + 8] = make_float2(m_run[1], l_run[1]);
        }
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < M_TILES * 16 * kHeadDim; idx += Cfg::kThreads) {
        const int c = idx & (kHeadDim - 1);
        const int hr = (idx >> 7) & 15;
        const int tile = idx >> 11;
        const int head = tile * 16 + hr;
        if (head >= h) continue;
        float top = -INFINITY;
#pragma unroll
        for (int w = 0; w < kRowWarps; ++w) top = fmaxf(top, sm_ml[(w * M_TILES + tile) * 16 + hr].x);
        float num = 0.f, den = 0.f;
#pragma unroll
        for (int w = 0; w < kRowWarps; ++w) {
            const int src = w * M_TILES + tile;                          // consumer warp (rw = w, mt = tile)
            const float2 ml = sm_ml[src * 16 + hr];
            const float wt = fast_exp2(ml.x - top);                      // a warp without tiles: exp2(-inf) = 0
            den = fmaf(wt, ml.y, den);
            num = fmaf(wt, sm_acc[((size_t)src * 16 + hr) * kHeadDim + c], num);
        }
        const size_t unit = (size_t)seq * h + head;
        if (n_splits == 1) {
            o[unit * kHeadDim + c] = num / den;
        } else {
            const size_t slot = unit * n_splits + split;
            part_acc[slot * kHeadDim + c] = num;
            if (c == 0) part_ml[slot] = make_float2(top, den);
        }
    }
}

}  // namespace mqa
