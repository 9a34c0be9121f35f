// Local multi-query attention, one decoding step (Section 4.1: a position attends to itself and the previous
// window - 1 positions; Section 4.3: the memory tensors padded to the window size).  The cache of a sequence is a
// ring of `window` rows: the new token's key/value row goes to row pos % window and the h heads attend over the
// min(pos + 1, window) rows that hold tokens (the order of rows does not matter to a softmax).
//
// A window is a few 32-row tiles (the paper's is one), so the work of a sequence is one warp's: 16 KiB of K and V
// per tile, brought in by the warp's own TMA copies into the warp's own stage of shared memory, and the same
// tensor-core tile routine as the fixed-split kernel (consume_tile: mma.sync m16n8k16 with the heads as M rows,
// online softmax in registers, P as bf16 hi + lo parts).  No CTA-wide barrier, no merge between warps: a warp
// loads its query fragments, walks its tiles and writes o from its accumulators.  A CTA is kLocalWarps independent
// warps, so a batch of a thousand sequences is one wave of CTAs (with one CTA per sequence and 64 KiB of stages each
// it was several).  More than 16 heads: the warp goes over the window once per 16 heads (the tiles come from L2).
#pragma once
#include "decode_mma.cuh"

namespace mqa {

constexpr int kLocalWarps = 8;                          // sequences per CTA
constexpr int kLocalThreads = kLocalWarps * 32;
constexpr int kLocalSmemBytes = kLocalWarps * kStageBytes + 1024 /* alignment slack */ + kLocalWarps * 8 /* barriers */;

__global__ void __launch_bounds__(kLocalThreads, 1)
mqa_decode_local_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                        const uint32_t* __restrict__ q, const uint4* __restrict__ k_new, const uint4* __restrict__ v_new,
                        uint4* __restrict__ K, uint4* __restrict__ V, int32_t* __restrict__ pos, float* __restrict__ o,
                        int32_t* __restrict__ status, int b, int h, int window, int advance) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int seq = blockIdx.x * kLocalWarps + warp;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* stages = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);     // the 128-byte swizzle repeats every 1 KiB
    const uint32_t stage_s = smem_addr(stages) + warp * kStageBytes;                    // this warp's K and V tile
    const uint32_t bar = smem_addr(stages + kLocalWarps * kStageBytes) + warp * 8;      // this warp's barrier
    if (lane == 0) {
        if (warp == 0) { prefetch_tensormap(&map_k); prefetch_tensormap(&map_v); }
        mbar_init(bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();
    grid_dependency_wait();          // pos, q and the new row may come from the kernel before
    grid_launch_dependents();
    if (seq >= b) return;            // (the whole warp: nothing is in flight)

    // the new row's pieces are asked for before pos (two loads in flight): lanes 0-15 the key row, 16-31 the value row
    const uint4 row_piece = (lane < 16 ? k_new : v_new)[(size_t)seq * (kRowBytes / 16) + (lane & 15)];
    const int raw = pos[seq];
    const size_t units = (size_t)seq * h;
    if (raw < 0) {                   // no token position: no row written, zeros, flagged
        if (lane == 0 && status) atomicOr(status, kStatusAppendNegative | kStatusLenClamped);
        for (int i = lane; i < h * (kHeadDim / 4); i += 32) reinterpret_cast<float4*>(o + units * kHeadDim)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        return;
    }
    {
        const size_t dst = ((size_t)seq * window + raw % window) * (kRowBytes / 16) + (lane & 15);
        if (lane < 16) K[dst] = row_piece; else V[dst] = row_piece;
        asm volatile("fence.proxy.async;" ::: "memory");    // the copy engine must see the row
        __syncwarp();
    }
    const int L = raw + 1 < window ? raw + 1 : window;       // rows that hold tokens
    const int n_tiles = (L + kTileRows - 1) / kTileRows;
    const int row_base = seq * window;                       // row coordinate in the [b * window, 128] view

    LaneOffsets off;
    off.init(lane);
    const int g = lane >> 2, t4 = lane & 3;
    bool ok = true;
    int use = 0;                                             // copies of a tile into the stage so far (parity of the barrier)
    for (int mt = 0; mt * 16 < h && ok; ++mt) {              // 16 heads at a time
        uint32_t qa[8][4];
        load_q_fragments(qa, q, (size_t)seq, h, mt, lane);
        WarpState st;
        st.reset();
        for (int i = 0; i < n_tiles && ok; ++i, ++use) {
            if (lane == 0) {
                mbar_expect_tx(bar, kStageBytes);
                const int y = row_base + i * kTileRows;      // (a tile may run past the window: rows masked by index below)
                tma_load_2d(stage_s, &map_k, 0, y, bar);
                tma_load_2d(stage_s + kBoxBytes, &map_k, kBoxCols, y, bar);
                tma_load_2d(stage_s + 2 * kBoxBytes, &map_v, 0, y, bar);
                tma_load_2d(stage_s + 3 * kBoxBytes, &map_v, kBoxCols, y, bar);
            }
            ok = mbar_wait(bar, use & 1);
            if (!ok) break;                                  // (the copy may still land: see the end of the kernel)
            consume_tile<true>(st, qa, off, stage_s, stage_s + 2 * kBoxBytes, kBoxBytes, i * kTileRows, L, lane);
            // the tile was read through the generic proxy and the next copy writes the stage through the async proxy
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
        }
        if (!ok) break;
        // sums over the four lanes that share a head, then o = accumulators / sum, straight from the registers
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            st.l[r] += __shfl_xor_sync(0xffffffffu, st.l[r], 1);
            st.l[r] += __shfl_xor_sync(0xffffffffu, st.l[r], 2);
        }
        const float inv0 = 1.f / st.l[0], inv1 = 1.f / st.l[1];
        const int head0 = mt * 16 + g, head1 = head0 + 8;
#pragma unroll
        for (int vt = 0; vt < 16; ++vt) {
            if (head0 < h)
                *reinterpret_cast<float2*>(o + (units + head0) * kHeadDim + vt * 8 + t4 * 2) = make_float2(st.acc[vt][0] * inv0, st.acc[vt][1] * inv0);
            if (head1 < h)
                *reinterpret_cast<float2*>(o + (units + head1) * kHeadDim + vt * 8 + t4 * 2) = make_float2(st.acc[vt][2] * inv1, st.acc[vt][3] * inv1);
        }
    }
    if (!ok) {
        // a wait ran out: before the warp leaves (and with it, perhaps, the CTA and its shared memory), give the copy
        // one more bounded wait; flag the status word; o of this sequence is not valid
        mbar_wait(bar, use & 1);
        if (lane == 0 && status) atomicOr(status, kStatusPipelineTimeout);
        return;
    }
    if (advance && lane == 0) pos[seq] = raw + 1;            // every lane read pos[seq] before the first __syncwarp above
}

}  // namespace mqa
