// kv_cache_append kernel: one CTA per sequence copies the new token's key and value row of
// every cache head into row lens[b] (the in-place form of the concatenation on the memory
// axis in Sections 2.4 and 3).  Rows move as 16-byte words and are never interpreted.
#pragma once
#include "common.cuh"

namespace mqa {

constexpr int kAppendThreads = 256;  // 8 warps: one (cache head) row pair per warp per pass

__global__ void __launch_bounds__(kAppendThreads)
kv_cache_append_kernel(uint4* __restrict__ K, uint4* __restrict__ V,
                       const uint4* __restrict__ k_new, const uint4* __restrict__ v_new,
                       int32_t* __restrict__ lens, int advance, int32_t* __restrict__ status,
                       int kv_heads, int m_max) {
    const int bi = blockIdx.x;
    grid_dependency_wait();          // lens may come from the kernel before this one
    grid_launch_dependents();        // the step that follows may set itself up; it waits before reading
    const int row = lens[bi];
    if (row < 0 || row >= m_max) {   // uniform over the CTA
        if (threadIdx.x == 0 && status)
            atomicOr(status, row < 0 ? kStatusAppendNegative : kStatusAppendFull);
        return;
    }
    constexpr int kVecPerRow = kRowBytes / 16;               // 16 uint4 per row
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int vec = lane & (kVecPerRow - 1);
    const bool is_v = lane >= kVecPerRow;                    // lanes 0-15 copy K, 16-31 copy V
    for (int g = warp; g < kv_heads; g += kAppendThreads / 32) {
        const size_t src = ((size_t)bi * kv_heads + g) * kVecPerRow + vec;
        const size_t dst = (((size_t)bi * kv_heads + g) * m_max + row) * kVecPerRow + vec;
        if (is_v) V[dst] = v_new[src]; else K[dst] = k_new[src];
    }
    if (advance) {
        __syncthreads();             // every warp has read lens[bi] before it moves
        if (threadIdx.x == 0) lens[bi] = row + 1;
    }
}

// The host-buffer step's inputs (q, the new key row, the new value row) from pinned host memory that the device can
// address into the staging buffer, 16 bytes per thread and turn.  A kernel rather than a copy-engine transfer so that the
// attention kernel behind it may set itself up and fetch its first stages meanwhile: like every kernel here it waits for
// what is older, then lets its dependent start, and writes nothing but the staging buffer.
constexpr int kStageInThreads = 256;
struct StageInPart { const uint4* src; uint4* dst; unsigned n16; };

__global__ void __launch_bounds__(kStageInThreads)
stage_in_kernel(StageInPart q, StageInPart k_new, StageInPart v_new) {
    grid_dependency_wait();          // the step before may still read the staging buffer
    grid_launch_dependents();
    const unsigned stride = gridDim.x * kStageInThreads;
    const StageInPart parts[3] = {q, k_new, v_new};
#pragma unroll
    for (int p = 0; p < 3; ++p)
        for (unsigned i = blockIdx.x * kStageInThreads + threadIdx.x; i < parts[p].n16; i += stride)
            parts[p].dst[i] = __ldcv(parts[p].src + i);      // (host memory: read afresh, never from a cache line of an earlier step)
}

}  // namespace mqa
