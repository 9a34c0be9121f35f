// Second pass of the split-m step: merge the per-split (max, sum, weighted sum) partials of
// one (sequence, head) into o.  With M = max_s M_s,
//     o = sum_s e^{M_s - M} acc_s / sum_s e^{M_s - M} l_s,
// (maxima are stored multiplied by log2(e), so each weight is one exp2 of a difference)
// the same softmax re-associated; splits that start at or beyond lens[b] hold nothing and are
// skipped.  One CTA per (sequence, head).
#pragma once
#include "common.cuh"

namespace mqa {

// Partials layout in the workspace (units = b*h, S = n_splits):
//   ml  : float2 [units][S]        (M_s * log2(e), l_s)
//   acc : float  [units][S][128]
__host__ __device__ inline size_t partial_ml_bytes(size_t units, int S) {
    size_t bytes = units * (size_t)S * 2 * sizeof(float);
    return (bytes + 255) & ~(size_t)255;
}
__host__ __device__ inline size_t partial_acc_bytes(size_t units, int S) {
    return units * (size_t)S * kHeadDim * sizeof(float);
}

// Threads: 128 columns x GROUPS piece groups.  Group g takes pieces g, g + GROUPS, ...;
// a thread fetches its column of up to kCombineEager of them in one go (the addresses do not depend
// on the weights), so merging a few dozen pieces costs one round trip to L2, not one per piece.
// The host picks the shape by the most pieces a sequence can have: GROUPS = 1 (128 threads, 8 pieces in flight
// per thread) up to kCombineEager pieces, GROUPS = 4 (512 threads, 8 in flight) up to 4 * kCombineEager, and
// GROUPS = 5 (still 4 thread groups, 40 in flight per thread: 160 pieces in one go) beyond.
constexpr int kCombineEager = 8;
constexpr int kCombineManyGroups = 5;

// Merge `n` pieces of one (sequence, head).  ml_of(i) / acc_of(i) give piece i's (max, sum) and the address of
// its 128 accumulators; a piece whose max is -inf is skipped entirely (it may never have been written).
template <int kCombineShape, typename MlOf, typename AccOf>
__device__ __forceinline__ void merge_pieces(int n, MlOf ml_of, AccOf acc_of, float* __restrict__ out) {
    constexpr int kCombineGroups = kCombineShape >= 4 ? 4 : 1;
    constexpr int kCombineThreads = kHeadDim * kCombineGroups;
    constexpr int kCombineEager = kCombineShape == kCombineManyGroups ? 40 : 8;     // loads in flight per thread
    __shared__ float m_s[1024], l_s[1024];
    __shared__ float num_s[kCombineGroups][kHeadDim], den_s[kCombineGroups];
    const int c = threadIdx.x & (kHeadDim - 1), g = threadIdx.x >> 7;
    float a[kCombineEager];
#pragma unroll
    for (int e = 0; e < kCombineEager; ++e) {
        const int i = g + e * kCombineGroups;
        a[e] = i < n ? __ldcg(acc_of(i) + c) : 0.f;
    }
    for (int i = threadIdx.x; i < n; i += kCombineThreads) {
        const float2 ml = ml_of(i);
        m_s[i] = ml.x;
        l_s[i] = ml.y;
    }
    __syncthreads();
    float top = -INFINITY;
    for (int i = 0; i < n; ++i) top = fmaxf(top, m_s[i]);
    if (top == -INFINITY) {                                // nothing but empty pieces: the empty prefix gives zeros
        if (g == 0) out[c] = 0.f;
        return;
    }
    float num = 0.f, den = 0.f;
#pragma unroll
    for (int e = 0; e < kCombineEager; ++e) {
        const int i = g + e * kCombineGroups;
        if (i < n) {
            const float w = fast_exp2(m_s[i] - top);
            if (w != 0.f) { den = fmaf(w, l_s[i], den); num = fmaf(w, a[e], num); }   // never multiply an unwritten slot
        }
    }
    for (int i0 = g + kCombineEager * kCombineGroups; i0 < n; i0 += kCombineEager * kCombineGroups) {
#pragma unroll
        for (int e = 0; e < kCombineEager; ++e) {
            const int i = i0 + e * kCombineGroups;
            a[e] = i < n ? __ldcg(acc_of(i) + c) : 0.f;
        }
#pragma unroll
        for (int e = 0; e < kCombineEager; ++e) {
            const int i = i0 + e * kCombineGroups;
            if (i < n) {
                const float w = fast_exp2(m_s[i] - top);
                if (w != 0.f) { den = fmaf(w, l_s[i], den); num = fmaf(w, a[e], num); }
            }
        }
    }
    num_s[g][c] = num;
    if (c == 0) den_s[g] = den;
    __syncthreads();
    if (g == 0) {
#pragma unroll
        for (int k = 1; k < kCombineGroups; ++k) { num += num_s[k][c]; den += den_s[k]; }
        out[c] = num / den;
    }
}

template <int GROUPS>
__global__ void __launch_bounds__(kHeadDim * (GROUPS >= 4 ? 4 : 1))
combine_splits_kernel(const float2* __restrict__ part_ml, const float* __restrict__ part_acc,
                      const int32_t* __restrict__ lens, float* __restrict__ o,
                      int h, int m_max, int chunk_rows, int n_splits, int len_bias, int32_t* __restrict__ lens_advance) {
    const size_t u = blockIdx.x;
    grid_dependency_wait();          // the partials come from the kernel before this one
    // lens == nullptr: every split wrote its piece (an empty one has max = -inf) and nobody here looks at lens, so
    // the CTA of a sequence's first head may move it on (lens_advance: the append-and-attend step)
    int live = n_splits;
    if (lens != nullptr) {
        int L = biased_len(lens[u / h], m_max, len_bias);
        L = L < 0 ? 0 : (L > m_max ? m_max : L);
        live = (L + chunk_rows - 1) / chunk_rows;
        if (live > n_splits) live = n_splits;
    } else if (lens_advance != nullptr && u % h == 0 && threadIdx.x == 0) {
        const int raw = lens_advance[u / h];
        if (raw >= 0 && raw < m_max) lens_advance[u / h] = raw + 1;
    }
    if (live == 0) {
        if (threadIdx.x < kHeadDim) o[u * kHeadDim + threadIdx.x] = 0.f;
        return;
    }
    const float2* ml = part_ml + u * n_splits;
    const float* acc = part_acc + u * (size_t)n_splits * kHeadDim;
    merge_pieces<GROUPS>(live, [&](int i) { return __ldcg(ml + i); }, [&](int i) { return acc + (size_t)i * kHeadDim; },
                 o + u * kHeadDim);
}

// The same second pass for up to kCombineEager pieces per (sequence, head), one WARP per (sequence, head): a lane takes four
// of the 128 columns, asks for its part of every piece and for the (maximum, sum) pairs in one go, and merges them in piece
// order with the arithmetic of merge_pieces (the same bits).  No shared memory, no barrier: eight units per CTA, so the
// 4096 units of 32 sequences x 128 query rows are one wave of 512 CTAs (one CTA per unit took 7.5 us there, this 2-3).
constexpr int kCombineFewWarps = 8;
__global__ void __launch_bounds__(kCombineFewWarps * 32)
combine_few_kernel(const float2* __restrict__ part_ml, const float* __restrict__ part_acc, const int32_t* __restrict__ lens,
                   float* __restrict__ o, int h, int m_max, int chunk_rows, int n_splits, int len_bias,
                   int32_t* __restrict__ lens_advance, size_t units) {
    const int lane = threadIdx.x & 31;
    const size_t u = (size_t)blockIdx.x * kCombineFewWarps + (threadIdx.x >> 5);
    grid_dependency_wait();          // the partials come from the kernel before this one
    if (u >= units) return;
    int live = n_splits;
    if (lens != nullptr) {
        int L = biased_len(lens[u / h], m_max, len_bias);
        L = L < 0 ? 0 : (L > m_max ? m_max : L);
        live = (L + chunk_rows - 1) / chunk_rows;
        if (live > n_splits) live = n_splits;
    } else if (lens_advance != nullptr && u % h == 0 && lane == 0) {
        const int raw = lens_advance[u / h];
        if (raw >= 0 && raw < m_max) lens_advance[u / h] = raw + 1;
    }
    float4* out = reinterpret_cast<float4*>(o + u * kHeadDim) + lane;
    const float2* ml_p = part_ml + u * n_splits;
    const float4* acc_p = reinterpret_cast<const float4*>(part_acc + u * (size_t)n_splits * kHeadDim) + lane;
    float2 ml[kCombineEager];
    float4 a[kCombineEager];
#pragma unroll
    for (int i = 0; i < kCombineEager; ++i) {
        ml[i] = make_float2(-INFINITY, 0.f);
        a[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (i < live) {
            ml[i] = __ldcg(ml_p + i);
            a[i] = __ldcg(acc_p + (size_t)i * (kHeadDim / 4));
        }
    }
    float top = -INFINITY;
#pragma unroll
    for (int i = 0; i < kCombineEager; ++i) top = fmaxf(top, ml[i].x);
    if (live == 0 || top == -INFINITY) {               // the empty prefix, or nothing but empty pieces: zeros
        *out = make_float4(0.f, 0.f, 0.f, 0.f);
        return;
    }
    float den = 0.f;
    float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int i = 0; i < kCombineEager; ++i) {
        if (i < live) {
            const float w = fast_exp2(ml[i].x - top);
            if (w != 0.f) {                               // never multiply an unwritten slot
                den = fmaf(w, ml[i].y, den);
                num.x = fmaf(w, a[i].x, num.x); num.y = fmaf(w, a[i].y, num.y);
                num.z = fmaf(w, a[i].z, num.z); num.w = fmaf(w, a[i].w, num.w);
            }
        }
    }
    *out = make_float4(num.x / den, num.y / den, num.z / den, num.w / den);
}

}  // namespace mqa
