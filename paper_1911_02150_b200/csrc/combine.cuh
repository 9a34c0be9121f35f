// Second pass of the split-m step: merge the per-split (max, sum, weighted sum) partials of
// one (sequence, head) into o.  With M = max_s M_s,
//     o = sum_s e^{M_s - M} acc_s / sum_s e^{M_s - M} l_s,
// (maxima are stored multiplied by log2(e), so each weight is one exp2 of a difference)
// the same softmax re-associated; splits that start at or beyond lens[b] hold nothing and are
// skipped.  One CTA of 128 threads per (sequence, head): thread c owns output column c.
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

__global__ void __launch_bounds__(kHeadDim)
combine_splits_kernel(const float2* __restrict__ part_ml, const float* __restrict__ part_acc,
                      const int32_t* __restrict__ lens, float* __restrict__ o,
                      int h, int m_max, int chunk_rows, int n_splits, int len_bias) {
    const size_t u = blockIdx.x;
    const int c = threadIdx.x;
    grid_dependency_wait();          // the partials come from the kernel before this one
    int L = biased_len(lens[u / h], m_max, len_bias);
    L = L < 0 ? 0 : (L > m_max ? m_max : L);
    int live = (L + chunk_rows - 1) / chunk_rows;
    if (live > n_splits) live = n_splits;
    if (live == 0) {
        o[u * kHeadDim + c] = 0.f;
        return;
    }
    const float2* ml = part_ml + u * n_splits;
    const float* acc = part_acc + u * (size_t)n_splits * kHeadDim;
    float top = -INFINITY;
    for (int s = 0; s < live; ++s) top = fmaxf(top, ml[s].x);
    float num = 0.f, den = 0.f;
    for (int s = 0; s < live; ++s) {
        const float2 p = ml[s];
        const float w = fast_exp2(p.x - top);
        den = fmaf(w, p.y, den);
        num = fmaf(w, acc[(size_t)s * kHeadDim + c], num);
    }
    o[u * kHeadDim + c] = num / den;
}

}  // namespace mqa
