// Split-m decode kernel on the CUDA cores: one CTA handles one split of the memory axis for
// one (sequence, head) "unit".  It is the multi-head step (Section 2.4: every head scans its
// own cache, 1 flop per byte, purely HBM-bound) and the general-h form of the multi-query step
// (Section 3), where `heads_per_cache` = h heads map onto the same cache.
//
// Mapping: a cache row is 256 bytes = 16 lanes x 16 bytes, so one warp-wide 16-byte load
// brings in two consecutive rows (lanes 0-15 row r, lanes 16-31 row r+1), fully coalesced.
// A lane keeps the 8 query values of its column chunk in registers, forms its 8-term share of
// q.K[row], and a 4-step butterfly over the 16 lanes of a half-warp finishes the dot.  The
// warp walks 16 rows per iteration (8 K loads + 8 V loads in flight per lane), keeps a
// running maximum and sum (online softmax, fp32; logits are scaled by log2(e) once so that
// every exponential is a bare exp2 and the maximum's weight is exactly 1) and a running
// weighted sum of V rows, its lane holding 8 of the 128 output columns.  Warps of a CTA are merged through shared memory
// at the end, and the CTA writes either the final o (single split) or its partial.
#pragma once
#include "combine.cuh"
#include "common.cuh"

namespace mqa {

constexpr int kSimtWarps = 4;
constexpr int kSimtThreads = kSimtWarps * 32;
constexpr int kSimtRowsPerIter = 16;   // rows one warp consumes per loop iteration

__global__ void __launch_bounds__(kSimtThreads)
decode_split_simt_kernel(const uint4* __restrict__ q, const uint4* __restrict__ K,
                         const uint4* __restrict__ V, const int32_t* __restrict__ lens,
                         float* __restrict__ o, float2* __restrict__ part_ml,
                         float* __restrict__ part_acc, int32_t* __restrict__ status,
                         int h, int heads_per_cache, int m_max, int chunk_rows, int n_splits, int len_bias) {
    const size_t u = blockIdx.x / n_splits;            // unit = sequence * h + head
    const int split = blockIdx.x % n_splits;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int half = lane >> 4, cl = lane & 15;

    grid_dependency_wait();          // lens and the newest cache row may come from the kernel before
    grid_launch_dependents();
    const int L = clamp_len(biased_len(lens[u / h], m_max, len_bias), m_max, threadIdx.x == 0 ? status : nullptr);
    const int r0 = split * chunk_rows;
    const int r1 = min(L, r0 + chunk_rows);
    if (r0 >= L) {                                     // nothing valid in this split
        if (n_splits == 1) o[u * kHeadDim + threadIdx.x] = 0.f;   // L == 0
        return;
    }

    constexpr int kVecPerRow = kRowBytes / 16;
    const uint4* Kc = K + (u / heads_per_cache) * (size_t)m_max * kVecPerRow + cl;
    const uint4* Vc = V + (u / heads_per_cache) * (size_t)m_max * kVecPerRow + cl;

    float qf[8];
    {
        const uint4 qv = q[u * kVecPerRow + cl];
        qf[0] = bf16_lo(qv.x); qf[1] = bf16_hi(qv.x); qf[2] = bf16_lo(qv.y); qf[3] = bf16_hi(qv.y);
        qf[4] = bf16_lo(qv.z); qf[5] = bf16_hi(qv.z); qf[6] = bf16_lo(qv.w); qf[7] = bf16_hi(qv.w);
    }

    float m_run = -INFINITY, l_run = 0.f;
    float acc[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) acc[c] = 0.f;

    for (int base = r0 + warp * kSimtRowsPerIter; base < r1; base += kSimtWarps * kSimtRowsPerIter) {
        uint4 kr[8], vr[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int row = base + 2 * i + half;
            if (row < r1) {
                kr[i] = ldg_stream(Kc + (size_t)row * kVecPerRow);
                vr[i] = ldg_stream(Vc + (size_t)row * kVecPerRow);
            } else {                                   // never touch rows past the prefix
                kr[i] = make_uint4(0, 0, 0, 0);
                vr[i] = make_uint4(0, 0, 0, 0);
            }
        }
        float s[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            float d = qf[0] * bf16_lo(kr[i].x);
            d = fmaf(qf[1], bf16_hi(kr[i].x), d);
            d = fmaf(qf[2], bf16_lo(kr[i].y), d);
            d = fmaf(qf[3], bf16_hi(kr[i].y), d);
            d = fmaf(qf[4], bf16_lo(kr[i].z), d);
            d = fmaf(qf[5], bf16_hi(kr[i].z), d);
            d = fmaf(qf[6], bf16_lo(kr[i].w), d);
            d = fmaf(qf[7], bf16_hi(kr[i].w), d);
            s[i] = d;
        }
#pragma unroll
        for (int off = 8; off >= 1; off >>= 1) {
#pragma unroll
            for (int i = 0; i < 8; ++i) s[i] += __shfl_xor_sync(0xffffffffu, s[i], off);
        }
        float top = -INFINITY;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            s[i] = (base + 2 * i + half < r1) ? s[i] * kLog2e : -INFINITY;   // select, never multiply
            top = fmaxf(top, s[i]);
        }
        top = fmaxf(top, __shfl_xor_sync(0xffffffffu, top, 16));  // row `base` is valid: finite
        const float m_new = fmaxf(m_run, top);
        const float rescale = fast_exp2(m_run - m_new);            // 0 on the first iteration
        m_run = m_new;
        l_run *= rescale;
#pragma unroll
        for (int c = 0; c < 8; ++c) acc[c] *= rescale;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float p = fast_exp2(s[i] - m_new);               // exactly 1 at the maximum, 0 when masked
            l_run += p;
            acc[0] = fmaf(p, bf16_lo(vr[i].x), acc[0]); acc[1] = fmaf(p, bf16_hi(vr[i].x), acc[1]);
            acc[2] = fmaf(p, bf16_lo(vr[i].y), acc[2]); acc[3] = fmaf(p, bf16_hi(vr[i].y), acc[3]);
            acc[4] = fmaf(p, bf16_lo(vr[i].z), acc[4]); acc[5] = fmaf(p, bf16_hi(vr[i].z), acc[5]);
            acc[6] = fmaf(p, bf16_lo(vr[i].w), acc[6]); acc[7] = fmaf(p, bf16_hi(vr[i].w), acc[7]);
        }
    }
    // the two half-warps saw different rows under the same running maximum
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 16);
#pragma unroll
    for (int c = 0; c < 8; ++c) acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], 16);

    __shared__ float sm_m[kSimtWarps], sm_l[kSimtWarps];
    __shared__ __align__(16) float sm_acc[kSimtWarps][kHeadDim];
    if (lane == 0) { sm_m[warp] = m_run; sm_l[warp] = l_run; }
    if (half == 0) {
        float4* dst = reinterpret_cast<float4*>(&sm_acc[warp][cl * 8]);
        dst[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
        dst[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
    }
    __syncthreads();

    const int c = threadIdx.x;                          // 128 threads, 128 output columns
    float top = sm_m[0];
#pragma unroll
    for (int w = 1; w < kSimtWarps; ++w) top = fmaxf(top, sm_m[w]);   // warp 0 always had rows
    float num = 0.f, den = 0.f;
#pragma unroll
    for (int w = 0; w < kSimtWarps; ++w) {
        const float wt = fast_exp2(sm_m[w] - top);                    // idle warp: exp2(-inf) = 0
        den = fmaf(wt, sm_l[w], den);
        num = fmaf(wt, sm_acc[w][c], num);
    }
    if (n_splits == 1) {
        o[u * kHeadDim + c] = num / den;
    } else {
        const size_t slot = u * n_splits + split;
        part_acc[slot * kHeadDim + c] = num;
        if (c == 0) part_ml[slot] = make_float2(top, den);
    }
}

}  // namespace mqa
