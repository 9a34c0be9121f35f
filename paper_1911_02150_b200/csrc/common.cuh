// Shared device helpers for the decode-attention kernels (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace mqa {

constexpr int kHeadDim = 128;                 // k == v == 128 (Section 4.1: d_k = d_v = 128)
constexpr int kRowBytes = kHeadDim * 2;       // one bf16 cache row
constexpr float kLog2e = 1.4426950408889634f;

// status bits (mirrors include/mqa_decode.h)
constexpr int kStatusAppendFull = 1;
constexpr int kStatusAppendNegative = 2;
constexpr int kStatusLenClamped = 4;
constexpr int kStatusPipelineTimeout = 8;

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// 16-byte read-only global load that does not allocate in L1 (each cache byte is used once).
__device__ __forceinline__ uint4 ldg_stream(const void* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}

// Programmatic dependent launch.  grid_dependency_wait(): block until the kernels this launch was
// made dependent on have finished and their writes are visible (a no-op for an ordinary launch).
// grid_launch_dependents(): allow the next kernel in the stream, if it was launched as a
// programmatic dependent, to start its prologue while this grid is still running.  Every kernel
// here waits first and lets its dependents start afterwards: with second-pass kernels that let
// theirs start before their own wait, a decoding loop of four kernels per step gave results that
// differed from run to run.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;"); }

// Clamp a sequence length into [0, m_max]; flag the status word if it had to move.
__device__ __forceinline__ int clamp_len(int L, int m_max, int32_t* status) {
    if (L < 0 || L > m_max) {
        if (status) atomicOr(status, kStatusLenClamped);
        L = L < 0 ? 0 : m_max;
    }
    return L;
}

// Rows to attend over when the caller's lens[] still holds the count from before this step's append
// (bias = 1): a sequence that could take the new row (0 <= lens < m_max) has one more row than lens says.
__device__ __forceinline__ int biased_len(int raw, int m_max, int bias) {
    return (bias && raw >= 0 && raw < m_max) ? raw + 1 : raw;
}

}  // namespace mqa
