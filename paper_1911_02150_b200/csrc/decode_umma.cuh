// Persistent multi-query decode kernel on the 5th-generation tensor cores (tcgen05 + TMEM) for
// head counts where the register-fragment mma.sync path runs out of issue slots and shared-memory
// bandwidth (h > 16).  Same step as the other kernels (Section 3: logits = einsum(bhk,bmk->bhm),
// softmax over m, o = einsum(bhm,bmv->bhv)), same equal-share scheduling, slots and second pass
// as mqa_decode_stream_mma_kernel; what changes is who does the two contractions:
//
//   producer warp   TMA: the segment's Q (64 head rows x 128) once, then K and V in 64-row stages
//   MMA warps       one thread each issues the tcgen05.mma of   S[64 heads x 64 rows] = Q K_stage^T   (TMEM)
//                                                    O[64 heads x 128]    += P V_stage     (TMEM)
//                   operands are read by the tensor core straight from the TMA-written shared
//                   memory (K row-major = K-major B; V row-major = MN-major B), so K and V are
//                   read from shared memory once for all heads and no fragment ever enters a register
//   softmax warps   the M=64 accumulator puts row r in TMEM lane 32*(r/16) + r%16, one row per thread
//                   of warp r/16: tcgen05.ld the logits, exact online softmax in fp32 registers, P
//                   written to shared memory as bf16 hi + lo (K-major A operand), O rescaled in TMEM
//                   on the rare stages where a row's maximum moves.  With 32 heads or fewer the 64
//                   rows hold R = 2 or 4 copies of the heads (Q is loaded R times); copy c takes the
//                   c-th part of each stage's 64 cache rows, so every softmax warp has work and a
//                   thread handles 64/R logits per stage.  The R partial results of a head are
//                   merged when the segment ends.
//
// Everything between the roles is an mbarrier; every wait is bounded (see mbar_wait).
#pragma once
#include <cuda.h>

#include "decode_mma.cuh"

namespace mqa {

constexpr int kUmmaStageRows = 64;                               // cache rows per stage
constexpr int kUmmaBoxBytes = kUmmaStageRows * 128;              // 8 KiB: 64 rows x 128 bytes
constexpr int kUmmaStageBytes = 4 * kUmmaBoxBytes;               // K lo, K hi, V lo, V hi = 32 KiB
constexpr int kUmmaStages = 5;
constexpr int kUmmaQBytes = 2 * 64 * 128;                        // 64 head rows x 128 columns bf16 = 16 KiB
constexpr int kUmmaSoftmaxWarps = 4;                             // heads 0..63
constexpr int kUmmaProducerWarp = 4, kUmmaMmaWarp = 5, kUmmaPvWarp = 6;   // two issuing threads: S = Q K^T, and O += P V
constexpr int kUmmaThreads = 7 * 32;
// TMEM columns: S0 [0,64) S1 [64,128) O [128,256); P as bf16 pairs, two buffers of hi [32 cols] + lo [32 cols]
constexpr int kUmmaTmemCols = 512;
constexpr int kTmemO = 128, kTmemP = 256;
constexpr int kUmmaPrefixBytes = (kStreamMaxSeqs + 1) * 4 + 12;
constexpr int kUmmaXchgBytes = 48 * 32 * 4 + 48 * 8;              // merge of the head copies: 48 rows x (32 columns + (m, l))
constexpr int kUmmaSmemBytes = kUmmaStages * kUmmaStageBytes + 2 * kUmmaQBytes + kUmmaPrefixBytes +
                               kUmmaXchgBytes + 512 /* barriers */ + 1024 /* alignment slack */;
static_assert(kUmmaSmemBytes <= 227 * 1024, "exceeds the shared memory of one SM");

// ---- tcgen05 wrappers ----------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem desc] * B[smem desc]; bf16 inputs, fp32 accumulate
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// D[tmem] (+)= A[tmem, bf16 pairs, one row per lane] * B[smem desc]
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t (&r)[8]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]) : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
                   "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,"
        "%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,"
        "%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
          "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
          "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}
// COLS (16, 32 or 64) consecutive fp32 columns of this thread's TMEM lane
template <int COLS>
__device__ __forceinline__ void tmem_ld_cols(uint32_t taddr, uint32_t (&r)[COLS]) {
    if constexpr (COLS == 16) {
        tmem_ld16(taddr, r);
    } else {
#pragma unroll
        for (int c = 0; c < COLS / 32; ++c) tmem_ld32(taddr + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&r[c * 32]));
    }
}
template <int WORDS>
__device__ __forceinline__ void tmem_st_words(uint32_t taddr, const uint32_t (&r)[WORDS]) {
    if constexpr (WORDS == 8) tmem_st8(taddr, r);
    else if constexpr (WORDS == 16) tmem_st16(taddr, r);
    else tmem_st32(taddr, r);
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle (layout type 2), descriptor version 1.
// lbo/sbo in bytes.  K-major operand: 8-row groups `sbo` apart (lbo unused, 16).  MN-major operand:
// 64-element blocks along M/N `lbo` apart, 8-row groups along K `sbo` apart.
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_byte_addr, uint32_t lbo, uint32_t sbo) {
    const uint64_t lo = (uint64_t)((smem_byte_addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo >> 4) & 0x3FFFu) << 16);
    const uint64_t hi = (uint64_t)((sbo >> 4) & 0x3FFFu) | (1ull << 14) | (2ull << 29);
    return lo | (hi << 32);
}
// Instruction descriptor: fp32 accumulator, bf16 A and B, M x N tile, B optionally MN-major.
__host__ __device__ constexpr uint32_t umma_idesc(int M, int N, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(N >> 3) << 17) |
           ((uint32_t)(M >> 4) << 24);
}

// R = copies of the heads among the 64 accumulator rows: 4 (h <= 16), 2 (h <= 32) or 1 (h <= 64).
template <int R>
__global__ void __launch_bounds__(kUmmaThreads, 1)
mqa_decode_stream_umma_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                              const __grid_constant__ CUtensorMap map_k_sub, const __grid_constant__ CUtensorMap map_v_sub,
                              const __grid_constant__ CUtensorMap map_q,
                              const int32_t* __restrict__ lens, float* __restrict__ o, int2* __restrict__ seq_span,
                              float2* __restrict__ part_ml, float* __restrict__ part_acc, int32_t* __restrict__ status,
                              int b, int h, int m_max) {
    const int cta = blockIdx.x, G = gridDim.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int H16 = R == 4 ? 16 : (R == 2 ? 32 : ((h + 15) & ~15));   // rows one copy of the heads takes
    const int n_sm_warps = R > 1 ? 4 : (H16 >> 4);          // softmax warps whose rows hold real heads
    constexpr int kCpr = kUmmaStageRows / R;                // stage columns (cache rows) per copy

    extern __shared__ uint8_t smem_raw[];
    uint8_t* stages = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);
    uint8_t* q_buf = stages + kUmmaStages * kUmmaStageBytes;            // 2 x 16 KiB
    int* prefix = reinterpret_cast<int*>(q_buf + 2 * kUmmaQBytes);      // [b + 1]
    float* xchg_o = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(prefix) + kUmmaPrefixBytes / 8 * 8);   // [48][32]
    float2* xchg_ml = reinterpret_cast<float2*>(xchg_o + 48 * 32);                                              // [48]
    uint64_t* bars = reinterpret_cast<uint64_t*>(xchg_ml + 48);
    const uint32_t stages_s = smem_addr(stages), q_s = smem_addr(q_buf);
    // barrier table
    const uint32_t kv_full = smem_addr(bars), kv_empty = kv_full + kUmmaStages * 8;
    const uint32_t q_full = kv_empty + kUmmaStages * 8, q_empty = q_full + 16;
    const uint32_t s_ready = q_empty + 16, s_free = s_ready + 16;
    const uint32_t p_ready = s_free + 16, pv_done = p_ready + 16, o_free = pv_done + 16;
    __shared__ int timed_out, issued;
    __shared__ uint32_t tmem_base_slot;

    if (warp == kUmmaProducerWarp && lane == 0) {
        prefetch_tensormap(&map_k); prefetch_tensormap(&map_v); prefetch_tensormap(&map_k_sub);
        prefetch_tensormap(&map_v_sub); prefetch_tensormap(&map_q);
    }
    if (threadIdx.x == 0) {
        timed_out = 0;
        issued = 0;
        for (int s = 0; s < kUmmaStages; ++s) { mbar_init(kv_full + s * 8, 1); mbar_init(kv_empty + s * 8, 1); }
        for (int s = 0; s < 2; ++s) {
            mbar_init(q_full + s * 8, 1); mbar_init(q_empty + s * 8, 1);
            mbar_init(s_ready + s * 8, 1); mbar_init(s_free + s * 8, n_sm_warps);
            mbar_init(p_ready + s * 8, n_sm_warps); mbar_init(pv_done + s * 8, 1);
        }
        mbar_init(o_free, n_sm_warps);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == kUmmaMmaWarp) {                             // one warp owns the TMEM allocation
        tmem_alloc(smem_addr(&tmem_base_slot), kUmmaTmemCols);
        tmem_relinquish();
    }
    grid_dependency_wait();
    grid_launch_dependents();

    // ---- 32-row sub-tiles per sequence and their running sum (as in the mma.sync persistent kernel)
    for (int s = threadIdx.x; s < b; s += kUmmaThreads) {
        const int L = clamp_len(lens[s], m_max, cta == 0 ? status : nullptr);
        prefix[s + 1] = L > 0 ? (L + kTileRows - 1) / kTileRows + kBoundaryPenalty : 0;
        if (L == 0 && s % G == cta)
            for (int i = 0; i < h * kHeadDim; ++i) o[(size_t)s * h * kHeadDim + i] = 0.f;
    }
    if (threadIdx.x == 0) prefix[0] = 0;
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    if (warp < 4) {
        // a row of P is written only in the columns of its own copy; the rest stays zero for the whole kernel
        uint32_t z[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) z[i] = 0u;
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_st32(tmem_base + ((uint32_t)(warp * 32) << 16) + kTmemP + c * 32, z);
        tmem_wait_st();
        tc_fence_before();
    }
    if (warp == 0) {
        const int per = (b + 31) / 32;
        const int lo = 1 + lane * per, hi = min(b, lo + per - 1);
        int sum = 0;
        for (int s = lo; s <= hi; ++s) sum += prefix[s];
        int incl = sum;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int up = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += up;
        }
        int run = incl - sum;
        for (int s = lo; s <= hi; ++s) { run += prefix[s]; prefix[s] = run; }
    }
    __syncthreads();
    const long long T = prefix[b];
    const long long t_begin = (long long)cta * T / G, t_end = (long long)(cta + 1) * T / G;
    int s_first = 0;
    if (t_begin < t_end) {
        int lo = 0, hi = b - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (prefix[mid] <= t_begin) lo = mid; else hi = mid - 1;
        }
        s_first = lo;
        while (prefix[s_first + 1] <= t_begin) ++s_first;
    }
    constexpr int kSubs = kUmmaStageRows / kTileRows;       // 2 sub-tiles of 32 rows per stage

    if (warp == kUmmaProducerWarp) {
        // =============================================================== TMA producer
        if (lane == 0 && t_begin < t_end) {
            bool ok = true;
            int j = 0, seg = 0;
            ShareWalker walk{prefix, t_begin, t_end, s_first};
            Segment g;
            for (; ok && walk.next(g); ++seg) {
                const int s = g.s;
                const int qi = seg & 1;
                if (seg >= 2) ok = mbar_wait(q_empty + qi * 8, ((seg >> 1) - 1) & 1);
                if (!ok) break;
                mbar_expect_tx(q_full + qi * 8, R * H16 * kRowBytes);
#pragma unroll
                for (int c = 0; c < R; ++c) {               // R copies of the sequence's head rows (box = H16 rows x 64 columns)
                    const uint32_t d = q_s + qi * kUmmaQBytes + c * H16 * 128;
                    tma_load_2d(d, &map_q, 0, s * h, q_full + qi * 8);
                    tma_load_2d(d + kUmmaQBytes / 2, &map_q, kBoxCols, s * h, q_full + qi * 8);
                }
                for (int u = g.lo; u < g.hi && ok; u += kSubs, ++j) {
                    const int nsub = min(kSubs, g.hi - u);
                    const int stg = j % kUmmaStages;
                    if (j >= kUmmaStages) ok = mbar_wait(kv_empty + stg * 8, ((j / kUmmaStages) - 1) & 1);
                    if (!ok) break;
                    const uint32_t bar = kv_full + stg * 8;
                    const uint32_t dst = stages_s + stg * kUmmaStageBytes;
                    mbar_expect_tx(bar, nsub * kStageBytes);
                    const int y = s * m_max + u * kTileRows;
                    if (nsub == kSubs) {
                        tma_load_2d(dst, &map_k, 0, y, bar);
                        tma_load_2d(dst + kUmmaBoxBytes, &map_k, kBoxCols, y, bar);
                        tma_load_2d(dst + 2 * kUmmaBoxBytes, &map_v, 0, y, bar);
                        tma_load_2d(dst + 3 * kUmmaBoxBytes, &map_v, kBoxCols, y, bar);
                    } else {
                        tma_load_2d(dst, &map_k_sub, 0, y, bar);
                        tma_load_2d(dst + kUmmaBoxBytes, &map_k_sub, kBoxCols, y, bar);
                        tma_load_2d(dst + 2 * kUmmaBoxBytes, &map_v_sub, 0, y, bar);
                        tma_load_2d(dst + 3 * kUmmaBoxBytes, &map_v_sub, kBoxCols, y, bar);
                    }
                    issued = j + 1;
                }
            }
            if (!ok) atomicExch(&timed_out, 1);
        }
    } else if (warp == kUmmaMmaWarp) {
        // =============================================================== issuer of S = Q K^T
        // (one tcgen05.mma or commit costs this thread ~45 ns, measured; the two contractions of a stage are
        // therefore issued by two threads)
        if (lane == 0 && t_begin < t_end) {
            constexpr uint32_t kIdescS = umma_idesc(64, kUmmaStageRows, false);
            bool ok = true;
            int j = 0, seg = 0;
            ShareWalker walk{prefix, t_begin, t_end, s_first};
            Segment g;
            for (; walk.next(g); ++seg) {
                const int qi = seg & 1;
                if (ok) ok = mbar_wait(q_full + qi * 8, (seg >> 1) & 1);
                for (int u = g.lo; u < g.hi; u += kSubs, ++j) {
                    const int stg = j % kUmmaStages, sb = j & 1;
                    if (ok) ok = mbar_wait(kv_full + stg * 8, (j / kUmmaStages) & 1);
                    if (ok && j >= 2) ok = mbar_wait(s_free + sb * 8, ((j >> 1) - 1) & 1);
                    tc_fence_after();
                    if (ok) {
                        const uint32_t k_s = stages_s + stg * kUmmaStageBytes;
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks) {             // 8 k-steps of 16 columns; 4 per 64-column box
                            const uint64_t a = umma_desc(q_s + qi * kUmmaQBytes + (ks >> 2) * (kUmmaQBytes / 2) + (ks & 3) * 32, 16, 1024);
                            const uint64_t bd = umma_desc(k_s + (ks >> 2) * kUmmaBoxBytes + (ks & 3) * 32, 16, 1024);
                            umma_ss(tmem_base + sb * 64, a, bd, kIdescS, ks ? 1u : 0u);
                        }
                    }
                    tc_commit(s_ready + sb * 8);
                    if (u + kSubs >= g.hi) tc_commit(q_empty + qi * 8);   // last use of this segment's Q
                }
            }
            if (!ok) atomicExch(&timed_out, 1);
        }
    } else if (warp == kUmmaPvWarp) {
        // =============================================================== issuer of O += P V
        if (lane == 0 && t_begin < t_end) {
            constexpr uint32_t kIdescO = umma_idesc(64, kHeadDim, true);
            bool ok = true;
            int j = 0, seg = 0;
            ShareWalker walk{prefix, t_begin, t_end, s_first};
            Segment g;
            for (; walk.next(g); ++seg) {
                const int L = min(max(__ldg(lens + g.s), 0), m_max);
                const int parts = L >= kSingleRoundingMinRows ? 1 : 2;   // P hi only, or hi then lo (as the softmax warps wrote it)
                for (int u = g.lo; u < g.hi; u += kSubs, ++j) {
                    const int pb = j & 1;
                    if (ok) ok = mbar_wait(p_ready + pb * 8, (j >> 1) & 1);
                    if (ok && u == g.lo && seg >= 1) ok = mbar_wait(o_free, (seg - 1) & 1);   // the segment before has read O out
                    tc_fence_after();
                    const uint32_t v_s = stages_s + (j % kUmmaStages) * kUmmaStageBytes + 2 * kUmmaBoxBytes;
                    if (ok) {
                        for (int part = 0; part < parts; ++part) {
#pragma unroll
                            for (int kk = 0; kk < kUmmaStageRows / 16; ++kk) {
                                const uint32_t a = tmem_base + kTmemP + pb * 64 + part * 32 + kk * 8;   // 16 bf16 = 8 columns
                                const uint64_t bd = umma_desc(v_s + kk * 2048, kUmmaBoxBytes, 1024);
                                umma_ts(tmem_base + kTmemO, a, bd, kIdescO, (u == g.lo && part == 0 && kk == 0) ? 0u : 1u);
                            }
                        }
                    }
                    // S = Q K^T of this stage finished before its softmax began, so both K and V are free now
                    tc_commit(kv_empty + (j % kUmmaStages) * 8);
                    tc_commit(pv_done + pb * 8);                        // this P buffer is free, O is up to date
                }
            }
            if (!ok) atomicExch(&timed_out, 1);
        }
    } else {
        // =============================================================== softmax warps
        if (warp == 0) {                                    // second-pass bookkeeping, spread over the CTAs
            for (int s = cta + lane * G; s < b; s += G * 32) {
                const int t0 = prefix[s] + kBoundaryPenalty, t1 = prefix[s + 1];     // its real tiles on the line
                seq_span[s] = t1 > t0 ? make_int2(stream_owner(t0, T, G), stream_owner(t1 - 1, T, G)) : make_int2(0, 0);
            }
            if (cta == 0 && lane == 0) seq_span[b] = make_int2((int)T, G);
        }
        if (warp < n_sm_warps && t_begin < t_end) {
            const int row = warp * 16 + (lane & 15);        // accumulator row of this thread (lanes 16..31 hold none)
            const int head = row % H16, copy = row / H16;   // the copy is the same for a whole warp
            const bool live = lane < 16 && head < h;
            const int col0 = copy * kCpr;                   // this copy's columns of every stage
            const uint32_t lane_base = tmem_base + ((uint32_t)(warp * 32) << 16);
            const int sm_threads = n_sm_warps * 32, sm_tid = warp * 32 + lane;
                        bool ok = true;
            int j = 0, seg = 0;
            ShareWalker walk{prefix, t_begin, t_end, s_first};
            Segment g;
            for (; walk.next(g); ++seg) {
                const int s = g.s;
                const int L = min(max(__ldg(lens + s), 0), m_max);
                const bool whole = g.whole;
                const bool hilo = L < kSingleRoundingMinRows;    // long prefixes: one bf16 rounding of P is enough
                float m_run = -INFINITY, l_run = 0.f;
                for (int u = g.lo; u < g.hi; u += kSubs, ++j) {
                    const int sb = j & 1, stg = j % kUmmaStages;
                    // rows of this stage that count: what was fetched (the share may end mid-stage) and
                    // lies inside the prefix; always >= 1
                    const int fetched = min(kSubs, g.hi - u) * kTileRows;
                    const int valid = min(fetched, L - u * kTileRows);
                    if (ok) ok = mbar_wait(s_ready + sb * 8, (j >> 1) & 1);
                    tc_fence_after();
                    uint32_t r[kCpr];
                    tmem_ld_cols<kCpr>(lane_base + sb * 64 + col0, r);
                    tmem_wait_ld();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(s_free + sb * 8);             // S is in registers now
                    // ---- the stage's maximum for this row (its own columns only)
                    float top = -INFINITY;
#pragma unroll
                    for (int i = 0; i < kCpr; ++i)
                        if (col0 + i < valid) top = fmaxf(top, __uint_as_float(r[i]));   // select by index
                    // same rounding as below: the maximum's weight is exactly 1.  A copy whose columns
                    // are all beyond the prefix keeps its state.
                    const float m_new = fmaxf(m_run, __fmul_rn(top, kLog2e));
                    const float rescale = m_new == -INFINITY ? 1.f : fast_exp2(m_run - m_new);   // 0 on a copy's first columns
                    const bool moved = live && m_new > m_run && u != g.lo;   // O holds something to rescale
                    l_run *= rescale;
                    m_run = m_new;
                    // ---- P = exp2(S - max) as bf16 hi + lo pairs (two cache rows per 32-bit TMEM column)
                    uint32_t p_hi[kCpr / 2], p_lo[kCpr / 2];
#pragma unroll
                    for (int i = 0; i < kCpr; i += 2) {
                        const float p0 = col0 + i < valid ? fast_exp2(__fmul_rn(__uint_as_float(r[i]), kLog2e) - m_new) : 0.f;
                        const float p1 = col0 + i + 1 < valid ? fast_exp2(__fmul_rn(__uint_as_float(r[i + 1]), kLog2e) - m_new) : 0.f;
                        l_run += p0 + p1;
                        p_hi[i / 2] = pack_bf16(p0, p1);
                        if (hilo) p_lo[i / 2] = pack_bf16(p0 - bf16_lo(p_hi[i / 2]), p1 - bf16_hi(p_hi[i / 2]));
                    }
                    // this P buffer was last read by the P V of stage j-2
                    const int pb = j & 1;
                    if (j >= 2 && ok) ok = mbar_wait(pv_done + pb * 8, ((j >> 1) - 1) & 1);
                    if (__any_sync(0xffffffffu, moved)) {
                        // rare after the first stages: rescale this row of O in TMEM, between the P V of the
                        // stage before (waited for here) and the P V of this stage (not yet released)
                        if (ok) ok = mbar_wait(pv_done + (pb ^ 1) * 8, ((j - 1) >> 1) & 1);
                        tc_fence_after();
                        uint32_t x[32];
#pragma unroll 1
                        for (int c = 0; c < 4; ++c) {
                            tmem_ld32(lane_base + kTmemO + c * 32, x);
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i) x[i] = __float_as_uint(__uint_as_float(x[i]) * (moved ? rescale : 1.f));
                            tmem_st32(lane_base + kTmemO + c * 32, x);
                        }
                    }
                    tc_fence_after();
                    tmem_st_words<kCpr / 2>(lane_base + kTmemP + pb * 64 + (col0 >> 1), p_hi);
                    if (hilo) tmem_st_words<kCpr / 2>(lane_base + kTmemP + pb * 64 + 32 + (col0 >> 1), p_lo);
                    // a stage that runs past the prefix: the tensor core would multiply the zero weights
                    // with whatever lies there (NaN * 0 = NaN), so those V rows are cleared first
                    if (valid < kUmmaStageRows) {
                        const uint32_t v_s = stages_s + stg * kUmmaStageBytes + 2 * kUmmaBoxBytes;
                        for (int i = sm_tid; i < (kUmmaStageRows - valid) * 16; i += sm_threads) {
                            const int vrow = valid + (i >> 4), ch = i & 15;  // 16 chunks of 16 bytes per row
                            const uint32_t a = v_s + (ch >> 3) * kUmmaBoxBytes + vrow * 128 + ((ch & 7) << 4);
                            asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0u) : "memory");
                        }
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // cleared V visible to the tensor core
                    }
                    tmem_wait_st();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(p_ready + pb * 8);
                }
                // ---- segment done: wait for its last P V, merge the copies of each head, read O out of TMEM
                if (j >= 2 && ok) ok = mbar_wait(pv_done + (j & 1) * 8, ((j - 2) >> 1) & 1);        // P V of stage j-2 ...
                if (ok) ok = mbar_wait(pv_done + ((j - 1) & 1) * 8, ((j - 1) >> 1) & 1);           // ... and of the last stage
                tc_fence_after();
                const size_t slot = (size_t)cta + s;
                float w_own = 1.f, m_tot = m_run, l_tot = l_run;
                float w_other[R > 1 ? R - 1 : 1];
                if constexpr (R > 1) {
                    if (lane < 16 && copy > 0) xchg_ml[(copy - 1) * H16 + head] = make_float2(m_run, l_run);
                    named_barrier(2, 128);
                    if (copy == 0) {
#pragma unroll
                        for (int c = 1; c < R; ++c) m_tot = fmaxf(m_tot, xchg_ml[(c - 1) * H16 + head].x);
                        w_own = m_run == -INFINITY ? 0.f : fast_exp2(m_run - m_tot);   // copy 0 always holds the first row: finite
                        l_tot = l_run * w_own;
#pragma unroll
                        for (int c = 1; c < R; ++c) {
                            const float2 ml = xchg_ml[(c - 1) * H16 + head];
                            w_other[c - 1] = ml.x == -INFINITY ? 0.f : fast_exp2(ml.x - m_tot);
                            l_tot = fmaf(w_other[c - 1], ml.y, l_tot);
                        }
                    }
                }
                float* dst = whole ? o + ((size_t)s * h + head) * kHeadDim : part_acc + (slot * h + head) * kHeadDim;
                const float inv = whole ? 1.f / l_tot : 1.f;
                uint32_t x[32];
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    tmem_ld32(lane_base + kTmemO + c * 32, x);
                    tmem_wait_ld();
                    if constexpr (R > 1) {
                        if (lane < 16 && copy > 0) {
                            float4* put = reinterpret_cast<float4*>(xchg_o + ((copy - 1) * H16 + head) * 32);
#pragma unroll
                            for (int i = 0; i < 8; ++i) put[i] = make_float4(__uint_as_float(x[4 * i]), __uint_as_float(x[4 * i + 1]), __uint_as_float(x[4 * i + 2]), __uint_as_float(x[4 * i + 3]));
                        }
                        named_barrier(2, 128);
                        if (copy == 0) {
#pragma unroll
                            for (int cc = 1; cc < R; ++cc) {
                                const float4* get = reinterpret_cast<const float4*>(xchg_o + ((cc - 1) * H16 + head) * 32);
#pragma unroll
                                for (int i = 0; i < 8; ++i) {
                                    const float4 v4 = get[i];
                                    const float wgt = w_other[cc - 1];
                                    x[4 * i] = __float_as_uint(fmaf(wgt, v4.x, __uint_as_float(x[4 * i]) * (cc == 1 ? w_own : 1.f)));
                                    x[4 * i + 1] = __float_as_uint(fmaf(wgt, v4.y, __uint_as_float(x[4 * i + 1]) * (cc == 1 ? w_own : 1.f)));
                                    x[4 * i + 2] = __float_as_uint(fmaf(wgt, v4.z, __uint_as_float(x[4 * i + 2]) * (cc == 1 ? w_own : 1.f)));
                                    x[4 * i + 3] = __float_as_uint(fmaf(wgt, v4.w, __uint_as_float(x[4 * i + 3]) * (cc == 1 ? w_own : 1.f)));
                                }
                            }
                        }
                    }
                    if (live && copy == 0) {
#pragma unroll
                        for (int i = 0; i < 32; i += 4)
                            *reinterpret_cast<float4*>(dst + c * 32 + i) =
                                make_float4(__uint_as_float(x[i]) * inv, __uint_as_float(x[i + 1]) * inv,
                                            __uint_as_float(x[i + 2]) * inv, __uint_as_float(x[i + 3]) * inv);
                    }
                    if constexpr (R > 1) named_barrier(2, 128);              // the exchange buffer is free again
                }
                if (live && copy == 0 && !whole) part_ml[slot * h + head] = make_float2(m_tot, l_tot);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(o_free);         // the next segment may overwrite O
            }
            if (!ok) atomicExch(&timed_out, 1);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (timed_out && threadIdx.x == 0) {
        for (int s = 0; s < kUmmaStages && s < issued; ++s) {
            const int last_use = (issued - 1 - s) / kUmmaStages;
            mbar_wait(kv_full + s * 8, last_use & 1);
        }
        if (status) atomicOr(status, kStatusPipelineTimeout);
    }
    __syncthreads();
    if (warp == kUmmaMmaWarp) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kUmmaTmemCols);
    }
}

}  // namespace mqa
