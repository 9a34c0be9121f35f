// Multi-query decode kernels on the tensor cores (Section 3: logits = einsum(bhk,bmk->bhm),
// softmax over m, o = einsum(bhm,bmv->bhv)) for sm_100a.
//
// A producer warp streams K and V rows HBM -> shared memory with TMA (cp.async.bulk.tensor,
// 128-byte swizzle) through a ring of stages guarded by full/empty mbarriers; every K/V byte is
// fetched from HBM once and is then used for ALL h heads, which is the whole point of the
// multi-query layout (h flops per byte instead of 1).  At h flops per byte the CUDA cores
// cannot keep up with HBM, so the two contractions run on the tensor cores with the heads as
// the M rows:
//     S[h x rows]   = Q[h x k] * K_tile^T          (bf16 mma, fp32 accumulate)
//     O[h x v]     += P[h x rows] * V_tile         (P = exp2(S - max), split into bf16 hi + lo
//                                                  parts so that the weights keep ~16 bits)
// Each consumer warp takes whole 32-row tiles round-robin and keeps its own online-softmax
// state (running max, running sum, fp32 accumulators) in registers.
//
// mqa_decode_split_mma_kernel runs one CTA per (sequence, fixed-size split) and is used when the
// whole problem is small (short caches, few sequences); large batches go to the persistent
// tcgen05 kernel (decode_umma.cuh).  The second half of this file is what the persistent kernel's
// schedule is made of: the line of 32-row tiles, its equal shares, segments, slots and the
// second-pass kernel that merges the slots of a sequence cut into many pieces.
//
// Rows at or beyond lens[b] are never used: their logits are replaced by -inf by index and
// their V fragments are zeroed by index (a NaN times a zero weight would still be a NaN).
#pragma once
#include <cuda.h>

#include "combine.cuh"
#include "common.cuh"

namespace mqa {

#ifdef MQA_DEBUG_TS
__device__ unsigned long long g_ts[256 * 32];
__device__ __forceinline__ unsigned long long dbg_ns() { unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t; }
#define TS(k) do { g_ts[blockIdx.x * 32 + (k)] = dbg_ns(); } while (0)
__device__ unsigned long long g_st[64 * 8];
#define ST(j, k) do { if (blockIdx.x == MQA_DEBUG_CTA && (j) < 64) g_st[(j) * 8 + (k)] = dbg_ns(); } while (0)
#else
#define TS(k) do { } while (0)
#define ST(j, k) do { } while (0)
#endif

constexpr int kTileRows = 32;                          // cache rows per pipeline stage
constexpr int kBoxCols = 64;                           // 64 bf16 = 128 bytes = one swizzle span
constexpr int kBoxBytes = kTileRows * kBoxCols * 2;    // 4 KiB
constexpr int kStageBytes = 4 * kBoxBytes;             // K lo, K hi, V lo, V hi = 16 KiB
constexpr int kRowWarps = 4;                           // consumer warps that share the tiles
constexpr long long kWaitLimitCycles = 2000000000ll;   // every mbarrier wait gives up after ~1 s of SM clock ...
constexpr uint32_t kWaitRounds = 1u << 24;             // ... or after this many polling rounds
// The limit in force, in SM clock cycles (mqa_set_wait_limit_cycles: a test shortens it to see a wait run out).
__device__ long long g_wait_limit_cycles = kWaitLimitCycles;
constexpr int kSingleRoundingMinRows = 1024;            // prefixes this long feed P to the tensor cores in one bf16 rounding
constexpr int kStreamMaxSeqs = 1024;                   // sequences the persistent kernel can index in shared memory

// Ring depth must be a multiple of kRowWarps: tile i lives in stage i % kStages and belongs to
// row-warp i % kRowWarps, so with this rule every use of a stage is waited on by the same warp.
// A parity wait can only tell the current phase from the one before it; a warp that skipped a
// use of a stage could mistake an old phase for the one it needs.
template <int M_TILES>
struct MmaCfg {                                        // fixed-split kernel
    static constexpr int kConsumerWarps = M_TILES * kRowWarps;
    static constexpr int kThreads = (kConsumerWarps + 1) * 32;
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
    const long long limit = g_wait_limit_cycles;
    for (uint32_t round = 0; round < kWaitRounds; ++round) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (clock64() - t0 > limit && clock64() - t0 > limit) return false;
    }
    return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
// The same copy with an L2 eviction policy for the lines it brings in (see l2_stream_policy).
__device__ __forceinline__ void tma_load_2d_hint(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar), "l"(policy) : "memory");
}
// Ask for a box of a tensor to be brought into L2 (nothing lands in shared memory, nothing to wait for).
__device__ __forceinline__ void tma_prefetch_l2_2d(const CUtensorMap* map, int x, int y) {
    asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(map), "r"(x), "r"(y) : "memory");
}
// Policy for data that is read once (read_once): its lines are the first to go, so that a pass over a cache larger
// than L2 does not push out what every launch needs again (q, lens, the workspace, the kernel's own code and
// parameters).  Otherwise the ordinary policy: a cache that fits in L2 is found there by the next step.
__device__ __forceinline__ uint64_t l2_stream_policy(bool read_once) {
    uint64_t policy;
    if (read_once)
        asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    else
        asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(policy));
    return policy;
}
// Bring a tensor map into the descriptor cache ahead of its first use by a copy.
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
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
__device__ __forceinline__ void named_barrier(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
// Counts towards a named barrier of `threads` threads without waiting for it.
__device__ __forceinline__ void named_barrier_arrive(int id, int threads) {
    asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// The append-and-attend step: the kernel that owns a sequence's last tile also writes the new token's key
// and value row (row lens[b]) into the cache before it fetches that tile, so the step attends over
// lens[b] + 1 rows without a separate append launch.
struct FusedArgs {
    const uint4* k_new;      // [b, 128] bf16 rows as 16-byte words; null = nothing to append
    const uint4* v_new;
    uint4* K;                // the cache, written at row lens[b]
    uint4* V;
};

// ---- the consumer warp's state and inner loop ------------------------------------------------
// Layout of a K or V tile in shared memory as TMA writes it: two 64-column boxes of 32 rows x
// 128 bytes; inside a box the 16-byte chunk index (0..7) is XORed with (row mod 8).
// An ldmatrix lane addresses row (8*j + lane%8) of its matrix, so (row mod 8) == lane%8 for every
// access and the swizzle folds into four per-lane offsets (one per chunk pair).
struct LaneOffsets {
    uint32_t k[4];   // K: [(lane/16)*8 + lane%8] row, chunk pair c -> byte offset (without box/tile-row parts)
    uint32_t v[4];   // V: [((lane/8)&1)*8 + lane%8] row, chunk pair c
    __device__ __forceinline__ void init(int lane) {
        const int lm = lane >> 3, lr = lane & 7;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            k[c] = (uint32_t)((((lm >> 1) * 8 + lr) * 128) + ((((c * 2) | (lm & 1)) ^ lr) << 4));
            v[c] = (uint32_t)((((lm & 1) * 8 + lr) * 128) + ((((c * 2) | (lm >> 1)) ^ lr) << 4));
        }
    }
};

struct WarpState {
    float acc[16][4];     // O fragments: [8-column tile][c0 c1 (head g) | c2 c3 (head g+8)]
    float m[2];           // running maxima (log2 units) of heads g and g+8
    float l[2];           // this thread's share of the running sums
    __device__ __forceinline__ void reset() {
#pragma unroll
        for (int i = 0; i < 16; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;
        m[0] = m[1] = -INFINITY;
        l[0] = l[1] = 0.f;
    }
};

// Q fragments (A operand, 16 heads x 128 columns) of head tile mt of sequence seq, straight from
// global memory; heads >= h are zero.
__device__ __forceinline__ void load_q_fragments(uint32_t (&qa)[8][4], const uint32_t* __restrict__ q, size_t seq,
                                                 int h, int mt, int lane) {
    const int g = lane >> 2, t4 = lane & 3;
    const int head0 = mt * 16 + g, head1 = head0 + 8;
    const uint32_t* q0 = q + (seq * h + head0) * (kHeadDim / 2);
    const uint32_t* q1 = q + (seq * h + head1) * (kHeadDim / 2);
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
        const int w0 = ks * 8 + t4;                    // 32-bit word: columns ks*16 + t4*2 + {0,1}
        qa[ks][0] = head0 < h ? __ldg(q0 + w0) : 0u;
        qa[ks][1] = head1 < h ? __ldg(q1 + w0) : 0u;
        qa[ks][2] = head0 < h ? __ldg(q0 + w0 + 4) : 0u;   // columns + 8
        qa[ks][3] = head1 < h ? __ldg(q1 + w0 + 4) : 0u;
    }
}

// One 32-row tile (cache rows row0 .. row0+31 of the sequence, of which rows < r1 are valid) for
// 16 heads: S = Q K^T, online softmax update, O += P V.
// HILO: feed P to the tensor cores as bf16 hi + lo parts (weights good to ~2^-17) instead of one
// bf16 rounding (2^-9 per weight).  One rounding is enough once the prefix is long: the output
// is then an average over many rows, of size ~1/sqrt(rows), and so is the rounding error.
// half_stride: bytes between the box holding columns 0..63 and the box holding columns 64..127.
template <bool HILO>
__device__ __forceinline__ void consume_tile(WarpState& st, const uint32_t (&qa)[8][4], const LaneOffsets& off,
                                             uint32_t k_s, uint32_t v_s, uint32_t half_stride, int row0, int r1, int lane) {
    const int t4 = lane & 3;
    const bool ragged = row0 + kTileRows > r1;

    // S = Q K^T: 4 n-tiles of 8 rows, 8 k-steps of 16 columns
    float sc[4][4];
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
        const uint32_t a = k_s + off.k[ks & 3] + (ks >> 2) * half_stride;
#pragma unroll
        for (int np = 0; np < 2; ++np) {               // n-tile pairs (0,1) and (2,3): 16 rows = 2 KiB apart
            uint32_t b0, b1, b2, b3;
            ldmatrix_x4(a + np * 2048, b0, b1, b2, b3);
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
            const float x = sc[nt][j] * kLog2e;
            sc[nt][j] = (!ragged || row0 + nt * 8 + t4 * 2 + (j & 1) < r1) ? x : -INFINITY;   // select, never multiply
            top[j >> 1] = fmaxf(top[j >> 1], sc[nt][j]);
        }
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        top[r] = fmaxf(top[r], __shfl_xor_sync(0xffffffffu, top[r], 1));
        top[r] = fmaxf(top[r], __shfl_xor_sync(0xffffffffu, top[r], 2));
    }
    // a new maximum rescales what has been accumulated; most tiles do not bring one
    if (__any_sync(0xffffffffu, top[0] > st.m[0] || top[1] > st.m[1])) {
        float rescale[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const float m_new = fmaxf(st.m[r], top[r]);     // the tile's first row is valid: finite
            rescale[r] = fast_exp2(st.m[r] - m_new);        // 0 on the first tile, 1 if unchanged
            st.m[r] = m_new;
            st.l[r] *= rescale[r];
        }
#pragma unroll
        for (int vt = 0; vt < 16; ++vt) {
            st.acc[vt][0] *= rescale[0]; st.acc[vt][1] *= rescale[0];
            st.acc[vt][2] *= rescale[1]; st.acc[vt][3] *= rescale[1];
        }
    }
    // P = exp2(S - max) as bf16 hi + lo A-fragments for the two 16-row k-steps
    uint32_t p_hi[2][4], p_lo[2][4];
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
        float p[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            p[j] = fast_exp2(sc[nt][j] - st.m[j >> 1]);     // exactly 1 at the maximum, 0 when masked
            st.l[j >> 1] += p[j];
        }
        const uint32_t hi01 = pack_bf16(p[0], p[1]), hi23 = pack_bf16(p[2], p[3]);
        const int kk = nt >> 1, hf = (nt & 1) * 2;          // A regs: {g,k}, {g+8,k}, {g,k+8}, {g+8,k+8}
        p_hi[kk][hf] = hi01; p_hi[kk][hf + 1] = hi23;
        if (HILO) {
            p_lo[kk][hf] = pack_bf16(p[0] - bf16_lo(hi01), p[1] - bf16_hi(hi01));
            p_lo[kk][hf + 1] = pack_bf16(p[2] - bf16_lo(hi23), p[3] - bf16_hi(hi23));
        }
    }
    // O += P V : 2 k-steps of 16 rows x 16 n-tiles of 8 columns
#pragma unroll
    for (int kk = 0; kk < 2; ++kk) {
        uint32_t keep_lo = 0xffffffffu, keep_hi = 0xffffffffu;   // per-register row masks (ragged tile)
        if (ragged) {
            const int ra = row0 + kk * 16 + t4 * 2;              // rows held by b0/b2: ra, ra+1; b1/b3: +8
            keep_lo = (ra < r1 ? 0x0000ffffu : 0u) | (ra + 1 < r1 ? 0xffff0000u : 0u);
            keep_hi = (ra + 8 < r1 ? 0x0000ffffu : 0u) | (ra + 9 < r1 ? 0xffff0000u : 0u);
        }
#pragma unroll
        for (int vp = 0; vp < 8; ++vp) {                         // pairs of 8-column n-tiles
            uint32_t b0, b1, b2, b3;
            ldmatrix_x4_trans(v_s + off.v[vp & 3] + (vp >> 2) * half_stride + kk * 2048, b0, b1, b2, b3);
            if (ragged) { b0 &= keep_lo; b1 &= keep_hi; b2 &= keep_lo; b3 &= keep_hi; }
            mma_bf16(st.acc[vp * 2], p_hi[kk], b0, b1);
            mma_bf16(st.acc[vp * 2 + 1], p_hi[kk], b2, b3);
            if (HILO) {
                mma_bf16(st.acc[vp * 2], p_lo[kk], b0, b1);
                mma_bf16(st.acc[vp * 2 + 1], p_lo[kk], b2, b3);
            }
        }
    }
}

// Merge `other` (the same heads over other rows) into `st`.  Either side may be empty (m = -inf).
__device__ __forceinline__ void merge_state(WarpState& st, const float* __restrict__ other, int lane) {
    // `other` is thread-private storage: float index r * 32 + lane, r = 0..63 acc, 64..65 m, 66..67 l
    float wa[2], wb[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const float mb = other[(64 + r) * 32 + lane];
        const float lb = other[(66 + r) * 32 + lane];
        const float m_new = fmaxf(st.m[r], mb);
        wa[r] = st.m[r] == -INFINITY ? 0.f : fast_exp2(st.m[r] - m_new);
        wb[r] = mb == -INFINITY ? 0.f : fast_exp2(mb - m_new);
        st.m[r] = m_new;
        st.l[r] = st.l[r] * wa[r] + lb * wb[r];
    }
#pragma unroll
    for (int vt = 0; vt < 16; ++vt) {
#pragma unroll
        for (int j = 0; j < 4; ++j)
            st.acc[vt][j] = st.acc[vt][j] * wa[j >> 1] + other[(vt * 4 + j) * 32 + lane] * wb[j >> 1];
    }
}

__device__ __forceinline__ void store_state(const WarpState& st, float* __restrict__ dst, int lane) {
#pragma unroll
    for (int vt = 0; vt < 16; ++vt) {
#pragma unroll
        for (int j = 0; j < 4; ++j) dst[(vt * 4 + j) * 32 + lane] = st.acc[vt][j];
    }
    dst[64 * 32 + lane] = st.m[0]; dst[65 * 32 + lane] = st.m[1];
    dst[66 * 32 + lane] = st.l[0]; dst[67 * 32 + lane] = st.l[1];
}

// =============================================================================================
// Fixed-split kernel: one CTA per (sequence, split of chunk_rows rows).
// =============================================================================================
template <int M_TILES, bool EARLY = false>
__global__ void __launch_bounds__(MmaCfg<M_TILES>::kThreads, MmaCfg<M_TILES>::kMinBlocks)
mqa_decode_split_mma_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                            const __grid_constant__ CUtensorMap map_k_big, const __grid_constant__ CUtensorMap map_v_big,
                            const uint32_t* __restrict__ q, const int32_t* __restrict__ lens,
                            float* __restrict__ o, float2* __restrict__ part_ml, float* __restrict__ part_acc,
                            int32_t* __restrict__ status, int h, int m_max, int chunk_rows, int n_splits, int len_bias,
                            const FusedArgs fa, int32_t* __restrict__ lens_advance, int mode) {
    using Cfg = MmaCfg<M_TILES>;
    const bool withhold = (mode & 2) != 0;                 // for tests: one copy is never started, so that a wait runs out (bit 0: unused)
    constexpr int kStages = Cfg::kStages;
    const int seq = blockIdx.x / n_splits;
    const int split = blockIdx.x % n_splits;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    extern __shared__ uint8_t smem_raw[];
    // 1 KiB alignment in the shared window: the 128-byte swizzle repeats every 8 rows x 128 bytes
    uint8_t* stages = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);
    uint64_t* bars = reinterpret_cast<uint64_t*>(stages + kStages * kStageBytes);   // full[kStages], empty[kStages]
    const uint32_t stages_s = smem_addr(stages);
    const uint32_t full_s = smem_addr(bars), empty_s = full_s + kStages * 8;
    __shared__ int timed_out, issued;   // a wait ran out; tiles whose copies were started

    // set up by the thread that issues the copies (it may issue some before the first CTA-wide barrier)
    if (warp == Cfg::kConsumerWarps && lane == 0) {
        prefetch_tensormap(&map_k); prefetch_tensormap(&map_v);
        timed_out = 0;
        issued = 0;
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full_s + s * 8, 1);                  // the producer's arrive + the TMA bytes
            mbar_init(empty_s + s * 8, M_TILES);           // one arrive per warp that read the tile
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    const int row_base = seq * m_max + split * chunk_rows; // row coordinate in the [b*m_max, 128] view
    auto issue_tile = [&](int i) {
        const int s = i % kStages;
        const uint32_t bar = full_s + s * 8;
        const uint32_t dst = stages_s + s * kStageBytes;
        mbar_expect_tx(bar, kStageBytes);
        const int y = row_base + i * kTileRows;
        tma_load_2d(dst, &map_k, 0, y, bar);
        tma_load_2d(dst + kBoxBytes, &map_k, kBoxCols, y, bar);
        tma_load_2d(dst + 2 * kBoxBytes, &map_v, 0, y, bar);
        if (!(withhold && blockIdx.x == 0 && i == 1)) tma_load_2d(dst + 3 * kBoxBytes, &map_v, kBoxCols, y, bar);
        issued = i + 1;
    };
    // EARLY (the caller's promise that only this library's steps have written the cache and lens since its last step
    // on them): one CTA owns the sequence, its tiles are tiles 0, 1, ... whatever lens says, so those that lie wholly
    // below the prefix's last two rows -- by lens as it reads now, which the step ahead may be about to advance -- are
    // fetched while that step is still finishing.  Only their number is a guess: should fewer tiles count in the end,
    // the surplus is left to land and ignored.
    int pre = 0;
    if (EARLY && n_splits == 1 && warp == Cfg::kConsumerWarps && lane == 0) {
        const int raw_guess = __ldcg(lens + seq);
        const int rows_guess = min(max(raw_guess, 0) + (fa.k_new != nullptr ? 1 : 0), m_max);
        pre = min((rows_guess - 2) / kTileRows, kStages);
        if (pre < 0) pre = 0;
        for (int i = 0; i < pre; ++i) issue_tile(i);
    }
    // everything above overlaps the tail of the kernel before this one
    grid_dependency_wait();          // lens and the newest cache row may come from the kernel before
    grid_launch_dependents();
    // With one CTA per sequence (n_splits == 1) the CTA may do the whole decoding step: write the new row
    // (fa.k_new given), attend over one row more, and move lens[seq] on at the end (lens_advance given) --
    // nobody else reads this sequence's length.
    // A sequence cut into several splits (n_splits > 1) may take its new row too: the CTA whose rows hold it writes
    // it, every split attends over one row more, and lens is left to the second-pass kernel.
    // (the new row's pieces do not depend on lens: asked for first, so that the two loads are in flight together)
    uint4 row_piece = make_uint4(0u, 0u, 0u, 0u);
    if (fa.k_new != nullptr && warp == 0)                 // lanes 0-15 move the key row, 16-31 the value row
        row_piece = (lane < 16 ? fa.k_new : fa.v_new)[(size_t)seq * (kRowBytes / 16) + (lane & 15)];
    const int raw = lens[seq];
    const bool appended = fa.k_new != nullptr && raw >= 0 && raw < m_max;
    if (fa.k_new != nullptr) {
        if (!appended && threadIdx.x == 0 && status) atomicOr(status, raw < 0 ? kStatusAppendNegative : kStatusAppendFull);
        if (appended && warp == 0 && (n_splits == 1 || raw / chunk_rows == split)) {
            const size_t dst = ((size_t)seq * m_max + raw) * (kRowBytes / 16) + (lane & 15);
            if (lane < 16) fa.K[dst] = row_piece; else fa.V[dst] = row_piece;
            asm volatile("fence.proxy.async;" ::: "memory");   // the copy engine must see the row (a barrier follows)
        }
    }
    const int L = clamp_len(appended ? raw + 1 : biased_len(raw, m_max, len_bias), m_max,
                            threadIdx.x == 0 ? status : nullptr);
    const int r0 = split * chunk_rows;
    const int r1 = min(L, r0 + chunk_rows);
    if (r0 >= L) {                                         // nothing valid in this split (uniform)
        if (n_splits == 1)                                 // L == 0: the empty prefix gives zeros
            for (int i = threadIdx.x; i < h * kHeadDim; i += Cfg::kThreads) o[(size_t)seq * h * kHeadDim + i] = 0.f;
        else                                               // an empty piece, for a second pass that does not look at lens
            for (int i = threadIdx.x; i < h; i += Cfg::kThreads)
                part_ml[((size_t)seq * h + i) * n_splits + split] = make_float2(-INFINITY, 0.f);
        for (int i = 0; i < pre; ++i) mbar_wait(full_s + i * 8, 0);   // copies started on a guess land before the CTA leaves
        return;
    }
    const int n_tiles = (r1 - r0 + kTileRows - 1) / kTileRows;
    // a few tiles (each has a stage of its own), beginning at a multiple of 128 rows: fetched four tiles per copy
    // (from three tiles on: a copy moves all 128 rows of its box, and one or two tiles are quicker on their own)
    const bool big = !EARLY && !withhold && n_tiles >= 3 && n_tiles <= kStages && (r0 & (4 * kTileRows - 1)) == 0;

    __syncthreads();

    const int mt = warp % M_TILES;                         // which 16-head tile this warp serves
    const int rw = warp / M_TILES;                         // which tiles (round-robin over kRowWarps)
    WarpState st;

    if (warp == Cfg::kConsumerWarps) {
        // ------------------------------------------------------------------ producer warp
        if (lane == 0 && big) {
            // four tiles per copy: boxes of 128 rows (K columns 0-63, 64-127, V likewise), a quarter of the copies
            for (int grp = 0; grp * 4 < n_tiles; ++grp) {
                const uint32_t bar = full_s + grp * 8, dst = stages_s + grp * 4 * kStageBytes;
                mbar_expect_tx(bar, 4 * kStageBytes);
                const int y = row_base + grp * 4 * kTileRows;
                tma_load_2d(dst, &map_k_big, 0, y, bar);
                tma_load_2d(dst + 4 * kBoxBytes, &map_k_big, kBoxCols, y, bar);
                tma_load_2d(dst + 8 * kBoxBytes, &map_v_big, 0, y, bar);
                tma_load_2d(dst + 12 * kBoxBytes, &map_v_big, kBoxCols, y, bar);
                issued = grp + 1;
            }
        } else if (lane == 0) {
            bool ok = true;
            for (int i = pre; i < n_tiles && ok; ++i) {
                const int s = i % kStages;
                if (i >= kStages) ok = mbar_wait(empty_s + s * 8, ((i / kStages) - 1) & 1);
                if (!ok) break;
                issue_tile(i);
            }
            for (int i = n_tiles; i < pre; ++i) ok = mbar_wait(full_s + i * 8, 0) && ok;   // a surplus of the guess
            if (!ok) atomicExch(&timed_out, 1);
        }
    } else {
        // --------------------------------------------------------------- consumer warps
        st.reset();
        uint32_t qa[8][4];
        load_q_fragments(qa, q, (size_t)seq, h, mt, lane);
        LaneOffsets off;
        off.init(lane);
        bool ok = true;
        for (int i = rw; i < n_tiles; i += kRowWarps) {
            const int s = i % kStages;
            ok = big ? mbar_wait(full_s + (i >> 2) * 8, 0) : mbar_wait(full_s + s * 8, (i / kStages) & 1);
            if (!ok) break;
            // a tile's K boxes, then its V boxes; in a copy of four tiles the tile is 32 of a box's 128 rows
            const uint32_t k_s = big ? stages_s + (i >> 2) * 4 * kStageBytes + (i & 3) * kBoxBytes : stages_s + s * kStageBytes;
            const uint32_t half = big ? 4 * kBoxBytes : kBoxBytes;
            consume_tile<true>(st, qa, off, k_s, k_s + 2 * half, half, r0 + i * kTileRows, r1, lane);
            // The tile was read through the generic proxy (ldmatrix) and the copy engine will write the stage
            // again through the async proxy: without this fence the last ldmatrix of a tile now and then saw
            // rows of the tile that came four tiles later (one run in a few hundred, 16 output columns off).
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
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
    const int g = lane >> 2, t4 = lane & 3;
    float* sm_acc = reinterpret_cast<float*>(stages);                   // [consumer warp][16][128]
    float2* sm_ml = reinterpret_cast<float2*>(stages + Cfg::kConsumerWarps * 16 * kHeadDim * 4);  // [cw][16]
    if (warp < Cfg::kConsumerWarps) {
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            st.l[r] += __shfl_xor_sync(0xffffffffu, st.l[r], 1);
            st.l[r] += __shfl_xor_sync(0xffffffffu, st.l[r], 2);
        }
        float* mine = sm_acc + (size_t)warp * 16 * kHeadDim;
#pragma unroll
        for (int vt = 0; vt < 16; ++vt) {
            *reinterpret_cast<float2*>(mine + g * kHeadDim + vt * 8 + t4 * 2) = make_float2(st.acc[vt][0], st.acc[vt][1]);
            *reinterpret_cast<float2*>(mine + (g + 8) * kHeadDim + vt * 8 + t4 * 2) = make_float2(st.acc[vt][2], st.acc[vt][3]);
        }
        if (t4 == 0) {
            sm_ml[warp * 16 + g] = make_float2(st.m[0], st.l[0]);
            sm_ml[warp * 16 + g + 8] = make_float2(st.m[1], st.l[1]);
        }
    }
    __syncthreads();
    // per head, once: the largest of the row-warps' maxima, each warp's weight, the sum
    float* sm_w = reinterpret_cast<float*>(sm_ml + Cfg::kConsumerWarps * 16);   // [M_TILES * 16][8]: kRowWarps weights, max, sum
    if (threadIdx.x < M_TILES * 16) {
        const int tile = threadIdx.x >> 4, hr = threadIdx.x & 15;
        float2 ml[kRowWarps];
        float top = -INFINITY;
#pragma unroll
        for (int w = 0; w < kRowWarps; ++w) {
            ml[w] = sm_ml[(w * M_TILES + tile) * 16 + hr];              // consumer warp (rw = w, mt = tile)
            top = fmaxf(top, ml[w].x);
        }
        float den = 0.f;
#pragma unroll
        for (int w = 0; w < kRowWarps; ++w) {
            const float wt = ml[w].x == -INFINITY ? 0.f : fast_exp2(ml[w].x - top);   // a warp without tiles counts for nothing
            den = fmaf(wt, ml[w].y, den);
            sm_w[threadIdx.x * 8 + w] = wt;
        }
        sm_w[threadIdx.x * 8 + kRowWarps] = top;
        sm_w[threadIdx.x * 8 + kRowWarps + 1] = den;
    }
    __syncthreads();
    // then 16 bytes of a head's 128 outputs per thread and round
    for (int idx = threadIdx.x; idx < h * (kHeadDim / 4); idx += Cfg::kThreads) {
        const int head = idx >> 5, c4 = idx & 31;
        const int tile = head >> 4, hr = head & 15;
        const float* wts = sm_w + head * 8;
        float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int w = 0; w < kRowWarps; ++w) {
            const float4 a = *reinterpret_cast<const float4*>(sm_acc + ((size_t)(w * M_TILES + tile) * 16 + hr) * kHeadDim + c4 * 4);
            const float wt = wts[w];
            num.x = fmaf(wt, a.x, num.x); num.y = fmaf(wt, a.y, num.y); num.z = fmaf(wt, a.z, num.z); num.w = fmaf(wt, a.w, num.w);
        }
        const size_t unit = (size_t)seq * h + head;
        if (n_splits == 1) {
            const float inv = 1.f / wts[kRowWarps + 1];
            *reinterpret_cast<float4*>(o + unit * kHeadDim + c4 * 4) = make_float4(num.x * inv, num.y * inv, num.z * inv, num.w * inv);
        } else {
            const size_t slot = unit * n_splits + split;
            *reinterpret_cast<float4*>(part_acc + slot * kHeadDim + c4 * 4) = num;
            if (c4 == 0) part_ml[slot] = make_float2(wts[kRowWarps], wts[kRowWarps + 1]);
        }
    }
    if (lens_advance && appended && threadIdx.x == 0) lens_advance[seq] = raw + 1;   // every thread read lens[seq] barriers ago
}

// =============================================================================================
// Persistent kernel: the valid 32-row tiles of all sequences, in sequence order, form one line
// of T tiles; CTA c of G takes tiles [c*T/G, (c+1)*T/G).  A CTA's share is a run of segments,
// each a contiguous run of tiles of one sequence.  A segment that covers its whole sequence
// writes the final o; any other segment writes a partial into slot (c + sequence) -- along the
// line every step moves to the next CTA, the next sequence, or both, so that sum never repeats
// -- and the slots of each sequence that was cut are merged, inside the kernel by the CTA that
// delivers the last one or by the second-pass kernel below.
// =============================================================================================
// Crossing from one sequence to the next inside a share is not free (sums are added up, a partial or
// the result is written, the next sequence's Q is fetched), so the line carries, in front of each
// sequence's tiles, PENALTY virtual tiles that cost nothing to "process": a CTA whose share contains a
// crossing gets that many fewer real tiles, and all CTAs finish together.

// Share c of G of a line of T positions: [c*T/G, (c+1)*T/G).  The division by the run-time grid size is
// a multiplication by magic = ceil(2^64 / G), computed on the host (exact for c*T < 2^48, G <= 256; a
// division in the kernel would be a long dependent sequence at the head of every CTA).  magic = 0: G = 1.
__host__ __device__ inline unsigned long long share_magic(int G) { return G <= 1 ? 0ull : ~0ull / (unsigned long long)G + 1ull; }
__device__ __forceinline__ int share_begin(int c, int T, unsigned long long magic) {
    const unsigned long long n = (unsigned long long)(unsigned int)c * (unsigned int)T;
    return magic ? (int)__umul64hi(n, magic) : (int)n;
}

// A run of 32-row tiles [lo, hi) of sequence s inside one CTA's share.
struct Segment {
    int s, lo, hi;
    bool whole;           // the share holds every tile of the sequence: it writes the final o
};

// Walks one CTA's share [t, t_end) of the line.  prefix[s] = position of sequence s's block (its penalty
// tiles, then its real tiles); sequences without rows have no block.
template <int PENALTY>
struct ShareWalker {
    const int* prefix;
    int t, t_end;
    int s;
    __device__ __forceinline__ bool next(Segment& g) {
        while (t < t_end) {
            while (prefix[s + 1] <= t) ++s;
            const int v0 = prefix[s], v1 = prefix[s + 1];
            const int n = v1 - v0 - PENALTY;                                    // real tiles, >= 1
            const int end = v1 < t_end ? v1 : t_end;
            const int lo = t - v0 - PENALTY, hi = end - v0 - PENALTY;
            t = end;
            g.s = s;
            g.lo = lo > 0 ? lo : 0;
            g.hi = hi < n ? hi : n;
            g.whole = g.lo == 0 && g.hi == n;
            if (g.hi > g.lo) return true;
        }
        return false;
    }
};

// cta that owns global tile t when T tiles are cut into G shares [c*T/G, (c+1)*T/G)
__host__ __device__ inline int stream_owner(long long t, long long T, int G) {
    return (int)(((t + 1) * G + T - 1) / T - 1);
}

// Workspace layout of the persistent kernel
__host__ __device__ inline size_t stream_span_bytes(int b) { return (((size_t)(b + 1) * sizeof(int2)) + 255) & ~(size_t)255; }
__host__ __device__ inline size_t stream_ml_bytes(int slots, int h) {
    return (((size_t)slots * h * sizeof(float2)) + 255) & ~(size_t)255;
}
__host__ __device__ inline size_t stream_acc_bytes(int slots, int h) { return (size_t)slots * h * kHeadDim * sizeof(float); }

// Rows of its cache that sequence s may look at, as lens says (read from L2: the kernels before and after this one may
// write lens).
template <bool FUSED>
__device__ __forceinline__ int read_len(const int32_t* lens, int s) { return __ldcg(lens + s); }

// Rows of sequence s this launch attends over, and whether the step appends to it.
__device__ __forceinline__ int fused_rows(int raw, int m_max, bool appending, bool* can_append) {
    const bool ok = appending && raw >= 0 && raw < m_max;
    if (can_append) *can_append = ok;
    const int L = raw < 0 ? 0 : (raw > m_max ? m_max : raw);
    return ok ? L + 1 : L;
}

constexpr int kAppendBit = 1 << 30;                    // in rows_of[]: this step appends a row to the sequence

// The schedule of a persistent kernel, computed by every CTA for itself (all THREADS threads call this):
// prefix[s] = position on the line of sequence s's block (PENALTY virtual tiles, then its 32-row
// tiles; no block for an empty prefix, whose output is zeroed here), rows_of[s] = rows to attend over
// (kAppendBit set when this step appends one).  Returns T = length of the line, [t_begin, t_end) = this
// CTA's share, s_first = the sequence that holds position t_begin, equal = every sequence has the same, non-zero
// number of tiles (then G shares of a batch that divides G fall on sequence boundaries).  plan_sm: 8 ints of
// shared memory.
struct SharePlan { int T, t_begin, t_end, s_first; bool equal; };

// solo_warp: a warp (the one that issues the copies) that takes no part in building the tables, so that the other
// warps do not wait for it: it must have arrived on barrier kPlanBarInit (named_barrier_arrive over THREADS) once what it
// initialises in shared memory is in place, and it returns from here when the tables are complete.  -1: none.
constexpr int kPlanBarInit = 3, kPlanBarScan = 4, kPlanBarDone = 5;
template <bool FUSED, int THREADS, int PENALTY>
__device__ __forceinline__ SharePlan stream_plan(const int32_t* __restrict__ lens, float* __restrict__ o,
                                                 int32_t* __restrict__ status, int b, int h, int m_max, bool appending,
                                                 unsigned long long magic, int* prefix, int* rows_of, int* plan_sm,
                                                 int solo_warp = -1) {
    const int cta = blockIdx.x, G = gridDim.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int planners = solo_warp >= 0 ? THREADS - 32 : THREADS;
    const int tix = (solo_warp >= 0 && warp > solo_warp) ? (int)threadIdx.x - 32 : (int)threadIdx.x;
    if (warp == solo_warp) {
        named_barrier(kPlanBarDone, THREADS);
    } else {
    for (int s = tix; s < b; s += planners) {
        const int raw = read_len<FUSED>(lens, s);
        clamp_len(raw, m_max, cta == 0 ? status : nullptr);
        bool can_append;
        const int L = fused_rows(raw, m_max, appending, &can_append);
        if (appending && !can_append && cta == 0 && status)
            atomicOr(status, raw < 0 ? kStatusAppendNegative : kStatusAppendFull);
        prefix[s + 1] = L > 0 ? (L + kTileRows - 1) / kTileRows + PENALTY : 0;
        rows_of[s] = L | (appending && can_append ? kAppendBit : 0);
    }
    if (threadIdx.x == 0) { prefix[0] = 0; plan_sm[3] = 0; }
    if (solo_warp >= 0) named_barrier(kPlanBarInit, THREADS); else __syncthreads();
    for (int s = cta; s < b; s += G) {                     // the empty prefix gives zeros: all threads, 16 bytes each
        if ((rows_of[s] & (kAppendBit - 1)) != 0) continue;
        float4* dst = reinterpret_cast<float4*>(o + (size_t)s * h * kHeadDim);
        for (int i = tix; i < h * (kHeadDim / 4); i += planners) dst[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    if (warp == 0) {
        // inclusive scan of prefix[1..b] by one warp; the lane whose chunk holds this CTA's first position
        // also notes which sequence that is
        const int per = (b + 31) >> 5;
        const int lo = 1 + lane * per, hi = min(b, lo + per - 1);
        int sum = 0;
        for (int s = lo; s <= hi; ++s) sum += prefix[s];
        int incl = sum;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int up = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += up;
        }
        const int T = __shfl_sync(0xffffffffu, incl, 31);
        const int tb = share_begin(cta, T, magic), te = share_begin(cta + 1, T, magic);
        const int first_count = prefix[1];
        int run = incl - sum;
        bool same = true;
        for (int s = lo; s <= hi; ++s) {
            const int before = run;
            same = same && prefix[s] == first_count;
            run += prefix[s];
            prefix[s] = run;
            if (before <= tb && tb < run) plan_sm[3] = s - 1;     // sequence s-1 occupies [before, run)
        }
        same = __all_sync(0xffffffffu, same) && first_count > 0;
        if (lane == 0) { plan_sm[0] = T; plan_sm[1] = tb; plan_sm[2] = te; plan_sm[4] = same ? 1 : 0; }
    }
    if (solo_warp >= 0) {
        named_barrier(kPlanBarScan, planners);
        named_barrier_arrive(kPlanBarDone, THREADS);
    } else {
        __syncthreads();
    }
    }
    SharePlan p;
    p.T = plan_sm[0]; p.t_begin = plan_sm[1]; p.t_end = plan_sm[2]; p.s_first = plan_sm[3]; p.equal = plan_sm[4] != 0;
    return p;
}

// The producer warp's short cut to its first copies (all 32 lanes call this): for up to kFastSeqs sequences
// the warp reads lens itself, scans the tile counts in registers and finds the first segment of this
// CTA's share, so that the first copies start one L2 round trip after the wait for the kernel before,
// while the other warps build the shared tables (stream_plan, which gives the same segment again).
// Returns false when there is nothing to start early (more sequences, an empty share, or a share that
// begins between two sequences); *rows = rows_of[] entry of the segment's sequence.
constexpr int kFastSeqs = 256;
// cluster > 1: the grid was launched as clusters of `cluster` CTAs with cluster * b == gridDim.x, this CTA has rank
// `rank` in its cluster, and a stage is `stage_tiles` tiles.  If every sequence has the same, non-zero number of tiles,
// cluster c holds sequence c and its CTAs take the sequence's stages in turn (rank r: stages r, r + cluster, ...):
// then *strided is set and the segment returned is (sequence, first tile of stage r, all tiles of the sequence).
template <bool FUSED, int PENALTY>
__device__ __forceinline__ bool first_segment(const int32_t* __restrict__ lens, int b, int m_max, bool appending,
                                              unsigned long long magic, Segment* g, int* rows, int cluster = 1, int rank = 0,
                                              int stage_tiles = 4, bool* strided = nullptr) {
    if (strided) *strided = false;
    if (b > kFastSeqs) return false;
    const int cta = blockIdx.x, lane = threadIdx.x & 31;
    const int per = (b + 31) >> 5, base = lane * per;
    int tl[kFastSeqs / 32], rw[kFastSeqs / 32];
    int sum = 0;
#pragma unroll
    for (int i = 0; i < kFastSeqs / 32; ++i) {
        tl[i] = 0; rw[i] = 0;
        if (i < per && base + i < b) {
            bool can_append;
            const int L = fused_rows(read_len<FUSED>(lens, base + i), m_max, appending, &can_append);
            tl[i] = L > 0 ? (L + kTileRows - 1) / kTileRows + PENALTY : 0;
            rw[i] = L | (appending && can_append ? kAppendBit : 0);
        }
        sum += tl[i];
    }
    if (sum >= 0 && lane == 0) TS(28);
    if (cluster > 1) {
        const int first = __shfl_sync(0xffffffffu, tl[0], 0);
        bool same = first > 0;
#pragma unroll
        for (int i = 0; i < kFastSeqs / 32; ++i)
            if (i < per && base + i < b) same = same && tl[i] == first;
        if (__all_sync(0xffffffffu, same)) {
            const int s = cta / cluster;
            int fr = 0;
#pragma unroll
            for (int i = 0; i < kFastSeqs / 32; ++i)
                if (i == s % per) fr = rw[i];
            fr = __shfl_sync(0xffffffffu, fr, s / per);
            g->s = s;
            g->lo = rank * stage_tiles;
            g->hi = first - PENALTY;
            g->whole = false;
            *rows = fr;
            if (strided) *strided = true;
            if (lane == 0) TS(29);
            return g->lo < g->hi;
        }
    }
    int incl = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += up;
    }
    const int T = __shfl_sync(0xffffffffu, incl, 31);
    const int tb = share_begin(cta, T, magic), te = share_begin(cta + 1, T, magic);
    int run = incl - sum, fs = -1, v0 = 0, v1 = 0, fr = 0;
#pragma unroll
    for (int i = 0; i < kFastSeqs / 32; ++i) {
        const int before = run;
        run += tl[i];
        if (before <= tb && tb < run) { fs = base + i; v0 = before; v1 = run; fr = rw[i]; }
    }
    const unsigned found = __ballot_sync(0xffffffffu, fs >= 0);
    if (tb >= te || found == 0) return false;
    const int src = __ffs(found) - 1;
    fs = __shfl_sync(0xffffffffu, fs, src); v0 = __shfl_sync(0xffffffffu, v0, src);
    v1 = __shfl_sync(0xffffffffu, v1, src); fr = __shfl_sync(0xffffffffu, fr, src);
    const int n = v1 - v0 - PENALTY;
    const int end = v1 < te ? v1 : te;
    const int lo = tb - v0 - PENALTY, hi = end - v0 - PENALTY;
    g->s = fs;
    g->lo = lo > 0 ? lo : 0;
    g->hi = hi < n ? hi : n;
    g->whole = g->lo == 0 && g->hi == n;
    *rows = fr;
    return g->hi > g->lo;
}

// Second pass of the persistent kernel: one CTA per (sequence, head) merges the slots of the
// CTAs that hold pieces of the sequence (nothing to do when a single CTA had the whole sequence,
// or it is empty).  seq_span[b] holds (T, G): a CTA whose share of the T tiles is empty wrote no
// slot and is skipped.
template <int GROUPS>
__global__ void __launch_bounds__(kHeadDim * (GROUPS >= 4 ? 4 : 1))
stream_combine_kernel(const int2* __restrict__ seq_span, const float2* __restrict__ part_ml,
                      const float* __restrict__ part_acc, float* __restrict__ o, int b, int h,
                      int32_t* lens_advance, int m_max, unsigned long long magic) {
    const int s = blockIdx.x / h, head = blockIdx.x % h;
    grid_dependency_wait();          // the slots come from the kernel before this one
    // append-and-attend step: lens += 1 for a sequence that took a row
    if (lens_advance && head == 0 && threadIdx.x == 0) {
        const int raw = lens_advance[s];
        if (raw >= 0 && raw < m_max) lens_advance[s] = raw + 1;
    }
    const int2 span = seq_span[s];
    if (span.y <= span.x) return;
    const int T = seq_span[b].x;                        // length of the line (magic: the first pass's grid size, see share_begin)
    const int n_cta = span.y - span.x + 1;              // at most the grid of the first pass (<= 256 SMs)
    // piece i is the slot of CTA span.x + i; a CTA whose share of the line is empty wrote none (max = -inf)
    merge_pieces<GROUPS>(
        n_cta,
        [&](int i) {
            const int cta = span.x + i;
            const bool live = share_begin(cta, T, magic) != share_begin(cta + 1, T, magic);
            return live ? __ldcg(part_ml + ((size_t)cta + s) * h + head) : make_float2(-INFINITY, 0.f);
        },
        [&](int i) { return part_acc + (((size_t)span.x + i + s) * h + head) * kHeadDim; },
        o + ((size_t)s * h + head) * kHeadDim);
}

}  // namespace mqa
