// Persistent multi-query decode kernel on the 5th-generation tensor cores (tcgen05 + TMEM): one CTA
// per SM, every CTA an equal share of the line of valid 32-row tiles of the whole batch (see the
// second half of decode_mma.cuh).  The step is the three lines of Section 3: logits =
// einsum(bhk,bmk->bhm), softmax over m, o = einsum(bhm,bmv->bhv).  The cache rows are the M dimension
// of both products and the heads are N:
//
//     S^T[128 cache rows x HP heads]  = K_stage[128 x 128] * Q^T          A = the TMA-written K rows (K-major),
//                                                                          B = the sequence's Q rows (K-major)
//     O^T[128 columns x HP heads]    += V_stage^T[128 x 128 rows] * P^T   A = the TMA-written V rows (MN-major),
//                                                                          B = P^T, written by the softmax warps
//
// so K and V are read from shared memory by the tensor core itself, once for all heads; the work
// per stage grows with the padded head count HP (16 or 32; more query rows per sequence run on decode_wide.cuh) and nothing is replicated.  In TMEM
// a cache row of S^T is a lane, so a softmax thread owns one cache row of the stage (two threads
// share a row's heads): masking by index is a per-thread decision and the weights need no exchange
// between threads.  The reference maximum of a head is shared by all rows and moves only when some
// logit exceeds it by more than 2^kMaxLead (always on a segment's first stage): then the warps find
// the stage's maxima together, rescale their sums and the O^T accumulator, and go on.  Softmax is
// shift invariant, so a reference that lags the true maximum by a bounded amount changes nothing but
// the common scale of numerator and denominator.
//
//   producer warp      TMA: a segment's Q rows once, then K and V rows in 128-row stages (separate
//                      rings: a K slot is free again as soon as S^T is done).  It finds its first
//                      copies from its own scan of lens, before the shared tables exist, and in the
//                      append-and-attend step moves the new key/value row into the cache.
//   two MMA warps      one thread each issues the tcgen05.mma of S^T, and of O^T
//   8 softmax warps    tcgen05.ld the logits of their row, P = exp2(S - reference) as bf16 (hi, and lo
//                      for short prefixes) into shared memory, per-thread partial sums.  Two O^T
//                      buffers: a finished segment is read out of TMEM after the next one's first stage.
//
// A sequence cut over several CTAs leaves one piece per CTA in the workspace.  With a control block
// (see below) the CTA that delivers the last piece merges them inside this kernel; without one the
// second-pass kernel does.  Everything between the roles is an mbarrier; every wait is bounded (see
// mbar_wait); no CTA ever waits for another CTA.
#pragma once
#include <cuda.h>

#include "decode_mma.cuh"

namespace mqa {

constexpr int kUmmaStageRows = 128;                              // cache rows per stage
constexpr int kUmmaHalfBytes = kUmmaStageRows * 128;             // 16 KiB: one 64-column box of 128 rows
constexpr int kUmmaSlotBytes = 2 * kUmmaHalfBytes;               // 32 KiB: the K (or the V) rows of a stage
constexpr int kUmmaSoftmaxWarps = 8;                             // warp w: TMEM lanes 32 * (w % 4) .., heads of half w / 4
constexpr int kUmmaSoftmaxThreads = kUmmaSoftmaxWarps * 32;
constexpr int kUmmaProducerWarp = 8, kUmmaSWarp = 9, kUmmaPvWarp = 10;
constexpr int kUmmaThreads = 11 * 32;
// virtual tiles in front of each sequence on the line: what crossing from one sequence to the next costs this kernel
constexpr int kUmmaBoundaryPenalty = 8;
constexpr int kGuessL2Stages = 2;                                // stages asked into L2 on a guess, beyond those the rings take
constexpr float kMaxLead = 16.f;                                 // log2 units a logit may exceed the reference maximum by

template <int HP>
struct UmmaCfg {
    static_assert(HP == 16 || HP == 32, "padded head count (more query rows than 32: decode_wide.cuh)");
    static constexpr int kKSlots = 2, kVSlots = 3;
    static constexpr int kQBytes = HP * 256;                     // HP head rows x 128 columns bf16, two 64-column boxes
    // P^T tile: 128 cache rows x 128 bytes (64 bf16 head slots, HP used), 128-byte swizzle: an MN-major B
    // operand, so that a softmax thread writes the weights of its cache row with 16-byte stores.  Two tiles:
    // the hi parts of two buffers (one rounding of P), or hi and lo of a single buffer (short prefixes).
    static constexpr int kPBytes = kUmmaStageRows * 128;
    static constexpr int kPTiles = 2;
    static constexpr int kQBufs = 2;
    static constexpr int kHeadsPerThread = HP / 2;               // a cache row's heads are split over two warps
    static constexpr int kChunk = kHeadsPerThread < 32 ? kHeadsPerThread : 32;   // heads handled per TMEM load
    // per-quarter maxima and sums [4][HP] each, reference maxima, factors of the last move, 1/sum of two segments
    static constexpr int kRedBytes = (2 * 4 + 4) * HP * 4;
    static constexpr int kPlanBytes = (2 * kStreamMaxSeqs + 1) * 4 + 12;   // line positions + rows per sequence
    static constexpr int kBarriers = 2 * kKSlots + 2 * kVSlots + 15;
    static constexpr int kSmemBytes = (kKSlots + kVSlots) * kUmmaSlotBytes + kQBufs * kQBytes + kPTiles * kPBytes + kRedBytes +
                                      kPlanBytes + kBarriers * 8 + 1024 /* alignment slack */;
    static_assert(kSmemBytes <= 227 * 1024, "exceeds the shared memory of one SM");
    static constexpr int kTmemCols = 4 * HP;                     // S^T twice, O^T twice (64, 128 or 256 columns)
};

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
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t (&r)[8]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr) : "memory");
}
// COLS (8, 16, 32 or 64) consecutive fp32 columns of this thread's TMEM lane
template <int COLS>
__device__ __forceinline__ void tmem_ld_cols(uint32_t taddr, uint32_t (&r)[COLS]) {
    if constexpr (COLS == 8) {
        tmem_ld8(taddr, r);
    } else if constexpr (COLS == 16) {
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
// Instruction descriptor: fp32 accumulator, bf16 A and B, M x N tile, A and B K-major unless said otherwise.
__host__ __device__ constexpr uint32_t umma_idesc(int M, int N, bool a_mn_major, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn_major ? 1u : 0u) << 15) | ((b_mn_major ? 1u : 0u) << 16) |
           ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// ---- control block of the single-launch step ---------------------------------------------------
// When a control block is given, the CTA that is last to deliver a piece of a sequence merges the pieces
// itself (no second-pass kernel), and one CTA advances lens at the end.  The block is the first
// kStreamCtrlBytes of the caller's workspace -- the same place and size whatever the batch, the head count
// and the grid, and no other kernel of the library writes there -- so every launch that uses a workspace
// finds the epoch word of the launch before it, of whatever shape that was.  Its contents are arbitrary
// the first time and nothing in it is ever reset: every launch works under a new epoch E = the epoch word
// as found + 1 (44 bits), read by every CTA before anything in the block is written, and a word counts only
// if it carries E.
//   ctrl[1]            epoch of the last launch (whatever the memory held, the first time)
//   ctrl[8 + c]        = E once CTA c has read the epoch and lens      ("started")
//   ctrl[8 + 256 + s]  = E << 20 | pieces of sequence s delivered so far
// The epoch is moved on by the first CTA that finds every CTA started (at least the CTA that started
// last does: the store of its own mark, a fence.sc and then the reads).  Until then nobody leaves
// the old epoch behind, so all CTAs of a launch agree on E.  A launch whose waits ran out still moves the
// epoch on (every CTA marks itself before its loop), so the block needs no repair afterwards.
constexpr unsigned long long kCtrlEpochMask = (1ull << 44) - 1;
constexpr int kCtrlCountBits = 20;
constexpr int kCtrlStarted = 8, kCtrlCounters = 8 + 256;
constexpr size_t kStreamCtrlBytes = (((size_t)(kCtrlCounters + kStreamMaxSeqs) * 8) + 255) & ~(size_t)255;

// One more piece of a sequence delivered: returns how many were delivered before it in this launch.
__device__ __forceinline__ unsigned int ctrl_arrive(unsigned long long* word, unsigned long long E) {
    const unsigned long long cmask = (1ull << kCtrlCountBits) - 1;
    unsigned long long old = atomicAdd(word, 1ull);
    if ((old >> kCtrlCountBits) == E) return (unsigned int)(old & cmask);
    // the word is from an earlier launch (or was never written): put this launch's tag on it, counting this piece
    unsigned long long expected = old + 1;
    for (int tries = 0; tries < 1024; ++tries) {
        const unsigned long long prev = atomicCAS(word, expected, (E << kCtrlCountBits) | 1ull);
        if (prev == expected) return 0u;
        if ((prev >> kCtrlCountBits) == E) return (unsigned int)(atomicAdd(word, 1ull) & cmask);   // another CTA tagged it meanwhile
        expected = prev;                                   // another CTA's add to the old word came in between
    }
    return 0xffffffffu;                                    // never seen; the caller then does not merge
}

// ---- thread-block cluster helpers (the pieces of a sequence, and the head groups of the output projection, are summed
// through distributed shared memory)
__device__ __forceinline__ uint32_t cluster_cta_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_size() {
    uint32_t n;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(n));
    return n;
}
// every thread of every CTA of the cluster, the same number of times on every path: what a CTA wrote to its shared
// memory before is visible to the others after
__device__ __forceinline__ void cluster_sync() {
    __syncwarp();                    // the aligned forms want the whole warp at the same instruction
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ float ld_cluster_f32(uint32_t local_addr, uint32_t rank) {
    uint32_t remote;
    float v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
    return v;
}
// The address, in the cluster's shared window, of this CTA's shared address `local` in the CTA of rank `rank`.
__device__ __forceinline__ uint32_t cluster_map(uint32_t local, uint32_t rank) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(rank));
    return remote;
}
__device__ __forceinline__ float4 cluster_ld_f4(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ float2 cluster_ld_f2(uint32_t addr) {
    float2 v;
    asm volatile("ld.shared::cluster.v2.f32 {%0,%1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr) : "memory");
    return v;
}

// Barrier over `threads` threads that also ORs a predicate over them.
__device__ __forceinline__ bool named_barrier_or(int id, int threads, bool pred) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 q, %1, 0;\n\t"
        "bar.red.or.pred p, %2, %3, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(out) : "r"((uint32_t)pred), "r"(id), "r"(threads) : "memory");
    return out != 0;
}

// Reduces N (8, 16 or 32) values per lane over the 32 lanes of a warp, all at once: afterwards lane l holds
// the total (sum, or maximum) of value number l % N.  v is used up.
template <int N, bool MAX>
__device__ __forceinline__ float warp_reduce_scatter(float (&v)[N], int lane) {
#pragma unroll
    for (int d = N / 2; d >= 1; d >>= 1) {
        const bool up = (lane & d) != 0;
#pragma unroll
        for (int i = 0; i < d; ++i) {
            const float send = up ? v[i] : v[i + d];
            const float keep = up ? v[i + d] : v[i];
            const float got = __shfl_xor_sync(0xffffffffu, send, d);
            v[i] = MAX ? fmaxf(keep, got) : keep + got;
        }
    }
#pragma unroll
    for (int d = N; d < 32; d <<= 1) {
        const float got = __shfl_xor_sync(0xffffffffu, v[0], d);
        v[0] = MAX ? fmaxf(v[0], got) : v[0] + got;
    }
    return v[0];
}

// All the softmax threads of the CTA that delivered the last piece of sequence s: o[s] = the pieces held by
// the CTAs lo..hi (those with a share of the line), merged in CTA order.  8 threads per head, 16 columns each.
// o_rows: the sequence's rows of o (its first query row onwards), n_rows of them.
__device__ __forceinline__ void merge_sequence_pieces(const float2* __restrict__ part_ml, const float* __restrict__ part_acc,
                                                   float* __restrict__ o_rows, int n_rows, int s, int h, int lo, int hi, int T,
                                                   unsigned long long magic, int tid) {
    const int g8 = tid & 7;
    for (int head = tid >> 3; head < n_rows; head += kUmmaSoftmaxThreads / 8) {
        float top = -INFINITY, den = 0.f;
        float4 num[4];
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) num[q4] = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int c0 = lo; c0 <= hi; c0 += 6) {
            float2 ml[6];
            float4 a[6][4];
#pragma unroll
            for (int k = 0; k < 6; ++k) {
                const int c = c0 + k;
                const bool live = c <= hi && share_begin(c, T, magic) != share_begin(c + 1, T, magic);
                ml[k] = make_float2(-INFINITY, 0.f);
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) a[k][q4] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (live) {
                    const size_t unit = ((size_t)c + s) * h + head;
                    ml[k] = __ldcg(part_ml + unit);
                    const float4* src = reinterpret_cast<const float4*>(part_acc + unit * kHeadDim) + g8;
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) a[k][q4] = __ldcg(src + q4 * 8);
                }
            }
            float top_new = top;
#pragma unroll
            for (int k = 0; k < 6; ++k) top_new = fmaxf(top_new, ml[k].x);
            const float keep = top == -INFINITY ? 0.f : fast_exp2(top - top_new);
            den *= keep;
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) { num[q4].x *= keep; num[q4].y *= keep; num[q4].z *= keep; num[q4].w *= keep; }
#pragma unroll
            for (int k = 0; k < 6; ++k) {
                const float w = ml[k].x == -INFINITY ? 0.f : fast_exp2(ml[k].x - top_new);
                den = fmaf(w, ml[k].y, den);
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                    num[q4].x = fmaf(w, a[k][q4].x, num[q4].x); num[q4].y = fmaf(w, a[k][q4].y, num[q4].y);
                    num[q4].z = fmaf(w, a[k][q4].z, num[q4].z); num[q4].w = fmaf(w, a[k][q4].w, num[q4].w);
                }
            }
            top = top_new;
        }
        const float inv = 1.f / den;
        float4* dst = reinterpret_cast<float4*>(o_rows + (size_t)head * kHeadDim) + g8;
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4)
            dst[q4 * 8] = make_float4(num[q4].x * inv, num[q4].y * inv, num[q4].z * inv, num[q4].w * inv);
    }
}

// HP = head rows of the Q tile (h rounded up to 16, 32 or 64).  GUESS: built with the code that starts copies on a
// guess before the wait (GUESS && early >= 2 below); kernels without it take early 0 or 1 only.
template <int HP, bool FUSED, bool GUESS = false>
__global__ void __launch_bounds__(kUmmaThreads, 1)
mqa_decode_stream_umma_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                              const __grid_constant__ CUtensorMap map_k_sub, const __grid_constant__ CUtensorMap map_v_sub,
                              const __grid_constant__ CUtensorMap map_q,
                              const int32_t* __restrict__ lens, float* __restrict__ o, int2* __restrict__ seq_span,
                              float2* __restrict__ part_ml, float* __restrict__ part_acc, int32_t* __restrict__ status,
                              int b, int h, int m_max, unsigned long long magic, const FusedArgs fa,
                              unsigned long long* __restrict__ ctrl, int32_t* __restrict__ lens_advance, int early_arg,
                              int read_once) {
    using Cfg = UmmaCfg<HP>;
    const int early = GUESS ? early_arg : (early_arg == 1 ? 1 : 0);
    constexpr int NK = Cfg::kKSlots, NV = Cfg::kVSlots, NQ = Cfg::kQBufs, CH = Cfg::kChunk, NCH = Cfg::kHeadsPerThread / CH;
    constexpr int kSubs = kUmmaStageRows / kTileRows;       // 4 sub-tiles of 32 rows per stage
    const bool appending = FUSED && fa.k_new != nullptr;
    const int cta = blockIdx.x, G = gridDim.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* ring = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);   // K slots, then V slots
    uint8_t* q_buf = ring + (NK + NV) * kUmmaSlotBytes;                 // 2 x Q
    uint8_t* p_buf = q_buf + Cfg::kQBufs * Cfg::kQBytes;                // P^T tiles
    float* red_m = reinterpret_cast<float*>(p_buf + Cfg::kPTiles * Cfg::kPBytes);   // [4 lane quarters][HP]
    float* red_l = red_m + 4 * HP;                                                  // [4 lane quarters][HP]
    float* m_sm = red_l + 4 * HP;                                   // [HP] reference maxima (log2 units) of the segment
    float* f_sm = m_sm + HP;                                                        // [HP] factor of the last move
    float* inv_sm = f_sm + HP;                                                      // [2][HP] 1 / sum of weights (1 for a partial), by segment parity
    int* prefix = reinterpret_cast<int*>(inv_sm + 2 * HP);                          // [b + 1]
    int* rows_of = prefix + kStreamMaxSeqs + 1;                                     // [b]
    uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(prefix) + (Cfg::kPlanBytes + 7) / 8 * 8);
    const uint32_t k_ring = smem_addr(ring), v_ring = k_ring + NK * kUmmaSlotBytes;
    const uint32_t q_s = smem_addr(q_buf), p_s = smem_addr(p_buf);
    // barrier table
    const uint32_t k_full = smem_addr(bars), k_empty = k_full + NK * 8;
    const uint32_t v_full = k_empty + NK * 8, v_empty = v_full + NV * 8;
    const uint32_t q_full = v_empty + NV * 8, q_empty = q_full + 16;
    const uint32_t s_ready = q_empty + 16, s_free = s_ready + 16;
    const uint32_t p_ready = s_free + 16, pv_done = p_ready + 16, o_free = pv_done + 16;   // o_free: one per O^T buffer
    const uint32_t go = o_free + 16;                        // the share's first segment is settled (see early below)
    __shared__ int timed_out, issued[2], plan_sm[8], merge_sm[8];   // merge_sm: count, then (sequence, first CTA, last CTA) x 2
    __shared__ unsigned long long epoch_sm[2];              // this launch's epoch; the epoch word as found
    __shared__ uint32_t tmem_base_slot;
    __shared__ int waited_sm;                                // 1 once a warp of this CTA has come back from the wait on the kernel before

    // set up by the thread that issues the copies: it may start some before the first CTA-wide barrier, and
    // program order is what puts the initialisation before them; every other thread first passes that barrier
    if (warp == kUmmaProducerWarp && lane == 0) {
        if (GUESS) asm volatile("st.volatile.shared.u32 [%0], %1;" ::"r"(smem_addr(&waited_sm)), "r"(0) : "memory");
        TS(0);
        prefetch_tensormap(&map_k); prefetch_tensormap(&map_v); prefetch_tensormap(&map_k_sub);
        prefetch_tensormap(&map_v_sub); prefetch_tensormap(&map_q);
        timed_out = 0;
        issued[0] = issued[1] = 0;
        merge_sm[0] = 0;
        for (int s = 0; s < NK; ++s) { mbar_init(k_full + s * 8, 1); mbar_init(k_empty + s * 8, 1); }
        for (int s = 0; s < NV; ++s) { mbar_init(v_full + s * 8, 1); mbar_init(v_empty + s * 8, 1); }
        for (int s = 0; s < 2; ++s) {
            mbar_init(q_full + s * 8, 1); mbar_init(q_empty + s * 8, 1);
            mbar_init(s_ready + s * 8, 1); mbar_init(s_free + s * 8, kUmmaSoftmaxWarps);
            mbar_init(p_ready + s * 8, kUmmaSoftmaxWarps); mbar_init(pv_done + s * 8, 1);
            mbar_init(o_free + s * 8, kUmmaSoftmaxWarps);
        }
        mbar_init(go, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        TS(10);
    }
    // what the producer thread set up is in place: the other warps pass this barrier inside stream_plan, before
    // they touch any of it, and do not wait for this warp again until the tables are built
    if (warp == kUmmaProducerWarp) { __syncwarp(); named_barrier_arrive(kPlanBarInit, kUmmaThreads); }
    if (warp == kUmmaSWarp) {                               // one warp owns the TMEM allocation
        tmem_alloc(smem_addr(&tmem_base_slot), Cfg::kTmemCols);
        tmem_relinquish();
    }
    // ---- the append inside the pass, by the 32 lanes of the producer warp: lane l < 16 moves 16 bytes of the
    // new key row, lane l >= 16 of the new value row.  The row is loaded when its segment begins and stored (and
    // made visible to the copy engine) before the stage that contains it is fetched.
    auto row_load = [&](int s) -> uint4 {
        const uint4* src = (lane < 16 ? fa.k_new : fa.v_new) + (size_t)s * (kRowBytes / 16) + (lane & 15);
        return __ldg(src);
    };
    auto row_store = [&](int s, int new_row, uint4 value) {
        uint4* dst = (lane < 16 ? fa.K : fa.V) + ((size_t)s * m_max + new_row) * (kRowBytes / 16) + (lane & 15);
        *dst = value;
        asm volatile("fence.proxy.async;" ::: "memory");   // the copy engine must see the row
        __syncwarp();
        asm volatile("fence.proxy.async;" ::: "memory");
    };
    // ---- what the producer warp does for a segment and for a stage.  A copy instruction takes a tenth of a
    // microsecond to issue, so the boxes of a stage go out in one instruction executed by four lanes: lane =
    // 2 * (0: the K rows, 1: the V rows) + (which 64-column half); the two boxes of Q by lanes 0 and 1.
    bool p_ok = true;                                       // no producer wait has run out
    auto issue_q = [&](int s, int seg) {                    // lanes 0 and 1
        const int qi = seg % NQ;
        if (seg >= NQ) p_ok = p_ok && mbar_wait(q_empty + qi * 8, ((seg / NQ) - 1) & 1);
        if (!p_ok) return;
        // the sequence's head rows (rows past h belong to the next sequence or read as zero: their
        // columns of S^T and O^T are never stored)
        if (lane == 0) mbar_expect_tx(q_full + qi * 8, Cfg::kQBytes);
        tma_load_2d(q_s + qi * Cfg::kQBytes + lane * (Cfg::kQBytes / 2), &map_q, lane * kBoxCols, s * h, q_full + qi * 8);
    };
    const uint64_t stream_policy = l2_stream_policy((read_once & 1) != 0);
    const bool withhold = (read_once & 2) != 0;             // for tests: one copy is never started, so that a wait runs out
    auto issue_stage = [&](int s, int u, int hi, int j) {   // lanes 0 to 3
        const int kv = lane >> 1, half = lane & 1;          // the K rows, then the V rows, each into its own ring
        const int nsub = min(kSubs, hi - u);
        const int y = s * m_max + u * kTileRows;
        const int n_slots = kv ? NV : NK;
        const int slot = j % n_slots;
        const uint32_t full = (kv ? v_full : k_full) + slot * 8;
        if (j >= n_slots) p_ok = p_ok && mbar_wait((kv ? v_empty : k_empty) + slot * 8, ((j / n_slots) - 1) & 1);
        if (!p_ok) return;
        const uint32_t dst = (kv ? v_ring : k_ring) + slot * kUmmaSlotBytes + half * kUmmaHalfBytes;
        if (half == 0) mbar_expect_tx(full, nsub * 2 * kBoxBytes);
        if (withhold && cta == 0 && j == 1 && lane == 3) {
            // (the V rows' second half of this CTA's second stage stays away)
        } else if (nsub == kSubs) {
            tma_load_2d_hint(dst, kv ? &map_v : &map_k, half * kBoxCols, y, full, stream_policy);
        } else {
            for (int i = 0; i < nsub; ++i)
                tma_load_2d_hint(dst + i * kBoxBytes, kv ? &map_v_sub : &map_k_sub, half * kBoxCols, y + i * kTileRows, full, stream_policy);
        }
        if (half == 0) issued[kv] = j + 1;                  // stages whose K (V) copies were started
    };

    // ---- what may start before the wait on the kernel before this one (early):
    // 0  nothing.
    // 1  that kernel writes nothing but q and the new key/value row (the input projection of the layer step) and,
    //    like every kernel here, lets this one start only after its own wait -- so everything older is complete,
    //    lens included, and only the producer warp has to wait, before it touches q or the new row.
    // 2  that kernel may be a step of this library on the same cache (a decoding loop): it writes one row per
    //    sequence, at or just below the end of the prefix, and moves lens on by one.  The producer warp works out
    //    its first segment from lens as it reads now and starts the copies of the stages that lie wholly below the
    //    last two rows of that prefix; right after the wait it asks for that sequence's q, then works the segment
    //    out again, and if the first stages are no longer the same (lens moved under it and a tile boundary was
    //    crossed) the copies are left to land and everything is started again.  The warp that issues S^T = K Q^T,
    //    whose results everything else waits for, starts only when told that the segment is settled (go).
    // 3  as 2 with a guess that is wrong on purpose, so that tests reach the recovery.
    int pre_issued = 0;                                     // stages whose copies were started here
    // The launch is made of clusters of C CTAs when the batch divides the grid (C = G / b) and the step is a single
    // launch.  With sequences of equal tile counts cluster c then holds sequence c: its CTAs take the sequence's stages
    // in turn (rank r: stages r, r + C, ...: "strided"), leave one piece each in their own shared memory and merge the
    // pieces through the cluster's shared window, with no partial result, fence or counter in global memory.  Whether
    // the sequences are equal is decided from lens, by every CTA alike (stream_plan); until then it is a guess.
    const uint32_t C = cluster_size();
    const int crank = (int)cluster_cta_rank();
    const int cl = (ctrl != nullptr && C > 1 && (long long)C * b == G) ? (int)C : 1;
    if (warp == kUmmaProducerWarp) {
        // One loop body serves both sides of the wait (with a guess it runs twice, and the second time its
        // instructions are already on the SM): work out the share's first segment, start what may be started.
        Segment g0 = {};
        int r0 = 0;
        bool have = false, q_started = false, strided0 = false;
        // A CTA that starts only when the kernel before has already completed (its SM was that kernel's last to become
        // free) gains nothing from a guess: by then a warp that went straight to the wait has come back and said so
        // (waited_sm, zeroed by this thread first, so that a 1 can only be that warp's), lens as it reads now is final,
        // and one pass does.
        int late = 0;
        if (GUESS && early >= 2) {
            if (lane == 0) asm volatile("ld.acquire.cta.shared.u32 %0, [%1];" : "=r"(late) : "r"(smem_addr(&waited_sm)) : "memory");
            late = __shfl_sync(0xffffffffu, late, 0);
        }
        const bool lensfree = GUESS && early >= 2 && cl > 1;
        const int passes = late ? 1 : early >= 1 ? 2 : 1;
#pragma unroll 1
        for (int pass = 0; pass < passes; ++pass) {
            const bool before = pass + 1 < passes;          // this pass runs ahead of the wait
            if (!before) {
                if (lane == 0) TS(11);
                grid_dependency_wait();                     // q, the new row, lens: all there now
                grid_launch_dependents();
                if (lane == 0) TS(1);
                if (GUESS && early >= 2 && have) {                   // q of the guessed sequence, while the guess is checked
                    if (lane < 2) issue_q(g0.s, 0);
                    q_started = true;
                }
                if (lane == 0) TS(12);
            }
            if (lensfree && before) {
                // A guess that needs no look at lens (a round trip to L2 saved on the way to the first copies): the
                // sequences are equal and long, so this CTA's first stages are stages crank and crank + C of sequence
                // cta / C.  Checked against lens after the wait like any guess.
                g0.s = cta / cl;
                g0.lo = crank * kSubs + (early == 3 ? kSubs : 0);    // (3, for tests: one stage off)
                g0.hi = m_max / kTileRows;                           // whole tiles of a full cache
                g0.whole = false;
                r0 = m_max + 2;                                      // rows below m_max may be asked for
                have = g0.lo < g0.hi;
                strided0 = true;
            } else if (before || early != 1) {              // (early == 1: lens cannot have moved)
                Segment g = {};
                int r = 0;
                bool strided = false;
                const bool found = first_segment<FUSED, kUmmaBoundaryPenalty>(lens, b, m_max, appending, magic, &g, &r, cl, crank, kSubs, &strided);
                if (before && lane == 0) TS(8);
                if (GUESS && before && early == 3) g.lo += kSubs;    // for tests: a guess that is one stage off
                if (!before && GUESS && early >= 2) {
                    // the stages started on the guess stand if this is how the share begins and each of them is a
                    // whole stage below the prefix's last two rows (which the step before may have been writing)
                    bool keep = have && found && g.s == g0.s && g.lo == g0.lo && strided == strided0;
                    const int ust = strided ? kSubs * cl : kSubs;
                    for (int i = 0; i < pre_issued; ++i)
                        keep = keep && g.lo + i * ust + kSubs <= g.hi && (g.lo + i * ust + kSubs) * kTileRows <= (r & (kAppendBit - 1)) - 2;
                    if (have && !keep) {
                        // what was started on the guess is not how this share begins: each of those barriers has
                        // completed one phase when its copy has landed; one more arrival completes a second,
                        // empty one, and the slot is as new (no consumer has looked: the first of them waits for go)
                        if (lane == 0) {
                            p_ok = p_ok && mbar_wait(q_full, 0);
                            if (p_ok) mbar_arrive(q_full);
                            for (int i = 0; i < pre_issued; ++i) {
                                p_ok = p_ok && mbar_wait(k_full + i * 8, 0) && mbar_wait(v_full + i * 8, 0);
                                if (p_ok) { mbar_arrive(k_full + i * 8); mbar_arrive(v_full + i * 8); }
                            }
                        }
                        p_ok = __shfl_sync(0xffffffffu, (int)p_ok, 0) != 0;
                        pre_issued = 0;
                        q_started = false;
                    }
                    if (lane == 0) mbar_arrive(go);
                    if (lane == 0) TS(13);
                }
                have = found;
                g0 = g;
                r0 = r;
                strided0 = strided;
            }
            if (have) {
                const int L = r0 & (kAppendBit - 1);
                const int new_row = (r0 & kAppendBit) ? L - 1 : -1;          // row this step appends
                const int ust = strided0 ? kSubs * cl : kSubs;               // tiles from one of this CTA's stages to the next
                // rows that may be fetched now lie below stop_row: ahead of the wait not this step's new row
                // (early == 1) or, on a guess, the prefix's last two rows, and then whole stages only
                const int stop_row = !before ? 0x7fffffff : early == 1 ? (new_row >= 0 ? new_row : 0x7fffffff) : L - 2;
                const int n_pre = min((g0.hi - g0.lo + ust - 1) / ust, NK < NV ? NK : NV);   // what the rings hold without a wait
                // which of this segment's stages holds the new row (-1: none)
                int p_row = -1;
                if (new_row >= 0) {
                    const int tile = new_row / kTileRows;
                    if (tile >= g0.lo && tile < g0.hi && (tile - g0.lo) % ust < kSubs) p_row = (tile - g0.lo) / ust;
                }
                if (!before && appending && p_row >= pre_issued && p_row < n_pre)
                    row_store(g0.s, new_row, row_load(g0.s));   // the new row lies in the stages started now
                if (lane < 4) {
                    if (lane < 2 && !before && !q_started) issue_q(g0.s, 0);
                    for (int u = g0.lo + pre_issued * ust; pre_issued < n_pre && (u + kSubs) * kTileRows <= stop_row &&
                                     !(before && GUESS && early >= 2 && u + kSubs > g0.hi);
                         u += ust, ++pre_issued)
                        issue_stage(g0.s, u, g0.hi, pre_issued);
                    if (before && lensfree) {
                        // and the stages after those are asked into L2 (measured at 32 sequences x 8192 rows on 128
                        // CTAs: 26.9 us per step without, 26.2 / 26.0 / 26.5 / 27.2 us with 1 / 2 / 3 / 4 stages)
                        int u = g0.lo + pre_issued * ust;
                        for (int p = 0; p < kGuessL2Stages && (u + kSubs) * kTileRows <= stop_row && u + kSubs <= g0.hi; ++p, u += ust) {
                            tma_prefetch_l2_2d((lane >> 1) ? &map_v : &map_k, (lane & 1) * kBoxCols, g0.s * m_max + u * kTileRows);
                        }
                    }
                }
                pre_issued = __shfl_sync(0xffffffffu, pre_issued, 0);
                p_ok = __all_sync(0xffffffffu, p_ok);
            }
        }
    } else if (early != 1) {
        grid_dependency_wait();      // lens and the newest cache row may come from the kernel before
        grid_launch_dependents();
        if (GUESS && threadIdx.x == kUmmaSWarp * 32)
            asm volatile("st.release.cta.shared.u32 [%0], %1;" ::"r"(smem_addr(&waited_sm)), "r"(1) : "memory");
    }
    if (ctrl && threadIdx.x == kUmmaPvWarp * 32) {          // (a thread with nothing else to do at this point)
        const unsigned long long was = __ldcg(ctrl + 1);
        unsigned long long E = (was + 1) & kCtrlEpochMask;
        if (E == 0) E = 1;
        epoch_sm[0] = E;
        epoch_sm[1] = was;
    }

    tc_fence_before();
    const SharePlan plan = stream_plan<FUSED, kUmmaThreads, kUmmaBoundaryPenalty>(lens, o, status, b, h, m_max, appending, magic, prefix,
                                                            rows_of, plan_sm, kUmmaProducerWarp);
    const int T = plan.T, t_begin = plan.t_begin, t_end = plan.t_end, s_first = plan.s_first;
    tc_fence_after();
    // sequences of equal tile counts in a launch made of clusters: strided stages, pieces merged through the cluster
    const bool via_cluster = cl > 1 && plan.equal;
    const int ustep = via_cluster ? kSubs * cl : kSubs;     // tiles from one of this CTA's stages to the next
    // the next segment of this CTA's share: a run of its line share, or the whole sequence of its cluster taken in strides
    auto next_segment = [&](ShareWalker<kUmmaBoundaryPenalty>& walk, Segment& g, int seg) -> bool {
        if (!via_cluster) return walk.next(g);
        if (seg > 0) return false;
        g.s = cta / cl;
        g.lo = crank * kSubs;
        g.hi = prefix[g.s + 1] - prefix[g.s] - kUmmaBoundaryPenalty;
        g.whole = false;
        return g.lo < g.hi;
    };
    float* piece_acc = reinterpret_cast<float*>(ring);                        // [h][128] in the first K slot (free by then)
    float2* piece_ml = reinterpret_cast<float2*>(ring + kUmmaSlotBytes);      // [h] (reference maximum, sum) in the second
    bool piece_left = false;                                // (softmax warps) this CTA has left a piece there
    const uint32_t tmem_base = tmem_base_slot;
    const uint32_t tmem_o = tmem_base + 2 * HP;             // S^T buffers at columns 0 and HP, two O^T buffers after them

    if (warp == kUmmaProducerWarp) {
        // =============================================================== TMA producer
        const unsigned long long E = ctrl ? epoch_sm[0] : 0ull;
        if (ctrl && lane == 0) __stcg(ctrl + kCtrlStarted + cta, E);   // this CTA has read the epoch and lens
        if (t_begin < t_end) {                              // all lanes walk the share; lane 0 waits and issues the copies
            int j = 0, seg = 0;
            ShareWalker<kUmmaBoundaryPenalty> walk{prefix, t_begin, t_end, s_first};
            Segment g;
            for (; p_ok && next_segment(walk, g, seg); ++seg) {
                if (lane < 2 && !(seg == 0 && pre_issued > 0)) issue_q(g.s, seg);
                const int rows_entry = rows_of[g.s];
                const int new_row = (rows_entry & kAppendBit) ? (rows_entry & (kAppendBit - 1)) - 1 : -1;   // row this step appends
                // which of the segment's stages holds the new row (-1: none, it is not this CTA's to write)
                int p_row = -1;
                if (new_row >= 0) {
                    const int tile = new_row / kTileRows;
                    if (tile >= g.lo && tile < g.hi && (tile - g.lo) % ustep < kSubs) p_row = (tile - g.lo) / ustep;
                }
                // the new row is in this segment and was not written on the way to the first stages
                bool row_due = appending && p_row >= 0 && !(seg == 0 && p_row < pre_issued);
                uint4 row = make_uint4(0u, 0u, 0u, 0u);
                if (row_due) row = row_load(g.s);
                for (int u = g.lo; u < g.hi && p_ok; u += ustep, ++j) {
                    // stored once the segment's first stage is on its way, or earlier if that stage holds the row
                    if (row_due && (u > g.lo || p_row == 0)) {
                        row_store(g.s, new_row, row);
                        row_due = false;
                    }
                    if (lane < 4 && j >= pre_issued) issue_stage(g.s, u, g.hi, j);
                    p_ok = __all_sync(0xffffffffu, p_ok);
                }
            }
            if (lane == 0 && !p_ok) atomicExch(&timed_out, 1);
        }
        if (ctrl) {
            // Has every CTA started?  Then nobody will read the epoch word or lens again: the first CTA to
            // see that moves the epoch on and, in the append-and-attend step, advances lens.
            __syncwarp();
            asm volatile("fence.sc.gpu;" ::: "memory");
            bool all = true;
            for (int c = lane; c < G; c += 32) all = all && __ldcg(ctrl + kCtrlStarted + c) == E;
            all = __all_sync(0xffffffffu, all);
            int won = 0;
            if (all && lane == 0) won = atomicCAS(ctrl + 1, epoch_sm[1], E) == epoch_sm[1];
            won = __shfl_sync(0xffffffffu, won, 0);
            if (won) {
                if (lens_advance)
                    for (int s = lane; s < b; s += 32)
                        if (rows_of[s] & kAppendBit) lens_advance[s] = rows_of[s] & (kAppendBit - 1);
            }
        }
    } else if (warp == kUmmaSWarp) {
        // =============================================================== issuer of S^T = K Q^T
        if (lane == 0 && t_begin < t_end) {
            constexpr uint32_t kIdescS = umma_idesc(128, HP, false, false);
            bool ok = !(GUESS && early >= 2) || mbar_wait(go, 0);
            TS(14);
            int j = 0, seg = 0;
            ShareWalker<kUmmaBoundaryPenalty> walk{prefix, t_begin, t_end, s_first};
            Segment g;
            for (; next_segment(walk, g, seg); ++seg) {
                const int qi = seg % NQ;
                if (ok) ok = mbar_wait(q_full + qi * 8, (seg / NQ) & 1);
                if (seg == 0) TS(15);
                for (int u = g.lo; u < g.hi; u += ustep, ++j) {
                    const int slot = j % NK, sb = j & 1;
                    if (ok) ok = mbar_wait(k_full + slot * 8, (j / NK) & 1);
                    if (j == 0) TS(2);
                    TS(3);
                    ST(j, 0);
                    if (ok && j >= 2) ok = mbar_wait(s_free + sb * 8, ((j >> 1) - 1) & 1);
                    ST(j, 1);
                    tc_fence_after();
                    if (ok) {
                        const uint32_t k_s = k_ring + slot * kUmmaSlotBytes;
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks) {             // 8 k-steps of 16 columns; 4 per 64-column box
                            const uint64_t a = umma_desc(k_s + (ks >> 2) * kUmmaHalfBytes + (ks & 3) * 32, 16, 1024);
                            const uint64_t bd = umma_desc(q_s + qi * Cfg::kQBytes + (ks >> 2) * (Cfg::kQBytes / 2) + (ks & 3) * 32, 16, 1024);
                            umma_ss(tmem_base + sb * HP, a, bd, kIdescS, ks ? 1u : 0u);
                        }
                    }
                    tc_commit(s_ready + sb * 8);
                    tc_commit(k_empty + slot * 8);                   // the K rows are not needed again
                    if (u + ustep >= g.hi) tc_commit(q_empty + qi * 8);   // last use of this segment's Q
                }
            }
            if (!ok) atomicExch(&timed_out, 1);
        }
    } else if (warp == kUmmaPvWarp) {
        // =============================================================== issuer of O^T += V^T P^T
        if (lane == 0 && t_begin < t_end) {
            constexpr uint32_t kIdescO = umma_idesc(128, HP, true, true);
            bool ok = true;
            int j = 0, seg = 0;
            ShareWalker<kUmmaBoundaryPenalty> walk{prefix, t_begin, t_end, s_first};
            Segment g;
            for (; next_segment(walk, g, seg); ++seg) {
                const int L = rows_of[g.s] & (kAppendBit - 1);
                const int parts = L >= kSingleRoundingMinRows ? 1 : 2;   // P hi only, or hi then lo (as the softmax warps wrote it)
                for (int u = g.lo; u < g.hi; u += ustep, ++j) {
                    const int pb = j & 1, slot = j % NV;
                    // the weights first: they exist only once q has arrived, and before that a slot's barrier may
                    // still be on its way back from copies started on a guess (see early above)
                    if (ok) ok = mbar_wait(p_ready + pb * 8, (j >> 1) & 1);
                    ST(j, 5);
                    if (ok) ok = mbar_wait(v_full + slot * 8, (j / NV) & 1);
                    ST(j, 6);
                    // segments alternate between the two O^T buffers; the segment before the last has read this one out
                    if (ok && u == g.lo && seg >= 2) ok = mbar_wait(o_free + (seg & 1) * 8, ((seg >> 1) - 1) & 1);
                    tc_fence_after();
                    if (ok) {
                        const uint32_t v_s = v_ring + slot * kUmmaSlotBytes;
                        for (int part = 0; part < parts; ++part) {
                            const uint32_t pt = p_s + (parts == 2 ? part : pb) * Cfg::kPBytes;
#pragma unroll
                            for (int kk = 0; kk < 8; ++kk) {         // 8 k-steps of 16 cache rows
                                const uint64_t a = umma_desc(v_s + kk * 2048, kUmmaHalfBytes, 1024);
                                const uint64_t bd = umma_desc(pt + kk * 2048, Cfg::kPBytes, 1024);
                                umma_ss(tmem_o + (seg & 1) * HP, a, bd, kIdescO, (u == g.lo && part == 0 && kk == 0) ? 0u : 1u);
                            }
                        }
                    }
                    tc_commit(v_empty + slot * 8);
                    tc_commit(pv_done + pb * 8);                     // this P^T buffer is free, O^T is up to date
                }
            }
            if (!ok) atomicExch(&timed_out, 1);
        }
    } else {
        // =============================================================== softmax warps
        if (warp == 0) {                                    // second-pass bookkeeping, spread over the CTAs
            for (int s = cta + lane * G; s < b; s += G * 32) {
                const int t0 = prefix[s] + kUmmaBoundaryPenalty, t1 = prefix[s + 1];     // its real tiles on the line
                seq_span[s] = t1 > t0 ? make_int2(stream_owner(t0, T, G), stream_owner(t1 - 1, T, G)) : make_int2(0, 0);
            }
            if (cta == 0 && lane == 0) seq_span[b] = make_int2((int)T, G);
        }
        if (t_begin < t_end) {
            constexpr int HH = Cfg::kHeadsPerThread;
            const int quarter = warp & 3, half = warp >> 2;
            const int t = quarter * 32 + lane;              // this thread's cache row of every stage = its TMEM lane;
                                                            // when a segment is read out, its column of O^T
            const int tid = warp * 32 + lane;               // 0 .. 255 among the softmax threads
            const int head0 = half * HH;                    // this thread's heads: head0 .. head0 + HH - 1
            const uint32_t lane_base = tmem_base + ((uint32_t)(quarter * 32) << 16);
            // where this row's weights go in a P^T tile (128 cache rows x 128 bytes, 128-byte swizzle): the 16
            // bytes of heads 8c .. 8c+7 at row * 128 + ((c ^ (row & 7)) << 4)
            const uint32_t p_row = (uint32_t)(t * 128), p_xor = (uint32_t)((t & 7) << 4);
            bool ok = true;
            int j = 0, seg = 0;
            // a finished segment whose O^T has not been read out of TMEM yet (done after the next segment's first stage)
            bool pend = false;
            bool prev_hilo = false;                         // the stage before wrote hi and lo parts of P
            float* pend_dst = nullptr;
            int pend_par = 0, pend_j = 0, pend_s = 0, pend_rows = 0;
            bool pend_whole = false;
            auto read_out = [&]() {
                // O^T[column t][head] of the finished segment -> o (divided by the sum) or its partial slot
                if (ok) ok = mbar_wait(pv_done + (pend_j & 1) * 8, (pend_j >> 1) & 1);   // the segment's last product
                tc_fence_after();
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    uint32_t y[CH];
                    tmem_ld_cols<CH>(lane_base + 2 * HP + pend_par * HP + head0 + c * CH, y);
                    float inv[CH];
#pragma unroll
                    for (int i = 0; i < CH; i += 4) {
                        const float4 v4 = *reinterpret_cast<const float4*>(inv_sm + pend_par * HP + head0 + c * CH + i);
                        inv[i] = v4.x; inv[i + 1] = v4.y; inv[i + 2] = v4.z; inv[i + 3] = v4.w;
                    }
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < CH; ++i)
                        if (head0 + c * CH + i < pend_rows) pend_dst[(size_t)(head0 + c * CH + i) * kHeadDim] = __uint_as_float(y[i]) * inv[i];
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(o_free + pend_par * 8);   // this O^T buffer may be overwritten
                pend = false;
                if (ctrl && !pend_whole && !via_cluster) {
                    // ---- single-launch step: the piece is delivered; the CTA that delivers a sequence's
                    // last piece merges them all into o (pieces in CTA order whoever merges: deterministic)
                    const int s = pend_s;
                    __threadfence();
                    named_barrier(2, kUmmaSoftmaxThreads);
                    if (warp == 0) {
                        const int t0 = prefix[s] + kUmmaBoundaryPenalty, t1 = prefix[s + 1];
                        const int lo = stream_owner(t0, T, G), hi = stream_owner(t1 - 1, T, G);
                        int n = 0;
                        for (int c = lo + lane; c <= hi; c += 32) n += share_begin(c, T, magic) != share_begin(c + 1, T, magic);
#pragma unroll
                        for (int d = 16; d >= 1; d >>= 1) n += __shfl_xor_sync(0xffffffffu, n, d);
                        if (lane == 0) {
                            const unsigned int before = ctrl_arrive(ctrl + kCtrlCounters + s, epoch_sm[0]);
                            if (before + 1 == (unsigned int)n) {        // the last piece: note the merge, done when the share is finished
                                const int k = merge_sm[0]++;
                                merge_sm[1 + 3 * k] = s;
                                merge_sm[2 + 3 * k] = lo;
                                merge_sm[3 + 3 * k] = hi;
                            }
                        }
                    }
                }
            };
            ShareWalker<kUmmaBoundaryPenalty> walk{prefix, t_begin, t_end, s_first};
            Segment g;
            for (; next_segment(walk, g, seg); ++seg) {
                const int s = g.s;
                const int L = rows_of[s] & (kAppendBit - 1);
                const bool whole = g.whole;
                const bool hilo = L < kSingleRoundingMinRows;    // long prefixes: one bf16 rounding of P is enough
                const int par = seg & 1;                    // O^T buffer of this segment
                float l_sum[HH];                            // this row's share of its heads' sums of weights
#pragma unroll
                for (int i = 0; i < HH; ++i) l_sum[i] = 0.f;
                for (int u = g.lo; u < g.hi; u += ustep, ++j) {
                    const int sb = j & 1, pb = j & 1;
                    const bool first = u == g.lo;           // nothing accumulated yet: no reference maxima, O^T not started
                    // rows of this stage that count: what was fetched (the share may end mid-stage) and
                    // lies inside the prefix; always >= 1
                    const int fetched = min(kSubs, g.hi - u) * kTileRows;
                    const int valid = min(fetched, L - u * kTileRows);
                    const bool row_ok = t < valid;
                    if (ok) ok = mbar_wait(s_ready + sb * 8, (j >> 1) & 1);
                    if (tid == 0) ST(j, 2);
                    tc_fence_after();
                    uint32_t xr[HH];
#pragma unroll
                    for (int c = 0; c < NCH; ++c) {
                        uint32_t part[CH];
                        tmem_ld_cols<CH>(lane_base + sb * HP + head0 + c * CH, part);
#pragma unroll
                        for (int i = 0; i < CH; ++i) xr[c * CH + i] = part[i];
                    }
                    tmem_wait_ld();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(s_free + sb * 8);             // S^T is in registers now
                    // ---- logits in log2 units, masked by index; how far the largest leads its reference
                    float x[HH];
                    float lead = -INFINITY;
#pragma unroll
                    for (int i = 0; i < HH; i += 4) {
                        const float4 m4 = first ? make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY)
                                                : *reinterpret_cast<const float4*>(m_sm + head0 + i);
                        const float mv[4] = {m4.x, m4.y, m4.z, m4.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            x[i + e] = row_ok ? __fmul_rn(__uint_as_float(xr[i + e]), kLog2e) : -INFINITY;   // select, never multiply
                            lead = fmaxf(lead, x[i + e] - mv[e]);           // (-inf) - (-inf) = NaN is ignored by fmaxf
                        }
                    }
                    if (named_barrier_or(1, kUmmaSoftmaxThreads, lead > kMaxLead)) {
                        // ---- some logit leads by too much (always on a segment's first stage): every head's
                        // reference moves to the largest logit seen so far; sums and O^T are rescaled
#pragma unroll
                        for (int c = 0; c < NCH; ++c) {
                            float r[CH];
#pragma unroll
                            for (int i = 0; i < CH; ++i) r[i] = x[c * CH + i];
                            const float top = warp_reduce_scatter<CH, true>(r, lane);
                            if (lane < CH) red_m[quarter * HP + head0 + c * CH + lane] = top;
                        }
                        named_barrier(2, kUmmaSoftmaxThreads);
                        if (tid < HP) {
                            const float m_old = first ? -INFINITY : m_sm[tid];
                            float m_new = m_old;
#pragma unroll
                            for (int w = 0; w < 4; ++w) m_new = fmaxf(m_new, red_m[w * HP + tid]);   // finite: the stage has a valid row
                            f_sm[tid] = fast_exp2(m_old - m_new);            // 0 on the first stage, 1 if unchanged
                            m_sm[tid] = m_new;
                        }
                        named_barrier(2, kUmmaSoftmaxThreads);
                        if (!first) {
#pragma unroll
                            for (int i = 0; i < HH; i += 4) {
                                const float4 f4 = *reinterpret_cast<const float4*>(f_sm + head0 + i);
                                l_sum[i] *= f4.x; l_sum[i + 1] *= f4.y; l_sum[i + 2] *= f4.z; l_sum[i + 3] *= f4.w;
                            }
                            // O^T holds the stages before this one: wait for the last of their products, scale
                            // column (head) i of this thread's lane by f[i]
                            if (ok) ok = mbar_wait(pv_done + ((j - 1) & 1) * 8, ((j - 1) >> 1) & 1);
                            tc_fence_after();
#pragma unroll
                            for (int c = 0; c < NCH; ++c) {
                                uint32_t y[CH];
                                const uint32_t at = lane_base + 2 * HP + par * HP + head0 + c * CH;
                                tmem_ld_cols<CH>(at, y);
                                tmem_wait_ld();
#pragma unroll
                                for (int i = 0; i < CH; i += 4) {
                                    const float4 f4 = *reinterpret_cast<const float4*>(f_sm + head0 + c * CH + i);
                                    y[i] = __float_as_uint(__uint_as_float(y[i]) * f4.x);
                                    y[i + 1] = __float_as_uint(__uint_as_float(y[i + 1]) * f4.y);
                                    y[i + 2] = __float_as_uint(__uint_as_float(y[i + 2]) * f4.z);
                                    y[i + 3] = __float_as_uint(__uint_as_float(y[i + 3]) * f4.w);
                                }
                                tmem_st_words<CH>(at, y);
                            }
                            tmem_wait_st();
                            tc_fence_before();
                        }
                    }
                    // this P^T tile was last read by the product of stage j-2 (of stage j-1 when that stage or
                    // this one has hi and lo parts, which take both tiles)
                    if (tid == 0) ST(j, 3);
                    if (j >= 2 && ok) ok = mbar_wait(pv_done + pb * 8, ((j >> 1) - 1) & 1);
                    if ((hilo || prev_hilo) && j >= 1 && ok) ok = mbar_wait(pv_done + ((j - 1) & 1) * 8, ((j - 1) >> 1) & 1);
                    prev_hilo = hilo;
                    tc_fence_after();                       // the tensor core's reads of the tile come before the stores below
                    // ---- P = exp2(S - reference): 0 for a masked row; bf16 hi (and lo) into the P^T tiles
                    const uint32_t p_hi = p_s + (hilo ? 0 : pb) * Cfg::kPBytes + p_row, p_lo = p_s + Cfg::kPBytes + p_row;
#pragma unroll
                    for (int c = 0; c < HH / 8; ++c) {
                        const float4 ma = *reinterpret_cast<const float4*>(m_sm + head0 + c * 8);
                        const float4 mb = *reinterpret_cast<const float4*>(m_sm + head0 + c * 8 + 4);
                        const float mv[8] = {ma.x, ma.y, ma.z, ma.w, mb.x, mb.y, mb.z, mb.w};
                        float pw[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            pw[e] = fast_exp2(x[c * 8 + e] - mv[e]);
                            l_sum[c * 8 + e] += pw[e];
                        }
                        uint32_t hi[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) hi[e] = pack_bf16(pw[2 * e], pw[2 * e + 1]);
                        const uint32_t at = ((uint32_t)((half * (HH / 8) + c) << 4)) ^ p_xor;
                        asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(p_hi + at), "r"(hi[0]), "r"(hi[1]), "r"(hi[2]), "r"(hi[3]));
                        if (hilo) {
                            uint32_t lo[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                lo[e] = pack_bf16(pw[2 * e] - bf16_lo(hi[e]), pw[2 * e + 1] - bf16_hi(hi[e]));
                            asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(p_lo + at), "r"(lo[0]), "r"(lo[1]), "r"(lo[2]), "r"(lo[3]));
                        }
                    }
                    // a stage that runs past the prefix: the tensor core would multiply the zero weights
                    // with whatever lies there (NaN * 0 = NaN), so those V rows are cleared first
                    if (valid < kUmmaStageRows) {
                        const int slot = j % NV;
                        if (ok) ok = mbar_wait(v_full + slot * 8, (j / NV) & 1);
                        const uint32_t v_s = v_ring + slot * kUmmaSlotBytes;
                        for (int i = tid; i < (kUmmaStageRows - valid) * 16; i += kUmmaSoftmaxThreads) {
                            const int vrow = valid + (i >> 4), ch = i & 15;  // 16 chunks of 16 bytes per row
                            const uint32_t a = v_s + (ch >> 3) * kUmmaHalfBytes + vrow * 128 + ((ch & 7) << 4);
                            asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0u) : "memory");
                        }
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // P^T (and cleared V) visible to the tensor core
                    __syncwarp();
                    if (lane == 0) mbar_arrive(p_ready + pb * 8);
                    if (tid == 0) ST(j, 4);
                    // the segment before this one is read out of its own O^T buffer now, after this
                    // segment's first stage is on its way (its last product has long finished)
                    if (pend) read_out();
                }
                // ---- segment done: add up the rows' sums; thread i < HP keeps head i's 1/sum for the read-out
                // and writes (maximum, sum) of a partial result.  O^T itself is read out later (see above).
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    float r[CH];
#pragma unroll
                    for (int i = 0; i < CH; ++i) r[i] = l_sum[c * CH + i];
                    const float tot = warp_reduce_scatter<CH, false>(r, lane);
                    if (lane < CH) red_l[quarter * HP + head0 + c * CH + lane] = tot;
                }
                named_barrier(2, kUmmaSoftmaxThreads);
                const size_t slot = (size_t)cta + s;
                if (tid < HP) {
                    float tot = 0.f;
#pragma unroll
                    for (int w = 0; w < 4; ++w) tot += red_l[w * HP + tid];
                    inv_sm[par * HP + tid] = whole ? 1.f / tot : 1.f;
                    if (!whole && tid < h) {
                        if (via_cluster) piece_ml[tid] = make_float2(m_sm[tid], tot);
                        else part_ml[slot * h + tid] = make_float2(m_sm[tid], tot);
                    }
                }
                piece_left = true;
                pend = true;
                pend_dst = (whole ? o + (size_t)s * h * kHeadDim : via_cluster ? piece_acc : part_acc + slot * h * kHeadDim) + t;
                pend_rows = h;
                pend_par = par;
                pend_j = j - 1;
                pend_s = s;
                pend_whole = whole;
            }
            if (tid == 0) TS(4);
            if (pend) {
                named_barrier(2, kUmmaSoftmaxThreads);      // the last segment's 1/sum values are in shared memory
                read_out();
            }
            if (tid == 0) TS(5);
            if (ctrl && !via_cluster) {
                // sequences whose last piece this CTA delivered (a share has at most two cut segments)
                named_barrier(2, kUmmaSoftmaxThreads);
                const int n_merge = merge_sm[0];
                if (n_merge > 0) __threadfence();
                for (int k = 0; k < n_merge; ++k)
                    merge_sequence_pieces(part_ml, part_acc, o + (size_t)merge_sm[1 + 3 * k] * h * kHeadDim,
                                          h, merge_sm[1 + 3 * k], h, merge_sm[2 + 3 * k],
                                          merge_sm[3 + 3 * k], T, magic, tid);
            }
            if (!ok) atomicExch(&timed_out, 1);
        }
    }

    if (via_cluster) {
        // a CTA whose share holds none of the sequence's rows (short sequences: nothing but the virtual tiles in
        // front of them) leaves an empty piece
        if (warp < kUmmaSoftmaxWarps && !piece_left && threadIdx.x < h) piece_ml[threadIdx.x] = make_float2(-INFINITY, 0.f);
        // every thread of the cluster: the C pieces lie in their CTAs' shared memory
        cluster_sync();
        if (threadIdx.x == 0) TS(6);
        if (warp < kUmmaSoftmaxWarps) {
            // CTA of rank r merges the heads [r * per, (r + 1) * per) of its sequence, pieces in rank (= row) order:
            // a thread takes 16 bytes of a head's 128 outputs
            const uint32_t rank = cluster_cta_rank();
            const int per = (h + (int)C - 1) / (int)C;
            const int s = cta / (int)C;
            const int tid = threadIdx.x;
            const uint32_t acc_s = smem_addr(piece_acc), ml_s = smem_addr(piece_ml);
            for (int item = tid; item < per * (kHeadDim / 4); item += kUmmaSoftmaxThreads) {
                const int head = (int)rank * per + (item >> 5), c4 = item & 31;
                if (head >= h) break;
                // the (maximum, sum) pairs of all pieces first, then the sums eight pieces at a time (a cluster has up to 16)
                float top = -INFINITY;
                float2 ml[16];
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    ml[c] = make_float2(-INFINITY, 0.f);
                    if (c < (int)C) ml[c] = cluster_ld_f2(cluster_map(ml_s + head * 8, c));
                    top = fmaxf(top, ml[c].x);
                }
                float den = 0.f;
                float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int c0 = 0; c0 < 16; c0 += 8) {
                    if (c0 >= (int)C) break;
                    float4 a[8];
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        a[c] = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (c0 + c < (int)C) a[c] = cluster_ld_f4(cluster_map(acc_s + (head * kHeadDim + c4 * 4) * 4, c0 + c));
                    }
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        if (ml[c0 + c].x == -INFINITY) continue;  // an empty piece (its sums were never written) is skipped, not multiplied
                        const float w = fast_exp2(ml[c0 + c].x - top);
                        den = fmaf(w, ml[c0 + c].y, den);
                        num.x = fmaf(w, a[c].x, num.x); num.y = fmaf(w, a[c].y, num.y);
                        num.z = fmaf(w, a[c].z, num.z); num.w = fmaf(w, a[c].w, num.w);
                    }
                }
                const float inv = 1.f / den;
                *reinterpret_cast<float4*>(o + ((size_t)s * h + head) * kHeadDim + c4 * 4) =
                    make_float4(num.x * inv, num.y * inv, num.z * inv, num.w * inv);
            }
        }
        if (threadIdx.x == 0) TS(7);
        cluster_sync();                                 // nobody leaves while its shared memory is being read
    }
    tc_fence_before();
    __syncthreads();
    if (timed_out && threadIdx.x == 0) {
        // before the CTA leaves: the last copy started into each ring slot has to land
        const int n_k = issued[0], n_v = issued[1];
        for (int s = 0; s < NK && s < n_k; ++s) mbar_wait(k_full + s * 8, ((n_k - 1 - s) / NK) & 1);
        for (int s = 0; s < NV && s < n_v; ++s) mbar_wait(v_full + s * 8, ((n_v - 1 - s) / NV) & 1);
        if (status) atomicOr(status, kStatusPipelineTimeout);
    }
    __syncthreads();
    if (warp == kUmmaSWarp) {
        tc_fence_after();
        tmem_dealloc(tmem_base, Cfg::kTmemCols);
    }
    if (threadIdx.x == 0) TS(9);
}

}  // namespace mqa
