// Multi-query attention over many query positions at once (Section 3, the attention lines of the batched function:
// logits = einsum(bhnk,bmk->bhnm), weights = softmax(logits + mask), O = einsum(bhnm,bmv->bhnv)) under the mask of
// Section 2.3 for an autoregressive model.  This is the one part of the method whose arithmetic intensity is high:
// every K/V row is used by all h heads and by every later position, so it runs against the tensor-core roofline.
//
// Shape of the work on sm_100a.  A CTA takes 128 consecutive positions of TWO heads of one sequence (multi-query: the
// heads share K and V, so one staged K/V tile of 128 rows serves 256 query rows) and walks the cache rows up to its
// last position in stages of 128:
//     S_w   = Q_w K_j^T       tcgen05.mma, M = 128 query rows (TMEM lanes), N = 128 cache rows, fp32 in TMEM
//     P_w   = exp2(S_w log2e - m)   one thread per query row: the row's maximum and sum need no other thread
//     O_w  += P_w V_j         tcgen05.mma with A = P_w read from TMEM (bf16 pairs written over S_w), B = V_j (MN-major)
// for w = 0, 1.  While the four softmax warps of one head work on S_w, the tensor core computes the other head's
// products: the issue order is S_0 S_1 | PV_0 S_0' | PV_1 S_1' | ...  TMEM: S_0, S_1, O_0, O_1 of 128 columns each
// (all 512).  The reference maximum of a row moves only when the row's largest logit leads it by more than
// kPfMaxLead (then O_w's row is rescaled in TMEM by the row's own thread); P is bounded by 2^kPfMaxLead.
// Rows of a tile whose memory is shorter than 1024 rows feed P as bf16 hi + lo parts (two products), like the
// decoding kernels, so that the rounding of few large weights stays inside the tolerance.
//
// Roles: warps 0-3 softmax of head 0, warps 4-7 softmax of head 1, warp 8 TMA producer, warp 9 MMA issuer.
// Every wait is bounded; a wait that runs out flags PIPELINE_TIMEOUT and the CTA drains and leaves.
#pragma once
#include "decode_umma.cuh"

namespace mqa {

constexpr int kPfRows = 128;                                   // query positions per tile = cache rows per stage
constexpr int kPfTileBytes = kPfRows * kRowBytes;              // 32 KiB: 128 rows x 128 bf16, two 64-column boxes
constexpr int kPfHalfBytes = kPfTileBytes / 2;
constexpr int kPfKSlots = 2, kPfVSlots = 2;
constexpr int kPfThreads = 12 * 32;                            // (warps 10 and 11 only complete the third warpgroup)
constexpr int kPfProducerWarp = 8, kPfMmaWarp = 9;
constexpr int kPfRegsSoftmax = 216, kPfRegsOther = 72;
constexpr float kPfMaxLead = 8.f;                              // log2 units a logit may exceed its row's reference by
// barriers: q_full, k_full/k_empty[2], v_full/v_empty[2], s_ready[2], p_ready[2], pv_done[2]
constexpr int kPfBarriers = 1 + 2 * kPfKSlots + 2 * kPfVSlots + 6 + 1;       // (+ q_empty)
constexpr int kPfSmemBytes = (2 + kPfKSlots + kPfVSlots) * kPfTileBytes + kPfBarriers * 8 + 16 + 1024 /* alignment slack */;
static_assert(kPfSmemBytes <= 227 * 1024, "exceeds the shared memory of one SM");

// two fp32 values in one 64-bit register: packed multiply-add and add (one instruction for two elements)
__device__ __forceinline__ unsigned long long f2_pack(float lo, float hi) {
    unsigned long long d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
    return d;
}
__device__ __forceinline__ void f2_unpack(unsigned long long v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ unsigned long long f2_fma(unsigned long long a, unsigned long long b, unsigned long long c) {
    unsigned long long d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ unsigned long long f2_add(unsigned long long a, unsigned long long b) {
    unsigned long long d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// For tests (mqa_set_test_withhold_copy): when non-zero, CTA 0 never starts one copy of the second stage of its first
// unit, so that a bounded wait runs out.
__device__ int g_test_withhold = 0;

// One unit of work: 128 positions of a pair of heads of one sequence.  Units are numbered ((n_tiles - 1 - position tile) *
// b + sequence) * head pairs + pair, the longest first; CTA c takes units c, c + grid, c + 2 grid, ... one after the other
// (a persistent kernel: barriers, tensor memory and the K/V rings are set up once, and the next unit's Q and first stages
// are fetched, and its first logits computed, while the softmax warps still write the unit before out).
struct PfItem {
    int seq, p0, head0, n_act, raw, L, n_kv;
    bool hilo;
    long long q_row0;
};
__device__ __forceinline__ PfItem pf_item(int item, const int32_t* __restrict__ start, int b, int h, int n, int m_max) {
    PfItem it;
    const int pairs = (h + 1) >> 1, n_tiles = (n + kPfRows - 1) / kPfRows;
    const int pair = item % pairs;
    it.seq = (item / pairs) % b;
    it.p0 = (n_tiles - 1 - item / (pairs * b)) * kPfRows;        // first query position of the tile
    it.head0 = 2 * pair;
    it.n_act = it.head0 + 1 < h ? 2 : 1;                         // heads of the unit (an odd head count leaves one alone)
    it.raw = start ? __ldg(start + it.seq) : 0;
    // rows of the memory the tile's last position sees (the last tile of a head may hold fewer than 128 positions: the
    // rows after them are computed on whatever the Q tile holds there and never stored); a memory that would pass m_max
    // is cut there
    it.L = it.raw + min(it.p0 + kPfRows, n);
    if (it.L > m_max) it.L = m_max;
    const bool empty = it.raw < 0 || it.L <= 0;                  // nothing to look at: zeros (like a bad lens)
    it.n_kv = empty ? 0 : (it.L + kPfRows - 1) / kPfRows;        // stages
    it.hilo = it.L < kSingleRoundingMinRows;
    it.q_row0 = ((long long)it.seq * h + it.head0) * n + it.p0;  // row of head 0's first query in [b h n, 128]
    return it;
}

__global__ void __launch_bounds__(kPfThreads, 1)
mqa_prefill_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                   const __grid_constant__ CUtensorMap map_v, const int32_t* __restrict__ start, float* __restrict__ O,
                   int32_t* __restrict__ status, int b, int h, int n, int m_max, int n_items) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);     // the 128-byte swizzle repeats every 1 KiB
    const uint32_t q_s = smem_addr(base);
    const uint32_t k_ring = q_s + 2 * kPfTileBytes, v_ring = k_ring + kPfKSlots * kPfTileBytes;
    const uint32_t bars = v_ring + kPfVSlots * kPfTileBytes;
    const uint32_t q_empty = bars + 8 * (kPfBarriers - 1);       // the unit's Q tiles have been read for the last time
    const uint32_t q_full = bars, k_full = bars + 8, k_empty = k_full + 8 * kPfKSlots, v_full = k_empty + 8 * kPfKSlots,
                   v_empty = v_full + 8 * kPfVSlots, s_ready = v_empty + 8 * kPfVSlots, p_ready = s_ready + 16,
                   pv_done = p_ready + 16;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base + (2 + kPfKSlots + kPfVSlots) * kPfTileBytes + kPfBarriers * 8);
    __shared__ int timed_out;

    if (threadIdx.x == 0) {
        prefetch_tensormap(&map_q); prefetch_tensormap(&map_k); prefetch_tensormap(&map_v);
        mbar_init(q_full, 1);
        mbar_init(q_empty, 1);
        for (int i = 0; i < kPfKSlots; ++i) { mbar_init(k_full + 8 * i, 1); mbar_init(k_empty + 8 * i, 1); }
        for (int i = 0; i < kPfVSlots; ++i) { mbar_init(v_full + 8 * i, 1); mbar_init(v_empty + 8 * i, 1); }
        for (int w = 0; w < 2; ++w) { mbar_init(s_ready + 8 * w, 1); mbar_init(p_ready + 8 * w, 4); mbar_init(pv_done + 8 * w, 1); }
        timed_out = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == kPfMmaWarp) {
        tmem_alloc(smem_addr(tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    grid_dependency_wait();              // Q, K, V and start may come from the kernel before
    grid_launch_dependents();
    // the units of this CTA: c, 2G - 1 - c, 2G + c, 4G - 1 - c, ... (G CTAs; the units come longest first, so taking them
    // forwards and backwards in turn evens the CTAs' totals out)
    auto pf_unit = [&](int round) -> int {
        const int G = (int)gridDim.x, c = (int)blockIdx.x;
        return round * G + ((round & 1) ? G - 1 - c : c);
    };
    if (start && threadIdx.x < 32) {
        // a start that is negative or leaves too little room is flagged once (its rows are zeros, or the memory is cut at m_max)
        bool bad = false;
        for (int i = blockIdx.x * 32 + threadIdx.x; i < b; i += gridDim.x * 32) bad = bad || start[i] < 0 || start[i] + n > m_max;
        if (bad && status) atomicOr(status, kStatusLenClamped);
    }

    if (warp >= 8) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kPfRegsOther));
    if (warp == kPfProducerWarp) {
        // =============================================================== TMA producer
        if (lane == 0) {
            bool ok = true;
            int g = 0, qi = 0;                                   // stages and units so far (they number the barriers' phases)
            int issued_k = 0, issued_v = 0, issued_q = 0;
            const bool withhold = blockIdx.x == 0 && *reinterpret_cast<volatile int*>(&g_test_withhold) != 0;
            for (int round = 0, item; (item = pf_unit(round)) < n_items && ok; ++round) {
                const PfItem it = pf_item(item, start, b, h, n, m_max);
                if (it.n_kv == 0) continue;
                if (qi > 0) ok = mbar_wait(q_empty, (qi - 1) & 1);            // the unit before has read its Q for the last time
                if (!ok) break;
                mbar_expect_tx(q_full, it.n_act * kPfTileBytes);
                for (int w = 0; w < it.n_act; ++w)
                    for (int half = 0; half < 2; ++half)
                        tma_load_2d(q_s + w * kPfTileBytes + half * kPfHalfBytes, &map_q, half * kBoxCols, (int)(it.q_row0 + (long long)w * n), q_full);
                issued_q = qi + 1;
                for (int j = 0; j < it.n_kv && ok; ++j) {
                    const int G = g + j;
                    const int y = it.seq * m_max + j * kPfRows;
                    const int ks = G % kPfKSlots, vs = G % kPfVSlots;
                    if (G >= kPfKSlots) ok = mbar_wait(k_empty + 8 * ks, ((G / kPfKSlots) - 1) & 1);
                    if (!ok) break;
                    mbar_expect_tx(k_full + 8 * ks, kPfTileBytes);
                    tma_load_2d(k_ring + ks * kPfTileBytes, &map_k, 0, y, k_full + 8 * ks);
                    tma_load_2d(k_ring + ks * kPfTileBytes + kPfHalfBytes, &map_k, kBoxCols, y, k_full + 8 * ks);
                    issued_k = G + 1;
                    if (G >= kPfVSlots) ok = mbar_wait(v_empty + 8 * vs, ((G / kPfVSlots) - 1) & 1);
                    if (!ok) break;
                    mbar_expect_tx(v_full + 8 * vs, kPfTileBytes);
                    tma_load_2d(v_ring + vs * kPfTileBytes, &map_v, 0, y, v_full + 8 * vs);
                    if (!(withhold && G == 1)) tma_load_2d(v_ring + vs * kPfTileBytes + kPfHalfBytes, &map_v, kBoxCols, y, v_full + 8 * vs);
                    issued_v = G + 1;
                }
                g += it.n_kv;
                ++qi;
            }
            if (!ok) {
                // a wait ran out: the copies already started are given a bounded wait each before the CTA may leave
                atomicExch(&timed_out, 1);
                if (issued_q > 0) mbar_wait(q_full, (issued_q - 1) & 1);
                for (int G = max(0, issued_k - kPfKSlots); G < issued_k; ++G) mbar_wait(k_full + 8 * (G % kPfKSlots), (G / kPfKSlots) & 1);
                for (int G = max(0, issued_v - kPfVSlots); G < issued_v; ++G) mbar_wait(v_full + 8 * (G % kPfVSlots), (G / kPfVSlots) & 1);
            }
        }
    } else if (warp == kPfMmaWarp) {
        // =============================================================== issuer of both products
        if (lane == 0) {
            constexpr uint32_t kIdescS = umma_idesc(128, 128, false, false);
            constexpr uint32_t kIdescO = umma_idesc(128, 128, false, true);
            bool ok = true;
            int g = 0, qi = 0, c_done[2] = {0, 0};               // stages, units, and stages of each head so far
            for (int round = 0, item; (item = pf_unit(round)) < n_items && ok; ++round) {
                const PfItem it = pf_item(item, start, b, h, n, m_max);
                if (it.n_kv == 0) continue;
                const int n_act = it.n_act, n_kv = it.n_kv;
                auto issue_s = [&](int w, int G) {              // S_w = Q_w K^T into its 128 columns
                    const uint32_t k_s = k_ring + (G % kPfKSlots) * kPfTileBytes, qw = q_s + w * kPfTileBytes;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {            // 8 k-steps of 16 columns; 4 per 64-column box
                        const uint32_t off = (ks >> 2) * kPfHalfBytes + (ks & 3) * 32;
                        umma_ss(tmem_base + w * 128, umma_desc(qw + off, 16, 1024), umma_desc(k_s + off, 16, 1024), kIdescS, ks ? 1u : 0u);
                    }
                    tc_commit(s_ready + 8 * w);
                };
                auto issue_pv = [&](int w, int G, bool first) {  // O_w += P_w V: P from TMEM (bf16 pairs: 8 columns per 16 rows of V)
                    const uint32_t v_s = v_ring + (G % kPfVSlots) * kPfTileBytes;
                    for (int part = 0; part < (it.hilo ? 2 : 1); ++part) {
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk)
                            umma_ts(tmem_base + 256 + w * 128, tmem_base + w * 128 + (kk >> 1) * 32 + part * 16 + (kk & 1) * 8,
                                    umma_desc(v_s + kk * 2048, kPfHalfBytes, 1024), kIdescO, (first && part == 0 && kk == 0) ? 0u : 1u);
                    }
                    tc_commit(pv_done + 8 * w);
                };
                ok = mbar_wait(q_full, qi & 1);
                if (ok) ok = mbar_wait(k_full + 8 * (g % kPfKSlots), (g / kPfKSlots) & 1);
                if (!ok) break;
                tc_fence_after();
                for (int w = 0; w < n_act; ++w) issue_s(w, g);
                tc_commit(k_empty + 8 * (g % kPfKSlots));
                if (n_kv == 1) tc_commit(q_empty);
                for (int j = 0; j < n_kv && ok; ++j) {
                    const bool more = j + 1 < n_kv;
                    const int G = g + j;
                    for (int w = 0; w < n_act && ok; ++w) {
                        ok = mbar_wait(p_ready + 8 * w, (c_done[w] + j) & 1);
                        if (ok && w == 0) ok = mbar_wait(v_full + 8 * (G % kPfVSlots), (G / kPfVSlots) & 1);
                        if (ok && w == 0 && more) ok = mbar_wait(k_full + 8 * ((G + 1) % kPfKSlots), ((G + 1) / kPfKSlots) & 1);
                        if (!ok) break;
                        tc_fence_after();
                        issue_pv(w, G, j == 0);
                        if (w == n_act - 1) tc_commit(v_empty + 8 * (G % kPfVSlots));
                        if (more) {
                            issue_s(w, G + 1);
                            if (w == n_act - 1) {
                                tc_commit(k_empty + 8 * ((G + 1) % kPfKSlots));
                                if (j + 2 == n_kv) tc_commit(q_empty);       // the unit's last logits are on their way
                            }
                        }
                    }
                }
                g += n_kv;
                ++qi;
                for (int w = 0; w < n_act; ++w) c_done[w] += n_kv;
            }
            if (!ok) atomicExch(&timed_out, 1);
        }
    }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kPfRegsSoftmax));
        // =============================================================== softmax warps: one thread per query row
        const int w = warp >> 2, quarter = warp & 3, r = quarter * 32 + lane;
        const uint32_t lane_base = tmem_base + ((uint32_t)(quarter * 32) << 16);
        const uint32_t s_t = lane_base + w * 128, o_t = lane_base + 256 + w * 128;
        bool ok = true;
        int g = 0, c_done = 0;                                   // stages of the CTA and of this head so far
        for (int round = 0, item; (item = pf_unit(round)) < n_items; ++round) {
            const PfItem it = pf_item(item, start, b, h, n, m_max);
            if (w >= it.n_act) { g += it.n_kv; continue; }       // (an odd head count: the unit has one head)
            const int p0 = it.p0, raw = it.raw;
            float* dst = O + (size_t)(it.q_row0 + (long long)w * n + r) * kHeadDim;
            const bool stored = p0 + r < n;                      // (a position of this head)
            if (it.n_kv == 0) {
                if (stored)
                    for (int i = 0; i < kHeadDim; i += 4) *reinterpret_cast<float4*>(dst + i) = make_float4(0.f, 0.f, 0.f, 0.f);
                continue;
            }
            const int lim_first = min(raw + p0 + 1, it.L);       // rows the tile's first position sees
            const int lim = min(raw + p0 + r + 1, it.L);         // rows this thread's position sees: >= 1
            float m = -INFINITY, l = 0.f;                        // reference maximum (log2 units), sum of weights
            for (int j = 0; j < it.n_kv; ++j) {
                const int k0 = j * kPfRows;
                if (ok) ok = mbar_wait(s_ready + 8 * w, (c_done + j) & 1);
                tc_fence_after();
                const bool diag = k0 + kPfRows > lim_first;           // some position of the tile cannot see all of this stage
                // ---- the row's 128 logits, read once and kept in registers.  The mask of Section 2.3 is applied
                // by index, as a select: what lies behind a masked logit is never used.
                uint32_t x[128];
                tmem_ld_cols<128>(s_t, x);
                tmem_wait_ld();
                if (diag) {
#pragma unroll
                    for (int i = 0; i < 128; ++i)
                        if (k0 + i >= lim) x[i] = 0xff800000u;        // -inf
                }
                float mx8[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) mx8[i] = fmaxf(__uint_as_float(x[2 * i]), __uint_as_float(x[2 * i + 1]));
#pragma unroll
                for (int i = 8; i < 64; ++i) mx8[i & 7] = max3(mx8[i & 7], __uint_as_float(x[2 * i]), __uint_as_float(x[2 * i + 1]));
                const float mx = max3(max3(mx8[0], mx8[1], mx8[2]), max3(mx8[3], mx8[4], mx8[5]), fmaxf(mx8[6], mx8[7])) * kLog2e;
                if (__any_sync(0xffffffffu, mx > m + kPfMaxLead)) {
                    const float m_new = fmaxf(m, mx);
                    if (j > 0) {
                        const float f = fast_exp2(m - m_new);         // (m is finite from the first stage on)
                        l *= f;
                        if (ok) ok = mbar_wait(pv_done + 8 * w, (c_done + j - 1) & 1);    // O holds the stages before this one
                        tc_fence_after();
#pragma unroll 1
                        for (int c = 0; c < 16; ++c) {
                            uint32_t y[8];
                            tmem_ld8(o_t + c * 8, y);
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 8; ++i) y[i] = __float_as_uint(__uint_as_float(y[i]) * f);
                            tmem_st8(o_t + c * 8, y);
                        }
                    }
                    m = m_new;
                }
                const unsigned long long neg_m2 = f2_pack(-m, -m), log2e2 = f2_pack(kLog2e, kLog2e);
                unsigned long long sum2[2] = {0ull, 0ull};
                if (it.hilo) {
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint32_t hi[16];
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            float a0, a1;
                            f2_unpack(f2_fma(f2_pack(__uint_as_float(x[c * 32 + 2 * i]), __uint_as_float(x[c * 32 + 2 * i + 1])), log2e2, neg_m2), a0, a1);
                            const float pa = fast_exp2(a0), pb = fast_exp2(a1);
                            sum2[i & 1] = f2_add(sum2[i & 1], f2_pack(pa, pb));
                            hi[i] = pack_bf16(pa, pb);
                            x[c * 32 + i] = pack_bf16(pa - bf16_lo(hi[i]), pb - bf16_hi(hi[i]));
                        }
                        tmem_st16(s_t + c * 32, hi);
                        tmem_st16(s_t + c * 32 + 16, *reinterpret_cast<uint32_t(*)[16]>(&x[c * 32]));
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint32_t hi[16];
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            float a0, a1;
                            f2_unpack(f2_fma(f2_pack(__uint_as_float(x[c * 32 + 2 * i]), __uint_as_float(x[c * 32 + 2 * i + 1])), log2e2, neg_m2), a0, a1);
                            const float pa = fast_exp2(a0), pb = fast_exp2(a1);
                            sum2[i & 1] = f2_add(sum2[i & 1], f2_pack(pa, pb));
                            hi[i] = pack_bf16(pa, pb);
                        }
                        tmem_st16(s_t + c * 32, hi);
                    }
                }
                {
                    float s0, s1;
                    f2_unpack(f2_add(sum2[0], sum2[1]), s0, s1);
                    l += s0 + s1;
                }
                tmem_wait_st();
                tc_fence_before();
                if (w == 0 && j == it.n_kv - 1 && it.L < k0 + kPfRows) {
                    // the last stage runs past the memory: the tensor core would multiply the zero weights with
                    // whatever lies there (NaN * 0 = NaN), so those V rows are cleared first
                    const int vs = (g + j) % kPfVSlots;
                    if (ok) ok = mbar_wait(v_full + 8 * vs, ((g + j) / kPfVSlots) & 1);
                    const uint32_t v_s = v_ring + vs * kPfTileBytes;
                    const int first = it.L - k0;
                    for (int i = r; i < (kPfRows - first) * 16; i += 128) {
                        const int vrow = first + (i >> 4), ch = i & 15;
                        const uint32_t a = v_s + (ch >> 3) * kPfHalfBytes + vrow * 128 + ((ch & 7) << 4);
                        asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0u) : "memory");
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(p_ready + 8 * w);
            }
            // ---- the row of O, divided by the sum of its weights
            if (ok) ok = mbar_wait(pv_done + 8 * w, (c_done + it.n_kv - 1) & 1);
            tc_fence_after();
            const float inv = 1.f / l;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t y[32];
                tmem_ld32(o_t + c * 32, y);
                tmem_wait_ld();
                if (stored) {
#pragma unroll
                    for (int i = 0; i < 32; i += 4)
                        *reinterpret_cast<float4*>(dst + c * 32 + i) =
                            make_float4(__uint_as_float(y[i]) * inv, __uint_as_float(y[i + 1]) * inv, __uint_as_float(y[i + 2]) * inv,
                                        __uint_as_float(y[i + 3]) * inv);
                }
            }
            tc_fence_before();                                   // (the next unit's first product overwrites O once its weights are in)
            g += it.n_kv;
            c_done += it.n_kv;
        }
        if (!ok) atomicExch(&timed_out, 1);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kPfMmaWarp) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
    if (threadIdx.x == 0 && timed_out && status) atomicOr(status, kStatusPipelineTimeout);
}

}  // namespace mqa
