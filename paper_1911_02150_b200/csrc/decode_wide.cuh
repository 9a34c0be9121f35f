// Multi-query decoding step for MANY query rows per sequence (33 and more: many heads, or beams x heads over one shared
// memory, Section 4.2; 128 rows per CTA, more as grid.y row tiles over the same cache rows) -- the same three lines of Section 3 (logits = einsum(bhk,bmk->bhm), softmax over the valid
// prefix, o = einsum(bhm,bmv->bhv)), with the query rows as the ROWS of the tensor-core tiles.
//
// The streaming kernel (decode_umma.cuh) puts the cache rows on the TMEM lanes and the heads on the columns, which is
// right for a few heads (N = 16 .. 32) but makes the softmax a cross-thread affair; from 64 query rows on that kernel
// is bound by its softmax warps, not by HBM.  Here a CTA holds all the sequence's query rows as ONE 128-row Q tile
// (rows past h belong to the next sequence or read as zero: computed, never stored) and walks a fixed split of the
// sequence's cache rows in stages of 128:
//     S   = Q K_j^T        tcgen05.mma, M = 128 query rows (TMEM lanes), N = 128 cache rows, fp32 in TMEM
//     P   = exp2(S log2e - m)   one thread per query row: the row's maximum and sum need no other thread
//     O  += P V_j          tcgen05.mma with A = P read from TMEM (bf16 pairs written over S), B = V_j (MN-major)
// The two softmax warpgroups take the stages in turn (warpgroup w: stages w, w + 2, ...), each with an S buffer, an
// O accumulator, reference maxima and sums of its own -- two partial softmaxes over interleaved rows of the cache,
// merged exactly at the end (the same recombination as between splits) -- so the logits of a stage are computed and
// its weights formed while the other warpgroup's stage is multiplied with V.  TMEM: S_0, S_1, O_0, O_1 (512 columns).
// A CTA writes o itself when the sequence has one split, else a piece (maximum, sum, unnormalised rows) for the
// second-pass kernel (combine.cuh).  Valid prefix: rows >= lens are never fetched except in a split's last stage,
// where they are masked by index (select) and their V rows cleared in shared memory.
//
// Roles: warps 0-3 and 4-7 the two softmax warpgroups, warp 8 TMA producer, warp 9 MMA issuer (warps 10, 11 only
// complete the third warpgroup, which hands most of its registers to the other two).  Every wait is bounded.
#pragma once
#include "prefill.cuh"

namespace mqa {

constexpr int kWideRows = 128;                                 // query rows of the tile = cache rows per stage
constexpr int kWideKSlots = 3, kWideVSlots = 3;
constexpr int kWideThreads = 12 * 32;
constexpr int kWideProducerWarp = 8, kWideMmaWarp = 9;
// barriers: q_full, k_full/k_empty, v_full/v_empty per slot, s_ready[2], p_ready[2], pv_done[2]
constexpr int kWideBarriers = 1 + 2 * kWideKSlots + 2 * kWideVSlots + 6;
constexpr int kWideSmemBytes = (1 + kWideKSlots + kWideVSlots) * kPfTileBytes + kWideBarriers * 8 + 16 + 1024 /* alignment slack */;
static_assert(kWideSmemBytes + 1024 + 16 /* static */ <= 227 * 1024, "exceeds the shared memory of one SM");

// grid: x = sequence * n_splits + split, y = tile of 128 query rows.  part_ml [b * h][n_splits], part_acc [b * h][n_splits][128] (combine.cuh).
__global__ void __launch_bounds__(kWideThreads, 1)
mqa_decode_wide_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                       const __grid_constant__ CUtensorMap map_v, const int32_t* __restrict__ lens, float* __restrict__ o,
                       float2* __restrict__ part_ml, float* __restrict__ part_acc, int32_t* __restrict__ status, int h,
                       int m_max, int chunk_rows, int n_splits, int len_bias, const FusedArgs fa, int32_t* __restrict__ lens_advance,
                       int withhold) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int seq = blockIdx.x / n_splits, split = blockIdx.x % n_splits;
    const int row0 = blockIdx.y * kWideRows;                   // this CTA's first query row of the sequence (more than 128: grid.y tiles)

    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);     // the 128-byte swizzle repeats every 1 KiB
    const uint32_t q_s = smem_addr(base);
    const uint32_t k_ring = q_s + kPfTileBytes, v_ring = k_ring + kWideKSlots * kPfTileBytes;
    const uint32_t bars = v_ring + kWideVSlots * kPfTileBytes;
    const uint32_t q_full = bars, k_full = bars + 8, k_empty = k_full + 8 * kWideKSlots, v_full = k_empty + 8 * kWideKSlots,
                   v_empty = v_full + 8 * kWideVSlots, s_ready = v_empty + 8 * kWideVSlots, p_ready = s_ready + 16,
                   pv_done = p_ready + 16;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base + (1 + kWideKSlots + kWideVSlots) * kPfTileBytes + kWideBarriers * 8);
    __shared__ int timed_out;
    __shared__ float2 ex_ml[kWideRows];                       // (maximum, sum) of warpgroup 1's rows, for the merge at the end

    if (threadIdx.x == 0) {
        prefetch_tensormap(&map_q); prefetch_tensormap(&map_k); prefetch_tensormap(&map_v);
        mbar_init(q_full, 1);
        for (int i = 0; i < kWideKSlots; ++i) { mbar_init(k_full + 8 * i, 1); mbar_init(k_empty + 8 * i, 1); }
        for (int i = 0; i < kWideVSlots; ++i) { mbar_init(v_full + 8 * i, 1); mbar_init(v_empty + 8 * i, 1); }
        for (int w = 0; w < 2; ++w) { mbar_init(s_ready + 8 * w, 1); mbar_init(p_ready + 8 * w, 4); mbar_init(pv_done + 8 * w, 1); }
        timed_out = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == kWideMmaWarp) {
        tmem_alloc(smem_addr(tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    grid_dependency_wait();              // q, lens and the newest cache row may come from the kernel before
    grid_launch_dependents();
    // The append-and-attend step (fa.k_new given): the CTA whose rows hold row lens[seq] writes the new key/value row
    // there before it fetches it (its producer warp: store, proxy fence, then the copies), every split attends over one
    // row more, and lens moves on at the end -- here when the sequence has one split (lens_advance given), else in the
    // second-pass kernel.
    const int raw = __ldcg(lens + seq);
    const bool appended = fa.k_new != nullptr && raw >= 0 && raw < m_max;
    if (fa.k_new != nullptr && !appended && split == 0 && blockIdx.y == 0 && threadIdx.x == 0 && status)
        atomicOr(status, raw < 0 ? kStatusAppendNegative : kStatusAppendFull);
    const int L = clamp_len(appended ? raw + 1 : biased_len(raw, m_max, len_bias), m_max, (split == 0 && blockIdx.y == 0 && threadIdx.x == 0) ? status : nullptr);
    const int r0 = split * chunk_rows, r1 = min(r0 + chunk_rows, L);           // this CTA's rows of the sequence's cache
    const int n_kv = r1 > r0 ? (r1 - r0 + kWideRows - 1) / kWideRows : 0;      // stages
    const bool hilo = L < kSingleRoundingMinRows;

    if (warp >= 8) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kPfRegsOther));
        if (warp == kWideProducerWarp) {
            // =========================================================== TMA producer
            if (appended && raw >= split * chunk_rows && raw < (split + 1) * chunk_rows) {
                const uint4 piece = (lane < 16 ? fa.k_new : fa.v_new)[(size_t)seq * (kRowBytes / 16) + (lane & 15)];
                const size_t at = ((size_t)seq * m_max + raw) * (kRowBytes / 16) + (lane & 15);
                if (lane < 16) fa.K[at] = piece; else fa.V[at] = piece;
                asm volatile("fence.proxy.async;" ::: "memory");    // the copy engine must see the row
                __syncwarp();
            }
            if (lane == 0 && n_kv > 0) {
                bool ok = true;
                mbar_expect_tx(q_full, kPfTileBytes);
                for (int half = 0; half < 2; ++half)
                    tma_load_2d(q_s + half * kPfHalfBytes, &map_q, half * kBoxCols, seq * h + row0, q_full);
                const uint64_t policy = l2_stream_policy(true);     // the cache is read once per step
                int issued_k = 0, issued_v = 0;
                for (int j = 0; j < n_kv && ok; ++j) {
                    const int y = seq * m_max + r0 + j * kWideRows;
                    const int ks = j % kWideKSlots, vs = j % kWideVSlots;
                    if (j >= kWideKSlots) ok = mbar_wait(k_empty + 8 * ks, ((j / kWideKSlots) - 1) & 1);
                    if (!ok) break;
                    mbar_expect_tx(k_full + 8 * ks, kPfTileBytes);
                    tma_load_2d_hint(k_ring + ks * kPfTileBytes, &map_k, 0, y, k_full + 8 * ks, policy);
                    tma_load_2d_hint(k_ring + ks * kPfTileBytes + kPfHalfBytes, &map_k, kBoxCols, y, k_full + 8 * ks, policy);
                    issued_k = j + 1;
                    if (j >= kWideVSlots) ok = mbar_wait(v_empty + 8 * vs, ((j / kWideVSlots) - 1) & 1);
                    if (!ok) break;
                    mbar_expect_tx(v_full + 8 * vs, kPfTileBytes);
                    tma_load_2d_hint(v_ring + vs * kPfTileBytes, &map_v, 0, y, v_full + 8 * vs, policy);
                    // (for tests: one copy of the first CTA's second stage is never started, so that a wait runs out)
                    if (!(withhold && blockIdx.x == 0 && blockIdx.y == 0 && j == 1))
                        tma_load_2d_hint(v_ring + vs * kPfTileBytes + kPfHalfBytes, &map_v, kBoxCols, y, v_full + 8 * vs, policy);
                    issued_v = j + 1;
                }
                if (!ok) {
                    // a wait ran out: the copies already started are given a bounded wait each before the CTA may leave
                    atomicExch(&timed_out, 1);
                    mbar_wait(q_full, 0);
                    for (int j = max(0, issued_k - kWideKSlots); j < issued_k; ++j) mbar_wait(k_full + 8 * (j % kWideKSlots), (j / kWideKSlots) & 1);
                    for (int j = max(0, issued_v - kWideVSlots); j < issued_v; ++j) mbar_wait(v_full + 8 * (j % kWideVSlots), (j / kWideVSlots) & 1);
                }
            }
        } else if (warp == kWideMmaWarp) {
            // =========================================================== issuer of both products
            if (lane == 0 && n_kv > 0) {
                constexpr uint32_t kIdescS = umma_idesc(128, 128, false, false);
                constexpr uint32_t kIdescO = umma_idesc(128, 128, false, true);
                bool ok = mbar_wait(q_full, 0);
                auto issue_s = [&](int j) {                     // S = Q K_j^T into the buffer of warpgroup j mod 2
                    const uint32_t k_s = k_ring + (j % kWideKSlots) * kPfTileBytes;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {            // 8 k-steps of 16 columns; 4 per 64-column box
                        const uint32_t off = (ks >> 2) * kPfHalfBytes + (ks & 3) * 32;
                        umma_ss(tmem_base + (j & 1) * 128, umma_desc(q_s + off, 16, 1024), umma_desc(k_s + off, 16, 1024), kIdescS, ks ? 1u : 0u);
                    }
                    tc_commit(s_ready + 8 * (j & 1));
                    tc_commit(k_empty + 8 * (j % kWideKSlots));
                };
                auto issue_pv = [&](int j) {                    // O_w += P V_j: P from TMEM (bf16 pairs: 8 columns per 16 rows of V)
                    const uint32_t v_s = v_ring + (j % kWideVSlots) * kPfTileBytes;
                    const int w = j & 1;
                    for (int part = 0; part < (hilo ? 2 : 1); ++part) {
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk)
                            umma_ts(tmem_base + 256 + w * 128, tmem_base + w * 128 + part * 64 + kk * 8,
                                    umma_desc(v_s + kk * 2048, kPfHalfBytes, 1024), kIdescO, (j < 2 && part == 0 && kk == 0) ? 0u : 1u);
                    }
                    tc_commit(pv_done + 8 * w);
                    tc_commit(v_empty + 8 * (j % kWideVSlots));
                };
                for (int j = 0; j < 2 && j < n_kv && ok; ++j) {
                    ok = mbar_wait(k_full + 8 * j, 0);
                    if (!ok) break;
                    tc_fence_after();
                    issue_s(j);
                }
                for (int j = 0; j < n_kv && ok; ++j) {
                    ok = mbar_wait(p_ready + 8 * (j & 1), (j >> 1) & 1);
                    if (ok) ok = mbar_wait(v_full + 8 * (j % kWideVSlots), (j / kWideVSlots) & 1);
                    if (ok && j + 2 < n_kv) ok = mbar_wait(k_full + 8 * ((j + 2) % kWideKSlots), ((j + 2) / kWideKSlots) & 1);
                    if (!ok) break;
                    tc_fence_after();
                    issue_pv(j);
                    if (j + 2 < n_kv) issue_s(j + 2);           // the buffer these weights were in takes the logits of stage j + 2
                }
                if (!ok) atomicExch(&timed_out, 1);
            }
        }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kPfRegsSoftmax));
        // =============================================================== softmax warpgroups: one thread per query row
        const int w = warp >> 2, quarter = warp & 3, r = quarter * 32 + lane;
        const uint32_t lane_base = tmem_base + ((uint32_t)(quarter * 32) << 16);
        const uint32_t s_t = lane_base + w * 128, o_t = lane_base + 256 + w * 128;
        float m = -INFINITY, l = 0.f;                                 // reference maximum (log2 units), sum of weights
        bool ok = true;
        int last_phase = -1;                                          // phase of this warpgroup's last product
        for (int j = w; j < n_kv; j += 2) {
            const int ph = j >> 1;
            const int valid = r1 - (r0 + j * kWideRows);              // rows of the stage inside this split's prefix (> 0)
            if (ok) ok = mbar_wait(s_ready + 8 * w, ph & 1);
            tc_fence_after();
            // ---- the row's 128 logits, read once and kept in registers; rows past the prefix masked by index (a select)
            uint32_t x[128];
            tmem_ld_cols<128>(s_t, x);
            tmem_wait_ld();
            if (valid < kWideRows) {
#pragma unroll
                for (int i = 0; i < 128; ++i)
                    if (i >= valid) x[i] = 0xff800000u;               // -inf
            }
            float mx8[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) mx8[i] = fmaxf(__uint_as_float(x[2 * i]), __uint_as_float(x[2 * i + 1]));
#pragma unroll
            for (int i = 8; i < 64; ++i) mx8[i & 7] = max3(mx8[i & 7], __uint_as_float(x[2 * i]), __uint_as_float(x[2 * i + 1]));
            const float mx = max3(max3(mx8[0], mx8[1], mx8[2]), max3(mx8[3], mx8[4], mx8[5]), fmaxf(mx8[6], mx8[7])) * kLog2e;
            if (__any_sync(0xffffffffu, mx > m + kPfMaxLead)) {
                // ---- a row of this warp leads its reference by too much: every row of the warp moves its reference
                // to its largest logit so far and rescales its sum and its row of O
                const float m_new = fmaxf(m, mx);
                if (ph > 0) {
                    const float f = fast_exp2(m - m_new);             // (m is finite from the warpgroup's first stage on)
                    l *= f;
                    if (ok) ok = mbar_wait(pv_done + 8 * w, (ph - 1) & 1);   // O holds the warpgroup's stages before this one
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
            // ---- P = exp2(S log2e - m) as bf16 pairs over the first 64 columns of S (hi) and, for a short prefix, their
            // remainders over the other 64 (lo)
            const unsigned long long neg_m2 = f2_pack(-m, -m), log2e2 = f2_pack(kLog2e, kLog2e);
            unsigned long long sum2[2] = {0ull, 0ull};
            if (hilo) {
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
                    tmem_st16(s_t + c * 16, hi);
                }
#pragma unroll
                for (int c = 0; c < 4; ++c) tmem_st16(s_t + 64 + c * 16, *reinterpret_cast<uint32_t(*)[16]>(&x[c * 32]));
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
                    tmem_st16(s_t + c * 16, hi);
                }
            }
            {
                float s0, s1;
                f2_unpack(f2_add(sum2[0], sum2[1]), s0, s1);
                l += s0 + s1;
            }
            tmem_wait_st();
            tc_fence_before();
            if (valid < kWideRows) {
                // the stage runs past the prefix: the tensor core would multiply the zero weights with whatever lies
                // there (NaN * 0 = NaN), so those V rows are cleared first
                const int vs = j % kWideVSlots;
                if (ok) ok = mbar_wait(v_full + 8 * vs, (j / kWideVSlots) & 1);
                const uint32_t v_s = v_ring + vs * kPfTileBytes;
                for (int i = r; i < (kWideRows - valid) * 16; i += 128) {
                    const int vrow = valid + (i >> 4), ch = i & 15;
                    const uint32_t a = v_s + (ch >> 3) * kPfHalfBytes + vrow * 128 + ((ch & 7) << 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0u) : "memory");
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(p_ready + 8 * w);
            last_phase = ph;
        }
        if (last_phase >= 0 && ok) ok = mbar_wait(pv_done + 8 * w, last_phase & 1);
        tc_fence_after();
        // ---- the two warpgroups' partial results become one: warpgroup 1 leaves (maximum, sum) and its rows of O in
        // shared memory (the K ring: every S product has completed by now), warpgroup 0 merges and writes out
        const uint32_t ex_o = k_ring + r * 512;                                        // [128][128] fp32, 16-byte pieces swizzled by row
        if (w == 1) {
            if (n_kv > 0) {
                ex_ml[r] = make_float2(m, l);
                if (last_phase >= 0) {
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");       // (the ring was the copy engine's and the tensor core's)
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint32_t y[32];
                        tmem_ld32(o_t + c * 32, y);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; i += 4)
                            asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(ex_o + ((((c * 8 + (i >> 2)) ^ (r & 31)) << 4))),
                                         "r"(y[i]), "r"(y[i + 1]), "r"(y[i + 2]), "r"(y[i + 3]) : "memory");
                    }
                }
            }
            named_barrier_arrive(1, 256);
        } else {
            named_barrier(1, 256);
            // (the loads from tensor memory below are warp-wide instructions: every lane executes them, whether or not
            // its row is one of the sequence's h query rows)
            const bool stored = row0 + r < h;
            const size_t unit = (size_t)seq * h + (stored ? row0 + r : 0);
            if (n_kv == 0) {
                // nothing of this split lies inside the prefix: zeros (one split, written below) or an empty piece
                if (stored && n_splits > 1) part_ml[unit * n_splits + split] = make_float2(-INFINITY, 0.f);
            } else {
                const float2 other = ex_ml[r];
                const bool two = other.x != -INFINITY;                                 // warpgroup 1 had a stage
                const float top = fmaxf(m, other.x);
                const float f0 = fast_exp2(m - top), f1 = two ? fast_exp2(other.x - top) : 0.f;
                const float tot = f0 * l + f1 * other.y;
                const float scale = n_splits == 1 ? 1.f / tot : 1.f;
                const float g0 = f0 * scale, g1 = f1 * scale;
                // the merged row goes back to shared memory, in place of warpgroup 1's: a thread's row is 512 bytes, and
                // stored from here it would leave as 32 separate 16-byte pieces per instruction (measured: 4.7 us for the
                // CTA's 64 KB); all eight warps then copy whole rows out, 512 contiguous bytes per instruction
                float4* my_row = reinterpret_cast<float4*>(base + kPfTileBytes + r * 512);   // (plain accesses: the eight loads of a
                                                                                            // block go out together, ahead of its stores)
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t y[32];
                    tmem_ld32(o_t + c * 32, y);
                    float4 u[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) u[i] = two ? my_row[(c * 8 + i) ^ (r & 31)] : make_float4(0.f, 0.f, 0.f, 0.f);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        float4 v;
                        v.x = fmaf(u[i].x, g1, __uint_as_float(y[4 * i]) * g0);
                        v.y = fmaf(u[i].y, g1, __uint_as_float(y[4 * i + 1]) * g0);
                        v.z = fmaf(u[i].z, g1, __uint_as_float(y[4 * i + 2]) * g0);
                        v.w = fmaf(u[i].w, g1, __uint_as_float(y[4 * i + 3]) * g0);
                        my_row[(c * 8 + i) ^ (r & 31)] = v;
                    }
                }
                if (stored && n_splits > 1) part_ml[unit * n_splits + split] = make_float2(top, tot);
            }
        }
        // ---- all eight warps: the CTA's rows from shared memory to o (one split) or to its piece
        named_barrier(2, 256);
        if (n_kv > 0 || n_splits == 1) {
            for (int item = threadIdx.x; item < kWideRows * 32; item += 256) {
                const int row = item >> 5, c16 = item & 31;                             // (a warp: one row, its 32 pieces of 16 bytes)
                if (row0 + row >= h) break;
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                if (n_kv > 0) v = reinterpret_cast<const float4*>(base + kPfTileBytes + row * 512)[c16 ^ (row & 31)];
                const size_t unit = (size_t)seq * h + row0 + row;
                float* dst = n_splits == 1 ? o + unit * kHeadDim : part_acc + (unit * n_splits + split) * kHeadDim;
                reinterpret_cast<float4*>(dst)[c16] = v;
            }
        }
        if (!ok) atomicExch(&timed_out, 1);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kWideMmaWarp) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
    if (threadIdx.x == 0 && timed_out && status) atomicOr(status, kStatusPipelineTimeout);
    // (one split: lens is this CTA's to move on -- with several row tiles, the sequence's other CTAs read it too, so then the
    // host leaves it to a kernel of its own)
    if (lens_advance && appended && n_splits == 1 && threadIdx.x == 0) lens_advance[seq] = raw + 1;
}

}  // namespace mqa
