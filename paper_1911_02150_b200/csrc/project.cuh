// The projections either side of the multi-query step (Section 3, MultiquerySelfAttentionIncremental):
//
//     q     = einsum("bd,hdk->bhk", x, P_q)     k_new = einsum("bd,dk->bk", x, P_k)     v_new = einsum("bd,dv->bv", x, P_v)
//     y     = einsum("bhv,hdv->bd", o, P_o)
//
// as bf16 tensor-core products with fp32 accumulation (tcgen05, accumulators in TMEM).  A decoding
// step has few rows (b sequences) and large weights, so the weights are the M operand and the
// batch is N ("swap A and B"): a CTA streams a 128-wide slab of a weight matrix through shared
// memory with TMA, once, and multiplies it with the batch's activations:
//
//   project_in_kernel    slab s < h: P_q[s] = [d rows x 128]; s = h: P_k; s = h + 1: P_v  (each [d x 128], d contiguous
//                        rows of 256 bytes -- the layout of a 128-column cache, fetched the same way)
//                        Out^T[128 features x NB] = sum over d in chunks of 128:  W_chunk^T (MN-major A) * x_chunk^T (K-major B)
//   project_out_kernel   CTA (d tile j, head group g): Y^T[128 x NB] = sum over the group's heads:
//                        P_o[head][128 d-rows of tile j x 128] (K-major A) * o[:, head, :]^T (K-major B, converted
//                        from fp32 to bf16 by the CTA); the head groups of a tile are one thread-block cluster and
//                        add their sums up through distributed shared memory, in a fixed order (no float atomics)
//
// NB = batch columns of a tile (the batch rounded up to 16, 32, 64 or 128; larger batches take
// several tiles of 128).  Every wait is bounded (mbar_wait); TMEM is freed on every path.
#pragma once
#include <cuda_bf16.h>

#include "decode_umma.cuh"

namespace mqa {

constexpr int kProjThreads = 6 * 32;           // warps 0-3: convert / read out, warp 4: TMA, warp 5: MMA issue
constexpr int kProjChunkBytes = 128 * 256;     // 128 rows x 128 bf16 of a weight matrix: 32 KiB, two 64-column boxes
constexpr int kProjMaxGroups = 16;             // project_out: head groups of a tile = CTAs of one cluster (16: the
                                               // non-portable cluster size, which the B200 offers; two heads per CTA at h = 32)

template <int NB>
struct ProjCfg {
    static_assert(NB == 16 || NB == 32 || NB == 64 || NB == 128, "batch columns of a tile");
    static constexpr int kActBytes = NB * 256;                 // NB rows x 128 bf16, two 64-column boxes
    static constexpr int kStages = NB == 128 ? 3 : 4;
    static constexpr int kStageBytes = kProjChunkBytes + kActBytes;
    static constexpr int kSmemBytes = kStages * kStageBytes + 256 /* barriers */ + 1024 /* alignment slack */;
    static constexpr int kTmemCols = NB < 32 ? 32 : NB;
    static_assert(kSmemBytes <= 227 * 1024, "exceeds the shared memory of one SM");
};

// NB consecutive fp32 columns of this thread's TMEM lane, in pieces of at most 32
template <int NB>
__device__ __forceinline__ void tmem_ld_row(uint32_t taddr, uint32_t (&r)[NB]) {
    constexpr int CH = NB < 32 ? NB : 32;
#pragma unroll
    for (int c = 0; c < NB / CH; ++c) {
        uint32_t part[CH];
        tmem_ld_cols<CH>(taddr + c * CH, part);
#pragma unroll
        for (int i = 0; i < CH; ++i) r[c * CH + i] = part[i];
    }
    tmem_wait_ld();
}

template <int NB>
__global__ void __launch_bounds__(kProjThreads, 1)
project_in_kernel(const __grid_constant__ CUtensorMap map_pq, const __grid_constant__ CUtensorMap map_pk,
                  const __grid_constant__ CUtensorMap map_pv, const __grid_constant__ CUtensorMap map_x,
                  __nv_bfloat16* __restrict__ q, __nv_bfloat16* __restrict__ k_new, __nv_bfloat16* __restrict__ v_new,
                  int32_t* __restrict__ status, int b, int h, int d) {
    using Cfg = ProjCfg<NB>;
    constexpr int S = Cfg::kStages;
    const int slab = blockIdx.x, row0 = blockIdx.y * 128;          // weight slab; first batch row of this tile
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_chunks = d / 128;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* stages = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);
    const uint32_t stages_s = smem_addr(stages);
    const uint32_t full_s = stages_s + S * Cfg::kStageBytes, empty_s = full_s + S * 8, done_s = empty_s + S * 8;
    __shared__ uint32_t tmem_slot;
    __shared__ int timed_out, issued;

    // The weights do not depend on the kernel before this one, x does: a stage's barrier takes two arrivals, one with
    // the weight chunk's bytes and one with the x chunk's, and the weight copies of the first stages start before the wait.
    const CUtensorMap* wmap = slab < h ? &map_pq : (slab == h ? &map_pk : &map_pv);
    const int wrow0 = slab < h ? slab * d : 0;
    auto issue_weights = [&](int c) {
        const uint32_t bar = full_s + (c % S) * 8, w_s = stages_s + (c % S) * Cfg::kStageBytes;
        mbar_expect_tx(bar, kProjChunkBytes);
        tma_load_2d(w_s, wmap, 0, wrow0 + c * 128, bar);
        tma_load_2d(w_s + kProjChunkBytes / 2, wmap, kBoxCols, wrow0 + c * 128, bar);
    };
    auto issue_x = [&](int c) {
        const uint32_t bar = full_s + (c % S) * 8, x_s = stages_s + (c % S) * Cfg::kStageBytes + kProjChunkBytes;
        mbar_expect_tx(bar, Cfg::kActBytes);
        tma_load_2d(x_s, &map_x, c * 128, row0, bar);                         // rows past b read as zero
        tma_load_2d(x_s + Cfg::kActBytes / 2, &map_x, c * 128 + kBoxCols, row0, bar);
        issued = c + 1;
    };
    if (warp == 4 && lane == 0) {                                  // by the thread that issues the copies
        prefetch_tensormap(&map_pq); prefetch_tensormap(&map_pk); prefetch_tensormap(&map_pv); prefetch_tensormap(&map_x);
        timed_out = 0;
        issued = 0;
        for (int s = 0; s < S; ++s) { mbar_init(full_s + s * 8, 2); mbar_init(empty_s + s * 8, 1); }
        mbar_init(done_s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        for (int c = 0; c < n_chunks && c < S; ++c) issue_weights(c);
    }
    if (warp == 5) { tmem_alloc(smem_addr(&tmem_slot), Cfg::kTmemCols); tmem_relinquish(); }
    grid_dependency_wait();          // x may come from the kernel before this one
    grid_launch_dependents();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;

    if (warp == 4) {
        if (lane == 0) {
            bool ok = true;
            for (int c = 0; c < n_chunks && ok; ++c) {
                if (c >= S) {
                    ok = mbar_wait(empty_s + (c % S) * 8, ((c / S) - 1) & 1);
                    if (!ok) break;
                    issue_weights(c);
                }
                issue_x(c);
            }
            if (!ok) atomicExch(&timed_out, 1);
        }
    } else if (warp == 5) {
        if (lane == 0) {
            constexpr uint32_t kIdesc = umma_idesc(128, NB, true, false);
            bool ok = true;
            for (int c = 0; c < n_chunks; ++c) {
                const int st = c % S;
                if (ok) ok = mbar_wait(full_s + st * 8, (c / S) & 1);
                tc_fence_after();
                if (ok) {
                    const uint32_t w_s = stages_s + st * Cfg::kStageBytes, x_s = w_s + kProjChunkBytes;
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {                         // 8 k-steps of 16 rows of the weight chunk
                        const uint64_t a = umma_desc(w_s + kk * 2048, kProjChunkBytes / 2, 1024);
                        const uint64_t bd = umma_desc(x_s + (kk >> 2) * (Cfg::kActBytes / 2) + (kk & 3) * 32, 16, 1024);
                        umma_ss(tmem, a, bd, kIdesc, (c > 0 || kk > 0) ? 1u : 0u);
                    }
                }
                tc_commit(empty_s + st * 8);
            }
            tc_commit(done_s);
            if (!ok) atomicExch(&timed_out, 1);
        }
    } else {
        // read-out: thread t = feature t of the slab, one TMEM lane; a column is a batch row
        const int t = warp * 32 + lane;
        const bool ok = mbar_wait(done_s, 0);
        tc_fence_after();
        if (ok) {
            uint32_t acc[NB];
            tmem_ld_row<NB>(tmem + ((uint32_t)(warp * 32) << 16), acc);
            __nv_bfloat16* out = slab < h ? q + (size_t)slab * 128 + t : (slab == h ? k_new : v_new) + t;
            const size_t stride = slab < h ? (size_t)h * 128 : 128;
#pragma unroll
            for (int i = 0; i < NB; ++i)
                if (row0 + i < b) out[(size_t)(row0 + i) * stride] = __float2bfloat16_rn(__uint_as_float(acc[i]));
        } else {
            atomicExch(&timed_out, 1);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (timed_out && threadIdx.x == 0) {
        // before the CTA leaves: the last copy started into each stage has to land
        for (int s = 0; s < S && s < issued; ++s) mbar_wait(full_s + s * 8, ((issued - 1 - s) / S) & 1);
        if (status) atomicOr(status, kStatusPipelineTimeout);
    }
    __syncthreads();
    if (warp == 5) { tc_fence_after(); tmem_dealloc(tmem, Cfg::kTmemCols); }
}

// The head groups of one (d tile, batch tile) form one thread-block cluster (gridDim.y CTAs, at most 16): each CTA
// accumulates Y^T over its heads in TMEM, leaves it in its shared memory, and after a cluster barrier every CTA adds up,
// in group order, the batch rows that fall to it (row n to CTA n mod cluster size) out of all the CTAs' shared memory
// and stores them to y.  No partial sums pass through global memory and no float atomics are used.
template <int NB>
__global__ void __launch_bounds__(kProjThreads, 1)
project_out_kernel(const __grid_constant__ CUtensorMap map_po, const float* __restrict__ o, float* __restrict__ y,
                   int32_t* __restrict__ status, int b, int h, int d, int heads_per_cta) {
    using Cfg = ProjCfg<NB>;
    constexpr int S = 2;                                           // ring of two stages: a head's weights and its o tile
    const int tile = blockIdx.x, group = blockIdx.y, row0 = blockIdx.z * 128;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int head0 = group * heads_per_cta;
    const int n_heads = max(0, min(heads_per_cta, h - head0));

    extern __shared__ uint8_t smem_raw[];
    uint8_t* stages = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);
    const uint32_t stages_s = smem_addr(stages);
    const uint32_t w_full = stages_s + S * Cfg::kStageBytes, o_full = w_full + S * 8, empty_s = o_full + S * 8, done_s = empty_s + S * 8;
    __shared__ uint32_t tmem_slot;
    __shared__ int timed_out, issued;

    if (warp == 4 && lane == 0) {                                  // by the thread that issues the copies
        prefetch_tensormap(&map_po);
        timed_out = 0;
        issued = 0;
        for (int s = 0; s < S; ++s) { mbar_init(w_full + s * 8, 1); mbar_init(o_full + s * 8, 4); mbar_init(empty_s + s * 8, 1); }
        mbar_init(done_s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 5) { tmem_alloc(smem_addr(&tmem_slot), Cfg::kTmemCols); tmem_relinquish(); }
    auto issue_weights = [&](int i) {
        const int st = i % S;
        const uint32_t bar = w_full + st * 8, w_s = stages_s + st * Cfg::kStageBytes;
        mbar_expect_tx(bar, kProjChunkBytes);
        const int yrow = (head0 + i) * d + tile * 128;
        tma_load_2d(w_s, &map_po, 0, yrow, bar);
        tma_load_2d(w_s + kProjChunkBytes / 2, &map_po, kBoxCols, yrow, bar);
        issued = i + 1;
    };
    // the weights do not depend on the kernel before this one: the first copies start at once
    if (warp == 4 && lane == 0)
        for (int i = 0; i < n_heads && i < S; ++i) issue_weights(i);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    grid_dependency_wait();          // o comes from the kernel before this one
    grid_launch_dependents();

    if (warp == 4) {
        if (lane == 0) {
            bool ok = true;
            for (int i = S; i < n_heads && ok; ++i) {
                ok = mbar_wait(empty_s + (i % S) * 8, ((i / S) - 1) & 1);
                if (ok) issue_weights(i);
            }
            if (!ok) atomicExch(&timed_out, 1);
        }
    } else if (warp == 5) {
        if (lane == 0) {
            constexpr uint32_t kIdesc = umma_idesc(128, NB, false, false);
            bool ok = true;
            for (int i = 0; i < n_heads; ++i) {
                const int st = i % S;
                if (ok) ok = mbar_wait(w_full + st * 8, (i / S) & 1);
                if (ok) ok = mbar_wait(o_full + st * 8, (i / S) & 1);
                tc_fence_after();
                if (ok) {
                    const uint32_t w_s = stages_s + st * Cfg::kStageBytes, o_s = w_s + kProjChunkBytes;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {                         // 8 k-steps of 16 columns; 4 per 64-column box
                        const uint64_t a = umma_desc(w_s + (ks >> 2) * (kProjChunkBytes / 2) + (ks & 3) * 32, 16, 1024);
                        const uint64_t bd = umma_desc(o_s + (ks >> 2) * (Cfg::kActBytes / 2) + (ks & 3) * 32, 16, 1024);
                        umma_ss(tmem, a, bd, kIdesc, (i > 0 || ks > 0) ? 1u : 0u);
                    }
                }
                tc_commit(empty_s + st * 8);                                 // the stage may be filled again
            }
            tc_commit(done_s);
            if (!ok) atomicExch(&timed_out, 1);
        }
    } else {
        // ---- o[:, head, :] (fp32) -> bf16 tile [NB rows x 128 columns], K-major with the 128-byte swizzle:
        // row n, 16-byte chunk c of its 64-column half at n * 128 + ((c ^ (n & 7)) << 4)
        const int tid = warp * 32 + lane;
        bool ok = true;
        for (int i = 0; i < n_heads; ++i) {
            const int st = i % S;
            if (i >= S && ok) ok = mbar_wait(empty_s + st * 8, ((i / S) - 1) & 1);   // the product that read this tile is done
            const uint32_t o_s = stages_s + st * Cfg::kStageBytes + kProjChunkBytes;
            for (int item = tid; item < NB * 16; item += 128) {
                const int n = item >> 4, ch = item & 15;                     // batch row of the tile, 8-column chunk
                uint32_t w[4] = {0u, 0u, 0u, 0u};
                if (row0 + n < b) {
                    const float4* src = reinterpret_cast<const float4*>(o + ((size_t)(row0 + n) * h + head0 + i) * kHeadDim + ch * 8);
                    const float4 lo = src[0], hi = src[1];
                    w[0] = pack_bf16(lo.x, lo.y); w[1] = pack_bf16(lo.z, lo.w);
                    w[2] = pack_bf16(hi.x, hi.y); w[3] = pack_bf16(hi.z, hi.w);
                }
                const uint32_t at = o_s + (ch >> 3) * (Cfg::kActBytes / 2) + n * 128 + (((ch & 7) ^ (n & 7)) << 4);
                asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(at), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // the tile is read by the tensor core
            __syncwarp();
            if (lane == 0) mbar_arrive(o_full + st * 8);
        }
        // ---- this CTA's Y^T (thread t = row t of the d tile, one TMEM lane; a TMEM column is a batch row) into its
        // shared memory as [NB batch rows][128]: the stages are free once the last product has completed
        const int t = warp * 32 + lane;
        if (ok) ok = mbar_wait(done_s, 0);
        tc_fence_after();
        if (ok && n_heads > 0) {
            uint32_t acc[NB];
            tmem_ld_row<NB>(tmem + ((uint32_t)(warp * 32) << 16), acc);
#pragma unroll
            for (int i = 0; i < NB; ++i)
                asm volatile("st.shared.b32 [%0], %1;" ::"r"(stages_s + (uint32_t)(i * 128 + t) * 4), "r"(acc[i]) : "memory");
        } else {
#pragma unroll
            for (int i = 0; i < NB; ++i)
                asm volatile("st.shared.b32 [%0], %1;" ::"r"(stages_s + (uint32_t)(i * 128 + t) * 4), "r"(0u) : "memory");
        }
        if (!ok) atomicExch(&timed_out, 1);
    }
    tc_fence_before();
    __syncthreads();
    if (timed_out && threadIdx.x == 0) {
        // before anything else: the last copy started into each stage has to land
        for (int s = 0; s < S && s < issued; ++s) mbar_wait(w_full + s * 8, ((issued - 1 - s) / S) & 1);
        if (status) atomicOr(status, kStatusPipelineTimeout);
    }
    __syncthreads();
    cluster_sync();                  // every group's Y^T is in its shared memory
    if (warp < 4) {
        const int t = warp * 32 + lane;
        const uint32_t rank = cluster_cta_rank(), n_groups = cluster_size();
        for (int n = (int)rank; n < NB && row0 + n < b; n += (int)n_groups) {
            float sum = 0.f;
            for (uint32_t g = 0; g < n_groups; ++g) sum += ld_cluster_f32(stages_s + (uint32_t)(n * 128 + t) * 4, g);
            y[(size_t)(row0 + n) * d + (size_t)tile * 128 + t] = sum;
        }
    }
    cluster_sync();                  // nobody leaves while its shared memory is being read
    if (warp == 5) { tc_fence_after(); tmem_dealloc(tmem, Cfg::kTmemCols); }
}

}  // namespace mqa
