// C-ABI entry points of the decode-attention library (declared in include/mqa_decode.h):
// argument validation, the launch plan, and the kernel launches.  Host code here never
// synchronises, allocates or frees device memory.
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <cstdlib>

#include "../../include/mqa_decode.h"
#include "append.cuh"
#include "combine.cuh"
#include "common.cuh"
#include "decode_mma.cuh"
#include "project.cuh"
#include "decode_simt.cuh"
#include "decode_umma.cuh"
#include "decode_local.cuh"
#include "prefill.cuh"
#include "decode_wide.cuh"

namespace mqa {
namespace {

constexpr int kMaxDevices = 64;
std::atomic<int> g_sm_count[kMaxDevices];

// Number of SMs of the current device (148 on a B200); 148 when no device can be queried,
// so that the host-only planning calls still answer on a machine without a GPU.
int sm_count() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return 148; }
    if (dev < 0 || dev >= kMaxDevices) return 148;
    int n = g_sm_count[dev].load(std::memory_order_relaxed);
    if (n > 0) return n;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
        cudaGetLastError();
        return 148;
    }
    g_sm_count[dev].store(n, std::memory_order_relaxed);
    return n;
}

enum class Kernel { kSimt, kMma1, kMma2, kUmma, kWide };
constexpr int kMergeInKernelMaxPieces = 10;
constexpr int kMaxClusterCtas = 4;            // a sequence's CTAs as one thread-block cluster.  Measured per step: clusters of 8
                                              // (16 sequences x 16384 rows) 43 us against 29 us without, clusters of 16
                                              // (8 x 32768) 43 against 30: too few of them fit the GPCs at once

struct Plan {
    int n_splits = 0;     // 0 = invalid.  Fixed-split kernels: splits per sequence.  Persistent kernel: the
                          // most CTAs that can hold pieces of one sequence.
    int chunk_rows = 0;   // rows of the memory axis per split (persistent kernel: per CTA for full caches)
    size_t units = 0;     // b * h
    int b = 0, h = 0;
    int grid = 0;         // persistent kernel: number of CTAs
    Kernel kernel = Kernel::kSimt;
    bool merge_in_kernel = false;   // tcgen05 plan: pieces merged by the CTA that delivers a sequence's last one (single launch)
    bool stream() const { return kernel == Kernel::kUmma; }
};

bool dims_ok(int b, int h, int m_max) { return b > 0 && h > 0 && m_max > 0; }

// Split plan for the CUDA-core kernel (one CTA per (unit, split)): enough CTAs to fill every
// SM several times over, but never chunks shorter than 256 rows, and a single split (no
// combine launch) when the cache is short.
Plan plan_simt(int b, int h, int m_max) {
    Plan p;
    p.units = (size_t)b * h;
    p.b = b; p.h = h;
    const long target_ctas = (long)sm_count() * 16;
    long want = (target_ctas + (long)p.units - 1) / (long)p.units;
    const long cap = m_max / 256 > 1 ? m_max / 256 : 1;
    if (want > cap) want = cap;
    if (want > 1024) want = 1024;                 // the second pass keeps one (max, sum) per split in shared memory
    if (want < 1) want = 1;
    int chunk = (int)((m_max + want - 1) / want);
    chunk = (chunk + 63) / 64 * 64;
    p.chunk_rows = chunk;
    p.n_splits = (m_max + chunk - 1) / chunk;
    return p;
}

// Split plan for the tensor-core multi-query kernel (one CTA per (sequence, split), every CTA
// serving all h heads).  A small cost model in units of "cache rows streamed by one SM":
// CTAs run in waves over the resident slots, every CTA pays a fixed start-up/merge cost, and
// every split adds partial results that are written once and read once by the combine pass.
Plan plan_mma(int b, int h, int m_max) {
    Plan p;
    p.units = (size_t)b * h;
    p.b = b; p.h = h;
    p.kernel = h <= 16 ? Kernel::kMma1 : Kernel::kMma2;
    const int ctas_per_sm = h <= 16 ? MmaCfg<1>::kMinBlocks : MmaCfg<2>::kMinBlocks;
    const int sms = sm_count();
    const long slots = (long)sms * ctas_per_sm;
    const double overhead_rows = 128.0;                               // start-up + merge, per CTA
    const double partial_rows = (double)h * (kHeadDim + 2) * 4 * 2 / (2.0 * kRowBytes);   // per split
    const int max_splits = m_max / 128 > 1 ? (m_max / 128 < 256 ? m_max / 128 : 256) : 1;
    double best = 0;
    for (int s = 1; s <= max_splits; ++s) {
        int chunk = (m_max + s - 1) / s;
        chunk = (chunk + kTileRows - 1) / kTileRows * kTileRows;
        const int n = (m_max + chunk - 1) / chunk;
        if (n != s) continue;                                         // same plan as a smaller s
        const long ctas = (long)b * n;
        const long waves = (ctas + slots - 1) / slots;
        double cost = (double)waves * (chunk + overhead_rows) * ctas_per_sm;
        if (n > 1) cost += (double)ctas * partial_rows / sms;
        if (p.n_splits == 0 || cost < best) {
            best = cost;
            p.n_splits = n;
            p.chunk_rows = chunk;
        }
    }
    return p;
}

// Persistent tensor-core kernel: one CTA per SM, equal shares of the line of valid tiles.
Plan plan_stream(int b, int h, int m_max) {
    Plan p;
    p.units = (size_t)b * h;
    p.b = b; p.h = h;
    p.kernel = Kernel::kUmma;
    // One CTA per SM -- or a few fewer, when that makes the grid a multiple or a divisor of the batch: with
    // sequences of equal length every share then starts at a sequence's beginning, a sequence has the fewest
    // pieces (none when CTAs take whole sequences) and the CTAs that hold them finish together.  HBM is
    // saturated from about three quarters of the SMs on (measured: same pass time with 112..148 CTAs).
    // Among the multiples of the batch, first one that makes a sequence's CTAs a thread-block cluster.
    const int sms = sm_count();
    p.grid = sms;
    bool found = false;
    for (int g = sms; g >= (3 * sms + 3) / 4 && !found; --g)
        if (b % g == 0 || (g % b == 0 && g / b <= kMaxClusterCtas)) { p.grid = g; found = true; }
    for (int g = sms; g >= (3 * sms + 3) / 4 && !found; --g)
        if (g % b == 0) { p.grid = g; found = true; }
    const long long tiles = (long long)b * ((m_max + kTileRows - 1) / kTileRows);
    p.chunk_rows = (int)((tiles + p.grid - 1) / p.grid) * kTileRows;
    int parts = (p.grid + b - 1) / b + 1;
    p.n_splits = parts < p.grid ? parts : p.grid;
    // a sequence cut into a few pieces is merged by one CTA inside the kernel; many pieces (few, long
    // sequences) are better spread over all SMs by the second-pass kernel
    // ... unless the batch divides the grid into clusters: then, with sequences
    // of equal length, a cluster merges its sequence through its shared memory however many pieces that is
    p.merge_in_kernel = p.kernel == Kernel::kUmma &&
                        (p.n_splits <= kMergeInKernelMaxPieces || (p.grid % b == 0 && p.grid / b >= 2 && p.grid / b <= kMaxClusterCtas));
    return p;
}

// Fixed splits for the kernel with the query rows as tile rows (decode_wide.cuh: 33 .. 128 query rows per sequence): one
// CTA per (sequence, split), about one CTA per SM, splits of whole 128-row stages and never shorter than two of them.
Plan plan_wide(int b, int h, int m_max) {
    Plan p;
    p.units = (size_t)b * h;
    p.b = b; p.h = h;
    p.kernel = Kernel::kWide;
    const int tiles = (h + kWideRows - 1) / kWideRows;           // row tiles of 128 query rows (grid.y)
    int want = sm_count() / (b * tiles);
    const int cap = m_max / (2 * kWideRows);
    if (want > cap) want = cap;
    if (want > 160) want = 160;                    // (the second pass merges up to 160 pieces in one go)
    if (want < 1) want = 1;
    int chunk = (m_max + want - 1) / want;
    chunk = (chunk + kWideRows - 1) / kWideRows * kWideRows;
    p.chunk_rows = chunk;
    p.n_splits = (m_max + chunk - 1) / chunk;
    return p;
}

Plan make_plan(bool multi_query, int b, int h, int m_max) {
    // a row space too large for the 32-bit TMA coordinates goes to the general CUDA-core kernel
    if (!(multi_query && (long long)b * m_max < 0x7fffffffLL)) return plan_simt(b, h, m_max);
    // More than 32 query rows per sequence: the kernel with the query rows as tile rows, 128 rows per CTA and more as row
    // tiles over the same cache rows.  (The streaming kernel used to take up to 64 rows on a tile of its own and more as
    // groups of 64: measured against that, per step, 32 x 64 rows x 8192: 30.5 vs 35.0 us; 128 x 64 x 2048: 26.2 vs 32.8;
    // 4 x 48 x 4096: 10.8 vs 20.7; 32 x 128 x 8192: 34.9 vs 68.8; 32 x 256 x 8192: 43.6 vs 122.7; 128 x 160 x 2048: 50.1 vs
    // 103.2 -- that tile and the groups are gone.)
    if (h > 32 && (h + kWideRows - 1) / kWideRows <= 65535 && (long long)b * h < 0x7fffffffLL) return plan_wide(b, h, m_max);
    // enough tiles to give every SM a real share: the persistent kernels; otherwise fixed splits
    const long long tiles = (long long)b * ((m_max + kTileRows - 1) / kTileRows);
    const int sms = sm_count();
    if (b <= kStreamMaxSeqs && tiles >= 2LL * sms && m_max >= 1024 && sms <= 256) {
        const Plan p = plan_stream(b, h, m_max);
        // few, long sequences, each cut into more pieces than one CTA merges inside the kernel: the streaming kernel would
        // need its second pass as well, and the kernel with the query rows as tile rows (fixed splits, second pass) is
        // then the quicker of the two (measured per step: 1 x 32 heads x 32768 rows 16.2 vs 18.5 us, 4 x 32 x 4096 10.5 vs
        // 14.2, 8 x 32 x 32768 29.2 vs 30.6, 8 x 16 x 8192 16.1 vs 16.4)
        if (!p.merge_in_kernel) return plan_wide(b, h, m_max);
        return p;
    }
    return h <= 32 ? plan_mma(b, h, m_max) : plan_simt(b, h, m_max);
}

// Every workspace begins with the control block of the single-launch step (kStreamCtrlBytes: see decode_umma.cuh),
// whatever the plan: a workspace that serves several shapes then keeps one epoch for all of them, and the kernels of
// the other plans never write over it.  The plan's own scratch follows.
size_t plan_workspace_bytes(const Plan& p) {
    if (p.stream()) {
        const int slots = p.grid + p.b;
        return kStreamCtrlBytes + stream_span_bytes(p.b) + stream_ml_bytes(slots, p.h) + stream_acc_bytes(slots, p.h);
    }
    if (p.n_splits <= 1) return 0;
    return kStreamCtrlBytes + partial_ml_bytes(p.units, p.n_splits) + partial_acc_bytes(p.units, p.n_splits);
}

// Fixed-split plans: (max, sum) pairs, then the accumulators, after the control block.
float2* partials_ml(const void* workspace) {
    return workspace ? reinterpret_cast<float2*>(static_cast<char*>(const_cast<void*>(workspace)) + kStreamCtrlBytes) : nullptr;
}
float* partials_acc(const Plan& p, const void* workspace) {
    return workspace ? reinterpret_cast<float*>(static_cast<char*>(const_cast<void*>(workspace)) + kStreamCtrlBytes +
                                                partial_ml_bytes(p.units, p.n_splits))
                     : nullptr;
}

struct StreamWorkspace {
    int2* span;
    float2* ml;
    float* acc;
    unsigned long long* ctrl;     // control block of the single-launch step (tcgen05 kernel)
};
StreamWorkspace stream_workspace(const Plan& p, const void* workspace) {
    char* base = static_cast<char*>(const_cast<void*>(workspace));
    const int slots = p.grid + p.b;
    StreamWorkspace w;
    w.ctrl = reinterpret_cast<unsigned long long*>(base);
    base += kStreamCtrlBytes;
    w.span = reinterpret_cast<int2*>(base);
    w.ml = reinterpret_cast<float2*>(base + stream_span_bytes(p.b));
    w.acc = reinterpret_cast<float*>(base + stream_span_bytes(p.b) + stream_ml_bytes(slots, p.h));
    return w;
}

// Launch `kernel` so that it may begin while the kernel before it in the stream is still running
// (programmatic dependent launch).  Every kernel of this library waits (griddepcontrol.wait)
// before it touches memory an earlier kernel may write, so the only effect is that launch
// latency and set-up overlap the tail of the previous kernel.
template <typename... Params, typename... Args>
cudaError_t launch_dependent_clusters(unsigned cluster, void (*kernel)(Params...), unsigned grid, unsigned block, size_t smem,
                                      cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cluster > 1) {
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = cluster; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
        cfg.numAttrs = 2;
    }
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<Params>(args)...);
}

template <typename... Params, typename... Args>
cudaError_t launch_dependent_2d(void (*kernel)(Params...), unsigned grid_x, unsigned grid_y, unsigned block, size_t smem,
                                cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid_x, grid_y);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<Params>(args)...);
}

template <typename... Params, typename... Args>
cudaError_t launch_dependent(void (*kernel)(Params...), unsigned grid, unsigned block, size_t smem,
                             cudaStream_t stream, Args... args) {
    return launch_dependent_clusters(1u, kernel, grid, block, smem, stream, args...);
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool aligned4(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 3u) == 0; }

int check_step_args(const void* q, const void* K, const void* V, const int32_t* lens, const float* o,
                    const int32_t* status, int b, int h, int m_max, int k, int v) {
    if (!q || !K || !V || !lens || !o) return MQA_ERR_INVALID_ARG;
    if (!dims_ok(b, h, m_max) || k <= 0 || v <= 0) return MQA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(K) || !aligned16(V) || !aligned16(o) || !aligned4(lens) ||
        !aligned4(status))
        return MQA_ERR_INVALID_ARG;
    if (k != kHeadDim || v != kHeadDim) return MQA_ERR_UNSUPPORTED;
    return MQA_OK;
}

int check_workspace(const Plan& p, const void* workspace, size_t workspace_bytes) {
    const size_t need = plan_workspace_bytes(p);
    if (need == 0) return MQA_OK;
    if (!workspace || !aligned16(workspace)) return MQA_ERR_INVALID_ARG;
    if (workspace_bytes < need) return MQA_ERR_WORKSPACE_TOO_SMALL;
    return MQA_OK;
}

// cuTensorMapEncodeTiled through the runtime's driver entry point (no link against libcuda).
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
std::atomic<EncodeTiledFn> g_encode{nullptr};

EncodeTiledFn encode_fn() {
    EncodeTiledFn f = g_encode.load(std::memory_order_acquire);
    if (f) return f;
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !sym) {
        cudaGetLastError();
        return nullptr;
    }
    f = reinterpret_cast<EncodeTiledFn>(sym);
    g_encode.store(f, std::memory_order_release);
    return f;
}

// A row-major bf16 matrix [rows][cols] fetched in boxes of box_rows rows x 64 columns (128-byte swizzle).
// A decoding loop asks for the same few maps at every step (the cache, the weights) and encoding one costs about a
// microsecond of host time, so every thread keeps the maps it encoded last, by (address, shape, box): a map describes
// nothing but those, so it stays valid whatever the memory holds.
bool encode_matrix_map(CUtensorMap* map, const void* base, long long rows, long long cols, int box_rows) {
    struct Entry { const void* base; long long rows, cols; int box_rows; bool used; CUtensorMap map; };
    constexpr int kEntries = 32;
    thread_local Entry kept[kEntries] = {};
    size_t hash = reinterpret_cast<size_t>(base) >> 8;
    hash = (hash ^ (hash >> 7) ^ (size_t)rows * 31u ^ (size_t)cols * 131u ^ (size_t)box_rows * 7u) % kEntries;
    Entry& e = kept[hash];
    if (e.used && e.base == base && e.rows == rows && e.cols == cols && e.box_rows == box_rows) {
        *map = e.map;
        return true;
    }
    EncodeTiledFn enc = encode_fn();
    if (!enc) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kBoxCols, (cuuint32_t)box_rows};
    const cuuint32_t elem[2] = {1, 1};
    if (enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, elem,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    e.base = base; e.rows = rows; e.cols = cols; e.box_rows = box_rows; e.map = *map; e.used = true;
    return true;
}

// The cache of one tensor (K or V) as a 2-D bf16 tensor [rows = b * m_max][128 columns], fetched in
// boxes of kTileRows rows x 64 columns (128 bytes, the span of the 128-byte swizzle).
bool encode_cache_map(CUtensorMap* map, const void* base, long long rows, int box_rows = kTileRows) {
    return encode_matrix_map(map, base, rows, kHeadDim, box_rows);
}

std::atomic<int> g_smem_opt_in[kMaxDevices][4];

template <int M_TILES, bool EARLY = false>
int launch_mma(const Plan& p, const void* q, const void* K, const void* V, const int32_t* lens, float* o,
               float2* part_ml, float* part_acc, int32_t* status, int b, int h, int m_max, cudaStream_t stream, int len_bias,
               const void* k_new = nullptr, const void* v_new = nullptr, int32_t* lens_advance = nullptr,
               bool withhold = false) {
    using Cfg = MmaCfg<M_TILES>;
    auto kernel = mqa_decode_split_mma_kernel<M_TILES, EARLY>;
    constexpr int kSlot = (M_TILES - 1) * 2 + (EARLY ? 1 : 0);
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return MQA_ERR_CUDA; }
    if (!g_smem_opt_in[dev][kSlot].load(std::memory_order_acquire)) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes) != cudaSuccess) {
            cudaGetLastError();
            return MQA_ERR_CUDA;
        }
        g_smem_opt_in[dev][kSlot].store(1, std::memory_order_release);
    }
    alignas(64) CUtensorMap map_k, map_v, map_k_big, map_v_big;
    if (!encode_cache_map(&map_k, K, (long long)b * m_max) || !encode_cache_map(&map_v, V, (long long)b * m_max) ||
        !encode_cache_map(&map_k_big, K, (long long)b * m_max, 4 * kTileRows) ||
        !encode_cache_map(&map_v_big, V, (long long)b * m_max, 4 * kTileRows))
        return MQA_ERR_CUDA;
    FusedArgs fa = {};
    if (k_new) {                                       // the whole decoding step in this launch (one CTA per sequence)
        fa.k_new = static_cast<const uint4*>(k_new);
        fa.v_new = static_cast<const uint4*>(v_new);
        fa.K = static_cast<uint4*>(const_cast<void*>(K));
        fa.V = static_cast<uint4*>(const_cast<void*>(V));
    }
    launch_dependent(kernel, (unsigned)((size_t)b * p.n_splits), Cfg::kThreads, Cfg::kSmemBytes, stream, map_k, map_v,
                     map_k_big, map_v_big, static_cast<const uint32_t*>(q), lens, o, part_ml, part_acc, status, h, m_max, p.chunk_rows,
                     p.n_splits, len_bias, fa, lens_advance, withhold ? 2 : 0);
    return cudaGetLastError() == cudaSuccess ? MQA_OK : MQA_ERR_CUDA;
}

constexpr int kLocalMaxWindow = 4096;         // the longest window the local step takes (a warp per sequence: decode_local.cuh)
constexpr size_t kL2KeepBytes = 64u << 20;   // K and V together: half of the 126 MB L2
constexpr int kEarlyTestWithhold = 1 << 8;    // rides on `early`: MQA_STEP_TEST_WITHHOLD_COPY
std::atomic<int> g_umma_opt_in[kMaxDevices][13];

// The streaming kernel serves up to 32 query rows per sequence (HP = 16 or 32); more go to decode_wide.cuh.
template <int HP, bool FUSED, bool GUESS = false>
int launch_umma(const Plan& p, const void* q, const void* K, const void* V, const int32_t* lens, float* o,
                void* workspace, int32_t* status, int b, int h, int m_max, cudaStream_t stream, bool merge,
                const void* k_new = nullptr, const void* v_new = nullptr, int32_t* lens_advance = nullptr,
                int early = 0) {
    using Cfg = UmmaCfg<HP>;
    auto kernel = mqa_decode_stream_umma_kernel<HP, FUSED, GUESS>;
    static_assert(HP == 16 || HP == 32, "padded head count");
    constexpr int kSlot = (HP == 16 ? 0 : 1) * 3 + (GUESS ? 2 : FUSED ? 1 : 0);
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return MQA_ERR_CUDA; }
    if (!g_umma_opt_in[dev][kSlot].load(std::memory_order_acquire)) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes) != cudaSuccess ||
            cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess) {
            cudaGetLastError();
            return MQA_ERR_CUDA;
        }
        g_umma_opt_in[dev][kSlot].store(1, std::memory_order_release);
    }
    FusedArgs fa = {};
    if (FUSED) {
        fa.k_new = static_cast<const uint4*>(k_new);
        fa.v_new = static_cast<const uint4*>(v_new);
        fa.K = static_cast<uint4*>(const_cast<void*>(K));
        fa.V = static_cast<uint4*>(const_cast<void*>(V));
    }
    alignas(64) CUtensorMap map_k, map_v, map_k_sub, map_v_sub, map_q;
    const long long rows = (long long)b * m_max;
    if (!encode_cache_map(&map_k, K, rows, kUmmaStageRows) || !encode_cache_map(&map_v, V, rows, kUmmaStageRows) ||
        !encode_cache_map(&map_k_sub, K, rows) || !encode_cache_map(&map_v_sub, V, rows) ||
        !encode_cache_map(&map_q, q, (long long)b * h, HP))
        return MQA_ERR_CUDA;
    const StreamWorkspace w = stream_workspace(p, workspace);
    // a cache that cannot stay in L2 from one step to the next is streamed through it with the evict-first policy
    const int read_once = ((size_t)b * m_max * 2 * kRowBytes > kL2KeepBytes ? 1 : 0) | ((early & kEarlyTestWithhold) ? 2 : 0);
    early &= ~kEarlyTestWithhold;
    // The single-launch step of a batch that divides the grid runs as clusters of grid / b CTAs (2 to 4): with sequences of equal length a cluster then holds exactly one sequence's pieces and merges
    // them through its shared memory (the kernel decides from lens; otherwise the clusters change nothing).
    unsigned cluster = 1;
    if (merge && p.grid % p.b == 0 && p.grid / p.b >= 2 && p.grid / p.b <= kMaxClusterCtas) cluster = (unsigned)(p.grid / p.b);
    launch_dependent_clusters(cluster, kernel, (unsigned)p.grid, kUmmaThreads, Cfg::kSmemBytes, stream, map_k, map_v, map_k_sub,
                              map_v_sub, map_q, lens, o, w.span, w.ml, w.acc, status, p.b, p.h, m_max, share_magic(p.grid), fa,
                              merge ? w.ctrl : nullptr, lens_advance, early, read_once);
    return cudaGetLastError() == cudaSuccess ? MQA_OK : MQA_ERR_CUDA;
}

template <bool FUSED>
int launch_umma_for(const Plan& p, const void* q, const void* K, const void* V, const int32_t* lens, float* o,
                    void* workspace, int32_t* status, int b, int h, int m_max, cudaStream_t stream, bool merge,
                    const void* k_new = nullptr, const void* v_new = nullptr, int32_t* lens_advance = nullptr,
                    int early = 0) {
#define MQA_UMMA_ARGS p, q, K, V, lens, o, workspace, status, b, h, m_max, stream, merge, k_new, v_new, lens_advance, early
    if constexpr (FUSED) {
        if ((early & ~kEarlyTestWithhold) >= 2) {           // the kernels that carry the code for copies started on a guess
            if (p.h <= 16) return launch_umma<16, true, true>(MQA_UMMA_ARGS);
            return launch_umma<32, true, true>(MQA_UMMA_ARGS);
        }
    }
    if (p.h <= 16) return launch_umma<16, FUSED>(MQA_UMMA_ARGS);
    return launch_umma<32, FUSED>(MQA_UMMA_ARGS);
#undef MQA_UMMA_ARGS
}

int launch_status() { return cudaGetLastError() == cudaSuccess ? MQA_OK : MQA_ERR_CUDA; }

int launch_wide(const Plan& p, const void* q, const void* K, const void* V, const int32_t* lens, float* o, float2* part_ml,
                float* part_acc, int32_t* status, int b, int h, int m_max, cudaStream_t stream, int len_bias,
                const void* k_new = nullptr, const void* v_new = nullptr, int32_t* lens_advance = nullptr, bool withhold = false) {
    FusedArgs fa = {};
    if (k_new) {
        fa.k_new = static_cast<const uint4*>(k_new);
        fa.v_new = static_cast<const uint4*>(v_new);
        fa.K = static_cast<uint4*>(const_cast<void*>(K));
        fa.V = static_cast<uint4*>(const_cast<void*>(V));
    }
    static std::atomic<int> opt_in[kMaxDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return MQA_ERR_CUDA; }
    if (!opt_in[dev].load(std::memory_order_acquire)) {
        if (cudaFuncSetAttribute(mqa_decode_wide_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kWideSmemBytes) != cudaSuccess) {
            cudaGetLastError();
            return MQA_ERR_CUDA;
        }
        opt_in[dev].store(1, std::memory_order_release);
    }
    alignas(64) CUtensorMap map_q, map_k, map_v;
    if (!encode_cache_map(&map_q, q, (long long)b * h, kWideRows) || !encode_cache_map(&map_k, K, (long long)b * m_max, kWideRows) ||
        !encode_cache_map(&map_v, V, (long long)b * m_max, kWideRows))
        return MQA_ERR_CUDA;
    launch_dependent_2d(mqa_decode_wide_kernel, (unsigned)((size_t)b * p.n_splits), (unsigned)((h + kWideRows - 1) / kWideRows),
                        (unsigned)kWideThreads, (size_t)kWideSmemBytes, stream, map_q,
                     map_k, map_v, lens, o, part_ml, part_acc, status, h, m_max, p.chunk_rows, p.n_splits, len_bias, fa, lens_advance,
                     withhold ? 1 : 0);
    return launch_status();
}

int run_split(bool multi_query, const void* q, const void* K, const void* V, const int32_t* lens, float* o,
              void* workspace, size_t workspace_bytes, int32_t* status,
              int b, int h, int m_max, int k, int v, cudaStream_t stream, int len_bias = 0, bool merge_in_kernel = false) {
    int rc = check_step_args(q, K, V, lens, o, status, b, h, m_max, k, v);
    if (rc) return rc;
    const Plan p = make_plan(multi_query, b, h, m_max);
    if (p.units * (size_t)p.n_splits > 0x7fffffffull) return MQA_ERR_UNSUPPORTED;
    rc = check_workspace(p, workspace, workspace_bytes);
    if (rc) return rc;
    if (p.kernel == Kernel::kUmma)
        return launch_umma_for<false>(p, q, K, V, lens, o, workspace, status, b, h, m_max, stream, merge_in_kernel);
    float2* part_ml = partials_ml(workspace);
    float* part_acc = partials_acc(p, workspace);
    if (p.kernel == Kernel::kWide) return launch_wide(p, q, K, V, lens, o, part_ml, part_acc, status, b, h, m_max, stream, len_bias);
    if (p.kernel == Kernel::kMma1)
        return launch_mma<1>(p, q, K, V, lens, o, part_ml, part_acc, status, b, h, m_max, stream, len_bias);
    if (p.kernel == Kernel::kMma2)
        return launch_mma<2>(p, q, K, V, lens, o, part_ml, part_acc, status, b, h, m_max, stream, len_bias);
    const unsigned grid = (unsigned)(p.units * (size_t)p.n_splits);
    launch_dependent(decode_split_simt_kernel, grid, kSimtThreads, 0, stream, static_cast<const uint4*>(q),
                     static_cast<const uint4*>(K), static_cast<const uint4*>(V), lens, o, part_ml, part_acc, status, h,
                     multi_query ? h : 1, m_max, p.chunk_rows, p.n_splits, len_bias);
    return launch_status();
}

// Second pass of the persistent kernel: one CTA per (schedule sequence, query row) merges the sequence's pieces.
int launch_stream_combine(const Plan& p, const void* workspace, float* o, int32_t* lens_advance, int m_max, cudaStream_t stream) {
    const StreamWorkspace w = stream_workspace(p, workspace);
    const unsigned grid = (unsigned)((size_t)p.b * p.h);
    if (p.n_splits <= kCombineEager)
        launch_dependent(stream_combine_kernel<1>, grid, kHeadDim, 0, stream, w.span, w.ml, w.acc, o, p.b, p.h, lens_advance,
                         m_max, share_magic(p.grid));
    else if (p.n_splits <= 4 * kCombineEager)
        launch_dependent(stream_combine_kernel<4>, grid, 4 * kHeadDim, 0, stream, w.span, w.ml, w.acc, o, p.b, p.h,
                         lens_advance, m_max, share_magic(p.grid));
    else
        launch_dependent(stream_combine_kernel<kCombineManyGroups>, grid, 4 * kHeadDim, 0, stream, w.span, w.ml, w.acc, o,
                         p.b, p.h, lens_advance, m_max, share_magic(p.grid));
    return launch_status();
}

int run_combine(bool multi_query, const int32_t* lens, float* o, const void* workspace, size_t workspace_bytes,
                int b, int h, int m_max, int k, int v, cudaStream_t stream, int len_bias = 0,
                int32_t* lens_advance = nullptr, bool fused = false) {
    if (!lens || !o || !dims_ok(b, h, m_max) || !aligned16(o) || !aligned4(lens)) return MQA_ERR_INVALID_ARG;
    if (k != kHeadDim || v != kHeadDim) return MQA_ERR_UNSUPPORTED;
    const Plan p = make_plan(multi_query, b, h, m_max);
    if (p.units > 0x7fffffffull) return MQA_ERR_UNSUPPORTED;
    int rc = check_workspace(p, workspace, workspace_bytes);
    if (rc) return rc;
    if (p.stream()) {
        return launch_stream_combine(p, workspace, o, lens_advance, m_max, stream);
    }
    if (p.n_splits <= 1) return MQA_OK;
    const float2* part_ml = partials_ml(workspace);
    const float* part_acc = partials_acc(p, workspace);
    // fused (the append-and-attend step of a sequence cut into fixed splits): the pass wrote a piece for every split,
    // the second pass does not look at lens and moves it on when asked to
    const int32_t* lens_read = fused ? nullptr : lens;
    if (p.n_splits <= kCombineEager)
        launch_dependent(combine_few_kernel, (unsigned)((p.units + kCombineFewWarps - 1) / kCombineFewWarps), (unsigned)(kCombineFewWarps * 32),
                         0, stream, part_ml, part_acc, lens_read, o, h, m_max, p.chunk_rows, p.n_splits, len_bias,
                         fused ? lens_advance : static_cast<int32_t*>(nullptr), p.units);
    else
        launch_dependent(combine_splits_kernel<4>, (unsigned)p.units, 4 * kHeadDim, 0, stream, part_ml, part_acc, lens_read, o, h,
                         m_max, p.chunk_rows, p.n_splits, len_bias, fused ? lens_advance : static_cast<int32_t*>(nullptr));
    return launch_status();
}

int run_step(bool multi_query, const void* q, const void* K, const void* V, const int32_t* lens, float* o,
             void* workspace, size_t workspace_bytes, int32_t* status,
             int b, int h, int m_max, int k, int v, cudaStream_t stream) {
    // the tcgen05 plan is a single launch: the CTA that delivers the last piece of a sequence merges the pieces
    const bool one_launch = dims_ok(b, h, m_max) && make_plan(multi_query, b, h, m_max).merge_in_kernel;
    int rc = run_split(multi_query, q, K, V, lens, o, workspace, workspace_bytes, status, b, h, m_max, k, v, stream, 0,
                       one_launch);
    if (rc || one_launch) return rc;
    return run_combine(multi_query, lens, o, workspace, workspace_bytes, b, h, m_max, k, v, stream);
}

// lens[i] += 1 for the sequences that took a row (the multi-launch form of mqa_decode_append_step
// advances lens last, after the kernels that read the old value).
__global__ void lens_advance_kernel(int32_t* lens, int b, int m_max) {
    grid_dependency_wait();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < b && lens[i] >= 0 && lens[i] < m_max) lens[i] += 1;
}

// ---- the whole layer step: projections, append + attention, output projection ---------------------
size_t align256(size_t n) { return (n + 255) & ~(size_t)255; }

struct LayerWorkspace {
    size_t q, k_new, v_new, o, step, total;             // byte offsets
};
LayerWorkspace layer_workspace(int b, int h, int d, int m_max) {
    LayerWorkspace w;
    size_t at = 0;
    w.q = at;      at += align256((size_t)b * h * kHeadDim * 2);
    w.k_new = at;  at += align256((size_t)b * kHeadDim * 2);
    w.v_new = at;  at += align256((size_t)b * kHeadDim * 2);
    w.o = at;      at += align256((size_t)b * h * kHeadDim * 4);
    w.step = at;   at += align256(plan_workspace_bytes(make_plan(true, b, h, m_max)));
    w.total = at;
    return w;
}

std::atomic<int> g_proj_opt_in[kMaxDevices][8];

template <int NB>
int launch_projections_in(const void* x, const void* P_q, const void* P_k, const void* P_v, void* q, void* k_new, void* v_new,
                          int32_t* status, int b, int h, int d, cudaStream_t stream) {
    using Cfg = ProjCfg<NB>;
    auto kernel = project_in_kernel<NB>;
    constexpr int kSlot = NB == 16 ? 0 : (NB == 32 ? 1 : (NB == 64 ? 2 : 3));
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return MQA_ERR_CUDA; }
    if (!g_proj_opt_in[dev][kSlot].load(std::memory_order_acquire)) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes) != cudaSuccess) {
            cudaGetLastError();
            return MQA_ERR_CUDA;
        }
        g_proj_opt_in[dev][kSlot].store(1, std::memory_order_release);
    }
    alignas(64) CUtensorMap map_pq, map_pk, map_pv, map_x;
    if (!encode_matrix_map(&map_pq, P_q, (long long)h * d, kHeadDim, 128) || !encode_matrix_map(&map_pk, P_k, d, kHeadDim, 128) ||
        !encode_matrix_map(&map_pv, P_v, d, kHeadDim, 128) || !encode_matrix_map(&map_x, x, b, d, NB))
        return MQA_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(h + 2), (unsigned)((b + 127) / 128));
    cfg.blockDim = dim3(kProjThreads);
    cfg.dynamicSmemBytes = Cfg::kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kernel, map_pq, map_pk, map_pv, map_x, static_cast<__nv_bfloat16*>(q),
                       static_cast<__nv_bfloat16*>(k_new), static_cast<__nv_bfloat16*>(v_new), status, b, h, d);
    return launch_status();
}

// The output projection: the head groups of a (d tile, batch tile) are the CTAs of one thread-block cluster (see
// project_out_kernel), so there are at most kProjMaxGroups of them, each with ceil(h / groups) heads.
template <int NB>
int launch_projection_out(const void* P_o, const float* o, float* y, int32_t* status, int b, int h, int d, cudaStream_t stream) {
    using Cfg = ProjCfg<NB>;
    auto kernel = project_out_kernel<NB>;
    constexpr int kSlot = 4 + (NB == 16 ? 0 : (NB == 32 ? 1 : (NB == 64 ? 2 : 3)));
    constexpr int kSmem = 2 * Cfg::kStageBytes + 256 + 1024;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return MQA_ERR_CUDA; }
    if (!g_proj_opt_in[dev][kSlot].load(std::memory_order_acquire)) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem) != cudaSuccess ||
            (kProjMaxGroups > 8 && cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess)) {
            cudaGetLastError();
            return MQA_ERR_CUDA;
        }
        g_proj_opt_in[dev][kSlot].store(1, std::memory_order_release);
    }
    alignas(64) CUtensorMap map_po;
    if (!encode_matrix_map(&map_po, P_o, (long long)h * d, kHeadDim, 128)) return MQA_ERR_CUDA;
    const int heads_per_cta = (h + kProjMaxGroups - 1) / kProjMaxGroups;
    const int groups = (h + heads_per_cta - 1) / heads_per_cta;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(d / 128), (unsigned)groups, (unsigned)((b + 127) / 128));
    cfg.blockDim = dim3(kProjThreads);
    cfg.dynamicSmemBytes = kSmem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 1;
    attr[1].val.clusterDim.y = (unsigned)groups;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    cudaLaunchKernelEx(&cfg, kernel, map_po, o, y, status, b, h, d, heads_per_cta);
    return launch_status();
}

}  // namespace
}  // namespace mqa

using namespace mqa;

extern "C" {
#ifdef MQA_DEBUG_TS
void mqa_debug_ts(unsigned long long* t) { cudaMemcpyFromSymbol(t, mqa::g_ts, sizeof(mqa::g_ts)); }
void mqa_debug_st(unsigned long long* t) { cudaMemcpyFromSymbol(t, mqa::g_st, sizeof(mqa::g_st)); }
#endif

int kv_cache_append(void* K, void* V, const void* k_new, const void* v_new, int32_t* lens, int advance,
                    int32_t* status, int b, int kv_heads, int m_max, int k, int v, mqa_stream_t stream) {
    if (!K || !V || !k_new || !v_new || !lens) return MQA_ERR_INVALID_ARG;
    if (b <= 0 || kv_heads <= 0 || m_max <= 0 || k <= 0 || v <= 0) return MQA_ERR_INVALID_ARG;
    if (!aligned16(K) || !aligned16(V) || !aligned16(k_new) || !aligned16(v_new) || !aligned4(lens) ||
        !aligned4(status))
        return MQA_ERR_INVALID_ARG;
    if (k != kHeadDim || v != kHeadDim) return MQA_ERR_UNSUPPORTED;
    launch_dependent(kv_cache_append_kernel, (unsigned)b, kAppendThreads, 0, static_cast<cudaStream_t>(stream),
                     static_cast<uint4*>(K), static_cast<uint4*>(V), static_cast<const uint4*>(k_new),
                     static_cast<const uint4*>(v_new), lens, advance, status, kv_heads, m_max);
    return launch_status();
}

int mqa_decode_step(const void* q, const void* K, const void* V, const int32_t* lens, float* o, void* workspace,
                    size_t workspace_bytes, int32_t* status, int b, int h, int m_max, int k, int v,
                    mqa_stream_t stream) {
    return run_step(true, q, K, V, lens, o, workspace, workspace_bytes, status, b, h, m_max, k, v,
                    static_cast<cudaStream_t>(stream));
}

int mha_decode_step(const void* q, const void* K, const void* V, const int32_t* lens, float* o, void* workspace,
                    size_t workspace_bytes, int32_t* status, int b, int h, int m_max, int k, int v,
                    mqa_stream_t stream) {
    return run_step(false, q, K, V, lens, o, workspace, workspace_bytes, status, b, h, m_max, k, v,
                    static_cast<cudaStream_t>(stream));
}

int mqa_decode_step_split(const void* q, const void* K, const void* V, const int32_t* lens, float* o,
                          void* workspace, size_t workspace_bytes, int32_t* status, int b, int h, int m_max,
                          int k, int v, mqa_stream_t stream) {
    return run_split(true, q, K, V, lens, o, workspace, workspace_bytes, status, b, h, m_max, k, v,
                     static_cast<cudaStream_t>(stream));
}

int mqa_decode_step_combine(const int32_t* lens, float* o, const void* workspace, size_t workspace_bytes, int b,
                            int h, int m_max, int k, int v, mqa_stream_t stream) {
    return run_combine(true, lens, o, workspace, workspace_bytes, b, h, m_max, k, v,
                       static_cast<cudaStream_t>(stream));
}

int mha_decode_step_split(const void* q, const void* K, const void* V, const int32_t* lens, float* o,
                          void* workspace, size_t workspace_bytes, int32_t* status, int b, int h, int m_max,
                          int k, int v, mqa_stream_t stream) {
    return run_split(false, q, K, V, lens, o, workspace, workspace_bytes, status, b, h, m_max, k, v,
                     static_cast<cudaStream_t>(stream));
}

int mha_decode_step_combine(const int32_t* lens, float* o, const void* workspace, size_t workspace_bytes, int b,
                            int h, int m_max, int k, int v, mqa_stream_t stream) {
    return run_combine(false, lens, o, workspace, workspace_bytes, b, h, m_max, k, v,
                       static_cast<cudaStream_t>(stream));
}

// early: what the persistent kernel may do before it waits for the kernel before it (see early in
// mqa_decode_stream_umma_kernel): kEarlyAfterProjection inside the layer step, kEarlyChained when the caller set
// MQA_STEP_CHAINED.  flags: MQA_STEP_ADVANCE | MQA_STEP_CHAINED.
constexpr int kEarlyNone = 0, kEarlyAfterProjection = 1, kEarlyChained = 2, kEarlyChainedWrongGuess = 3;
constexpr int kGuessMaxPieces = 6, kGuessMinShareRows = 8 * kUmmaStageRows;
// Every check of mqa_decode_append_step that needs no launch: flags, pointers, sizes, the plan, the workspace.
static int check_append_step(const void* q, const void* K, const void* V, const void* k_new, const void* v_new,
                             const int32_t* lens, int flags, const float* o, const void* workspace, size_t workspace_bytes,
                             const int32_t* status, int b, int h, int m_max, int k, int v, Plan* plan) {
    if (flags & ~(MQA_STEP_ADVANCE | MQA_STEP_CHAINED | MQA_STEP_TEST_WRONG_GUESS | MQA_STEP_TEST_WITHHOLD_COPY)) return MQA_ERR_INVALID_ARG;
    int rc = check_step_args(q, K, V, lens, o, status, b, h, m_max, k, v);
    if (rc) return rc;
    if (!k_new || !v_new || !aligned16(k_new) || !aligned16(v_new)) return MQA_ERR_INVALID_ARG;
    *plan = make_plan(true, b, h, m_max);
    if (plan->units * (size_t)plan->n_splits > 0x7fffffffull) return MQA_ERR_UNSUPPORTED;
    return check_workspace(*plan, workspace, workspace_bytes);
}

static int append_step_impl(const void* q, void* K, void* V, const void* k_new, const void* v_new, int32_t* lens,
                            int flags, float* o, void* workspace, size_t workspace_bytes, int32_t* status, int b,
                            int h, int m_max, int k, int v, mqa_stream_t stream_, bool after_projection,
                            const Plan* checked = nullptr) {
    // (checked: the caller has run check_append_step on these very arguments and passes the plan it gave)
    Plan p;
    int rc = MQA_OK;
    if (checked) p = *checked;
    else if ((rc = check_append_step(q, K, V, k_new, v_new, lens, flags, o, workspace, workspace_bytes, status, b, h, m_max, k, v, &p))) return rc;
    const int advance = flags & MQA_STEP_ADVANCE;
    int early = after_projection ? kEarlyAfterProjection
                : !(flags & MQA_STEP_CHAINED) ? kEarlyNone
                : (flags & MQA_STEP_TEST_WRONG_GUESS) ? kEarlyChainedWrongGuess : kEarlyChained;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const bool withhold = (flags & MQA_STEP_TEST_WITHHOLD_COPY) != 0;
    if (p.kernel == Kernel::kUmma) {
        // copies started on a guess pay where the step is one launch over long shares (measured: 0.4-0.7 us gained with
        // up to 6 pieces per sequence, 0.3-2.5 us lost with more pieces, short shares or a second-pass kernel)
        if (early == kEarlyChained && !(p.merge_in_kernel && p.n_splits <= kGuessMaxPieces && p.chunk_rows >= kGuessMinShareRows))
            early = kEarlyNone;
        if (withhold) early |= kEarlyTestWithhold;
        // one launch: append inside the pass, pieces merged by the last CTA to deliver one, lens advanced at the end
        if (p.merge_in_kernel)
            return launch_umma_for<true>(p, q, K, V, lens, o, workspace, status, b, h, m_max, stream, true, k_new, v_new,
                                         advance ? lens : nullptr, early);
        rc = launch_umma_for<true>(p, q, K, V, lens, o, workspace, status, b, h, m_max, stream, false, k_new, v_new, nullptr,
                                   early);
        if (rc) return rc;
        return run_combine(true, lens, o, workspace, workspace_bytes, b, h, m_max, k, v, stream, 0, advance ? lens : nullptr);
    }
    // other plans: the same step as separate launches.  Without `advance` the append leaves lens alone and
    // the step is told that a sequence which took a row has one more row than lens says.
    if ((p.kernel == Kernel::kMma1 || p.kernel == Kernel::kMma2) && p.n_splits == 1) {
        // one CTA per sequence: it writes the row, attends and moves lens on, all in one launch
        // tiles below the prefix's last rows are fetched ahead of the wait (measured: 5.70 -> 5.45 us per step over the
        // 128 steps of a cache growing to 128 rows; nothing gained, 0.2 us lost, at 512 rows)
        if (early == kEarlyChained && m_max <= 8 * kTileRows && !withhold)
            return p.kernel == Kernel::kMma1
                       ? launch_mma<1, true>(p, q, K, V, lens, o, nullptr, nullptr, status, b, h, m_max, stream, 0, k_new, v_new,
                                             advance ? lens : nullptr)
                       : launch_mma<2, true>(p, q, K, V, lens, o, nullptr, nullptr, status, b, h, m_max, stream, 0, k_new, v_new,
                                             advance ? lens : nullptr);
        return p.kernel == Kernel::kMma1
                   ? launch_mma<1>(p, q, K, V, lens, o, nullptr, nullptr, status, b, h, m_max, stream, 0, k_new, v_new,
                                   advance ? lens : nullptr, withhold)
                   : launch_mma<2>(p, q, K, V, lens, o, nullptr, nullptr, status, b, h, m_max, stream, 0, k_new, v_new,
                                   advance ? lens : nullptr, withhold);
    }
    if (p.kernel == Kernel::kWide) {
        // many query rows: the CTA whose rows hold the new one writes it; one split per sequence moves lens on itself,
        // otherwise the second pass does.  One or two launches.
        float2* part_ml = partials_ml(workspace);
        float* part_acc = partials_acc(p, workspace);
        // (one split and one tile of 128 rows: the CTA moves lens on itself)
        const bool alone = p.n_splits == 1 && h <= kWideRows;
        rc = launch_wide(p, q, K, V, lens, o, part_ml, part_acc, status, b, h, m_max, stream, 0, k_new, v_new,
                         alone && advance ? lens : nullptr, withhold);
        if (rc || alone) return rc;
        if (p.n_splits == 1) {                                   // several row tiles read lens: moved on by a kernel of its own
            if (advance) launch_dependent(lens_advance_kernel, (unsigned)((b + 255) / 256), 256u, 0, stream, lens, b, m_max);
            return launch_status();
        }
        return run_combine(true, lens, o, workspace, workspace_bytes, b, h, m_max, k, v, stream, 0, advance ? lens : nullptr, true);
    }
    if ((p.kernel == Kernel::kMma1 || p.kernel == Kernel::kMma2) && p.n_splits > 1) {
        // fixed splits: the CTA whose rows hold the new one writes it; the second pass moves lens on.  Two launches.
        float2* part_ml = partials_ml(workspace);
        float* part_acc = partials_acc(p, workspace);
        rc = p.kernel == Kernel::kMma1
                 ? launch_mma<1>(p, q, K, V, lens, o, part_ml, part_acc, status, b, h, m_max, stream, 0, k_new, v_new, nullptr, withhold)
                 : launch_mma<2>(p, q, K, V, lens, o, part_ml, part_acc, status, b, h, m_max, stream, 0, k_new, v_new, nullptr, withhold);
        if (rc) return rc;
        return run_combine(true, lens, o, workspace, workspace_bytes, b, h, m_max, k, v, stream, 0, advance ? lens : nullptr, true);
    }
    rc = kv_cache_append(K, V, k_new, v_new, lens, 0, status, b, 1, m_max, k, v, stream_);
    if (rc) return rc;
    rc = run_split(true, q, K, V, lens, o, workspace, workspace_bytes, status, b, h, m_max, k, v, stream, 1);
    if (rc) return rc;
    rc = run_combine(true, lens, o, workspace, workspace_bytes, b, h, m_max, k, v, stream, 1);
    if (rc) return rc;
    if (advance) {
        launch_dependent(lens_advance_kernel, (unsigned)((b + 255) / 256), 256u, 0, stream, lens, b, m_max);
        return launch_status();
    }
    return MQA_OK;
}

int mqa_decode_append_step(const void* q, void* K, void* V, const void* k_new, const void* v_new, int32_t* lens,
                           int advance, float* o, void* workspace, size_t workspace_bytes, int32_t* status, int b,
                           int h, int m_max, int k, int v, mqa_stream_t stream) {
    return append_step_impl(q, K, V, k_new, v_new, lens, advance, o, workspace, workspace_bytes, status, b, h, m_max, k, v,
                            stream, false);
}

int mqa_decode_local_step(const void* q, void* K, void* V, const void* k_new, const void* v_new, int32_t* pos, int advance,
                          float* o, int32_t* status, int b, int h, int window, int k, int v, mqa_stream_t stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    int rc = check_step_args(q, K, V, pos, o, status, b, h, window, k, v);
    if (rc) return rc;
    if (!k_new || !v_new || !aligned16(k_new) || !aligned16(v_new)) return MQA_ERR_INVALID_ARG;
    if ((long long)b * window >= 0x7fffffffLL) return MQA_ERR_UNSUPPORTED;
    if (window <= kLocalMaxWindow) {
        // a warp per sequence: windows of a few tiles (the paper's is one), any number of heads
        static std::atomic<int> opted[kMaxDevices];
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return MQA_ERR_CUDA; }
        if (!opted[dev].load(std::memory_order_acquire)) {
            if (cudaFuncSetAttribute(mqa_decode_local_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kLocalSmemBytes) != cudaSuccess) {
                cudaGetLastError();
                return MQA_ERR_CUDA;
            }
            opted[dev].store(1, std::memory_order_release);
        }
        alignas(64) CUtensorMap map_k, map_v;
        if (!encode_cache_map(&map_k, K, (long long)b * window) || !encode_cache_map(&map_v, V, (long long)b * window)) return MQA_ERR_CUDA;
        launch_dependent(mqa_decode_local_kernel, (unsigned)((b + kLocalWarps - 1) / kLocalWarps), kLocalThreads, kLocalSmemBytes, stream,
                         map_k, map_v, static_cast<const uint32_t*>(q), static_cast<const uint4*>(k_new), static_cast<const uint4*>(v_new),
                         static_cast<uint4*>(K), static_cast<uint4*>(V), pos, o, status, b, h, window, advance ? 1 : 0);
        return launch_status();
    }
    return MQA_ERR_UNSUPPORTED;   // a window that long is the ordinary step's business
}

size_t mqa_host_staging_bytes(int b, int h, int k, int v) {
    if (b <= 0 || h <= 0 || k != kHeadDim || v != kHeadDim) return 0;
    return align256((size_t)b * h * k * 2) + 2 * align256((size_t)b * kHeadDim * 2) + align256((size_t)b * h * v * 4);
}

// The device's address of pinned host memory that it can reach (16-byte aligned), or null.
static const void* host_device_pointer(const void* host) {
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, host) == cudaSuccess && attr.type == cudaMemoryTypeHost && attr.devicePointer &&
        aligned16(attr.devicePointer))
        return attr.devicePointer;
    cudaGetLastError();
    return nullptr;
}

int mqa_decode_append_step_host(const void* q_host, const void* k_new_host, const void* v_new_host, float* o_host,
                                void* K, void* V, int32_t* lens, int advance, void* staging, size_t staging_bytes,
                                void* workspace, size_t workspace_bytes, int32_t* status, int b, int h, int m_max, int k,
                                int v, mqa_stream_t stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (!q_host || !k_new_host || !v_new_host || !o_host || !staging) return MQA_ERR_INVALID_ARG;
    if (!dims_ok(b, h, m_max) || k <= 0 || v <= 0 || !aligned16(staging)) return MQA_ERR_INVALID_ARG;
    if (k != kHeadDim || v != kHeadDim) return MQA_ERR_UNSUPPORTED;
    if (staging_bytes < mqa_host_staging_bytes(b, h, k, v)) return MQA_ERR_WORKSPACE_TOO_SMALL;
    const size_t q_bytes = (size_t)b * h * k * 2, row_bytes = (size_t)b * kHeadDim * 2, o_bytes = (size_t)b * h * v * 4;
    char* base = static_cast<char*>(staging);
    char* q_dev = base;
    char* k_dev = q_dev + align256(q_bytes);
    char* v_dev = k_dev + align256(row_bytes);
    float* o_dev = reinterpret_cast<float*>(v_dev + align256(row_bytes));
    // everything that can be refused is refused before the first copy is enqueued
    Plan plan;
    const int bad = check_append_step(q_dev, K, V, k_dev, v_dev, lens, advance, o_dev, workspace, workspace_bytes, status, b, h,
                                      m_max, k, v, &plan);
    if (bad) return bad;
    // the step's inputs.  Pinned memory that this device can address: a kernel fetches them, and the attention kernel
    // sets itself up and asks for its first stages while it does (what the layer step does behind its input projection).
    // Otherwise copy-engine transfers: one when the caller packed them back to back (256-byte aligned parts), else three.
    const char* qh = static_cast<const char*>(q_host);
    const void* q_map = host_device_pointer(q_host);
    const void* k_map = host_device_pointer(k_new_host);
    const void* v_map = host_device_pointer(v_new_host);
    const bool by_kernel = q_map && k_map && v_map && q_bytes / 16 <= 0xffffffffull;
    if (by_kernel) {
        const StageInPart pq = {static_cast<const uint4*>(q_map), reinterpret_cast<uint4*>(q_dev), (unsigned)(q_bytes / 16)};
        const StageInPart pk = {static_cast<const uint4*>(k_map), reinterpret_cast<uint4*>(k_dev), (unsigned)(row_bytes / 16)};
        const StageInPart pv = {static_cast<const uint4*>(v_map), reinterpret_cast<uint4*>(v_dev), (unsigned)(row_bytes / 16)};
        const size_t turns = (q_bytes / 16 + kStageInThreads - 1) / kStageInThreads;
        const unsigned grid = (unsigned)(turns < (size_t)(2 * sm_count()) ? (turns ? turns : 1) : 2 * sm_count());
        if (launch_dependent(stage_in_kernel, grid, (unsigned)kStageInThreads, 0, stream, pq, pk, pv) != cudaSuccess) {
            cudaGetLastError();
            return MQA_ERR_CUDA;
        }
    } else {
        const bool packed = static_cast<const char*>(k_new_host) == qh + align256(q_bytes) &&
                            static_cast<const char*>(v_new_host) == qh + align256(q_bytes) + align256(row_bytes);
        if (packed) {
            if (cudaMemcpyAsync(q_dev, qh, align256(q_bytes) + align256(row_bytes) + row_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess) {
                cudaGetLastError();
                return MQA_ERR_CUDA;
            }
        } else {
            if (cudaMemcpyAsync(q_dev, q_host, q_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
                cudaMemcpyAsync(k_dev, k_new_host, row_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
                cudaMemcpyAsync(v_dev, v_new_host, row_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess) {
                cudaGetLastError();
                return MQA_ERR_CUDA;
            }
        }
    }
    // the result: where o_host is pinned memory that this device can address, the kernels store o there themselves
    // (posted writes that overlap the end of the step); otherwise it goes through the staging buffer and a copy
    float* o_direct = static_cast<float*>(const_cast<void*>(host_device_pointer(o_host)));
    const int rc = append_step_impl(q_dev, K, V, k_dev, v_dev, lens, advance, o_direct ? o_direct : o_dev, workspace,
                                    workspace_bytes, status, b, h, m_max, k, v, stream_, by_kernel, &plan);
    if (rc || o_direct) return rc;
    if (cudaMemcpyAsync(o_host, o_dev, o_bytes, cudaMemcpyDeviceToHost, stream) != cudaSuccess) {
        cudaGetLastError();
        return MQA_ERR_CUDA;
    }
    return MQA_OK;
}

size_t mqa_layer_workspace_bytes(int b, int h, int d, int m_max, int k, int v) {
    if (!dims_ok(b, h, m_max) || d <= 0 || d % 128 != 0 || k != kHeadDim || v != kHeadDim) return 0;
    return layer_workspace(b, h, d, m_max).total;
}

int mqa_layer_decode_step(const void* x, const void* P_q, const void* P_k, const void* P_v, const void* P_o, void* K, void* V,
                          int32_t* lens, int advance, float* y, void* workspace, size_t workspace_bytes, int32_t* status,
                          int b, int h, int d, int m_max, int k, int v, mqa_stream_t stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (!x || !P_q || !P_k || !P_v || !P_o || !K || !V || !lens || !y || !workspace) return MQA_ERR_INVALID_ARG;
    if (!dims_ok(b, h, m_max) || d <= 0 || k <= 0 || v <= 0) return MQA_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(P_q) || !aligned16(P_k) || !aligned16(P_v) || !aligned16(P_o) || !aligned16(K) ||
        !aligned16(V) || !aligned16(y) || !aligned16(workspace) || !aligned4(lens) || !aligned4(status))
        return MQA_ERR_INVALID_ARG;
    if (k != kHeadDim || v != kHeadDim || d % 128 != 0 || (long long)h * d >= 0x7fffffffLL) return MQA_ERR_UNSUPPORTED;
    const LayerWorkspace w = layer_workspace(b, h, d, m_max);
    if (workspace_bytes < w.total) return MQA_ERR_WORKSPACE_TOO_SMALL;
    char* base = static_cast<char*>(workspace);
    void* q = base + w.q;
    void* k_new = base + w.k_new;
    void* v_new = base + w.v_new;
    float* o = reinterpret_cast<float*>(base + w.o);
    const int nb = b >= 128 ? 128 : (b > 64 ? 128 : (b > 32 ? 64 : (b > 16 ? 32 : 16)));
    int rc;
    switch (nb) {
        case 16: rc = launch_projections_in<16>(x, P_q, P_k, P_v, q, k_new, v_new, status, b, h, d, stream); break;
        case 32: rc = launch_projections_in<32>(x, P_q, P_k, P_v, q, k_new, v_new, status, b, h, d, stream); break;
        case 64: rc = launch_projections_in<64>(x, P_q, P_k, P_v, q, k_new, v_new, status, b, h, d, stream); break;
        default: rc = launch_projections_in<128>(x, P_q, P_k, P_v, q, k_new, v_new, status, b, h, d, stream); break;
    }
    if (rc) return rc;
    rc = append_step_impl(q, K, V, k_new, v_new, lens, advance ? MQA_STEP_ADVANCE : 0, o, base + w.step, w.total - w.step, status,
                          b, h, m_max, k, v, stream_, true);
    if (rc) return rc;
    switch (nb) {
        case 16: return launch_projection_out<16>(P_o, o, y, status, b, h, d, stream);
        case 32: return launch_projection_out<32>(P_o, o, y, status, b, h, d, stream);
        case 64: return launch_projection_out<64>(P_o, o, y, status, b, h, d, stream);
        default: return launch_projection_out<128>(P_o, o, y, status, b, h, d, stream);
    }
}

size_t mqa_workspace_bytes(int b, int h, int m_max, int k, int v) {
    if (!dims_ok(b, h, m_max) || k != kHeadDim || v != kHeadDim) return 0;
    const size_t a = plan_workspace_bytes(make_plan(true, b, h, m_max));
    const size_t c = plan_workspace_bytes(make_plan(false, b, h, m_max));
    return a > c ? a : c;
}

int mqa_append_step_launches(int b, int h, int m_max, int k, int v) {
    if (!dims_ok(b, h, m_max) || k != kHeadDim || v != kHeadDim) return 0;
    const Plan p = make_plan(true, b, h, m_max);
    if (p.merge_in_kernel) return 1;                   // append, pass, merge and lens advance in one kernel
    if ((p.kernel == Kernel::kMma1 || p.kernel == Kernel::kMma2) && p.n_splits == 1) return 1;   // one CTA per sequence does it all
    if (p.stream()) return 2;                          // pass with the append inside, second pass
    if (p.kernel == Kernel::kMma1 || p.kernel == Kernel::kMma2) return 2;   // fixed splits: the same two
    if (p.kernel == Kernel::kWide) return p.n_splits == 1 && h <= kWideRows ? 1 : 2;
    return 2 + (p.n_splits > 1 ? 1 : 0) + 1;           // append, pass, (second pass), lens advance
}

int mqa_plan_splits(int multi_query, int b, int h, int m_max, int k, int v, int* chunk_rows) {
    if (!dims_ok(b, h, m_max) || k != kHeadDim || v != kHeadDim) return 0;
    const Plan p = make_plan(multi_query != 0, b, h, m_max);
    if (chunk_rows) *chunk_rows = p.chunk_rows;
    return p.n_splits;
}

// ---- the batched form (prefill) ---------------------------------------------------------------------------------
static int check_prefill_dims(int b, int h, int n, int m_max, int k, int v) {
    if (!dims_ok(b, h, m_max) || n <= 0 || k <= 0 || v <= 0) return MQA_ERR_INVALID_ARG;
    if (k != kHeadDim || v != kHeadDim || n > m_max) return MQA_ERR_UNSUPPORTED;
    const long long ctas = (long long)((n + kPfRows - 1) / kPfRows) * b * ((h + 1) / 2);
    if ((long long)b * m_max >= 0x7fffffffLL || (long long)b * h * n >= 0x7fffffffLL - kPfRows || ctas >= 0x7fffffffLL) return MQA_ERR_UNSUPPORTED;
    return MQA_OK;
}

size_t mqa_prefill_workspace_bytes(int b, int h, int n, int m_max, int k, int v) {
    return check_prefill_dims(b, h, n, m_max, k, v) == MQA_OK ? 16 : 0;     // (the kernel keeps everything on chip)
}

int mqa_prefill_attention(const void* Q, const void* K, const void* V, const int32_t* start, float* O, void* workspace,
                          size_t workspace_bytes, int32_t* status, int b, int h, int n, int m_max, int k, int v,
                          mqa_stream_t stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (!Q || !K || !V || !O || !workspace) return MQA_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(workspace) || !aligned4(start) ||
        !aligned4(status))
        return MQA_ERR_INVALID_ARG;
    const int rc = check_prefill_dims(b, h, n, m_max, k, v);
    if (rc) return rc;
    if (workspace_bytes < mqa_prefill_workspace_bytes(b, h, n, m_max, k, v)) return MQA_ERR_WORKSPACE_TOO_SMALL;
    static std::atomic<int> opt_in[kMaxDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return MQA_ERR_CUDA; }
    if (!opt_in[dev].load(std::memory_order_acquire)) {
        if (cudaFuncSetAttribute(mqa_prefill_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPfSmemBytes) != cudaSuccess) {
            cudaGetLastError();
            return MQA_ERR_CUDA;
        }
        opt_in[dev].store(1, std::memory_order_release);
    }
    // a unit of work per (tile of 128 positions, pair of heads, sequence); the last tile of a head may be partly filled.
    // One CTA per SM walks the units, longest first.
    const long long ctas = (long long)((n + kPfRows - 1) / kPfRows) * b * ((h + 1) / 2);
    const unsigned grid = (unsigned)(ctas < sm_count() ? ctas : sm_count());
    alignas(64) CUtensorMap map_q, map_k, map_v;
    if (!encode_cache_map(&map_q, Q, (long long)b * h * n, kPfRows) || !encode_cache_map(&map_k, K, (long long)b * m_max, kPfRows) ||
        !encode_cache_map(&map_v, V, (long long)b * m_max, kPfRows))
        return MQA_ERR_CUDA;
    launch_dependent(mqa_prefill_kernel, grid, (unsigned)kPfThreads, (size_t)kPfSmemBytes, stream, map_q, map_k, map_v, start, O,
                     status, b, h, n, m_max, (int)ctas);
    return launch_status();
}

int mqa_set_test_withhold_copy(int on) {
    const int value = on ? 1 : 0;
    if (cudaMemcpyToSymbol(g_test_withhold, &value, sizeof value) != cudaSuccess) {
        cudaGetLastError();
        return MQA_ERR_CUDA;
    }
    return MQA_OK;
}

int mqa_set_wait_limit_cycles(long long cycles) {
    const long long value = cycles > 0 ? cycles : kWaitLimitCycles;
    if (cudaMemcpyToSymbol(g_wait_limit_cycles, &value, sizeof value) != cudaSuccess) {
        cudaGetLastError();
        return MQA_ERR_CUDA;
    }
    return MQA_OK;
}

const char* mqa_plan_kernel_name(int multi_query, int whole_step, int b, int h, int m_max, int k, int v) {
    if (!dims_ok(b, h, m_max) || k != kHeadDim || v != kHeadDim) return "";
    const Plan p = make_plan(multi_query != 0, b, h, m_max);
    switch (p.kernel) {
        case Kernel::kUmma: {
            const bool guess = whole_step && p.merge_in_kernel && p.n_splits <= kGuessMaxPieces && p.chunk_rows >= kGuessMinShareRows;
            if (h <= 16) return !whole_step ? "mqa_decode_stream_umma_kernel<16>" : guess ? "mqa_decode_stream_umma_kernel<16, fused, guess>" : "mqa_decode_stream_umma_kernel<16, fused>";
            return !whole_step ? "mqa_decode_stream_umma_kernel<32>" : guess ? "mqa_decode_stream_umma_kernel<32, fused, guess>" : "mqa_decode_stream_umma_kernel<32, fused>";
        }
        case Kernel::kMma1: return "mqa_decode_split_mma_kernel<1>";
        case Kernel::kMma2: return "mqa_decode_split_mma_kernel<2>";
        case Kernel::kWide: return "mqa_decode_wide_kernel";
        default: return "decode_split_simt_kernel";
    }
}

const char* mqa_status_string(int code) {
    switch (code) {
        case MQA_OK: return "ok";
        case MQA_ERR_INVALID_ARG: return "invalid argument (null or misaligned pointer, non-positive dimension)";
        case MQA_ERR_UNSUPPORTED: return "unsupported configuration (k and v must be 128)";
        case MQA_ERR_WORKSPACE_TOO_SMALL: return "workspace too small (see mqa_workspace_bytes)";
        case MQA_ERR_CUDA: return "CUDA launch error";
        case MQA_ERR_STATIC_SCRATCH_TOO_SMALL:
            return "these sizes need more scratch than the built-in array of mqa_decode_step_noalloc";
        default: return "unknown status code";
    }
}

}  // extern "C"
