// mqa_decode_step_noalloc: the multi-query decode step for callers that cannot hand the
// library a workspace because they cannot allocate one.
//
// Who that is: code that runs inside someone else's executor -- an inference-server plugin, a
// custom op in a framework whose memory plan was frozen at start-up, a real-time decode loop --
// where every buffer was planned ahead and cudaMalloc is off the table, either because it
// would stall every stream of the device while it runs, or because the host application has
// already reserved all device memory and the call would simply fail.  Such a caller has its
// inputs and outputs, but no spare scratch buffer and no allocator.
//
// The scratch for the per-piece partial results therefore lives in this library's own image:
// a fixed array in device global memory, reserved on every GPU that loads the library for as
// long as the process lives.  The step itself is the same pair of kernels that
// mqa_decode_step launches; only the home of the scratch differs.
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "../../include/mqa_decode.h"

namespace {

// 8 MiB: covers every multi-query shape this build is measured on (the largest, 256 sequences
// of 32768 rows with 16 heads, needs 3.4 MB) with room to spare, and stays small next to a
// 180 GB device.
constexpr size_t kStaticScratchBytes = MQA_NOALLOC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::atomic<void*> g_scratch_address[kMaxDevices];

// Device address of the array on the CURRENT device.  In host code the array's name is only a
// handle for the runtime, not a pointer a kernel could use; the address has to be asked for,
// once per device, with that device current.
int static_scratch(void** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        cudaGetLastError();
        return MQA_ERR_CUDA;
    }
    void* p = g_scratch_address[dev].load(std::memory_order_acquire);
    if (!p) {
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return MQA_ERR_CUDA;
        }
        g_scratch_address[dev].store(p, std::memory_order_release);
    }
    *out = p;
    return MQA_OK;
}

}  // namespace

extern "C" int mqa_decode_step_noalloc(const void* q, const void* K, const void* V, const int32_t* lens, float* o,
                                       int32_t* status, int b, int h, int m_max, int k, int v,
                                       mqa_stream_t stream) {
    // Arguments the ordinary entry point would refuse are refused by it below, before any launch;
    // here only the one extra condition is checked: the plan's scratch must fit the fixed array.
    if (b > 0 && h > 0 && m_max > 0 && k == 128 && v == 128 &&
        mqa_workspace_bytes(b, h, m_max, k, v) > kStaticScratchBytes)
        return MQA_ERR_STATIC_SCRATCH_TOO_SMALL;
    void* scratch = nullptr;
    const int rc = static_scratch(&scratch);
    if (rc != MQA_OK) return rc;
    return mqa_decode_step(q, K, V, lens, o, scratch, kStaticScratchBytes, status, b, h, m_max, k, v, stream);
}
