// spark_decode_attn_noalloc: the decode step for callers that cannot allocate device memory.
//
// Some hosts of this library run where cudaMalloc is off limits: inside a serving loop whose memory
// was carved up once at start-up, inside a plug-in that is handed tensors but no allocator, or under a
// framework that forbids allocation while it records work.  Such a caller can still pass inputs and
// outputs, but has nowhere to get the scratch that split decoding needs for its partial results and
// arrival tickets.  This entry point brings its own: a fixed array in device memory that is part of
// the loaded library image (every GPU that loads the library holds it until the process exits).
//
// The array's name is only a host-side handle.  Its device address is looked up once per device with
// cudaGetSymbolAddress (with that device current) and that address is what the kernel receives.
#include <mutex>

#include "spark_common.cuh"

namespace spark {

// Largest problem the built-in scratch serves: batch * n_kv_heads <= 64 (any G <= 8).
constexpr int kNoAllocMaxUnits = 64;
constexpr size_t kNoAllocScratchBytes =
    kWorkspaceHeader + 256 /* tickets */ +
    static_cast<size_t>(kMaxCtas + kNoAllocMaxUnits) * kMaxGroup * (kHeadDim + 4) * sizeof(float);   // ~1.3 MB

static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

constexpr int kMaxDevices = 64;
static std::mutex g_setup_mutex;
static void* g_scratch_addr[kMaxDevices] = {};

// Device address of the scratch array on the current device (looked up on first use per device).
static spark_status noalloc_scratch(void** out)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SPARK_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[dev]) {
        void* addr = nullptr;
        if (cudaGetSymbolAddress(&addr, g_noalloc_scratch) != cudaSuccess || !addr) return SPARK_ERR_CUDA;
        g_scratch_addr[dev] = addr;
    }
    *out = g_scratch_addr[dev];
    return SPARK_OK;
}

}  // namespace spark

using namespace spark;

extern "C" spark_status spark_decode_attn_noalloc(const spark_params* p, const void* q, const void* pages,
                                                  const int32_t* block_table, int32_t max_blocks,
                                                  const int32_t* packed_lens, const float* qnorm,
                                                  float* out, float* lse, spark_stream_t stream)
{
    spark_status st = check_params(p);
    if (st != SPARK_OK) return st;
    if (!q || !pages || !packed_lens || !qnorm || !out) return SPARK_ERR_NULL;
    if (max_blocks < 0 || max_blocks > INT32_MAX / kPageTokens) return SPARK_ERR_BAD_SHAPE;
    if ((reinterpret_cast<uintptr_t>(pages) & 15) || (reinterpret_cast<uintptr_t>(q) & 15) ||
        (reinterpret_cast<uintptr_t>(qnorm) & 15) || (reinterpret_cast<uintptr_t>(out) & 15) ||
        (reinterpret_cast<uintptr_t>(lse) & 3))
        return SPARK_ERR_BAD_SHAPE;
    if (!block_table && static_cast<int64_t>(p->batch) * p->n_kv_heads * max_blocks > p->n_pool_pages)
        return SPARK_ERR_BAD_SHAPE;
    // the built-in scratch has a fixed size: refuse anything it cannot hold
    if (static_cast<int64_t>(p->batch) * p->n_kv_heads > kNoAllocMaxUnits ||
        decode_workspace_bytes(*p) > kNoAllocScratchBytes)
        return SPARK_ERR_WORKSPACE;
    void* scratch = nullptr;
    st = noalloc_scratch(&scratch);
    if (st != SPARK_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // status word and tickets must start at zero; the array keeps whatever the last call left
    if (cudaMemsetAsync(scratch, 0, kWorkspaceHeader + 256, s) != cudaSuccess) return SPARK_ERR_CUDA;
    int launches = 0;
    return launch_decode(*p, q, pages, block_table, max_blocks, packed_lens, qnorm, out, lse, scratch,
                         kNoAllocScratchBytes, s, &launches);
}
