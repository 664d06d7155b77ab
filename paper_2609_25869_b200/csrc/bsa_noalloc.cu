// Mask statistics without any allocation: for callers that must not touch the CUDA allocator.
//
// The regular path (bsa_plan_create) sizes its buffers from the request and takes them from the
// stream-ordered allocator.  Some hosts cannot do that: a serving process that handed the whole
// device to its own memory pool at start-up, a plug-in running under somebody else's allocator
// policy, a control loop in which a cudaMalloc (an implicit device-wide synchronisation, and a
// call that can fail late) is not acceptable.  For them this file offers the mask-state statistics
// kernel with its scratch (one counter per mask row plus the three accumulators) in a fixed
// device-resident array that lives as long as the library is loaded.
#include <atomic>

#include "bsa_common.h"

namespace bsa {
namespace {

constexpr int kAccumBytes = 256;  // accumulators (MaskStatsDev) in front, 256-byte aligned rows behind
constexpr size_t kScratchBytes = kAccumBytes + sizeof(int32_t) * (size_t)BSA_NOALLOC_MAX_ROWS;

// Scratch of the no-allocation entry point: [accumulators | row_nnz[BSA_NOALLOC_MAX_ROWS]].
// In HOST code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

// Device address of the array, per device.  Host threads that make their first call on a device at the same time
// all resolve the same address and store the same value.
std::atomic<unsigned char*> g_scratch_addr[kMaxDevices];

// Copies the accumulators to the caller's buffer and counts rows without any active block.
__global__ void __launch_bounds__(256) noalloc_finalize_kernel(const MaskStatsDev* stats, const int32_t* row_nnz,
                                                                int nrows, long long* out) {
    __shared__ int warp_cnt[8];
    int empty = 0;
    for (int i = threadIdx.x; i < nrows; i += blockDim.x) empty += (row_nnz[i] == 0);
    for (int o = 16; o > 0; o >>= 1) empty += __shfl_down_sync(0xffffffffu, empty, o);
    if ((threadIdx.x & 31) == 0) warp_cnt[threadIdx.x >> 5] = empty;
    __syncthreads();
    if (threadIdx.x == 0) {
        int tot = 0;
        for (int w = 0; w < 8; ++w) tot += warp_cnt[w];
        out[0] = (long long)stats->nnz;
        out[1] = (long long)stats->in_runs;
        out[2] = (long long)stats->max_row_nnz;
        out[3] = tot;
    }
}

}  // namespace
}  // namespace bsa

using namespace bsa;

extern "C" bsa_status_t bsa_mask_stats_noalloc(const uint8_t* mask_dev, int heads, int nQb, int nKb,
                                               int64_t* stats_out_dev, void* stream_v) {
    if (!mask_dev || !stats_out_dev || heads <= 0 || nQb <= 0 || nKb <= 0) return BSA_ERR_INVALID_ARG;
    const int64_t nrows = (int64_t)heads * nQb;
    if (nrows > BSA_NOALLOC_MAX_ROWS) return BSA_ERR_UNSUPPORTED;  // scratch holds one counter per mask row
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_v);
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return BSA_ERR_CUDA;
    unsigned char* base = g_scratch_addr[dev].load(std::memory_order_acquire);
    if (!base) {
        // Set-up, once per device, with that device current: resolve the array's device address.  With CUDA's lazy
        // module loading this is also the moment the driver loads this file's module onto the device and reserves
        // the array there, which is why it can still fail, and why it belongs at start-up.
        void* addr = nullptr;
        if (cudaGetSymbolAddress(&addr, g_noalloc_scratch) != cudaSuccess || !addr) return BSA_ERR_CUDA;
        base = static_cast<unsigned char*>(addr);
        g_scratch_addr[dev].store(base, std::memory_order_release);
    }
    MaskStatsDev* stats = reinterpret_cast<MaskStatsDev*>(base);
    int32_t* row_nnz = reinterpret_cast<int32_t*>(base + kAccumBytes);
    // the array keeps the previous call's contents: the accumulators must start at zero
    // (row_nnz is fully overwritten for the rows in use)
    if (cudaMemsetAsync(stats, 0, kAccumBytes, stream) != cudaSuccess) return BSA_ERR_CUDA;
    if (launch_mask_row_stats(mask_dev, (int)nrows, nKb, row_nnz, stats, stream) != cudaSuccess) return BSA_ERR_CUDA;
    noalloc_finalize_kernel<<<1, 256, 0, stream>>>(stats, row_nnz, (int)nrows,
                                                   reinterpret_cast<long long*>(stats_out_dev));
    count_launch();
    return cudaGetLastError() == cudaSuccess ? BSA_OK : BSA_ERR_CUDA;
}
