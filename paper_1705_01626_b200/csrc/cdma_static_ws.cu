// cdma_zvc_compress_static_ws: the compression call for callers that cannot
// allocate device memory.
//
// Some callers of this library are not allowed to call cudaMalloc (or to ask a
// framework allocator for memory) at the point where they need to compress:
// code running inside a memory manager's own eviction path, where an allocation
// could re-enter the manager or fail because the device is full (which is
// exactly when activations get offloaded); plug-ins that are handed buffers by
// their host application and own none; start-up and tear-down hooks that run
// when the allocator is not usable.  They can pass the tensor, the payload
// buffer and the table, but they have no place to get the kernel's workspace
// from.  For them the workspace lives here, in a file-scope device array that
// every GPU loading this library holds until the process exits.
//
// Host code must not hand the array's name to a kernel: in host code the name
// is only a host-side stand-in for the symbol, not a device address.  The
// device address is looked up once per device with cudaGetSymbolAddress, with
// that device current, and that pointer is what the kernel receives.
#include <mutex>

#include "zvc_common.cuh"

namespace {

// Largest tensor the built-in workspace serves: 2^28 elements (1 GiB of fp32).
constexpr uint64_t kStaticMaxElements = 1ull << 28;
constexpr uint64_t kStaticWsBytes =
    (cdma::kWsHeaderBytes + 8 * cdma::kDescStride * ((kStaticMaxElements / cdma::kChunk + cdma::kTileChunks - 1) / cdma::kTileChunks) +
     255) / 256 * 256;                                   // 1,048,832 bytes

static __device__ __align__(256) unsigned char g_static_ws[kStaticWsBytes];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
uint64_t* g_ws_ptr[kMaxDevices] = {};

// Device address of the workspace on the current device; looked up on the
// first call made with that device current.  Returns nullptr on failure.
uint64_t* static_ws_for_current_device() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (g_ws_ptr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_ws) != cudaSuccess || p == nullptr) {
            cudaGetLastError();
            return nullptr;
        }
        g_ws_ptr[dev] = static_cast<uint64_t*>(p);
    }
    return g_ws_ptr[dev];
}

inline bool aligned_to(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

}  // namespace

extern "C" int64_t cdma_zvc_compress_static_ws(const void* d_src, uint64_t n, int dtype, int layout,
                                               void* d_dst, uint64_t dst_capacity, uint64_t* d_table,
                                               void* cuda_stream) {
    using namespace cdma;
    const uint32_t s = cdma_dtype_size(dtype);
    if (s == 0) return -static_cast<int64_t>(CDMA_ERR_UNSUPPORTED_DTYPE);
    if (layout != CDMA_NCHW && layout != CDMA_NHWC && layout != CDMA_CHWN)
        return -static_cast<int64_t>(CDMA_ERR_UNSUPPORTED_LAYOUT);
    // the built-in workspace has a fixed size: larger tensors are refused, never truncated
    if (n > kStaticMaxElements) return -static_cast<int64_t>(CDMA_ERR_BUFFER_TOO_SMALL);
    if (d_table == nullptr || (n != 0 && d_src == nullptr) || (dst_capacity != 0 && d_dst == nullptr))
        return -static_cast<int64_t>(CDMA_ERR_INVALID_ARG);
    if (!aligned_to(d_src, 16) || !aligned_to(d_dst, 16) || !aligned_to(d_table, 8))
        return -static_cast<int64_t>(CDMA_ERR_ALIGNMENT);
    {
        const uintptr_t a0 = reinterpret_cast<uintptr_t>(d_src), b0 = reinterpret_cast<uintptr_t>(d_dst);
        if (n != 0 && dst_capacity != 0 && a0 < b0 + dst_capacity && b0 < a0 + n * s)
            return -static_cast<int64_t>(CDMA_ERR_INVALID_ARG);
    }
    uint64_t* ws = static_ws_for_current_device();
    if (ws == nullptr) return -static_cast<int64_t>(CDMA_ERR_CUDA);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

    // The array keeps whatever the previous call left: ticket, result words and
    // the descriptors of every tile this call uses must start at zero.
    if (cudaMemsetAsync(ws, 0, kWsHeaderBytes + 8 * kDescStride * num_tiles_of(n), stream) != cudaSuccess)
        return -static_cast<int64_t>(CDMA_ERR_CUDA);
    if (n == 0) {
        if (cudaMemsetAsync(d_table, 0, 8, stream) != cudaSuccess) return -static_cast<int64_t>(CDMA_ERR_CUDA);
    } else if (launch_zvc_compress(d_src, n, s, d_dst, dst_capacity, d_table, ws, stream) != cudaSuccess) {
        return -static_cast<int64_t>(CDMA_ERR_CUDA);
    }
    uint64_t result[2] = {0, 0};
    if (cudaMemcpyAsync(result, ws + kWsBytes, 16, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess)
        return -static_cast<int64_t>(CDMA_ERR_CUDA);
    if (result[1] != 0) return -static_cast<int64_t>(result[1]);
    return static_cast<int64_t>(result[0]);
}
