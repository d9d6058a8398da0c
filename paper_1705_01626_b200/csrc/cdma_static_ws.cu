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
// device address is looked up with cudaGetSymbolAddress, with the calling
// device current, and that pointer is what the kernel receives.
#include "zvc_common.cuh"

namespace {

// Largest tensor the built-in workspace serves: 2^28 elements (1 GiB of fp32).
constexpr uint64_t kStaticMaxElements = 1ull << 28;
constexpr uint64_t kStaticWsBytes =
    (cdma::kWsHeaderBytes + 8 * cdma::kDescStride * ((kStaticMaxElements / cdma::kChunk + cdma::kTileChunks - 1) / cdma::kTileChunks) +
     255) / 256 * 256;                                   // 1,048,832 bytes

static __device__ __align__(256) unsigned char g_static_ws[kStaticWsBytes];

// Device address of the workspace on the current device.  Looked up on every call
// (after the first time on a device this is a table look-up inside the runtime),
// so that a pointer from before a cudaDeviceReset is never reused.  The first
// look-up on a device loads this module, which is when the array's memory is
// reserved there: it can fail for lack of memory on a full device.
int static_ws_for_current_device(uint64_t** out) {
    void* p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, g_static_ws);
    if (e != cudaSuccess || p == nullptr) {
        (void)cudaGetLastError();
        return e == cudaErrorMemoryAllocation ? CDMA_ERR_OUT_OF_MEMORY : CDMA_ERR_CUDA;
    }
    *out = static_cast<uint64_t*>(p);
    return CDMA_OK;
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
    uint64_t* ws = nullptr;
    const int ws_status = static_ws_for_current_device(&ws);
    if (ws_status != CDMA_OK) return -static_cast<int64_t>(ws_status);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

    // The array keeps whatever the previous call left.  Nothing in it has to start
    // at zero: the look-back descriptors of this launch carry a tag of their own,
    // and the result words are written by the launch before they are read.
    uint64_t result[2] = {0, 0};
    LaunchCtl ctl = make_launch_ctl(nullptr);            // result words come back by the copy below
    if (n == 0) {
        if (cudaMemsetAsync(d_table, 0, 8, stream) != cudaSuccess || cudaStreamSynchronize(stream) != cudaSuccess)
            return -static_cast<int64_t>(CDMA_ERR_CUDA);
        return 0;
    }
    // a source in page-locked host memory is read over the host link: no L2 prefetches for it
    if (launch_zvc_compress(d_src, n, s, d_dst, dst_capacity, d_table, ws, ctl, stream, !in_host_memory(d_src)) !=
        cudaSuccess)
        return -static_cast<int64_t>(CDMA_ERR_CUDA);
    if (cudaMemcpyAsync(result, ws + kWsBytes, 16, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess)
        return -static_cast<int64_t>(CDMA_ERR_CUDA);
    if (result[1] != 0) return -static_cast<int64_t>(result[1]);
    return static_cast<int64_t>(result[0]);
}
