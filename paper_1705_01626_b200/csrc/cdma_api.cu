// extern "C" codec entry points: argument checking, launch, result hand-over.
// Declarations and contracts are in include/cdma.h.
#include <atomic>
#include <chrono>
#include <cstring>
#include <mutex>
#include <random>
#include <utility>
#include <vector>

#include "zvc_common.cuh"

namespace cdma {

static inline bool aligned_u64(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 7) == 0; }

static std::atomic<uint64_t> g_kernel_launches{0};
void count_kernel_launch() { g_kernel_launches.fetch_add(1, std::memory_order_relaxed); }

// One-shot pair of events that the next codec kernel launch of this thread is bracketed with.
static thread_local cudaEvent_t t_time_start = nullptr;
static thread_local cudaEvent_t t_time_stop = nullptr;
void timing_before_launch(cudaStream_t stream) {
    if (t_time_start != nullptr) cudaEventRecord(t_time_start, stream);
}
void timing_after_launch(cudaStream_t stream) {
    if (t_time_stop != nullptr) cudaEventRecord(t_time_stop, stream);
    t_time_start = nullptr;
    t_time_stop = nullptr;
}

// Tags of launches: a process-wide counter started at a value that differs from
// run to run, so that a workspace written by another process (or left dirty by the
// caller) does not hold a matching tag either.
static std::atomic<uint64_t> g_next_tag{0};
static uint64_t fresh_tag() {
    uint64_t t = g_next_tag.load(std::memory_order_relaxed);
    if (t == 0) {
        const uint64_t seed = (static_cast<uint64_t>(std::chrono::steady_clock::now().time_since_epoch().count()) *
                               0x9E3779B97F4A7C15ull) ^ (static_cast<uint64_t>(std::random_device{}()) << 20);
        uint64_t expected = 0;
        g_next_tag.compare_exchange_strong(expected, (seed & kTagMask) | 1ull);
    }
    do {
        t = g_next_tag.fetch_add(1, std::memory_order_relaxed) & kTagMask;
    } while (t == 0);
    return t;
}

// True when p lies in page-locked host memory (which kernels reach over the host link).
bool in_host_memory(const void* p) {
    cudaPointerAttributes attr;
    if (p == nullptr || cudaPointerGetAttributes(&attr, p) != cudaSuccess) {
        (void)cudaGetLastError();
        return false;
    }
    return attr.type == cudaMemoryTypeHost;
}

// Page-locked host memory is addressable from the device, so the kernel that knows
// the result stores the two words there itself: no extra operation on the stream.
LaunchCtl make_launch_ctl(uint64_t* h_result) {
    LaunchCtl ctl{fresh_tag(), nullptr, kWaitLimitNs, kNoTile};
    cudaPointerAttributes attr;
    if (h_result != nullptr && cudaPointerGetAttributes(&attr, h_result) == cudaSuccess &&
        attr.type == cudaMemoryTypeHost && attr.devicePointer != nullptr && aligned_u64(attr.devicePointer))
        ctl.result_out = static_cast<uint64_t*>(attr.devicePointer);
    else
        (void)cudaGetLastError();   // an unregistered pointer is not an error here
    return ctl;
}

// Any other destination takes an ordinary 16-byte copy behind the kernel.
cudaError_t finish_result(const uint64_t* d_ws, const LaunchCtl& ctl, uint64_t* h_result, cudaStream_t stream) {
    if (ctl.result_out != nullptr) return cudaSuccess;
    return cudaMemcpyAsync(h_result, d_ws + kWsBytes, 16, cudaMemcpyDeviceToHost, stream);
}

cudaError_t result_without_kernel(uint64_t* d_ws, uint64_t bytes, uint64_t* h_result, cudaStream_t stream) {
    // only n = 0 comes here, where bytes is 0 too: both words are zero
    (void)bytes;
    const cudaError_t e = cudaMemsetAsync(d_ws + kWsBytes, 0, 16, stream);
    if (e != cudaSuccess) return e;
    return cudaMemcpyAsync(h_result, d_ws + kWsBytes, 16, cudaMemcpyDeviceToHost, stream);
}

cudaError_t opt_in_shared_memory(const void* kernel, uint32_t bytes) {
    static std::mutex mu;
    static std::vector<std::pair<const void*, int>> done;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(mu);
    for (const auto& d : done)
        if (d.first == kernel && d.second == dev) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes));
    if (e == cudaSuccess) done.emplace_back(kernel, dev);
    return e;
}

static inline bool aligned(const void* p, uintptr_t a) {
    return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0;
}
static inline bool overlaps(const void* a, uint64_t na, const void* b, uint64_t nb) {
    const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
    return na != 0 && nb != 0 && a0 < b0 + nb && b0 < a0 + na;
}

static int check_common(uint64_t n, int dtype, int layout, const void* dense, const void* packed,
                        const uint64_t* table, const void* ws, uint64_t ws_bytes) {
    const uint32_t s = cdma_dtype_size(dtype);
    if (s == 0) return CDMA_ERR_UNSUPPORTED_DTYPE;
    if (layout != CDMA_NCHW && layout != CDMA_NHWC && layout != CDMA_CHWN)
        return CDMA_ERR_UNSUPPORTED_LAYOUT;
    if (n > (1ull << 40)) return CDMA_ERR_INVALID_ARG;
    if (table == nullptr || ws == nullptr) return CDMA_ERR_INVALID_ARG;
    if (n != 0 && dense == nullptr) return CDMA_ERR_INVALID_ARG;
    if (!aligned(dense, 16) || !aligned(packed, 16) || !aligned(ws, 16) || !aligned(table, 8))
        return CDMA_ERR_ALIGNMENT;
    if (ws_bytes < cdma_zvc_workspace_bytes(n, dtype)) return CDMA_ERR_BUFFER_TOO_SMALL;
    return CDMA_OK;
}

}  // namespace cdma

using namespace cdma;

extern "C" {

const char* cdma_status_string(int status) {
    switch (status < 0 ? -status : status) {
        case CDMA_OK: return "ok";
        case CDMA_ERR_INVALID_ARG: return "invalid argument";
        case CDMA_ERR_UNSUPPORTED_DTYPE: return "unsupported dtype";
        case CDMA_ERR_UNSUPPORTED_LAYOUT: return "unsupported layout";
        case CDMA_ERR_ALIGNMENT: return "buffer not 16-byte aligned";
        case CDMA_ERR_BUFFER_TOO_SMALL: return "buffer too small";
        case CDMA_ERR_CORRUPT_STREAM: return "corrupt stream or offset table";
        case CDMA_ERR_TIMEOUT: return "device-side wait ran out";
        case CDMA_ERR_CUDA: return "CUDA runtime error";
        case CDMA_ERR_OUT_OF_MEMORY: return "out of memory";
        case CDMA_ERR_BAD_TICKET: return "unknown or consumed ticket";
        default: return "unknown status";
    }
}

uint32_t cdma_dtype_size(int dtype) {
    switch (dtype) {
        case CDMA_F32: return 4;
        case CDMA_F16: return 2;
        case CDMA_BF16: return 2;
        case CDMA_U8: return 1;
        default: return 0;
    }
}

uint64_t cdma_zvc_max_compressed_bytes(uint64_t n, int dtype) {
    const uint64_t s = cdma_dtype_size(dtype);
    if (s == 0) return 0;
    const uint64_t bytes = 4 * ((n + kWindow - 1) / kWindow) + s * n;
    return (bytes + 15) & ~15ull;
}

uint64_t cdma_zvc_table_entries(uint64_t n) { return num_chunks_of(n) + 1; }

uint64_t cdma_zvc_workspace_bytes(uint64_t n, int dtype) {
    (void)dtype;
    const uint64_t bytes = kWsHeaderBytes + 8 * kDescStride * num_tiles_of(n);
    return (bytes + 255) & ~255ull;
}

// Launch and result hand-over shared by every compression entry point.
static int compress_launch(const void* d_src, uint64_t n, int dtype, bool relu, void* d_relu_out, void* d_dst,
                           uint64_t dst_capacity, uint64_t* d_table, uint64_t* ws, const LaunchCtl& ctl,
                           cudaStream_t stream, uint64_t* h_result) {
    const uint32_t s = cdma_dtype_size(dtype);
    if (n == 0) {
        if (cudaMemsetAsync(d_table, 0, 8, stream) != cudaSuccess) return CDMA_ERR_CUDA;
        if (result_without_kernel(ws, 0, h_result, stream) != cudaSuccess) return CDMA_ERR_CUDA;
        return CDMA_OK;
    }
    const bool on_device = !in_host_memory(d_src);
    const uint32_t nan_above = (dtype == CDMA_F32) ? 0x7f800000u : (dtype == CDMA_F16 ? 0x7c00u : 0x7f80u);
    const cudaError_t e =
        relu ? launch_zvc_relu_compress(d_src, n, s, nan_above, d_relu_out, d_dst, dst_capacity, d_table, ws, ctl,
                                        stream, on_device)
             : launch_zvc_compress(d_src, n, s, d_dst, dst_capacity, d_table, ws, ctl, stream, on_device);
    if (e != cudaSuccess) return CDMA_ERR_CUDA;
    if (finish_result(ws, ctl, h_result, stream) != cudaSuccess) return CDMA_ERR_CUDA;
    return CDMA_OK;
}

// Shared body of the plain and the ReLU-fused compression calls.
static int compress_enqueue(const void* d_src, uint64_t n, int dtype, int layout, bool relu, void* d_relu_out,
                            void* d_dst, uint64_t dst_capacity, uint64_t* d_table, void* d_workspace,
                            uint64_t workspace_bytes, void* cuda_stream, uint64_t* h_result) {
    const int st = check_common(n, dtype, layout, d_src, d_dst, d_table, d_workspace, workspace_bytes);
    if (st != CDMA_OK) return st;
    if (dst_capacity != 0 && d_dst == nullptr) return CDMA_ERR_INVALID_ARG;
    if (h_result == nullptr) return CDMA_ERR_INVALID_ARG;
    const uint32_t s = cdma_dtype_size(dtype);
    if (overlaps(d_src, n * s, d_dst, dst_capacity)) return CDMA_ERR_INVALID_ARG;
    if (relu && s == 1) return CDMA_ERR_UNSUPPORTED_DTYPE;
    if (relu && d_relu_out != nullptr) {
        if (!aligned(d_relu_out, 16)) return CDMA_ERR_ALIGNMENT;
        // writing the activation map over its own input is fine; over the payload it is not
        if (overlaps(d_relu_out, n * s, d_dst, dst_capacity)) return CDMA_ERR_INVALID_ARG;
        if (d_relu_out != d_src && overlaps(d_relu_out, n * s, d_src, n * s)) return CDMA_ERR_INVALID_ARG;
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    uint64_t* ws = static_cast<uint64_t*>(d_workspace);

    const LaunchCtl ctl = make_launch_ctl(h_result);
    return compress_launch(d_src, n, dtype, relu, d_relu_out, d_dst, dst_capacity, d_table, ws, ctl, stream, h_result);
}

int cdma_zvc_compress_async(const void* d_src, uint64_t n, int dtype, int layout, void* d_dst,
                            uint64_t dst_capacity, uint64_t* d_table, void* d_workspace,
                            uint64_t workspace_bytes, void* cuda_stream, uint64_t* h_result) {
    return compress_enqueue(d_src, n, dtype, layout, false, nullptr, d_dst, dst_capacity, d_table, d_workspace,
                            workspace_bytes, cuda_stream, h_result);
}

int cdma_zvc_relu_compress_async(const void* d_src, uint64_t n, int dtype, int layout, void* d_relu_out,
                                 void* d_dst, uint64_t dst_capacity, uint64_t* d_table, void* d_workspace,
                                 uint64_t workspace_bytes, void* cuda_stream, uint64_t* h_result) {
    return compress_enqueue(d_src, n, dtype, layout, true, d_relu_out, d_dst, dst_capacity, d_table, d_workspace,
                            workspace_bytes, cuda_stream, h_result);
}

int64_t cdma_zvc_relu_compress(const void* d_src, uint64_t n, int dtype, int layout, void* d_relu_out,
                               void* d_dst, uint64_t dst_capacity, uint64_t* d_table, void* d_workspace,
                               uint64_t workspace_bytes, void* cuda_stream) {
    uint64_t result[2] = {0, 0};
    const int st = compress_enqueue(d_src, n, dtype, layout, true, d_relu_out, d_dst, dst_capacity, d_table,
                                    d_workspace, workspace_bytes, cuda_stream, result);
    if (st != CDMA_OK) return -static_cast<int64_t>(st);
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return -static_cast<int64_t>(CDMA_ERR_CUDA);
    if (result[1] != 0) return -static_cast<int64_t>(result[1]);
    return static_cast<int64_t>(result[0]);
}

int64_t cdma_zvc_compress(const void* d_src, uint64_t n, int dtype, int layout, void* d_dst,
                          uint64_t dst_capacity, uint64_t* d_table, void* d_workspace,
                          uint64_t workspace_bytes, void* cuda_stream) {
    uint64_t result[2] = {0, 0};
    const int st = cdma_zvc_compress_async(d_src, n, dtype, layout, d_dst, dst_capacity, d_table,
                                           d_workspace, workspace_bytes, cuda_stream, result);
    if (st != CDMA_OK) return -static_cast<int64_t>(st);
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return -static_cast<int64_t>(CDMA_ERR_CUDA);
    if (result[1] != 0) return -static_cast<int64_t>(result[1]);
    return static_cast<int64_t>(result[0]);
}

int cdma_zvc_decompress_async(const void* d_src, uint64_t src_bytes, const uint64_t* d_table,
                              uint64_t n, int dtype, int layout, void* d_dst, void* d_workspace,
                              uint64_t workspace_bytes, void* cuda_stream, uint64_t* h_result) {
    const int st = check_common(n, dtype, layout, d_dst, d_src, d_table, d_workspace, workspace_bytes);
    if (st != CDMA_OK) return st;
    if (src_bytes != 0 && d_src == nullptr) return CDMA_ERR_INVALID_ARG;
    if (h_result == nullptr) return CDMA_ERR_INVALID_ARG;
    const uint32_t s = cdma_dtype_size(dtype);
    if (overlaps(d_dst, n * s, d_src, src_bytes)) return CDMA_ERR_INVALID_ARG;
    // sizes the format cannot produce are refused before anything is launched
    const uint64_t windows = (n + kWindow - 1) / kWindow;
    if (src_bytes < 4 * windows || src_bytes > 4 * windows + static_cast<uint64_t>(s) * n ||
        src_bytes % s != 0)
        return CDMA_ERR_CORRUPT_STREAM;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    uint64_t* ws = static_cast<uint64_t*>(d_workspace);

    if (n == 0) return result_without_kernel(ws, 0, h_result, stream) == cudaSuccess ? CDMA_OK : CDMA_ERR_CUDA;
    const LaunchCtl ctl = make_launch_ctl(h_result);
    if (launch_zvc_decompress(d_src, src_bytes, d_table, n, s, d_dst, ws, ctl, stream, !in_host_memory(d_src)) != cudaSuccess)
        return CDMA_ERR_CUDA;
    if (finish_result(ws, ctl, h_result, stream) != cudaSuccess) return CDMA_ERR_CUDA;
    return CDMA_OK;
}

int64_t cdma_zvc_decompress(const void* d_src, uint64_t src_bytes, const uint64_t* d_table,
                            uint64_t n, int dtype, int layout, void* d_dst, void* d_workspace,
                            uint64_t workspace_bytes, void* cuda_stream) {
    uint64_t result[2] = {0, 0};
    const int st = cdma_zvc_decompress_async(d_src, src_bytes, d_table, n, dtype, layout, d_dst,
                                             d_workspace, workspace_bytes, cuda_stream, result);
    if (st != CDMA_OK) return -static_cast<int64_t>(st);
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return -static_cast<int64_t>(CDMA_ERR_CUDA);
    if (result[1] != 0) return -static_cast<int64_t>(result[1]);
    return static_cast<int64_t>(n) * cdma_dtype_size(dtype);
}

// ---- backward pass of the activation function from the compressed map ----------------

int cdma_zvc_relu_backward_async(const void* d_src, uint64_t src_bytes, const uint64_t* d_table, uint64_t n,
                                 int dtype, int layout, const void* d_dy, void* d_dx, void* d_workspace,
                                 uint64_t workspace_bytes, void* cuda_stream, uint64_t* h_result) {
    const int st = check_common(n, dtype, layout, d_dx, d_src, d_table, d_workspace, workspace_bytes);
    if (st != CDMA_OK) return st;
    if ((src_bytes != 0 && d_src == nullptr) || (n != 0 && d_dy == nullptr) || h_result == nullptr)
        return CDMA_ERR_INVALID_ARG;
    if (!aligned(d_dy, 16)) return CDMA_ERR_ALIGNMENT;
    const uint32_t s = cdma_dtype_size(dtype);
    // dx may be dy itself (in place); any other overlap, or one with the payload, is refused
    if (overlaps(d_dx, n * s, d_src, src_bytes) || overlaps(d_dy, n * s, d_src, src_bytes)) return CDMA_ERR_INVALID_ARG;
    if (d_dx != d_dy && overlaps(d_dx, n * s, d_dy, n * s)) return CDMA_ERR_INVALID_ARG;
    const uint64_t windows = (n + kWindow - 1) / kWindow;
    if (src_bytes < 4 * windows || src_bytes > 4 * windows + static_cast<uint64_t>(s) * n || src_bytes % s != 0)
        return CDMA_ERR_CORRUPT_STREAM;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    uint64_t* ws = static_cast<uint64_t*>(d_workspace);
    if (n == 0) return result_without_kernel(ws, 0, h_result, stream) == cudaSuccess ? CDMA_OK : CDMA_ERR_CUDA;
    const LaunchCtl ctl = make_launch_ctl(h_result);
    if (launch_zvc_relu_backward(d_src, src_bytes, d_table, n, s, d_dy, d_dx, ws, ctl, stream) != cudaSuccess)
        return CDMA_ERR_CUDA;
    if (finish_result(ws, ctl, h_result, stream) != cudaSuccess) return CDMA_ERR_CUDA;
    return CDMA_OK;
}

int64_t cdma_zvc_relu_backward(const void* d_src, uint64_t src_bytes, const uint64_t* d_table, uint64_t n, int dtype,
                               int layout, const void* d_dy, void* d_dx, void* d_workspace, uint64_t workspace_bytes,
                               void* cuda_stream) {
    uint64_t result[2] = {0, 0};
    const int st = cdma_zvc_relu_backward_async(d_src, src_bytes, d_table, n, dtype, layout, d_dy, d_dx, d_workspace,
                                                workspace_bytes, cuda_stream, result);
    if (st != CDMA_OK) return -static_cast<int64_t>(st);
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return -static_cast<int64_t>(CDMA_ERR_CUDA);
    if (result[1] != 0) return -static_cast<int64_t>(result[1]);
    return static_cast<int64_t>(n) * cdma_dtype_size(dtype);
}

// ---- run-length comparison codec (4-byte elements) -----------------------------------

int cdma_rle_compress_async(const void* d_src, uint64_t n, int dtype, int layout, void* d_dst,
                            uint64_t dst_capacity, uint64_t* d_table, void* d_workspace,
                            uint64_t workspace_bytes, void* cuda_stream, uint64_t* h_result) {
    const int st = check_common(n, dtype, layout, d_src, d_dst, d_table, d_workspace, workspace_bytes);
    if (st != CDMA_OK) return st;
    if (dtype != CDMA_F32) return CDMA_ERR_UNSUPPORTED_DTYPE;
    if ((dst_capacity != 0 && d_dst == nullptr) || h_result == nullptr) return CDMA_ERR_INVALID_ARG;
    if (overlaps(d_src, n * 4, d_dst, dst_capacity)) return CDMA_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    uint64_t* ws = static_cast<uint64_t*>(d_workspace);
    if (n == 0) {
        if (cudaMemsetAsync(d_table, 0, 8, stream) != cudaSuccess) return CDMA_ERR_CUDA;
        return result_without_kernel(ws, 0, h_result, stream) == cudaSuccess ? CDMA_OK : CDMA_ERR_CUDA;
    }
    const LaunchCtl ctl = make_launch_ctl(h_result);
    if (launch_rle_compress(d_src, n, d_dst, dst_capacity, d_table, ws, ctl, stream) != cudaSuccess) return CDMA_ERR_CUDA;
    if (finish_result(ws, ctl, h_result, stream) != cudaSuccess) return CDMA_ERR_CUDA;
    return CDMA_OK;
}

int64_t cdma_rle_compress(const void* d_src, uint64_t n, int dtype, int layout, void* d_dst,
                          uint64_t dst_capacity, uint64_t* d_table, void* d_workspace,
                          uint64_t workspace_bytes, void* cuda_stream) {
    uint64_t result[2] = {0, 0};
    const int st = cdma_rle_compress_async(d_src, n, dtype, layout, d_dst, dst_capacity, d_table, d_workspace,
                                           workspace_bytes, cuda_stream, result);
    if (st != CDMA_OK) return -static_cast<int64_t>(st);
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return -static_cast<int64_t>(CDMA_ERR_CUDA);
    if (result[1] != 0) return -static_cast<int64_t>(result[1]);
    return static_cast<int64_t>(result[0]);
}

int cdma_rle_decompress_async(const void* d_src, uint64_t src_bytes, const uint64_t* d_table, uint64_t n,
                              int dtype, int layout, void* d_dst, void* d_workspace, uint64_t workspace_bytes,
                              void* cuda_stream, uint64_t* h_result) {
    const int st = check_common(n, dtype, layout, d_dst, d_src, d_table, d_workspace, workspace_bytes);
    if (st != CDMA_OK) return st;
    if (dtype != CDMA_F32) return CDMA_ERR_UNSUPPORTED_DTYPE;
    if ((src_bytes != 0 && d_src == nullptr) || h_result == nullptr) return CDMA_ERR_INVALID_ARG;
    if (overlaps(d_dst, n * 4, d_src, src_bytes)) return CDMA_ERR_INVALID_ARG;
    // sizes the format cannot produce are refused before anything is launched:
    // at least one token per chunk, at most 1025 words per chunk
    const uint64_t chunks = num_chunks_of(n);
    if (src_bytes < 4 * chunks || src_bytes > 4 * (n + chunks) || src_bytes % 4 != 0) return CDMA_ERR_CORRUPT_STREAM;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    uint64_t* ws = static_cast<uint64_t*>(d_workspace);
    if (n == 0) return result_without_kernel(ws, 0, h_result, stream) == cudaSuccess ? CDMA_OK : CDMA_ERR_CUDA;
    const LaunchCtl ctl = make_launch_ctl(h_result);
    if (launch_rle_decompress(d_src, src_bytes, d_table, n, d_dst, ws, ctl, stream) != cudaSuccess) return CDMA_ERR_CUDA;
    if (finish_result(ws, ctl, h_result, stream) != cudaSuccess) return CDMA_ERR_CUDA;
    return CDMA_OK;
}

int64_t cdma_rle_decompress(const void* d_src, uint64_t src_bytes, const uint64_t* d_table, uint64_t n,
                            int dtype, int layout, void* d_dst, void* d_workspace, uint64_t workspace_bytes,
                            void* cuda_stream) {
    uint64_t result[2] = {0, 0};
    const int st = cdma_rle_decompress_async(d_src, src_bytes, d_table, n, dtype, layout, d_dst, d_workspace,
                                             workspace_bytes, cuda_stream, result);
    if (st != CDMA_OK) return -static_cast<int64_t>(st);
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return -static_cast<int64_t>(CDMA_ERR_CUDA);
    if (result[1] != 0) return -static_cast<int64_t>(result[1]);
    return static_cast<int64_t>(n) * 4;
}

// Test hook, deliberately not declared in cdma.h: cdma_zvc_compress with one tile
// that never publishes its look-back descriptor and a short bound on the device-side
// waits, so that the tiles behind it run into the bound.  Every wait is bounded, the
// kernel returns normally and the call reports -CDMA_ERR_TIMEOUT; nothing traps or
// spins without limit.  stall_tile >= the number of tiles stalls nothing.
int64_t cdma_test_compress_stalled(const void* d_src, uint64_t n, int dtype, void* d_dst, uint64_t dst_capacity,
                                   uint64_t* d_table, void* d_workspace, uint64_t workspace_bytes,
                                   void* cuda_stream, uint32_t stall_tile, uint64_t wait_limit_ns) {
    const int st = check_common(n, dtype, CDMA_NCHW, d_src, d_dst, d_table, d_workspace, workspace_bytes);
    if (st != CDMA_OK) return -static_cast<int64_t>(st);
    if (n == 0 || wait_limit_ns == 0 || wait_limit_ns > kWaitLimitNs) return -static_cast<int64_t>(CDMA_ERR_INVALID_ARG);
    uint64_t result[2] = {0, 0};
    LaunchCtl ctl = make_launch_ctl(result);
    ctl.stall_tile = stall_tile;
    ctl.wait_limit_ns = wait_limit_ns;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int ls = compress_launch(d_src, n, dtype, false, nullptr, d_dst, dst_capacity, d_table,
                                   static_cast<uint64_t*>(d_workspace), ctl, stream, result);
    if (ls != CDMA_OK) return -static_cast<int64_t>(ls);
    if (cudaStreamSynchronize(stream) != cudaSuccess) return -static_cast<int64_t>(CDMA_ERR_CUDA);
    if (result[1] != 0) return -static_cast<int64_t>(result[1]);
    return static_cast<int64_t>(result[0]);
}

void cdma_time_next_kernel(void* start_event, void* stop_event) {
    t_time_start = static_cast<cudaEvent_t>(start_event);
    t_time_stop = static_cast<cudaEvent_t>(stop_event);
}

uint64_t cdma_kernel_launch_count(void) { return g_kernel_launches.load(std::memory_order_relaxed); }

}  // extern "C"
