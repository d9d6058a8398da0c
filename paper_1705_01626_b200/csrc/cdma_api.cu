// extern "C" codec entry points: argument checking, workspace reset, launch,
// result read-back.  Declarations and contracts are in include/cdma.h.
#include <atomic>
#include <cstring>

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

// Result words of a launch, handed to the host.  Page-locked host memory is
// addressable from the device, so a one-warp kernel stores the two words there
// (the next thing on the stream, with no copy-engine hand-over, which costs about
// 10 us per call); any other destination takes an ordinary 16-byte copy.
__global__ void publish_result_kernel(const uint64_t* __restrict__ ws, uint64_t* __restrict__ out) {
    if (threadIdx.x < 2) out[threadIdx.x] = ws[kWsBytes + threadIdx.x];
}

static cudaError_t enqueue_result(const uint64_t* ws, uint64_t* h_result, cudaStream_t stream) {
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, h_result) == cudaSuccess && attr.type == cudaMemoryTypeHost &&
        attr.devicePointer != nullptr && aligned_u64(attr.devicePointer)) {
        publish_result_kernel<<<1, 32, 0, stream>>>(ws, static_cast<uint64_t*>(attr.devicePointer));
        count_kernel_launch();
        return cudaGetLastError();
    }
    (void)cudaGetLastError();   // an unregistered pointer is not an error here
    return cudaMemcpyAsync(h_result, ws + kWsBytes, 16, cudaMemcpyDeviceToHost, stream);
}

// True when p lies in page-locked host memory (which kernels reach over the host link).
static bool in_host_memory(const void* p) {
    cudaPointerAttributes attr;
    if (p == nullptr || cudaPointerGetAttributes(&attr, p) != cudaSuccess) {
        (void)cudaGetLastError();
        return false;
    }
    return attr.type == cudaMemoryTypeHost;
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
    if (relu && d_relu_out != nullptr) {
        if (!aligned(d_relu_out, 16)) return CDMA_ERR_ALIGNMENT;
        // writing the activation map over its own input is fine; over the payload it is not
        if (overlaps(d_relu_out, n * s, d_dst, dst_capacity)) return CDMA_ERR_INVALID_ARG;
        if (d_relu_out != d_src && overlaps(d_relu_out, n * s, d_src, n * s)) return CDMA_ERR_INVALID_ARG;
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    uint64_t* ws = static_cast<uint64_t*>(d_workspace);

    // result words and every tile descriptor start at zero
    if (cudaMemsetAsync(ws, 0, kWsHeaderBytes + 8 * kDescStride * num_tiles_of(n), stream) != cudaSuccess)
        return CDMA_ERR_CUDA;
    if (n == 0) {
        if (cudaMemsetAsync(d_table, 0, 8, stream) != cudaSuccess) return CDMA_ERR_CUDA;
    } else {
        const bool on_device = !in_host_memory(d_src);
        const uint32_t nan_above = (dtype == CDMA_F32) ? 0x7f800000u : (dtype == CDMA_F16 ? 0x7c00u : 0x7f80u);
        const cudaError_t e =
            relu ? launch_zvc_relu_compress(d_src, n, s, nan_above, d_relu_out, d_dst, dst_capacity, d_table, ws, stream,
                                            on_device)
                 : launch_zvc_compress(d_src, n, s, d_dst, dst_capacity, d_table, ws, stream, on_device);
        if (e != cudaSuccess) return CDMA_ERR_CUDA;
    }
    if (enqueue_result(ws, h_result, stream) != cudaSuccess) return CDMA_ERR_CUDA;
    return CDMA_OK;
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

    if (cudaMemsetAsync(ws, 0, kWsHeaderBytes, stream) != cudaSuccess) return CDMA_ERR_CUDA;
    if (launch_zvc_decompress(d_src, src_bytes, d_table, n, s, d_dst, ws, stream, !in_host_memory(d_src)) != cudaSuccess)
        return CDMA_ERR_CUDA;
    if (enqueue_result(ws, h_result, stream) != cudaSuccess) return CDMA_ERR_CUDA;
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
    if (cudaMemsetAsync(ws, 0, kWsHeaderBytes + 8 * kDescStride * num_tiles_of(n), stream) != cudaSuccess)
        return CDMA_ERR_CUDA;
    if (n == 0) {
        if (cudaMemsetAsync(d_table, 0, 8, stream) != cudaSuccess) return CDMA_ERR_CUDA;
    } else if (launch_rle_compress(d_src, n, d_dst, dst_capacity, d_table, ws, stream) != cudaSuccess) {
        return CDMA_ERR_CUDA;
    }
    if (enqueue_result(ws, h_result, stream) != cudaSuccess) return CDMA_ERR_CUDA;
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
    if (cudaMemsetAsync(ws, 0, kWsHeaderBytes, stream) != cudaSuccess) return CDMA_ERR_CUDA;
    if (launch_rle_decompress(d_src, src_bytes, d_table, n, d_dst, ws, stream) != cudaSuccess) return CDMA_ERR_CUDA;
    if (enqueue_result(ws, h_result, stream) != cudaSuccess) return CDMA_ERR_CUDA;
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

void cdma_time_next_kernel(void* start_event, void* stop_event) {
    t_time_start = static_cast<cudaEvent_t>(start_event);
    t_time_stop = static_cast<cudaEvent_t>(stop_event);
}

uint64_t cdma_kernel_launch_count(void) { return g_kernel_launches.load(std::memory_order_relaxed); }

}  // extern "C"
