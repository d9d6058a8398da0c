// Shared definitions of the CUDA codec: constants of the stream format, the
// workspace layout, the per-launch control block and small device helpers.
// sm_100a only.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

#include "../../include/cdma.h"
#include "lookback_protocol.h"

namespace cdma {

// Format constants (Section V-A: 32-element window, 32-bit mask; the 4 KB
// block of the compression study is the offset-table granularity).
constexpr uint32_t kWindow = 32;
constexpr uint32_t kChunkWindows = 32;
constexpr uint32_t kChunk = kWindow * kChunkWindows;   // 1024 elements

// Compression tiling: one CTA = one tile of 32 KB of input (8 chunks of 4-byte
// elements, 16 chunks of 2-byte elements), 256 threads.
constexpr uint32_t kTileChunks = 8;
constexpr uint32_t kMinCtasPerSm = 5;
constexpr uint32_t kTileThreads = 32 * kTileChunks;
constexpr uint32_t kTileBytes = kTileChunks * kChunk * 4;

// Workspace layout, in uint64 words.  Nothing in it has to be cleared between
// calls: every word a launch reads was either written by that same launch or
// carries the launch's tag (see LaunchCtl), so whatever an earlier call -- or
// the caller -- left there is ignored.
constexpr uint32_t kWsReserved = 0;
constexpr uint32_t kWsFlag = 1;        // decompress: result words below have been initialised (holds the tag)
constexpr uint32_t kWsBytes = 2;       // result: payload bytes (compress) / dense bytes (decompress)
constexpr uint32_t kWsStatus = 3;      // result: error code, 0 = none
constexpr uint32_t kWsDescriptors = 4; // prefix descriptors follow
constexpr uint64_t kWsHeaderBytes = 8 * kWsDescriptors;
// One descriptor per 32-byte sector (16 bytes used), so that a tile publishing
// its descriptor does not contend in L2 with the walks that are reading its
// neighbours' (packed descriptors cost 10 % of the kernel's time).
constexpr uint32_t kDescStride = 4;    // uint64 words between descriptors

// Default bound of every device-side wait.
constexpr uint64_t kWaitLimitNs = 2000000000ull;  // 2 s
constexpr uint32_t kWaitLimitPolls = 1u << 24;    // backstop if the timer stalls
constexpr uint32_t kNoTile = 0xffffffffu;

// Per-launch control block, passed to the kernels by value.
struct LaunchCtl {
    uint64_t tag;            // unique per launch (62 bits, never 0): validates descriptors and flags
    uint64_t* result_out;    // device view of two page-locked host words {bytes, status}, or nullptr
    uint64_t wait_limit_ns;  // bound of the look-back / flag waits
    uint32_t stall_tile;     // test hook: this tile never publishes its descriptor (kNoTile: none)
};

__host__ __device__ inline uint64_t num_chunks_of(uint64_t n) { return (n + kChunk - 1) / kChunk; }
// upper bound of the tiles of a compression launch (a tile is never less than kTileChunks chunks):
// sizes the workspace
__host__ __device__ inline uint64_t num_tiles_of(uint64_t n) {
    return (num_chunks_of(n) + kTileChunks - 1) / kTileChunks;
}

struct Desc {
    uint64_t head;   // state | tag
    uint64_t value;
};
__device__ __forceinline__ Desc ld_desc(const uint64_t* p) {
    Desc d;
    asm volatile("ld.relaxed.gpu.global.v2.u64 {%0,%1}, [%2];" : "=l"(d.head), "=l"(d.value) : "l"(p) : "memory");
    return d;
}
__device__ __forceinline__ void st_desc(uint64_t* p, uint64_t head, uint64_t value) {
    asm volatile("st.relaxed.gpu.global.v2.u64 [%0], {%1,%2};" ::"l"(p), "l"(head), "l"(value) : "memory");
}
__device__ __forceinline__ uint64_t* desc_slot(uint64_t* ws, uint32_t tile) {
    return ws + kWsDescriptors + static_cast<uint64_t>(tile) * kDescStride;
}
__device__ __forceinline__ uint64_t ld_acquire_u64(const uint64_t* p) {
    uint64_t v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_u64(uint64_t* p, uint64_t v) {
    asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ uint64_t global_timer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ uint32_t lane_id() { return threadIdx.x & 31u; }
__device__ __forceinline__ uint32_t lanemask_lt() {
    uint32_t m;
    asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
    return m;
}

// Result words of a compression launch: written once, by the tile that closes
// the stream (it alone knows the total size, and every failure of a launch --
// a wait that ran out anywhere in front of it, a payload that outgrew its
// buffer -- is visible to it).
__device__ __forceinline__ void publish_result(uint64_t* ws, const LaunchCtl& ctl, uint64_t bytes, uint64_t status) {
    ws[kWsBytes] = bytes;
    ws[kWsStatus] = status;
    if (ctl.result_out != nullptr) {
        ctl.result_out[0] = bytes;
        ctl.result_out[1] = status;
    }
}

// Result words of a decompression launch.  Block 0 writes {dense bytes, 0} first
// thing and then raises the tagged flag; a block that finds the stream malformed
// waits (bounded) for that flag, so that its error code lands after the zero.
__device__ __forceinline__ void init_decode_result(uint64_t* ws, const LaunchCtl& ctl, uint64_t bytes) {
    publish_result(ws, ctl, bytes, 0);
    __threadfence_system();
    st_release_u64(ws + kWsFlag, ctl.tag);
}
__device__ inline void report_decode_error(uint64_t* ws, const LaunchCtl& ctl, uint32_t code) {
    const uint64_t t0 = global_timer_ns();
    uint32_t polls = 0;
    while (ld_acquire_u64(ws + kWsFlag) != ctl.tag) {
        if (++polls > kWaitLimitPolls || global_timer_ns() - t0 > ctl.wait_limit_ns) break;
        __nanosleep(200);
    }
    ws[kWsStatus] = code;
    if (ctl.result_out != nullptr) ctl.result_out[1] = code;
    __threadfence_system();
}

// Launchers (defined next to their kernels).  elem_size is 1, 2 or 4.  src_on_device
// is false when the input lies in mapped host memory: the kernels then leave out
// their L2 prefetches, which would fetch every line over the host link twice,
// and compression takes the kernel that loads with plain instructions.
cudaError_t launch_zvc_compress(const void* d_src, uint64_t n, uint32_t elem_size, void* d_dst,
                                uint64_t cap, uint64_t* d_table, uint64_t* d_ws, const LaunchCtl& ctl,
                                cudaStream_t stream, bool src_on_device = true);
// The row-per-thread kernel for 2-byte and 1-byte elements (zvc_compress_rows.cu).  With use_tma (device
// memory, at least one tile) the tile comes in by one TMA tensor copy; without, by plain loads.
bool zvc_compress_rows_tma_usable(const void* d_src, uint64_t n, uint32_t elem_size);
cudaError_t launch_zvc_compress_rows(const void* d_src, uint64_t n, uint32_t elem_size, void* d_dst, uint64_t cap,
                                     uint64_t* d_table, uint64_t* d_ws, const LaunchCtl& ctl, cudaStream_t stream,
                                     bool use_tma);
void preload_compress_rows_kernel();
void preload_compress_kernels();     // load every compression kernel now rather than at its first launch
cudaError_t launch_zvc_relu_compress(const void* d_src, uint64_t n, uint32_t elem_size, uint32_t nan_above,
                                     void* d_relu_out, void* d_dst, uint64_t cap, uint64_t* d_table,
                                     uint64_t* d_ws, const LaunchCtl& ctl, cudaStream_t stream,
                                     bool src_on_device = true);
cudaError_t launch_zvc_decompress(const void* d_src, uint64_t src_bytes, const uint64_t* d_table,
                                  uint64_t n, uint32_t elem_size, void* d_dst, uint64_t* d_ws,
                                  const LaunchCtl& ctl, cudaStream_t stream, bool src_on_device = true);
// 2-byte and 1-byte elements (zvc_decompress_groups.cu); the caller brackets the launch with the timing hooks
cudaError_t launch_zvc_decompress_groups(const void* d_src, uint64_t src_bytes, const uint64_t* d_table, uint64_t n,
                                         uint32_t elem_size, void* d_dst, uint64_t* d_ws, const LaunchCtl& ctl,
                                         cudaStream_t stream, bool src_on_device);
cudaError_t launch_zvc_gate_u32(const void* d_src, uint64_t src_bytes, const uint64_t* d_table, uint64_t n,
                                const void* d_gate, void* d_dst, uint64_t* d_ws, const LaunchCtl& ctl,
                                cudaStream_t stream);
cudaError_t launch_zvc_gate_groups(const void* d_src, uint64_t src_bytes, const uint64_t* d_table, uint64_t n,
                                   uint32_t elem_size, const void* d_gate, void* d_dst, uint64_t* d_ws,
                                   const LaunchCtl& ctl, cudaStream_t stream);
cudaError_t launch_zvc_relu_backward(const void* d_src, uint64_t src_bytes, const uint64_t* d_table, uint64_t n,
                                     uint32_t elem_size, const void* d_dy, void* d_dx, uint64_t* d_ws,
                                     const LaunchCtl& ctl, cudaStream_t stream);
cudaError_t launch_rle_compress(const void* d_src, uint64_t n, void* d_dst, uint64_t cap, uint64_t* d_table,
                                uint64_t* d_ws, const LaunchCtl& ctl, cudaStream_t stream);
cudaError_t launch_rle_decompress(const void* d_src, uint64_t src_bytes, const uint64_t* d_table, uint64_t n,
                                  void* d_dst, uint64_t* d_ws, const LaunchCtl& ctl, cudaStream_t stream);

// Host side of a call (cdma_api.cu).
LaunchCtl make_launch_ctl(uint64_t* h_result);                  // fresh tag; result_out if h_result is page-locked
bool in_host_memory(const void* p);                              // p lies in page-locked host memory
// After the kernel: hand the result words to h_result unless the kernel stores them there itself.
cudaError_t finish_result(const uint64_t* d_ws, const LaunchCtl& ctl, uint64_t* h_result, cudaStream_t stream);
// A call that launches no kernel (n = 0): result words {bytes, 0} by plain stream operations.
cudaError_t result_without_kernel(uint64_t* d_ws, uint64_t bytes, uint64_t* h_result, cudaStream_t stream);
// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) once per kernel and device instead of on every launch.
cudaError_t opt_in_shared_memory(const void* kernel, uint32_t bytes);
void count_kernel_launch();
void timing_before_launch(cudaStream_t stream);   // measurement hook, see cdma_time_next_kernel
void timing_after_launch(cudaStream_t stream);

}  // namespace cdma
