// Shared definitions of the CUDA codec: constants of the stream format, the
// workspace layout and small device helpers.  sm_100a only.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

#include "../../include/cdma.h"

namespace cdma {

// Format constants (Section V-A: 32-element window, 32-bit mask; the 4 KB
// block of the compression study is the offset-table granularity).
constexpr uint32_t kWindow = 32;
constexpr uint32_t kChunkWindows = 32;
constexpr uint32_t kChunk = kWindow * kChunkWindows;   // 1024 elements

// Compression tiling: one CTA = one tile = kTileChunks chunks, one warp per chunk.
#ifndef CDMA_TILE_CHUNKS
#define CDMA_TILE_CHUNKS 8
#endif
#ifndef CDMA_MIN_CTAS
#define CDMA_MIN_CTAS 5
#endif
constexpr uint32_t kTileChunks = CDMA_TILE_CHUNKS;
constexpr uint32_t kMinCtasPerSm = CDMA_MIN_CTAS;
constexpr uint32_t kTileThreads = 32 * kTileChunks;

// Workspace layout, in uint64 words.
constexpr uint32_t kWsTicket = 0;      // reserved (tiles are taken in block-index order)
constexpr uint32_t kWsReserved = 1;
constexpr uint32_t kWsBytes = 2;       // result: payload bytes (compress) / dense bytes (decompress)
constexpr uint32_t kWsStatus = 3;      // result: first error code, 0 = none
constexpr uint32_t kWsDescriptors = 4; // prefix descriptors follow, one 64-bit word per tile every kDescStride words
constexpr uint64_t kWsHeaderBytes = 8 * kWsDescriptors;
// Descriptors are kDescStride words apart: one per 32-byte sector, so that a tile
// publishing its descriptor does not contend in L2 with the walks that are
// reading its neighbours' (packed descriptors cost 10 % of the kernel's time).
#ifndef CDMA_DESC_STRIDE
#define CDMA_DESC_STRIDE 4
#endif
constexpr uint32_t kDescStride = CDMA_DESC_STRIDE;

// Inter-tile prefix descriptor: {state:2 | value:62} in one 64-bit word so
// that state and value are published by a single store.
constexpr uint64_t kDescValueMask = (1ull << 62) - 1;
constexpr uint64_t kDescAggregate = 1ull << 62;   // value = this tile's bytes
constexpr uint64_t kDescPrefix = 2ull << 62;      // value = bytes of tiles 0..this
constexpr uint64_t kDescError = 3ull << 62;       // a predecessor gave up; give up too

// Bounded waiting: a look-back poll loop gives up after this long.
constexpr uint64_t kWaitLimitNs = 2000000000ull;  // 2 s
constexpr uint32_t kWaitLimitPolls = 1u << 24;    // backstop if the timer stalls

__host__ __device__ inline uint64_t num_chunks_of(uint64_t n) { return (n + kChunk - 1) / kChunk; }
__host__ __device__ inline uint64_t num_tiles_of(uint64_t n) {
    return (num_chunks_of(n) + kTileChunks - 1) / kTileChunks;
}

__device__ __forceinline__ uint64_t ld_relaxed_u64(const uint64_t* p) {
    uint64_t v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed_u64(uint64_t* p, uint64_t v) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
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

// Record the first failure of a launch; later ones are dropped.
__device__ __forceinline__ void report_status(uint64_t* ws, uint32_t code) {
    atomicCAS(reinterpret_cast<unsigned long long*>(ws + kWsStatus), 0ull,
              static_cast<unsigned long long>(code));
}

// Launchers (defined next to their kernels).  elem_size is 2 or 4.  src_on_device
// is false when the input lies in mapped host memory: the kernels then leave out
// their L2 prefetches, which would fetch every line over the host link twice.
cudaError_t launch_zvc_compress(const void* d_src, uint64_t n, uint32_t elem_size, void* d_dst,
                                uint64_t cap, uint64_t* d_table, uint64_t* d_ws,
                                cudaStream_t stream, bool src_on_device = true);
cudaError_t launch_zvc_relu_compress(const void* d_src, uint64_t n, uint32_t elem_size, uint32_t nan_above,
                                     void* d_relu_out, void* d_dst, uint64_t cap, uint64_t* d_table,
                                     uint64_t* d_ws, cudaStream_t stream, bool src_on_device = true);
cudaError_t launch_zvc_decompress(const void* d_src, uint64_t src_bytes, const uint64_t* d_table,
                                  uint64_t n, uint32_t elem_size, void* d_dst, uint64_t* d_ws,
                                  cudaStream_t stream, bool src_on_device = true);
cudaError_t launch_rle_compress(const void* d_src, uint64_t n, void* d_dst, uint64_t cap, uint64_t* d_table,
                                uint64_t* d_ws, cudaStream_t stream);
cudaError_t launch_rle_decompress(const void* d_src, uint64_t src_bytes, const uint64_t* d_table, uint64_t n,
                                  void* d_dst, uint64_t* d_ws, cudaStream_t stream);
void count_kernel_launch();
void timing_before_launch(cudaStream_t stream);   // measurement hook, see cdma_time_next_kernel
void timing_after_launch(cudaStream_t stream);

}  // namespace cdma
