// Zero-value compression (Section V-A) of 2-byte and 1-byte elements that live in
// device memory: one thread owns one row of 128 bytes of the input -- two windows
// of 32 two-byte elements, or four of 32 one-byte elements -- so that the whole
// record of a window (compare, count, shift, append: the stages of Section V-B,
// Fig. 10a) is built by one thread from its own registers, with no work repeated
// across lanes and no cross-lane traffic.  With fewer bytes per element, the
// per-element cost is what bounds these widths; 4-byte elements stay with the
// kernel in zvc_compress.cu, which is faster there.
//
// A CTA compresses a tile of 256 rows (32 KB: 16 or 32 chunks).  Order of work:
//   1. load: one TMA tensor copy brings the tile into shared memory (128-byte
//      swizzle, so that thread t's reads of row t do not collide with its
//      neighbours'); each thread then takes its row into 32 registers;
//   2. count: the row's masks and number of non-zero elements per thread; a scan
//      over the CTA gives every record its place in the tile, and the tile's
//      size is published at once for the tiles behind it (single-pass decoupled
//      look-back);
//   3. assemble: each thread appends its masks and its non-zero elements to the
//      staged tile (in place of the input, which now lives in registers);
//   4. look back: warp 0 finds the tile's place in the stream;
//   5. copy: the CTA moves the staged bytes to the payload with aligned 16-byte
//      stores, realigning in registers.
#include <cuda.h>

#include <cstring>

#include "zvc_common.cuh"
#include "lookback.cuh"
#include "copy_out.cuh"

namespace cdma {

namespace {

constexpr uint32_t kRows = kTileThreads;               // rows of 128 bytes per tile, one per thread
constexpr uint32_t kRowBytes = 128;
// largest tile output (every element non-zero: a mask per window and the row itself) + slack
constexpr uint32_t stage_bytes(uint32_t elem_size) { return kRows * (kRowBytes + 4 * (4 / elem_size)) + 32; }
// Tiles follow the block index and blocks are dispatched in that order, so the tile this many places
// further on will be picked up by a CTA that starts about half a CTA lifetime from now.
constexpr uint32_t kPrefetchAheadTiles = 370;
constexpr uint32_t kTryWaitHintNs = 100000;            // 100 us

// flags of the two halves of w at bits J and 16 + J: two instructions
template <uint32_t J>
__device__ __forceinline__ void flag_pair(uint32_t& acc, uint32_t w) {
    asm("{\n\t.reg .b32 d;\n\tmin.u16x2 d, %1, %2;\n\tmad.lo.u32 %0, d, %3, %0;\n\t}"
        : "+r"(acc) : "r"(w), "r"(0x00010001u), "n"(1u << J));
}
// {flags of the low halves of 16 words | flags of their high halves} of one window
__device__ __forceinline__ uint32_t flags_of(const uint32_t* w) {
    uint32_t f = 0;
    flag_pair<0>(f, w[0]);   flag_pair<1>(f, w[1]);   flag_pair<2>(f, w[2]);   flag_pair<3>(f, w[3]);
    flag_pair<4>(f, w[4]);   flag_pair<5>(f, w[5]);   flag_pair<6>(f, w[6]);   flag_pair<7>(f, w[7]);
    flag_pair<8>(f, w[8]);   flag_pair<9>(f, w[9]);   flag_pair<10>(f, w[10]); flag_pair<11>(f, w[11]);
    flag_pair<12>(f, w[12]); flag_pair<13>(f, w[13]); flag_pair<14>(f, w[14]); flag_pair<15>(f, w[15]);
    return f;
}
// bits 0..15 of x to the even positions, bits 16..31 to the odd ones (a perfect shuffle):
// turns flags_of() into the window's mask
__device__ __forceinline__ uint32_t interleave16(uint32_t x) {
    uint32_t t;
    t = (x ^ (x >> 8)) & 0x0000ff00u;  x ^= t ^ (t << 8);
    t = (x ^ (x >> 4)) & 0x00f000f0u;  x ^= t ^ (t << 4);
    t = (x ^ (x >> 2)) & 0x0c0c0c0cu;  x ^= t ^ (t << 2);
    t = (x ^ (x >> 1)) & 0x22222222u;  x ^= t ^ (t << 1);
    return x;
}
// append the non-zero halves of w (low half first) at q + 4
__device__ __forceinline__ void append_pair(uint32_t& q, uint32_t w) {
    asm volatile("{\n\t.reg .pred p, r;\n\t.reg .b32 t, h;\n\t"
                 "and.b32 t, %1, 0xffff;\n\tsetp.ne.u32 p, t, 0;\n\t"
                 "@p st.shared.u16 [%0+4], %1;\n\t@p add.u32 %0, %0, 2;\n\t"
                 "shr.u32 h, %1, 16;\n\tsetp.ne.u32 r, h, 0;\n\t"
                 "@r st.shared.u16 [%0+4], h;\n\t@r add.u32 %0, %0, 2;\n\t}"
                 : "+r"(q) : "r"(w) : "memory");
}
// a mask word at a 2-byte aligned shared address
__device__ __forceinline__ void sts_mask(uint32_t q, uint32_t m) {
    asm volatile("{\n\t.reg .b32 h;\n\tshr.u32 h, %1, 16;\n\tst.shared.u16 [%0], %1;\n\tst.shared.u16 [%0+2], h;\n\t}"
                 ::"r"(q), "r"(m) : "memory");
}

// ---- 1-byte elements ---------------------------------------------------------------------------
// the 4 "byte is non-zero" bits of a word (byte 0 = bit 0)
__device__ __forceinline__ uint32_t nonzero_bytes(uint32_t w) {
    const uint32_t t = (((w & 0x7f7f7f7fu) + 0x7f7f7f7fu) | w) & 0x80808080u;   // 0x80 in every non-zero byte
    return (((t >> 7) * 0x00204081u) >> 21) & 15u;                               // bits 0, 8, 16, 24 -> 0, 1, 2, 3
}
// mask of a window of 32 one-byte elements held in 8 words
__device__ __forceinline__ uint32_t mask_of_bytes(const uint32_t* w) {
    uint32_t m = 0;
#pragma unroll
    for (uint32_t j = 0; j < 8; ++j) m |= nonzero_bytes(w[j]) << (4 * j);
    return m;
}
// append the non-zero bytes of w (lowest first) at q + 4
__device__ __forceinline__ void append_bytes(uint32_t& q, uint32_t w) {
    asm volatile("{\n\t.reg .pred p;\n\t.reg .b32 h;\n\t"
                 "prmt.b32 h, %1, 0, 0x4440;\n\tsetp.ne.u32 p, h, 0;\n\t@p st.shared.u8 [%0+4], h;\n\t@p add.u32 %0, %0, 1;\n\t"
                 "prmt.b32 h, %1, 0, 0x4441;\n\tsetp.ne.u32 p, h, 0;\n\t@p st.shared.u8 [%0+4], h;\n\t@p add.u32 %0, %0, 1;\n\t"
                 "prmt.b32 h, %1, 0, 0x4442;\n\tsetp.ne.u32 p, h, 0;\n\t@p st.shared.u8 [%0+4], h;\n\t@p add.u32 %0, %0, 1;\n\t"
                 "prmt.b32 h, %1, 0, 0x4443;\n\tsetp.ne.u32 p, h, 0;\n\t@p st.shared.u8 [%0+4], h;\n\t@p add.u32 %0, %0, 1;\n\t}"
                 : "+r"(q) : "r"(w) : "memory");
}
// a mask word at any shared byte address
__device__ __forceinline__ void sts_mask_bytes(uint32_t q, uint32_t m) {
    asm volatile("{\n\t.reg .b32 h;\n\tst.shared.u8 [%0], %1;\n\tshr.u32 h, %1, 8;\n\tst.shared.u8 [%0+1], h;\n\t"
                 "shr.u32 h, %1, 16;\n\tst.shared.u8 [%0+2], h;\n\tshr.u32 h, %1, 24;\n\tst.shared.u8 [%0+3], h;\n\t}"
                 ::"r"(q), "r"(m) : "memory");
}

// Bounded wait for the tile to land.  Returns false when the limit ran out.
__device__ __forceinline__ bool wait_tile(uint32_t mbar, uint64_t limit_ns) {
    uint32_t done = 0;
    uint32_t polls = 0;
    uint64_t t0 = 0;
    while (true) {
        // (the last operand lets the hardware hold the thread for up to that many nanoseconds before
        // it answers "not yet": the loop runs once or twice, not hundreds of times)
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0, %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(mbar), "r"(kTryWaitHintNs) : "memory");
        if (done) return true;
        const uint64_t now = global_timer_ns();
        if (t0 == 0) t0 = now;
        else if (now - t0 > limit_ns || ++polls > kWaitLimitPolls) return false;
    }
}

// The grid is one CTA per tile; tiles follow the block index and blocks are dispatched in
// that order, so a tile only ever waits for blocks that were dispatched before it (the
// assumption single-pass scans rest on); should it ever not hold, the bounded wait in the
// walk turns it into CDMA_ERR_TIMEOUT.
// S = element size (2 or 1).
template <uint32_t S>
__global__ void __launch_bounds__(kTileThreads, kMinCtasPerSm)
zvc_compress_rows_kernel(const __grid_constant__ CUtensorMap tmap, const uint8_t* __restrict__ src, uint64_t n,
                         uint8_t* __restrict__ dst, uint64_t cap, uint64_t* __restrict__ table,
                         uint64_t* __restrict__ ws, const LaunchCtl ctl, uint32_t num_tiles, uint64_t num_chunks,
                         uint64_t full_rows, uint32_t use_tma) {
    constexpr uint32_t WPR = 4 / S;                              // windows per row: 2 or 4
    constexpr uint32_t WW = 8 * S;                               // words per window: 16 or 8
    extern __shared__ __align__(1024) uint8_t smem_raw[];          // input tile, then the staged output
    __shared__ __align__(8) uint64_t s_mbar;
    __shared__ uint32_t s_warp_bytes[kTileThreads / 32];
    __shared__ uint64_t s_base;
    __shared__ uint32_t s_failed;
    __shared__ uint32_t s_room;
    __shared__ uint32_t s_late;

    const uint32_t tid = threadIdx.x;
    const uint32_t lane = tid & 31u;
    const uint32_t warp = tid >> 5;
    const uint32_t tile = blockIdx.x;
    const uint32_t s_stage = smem_u32(smem_raw);
    const uint32_t mbar = smem_u32(&s_mbar);
    const uint64_t row0 = static_cast<uint64_t>(tile) * kRows;

    // ---- 1. load -------------------------------------------------------------------------------
    // (use_tma is 0 for tensors the tensor copy cannot serve -- less than one row, or in host memory:
    // every thread then fetches its row with plain loads further down)
    if (tid == 0) {
        s_late = 0;
        prefetch_future_descriptor(ws, tile, num_tiles);
        if (use_tma) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(mbar) : "memory");
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        }
    }
    __syncthreads();
    uint32_t e[32];
    if (use_tma) {
        if (tid == 0) {
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(mbar), "r"(kTileBytes) : "memory");
            // rows past the end of the tensor map (the last tile only) arrive as zeros
            asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                         ::"r"(s_stage), "l"(&tmap), "r"(0), "r"(static_cast<int32_t>(row0)), "r"(mbar) : "memory");
        } else if (tid == 32) {
            // asking L2 for a later tile now turns that tile's load into L2 hits; every line still comes
            // from DRAM exactly once
            const uint64_t prow = row0 + static_cast<uint64_t>(kPrefetchAheadTiles) * kRows;
            if (prow + kRows <= full_rows)
                asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];"
                             ::"l"(&tmap), "r"(0), "r"(static_cast<int32_t>(prow)) : "memory");
        }
        // (a thread whose wait ran out goes on with whatever shared memory holds; the CTA decides
        // together behind the next barrier)
        if (!wait_tile(mbar, ctl.wait_limit_ns)) s_late = 1;

        // thread t takes row t: eight 16-byte pieces, piece i stored at position i ^ (t & 7) by the swizzle
        const uint32_t row_addr = s_stage + kRowBytes * tid;
        const uint32_t sw = tid & 7u;
#pragma unroll
        for (uint32_t i = 0; i < 8; ++i) {
            const uint4 v = lds128(row_addr + 16u * (i ^ sw));
            e[4 * i + 0] = v.x; e[4 * i + 1] = v.y; e[4 * i + 2] = v.z; e[4 * i + 3] = v.w;
        }
    } else {
#pragma unroll
        for (uint32_t i = 0; i < 32; ++i) e[i] = 0;
        if (row0 + tid < full_rows) {
            const uint4* rp = reinterpret_cast<const uint4*>(src + (row0 + tid) * kRowBytes);
#pragma unroll
            for (uint32_t i = 0; i < 8; ++i) {
                const uint4 v = __ldcs(rp + i);
                e[4 * i + 0] = v.x; e[4 * i + 1] = v.y; e[4 * i + 2] = v.z; e[4 * i + 3] = v.w;
            }
        }
    }
    const uint64_t row = row0 + tid;
    // windows of this row that exist (the tensor may end inside the last tile)
    const uint64_t total_windows = (n + kWindow - 1) / kWindow;
    const uint64_t w_first = WPR * row;
    const uint32_t nwin = w_first >= total_windows ? 0u
                          : (total_windows - w_first >= WPR ? WPR : static_cast<uint32_t>(total_windows - w_first));
    if (row >= full_rows && nwin != 0) {
        // the one row that is only partly inside the tensor: plain guarded loads, byte by byte
        const uint64_t b0 = row * kRowBytes, nbytes = n * S;
#pragma unroll
        for (uint32_t i = 0; i < 32; ++i) {
            uint32_t v = 0;
            for (uint32_t b = 0; b < 4; ++b)
                if (b0 + 4 * i + b < nbytes) v |= static_cast<uint32_t>(src[b0 + 4 * i + b]) << (8 * b);
            e[i] = v;
        }
    }

    // ---- 2. count ------------------------------------------------------------------------------
    uint32_t mask[WPR];
    uint32_t rec_bytes = 0;
#pragma unroll
    for (uint32_t k = 0; k < WPR; ++k) {
        mask[k] = (S == 2) ? interleave16(flags_of(e + WW * k)) : mask_of_bytes(e + WW * k);
        if (k < nwin) rec_bytes += 4u + S * __popc(mask[k]);
    }
    // place of every thread's records in the tile: scan over the warp, then over the warps
    uint32_t incl = rec_bytes;
#pragma unroll
    for (uint32_t o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) s_warp_bytes[warp] = incl;
    __syncthreads();                       // also: every thread has its row in registers, the tile may be overwritten
    if (s_late) {
        // The copy is late beyond the limit.  One more bounded wait, so that it cannot write into shared
        // memory this CTA has already handed back; then the launch fails the way a look-back time-out
        // does: the tile marks itself, so that the tiles behind it stop as well.
        if (use_tma) (void)wait_tile(mbar, ctl.wait_limit_ns);
        if (tid == 0) {
            publish_prefix(ws, ctl, tile, true, 0);
            if (tile == num_tiles - 1) publish_result(ws, ctl, 0, CDMA_ERR_TIMEOUT);
        }
        return;
    }
    const uint32_t wb = (lane < kTileThreads / 32) ? s_warp_bytes[lane] : 0u;
    const uint32_t warp_off = __reduce_add_sync(0xffffffffu, lane < warp ? wb : 0u);
    uint64_t tile_bytes = 0;
    if (warp == 0) {
        tile_bytes = __reduce_add_sync(0xffffffffu, wb);
        // the tile's size is public before any record is assembled
        if (lane == 0) publish_aggregate(ws, ctl, tile, tile_bytes);
    }
    const uint32_t rec_off = warp_off + incl - rec_bytes;       // byte offset of my records in the staged tile

    // ---- 3. assemble -----------------------------------------------------------------------------
    uint32_t q = s_stage + rec_off;
#pragma unroll
    for (uint32_t k = 0; k < WPR; ++k) {
        if (k < nwin) {
            if (S == 2) sts_mask(q, mask[k]);
            else sts_mask_bytes(q, mask[k]);
#pragma unroll
            for (uint32_t i = 0; i < WW; ++i) {
                if (S == 2) append_pair(q, e[WW * k + i]);
                else append_bytes(q, e[WW * k + i]);
            }
            q += 4;
        }
    }

    // ---- 4. the tile's place in the stream -------------------------------------------------------
    if (warp == 0)
        resolve_tile(ws, ctl, tile, num_tiles, tile_bytes, cap, table, num_chunks, &s_base, &s_failed, &s_room);
    __syncthreads();
    if (s_failed) return;
    const uint64_t base = s_base;

    // offset-table entries: a chunk is 32 windows = 32 / WPR rows
    constexpr uint32_t kChunkRows = 32 / WPR;
    const uint64_t chunk = static_cast<uint64_t>(tile) * (kRows / kChunkRows) + WPR * warp + lane / kChunkRows;
    if (lane % kChunkRows == 0 && chunk < num_chunks) table[chunk] = base + rec_off;

    // ---- 5. copy the staged bytes to their place, below the capacity ------------------------------
    copy_out<S, kTileThreads>(s_stage, smem_raw, dst, base, s_room);
}

// The driver's tensor-map encoder, looked up once (no link-time dependency on the driver library).
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess) {
            (void)cudaGetLastError();
            p = nullptr;
        }
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

}  // namespace

void preload_compress_rows_kernel() {
    cudaFuncAttributes a;
    (void)cudaFuncGetAttributes(&a, zvc_compress_rows_kernel<2>);
    (void)cudaFuncGetAttributes(&a, zvc_compress_rows_kernel<1>);
    (void)encode_tiled();
}

bool zvc_compress_rows_tma_usable(const void* d_src, uint64_t n, uint32_t elem_size) {
    // 2-byte or 1-byte elements, at least one whole tile, rows addressable with 32-bit coordinates, and an
    // encoder to describe them
    const uint64_t full_rows = n * elem_size / kRowBytes;
    return (elem_size == 2 || elem_size == 1) && full_rows >= kRows && full_rows < (1ull << 31) &&
           (reinterpret_cast<uintptr_t>(d_src) & 15) == 0 && encode_tiled() != nullptr;
}

cudaError_t launch_zvc_compress_rows(const void* d_src, uint64_t n, uint32_t elem_size, void* d_dst, uint64_t cap,
                                     uint64_t* d_table, uint64_t* d_ws, const LaunchCtl& ctl, cudaStream_t stream,
                                     bool use_tma) {
    const uint64_t bytes = n * elem_size;
    const uint64_t full_rows = bytes / kRowBytes;
    const uint64_t tiles = (bytes + kTileBytes - 1) / kTileBytes;
    CUtensorMap tmap;
    memset(&tmap, 0, sizeof(tmap));
    if (use_tma) {
        // the tensor as rows of 32 words; a box is one tile; 128-byte swizzle
        const cuuint64_t dims[2] = {kRowBytes / 4, full_rows};
        const cuuint64_t strides[1] = {kRowBytes};
        const cuuint32_t box[2] = {kRowBytes / 4, kRows};
        const cuuint32_t estr[2] = {1, 1};
        const CUresult r = encode_tiled()(&tmap, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<void*>(d_src), dims,
                                          strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                          CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    }
    auto kernel = elem_size == 2 ? zvc_compress_rows_kernel<2> : zvc_compress_rows_kernel<1>;
    const uint32_t smem = stage_bytes(elem_size);
    const cudaError_t oe = opt_in_shared_memory(reinterpret_cast<const void*>(kernel), smem);
    if (oe != cudaSuccess) return oe;
    timing_before_launch(stream);
    kernel<<<static_cast<unsigned>(tiles), kTileThreads, smem, stream>>>(
        tmap, static_cast<const uint8_t*>(d_src), n, static_cast<uint8_t*>(d_dst), cap, d_table, d_ws, ctl,
        static_cast<uint32_t>(tiles), num_chunks_of(n), full_rows, use_tma ? 1u : 0u);
    timing_after_launch(stream);
    count_kernel_launch();
    return cudaGetLastError();
}

}  // namespace cdma
