// Zero-value decompression of 1-byte elements (Section V-B, Fig. 10b: the
// pop-count of a mask tells how many payload values its window takes; values or
// zeros are steered into the window's 32 places).
//
// One warp expands one chunk (1024 elements).  The chunk's payload bytes are staged
// in shared memory; the warp walks the records -- a record is 4 + popc(mask) bytes,
// so masks sit at any byte address and are read as two aligned words and a funnel
// shift -- and lane w keeps {position, mask} of window w.  A lane then expands 4
// consecutive elements (one output word; 8 lanes per window, 4 windows per round):
// the pop-count of the mask bits below them is where their values start, and one
// byte permute with a selector from a 16-entry table (indexed by the lane's 4 mask
// bits) puts values and zeros in place.  The table and every record are validated;
// nothing is read outside the payload or written outside the tensor whatever the
// input holds.
#include "zvc_common.cuh"

namespace cdma {

namespace {

constexpr uint32_t kWarps = 8;
constexpr uint32_t kMaxChunkBytes = 4 * kChunkWindows + kChunk;      // 1152
// 16-byte phase in front; behind, room for the 8 bytes a lane reads past the end of a malformed chunk
constexpr uint32_t kBuf = (kMaxChunkBytes + 16 + 64 + 15) / 16 * 16;

// Selector of the byte permute that expands up to 4 values into 4 places, by the 4 mask bits:
// place k takes value number popc(bits below k) if bit k is set, else a zero byte (index 4).
__constant__ uint16_t kExpandSel[16] = {
    0x4444, 0x4440, 0x4404, 0x4410, 0x4044, 0x4140, 0x4104, 0x4210,
    0x0444, 0x1440, 0x1404, 0x2410, 0x1044, 0x2140, 0x2104, 0x3210,
};

// the 4 bytes at byte address p of the staged words
__device__ __forceinline__ uint32_t load_unaligned(const uint32_t* words, uint32_t p) {
    const uint32_t lo = words[p >> 2], hi = words[(p >> 2) + 1];
    return __funnelshift_r(lo, hi, 8u * (p & 3u));
}

__global__ void __launch_bounds__(32 * kWarps)
zvc_decompress_kernel_u8(const uint8_t* __restrict__ src, uint64_t src_bytes, const uint64_t* __restrict__ table,
                         uint64_t n, uint8_t* __restrict__ dst, uint64_t* __restrict__ ws, const LaunchCtl ctl,
                         uint64_t num_chunks) {
    __shared__ __align__(16) uint8_t s_buf[kWarps][kBuf];
    __shared__ uint16_t s_sel[16];
    if (threadIdx.x < 16) s_sel[threadIdx.x] = kExpandSel[threadIdx.x];
    __syncthreads();

    const uint32_t lane = lane_id();
    const uint32_t warp = threadIdx.x >> 5;
    const uint64_t chunk = static_cast<uint64_t>(blockIdx.x) * kWarps + warp;
    if (blockIdx.x == 0 && threadIdx.x == 0) init_decode_result(ws, ctl, n);
    if (chunk >= num_chunks) return;

    const uint64_t e0 = chunk * kChunk;
    const uint32_t nelem = (n - e0 < kChunk) ? static_cast<uint32_t>(n - e0) : kChunk;
    const uint32_t nwin = (nelem + kWindow - 1) / kWindow;

    // ---- the chunk's byte range, validated ----------------------------------------------------------
    const uint64_t lo = __ldg(table + chunk);
    const uint64_t hi = __ldg(table + chunk + 1);
    bool ok = (lo <= hi) && (hi <= src_bytes) && (hi - lo >= 4ull * nwin) && (hi - lo <= 4ull * nwin + nelem);
    if (chunk == 0 && lo != 0) ok = false;
    if (chunk == num_chunks - 1 && hi != src_bytes) ok = false;
    if (!ok) {
        if (lane == 0) report_decode_error(ws, ctl, CDMA_ERR_CORRUPT_STREAM);
        return;
    }

    // ---- stage payload bytes [lo, hi) in shared memory (same 16-byte phase) ----------------------------
    uint8_t* buf = s_buf[warp];
    const uint64_t a0 = lo & ~15ull;              // buf[0] corresponds to payload byte a0
    for (uint64_t a = a0 + 16ull * lane; a < hi; a += 16ull * 32) {
        uint4 q;
        if (a + 16 <= src_bytes) {
            q = __ldcs(reinterpret_cast<const uint4*>(src + a));
        } else {
            // last, partial 16 bytes of the payload: never read past src_bytes
            uint32_t wds[4] = {0, 0, 0, 0};
            for (uint32_t b = 0; b < 16; ++b)
                if (a + b < src_bytes) wds[b >> 2] |= static_cast<uint32_t>(src[a + b]) << (8 * (b & 3));
            q = make_uint4(wds[0], wds[1], wds[2], wds[3]);
        }
        *reinterpret_cast<uint4*>(buf + (a - a0)) = q;
    }
    __syncwarp();

    // ---- walk the records: lane w keeps {position, mask} of window w ------------------------------------
    const uint32_t* words = reinterpret_cast<const uint32_t*>(buf);
    uint32_t p = static_cast<uint32_t>(lo - a0);
    const uint32_t end = static_cast<uint32_t>(hi - a0);
    uint32_t my_p = 0, my_m = 0;
    bool bad = false;
    for (uint32_t w = 0; w < nwin; ++w) {
        if (p + 4 > end) { bad = true; break; }
        const uint32_t m = load_unaligned(words, p);
        if (lane == w) { my_p = p; my_m = m; }
        p += 4u + __popc(m);
    }
    if (!bad && p != end) bad = true;
    if (!bad && nelem != kChunk) {
        // a short last window must not name elements beyond n
        const uint32_t tail = nelem & 31u;
        const uint32_t last_mask = __shfl_sync(0xffffffffu, my_m, nwin - 1);
        if (tail != 0 && (last_mask >> tail) != 0) bad = true;
    }
    if (bad) {
        if (lane == 0) report_decode_error(ws, ctl, CDMA_ERR_CORRUPT_STREAM);
        return;
    }

    // ---- expand -------------------------------------------------------------------------------------------
    if (nelem == kChunk) {
        uint32_t* out = reinterpret_cast<uint32_t*>(dst + e0) + lane;
        const uint32_t sh = 4u * (lane & 7u);
        const uint32_t below = (1u << sh) - 1u;
#pragma unroll
        for (uint32_t r = 0; r < kChunkWindows / 4; ++r) {
            const uint32_t w = 4 * r + (lane >> 3);
            const uint32_t m = __shfl_sync(0xffffffffu, my_m, w);
            const uint32_t pw = __shfl_sync(0xffffffffu, my_p, w);
            const uint32_t v = load_unaligned(words, pw + 4u + __popc(m & below));      // my (up to) four values
            uint32_t o;
            asm("prmt.b32 %0, %1, 0, %2;" : "=r"(o) : "r"(v), "r"(static_cast<uint32_t>(s_sel[(m >> sh) & 15u])));
            __stcs(out + 32 * r, o);
        }
    } else {
        // ragged last chunk: lane = element, one window per step
        const uint32_t lt = lanemask_lt();
        for (uint32_t w = 0; w < nwin; ++w) {
            const uint32_t m = __shfl_sync(0xffffffffu, my_m, w);
            const uint32_t pw = __shfl_sync(0xffffffffu, my_p, w);
            const uint64_t j = e0 + w * kWindow + lane;
            if (j < n) dst[j] = ((m >> lane) & 1u) ? buf[pw + 4u + __popc(m & lt)] : uint8_t(0);
        }
    }
}

}  // namespace

cudaError_t launch_zvc_decompress_u8(const void* d_src, uint64_t src_bytes, const uint64_t* d_table, uint64_t n,
                                     void* d_dst, uint64_t* d_ws, const LaunchCtl& ctl, cudaStream_t stream) {
    const uint64_t chunks = num_chunks_of(n);
    const dim3 grid(static_cast<unsigned>((chunks + kWarps - 1) / kWarps));
    zvc_decompress_kernel_u8<<<grid, 32 * kWarps, 0, stream>>>(static_cast<const uint8_t*>(d_src), src_bytes, d_table, n,
                                                               static_cast<uint8_t*>(d_dst), d_ws, ctl, chunks);
    return cudaGetLastError();
}

}  // namespace cdma
