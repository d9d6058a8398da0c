// Zero-value decompression (Section V-B, Fig. 10b): the pop-count of a mask
// tells how many payload values its window takes; values or zeros are steered
// into the window's 32 places.
//
// One warp expands one chunk (1024 elements).  The offset table gives the
// chunk's byte range in the payload; the warp copies that range into shared
// memory with 16-byte loads, then walks the records: the position of window
// w+1's mask is the position of window w's mask plus 4 plus s times the
// pop-count of that mask (the stream is self-delimiting, Section V-A).  A lane
// expands 4 consecutive elements, so one warp store covers 4 windows (8 lanes
// per window): the lane takes its 4 mask bits, the pop-count of the mask bits
// below them is where its first value sits, it reads 4 candidate values and
// selects value-or-zero for each element, then stores them as one vector.
// The table and every record are validated; nothing is read outside the
// payload or written outside the tensor whatever the input holds.
#include "zvc_common.cuh"

namespace cdma {

namespace {

constexpr uint32_t kDecWarps = 8;
constexpr uint32_t kDecThreads = 32 * kDecWarps;
#ifndef CDMA_DEC_PREFETCH_CTAS
#define CDMA_DEC_PREFETCH_CTAS 888
#endif
constexpr uint32_t kPrefetchAheadCtas = CDMA_DEC_PREFETCH_CTAS;   // 6 CTAs x 148 SMs resident at a time

__device__ __forceinline__ void store4(uint32_t* p, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    __stcs(reinterpret_cast<uint4*>(p), make_uint4(a, b, c, d));
}
__device__ __forceinline__ void store4(uint16_t* p, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    __stcs(reinterpret_cast<uint2*>(p), make_uint2(a | (b << 16), c | (d << 16)));
}

template <typename T, bool PREFETCH>
__global__ void __launch_bounds__(kDecThreads)
zvc_decompress_kernel(const uint8_t* __restrict__ src, uint64_t src_bytes,
                      const uint64_t* __restrict__ table, uint64_t n, T* __restrict__ dst,
                      uint64_t* __restrict__ ws, uint64_t num_chunks) {
    constexpr uint32_t S = sizeof(T);
    constexpr uint32_t MU = 4 / S;                               // units of T per mask
    constexpr uint32_t kMaxChunkBytes = 4 * kChunkWindows + S * kChunk;
    // 16-byte phase in front; behind, room for the reads of a walk that has left
    // a malformed record.  4-byte elements: the position is pulled back to `end`
    // after every window (one more instruction per window, but the smaller buffer
    // lets a sixth CTA fit per SM); 2-byte elements: after every group of 4
    // windows, so the walk can run 4 records past `end`.  Either way a lane then
    // reads a mask and up to 35 values from there.
    constexpr bool kClampEveryWindow = (S == 4);
    constexpr uint32_t kOverrun = kClampEveryWindow ? 0u : 4u * (MU + 32u);
    constexpr uint32_t kBuf = (kMaxChunkBytes + 16 + S * (kOverrun + MU + 36) + 15) / 16 * 16;
    static_assert(kBuf % 16 == 0, "rows of s_buf must keep 16-byte alignment for the vector stores");
    __shared__ __align__(16) uint8_t s_buf[kDecWarps][kBuf];

    const uint32_t lane = lane_id();
    const uint32_t warp = threadIdx.x >> 5;
    const uint64_t chunk = static_cast<uint64_t>(blockIdx.x) * kDecWarps + warp;
    if (blockIdx.x == 0 && threadIdx.x == 0) ws[kWsBytes] = n * S;
    if (chunk >= num_chunks) return;

    const uint64_t e0 = chunk * kChunk;
    const uint32_t nelem = (n - e0 < kChunk) ? static_cast<uint32_t>(n - e0) : kChunk;
    const uint32_t nwin = (nelem + kWindow - 1) / kWindow;

    // ---- the chunk's byte range, validated ----------------------------------
    const uint64_t lo = __ldg(table + chunk);
    const uint64_t hi = __ldg(table + chunk + 1);
    bool ok = (lo <= hi) && (hi <= src_bytes) && (hi - lo >= 4ull * nwin) &&
              (hi - lo <= 4ull * nwin + static_cast<uint64_t>(S) * nelem) && (lo % S == 0) &&
              ((hi - lo) % S == 0);
    if (chunk == 0 && lo != 0) ok = false;
    if (chunk == num_chunks - 1 && hi != src_bytes) ok = false;
    if (!ok) {
        if (lane == 0) report_status(ws, CDMA_ERR_CORRUPT_STREAM);
        return;
    }

    // ---- stage payload bytes [lo, hi) in shared memory -----------------------
    uint8_t* buf = s_buf[warp];
    const uint64_t a0 = lo & ~15ull;              // buf[0] corresponds to payload byte a0
    for (uint64_t a = a0 + 16ull * lane; a < hi; a += 16ull * 32) {
        uint4 q;
        if (a + 16 <= src_bytes) {
            q = __ldcs(reinterpret_cast<const uint4*>(src + a));
        } else {
            // last, partial 16 bytes of the payload: never read past src_bytes
            uint32_t wds[4] = {0, 0, 0, 0};
            for (uint32_t b = 0; b < 16; b += 2) {
                if (a + b + 2 <= src_bytes) {
                    const uint32_t h = *reinterpret_cast<const uint16_t*>(src + a + b);
                    wds[b >> 2] |= h << (8 * (b & 2));
                }
            }
            q = make_uint4(wds[0], wds[1], wds[2], wds[3]);
        }
        *reinterpret_cast<uint4*>(buf + (a - a0)) = q;
    }
    // Blocks are dispatched in index order, so the chunk `kPrefetchAheadCtas` blocks
    // further on will be expanded by a warp that starts about one CTA lifetime from
    // now: ask L2 for its table entries (by reading them) and its payload bytes now.
    // Nothing depends on this and every line still comes from DRAM exactly once.
    // Worth its instructions only where the payload is a sizeable part of the traffic:
    // the launcher picks this variant by the payload-to-dense ratio.
    if (PREFETCH && kPrefetchAheadCtas != 0) {
        const uint64_t cf = chunk + static_cast<uint64_t>(kPrefetchAheadCtas) * kDecWarps;
        if (cf < num_chunks) {
            const uint64_t flo = __ldg(table + cf);
            const uint64_t fhi = __ldg(table + cf + 1);
            if (flo <= fhi && fhi <= src_bytes && fhi - flo <= kMaxChunkBytes) {
                for (uint64_t a = (flo & ~127ull) + 128ull * lane; a < fhi; a += 128ull * 32)
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(src + a));
            }
        }
    }
    __syncwarp();

    // ---- walk the records and expand ----------------------------------------
    const T* units = reinterpret_cast<const T*>(buf);
    uint32_t p = static_cast<uint32_t>(lo - a0) / S;        // position in units of S bytes
    const uint32_t end = static_cast<uint32_t>(hi - a0) / S;
    bool bad = false;

    if (nelem == kChunk && S == 2) {
        // full chunk of 2-byte elements: 16 rounds of 2 windows; a half-warp expands a
        // window, a lane 2 consecutive elements (one 4-byte store per lane, 128
        // contiguous bytes per warp).  Fewer instructions per element than the 4-byte
        // scheme below, which matters here: with half the bytes per element this
        // kernel is bound by instruction issue, not by DRAM.
        const uint32_t half = lane >> 4;
        const uint32_t sh = 2u * (lane & 15u);
        const uint32_t below = (1u << sh) - 1u;
        uint32_t* out = reinterpret_cast<uint32_t*>(dst + e0) + lane;
#pragma unroll
        for (uint32_t g = 0; g < kChunkWindows / 2; ++g) {
            const uint32_t pa = p;
            const uint32_t ma = static_cast<uint32_t>(units[p]) | (static_cast<uint32_t>(units[p + 1]) << 16);
            p += MU + __popc(ma);
            const uint32_t pb = p;
            const uint32_t mb = static_cast<uint32_t>(units[p]) | (static_cast<uint32_t>(units[p + 1]) << 16);
            p += MU + __popc(mb);
            // a malformed record may carry the walk past the chunk: flag it and pull the
            // position back (every second round) so that no later read leaves the buffer
            if (g & 1u) { bad |= (p > end); p = min(p, end); }
            const uint32_t my_m = half ? mb : ma;
            const uint32_t q = (half ? pb : pa) + MU + __popc(my_m & below);
            const uint32_t two = (my_m >> sh) & 3u;
            const uint32_t v0 = units[q], v1 = units[q + (two & 1u)];
            __stcs(out + g * 32, ((two & 1u) ? v0 : 0u) | ((two & 2u) ? (v1 << 16) : 0u));
        }
    } else if (nelem == kChunk) {
        // full chunk: 8 rounds of 4 windows; lane = 4 consecutive elements
        const uint32_t sub = lane & 7u;
        const uint32_t wj = lane >> 3;
        const uint32_t below = (1u << (4 * sub)) - 1u;
        T* out = dst + e0 + 4 * lane;
#pragma unroll
        for (uint32_t g = 0; g < kChunk / 128; ++g) {
            // four serial steps of the self-delimiting walk; every lane sees all four
            uint32_t pw[4], mw[4];
#pragma unroll
            for (uint32_t j = 0; j < 4; ++j) {
                pw[j] = p;
                if (S == 4) mw[j] = units[p];
                else mw[j] = static_cast<uint32_t>(units[p]) | (static_cast<uint32_t>(units[p + 1]) << 16);
                p += MU + __popc(mw[j]);
                // a malformed record may carry the walk past the chunk: flag it and pull
                // the position back so that no later read leaves the staged bytes
                if (kClampEveryWindow) { bad |= (p > end); p = min(p, end); }
            }
            if (!kClampEveryWindow) { bad |= (p > end); p = min(p, end); }
            const uint32_t my_p = (wj == 0) ? pw[0] : (wj == 1) ? pw[1] : (wj == 2) ? pw[2] : pw[3];
            const uint32_t my_m = (wj == 0) ? mw[0] : (wj == 1) ? mw[1] : (wj == 2) ? mw[2] : mw[3];
            const uint32_t nib = (my_m >> (4 * sub)) & 15u;
            const uint32_t q = my_p + MU + __popc(my_m & below);
            // element k takes the value numbered by the set bits below bit k
            const uint32_t c1 = nib & 1u, c2 = __popc(nib & 3u), c3 = __popc(nib & 7u);
            const uint32_t a0v = units[q], a1v = units[q + c1], a2v = units[q + c2], a3v = units[q + c3];
            store4(out + g * 128, (nib & 1u) ? a0v : 0u, (nib & 2u) ? a1v : 0u, (nib & 4u) ? a2v : 0u,
                   (nib & 8u) ? a3v : 0u);
        }
    } else {
        // ragged last chunk: lane = element, one window per round
        const uint32_t lt = lanemask_lt();
        T* out = dst + e0 + lane;
        for (uint32_t w = 0; w < nwin; ++w) {
            if (p + MU > end) { bad = true; break; }
            uint32_t m;
            if (S == 4) m = units[p];
            else m = static_cast<uint32_t>(units[p]) | (static_cast<uint32_t>(units[p + 1]) << 16);
            const uint32_t cnt = __popc(m);
            const uint32_t left = nelem - w * kWindow;           // elements this window really has
            if (p + MU + cnt > end || (left < kWindow && (m >> left) != 0)) { bad = true; break; }
            const bool bit = (m >> lane) & 1u;
            const T val = bit ? units[p + MU + __popc(m & lt)] : T(0);
            if (lane < left) out[w * kWindow] = val;
            p += MU + cnt;
        }
    }
    if (!bad && p != end) bad = true;
    if (bad && lane == 0) report_status(ws, CDMA_ERR_CORRUPT_STREAM);
}

}  // namespace

cudaError_t launch_zvc_decompress(const void* d_src, uint64_t src_bytes, const uint64_t* d_table,
                                  uint64_t n, uint32_t elem_size, void* d_dst, uint64_t* d_ws,
                                  cudaStream_t stream, bool src_on_device) {
    const uint64_t chunks = num_chunks_of(n);
    if (chunks == 0) return cudaSuccess;
    const dim3 grid(static_cast<unsigned>((chunks + kDecWarps - 1) / kDecWarps));
    timing_before_launch(stream);
    if (elem_size == 4) {
        // payload at least a fifth of the dense bytes: reading it is a real share of the traffic
        const bool prefetch = src_on_device && src_bytes >= (n * 4) / 5;
        auto kernel = prefetch ? zvc_decompress_kernel<uint32_t, true> : zvc_decompress_kernel<uint32_t, false>;
        kernel<<<grid, kDecThreads, 0, stream>>>(static_cast<const uint8_t*>(d_src), src_bytes, d_table, n,
                                                 static_cast<uint32_t*>(d_dst), d_ws, chunks);
    } else {
        zvc_decompress_kernel<uint16_t, false><<<grid, kDecThreads, 0, stream>>>(
            static_cast<const uint8_t*>(d_src), src_bytes, d_table, n, static_cast<uint16_t*>(d_dst),
            d_ws, chunks);
    }
    timing_after_launch(stream);
    count_kernel_launch();
    return cudaGetLastError();
}

}  // namespace cdma
