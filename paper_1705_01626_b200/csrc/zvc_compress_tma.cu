// Zero-value compression (Section V-A), the kernel for tensors that live in device
// memory: one thread owns one row of 128 bytes of the input -- one window of 32
// four-byte elements, or two windows of 32 two-byte elements -- so that the whole
// record of a window (compare, count, shift, append: the stages of Section V-B,
// Fig. 10a) is built by one thread from its own registers, with no work repeated
// across lanes.
//
// A CTA compresses a tile of 256 rows (32 KB).  Order of work:
//   1. load: one TMA tensor copy brings the tile into shared memory (128-byte
//      swizzle, so that thread t's reads of row t do not collide with its
//      neighbours'); each thread then takes its row into 32 registers;
//   2. count: mask(s) and number of non-zero elements per thread; a scan over the
//      CTA gives every record its place in the tile, and the tile's size is
//      published at once for the tiles behind it (single-pass decoupled look-back);
//   3. assemble: each thread appends its mask and its non-zero elements to the
//      staged tile (in place of the input, which now lives in registers);
//   4. look back: warp 0 finds the tile's place in the stream;
//   5. copy: the CTA moves the staged bytes to the payload with aligned 16-byte
//      stores, realigning in registers (the payload offset of a tile is only a
//      multiple of the element size).
#include <cuda.h>

#include "zvc_common.cuh"
#include "lookback.cuh"

namespace cdma {

namespace {

constexpr uint32_t kRows = kTileThreads;               // rows of 128 bytes per tile, one per thread
constexpr uint32_t kRowBytes = 128;
constexpr uint32_t kStageBytes = kRows * 136 + 32;     // largest tile output (2-byte elements, all non-zero) + slack
constexpr uint32_t kTmaPrefetchAhead = 370;            // tiles; see prefetch note in the kernel

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

// ---- 4-byte elements -------------------------------------------------------------------------
// mask bit I and the running count of element e: two instructions
template <uint32_t I>
__device__ __forceinline__ void flag_u32(uint32_t& mask, uint32_t e) {
    asm("{\n\t.reg .b32 d;\n\tmin.u32 d, %1, 1;\n\tmad.lo.u32 %0, d, %2, %0;\n\t}" : "+r"(mask) : "r"(e), "n"(1u << I));
}
// append element e at q + 4 if it is non-zero: three instructions
__device__ __forceinline__ void append_u32(uint32_t& q, uint32_t e) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %1, 0;\n\t@p st.shared.u32 [%0+4], %1;\n\t@p add.u32 %0, %0, 4;\n\t}"
                 : "+r"(q) : "r"(e) : "memory");
}

// ---- 2-byte elements -------------------------------------------------------------------------
// flags of the two halves of w at bits J and 16 + J: two instructions
template <uint32_t J>
__device__ __forceinline__ void flag_pair_u16(uint32_t& acc, uint32_t w) {
    asm("{\n\t.reg .b32 d;\n\tmin.u16x2 d, %1, %2;\n\tmad.lo.u32 %0, d, %3, %0;\n\t}"
        : "+r"(acc) : "r"(w), "r"(0x00010001u), "n"(1u << J));
}
// bits 0..15 of x to the even positions, bits 16..31 to the odd ones (a perfect shuffle):
// turns {flags of the low halves | flags of the high halves} into the window's mask
__device__ __forceinline__ uint32_t interleave16(uint32_t x) {
    uint32_t t;
    t = (x ^ (x >> 8)) & 0x0000ff00u;  x ^= t ^ (t << 8);
    t = (x ^ (x >> 4)) & 0x00f000f0u;  x ^= t ^ (t << 4);
    t = (x ^ (x >> 2)) & 0x0c0c0c0cu;  x ^= t ^ (t << 2);
    t = (x ^ (x >> 1)) & 0x22222222u;  x ^= t ^ (t << 1);
    return x;
}
// append the non-zero halves of w (low half first) at q + 4
__device__ __forceinline__ void append_pair_u16(uint32_t& q, uint32_t w) {
    asm volatile("{\n\t.reg .pred p, r;\n\t.reg .b32 t, h;\n\t"
                 "and.b32 t, %1, 0xffff;\n\tsetp.ne.u32 p, t, 0;\n\t"
                 "@p st.shared.u16 [%0+4], %1;\n\t@p add.u32 %0, %0, 2;\n\t"
                 "shr.u32 h, %1, 16;\n\tsetp.ne.u32 r, h, 0;\n\t"
                 "@r st.shared.u16 [%0+4], h;\n\t@r add.u32 %0, %0, 2;\n\t}"
                 : "+r"(q) : "r"(w) : "memory");
}
__device__ __forceinline__ void sts_mask_u16(uint32_t q, uint32_t m) {
    asm volatile("{\n\t.reg .b32 h;\n\tshr.u32 h, %1, 16;\n\tst.shared.u16 [%0], %1;\n\tst.shared.u16 [%0+2], h;\n\t}"
                 ::"r"(q), "r"(m) : "memory");
}

// Bounded wait for the tile to land.  Returns false when the limit ran out.
__device__ __forceinline__ bool wait_tile(uint32_t mbar, uint64_t limit_ns) {
    uint32_t done = 0;
    uint32_t polls = 0;
    uint64_t t0 = 0;
    while (true) {
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(mbar) : "memory");
        if (done) return true;
        if ((++polls & 63u) == 0) {
            const uint64_t now = global_timer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit_ns || polls > kWaitLimitPolls) return false;
        }
    }
}

// Aligned 16-byte vector j of the payload region this tile writes, taken from the
// staged bytes: the staged tile starts `ph` bytes into vector 0, so vector j is the
// 16 bytes at staged offset 16 j - ph, i.e. the words a .. a+3 (plus a 16-bit shift
// for 2-byte elements) of the two aligned shared-memory vectors around it.
template <uint32_t A, bool HALF>
__device__ __forceinline__ uint4 realign(const uint4& lo, const uint4& hi) {
    const uint32_t w[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
    if (!HALF) return make_uint4(w[A], w[A + 1], w[A + 2], w[A + 3]);
    // A + 4 <= 7 for A <= 3; the half shift never comes with A = 4 (ph = 0 has no shift)
    return make_uint4(__funnelshift_r(w[A], w[A + 1], 16), __funnelshift_r(w[A + 1], w[A + 2], 16),
                      __funnelshift_r(w[A + 2], w[A + 3], 16), __funnelshift_r(w[A + 3], w[(A + 4) & 7], 16));
}

template <uint32_t A, bool HALF>
__device__ __forceinline__ void copy_body(uint32_t s_stage, uint4* __restrict__ g, uint32_t j0, uint32_t j1) {
    // vector j needs the aligned shared-memory vectors j - 1 and j (only j when the phase is zero)
    for (uint32_t j = j0 + threadIdx.x; j < j1; j += kTileThreads) {
        const uint4 hi = lds128(s_stage + 16u * j);
        uint4 out = hi;
        if (A != 4 || HALF) {
            const uint4 lo = lds128(s_stage + 16u * j - 16u);
            out = realign<A, HALF>(lo, hi);
        }
        g[j] = out;
    }
}

// S = element size.  The grid is one CTA per tile; tiles follow the block index and
// blocks are dispatched in that order, so a tile only ever waits for blocks that were
// dispatched before it (the assumption single-pass scans rest on); should it ever not
// hold, the bounded wait in the walk turns it into CDMA_ERR_TIMEOUT.
template <uint32_t S>
__global__ void __launch_bounds__(kTileThreads, 4)
zvc_compress_tma_kernel(const __grid_constant__ CUtensorMap tmap, const uint8_t* __restrict__ src, uint64_t n,
                        uint8_t* __restrict__ dst, uint64_t cap, uint64_t* __restrict__ table,
                        uint64_t* __restrict__ ws, const LaunchCtl ctl, uint32_t num_tiles, uint64_t num_chunks,
                        uint64_t full_rows) {
    constexpr uint32_t kWinPerRow = 4 / S;                       // 1 or 2 windows per 128-byte row
    constexpr uint32_t kElemPerRow = kRowBytes / S;
    extern __shared__ __align__(1024) uint8_t smem_raw[];          // input tile, then the staged output
    __shared__ __align__(8) uint64_t s_mbar;
    __shared__ uint32_t s_warp_bytes[kTileThreads / 32];
    __shared__ uint64_t s_base;
    __shared__ uint32_t s_failed;
    __shared__ uint32_t s_room;

    const uint32_t tid = threadIdx.x;
    const uint32_t lane = tid & 31u;
    const uint32_t warp = tid >> 5;
    const uint32_t tile = blockIdx.x;
    const uint32_t s_stage = smem_u32(smem_raw);
    const uint32_t mbar = smem_u32(&s_mbar);
    const uint64_t row0 = static_cast<uint64_t>(tile) * kRows;

    // ---- 1. load -------------------------------------------------------------------------------
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(mbar) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    if (tid == 0) {
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(mbar), "r"(kTileBytes) : "memory");
        // rows past the end of the tensor map (the last tile only) arrive as zeros
        asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                     ::"r"(s_stage), "l"(&tmap), "r"(0), "r"(static_cast<int32_t>(row0)), "r"(mbar) : "memory");
    } else if (tid == 32) {
        // The tile kTmaPrefetchAhead places further on will be picked up by a CTA that starts about half
        // a CTA lifetime from now; asking L2 for it now turns that CTA's load into L2 hits.  Every line
        // still comes from DRAM exactly once.
        const uint64_t prow = row0 + static_cast<uint64_t>(kTmaPrefetchAhead) * kRows;
        if (prow + kRows <= full_rows)
            asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];"
                         ::"l"(&tmap), "r"(0), "r"(static_cast<int32_t>(prow)) : "memory");
    }
    bool landed = wait_tile(mbar, ctl.wait_limit_ns);
    if (!landed) {
        // the copy is late beyond the limit: give it one more bounded wait so that it cannot write into
        // shared memory this CTA has already handed back, then fail the launch the way a look-back
        // time-out does (the tile marks itself so that the tiles behind it stop as well)
        landed = wait_tile(mbar, ctl.wait_limit_ns);
        if (tid == 0) {
            publish_prefix(ws, ctl, tile, true, 0);
            if (tile == num_tiles - 1) publish_result(ws, ctl, 0, CDMA_ERR_TIMEOUT);
        }
        return;
    }

    // thread t takes row t: eight 16-byte pieces, piece i stored at position i ^ (t & 7) by the swizzle
    uint32_t e[32];
    {
        const uint32_t row_addr = s_stage + kRowBytes * tid;
        const uint32_t sw = tid & 7u;
#pragma unroll
        for (uint32_t i = 0; i < 8; ++i) {
            const uint4 v = lds128(row_addr + 16u * (i ^ sw));
            e[4 * i + 0] = v.x; e[4 * i + 1] = v.y; e[4 * i + 2] = v.z; e[4 * i + 3] = v.w;
        }
    }
    const uint64_t row = row0 + tid;
    // windows of this row that exist (the tensor may end inside the last tile)
    const uint64_t total_windows = (n + kWindow - 1) / kWindow;
    const uint64_t w_first = row * kWinPerRow;
    const uint32_t nwin = w_first >= total_windows ? 0u
                          : (total_windows - w_first >= kWinPerRow ? kWinPerRow : static_cast<uint32_t>(total_windows - w_first));
    if (row >= full_rows && nwin != 0) {
        // the one row that is only partly inside the tensor: plain guarded loads
        const uint64_t e0 = row * kElemPerRow;
#pragma unroll
        for (uint32_t i = 0; i < 32; ++i) {
            if (S == 4) {
                const uint64_t j = e0 + i;
                e[i] = j < n ? reinterpret_cast<const uint32_t*>(src)[j] : 0u;
            } else {
                const uint64_t j = e0 + 2 * i;
                const uint32_t lo = j < n ? reinterpret_cast<const uint16_t*>(src)[j] : 0u;
                const uint32_t hi = j + 1 < n ? reinterpret_cast<const uint16_t*>(src)[j + 1] : 0u;
                e[i] = lo | (hi << 16);
            }
        }
    }

    // ---- 2. count ------------------------------------------------------------------------------
    uint32_t mask_a = 0, mask_b = 0;
    uint32_t rec_bytes;
    if (S == 4) {
        flag_u32<0>(mask_a, e[0]);   flag_u32<1>(mask_a, e[1]);   flag_u32<2>(mask_a, e[2]);   flag_u32<3>(mask_a, e[3]);
        flag_u32<4>(mask_a, e[4]);   flag_u32<5>(mask_a, e[5]);   flag_u32<6>(mask_a, e[6]);   flag_u32<7>(mask_a, e[7]);
        flag_u32<8>(mask_a, e[8]);   flag_u32<9>(mask_a, e[9]);   flag_u32<10>(mask_a, e[10]); flag_u32<11>(mask_a, e[11]);
        flag_u32<12>(mask_a, e[12]); flag_u32<13>(mask_a, e[13]); flag_u32<14>(mask_a, e[14]); flag_u32<15>(mask_a, e[15]);
        flag_u32<16>(mask_a, e[16]); flag_u32<17>(mask_a, e[17]); flag_u32<18>(mask_a, e[18]); flag_u32<19>(mask_a, e[19]);
        flag_u32<20>(mask_a, e[20]); flag_u32<21>(mask_a, e[21]); flag_u32<22>(mask_a, e[22]); flag_u32<23>(mask_a, e[23]);
        flag_u32<24>(mask_a, e[24]); flag_u32<25>(mask_a, e[25]); flag_u32<26>(mask_a, e[26]); flag_u32<27>(mask_a, e[27]);
        flag_u32<28>(mask_a, e[28]); flag_u32<29>(mask_a, e[29]); flag_u32<30>(mask_a, e[30]); flag_u32<31>(mask_a, e[31]);
        rec_bytes = nwin ? 4u + 4u * __popc(mask_a) : 0u;
    } else {
        uint32_t fa = 0, fb = 0;
        flag_pair_u16<0>(fa, e[0]);   flag_pair_u16<1>(fa, e[1]);   flag_pair_u16<2>(fa, e[2]);   flag_pair_u16<3>(fa, e[3]);
        flag_pair_u16<4>(fa, e[4]);   flag_pair_u16<5>(fa, e[5]);   flag_pair_u16<6>(fa, e[6]);   flag_pair_u16<7>(fa, e[7]);
        flag_pair_u16<8>(fa, e[8]);   flag_pair_u16<9>(fa, e[9]);   flag_pair_u16<10>(fa, e[10]); flag_pair_u16<11>(fa, e[11]);
        flag_pair_u16<12>(fa, e[12]); flag_pair_u16<13>(fa, e[13]); flag_pair_u16<14>(fa, e[14]); flag_pair_u16<15>(fa, e[15]);
        flag_pair_u16<0>(fb, e[16]);  flag_pair_u16<1>(fb, e[17]);  flag_pair_u16<2>(fb, e[18]);  flag_pair_u16<3>(fb, e[19]);
        flag_pair_u16<4>(fb, e[20]);  flag_pair_u16<5>(fb, e[21]);  flag_pair_u16<6>(fb, e[22]);  flag_pair_u16<7>(fb, e[23]);
        flag_pair_u16<8>(fb, e[24]);  flag_pair_u16<9>(fb, e[25]);  flag_pair_u16<10>(fb, e[26]); flag_pair_u16<11>(fb, e[27]);
        flag_pair_u16<12>(fb, e[28]); flag_pair_u16<13>(fb, e[29]); flag_pair_u16<14>(fb, e[30]); flag_pair_u16<15>(fb, e[31]);
        mask_a = interleave16(fa);
        mask_b = interleave16(fb);
        rec_bytes = (nwin > 0 ? 4u + 2u * __popc(mask_a) : 0u) + (nwin > 1 ? 4u + 2u * __popc(mask_b) : 0u);
    }
    // place of every thread's record(s) in the tile: scan over the warp, then over the warps
    uint32_t incl = rec_bytes;
#pragma unroll
    for (uint32_t o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) s_warp_bytes[warp] = incl;
    __syncthreads();                       // also: every thread has its row in registers, the tile may be overwritten
    const uint32_t wb = (lane < kTileThreads / 32) ? s_warp_bytes[lane] : 0u;
    const uint32_t warp_off = __reduce_add_sync(0xffffffffu, lane < warp ? wb : 0u);
    uint64_t tile_bytes = 0;
    if (warp == 0) {
        tile_bytes = __reduce_add_sync(0xffffffffu, wb);
        // the tile's size is public before any record is assembled
        if (lane == 0) publish_aggregate(ws, ctl, tile, tile_bytes);
    }
    const uint32_t rec_off = warp_off + incl - rec_bytes;       // byte offset of my record(s) in the staged tile

    // ---- 3. assemble -----------------------------------------------------------------------------
    uint32_t q = s_stage + rec_off;
    if (S == 4) {
        if (nwin) {
            asm volatile("st.shared.u32 [%0], %1;" ::"r"(q), "r"(mask_a) : "memory");
#pragma unroll
            for (uint32_t i = 0; i < 32; ++i) append_u32(q, e[i]);
        }
    } else {
        if (nwin > 0) {
            sts_mask_u16(q, mask_a);
#pragma unroll
            for (uint32_t i = 0; i < 16; ++i) append_pair_u16(q, e[i]);
            q += 4;
        }
        if (nwin > 1) {
            sts_mask_u16(q, mask_b);
#pragma unroll
            for (uint32_t i = 16; i < 32; ++i) append_pair_u16(q, e[i]);
        }
    }

    // ---- 4. the tile's place in the stream -------------------------------------------------------
    if (warp == 0)
        resolve_tile(ws, ctl, tile, num_tiles, tile_bytes, cap, table, num_chunks, &s_base, &s_failed, &s_room);
    __syncthreads();
    if (s_failed) return;
    const uint64_t base = s_base;

    // offset-table entries: a chunk is 32 windows = 32 rows (4-byte elements) or 16 rows (2-byte)
    if (S == 4) {
        const uint64_t chunk = static_cast<uint64_t>(tile) * (kRows / 32) + warp;
        if (lane == 0 && chunk < num_chunks) table[chunk] = base + rec_off;
    } else {
        const uint64_t chunk = static_cast<uint64_t>(tile) * (kRows / 16) + 2 * warp + (lane >> 4);
        if ((lane & 15u) == 0 && chunk < num_chunks) table[chunk] = base + rec_off;
    }

    // ---- 5. copy the staged bytes to their place, below the capacity ------------------------------
    const uint32_t room = s_room & ~(S - 1u);                    // whole elements
    const uint32_t ph = static_cast<uint32_t>(base) & 15u;        // where the tile starts inside its first vector
    uint8_t* gdst = dst + base;
    // head: the bytes in front of the first aligned vector; tail: those behind the last one
    const uint32_t head = ph ? min(16u - ph, room) : 0u;
    const uint32_t nvec = (room - head) / 16u;
    const uint32_t tail = room - head - 16u * nvec;
    if (tid < head / S) {
        if (S == 4) reinterpret_cast<uint32_t*>(gdst)[tid] = reinterpret_cast<const uint32_t*>(smem_raw)[tid];
        else reinterpret_cast<uint16_t*>(gdst)[tid] = reinterpret_cast<const uint16_t*>(smem_raw)[tid];
    } else if (tid >= 32 && tid - 32 < tail / S) {
        const uint32_t o = (head + 16u * nvec) / S + (tid - 32);
        if (S == 4) reinterpret_cast<uint32_t*>(gdst)[o] = reinterpret_cast<const uint32_t*>(smem_raw)[o];
        else reinterpret_cast<uint16_t*>(gdst)[o] = reinterpret_cast<const uint16_t*>(smem_raw)[o];
    }
    // body: aligned vector j of the payload (counted from the vector the tile starts in) holds the
    // staged bytes 16 j - ph .. 16 j - ph + 15
    uint4* g = reinterpret_cast<uint4*>(gdst - ph);
    const uint32_t j0 = ph ? 1u : 0u, j1 = j0 + nvec;
    switch (ph >> 1) {
        case 0: copy_body<4, false>(s_stage, g, j0, j1); break;
        case 2: copy_body<3, false>(s_stage - 16u + 16u, g, j0, j1); break;   // ph = 4: words 3.. of vector j - 1
        case 4: copy_body<2, false>(s_stage, g, j0, j1); break;              // ph = 8
        case 6: copy_body<1, false>(s_stage, g, j0, j1); break;              // ph = 12
        default:
            if (S == 2) {
                switch (ph >> 1) {
                    case 1: copy_body<3, true>(s_stage, g, j0, j1); break;   // ph = 2
                    case 3: copy_body<2, true>(s_stage, g, j0, j1); break;   // ph = 6
                    case 5: copy_body<1, true>(s_stage, g, j0, j1); break;   // ph = 10
                    case 7: copy_body<0, true>(s_stage, g, j0, j1); break;   // ph = 14
                }
            }
    }
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

bool zvc_compress_tma_usable(const void* d_src, uint64_t n, uint32_t elem_size) {
    // at least one whole tile, rows addressable with 32-bit coordinates, and an encoder to describe them
    const uint64_t full_rows = n * elem_size / kRowBytes;
    return full_rows >= kRows && full_rows < (1ull << 31) && (reinterpret_cast<uintptr_t>(d_src) & 15) == 0 &&
           encode_tiled() != nullptr;
}

cudaError_t launch_zvc_compress_tma(const void* d_src, uint64_t n, uint32_t elem_size, void* d_dst, uint64_t cap,
                                    uint64_t* d_table, uint64_t* d_ws, const LaunchCtl& ctl, cudaStream_t stream) {
    const uint64_t bytes = n * elem_size;
    const uint64_t full_rows = bytes / kRowBytes;
    const uint64_t tiles = (bytes + kTileBytes - 1) / kTileBytes;
    // the tensor as rows of 32 words; a box is one tile; 128-byte swizzle
    CUtensorMap tmap;
    const cuuint64_t dims[2] = {kRowBytes / 4, full_rows};
    const cuuint64_t strides[1] = {kRowBytes};
    const cuuint32_t box[2] = {kRowBytes / 4, kRows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = encode_tiled()(&tmap, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<void*>(d_src), dims, strides,
                                      box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                      CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    auto kernel = elem_size == 4 ? zvc_compress_tma_kernel<4> : zvc_compress_tma_kernel<2>;
    const cudaError_t oe = opt_in_shared_memory(reinterpret_cast<const void*>(kernel), kStageBytes);
    if (oe != cudaSuccess) return oe;
    timing_before_launch(stream);
    kernel<<<static_cast<unsigned>(tiles), kTileThreads, kStageBytes, stream>>>(
        tmap, static_cast<const uint8_t*>(d_src), n, static_cast<uint8_t*>(d_dst), cap, d_table, d_ws, ctl,
        static_cast<uint32_t>(tiles), num_chunks_of(n), full_rows);
    timing_after_launch(stream);
    count_kernel_launch();
    return cudaGetLastError();
}

}  // namespace cdma
