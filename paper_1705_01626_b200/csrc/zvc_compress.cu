// Zero-value compression, one pass over the input (Section V-A; the compare /
// prefix-sum / shift / append stages of the engine in Section V-B, Fig. 10a).
//
// One CTA compresses one tile of kTileChunks chunks; one warp owns one chunk
// (32 windows of 32 elements).  Lane = element: a warp load of 32 consecutive
// elements is one window, __ballot_sync of "bit pattern != 0" is its mask,
// __popc of the mask below a lane is that element's slot among the window's
// non-zeros.  Record sizes are scanned inside the warp and the CTA; the
// running byte offset across tiles comes from a single-pass decoupled
// look-back over 64-bit {state,value} descriptors, in ticket order so that a
// tile only ever waits for tiles that are already running.  The tile's records
// are assembled in shared memory at the same 16-byte phase as their place in
// the payload and written out with 16-byte stores.
#include "zvc_common.cuh"

namespace cdma {

namespace {

struct LookbackResult {
    uint64_t exclusive;   // bytes of all earlier tiles
    bool failed;
};

// Warp-wide look-back executed by warp 0 of the CTA.  Every lane inspects one
// predecessor per round.  Waiting is bounded: when the limit is hit the tile
// marks itself failed so that every later tile stops waiting too.
__device__ LookbackResult decoupled_lookback(uint64_t* desc, uint64_t* ws, uint32_t tile,
                                             uint64_t aggregate) {
    const uint32_t lane = lane_id();
    LookbackResult r{0, false};
    if (tile == 0) {
        if (lane == 0) st_relaxed_u64(desc, kDescPrefix | aggregate);
        return r;
    }
    if (lane == 0) st_relaxed_u64(desc + tile, kDescAggregate | aggregate);

    int64_t look = static_cast<int64_t>(tile) - 1;   // lane l inspects tile look - l
    uint32_t polls = 0;
    uint64_t t_start = 0;
    while (true) {
        const int64_t idx = look - static_cast<int64_t>(lane);
        // before tile 0 there is nothing: an inclusive prefix of zero
        const uint64_t d = (idx >= 0) ? ld_relaxed_u64(desc + idx) : kDescPrefix;
        const uint32_t state = static_cast<uint32_t>(d >> 62);
        const uint32_t is_invalid = __ballot_sync(0xffffffffu, state == 0);
        const uint32_t is_prefix = __ballot_sync(0xffffffffu, state == 2);
        const uint32_t is_error = __ballot_sync(0xffffffffu, state == 3);
        // lanes up to and including the nearest tile that already knows its prefix
        const uint32_t first = is_prefix & (0u - is_prefix);
        const uint32_t upto = is_prefix ? (first | (first - 1u)) : 0xffffffffu;
        if (is_error & upto) {
            r.failed = true;
            break;
        }
        if (is_invalid & upto) {
            if (polls == 0) t_start = global_timer_ns();
            ++polls;
            if (polls > kWaitLimitPolls || (global_timer_ns() - t_start) > kWaitLimitNs) {
                if (lane == 0) report_status(ws, CDMA_ERR_TIMEOUT);
                r.failed = true;
                break;
            }
            __nanosleep(polls < 16 ? 32 : 256);
            continue;
        }
        uint64_t v = ((upto >> lane) & 1u) ? (d & kDescValueMask) : 0ull;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        r.exclusive += v;
        if (is_prefix) break;
        look -= 32;
    }
    if (lane == 0) {
        st_relaxed_u64(desc + tile, r.failed ? kDescError
                                             : (kDescPrefix | (r.exclusive + aggregate)));
    }
    return r;
}

template <typename T>
__global__ void __launch_bounds__(kTileThreads)
zvc_compress_kernel(const T* __restrict__ src, uint64_t n, uint8_t* __restrict__ dst, uint64_t cap,
                    uint64_t* __restrict__ table, uint64_t* __restrict__ ws, uint32_t num_tiles,
                    uint64_t num_chunks) {
    constexpr uint32_t S = sizeof(T);
    constexpr uint32_t kMaxChunkBytes = 4 * kChunkWindows + S * kChunk;
    __shared__ __align__(16) uint8_t stage[kTileChunks * kMaxChunkBytes + 16];
    __shared__ uint32_t s_tile;
    __shared__ uint32_t s_chunk_bytes[kTileChunks];
    __shared__ uint32_t s_chunk_off[kTileChunks];
    __shared__ uint32_t s_tile_bytes;
    __shared__ uint64_t s_base;
    __shared__ uint32_t s_failed;

    const uint32_t lane = lane_id();
    const uint32_t warp = threadIdx.x >> 5;
    uint64_t* desc = ws + kWsDescriptors;

    // Tiles are handed out in the order CTAs start running.
    if (threadIdx.x == 0) s_tile = atomicAdd(reinterpret_cast<unsigned int*>(ws + kWsTicket), 1u);
    __syncthreads();
    const uint32_t tile = s_tile;
    if (tile >= num_tiles) return;

    // ---- load: 32 windows of this warp's chunk, lane = element -------------
    const uint64_t chunk = static_cast<uint64_t>(tile) * kTileChunks + warp;
    const uint64_t e0 = chunk * kChunk;
    uint32_t nwin;   // windows this chunk really has
    T v[kChunkWindows];
    if (e0 + kChunk <= n) {
        nwin = kChunkWindows;
        const T* p = src + e0 + lane;
#pragma unroll
        for (uint32_t w = 0; w < kChunkWindows; ++w) v[w] = __ldcs(p + w * kWindow);
    } else {
        const uint64_t left = (e0 < n) ? (n - e0) : 0;
        nwin = static_cast<uint32_t>((left + kWindow - 1) / kWindow);
#pragma unroll
        for (uint32_t w = 0; w < kChunkWindows; ++w) {
            const uint64_t j = static_cast<uint64_t>(w) * kWindow + lane;
            v[w] = (j < left) ? __ldcs(src + e0 + j) : T(0);
        }
    }

    // ---- masks: lane w keeps the mask of window w ---------------------------
    uint32_t my_mask = 0;
#pragma unroll
    for (uint32_t w = 0; w < kChunkWindows; ++w) {
        const uint32_t m = __ballot_sync(0xffffffffu, v[w] != T(0));
        if (lane == w) my_mask = m;
    }

    // ---- record sizes and their exclusive scan inside the chunk -------------
    const uint32_t my_rec = (lane < nwin) ? (4u + S * __popc(my_mask)) : 0u;
    uint32_t incl = my_rec;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= static_cast<uint32_t>(o)) incl += t;
    }
    const uint32_t my_off = incl - my_rec;
    if (lane == 31) s_chunk_bytes[warp] = incl;
    __syncthreads();

    // ---- chunk offsets inside the tile, then the tile's place in the stream -
    if (warp == 0) {
        const uint32_t cb = (lane < kTileChunks) ? s_chunk_bytes[lane] : 0u;
        uint32_t ci = cb;
#pragma unroll
        for (int o = 1; o < static_cast<int>(kTileChunks); o <<= 1) {
            const uint32_t t = __shfl_up_sync(0xffffffffu, ci, o);
            if (lane >= static_cast<uint32_t>(o)) ci += t;
        }
        if (lane < kTileChunks) s_chunk_off[lane] = ci - cb;
        const uint32_t tile_bytes = __shfl_sync(0xffffffffu, ci, kTileChunks - 1);
        const LookbackResult lb = decoupled_lookback(desc, ws, tile, tile_bytes);
        if (lane == 0) {
            s_tile_bytes = tile_bytes;
            s_base = lb.exclusive;
            s_failed = lb.failed ? 1u : 0u;
        }
    }
    __syncthreads();
    if (s_failed) return;

    const uint64_t base = s_base;
    const uint32_t tile_bytes = s_tile_bytes;
    const uint32_t chunk_off = s_chunk_off[warp];

    if (lane == 0 && chunk < num_chunks) table[chunk] = base + chunk_off;
    if (tile == num_tiles - 1 && threadIdx.x == 0) {
        table[num_chunks] = base + tile_bytes;
        ws[kWsBytes] = base + tile_bytes;
    }
    if (threadIdx.x == 0 && base + tile_bytes > cap) report_status(ws, CDMA_ERR_BUFFER_TOO_SMALL);

    // ---- assemble the records in shared memory ------------------------------
    // Byte b of the tile's output sits at stage[phase + b], phase = base mod 16,
    // so that 16-byte groups of the payload are 16-byte groups of `stage`.
    const uint32_t phase = static_cast<uint32_t>(base & 15u);
    T* out = reinterpret_cast<T*>(stage + phase + chunk_off);   // S divides every offset
    const uint32_t lt = lanemask_lt();
#pragma unroll
    for (uint32_t w = 0; w < kChunkWindows; ++w) {
        const uint32_t m = __shfl_sync(0xffffffffu, my_mask, w);
        const uint32_t off = __shfl_sync(0xffffffffu, my_off, w) / S;
        if (w < nwin) {
            if (S == 4) {
                if (lane == 0) out[off] = static_cast<T>(m);
            } else {
                if (lane < 2) out[off + lane] = static_cast<T>(m >> (16 * lane));
            }
            if ((m >> lane) & 1u) out[off + 4 / S + __popc(m & lt)] = v[w];
        }
    }
    __syncthreads();

    // ---- write the tile's bytes [base, base + tile_bytes) below cap ---------
    const uint64_t g0 = base;
    const uint64_t g1 = (base + tile_bytes < cap) ? (base + tile_bytes) : cap;
    if (g0 >= g1) return;
    const uint64_t a0 = g0 & ~15ull;                 // stage[0] corresponds to payload byte a0
    const uint32_t nvec = static_cast<uint32_t>((g1 - a0 + 15) >> 4);
    for (uint32_t i = threadIdx.x; i < nvec; i += kTileThreads) {
        const uint64_t ga = a0 + 16ull * i;
        if (ga >= g0 && ga + 16 <= g1) {
            __stcs(reinterpret_cast<uint4*>(dst + ga), *reinterpret_cast<const uint4*>(stage + 16u * i));
        } else {
            // ragged edge of the tile: element-sized stores, clipped to [g0, g1)
#pragma unroll
            for (uint32_t b = 0; b < 16; b += S) {
                const uint64_t gb = ga + b;
                if (gb >= g0 && gb < g1)
                    *reinterpret_cast<T*>(dst + gb) = *reinterpret_cast<const T*>(stage + 16u * i + b);
            }
        }
    }
}

}  // namespace

cudaError_t launch_zvc_compress(const void* d_src, uint64_t n, uint32_t elem_size, void* d_dst,
                                uint64_t cap, uint64_t* d_table, uint64_t* d_ws,
                                cudaStream_t stream) {
    const uint64_t chunks = num_chunks_of(n);
    const uint64_t tiles = num_tiles_of(n);
    if (tiles == 0) return cudaSuccess;
    const dim3 grid(static_cast<unsigned>(tiles));
    if (elem_size == 4) {
        zvc_compress_kernel<uint32_t><<<grid, kTileThreads, 0, stream>>>(
            static_cast<const uint32_t*>(d_src), n, static_cast<uint8_t*>(d_dst), cap, d_table, d_ws,
            static_cast<uint32_t>(tiles), chunks);
    } else {
        zvc_compress_kernel<uint16_t><<<grid, kTileThreads, 0, stream>>>(
            static_cast<const uint16_t*>(d_src), n, static_cast<uint8_t*>(d_dst), cap, d_table, d_ws,
            static_cast<uint32_t>(tiles), chunks);
    }
    count_kernel_launch();
    return cudaGetLastError();
}

}  // namespace cdma
