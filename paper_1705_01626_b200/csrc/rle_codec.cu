// Run-length comparison codec (Section V-A, "Run-length encoding compression";
// its layout sensitivity is the subject of Section VI-A, Fig. 11), 4-byte elements.
//
// The paper gives no format.  Ours, on the framing of the zero-value codec
// (independent chunks of 1024 elements, offset table outside the payload): a
// chunk is a sequence of records {token, literals}; the 32-bit token holds the
// number of zero elements in front (low 16 bits) and the number of non-zero
// elements that follow (high 16 bits); a record is written for every maximal run
// of non-zero elements, and a chunk that ends in zeros gets a last record with
// no literals.  Chunk size = 4 * records + 4 * non-zero elements.
//
// Compression uses the tile / look-back skeleton of the zero-value kernel: one
// CTA per 8-chunk tile, a warp per chunk, a lane holds one element of each of
// the chunk's 32 windows, window masks by ballot.  Decompression: a warp per
// chunk walks the tokens (the walk is serial: a token says where the next one
// is), zero-fills its chunk of the output and stores each record's literals over
// the zeros (never outside the chunk, whatever the stream holds).
#include "zvc_common.cuh"
#include "lookback.cuh"

namespace cdma {

namespace {

// r runs need r non-zeros and r - 1 zeros between them, so tokens + literals <= 1025 words per chunk
constexpr uint32_t kRleMaxChunkUnits = kChunk + 1;
constexpr uint32_t kBig = 0x7fffffffu;

__global__ void __launch_bounds__(kTileThreads, 4)
rle_compress_kernel(const uint32_t* __restrict__ src, uint64_t n, uint8_t* __restrict__ dst, uint64_t cap,
                    uint64_t* __restrict__ table, uint64_t* __restrict__ ws, const LaunchCtl ctl,
                    uint32_t num_tiles, uint64_t num_chunks) {
    extern __shared__ __align__(16) uint8_t smem_raw[];
    uint32_t* s_tile = reinterpret_cast<uint32_t*>(smem_raw);       // the tile's records, contiguous
    __shared__ uint32_t s_chunk_units[kTileChunks];
    __shared__ uint32_t s_next_zero[kTileChunks][kChunkWindows];    // first zero at or after window w + 1
    __shared__ uint64_t s_base;
    __shared__ uint32_t s_failed;
    __shared__ uint32_t s_room;

    const uint32_t lane = lane_id();
    const uint32_t warp = threadIdx.x >> 5;
    const uint32_t lt = lanemask_lt();
    const uint32_t tile = blockIdx.x;          // block-index order, as in the zero-value kernel
    if (tile >= num_tiles) return;
    if (threadIdx.x == 0) prefetch_future_descriptor(ws, tile, num_tiles);

    // ---- load: lane l takes element l of every window; beyond n: zeros -------------
    const uint64_t chunk = static_cast<uint64_t>(tile) * kTileChunks + warp;
    const uint64_t e0 = chunk * kChunk;
    const uint32_t nelem = (e0 >= n) ? 0u : (n - e0 < kChunk ? static_cast<uint32_t>(n - e0) : kChunk);
    uint32_t e[kChunkWindows];
#pragma unroll
    for (uint32_t w = 0; w < kChunkWindows; ++w) {
        const uint32_t j = w * kWindow + lane;
        e[w] = (j < nelem) ? __ldcs(src + e0 + j) : 0u;
    }

    // ---- 1. count: window masks by ballot, lane w keeps the mask of window w --------
    uint32_t mine = 0;
#pragma unroll
    for (uint32_t w = 0; w < kChunkWindows; ++w) {
        const uint32_t m = __ballot_sync(0xffffffffu, e[w] != 0u);
        if (lane == w) mine = m;
    }
    // lane = window from here: run starts are non-zero elements whose predecessor is zero
    uint32_t carry = __shfl_up_sync(0xffffffffu, mine >> 31, 1);
    if (lane == 0) carry = 0;
    const uint32_t starts = mine & ~((mine << 1) | carry);
    const uint32_t nnz = __reduce_add_sync(0xffffffffu, __popc(mine));
    const uint32_t runs = __reduce_add_sync(0xffffffffu, __popc(starts));
    uint32_t trailing = 0;                                          // the chunk ends in zeros
    if (nelem != 0) {
        const uint32_t last_mask = __shfl_sync(0xffffffffu, mine, (nelem - 1) >> 5);
        trailing = ((last_mask >> ((nelem - 1) & 31u)) & 1u) ^ 1u;
    }
    const uint32_t units = runs + trailing + nnz;
    // first zero at or after each window (suffix minimum), for the run lengths
    uint32_t fz = (mine != 0xffffffffu) ? lane * kWindow + (__ffs(~mine) - 1) : kBig;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_down_sync(0xffffffffu, fz, o);
        if (lane + o < 32) fz = min(fz, t);
    }
    uint32_t after = __shfl_down_sync(0xffffffffu, fz, 1);          // from window lane + 1 on
    if (lane == 31) after = kBig;
    s_next_zero[warp][lane] = min(after, nelem);
    if (lane == 0) s_chunk_units[warp] = units;
    __syncthreads();
    const uint32_t cu = (lane < kTileChunks) ? s_chunk_units[lane] : 0u;
    const uint32_t chunk_off = __reduce_add_sync(0xffffffffu, lane < warp ? cu : 0u);
    uint64_t tile_bytes = 0;
    if (warp == 0) {
        tile_bytes = static_cast<uint64_t>(__reduce_add_sync(0xffffffffu, cu)) * 4u;
        if (lane == 0) publish_aggregate(ws, ctl, tile, tile_bytes);
    }

    // ---- 2. assemble the chunk's records in the staged tile --------------------------
    uint32_t* st = s_tile + chunk_off;
    uint32_t nnz_run = 0, runs_run = 0;          // non-zeros and run starts in front of this window
    int32_t last_nz = -1;                        // index of the last non-zero element in front of it
    uint32_t prev_top = 0;                       // bit 31 of the previous window's mask
#pragma unroll
    for (uint32_t w = 0; w < kChunkWindows; ++w) {
        const uint32_t m = __ballot_sync(0xffffffffu, e[w] != 0u);
        const uint32_t sw = m & ~((m << 1) | prev_top);
        const uint32_t i = w * kWindow + lane;                      // my element's index in the chunk
        // my place: one word per record started up to and including me, one per non-zero before me
        const uint32_t pos = runs_run + __popc(sw & (lt | (1u << lane))) + nnz_run + __popc(m & lt);
        // (no branch: every lane works out the token its element would start; only run starts store it)
        const uint32_t lower = m & lt;
        const uint32_t zeros = lower ? (lane - 1u - (31u - __clz(lower)))
                                     : static_cast<uint32_t>(static_cast<int32_t>(i) - 1 - last_nz);
        const uint32_t higher_zeros = ~m & ~(lt | (1u << lane));
        const uint32_t beyond = s_next_zero[warp][w];
        const uint32_t run_end = higher_zeros ? w * kWindow + (__ffs(higher_zeros) - 1) : beyond;
        const uint32_t s_addr = static_cast<uint32_t>(__cvta_generic_to_shared(st + pos));
        asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 p, %1, 0;\n\t@p st.shared.u32 [%0], %1;\n\t"
                     "setp.ne.u32 q, %3, 0;\n\t@q st.shared.u32 [%0+-4], %2;\n\t}"
                     ::"r"(s_addr), "r"(e[w]), "r"(zeros | ((run_end - i) << 16)), "r"((sw >> lane) & 1u) : "memory");
        nnz_run += __popc(m);
        runs_run += __popc(sw);
        if (m) last_nz = static_cast<int32_t>(w * kWindow + 31u - __clz(m));
        prev_top = m >> 31;
    }
    if (trailing && lane == 0) st[units - 1] = nelem - 1u - static_cast<uint32_t>(last_nz);   // zeros only

    // ---- 3. the tile's place in the stream ------------------------------------------
    if (warp == 0)
        resolve_tile(ws, ctl, tile, num_tiles, tile_bytes, cap, table, num_chunks, &s_base, &s_failed, &s_room);
    __syncthreads();
    if (s_failed) return;

    // ---- 4. the CTA writes the tile's words to their place, below cap ----------------
    const uint64_t first_unit = s_base / 4u;
    if (lane == 0 && chunk < num_chunks) table[chunk] = (first_unit + chunk_off) * 4u;
    const uint32_t room = s_room / 4u;           // whole words below the capacity
    uint32_t* out = reinterpret_cast<uint32_t*>(dst) + first_unit;
    for (uint32_t u = threadIdx.x; u < room; u += kTileThreads) out[u] = s_tile[u];
}

constexpr uint32_t kRleDecWarps = 8;

__global__ void __launch_bounds__(32 * kRleDecWarps)
rle_decompress_kernel(const uint8_t* __restrict__ src, uint64_t src_bytes, const uint64_t* __restrict__ table,
                      uint64_t n, uint32_t* __restrict__ dst, uint64_t* __restrict__ ws, const LaunchCtl ctl,
                      uint64_t num_chunks) {
    // staged payload (16-byte phase in front)
    constexpr uint32_t kStageWords = kRleMaxChunkUnits + 4 + 3;
    __shared__ __align__(16) uint32_t s_stage[kRleDecWarps][(kStageWords + 3) / 4 * 4];

    const uint32_t lane = lane_id();
    const uint32_t warp = threadIdx.x >> 5;
    const uint64_t chunk = static_cast<uint64_t>(blockIdx.x) * kRleDecWarps + warp;
    if (blockIdx.x == 0 && threadIdx.x == 0) init_decode_result(ws, ctl, n * 4u);
    if (chunk >= num_chunks) return;
    const uint64_t e0 = chunk * kChunk;
    const uint32_t nelem = (n - e0 < kChunk) ? static_cast<uint32_t>(n - e0) : kChunk;

    // ---- the chunk's byte range, validated ---------------------------------------------
    const uint64_t lo = __ldg(table + chunk);
    const uint64_t hi = __ldg(table + chunk + 1);
    const uint64_t len64 = hi - lo;
    bool ok = (lo <= hi) && (hi <= src_bytes) && (len64 >= 4) && (len64 <= 4ull * kRleMaxChunkUnits) &&
              (((static_cast<uint32_t>(lo) | static_cast<uint32_t>(len64)) & 3u) == 0u);
    if (chunk == 0 && lo != 0) ok = false;
    if (chunk == num_chunks - 1 && hi != src_bytes) ok = false;
    if (!ok) {
        if (lane == 0) report_decode_error(ws, ctl, CDMA_ERR_CORRUPT_STREAM);
        return;
    }

    // ---- stage payload bytes [lo, hi); zero the dense chunk -----------------------------
    uint32_t* buf = s_stage[warp];
    uint32_t* dense = dst + e0;                  // zero-filled first, literals stored over the zeros
    const uint64_t a0 = lo & ~15ull;
    const uint32_t span = static_cast<uint32_t>(hi - a0);
    for (uint32_t off = 16u * lane; off < span; off += 16u * 32u) {
        uint4 q = make_uint4(0, 0, 0, 0);
        if (a0 + off + 16 <= src_bytes) {
            q = __ldcs(reinterpret_cast<const uint4*>(src + a0 + off));
        } else {
            uint32_t wds[4] = {0, 0, 0, 0};
            for (uint32_t b = 0; b < 16; b += 4)
                if (a0 + off + b + 4 <= src_bytes) wds[b >> 2] = *reinterpret_cast<const uint32_t*>(src + a0 + off + b);
            q = make_uint4(wds[0], wds[1], wds[2], wds[3]);
        }
        *reinterpret_cast<uint4*>(buf + off / 4) = q;
    }
    if (nelem == kChunk) {
#pragma unroll
        for (uint32_t k = 0; k < kChunk / 128; ++k) reinterpret_cast<uint4*>(dense)[k * 32 + lane] = make_uint4(0, 0, 0, 0);
    } else {
        for (uint32_t j = lane; j < nelem; j += 32) dense[j] = 0u;
    }
    __syncwarp();                                // the zeros are ordered before this warp's literal stores

    // ---- walk the records: every lane sees every token; lanes share a record's literals ----
    uint32_t p = static_cast<uint32_t>(lo - a0) / 4u;
    const uint32_t end = span / 4u;
    uint32_t pos = 0;
    bool bad = false;
    uint32_t zero_literal = 0;                   // per lane: a literal that is zero was seen
    while (pos < nelem) {
        // (reading one word past `end` is harmless: the staging buffer has room and the
        // checks below refuse whatever it holds)
        const uint32_t token = buf[min(p, end)];
        const uint32_t zeros = token & 0xffffu, count = token >> 16;
        if (p >= end || token == 0u || pos + zeros + count > nelem || p + 1 + count > end) { bad = true; break; }
        const uint32_t from = p + 1 + lane, to = pos + zeros + lane;
        if (lane < count) {                      // runs of up to 32 literals: one step
            const uint32_t v = buf[from];
            zero_literal |= (v == 0u) ? 1u : 0u;
            dense[to] = v;
        }
        for (uint32_t j = 32; j < count; j += 32) {
            if (lane + j < count) {
                const uint32_t v = buf[from + j];
                zero_literal |= (v == 0u) ? 1u : 0u;
                dense[to + j] = v;
            }
        }
        p += 1 + count;
        pos += zeros + count;
    }
    bad |= zero_literal != 0u;
    bad = __any_sync(0xffffffffu, bad) || p != end;
    if (bad && lane == 0) report_decode_error(ws, ctl, CDMA_ERR_CORRUPT_STREAM);
}

}  // namespace

cudaError_t launch_rle_compress(const void* d_src, uint64_t n, void* d_dst, uint64_t cap, uint64_t* d_table,
                                uint64_t* d_ws, const LaunchCtl& ctl, cudaStream_t stream) {
    const uint64_t chunks = num_chunks_of(n);
    const uint64_t tiles = num_tiles_of(n);
    if (tiles == 0) return cudaSuccess;
    constexpr uint32_t kSmem = kTileChunks * kRleMaxChunkUnits * 4;
    const cudaError_t e = opt_in_shared_memory(reinterpret_cast<const void*>(rle_compress_kernel), kSmem);
    if (e != cudaSuccess) return e;
    timing_before_launch(stream);
    rle_compress_kernel<<<static_cast<unsigned>(tiles), kTileThreads, kSmem, stream>>>(
        static_cast<const uint32_t*>(d_src), n, static_cast<uint8_t*>(d_dst), cap, d_table, d_ws, ctl,
        static_cast<uint32_t>(tiles), chunks);
    timing_after_launch(stream);
    count_kernel_launch();
    return cudaGetLastError();
}

cudaError_t launch_rle_decompress(const void* d_src, uint64_t src_bytes, const uint64_t* d_table, uint64_t n,
                                  void* d_dst, uint64_t* d_ws, const LaunchCtl& ctl, cudaStream_t stream) {
    const uint64_t chunks = num_chunks_of(n);
    if (chunks == 0) return cudaSuccess;
    const dim3 grid(static_cast<unsigned>((chunks + kRleDecWarps - 1) / kRleDecWarps));
    timing_before_launch(stream);
    rle_decompress_kernel<<<grid, 32 * kRleDecWarps, 0, stream>>>(static_cast<const uint8_t*>(d_src), src_bytes,
                                                                   d_table, n, static_cast<uint32_t*>(d_dst), d_ws,
                                                                   ctl, chunks);
    timing_after_launch(stream);
    count_kernel_launch();
    return cudaGetLastError();
}

}  // namespace cdma
