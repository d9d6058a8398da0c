// Zero-value compression, one pass over the input (Section V-A; the compare /
// prefix-sum / shift / append stages of the engine in Section V-B, Fig. 10a).
//
// One CTA compresses one tile of kTileChunks chunks; one warp owns one chunk
// (32 windows of 32 elements).  4-byte elements: a lane holds one element of
// every window, so a window's mask is one warp ballot.  2-byte elements: a lane
// holds 8 consecutive elements (4 lanes per window, masks by xor-shuffles) and
// a warp owns two chunks.
//
// Order of work inside a CTA, chosen so that the one step that depends on other
// CTAs (the running byte offset across tiles) waits as little as possible:
//   1. count: the tile's size needs only the number of non-zeros, so it is
//      reduced and published at once, before any record exists;
//   2. assemble: mask words and non-zero values go to shared memory; the
//      pop-count of the mask bits below an element is the slot of its value;
//   3. look back: warp 0 walks the 64-bit {state,value} descriptors of earlier
//      tiles (single-pass decoupled look-back, 32 per round); tiles follow the
//      block index, so a tile only ever waits for blocks dispatched before it;
//      by now its predecessors have had the whole of step 2 to publish;
//   4. copy: the staged bytes go to their place in the payload with coalesced
//      stores.
#include "zvc_common.cuh"
#include "lookback.cuh"

namespace cdma {

namespace {

// Tiles follow the block index and blocks are dispatched in that order, so the
// tile `kPrefetchAhead` places further on will be picked up by a CTA that starts
// about half a CTA lifetime from now (5 CTAs x 148 SMs are resident at a time).
// Asking L2 for it now turns that CTA's DRAM-latency load phase into L2 hits;
// every line is still fetched from DRAM exactly once.
constexpr uint32_t kPrefetchAhead = 370;

__device__ __forceinline__ void prefetch_future_tile(const void* src, uint64_t total_bytes, uint32_t tile) {
    const uint64_t off = (static_cast<uint64_t>(tile) + kPrefetchAhead) * kTileBytes + 128ull * threadIdx.x;
    if (off + 128 <= total_bytes)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(static_cast<const uint8_t*>(src) + off));
}

// ReLU on bit patterns, NaN-propagating: an element is kept when it is greater
// than zero or a NaN (of either sign); everything else -- negatives, -0.0, +0.0,
// -Inf -- becomes +0.  `nan_above` is the largest magnitude pattern that is not a
// NaN (0x7f800000 for fp32, 0x7c00 for fp16, 0x7f80 for bf16).
__device__ __forceinline__ uint32_t relu_bits32(uint32_t e) {
    const bool keep = (static_cast<int32_t>(e) > 0) || ((e & 0x7fffffffu) > 0x7f800000u);
    return keep ? e : 0u;
}
__device__ __forceinline__ uint32_t relu_bits16(uint32_t h, uint32_t nan_above) {
    const bool keep = ((h & 0x8000u) == 0u && h != 0u) || ((h & 0x7fffu) > nan_above);
    return keep ? h : 0u;
}

// Records of one chunk into shared memory, one window per step: the ballot of
// "my element is non-zero" IS the window's mask (compare stage), the pop-count of
// the mask bits below a lane is the slot of its value (prefix-sum and shift
// stages), lane 0 appends the mask word itself.  Returns the units written.
// One window of a chunk, written as one block of PTX so that it stays at nine
// instructions (the kernel is bound by instruction issue, not by DRAM, once the
// loads are prefetched): compare, ballot, mask store (all lanes, same address,
// same value), rank = popc(mask & lanes below), predicated value store, record
// length.  `a` is the shared-memory byte address of the window's record minus
// 4*W, so that the 4 bytes of every mask word in front fold into the immediate
// offsets; no branch, hence no reconvergence point in front of the ballot.
template <uint32_t W>
__device__ __forceinline__ void assemble_window(uint32_t& a, uint32_t e, uint32_t lt) {
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        ".reg .b32 m, t, q;\n\t"
        "setp.ne.u32 p, %1, 0;\n\t"
        "vote.sync.ballot.b32 m, p, 0xffffffff;\n\t"
        "st.shared.u32 [%0+%3], m;\n\t"
        "and.b32 t, m, %2;\n\t"
        "popc.b32 t, t;\n\t"
        "mad.lo.u32 q, t, 4, %0;\n\t"
        "@p st.shared.u32 [q+%4], %1;\n\t"
        "popc.b32 t, m;\n\t"
        "mad.lo.u32 %0, t, 4, %0;\n\t"
        "}"
        : "+r"(a)
        : "r"(e), "r"(lt), "n"(4 * W), "n"(4 * W + 4)
        : "memory");
}

template <uint32_t W>
__device__ __forceinline__ void assemble_windows(uint32_t& a, const uint32_t (&e)[kChunkWindows], uint32_t nwin,
                                                 uint32_t lt) {
    if constexpr (W < kChunkWindows) {
        if (W < nwin) {                     // uniform; always true for a full chunk
            assemble_window<W>(a, e[W], lt);
            assemble_windows<W + 1>(a, e, nwin, lt);
        }
    }
}

// Number of non-zero elements among a lane's 32: min(e, 1) added up (a compare and a
// predicated add per element came out at more than twice the instructions).
__device__ __forceinline__ void count_nonzero(uint32_t& cnt, uint32_t e) {
    asm("{\n\t.reg .b32 d;\n\tmin.u32 d, %1, 1;\n\tadd.u32 %0, %0, d;\n\t}" : "+r"(cnt) : "r"(e));
}

// 4-byte elements.  A lane holds one element of each of the chunk's 32 windows
// (warp loads are 128 contiguous bytes), so a window's mask is one warp ballot.
// The tile's records are staged contiguously in shared memory -- each chunk at
// the offset the count step gave it -- and the whole CTA then copies them out
// with stores that each cover one aligned 128-byte line.
//
// When RELU is set the kernel compresses max(x, 0) instead of x (the activation
// function whose output the paper offloads, Section IV) and, if relu_out is not
// null, also writes the dense activation map for the next layer -- the input is
// read once for both.
// FULL: every chunk of the tile has all 1024 elements (true for every tile but
// possibly the last); the two cases are separate straight-line instantiations so
// that the common one carries no trace of the ragged one.
template <bool RELU, bool FULL>
__device__ __forceinline__ void compress_tile_u32(const uint32_t* __restrict__ src, uint64_t n,
                                                  uint8_t* __restrict__ dst, uint64_t cap,
                                                  uint64_t* __restrict__ table, uint64_t* __restrict__ ws,
                                                  const LaunchCtl& ctl, uint32_t num_tiles, uint64_t num_chunks,
                                                  uint32_t* __restrict__ relu_out, uint32_t tile) {
    constexpr uint32_t S = 4;
    extern __shared__ __align__(16) uint8_t smem_raw[];
    uint32_t* s_tile = reinterpret_cast<uint32_t*>(smem_raw);   // up to kTileChunks * 1056 units
    __shared__ uint32_t s_chunk_units[kTileChunks];
    __shared__ uint64_t s_base;
    __shared__ uint32_t s_failed;
    __shared__ uint32_t s_room;

    const uint32_t lane = lane_id();
    const uint32_t warp = threadIdx.x >> 5;
    const uint32_t lt = lanemask_lt();

    // ---- load the warp's chunk: 32 loads per lane, all in flight --------------
    const uint64_t chunk = static_cast<uint64_t>(tile) * kTileChunks + warp;
    const uint64_t e0 = chunk * kChunk;
    uint32_t nwin = kChunkWindows;   // windows this chunk really has
    uint32_t e[kChunkWindows];
    if (FULL) {
        const uint32_t* p = src + e0 + lane;
#pragma unroll
        for (uint32_t w = 0; w < kChunkWindows; ++w) e[w] = __ldcs(p + w * kWindow);
        if (RELU) {
#pragma unroll
            for (uint32_t w = 0; w < kChunkWindows; ++w) {
                e[w] = relu_bits32(e[w]);
                if (relu_out != nullptr) relu_out[e0 + lane + w * kWindow] = e[w];
            }
        }
    } else {
        const uint64_t left = (e0 < n) ? (n - e0) : 0;
        nwin = static_cast<uint32_t>(((left < kChunk ? left : kChunk) + kWindow - 1) / kWindow);
#pragma unroll
        for (uint32_t w = 0; w < kChunkWindows; ++w) {
            const uint64_t j = static_cast<uint64_t>(w) * kWindow + lane;
            e[w] = (j < left) ? __ldcs(src + e0 + j) : 0u;
            if (RELU) {
                e[w] = relu_bits32(e[w]);
                if (relu_out != nullptr && j < left) relu_out[e0 + j] = e[w];
            }
        }
    }

    // ---- 1. count: the tile's size needs only the number of non-zeros ---------
    uint32_t mine = 0;
#pragma unroll
    for (uint32_t w = 0; w < kChunkWindows; ++w) count_nonzero(mine, e[w]);
    const uint32_t units = nwin + __reduce_add_sync(0xffffffffu, mine);
    if (lane == 0) s_chunk_units[warp] = units;
    __syncthreads();
    // every warp sums the chunks in front of its own; warp 0 also needs the total
    const uint32_t cu = (lane < kTileChunks) ? s_chunk_units[lane] : 0u;
    const uint32_t chunk_off = __reduce_add_sync(0xffffffffu, lane < warp ? cu : 0u);
    uint64_t tile_bytes = 0;
    if (warp == 0) {
        tile_bytes = static_cast<uint64_t>(__reduce_add_sync(0xffffffffu, cu)) * S;
        // the tile's size is public before any record is assembled
        if (lane == 0) publish_aggregate(ws, ctl, tile, tile_bytes);
    }

    // ---- 2. assemble the chunk's records at its place in the staged tile ------
    // (a recursive template rather than a loop, so that the window number is an immediate)
    uint32_t a = static_cast<uint32_t>(__cvta_generic_to_shared(s_tile + chunk_off));
    assemble_windows<0>(a, e, FULL ? kChunkWindows : nwin, lt);

    // ---- 3. the tile's place in the stream ------------------------------------
    if (warp == 0)
        resolve_tile(ws, ctl, tile, num_tiles, tile_bytes, cap, table, num_chunks, &s_base, &s_failed, &s_room);
    __syncthreads();
    if (s_failed) return;

    // ---- 4. the CTA writes the tile's bytes to their place, below cap ---------
    const uint64_t first_unit = s_base / S;
    if (lane == 0 && chunk < num_chunks) table[chunk] = (first_unit + chunk_off) * S;
    const uint32_t room = s_room / S;                            // whole units below the capacity
    // Row r of the copy is the aligned 128-byte line r of the destination that the
    // tile touches: thread t moves unit u = t - mis + r * kTileThreads, where mis is
    // how far the tile's first unit sits inside its line; only row 0 can have u < 0.
    const uint32_t mis = static_cast<uint32_t>(first_unit) & 31u;
    const uint32_t* sp = s_tile + threadIdx.x - mis;            // never dereferenced below s_tile
    uint32_t* gp = reinterpret_cast<uint32_t*>(dst) + first_unit + threadIdx.x - mis;
    int32_t left = static_cast<int32_t>(room) + static_cast<int32_t>(mis) - static_cast<int32_t>(threadIdx.x);
    // `left` > 0 <=> this thread's unit of the current row is below the end of the tile
    if (threadIdx.x >= mis && left > 0) *gp = *sp;
    left -= kTileThreads; sp += kTileThreads; gp += kTileThreads;
    while (left > 3 * static_cast<int32_t>(kTileThreads)) {
        const uint32_t v0 = sp[0], v1 = sp[kTileThreads], v2 = sp[2 * kTileThreads], v3 = sp[3 * kTileThreads];
        gp[0] = v0; gp[kTileThreads] = v1; gp[2 * kTileThreads] = v2; gp[3 * kTileThreads] = v3;
        left -= 4 * kTileThreads; sp += 4 * kTileThreads; gp += 4 * kTileThreads;
    }
    while (left > 0) {
        *gp = *sp;
        left -= kTileThreads; sp += kTileThreads; gp += kTileThreads;
    }
}

template <typename T, bool RELU>
__global__ void __launch_bounds__(kTileThreads, kMinCtasPerSm)
zvc_compress_kernel(const T* __restrict__ src, uint64_t n, uint8_t* __restrict__ dst, uint64_t cap,
                    uint64_t* __restrict__ table, uint64_t* __restrict__ ws, const LaunchCtl ctl,
                    uint32_t num_tiles, uint64_t num_chunks, T* __restrict__ relu_out, uint32_t nan_above,
                    uint64_t prefetch_bytes) {
    static_assert(sizeof(T) == 4, "2-byte elements have a kernel of their own");
    // Tile = block index.  Thread blocks are dispatched in increasing index order,
    // so every tile this one will wait for belongs to a block that is already
    // running or finished (the assumption single-pass scans rest on); should it
    // ever not hold, the bounded wait in the walk turns it into CDMA_ERR_TIMEOUT.
    const uint32_t tile = blockIdx.x;
    if (tile >= num_tiles) return;
    prefetch_future_tile(src, prefetch_bytes, tile);
    if (threadIdx.x == 0) prefetch_future_descriptor(ws, tile, num_tiles);
    if ((static_cast<uint64_t>(tile) + 1) * (kTileChunks * kChunk) <= n)
        compress_tile_u32<RELU, true>(src, n, dst, cap, table, ws, ctl, num_tiles, num_chunks, relu_out, tile);
    else
        compress_tile_u32<RELU, false>(src, n, dst, cap, table, ws, ctl, num_tiles, num_chunks, relu_out, tile);
}

// 2-byte elements: a lane holds 8 consecutive elements (one 16-byte load), so a
// warp instruction covers 8 windows (4 lanes per window), and a warp owns two
// chunks, so that a tile is as many bytes (32 KB) as in the 4-byte kernel.  The
// steps are the same; masks come from xor-shuffles over the 4 lanes of a window,
// record positions from a shuffle-up scan over the 8 windows of a group.  The
// inner pieces are blocks of PTX for the same reason as in the 4-byte kernel:
// with half the bytes per element this kernel is bound by instruction issue.
constexpr uint32_t kTileChunksU16 = 2 * kTileChunks;
constexpr uint32_t kGroupsU16 = kChunk / 256;                   // 256 elements per warp load

// "Non-zero" flags of the two halves of w, or-ed into bits at LO and HI.
template <uint32_t LO, uint32_t HI>
__device__ __forceinline__ void flag_pair_u16(uint32_t& bits, uint32_t w) {
    asm("{\n\t.reg .pred p, q;\n\t.reg .b32 t;\n\t"
        "and.b32 t, %1, 0xffff;\n\tsetp.ne.u32 p, t, 0;\n\t@p or.b32 %0, %0, %2;\n\t"
        "setp.gt.u32 q, %1, 0xffff;\n\t@q or.b32 %0, %0, %3;\n\t}"
        : "+r"(bits) : "r"(w), "n"(LO), "n"(HI));
}

// Append the non-zero halves of w (low half first) at shared byte address q + 4
// (q points at the window's mask word), advancing q by 2 per value stored.  The
// 16-bit stores take 32-bit registers (the low half is stored), and the position
// advances by 2 * min(half, 1): both measurably cheaper than 16-bit registers and
// predicated adds (18 -> 11 instructions per pair).
__device__ __forceinline__ void append_pair_u16(uint32_t& q, uint32_t w) {
    asm volatile("{\n\t.reg .pred p, r;\n\t.reg .b32 t, h, d;\n\t"
                 "and.b32 t, %1, 0xffff;\n\tsetp.ne.u32 p, t, 0;\n\t"
                 "@p st.shared.u16 [%0+4], %1;\n\t"
                 "min.u32 d, t, 1;\n\tmad.lo.u32 %0, d, 2, %0;\n\t"
                 "shr.u32 h, %1, 16;\n\tsetp.ne.u32 r, h, 0;\n\t"
                 "@r st.shared.u16 [%0+4], h;\n\t"
                 "min.u32 d, h, 1;\n\tmad.lo.u32 %0, d, 2, %0;\n\t}"
                 : "+r"(q) : "r"(w) : "memory");
}

// A 32-bit mask word at a 2-byte aligned shared address, by the lanes with `on` set
// (predicated stores, no branch in front of the next shuffles).
__device__ __forceinline__ void sts_mask_u16(uint32_t saddr, uint32_t v, uint32_t on) {
    asm volatile("{\n\t.reg .pred p;\n\t.reg .b32 h;\n\tsetp.ne.u32 p, %2, 0;\n\tshr.u32 h, %1, 16;\n\t"
                 "@p st.shared.u16 [%0], %1;\n\t@p st.shared.u16 [%0+2], h;\n\t}"
                 ::"r"(saddr), "r"(v), "r"(on) : "memory");
}

// Records of one chunk from its 32 flag bits per lane and the lane's 32 elements;
// `a` = shared byte address where the chunk's records start.  FULL: all 32
// windows exist; otherwise only the first nwin do (elements past the end were
// loaded as zeros, so only their mask records have to be suppressed).
template <bool FULL>
__device__ __forceinline__ void assemble_chunk_u16(uint32_t a, uint32_t bits, const uint32_t (&w)[kGroupsU16][4],
                                                   uint32_t lane, uint32_t nwin) {
    const uint32_t sub = lane & 3u;                       // which byte of the window's mask is mine
    const uint32_t below = (1u << (8u * sub)) - 1u;
    const uint32_t first = sub == 0u ? 1u : 0u;
#pragma unroll
    for (uint32_t g = 0; g < kGroupsU16; ++g) {
        uint32_t m = ((bits >> (8u * g)) & 0xffu) << (8u * sub);
        m |= __shfl_xor_sync(0xffffffffu, m, 1);
        m |= __shfl_xor_sync(0xffffffffu, m, 2);           // the window's 32-bit mask
        const bool live = FULL || (8u * g + (lane >> 2)) < nwin;
        const uint32_t rec = live ? 4u + 2u * __popc(m) : 0u;   // record length in bytes, same in 4 lanes
        uint32_t incl = rec;
        uint32_t t = __shfl_up_sync(0xffffffffu, incl, 4);
        if (lane >= 4) incl += t;
        t = __shfl_up_sync(0xffffffffu, incl, 8);
        if (lane >= 8) incl += t;
        t = __shfl_up_sync(0xffffffffu, incl, 16);
        if (lane >= 16) incl += t;                          // records of windows up to mine
        const uint32_t mine = a + incl - rec;               // where my window's record starts
        a += __shfl_sync(0xffffffffu, incl, 31);
        sts_mask_u16(mine, m, (FULL || live) ? first : 0u);
        uint32_t q = mine + 2u * __popc(m & below);
        append_pair_u16(q, w[g][0]);
        append_pair_u16(q, w[g][1]);
        append_pair_u16(q, w[g][2]);
        append_pair_u16(q, w[g][3]);
    }
}

template <bool RELU, bool FULL>
__device__ __forceinline__ void compress_tile_u16(const uint16_t* __restrict__ src, uint64_t n,
                                                  uint8_t* __restrict__ dst, uint64_t cap,
                                                  uint64_t* __restrict__ table, uint64_t* __restrict__ ws,
                                                  const LaunchCtl& ctl, uint32_t num_tiles, uint64_t num_chunks,
                                                  uint16_t* __restrict__ relu_out, uint32_t nan_above,
                                                  uint32_t tile) {
    constexpr uint32_t S = 2;
    extern __shared__ __align__(16) uint8_t smem_raw[];          // the tile's records, contiguous
    __shared__ uint32_t s_chunk_units[kTileChunksU16];
    __shared__ uint64_t s_base;
    __shared__ uint32_t s_failed;
    __shared__ uint32_t s_room;

    const uint32_t lane = lane_id();
    const uint32_t warp = threadIdx.x >> 5;

    // ---- load the warp's two chunks ------------------------------------------
    uint32_t nwin[2] = {kChunkWindows, kChunkWindows};
    uint32_t w[2][kGroupsU16][4];         // 8 elements of a group = 4 words of two halves
#pragma unroll
    for (uint32_t c = 0; c < 2; ++c) {
        const uint64_t e0 = (static_cast<uint64_t>(tile) * kTileChunksU16 + 2 * warp + c) * kChunk;
        if (FULL) {
            const uint16_t* p = src + e0 + 8 * lane;
#pragma unroll
            for (uint32_t g = 0; g < kGroupsU16; ++g) {
                const uint4 q = __ldcs(reinterpret_cast<const uint4*>(p + g * 256));
                w[c][g][0] = q.x; w[c][g][1] = q.y; w[c][g][2] = q.z; w[c][g][3] = q.w;
                if (RELU) {
#pragma unroll
                    for (uint32_t k = 0; k < 4; ++k)
                        w[c][g][k] = relu_bits16(w[c][g][k] & 0xffffu, nan_above) |
                                     (relu_bits16(w[c][g][k] >> 16, nan_above) << 16);
                    if (relu_out != nullptr)
                        *reinterpret_cast<uint4*>(relu_out + e0 + 8 * lane + g * 256) =
                            make_uint4(w[c][g][0], w[c][g][1], w[c][g][2], w[c][g][3]);
                }
            }
        } else {
            const uint64_t left = (e0 < n) ? (n - e0) : 0;
            nwin[c] = static_cast<uint32_t>(((left < kChunk ? left : kChunk) + kWindow - 1) / kWindow);
#pragma unroll
            for (uint32_t g = 0; g < kGroupsU16; ++g) {
#pragma unroll
                for (uint32_t k = 0; k < 4; ++k) {
                    const uint64_t j = static_cast<uint64_t>(g) * 256 + 8 * lane + 2 * k;
                    uint32_t lo = (j < left) ? static_cast<uint32_t>(__ldcs(src + e0 + j)) : 0u;
                    uint32_t hi = (j + 1 < left) ? static_cast<uint32_t>(__ldcs(src + e0 + j + 1)) : 0u;
                    if (RELU) {
                        lo = relu_bits16(lo, nan_above);
                        hi = relu_bits16(hi, nan_above);
                        if (relu_out != nullptr && j < left) relu_out[e0 + j] = static_cast<uint16_t>(lo);
                        if (relu_out != nullptr && j + 1 < left) relu_out[e0 + j + 1] = static_cast<uint16_t>(hi);
                    }
                    w[c][g][k] = lo | (hi << 16);
                }
            }
        }
    }

    // ---- 1. count: 8 "non-zero" bits per group, 4 groups in one word -----------
    uint32_t bits[2] = {0u, 0u};
    uint32_t units[2];
#pragma unroll
    for (uint32_t c = 0; c < 2; ++c) {
        flag_pair_u16<1u << 0, 1u << 1>(bits[c], w[c][0][0]);   flag_pair_u16<1u << 2, 1u << 3>(bits[c], w[c][0][1]);
        flag_pair_u16<1u << 4, 1u << 5>(bits[c], w[c][0][2]);   flag_pair_u16<1u << 6, 1u << 7>(bits[c], w[c][0][3]);
        flag_pair_u16<1u << 8, 1u << 9>(bits[c], w[c][1][0]);   flag_pair_u16<1u << 10, 1u << 11>(bits[c], w[c][1][1]);
        flag_pair_u16<1u << 12, 1u << 13>(bits[c], w[c][1][2]); flag_pair_u16<1u << 14, 1u << 15>(bits[c], w[c][1][3]);
        flag_pair_u16<1u << 16, 1u << 17>(bits[c], w[c][2][0]); flag_pair_u16<1u << 18, 1u << 19>(bits[c], w[c][2][1]);
        flag_pair_u16<1u << 20, 1u << 21>(bits[c], w[c][2][2]); flag_pair_u16<1u << 22, 1u << 23>(bits[c], w[c][2][3]);
        flag_pair_u16<1u << 24, 1u << 25>(bits[c], w[c][3][0]); flag_pair_u16<1u << 26, 1u << 27>(bits[c], w[c][3][1]);
        flag_pair_u16<1u << 28, 1u << 29>(bits[c], w[c][3][2]); flag_pair_u16<1u << 30, 1u << 31>(bits[c], w[c][3][3]);
        units[c] = 2 * nwin[c] + __reduce_add_sync(0xffffffffu, __popc(bits[c]));
        if (lane == 0) s_chunk_units[2 * warp + c] = units[c];
    }
    __syncthreads();
    // every warp sums the chunks in front of its own; warp 0 also needs the total
    const uint32_t cu = (lane < kTileChunksU16) ? s_chunk_units[lane] : 0u;
    const uint32_t chunk_off = __reduce_add_sync(0xffffffffu, lane < 2 * warp ? cu : 0u);
    uint64_t tile_bytes = 0;
    if (warp == 0) {
        tile_bytes = static_cast<uint64_t>(__reduce_add_sync(0xffffffffu, cu)) * S;
        // the tile's size is public before any record is assembled
        if (lane == 0) publish_aggregate(ws, ctl, tile, tile_bytes);
    }

    // ---- 2. assemble both chunks' records at their place in the staged tile ----
    const uint32_t s_addr = static_cast<uint32_t>(__cvta_generic_to_shared(smem_raw));
    assemble_chunk_u16<FULL>(s_addr + S * chunk_off, bits[0], w[0], lane, nwin[0]);
    assemble_chunk_u16<FULL>(s_addr + S * (chunk_off + units[0]), bits[1], w[1], lane, nwin[1]);

    // ---- 3. the tile's place in the stream ------------------------------------
    if (warp == 0)
        resolve_tile(ws, ctl, tile, num_tiles, tile_bytes, cap, table, num_chunks, &s_base, &s_failed, &s_room);
    __syncthreads();
    if (s_failed) return;

    // ---- 4. the CTA writes the tile's bytes to their place, below cap ---------
    const uint64_t base = s_base;
    if (lane < 2) {
        const uint64_t chunk = static_cast<uint64_t>(tile) * kTileChunksU16 + 2 * warp + lane;
        if (chunk < num_chunks) table[chunk] = base + S * (chunk_off + (lane ? units[0] : 0u));
    }
    const uint32_t room = s_room & ~1u;                             // bytes, whole units
    // The payload is only 2-byte aligned.  A halfword in front brings the destination
    // to a 4-byte boundary; the body goes out as 32-bit words, each warp store one
    // aligned 128-byte line; a halfword may remain at the end.  When the head halfword
    // exists the staged words straddle two shared-memory words: funnel shift.
    const uint32_t hb = (static_cast<uint32_t>(base) & 2u) ? min(2u, room) : 0u;
    const uint32_t nw = (room - hb) / 4u;
    const uint32_t tb = room - hb - 4u * nw;                        // 0 or 2 bytes behind the body
    const uint16_t* s16 = reinterpret_cast<const uint16_t*>(smem_raw);
    if (threadIdx.x == 0 && hb) *reinterpret_cast<uint16_t*>(dst + base) = s16[0];
    if (threadIdx.x == 32 && tb) *reinterpret_cast<uint16_t*>(dst + base + hb + 4ull * nw) = s16[(hb + 4u * nw) / 2u];
    const uint64_t body = base + hb;                                // 4-byte aligned
    const uint32_t mis = static_cast<uint32_t>(body >> 2) & 31u;    // first word's place in its 128-byte line
    const uint32_t* sp = reinterpret_cast<const uint32_t*>(smem_raw) + threadIdx.x - mis;
    uint32_t* gp = reinterpret_cast<uint32_t*>(dst + body) + threadIdx.x - mis;
    int32_t left = static_cast<int32_t>(nw) + static_cast<int32_t>(mis) - static_cast<int32_t>(threadIdx.x);
    if (hb == 0) {
        if (threadIdx.x >= mis && left > 0) *gp = *sp;
        left -= kTileThreads; sp += kTileThreads; gp += kTileThreads;
        while (left > 0) {
            *gp = *sp;
            left -= kTileThreads; sp += kTileThreads; gp += kTileThreads;
        }
    } else {
        if (threadIdx.x >= mis && left > 0) *gp = __funnelshift_r(sp[0], sp[1], 16);
        left -= kTileThreads; sp += kTileThreads; gp += kTileThreads;
        while (left > 0) {
            *gp = __funnelshift_r(sp[0], sp[1], 16);
            left -= kTileThreads; sp += kTileThreads; gp += kTileThreads;
        }
    }
}

template <bool RELU>
__global__ void __launch_bounds__(kTileThreads, kMinCtasPerSm)
zvc_compress_kernel_u16(const uint16_t* __restrict__ src, uint64_t n, uint8_t* __restrict__ dst,
                        uint64_t cap, uint64_t* __restrict__ table, uint64_t* __restrict__ ws,
                        const LaunchCtl ctl, uint32_t num_tiles, uint64_t num_chunks, uint16_t* __restrict__ relu_out,
                        uint32_t nan_above, uint64_t prefetch_bytes) {
    const uint32_t tile = blockIdx.x;     // block-index order, as in the 4-byte kernel
    if (tile >= num_tiles) return;
    prefetch_future_tile(src, prefetch_bytes, tile);
    if (threadIdx.x == 0) prefetch_future_descriptor(ws, tile, num_tiles);
    if ((static_cast<uint64_t>(tile) + 1) * (kTileChunksU16 * kChunk) <= n)
        compress_tile_u16<RELU, true>(src, n, dst, cap, table, ws, ctl, num_tiles, num_chunks, relu_out, nan_above, tile);
    else
        compress_tile_u16<RELU, false>(src, n, dst, cap, table, ws, ctl, num_tiles, num_chunks, relu_out, nan_above, tile);
}

template <typename T, uint32_t TILE_CHUNKS, typename Kernel>
cudaError_t launch_typed(Kernel kernel, const void* d_src, uint64_t n, void* d_dst, uint64_t cap,
                         uint64_t* d_table, uint64_t* d_ws, const LaunchCtl& ctl, void* d_relu_out,
                         uint32_t nan_above, cudaStream_t stream, bool src_on_device) {
    constexpr uint32_t kSmem = TILE_CHUNKS * (4 * kChunkWindows + sizeof(T) * kChunk);
    const cudaError_t oe = opt_in_shared_memory(reinterpret_cast<const void*>(kernel), kSmem);
    if (oe != cudaSuccess) return oe;
    const uint64_t chunks = num_chunks_of(n);
    const uint64_t tiles = (chunks + TILE_CHUNKS - 1) / TILE_CHUNKS;   // never more than num_tiles_of(n)
    timing_before_launch(stream);
    kernel<<<static_cast<unsigned>(tiles), kTileThreads, kSmem, stream>>>(
        static_cast<const T*>(d_src), n, static_cast<uint8_t*>(d_dst), cap, d_table, d_ws, ctl,
        static_cast<uint32_t>(tiles), chunks, static_cast<T*>(d_relu_out), nan_above,
        src_on_device ? n * sizeof(T) : 0ull);
    timing_after_launch(stream);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_zvc_compress(const void* d_src, uint64_t n, uint32_t elem_size, void* d_dst,
                                uint64_t cap, uint64_t* d_table, uint64_t* d_ws, const LaunchCtl& ctl,
                                cudaStream_t stream, bool src_on_device) {
    if (num_tiles_of(n) == 0) return cudaSuccess;
    // 2-byte and 1-byte elements in device memory, at least one tile: the row-per-thread kernel with TMA loads;
    // 1-byte elements have no other kernel and take it without the tensor copy otherwise
    const bool tma = src_on_device && zvc_compress_rows_tma_usable(d_src, n, elem_size);
    if (tma || elem_size == 1)
        return launch_zvc_compress_rows(d_src, n, elem_size, d_dst, cap, d_table, d_ws, ctl, stream, tma);
    const cudaError_t e =
        (elem_size == 4)
            ? launch_typed<uint32_t, kTileChunks>(zvc_compress_kernel<uint32_t, false>, d_src, n, d_dst, cap,
                                                  d_table, d_ws, ctl, nullptr, 0, stream, src_on_device)
            : launch_typed<uint16_t, kTileChunksU16>(zvc_compress_kernel_u16<false>, d_src, n, d_dst, cap,
                                                     d_table, d_ws, ctl, nullptr, 0, stream, src_on_device);
    count_kernel_launch();
    return e;
}

// With lazy module loading the first launch of a kernel in a process can wait for the device
// to go idle; a context that promises not to make the host wait loads its kernels up front.
void preload_compress_kernels() {
    cudaFuncAttributes a;
    (void)cudaFuncGetAttributes(&a, zvc_compress_kernel<uint32_t, false>);
    (void)cudaFuncGetAttributes(&a, zvc_compress_kernel_u16<false>);
    preload_compress_rows_kernel();
    (void)cudaGetLastError();
}

cudaError_t launch_zvc_relu_compress(const void* d_src, uint64_t n, uint32_t elem_size, uint32_t nan_above,
                                     void* d_relu_out, void* d_dst, uint64_t cap, uint64_t* d_table,
                                     uint64_t* d_ws, const LaunchCtl& ctl, cudaStream_t stream,
                                     bool src_on_device) {
    if (num_tiles_of(n) == 0) return cudaSuccess;
    const cudaError_t e =
        (elem_size == 4)
            ? launch_typed<uint32_t, kTileChunks>(zvc_compress_kernel<uint32_t, true>, d_src, n, d_dst, cap,
                                                  d_table, d_ws, ctl, d_relu_out, nan_above, stream, src_on_device)
            : launch_typed<uint16_t, kTileChunksU16>(zvc_compress_kernel_u16<true>, d_src, n, d_dst, cap,
                                                     d_table, d_ws, ctl, d_relu_out, nan_above, stream, src_on_device);
    count_kernel_launch();
    return e;
}

}  // namespace cdma
