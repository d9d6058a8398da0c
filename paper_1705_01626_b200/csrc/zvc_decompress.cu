// Zero-value decompression of 4-byte elements (Section V-B, Fig. 10b): the
// pop-count of a mask tells how many payload values its window takes; values or
// zeros are steered into the window's 32 places.  (2-byte and 1-byte elements
// have a kernel of their own, in zvc_decompress_groups.cu.)
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
constexpr uint32_t kPrefetchAheadCtas = 888;   // 6 CTAs x 148 SMs resident at a time

// Shared-memory loads by 32-bit address + immediate: positions in the staged
// array are kept as byte addresses so that no index has to be scaled.
template <uint32_t IMM>
__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1+%2];" : "=r"(v) : "r"(addr), "n"(IMM));
    return v;
}

// Per-lane constants of the 4-byte expansion.
struct U32Lane {
    uint32_t sh;         // 4 * (lane & 7): where my 4 mask bits start
    uint32_t below;      // mask bits of the elements in front of mine
    uint32_t off;        // 4 * (lane >> 3) + 4: my window's place in the round, past its mask word
    bool w_hi, w_odd;    // bits of lane >> 3
};

// One round = windows 4G .. 4G+3 of a full chunk of 4-byte elements.  `a` is the
// shared byte address of the next mask word minus 4 bytes per window already
// passed (folded into the immediates).  The walk is pulled back to the chunk's
// end after every second window, so that nothing is read beyond the staged bytes
// plus two records; a walk that was pulled back once overshoots again at every
// later step, so the caller only has to look at the last one.
// GATE: instead of the values of the stream, the elements of `gate` (the incoming gradient of the
// backward pass) go to the places the masks mark; the values are not even read.
template <uint32_t G, bool GATE>
__device__ __forceinline__ void expand_round_u32(uint32_t& a, uint32_t a_end, uint32_t& last, const U32Lane& c,
                                                 uint4* __restrict__ out, const uint4& g) {
    // four serial steps of the self-delimiting walk; every lane sees all four
    const uint32_t a0 = a;
    const uint32_t m0 = lds32<16 * G + 0>(a0);
    const uint32_t a1 = a0 + 4u * __popc(m0);
    const uint32_t m1 = lds32<16 * G + 4>(a1);
    const uint32_t a2 = min(a1 + 4u * __popc(m1), a_end - (16u * G + 8u));
    const uint32_t m2 = lds32<16 * G + 8>(a2);
    const uint32_t a3 = a2 + 4u * __popc(m2);
    const uint32_t m3 = lds32<16 * G + 12>(a3);
    last = a3 + 4u * __popc(m3);
    a = min(last, a_end - (16u * G + 16u));
    const uint32_t my_a = c.w_hi ? (c.w_odd ? a3 : a2) : (c.w_odd ? a1 : a0);
    const uint32_t my_m = c.w_hi ? (c.w_odd ? m3 : m2) : (c.w_odd ? m1 : m0);
    const uint32_t nib = my_m >> c.sh;
    const bool b0 = nib & 1u, b1 = nib & 2u, b2 = nib & 4u, b3 = nib & 8u;
    if (GATE) {
        (void)my_a;
        __stcs(out + 32 * G, make_uint4(b0 ? g.x : 0u, b1 ? g.y : 0u, b2 ? g.z : 0u, b3 ? g.w : 0u));
        return;
    }
    // the next four values in front of my elements
    const uint32_t q = my_a + 4u * __popc(my_m & c.below) + c.off;
    const uint32_t v0 = lds32<16 * G + 0>(q), v1 = lds32<16 * G + 4>(q), v2 = lds32<16 * G + 8>(q),
                   v3 = lds32<16 * G + 12>(q);
    // element k takes the value numbered by the set bits below bit k
    const uint32_t t1 = b0 ? v1 : v0, u = b0 ? v2 : v1, w = b0 ? v3 : v2;
    const uint32_t t2 = b1 ? u : t1, x = b1 ? w : u;
    const uint32_t t3 = b2 ? x : t2;
    __stcs(out + 32 * G, make_uint4(b0 ? v0 : 0u, b1 ? t1 : 0u, b2 ? t2 : 0u, b3 ? t3 : 0u));
}

template <uint32_t G, bool GATE>
__device__ __forceinline__ void expand_rounds_u32(uint32_t& a, uint32_t a_end, uint32_t& last, const U32Lane& c,
                                                  uint4* __restrict__ out, const uint4* __restrict__ gate) {
    // four rounds at a time; in the gate form their four loads of the gradient are issued together, in front
    if constexpr (G < kChunkWindows / 4) {
        uint4 g[4];
#pragma unroll
        for (uint32_t i = 0; i < 4; ++i) g[i] = GATE ? __ldcs(gate + 32 * (G + i)) : make_uint4(0, 0, 0, 0);
        expand_round_u32<G + 0, GATE>(a, a_end, last, c, out, g[0]);
        expand_round_u32<G + 1, GATE>(a, a_end, last, c, out, g[1]);
        expand_round_u32<G + 2, GATE>(a, a_end, last, c, out, g[2]);
        expand_round_u32<G + 3, GATE>(a, a_end, last, c, out, g[3]);
        expand_rounds_u32<G + 4, GATE>(a, a_end, last, c, out, gate);
    }
}

// GATE = false: decompression.  GATE = true: the backward pass of the activation function from the
// compressed map (Section II-B: the backward pass reuses the map; for y = max(x, 0) only its non-zero
// pattern matters): dst = gate where the map's element is non-zero, else 0 -- the same table checks,
// staging and walk, but the masks alone are used.
template <typename T, bool PREFETCH, bool GATE>
__global__ void __launch_bounds__(kDecThreads, 6)
zvc_decompress_kernel(const uint8_t* __restrict__ src, uint64_t src_bytes,
                      const uint64_t* __restrict__ table, uint64_t n, T* __restrict__ dst,
                      uint64_t* __restrict__ ws, const LaunchCtl ctl, uint64_t num_chunks,
                      const T* __restrict__ gate) {
    constexpr uint32_t S = sizeof(T);
    constexpr uint32_t MU = 4 / S;                               // units of T per mask
    constexpr uint32_t kMaxChunkBytes = 4 * kChunkWindows + S * kChunk;
    static_assert(S == 4, "2-byte elements have a kernel of their own");
    // 16-byte phase in front; behind, room for the reads of a walk that has left
    // a malformed record: the position is pulled back to `end` after every second
    // window (the buffer then still lets six CTAs fit per SM), so the walk can run
    // 2 records past `end`, and a lane reads a mask and up to 35 values from there.
    constexpr uint32_t kOverrun = 2u * (MU + 32u);
    constexpr uint32_t kBuf = (kMaxChunkBytes + 16 + S * (kOverrun + MU + 36) + 15) / 16 * 16;
    static_assert(kBuf % 16 == 0, "rows of s_buf must keep 16-byte alignment for the vector stores");
    __shared__ __align__(16) uint8_t s_buf[kDecWarps][kBuf];

    const uint32_t lane = lane_id();
    const uint32_t warp = threadIdx.x >> 5;
    const uint64_t chunk = static_cast<uint64_t>(blockIdx.x) * kDecWarps + warp;
    if (blockIdx.x == 0 && threadIdx.x == 0) init_decode_result(ws, ctl, n * S);
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
        if (lane == 0) report_decode_error(ws, ctl, CDMA_ERR_CORRUPT_STREAM);
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
    if (PREFETCH) {
        const uint64_t cf = chunk + static_cast<uint64_t>(kPrefetchAheadCtas) * kDecWarps;
        if (cf < num_chunks) {
            const uint64_t flo = __ldg(table + cf);
            const uint64_t fhi = __ldg(table + cf + 1);
            // at most 34 lines of 128 bytes: one per lane, a second one for the first lanes
            const uint64_t line0 = flo & ~127ull;
            const uint64_t span = fhi - line0;                 // garbage if the entries are bad: checked next
            if (flo <= fhi && fhi <= src_bytes && span <= kMaxChunkBytes + 127) {
                const uint32_t off = 128u * lane;
                if (off < static_cast<uint32_t>(span)) asm volatile("prefetch.global.L2 [%0];" ::"l"(src + line0 + off));
                if (off + 4096u < static_cast<uint32_t>(span))
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(src + line0 + off + 4096u));
            }
        }
    }
    __syncwarp();

    // ---- walk the records and expand ----------------------------------------
    const T* units = reinterpret_cast<const T*>(buf);
    uint32_t p = static_cast<uint32_t>(lo - a0) / S;        // position in units of S bytes
    const uint32_t end = static_cast<uint32_t>(hi - a0) / S;
    bool bad = false;

    if (nelem == kChunk) {
        // full chunk: 8 rounds of 4 windows; lane = 4 consecutive elements
        U32Lane c;
        c.sh = 4u * (lane & 7u);
        c.below = (1u << c.sh) - 1u;
        c.off = 4u * (lane >> 3) + 4u;
        c.w_hi = (lane & 16u) != 0u;
        c.w_odd = (lane & 8u) != 0u;
        const uint32_t t_addr = static_cast<uint32_t>(__cvta_generic_to_shared(buf));
        uint32_t a = t_addr + 4u * p, last = 0;
        expand_rounds_u32<0, GATE>(a, t_addr + 4u * end, last, c, reinterpret_cast<uint4*>(dst + e0) + lane,
                                   GATE ? reinterpret_cast<const uint4*>(gate + e0) + lane : nullptr);
        // `last` is the final position before it was pulled back, with 4 bytes per window folded out
        p = (last - t_addr) / 4u + kChunkWindows;
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
            if (lane < left) {
                const T val = bit ? (GATE ? gate[e0 + lane + w * kWindow] : units[p + MU + __popc(m & lt)]) : T(0);
                out[w * kWindow] = val;
            }
            p += MU + cnt;
        }
    }
    if (!bad && p != end) bad = true;
    if (bad && lane == 0) report_decode_error(ws, ctl, CDMA_ERR_CORRUPT_STREAM);
}

}  // namespace

cudaError_t launch_zvc_decompress(const void* d_src, uint64_t src_bytes, const uint64_t* d_table,
                                  uint64_t n, uint32_t elem_size, void* d_dst, uint64_t* d_ws,
                                  const LaunchCtl& ctl, cudaStream_t stream, bool src_on_device) {
    const uint64_t chunks = num_chunks_of(n);
    if (chunks == 0) return cudaSuccess;
    const dim3 grid(static_cast<unsigned>((chunks + kDecWarps - 1) / kDecWarps));
    timing_before_launch(stream);
    if (elem_size == 4) {
        // payload at least a fifth of the dense bytes: reading it is a real share of the traffic
        const bool prefetch = src_on_device && src_bytes >= (n * 4) / 5;
        auto kernel = prefetch ? zvc_decompress_kernel<uint32_t, true, false> : zvc_decompress_kernel<uint32_t, false, false>;
        kernel<<<grid, kDecThreads, 0, stream>>>(static_cast<const uint8_t*>(d_src), src_bytes, d_table, n,
                                                 static_cast<uint32_t*>(d_dst), d_ws, ctl, chunks, nullptr);
    } else {
        const cudaError_t e = launch_zvc_decompress_groups(d_src, src_bytes, d_table, n, elem_size, d_dst, d_ws, ctl,
                                                           stream, src_on_device);
        if (e != cudaSuccess) return e;
    }
    timing_after_launch(stream);
    count_kernel_launch();
    return cudaGetLastError();
}

// Backward gate for 4-byte elements: the decompression kernel with the masks steering the gradient.
cudaError_t launch_zvc_gate_u32(const void* d_src, uint64_t src_bytes, const uint64_t* d_table, uint64_t n,
                                const void* d_gate, void* d_dst, uint64_t* d_ws, const LaunchCtl& ctl,
                                cudaStream_t stream) {
    const uint64_t chunks = num_chunks_of(n);
    if (chunks == 0) return cudaSuccess;
    const dim3 grid(static_cast<unsigned>((chunks + kDecWarps - 1) / kDecWarps));
    timing_before_launch(stream);
    // (the payload is asked for ahead of time under the same condition as in decompression)
    const bool prefetch = !in_host_memory(d_src) && src_bytes >= (n * 4) / 5;
    auto kernel = prefetch ? zvc_decompress_kernel<uint32_t, true, true> : zvc_decompress_kernel<uint32_t, false, true>;
    kernel<<<grid, kDecThreads, 0, stream>>>(
        static_cast<const uint8_t*>(d_src), src_bytes, d_table, n, static_cast<uint32_t*>(d_dst), d_ws, ctl, chunks,
        static_cast<const uint32_t*>(d_gate));
    timing_after_launch(stream);
    count_kernel_launch();
    return cudaGetLastError();
}

// The backward pass of the activation function straight from the compressed map: every element width takes
// its decompression kernel in the gate form.
cudaError_t launch_zvc_relu_backward(const void* d_src, uint64_t src_bytes, const uint64_t* d_table, uint64_t n,
                                     uint32_t elem_size, const void* d_dy, void* d_dx, uint64_t* d_ws,
                                     const LaunchCtl& ctl, cudaStream_t stream) {
    if (elem_size == 4) return launch_zvc_gate_u32(d_src, src_bytes, d_table, n, d_dy, d_dx, d_ws, ctl, stream);
    return launch_zvc_gate_groups(d_src, src_bytes, d_table, n, elem_size, d_dy, d_dx, d_ws, ctl, stream);
}

}  // namespace cdma
