// Zero-value decompression of 2-byte and 1-byte elements (Section V-B, Fig. 10b:
// the pop-count of a mask tells how many payload values its window takes; values
// or zeros are steered into the window's 32 places).
//
// With fewer bytes per element, these widths are bound by the instructions and the
// shared-memory accesses spent per chunk, not by DRAM.  Three choices keep both low:
//
//   - A warp expands several consecutive chunks at once: four chunks of 2-byte
//     elements (eight lanes per chunk) or eight chunks of 1-byte elements (four
//     lanes per chunk).  The walk from mask to mask (the stream is self-delimiting,
//     Section V-A) is serial within a chunk and every lane of a warp repeats it, so
//     its instructions cost the same whatever the lanes hold: one walk step now
//     advances all the warp's chunks.  A lane's window is simply the one its group
//     of lanes has just reached.
//   - Those chunks are one contiguous piece of the payload.  One bulk copy
//     (cp.async.bulk, completion on an mbarrier) brings it into shared memory: no
//     load or store instruction of the warp is spent on staging.  Masks and values
//     sit at element boundaries there: 2-byte elements are read as 2-byte halves,
//     1-byte elements as two aligned words and a funnel shift.
//   - A lane fetches only as many values as it has non-zero elements (predicated
//     loads): fewer lanes per access, fewer bank conflicts between the four chunks.
//
// A lane expands 8 bytes of the tensor per round (4 two-byte or 8 one-byte
// elements): the pop-count of the mask bits below them is where its values start,
// and byte permutes with selectors from a 16-entry table (indexed by 4 mask bits)
// put values and zeros in place; one 8-byte store per lane, a window's 64 or 32
// bytes contiguous.  The table and
// every record are validated; nothing is read outside the payload or written
// outside the tensor whatever the input holds.
//
// The gate form of the kernel is the backward pass of the activation function
// straight from the compressed map (Section II-B: the backward pass reuses the
// map; for y = max(x, 0) all it needs is which elements are non-zero, and that
// is what the masks say): dst = gate where the map's element is non-zero, else 0.
// The dense y never has to be rebuilt in memory (the direction Section IX leaves
// as future work: keeping activations compressed).
#include "zvc_common.cuh"

namespace cdma {

namespace {

constexpr uint32_t kTryWaitHintNs = 100000;

// Sizes by element width S.
template <uint32_t S>
struct Geometry {
    // a lane expands 8 bytes of the tensor per round: 4 two-byte or 8 one-byte elements; a window takes 8 or 4
    // lanes, so a warp walks 4 or 8 chunks at once
    static constexpr uint32_t kLaneElems = 8 / S;
    static constexpr uint32_t kLanesPerChunk = kWindow / kLaneElems;
    static constexpr uint32_t kQ = 32 / kLanesPerChunk;                  // chunks per warp
    static constexpr uint32_t kMaxChunkBytes = 4 * kChunkWindows + S * kChunk;
    // The walk is pulled back to the chunk's end after every second window, so it can run two records past
    // it, and a lane reads a mask and up to 4 values (two words) from there.
    static constexpr uint32_t kOverrunBytes = 2 * (4 + S * kWindow);
    static constexpr uint32_t kBufBytes = (16 + kQ * kMaxChunkBytes + kOverrunBytes + 4 + S * 36 + 16 + 15) / 16 * 16;
    // CTAs of one warp: what shared memory allows, at most 32
    static constexpr uint32_t kCtasBySmem = (227u * 1024u) / (kBufBytes + 1024u + 128u);
    static constexpr uint32_t kCtasPerSm = kCtasBySmem > 32 ? 32 : kCtasBySmem;
    static constexpr uint32_t kPrefetchGroups = 148 * kCtasPerSm;       // the groups resident at a time
};

// Selectors of the byte permutes, by a lane's 4 mask bits.  Element k takes value number popc(bits below k).
// 2-byte elements: with v01 / v23 the next four values, elements 0,1 = prmt(v01, 0, low half) (selector
// nibble 4 picks a zero byte), elements 2,3 = prmt(v01, v23, high half), cleared where their bits are clear.
__constant__ uint32_t kExpandSel2[16] = {
    0x10104444u, 0x32324410u, 0x32321044u, 0x54543210u, 0x32104444u, 0x54324410u, 0x54321044u, 0x76543210u,
    0x10104444u, 0x32324410u, 0x32321044u, 0x54543210u, 0x32104444u, 0x54324410u, 0x54321044u, 0x76543210u,
};
// 1-byte elements: the four elements = prmt(next four values, 0, selector).
__constant__ uint32_t kExpandSel1[16] = {
    0x4444, 0x4440, 0x4404, 0x4410, 0x4044, 0x4140, 0x4104, 0x4210,
    0x0444, 0x1440, 0x1404, 0x2410, 0x1044, 0x2140, 0x2104, 0x3210,
};

template <uint32_t IMM>
__device__ __forceinline__ uint32_t lds16(uint32_t addr) {
    uint32_t v;
    asm("ld.shared.u16 %0, [%1+%2];" : "=r"(v) : "r"(addr), "n"(IMM));
    return v;
}
template <uint32_t IMM>
__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
    uint32_t v;
    asm("ld.shared.u32 %0, [%1+%2];" : "=r"(v) : "r"(addr), "n"(IMM));
    return v;
}
// the same for the lanes where a > K; the others keep a zero
template <uint32_t IMM, uint32_t K>
__device__ __forceinline__ uint32_t lds16_if_more(uint32_t addr, uint32_t a) {
    uint32_t v = 0;
    asm("{\n\t.reg .pred p;\n\tsetp.gt.u32 p, %2, %3;\n\t@p ld.shared.u16 %0, [%1+%4];\n\t}"
        : "+r"(v) : "r"(addr), "r"(a), "n"(K), "n"(IMM));
    return v;
}
template <uint32_t IMM, uint32_t K>
__device__ __forceinline__ uint32_t lds32_if_more(uint32_t addr, uint32_t a) {
    uint32_t v = 0;
    asm("{\n\t.reg .pred p;\n\tsetp.gt.u32 p, %2, %3;\n\t@p ld.shared.u32 %0, [%1+%4];\n\t}"
        : "+r"(v) : "r"(addr), "r"(a), "n"(K), "n"(IMM));
    return v;
}
__device__ __forceinline__ uint32_t lds32_at(uint32_t addr) {
    uint32_t v;
    asm("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t v;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(v) : "r"(a), "r"(b), "r"(sel));   // the low 16 bits of sel are used
    return v;
}

// Bounded wait for the bulk copy.  Returns false when the limit ran out.
__device__ __forceinline__ bool wait_copy(uint32_t mbar, uint64_t limit_ns) {
    uint32_t done = 0, polls = 0;
    uint64_t t0 = 0;
    while (true) {
        // (the last operand lets the hardware hold the thread for up to that many nanoseconds before it
        // answers "not yet")
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0, %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(mbar), "r"(kTryWaitHintNs) : "memory");
        if (done) return true;
        const uint64_t now = global_timer_ns();
        if (t0 == 0) t0 = now;
        else if (now - t0 > limit_ns || ++polls > kWaitLimitPolls) return false;
    }
}

struct LaneConst {
    uint32_t sh;         // where my 4 (8) mask bits start
    uint32_t below;      // mask bits of the elements in front of mine
    uint32_t tbl;        // shared address of the selector table
};

// One round = window G of each of the warp's chunks.  `a` is the shared byte address of the chunk's next mask
// minus 4 bytes per window already passed (folded into the immediates).  A walk that was pulled back once
// overshoots again at every later step, so the caller only has to look at `last`.
// A lane's share of one round: 8 bytes (4 two-byte or 8 one-byte elements).
template <uint32_t S> struct LaneWord { using type = uint2; };

// One round = window G of each of the warp's chunks.  `a` is the shared byte address of the chunk's next mask
// minus 4 bytes per window already passed (folded into the immediates).  A walk that was pulled back once
// overshoots again at every later step, so the caller only has to look at `last`.
// GATE: instead of the values of the stream, the elements of `gate` (the incoming gradient of the backward
// pass) go to the places the masks mark; the values are not even read.
template <uint32_t S, uint32_t G, bool GATE>
__device__ __forceinline__ void expand_round(uint32_t& a, uint32_t a_end, uint32_t& last, const LaneConst& c,
                                             typename LaneWord<S>::type* __restrict__ out,
                                             const typename LaneWord<S>::type& g) {
    uint32_t m;
    if (S == 2) {
        m = prmt(lds16<4 * G>(a), lds16<4 * G + 2>(a), 0x5410u);
    } else {
        // a mask at any byte address: the two aligned words around it
        const uint32_t al = a & ~3u;
        m = __funnelshift_r(lds32<4 * G>(al), lds32<4 * G + 4>(al), 8u * (a & 3u));
    }
    last = a + S * __popc(m);
    const uint32_t nib = (m >> c.sh) & 15u;
    // 0xff.. where a mask bit is set: the four bits go to the sign positions of the four bytes of x, which a
    // permute replicates
    const uint32_t x = nib * 0x10204080u;
    if constexpr (S == 2) {
        if (GATE) {
            __stcs(out + 8 * G, make_uint2(g.x & prmt(x, x, 0x9988u), g.y & prmt(x, x, 0xbbaau)));
        } else {
            // my (up to) four values: 2-byte halves behind the mask, only as many as I have non-zero elements
            const uint32_t q = a + 2u * __popc(m & c.below);
            const uint32_t cnt = __popc(nib);
            const uint32_t v01 = prmt(lds16_if_more<4 * G + 4, 0>(q, cnt), lds16_if_more<4 * G + 6, 1>(q, cnt), 0x5410u);
            const uint32_t v23 = prmt(lds16_if_more<4 * G + 8, 2>(q, cnt), lds16_if_more<4 * G + 10, 3>(q, cnt), 0x5410u);
            const uint32_t sel = lds32_at(c.tbl + 4u * nib);
            __stcs(out + 8 * G, make_uint2(prmt(v01, 0u, sel), prmt(v01, v23, sel >> 16) & prmt(x, x, 0xbbaau)));
        }
    } else {
        // eight elements: two groups of four, the second group's values right behind the first's
        const uint32_t nib_hi = (m >> (c.sh + 4u)) & 15u;
        const uint32_t x_hi = nib_hi * 0x10204080u;
        if (GATE) {
            __stcs(out + 4 * G, make_uint2(g.x & prmt(x, x, 0xba98u), g.y & prmt(x_hi, x_hi, 0xba98u)));
        } else {
            // my (up to) eight values: the bytes behind the mask, from the aligned word they start in and, as far
            // as they reach, the next two
            const uint32_t q = a + __popc(m & c.below);
            const uint32_t qa = q & ~3u, ph = q & 3u;
            const uint32_t c0 = __popc(nib);
            const uint32_t reach = ph + c0 + __popc(nib_hi);
            const uint32_t w0 = lds32_if_more<4 * G + 4, 0>(qa, reach - ph);
            const uint32_t w1 = lds32_if_more<4 * G + 8, 4>(qa, reach);
            const uint32_t w2 = lds32_if_more<4 * G + 12, 8>(qa, reach);
            const uint32_t v_lo = __funnelshift_r(w0, w1, 8u * ph), v_hi = __funnelshift_r(w1, w2, 8u * ph);
            const uint32_t sel_lo = lds32_at(c.tbl + 4u * nib), sel_hi = lds32_at(c.tbl + 4u * nib_hi);
            __stcs(out + 4 * G, make_uint2(prmt(v_lo, 0u, sel_lo), prmt(__funnelshift_rc(v_lo, v_hi, 8u * c0), 0u, sel_hi)));
        }
    }
    a = (G & 1u) ? min(last, a_end - 4u * (G + 1u)) : last;
}

// Eight rounds at a time; in the gate form their eight loads of the gradient are issued together, in front.
template <uint32_t S, uint32_t G, bool GATE>
__device__ __forceinline__ void expand_rounds(uint32_t& a, uint32_t a_end, uint32_t& last, const LaneConst& c,
                                              typename LaneWord<S>::type* __restrict__ out,
                                              const typename LaneWord<S>::type* __restrict__ gate) {
    if constexpr (G < kChunkWindows) {
        typename LaneWord<S>::type g[8];
#pragma unroll
        for (uint32_t i = 0; i < 8; ++i)
            g[i] = GATE ? __ldcs(gate + Geometry<S>::kLanesPerChunk * (G + i)) : typename LaneWord<S>::type{};
        expand_round<S, G + 0, GATE>(a, a_end, last, c, out, g[0]);
        expand_round<S, G + 1, GATE>(a, a_end, last, c, out, g[1]);
        expand_round<S, G + 2, GATE>(a, a_end, last, c, out, g[2]);
        expand_round<S, G + 3, GATE>(a, a_end, last, c, out, g[3]);
        expand_round<S, G + 4, GATE>(a, a_end, last, c, out, g[4]);
        expand_round<S, G + 5, GATE>(a, a_end, last, c, out, g[5]);
        expand_round<S, G + 6, GATE>(a, a_end, last, c, out, g[6]);
        expand_round<S, G + 7, GATE>(a, a_end, last, c, out, g[7]);
        expand_rounds<S, G + 8, GATE>(a, a_end, last, c, out, gate);
    }
}

// S: element size (2 or 1).  BULK: the group's bytes come in by one bulk copy (the payload lies in device
// memory); otherwise by the warp's own loads.  PREFETCH: ask L2 for the bytes of the group a later CTA will
// expand.  GATE: the backward gate -- the same table checks, staging and walk, but the masks alone are used.
template <uint32_t S, bool BULK, bool PREFETCH, bool GATE>
__global__ void __launch_bounds__(32, Geometry<S>::kCtasPerSm)
zvc_decompress_groups_kernel(const uint8_t* __restrict__ src, uint64_t src_bytes, const uint64_t* __restrict__ table,
                             uint64_t n, uint8_t* __restrict__ dst, uint64_t* __restrict__ ws, const LaunchCtl ctl,
                             uint64_t num_chunks, const uint8_t* __restrict__ gate) {
    using Word = typename LaneWord<S>::type;
    constexpr uint32_t kQ = Geometry<S>::kQ;
    constexpr uint32_t kLanesPerChunk = Geometry<S>::kLanesPerChunk;
    constexpr uint32_t kMaxChunkBytes = Geometry<S>::kMaxChunkBytes;
    constexpr uint32_t kBufBytes = Geometry<S>::kBufBytes;
    constexpr uint32_t kPrefetchGroups = Geometry<S>::kPrefetchGroups;
    __shared__ __align__(128) uint8_t s_buf[kBufBytes];
    __shared__ uint32_t s_sel[16];
    __shared__ __align__(8) uint64_t s_mbar;
    const uint32_t lane = lane_id();
    const uint32_t mbar = static_cast<uint32_t>(__cvta_generic_to_shared(&s_mbar));
    if (lane < 16) s_sel[lane] = (S == 2) ? kExpandSel2[lane] : kExpandSel1[lane];
    if (BULK && lane == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(mbar) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();

    const uint64_t c0 = static_cast<uint64_t>(blockIdx.x) * kQ;          // first chunk of the group (exists: grid size)
    if (blockIdx.x == 0 && lane == 0) init_decode_result(ws, ctl, n * S);
    const uint32_t nchunks = (num_chunks - c0 < kQ) ? static_cast<uint32_t>(num_chunks - c0) : kQ;
    // lanes of a chunk the tensor does not have shadow the group's last chunk (their checks then agree with it)
    const uint32_t mine = min(lane / kLanesPerChunk, nchunks - 1u);
    const uint64_t chunk = c0 + mine;
    const uint64_t e0 = chunk * kChunk;
    const uint32_t nelem = (n - e0 < kChunk) ? static_cast<uint32_t>(n - e0) : kChunk;
    const uint32_t nwin = (nelem + kWindow - 1) / kWindow;

    // ---- the chunks' byte ranges, validated -----------------------------------------------------
    const uint64_t lo = __ldg(table + chunk);
    const uint64_t hi = __ldg(table + chunk + 1);
    const uint64_t len64 = hi - lo;
    const uint32_t len = static_cast<uint32_t>(len64);                      // trusted only once len64 is known small
    bool ok = (lo <= hi) && (hi <= src_bytes) && (len64 <= kMaxChunkBytes) && (len >= 4u * nwin) &&
              (len <= 4u * nwin + S * nelem) && (((static_cast<uint32_t>(lo) | len) & (S - 1u)) == 0u);
    if (chunk == 0 && lo != 0) ok = false;
    if (chunk == num_chunks - 1 && hi != src_bytes) ok = false;
    if (!__all_sync(0xffffffffu, ok)) {
        if (lane == 0) report_decode_error(ws, ctl, CDMA_ERR_CORRUPT_STREAM);
        return;
    }
    // the group's bytes: from the first chunk's start to the last chunk's end (consecutive table entries,
    // every piece at most one chunk long: at most four chunks' worth)
    const uint64_t glo = __shfl_sync(0xffffffffu, lo, 0);
    const uint64_t ghi = __shfl_sync(0xffffffffu, hi, 31);

    // ---- stage payload bytes [glo, ghi); s_buf[0] is payload byte a0 -------------------------------------
    const uint64_t a0 = glo & ~15ull;
    const uint32_t span = static_cast<uint32_t>(ghi - a0);                 // bytes from a0 to the group's end
    const uint32_t span16 = (span + 15u) & ~15u;
    // the bulk copy moves whole 16-byte pieces: the tensor's last group may not have them inside the payload
    const bool bulk = BULK && a0 + span16 <= src_bytes;
    if (bulk) {
        if (lane == 0 && span16 != 0) {
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(mbar), "r"(span16) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(s_buf))), "l"(src + a0), "r"(span16), "r"(mbar)
                         : "memory");
        }
    } else {
        const uint32_t avail = (src_bytes - a0 > 32768ull) ? 32768u : static_cast<uint32_t>(src_bytes - a0);
        const uint8_t* from = src + a0;
        for (uint32_t off = 16u * lane; off < span; off += 16u * 32u) {
            uint4 q;
            if (off + 16u <= avail) {
                q = __ldcs(reinterpret_cast<const uint4*>(from + off));
            } else {
                // the payload's last bytes: never read past src_bytes
                uint32_t wds[4] = {0, 0, 0, 0};
                for (uint32_t b = 0; b < 16; ++b)
                    if (off + b < avail) wds[b >> 2] |= static_cast<uint32_t>(from[off + b]) << (8 * (b & 3));
                q = make_uint4(wds[0], wds[1], wds[2], wds[3]);
            }
            *reinterpret_cast<uint4*>(s_buf + off) = q;
        }
    }
    if (PREFETCH) {
        // ask L2 for the payload of the group a CTA kPrefetchGroups blocks later will expand
        // (blocks are dispatched in index order; every line still comes from DRAM once)
        const uint64_t cf = c0 + static_cast<uint64_t>(kPrefetchGroups) * kQ;
        if (cf < num_chunks) {
            const uint64_t cl = (num_chunks - cf < kQ) ? num_chunks : cf + kQ;
            const uint64_t flo = __ldg(table + cf);
            const uint64_t fhi = __ldg(table + cl);
            const uint64_t line0 = flo & ~127ull;
            const uint64_t fspan = fhi - line0;                // garbage if the entries are bad: checked next
            if (flo <= fhi && fhi <= src_bytes && fspan <= kQ * kMaxChunkBytes + 127) {
                for (uint32_t o = 128u * lane; o < static_cast<uint32_t>(fspan); o += 4096u)
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(src + line0 + o));
            }
        }
    }
    if (bulk && span16 != 0) {
        if (!wait_copy(mbar, ctl.wait_limit_ns)) {
            // late beyond the limit: one more bounded wait, so that the copy cannot write into shared memory
            // this CTA has already handed back; then the launch fails
            (void)wait_copy(mbar, ctl.wait_limit_ns);
            if (lane == 0) report_decode_error(ws, ctl, CDMA_ERR_TIMEOUT);
            return;
        }
    }
    __syncwarp();

    // ---- walk the records and expand ----------------------------------------------------------------
    // (the shared loads below are plain functions of their address to the compiler: the address is made to
    // depend on this point of the program, behind the wait for the staged bytes)
    uint32_t buf_addr = static_cast<uint32_t>(__cvta_generic_to_shared(s_buf));
    uint32_t sel_addr = static_cast<uint32_t>(__cvta_generic_to_shared(s_sel));
    asm volatile("" : "+r"(buf_addr), "+r"(sel_addr) : : "memory");
    if (nchunks == kQ && n - c0 * kChunk >= kQ * kChunk) {
        // four full chunks: every group of eight lanes walks its own chunk
        LaneConst c;
        c.sh = Geometry<S>::kLaneElems * (lane % kLanesPerChunk);
        c.below = (1u << c.sh) - 1u;
        c.tbl = sel_addr;
        const uint32_t a_end = buf_addr + static_cast<uint32_t>(hi - a0);
        uint32_t a = buf_addr + static_cast<uint32_t>(lo - a0), last = 0;
        expand_rounds<S, 0, GATE>(a, a_end, last, c, reinterpret_cast<Word*>(dst + e0 * S) + (lane % kLanesPerChunk),
                                  GATE ? reinterpret_cast<const Word*>(gate + e0 * S) + (lane % kLanesPerChunk) : nullptr);
        // `last` has 4 bytes per window folded out
        const bool bad = last + 4u * kChunkWindows != a_end;
        if (__any_sync(0xffffffffu, bad) && lane == 0) report_decode_error(ws, ctl, CDMA_ERR_CORRUPT_STREAM);
        return;
    }
    // the tensor's last group: chunk after chunk, lane = element, one window per round
    bool bad = false;
    const uint32_t lt = lanemask_lt();
    for (uint32_t k = 0; k < nchunks && !bad; ++k) {
        const uint64_t klo = __shfl_sync(0xffffffffu, lo, k * kLanesPerChunk);
        const uint64_t khi = __shfl_sync(0xffffffffu, hi, k * kLanesPerChunk);
        const uint64_t ke0 = (c0 + k) * kChunk;
        const uint32_t knelem = (n - ke0 < kChunk) ? static_cast<uint32_t>(n - ke0) : kChunk;
        const uint32_t knwin = (knelem + kWindow - 1) / kWindow;
        uint32_t p = static_cast<uint32_t>(klo - a0);                       // byte position in the staged bytes
        const uint32_t end = static_cast<uint32_t>(khi - a0);
        for (uint32_t w = 0; w < knwin; ++w) {
            if (p + 4u > end) { bad = true; break; }
            const uint32_t m = static_cast<uint32_t>(s_buf[p]) | (static_cast<uint32_t>(s_buf[p + 1]) << 8) |
                               (static_cast<uint32_t>(s_buf[p + 2]) << 16) | (static_cast<uint32_t>(s_buf[p + 3]) << 24);
            const uint32_t cnt = __popc(m);
            const uint32_t left = knelem - w * kWindow;           // elements this window really has
            if (p + 4u + S * cnt > end || (left < kWindow && (m >> left) != 0)) { bad = true; break; }
            if (lane < left) {
                const uint64_t j = ke0 + w * kWindow + lane;
                const bool bit = (m >> lane) & 1u;
                const uint8_t* from_b = GATE ? gate + j * S : s_buf + p + 4u + S * __popc(m & lt);
                for (uint32_t b = 0; b < S; ++b) dst[j * S + b] = bit ? from_b[b] : uint8_t(0);
            }
            p += 4u + S * cnt;
        }
        if (!bad && p != end) bad = true;
    }
    if (bad && lane == 0) report_decode_error(ws, ctl, CDMA_ERR_CORRUPT_STREAM);
}

}  // namespace

namespace {

template <uint32_t S>
cudaError_t launch_groups(const void* d_src, uint64_t src_bytes, const uint64_t* d_table, uint64_t n, void* d_dst,
                          uint64_t* d_ws, const LaunchCtl& ctl, cudaStream_t stream, bool src_on_device,
                          const void* d_gate) {
    const uint64_t chunks = num_chunks_of(n);
    constexpr uint32_t kQ = Geometry<S>::kQ;
    const dim3 grid(static_cast<unsigned>((chunks + kQ - 1) / kQ));
    // payload at least a fifth of the dense bytes: reading it is a real share of the traffic
    const bool prefetch = src_on_device && src_bytes >= (n * S) / 5;
    const bool bulk = src_on_device && (reinterpret_cast<uintptr_t>(d_src) & 15) == 0;
    auto kernel = d_gate != nullptr ? (bulk ? (prefetch ? zvc_decompress_groups_kernel<S, true, true, true>
                                                        : zvc_decompress_groups_kernel<S, true, false, true>)
                                            : zvc_decompress_groups_kernel<S, false, false, true>)
                  : bulk ? (prefetch ? zvc_decompress_groups_kernel<S, true, true, false>
                                     : zvc_decompress_groups_kernel<S, true, false, false>)
                         : zvc_decompress_groups_kernel<S, false, false, false>;
    kernel<<<grid, 32, 0, stream>>>(static_cast<const uint8_t*>(d_src), src_bytes, d_table, n,
                                    static_cast<uint8_t*>(d_dst), d_ws, ctl, chunks, static_cast<const uint8_t*>(d_gate));
    return cudaGetLastError();
}

}  // namespace

// Decompression of 2-byte (elem_size 2) and 1-byte (elem_size 1) elements.  The caller brackets the launch
// with the timing hooks and counts it.
cudaError_t launch_zvc_decompress_groups(const void* d_src, uint64_t src_bytes, const uint64_t* d_table, uint64_t n,
                                         uint32_t elem_size, void* d_dst, uint64_t* d_ws, const LaunchCtl& ctl,
                                         cudaStream_t stream, bool src_on_device) {
    return elem_size == 2 ? launch_groups<2>(d_src, src_bytes, d_table, n, d_dst, d_ws, ctl, stream, src_on_device, nullptr)
                          : launch_groups<1>(d_src, src_bytes, d_table, n, d_dst, d_ws, ctl, stream, src_on_device, nullptr);
}

// Backward gate for 2-byte and 1-byte elements: the same kernel with the masks steering the gradient.
cudaError_t launch_zvc_gate_groups(const void* d_src, uint64_t src_bytes, const uint64_t* d_table, uint64_t n,
                                   uint32_t elem_size, const void* d_gate, void* d_dst, uint64_t* d_ws,
                                   const LaunchCtl& ctl, cudaStream_t stream) {
    if (num_chunks_of(n) == 0) return cudaSuccess;
    const bool on_device = !in_host_memory(d_src);
    timing_before_launch(stream);
    const cudaError_t e =
        elem_size == 2 ? launch_groups<2>(d_src, src_bytes, d_table, n, d_dst, d_ws, ctl, stream, on_device, d_gate)
                       : launch_groups<1>(d_src, src_bytes, d_table, n, d_dst, d_ws, ctl, stream, on_device, d_gate);
    timing_after_launch(stream);
    count_kernel_launch();
    return e;
}

}  // namespace cdma
