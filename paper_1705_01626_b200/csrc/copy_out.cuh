// The last step of a compression tile: the records staged in shared memory go to
// their place in the payload.  The payload offset of a tile is only a multiple of
// the element size, so the staged bytes are realigned in registers and leave as
// aligned 16-byte stores (a few elements in front and behind go one by one).
#pragma once

#include "zvc_common.cuh"

namespace cdma {

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

// Aligned 16-byte vector j of the payload region this tile writes, taken from the
// staged bytes: the staged tile starts `ph` bytes into vector 0, so vector j is the
// 16 bytes at staged offset 16 j - ph, i.e. at byte START = 16 - ph of the two
// aligned shared-memory vectors around it (START = 16: the second one as it is).
template <uint32_t START>
__device__ __forceinline__ uint4 realign(const uint4& lo, const uint4& hi) {
    constexpr uint32_t A = START / 4, BITS = 8 * (START % 4);
    const uint32_t w[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
    if (BITS == 0) return make_uint4(w[A & 7], w[(A + 1) & 7], w[(A + 2) & 7], w[(A + 3) & 7]);
    // A <= 3 whenever there is a sub-word shift, so A + 4 <= 7
    return make_uint4(__funnelshift_r(w[A & 7], w[(A + 1) & 7], BITS), __funnelshift_r(w[(A + 1) & 7], w[(A + 2) & 7], BITS),
                      __funnelshift_r(w[(A + 2) & 7], w[(A + 3) & 7], BITS),
                      __funnelshift_r(w[(A + 3) & 7], w[(A + 4) & 7], BITS));
}

template <uint32_t START, uint32_t THREADS>
__device__ __forceinline__ void copy_body(uint32_t s_stage, uint4* __restrict__ g, uint32_t j0, uint32_t j1) {
    // vector j needs the aligned shared-memory vectors j - 1 and j (only j when the phase is zero)
    for (uint32_t j = j0 + threadIdx.x; j < j1; j += THREADS) {
        const uint4 hi = lds128(s_stage + 16u * j);
        uint4 out = hi;
        if (START != 16) {
            const uint4 lo = lds128(s_stage + 16u * j - 16u);
            out = realign<START>(lo, hi);
        }
        g[j] = out;
    }
}

template <uint32_t S, uint32_t THREADS, uint32_t PH>
__device__ __forceinline__ void copy_phase(uint32_t ph, uint32_t s_buf, uint4* g, uint32_t j0, uint32_t j1) {
    // a uniform chain over the 16 / S possible phases, each with its own straight-line body
    if constexpr (PH < 16) {
        if (ph == PH) copy_body<(PH == 0 ? 16 : 16 - PH), THREADS>(s_buf, g, j0, j1);
        else copy_phase<S, THREADS, PH + S>(ph, s_buf, g, j0, j1);
    }
}

// Staged bytes of one tile (shared address s_buf, generic pointer buf) to their place in the payload,
// below the capacity.  S = element size (1, 2 or 4): the granularity of the payload offset.
template <uint32_t S, uint32_t THREADS>
__device__ __forceinline__ void copy_out(uint32_t s_buf, const uint8_t* buf, uint8_t* __restrict__ dst, uint64_t base,
                                         uint32_t room_bytes) {
    const uint32_t tid = threadIdx.x;
    const uint32_t room = room_bytes & ~(S - 1u);                 // whole elements
    const uint32_t ph = static_cast<uint32_t>(base) & 15u;        // where the tile starts inside its first vector
    uint8_t* gdst = dst + base;
    // head: the bytes in front of the first aligned vector; tail: those behind the last one
    const uint32_t head = ph ? min(16u - ph, room) : 0u;
    const uint32_t nvec = (room - head) / 16u;
    const uint32_t tail = room - head - 16u * nvec;
    if (tid < head / S) {
        if (S == 4) reinterpret_cast<uint32_t*>(gdst)[tid] = reinterpret_cast<const uint32_t*>(buf)[tid];
        else if (S == 2) reinterpret_cast<uint16_t*>(gdst)[tid] = reinterpret_cast<const uint16_t*>(buf)[tid];
        else gdst[tid] = buf[tid];
    } else if (tid >= 32 && tid - 32 < tail / S) {
        const uint32_t o = (head + 16u * nvec) / S + (tid - 32);
        if (S == 4) reinterpret_cast<uint32_t*>(gdst)[o] = reinterpret_cast<const uint32_t*>(buf)[o];
        else if (S == 2) reinterpret_cast<uint16_t*>(gdst)[o] = reinterpret_cast<const uint16_t*>(buf)[o];
        else gdst[o] = buf[o];
    }
    // body: aligned vector j of the payload (counted from the vector the tile starts in) holds the
    // staged bytes 16 j - ph .. 16 j - ph + 15
    uint4* g = reinterpret_cast<uint4*>(gdst - ph);
    const uint32_t j0 = ph ? 1u : 0u, j1 = j0 + nvec;
    copy_phase<S, THREADS, 0>(ph, s_buf, g, j0, j1);
}

}  // namespace cdma
