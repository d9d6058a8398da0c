// The descriptor protocol of the single-pass compression kernels, as plain
// functions that compile for the device and for the host alike: how a
// descriptor is packed, when it counts, and what a tile does with one round of
// 32 predecessors' descriptors.  The kernels (lookback.cuh) call these; a
// host-thread simulation in the test suite drives the very same functions.
#pragma once

#include <stdint.h>

#if defined(__CUDACC__)
#define CDMA_HD __host__ __device__ __forceinline__
#else
#define CDMA_HD inline
#endif

namespace cdma {

// Inter-tile prefix descriptor, 16 bytes written and read as one unit:
//   head = state:2 | tag:62     value = bytes
// A descriptor counts only if its tag is the current launch's; anything else is
// "not published yet" (state 0), whatever an earlier launch or the caller left.
constexpr uint64_t kTagMask = (1ull << 62) - 1;
constexpr uint64_t kDescAggregate = 1ull << 62;   // value = this tile's bytes
constexpr uint64_t kDescPrefix = 2ull << 62;      // value = bytes of tiles 0..this
constexpr uint64_t kDescError = 3ull << 62;       // a predecessor gave up; give up too

CDMA_HD uint64_t desc_head(uint64_t state_bits, uint64_t tag) { return state_bits | (tag & kTagMask); }
CDMA_HD uint32_t desc_state(uint64_t head, uint64_t tag) {
    return ((head & kTagMask) == (tag & kTagMask)) ? static_cast<uint32_t>(head >> 62) : 0u;
}

// One round of the walk looks at 32 predecessors, lane 0 the nearest.  From the
// lanes whose descriptor holds an inclusive prefix (m_prefix), nothing yet
// (m_invalid) or the error mark (m_error):
enum : uint32_t {
    kRoundWait = 0,      // a descriptor that is needed has not been published: poll again
    kRoundFail = 1,      // a tile in front gave up
    kRoundContinue = 2,  // add the sizes of add_lanes, go 32 tiles further back
    kRoundDone = 3       // add the sizes of add_lanes and the prefix held by prefix_lane: finished
};
struct RoundPlan {
    uint32_t action;
    uint32_t add_lanes;    // lanes whose value is a tile size to add
    uint32_t prefix_lane;  // lane whose value is the inclusive prefix that ends the walk
};
CDMA_HD RoundPlan plan_round(uint32_t m_prefix, uint32_t m_invalid, uint32_t m_error) {
    // lanes up to and including the nearest tile that knows its prefix
    const uint32_t first = m_prefix & (0u - m_prefix);
    const uint32_t upto = m_prefix ? (first | (first - 1u)) : 0xffffffffu;
    RoundPlan p{kRoundContinue, upto & ~first, 0};
    if (m_error & upto) p.action = kRoundFail;
    else if (m_invalid & upto) p.action = kRoundWait;
    else if (m_prefix) {
        p.action = kRoundDone;
#if defined(__CUDA_ARCH__)
        p.prefix_lane = static_cast<uint32_t>(__ffs(static_cast<int>(first)) - 1);
#else
        p.prefix_lane = static_cast<uint32_t>(__builtin_ctz(first));
#endif
    }
    return p;
}

}  // namespace cdma
