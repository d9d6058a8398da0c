// Inter-tile part of the single-pass compression kernels: the decoupled look-back
// over the 64-bit {state:2 | value:62} descriptors of earlier tiles.  Shared by
// the zero-value and the run-length kernels.
#pragma once

#include "zvc_common.cuh"

namespace cdma {

struct LookbackResult {
    uint64_t exclusive;   // bytes of all earlier tiles
    bool failed;
};

// Warp-wide walk executed by warp 0 of the CTA: lane l inspects tile look - l;
// aggregates are added until a tile that already knows its inclusive prefix is
// met.  Waiting for a predecessor that has not published yet is bounded: when
// the limit is hit the tile marks itself failed so that every later tile stops
// waiting too.
__device__ inline LookbackResult lookback_walk(const uint64_t* desc, uint64_t* ws, uint32_t tile) {
    const uint32_t lane = lane_id();
    LookbackResult r{0, false};
    int64_t look = static_cast<int64_t>(tile) - 1;   // nearest tile not yet added
    uint32_t polls = 0;
    uint64_t t_start = 0;
    while (true) {
        const int64_t idx = look - static_cast<int64_t>(lane);
        // before tile 0 there is nothing: an inclusive prefix of zero
        const uint64_t d = (idx >= 0) ? ld_relaxed_u64(desc + idx * kDescStride) : kDescPrefix;
        const uint32_t state = static_cast<uint32_t>(d >> 62);
        const uint32_t m_prefix = __ballot_sync(0xffffffffu, state == 2);
        const uint32_t m_invalid = __ballot_sync(0xffffffffu, state == 0);
        const uint32_t m_error = __ballot_sync(0xffffffffu, state == 3);
        // lanes up to and including the nearest tile that knows its prefix
        const uint32_t f = m_prefix & (0u - m_prefix);
        const uint32_t upto = m_prefix ? (f | (f - 1u)) : 0xffffffffu;
        if (m_error & upto) {
            r.failed = true;
            break;
        }
        if (m_invalid & upto) {
            ++polls;
            if ((polls & 63u) == 0) {
                const uint64_t now = global_timer_ns();
                if (t_start == 0) t_start = now;
                else if (now - t_start > kWaitLimitNs || polls > kWaitLimitPolls) {
                    if (lane == 0) report_status(ws, CDMA_ERR_TIMEOUT);
                    r.failed = true;
                    break;
                }
            }
            if (polls > 2) __nanosleep(100);
            continue;
        }
        // A tile is at most 50,688 bytes, so the sizes of up to 32 tiles add up in
        // 32 bits: one warp reduction; the 64-bit prefix comes from the lane that
        // holds it.
        const uint32_t sizes = upto & ~f;                       // lanes holding a size to add
        const uint32_t part = ((sizes >> lane) & 1u) ? static_cast<uint32_t>(d) : 0u;
        r.exclusive += __reduce_add_sync(0xffffffffu, part);
        if (m_prefix) {
            r.exclusive += __shfl_sync(0xffffffffu, d, __ffs(m_prefix) - 1) & kDescValueMask;
            break;
        }
        look -= 32;
    }
    return r;
}

}  // namespace cdma
