// Inter-tile part of the single-pass compression kernels: the decoupled look-back
// over the {state | tag, value} descriptors of earlier tiles.  Shared by the
// zero-value and the run-length kernels.
#pragma once

#include "zvc_common.cuh"

namespace cdma {

struct LookbackResult {
    uint64_t exclusive;   // bytes of all earlier tiles
    bool failed;
};

// A tile makes its size public (before it has assembled anything).  The tile
// named by ctl.stall_tile stays silent: a test uses it to make the waits of the
// tiles behind it run out.
__device__ __forceinline__ void publish_aggregate(uint64_t* ws, const LaunchCtl& ctl, uint32_t tile, uint64_t tile_bytes) {
    if (tile == ctl.stall_tile) return;
    st_desc(desc_slot(ws, tile), desc_head(tile == 0 ? kDescPrefix : kDescAggregate, ctl.tag), tile_bytes);
}
__device__ __forceinline__ void publish_prefix(uint64_t* ws, const LaunchCtl& ctl, uint32_t tile, bool failed,
                                               uint64_t inclusive) {
    if (tile == ctl.stall_tile) return;
    st_desc(desc_slot(ws, tile), desc_head(failed ? kDescError : kDescPrefix, ctl.tag), inclusive);
}

// The workspace is not cleared between launches (the tag tells old descriptors from new ones), so the
// first read of a descriptor that has not been published yet would go all the way to DRAM.  A CTA
// therefore asks L2 for the descriptor of the tile `kDescAhead` places further on -- a generation of
// resident CTAs -- long before anybody publishes or inspects it (370 to 1110 places measure the same).
constexpr uint32_t kDescAhead = 740;
__device__ __forceinline__ void prefetch_future_descriptor(uint64_t* ws, uint32_t tile, uint32_t num_tiles) {
    if (tile + kDescAhead < num_tiles)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(desc_slot(ws, tile + kDescAhead)));
    // (the first tiles have nobody in front of them to do it)
    if (tile < kDescAhead) asm volatile("prefetch.global.L2 [%0];" ::"l"(desc_slot(ws, tile)));
}

// Warp-wide walk executed by one warp of the CTA: lane l inspects tile look - l;
// aggregates are added until a tile that already knows its inclusive prefix is
// met.  Waiting for a predecessor that has not published yet is bounded by
// ctl.wait_limit_ns: when the limit is hit the result says failed (the caller
// then marks its own descriptor so that every later tile stops waiting too).
// The decision to give up is taken by lane 0 and broadcast, so that the warp
// leaves the loop together.
__device__ inline LookbackResult lookback_walk(uint64_t* ws, const LaunchCtl& ctl, uint32_t tile) {
    const uint32_t lane = lane_id();
    LookbackResult r{0, false};
    int64_t look = static_cast<int64_t>(tile) - 1;   // nearest tile not yet added
    uint32_t polls = 0;
    uint64_t t_start = 0;
    while (true) {
        const int64_t idx = look - static_cast<int64_t>(lane);
        // before tile 0 there is nothing: an inclusive prefix of zero
        Desc d{desc_head(kDescPrefix, ctl.tag), 0};
        if (idx >= 0) d = ld_desc(desc_slot(ws, static_cast<uint32_t>(idx)));
        const uint32_t state = desc_state(d.head, ctl.tag);
        const RoundPlan plan = plan_round(__ballot_sync(0xffffffffu, state == 2), __ballot_sync(0xffffffffu, state == 0),
                                          __ballot_sync(0xffffffffu, state == 3));
        if (plan.action == kRoundFail) {
            r.failed = true;
            break;
        }
        if (plan.action == kRoundWait) {
            ++polls;
            if ((polls & 15u) == 0) {
                uint32_t expired = 0;
                if (lane == 0) {
                    const uint64_t now = global_timer_ns();
                    if (t_start == 0) t_start = now;
                    else if (now - t_start > ctl.wait_limit_ns || polls > kWaitLimitPolls) expired = 1;
                }
                if (__shfl_sync(0xffffffffu, expired, 0)) {
                    r.failed = true;
                    break;
                }
            }
            if (polls > 2) __nanosleep(100);
            continue;
        }
        // A tile is less than 2^16 bytes, so the sizes of up to 32 tiles add up in
        // 32 bits: one warp reduction; the 64-bit prefix comes from the lane that
        // holds it.
        const uint32_t part = ((plan.add_lanes >> lane) & 1u) ? static_cast<uint32_t>(d.value) : 0u;
        r.exclusive += __reduce_add_sync(0xffffffffu, part);
        if (plan.action == kRoundDone) {
            r.exclusive += __shfl_sync(0xffffffffu, d.value, plan.prefix_lane);
            break;
        }
        look -= 32;
    }
    return r;
}

// What warp 0 of a compression CTA does once the tile's records are assembled:
// find the tile's place in the stream, publish the inclusive prefix, and -- the
// last tile only -- close the stream: last table entry, result words.  Returns
// through the three shared words: base offset, "failed" and the bytes of the
// tile that fit below the capacity.
__device__ __forceinline__ void resolve_tile(uint64_t* ws, const LaunchCtl& ctl, uint32_t tile, uint32_t num_tiles,
                                             uint64_t tile_bytes, uint64_t cap, uint64_t* table, uint64_t num_chunks,
                                             uint64_t* s_base, uint32_t* s_failed, uint32_t* s_room_bytes) {
    LookbackResult lb{0, false};
    if (tile != 0) {
        lb = lookback_walk(ws, ctl, tile);
        if (lane_id() == 0) publish_prefix(ws, ctl, tile, lb.failed, lb.exclusive + tile_bytes);
    }
    if (lane_id() == 0) {
        *s_base = lb.exclusive;
        *s_failed = lb.failed ? 1u : 0u;
        const uint64_t end_bytes = lb.exclusive + tile_bytes;
        *s_room_bytes = static_cast<uint32_t>(cap >= end_bytes ? tile_bytes : (cap > lb.exclusive ? cap - lb.exclusive : 0));
        if (tile == num_tiles - 1) {
            if (lb.failed) {
                publish_result(ws, ctl, 0, CDMA_ERR_TIMEOUT);
            } else {
                table[num_chunks] = end_bytes;
                publish_result(ws, ctl, end_bytes, end_bytes > cap ? CDMA_ERR_BUFFER_TOO_SMALL : 0);
            }
        }
    }
}

}  // namespace cdma
