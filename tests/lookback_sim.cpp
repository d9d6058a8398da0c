// Host-thread simulation of the inter-tile descriptor protocol of the compression
// kernels.  Every simulated tile is a thread that does what a compression CTA does
// with its descriptor -- publish its size, work for a while, walk back over its
// predecessors 32 at a time until it meets an inclusive prefix, publish its own
// prefix (or the error mark when a wait ran out) -- using the very functions the
// kernels use for packing descriptors and for deciding what a round means
// (csrc/lookback_protocol.h).  The 32 lanes of the walking warp are a loop here and
// the 16-byte descriptor access is a locked copy.  Test infrastructure only.
#include <atomic>
#include <chrono>
#include <cstdint>
#include <mutex>
#include <thread>
#include <vector>

#include "lookback_protocol.h"

namespace {

struct Slot {
    std::mutex mu;
    uint64_t head = 0, value = 0;
};

struct Sim {
    std::vector<Slot> slots;
    uint64_t tag;
    uint32_t stall_tile;
    uint32_t poll_limit;
};

void store(Sim& s, uint32_t tile, uint64_t head, uint64_t value) {
    if (tile == s.stall_tile) return;   // the silent tile
    std::lock_guard<std::mutex> g(s.slots[tile].mu);
    s.slots[tile].head = head;
    s.slots[tile].value = value;
}

void tile_thread(Sim& s, uint32_t tile, uint64_t size, uint32_t delay_us, uint64_t* exclusive, uint32_t* failed,
                 uint32_t* polls_out) {
    using namespace cdma;
    std::this_thread::sleep_for(std::chrono::microseconds(delay_us));
    store(s, tile, desc_head(tile == 0 ? kDescPrefix : kDescAggregate, s.tag), size);
    std::this_thread::sleep_for(std::chrono::microseconds(delay_us / 2));   // "assembling"
    uint64_t sum = 0;
    bool fail = false;
    uint32_t polls = 0;
    if (tile != 0) {
        int64_t look = static_cast<int64_t>(tile) - 1;
        while (true) {
            uint64_t head[32], value[32];
            uint32_t m_prefix = 0, m_invalid = 0, m_error = 0;
            for (int lane = 0; lane < 32; ++lane) {
                const int64_t idx = look - lane;
                head[lane] = desc_head(kDescPrefix, s.tag);     // before tile 0: an inclusive prefix of zero
                value[lane] = 0;
                if (idx >= 0) {
                    std::lock_guard<std::mutex> g(s.slots[idx].mu);
                    head[lane] = s.slots[idx].head;
                    value[lane] = s.slots[idx].value;
                }
                const uint32_t st = desc_state(head[lane], s.tag);
                m_prefix |= (st == 2 ? 1u : 0u) << lane;
                m_invalid |= (st == 0 ? 1u : 0u) << lane;
                m_error |= (st == 3 ? 1u : 0u) << lane;
            }
            const RoundPlan plan = plan_round(m_prefix, m_invalid, m_error);
            if (plan.action == kRoundFail) { fail = true; break; }
            if (plan.action == kRoundWait) {
                if (++polls > s.poll_limit) { fail = true; break; }   // the bounded wait ran out
                std::this_thread::sleep_for(std::chrono::microseconds(20));
                continue;
            }
            for (int lane = 0; lane < 32; ++lane)
                if ((plan.add_lanes >> lane) & 1u) sum += value[lane];
            if (plan.action == kRoundDone) { sum += value[plan.prefix_lane]; break; }
            look -= 32;
        }
        store(s, tile, desc_head(fail ? kDescError : kDescPrefix, s.tag), sum + size);
    }
    *exclusive = sum;
    *failed = fail ? 1u : 0u;
    *polls_out = polls;
}

}  // namespace

// Runs `tiles` simulated tiles.  garbage_head / garbage_value fill every descriptor
// before the start (what an earlier launch or the caller may have left).  Returns 0.
extern "C" int lookback_sim_run(uint32_t tiles, const uint64_t* sizes, const uint32_t* delays_us, uint64_t tag,
                                uint32_t stall_tile, uint32_t poll_limit, uint64_t garbage_head,
                                uint64_t garbage_value, uint64_t* exclusive, uint32_t* failed, uint32_t* polls) {
    Sim s{std::vector<Slot>(tiles), tag, stall_tile, poll_limit};
    for (auto& sl : s.slots) { sl.head = garbage_head; sl.value = garbage_value; }
    std::vector<std::thread> th;
    th.reserve(tiles);
    for (uint32_t t = 0; t < tiles; ++t)
        th.emplace_back(tile_thread, std::ref(s), t, sizes[t], delays_us[t], exclusive + t, failed + t, polls + t);
    for (auto& t : th) t.join();
    return 0;
}

// The packing on its own: head and state for a (state, tag) pair, as the kernels compute them.
extern "C" uint64_t lookback_sim_head(uint32_t state, uint64_t tag) {
    return cdma::desc_head(static_cast<uint64_t>(state) << 62, tag);
}
extern "C" uint32_t lookback_sim_state(uint64_t head, uint64_t tag) { return cdma::desc_state(head, tag); }
extern "C" void lookback_sim_plan(uint32_t m_prefix, uint32_t m_invalid, uint32_t m_error, uint32_t* out3) {
    const cdma::RoundPlan p = cdma::plan_round(m_prefix, m_invalid, m_error);
    out3[0] = p.action; out3[1] = p.add_lanes; out3[2] = p.prefix_lane;
}
