// Offload / prefetch pipeline (Section III, Fig. 2b; Section V-D): OFF(n)
// compresses an activation map and copies the compressed bytes to pinned host
// memory, PRE(n) copies them back and expands them.  The codec kernels run on
// the caller's compute stream, the copies on a side stream owned by the
// context; two device staging slots let one tensor's copy overlap the next
// tensor's kernel.  Host code, plus the small copy kernel of the asynchronous
// offload; contracts are in include/cdma.h.
#include <map>
#include <new>
#include <unordered_map>
#include <vector>

#include "zvc_common.cuh"

namespace {

constexpr uint64_t kAlign = 256;
constexpr uint32_t kSlots = 2;
constexpr uint32_t kResultRing = 1024;   // pinned {bytes,status} pairs for asynchronous calls

inline uint64_t round_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }

// First-fit allocator over the pinned pool with merging of free neighbours.
class RegionPool {
public:
    void reset(uint64_t bytes) {
        free_.clear();
        if (bytes) free_[0] = bytes;
    }
    bool alloc(uint64_t bytes, uint64_t* off) {
        bytes = round_up(bytes ? bytes : 1, kAlign);
        for (auto it = free_.begin(); it != free_.end(); ++it) {
            if (it->second >= bytes) {
                *off = it->first;
                const uint64_t rest = it->second - bytes;
                const uint64_t rest_off = it->first + bytes;
                free_.erase(it);
                if (rest) free_[rest_off] = rest;
                return true;
            }
        }
        return false;
    }
    // Give back the tail of a region that turned out larger than needed.
    void shrink(uint64_t off, uint64_t old_bytes, uint64_t new_bytes) {
        old_bytes = round_up(old_bytes ? old_bytes : 1, kAlign);
        new_bytes = round_up(new_bytes ? new_bytes : 1, kAlign);
        if (new_bytes < old_bytes) release(off + new_bytes, old_bytes - new_bytes);
    }
    void release(uint64_t off, uint64_t bytes) {
        bytes = round_up(bytes ? bytes : 1, kAlign);
        auto it = free_.emplace(off, bytes).first;
        auto next = std::next(it);
        if (next != free_.end() && it->first + it->second == next->first) {
            it->second += next->second;
            free_.erase(next);
        }
        if (it != free_.begin()) {
            auto prev = std::prev(it);
            if (prev->first + prev->second == it->first) {
                prev->second += it->second;
                free_.erase(it);
            }
        }
    }

private:
    std::map<uint64_t, uint64_t> free_;
};

struct Slot {
    uint8_t* base = nullptr;
    uint64_t bytes = 0;
    cudaEvent_t idle = nullptr;     // last use of the slot has finished
    cudaEvent_t staged = nullptr;   // kernel (offload) / copy (prefetch) into the slot has finished
    bool used = false;
};

struct SlotPlan {
    uint64_t* table;
    uint64_t table_bytes;
    uint64_t* ws;
    uint64_t ws_bytes;
    uint8_t* payload;
    uint64_t capacity;
};

struct TicketRec {
    uint64_t n;
    int dtype, layout;
    uint64_t payload_bytes;
    uint64_t pool_off, pool_bytes;      // region of the pinned pool owned by the ticket
    uint64_t payload_off, table_off;    // where payload and table sit inside the pool
    // asynchronous offloads: the size is not known when the ticket is handed out
    bool resolved = true;
    const uint64_t* res = nullptr;      // pinned {bytes, status} written by the compression kernel
    cudaEvent_t done = nullptr;         // the ticket's bytes have landed in the pool
};

// Copy of an offloaded tensor from a device staging slot into the mapped pinned
// pool, for the case where the host does not know the payload size yet: the
// kernel reads the size (and the status) the compression kernel left in the
// slot's workspace and moves exactly that many payload bytes plus the offset
// table.  A few CTAs saturate the host link; the rest of the GPU stays free for
// the caller's compute stream.
constexpr uint32_t kCopyCtas = 48;
constexpr uint32_t kCopyThreads = 256;
__global__ void __launch_bounds__(kCopyThreads)
offload_copy_kernel(const uint64_t* __restrict__ ws, const uint4* __restrict__ payload, uint4* __restrict__ pool_payload,
                    const uint4* __restrict__ table, uint4* __restrict__ pool_table, uint64_t table_vecs,
                    uint64_t capacity) {
    const uint64_t bytes = ws[cdma::kWsBytes];
    const uint64_t status = ws[cdma::kWsStatus];
    if (status != 0 || bytes > capacity) return;          // nothing valid to move; the host sees the status
    const uint64_t vecs = (bytes + 15) / 16;               // the slot and the pool region are padded to 16 bytes
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    for (uint64_t i = static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < vecs; i += stride)
        pool_payload[i] = __ldcs(payload + i);
    for (uint64_t i = static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < table_vecs; i += stride)
        pool_table[i] = __ldcs(table + i);
}

}  // namespace

struct cdma_ctx {
    int device = 0;
    cudaStream_t side = nullptr;
    uint8_t* h_pool = nullptr;
    uint64_t pool_bytes = 0;
    RegionPool pool;
    uint8_t* d_staging = nullptr;
    Slot slots[kSlots];
    uint32_t next_slot = 0;
    std::unordered_map<uint64_t, TicketRec> tickets;
    uint64_t next_ticket = 1;
    uint64_t* h_results = nullptr;
    uint32_t next_result = 0;
    std::vector<uint64_t*> pending;   // results of asynchronous calls not yet inspected
    int deferred = 0;
    void* d_dense = nullptr;          // dense staging of the host-buffer calls
    uint64_t dense_bytes = 0;
    std::vector<uint64_t> unresolved; // asynchronous offload tickets whose size has not been read yet, oldest first
    std::vector<cudaEvent_t> spare_events;
    cudaEvent_t pool_read = nullptr;  // last side-stream copy that reads the pinned pool
    bool pool_read_used = false;
};

namespace {

bool plan_slot(const Slot& slot, uint64_t n, int dtype, SlotPlan* p) {
    p->table_bytes = 8 * cdma_zvc_table_entries(n);
    p->ws_bytes = cdma_zvc_workspace_bytes(n, dtype);
    const uint64_t head = round_up(p->table_bytes, kAlign) + round_up(p->ws_bytes, kAlign);
    if (slot.bytes < head) return false;
    p->table = reinterpret_cast<uint64_t*>(slot.base);
    p->ws = reinterpret_cast<uint64_t*>(slot.base + round_up(p->table_bytes, kAlign));
    p->payload = slot.base + head;
    const uint64_t room = (slot.bytes - head) & ~15ull;
    const uint64_t worst = cdma_zvc_max_compressed_bytes(n, dtype);
    p->capacity = room < worst ? room : worst;
    return true;
}

// Device view of a page-locked host buffer (mapped into the device's address space
// under unified addressing), or nullptr if p is anything else or not aligned to `align`.
void* mapped_view(const void* p, uintptr_t align) {
    cudaPointerAttributes attr;
    if (p == nullptr || cudaPointerGetAttributes(&attr, p) != cudaSuccess) {
        (void)cudaGetLastError();
        return nullptr;
    }
    if (attr.type != cudaMemoryTypeHost || attr.devicePointer == nullptr) return nullptr;
    if (reinterpret_cast<uintptr_t>(attr.devicePointer) & (align - 1)) return nullptr;
    return attr.devicePointer;
}

uint64_t* next_result_words(cdma_ctx* ctx) {
    uint64_t* r = ctx->h_results + 2 * (ctx->next_result % kResultRing);
    ++ctx->next_result;
    r[0] = 0;
    r[1] = 0;
    return r;
}

// Inspect finished asynchronous calls; keeps the first failure.
void collect_pending(cdma_ctx* ctx) {
    for (uint64_t* r : ctx->pending)
        if (r[1] != 0 && ctx->deferred == 0) ctx->deferred = static_cast<int>(r[1]);
    ctx->pending.clear();
}

int wait_all(cdma_ctx* ctx) {
    if (cudaStreamSynchronize(ctx->side) != cudaSuccess) return CDMA_ERR_CUDA;
    for (Slot& s : ctx->slots)
        if (s.used && cudaEventSynchronize(s.idle) != cudaSuccess) return CDMA_ERR_CUDA;
    collect_pending(ctx);
    return CDMA_OK;
}

bool settle_ticket(cdma_ctx* ctx, uint64_t id, bool block);
void settle_all(cdma_ctx* ctx, bool block);

int ensure_dense(cdma_ctx* ctx, uint64_t bytes) {
    if (bytes <= ctx->dense_bytes) return CDMA_OK;
    if (wait_all(ctx) != CDMA_OK) return CDMA_ERR_CUDA;
    if (ctx->d_dense) cudaFree(ctx->d_dense);
    ctx->d_dense = nullptr;
    ctx->dense_bytes = 0;
    if (cudaMalloc(&ctx->d_dense, round_up(bytes, kAlign)) != cudaSuccess) {
        cudaGetLastError();
        return CDMA_ERR_OUT_OF_MEMORY;
    }
    ctx->dense_bytes = round_up(bytes, kAlign);
    return CDMA_OK;
}

cudaEvent_t take_event(cdma_ctx* ctx) {
    if (!ctx->spare_events.empty()) {
        cudaEvent_t e = ctx->spare_events.back();
        ctx->spare_events.pop_back();
        return e;
    }
    cudaEvent_t e = nullptr;
    if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) {
        cudaGetLastError();
        return nullptr;
    }
    return e;
}

// An asynchronous offload hands out its ticket before the payload size exists.  The
// first caller that needs the size settles the ticket: waits (or, with block = false,
// only looks) for the ticket's bytes to have landed, reads the size the kernel stored
// in pinned memory, and gives the unused tail of the worst-case reservation back to
// the pool.  A ticket whose compression failed is dropped and its status deferred.
// Returns false if the ticket is still in flight (block = false only).
bool settle_ticket(cdma_ctx* ctx, uint64_t id, bool block) {
    auto it = ctx->tickets.find(id);
    if (it == ctx->tickets.end() || it->second.resolved) return true;
    TicketRec& rec = it->second;
    if (block) {
        if (cudaEventSynchronize(rec.done) != cudaSuccess) cudaGetLastError();
    } else if (cudaEventQuery(rec.done) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    ctx->spare_events.push_back(rec.done);
    rec.done = nullptr;
    rec.resolved = true;
    for (size_t i = 0; i < ctx->unresolved.size(); ++i)
        if (ctx->unresolved[i] == id) { ctx->unresolved.erase(ctx->unresolved.begin() + i); break; }
    const uint64_t status = rec.res[1];
    if (status != 0) {
        if (ctx->deferred == 0) ctx->deferred = static_cast<int>(status);
        ctx->pool.release(rec.pool_off, rec.pool_bytes);
        ctx->tickets.erase(it);
        return true;
    }
    rec.payload_bytes = rec.res[0];
    const uint64_t used = (rec.payload_off - rec.pool_off) + rec.payload_bytes;
    ctx->pool.shrink(rec.pool_off, rec.pool_bytes, used);
    rec.pool_bytes = used;
    return true;
}

void settle_all(cdma_ctx* ctx, bool block) {
    const std::vector<uint64_t> ids = ctx->unresolved;
    for (uint64_t id : ids) settle_ticket(ctx, id, block);
}

// Pool allocation that first gives back what finished asynchronous offloads over-reserved, and
// waits for the ones still in flight (oldest first) before it reports the pool exhausted.
bool pool_alloc(cdma_ctx* ctx, uint64_t bytes, uint64_t* off) {
    if (ctx->pool.alloc(bytes, off)) return true;
    settle_all(ctx, false);
    if (ctx->pool.alloc(bytes, off)) return true;
    while (!ctx->unresolved.empty()) {
        settle_ticket(ctx, ctx->unresolved.front(), true);
        if (ctx->pool.alloc(bytes, off)) return true;
    }
    return false;
}

}  // namespace

extern "C" {

int cdma_ctx_create(uint64_t pinned_bytes, uint64_t device_staging_bytes, cdma_ctx** out) {
    if (out == nullptr) return CDMA_ERR_INVALID_ARG;
    *out = nullptr;
    cdma_ctx* ctx = new (std::nothrow) cdma_ctx();
    if (ctx == nullptr) return CDMA_ERR_OUT_OF_MEMORY;
    int st = CDMA_OK;
    const uint64_t slot_bytes = (device_staging_bytes / kSlots) & ~(kAlign - 1);
    do {
        if (cudaGetDevice(&ctx->device) != cudaSuccess) { st = CDMA_ERR_CUDA; break; }
        if (cudaStreamCreateWithFlags(&ctx->side, cudaStreamNonBlocking) != cudaSuccess) {
            st = CDMA_ERR_CUDA; break;
        }
        if (pinned_bytes &&
            cudaHostAlloc(reinterpret_cast<void**>(&ctx->h_pool), pinned_bytes, cudaHostAllocMapped | cudaHostAllocPortable) !=
                cudaSuccess) {
            st = CDMA_ERR_OUT_OF_MEMORY; break;
        }
        ctx->pool_bytes = pinned_bytes;
        ctx->pool.reset(pinned_bytes);
        if (cudaHostAlloc(reinterpret_cast<void**>(&ctx->h_results), 16 * kResultRing,
                          cudaHostAllocDefault) != cudaSuccess) {
            st = CDMA_ERR_OUT_OF_MEMORY; break;
        }
        if (slot_bytes &&
            cudaMalloc(reinterpret_cast<void**>(&ctx->d_staging), slot_bytes * kSlots) != cudaSuccess) {
            st = CDMA_ERR_OUT_OF_MEMORY; break;
        }
        if (cudaEventCreateWithFlags(&ctx->pool_read, cudaEventDisableTiming) != cudaSuccess) {
            st = CDMA_ERR_CUDA; break;
        }
        // cdma_offload_async must not make the host wait: no kernel is loaded lazily at its first launch
        cdma::preload_compress_kernels();
        {
            cudaFuncAttributes attr;
            (void)cudaFuncGetAttributes(&attr, offload_copy_kernel);
            (void)cudaGetLastError();
        }
        for (uint32_t i = 0; i < kSlots && st == CDMA_OK; ++i) {
            ctx->slots[i].base = ctx->d_staging ? ctx->d_staging + i * slot_bytes : nullptr;
            ctx->slots[i].bytes = slot_bytes;
            if (cudaEventCreateWithFlags(&ctx->slots[i].idle, cudaEventDisableTiming) != cudaSuccess ||
                cudaEventCreateWithFlags(&ctx->slots[i].staged, cudaEventDisableTiming) != cudaSuccess)
                st = CDMA_ERR_CUDA;
        }
    } while (false);
    if (st != CDMA_OK) {
        cudaGetLastError();
        cdma_ctx_destroy(ctx);
        return st;
    }
    *out = ctx;
    return CDMA_OK;
}

int cdma_ctx_destroy(cdma_ctx* ctx) {
    if (ctx == nullptr) return CDMA_ERR_INVALID_ARG;
    if (ctx->side) cudaStreamSynchronize(ctx->side);
    for (Slot& s : ctx->slots) {
        if (s.used && s.idle) cudaEventSynchronize(s.idle);
        if (s.idle) cudaEventDestroy(s.idle);
        if (s.staged) cudaEventDestroy(s.staged);
    }
    for (auto& kv : ctx->tickets)
        if (kv.second.done) cudaEventDestroy(kv.second.done);
    for (cudaEvent_t e : ctx->spare_events) cudaEventDestroy(e);
    if (ctx->pool_read) cudaEventDestroy(ctx->pool_read);
    if (ctx->d_dense) cudaFree(ctx->d_dense);
    if (ctx->d_staging) cudaFree(ctx->d_staging);
    if (ctx->h_results) cudaFreeHost(ctx->h_results);
    if (ctx->h_pool) cudaFreeHost(ctx->h_pool);
    if (ctx->side) cudaStreamDestroy(ctx->side);
    delete ctx;
    return CDMA_OK;
}

int64_t cdma_offload(cdma_ctx* ctx, const void* d_src, uint64_t n, int dtype, int layout,
                     void* compute_stream, cdma_ticket* out) {
    if (ctx == nullptr || out == nullptr) return -static_cast<int64_t>(CDMA_ERR_INVALID_ARG);
    if (cdma_dtype_size(dtype) == 0) return -static_cast<int64_t>(CDMA_ERR_UNSUPPORTED_DTYPE);
    cudaStream_t compute = static_cast<cudaStream_t>(compute_stream);
    Slot& slot = ctx->slots[ctx->next_slot++ % kSlots];
    SlotPlan p;
    if (!plan_slot(slot, n, dtype, &p)) return -static_cast<int64_t>(CDMA_ERR_BUFFER_TOO_SMALL);

    // the slot's previous copy must have drained before the kernel overwrites it
    if (slot.used && cudaStreamWaitEvent(compute, slot.idle, 0) != cudaSuccess)
        return -static_cast<int64_t>(CDMA_ERR_CUDA);
    uint64_t* res = next_result_words(ctx);
    const int st = cdma_zvc_compress_async(d_src, n, dtype, layout, p.payload, p.capacity, p.table, p.ws,
                                           p.ws_bytes, compute, res);
    if (st != CDMA_OK) return -static_cast<int64_t>(st);
    if (cudaEventRecord(slot.staged, compute) != cudaSuccess ||
        cudaEventSynchronize(slot.staged) != cudaSuccess)
        return -static_cast<int64_t>(CDMA_ERR_CUDA);
    slot.used = true;
    cudaEventRecord(slot.idle, compute);
    if (res[1] != 0) return -static_cast<int64_t>(res[1]);
    const uint64_t c = res[0];

    // exactly C payload bytes and the table cross the link (Section V-D: the
    // compressed size is known on completion and sizes the host allocation)
    TicketRec rec{n, dtype, layout, c, 0, round_up(c, 16) + p.table_bytes, 0, 0};
    if (!pool_alloc(ctx, rec.pool_bytes, &rec.pool_off) ||
        rec.pool_off + rec.pool_bytes > ctx->pool_bytes)
        return -static_cast<int64_t>(CDMA_ERR_OUT_OF_MEMORY);
    rec.payload_off = rec.pool_off;
    rec.table_off = rec.pool_off + round_up(c, 16);
    uint8_t* h = ctx->h_pool + rec.pool_off;
    bool ok = true;
    if (c) ok &= cudaMemcpyAsync(h, p.payload, c, cudaMemcpyDeviceToHost, ctx->side) == cudaSuccess;
    ok &= cudaMemcpyAsync(h + round_up(c, 16), p.table, p.table_bytes, cudaMemcpyDeviceToHost,
                          ctx->side) == cudaSuccess;
    ok &= cudaEventRecord(slot.idle, ctx->side) == cudaSuccess;
    if (!ok) {
        ctx->pool.release(rec.pool_off, rec.pool_bytes);
        return -static_cast<int64_t>(CDMA_ERR_CUDA);
    }
    out->id = ctx->next_ticket++;
    ctx->tickets[out->id] = rec;
    return static_cast<int64_t>(c);
}

// OFF without a host-side wait (Fig. 2b: the offload of a layer's map overlaps the layers that
// follow; Section V-D: the size is reported on completion, not needed to start the copy).
int cdma_offload_async(cdma_ctx* ctx, const void* d_src, uint64_t n, int dtype, int layout, void* compute_stream,
                       cdma_ticket* out) {
    if (ctx == nullptr || out == nullptr) return CDMA_ERR_INVALID_ARG;
    if (cdma_dtype_size(dtype) == 0) return CDMA_ERR_UNSUPPORTED_DTYPE;
    cudaStream_t compute = static_cast<cudaStream_t>(compute_stream);
    // keep the ring of pinned result words ahead of the tickets that still point into it
    while (ctx->pending.size() + ctx->unresolved.size() + 2 >= kResultRing) {
        if (!ctx->unresolved.empty()) settle_ticket(ctx, ctx->unresolved.front(), true);
        else if (wait_all(ctx) != CDMA_OK) return CDMA_ERR_CUDA;
    }
    Slot& slot = ctx->slots[ctx->next_slot % kSlots];
    SlotPlan p;
    if (!plan_slot(slot, n, dtype, &p)) return CDMA_ERR_BUFFER_TOO_SMALL;
    // the size is not known yet: reserve the most this slot's payload can be; the rest comes back
    // when the ticket is settled
    const uint64_t table_room = round_up(p.table_bytes, kAlign);
    TicketRec rec{n, dtype, layout, 0, 0, table_room + round_up(p.capacity, 16), 0, 0};
    if (!pool_alloc(ctx, rec.pool_bytes, &rec.pool_off) || rec.pool_off + rec.pool_bytes > ctx->pool_bytes)
        return CDMA_ERR_OUT_OF_MEMORY;
    rec.table_off = rec.pool_off;
    rec.payload_off = rec.pool_off + table_room;
    void* m_payload = nullptr;
    void* m_table = nullptr;
    cudaEvent_t done = take_event(ctx);
    bool ok = done != nullptr;
    ok = ok && cudaHostGetDevicePointer(&m_payload, ctx->h_pool + rec.payload_off, 0) == cudaSuccess;
    ok = ok && cudaHostGetDevicePointer(&m_table, ctx->h_pool + rec.table_off, 0) == cudaSuccess;
    // the slot's previous copy must have drained before the kernel overwrites it
    ok = ok && (!slot.used || cudaStreamWaitEvent(compute, slot.idle, 0) == cudaSuccess);
    uint64_t* res = next_result_words(ctx);
    int st = ok ? cdma_zvc_compress_async(d_src, n, dtype, layout, p.payload, p.capacity, p.table, p.ws, p.ws_bytes,
                                          compute, res)
                : CDMA_ERR_CUDA;
    if (st == CDMA_OK) {
        ++ctx->next_slot;
        slot.used = true;
        ok = cudaEventRecord(slot.staged, compute) == cudaSuccess;
        ok = ok && cudaStreamWaitEvent(ctx->side, slot.staged, 0) == cudaSuccess;
        if (ok) {
            offload_copy_kernel<<<kCopyCtas, kCopyThreads, 0, ctx->side>>>(
                p.ws, reinterpret_cast<const uint4*>(p.payload), static_cast<uint4*>(m_payload),
                reinterpret_cast<const uint4*>(p.table), static_cast<uint4*>(m_table), (p.table_bytes + 15) / 16,
                p.capacity);
            cdma::count_kernel_launch();
            ok = cudaGetLastError() == cudaSuccess;
        }
        // whatever happened, the slot is busy until the work enqueued so far is through
        cudaEventRecord(slot.idle, ok ? ctx->side : compute);
        ok = ok && cudaEventRecord(done, ctx->side) == cudaSuccess;
        if (!ok) st = CDMA_ERR_CUDA;
    }
    if (st != CDMA_OK) {
        cudaGetLastError();
        if (done) ctx->spare_events.push_back(done);
        ctx->pool.release(rec.pool_off, rec.pool_bytes);
        return st;
    }
    rec.resolved = false;
    rec.res = res;
    rec.done = done;
    out->id = ctx->next_ticket++;
    ctx->tickets[out->id] = rec;
    ctx->unresolved.push_back(out->id);
    return CDMA_OK;
}

static int prefetch_enqueue(cdma_ctx* ctx, cdma_ticket ticket, void* d_dst, void* compute_stream,
                            Slot** used_slot, uint64_t** result, uint64_t* dense_bytes) {
    if (ctx == nullptr) return CDMA_ERR_INVALID_ARG;
    settle_ticket(ctx, ticket.id, true);      // an asynchronous offload's size is needed now
    auto it = ctx->tickets.find(ticket.id);
    if (it == ctx->tickets.end()) return CDMA_ERR_BAD_TICKET;
    const TicketRec rec = it->second;
    cudaStream_t compute = static_cast<cudaStream_t>(compute_stream);
    if (ctx->pending.size() + ctx->unresolved.size() + 2 >= kResultRing) {
        if (wait_all(ctx) != CDMA_OK) return CDMA_ERR_CUDA;
        settle_all(ctx, true);
    }
    Slot& slot = ctx->slots[ctx->next_slot++ % kSlots];
    SlotPlan p;
    if (!plan_slot(slot, rec.n, rec.dtype, &p) || p.capacity < rec.payload_bytes)
        return CDMA_ERR_BUFFER_TOO_SMALL;
    if (slot.used && cudaStreamWaitEvent(ctx->side, slot.idle, 0) != cudaSuccess) return CDMA_ERR_CUDA;
    bool ok = true;
    if (rec.payload_bytes)
        ok &= cudaMemcpyAsync(p.payload, ctx->h_pool + rec.payload_off, rec.payload_bytes,
                              cudaMemcpyHostToDevice, ctx->side) == cudaSuccess;
    ok &= cudaMemcpyAsync(p.table, ctx->h_pool + rec.table_off, p.table_bytes, cudaMemcpyHostToDevice,
                          ctx->side) == cudaSuccess;
    ok &= cudaEventRecord(slot.staged, ctx->side) == cudaSuccess;
    ok &= cudaStreamWaitEvent(compute, slot.staged, 0) == cudaSuccess;
    // the pool region is given back below while this copy may still be reading it: whoever
    // writes the pool from another stream waits for this event first
    ok &= cudaEventRecord(ctx->pool_read, ctx->side) == cudaSuccess;
    if (!ok) return CDMA_ERR_CUDA;
    ctx->pool_read_used = true;
    slot.used = true;
    cudaEventRecord(slot.idle, ctx->side);
    uint64_t* res = next_result_words(ctx);
    const int st = cdma_zvc_decompress_async(p.payload, rec.payload_bytes, p.table, rec.n, rec.dtype,
                                             rec.layout, d_dst, p.ws, p.ws_bytes, compute, res);
    if (st != CDMA_OK) return st;   // the ticket stays valid: nothing was consumed
    if (cudaEventRecord(slot.idle, compute) != cudaSuccess) return CDMA_ERR_CUDA;
    // The region can be recycled now: later copies into it are enqueued on the same
    // side stream, behind the copy just issued, and a kernel that writes the pool from
    // the caller's stream waits for pool_read first.
    ctx->pool.release(rec.pool_off, rec.pool_bytes);
    ctx->tickets.erase(it);
    *used_slot = &slot;
    *result = res;
    *dense_bytes = rec.n * cdma_dtype_size(rec.dtype);
    return CDMA_OK;
}

int cdma_prefetch_async(cdma_ctx* ctx, cdma_ticket ticket, void* d_dst, void* compute_stream) {
    Slot* slot = nullptr;
    uint64_t* res = nullptr;
    uint64_t dense = 0;
    const int st = prefetch_enqueue(ctx, ticket, d_dst, compute_stream, &slot, &res, &dense);
    if (st == CDMA_OK) ctx->pending.push_back(res);
    return st;
}

int64_t cdma_prefetch(cdma_ctx* ctx, cdma_ticket ticket, void* d_dst, void* compute_stream) {
    Slot* slot = nullptr;
    uint64_t* res = nullptr;
    uint64_t dense = 0;
    const int st = prefetch_enqueue(ctx, ticket, d_dst, compute_stream, &slot, &res, &dense);
    if (st != CDMA_OK) return -static_cast<int64_t>(st);
    if (cudaEventSynchronize(slot->idle) != cudaSuccess) return -static_cast<int64_t>(CDMA_ERR_CUDA);
    if (res[1] != 0) return -static_cast<int64_t>(res[1]);
    return static_cast<int64_t>(dense);
}


// ---- direct variants: the kernels read and write the pinned pool themselves ----------------------
// (Section V-D: one call that compresses while it copies and reports the size on completion; here the
// copy over the host link is the kernel's own stores into mapped host memory.)

int64_t cdma_offload_direct(cdma_ctx* ctx, const void* d_src, uint64_t n, int dtype, int layout,
                            void* compute_stream, cdma_ticket* out) {
    if (ctx == nullptr || out == nullptr) return -static_cast<int64_t>(CDMA_ERR_INVALID_ARG);
    if (cdma_dtype_size(dtype) == 0) return -static_cast<int64_t>(CDMA_ERR_UNSUPPORTED_DTYPE);
    cudaStream_t compute = static_cast<cudaStream_t>(compute_stream);
    // only the workspace lives on the device: take it from a staging slot
    Slot& slot = ctx->slots[ctx->next_slot++ % kSlots];
    const uint64_t ws_bytes = cdma_zvc_workspace_bytes(n, dtype);
    if (slot.bytes < ws_bytes) return -static_cast<int64_t>(CDMA_ERR_BUFFER_TOO_SMALL);
    // the size is unknown until the kernel is done: reserve the worst case, give the rest back after
    const uint64_t table_bytes = 8 * cdma_zvc_table_entries(n);
    const uint64_t cap = cdma_zvc_max_compressed_bytes(n, dtype);
    TicketRec rec{n, dtype, layout, 0, 0, round_up(table_bytes, kAlign) + cap, 0, 0};
    if (!pool_alloc(ctx, rec.pool_bytes, &rec.pool_off) || rec.pool_off + rec.pool_bytes > ctx->pool_bytes)
        return -static_cast<int64_t>(CDMA_ERR_OUT_OF_MEMORY);
    rec.table_off = rec.pool_off;
    rec.payload_off = rec.pool_off + round_up(table_bytes, kAlign);
    void* d_payload = nullptr;
    void* d_table = nullptr;
    if (cudaHostGetDevicePointer(&d_payload, ctx->h_pool + rec.payload_off, 0) != cudaSuccess ||
        cudaHostGetDevicePointer(&d_table, ctx->h_pool + rec.table_off, 0) != cudaSuccess) {
        cudaGetLastError();
        ctx->pool.release(rec.pool_off, rec.pool_bytes);
        return -static_cast<int64_t>(CDMA_ERR_CUDA);
    }
    // the kernel writes the pool from the caller's stream: a region recycled by an earlier
    // prefetch may still be read by that prefetch's copy on the side stream
    if ((slot.used && cudaStreamWaitEvent(compute, slot.idle, 0) != cudaSuccess) ||
        (ctx->pool_read_used && cudaStreamWaitEvent(compute, ctx->pool_read, 0) != cudaSuccess)) {
        ctx->pool.release(rec.pool_off, rec.pool_bytes);
        return -static_cast<int64_t>(CDMA_ERR_CUDA);
    }
    uint64_t* res = next_result_words(ctx);
    const int st = cdma_zvc_compress_async(d_src, n, dtype, layout, d_payload, cap, static_cast<uint64_t*>(d_table),
                                           slot.base, slot.bytes, compute, res);
    if (st != CDMA_OK) {
        ctx->pool.release(rec.pool_off, rec.pool_bytes);
        return -static_cast<int64_t>(st);
    }
    slot.used = true;
    if (cudaEventRecord(slot.idle, compute) != cudaSuccess || cudaEventSynchronize(slot.idle) != cudaSuccess) {
        ctx->pool.release(rec.pool_off, rec.pool_bytes);
        return -static_cast<int64_t>(CDMA_ERR_CUDA);
    }
    if (res[1] != 0) {
        ctx->pool.release(rec.pool_off, rec.pool_bytes);
        return -static_cast<int64_t>(res[1]);
    }
    rec.payload_bytes = res[0];
    const uint64_t used = round_up(table_bytes, kAlign) + rec.payload_bytes;
    ctx->pool.shrink(rec.pool_off, rec.pool_bytes, used);
    rec.pool_bytes = used;
    out->id = ctx->next_ticket++;
    ctx->tickets[out->id] = rec;
    return static_cast<int64_t>(rec.payload_bytes);
}

int64_t cdma_prefetch_direct(cdma_ctx* ctx, cdma_ticket ticket, void* d_dst, void* compute_stream) {
    if (ctx == nullptr) return -static_cast<int64_t>(CDMA_ERR_INVALID_ARG);
    settle_ticket(ctx, ticket.id, true);
    auto it = ctx->tickets.find(ticket.id);
    if (it == ctx->tickets.end()) return -static_cast<int64_t>(CDMA_ERR_BAD_TICKET);
    const TicketRec rec = it->second;
    cudaStream_t compute = static_cast<cudaStream_t>(compute_stream);
    Slot& slot = ctx->slots[ctx->next_slot++ % kSlots];
    if (slot.bytes < cdma_zvc_workspace_bytes(rec.n, rec.dtype)) return -static_cast<int64_t>(CDMA_ERR_BUFFER_TOO_SMALL);
    void* d_payload = nullptr;
    void* d_table = nullptr;
    if (cudaHostGetDevicePointer(&d_payload, ctx->h_pool + rec.payload_off, 0) != cudaSuccess ||
        cudaHostGetDevicePointer(&d_table, ctx->h_pool + rec.table_off, 0) != cudaSuccess) {
        cudaGetLastError();
        return -static_cast<int64_t>(CDMA_ERR_CUDA);
    }
    // earlier copies into this region were enqueued on the side stream: let them land first
    if (cudaStreamSynchronize(ctx->side) != cudaSuccess) return -static_cast<int64_t>(CDMA_ERR_CUDA);
    if (slot.used && cudaStreamWaitEvent(compute, slot.idle, 0) != cudaSuccess)
        return -static_cast<int64_t>(CDMA_ERR_CUDA);
    uint64_t* res = next_result_words(ctx);
    const int st = cdma_zvc_decompress_async(d_payload, rec.payload_bytes, static_cast<const uint64_t*>(d_table), rec.n,
                                             rec.dtype, rec.layout, d_dst, slot.base, slot.bytes, compute, res);
    if (st != CDMA_OK) return -static_cast<int64_t>(st);
    slot.used = true;
    if (cudaEventRecord(slot.idle, compute) != cudaSuccess || cudaEventSynchronize(slot.idle) != cudaSuccess)
        return -static_cast<int64_t>(CDMA_ERR_CUDA);
    ctx->pool.release(rec.pool_off, rec.pool_bytes);
    ctx->tickets.erase(it);
    if (res[1] != 0) return -static_cast<int64_t>(res[1]);
    return static_cast<int64_t>(rec.n * cdma_dtype_size(rec.dtype));
}

int cdma_ctx_synchronize(cdma_ctx* ctx) {
    if (ctx == nullptr) return CDMA_ERR_INVALID_ARG;
    const int st = wait_all(ctx);
    if (st != CDMA_OK) return st;
    settle_all(ctx, true);
    const int d = ctx->deferred;
    ctx->deferred = 0;
    return d;
}

int cdma_ticket_info(cdma_ctx* ctx, cdma_ticket ticket, uint64_t* payload_bytes, uint64_t* n) {
    if (ctx == nullptr) return CDMA_ERR_INVALID_ARG;
    settle_ticket(ctx, ticket.id, true);
    auto it = ctx->tickets.find(ticket.id);
    if (it == ctx->tickets.end()) return CDMA_ERR_BAD_TICKET;
    if (payload_bytes) *payload_bytes = it->second.payload_bytes;
    if (n) *n = it->second.n;
    return CDMA_OK;
}

int cdma_ticket_host_view(cdma_ctx* ctx, cdma_ticket ticket, const void** h_payload, const uint64_t** h_table) {
    if (ctx == nullptr) return CDMA_ERR_INVALID_ARG;
    settle_ticket(ctx, ticket.id, true);
    auto it = ctx->tickets.find(ticket.id);
    if (it == ctx->tickets.end()) return CDMA_ERR_BAD_TICKET;
    // copies into the pool are asynchronous on the side stream: let them land before the host looks
    if (cudaStreamSynchronize(ctx->side) != cudaSuccess) return CDMA_ERR_CUDA;
    if (h_payload) *h_payload = ctx->h_pool + it->second.payload_off;
    if (h_table) *h_table = reinterpret_cast<const uint64_t*>(ctx->h_pool + it->second.table_off);
    return CDMA_OK;
}

int64_t cdma_zvc_compress_host(cdma_ctx* ctx, const void* h_src, uint64_t n, int dtype, int layout,
                               void* h_dst, uint64_t dst_capacity, uint64_t* h_table) {
    if (ctx == nullptr || h_table == nullptr || (n && h_src == nullptr) ||
        (dst_capacity && h_dst == nullptr))
        return -static_cast<int64_t>(CDMA_ERR_INVALID_ARG);
    const uint32_t s = cdma_dtype_size(dtype);
    if (s == 0) return -static_cast<int64_t>(CDMA_ERR_UNSUPPORTED_DTYPE);
    int st;
    {
        // All three buffers page-locked: one kernel reads the tensor and writes payload and
        // table over the host link as it goes (both directions of the link busy at once),
        // with no device staging and no separate copies.
        void* m_src = n ? mapped_view(h_src, 16) : nullptr;
        void* m_dst = dst_capacity ? mapped_view(h_dst, 16) : nullptr;
        void* m_table = mapped_view(h_table, 8);
        if ((n == 0 || m_src) && (dst_capacity == 0 || m_dst) && m_table) {
            Slot& slot = ctx->slots[ctx->next_slot++ % kSlots];
            SlotPlan p;
            if (!plan_slot(slot, n, dtype, &p)) return -static_cast<int64_t>(CDMA_ERR_BUFFER_TOO_SMALL);
            if (slot.used && cudaStreamWaitEvent(ctx->side, slot.idle, 0) != cudaSuccess)
                return -static_cast<int64_t>(CDMA_ERR_CUDA);
            uint64_t* res = next_result_words(ctx);
            st = cdma_zvc_compress_async(m_src, n, dtype, layout, m_dst, dst_capacity,
                                         static_cast<uint64_t*>(m_table), p.ws, p.ws_bytes, ctx->side, res);
            if (st != CDMA_OK) return -static_cast<int64_t>(st);
            slot.used = true;
            cudaEventRecord(slot.idle, ctx->side);
            if (cudaStreamSynchronize(ctx->side) != cudaSuccess) return -static_cast<int64_t>(CDMA_ERR_CUDA);
            if (res[1] != 0) return -static_cast<int64_t>(res[1]);
            return static_cast<int64_t>(res[0]);
        }
    }
    st = ensure_dense(ctx, n * s);
    if (st != CDMA_OK) return -static_cast<int64_t>(st);
    Slot& slot = ctx->slots[ctx->next_slot++ % kSlots];
    SlotPlan p;
    if (!plan_slot(slot, n, dtype, &p)) return -static_cast<int64_t>(CDMA_ERR_BUFFER_TOO_SMALL);
    if (slot.used && cudaStreamWaitEvent(ctx->side, slot.idle, 0) != cudaSuccess)
        return -static_cast<int64_t>(CDMA_ERR_CUDA);
    if (n && cudaMemcpyAsync(ctx->d_dense, h_src, n * s, cudaMemcpyHostToDevice, ctx->side) != cudaSuccess)
        return -static_cast<int64_t>(CDMA_ERR_CUDA);
    uint64_t* res = next_result_words(ctx);
    st = cdma_zvc_compress_async(ctx->d_dense, n, dtype, layout, p.payload, p.capacity, p.table, p.ws,
                                 p.ws_bytes, ctx->side, res);
    if (st != CDMA_OK) return -static_cast<int64_t>(st);
    slot.used = true;
    cudaEventRecord(slot.idle, ctx->side);
    if (cudaStreamSynchronize(ctx->side) != cudaSuccess) return -static_cast<int64_t>(CDMA_ERR_CUDA);
    if (res[1] != 0) return -static_cast<int64_t>(res[1]);
    const uint64_t c = res[0];
    if (c > dst_capacity) return -static_cast<int64_t>(CDMA_ERR_BUFFER_TOO_SMALL);
    bool ok = true;
    if (c) ok &= cudaMemcpyAsync(h_dst, p.payload, c, cudaMemcpyDeviceToHost, ctx->side) == cudaSuccess;
    ok &= cudaMemcpyAsync(h_table, p.table, p.table_bytes, cudaMemcpyDeviceToHost, ctx->side) ==
          cudaSuccess;
    ok &= cudaEventRecord(slot.idle, ctx->side) == cudaSuccess;
    ok &= cudaStreamSynchronize(ctx->side) == cudaSuccess;
    if (!ok) return -static_cast<int64_t>(CDMA_ERR_CUDA);
    return static_cast<int64_t>(c);
}

int64_t cdma_zvc_decompress_host(cdma_ctx* ctx, const void* h_src, uint64_t src_bytes,
                                 const uint64_t* h_table, uint64_t n, int dtype, int layout,
                                 void* h_dst) {
    if (ctx == nullptr || h_table == nullptr || (src_bytes && h_src == nullptr) ||
        (n && h_dst == nullptr))
        return -static_cast<int64_t>(CDMA_ERR_INVALID_ARG);
    const uint32_t s = cdma_dtype_size(dtype);
    if (s == 0) return -static_cast<int64_t>(CDMA_ERR_UNSUPPORTED_DTYPE);
    int st;
    {
        // All three buffers page-locked: one kernel loads payload and table over the host
        // link and stores the dense tensor back over it.
        void* m_src = src_bytes ? mapped_view(h_src, 16) : nullptr;
        void* m_table = mapped_view(h_table, 8);
        void* m_dst = n ? mapped_view(h_dst, 16) : nullptr;
        if ((src_bytes == 0 || m_src) && (n == 0 || m_dst) && m_table) {
            Slot& slot = ctx->slots[ctx->next_slot++ % kSlots];
            SlotPlan p;
            if (!plan_slot(slot, n, dtype, &p)) return -static_cast<int64_t>(CDMA_ERR_BUFFER_TOO_SMALL);
            if (slot.used && cudaStreamWaitEvent(ctx->side, slot.idle, 0) != cudaSuccess)
                return -static_cast<int64_t>(CDMA_ERR_CUDA);
            uint64_t* res = next_result_words(ctx);
            st = cdma_zvc_decompress_async(m_src, src_bytes, static_cast<const uint64_t*>(m_table), n, dtype,
                                           layout, m_dst, p.ws, p.ws_bytes, ctx->side, res);
            if (st != CDMA_OK) return -static_cast<int64_t>(st);
            slot.used = true;
            cudaEventRecord(slot.idle, ctx->side);
            if (cudaStreamSynchronize(ctx->side) != cudaSuccess) return -static_cast<int64_t>(CDMA_ERR_CUDA);
            if (res[1] != 0) return -static_cast<int64_t>(res[1]);
            return static_cast<int64_t>(n * s);
        }
    }
    st = ensure_dense(ctx, n * s);
    if (st != CDMA_OK) return -static_cast<int64_t>(st);
    Slot& slot = ctx->slots[ctx->next_slot++ % kSlots];
    SlotPlan p;
    if (!plan_slot(slot, n, dtype, &p) || p.capacity < src_bytes)
        return -static_cast<int64_t>(src_bytes > cdma_zvc_max_compressed_bytes(n, dtype)
                                         ? CDMA_ERR_CORRUPT_STREAM
                                         : CDMA_ERR_BUFFER_TOO_SMALL);
    if (slot.used && cudaStreamWaitEvent(ctx->side, slot.idle, 0) != cudaSuccess)
        return -static_cast<int64_t>(CDMA_ERR_CUDA);
    bool ok = true;
    if (src_bytes)
        ok &= cudaMemcpyAsync(p.payload, h_src, src_bytes, cudaMemcpyHostToDevice, ctx->side) == cudaSuccess;
    ok &= cudaMemcpyAsync(p.table, h_table, p.table_bytes, cudaMemcpyHostToDevice, ctx->side) == cudaSuccess;
    if (!ok) return -static_cast<int64_t>(CDMA_ERR_CUDA);
    uint64_t* res = next_result_words(ctx);
    st = cdma_zvc_decompress_async(p.payload, src_bytes, p.table, n, dtype, layout, ctx->d_dense, p.ws,
                                   p.ws_bytes, ctx->side, res);
    slot.used = true;
    cudaEventRecord(slot.idle, ctx->side);
    if (st != CDMA_OK) return -static_cast<int64_t>(st);
    if (n) ok &= cudaMemcpyAsync(h_dst, ctx->d_dense, n * s, cudaMemcpyDeviceToHost, ctx->side) == cudaSuccess;
    ok &= cudaEventRecord(slot.idle, ctx->side) == cudaSuccess;
    ok &= cudaStreamSynchronize(ctx->side) == cudaSuccess;
    if (!ok) return -static_cast<int64_t>(CDMA_ERR_CUDA);
    if (res[1] != 0) return -static_cast<int64_t>(res[1]);
    return static_cast<int64_t>(n * s);
}

}  // extern "C"
