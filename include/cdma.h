/*
 * cdma.h -- C ABI of the compressing-DMA (cDMA) zero-value-compression library
 *           for NVIDIA B200 (sm_100a).
 *
 * The paper proposes a memory copy that compresses activation maps on their
 * way from GPU memory to host memory and expands them on the way back, and
 * that reports the compressed size when the copy completes (Section V-D,
 * "Software Interface": cudaMemcpyCompressed).  This library provides that
 * operation in software: the codec runs as CUDA kernels on the SMs, the copy
 * over the host link is a plain cudaMemcpyAsync of the compressed bytes.
 *
 * Stream format (Section V-A, "Zero-value compression"):
 *   elements are taken 32 at a time in memory order (a "window").  A window's
 *   record is a 32-bit mask, least-significant byte first, bit i set when
 *   element i of the window is non-zero, followed by the window's non-zero
 *   elements in ascending order, bytes unchanged.  "Non-zero" is a test of
 *   the element's bit pattern (Section V-B: words are compared to zero), so
 *   -0.0, NaNs, denormals and infinities are kept.  The payload is the
 *   concatenation of all records with no header and no padding; its size is
 *   4*ceil(n/32) + s*nnz bytes for n elements of s bytes of which nnz are
 *   non-zero.  A short last window has zero bits for the missing elements.
 *   For 2-byte and 1-byte elements the window is still 32 elements with a
 *   32-bit mask.
 *
 * Framing for parallel decoding (outside the payload): an offset table of
 *   ceil(n/1024)+1 little-endian uint64.  Entry k is the payload offset of
 *   the record of window 32k ("chunk" k = 1024 elements, the 4 KB block of the
 *   paper's compression study, Fig. 11 caption); the last entry equals the
 *   payload size.
 *
 * Conventions
 *   - "d_" pointers are device memory of the current CUDA device, "h_"
 *     pointers are host memory.  Streams are passed as void* holding a
 *     cudaStream_t (NULL = the legacy default stream).
 *   - The caller owns every buffer passed in; the codec calls allocate
 *     nothing.  A cdma_ctx owns its pinned host pool, its device staging and
 *     its side stream.
 *   - Dense tensors and compressed buffers must start on a 16-byte boundary
 *     and must not overlap each other.  The tensor must be dense in its
 *     physical layout; the layout argument is a tag that is validated and
 *     recorded but does not change the bytes: the codec compresses memory
 *     order (Section V-A: ZVC is insensitive to the layout).
 *   - Functions returning int64_t return a byte count >= 0, or -status on
 *     failure.  Functions returning int return a status (0 = success).
 *     Nothing aborts, throws or traps; device-side failures (capacity
 *     overflow, malformed stream, a wait that ran out) are written to a
 *     status word and come back as a negative return.
 *   - A call never writes beyond dst_capacity / n elements, whatever the
 *     input holds.  Bytes of the destination between the payload's end and
 *     dst_capacity, and the contents of workspaces, are unspecified.
 *   - Not thread-safe per context or per workspace: two calls that share a
 *     workspace (or a context) must not overlap in time.
 */
#ifndef CDMA_H_
#define CDMA_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* status codes; negative returns are the negated code */
enum {
    CDMA_OK = 0,
    CDMA_ERR_INVALID_ARG = 1,        /* null pointer, overlap, size mismatch            */
    CDMA_ERR_UNSUPPORTED_DTYPE = 2,
    CDMA_ERR_UNSUPPORTED_LAYOUT = 3,
    CDMA_ERR_ALIGNMENT = 4,          /* a buffer is not 16-byte aligned                 */
    CDMA_ERR_BUFFER_TOO_SMALL = 5,   /* payload, table, workspace or pool too small     */
    CDMA_ERR_CORRUPT_STREAM = 6,     /* table or payload fails validation in decompress */
    CDMA_ERR_TIMEOUT = 7,            /* a bounded device-side wait ran out              */
    CDMA_ERR_CUDA = 8,               /* a CUDA runtime call failed                      */
    CDMA_ERR_OUT_OF_MEMORY = 9,      /* context pool exhausted / allocation failed      */
    CDMA_ERR_BAD_TICKET = 10
};

/* element types: only the width matters to the codec (4, 2, 2, 1 bytes); CDMA_U8
 * stands for any one-byte element (int8, uint8, an 8-bit float) */
enum { CDMA_F32 = 0, CDMA_F16 = 1, CDMA_BF16 = 2, CDMA_U8 = 3 };

/* physical layouts of a 4-D activation map (Section II-C); a tag only */
enum { CDMA_NCHW = 0, CDMA_NHWC = 1, CDMA_CHWN = 2 };

#define CDMA_WINDOW 32u           /* elements per mask (Section V-A)              */
#define CDMA_CHUNK 1024u          /* elements per offset-table entry              */

const char* cdma_status_string(int status);

/* Element width in bytes for a dtype code, 0 for an unknown code. */
uint32_t cdma_dtype_size(int dtype);

/* Worst-case payload size, 4*ceil(n/32) + s*n (every element non-zero: the
 * all-ones mask plus 32 values per window, Section V-A), rounded up to a
 * multiple of 16.  0 for an unknown dtype. */
uint64_t cdma_zvc_max_compressed_bytes(uint64_t n, int dtype);

/* Number of uint64 entries of the offset table: ceil(n/1024) + 1. */
uint64_t cdma_zvc_table_entries(uint64_t n);

/* Bytes of device scratch a codec call on n elements needs (both directions;
 * a multiple of 256).  Holds the status/result words and the inter-tile
 * prefix descriptors (one per tile of 8192 elements, 32 bytes apart). */
uint64_t cdma_zvc_workspace_bytes(uint64_t n, int dtype);

/*
 * Compress n elements at d_src into d_dst (payload) and d_table (offsets).
 * One pass over the input: per window mask, per-window record sizes, running
 * prefix across tiles, compaction (Section V-A; the engine's compare /
 * prefix-sum / shift / append stages of Section V-B).
 *
 *   d_src           dense tensor, n*s bytes, 16-byte aligned, read only
 *   dtype, layout   CDMA_F32/F16/BF16/U8; CDMA_NCHW/NHWC/CHWN (tag)
 *   d_dst           payload out; dst_capacity bytes, 16-byte aligned.  Any
 *                   capacity is accepted; if the payload does not fit the
 *                   call fails with BUFFER_TOO_SMALL having written only
 *                   bytes below dst_capacity.
 *   d_table         cdma_zvc_table_entries(n) uint64, 8-byte aligned
 *   d_workspace     >= cdma_zvc_workspace_bytes(n, dtype), 16-byte aligned;
 *                   contents on entry are irrelevant and nothing is cleared
 *                   between calls (what a launch reads there carries its tag)
 *   cuda_stream     stream the work is enqueued on
 *
 * cdma_zvc_compress waits for the stream and returns the payload size C
 * (Section V-D: the size is returned on completion).  n = 0 gives C = 0 and
 * table = {0}.
 *
 * cdma_zvc_compress_async only enqueues.  h_result must point to two uint64
 * in host memory, 8-byte aligned; once the stream reaches that point
 * h_result[0] holds C and h_result[1] the status code (0 on success).  With
 * page-locked memory (recommended) the codec kernel stores the two words there
 * itself; pageable memory gets a 16-byte copy behind the kernel instead.
 * d_src, d_dst and d_table may also be device views of page-locked host
 * memory: the kernel then reads / writes over the host link directly.
 */
int64_t cdma_zvc_compress(const void* d_src, uint64_t n, int dtype, int layout,
                          void* d_dst, uint64_t dst_capacity, uint64_t* d_table,
                          void* d_workspace, uint64_t workspace_bytes,
                          void* cuda_stream);

int cdma_zvc_compress_async(const void* d_src, uint64_t n, int dtype, int layout,
                            void* d_dst, uint64_t dst_capacity, uint64_t* d_table,
                            void* d_workspace, uint64_t workspace_bytes,
                            void* cuda_stream, uint64_t* h_result);

/*
 * Activation function and compression in one pass.  The sparsity this method
 * exploits is produced by the ReLU layers (Section IV), and the paper leaves
 * compressing "on the way into DRAM" as future work (Section IX): here the
 * kernel reads the pre-activation tensor once, applies y = max(x, 0), and writes
 * the compressed form of y -- and, when d_relu_out is not NULL, also the dense y
 * for the next layer -- so y is never read back from memory to be compressed.
 *
 *   ReLU rule, on bit patterns: an element is kept unchanged when it is greater
 *   than zero or a NaN of either sign (NaNs propagate, as in the usual framework
 *   ReLU); every other value (negatives, -0.0, +0.0, -Inf) becomes +0.0.
 *   d_relu_out   NULL, or n*s bytes, 16-byte aligned; may be d_src itself
 *                (in-place activation) but must not overlap it otherwise, nor
 *                the payload.
 * Everything else, and the payload/table produced, is exactly that of
 * cdma_zvc_compress applied to y.  CDMA_U8 is refused (UNSUPPORTED_DTYPE): what
 * "greater than zero" means for a one-byte pattern depends on the type behind it.
 */
int64_t cdma_zvc_relu_compress(const void* d_src, uint64_t n, int dtype, int layout,
                               void* d_relu_out, void* d_dst, uint64_t dst_capacity,
                               uint64_t* d_table, void* d_workspace, uint64_t workspace_bytes,
                               void* cuda_stream);
int cdma_zvc_relu_compress_async(const void* d_src, uint64_t n, int dtype, int layout,
                                 void* d_relu_out, void* d_dst, uint64_t dst_capacity,
                                 uint64_t* d_table, void* d_workspace, uint64_t workspace_bytes,
                                 void* cuda_stream, uint64_t* h_result);

/*
 * The same compression for callers that cannot allocate device memory: code
 * inside a memory manager's eviction path (where an allocation could re-enter
 * the manager, or fail because the device is full -- which is when activations
 * get offloaded), plug-ins that only ever receive buffers from their host
 * application, start-up and tear-down hooks.  (The paper has no counterpart:
 * its engine needs no software workspace.)  The call takes no workspace; it
 * uses one built into the library, a fixed device array of 1,048,832 bytes, and
 * it calls no cudaMalloc, cudaFree or any other allocating routine.
 *
 *   - Serves tensors of at most 2^28 elements; a larger n is refused with
 *     -CDMA_ERR_BUFFER_TOO_SMALL (the built-in workspace is too small for it)
 *     before anything is enqueued.
 *   - The array belongs to the library's device code: its memory is taken on a
 *     device when that code is loaded there, which with CUDA's default lazy
 *     loading is the first call made with that device current (at process start
 *     with CUDA_MODULE_LOADING=EAGER).  Every call looks up the array's device
 *     address (a table look-up after the first time).  Make a first call -- one
 *     with n = 0 will do -- at start-up, while memory is available and outside
 *     any stream capture; on a device too full to load the code that first call
 *     returns -CDMA_ERR_OUT_OF_MEMORY.  The memory is held until the process
 *     exits.
 *   - All calls on a device share the one array, which keeps the previous
 *     call's contents.  Nothing in it has to be cleared: a launch only trusts
 *     look-back descriptors that carry its own tag and writes its result words
 *     before reading them.  Two calls that overlap in time on the same device
 *     (different streams or threads) still race on it and give undefined
 *     results: serialise them.
 *   - Otherwise identical to cdma_zvc_compress: same arguments and checks
 *     (d_src may be a device view of page-locked host memory), same payload and
 *     table, waits for the stream and returns C or -status.
 */
int64_t cdma_zvc_compress_static_ws(const void* d_src, uint64_t n, int dtype, int layout,
                                    void* d_dst, uint64_t dst_capacity, uint64_t* d_table,
                                    void* cuda_stream);

/*
 * Expand a payload back into n dense elements (Section V-B, decompression
 * engine: the pop-count of a mask tells how many values its window takes,
 * values or zeros are steered into place).
 *
 *   d_src, src_bytes   payload and its exact size C, 16-byte aligned
 *   d_table            the offset table produced by compression
 *   d_dst              n*s bytes out, 16-byte aligned
 *   d_workspace        >= cdma_zvc_workspace_bytes(n, dtype)
 *
 * The table and every record are validated: offsets must be non-decreasing,
 * inside the payload and a chunk must decode to exactly its byte range; a
 * mask must not name an element at index >= n.  A violation gives
 * CORRUPT_STREAM; no read leaves [d_src, d_src+src_bytes) and no write leaves
 * the n elements regardless.
 *
 * cdma_zvc_decompress waits for the stream and returns n*s.
 * cdma_zvc_decompress_async only enqueues; h_result as above, with
 * h_result[0] = n*s.
 */
int64_t cdma_zvc_decompress(const void* d_src, uint64_t src_bytes,
                            const uint64_t* d_table, uint64_t n, int dtype,
                            int layout, void* d_dst, void* d_workspace,
                            uint64_t workspace_bytes, void* cuda_stream);

int cdma_zvc_decompress_async(const void* d_src, uint64_t src_bytes,
                              const uint64_t* d_table, uint64_t n, int dtype,
                              int layout, void* d_dst, void* d_workspace,
                              uint64_t workspace_bytes, void* cuda_stream,
                              uint64_t* h_result);

/*
 * Backward pass of the activation function straight from the compressed map.
 * The offloaded maps are needed again in the backward pass (Section II-B); for a
 * ReLU layer all that is needed of y = max(x, 0) is which elements are non-zero,
 * and that is what the masks of the stream record (Section V-A).  The call
 * computes dx = dy where the element of the compressed tensor is non-zero, else
 * +0, reading the masks only: the dense y is never rebuilt in memory (Section IX
 * leaves keeping activations compressed as future work).
 *
 *   d_src, src_bytes, d_table   payload, its exact size and offset table, as for
 *                               cdma_zvc_decompress (validated the same way)
 *   d_dy        incoming gradient, n*s bytes, 16-byte aligned, same dtype
 *   d_dx        outgoing gradient, n*s bytes, 16-byte aligned; may be d_dy itself
 *               (in place), must not overlap it otherwise, nor the payload
 *   d_workspace >= cdma_zvc_workspace_bytes(n, dtype)
 *
 * For a payload produced from a ReLU output (cdma_zvc_relu_compress or
 * compression of y) this is the framework's ReLU backward, bit for bit: elements
 * whose y is a NaN pass dy on, as a comparison "y <= 0 ? 0 : dy" does.
 * cdma_zvc_relu_backward waits for the stream and returns n*s or -status;
 * the _async form only enqueues, h_result as for cdma_zvc_decompress_async.
 */
int64_t cdma_zvc_relu_backward(const void* d_src, uint64_t src_bytes, const uint64_t* d_table,
                               uint64_t n, int dtype, int layout, const void* d_dy, void* d_dx,
                               void* d_workspace, uint64_t workspace_bytes, void* cuda_stream);
int cdma_zvc_relu_backward_async(const void* d_src, uint64_t src_bytes, const uint64_t* d_table,
                                 uint64_t n, int dtype, int layout, const void* d_dy, void* d_dx,
                                 void* d_workspace, uint64_t workspace_bytes, void* cuda_stream,
                                 uint64_t* h_result);

/* ------------------------------------------------------------------------ *
 * Run-length comparison codec (Section V-A, "Run-length encoding compression";
 * its dependence on the activation layout is the subject of Section VI-A,
 * Fig. 11).  The paper names the scheme but gives no format; this one is the
 * library's own, on the framing of the zero-value codec: independent chunks of
 * 1024 elements, a table of cdma_zvc_table_entries(n) byte offsets outside the
 * payload.  A chunk is a sequence of records {token, literals}: the 32-bit
 * little-endian token holds the number of zero elements in front (low 16
 * bits) and the number of non-zero elements that follow (high 16 bits); one
 * record per maximal run of non-zero elements, plus a last record without
 * literals when the chunk ends in zeros.  Chunk size = 4 * records + 4 *
 * non-zero elements, at most 4100 bytes, so cdma_zvc_max_compressed_bytes()
 * and cdma_zvc_workspace_bytes() size its buffers too.  "Zero" is bitwise.
 *
 * dtype must be CDMA_F32 (CDMA_ERR_UNSUPPORTED_DTYPE otherwise).  Arguments,
 * ownership, alignment, capacity and error behaviour are those of
 * cdma_zvc_compress / cdma_zvc_decompress and their _async forms; a stream
 * in which a literal is zero or a token is zero is CDMA_ERR_CORRUPT_STREAM.
 * ------------------------------------------------------------------------ */
int64_t cdma_rle_compress(const void* d_src, uint64_t n, int dtype, int layout,
                          void* d_dst, uint64_t dst_capacity, uint64_t* d_table,
                          void* d_workspace, uint64_t workspace_bytes, void* cuda_stream);
int cdma_rle_compress_async(const void* d_src, uint64_t n, int dtype, int layout,
                            void* d_dst, uint64_t dst_capacity, uint64_t* d_table,
                            void* d_workspace, uint64_t workspace_bytes, void* cuda_stream,
                            uint64_t* h_result);
int64_t cdma_rle_decompress(const void* d_src, uint64_t src_bytes, const uint64_t* d_table,
                            uint64_t n, int dtype, int layout, void* d_dst,
                            void* d_workspace, uint64_t workspace_bytes, void* cuda_stream);
int cdma_rle_decompress_async(const void* d_src, uint64_t src_bytes, const uint64_t* d_table,
                              uint64_t n, int dtype, int layout, void* d_dst,
                              void* d_workspace, uint64_t workspace_bytes, void* cuda_stream,
                              uint64_t* h_result);

/* ------------------------------------------------------------------------ *
 * Offload pipeline (Section III, Fig. 2b: OFF(n) in the forward pass, PRE(n)
 * in reverse order in the backward pass; Section V-D: the compressed copy
 * replaces the cudaMemcpy calls of the memory manager).
 * ------------------------------------------------------------------------ */
typedef struct cdma_ctx cdma_ctx;
typedef struct { uint64_t id; } cdma_ticket;

/*
 * Create a context on the current device.
 *   pinned_bytes          size of the pinned host pool that holds offloaded
 *                         payloads and their tables
 *   device_staging_bytes  device memory for compressed staging; split into two
 *                         slots so that one tensor's copy overlaps the next
 *                         tensor's codec kernel.  A slot must hold the
 *                         tensor's payload, table and workspace; sizing a slot
 *                         for cdma_zvc_max_compressed_bytes of the largest
 *                         tensor never fails, a smaller one fails with
 *                         BUFFER_TOO_SMALL when a payload does not fit.
 * All allocation happens here (and, for the host-buffer calls below, on the
 * first call that needs a larger dense staging buffer).
 */
int cdma_ctx_create(uint64_t pinned_bytes, uint64_t device_staging_bytes, cdma_ctx** out);
int cdma_ctx_destroy(cdma_ctx* ctx);

/*
 * OFF: compress the tensor on compute_stream into a staging slot, wait for
 * the kernel (not for the copy), then enqueue the device-to-host copy of
 * exactly C payload bytes plus the table on the context's side stream, into
 * the pinned pool.  Returns C.  The copy proceeds while the caller continues;
 * the next cdma_offload's kernel overlaps it.  d_src may be reused as soon as
 * the call returns.
 */
int64_t cdma_offload(cdma_ctx* ctx, const void* d_src, uint64_t n, int dtype, int layout,
                     void* compute_stream, cdma_ticket* out);

/*
 * OFF without a host-side wait (Fig. 2b: the offload of layer n's map runs beside
 * the forward computation of the layers that follow; Section V-D: the compressed
 * size is reported on completion).  The call enqueues the compression on
 * compute_stream and, behind it on the context's side stream, a small copy kernel
 * that reads the payload size on the device and stores exactly that many bytes,
 * plus the table, into the (mapped) pinned pool; it returns a ticket at once,
 * without waiting for anything the caller has enqueued on compute_stream.
 * Returns a status.  The pinned pool holds a worst-case reservation for the
 * ticket until its size is first needed -- by cdma_ticket_info,
 * cdma_ticket_host_view, cdma_prefetch*, cdma_ctx_synchronize or a later
 * reservation that does not fit -- which waits for the ticket's bytes to have
 * landed and gives the unused part back.  A failure of the compression (for
 * instance a staging slot too small for the payload) drops the ticket and is
 * reported by cdma_ctx_synchronize; the ticket is then unknown.  d_src must stay
 * unchanged until the compression kernel has run (stream order on
 * compute_stream guarantees it for work enqueued later on that stream).
 */
int cdma_offload_async(cdma_ctx* ctx, const void* d_src, uint64_t n, int dtype, int layout,
                       void* compute_stream, cdma_ticket* out);

/*
 * PRE: enqueue the host-to-device copy of the ticket's payload and table on
 * the side stream, then the decompression into d_dst on compute_stream once
 * the copy has landed.  The ticket and its pinned bytes are released.
 * cdma_prefetch waits for the decompression and returns n*s (or -status);
 * cdma_prefetch_async returns at once so the next tensor's copy overlaps this
 * tensor's kernel; its outcome is reported by cdma_ctx_synchronize.
 */
int64_t cdma_prefetch(cdma_ctx* ctx, cdma_ticket ticket, void* d_dst, void* compute_stream);
int cdma_prefetch_async(cdma_ctx* ctx, cdma_ticket ticket, void* d_dst, void* compute_stream);

/*
 * The same OFF / PRE with no device staging and no second copy, closest to the
 * single compressed-copy call the paper envisions (Section V-D): the compress
 * kernel stores its payload and table straight into the context's pinned pool
 * (mapped into the device's address space), so the bytes cross the host link as
 * the kernel produces them, and the decompress kernel loads them from there.
 * Only the workspace is taken from a staging slot.  Both calls wait for their
 * kernel -- which now lasts as long as the transfer -- and return C / n*s.
 * cdma_offload_direct reserves the worst-case size in the pool while it runs
 * and gives the unused part back; tickets of either kind can be prefetched by
 * either cdma_prefetch or cdma_prefetch_direct.
 */
int64_t cdma_offload_direct(cdma_ctx* ctx, const void* d_src, uint64_t n, int dtype, int layout,
                            void* compute_stream, cdma_ticket* out);
int64_t cdma_prefetch_direct(cdma_ctx* ctx, cdma_ticket ticket, void* d_dst, void* compute_stream);

/* Wait for everything the context enqueued; returns the first deferred
 * failure of an asynchronous call since the last synchronize, else 0. */
int cdma_ctx_synchronize(cdma_ctx* ctx);

/* Size facts of a live ticket: payload bytes and element count. 0 on success. */
int cdma_ticket_info(cdma_ctx* ctx, cdma_ticket ticket, uint64_t* payload_bytes, uint64_t* n);

/* Host pointers to a live ticket's payload (payload_bytes long, see
 * cdma_ticket_info) and table inside the pinned pool, e.g. to write an offloaded
 * activation map to storage.  Waits for pending copies into the pool.  The
 * pointers stay valid until the ticket is prefetched or the context destroyed. */
int cdma_ticket_host_view(cdma_ctx* ctx, cdma_ticket ticket, const void** h_payload,
                          const uint64_t** h_table);

/*
 * The same compressed copies for callers whose tensors live in HOST memory.
 * When all three buffers are page-locked (cudaHostAlloc / cudaHostRegister,
 * tensor and payload 16-byte aligned) a single kernel reads the source over
 * the host link and writes the result back over it as it goes -- the software
 * form of the paper's one compressed-copy call (Section V-D), both directions
 * of the link busy at once and no device staging.  Otherwise h_src is copied
 * to the device, processed there and the result copied back.  Both run on the
 * context's side stream, wait for completion and return C / n*s.
 * h_table holds cdma_zvc_table_entries(n) uint64.  On CDMA_ERR_BUFFER_TOO_SMALL
 * the page-locked path may already have written payload bytes below
 * dst_capacity (never beyond it); the staged path leaves h_dst untouched.
 */
int64_t cdma_zvc_compress_host(cdma_ctx* ctx, const void* h_src, uint64_t n, int dtype,
                               int layout, void* h_dst, uint64_t dst_capacity,
                               uint64_t* h_table);
int64_t cdma_zvc_decompress_host(cdma_ctx* ctx, const void* h_src, uint64_t src_bytes,
                                 const uint64_t* h_table, uint64_t n, int dtype, int layout,
                                 void* h_dst);

/* Measurement hook: the next codec kernel this thread launches (compress or
 * decompress, through any entry point) is bracketed by cudaEventRecord of the
 * two given cudaEvent_t handles on the launch stream, around the kernel alone
 * (not the workspace reset or the result copy of the call).  One-shot: the pair
 * is forgotten after that launch.  Pass NULLs to cancel. */
void cdma_time_next_kernel(void* start_event, void* stop_event);

/* Number of kernel launches this library has issued in this process (codec
 * kernels and the copy kernel of cdma_offload_async; copies by the copy engines
 * are not counted). */
uint64_t cdma_kernel_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* CDMA_H_ */
