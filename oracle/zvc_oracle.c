/*
 * zvc_oracle.c -- plain, slow, byte-at-a-time CPU statement of zero-value
 * compression (ZVC).
 *
 * TEST INFRASTRUCTURE.  This file is the checker the CUDA library is compared
 * against and the timed CPU baseline.  Only the tests, the smoke check and the
 * benchmark's CPU-baseline leg may call it.  It shares no code, header, table
 * or helper with the CUDA path and must never be linked into it.
 *
 * What it states (paper Section V-A, "Zero-value compression", and the
 * decompression engine of Section V-B, Fig. 10b):
 *
 *   - The input is n elements of s bytes each (s = 4, 2 or 1), in memory order.
 *   - Elements are grouped into windows of 32 consecutive elements.  For each
 *     window a 32-bit mask is produced: bit i is 1 when element i of the
 *     window is non-zero, 0 when it is zero.  "Zero" means every byte of the
 *     element is 0x00 (the engine compares words to zero), so -0.0, NaN,
 *     denormals and infinities count as non-zero and survive unchanged.
 *   - After the mask, the window's non-zero elements are appended, in
 *     ascending element order.
 *   - The compressed stream is the concatenation of those records.  Since the
 *     population count of a mask tells how many values follow it, the
 *     position of the next mask is known from the stream alone.
 *
 * Readings where the paper is silent:
 * bit i (least significant = 0) belongs to element i of the window; the mask
 * is stored least-significant byte first; a short last window has zero bits
 * for the missing elements and no values for them; for 2-byte and 1-byte
 * elements the window is still 32 elements and the mask 32 bits, with no
 * padding (the paper's engine is 32-bit only, Section V-B), so the stream of n
 * elements with nnz non-zero ones is always 4*ceil(n/32) + s*nnz bytes.
 *
 * Framing for parallel decoders (ours, outside the payload): a table of
 * ceil(n/1024)+1 byte offsets, entry k being where the record of window 32k
 * starts, the last entry being the payload size.  1024 fp32 elements are the
 * 4 KB block the paper's compression study uses (Fig. 11 caption).
 *
 * Every function returns a non-negative byte count or a negative error:
 *   -1 bad argument, -5 destination too small, -6 malformed stream.
 */
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <pthread.h>

#define ORACLE_WINDOW 32u          /* elements per mask (Section V-A)          */
#define ORACLE_CHUNK_WINDOWS 32u   /* windows per table entry: 1024 elements   */

static int element_is_nonzero(const unsigned char *e, unsigned s)
{
    unsigned b;
    for (b = 0; b < s; ++b)
        if (e[b] != 0) return 1;
    return 0;
}

/* Size of the stream for n elements of which nnz are non-zero:
 * one 4-byte mask per window plus s bytes per non-zero element. */
uint64_t zvc_oracle_closed_form_bytes(uint64_t n, uint64_t nnz, unsigned s)
{
    uint64_t windows = (n + ORACLE_WINDOW - 1) / ORACLE_WINDOW;
    return 4 * windows + (uint64_t)s * nnz;
}

uint64_t zvc_oracle_table_entries(uint64_t n)
{
    uint64_t chunk = (uint64_t)ORACLE_WINDOW * ORACLE_CHUNK_WINDOWS;
    return (n + chunk - 1) / chunk + 1;
}

/*
 * Compress windows [w_begin, w_end) of the tensor, writing records starting at
 * dst[pos].  table may be NULL.  Returns the position after the last record.
 * A position beyond cap is still counted (so the caller learns the size) but
 * nothing is written past cap; *overflow is set in that case.
 */
static uint64_t compress_windows(const unsigned char *src, uint64_t n, unsigned s,
                                 uint64_t w_begin, uint64_t w_end,
                                 unsigned char *dst, uint64_t cap, uint64_t pos,
                                 uint64_t *table, int *overflow)
{
    uint64_t w;
    for (w = w_begin; w < w_end; ++w) {
        uint32_t mask = 0;
        unsigned i;
        uint64_t first = w * ORACLE_WINDOW;
        uint64_t p;

        if (table != NULL && (w % ORACLE_CHUNK_WINDOWS) == 0)
            table[w / ORACLE_CHUNK_WINDOWS] = pos;

        /* 1. the mask: one bit per element, 1 = non-zero */
        for (i = 0; i < ORACLE_WINDOW; ++i) {
            uint64_t j = first + i;
            if (j < n && element_is_nonzero(src + j * s, s))
                mask |= (uint32_t)1 << i;
        }
        /* 2. the mask goes first, least-significant byte first */
        p = pos;
        for (i = 0; i < 4; ++i) {
            if (p < cap) dst[p] = (unsigned char)((mask >> (8 * i)) & 0xffu);
            else *overflow = 1;
            ++p;
        }
        /* 3. then the non-zero elements, in ascending order, bytes verbatim */
        for (i = 0; i < ORACLE_WINDOW; ++i) {
            if ((mask >> i) & 1u) {
                uint64_t j = first + i;
                unsigned b;
                for (b = 0; b < s; ++b) {
                    if (p < cap) dst[p] = src[j * s + b];
                    else *overflow = 1;
                    ++p;
                }
            }
        }
        pos = p;
    }
    return pos;
}

/*
 * Whole-tensor compression, one thread, in stream order.
 * table must hold zvc_oracle_table_entries(n) values (or be NULL).
 */
int64_t zvc_oracle_compress(const void *src, uint64_t n, unsigned s,
                            void *dst, uint64_t cap, uint64_t *table)
{
    uint64_t windows, end;
    int overflow = 0;
    if (s != 1 && s != 2 && s != 4) return -1;
    if (n != 0 && src == NULL) return -1;
    if (cap != 0 && dst == NULL) return -1;
    windows = (n + ORACLE_WINDOW - 1) / ORACLE_WINDOW;
    end = compress_windows((const unsigned char *)src, n, s, 0, windows,
                           (unsigned char *)dst, cap, 0, table, &overflow);
    if (table != NULL) table[zvc_oracle_table_entries(n) - 1] = end;
    if (overflow) return -5;
    return (int64_t)end;
}

/*
 * Decompression: walk the stream from its first byte.  Read a mask, count its
 * ones to learn how many values follow, place each value (or s zero bytes) in
 * the window, move on to the next mask.  The offset table is NOT consulted.
 * Fails (-6) when the walk leaves the stream, does not end exactly at
 * src_bytes, or a mask claims an element at an index >= n.
 */
int64_t zvc_oracle_decompress(const void *src, uint64_t src_bytes, uint64_t n,
                              unsigned s, void *dst)
{
    const unsigned char *in = (const unsigned char *)src;
    unsigned char *out = (unsigned char *)dst;
    uint64_t windows, w, pos = 0;
    if (s != 1 && s != 2 && s != 4) return -1;
    if (n != 0 && dst == NULL) return -1;
    if (src_bytes != 0 && src == NULL) return -1;
    windows = (n + ORACLE_WINDOW - 1) / ORACLE_WINDOW;
    for (w = 0; w < windows; ++w) {
        uint32_t mask = 0;
        unsigned i;
        if (pos + 4 > src_bytes) return -6;
        for (i = 0; i < 4; ++i)
            mask |= (uint32_t)in[pos + i] << (8 * i);
        pos += 4;
        for (i = 0; i < ORACLE_WINDOW; ++i) {
            uint64_t j = w * ORACLE_WINDOW + i;
            unsigned b;
            if ((mask >> i) & 1u) {
                if (j >= n) return -6;
                if (pos + s > src_bytes) return -6;
                for (b = 0; b < s; ++b) out[j * s + b] = in[pos + b];
                pos += s;
            } else if (j < n) {
                for (b = 0; b < s; ++b) out[j * s + b] = 0;
            }
        }
    }
    if (pos != src_bytes) return -6;
    return (int64_t)(n * s);
}

/*
 * Check an offset table against the stream by walking the stream serially:
 * entry k must be the position at which window 32k's mask is met, and the last
 * entry must be the stream's size.  Returns 0 when it matches, -6 otherwise.
 */
int zvc_oracle_check_table(const void *src, uint64_t src_bytes, uint64_t n,
                           unsigned s, const uint64_t *table)
{
    const unsigned char *in = (const unsigned char *)src;
    uint64_t windows, w, pos = 0;
    if (s != 1 && s != 2 && s != 4) return -1;
    if (table == NULL) return -1;
    windows = (n + ORACLE_WINDOW - 1) / ORACLE_WINDOW;
    for (w = 0; w < windows; ++w) {
        uint32_t mask = 0;
        unsigned i, ones = 0;
        if ((w % ORACLE_CHUNK_WINDOWS) == 0 && table[w / ORACLE_CHUNK_WINDOWS] != pos)
            return -6;
        if (pos + 4 > src_bytes) return -6;
        for (i = 0; i < 4; ++i)
            mask |= (uint32_t)in[pos + i] << (8 * i);
        for (i = 0; i < 32; ++i) ones += (mask >> i) & 1u;
        pos += 4 + (uint64_t)s * ones;
    }
    if (pos != src_bytes) return -6;
    if (table[zvc_oracle_table_entries(n) - 1] != src_bytes) return -6;
    return 0;
}

/* ------------------------------------------------------------------------- *
 * Multi-core drivers for the timed CPU baseline.  They add no arithmetic of
 * their own: each thread runs the routines above on a contiguous range of
 * 1024-element chunks.  Compression first sizes every range (same routine,
 * writing nowhere), adds the sizes up, then runs again at the right offsets.
 * ------------------------------------------------------------------------- */
typedef struct {
    const unsigned char *src;
    unsigned char *dst;
    uint64_t n, cap, w_begin, w_end, pos, end;
    uint64_t *table;
    unsigned s;
    int overflow;
    int sizing;
} mt_job;

static void *mt_compress_worker(void *arg)
{
    mt_job *j = (mt_job *)arg;
    if (j->sizing) {
        int ignored = 0;
        j->end = compress_windows(j->src, j->n, j->s, j->w_begin, j->w_end,
                                  NULL, 0, 0, NULL, &ignored);
    } else {
        j->end = compress_windows(j->src, j->n, j->s, j->w_begin, j->w_end,
                                  j->dst, j->cap, j->pos, j->table, &j->overflow);
    }
    return NULL;
}

int64_t zvc_oracle_compress_mt(const void *src, uint64_t n, unsigned s,
                               void *dst, uint64_t cap, uint64_t *table,
                               unsigned threads)
{
    uint64_t windows, chunks, per, pos;
    unsigned t, used;
    int pass, overflow = 0;
    mt_job *jobs;
    pthread_t *tids;
    if (s != 1 && s != 2 && s != 4) return -1;
    if (threads == 0) return -1;
    windows = (n + ORACLE_WINDOW - 1) / ORACLE_WINDOW;
    chunks = (windows + ORACLE_CHUNK_WINDOWS - 1) / ORACLE_CHUNK_WINDOWS;
    if (chunks == 0) return zvc_oracle_compress(src, n, s, dst, cap, table);
    if (threads > chunks) threads = (unsigned)chunks;
    per = (chunks + threads - 1) / threads;
    jobs = (mt_job *)calloc(threads, sizeof(mt_job));
    tids = (pthread_t *)calloc(threads, sizeof(pthread_t));
    if (jobs == NULL || tids == NULL) { free(jobs); free(tids); return -1; }
    used = 0;
    for (t = 0; t < threads; ++t) {
        uint64_t c0 = (uint64_t)t * per, c1 = c0 + per;
        if (c0 >= chunks) break;
        if (c1 > chunks) c1 = chunks;
        jobs[t].src = (const unsigned char *)src;
        jobs[t].dst = (unsigned char *)dst;
        jobs[t].n = n; jobs[t].s = s; jobs[t].cap = cap; jobs[t].table = table;
        jobs[t].w_begin = c0 * ORACLE_CHUNK_WINDOWS;
        jobs[t].w_end = c1 * ORACLE_CHUNK_WINDOWS;
        if (jobs[t].w_end > windows) jobs[t].w_end = windows;
        ++used;
    }
    for (pass = 0; pass < 2; ++pass) {
        for (t = 0; t < used; ++t) {
            jobs[t].sizing = (pass == 0);
            pthread_create(&tids[t], NULL, mt_compress_worker, &jobs[t]);
        }
        for (t = 0; t < used; ++t) pthread_join(tids[t], NULL);
        if (pass == 0) {
            pos = 0;
            for (t = 0; t < used; ++t) { jobs[t].pos = pos; pos += jobs[t].end; }
        }
    }
    pos = jobs[used - 1].end;
    for (t = 0; t < used; ++t) overflow |= jobs[t].overflow;
    if (table != NULL) table[zvc_oracle_table_entries(n) - 1] = pos;
    free(jobs); free(tids);
    if (overflow) return -5;
    return (int64_t)pos;
}

typedef struct {
    const unsigned char *src;
    unsigned char *dst;
    uint64_t n_part, bytes_part;
    unsigned s;
    int64_t result;
} mt_djob;

static void *mt_decompress_worker(void *arg)
{
    mt_djob *j = (mt_djob *)arg;
    j->result = zvc_oracle_decompress(j->src, j->bytes_part, j->n_part, j->s, j->dst);
    return NULL;
}

/* Each thread decodes a contiguous range of chunks as a stream of its own,
 * found through the offset table. */
int64_t zvc_oracle_decompress_mt(const void *src, uint64_t src_bytes,
                                 const uint64_t *table, uint64_t n, unsigned s,
                                 void *dst, unsigned threads)
{
    uint64_t chunk = (uint64_t)ORACLE_WINDOW * ORACLE_CHUNK_WINDOWS;
    uint64_t chunks, per;
    unsigned t, used = 0;
    int bad = 0;
    mt_djob *jobs;
    pthread_t *tids;
    if (s != 1 && s != 2 && s != 4) return -1;
    if (threads == 0 || table == NULL) return -1;
    chunks = (n + chunk - 1) / chunk;
    if (chunks == 0) return zvc_oracle_decompress(src, src_bytes, n, s, dst);
    if (table[chunks] != src_bytes) return -6;
    if (threads > chunks) threads = (unsigned)chunks;
    per = (chunks + threads - 1) / threads;
    jobs = (mt_djob *)calloc(threads, sizeof(mt_djob));
    tids = (pthread_t *)calloc(threads, sizeof(pthread_t));
    if (jobs == NULL || tids == NULL) { free(jobs); free(tids); return -1; }
    for (t = 0; t < threads; ++t) {
        uint64_t c0 = (uint64_t)t * per, c1 = c0 + per, e0, e1;
        if (c0 >= chunks) break;
        if (c1 > chunks) c1 = chunks;
        if (table[c0] > table[c1] || table[c1] > src_bytes) { bad = 1; break; }
        e0 = c0 * chunk; e1 = c1 * chunk; if (e1 > n) e1 = n;
        jobs[t].src = (const unsigned char *)src + table[c0];
        jobs[t].bytes_part = table[c1] - table[c0];
        jobs[t].dst = (unsigned char *)dst + e0 * s;
        jobs[t].n_part = e1 - e0;
        jobs[t].s = s;
        ++used;
    }
    if (!bad) {
        for (t = 0; t < used; ++t)
            pthread_create(&tids[t], NULL, mt_decompress_worker, &jobs[t]);
        for (t = 0; t < used; ++t) pthread_join(tids[t], NULL);
        for (t = 0; t < used; ++t) if (jobs[t].result < 0) bad = 1;
    }
    free(jobs); free(tids);
    if (bad) return -6;
    return (int64_t)(n * s);
}
