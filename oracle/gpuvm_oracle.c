/*
 * CPU oracle for GPU-thread-driven demand paging (GPUVM, arXiv 2411.05309).
 *
 * TEST INFRASTRUCTURE ONLY.  Plain, slow C that shares no code with the CUDA path.
 * Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may call
 * it; the product never does.  As the tests build it (no OpenMP) it is
 * single-threaded.  The benchmark's all-core baseline compiles this same file with
 * -fopenmp: the pragmas below then split the outermost loop of four *_direct
 * functions over the host's threads; every element, block or bag is still computed
 * by one thread with the same operations in the same order, so those results are
 * bit-identical to the single-threaded build (a test compares the two).
 *
 * Two parts.
 *
 *  (R) Results.  The paging runtime is a cache in front of host memory
 *      (Section 3.1, Fig. 2: a thread computes page number and offset, consults
 *      the page table, and reads or writes the data in the frame), so what a
 *      workload computes through it equals what the same workload computes
 *      directly on the host arrays.  The *_direct functions are those plain
 *      definitions.
 *
 *  (P) Paging replay.  A sequential model of the runtime's bookkeeping that
 *      takes one access at a time, in program order: address split and
 *      page-table lookup (Fig. 2 steps 1-2), frame ring with a single head
 *      cursor (Section 3.3 "Eviction scheme", Fig. 4), eviction of the frame
 *      under the cursor, write-back of the victim, fetch of the new page.  Two
 *      policies: FIFO, which is the ring of the paper, and clock/second chance,
 *      which adds one reference bit per frame.  A dirty bit per frame decides
 *      whether a victim is copied back.  With move_bytes on, the replay owns a
 *      private frame buffer and every load and store of the paged workloads goes
 *      through it, so lost write-backs show up as wrong host contents.
 *
 * Readings where the paper is silent: a write miss fetches the page first; the
 * newly installed page has its reference bit set; the cursor moves past a frame
 * when that frame is filled; a hit sets the reference bit and, for a write, the
 * dirty bit.
 *
 * Pins (see tests): textbook reference strings with known FIFO and OPT fault
 * counts, a queue-formulated second-chance model, Belady lower bound, compulsory
 * misses, capacity, byte-exact host contents after flush, library BFS.
 */
#include <stdint.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------ (R) -- */

/* Streaming read-reduce: S = sum of a[i] as 64-bit integers. */
int64_t orc_stream_sum_i32_direct(const int32_t *a, uint64_t n)
{
    int64_t s = 0;
#pragma omp parallel for reduction(+ : s) schedule(static)
    for (uint64_t i = 0; i < n; ++i) s += (int64_t)a[i];
    return s;
}

/*
 * Random gather, one sum per block of `block` consecutive indices.
 *   fsum[b] = binary32( sum over the block, accumulated in binary64, index order )
 *   bsum[b] = sum over the block of the raw 32-bit patterns of the gathered
 *             values, taken as unsigned, accumulated in int64 (an exact,
 *             order-free fingerprint of WHICH elements were gathered).
 */
void orc_gather_block_sums_direct(const float *x, const int64_t *idx, uint64_t n_idx,
                                  uint64_t block, float *fsum, int64_t *bsum)
{
    uint64_t nb = (n_idx + block - 1) / block;
#pragma omp parallel for schedule(static)
    for (uint64_t b = 0; b < nb; ++b) {
        double acc = 0.0;
        int64_t bits = 0;
        uint64_t end = (b + 1) * block < n_idx ? (b + 1) * block : n_idx;
        for (uint64_t k = b * block; k < end; ++k) {
            float v = x[idx[k]];
            uint32_t u;
            memcpy(&u, &v, 4);
            acc += (double)v;
            bits += (int64_t)u;
        }
        fsum[b] = (float)acc;
        bsum[b] = bits;
    }
}

/* Hop distance from `source` over a directed CSR graph; -1 when unreachable. */
void orc_bfs_levels_direct(const int64_t *row_off, const int32_t *col, uint64_t nv,
                           uint64_t source, int32_t *level)
{
    for (uint64_t v = 0; v < nv; ++v) level[v] = -1;
    if (source >= nv) return;
    uint64_t *queue = (uint64_t *)malloc(nv * sizeof(uint64_t));
    uint64_t head = 0, tail = 0;
    level[source] = 0;
    queue[tail++] = source;
    while (head < tail) {
        uint64_t u = queue[head++];
        for (int64_t e = row_off[u]; e < row_off[u + 1]; ++e) {
            int32_t v = col[e];
            if (level[v] < 0) {
                level[v] = level[u] + 1;
                queue[tail++] = (uint64_t)v;
            }
        }
    }
    free(queue);
}

/*
 * Weakly connected components (Section 5.2 runs CC on the same graphs): label[v] = the
 * smallest vertex number in the component of v when edges count in both directions.
 * Union-find with the smaller root as the representative.
 */
static uint64_t uf_find(uint64_t *parent, uint64_t v)
{
    while (parent[v] != v) {
        parent[v] = parent[parent[v]];
        v = parent[v];
    }
    return v;
}

void orc_cc_labels_direct(const int64_t *row_off, const int32_t *col, uint64_t nv, int32_t *label)
{
    uint64_t *parent = (uint64_t *)malloc(nv * sizeof(uint64_t));
    for (uint64_t v = 0; v < nv; ++v) parent[v] = v;
    for (uint64_t u = 0; u < nv; ++u)
        for (int64_t e = row_off[u]; e < row_off[u + 1]; ++e) {
            uint64_t a = uf_find(parent, u), b = uf_find(parent, (uint64_t)col[e]);
            if (a < b) parent[b] = a;
            else if (b < a) parent[a] = b;
        }
    for (uint64_t v = 0; v < nv; ++v) label[v] = (int32_t)uf_find(parent, v);
    free(parent);
}

/*
 * Single-source shortest paths with non-negative int32 weights (Section 5.2 runs SSSP with a
 * separate weight array): Dijkstra with a binary heap of (distance, vertex) pairs and lazy
 * deletion.  dist[v] = 0x7FFFFFFF when v cannot be reached.
 */
typedef struct { int64_t d; uint64_t v; } orc_heap_item;

static void heap_push(orc_heap_item *h, uint64_t *n, orc_heap_item it)
{
    uint64_t i = (*n)++;
    while (i > 0 && h[(i - 1) / 2].d > it.d) { h[i] = h[(i - 1) / 2]; i = (i - 1) / 2; }
    h[i] = it;
}

static orc_heap_item heap_pop(orc_heap_item *h, uint64_t *n)
{
    orc_heap_item top = h[0], last = h[--(*n)];
    uint64_t i = 0;
    for (;;) {
        uint64_t c = 2 * i + 1;
        if (c >= *n) break;
        if (c + 1 < *n && h[c + 1].d < h[c].d) ++c;
        if (h[c].d >= last.d) break;
        h[i] = h[c];
        i = c;
    }
    h[i] = last;
    return top;
}

void orc_sssp_direct(const int64_t *row_off, const int32_t *col, const int32_t *weight, uint64_t nv, uint64_t source,
                     int32_t *dist)
{
    const int64_t INF = 0x7FFFFFFF;
    int64_t *d = (int64_t *)malloc(nv * sizeof(int64_t));
    for (uint64_t v = 0; v < nv; ++v) d[v] = INF;
    uint64_t cap = (uint64_t)row_off[nv] + 1, n = 0;
    orc_heap_item *heap = (orc_heap_item *)malloc(cap * sizeof(orc_heap_item));
    d[source] = 0;
    heap_push(heap, &n, (orc_heap_item){0, source});
    while (n) {
        orc_heap_item it = heap_pop(heap, &n);
        if (it.d != d[it.v]) continue;                  /* stale entry */
        for (int64_t e = row_off[it.v]; e < row_off[it.v + 1]; ++e) {
            int64_t nd = it.d + (int64_t)weight[e];
            uint64_t c = (uint64_t)col[e];
            if (nd < d[c]) { d[c] = nd; heap_push(heap, &n, (orc_heap_item){nd, c}); }
        }
    }
    for (uint64_t v = 0; v < nv; ++v) dist[v] = (int32_t)d[v];
    free(heap); free(d);
}

/* c[i] = a[i] + b[i], one correctly rounded binary32 addition per element. */
void orc_vadd_f32_direct(const float *a, const float *b, float *c, uint64_t n)
{
#pragma omp parallel for schedule(static)
    for (uint64_t i = 0; i < n; ++i) {
        volatile float s = a[i] + b[i];
        c[i] = s;
    }
}

/*
 * Embedding bag: out[g][d] = ((0 + t[r0][d]) + t[r1][d]) + ... in binary32, rows
 * of bag g taken in list order (rows[g*bag .. g*bag+bag-1]).
 */
void orc_embag_f32_direct(const float *table, uint64_t dims, const int64_t *rows,
                          uint64_t n_bags, uint64_t bag, float *out)
{
#pragma omp parallel for schedule(static)
    for (uint64_t g = 0; g < n_bags; ++g)
        for (uint64_t d = 0; d < dims; ++d) {
            volatile float acc = 0.0f;
            for (uint64_t k = 0; k < bag; ++k)
                acc = acc + table[(uint64_t)rows[g * bag + k] * dims + d];
            out[g * dims + d] = acc;
        }
}

/* ------------------------------------------------------------------ (P) -- */

enum { ORC_FIFO = 0, ORC_CLOCK = 1 };
#define ORC_NONE UINT64_MAX

typedef struct {
    uint8_t *host;            /* backing store: holds every page (Fig. 4, left)   */
    uint64_t bytes;
    uint64_t page_bytes;
    uint64_t n_pages;         /* ceil(bytes / page_bytes)                          */
    uint64_t n_frames;
    int policy;
    int move_bytes;
    uint64_t *map;            /* page table: page -> frame or ORC_NONE             */
    uint64_t *frame_page;     /* page map of the ring: frame -> page or ORC_NONE   */
    uint8_t *frame_dirty;
    uint8_t *frame_ref;
    uint8_t *frames;          /* private frame buffer (move_bytes only)            */
    uint64_t hand;            /* the ring's head cursor                            */
    /* counters */
    uint64_t accesses, hits, faults, evictions, writebacks;
    uint64_t bytes_in, bytes_out, resident, max_resident, hand_steps;
    /* optional record of the page numbers accessed, runs of one page collapsed to one entry */
    uint64_t *trace;
    uint64_t trace_cap, trace_len, trace_last;
} orc_pager;

static uint64_t page_len(const orc_pager *p, uint64_t vpn)
{
    uint64_t start = vpn * p->page_bytes;
    uint64_t left = p->bytes - start;
    return left < p->page_bytes ? left : p->page_bytes;
}

orc_pager *orc_pager_create(void *host, uint64_t bytes, uint64_t page_bytes,
                            uint64_t n_frames, int policy, int move_bytes)
{
    if (!host || !bytes || !page_bytes || !n_frames) return NULL;
    orc_pager *p = (orc_pager *)calloc(1, sizeof(orc_pager));
    p->host = (uint8_t *)host;
    p->bytes = bytes;
    p->page_bytes = page_bytes;
    p->n_pages = (bytes + page_bytes - 1) / page_bytes;
    p->n_frames = n_frames;
    p->policy = policy;
    p->move_bytes = move_bytes;
    p->map = (uint64_t *)malloc(p->n_pages * sizeof(uint64_t));
    p->frame_page = (uint64_t *)malloc(n_frames * sizeof(uint64_t));
    p->frame_dirty = (uint8_t *)calloc(n_frames, 1);
    p->frame_ref = (uint8_t *)calloc(n_frames, 1);
    for (uint64_t i = 0; i < p->n_pages; ++i) p->map[i] = ORC_NONE;
    for (uint64_t i = 0; i < n_frames; ++i) p->frame_page[i] = ORC_NONE;
    if (move_bytes) p->frames = (uint8_t *)malloc(n_frames * page_bytes);
    p->trace_last = ORC_NONE;
    return p;
}

/*
 * Record the sequence of page numbers that orc_pager_access sees from now on into buf (caller's
 * memory, cap entries).  Consecutive accesses to one page are recorded once: every access of such
 * a run after the first is a hit under any policy and leaves reference and dirty state as the
 * first access of the run left it (for read-only traces), so fault counts of the collapsed trace
 * equal those of the full one.  orc_pager_trace_len returns the number of entries the run would
 * have needed; entries beyond cap are counted but not stored.
 */
void orc_pager_trace(orc_pager *p, uint64_t *buf, uint64_t cap)
{
    p->trace = buf;
    p->trace_cap = cap;
    p->trace_len = 0;
    p->trace_last = ORC_NONE;
}

uint64_t orc_pager_trace_len(const orc_pager *p) { return p->trace_len; }

void orc_pager_destroy(orc_pager *p)
{
    if (!p) return;
    free(p->map); free(p->frame_page); free(p->frame_dirty); free(p->frame_ref);
    free(p->frames); free(p);
}

/* Copy a victim back to the host if it was written, then drop its mapping. */
static void evict_frame(orc_pager *p, uint64_t f)
{
    uint64_t q = p->frame_page[f];
    if (p->frame_dirty[f]) {
        p->writebacks++;
        p->bytes_out += page_len(p, q);
        if (p->move_bytes)
            memcpy(p->host + q * p->page_bytes, p->frames + f * p->page_bytes, page_len(p, q));
    }
    p->evictions++;
    p->map[q] = ORC_NONE;
    p->frame_page[f] = ORC_NONE;
    p->frame_dirty[f] = 0;
    p->frame_ref[f] = 0;
    p->resident--;
}

/* One access in program order.  Returns the frame that now holds the page. */
uint64_t orc_pager_access(orc_pager *p, uint64_t vpn, int is_write)
{
    p->accesses++;
    if (p->trace && vpn != p->trace_last) {
        if (p->trace_len < p->trace_cap) p->trace[p->trace_len] = vpn;
        p->trace_len++;
        p->trace_last = vpn;
    }
    uint64_t f = p->map[vpn];
    if (f != ORC_NONE) {                      /* Fig. 2 step 2: resident */
        p->hits++;
        p->frame_ref[f] = 1;
        if (is_write) p->frame_dirty[f] = 1;
        return f;
    }
    p->faults++;
    for (;;) {                                /* take the next ring slot */
        f = p->hand;
        p->hand = (p->hand + 1) % p->n_frames;
        p->hand_steps++;
        if (p->frame_page[f] == ORC_NONE) break;
        if (p->policy == ORC_CLOCK && p->frame_ref[f]) {
            p->frame_ref[f] = 0;              /* second chance */
            continue;
        }
        evict_frame(p, f);
        break;
    }
    p->bytes_in += page_len(p, vpn);
    if (p->move_bytes)
        memcpy(p->frames + f * p->page_bytes, p->host + vpn * p->page_bytes, page_len(p, vpn));
    p->map[vpn] = f;
    p->frame_page[f] = vpn;
    p->frame_ref[f] = 1;
    p->frame_dirty[f] = is_write ? 1 : 0;
    p->resident++;
    if (p->resident > p->max_resident) p->max_resident = p->resident;
    return f;
}

/* Replay a trace of (page, is_write) records. */
void orc_pager_replay(orc_pager *p, const uint64_t *vpn, const uint8_t *is_write, uint64_t n)
{
    for (uint64_t i = 0; i < n; ++i) orc_pager_access(p, vpn[i], is_write ? is_write[i] : 0);
}

/* Write every dirty frame back; mappings stay. */
void orc_pager_flush(orc_pager *p)
{
    for (uint64_t f = 0; f < p->n_frames; ++f)
        if (p->frame_page[f] != ORC_NONE && p->frame_dirty[f]) {
            uint64_t q = p->frame_page[f];
            p->writebacks++;
            p->bytes_out += page_len(p, q);
            if (p->move_bytes)
                memcpy(p->host + q * p->page_bytes, p->frames + f * p->page_bytes, page_len(p, q));
            p->frame_dirty[f] = 0;
        }
}

/* counters out: accesses, hits, faults, evictions, writebacks, bytes_in,
 * bytes_out, resident, max_resident, hand_steps */
void orc_pager_counters(const orc_pager *p, uint64_t out[10])
{
    out[0] = p->accesses; out[1] = p->hits; out[2] = p->faults; out[3] = p->evictions;
    out[4] = p->writebacks; out[5] = p->bytes_in; out[6] = p->bytes_out;
    out[7] = p->resident; out[8] = p->max_resident; out[9] = p->hand_steps;
}

/* Structural invariants of the replay's tables; 0 when they hold. */
int orc_pager_check(const orc_pager *p)
{
    uint64_t mapped = 0, used = 0;
    for (uint64_t v = 0; v < p->n_pages; ++v)
        if (p->map[v] != ORC_NONE) {
            mapped++;
            if (p->map[v] >= p->n_frames) return 1;
            if (p->frame_page[p->map[v]] != v) return 2;
        }
    for (uint64_t f = 0; f < p->n_frames; ++f)
        if (p->frame_page[f] != ORC_NONE) {
            used++;
            if (p->frame_page[f] >= p->n_pages) return 3;
            if (p->map[p->frame_page[f]] != f) return 4;
        }
    if (mapped != used || mapped != p->resident || mapped > p->n_frames) return 5;
    return 0;
}

/*
 * Test hook for the checker above: overwrite one word of the replay's tables so that a test can
 * see orc_pager_check report each kind of damage.  which: 0 = map[i] (page table), 1 =
 * frame_page[i] (ring), 2 = the resident counter (i ignored).  v = UINT64_MAX means "none".
 */
int orc_pager_debug_poke(orc_pager *p, int which, uint64_t i, uint64_t v)
{
    if (which == 0 && i < p->n_pages) { p->map[i] = v; return 0; }
    if (which == 1 && i < p->n_frames) { p->frame_page[i] = v; return 0; }
    if (which == 2) { p->resident = v; return 0; }
    return -1;
}

/*
 * Belady's optimal replacement (the lower bound of any policy, used next to the FIFO ring of
 * Section 3.3 and the clock variant): number of faults of `trace` with n_frames frames when, on
 * a fault with no free frame, the resident page whose next use lies farthest in the future (or
 * that is never used again) is evicted.  Plain form: next-use positions are computed by one
 * backward pass, the victim is found by a linear scan over the frames.
 */
uint64_t orc_belady_faults(const uint64_t *trace, uint64_t n, uint64_t n_pages, uint64_t n_frames)
{
    const uint64_t NEVER = UINT64_MAX;
    uint64_t *next = (uint64_t *)malloc((n ? n : 1) * sizeof(uint64_t));     /* next[i]: next position of trace[i] */
    uint64_t *last_seen = (uint64_t *)malloc((n_pages ? n_pages : 1) * sizeof(uint64_t));
    uint64_t *where = (uint64_t *)malloc((n_pages ? n_pages : 1) * sizeof(uint64_t)); /* page -> frame or NONE */
    uint64_t *frame_page = (uint64_t *)malloc(n_frames * sizeof(uint64_t));
    uint64_t *frame_next = (uint64_t *)malloc(n_frames * sizeof(uint64_t));
    for (uint64_t v = 0; v < n_pages; ++v) { last_seen[v] = NEVER; where[v] = ORC_NONE; }
    for (uint64_t i = n; i-- > 0;) { next[i] = last_seen[trace[i]]; last_seen[trace[i]] = i; }
    uint64_t used = 0, faults = 0;
    for (uint64_t i = 0; i < n; ++i) {
        uint64_t v = trace[i], f = where[v];
        if (f == ORC_NONE) {
            faults++;
            if (used < n_frames) f = used++;
            else {
                f = 0;
                for (uint64_t g = 1; g < n_frames; ++g)
                    if (frame_next[g] > frame_next[f]) f = g;
                where[frame_page[f]] = ORC_NONE;
            }
            frame_page[f] = v;
            where[v] = f;
        }
        frame_next[f] = next[i];
    }
    free(next); free(last_seen); free(where); free(frame_page); free(frame_next);
    return faults;
}

/* Element accessors through the pager.  An element never straddles a page
 * because page sizes are multiples of the element size and arrays start on page
 * boundaries.  Without move_bytes the data is read/written in place. */
static void paged_load(orc_pager *p, uint64_t byte_off, void *dst, uint64_t n)
{
    uint64_t vpn = byte_off / p->page_bytes, off = byte_off % p->page_bytes;
    uint64_t f = orc_pager_access(p, vpn, 0);
    if (p->move_bytes) memcpy(dst, p->frames + f * p->page_bytes + off, n);
    else memcpy(dst, p->host + byte_off, n);
}

static void paged_store(orc_pager *p, uint64_t byte_off, const void *src, uint64_t n)
{
    uint64_t vpn = byte_off / p->page_bytes, off = byte_off % p->page_bytes;
    uint64_t f = orc_pager_access(p, vpn, 1);
    if (p->move_bytes) memcpy(p->frames + f * p->page_bytes + off, src, n);
    else memcpy(p->host + byte_off, src, n);
}

/* The five workloads, element by element in canonical program order, every
 * paged operand going through the pager.  Offsets are byte offsets of the arrays
 * inside the backing store. */

int64_t orc_stream_sum_i32_paged(orc_pager *p, uint64_t a_off, uint64_t n)
{
    int64_t s = 0;
    for (uint64_t i = 0; i < n; ++i) {
        int32_t v;
        paged_load(p, a_off + 4 * i, &v, 4);
        s += (int64_t)v;
    }
    return s;
}

void orc_gather_block_sums_paged(orc_pager *p, uint64_t x_off, const int64_t *idx,
                                 uint64_t n_idx, uint64_t block, float *fsum, int64_t *bsum)
{
    uint64_t nb = (n_idx + block - 1) / block;
    for (uint64_t b = 0; b < nb; ++b) {
        double acc = 0.0;
        int64_t bits = 0;
        uint64_t end = (b + 1) * block < n_idx ? (b + 1) * block : n_idx;
        for (uint64_t k = b * block; k < end; ++k) {
            float v;
            uint32_t u;
            paged_load(p, x_off + 4 * (uint64_t)idx[k], &v, 4);
            memcpy(&u, &v, 4);
            acc += (double)v;
            bits += (int64_t)u;
        }
        fsum[b] = (float)acc;
        bsum[b] = bits;
    }
}

/* Level-synchronous BFS: level by level, vertices ascending inside a level; per
 * vertex row_off[v], row_off[v+1], then its edge range ascending.  The level
 * array is ordinary (unpaged) memory. */
void orc_bfs_levels_paged(orc_pager *p, uint64_t off_off, uint64_t col_off, uint64_t nv,
                          uint64_t source, int32_t *level)
{
    for (uint64_t v = 0; v < nv; ++v) level[v] = -1;
    if (source >= nv) return;
    level[source] = 0;
    for (int32_t cur = 0;; ++cur) {
        int found = 0;
        for (uint64_t u = 0; u < nv; ++u) {
            if (level[u] != cur) continue;
            int64_t lo, hi;
            paged_load(p, off_off + 8 * u, &lo, 8);
            paged_load(p, off_off + 8 * (u + 1), &hi, 8);
            for (int64_t e = lo; e < hi; ++e) {
                int32_t v;
                paged_load(p, col_off + 4 * (uint64_t)e, &v, 4);
                if (level[v] < 0) { level[v] = cur + 1; found = 1; }
            }
        }
        if (!found) break;
    }
}

void orc_vadd_f32_paged(orc_pager *p, uint64_t a_off, uint64_t b_off, uint64_t c_off, uint64_t n)
{
    for (uint64_t i = 0; i < n; ++i) {
        float a, b;
        paged_load(p, a_off + 4 * i, &a, 4);
        paged_load(p, b_off + 4 * i, &b, 4);
        volatile float s = a + b;
        float c = s;
        paged_store(p, c_off + 4 * i, &c, 4);
    }
}

void orc_embag_f32_paged(orc_pager *p, uint64_t t_off, uint64_t dims, const int64_t *rows,
                         uint64_t n_bags, uint64_t bag, float *out)
{
    for (uint64_t g = 0; g < n_bags; ++g) {
        for (uint64_t d = 0; d < dims; ++d) out[g * dims + d] = 0.0f;
        for (uint64_t k = 0; k < bag; ++k) {
            uint64_t r = (uint64_t)rows[g * bag + k];
            for (uint64_t d = 0; d < dims; ++d) {
                float v;
                paged_load(p, t_off + 4 * (r * dims + d), &v, 4);
                volatile float s = out[g * dims + d] + v;
                out[g * dims + d] = s;
            }
        }
    }
}

/* Threads the *_direct loops above run on in this build (1 without OpenMP). */
#ifdef _OPENMP
#include <omp.h>
int orc_threads(void) { return omp_get_max_threads(); }
#else
int orc_threads(void) { return 1; }
#endif

/* Oversubscription level, Eq. 1: workload size / available GPU memory - 1. */
double orc_oversubscription_level(double workload_bytes, double gpu_bytes)
{
    return workload_bytes / gpu_bytes - 1.0;
}

/* Queue depth by Little's law as used in Section 3.2: latency x throughput /
 * request size, all in binary units. */
double orc_queue_depth(double latency_s, double bytes_per_s, double request_bytes)
{
    return latency_s * bytes_per_s / request_bytes;
}
