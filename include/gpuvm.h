/*
 * gpuvm.h -- host C ABI of the GPU-thread-driven demand-paging runtime.
 *
 * The runtime keeps a large array in host memory ("backing store", the paper's
 * host region that holds every page, Section 3.3 / Fig. 4) and lets GPU threads
 * access it through a fixed pool of page frames in device memory.  All memory
 * is set up before any kernel runs (Section 3.3: no OS work at run time;
 * Section 4 "Constructing Virtual Memory"); page table, frame ring and counters
 * live in device memory and are modified only by GPU threads (Section 3.3 "Page
 * mapping").  The paper moves pages with an RDMA NIC; here the same GPU threads
 * copy pages between the pool and pinned, mapped host memory.
 *
 * Conventions
 *   - every function returns 0 on success or a negative gpuvm_status; nothing
 *     throws, aborts or traps.  gpuvm_strerror() names a status; the last CUDA
 *     error seen by a handle is kept in gpuvm_last_cuda_error().
 *   - "device pointer" means an address valid in kernels on the current CUDA
 *     device; "host pointer" an address valid on the CPU.
 *   - streams are passed as void* (a cudaStream_t; NULL is the default stream).
 *   - a handle belongs to the CUDA device that was current in gpuvm_create().
 *   - there is no CPU fallback: without a CUDA device every call fails.
 */
#ifndef GPUVM_H
#define GPUVM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct gpuvm_handle *gpuvm_t;

typedef enum gpuvm_status {
    GPUVM_OK = 0,
    GPUVM_E_ARG = -1,        /* NULL out pointer, zero size, bad handle               */
    GPUVM_E_PAGE = -2,       /* page_bytes not a power of two in [16, 2^30], or more
                                than 2^31-2 pages                                     */
    GPUVM_E_POOL = -3,       /* pool_bytes zero, not a multiple of page_bytes, or
                                more than 2^31-2 frames                               */
    GPUVM_E_ALIGN = -4,      /* host_backing not 16-byte aligned or bytes % 16 != 0   */
    GPUVM_E_PIN = -5,        /* pinning / mapping the host backing failed             */
    GPUVM_E_ALLOC = -6,      /* device allocation failed                              */
    GPUVM_E_CUDA = -7,       /* any other CUDA runtime failure                        */
    GPUVM_E_TIMEOUT = -8,    /* a device-side wait ran out (sticky, see gpuvm_stats)  */
    GPUVM_E_RANGE = -9,      /* a device accessor was given an offset past the end    */
    GPUVM_E_INVARIANT = -10, /* gpuvm_check found a broken page-table invariant       */
    GPUVM_E_NODEVICE = -11,  /* no CUDA device                                        */
    GPUVM_E_PINS = -12,      /* more than 2^23 simultaneous references to one page
                                (sticky): the request was refused before the 24-bit
                                reference counter could carry into the frame field    */
    GPUVM_E_FRAMES = -13     /* the pool has too few frames for the pages this
                                workload holds pinned at once (see gpuvm_safe_warps)  */
} gpuvm_status;

/* Eviction policy of the frame ring (Section 3.3 "Eviction scheme").
 * FIFO is the paper's ring: the frame under the head cursor is the victim.
 * CLOCK adds one reference bit per page: a referenced page is passed over once.
 * Under both, a page whose reference counter is not zero is never evicted. */
enum { GPUVM_POLICY_FIFO = 0, GPUVM_POLICY_CLOCK = 1 };

/*
 * Device view: a plain struct passed BY VALUE to kernels (the role of the
 * paper's array-like gpuvm<T> object of Listing 1).  All pointers are device
 * pointers; `host` is the device-visible address of the backing store.
 */
typedef struct gpuvm_dev {
    unsigned long long *pte;   /* page table, one 64-bit entry per page                 */
    unsigned int *frame_vpn;   /* frame ring: page held by each frame                   */
    unsigned char *pool;       /* n_frames * page_bytes of device memory                */
    unsigned char *host;       /* backing store (pinned host memory, mapped)            */
    unsigned long long *ctl;   /* head cursor, sticky error, counters                   */
    unsigned long long bytes;  /* size of the backing store                             */
    unsigned long long n_pages;
    unsigned int n_frames;
    unsigned int page_shift;   /* log2(page_bytes)                                      */
    unsigned int policy;       /* GPUVM_POLICY_*                                        */
    unsigned int spin_limit_us;/* upper bound of every device-side wait                 */
    unsigned int debug;        /* GPUVM_DEBUG_* flags                                   */
    unsigned int clean_ahead;  /* ring positions the cleaners may run ahead of the head
                                  cursor; 0: write-back only on the fault path          */
} gpuvm_dev_t;

/* Debug flags (gpuvm_set_debug).  POISON: whoever evicts a page fills its frame with the
 * byte pattern 0xA5 before the frame is handed on, so that a thread that still reads the
 * frame of a page it no longer holds sees the pattern instead of plausible old data (a
 * stale read then shows up as a wrong result in any parity check; the race checker of the
 * CUDA tools is not needed to see it).  Costs one extra write of the frame per eviction. */
/* FENCED_RELEASE: the batched engine releases the pages of read-only requests after a warp barrier and
 * a device fence (the form the PTX memory model orders by itself) instead of making the release depend
 * on the loaded values (the default, which leans on the hardware issuing an instruction only when its
 * operands exist).  Same results; a few per cent slower scans.  For cross-checking the default. */
enum { GPUVM_DEBUG_POISON = 1, GPUVM_DEBUG_FENCED_RELEASE = 2 };

/* Counters accumulated by GPU threads since the last gpuvm_reset(). */
typedef struct gpuvm_stats {
    uint64_t faults;          /* pages migrated host -> pool (one per serviced fault)  */
    uint64_t hits;            /* warp-level page requests that found the page resident */
    uint64_t waits;           /* warp-level requests that joined a fault in flight
                                 (inter-warp coalescing, Section 3.3)                  */
    uint64_t lanes_coalesced; /* threads that shared their warp leader's request
                                 (intra-warp coalescing)                               */
    uint64_t evictions;       /* pages unmapped to make room                           */
    uint64_t writebacks;      /* dirty victims copied pool -> host by the warp that
                                 needed their frame (on the fault path)               */
    uint64_t flush_writebacks;/* dirty pages copied by gpuvm_flush                     */
    uint64_t bytes_in;        /* host -> pool bytes                                    */
    uint64_t bytes_out;       /* pool -> host bytes (evictions + flush)                */
    uint64_t hand_steps;      /* frame-ring slots inspected                            */
    uint64_t retries;         /* wait-loop rounds that made no progress                */
    uint64_t resident;        /* pages resident now                                    */
    uint64_t cleaned;         /* dirty pages written back off the fault path, by idle
                                 warps, while they stayed resident                    */
    uint64_t bytes_direct;    /* bytes that kernels read in place from the backing store
                                 instead of fetching their page (sparse accesses of the
                                 graph sweeps to pages that are not resident)          */
    uint64_t ring_drops;      /* entries of a fault ring that were given up on after a
                                 bounded wait (slot never filled, slot never cleared, or
                                 a popped page that was not waiting for a migrator): each
                                 also sets the sticky GPUVM_E_TIMEOUT; 0 in a healthy run */
    int32_t error;            /* sticky device error: 0, GPUVM_E_TIMEOUT, _RANGE, _PINS */
    uint32_t reserved;
    uint64_t error_page;      /* page number the first error was raised for            */
} gpuvm_stats_t;

/* Result of the post-run invariant check. */
typedef struct gpuvm_check {
    uint64_t resident;        /* page-table entries in the VALID state                 */
    uint64_t frames_used;     /* frames that name a page                               */
    uint64_t bad_state;       /* entries left BUSY / EVICTING, or INVALID with stray bits */
    uint64_t bad_refcount;    /* entries whose reference counter is not zero           */
    uint64_t bad_backref;     /* VALID entry whose frame does not name it back, or a
                                 frame whose page is not VALID in that frame           */
    uint64_t bad_range;       /* frame number or page number out of range              */
    uint64_t dirty;           /* resident pages still marked dirty                     */
} gpuvm_check_t;

/*
 * Create a paged view of `bytes` bytes of host memory with pages of `page_bytes`
 * and a device pool of `pool_bytes` (Section 4 "Constructing Virtual Memory";
 * Section 3.3: GPU memory is a fixed ring of page frames).
 *   out          host pointer, receives the handle.
 *   host_backing host pointer, 16-byte aligned, owned by the caller and kept alive
 *                until gpuvm_destroy.  Pageable memory is pinned and mapped by the
 *                library (and unpinned at destroy); memory that is already pinned
 *                is used as is.  NULL: the library allocates pinned memory itself
 *                (see gpuvm_host_ptr) and frees it at destroy.
 *   bytes        multiple of 16.  The last page may be partial.
 *   page_bytes   power of two, 16 .. 2^30.
 *   pool_bytes   multiple of page_bytes, at least one page.
 * Allocates page table, frame ring, counters and the pool with cudaMalloc and
 * zeroes them.  Errors: GPUVM_E_ARG/PAGE/POOL/ALIGN are detected before any
 * CUDA call; GPUVM_E_PIN, GPUVM_E_ALLOC, GPUVM_E_NODEVICE.
 */
int gpuvm_create(gpuvm_t *out, void *host_backing, size_t bytes, size_t page_bytes,
                 size_t pool_bytes);

/* Flush dirty pages to the host, release device memory, unpin what create
 * pinned, free what create allocated.  The handle is dead afterwards. */
int gpuvm_destroy(gpuvm_t h);

/* Synchronise the device and copy the counters to *out (host pointer).  Returns
 * the sticky device error if one is set, else 0. */
int gpuvm_stats(gpuvm_t h, gpuvm_stats_t *out);

/* The same on a stream of the caller's choice: only `stream` is synchronised (not the
 * device), so a handle can be read out while other streams keep working. */
int gpuvm_stats_on(gpuvm_t h, gpuvm_stats_t *out, void *stream);

/* Copy the by-value device view to *out (host pointer). */
int gpuvm_device_view(gpuvm_t h, gpuvm_dev_t *out);

/* Host pointer of the backing store (the caller's, or the library's own). */
void *gpuvm_host_ptr(gpuvm_t h);

/* Write every dirty resident page back to the host on `stream` and clear the
 * dirty bits; mappings stay.  Synchronises the stream before returning, so the
 * host array is complete ("no dirty data is lost").  Must not run concurrently
 * with kernels that use the handle. */
int gpuvm_flush(gpuvm_t h, void *stream);

/* Forget all mappings (without write-back), zero the counters and the error.
 * Mappings otherwise persist across kernel launches (Section 4 "Multi-kernel
 * support"). */
int gpuvm_reset(gpuvm_t h);

/* gpuvm_reset enqueued on `stream` without any synchronisation: the three clears are
 * ordered after earlier work on that stream and before later work on it. */
int gpuvm_reset_on(gpuvm_t h, void *stream);

/* Run the invariant kernel: every resident page maps to exactly one frame and
 * that frame names it back, occupancy <= capacity, nothing left in a transient
 * state, all reference counters zero.  Fills *out (host pointer); returns
 * GPUVM_E_INVARIANT if any bad_* count is non-zero. */
int gpuvm_check(gpuvm_t h, gpuvm_check_t *out);

/* gpuvm_check on `stream`; synchronises that stream only. */
int gpuvm_check_on(gpuvm_t h, gpuvm_check_t *out, void *stream);

/* Options.  policy: GPUVM_POLICY_*; spin_limit_us: bound of device-side waits
 * (default 10 s).  Take effect for views fetched afterwards. */
int gpuvm_set_policy(gpuvm_t h, int policy);
int gpuvm_set_spin_limit_us(gpuvm_t h, unsigned int spin_limit_us);
int gpuvm_set_debug(gpuvm_t h, unsigned int flags);   /* GPUVM_DEBUG_*; 0 = off (default) */

/* Write-back off the fault path (Section 5.3 names synchronous write-back as the method's weak spot):
 * warps with nothing to do write back dirty pages that lie up to `frames` ring positions ahead of the
 * head cursor and would be its victims, so that the warp that takes the frame does not have to.  The
 * order of eviction is unchanged.  What it costs: a page that is written to again between its early
 * write-back and its eviction is written back twice.  Off by default (frames = 0): with thousands of
 * warps faulting at once, the write-backs of some overlap the fetches of others and both directions
 * of the link are busy anyway; measured on scattered updates over a thrashing pool it moved two thirds
 * of the write-backs off the fault path and made the run no faster (requesters migrate their own
 * pages) or slower by half (migrator warps: the extra write-backs take link time from the fetches).
 * A setting for workloads whose dirty pages are written once and whose faulting warps are few. */
int gpuvm_set_clean_ahead(gpuvm_t h, unsigned int frames);

/* Device scratch of the batched workload entry points (request tables, staging of gathered
 * rows; not pages of the backing store).  It belongs to the handle, is allocated at the first
 * call that needs it and grown on demand.  More scratch lets a kernel keep more page requests
 * registered at once, and so lets one migrated page serve more of them (the counterpart of the
 * paper's deeper queues, Section 3.2): gpuvm_set_scratch_limit bounds it (bytes; 0 = no bound,
 * the default), the workloads then choose the deepest batch that fits and never less than their
 * smallest one.  gpuvm_scratch_bytes returns what is allocated now. */
int gpuvm_set_scratch_limit(gpuvm_t h, size_t bytes);
size_t gpuvm_scratch_bytes(gpuvm_t h);

/* Advice: the pages that hold [byte_off, byte_off + bytes) are not to be evicted (keep != 0), or may be again
 * (keep == 0).  A kept page is fetched when it is first touched, like any other, and then stays in its frame
 * whatever the pressure on the pool; the evictor passes over it.  For small arrays that every part of a workload
 * comes back to (the row offsets of a graph beside its edge arrays).  At most half the pool's frames may be kept
 * (GPUVM_E_FRAMES beyond that; GPUVM_E_RANGE outside the backing store); the advice survives gpuvm_reset and is
 * dropped with the handle.  Synchronises the device. */
int gpuvm_advise_keep(gpuvm_t h, size_t byte_off, size_t bytes, int keep);

/* Reading rows in place instead of fetching their page (not in the paper, which fetches a page at its first
 * fault).  The batched row workloads (gpuvm_embag_f32) do not fetch a page for a few rows: pinned host memory is as
 * reachable for a load as for a page copy, so rows of pages with few lookups are read in place from the backing
 * store and the page stays where it is.  A page is worth fetching when its lookups would otherwise move at least
 * page_bytes / divisor over the link; limit = page_bytes / divisor / max(row_bytes, 128) lookups.  Rows read in
 * place are counted in gpuvm_stats as bytes_direct.  Only for reads, and only right for data that is not written
 * through the runtime while such a kernel runs.
 * divisor: 0 = off (every first touch fetches the page, as in the paper); GPUVM_INPLACE_AUTO (default) = 1 when
 * the rows read in place can be read page by page (see below), else 4.  Why: sequential reads over the link run
 * at 51.4 GB/s, and so do rows read page by page, so the break-even point is the page's own size; rows read one
 * lookup after the other are scattered over the table, and scattered reads over a 64 GiB pinned region were
 * measured at 24.5 GB/s however many were in flight (51.4 over 1 GiB, 33.4 over 8 GiB: address translation on the
 * host side), beside page copies at the full rate: the two streams finish together near a quarter of a page
 * (measured on the 64 GiB Zipf table, scattered: 70 / 61 / 77 ms for the divisors 2 / 4 / 8). */
#define GPUVM_INPLACE_AUTO 0xFFFFFFFFu
int gpuvm_set_inplace_divisor(gpuvm_t h, unsigned int divisor);

/* How the batched row workloads find the pages that are worth fetching.
 * counted = 1: a short kernel first counts, per page, the lookups of the whole list (the list is the kernel's
 * input, so the demand is known before the first access); rows of pages below the limit are read in place
 * without the page table being touched, as their lookups come up, and every other page is fetched at its first
 * touch: no row of a page that will be fetched anyway is read in place first.
 * counted = 2 (default): the same, and when every lookup has a staging slot of its own (all bags in flight at once:
 * the default without gpuvm_set_scratch_limit) the lookups of the pages that are not fetched are bucketed by page
 * and their rows read page by page, at the link's sequential rate; the pages that are fetched are handed to the
 * migrator warps before the first lookup (unless they would fill more than half the pool).  When those pages
 * fit the pool twice over they are also held in their frames for the length of the launch and their rows are
 * added up straight from the frames: no request tables, and only the rows read in place are staged (the call then
 * reads two counters back after its counting kernels, i.e. it synchronises with its stream once).  Where none of
 * that is possible it behaves like 1.
 * counted = 0: the online form, which needs no pass over the list: the first `limit` requests that find a page
 * absent read their rows in place (counted in the frame field of the invalid entry), the next one fetches the
 * page.  Other values: GPUVM_E_ARG. */
int gpuvm_set_inplace_counted(gpuvm_t h, int counted);

/* Largest number of simultaneously resident warps that can each hold
 * `pins_per_warp` pages pinned without exhausting the pool (a warp that holds
 * pins while faulting needs a free frame; Section 3.3: a frame is reused only
 * when its reference counter is zero).  Accessors that hold at most one page at
 * a time (gpuvm_read / gpuvm_write) are safe with any number of warps. */
int gpuvm_safe_warps(gpuvm_t h, int pins_per_warp);

/* Pages that must be in flight to keep a link of `bytes_per_s` busy at a fault
 * round-trip of `latency_s` (Little's law as applied in Section 3.2). */
double gpuvm_inflight_pages(double latency_s, double bytes_per_s, double page_bytes);

/* Test hook: overwrite one page-table entry with `value` (host-side injection of
 * a page that stays "being fetched" so that a bounded device wait can be seen to
 * expire with an error status instead of hanging). */
int gpuvm_debug_poke_pte(gpuvm_t h, uint64_t page, uint64_t value);

/* Test hook: read one page-table entry into *value (host pointer).  Synchronises the device. */
int gpuvm_debug_peek_pte(gpuvm_t h, uint64_t page, uint64_t *value);

const char *gpuvm_strerror(int status);
int gpuvm_last_cuda_error(gpuvm_t h);

#ifdef __cplusplus
}
#endif
#endif /* GPUVM_H */
