/*
 * gpuvm_batch.cuh -- batched access: one warp keeps thousands of page requests in flight.
 *
 * gpuvm_read / gpuvm_write return when the slowest of a warp's 32 requests has been
 * served, so a warp never has more than 32 requests outstanding.  For scattered
 * accesses that is what limits fault coalescing across warps (Section 3.3): the more
 * requests are registered in the page table at once, the more of them each migrated
 * page serves.  Here a warp stages a batch of page ids in a request table (8 bytes per
 * request, up to 64 rows of 32; shared or global memory), registers all of them in the
 * page table at once, and then runs the same fault state machine as the single-access
 * path over the whole table until every request has been served:
 *
 *   - row by row, the requests of a row are grouped with __match_any_sync; the leader
 *     of a group pins the page (atomicAdd on the entry) and becomes hit, waiter or
 *     owner exactly as in gpuvm_device.cuh; followers take the frame number from their
 *     leader by shuffle when the page is there (the grouping is redone over the unfinished
 *     lanes of the row each time: a group finishes as a whole, so it comes out the same);
 *   - every round, each unfinished row is visited: leaders re-read their entry; groups
 *     whose page is resident call `consume(i, ptr)` on each of their requests and the
 *     leader drops the reference at once (no page is held while frames are claimed:
 *     deadlock-free for any pool size);
 *   - faults the warp owns are handed to the thread block's ring of page ids in shared
 *     memory (gpuvm_fault_queue) and served by the block's migrator warps, which run
 *     gpuvm_migrator_loop: pop a page id, take a frame, write a dirty victim back, copy
 *     the page in, publish.  A warp that copies a page does not look at its table
 *     meanwhile, and pages published for it stay pinned that long; with thousands of
 *     warps that is what runs a pool dry.  Splitting the roles lets requesters come back
 *     to every resident page within one scan of their table.  Without a ring
 *     (queue == nullptr) the requesting warp migrates its pages itself, one per round.
 *
 * Use: all 32 lanes of a warp, converged.
 *     gpuvm_batch_set(vm, table, i, byte_offset)   for i < n, any lane may fill any i
 *     __syncwarp();
 *     gpuvm_batch_access(vm, table, n, GPUVM_READ or GPUVM_WRITE, consume, queue);
 * `consume(i, p)` is called exactly once per served request, by lane i % 32, with p
 * pointing at the requested byte inside its frame (use gpuvm_load / gpuvm_store on it);
 * it may overwrite table[i] (for instance with the value it read).  With WARP_CONSUME the
 * call is made by all 32 lanes together, one served request after the other, with the same
 * i and p in every lane: the shape for requests whose payload is a row that the warp reads
 * with coalesced 16-byte loads.  gpuvm_batch_skip(table, i) marks slot i as unused.  Requests that fail
 * (offset out of range, wait ran out) are not consumed; the sticky error is set as for the
 * other accessors.  Returns the number of requests served for the calling lane.
 * A consume function that only READS the page should return an unsigned value computed from
 * what it read (the value itself will do): in read mode the engine then makes the release of
 * the page depend on those values instead of issuing a fence per row, which is what bounded
 * the scan before (one third of all warp cycles).  A consume function that returns void, and
 * every consume function in write mode, gets a warp barrier and a fence before the release.
 * gpuvm_batch_run is the engine itself: longer tables, in any layout that a small accessor
 * type can read (for instance bare 32-bit element indices), with the per-lane state words in
 * memory the caller provides.
 * Reads in place (read mode, data that nobody writes through the runtime meanwhile): with inplace_limit != 0
 * a request for a page that is not resident need not fetch it; consume then gets a pointer into the backing
 * store (inplace_bytes: what one such request moves, for the bytes_direct counter).  Which requests: with
 * `demand` (one 32-bit count per page: how many requests of the whole launch name it, counted by the caller
 * beforehand) those of pages with fewer than inplace_limit requests, without the page table being touched at
 * all, and every other page is fetched at its first touch; without `demand` the first inplace_limit requests
 * that find a page absent, counted in the frame field of its entry, and the one after them fetches it.
 */
#ifndef GPUVM_BATCH_CUH
#define GPUVM_BATCH_CUH

#include <type_traits>

#include "gpuvm_device.cuh"

struct gpuvm_batch_entry {
    unsigned int vpn;       /* page number; 0xFFFFFFFF = rejected request */
    unsigned int offl;      /* offset in the page */
};

constexpr unsigned int GPUVM_BATCH_MAX = 2048;

/* Ring of owned faults of one thread block, in shared memory.  Zero it (all fields) before
 * use, set `requesters` to the number of requester warps, __syncthreads(). */
constexpr unsigned int GPUVM_FAULT_QUEUE_SLOTS = 2048;
constexpr unsigned int GPUVM_SHARED_QUEUE_SLOTS = 1u << 16;
constexpr unsigned int GPUVM_FAULT_QUEUE_SPILL = 8;       /* entries a block keeps for its own migrators */

/* Optional ring in device memory that all thread blocks of a grid share: a block whose own
 * ring already holds GPUVM_FAULT_QUEUE_SPILL entries pushes here instead, and migrator warps
 * that find their block's ring empty pop from here, so no block is left to move a long
 * backlog alone while the migrators of the others idle.  Zero it before the launch. */
struct gpuvm_shared_queue {
    unsigned int head;
    unsigned int pad0[31];
    unsigned int tail;
    unsigned int pad1[31];
    unsigned int slot[GPUVM_SHARED_QUEUE_SLOTS];  /* as gpuvm_fault_queue::slot */
};

struct gpuvm_fault_queue {
    unsigned int head;          /* next slot to pop  */
    unsigned int tail;          /* next slot to push */
    unsigned int requesters;    /* requester warps that have not called gpuvm_requester_done yet */
    unsigned int pad;
    gpuvm_shared_queue *shared; /* nullptr: none */
    unsigned int slot[GPUVM_FAULT_QUEUE_SLOTS];   /* 0 = empty, else (vpn + 1) | write << 31 */
};

namespace gpuvm {

constexpr unsigned int kNotReady = 0xFFFFFFFFu;   /* "frame" values a leader hands to its followers */
constexpr unsigned int kInPlaceFrame = 0xFFFFFFFEu; /* the group reads from the backing store, it holds no reference */
constexpr unsigned int kRejected = 0xFFFFFFFFu;   /* vpn of a request that was refused when it was set */
constexpr unsigned long long kColdWord = ~0ull;   /* stands for the entry of a page that is read in place unseen (no entry has all bits set) */

/* Any lane.  False when the ring is (nearly) full: the caller keeps the fault and retries. */
__device__ __forceinline__ bool fault_queue_push(gpuvm_fault_queue *q, unsigned int vpn, int mode,
                                                 const gpuvm_dev_t *vm_for_errors = nullptr)
{
    volatile unsigned int *vh = &q->head, *vt = &q->tail;
    const unsigned int item = (vpn + 1u) | (mode == kWrite ? 0x80000000u : 0u);
    gpuvm_shared_queue *g = q->shared;
    if (g && *vt - *vh >= GPUVM_FAULT_QUEUE_SPILL) {
        /* the block has enough of its own: the shared ring, unless that is full.  A slot is
         * reserved with a compare-and-swap on the tail, so the ring cannot be overrun however
         * many lanes of the grid push at the same moment; after 32 lost races the block's
         * own ring takes the fault. */
        for (int tries = 0; tries < 32; ++tries) {
            const unsigned int gt = ld_relaxed_u32(&g->tail);
            if (gt - ld_relaxed_u32(&g->head) >= GPUVM_SHARED_QUEUE_SLOTS - 1u) break;
            if (atomicCAS(&g->tail, gt, gt + 1u) == gt) {
                unsigned int *slot = &g->slot[gt % GPUVM_SHARED_QUEUE_SLOTS];
                unsigned int spins = 0;
                while (ld_relaxed_u32(slot) != 0u && ++spins < (1u << 20)) { }   /* its last reader has not cleared it yet */
                if (ld_relaxed_u32(slot) != 0u) {            /* still there: the entry under it is lost, say so */
                    if (vm_for_errors) { stat_add(*vm_for_errors, kRingDrops, 1); set_error(*vm_for_errors, GPUVM_E_TIMEOUT, vpn); }
                }
                st_relaxed_u32(slot, item);
                return true;
            }
        }
    }
    /* up to 1024 lanes may pass this check at the same moment: keep that many slots spare */
    if (*vt - *vh >= GPUVM_FAULT_QUEUE_SLOTS - 1024u) return false;
    const unsigned int pos = atomicAdd(&q->tail, 1u);
    volatile unsigned int *slot = &q->slot[pos % GPUVM_FAULT_QUEUE_SLOTS];
    *slot = item;
    return true;
}

/* All 32 lanes: frame `h` has been claimed for page `vpn` by lane `L` (steps 6 and 7 of the
 * access path): write a dirty victim back, unmap it, copy the page in, publish.  With `bulk`
 * (state held by lane L) the page comes in through the bulk-copy unit; false is returned when
 * that copy did not finish within the bound: the sticky error is set, the page's entry goes
 * back to INVALID and the frame is free again. */
__device__ __forceinline__ bool migrate_page(const gpuvm_dev_t &vm, unsigned long long vpn, int mode, unsigned int h,
                                             unsigned long long victim, int vdirty, unsigned int lane, unsigned int L,
                                             BulkStage *bulk = nullptr)
{
    unsigned char *fr = vm.pool + ((unsigned long long)h << vm.page_shift);
    retire_victim(vm, h, victim, vdirty, lane, 32, 0xFFFFFFFFu, lane == L);
    if (bulk) {
        int ok = 1;
        if (lane == L) {
            const unsigned long long limit_ns = (unsigned long long)vm.spin_limit_us * 1000ull;
            ok = bulk_copy_in(*bulk, fr, vm.host + (vpn << vm.page_shift), (unsigned int)page_len(vm, vpn), limit_ns);
            if (!ok) {
                /* Nothing may still be writing into the frame when it is given back: wait for the
                 * staging-to-frame copies that were committed, and (bounded) for the host-to-staging
                 * copies in flight, before the entry and the ring slot are released. */
                asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
                bulk_stage_drain(*bulk, limit_ns);
                set_error(vm, GPUVM_E_TIMEOUT, vpn);
                atomicXor(vm.pte + vpn, kBusy);                      /* BUSY -> INVALID */
                st_relaxed_u32(vm.frame_vpn + h, kFrameFree);
            }
        }
        if (!__shfl_sync(0xFFFFFFFFu, ok, L)) return false;
    } else {
        warp_copy<8, false>(fr, vm.host + (vpn << vm.page_shift), page_len(vm, vpn) >> 4, lane, 32);
    }
    __threadfence();
    __syncwarp();
    if (lane == L) publish(vm, vpn, h, mode);
    return true;
}

}  // namespace gpuvm

/* Called once by each requester warp (one lane) when it has no more batches to run. */
__device__ __forceinline__ void gpuvm_requester_done(gpuvm_fault_queue *q)
{
    __threadfence_block();
    atomicSub(&q->requesters, 1u);
}

/*
 * Body of a migrator warp (all 32 lanes, converged): serve the block's fault ring until
 * every requester warp is done and the ring is empty.  If no frame can be had for a page
 * within the bound, the sticky error is set and the page's entry goes back to INVALID, so
 * that its waiters give up instead of waiting forever.
 */
static __device__ __noinline__ void gpuvm_migrator_loop(const gpuvm_dev_t vm, gpuvm_fault_queue *q,
                                                        unsigned char *stage_buf = nullptr,
                                                        unsigned long long *stage_mbar = nullptr,
                                                        unsigned int chunk = 0, unsigned int stages = 0)
{
    using namespace gpuvm;
    const unsigned int lane = lane_id();
    BulkStage bulk{stage_buf, stage_mbar, chunk, stages, 0u, 0u};
    const bool use_bulk = stage_buf != nullptr && stages != 0u;
    if (use_bulk && lane == 0) bulk_stage_init(bulk);
    __syncwarp();
    volatile unsigned int *vh = &q->head, *vt = &q->tail, *vr = &q->requesters;
    unsigned int idle_ns = 32;
    for (;;) {
        unsigned int item = 0;
        if (lane == 0) {
            const unsigned int h = *vh;
            if (h != *vt && atomicCAS(&q->head, h, h + 1u) == h) {
                volatile unsigned int *slot = &q->slot[h % GPUVM_FAULT_QUEUE_SLOTS];
                unsigned int spins = 0;
                while ((item = *slot) == 0u && ++spins < (1u << 24)) { }   /* the pusher is between its two stores */
                *slot = 0u;
                if (item == 0u) { stat_add(vm, kRingDrops, 1); set_error(vm, GPUVM_E_TIMEOUT, ~0ull); }
            }
        }
        if (lane == 0 && item == 0u && q->shared) {
            gpuvm_shared_queue *g = q->shared;
            const unsigned int h = ld_relaxed_u32(&g->head);
            if (h != ld_relaxed_u32(&g->tail) && atomicCAS(&g->head, h, h + 1u) == h) {
                unsigned int *slot = &g->slot[h % GPUVM_SHARED_QUEUE_SLOTS];
                unsigned int spins = 0;
                while ((item = ld_relaxed_u32(slot)) == 0u && ++spins < (1u << 22)) { }   /* the pusher is between its two stores */
                st_relaxed_u32(slot, 0u);
                if (item == 0u) { stat_add(vm, kRingDrops, 1); set_error(vm, GPUVM_E_TIMEOUT, ~0ull); }
            }
        }
        /* An entry names a page that its pusher turned BUSY and nobody else may touch.  An entry
         * that was given up on above and filled in late can surface a ring cycle later, when its
         * page is long done: anything that is not BUSY is dropped, never migrated. */
        if (lane == 0 && item != 0u) {
            const unsigned long long w = ld_relaxed_u64(vm.pte + ((item & 0x7FFFFFFFu) - 1u));
            if ((w & kStMask) != kBusy) { stat_add(vm, kRingDrops, 1); set_error(vm, GPUVM_E_TIMEOUT, (item & 0x7FFFFFFFu) - 1u); item = 0u; }
        }
        item = __shfl_sync(0xFFFFFFFFu, item, 0);
        if (item == 0u) {
            /* no fault to serve: write back a dirty page that is about to become a victim, so that whoever needs a
             * frame next gets it without a write-back */
            if (clean_ahead(vm, 0xFFFFFFFFu, lane, 32, lane == 0)) { idle_ns = 32; continue; }
            const unsigned int done = (lane == 0) ? (unsigned int)(*vr == 0u && *vh == *vt &&
                                                                   (!q->shared || ld_relaxed_u32(&q->shared->head) ==
                                                                                      ld_relaxed_u32(&q->shared->tail))) : 0u;
            if (__shfl_sync(0xFFFFFFFFu, done, 0)) return;
            __nanosleep(idle_ns);
            if (idle_ns < 1024) idle_ns *= 2;
            continue;
        }
        idle_ns = 32;
        const unsigned long long vpn = (item & 0x7FFFFFFFu) - 1u;
        const int mode = (item >> 31) ? kWrite : kRead;
        unsigned int h = 0;
        unsigned long long victim = ~0ull;
        bool vdirty = false;
        int claimed = 0;
        unsigned long long t_start = 0;
        unsigned int sleep_ns = 32;
        for (;;) {
            if (lane == 0) claimed = try_claim(vm, vpn, 8, h, victim, vdirty);
            claimed = __shfl_sync(0xFFFFFFFFu, claimed, 0);
            if (claimed) break;
            const unsigned long long t = now_ns();
            if (t_start == 0) t_start = t;
            const bool expired = (t - t_start) > (unsigned long long)vm.spin_limit_us * 1000ull || has_error(vm);
            if (__any_sync(0xFFFFFFFFu, expired)) break;
            if (lane == 0) stat_add(vm, kRetries, 1);
            __nanosleep(sleep_ns);
            if (sleep_ns < 2048) sleep_ns *= 2;
        }
        if (!claimed) {
            if (lane == 0) {
                set_error(vm, GPUVM_E_TIMEOUT, vpn);
                atomicXor(vm.pte + vpn, kBusy);                  /* BUSY -> INVALID */
            }
            continue;
        }
        if (!migrate_page(vm, vpn, mode, __shfl_sync(0xFFFFFFFFu, h, 0), __shfl_sync(0xFFFFFFFFu, victim, 0),
                          __shfl_sync(0xFFFFFFFFu, (int)vdirty, 0), lane, 0, use_bulk ? &bulk : nullptr)) {
            /* the bulk copy ran out of time: the error is set, requesters give up; let the copies
             * still in flight land before the shared memory is given up, and stop serving */
            if (lane == 0) bulk_stage_drain(bulk, (unsigned long long)vm.spin_limit_us * 1000ull);
            __syncwarp();
            return;
        }
    }
}

__device__ __forceinline__ void gpuvm_batch_set(const gpuvm_dev_t &vm, gpuvm_batch_entry *table, unsigned int i,
                                                unsigned long long byte_off)
{
    gpuvm_batch_entry e;
    if (byte_off >= vm.bytes) {
        gpuvm::set_error(vm, GPUVM_E_RANGE, byte_off >> vm.page_shift);
        e.vpn = gpuvm::kRejected; e.offl = 0;
    } else {
        e.vpn = (unsigned int)(byte_off >> vm.page_shift);
        e.offl = (unsigned int)(byte_off & ((1ull << vm.page_shift) - 1ull));
    }
    table[i] = e;
}

__device__ __forceinline__ void gpuvm_batch_skip(gpuvm_batch_entry *table, unsigned int i)
{
    table[i].vpn = gpuvm::kRejected;
    table[i].offl = 0;
}

/* How the engine reads a request table.  valid(i): slot i holds a request; vpn(i) / off(i):
 * its page number and the offset inside the page.  The engine never writes the table. */
struct gpuvm_entry_table {
    const gpuvm_batch_entry *e;
    __device__ __forceinline__ bool valid(unsigned int i) const { return e[i].vpn != gpuvm::kRejected; }
    __device__ __forceinline__ unsigned int vpn(unsigned int i) const { return e[i].vpn; }
    __device__ __forceinline__ unsigned int off(unsigned int i) const { return e[i].offl; }
};

/*
 * The engine.  Table: see gpuvm_entry_table.  The table has up to GPUVM_BATCH_ROWS_MAX rows of
 * 32 requests.  The state of a lane's requests is two bits per row, kept in 64-bit words that
 * the caller provides: `masks` points at the calling lane's first word, word w of kind c
 * (0: todo, my request is not finished; 1: own, my group's page is BUSY by my compare-and-swap
 * and not handed to a migrator yet) is masks[(c * words + w) * mask_stride] with
 * words = ceil(rows / 64).  Shared memory with mask_stride = 32 and one base per lane, or a
 * per-thread array with mask_stride = 1, both work; gpuvm_batch_mask_words(n) gives the count
 * per lane.  Groups are formed with __match_any_sync when the requests are registered and
 * again, over the lanes that are not finished, whenever a row is visited: a group finishes as
 * a whole, so the lanes and the leader (lowest lane, it holds the group's reference) are the
 * same every time.
 * eager_push: a fault the warp comes to own goes to the ring while the rest of the table is
 * still being registered, instead of after the first round of visits.  Right when the table
 * holds all the requests the warp will ever make (the link starts at once); wrong when tables
 * follow one another, because pages that later rows of this table would have pinned are
 * still unprotected when the migrators look for victims (measured: 20-25 % more faults on the
 * Zipf embedding bag).
 */
constexpr unsigned int GPUVM_BATCH_ROWS_MAX = 1u << 16;
#ifndef GPUVM_BATCH_REGISTER_PER_ROUND
#define GPUVM_BATCH_REGISTER_PER_ROUND 1024u   /* words of 64 rows registered before each round of visits */
#endif
#ifndef GPUVM_BATCH_ACQ
#define GPUVM_BATCH_ACQ 1
#endif
#ifndef GPUVM_BATCH_ROWS_AT_ONCE
#define GPUVM_BATCH_ROWS_AT_ONCE 2     /* 1, 2, 4 or 8: rows whose memory accesses are issued together (2: no spills to speak
                                          of at 64 registers; 4 spilled ten times as much for the same speed, 8 was slower) */
#endif


__host__ __device__ __forceinline__ unsigned int gpuvm_batch_mask_words(unsigned int n)
{
    return 2u * ((((n + 31u) >> 5) + 63u) >> 6);
}

/*
 * A consume "function" for WARP_CONSUME that the engine carries out itself: request i asks for a row of
 * units16 x 16 bytes (at most 32 units), which goes to dst + i * units16 (in 16-byte units; ordinary device
 * memory).  Because the engine knows what is to be done it can have the rows of four requests in flight at
 * a time (four loads per lane, then four stores), which is what the rows that are read in place from the
 * backing store need: one such read takes a link round trip.
 */
struct gpuvm_row_copy {
    uint4 *dst;
    unsigned int units16;
    __device__ __forceinline__ unsigned int operator()(unsigned int, const unsigned char *) const { return 0u; }   /* (never called) */
};

namespace gpuvm {
/* call a consume function; what a non-void one returns is folded into `dep` */
template <class Consume>
__device__ __forceinline__ void call_consume(Consume &consume, unsigned int i, const unsigned char *p, unsigned int &dep)
{
    if constexpr (std::is_void<decltype(consume(i, p))>::value) consume(i, p);
    else dep ^= (unsigned int)consume(i, p);
}
}  // namespace gpuvm

template <bool WARP_CONSUME, class Table, class Consume>
static __device__ __noinline__ unsigned int gpuvm_batch_run(const gpuvm_dev_t vm, const Table table, unsigned int n,
                                                            int mode, Consume consume, gpuvm_fault_queue *queue,
                                                            unsigned long long *masks, unsigned int mask_stride,
                                                            bool eager_push = false, unsigned int inplace_limit = 0,
                                                            unsigned int inplace_bytes = 0, const unsigned int *demand = nullptr)
{
    using namespace gpuvm;
    const unsigned int lane = lane_id();
    if (mode != kRead) inplace_limit = 0;                   /* only reads can be served from the backing store */
    unsigned int n_inplace = 0;                             /* this lane's requests served in place */
    const unsigned int rows = (n + 31) >> 5;
    const unsigned int words = (rows + 63) >> 6;
    unsigned long long *const m_todo = masks, *const m_own = masks + (size_t)words * mask_stride;
    unsigned int served = 0;
    constexpr bool kConsumeReturns = !std::is_void<decltype(consume(0u, static_cast<const unsigned char *>(nullptr)))>::value;
    unsigned int n_hits = 0, n_waits = 0, n_lanes = 0;      /* this lane's share of the counters, added up at the end */
    constexpr int R = GPUVM_BATCH_ROWS_AT_ONCE;

    /*
     * R rows of word k, starting at row j0 of the word.  first: the requests are registered in the page
     * table (steps 1-4 of the access path: grouped, pinned by their leader, hit / wait / own); otherwise
     * the unfinished ones are looked at again.  Either way every group whose page is there is consumed
     * and released on the spot, so a request that hits costs one visit and one pin / unpin pair.
     * The R rows' table entries, page-table accesses and frame loads are issued together.
     * Returns true when something moved.
     */
    auto visit = [&](unsigned int k, unsigned int j0, unsigned int jn, bool first, unsigned long long &todo,
                     unsigned long long &own) -> bool {
        unsigned int rowmask[R], vpn[R], off[R], leader[R], gsize[R], any = 0;
        unsigned long long word[R];
        bool progress = false;
#pragma unroll
        for (int u = 0; u < R; ++u) {
            const unsigned int i = (64u * k + j0 + u) * 32 + lane;
            const bool mine = j0 + u < jn && (first ? (i < n && table.valid(i)) : ((todo >> (j0 + u)) & 1ull) != 0);
            rowmask[u] = __ballot_sync(0xFFFFFFFFu, mine);
            any |= rowmask[u];
        }
        if (!any) return false;
#pragma unroll
        for (int u = 0; u < R; ++u) {
            vpn[u] = 0; off[u] = 0;
            if ((rowmask[u] >> lane) & 1u) {
                const unsigned int i = (64u * k + j0 + u) * 32 + lane;
                vpn[u] = table.vpn(i);
                off[u] = table.off(i);
                if (first) todo |= 1ull << (j0 + u);
            }
        }
#pragma unroll
        for (int u = 0; u < R; ++u) {
            leader[u] = 32; word[u] = 0; gsize[u] = 1;
            if ((rowmask[u] >> lane) & 1u) {
                const unsigned int group = __match_any_sync(rowmask[u], vpn[u]);
                leader[u] = __ffs(group) - 1;
                gsize[u] = __popc(group);
                if (lane == leader[u]) {
                    if (first && demand && inplace_limit != 0u && demand[vpn[u]] < inplace_limit) {
                        word[u] = kColdWord;                /* known cold: read in place, the page table is not touched */
                    } else if (first) {
                        word[u] = pin_acquire(vm.pte + vpn[u]) + 1ull;
                        /* far too many references to one page: the sticky error ends every wait of the
                         * launch at its next idle round, long before the counter could carry */
                        if ((word[u] & kRcMask) > kRcLimit) set_error(vm, GPUVM_E_PINS, vpn[u]);
                        n_lanes += __popc(group) - 1;
                    } else if (!((own >> (j0 + u)) & 1ull)) {
                        word[u] = ld_relaxed_u64(vm.pte + vpn[u]);
                    }
                }
            }
        }
        /* leaders: what the entries say.  A pin is an acquire; on a later visit an entry that looks VALID is
         * read again with acquire (either pairs with the fence before the publish); a VALID that turns up
         * any other way gets a fence. */
        unsigned int frame[R];
        bool need_fence = false;
#pragma unroll
        for (int u = 0; u < R; ++u) {
            frame[u] = kNotReady;
            const unsigned long long bit = 1ull << (j0 + u);
            if (lane == leader[u] && (first || !(own & bit))) {
                unsigned long long w = word[u];
                const bool looks_valid = (w & kStMask) == kValid;
                if (!first && GPUVM_BATCH_ACQ == 1 && looks_valid) w = ld_acquire_u64(vm.pte + vpn[u]);
                unsigned int f;
                const int st = w == kColdWord ? (int)kInPlace
                                              : advance(vm, vm.pte + vpn[u], w, mode, f, demand ? 0u : inplace_limit, gsize[u]);
                if (st == kReady) {
                    frame[u] = f;
                    need_fence |= GPUVM_BATCH_ACQ == 2 || (GPUVM_BATCH_ACQ == 1 && !looks_valid);
                    if (first) ++n_hits;
                } else if (st == kInPlace) {
                    frame[u] = kInPlaceFrame;           /* served from the backing store; the reference is gone already */
                    n_inplace += gsize[u];
                } else if (st == kOwn) {
                    if (!(first && eager_push && queue && fault_queue_push(queue, vpn[u], mode, &vm))) own |= bit;
                    progress = true;
                } else if (first) {
                    ++n_waits;
                }
            }
        }
        if (__any_sync(0xFFFFFFFFu, need_fence)) __threadfence();
        /* followers take the frame from their leader; every ready request is consumed */
        bool any_ready = false;
        unsigned int dep = 0;          /* what consume returned, folded: see below */
#pragma unroll
        for (int u = 0; u < R; ++u) {
            if (!rowmask[u]) continue;
            const bool mine = ((rowmask[u] >> lane) & 1u) != 0;
            if (mine) frame[u] = __shfl_sync(rowmask[u], frame[u], leader[u]);
            const bool ready = mine && frame[u] != kNotReady;
            if constexpr (WARP_CONSUME && std::is_same<Consume, gpuvm_row_copy>::value) {
                unsigned int ready_lanes = __ballot_sync(0xFFFFFFFFu, ready);
                while (ready_lanes) {
                    constexpr int Q = 4;                    /* rows in flight per warp */
                    const unsigned char *src[Q];
                    unsigned int idx[Q];
                    uint4 v[Q];
                    int cnt = 0;
#pragma unroll
                    for (int q = 0; q < Q; ++q) {
                        src[q] = nullptr; idx[q] = 0;
                        if (ready_lanes) {
                            const unsigned int L = __ffs(ready_lanes) - 1;
                            ready_lanes &= ready_lanes - 1;
                            const unsigned int f = __shfl_sync(0xFFFFFFFFu, frame[u], L), o = __shfl_sync(0xFFFFFFFFu, off[u], L);
                            const unsigned int pv = __shfl_sync(0xFFFFFFFFu, vpn[u], L);
                            src[q] = (f == kInPlaceFrame ? vm.host + ((unsigned long long)pv << vm.page_shift)
                                                         : vm.pool + ((unsigned long long)f << vm.page_shift)) + o;
                            idx[q] = (64u * k + j0 + u) * 32 + L;
                            cnt = q + 1;
                        }
                    }
                    if (lane < consume.units16) {
#pragma unroll
                        for (int q = 0; q < Q; ++q)
                            if (q < cnt) v[q] = gpuvm_load16(src[q] + 16u * lane);
#pragma unroll
                        for (int q = 0; q < Q; ++q)
                            if (q < cnt) { consume.dst[(size_t)idx[q] * consume.units16 + lane] = v[q]; dep ^= v[q].x; }
                    }
                }
            } else if (WARP_CONSUME) {
                unsigned int ready_lanes = __ballot_sync(0xFFFFFFFFu, ready);
                while (ready_lanes) {
                    const unsigned int L = __ffs(ready_lanes) - 1;
                    ready_lanes &= ready_lanes - 1;
                    const unsigned int f = __shfl_sync(0xFFFFFFFFu, frame[u], L), o = __shfl_sync(0xFFFFFFFFu, off[u], L);
                    const unsigned int pv = __shfl_sync(0xFFFFFFFFu, vpn[u], L);
                    const unsigned char *src = f == kInPlaceFrame ? vm.host + ((unsigned long long)pv << vm.page_shift)
                                                                  : vm.pool + ((unsigned long long)f << vm.page_shift);
                    call_consume(consume, (64u * k + j0 + u) * 32 + L, src + o, dep);
                }
            } else if (ready) {
                const unsigned char *src = frame[u] == kInPlaceFrame ? vm.host + ((unsigned long long)vpn[u] << vm.page_shift)
                                                                     : vm.pool + ((unsigned long long)frame[u] << vm.page_shift);
                call_consume(consume, (64u * k + j0 + u) * 32 + lane, src + off[u], dep);
            }
            any_ready |= ready;
        }
        /* step 8 for all of them.  The decrements must not overtake the groups' accesses
         * to their frames.  A consume that only reads and returns (something computed
         * from) what it read gives the engine a value that does not exist before the
         * loads have returned: `hold` below is zero, but it is computed from those values
         * of all 32 lanes, so the decrement that adds it cannot be issued earlier (this leans on
         * the hardware executing a dependent instruction after its operands exist; the PTX memory
         * model by itself does not order a relaxed atomic after earlier loads).  Any
         * other consume, and write mode, get a warp barrier and a fence instead. */
        if (__any_sync(0xFFFFFFFFu, any_ready)) {
            unsigned long long hold = 0;
            if (kConsumeReturns && mode == kRead && !(vm.debug & GPUVM_DEBUG_FENCED_RELEASE)) {
                hold = __ballot_sync(0xFFFFFFFFu, (dep & (vm.n_frames >> 31)) != 0u);   /* n_frames < 2^31 */
            } else {
                __syncwarp();
                __threadfence();
            }
#pragma unroll
            for (int u = 0; u < R; ++u) {
                if (((rowmask[u] >> lane) & 1u) && frame[u] != kNotReady) {
                    todo &= ~(1ull << (j0 + u));
                    ++served;
                    if (lane == leader[u] && frame[u] != kInPlaceFrame) atomicAdd(vm.pte + vpn[u], ~0ull + hold);
                }
            }
            progress = true;
        }
        return progress;
    };

    /* Each round registers the next words of 64 rows and then visits every registered row that has
     * unfinished requests, so pages that are there are used and released while the rest of the
     * table is still being registered. */
    unsigned int registered = 0;
    unsigned long long t_start = 0;
    unsigned int sleep_ns = 64;
    for (;;) {
        bool progress = false, any_rows = false, has_own = false;
        const unsigned int first_new = registered;
        for (unsigned int r = 0; r < GPUVM_BATCH_REGISTER_PER_ROUND && registered < words; ++r) {
            const unsigned int k = registered++;
            unsigned long long todo = 0, own = 0;
            const unsigned int jn = rows - 64u * k < 64u ? rows - 64u * k : 64u;
            for (unsigned int j0 = 0; j0 < jn; j0 += R) visit(k, j0, jn, true, todo, own);
            m_todo[(size_t)k * mask_stride] = todo;
            m_own[(size_t)k * mask_stride] = own;
            progress = true;
        }
        for (unsigned int k = 0; k < registered; ++k) {
            unsigned long long todo = m_todo[(size_t)k * mask_stride], own = m_own[(size_t)k * mask_stride];
            if (!__any_sync(0xFFFFFFFFu, todo != 0ull)) continue;
            any_rows = true;
            const unsigned long long todo_in = todo, own_in = own;
            if (k < first_new) {                              /* (what was registered in this round has just been looked at) */
                const unsigned int jn = rows - 64u * k < 64u ? rows - 64u * k : 64u;
                for (unsigned int j0 = 0; j0 < jn; j0 += R) progress |= visit(k, j0, jn, false, todo, own);
            }
            if (queue) {
                /* hand owned faults to the migrator warps; afterwards wait for the page like anyone */
                while (own) {
                    const unsigned int jj = __ffsll((long long)own) - 1;
                    if (!fault_queue_push(queue, table.vpn((64u * k + jj) * 32 + lane), mode, &vm)) break;
                    own &= own - 1;
                    progress = true;
                }
            }
            has_own |= own != 0ull;
            if (todo != todo_in) m_todo[(size_t)k * mask_stride] = todo;
            if (own != own_in) m_own[(size_t)k * mask_stride] = own;
        }
        if (!any_rows && registered == words) break;

        if (!queue) {
            /* no helpers: the first lane that owns a fault takes a frame and the warp migrates the page */
            const unsigned int owners = __ballot_sync(0xFFFFFFFFu, has_own);
            if (owners) {
                const unsigned int L = __ffs(owners) - 1;
                unsigned int h = 0, vpn = 0, kk = 0;
                unsigned long long victim = ~0ull, word = 0;
                bool vdirty = false;
                int claimed = 0;
                if (lane == L) {
                    for (kk = 0; kk < registered; ++kk)
                        if ((word = m_own[(size_t)kk * mask_stride]) != 0ull) break;
                    if (word) {
                        vpn = table.vpn((64u * kk + (__ffsll((long long)word) - 1)) * 32 + lane);
                        claimed = try_claim(vm, vpn, 4, h, victim, vdirty);
                    }
                }
                if (__shfl_sync(0xFFFFFFFFu, claimed, L)) {
                    migrate_page(vm, __shfl_sync(0xFFFFFFFFu, vpn, L), mode, __shfl_sync(0xFFFFFFFFu, h, L),
                                 __shfl_sync(0xFFFFFFFFu, victim, L), __shfl_sync(0xFFFFFFFFu, (int)vdirty, L), lane, L);
                    if (lane == L) m_own[(size_t)kk * mask_stride] = word & (word - 1);
                    progress = true;
                }
            }
        }

        if (__any_sync(0xFFFFFFFFu, progress)) {
            sleep_ns = 64; t_start = 0;
            continue;
        }
        /* nothing moved: back off; give up when the bound is reached */
        const unsigned long long t = now_ns();
        if (t_start == 0) t_start = t;
        bool expired = (t - t_start) > (unsigned long long)vm.spin_limit_us * 1000ull || has_error(vm);
        expired = __any_sync(0xFFFFFFFFu, expired);
        if (expired) {
            /* every request that is left is abandoned: its group's leader drops the reference
             * (and takes back a fault it still owns), nobody consumes */
            for (unsigned int k = 0; k < registered; ++k) {
                const unsigned long long todo = m_todo[(size_t)k * mask_stride], own = m_own[(size_t)k * mask_stride];
                const unsigned int jn = rows - 64u * k < 64u ? rows - 64u * k : 64u;
                for (unsigned int jj = 0; jj < jn; ++jj) {
                    const bool mine = ((todo >> jj) & 1ull) != 0;
                    const unsigned int rowmask = __ballot_sync(0xFFFFFFFFu, mine);
                    if (!mine) continue;
                    const unsigned int vpn = table.vpn((64u * k + jj) * 32 + lane);
                    if (lane == (unsigned int)(__ffs(__match_any_sync(rowmask, vpn)) - 1)) {
                        set_error(vm, GPUVM_E_TIMEOUT, vpn);
                        if ((own >> jj) & 1ull) atomicXor(vm.pte + vpn, kBusy);   /* BUSY -> INVALID: never handed on */
                        unpin(vm.pte + vpn);
                    }
                }
                m_todo[(size_t)k * mask_stride] = 0ull;
                m_own[(size_t)k * mask_stride] = 0ull;
            }
            break;
        }
        if (lane == 0) stat_add(vm, kRetries, 1);
        if (clean_ahead(vm, 0xFFFFFFFFu, lane, 32, lane == 0)) continue;   /* idle: write back a page that is about to be a victim */
        __nanosleep(sleep_ns);
        if (sleep_ns < 4096) sleep_ns *= 2;
    }
    __syncwarp();
    for (int o = 16; o; o >>= 1) {
        n_hits += __shfl_down_sync(0xFFFFFFFFu, n_hits, o);
        n_waits += __shfl_down_sync(0xFFFFFFFFu, n_waits, o);
        n_lanes += __shfl_down_sync(0xFFFFFFFFu, n_lanes, o);
        n_inplace += __shfl_down_sync(0xFFFFFFFFu, n_inplace, o);
    }
    if (lane == 0) {
        if (n_inplace) stat_add(vm, kBytesDirect, (unsigned long long)n_inplace * inplace_bytes);
        if (GPUVM_COUNT_HITS && n_hits) stat_add(vm, kHits, n_hits);
        if (n_waits) stat_add(vm, kWaits, n_waits);
        if (n_lanes) stat_add(vm, kLanes, n_lanes);
    }
    return served;
}

/* One table of up to 2048 eight-byte entries (see the top of this file). */
template <bool WARP_CONSUME = false, class Consume>
static __device__ __forceinline__ unsigned int gpuvm_batch_access(const gpuvm_dev_t &vm, gpuvm_batch_entry *table,
                                                                  unsigned int n, int mode, Consume consume,
                                                                  gpuvm_fault_queue *queue = nullptr)
{
    unsigned long long masks[2] = {0ull, 0ull};
    return gpuvm_batch_run<WARP_CONSUME>(vm, gpuvm_entry_table{table}, n < GPUVM_BATCH_MAX ? n : GPUVM_BATCH_MAX, mode,
                                         consume, queue, masks, 1u);
}

#endif /* GPUVM_BATCH_CUH */
