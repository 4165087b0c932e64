/*
 * gpuvm_batch.cuh -- batched access: one warp keeps up to 2048 page requests in flight.
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
 * gpuvm_batch_run is the engine itself: tables of up to 64 * W rows in any layout that a
 * small accessor type can read (for instance bare 32-bit element indices).
 */
#ifndef GPUVM_BATCH_CUH
#define GPUVM_BATCH_CUH

#include "gpuvm_device.cuh"

struct gpuvm_batch_entry {
    unsigned int vpn;       /* page number; 0xFFFFFFFF = rejected request */
    unsigned int offl;      /* offset in the page */
};

constexpr unsigned int GPUVM_BATCH_MAX = 2048;

/* Ring of owned faults of one thread block, in shared memory.  Zero it (all fields) before
 * use, set `requesters` to the number of requester warps, __syncthreads(). */
constexpr unsigned int GPUVM_FAULT_QUEUE_SLOTS = 2048;
struct gpuvm_fault_queue {
    unsigned int head;          /* next slot to pop  */
    unsigned int tail;          /* next slot to push */
    unsigned int requesters;    /* requester warps that have not called gpuvm_requester_done yet */
    unsigned int pad;
    unsigned int slot[GPUVM_FAULT_QUEUE_SLOTS];   /* 0 = empty, else (vpn + 1) | write << 31 */
};

namespace gpuvm {

constexpr unsigned int kNotReady = 0xFFFFFFFFu;   /* "frame" values a leader hands to its followers */
constexpr unsigned int kFailed = 0xFFFFFFFEu;
constexpr unsigned int kRejected = 0xFFFFFFFFu;   /* vpn of a request that was refused when it was set */

/* Any lane.  False when the ring is (nearly) full: the caller keeps the fault and retries. */
__device__ __forceinline__ bool fault_queue_push(gpuvm_fault_queue *q, unsigned int vpn, int mode)
{
    volatile unsigned int *vh = &q->head, *vt = &q->tail;
    /* up to 1024 lanes may pass this check at the same moment: keep that many slots spare */
    if (*vt - *vh >= GPUVM_FAULT_QUEUE_SLOTS - 1024u) return false;
    const unsigned int pos = atomicAdd(&q->tail, 1u);
    volatile unsigned int *slot = &q->slot[pos % GPUVM_FAULT_QUEUE_SLOTS];
    *slot = (vpn + 1u) | (mode == kWrite ? 0x80000000u : 0u);
    return true;
}

/* All 32 lanes: frame `h` has been claimed for page `vpn` by lane `L` (steps 6 and 7 of the
 * access path): write a dirty victim back, unmap it, copy the page in, publish. */
__device__ __forceinline__ void migrate_page(const gpuvm_dev_t &vm, unsigned long long vpn, int mode, unsigned int h,
                                             unsigned long long victim, int vdirty, unsigned int lane, unsigned int L)
{
    unsigned char *fr = vm.pool + ((unsigned long long)h << vm.page_shift);
    if (victim != ~0ull) {
        if (vdirty) {
            warp_copy<8, true>(vm.host + (victim << vm.page_shift), fr, page_len(vm, victim) >> 4, lane, 32);
            __threadfence_system();
            __syncwarp();
        }
        if (lane == L) {
            atomicXor(vm.pte + victim, kEvicting | ((unsigned long long)h << kFrameShift) | (vdirty ? kDirty : 0ull));
            stat_add(vm, kEvictions, 1);
            if (vdirty) { stat_add(vm, kWritebacks, 1); stat_add(vm, kBytesOut, page_len(vm, victim)); }
        }
    }
    warp_copy<8, false>(fr, vm.host + (vpn << vm.page_shift), page_len(vm, vpn) >> 4, lane, 32);
    __threadfence();
    __syncwarp();
    if (lane == L) {
        st_relaxed_u32(vm.frame_vpn + h, (unsigned int)vpn);
        atomicXor(vm.pte + vpn, (kBusy ^ kValid) | ((unsigned long long)h << kFrameShift) |
                                    (vm.policy == GPUVM_POLICY_CLOCK ? kRef : 0ull) | (mode == kWrite ? kDirty : 0ull));
        stat_add(vm, kFaults, 1);
        stat_add(vm, kBytesIn, page_len(vm, vpn));
    }
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
static __device__ __noinline__ void gpuvm_migrator_loop(const gpuvm_dev_t vm, gpuvm_fault_queue *q)
{
    using namespace gpuvm;
    const unsigned int lane = lane_id();
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
            }
        }
        item = __shfl_sync(0xFFFFFFFFu, item, 0);
        if (item == 0u) {
            const unsigned int done = (lane == 0) ? (unsigned int)(*vr == 0u && *vh == *vt) : 0u;
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
        migrate_page(vm, vpn, mode, __shfl_sync(0xFFFFFFFFu, h, 0), __shfl_sync(0xFFFFFFFFu, victim, 0),
                     __shfl_sync(0xFFFFFFFFu, (int)vdirty, 0), lane, 0);
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
 * The engine.  W: the table has up to 64 * W rows of 32 requests (state of a lane's requests
 * is kept in W 64-bit masks per kind).  Table: see gpuvm_entry_table.  Groups are formed with
 * __match_any_sync when the requests are registered and again, over the lanes that are not
 * finished, whenever a row is visited: a group finishes as a whole, so the lanes and the
 * leader (lowest lane) are the same every time.
 */
template <int W, bool WARP_CONSUME, class Table, class Consume>
static __device__ __noinline__ unsigned int gpuvm_batch_run(const gpuvm_dev_t vm, const Table table, unsigned int n,
                                                            int mode, Consume consume, gpuvm_fault_queue *queue)
{
    using namespace gpuvm;
    const unsigned int lane = lane_id();
    const unsigned int rows = (n + 31) >> 5;
    unsigned long long todo[W], lead[W], own[W], failed[W];
    /* bit j of word k: row 64 k + j.  todo: my request is not finished; lead: I lead my group
     * (I hold its reference); own: my group's page is BUSY by my CAS and not handed on;
     * failed: I gave up on the row (leader only) */
#pragma unroll
    for (int k = 0; k < W; ++k) { todo[k] = 0; lead[k] = 0; own[k] = 0; failed[k] = 0; }
    unsigned int served = 0;

    /* register every request in the page table (steps 1-4 of the access path) */
#pragma unroll
    for (int k = 0; k < W; ++k) {
        for (unsigned int jj = 0; jj < 64 && 64u * k + jj < rows; ++jj) {
            const unsigned int i = (64u * k + jj) * 32 + lane;
            const bool active = i < n && table.valid(i);
            const unsigned int m = __ballot_sync(0xFFFFFFFFu, active);
            if (active) {
                const unsigned int vpn = table.vpn(i);
                const unsigned int group = __match_any_sync(m, vpn);
                if (lane == (unsigned int)(__ffs(group) - 1)) {
                    unsigned long long *pte = vm.pte + vpn;
                    unsigned int frame;
                    const int st = advance(vm, pte, pin_acquire(pte) + 1ull, mode, frame);
                    if (st == kReady) { if (GPUVM_COUNT_HITS) stat_add(vm, kHits, 1); }
                    else if (st == kWait) stat_add(vm, kWaits, 1);
                    else own[k] |= 1ull << jj;
                    if (group & (group - 1)) stat_add(vm, kLanes, __popc(group) - 1);
                    lead[k] |= 1ull << jj;
                }
                todo[k] |= 1ull << jj;
            }
        }
    }
    __syncwarp();

    unsigned long long t_start = 0;
    unsigned int sleep_ns = 64;
    for (;;) {
        bool progress = false, any_rows = false;
#pragma unroll
        for (int k = 0; k < W; ++k) {
            for (unsigned int jj = 0; jj < 64 && 64u * k + jj < rows; ++jj) {
                const unsigned long long bit = 1ull << jj;
                const bool mine = (todo[k] & bit) != 0;
                const unsigned int rowmask = __ballot_sync(0xFFFFFFFFu, mine);
                if (!rowmask) continue;
                any_rows = true;
                const unsigned int i = (64u * k + jj) * 32 + lane;
                unsigned int frame = kNotReady, off = 0;
                unsigned long long *pte = nullptr;
                bool is_leader = false;
                if (mine) {
                    const unsigned int vpn = table.vpn(i);
                    const unsigned int leader = __ffs(__match_any_sync(rowmask, vpn)) - 1;
                    off = table.off(i);
                    pte = vm.pte + vpn;
                    is_leader = (lead[k] & bit) != 0;            /* == (lane == leader) */
                    if (is_leader) {
                        if (failed[k] & bit) {
                            frame = kFailed;
                        } else if (!(own[k] & bit)) {
                            unsigned int f;
                            const int st = advance(vm, pte, ld_acquire_u64(pte), mode, f);   /* pairs with the publish */
                            if (st == kReady) frame = f;
                            else if (st == kOwn) { own[k] |= bit; progress = true; }
                        }
                    }
                    frame = __shfl_sync(rowmask, frame, leader);
                    if (frame == kFailed) todo[k] &= ~bit;
                }
                const bool ready = mine && frame < kFailed;
                if (WARP_CONSUME) {
                    unsigned int ready_lanes = __ballot_sync(0xFFFFFFFFu, ready);
                    while (ready_lanes) {
                        const unsigned int L = __ffs(ready_lanes) - 1;
                        ready_lanes &= ready_lanes - 1;
                        const unsigned int f = __shfl_sync(0xFFFFFFFFu, frame, L), o = __shfl_sync(0xFFFFFFFFu, off, L);
                        consume((64u * k + jj) * 32 + L, vm.pool + ((unsigned long long)f << vm.page_shift) + o);
                    }
                    __syncwarp();                               /* every group has used its frame */
                } else {
                    if (ready) consume(i, vm.pool + ((unsigned long long)frame << vm.page_shift) + off);
                    if (mine) __syncwarp(rowmask);              /* the whole group has used the frame */
                }
                if (ready) {
                    todo[k] &= ~bit;
                    ++served;
                    progress = true;
                    if (is_leader) unpin(pte);                  /* step 8 */
                }
            }
        }
        if (!any_rows) break;

        if (queue) {
            /* hand owned faults to the migrator warps; afterwards wait for the page like anyone */
#pragma unroll
            for (int k = 0; k < W; ++k)
                while (own[k]) {
                    const unsigned int jj = __ffsll((long long)own[k]) - 1;
                    if (!fault_queue_push(queue, table.vpn((64u * k + jj) * 32 + lane), mode)) break;
                    own[k] &= own[k] - 1;
                    progress = true;
                }
        } else {
            /* no helpers: the first lane that owns a fault takes a frame and the warp migrates the page */
            bool has_own = false;
#pragma unroll
            for (int k = 0; k < W; ++k) has_own |= own[k] != 0;
            const unsigned int owners = __ballot_sync(0xFFFFFFFFu, has_own);
            if (owners) {
                const unsigned int L = __ffs(owners) - 1;
                unsigned int h = 0, vpn = 0;
                unsigned long long victim = ~0ull;
                bool vdirty = false;
                int claimed = 0;
                if (lane == L) {
                    int kk = 0;
#pragma unroll
                    for (int k = W - 1; k >= 0; --k) if (own[k]) kk = k;
                    unsigned long long word = 0;
#pragma unroll
                    for (int k = 0; k < W; ++k) if (k == kk) word = own[k];
                    vpn = table.vpn((64u * kk + (__ffsll((long long)word) - 1)) * 32 + lane);
                    claimed = try_claim(vm, vpn, 4, h, victim, vdirty);
                }
                if (__shfl_sync(0xFFFFFFFFu, claimed, L)) {
                    migrate_page(vm, __shfl_sync(0xFFFFFFFFu, vpn, L), mode, __shfl_sync(0xFFFFFFFFu, h, L),
                                 __shfl_sync(0xFFFFFFFFu, victim, L), __shfl_sync(0xFFFFFFFFu, (int)vdirty, L), lane, L);
                    if (lane == L) {
                        bool cleared = false;
#pragma unroll
                        for (int k = 0; k < W; ++k)
                            if (!cleared && own[k]) { own[k] &= own[k] - 1; cleared = true; }
                    }
                    progress = true;
                }
            }
        }

        if (__any_sync(0xFFFFFFFFu, progress)) { sleep_ns = 64; t_start = 0; continue; }
        /* nothing moved: back off; give up when the bound is reached */
        const unsigned long long t = now_ns();
        if (t_start == 0) t_start = t;
        bool expired = (t - t_start) > (unsigned long long)vm.spin_limit_us * 1000ull || has_error(vm);
        expired = __any_sync(0xFFFFFFFFu, expired);
        if (expired) {
#pragma unroll
            for (int k = 0; k < W; ++k) {
                unsigned long long give_up = todo[k] & lead[k] & ~failed[k];
                while (give_up) {
                    const unsigned int jj = __ffsll((long long)give_up) - 1;
                    give_up &= give_up - 1;
                    const unsigned int vpn = table.vpn((64u * k + jj) * 32 + lane);
                    set_error(vm, GPUVM_E_TIMEOUT, vpn);
                    if ((own[k] >> jj) & 1ull) atomicXor(vm.pte + vpn, kBusy);   /* BUSY -> INVALID: never handed on */
                    unpin(vm.pte + vpn);
                    own[k] &= ~(1ull << jj);
                    failed[k] |= 1ull << jj;
                }
            }
            continue;                                           /* followers learn of it in the next round */
        }
        if (lane == 0) stat_add(vm, kRetries, 1);
        __nanosleep(sleep_ns);
        if (sleep_ns < 4096) sleep_ns *= 2;
    }
    return served;
}

/* One table of up to 2048 eight-byte entries (see the top of this file). */
template <bool WARP_CONSUME = false, class Consume>
static __device__ __forceinline__ unsigned int gpuvm_batch_access(const gpuvm_dev_t &vm, gpuvm_batch_entry *table,
                                                                  unsigned int n, int mode, Consume consume,
                                                                  gpuvm_fault_queue *queue = nullptr)
{
    return gpuvm_batch_run<1, WARP_CONSUME>(vm, gpuvm_entry_table{table}, n, mode, consume, queue);
}

#endif /* GPUVM_BATCH_CUH */
