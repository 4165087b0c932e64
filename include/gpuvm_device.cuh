/*
 * gpuvm_device.cuh -- device-side accessors of the demand-paging runtime.
 *
 * Include from CUDA code compiled for sm_100a.  A kernel receives a gpuvm_dev_t BY
 * VALUE (the role of the paper's array-like object, Listing 1) and touches the
 * paged array only through:
 *
 *   T     gpuvm_read <T>(vm, elem_index, base_byte_off)        pin, load, unpin
 *   void  gpuvm_read_n<T, N>(vm, elem[N], out[N], base, count) N such reads per lane with their round trips overlapped
 *   void  gpuvm_write<T>(vm, elem_index, value, base_byte_off) pin, mark dirty, store, unpin
 *   void* gpuvm_ptr(vm, byte_off, mode, &token)                pin and hand out a frame pointer
 *   void* gpuvm_ptr_if_resident(vm, byte_off, &token)          the same, but only if the page is there: no fault, no wait
 *   void  gpuvm_release(vm, token)                             unpin what gpuvm_ptr pinned
 *   void  gpuvm_clean(vm, token, p)                            write a pinned page back now (eager write-back)
 *   void  gpuvm_prefetch(vm, byte_off)                         fetch a page ahead of its use, unpinned
 *
 * What happens on an access (Section 3.1, Fig. 2; Section 3.3):
 *   1. address split: page number = byte offset >> page_shift, offset = the rest;
 *   2. translate: the page-table entry is read; a resident page is used in place;
 *   3. the threads of the warp that want the same page are grouped with
 *      __match_any_sync over __activemask() and the lowest lane of each group acts
 *      for it ("leader"); the reference counter of a page counts such warp-level
 *      requests, not threads;
 *   4. among the leaders of different warps only one gets to service a missing
 *      page: the one whose atomicCAS turns the entry from INVALID to BUSY.  The
 *      others have already added themselves to the entry's reference counter and
 *      simply wait for the entry to become VALID; the page cannot be evicted
 *      before they have used it because the counter is not zero;
 *   5. the owner takes the next slot of the frame ring with an atomic add on the
 *      head cursor.  A free slot is taken as is.  An occupied slot is passed over
 *      when its page is in use (counter != 0) or, under the clock policy, when its
 *      reference bit is set (the bit is cleared: second chance).  Otherwise the
 *      occupant is evicted: its entry goes VALID -> EVICTING with a CAS on the exact
 *      word, so a concurrent pin makes the CAS fail;
 *   6. a dirty victim is copied back to the host by the whole warp, 16 bytes per
 *      lane and instruction, followed by a system-scope fence; then its entry
 *      becomes INVALID;
 *   7. the warp copies the new page from the host into the frame the same way,
 *      fences, and the owner publishes the entry (BUSY -> VALID, frame number,
 *      reference bit) with one atomic XOR that leaves the counter untouched;
 *   8. each thread performs its load or store in the frame; the leader drops the
 *      group's reference with a release-ordered atomic.
 *
 * Rules for callers
 *   - Any subset of a warp may call an accessor; lanes that call together are
 *     handled together.
 *   - gpuvm_read / gpuvm_write never hold a page while waiting for a frame and are
 *     deadlock-free for any pool size and any number of warps.  gpuvm_ptr holds the
 *     page until gpuvm_release: a warp must not hold more pages than
 *     gpuvm_safe_warps() allows for the grid, and should ask for ONE page per call
 *     (all calling lanes in the same page) whenever the pool may be small.
 *   - Frames change identity when pages are evicted, so frame memory must be read
 *     with gpuvm_load / gpuvm_load16 and written with gpuvm_store / gpuvm_store16
 *     (L1-bypassing, device-coherent), never through a cached plain dereference.
 *   - Every wait is bounded by vm.spin_limit_us.  When a wait runs out, or an offset
 *     lies past the end of the array, a sticky error is recorded in the control
 *     block (reported by gpuvm_stats), reads return zero, writes are dropped and
 *     gpuvm_ptr returns nullptr.  Nothing traps.
 *   - Offsets are 64-bit.  An element must not straddle a page (arrays start on a
 *     multiple of the element size).
 */
#ifndef GPUVM_DEVICE_CUH
#define GPUVM_DEVICE_CUH

#include "gpuvm.h"

#ifndef GPUVM_COUNT_HITS
#define GPUVM_COUNT_HITS 1
#endif

namespace gpuvm {

/* ---- page-table entry: [state:2 @60][hold @59][keep @58][dirty @57][ref @56][frame:32 @24][refcount:24 @0]
 *      (while the state is INVALID the frame field counts the requests served in place, see advance) */
constexpr unsigned long long kRcMask = 0xFFFFFFull;
constexpr unsigned long long kRcLimit = 1ull << 23;   /* a pin that would take the counter beyond this is refused */
constexpr unsigned long long kPinRefused = ~0ull;     /* what a refused pin hands to its group instead of the entry */
constexpr int kFrameShift = 24;
constexpr unsigned long long kFrameMask = 0xFFFFFFFFull << kFrameShift;
constexpr unsigned long long kRef = 1ull << 56;
constexpr unsigned long long kDirty = 1ull << 57;
constexpr unsigned long long kKeep = 1ull << 58;    /* advice: not to be evicted (gpuvm_advise_keep); survives every state change */
constexpr unsigned long long kHold = 1ull << 59;    /* not to be evicted while the running kernel reads it without a reference (set and cleared by that kernel) */
constexpr unsigned long long kStMask = 3ull << 60;
constexpr unsigned long long kInvalid = 0ull;
constexpr unsigned long long kBusy = 1ull << 60;
constexpr unsigned long long kValid = 2ull << 60;
constexpr unsigned long long kEvicting = 3ull << 60;

/* ---- frame ring entry */
constexpr unsigned int kFrameFree = 0xFFFFFFFFu;
constexpr unsigned int kFrameLock = 0x80000000u;

/* ---- control block (64-bit words) */
constexpr int kCtlHand = 0;
constexpr int kCtlErr = 1;
constexpr int kCtlErrPage = 2;
constexpr int kCtlCounters = 16;      /* kStatSlots slots of 16 words, one 128-byte line each */
constexpr int kStatSlots = 32;
constexpr int kCtlCleanCursor = kCtlCounters + kStatSlots * 16;   /* ring position of the cleaners (a line of its own) */
constexpr int kCtlWords = kCtlCleanCursor + 16;
enum Stat { kFaults = 0, kHits, kWaits, kLanes, kEvictions, kWritebacks, kFlushWritebacks,
            kBytesIn, kBytesOut, kHandSteps, kRetries, kRingDrops, kCleaned, kBytesDirect, kNumStats };

enum Mode { kRead = 0, kWrite = 1, kWriteAll = 2 };

struct Token {
    unsigned long long vpn;
    unsigned int group;      /* lanes that share the pin */
    unsigned int leader;     /* 1 on the lane that owns the reference */
};

/* ------------------------------------------------------------ small primitives */

__device__ __forceinline__ unsigned int lane_id()
{
    unsigned int r;
    asm volatile("mov.u32 %0, %%laneid;" : "=r"(r));
    return r;
}

__device__ __forceinline__ unsigned int sm_id()
{
    unsigned int r;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(r));
    return r;
}

__device__ __forceinline__ unsigned long long now_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long *p)
{
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long *p)
{
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

/* take one reference; acquire order: what the publisher of a VALID entry wrote to the frame
 * before publishing is visible to the accesses that follow in this thread */
__device__ __forceinline__ unsigned long long pin_acquire(unsigned long long *pte)
{
    unsigned long long old;
    asm volatile("atom.acquire.gpu.global.add.u64 %0, [%1], 1;" : "=l"(old) : "l"(pte) : "memory");
    return old;
}

/* Leader only: `w` is the entry including the reference just taken.  When the counter has
 * left the range that 2^23 warp-level requests can reach, the reference is given back, the
 * sticky GPUVM_E_PINS is set and kPinRefused is returned: the 24-bit counter never carries
 * into the frame field. */
__device__ __forceinline__ unsigned long long set_error_pins(const gpuvm_dev_t &vm, unsigned long long *pte);

__device__ __forceinline__ unsigned long long guard_pin(const gpuvm_dev_t &vm, unsigned long long *pte, unsigned long long w)
{
    if ((w & kRcMask) <= kRcLimit) return w;
    return set_error_pins(vm, pte);
}

__device__ __forceinline__ unsigned int ld_relaxed_u32(const unsigned int *p)
{
    unsigned int v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ void st_relaxed_u32(unsigned int *p, unsigned int v)
{
    asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

/* drop one reference; release order makes this thread's (and, through the warp
 * barrier before it, its group's) frame accesses happen before the drop */
__device__ __forceinline__ void unpin(unsigned long long *pte)
{
    asm volatile("red.release.gpu.global.add.u64 [%0], %1;" ::"l"(pte), "l"(~0ull) : "memory");
}

__device__ __forceinline__ void stat_add(const gpuvm_dev_t &vm, int kind, unsigned long long v)
{
    unsigned long long *p = vm.ctl + kCtlCounters + (sm_id() & (kStatSlots - 1)) * 16 + kind;
    asm volatile("red.relaxed.gpu.global.add.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

__device__ __forceinline__ void set_error(const gpuvm_dev_t &vm, int code, unsigned long long vpn)
{
    if (atomicCAS(vm.ctl + kCtlErr, 0ull, (unsigned long long)(long long)code) == 0ull)
        vm.ctl[kCtlErrPage] = vpn;
}

__device__ __forceinline__ unsigned long long set_error_pins(const gpuvm_dev_t &vm, unsigned long long *pte)
{
    unpin(pte);
    set_error(vm, GPUVM_E_PINS, (unsigned long long)(pte - vm.pte));
    return kPinRefused;
}

__device__ __forceinline__ bool has_error(const gpuvm_dev_t &vm)
{
    return ld_relaxed_u64(vm.ctl + kCtlErr) != 0ull;
}

/* 16-byte accesses.  Host side: system scope.  Frame side: device scope, no L1. */
__device__ __forceinline__ uint4 ld_host16(const void *p)
{
    uint4 v;
    asm volatile("ld.relaxed.sys.global.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ void st_host16(void *p, uint4 v)
{
    asm volatile("st.relaxed.sys.global.v4.u32 [%0], {%1,%2,%3,%4};"
                 ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

__device__ __forceinline__ uint4 ld_frame16(const void *p)
{
    uint4 v;
    asm volatile("ld.relaxed.gpu.global.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ void st_frame16(void *p, uint4 v)
{
    asm volatile("st.relaxed.gpu.global.v4.u32 [%0], {%1,%2,%3,%4};"
                 ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

/* Bytes of page `vpn` that exist in the backing store, rounded up to 16. */
__device__ __forceinline__ unsigned int page_len(const gpuvm_dev_t &vm, unsigned long long vpn)
{
    unsigned long long start = vpn << vm.page_shift;
    unsigned long long left = vm.bytes - start;
    unsigned long long page = 1ull << vm.page_shift;
    return (unsigned int)(left < page ? left : page);
}

/*
 * Warp-cooperative page copy (steps 6 and 7): the `n` calling lanes (rank 0..n-1)
 * move `n16` 16-byte units; consecutive lanes touch consecutive units, U units per
 * lane are in flight before the first store.
 */
template <int U, bool TO_HOST>
__device__ __forceinline__ void warp_copy(unsigned char *dst, const unsigned char *src,
                                          unsigned int n16, unsigned int rank, unsigned int n)
{
    const uint4 *s = reinterpret_cast<const uint4 *>(src);
    uint4 *d = reinterpret_cast<uint4 *>(dst);
    for (unsigned int base = rank; base < n16; base += n * U) {
        uint4 v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            unsigned int i = base + u * n;
            if (i < n16) v[u] = TO_HOST ? ld_frame16(s + i) : ld_host16(s + i);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            unsigned int i = base + u * n;
            if (i < n16) {
                if (TO_HOST) st_host16(d + i, v[u]);
                else st_frame16(d + i, v[u]);
            }
        }
    }
}

/*
 * Page copy by the bulk-copy unit (cp.async.bulk): one thread moves a page host -> shared
 * memory -> frame in pieces of `chunk` bytes through `stages` staging buffers, each with its
 * own mbarrier.  The copies do not pass through the load/store unit or registers, so a single
 * thread keeps stages * chunk bytes in flight (a warp copying through registers has 4 KiB)
 * and the warps that issue ordinary loads are not queued behind the migration traffic.
 * The staging memory belongs to the calling warp; buf is 128-byte aligned, chunk a multiple
 * of 16.  All addresses and lengths of the path are multiples of 16 bytes by construction
 * (page sizes are powers of two >= 16, the backing store is 16-byte aligned and a multiple of
 * 16 bytes long).
 */
struct BulkStage {
    unsigned char *buf;            /* stages * chunk bytes of shared memory */
    unsigned long long *mbar;      /* `stages` mbarriers in shared memory   */
    unsigned int chunk, stages;
    unsigned int phases;           /* bit s: parity the next wait on mbar[s] uses */
    unsigned int pending;          /* bit s: a copy into stage s has been issued and not waited for */
};

__device__ __forceinline__ unsigned int smem_addr(const void *p) { return (unsigned int)__cvta_generic_to_shared(p); }

/* one thread, once, before the first copy */
__device__ __forceinline__ void bulk_stage_init(BulkStage &s)
{
    for (unsigned int i = 0; i < s.stages; ++i)
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_addr(s.mbar + i)) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    s.phases = 0;
    s.pending = 0;
}

/* one thread: wait for the copy into stage `st`; false when `limit_ns` went by first */
__device__ __forceinline__ bool bulk_stage_wait(BulkStage &s, unsigned int st, unsigned long long limit_ns)
{
    const unsigned int mb = smem_addr(s.mbar + st), parity = (s.phases >> st) & 1u;
    unsigned long long t0 = 0;
    for (unsigned int spins = 0;; ++spins) {
        unsigned int ok;
        asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                     : "=r"(ok) : "r"(mb), "r"(parity) : "memory");
        if (ok) break;
        if ((spins & 63u) == 63u) {
            const unsigned long long t = now_ns();
            if (t0 == 0) t0 = t;
            else if (t - t0 > limit_ns) return false;
        }
    }
    s.phases ^= 1u << st;
    s.pending &= ~(1u << st);
    return true;
}

/* one thread, after a failed copy: give the copies still in flight one more bounded wait each */
__device__ __forceinline__ void bulk_stage_drain(BulkStage &s, unsigned long long limit_ns)
{
    for (unsigned int st = 0; st < s.stages; ++st)
        if ((s.pending >> st) & 1u) bulk_stage_wait(s, st, limit_ns);
}

/*
 * One thread: copy `bytes` from the backing store to a frame.  Returns false when a wait ran
 * out; copies may then still be in flight into the staging buffers (the caller sets the
 * sticky error and waits once more, bounded, before it gives the shared memory up).
 * On success every byte is in the frame: the group wait covers the writes, the proxy fence
 * orders them before the generic-proxy publish that follows in the caller.
 */
__device__ __forceinline__ bool bulk_copy_in(BulkStage &s, unsigned char *frame, const unsigned char *src,
                                             unsigned int bytes, unsigned long long limit_ns)
{
    const unsigned int nchunks = (bytes + s.chunk - 1) / s.chunk;
    auto issue = [&](unsigned int c, unsigned int st) {
        const unsigned int len = bytes - c * s.chunk < s.chunk ? bytes - c * s.chunk : s.chunk;
        const unsigned int mb = smem_addr(s.mbar + st);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(mb), "r"(len) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(smem_addr(s.buf + (size_t)st * s.chunk)), "l"(__cvta_generic_to_global(src + (size_t)c * s.chunk)),
                       "r"(len), "r"(mb) : "memory");
        s.pending |= 1u << st;
    };
    unsigned int issued = 0;
    while (issued < nchunks && issued < s.stages) { issue(issued, issued); ++issued; }
    for (unsigned int done = 0; done < nchunks; ++done) {
        const unsigned int st = done % s.stages;
        const unsigned int len = bytes - done * s.chunk < s.chunk ? bytes - done * s.chunk : s.chunk;
        if (!bulk_stage_wait(s, st, limit_ns)) return false;
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                     ::"l"(__cvta_generic_to_global(frame + (size_t)done * s.chunk)), "r"(smem_addr(s.buf + (size_t)st * s.chunk)),
                       "r"(len) : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        if (issued < nchunks) {
            asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   /* the buffer has been read */
            issue(issued, st);
            ++issued;
        }
    }
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    asm volatile("fence.proxy.async.global;" ::: "memory");
    return true;
}

/*
 * Steps 6 and 6a for the `n` calling lanes (rank 0..n-1, all of `mask`, converged): the page
 * `victim` (EVICTING, exclusively ours) leaves frame `h`.  A dirty victim is copied to the
 * host, followed by a system-scope fence; then lane `L` turns its entry INVALID with one XOR
 * that returns the frame and dirty bits to zero and leaves the counter alone.  In the poison
 * debug mode the frame is then overwritten with a pattern before anybody gets it.
 */
__device__ __forceinline__ void retire_victim(const gpuvm_dev_t &vm, unsigned int h, unsigned long long victim, int vdirty,
                                              unsigned int rank, unsigned int n, unsigned int mask, bool is_L)
{
    if (victim == ~0ull) return;
    unsigned char *fr = vm.pool + ((unsigned long long)h << vm.page_shift);
    if (vdirty) {
        warp_copy<8, true>(vm.host + (victim << vm.page_shift), fr, page_len(vm, victim) >> 4, rank, n);
        __threadfence_system();
        __syncwarp(mask);
    }
    if (is_L) {
        atomicXor(vm.pte + victim, kEvicting | ((unsigned long long)h << kFrameShift) | (vdirty ? kDirty : 0ull));
        stat_add(vm, kEvictions, 1);
        if (vdirty) { stat_add(vm, kWritebacks, 1); stat_add(vm, kBytesOut, page_len(vm, victim)); }
    }
    if (vm.debug & GPUVM_DEBUG_POISON) {
        const uint4 pat = make_uint4(0xA5A5A5A5u, 0xA5A5A5A5u, 0xA5A5A5A5u, 0xA5A5A5A5u);
        const unsigned int n16 = 1u << (vm.page_shift - 4);
        for (unsigned int i = rank; i < n16; i += n) st_frame16(fr + 16ull * i, pat);
        __threadfence();
        __syncwarp(mask);
    }
}

/* Lane that publishes (step 7), after the warp barrier that follows the copy: the fence makes
 * this thread's atomic a release for the frame stores of all lanes that passed the barrier. */
__device__ __forceinline__ void publish(const gpuvm_dev_t &vm, unsigned long long vpn, unsigned int h, int mode)
{
    st_relaxed_u32(vm.frame_vpn + h, (unsigned int)vpn);
    __threadfence();
    atomicXor(vm.pte + vpn, (kBusy ^ kValid) | ((unsigned long long)h << kFrameShift) |
                                (vm.policy == GPUVM_POLICY_CLOCK ? kRef : 0ull) | (mode != kRead ? kDirty : 0ull));
    stat_add(vm, kFaults, 1);
    if (mode != kWriteAll) stat_add(vm, kBytesIn, page_len(vm, vpn));
}

/* ------------------------------------------------------------ fault machinery */

enum LaneState { kNew = 0, kWait, kOwn, kReady, kDone, kFail, kInPlace };

/*
 * Leader only.  `w` is a fresh value of the entry that includes this group's
 * reference.  VALID: note the reference/dirty bits, READY.  BUSY or EVICTING:
 * WAIT.  INVALID: try to become the owner (step 4).
 *
 * Rent or buy.  With inplace_limit != 0 (read mode only) a page that is not resident is not
 * fetched for its first requests: while fewer than inplace_limit requests have been served from it
 * since it was last resident, this one is counted (in the frame field of the entry, which means
 * nothing while the entry is INVALID), gives its reference back in the same compare-and-swap and
 * returns IN PLACE: the caller reads what it wants from the backing store, which is current for a
 * page that is not resident.  Only when a page has been asked for often enough that its requests
 * have moved a stated fraction of its size over the link does the next request fetch it.  Pages
 * that are touched a few times never cost a page of traffic; a page that turns out hot costs at
 * most that fraction more than if it had been fetched at once.
 */
__device__ __forceinline__ int advance(const gpuvm_dev_t &vm, unsigned long long *pte,
                                       unsigned long long w, int mode, unsigned int &frame,
                                       unsigned int inplace_limit = 0, unsigned int weight = 1)
{
    for (;;) {
        unsigned long long st = w & kStMask;
        if (st == kValid) {
            unsigned long long want = (mode != kRead ? kDirty : 0ull) |
                                      (vm.policy == GPUVM_POLICY_CLOCK ? kRef : 0ull);
            if ((w & want) != want) atomicOr(pte, want);
            frame = (unsigned int)((w & kFrameMask) >> kFrameShift);
            return kReady;
        }
        if (st != kInvalid) return kWait;
        unsigned long long next;
        int result;
        if (inplace_limit != 0u && ((w & kFrameMask) >> kFrameShift) < inplace_limit) {
            next = w + ((unsigned long long)weight << kFrameShift) - 1ull;      /* count it, drop the reference */
            result = kInPlace;
        } else {
            next = (w & ~kFrameMask) | kBusy;               /* ours to fetch; the count starts over */
            result = kOwn;
        }
        unsigned long long seen = atomicCAS(pte, w, next);
        if (seen == w) return result;
        w = seen;                      /* somebody pinned, unpinned, counted or took ownership */
    }
}

/*
 * Leader only, step 5: inspect up to `tries` ring slots.  On success the frame is
 * exclusively ours (its ring entry is locked) and `victim` names the page that
 * was in it and is now EVICTING (or ~0 when the frame was free).
 */
__device__ __forceinline__ bool try_claim(const gpuvm_dev_t &vm, unsigned long long vpn,
                                          int tries, unsigned int &frame,
                                          unsigned long long &victim, bool &victim_dirty, bool allow_dirty = true)
{
    for (int t = 0; t < tries; ++t) {
        unsigned long long ticket = atomicAdd(vm.ctl + kCtlHand, 1ull);
        unsigned int h = (unsigned int)(ticket % vm.n_frames);
        unsigned int e = ld_relaxed_u32(vm.frame_vpn + h);
        if (e == kFrameFree) {
            if (atomicCAS(vm.frame_vpn + h, kFrameFree, kFrameLock | (unsigned int)vpn) == kFrameFree) {
                frame = h; victim = ~0ull; victim_dirty = false;
                stat_add(vm, kHandSteps, t + 1);
                return true;
            }
            continue;
        }
        if (e & kFrameLock) continue;                       /* in transition */
        unsigned long long *qpte = vm.pte + e;
        unsigned long long w = ld_relaxed_u64(qpte);
        if ((w & kStMask) != kValid || (w & kRcMask) != 0ull ||
            (unsigned int)((w & kFrameMask) >> kFrameShift) != h)
            continue;                                       /* in use, or a stale ring read */
        if (w & (kKeep | kHold)) continue;                  /* the caller asked for this page to stay, or a kernel is reading it unpinned */
        if (vm.policy == GPUVM_POLICY_CLOCK && (w & kRef)) {
            atomicAnd(qpte, ~kRef);                         /* second chance */
            continue;
        }
        if ((w & kDirty) && !allow_dirty) continue;         /* a prefetch does not pay for a write-back */
        unsigned long long evicting = (w & ~(kStMask | kRef)) | kEvicting;
        if (atomicCAS(qpte, w, evicting) != w) continue;    /* lost against a pin or another evictor */
        st_relaxed_u32(vm.frame_vpn + h, kFrameLock | (unsigned int)vpn);
        frame = h; victim = e; victim_dirty = (w & kDirty) != 0ull;
        stat_add(vm, kHandSteps, t + 1);
        return true;
    }
    stat_add(vm, kHandSteps, tries);
    return false;
}

/*
 * Write-back off the fault path (the paper names synchronous write-back by the faulting thread as
 * its weak spot, Section 5.3, and eviction work inside the fault handler as the cause of the step at
 * oversubscription level 1, Section 5.4).  The frame ring has a second cursor that runs ahead of the
 * head cursor: warps of the batched kernels with nothing to do -- a migrator warp whose fault ring is
 * empty, a requester warp whose scan found nothing ready -- take the next ring position from it (the
 * single-access path does not: the call alone cost its kernels a third of their resident
 * throughput in registers), and if the page in that
 * frame would be the head cursor's victim when it gets there (resident, nobody holds it, not
 * referenced since its last chance, dirty) they write it back now.  One compare-and-swap on the
 * exact entry takes a reference and clears the dirty bit: all earlier writers have released the page,
 * and any later writer marks it dirty again.  Copy, system fence, drop the reference: the page stays
 * resident, and when the head cursor arrives its frame is handed on without a write-back.  The order
 * in which frames are claimed is untouched, so no fault is added; pages written back early and
 * written to again before they are evicted cost one more write-back.  Nothing depends on the
 * cleaners: a victim that is still dirty is written back by the warp that takes its frame, as before.
 */
/*
 * The `n` calling lanes (rank 0..n-1, all of `mask`, converged; `is_L` on the lowest of them): look
 * at the next ring position ahead of the head cursor and write its page back if it qualifies.
 * Returns true when a page was written back.
 */
static __device__ __noinline__ bool clean_ahead(const gpuvm_dev_t vm, unsigned int mask, unsigned int rank, unsigned int n,
                                                bool is_L)
{
    if (vm.clean_ahead == 0u) return false;
    const unsigned int L = __ffs(mask) - 1;
    unsigned int f = kFrameFree, e = kFrameFree;
    if (is_L) {
        const unsigned long long hand = ld_relaxed_u64(vm.ctl + kCtlHand);
        unsigned long long c = ld_relaxed_u64(vm.ctl + kCtlCleanCursor);
        const unsigned long long ahead = vm.clean_ahead;
        const unsigned long long pos = c < hand ? hand : c;              /* the head cursor has overtaken: start from it */
        if (hand >= vm.n_frames && pos < hand + ahead &&                 /* (a ring that has not filled once evicts nothing) */
            atomicCAS(vm.ctl + kCtlCleanCursor, c, pos + 1ull) == c) {
            f = (unsigned int)(pos % vm.n_frames);
            e = ld_relaxed_u32(vm.frame_vpn + f);
            if (e != kFrameFree && !(e & kFrameLock) && e < vm.n_pages) {
                const unsigned long long w = ld_relaxed_u64(vm.pte + e);
                const bool fits = (w & kStMask) == kValid && (w & kRcMask) == 0ull && (w & kDirty) &&
                                  !(vm.policy == GPUVM_POLICY_CLOCK && (w & kRef)) &&
                                  (unsigned int)((w & kFrameMask) >> kFrameShift) == f;
                if (!fits || atomicCAS(vm.pte + e, w, (w & ~kDirty) + 1ull) != w) e = kFrameFree;
            } else {
                e = kFrameFree;
            }
        }
    }
    f = __shfl_sync(mask, f, L);
    e = __shfl_sync(mask, e, L);
    if (e == kFrameFree) return false;
    __threadfence();                                          /* acquire side of the writers' releases */
    const unsigned int len = page_len(vm, e);
    warp_copy<8, true>(vm.host + ((unsigned long long)e << vm.page_shift), vm.pool + ((unsigned long long)f << vm.page_shift),
                       len >> 4, rank, n);
    __threadfence_system();
    __syncwarp(mask);
    if (is_L) {
        unpin(vm.pte + e);
        stat_add(vm, kCleaned, 1);
        stat_add(vm, kBytesOut, len);
    }
    return true;
}

/*
 * Out-of-line part of every accessor: entered by all calling lanes (`active`)
 * when at least one of their pages was not resident.  `w` is the entry value the
 * group's leader got back from its pin (broadcast to the group).
 *   op_bytes  0: hand out the frame (gpuvm_ptr); 1,2,4,8,16: load or store that
 *             many bytes at `off` inside the page, value in `val`.
 * Returns true when this lane's access was performed; `frame` is then its frame.
 */
static __device__ __noinline__ bool slow_path(const gpuvm_dev_t vm, unsigned long long vpn,
                                              unsigned int off, int mode, int op_bytes,
                                              unsigned int active, unsigned int group,
                                              unsigned long long w, uint4 &val,
                                              unsigned int &frame_out)
{
    const unsigned int lane = lane_id();
    const unsigned int leader = __ffs(group) - 1;
    const bool is_leader = lane == leader;
    const unsigned int rank = __popc(active & ((1u << lane) - 1u));
    const unsigned int nlanes = __popc(active);
    unsigned long long *pte = vm.pte + vpn;
    int st = kNew;
    unsigned int frame = 0;
    bool consumed = false, ok = false;
    unsigned long long t_start = 0;
    unsigned int sleep_ns = 32;

    if (is_leader) {
        if ((w & kRcMask) > kRcLimit) {                      /* too many references to this page: refused, nothing stays pinned */
            set_error_pins(vm, pte);
            st = kFail;
        } else {
            st = advance(vm, pte, w, mode, frame);
            if (st == kReady) { if (GPUVM_COUNT_HITS) stat_add(vm, kHits, 1); }
            else if (st == kWait) stat_add(vm, kWaits, 1);
        }
    }

    for (;;) {
        bool progress = false;
        /* waiting leaders look at their entry again */
        if (is_leader && st == kWait) {
            st = advance(vm, pte, ld_relaxed_u64(pte), mode, frame);
            progress = st != kWait;
        }
        /* groups whose page is resident and pinned perform their access */
        int gst = __shfl_sync(active, st, leader);
        unsigned int gframe = __shfl_sync(active, frame, leader);
        if (gst == kReady && !consumed) {
            __threadfence();                                 /* acquire side of the publish */
            unsigned char *p = vm.pool + ((unsigned long long)gframe << vm.page_shift) + off;
            if (op_bytes == 16) {
                if (mode == kWrite) st_frame16(p, val); else val = ld_frame16(p);
            } else if (op_bytes == 8) {
                if (mode == kWrite) asm volatile("st.relaxed.gpu.global.v2.u32 [%0], {%1,%2};" ::"l"(p), "r"(val.x), "r"(val.y) : "memory");
                else asm volatile("ld.relaxed.gpu.global.v2.u32 {%0,%1}, [%2];" : "=r"(val.x), "=r"(val.y) : "l"(p) : "memory");
            } else if (op_bytes == 4) {
                if (mode == kWrite) asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(val.x) : "memory");
                else asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(val.x) : "l"(p) : "memory");
            } else if (op_bytes == 2) {
                unsigned short h = (unsigned short)val.x;
                if (mode == kWrite) asm volatile("st.relaxed.gpu.global.u16 [%0], %1;" ::"l"(p), "h"(h) : "memory");
                else { asm volatile("ld.relaxed.gpu.global.u16 %0, [%1];" : "=h"(h) : "l"(p) : "memory"); val.x = h; }
            } else if (op_bytes == 1) {
                if (mode == kWrite) asm volatile("st.relaxed.gpu.global.u8 [%0], %1;" ::"l"(p), "r"(val.x) : "memory");
                else asm volatile("ld.relaxed.gpu.global.u8 %0, [%1];" : "=r"(val.x) : "l"(p) : "memory");
            }
            consumed = true; ok = true; frame_out = gframe; progress = true;
            if (op_bytes != 0) {                             /* step 8: drop the reference */
                __syncwarp(group);
                if (is_leader) { unpin(pte); st = kDone; }
            } else if (is_leader) {
                st = kDone;                                  /* reference kept until gpuvm_release */
            }
        }
        /* owners take frames (step 5) and the warp moves the pages (steps 6, 7) */
        bool claimed = false;
        unsigned int h = 0;
        unsigned long long victim = ~0ull;
        bool vdirty = false;
        if (is_leader && st == kOwn) claimed = try_claim(vm, vpn, 4, h, victim, vdirty);
        unsigned int got = __ballot_sync(active, claimed);
        while (got) {
            const int L = __ffs(got) - 1;
            got &= got - 1;
            progress = true;
            const unsigned int bh = __shfl_sync(active, h, L);
            const unsigned long long bq = __shfl_sync(active, victim, L);
            const int bd = __shfl_sync(active, (int)vdirty, L);
            const unsigned long long bv = __shfl_sync(active, vpn, L);
            const int bmode = __shfl_sync(active, mode, L);
            unsigned char *fr = vm.pool + ((unsigned long long)bh << vm.page_shift);
            retire_victim(vm, bh, bq, bd, rank, nlanes, active, (int)lane == L);
            if (bmode != kWriteAll) {                        /* a page that will be overwritten entirely is not fetched */
                warp_copy<8, false>(fr, vm.host + (bv << vm.page_shift), page_len(vm, bv) >> 4, rank, nlanes);
                __threadfence();
            }
            __syncwarp(active);
            if ((int)lane == L) {
                publish(vm, bv, bh, mode);                   /* step 7 */
                st = kReady; frame = bh;
            }
        }
        unsigned int pending = __ballot_sync(active, is_leader && st != kDone && st != kFail);
        if (!pending) break;
        if (__any_sync(active, progress)) { sleep_ns = 32; t_start = 0; continue; }
        /* nothing moved: back off, and give up when the bound is reached */
        unsigned long long t = now_ns();
        if (t_start == 0) t_start = t;
        bool expired = (t - t_start) > (unsigned long long)vm.spin_limit_us * 1000ull || has_error(vm);
        expired = __any_sync(active, expired);
        if (expired) {
            if (is_leader && (st == kWait || st == kOwn)) {
                set_error(vm, GPUVM_E_TIMEOUT, vpn);
                if (st == kOwn) atomicXor(pte, kBusy);        /* BUSY -> INVALID */
                unpin(pte);
                st = kFail;
            }
            continue;                                        /* READY groups still finish */
        }
        if (lane == (unsigned int)(__ffs(active) - 1)) stat_add(vm, kRetries, 1);
        __nanosleep(sleep_ns);
        if (sleep_ns < 2048) sleep_ns *= 2;
    }
    return ok;
}

template <typename T> struct always_false { static constexpr bool value = false; };

/* Shared front end: address split, grouping, optimistic pin (steps 1-3). */
template <int OP_BYTES>
__device__ __forceinline__ bool access(const gpuvm_dev_t &vm, unsigned long long byte_off, int mode,
                                       uint4 &val, Token *tok, unsigned char **ptr_out)
{
    if (byte_off + (OP_BYTES ? OP_BYTES : 1) > vm.bytes) {
        set_error(vm, GPUVM_E_RANGE, byte_off >> vm.page_shift);
        return false;
    }
    const unsigned long long vpn = byte_off >> vm.page_shift;
    const unsigned int off = (unsigned int)(byte_off & ((1ull << vm.page_shift) - 1ull));
    const unsigned int active = __activemask();
    const unsigned int group = __match_any_sync(active, vpn);
    const unsigned int leader = __ffs(group) - 1;
    const bool is_leader = lane_id() == leader;
    unsigned long long *pte = vm.pte + vpn;
    unsigned long long w = 0;
    if (is_leader) {
        w = pin_acquire(pte) + 1ull;                         /* pin first, look afterwards */
        if (group & (group - 1)) stat_add(vm, kLanes, __popc(group) - 1);
    }
    w = __shfl_sync(active, w, leader);
    unsigned int frame = (unsigned int)((w & kFrameMask) >> kFrameShift);
    /* (a counter beyond the limit is not a hit: the slow path refuses the request) */
    const bool hit = (w & kStMask) == kValid && (w & kRcMask) <= kRcLimit;
    if (__all_sync(active, hit)) {
        if (is_leader) {
            unsigned long long want = (mode != kRead ? kDirty : 0ull) |
                                      (vm.policy == GPUVM_POLICY_CLOCK ? kRef : 0ull);
            if ((w & want) != want) atomicOr(pte, want);
            if (GPUVM_COUNT_HITS) stat_add(vm, kHits, 1);
        }
        unsigned char *p = vm.pool + ((unsigned long long)frame << vm.page_shift) + off;
        if (OP_BYTES == 0) {
            *ptr_out = p;
        } else {
            if (OP_BYTES == 16) { if (mode == kWrite) st_frame16(p, val); else val = ld_frame16(p); }
            else if (OP_BYTES == 8) {
                if (mode == kWrite) asm volatile("st.relaxed.gpu.global.v2.u32 [%0], {%1,%2};" ::"l"(p), "r"(val.x), "r"(val.y) : "memory");
                else asm volatile("ld.relaxed.gpu.global.v2.u32 {%0,%1}, [%2];" : "=r"(val.x), "=r"(val.y) : "l"(p) : "memory");
            } else if (OP_BYTES == 4) {
                if (mode == kWrite) asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(val.x) : "memory");
                else asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(val.x) : "l"(p) : "memory");
            } else if (OP_BYTES == 2) {
                unsigned short hv = (unsigned short)val.x;
                if (mode == kWrite) asm volatile("st.relaxed.gpu.global.u16 [%0], %1;" ::"l"(p), "h"(hv) : "memory");
                else { asm volatile("ld.relaxed.gpu.global.u16 %0, [%1];" : "=h"(hv) : "l"(p) : "memory"); val.x = hv; }
            } else {
                if (mode == kWrite) asm volatile("st.relaxed.gpu.global.u8 [%0], %1;" ::"l"(p), "r"(val.x) : "memory");
                else asm volatile("ld.relaxed.gpu.global.u8 %0, [%1];" : "=r"(val.x) : "l"(p) : "memory");
            }
            __syncwarp(group);
            if (is_leader) unpin(pte);
        }
        if (tok) { tok->vpn = vpn; tok->group = group; tok->leader = is_leader; }
        return true;
    }
    bool ok = slow_path(vm, vpn, off, mode, OP_BYTES, active, group, w, val, frame);
    if (OP_BYTES == 0) {
        *ptr_out = ok ? vm.pool + ((unsigned long long)frame << vm.page_shift) + off : nullptr;
        if (tok) { tok->vpn = vpn; tok->group = group; tok->leader = ok && is_leader; }
    }
    return ok;
}

}  // namespace gpuvm

/* ------------------------------------------------------------------ public API */

typedef gpuvm::Token gpuvm_token;
enum { GPUVM_READ = gpuvm::kRead, GPUVM_WRITE = gpuvm::kWrite, GPUVM_WRITE_ALL = gpuvm::kWriteAll };

/* Element `elem` of an array of T that starts `base_off` bytes into the backing
 * store (Listing 1: A[i] on the right-hand side). */
template <typename T>
__device__ __forceinline__ T gpuvm_read(const gpuvm_dev_t &vm, unsigned long long elem,
                                        unsigned long long base_off = 0)
{
    static_assert(sizeof(T) == 1 || sizeof(T) == 2 || sizeof(T) == 4 || sizeof(T) == 8 || sizeof(T) == 16,
                  "element size must be 1, 2, 4, 8 or 16 bytes");
    uint4 v = make_uint4(0, 0, 0, 0);
    gpuvm::access<(int)sizeof(T)>(vm, base_off + elem * sizeof(T), gpuvm::kRead, v, nullptr, nullptr);
    T out;
    memcpy(&out, &v, sizeof(T));
    return out;
}

namespace gpuvm {
/* gpuvm_read as a call, for callers that reach it rarely and do not want its code in their loop */
template <typename T>
static __device__ __noinline__ T read_out_of_line(const gpuvm_dev_t vm, unsigned long long elem, unsigned long long base_off)
{
    return gpuvm_read<T>(vm, elem, base_off);
}
}  // namespace gpuvm

/*
 * N independent reads per lane, issued together: out[j] = element elem[j] of the array of T at base_off, for
 * j < count (count <= N may differ between lanes).  The resident case of gpuvm_read without its round trips in
 * series: every lane pins the pages of its own requests (no grouping: lanes that happen to ask for the same page
 * take one reference each), all N pins are in flight together, then the N loads, then the N unpins.  Ordering is
 * by dependency, as in the batched engine: a load's address is computed from the entry its pin returned, so it
 * is issued after the entry was seen VALID and is served by L2, where the publisher's stores already are; an
 * unpin adds a zero that is computed from the loaded value, so it is issued after the value has arrived.  (This
 * leans on the hardware executing a dependent instruction after its operands exist; the PTX memory model by
 * itself does not order relaxed operations by dependency.  With GPUVM_DEBUG_FENCED_RELEASE in vm.debug a fence
 * is placed on either side of the loads instead.)  A request whose page is not resident gives its reference
 * back, and the lanes that called together then repeat that slot through gpuvm_read, so nothing is held while
 * a frame is waited for (deadlock-free for any pool size, as gpuvm_read is).  Call it converged: `here` below
 * must name the same lanes in all of them.  Each served request counts as one hit.  T of 4, 8 or 16 bytes.
 */
template <typename T, int N>
__device__ __forceinline__ void gpuvm_read_n(const gpuvm_dev_t &vm, const unsigned long long (&elem)[N], T (&out)[N],
                                             unsigned long long base_off = 0, int count = N)
{
    using namespace gpuvm;
    static_assert(sizeof(T) == 4 || sizeof(T) == 8 || sizeof(T) == 16, "element size must be 4, 8 or 16 bytes");
    const bool fenced = (vm.debug & GPUVM_DEBUG_FENCED_RELEASE) != 0;
    unsigned long long w[N];
    unsigned int slots = 0, hits = 0;                           /* bit j: slot j holds a reference / was served */
#pragma unroll
    for (int j = 0; j < N; ++j) {
        const unsigned long long byte_off = base_off + elem[j] * sizeof(T);
        w[j] = 0;
        if (j < count && byte_off + sizeof(T) <= vm.bytes) {
            slots |= 1u << j;
            asm volatile("atom.relaxed.gpu.global.add.u64 %0, [%1], 1;" : "=l"(w[j]) : "l"(vm.pte + (byte_off >> vm.page_shift)) : "memory");
        }
    }
    if (fenced) __threadfence();
    uint4 v[N];
#pragma unroll
    for (int j = 0; j < N; ++j) {
        v[j] = make_uint4(0, 0, 0, 0);
        w[j] += 1ull;
        if (((slots >> j) & 1u) && (w[j] & kStMask) == kValid && (w[j] & kRcMask) <= kRcLimit) {
            const unsigned long long byte_off = base_off + elem[j] * sizeof(T);
            hits |= 1u << j;
            const unsigned char *p = vm.pool + (((w[j] & kFrameMask) >> kFrameShift) << vm.page_shift) +
                                     (byte_off & ((1ull << vm.page_shift) - 1ull));
            if (sizeof(T) == 16) v[j] = ld_frame16(p);
            else if (sizeof(T) == 8) asm volatile("ld.relaxed.gpu.global.v2.u32 {%0,%1}, [%2];" : "=r"(v[j].x), "=r"(v[j].y) : "l"(p) : "memory");
            else asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v[j].x) : "l"(p) : "memory");
        }
    }
    if (fenced) __threadfence();
#pragma unroll
    for (int j = 0; j < N; ++j)
        if ((slots >> j) & 1u) {
            unsigned long long *pte = vm.pte + ((base_off + elem[j] * sizeof(T)) >> vm.page_shift);
            if (((hits >> j) & 1u) && vm.policy == GPUVM_POLICY_CLOCK && !(w[j] & kRef)) atomicOr(pte, kRef);
            /* zero, but not before v[j] exists (n_frames < 2^31) */
            const unsigned long long hold = (unsigned long long)(v[j].x & (vm.n_frames >> 31));
            asm volatile("red.relaxed.gpu.global.add.u64 [%0], %1;" ::"l"(pte), "l"(~0ull + hold) : "memory");
        }
    if (GPUVM_COUNT_HITS && hits) {
        /* one counter update per warp instruction: the lowest lane adds up what the lanes with it served */
        const unsigned int active = __activemask();
        const unsigned int n = __reduce_add_sync(active, (unsigned int)__popc(hits));
        if (lane_id() == (unsigned int)__ffs(active) - 1u) stat_add(vm, kHits, n);
    }
    /* Slots that were not served (absent, in transit, out of range) take the full path.  All lanes that came in
     * together go there together, the served ones too: the warp that faults copies the page with the lanes it
     * has, and a few stragglers on their own would move a page sixteen bytes at a time. */
    const unsigned int here = __activemask();
#pragma unroll
    for (int j = 0; j < N; ++j) {
        const bool missed = j < count && !((hits >> j) & 1u);
        if ((hits >> j) & 1u) memcpy(&out[j], &v[j], sizeof(T));
        if (__any_sync(here, missed) && j < count) out[j] = gpuvm::read_out_of_line<T>(vm, elem[j], base_off);
    }
}

/* A[i] = value (Listing 1, left-hand side).  A write miss fetches the page first. */
template <typename T>
__device__ __forceinline__ void gpuvm_write(const gpuvm_dev_t &vm, unsigned long long elem, T value,
                                            unsigned long long base_off = 0)
{
    static_assert(sizeof(T) == 1 || sizeof(T) == 2 || sizeof(T) == 4 || sizeof(T) == 8 || sizeof(T) == 16,
                  "element size must be 1, 2, 4, 8 or 16 bytes");
    uint4 v = make_uint4(0, 0, 0, 0);
    memcpy(&v, &value, sizeof(T));
    gpuvm::access<(int)sizeof(T)>(vm, base_off + elem * sizeof(T), gpuvm::kWrite, v, nullptr, nullptr);
}

/* Pin the page that holds `byte_off` and return the address of that byte inside
 * its frame, valid up to the end of the page until gpuvm_release(token).
 * mode GPUVM_WRITE marks the page dirty.  GPUVM_WRITE_ALL is a promise that the caller
 * overwrites every byte of the page that lies inside the backing store before it releases
 * the page: a missing page is then given a frame without being fetched from the host (its
 * old contents would be overwritten anyway).  The page must stay pinned from this call to
 * gpuvm_release for the whole overwrite; whoever reads it meanwhile sees unspecified bytes.
 * nullptr after an error. */
__device__ __forceinline__ void *gpuvm_ptr(const gpuvm_dev_t &vm, unsigned long long byte_off, int mode,
                                           gpuvm_token *token)
{
    uint4 v;
    unsigned char *p = nullptr;
    token->leader = 0; token->group = 0; token->vpn = 0;
    gpuvm::access<0>(vm, byte_off, mode, v, token, &p);
    return p;
}

/*
 * gpuvm_ptr in read mode for callers that want a page only if it is there already: never faults,
 * never waits.  A resident page is pinned and its frame address returned (release it with
 * gpuvm_release, as after gpuvm_ptr); for a page that is absent or in transit nullptr is returned
 * and nothing stays pinned.  Lanes that call together may ask for different pages.  Used by the
 * graph sweeps to re-expand a vertex behind the sweep position while its pages are still in the pool.
 */
__device__ __forceinline__ void *gpuvm_ptr_if_resident(const gpuvm_dev_t &vm, unsigned long long byte_off,
                                                       gpuvm_token *token)
{
    using namespace gpuvm;
    token->leader = 0; token->group = 0; token->vpn = 0;
    if (byte_off >= vm.bytes) { set_error(vm, GPUVM_E_RANGE, byte_off >> vm.page_shift); return nullptr; }
    const unsigned long long vpn = byte_off >> vm.page_shift;
    const unsigned int active = __activemask();
    const unsigned int group = __match_any_sync(active, vpn);
    const unsigned int leader = __ffs(group) - 1;
    const bool is_leader = lane_id() == leader;
    unsigned long long *pte = vm.pte + vpn;
    unsigned long long w = 0;
    if (is_leader) {
        w = guard_pin(vm, pte, pin_acquire(pte) + 1ull);
        if (w == kPinRefused) w = 0;
        else if ((w & kStMask) != kValid) { unpin(pte); w = 0; }
        else {
            if (vm.policy == GPUVM_POLICY_CLOCK && !(w & kRef)) atomicOr(pte, kRef);
            if (GPUVM_COUNT_HITS) stat_add(vm, kHits, 1);
        }
    }
    w = __shfl_sync(group, w, leader);
    if ((w & kStMask) != kValid) return nullptr;
    token->vpn = vpn; token->group = group; token->leader = is_leader;
    return vm.pool + (((w & kFrameMask) >> kFrameShift) << vm.page_shift) + (byte_off & ((1ull << vm.page_shift) - 1ull));
}

/* Called by the same lanes that called gpuvm_ptr together. */
__device__ __forceinline__ void gpuvm_release(const gpuvm_dev_t &vm, const gpuvm_token &token)
{
    if (token.group == 0) return;
    __syncwarp(token.group);
    if (token.leader) gpuvm::unpin(vm.pte + token.vpn);
}

/*
 * Eager write-back: copy the page pinned by `token` to the host now and mark it clean, so
 * that its later eviction costs nothing and no fault has to wait for a write-back (the
 * paper names synchronous write-back on the fault path as its weak spot, Section 5.3).
 * Called by the lanes that pinned the page together (token.group), converged, before
 * gpuvm_release; `p` is any address inside the page's frame.  The dirty bit is cleared
 * before the copy starts, so a writer that pins the page after that marks it dirty again and
 * it is written back once more later.  A writer that pinned the page BEFORE the call and
 * stores during or after the copy is not covered (its pin saw the dirty bit already set and
 * did not set it again): clean only pages whose writers have all released them, or that
 * the calling warp alone writes, as the vector add does.
 */
__device__ __forceinline__ void gpuvm_clean(const gpuvm_dev_t &vm, const gpuvm_token &token, const void *p)
{
    if (token.group == 0 || p == nullptr) return;
    const unsigned int lane = gpuvm::lane_id();
    const unsigned int rank = __popc(token.group & ((1u << lane) - 1u)), n = __popc(token.group);
    unsigned long long *pte = vm.pte + token.vpn;
    __syncwarp(token.group);                                   /* the group's stores to the frame are done */
    bool dirty = false;
    if (token.leader) dirty = (atomicAnd(pte, ~gpuvm::kDirty) & gpuvm::kDirty) != 0ull;
    dirty = __shfl_sync(token.group, (int)dirty, __ffs(token.group) - 1);
    if (!dirty) return;
    const unsigned long long frame = (unsigned long long)(static_cast<const unsigned char *>(p) - vm.pool) >> vm.page_shift;
    const unsigned int len = gpuvm::page_len(vm, token.vpn);
    gpuvm::warp_copy<8, true>(vm.host + (token.vpn << vm.page_shift), vm.pool + (frame << vm.page_shift), len >> 4, rank, n);
    __threadfence_system();
    __syncwarp(token.group);
    if (token.leader) {
        gpuvm::stat_add(vm, gpuvm::kWritebacks, 1);
        gpuvm::stat_add(vm, gpuvm::kBytesOut, len);
    }
}

/*
 * Prefetch: if the page that holds `byte_off` is neither resident nor being fetched, the
 * calling lanes (which must all pass the same offset) fetch it now and leave it resident,
 * unpinned, with its reference bit set; otherwise they return at once.  Used by sweeps to
 * fetch pages ahead of the window in which all warps work: without it every warp of the
 * window waits for the same few pages and only those few are in flight on the link.  Gives
 * up quietly (page left INVALID) when no frame is free after a few ring slots.
 */
static __device__ __noinline__ void gpuvm_prefetch(const gpuvm_dev_t vm, unsigned long long byte_off)
{
    using namespace gpuvm;
    if (byte_off >= vm.bytes) return;
    const unsigned long long vpn = byte_off >> vm.page_shift;
    const unsigned int active = __activemask();
    const unsigned int lane = lane_id(), L = __ffs(active) - 1;
    const unsigned int rank = __popc(active & ((1u << lane) - 1u)), n = __popc(active);
    unsigned long long *pte = vm.pte + vpn;
    int go = 0;
    unsigned int h = 0;
    unsigned long long victim = ~0ull;
    bool vdirty = false;
    if (lane == L) {
        const unsigned long long w = ld_relaxed_u64(pte);
        if ((w & kStMask) == kInvalid && atomicCAS(pte, w, (w & ~kFrameMask) | kBusy) == w) {
            go = try_claim(vm, vpn, 8, h, victim, vdirty, /* allow_dirty = */ false) ? 1 : 0;
            if (!go) atomicXor(pte, kBusy);                       /* no frame at hand: BUSY -> INVALID */
        }
    }
    if (!__shfl_sync(active, go, L)) return;
    const unsigned int bh = __shfl_sync(active, h, L);
    const unsigned long long bq = __shfl_sync(active, victim, L);
    const int bd = __shfl_sync(active, (int)vdirty, L);
    unsigned char *fr = vm.pool + ((unsigned long long)bh << vm.page_shift);
    retire_victim(vm, bh, bq, bd, rank, n, active, lane == L);
    warp_copy<8, false>(fr, vm.host + (vpn << vm.page_shift), page_len(vm, vpn) >> 4, rank, n);
    __threadfence();
    __syncwarp(active);
    if (lane == L) publish(vm, vpn, bh, kRead);
}

/* Frame memory accessors (L1-bypassing, device-coherent). */
__device__ __forceinline__ uint4 gpuvm_load16(const void *p) { return gpuvm::ld_frame16(p); }
__device__ __forceinline__ void gpuvm_store16(void *p, uint4 v) { gpuvm::st_frame16(p, v); }

template <typename T>
__device__ __forceinline__ T gpuvm_load(const T *p)
{
    static_assert(sizeof(T) == 4 || sizeof(T) == 8, "4- or 8-byte elements");
    T out;
    if (sizeof(T) == 4) {
        unsigned int v;
        asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
        memcpy(&out, &v, 4);
    } else {
        unsigned long long v;
        asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
        memcpy(&out, &v, 8);
    }
    return out;
}

template <typename T>
__device__ __forceinline__ void gpuvm_store(T *p, T value)
{
    static_assert(sizeof(T) == 4 || sizeof(T) == 8, "4- or 8-byte elements");
    if (sizeof(T) == 4) {
        unsigned int v;
        memcpy(&v, &value, 4);
        asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
    } else {
        unsigned long long v;
        memcpy(&v, &value, 8);
        asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
    }
}

#endif /* GPUVM_DEVICE_CUH */
