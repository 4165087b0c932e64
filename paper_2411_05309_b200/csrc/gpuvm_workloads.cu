// Workload kernels written against the device accessors, plus the same kernels on
// plain pointers.  Each kernel is a template over a memory policy: Paged goes
// through the page table, Raw dereferences ordinary device-accessible memory.
#include <cuda_runtime.h>

#include <atomic>
#include <chrono>
#include <cstdint>
#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "gpuvm.h"
#include "gpuvm_batch.cuh"
#include "gpuvm_device.cuh"
#include "gpuvm_internal.h"
#include "gpuvm_workloads.h"

namespace {

std::atomic<unsigned long long> g_launches{0};

struct Paged {
    static constexpr int kSweepBlocksPerSm = 4;
    static constexpr bool kBehindQueue = true;
    gpuvm_dev_t vm;
    unsigned long long edges_hint = 0;
    __device__ __forceinline__ unsigned long long unit() const { return 1ull << vm.page_shift; }
    // what one lane group of a streaming kernel takes at a time: large pages are shared out in 64 KiB pieces
    // (one pin per piece), so that a few hundred pages still occupy the whole grid
    __device__ __forceinline__ unsigned long long stream_unit() const { return vm.page_shift > 16 ? 65536ull : 1ull << vm.page_shift; }
    // Host side.  Is it cheaper to read `vertices` scattered neighbour lists in place (about 256 bytes on the link
    // each: two row offsets, a short list, each rounded up to a 128-byte read) than to fetch the pages a full
    // sweep would miss (what does not fit the pool)?
    // Host side.  How many pages (at most `want`) may each of `warps` warps hold pinned at the same time?
    int pins_per_warp(int warps, int want) const
    {
        int g = want;
        while (g > 1 && (unsigned long long)warps * g > vm.n_frames) g >>= 1;
        return g;
    }
    bool sparse_sweep(unsigned long long vertices) const
    {
        const unsigned long long missing = vm.n_pages > vm.n_frames ? vm.n_pages - vm.n_frames : 0ull;
        return vertices * 256ull < (missing << vm.page_shift);
    }
    template <typename T>
    __device__ __forceinline__ T read(unsigned long long base, unsigned long long i) const { return gpuvm_read<T>(vm, i, base); }
    template <typename T, int N>
    __device__ __forceinline__ void read_n(unsigned long long base, const unsigned long long (&i)[N], T (&out)[N], int count) const
    {
        gpuvm_read_n<T, N>(vm, i, out, base, count);
    }
    template <typename T>
    __device__ __forceinline__ void write(unsigned long long base, unsigned long long i, T v) const { gpuvm_write<T>(vm, i, v, base); }
    __device__ __forceinline__ unsigned char *pin(unsigned long long off, int mode, gpuvm_token &t) const
    {
        return static_cast<unsigned char *>(gpuvm_ptr(vm, off, mode, &t));
    }
    __device__ __forceinline__ unsigned char *pin_if_resident(unsigned long long off, gpuvm_token &t) const
    {
        return static_cast<unsigned char *>(gpuvm_ptr_if_resident(vm, off, &t));
    }
    // The backing-store copy of a byte, read in place over the link.  Current for arrays that are not written
    // through the runtime during the launch (the graph arrays never are).
    __device__ __forceinline__ const unsigned char *through(unsigned long long off) const { return vm.host + off; }
    __device__ __forceinline__ void note_direct(unsigned long long bytes) const { gpuvm::stat_add(vm, gpuvm::kBytesDirect, bytes); }
    __device__ __forceinline__ void release(const gpuvm_token &t) const { gpuvm_release(vm, t); }
    __device__ __forceinline__ void clean(const gpuvm_token &t, const void *p) const { gpuvm_clean(vm, t, p); }
    __device__ __forceinline__ void prefetch(unsigned long long off) const { gpuvm_prefetch(vm, off); }
    __device__ __forceinline__ unsigned long long wait_ns() const { return (unsigned long long)vm.spin_limit_us * 1000ull; }
    __device__ __forceinline__ void wait_ran_out(unsigned long long where) const { gpuvm::set_error(vm, GPUVM_E_TIMEOUT, where); }
    static __device__ __forceinline__ uint4 load16(const void *p) { return gpuvm_load16(p); }
    static __device__ __forceinline__ void store16(void *p, uint4 v) { gpuvm_store16(p, v); }
    static __device__ __forceinline__ int load_i32(const void *p) { return gpuvm_load(static_cast<const int *>(p)); }
    static __device__ __forceinline__ long long load_i64(const void *p) { return gpuvm_load(static_cast<const long long *>(p)); }
};

struct Raw {
    static constexpr int kSweepBlocksPerSm = 2;
    static constexpr bool kBehindQueue = false;
    unsigned char *base;
    unsigned long long unit_bytes;
    unsigned long long edges_hint = 0;
    __device__ __forceinline__ unsigned long long unit() const { return unit_bytes; }
    __device__ __forceinline__ unsigned long long stream_unit() const { return unit_bytes; }
    int pins_per_warp(int, int) const { return 1; }
    bool sparse_sweep(unsigned long long) const { return false; }
    template <typename T>
    __device__ __forceinline__ T read(unsigned long long off, unsigned long long i) const { return reinterpret_cast<const T *>(base + off)[i]; }
    template <typename T, int N>
    __device__ __forceinline__ void read_n(unsigned long long off, const unsigned long long (&i)[N], T (&out)[N], int count) const
    {
#pragma unroll
        for (int j = 0; j < N; ++j)
            if (j < count) out[j] = reinterpret_cast<const T *>(base + off)[i[j]];
    }
    template <typename T>
    __device__ __forceinline__ void write(unsigned long long off, unsigned long long i, T v) const { reinterpret_cast<T *>(base + off)[i] = v; }
    __device__ __forceinline__ unsigned char *pin(unsigned long long off, int, gpuvm_token &) const { return base + off; }
    __device__ __forceinline__ unsigned char *pin_if_resident(unsigned long long off, gpuvm_token &) const { return base + off; }
    __device__ __forceinline__ const unsigned char *through(unsigned long long off) const { return base + off; }
    __device__ __forceinline__ void note_direct(unsigned long long) const {}
    __device__ __forceinline__ void release(const gpuvm_token &) const {}
    __device__ __forceinline__ void clean(const gpuvm_token &, const void *) const {}
    __device__ __forceinline__ void prefetch(unsigned long long) const {}
    __device__ __forceinline__ unsigned long long wait_ns() const { return 10000000000ull; }
    __device__ __forceinline__ void wait_ran_out(unsigned long long) const {}
    static __device__ __forceinline__ uint4 load16(const void *p) { return *static_cast<const uint4 *>(p); }
    static __device__ __forceinline__ void store16(void *p, uint4 v) { *static_cast<uint4 *>(p) = v; }
    static __device__ __forceinline__ int load_i32(const void *p) { return *static_cast<const int *>(p); }
    static __device__ __forceinline__ long long load_i64(const void *p) { return *static_cast<const long long *>(p); }
};

__device__ __forceinline__ unsigned int warp_in_grid() { return (blockIdx.x * blockDim.x + threadIdx.x) >> 5; }
__device__ __forceinline__ unsigned int warps_in_grid() { return (gridDim.x * blockDim.x) >> 5; }

// ------------------------------------------------------------- streaming sum
// G units (pages) per warp at a time, 32 / G lanes each: the G pins are issued together, so the round trip of
// the translation is paid once per G pages, and every lane group streams its own page.
template <class Mem, int G>
__global__ void __launch_bounds__(256) stream_sum_kernel(Mem m, unsigned long long a_off, unsigned long long n,
                                                         unsigned long long *out)
{
    constexpr unsigned int L = 32 / G;                            // lanes per page
    const unsigned int lane = threadIdx.x & 31, sub = lane / L, sl = lane % L;
    const unsigned long long unit = m.stream_unit();             // a page, or a 64 KiB piece of a larger one
    const unsigned long long start = a_off, end = a_off + 4ull * n;
    const unsigned long long first = start / unit, units = (end + unit - 1) / unit - first;
    long long acc = 0;
    for (unsigned long long u0 = (unsigned long long)warp_in_grid() * G; u0 < units; u0 += (unsigned long long)warps_in_grid() * G) {
        const unsigned long long u = u0 + sub;
        if (u >= units) continue;
        unsigned long long lo = (first + u) * unit, hi = lo + unit;
        if (lo < start) lo = start;
        if (hi > end) hi = end;
        gpuvm_token tok;
        const unsigned char *p = m.pin(lo, GPUVM_READ, tok);
        if (!p) continue;
        const unsigned int len = (unsigned int)(hi - lo), n16 = len >> 4;
#pragma unroll 8
        for (unsigned int i = sl; i < n16; i += L) {
            uint4 v = Mem::load16(p + 16ull * i);
            acc += (long long)(int)v.x + (long long)(int)v.y + (long long)(int)v.z + (long long)(int)v.w;
        }
        const unsigned int tail = (len & 15u) >> 2;
        if (sl < tail) acc += (long long)Mem::load_i32(p + 16ull * n16 + 4u * sl);
        m.release(tok);
    }
    __syncwarp();
    for (int o = 16; o; o >>= 1) acc += __shfl_down_sync(0xFFFFFFFFu, acc, o);
    if (lane == 0 && acc != 0) atomicAdd(out, (unsigned long long)acc);
}

// -------------------------------------------------------------- random gather
// One request per lane and slot, kGatherSlots slots at a time (gpuvm_read_n): a thread block adds up one index
// block at a time.
// Two blocks of 256 threads per SM at up to 128 registers: with four blocks at 64 registers the loop spills and
// a resident gather is a quarter slower (23.8 against 31.8 G accesses/s), the cold one the same.
constexpr int kGatherSlots = 4;
constexpr int kGatherPlainBlocksPerSm = 2;
template <class Mem>
__global__ void __launch_bounds__(256, kGatherPlainBlocksPerSm) gather_kernel(Mem m, unsigned long long x_off, const long long *__restrict__ idx,
                                                        unsigned long long n_idx, unsigned long long block,
                                                        float *__restrict__ fsum, long long *__restrict__ bsum)
{
    __shared__ double s_f[8];
    __shared__ long long s_b[8];
    const unsigned int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned long long nb = (n_idx + block - 1) / block;
    for (unsigned long long b = blockIdx.x; b < nb; b += gridDim.x) {
        const unsigned long long lo = b * block;
        const unsigned long long hi = lo + block < n_idx ? lo + block : n_idx;
        double f = 0.0;
        long long bits = 0;
        for (unsigned long long k = lo + threadIdx.x; k < hi; k += (unsigned long long)kGatherSlots * blockDim.x) {
            unsigned long long e[kGatherSlots];
            float v[kGatherSlots];
            int count = 0;
#pragma unroll
            for (int j = 0; j < kGatherSlots; ++j) {
                const unsigned long long kj = k + (unsigned long long)j * blockDim.x;
                e[j] = kj < hi ? (unsigned long long)idx[kj] : 0ull;
                count += kj < hi;
            }
            m.template read_n<float, kGatherSlots>(x_off, e, v, count);
#pragma unroll
            for (int j = 0; j < kGatherSlots; ++j)
                if (j < count) { f += (double)v[j]; bits += (long long)__float_as_uint(v[j]); }
        }
        __syncwarp();
        for (int o = 16; o; o >>= 1) {
            f += __shfl_down_sync(0xFFFFFFFFu, f, o);
            bits += __shfl_down_sync(0xFFFFFFFFu, bits, o);
        }
        if (lane == 0) { s_f[warp] = f; s_b[warp] = bits; }
        __syncthreads();
        if (warp == 0) {
            const unsigned int nw = blockDim.x >> 5;
            f = lane < nw ? s_f[lane] : 0.0;
            bits = lane < nw ? s_b[lane] : 0;
            for (int o = 4; o; o >>= 1) {
                f += __shfl_down_sync(0xFFFFFFFFu, f, o);
                bits += __shfl_down_sync(0xFFFFFFFFu, bits, o);
            }
            if (lane == 0) { fsum[b] = (float)f; bsum[b] = bits; }
        }
        __syncthreads();
    }
}

// A requester warp takes a run of consecutive indices (whole index blocks when they fit) and
// registers them all in the page table (gpuvm_batch.cuh).  Table form: their element indices are
// staged in the warp's request table (handle-owned device scratch), each index is replaced by the
// value it asked for as the pages arrive, and the values are added up block by block afterwards.
// Direct form: see the template parameter below.  The faults a warp owns go to the thread block's
// ring of page ids in shared memory, which the block's migrator warps serve.  No block-wide barrier
// after start-up: warps never wait for one another.
constexpr int kGatherRequesters = 28;
constexpr int kGatherMigrators = 4;
constexpr int kGatherMaxWarps = 32;
constexpr unsigned int kGatherBatch = 16384;             // most requests per requester warp: 512 rows of 32
constexpr unsigned int kNoIndex = 0xFFFFFFFFu;
constexpr unsigned int kGatherChunk = 8192;              // bytes per bulk copy of a migrator warp
constexpr unsigned int kGatherStages = 1;                // staging buffers per migrator warp (more in flight only delays each page)

// Request table of the gather: one 32-bit element index per request (the array has fewer than
// 2^32 - 1 elements), replaced by the value's bit pattern when the request is served.
struct GatherTable {
    unsigned int *e;
    unsigned long long x_off;
    unsigned int page_shift;
    __device__ __forceinline__ bool valid(unsigned int i) const { return e[i] != kNoIndex; }
    __device__ __forceinline__ unsigned int vpn(unsigned int i) const { return (unsigned int)((x_off + 4ull * e[i]) >> page_shift); }
    __device__ __forceinline__ unsigned int off(unsigned int i) const
    {
        return (unsigned int)((x_off + 4ull * e[i]) & ((1ull << page_shift) - 1ull));
    }
};

// The index list itself as the request table (no copy): request i of a piece is idx[i].
struct GatherIndexTable {
    const long long *idx;
    unsigned long long x_off, n_elems;
    gpuvm_dev_t vm;
    __device__ __forceinline__ bool valid(unsigned int i) const
    {
        const unsigned long long e = (unsigned long long)idx[i];
        if (e >= n_elems) gpuvm::set_error(vm, GPUVM_E_RANGE, (x_off + 4 * e) >> vm.page_shift);
        return e < n_elems;
    }
    __device__ __forceinline__ unsigned int vpn(unsigned int i) const { return (unsigned int)((x_off + 4ull * (unsigned long long)idx[i]) >> vm.page_shift); }
    __device__ __forceinline__ unsigned int off(unsigned int i) const
    {
        return (unsigned int)((x_off + 4ull * (unsigned long long)idx[i]) & ((1ull << vm.page_shift) - 1ull));
    }
};

constexpr unsigned int kGatherAcc = 64;                  // index blocks a requester warp sums at a time without a table
constexpr unsigned int kGatherDirectMinBlock = kGatherBatch / kGatherAcc;

// DIRECT: the requests are read from the index list in place and every value is added to the sums of
// its index block as it is gathered (shared-memory accumulators, double and int64): no request table,
// no scratch.  Needs index blocks of at least kGatherDirectMinBlock.  The double sum is then taken in
// the order of arrival; its float rounding is the oracle's unless the sum lies within 1e-13 of a
// rounding boundary.
template <bool DIRECT>
__global__ void __launch_bounds__(kGatherMaxWarps * 32, 1) gather_batch_kernel(gpuvm_dev_t vm, unsigned long long x_off,
                                                                               const long long *__restrict__ idx,
                                                                               unsigned long long n_idx, unsigned long long block,
                                                                               float *__restrict__ fsum, long long *__restrict__ bsum,
                                                                               int requesters, unsigned int batch,
                                                                               unsigned int *g_tables, unsigned int stage_chunk,
                                                                               unsigned int stage_count, bool one_pass,
                                                                               gpuvm_shared_queue *shared_queue)
{
    __shared__ gpuvm_fault_queue queue_s;
    // dynamic: per requester warp its mask words x 32 lanes; per migrator warp its staging
    // buffers for the bulk copies; the mbarriers of those
    extern __shared__ __align__(128) unsigned long long gather_masks[];
    gpuvm_fault_queue *queue = &queue_s;
    const unsigned int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (unsigned int k = threadIdx.x; k < sizeof(gpuvm_fault_queue) / 4; k += blockDim.x)
        reinterpret_cast<unsigned int *>(queue)[k] = 0;
    __syncthreads();
    if (threadIdx.x == 0) { queue->requesters = (unsigned int)requesters; queue->shared = shared_queue; }
    __syncthreads();
    if ((int)warp >= requesters) {
        const unsigned int mig = warp - requesters, n_mig = (blockDim.x >> 5) - requesters;
        unsigned char *stage0 = reinterpret_cast<unsigned char *>(gather_masks + (size_t)requesters * gpuvm_batch_mask_words(batch) * 32);
        unsigned long long *mbar0 = reinterpret_cast<unsigned long long *>(stage0 + (size_t)n_mig * stage_count * stage_chunk);
        gpuvm_migrator_loop(vm, queue, stage_count ? stage0 + (size_t)mig * stage_count * stage_chunk : nullptr,
                            mbar0 + (size_t)mig * stage_count, stage_chunk, stage_count);
        return;
    }
    unsigned long long *masks = gather_masks + (size_t)warp * gpuvm_batch_mask_words(batch) * 32 + lane;
    unsigned int *table = DIRECT ? nullptr : g_tables + ((size_t)blockIdx.x * requesters + warp) * batch;
    // DIRECT: this warp's accumulators, behind the masks, the staging buffers and their mbarriers
    const unsigned int n_mig_w = (blockDim.x >> 5) - requesters;
    unsigned char *acc0 = reinterpret_cast<unsigned char *>(gather_masks + (size_t)requesters * gpuvm_batch_mask_words(batch) * 32) +
                          (size_t)n_mig_w * stage_count * (stage_chunk + sizeof(unsigned long long));
    double *acc_f = reinterpret_cast<double *>(acc0) + (size_t)warp * 2 * kGatherAcc;
    unsigned long long *acc_b = reinterpret_cast<unsigned long long *>(acc_f + kGatherAcc);
    const unsigned long long n_elems = (vm.bytes - x_off) / 4;
    const unsigned long long nb = (n_idx + block - 1) / block;
    const unsigned long long per = block <= batch ? batch / block : 1;      // index blocks per work item
    const unsigned long long items = (nb + per - 1) / per;
    const unsigned long long stride = (unsigned long long)gridDim.x * requesters;
    for (unsigned long long t = (unsigned long long)blockIdx.x * requesters + warp; t < items; t += stride) {
        const unsigned long long lo = t * per * block;
        const unsigned long long hi = (t + 1) * per * block < n_idx ? (t + 1) * per * block : n_idx;
        double carry_f = 0.0;               // a block longer than one batch is summed piece by piece
        long long carry_b = 0;
        for (unsigned long long base = lo; base < hi; base += batch) {
            const unsigned int n = (unsigned int)(hi - base < batch ? hi - base : batch);
            if constexpr (DIRECT) {
                // blocks of this piece: whole ones (block <= batch: pieces start on a block boundary) or a part of one
                const unsigned int nblk = block <= batch ? (unsigned int)((n + block - 1) / block) : 1u;
                const unsigned int blk32 = (unsigned int)block;
                for (unsigned int k = lane; k < nblk; k += 32) { acc_f[k] = 0.0; acc_b[k] = 0ull; }
                __syncwarp();
                gpuvm_batch_run<false>(vm, GatherIndexTable{idx + base, x_off, n_elems, vm}, n, GPUVM_READ,
                                       [=](unsigned int i, const unsigned char *p) {
                                           const unsigned int v = gpuvm_load(reinterpret_cast<const unsigned int *>(p));
                                           const unsigned int k = nblk > 1 ? i / blk32 : 0u;
                                           atomicAdd(acc_f + k, (double)__uint_as_float(v));
                                           atomicAdd(acc_b + k, (unsigned long long)v);
                                           return v;              // read-only consume: lets the engine skip its fence
                                       }, queue, masks, 32u, one_pass);
                __syncwarp();
                if (block <= batch) {
                    for (unsigned int k = lane; k < nblk; k += 32) {
                        fsum[base / block + k] = (float)acc_f[k];
                        bsum[base / block + k] = (long long)acc_b[k];
                    }
                } else {                                          // one long block, piece by piece
                    carry_f += acc_f[0];
                    carry_b += (long long)acc_b[0];
                    if (base + n == hi) {
                        if (lane == 0) { fsum[base / block] = (float)carry_f; bsum[base / block] = carry_b; }
                        carry_f = 0.0;
                        carry_b = 0;
                    }
                }
                __syncwarp();
            } else {
            for (unsigned int k = lane; k < n; k += 32) {
                const unsigned long long i = (unsigned long long)idx[base + k];
                if (i >= n_elems) gpuvm::set_error(vm, GPUVM_E_RANGE, (x_off + 4 * i) >> vm.page_shift);
                table[k] = i < n_elems ? (unsigned int)i : kNoIndex;
            }
            __syncwarp();
            gpuvm_batch_run<false>(vm, GatherTable{table, x_off, vm.page_shift}, n, GPUVM_READ,
                                   [table](unsigned int i, const unsigned char *p) {
                                       const unsigned int v = gpuvm_load(reinterpret_cast<const unsigned int *>(p));
                                       table[i] = v;
                                       return v;                  // read-only consume: lets the engine skip its fence
                                   }, queue, masks, 32u, one_pass);
            __syncwarp();
            // sum the values of this piece, index block by index block (a rejected index left
            // kNoIndex in its slot and has set the sticky error: the sums are then meaningless)
            unsigned long long pos = base;
            while (pos < base + n) {
                const unsigned long long b = pos / block;
                unsigned long long end = (b + 1) * block;
                if (end > base + n) end = base + n;
                double f = 0.0;
                long long bits = 0;
                for (unsigned long long k = pos + lane; k < end; k += 32) {
                    const unsigned int v = table[k - base];
                    f += (double)__uint_as_float(v);
                    bits += (long long)v;
                }
                for (int o = 16; o; o >>= 1) {
                    f += __shfl_down_sync(0xFFFFFFFFu, f, o);
                    bits += __shfl_down_sync(0xFFFFFFFFu, bits, o);
                }
                carry_f += f;
                carry_b += bits;
                if (end == (b + 1) * block || end == n_idx) {    // the index block is complete
                    if (lane == 0) { fsum[b] = (float)carry_f; bsum[b] = carry_b; }
                    carry_f = 0.0;
                    carry_b = 0;
                }
                pos = end;
            }
            __syncwarp();
            }   // table path
        }
    }
    if (lane == 0) gpuvm_requester_done(queue);
}

// ------------------------------------------------------- graph sweeps (BFS, CC, SSSP)
constexpr long long kBigDegree = 4096;     // neighbour lists at least this long are spread over the grid
constexpr unsigned int kBigQueue = 65536;  // entries of the span queue (four int64 each: first edge, end, vertex, -)
constexpr unsigned int kChunksPerTicket = 2;  // consecutive chunks of 32 vertices a warp draws at a time
constexpr unsigned int kSpanPoll = 4;       // a warp looks into the span queue before every kSpanPoll-th chunk
constexpr long long kAhead = 16;           // pages of look-ahead of the sweeps' prefetches
constexpr unsigned int kNoVertex = 0xFFFFFFFFu;

// counters of a sweep, each in a 128-byte line of its own (the chunk ticket is hit by every warp all
// the time; a load of a word in the same line would queue behind those atomics)
constexpr int kCntUpdates = 0;       // updates made in this sweep
constexpr int kCntPushed = 32;       // span queue entries reserved
constexpr int kCntTicket = 64;       // chunk ticket
constexpr int kCntTaken = 96;        // span ticket
constexpr int kCntDone = 128;        // chunks finished
constexpr int kCntBehindTail = 160;  // entries reserved in the queue of vertices that changed behind the sweep position
constexpr int kCntBehindHead = 192;  // entries of that queue taken
constexpr int kCntMax = 224;         // largest label (written by the finishing kernel)
constexpr int kCntWords = 256;

// What a sweep does with a vertex and with each of its edges.
//   active(v)   does the sweep expand v?
//   begin(v)    called once by the lane that owns an active v before its edges are visited; returns the
//               value of v that its edges are visited with
//   value(u)    the same value without side effects (for pieces of a long list that are expanded later)
//   peek(c)     what the edge's other end holds now (a plain load: several edges' peeks are issued together)
//   edge(...)   decides and updates; returns 1 when it changed something.  `pos` is how far the sweep has
//               got (in chunks, in sweep order), for operations that care what lies behind it
struct BfsOp {                              // level-synchronous BFS: expand the vertices of the current level
    static constexpr bool kBehind = false;
    int *level;
    int depth;
    __device__ __forceinline__ bool active(unsigned long long v) const { return level[v] == depth; }
    __device__ __forceinline__ int begin(unsigned long long) const { return depth; }
    __device__ __forceinline__ int value(unsigned long long) const { return depth; }
    __device__ __forceinline__ int peek(int c) const { return level[c]; }
    __device__ __forceinline__ unsigned int edge(int, long long, int c, int, int seen, unsigned int) const
    {
        return seen == -1 && atomicCAS(level + c, -1, depth + 1) == -1;
    }
};

// Connected components by concurrent union-find in ONE pass over the edges (the lock-free scheme of
// Anderson and Woll as used by ECL-CC): parent[] starts as the identity; for every edge the roots of its
// two ends are found (with path halving) and the larger root is hooked under the smaller one with a
// compare-and-swap that only succeeds while it still is a root.  Parents only ever decrease, so the root
// of a tree is the smallest vertex in it; a finishing kernel replaces every parent by its root.
struct CcOp {
    static constexpr bool kBehind = false;
    int *parent;
    __device__ __forceinline__ static int ld(const int *p) { return __ldcg(p); }
    __device__ __forceinline__ int find(int x) const
    {
        int p = ld(parent + x);
        while (p != x) {
            const int gp = ld(parent + p);
            if (gp != p) parent[x] = gp;                 // path halving: any ancestor is a valid parent
            x = p;
            p = gp;
        }
        return x;
    }
    __device__ __forceinline__ int find_read_only(int x) const
    {
        for (int p = ld(parent + x); p != x; p = ld(parent + x)) x = p;
        return x;
    }
    __device__ __forceinline__ bool active(unsigned long long) const { return true; }
    __device__ __forceinline__ int begin(unsigned long long v) const { return (int)v; }
    __device__ __forceinline__ int value(unsigned long long u) const { return (int)u; }
    __device__ __forceinline__ int peek(int c) const { return ld(parent + c); }
    __device__ __forceinline__ unsigned int edge(int, long long u, int c, int, int pc, unsigned int) const
    {
        int ra = find((int)u), rb = pc == c ? c : find(pc);
        while (ra != rb) {
            if (ra < rb) { const int t = ra; ra = rb; rb = t; }          // ra is the larger root: it goes under rb
            const int old = atomicCAS(parent + ra, ra, rb);
            if (old == ra) return 1;
            ra = find(old);                                              // ra was no longer a root
            rb = find(rb);
        }
        return 0;
    }
};

// Label-correcting relaxation: BFS (every edge has length 1) and SSSP (edge weights).  dist[v] holds
// (distance << 1) | dirty.  A vertex is expanded when its dirty bit is set; expanding clears the bit with
// an atomic AND whose return value is the distance the edges are relaxed with; lowering a distance is an
// atomicMin with the bit set, so whoever is lowered is expanded (again) later.  The fixed point is the
// shortest distance.  One sweep carries as many hops as the order of the vertices allows, and a vertex
// that is lowered BEHIND the sweep position goes to a queue from which idle moments of all warps
// re-expand it in the same sweep, provided its pages are still resident (no fault is taken for it;
// otherwise it simply stays dirty for the next sweep).  Level-synchronous sweeps fetch most of the graph
// once per level; this way almost every page is fetched once per run.
constexpr int kLcInf = 0x7FFFFFFE;          // unreached, not dirty
template <bool WEIGHTED>
struct LcOp {
    static constexpr bool kBehind = true;
    int *dist;
    unsigned int *behind_q;                 // vertex numbers, kNoVertex = not written yet
    unsigned int *counters;
    unsigned int behind_cap, n_chunks;
    int backward;
    unsigned int only;                      // kNoVertex, or the one vertex this sweep expands (the first sweep: the source)
    int through_main;                       // a sparse sweep: pages that are not resident are read in place, not fetched
    __device__ __forceinline__ bool active(unsigned long long v) const
    {
        return only == kNoVertex ? (__ldcg(dist + v) & 1) != 0 : v == only;
    }
    __device__ __forceinline__ int begin(unsigned long long v) const { return atomicAnd(dist + v, ~1) >> 1; }
    __device__ __forceinline__ void redirty(unsigned long long v) const { atomicOr(dist + v, 1); }
    __device__ __forceinline__ int value(unsigned long long u) const { return __ldcg(dist + u) >> 1; }
    __device__ __forceinline__ int peek(int c) const { return dist[c]; }
    // could an edge of weight >= 0 from a vertex at distance du lower a vertex whose entry reads `seen`?
    __device__ __forceinline__ bool could_lower(int du, int seen) const { return ((du << 1) | 1) < seen; }
    __device__ __forceinline__ unsigned int edge(int du, long long, int c, int w, int seen, unsigned int pos) const
    {
        const int nd = ((du + (WEIGHTED ? w : 1)) << 1) | 1;
        if (nd >= seen || atomicMin(dist + c, nd) <= nd) return 0;
        // lowered.  Has the sweep passed c already (or is it just about to)?  Then nobody will look at it
        // again in this sweep unless it is queued.
        const unsigned int ci = (unsigned int)c >> 5, si = backward ? n_chunks - 1u - ci : ci;
        if (si < pos && only == kNoVertex && behind_cap != 0u) {
            const unsigned int m = __activemask(), lane = gpuvm::lane_id(), leader = __ffs(m) - 1;
            unsigned int base = 0;
            if (lane == leader) base = atomicAdd(counters + kCntBehindTail, (unsigned int)__popc(m));
            base = __shfl_sync(m, base, leader);
            const unsigned int slot = base + __popc(m & ((1u << lane) - 1u));
            if (slot < behind_cap) gpuvm::st_relaxed_u32(behind_q + slot, (unsigned int)c);   // full: c stays dirty for the next sweep
        }
        return 1;
    }
};

// Visit the edges [elo, ehi) of vertex u that lie inside the pinned unit starting at edge `first`,
// four per lane at a time: the column (and weight) loads of the four are issued together, then
// the peeks at their other ends, then the updates.
// LAZY_W (weights that would be read in place over the link): a weight is loaded only for an edge that could
// lower its other end at all, i.e. with the weight 0; where no edge of a 128-byte line can, the line is not
// requested.  Most edges of a vertex that is expanded again cannot, and what reads in place cost is requests.
template <class Mem, class Op, bool WEIGHTED, bool LAZY_W = false>
__device__ __forceinline__ unsigned int visit_edges(const Op &op, const unsigned char *col_unit, const unsigned char *w_unit,
                                                    long long first, long long u, int uval, long long elo, long long ehi,
                                                    unsigned int lane, unsigned int pos, unsigned long long *lazy_bytes = nullptr)
{
    constexpr int U = 4;
    unsigned int found = 0;
    for (long long e0 = elo + lane; e0 < ehi; e0 += 32 * U) {
        int c[U], w[U], seen[U];
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const long long e = e0 + 32 * k;
            c[k] = e < ehi ? Mem::load_i32(col_unit + 4 * (e - first)) : -1;
            w[k] = (WEIGHTED && !LAZY_W && e < ehi) ? Mem::load_i32(w_unit + 4 * (e - first)) : 0;
        }
#pragma unroll
        for (int k = 0; k < U; ++k) seen[k] = c[k] >= 0 ? op.peek(c[k]) : 0;
        if constexpr (WEIGHTED && LAZY_W) {
#pragma unroll
            for (int k = 0; k < U; ++k) {
                if (c[k] >= 0 && !op.could_lower(uval, seen[k])) c[k] = -1;
                if (c[k] >= 0) { w[k] = Mem::load_i32(w_unit + 4 * (e0 + 32 * k - first)); if (lazy_bytes) *lazy_bytes += 4; }
            }
        }
#pragma unroll
        for (int k = 0; k < U; ++k)
            if (c[k] >= 0) found += op.edge(uval, u, c[k], w[k], seen[k], pos);
    }
    return found;
}

__device__ __forceinline__ unsigned int ld_volatile_u32(const unsigned int *p) { return *reinterpret_cast<const volatile unsigned int *>(p); }

// How far the sweep has got, for operations that queue what changes behind it: the chunk ticket (chunks
// below it are drawn) plus the chunks that may be drawn while a unit of edges is being visited.
__device__ __forceinline__ unsigned int sweep_pos(const unsigned int *counters, unsigned int n_chunks)
{
    const unsigned int t = ld_volatile_u32(counters + kCntTicket), margin = 2u * kChunksPerTicket * warps_in_grid();
    return t >= n_chunks || t + margin >= n_chunks ? n_chunks : t + margin;
}

// Expand one queued piece of a long neighbour list (all 32 lanes).  Returns this lane's number of
// updates, or -1 when a wait ran out.  Out of line: it is the rare path of the sweep kernel and
// would only add to the register pressure of the common one.
template <class Mem, class Op, bool WEIGHTED>
__device__ __noinline__ int expand_piece(const Mem m, const Op op, unsigned long long col_off, unsigned long long w_off,
                                         const long long *span_q, unsigned int *counters, unsigned int n_chunks,
                                         unsigned int piece, long long epoch, unsigned int lane)
{
    // its producer is between reserving the slot and publishing it
    const volatile long long *ready = span_q + 4 * (size_t)piece + 3;
    unsigned long long t0 = 0;
    bool ok = true;
    while (*ready != epoch) {
        const unsigned long long t = gpuvm::now_ns();
        if (t0 == 0) t0 = t;
        else if (t - t0 > m.wait_ns()) { ok = false; break; }
        __nanosleep(64);
    }
    if (!__all_sync(0xFFFFFFFFu, ok)) { if (lane == 0) m.wait_ran_out(0); return -1; }
    __threadfence();                                      // the entry's fields were written before its ready word
    const long long elo = span_q[4 * (size_t)piece], ehi = span_q[4 * (size_t)piece + 1], u = span_q[4 * (size_t)piece + 2];
    if (ehi <= elo) return 0;
    gpuvm_token tok, tok_w;
    const unsigned char *p = m.pin(col_off + 4ull * elo, GPUVM_READ, tok);
    if (!p) return -1;
    const unsigned char *pw = nullptr;
    if (WEIGHTED) {
        pw = m.pin(w_off + 4ull * elo, GPUVM_READ, tok_w);
        if (!pw) { m.release(tok); return -1; }
    }
    const unsigned int pos = Op::kBehind ? sweep_pos(counters, n_chunks) : 0u;
    const unsigned int found = visit_edges<Mem, Op, WEIGHTED>(op, p, pw, elo, u, op.value((unsigned long long)u), elo, ehi, lane, pos);
    if (WEIGHTED) m.release(tok_w);
    m.release(tok);
    return (int)found;
}

// All 32 lanes: claim the next queued piece; 0xFFFFFFFF when none is waiting.
__device__ __forceinline__ unsigned int take_piece(unsigned int *counters, unsigned int lane)
{
    unsigned int piece = 0xFFFFFFFFu;
    if (lane == 0) {
        unsigned int pushed = ld_volatile_u32(counters + kCntPushed);
        if (pushed > kBigQueue) pushed = kBigQueue;
        const unsigned int taken = ld_volatile_u32(counters + kCntTaken);
        if (taken < pushed && atomicCAS(counters + kCntTaken, taken, taken + 1u) == taken) piece = taken;
    }
    return __shfl_sync(0xFFFFFFFFu, piece, 0);
}

// All 32 lanes: take up to 32 vertices from the queue of vertices that were lowered behind the sweep
// position and re-expand them.  Returns this lane's number of updates, or -1 when the queue was empty.
// No fault is taken for such a vertex: what it needs (two row offsets, its edges: a hundred bytes or so)
// is read from the frame when its page is in the pool and in place from the backing store when it is not
// (the CSR arrays are never written, so the backing store is current).  One with a very long list is left
// dirty for the next sweep.
template <class Mem, class Op, bool WEIGHTED>
__device__ __noinline__ int expand_behind(const Mem m, const Op op, unsigned long long off_off, unsigned long long col_off,
                                          unsigned long long w_off, unsigned int nv, unsigned int *counters, unsigned int lane)
{
    // 32 slots are reserved with one fetch-and-add, and only when the queue was seen non-empty: no retry
    // storms when thousands of warps come here at once.  Warps that saw the same state may reserve slots past
    // the tail; such a slot is read if its producer fills it within a short wait and is given up otherwise
    // (its vertex stays dirty and is found by the next sweep).
    unsigned int n = 0xFFFFFFFFu, h = 0;
    if (lane == 0) {
        unsigned int t = ld_volatile_u32(counters + kCntBehindTail);
        if (t > op.behind_cap) t = op.behind_cap;
        if (ld_volatile_u32(counters + kCntBehindHead) < t) {
            h = atomicAdd(counters + kCntBehindHead, 32u);
            n = h < op.behind_cap ? (op.behind_cap - h < 32u ? op.behind_cap - h : 32u) : 0u;
        }
    }
    n = __shfl_sync(0xFFFFFFFFu, n, 0);
    h = __shfl_sync(0xFFFFFFFFu, h, 0);
    if (n == 0xFFFFFFFFu) return -1;
    unsigned int u = kNoVertex;
    if (lane < n) {
        unsigned int spins = 0;                               // its producer is between reserving the slot and filling it
        while ((u = gpuvm::ld_relaxed_u32(op.behind_q + h + lane)) == kNoVertex && ++spins < 256u) __nanosleep(32);
    }
    bool have = u != kNoVertex && u < nv && op.active(u);
    long long lo = 0, hi = 0;
    unsigned long long direct = 0;                            // bytes read in place from the backing store
    // The two row offsets of each vertex: from their frame when the page is resident, else in place from the
    // backing store (no page is fetched for a vertex behind the sweep).
    bool got = false;
    if (have) {
        const unsigned long long ob = off_off + 8ull * u, unit_o = m.unit();
        if (ob / unit_o == (ob + 8) / unit_o) {                // both in one page: one pin
            gpuvm_token tok;
            const unsigned char *p = m.pin_if_resident(ob, tok);
            if (p) { lo = Mem::load_i64(p); hi = Mem::load_i64(p + 8); m.release(tok); got = true; }
        }
    }
    // In place, two lanes per vertex, so that the pair's loads are one instruction and, the two offsets lying
    // side by side, one request on the link (issued by one lane one after the other they were two): what these
    // reads cost is requests.
    const unsigned int in_place = __ballot_sync(0xFFFFFFFFu, have && !got);
#pragma unroll
    for (unsigned int r = 0; r < 2 && in_place; ++r) {
        const unsigned int src = (lane >> 1) + 16u * r;
        const unsigned int uu = __shfl_sync(0xFFFFFFFFu, u, src);
        long long val = 0;
        if ((in_place >> src) & 1u) val = Mem::load_i64(m.through(off_off + 8ull * ((unsigned long long)uu + (lane & 1u))));
        const long long a = __shfl_sync(0xFFFFFFFFu, val, (lane & 15u) * 2u), b = __shfl_sync(0xFFFFFFFFu, val, (lane & 15u) * 2u + 1u);
        if ((lane >> 4) == r && ((in_place >> lane) & 1u)) { lo = a; hi = b; direct += 16; }
    }
    if (have) {
        if (hi <= lo) { op.begin(u); have = false; }          // nothing to expand: just not dirty any more
        if (have && hi - lo >= kBigDegree) have = false;      // a hub: left dirty, the next sweep cuts it into pieces
    }
    unsigned int found = 0;
    unsigned int todo = __ballot_sync(0xFFFFFFFFu, have);
    const unsigned long long unit = m.unit();
    const unsigned int pos = sweep_pos(counters, op.n_chunks);
    while (todo) {
        const int L = __ffs(todo) - 1;
        todo &= todo - 1;
        const long long bu = __shfl_sync(0xFFFFFFFFu, u, L), bhi = __shfl_sync(0xFFFFFFFFu, hi, L);
        long long first = __shfl_sync(0xFFFFFFFFu, lo, L);
        int uval = 0;
        if (lane == 0) uval = op.begin((unsigned long long)bu);
        uval = __shfl_sync(0xFFFFFFFFu, uval, 0);
        while (first < bhi) {
            const unsigned long long byte = col_off + 4ull * first;
            long long last = (long long)(((byte / unit + 1) * unit - col_off) / 4);
            if (last > bhi) last = bhi;
            // this part of the list: from its frame when the page is resident, else in place from the backing store
            gpuvm_token tok, tok_w;
            const unsigned char *p = m.pin_if_resident(byte, tok);
            const bool held = p != nullptr;
            if (!held) { p = m.through(byte); if (lane == 0) direct += 4ull * (unsigned long long)(last - first); }
            const unsigned char *pw = nullptr;
            bool held_w = false;
            if (WEIGHTED) {
                pw = m.pin_if_resident(w_off + 4ull * first, tok_w);
                held_w = pw != nullptr;
                if (!held_w) pw = m.through(w_off + 4ull * first);      // (its bytes are counted as they are loaded)
            }
            if (WEIGHTED && !held_w) found += visit_edges<Mem, Op, WEIGHTED, true>(op, p, pw, first, bu, uval, first, last, lane, pos, &direct);
            else found += visit_edges<Mem, Op, WEIGHTED>(op, p, pw, first, bu, uval, first, last, lane, pos);
            if (held_w) m.release(tok_w);
            if (held) m.release(tok);
            first = last;
        }
    }
    for (int o = 16; o; o >>= 1) direct += __shfl_down_sync(0xFFFFFFFFu, direct, o);
    if (lane == 0 && direct) m.note_direct(direct);
    return (int)found;
}

// End of a warp's sweep (all 32 lanes): expand pieces (and vertices lowered behind the sweep) until every
// chunk of the sweep is finished and every piece is taken.  Returns this lane's number of updates.  The wait is bounded.
template <class Mem, class Op, bool WEIGHTED>
__device__ __noinline__ unsigned int drain_pieces(const Mem m, const Op op, unsigned long long off_off, unsigned long long col_off,
                                                  unsigned long long w_off, unsigned int nv, const long long *span_q,
                                                  unsigned int *counters, unsigned int n_chunks, long long epoch, unsigned int lane)
{
    unsigned int found = 0, sleep_ns = 64;
    unsigned long long idle_since = 0;
    for (;;) {
        const unsigned int piece = take_piece(counters, lane);
        if (piece != 0xFFFFFFFFu) {
            const int r = expand_piece<Mem, Op, WEIGHTED>(m, op, col_off, w_off, span_q, counters, n_chunks, piece, epoch, lane);
            if (r < 0) return found;
            found += (unsigned int)r;
            idle_since = 0;
            sleep_ns = 64;
            continue;
        }
        if constexpr (Op::kBehind) {
            const int r = expand_behind<Mem, Op, WEIGHTED>(m, op, off_off, col_off, w_off, nv, counters, lane);
            if (r >= 0) {
                found += (unsigned int)r;
                idle_since = 0;
                sleep_ns = 64;
                continue;
            }
        }
        int state = 0;                                        // 0 wait, 1 done, 2 gave up
        if (lane == 0) {
            unsigned int pushed = ld_volatile_u32(counters + kCntPushed);
            if (pushed > kBigQueue) pushed = kBigQueue;
            const unsigned int queued_behind = Op::kBehind ? ld_volatile_u32(counters + kCntBehindTail) : 0u;
            // Nothing queued in this sweep so far: leave at once (a warp that queues pieces later also
            // comes through here and sees to them); thousands of idle warps polling would only be in
            // the way of the ones still at work.  Otherwise stay and help until all chunks are finished.
            if (pushed == 0u && queued_behind == 0u) state = 1;
            else if (ld_volatile_u32(counters + kCntDone) >= n_chunks && ld_volatile_u32(counters + kCntTaken) >= pushed) state = 1;
            else {
                const unsigned long long t = gpuvm::now_ns();
                if (idle_since == 0) idle_since = t;
                else if (t - idle_since > m.wait_ns()) { m.wait_ran_out(0); state = 2; }
            }
        }
        if (__shfl_sync(0xFFFFFFFFu, state, 0)) return found;
        __nanosleep(sleep_ns);
        if (sleep_ns < 16384) sleep_ns *= 2;
    }
}

// One sweep over the vertices in address order: a warp draws the next chunk of 32 consecutive
// vertices from a ticket counter, so at any moment the whole grid works inside a narrow window
// of the row-offset and column arrays and a sweep touches every page at most about once.
// Per chunk the warp reads the 33 row offsets with two accessor calls and then walks the
// column pages that the chunk's edges span, holding one page at a time (two with weights, which
// sit at the same offset inside their own page): one pin per page and chunk instead of one per
// neighbour list, which keeps the atomic traffic on the entries of the few pages under the
// window low.  Odd sweeps run downwards: the pages a sweep used last are still resident when the
// next one starts with them (a one-directional cyclic sweep defeats any LRU-like policy).
// Very long neighbour lists are cut at unit boundaries into pieces that go to a queue; every warp
// looks into that queue before it draws its next chunk, so the pieces are expanded by the whole
// grid while their pages are still under (or just ahead of) the sweep window.  An entry is
// published by its `ready` word (= sweep + 1, written after a fence; the queue is zeroed once per
// call).  Operations with kBehind also keep a queue of vertices that changed behind the sweep position
// (see LcOp), served in the same way.  A warp leaves when all chunks are finished and all pieces are
// taken; every wait is bounded.
template <class Mem, class Op, bool WEIGHTED>
__global__ void __launch_bounds__(256, 4) graph_sweep_kernel(Mem m, Op op, unsigned long long off_off, unsigned long long col_off,
                                                          unsigned long long w_off, unsigned int nv,
                                                          unsigned long long n_edges, long long *__restrict__ span_q,
                                                          unsigned int *__restrict__ counters, int sweep, int backward)
{
    const unsigned int lane = threadIdx.x & 31;
    const unsigned long long unit = m.unit();
    const unsigned int n_chunks = (nv + 31) / 32;
    const long long epoch = sweep + 1;
    unsigned int found = 0, my_done = 0, iter = 0, next_chunk = 0, last_chunk = 0;
    unsigned long long direct = 0;                           // bytes this lane read in place from the backing store
    unsigned long long direct_w = 0;                         // weights this lane loaded in place, in bytes (all lanes count)
    for (;;) {
        // ---- a piece of a long neighbour list, if one is waiting (looked for before every kSpanPoll-th chunk)
        if ((iter++ & (kSpanPoll - 1)) == 0) {
            const unsigned int piece = take_piece(counters, lane);
            if (piece != 0xFFFFFFFFu) {
                const int r = expand_piece<Mem, Op, WEIGHTED>(m, op, col_off, w_off, span_q, counters, n_chunks, piece, epoch, lane);
                if (r < 0) break;
                found += (unsigned int)r;
                continue;
            }
        }
        // ---- vertices that were lowered behind the sweep position, while their pages are still there
        if constexpr (Op::kBehind) {
            if ((iter & (kSpanPoll - 1)) == 1) {
                const int r = expand_behind<Mem, Op, WEIGHTED>(m, op, off_off, col_off, w_off, nv, counters, lane);
                if (r > 0) found += (unsigned int)r;
            }
        }
        // ---- the next chunk of 32 vertices (a ticket is good for kChunksPerTicket consecutive chunks)
        if (next_chunk == last_chunk) {
            unsigned int t = 0;
            if (lane == 0) t = atomicAdd(counters + kCntTicket, kChunksPerTicket);
            t = __shfl_sync(0xFFFFFFFFu, t, 0);
            if (t >= n_chunks) {
                // no chunk left: report the finished ones, then help with the pieces until all chunks
                // are finished and all pieces taken
                if (lane == 0 && my_done) { __threadfence(); atomicAdd(counters + kCntDone, my_done); }
                found += drain_pieces<Mem, Op, WEIGHTED>(m, op, off_off, col_off, w_off, nv, span_q, counters, n_chunks, epoch, lane);
                break;
            }
            next_chunk = t;
            last_chunk = t + kChunksPerTicket < n_chunks ? t + kChunksPerTicket : n_chunks;
        }
        const unsigned int chunk = next_chunk++;
        ++my_done;
        const unsigned long long v0 = 32ull * (backward ? n_chunks - 1 - chunk : chunk);
        const unsigned long long v = v0 + lane;
        const bool active = v < nv && op.active(v);
        if (!__any_sync(0xFFFFFFFFu, active)) continue;
        // fetch the row-offset page the sweep will reach kAhead pages from now (one warp wins the
        // page, the others return at once), so that the window does not stall on one page at a time
        const bool dense = __popc(__ballot_sync(0xFFFFFFFFu, active)) >= 8;   // a sparse frontier may never get there
        if (dense) {
            const long long ahead = (long long)(off_off + 8ull * v0) + (backward ? -kAhead : kAhead) * (long long)unit;
            if (ahead >= (long long)off_off && ahead < (long long)(off_off + 8ull * nv)) m.prefetch((unsigned long long)ahead);
        }
        // row offsets of the chunk: off[v0 .. v0+32], clamped to the nv + 1 entries that exist
        // (one pin for all 33 when they lie in one unit, which they do except at unit ends and at the last chunk)
        long long lo, hi;
        const unsigned long long ob = off_off + 8ull * v0;
        // a sparse sweep (few vertices left to expand, scattered over the graph) does not fetch pages: what is
        // resident is read from its frame, the rest in place from the backing store
        bool thru = false;
        if constexpr (Op::kBehind) thru = op.through_main != 0;
        if (v0 + 32 <= nv && ob % unit + 33 * 8 <= unit) {
            gpuvm_token tok_o;
            const unsigned char *po = thru ? m.pin_if_resident(ob, tok_o) : m.pin(ob, GPUVM_READ, tok_o);
            const bool held = po != nullptr;
            if (!held) {
                if (!thru) break;
                po = m.through(ob);
                if (lane == 0) direct += 33 * 8;
            }
            lo = Mem::load_i64(po + 8 * lane);
            hi = __shfl_down_sync(0xFFFFFFFFu, lo, 1);
            if (lane == 31) hi = Mem::load_i64(po + 8 * 32);
            if (held) m.release(tok_o);
        } else if (thru) {
            lo = Mem::load_i64(m.through(off_off + 8ull * (v < nv ? v : nv)));
            hi = __shfl_down_sync(0xFFFFFFFFu, lo, 1);
            if (lane == 31) hi = Mem::load_i64(m.through(off_off + 8ull * (v + 1 < nv ? v + 1 : nv)));
            if (lane == 0) direct += 33 * 8;
        } else {
            lo = m.template read<long long>(off_off, v < nv ? v : nv);
            hi = __shfl_down_sync(0xFFFFFFFFu, lo, 1);
            if (lane == 31) hi = m.template read<long long>(off_off, v + 1 < nv ? v + 1 : nv);
        }
        if (!active) { lo = 0; hi = 0; }
        const int uval = active ? op.begin(v) : 0;          // the value this vertex's edges are visited with
        // long neighbour lists: cut them at unit boundaries and queue the pieces for the grid
        unsigned int bigs = __ballot_sync(0xFFFFFFFFu, hi - lo >= kBigDegree);
        while (bigs) {
            const int L = __ffs(bigs) - 1;
            bigs &= bigs - 1;
            const long long blo = __shfl_sync(0xFFFFFFFFu, lo, L), bhi = __shfl_sync(0xFFFFFFFFu, hi, L);
            const unsigned long long b0 = (col_off + 4ull * blo) / unit, b1 = (col_off + 4ull * bhi - 1) / unit;
            const unsigned int pieces = (unsigned int)(b1 - b0 + 1);
            unsigned int slot = 0;
            if (lane == 0) slot = atomicAdd(counters + kCntPushed, pieces);
            slot = __shfl_sync(0xFFFFFFFFu, slot, 0);
            const bool fits = slot + pieces <= kBigQueue;
            const unsigned int n_write = fits ? pieces : (slot < kBigQueue ? kBigQueue - slot : 0u);
            for (unsigned int k = lane; k < n_write; k += 32) {
                const long long s = (long long)(((b0 + k) * unit - col_off + 3) / 4);
                const long long t = (long long)(((b0 + k + 1) * unit - col_off) / 4);
                // queue full: the slots that were reserved are published empty and the list is expanded here
                span_q[4 * (size_t)(slot + k)] = fits ? (k == 0 ? blo : s) : 0;
                span_q[4 * (size_t)(slot + k) + 1] = fits ? (t < bhi ? t : bhi) : 0;
                span_q[4 * (size_t)(slot + k) + 2] = (long long)(v0 + L);
            }
            __threadfence();
            __syncwarp();
            for (unsigned int k = lane; k < n_write; k += 32)
                *reinterpret_cast<volatile long long *>(span_q + 4 * (size_t)(slot + k) + 3) = epoch;
            if (fits && (int)lane == L) { lo = 0; hi = 0; }
        }
        // the edges of this chunk, unit by unit
        long long rlo = hi > lo ? lo : 0x7FFFFFFFFFFFFFFFll, rhi = hi > lo ? hi : 0;
        for (int o = 16; o; o >>= 1) {
            const long long a = __shfl_xor_sync(0xFFFFFFFFu, rlo, o), b = __shfl_xor_sync(0xFFFFFFFFu, rhi, o);
            rlo = a < rlo ? a : rlo;
            rhi = b > rhi ? b : rhi;
        }
        if (dense && rhi > rlo) {                        // and the column page the sweep will reach
            const long long ahead = (long long)(col_off + 4ull * (backward ? rlo : rhi)) +
                                    (backward ? -kAhead : kAhead) * (long long)unit;
            if (ahead >= (long long)col_off && ahead < (long long)(col_off + 4ull * n_edges)) {
                m.prefetch((unsigned long long)ahead);
                if (WEIGHTED) m.prefetch((unsigned long long)ahead - col_off + w_off);
            }
        }
        long long first = rlo;
        bool failed = false;
        while (first < rhi) {
            const unsigned long long byte = col_off + 4ull * first;
            long long last = (long long)(((byte / unit + 1) * unit - col_off) / 4);   // first edge of the next unit
            if (last > rhi) last = rhi;
            unsigned int touch = __ballot_sync(0xFFFFFFFFu, lo < last && hi > first);
            if (touch) {
                gpuvm_token tok, tok_w;
                const unsigned char *p = thru ? m.pin_if_resident(byte, tok) : m.pin(byte, GPUVM_READ, tok);
                const bool held = p != nullptr;
                if (!held) {
                    if (!thru) { failed = true; break; }
                    p = m.through(byte);
                }
                const unsigned char *pw = nullptr;
                bool held_w = false;
                if (WEIGHTED) {
                    pw = thru ? m.pin_if_resident(w_off + 4ull * first, tok_w) : m.pin(w_off + 4ull * first, GPUVM_READ, tok_w);
                    held_w = pw != nullptr;
                    if (!held_w) {
                        if (!thru) { m.release(tok); failed = true; break; }
                        pw = m.through(w_off + 4ull * first);
                    }
                }
                const unsigned int pos = Op::kBehind ? sweep_pos(counters, n_chunks) : 0u;
                while (touch) {
                    const int L = __ffs(touch) - 1;
                    touch &= touch - 1;
                    long long blo = __shfl_sync(0xFFFFFFFFu, lo, L), bhi = __shfl_sync(0xFFFFFFFFu, hi, L);
                    const int bval = __shfl_sync(0xFFFFFFFFu, uval, L);
                    if (blo < first) blo = first;
                    if (bhi > last) bhi = last;
                    if (WEIGHTED && !held_w)
                        found += visit_edges<Mem, Op, WEIGHTED, true>(op, p, pw, first, (long long)(v0 + L), bval, blo, bhi, lane, pos, &direct_w);
                    else
                        found += visit_edges<Mem, Op, WEIGHTED>(op, p, pw, first, (long long)(v0 + L), bval, blo, bhi, lane, pos);
                    if (lane == 0 && !held) direct += 4ull * (unsigned long long)(bhi - blo);   // (weights: direct_w, as they are loaded)
                }
                if (held_w) m.release(tok_w);
                if (held) m.release(tok);
            }
            first = last;
        }
        if (failed) break;                               // a wait ran out: the sticky error is set, the others give up too
    }
    for (int o = 16; o; o >>= 1) found += __shfl_down_sync(0xFFFFFFFFu, found, o);
    if (lane == 0 && found) atomicAdd(counters + kCntUpdates, found);
    for (int o = 16; o; o >>= 1) direct_w += __shfl_down_sync(0xFFFFFFFFu, direct_w, o);
    if (lane == 0 && direct + direct_w) m.note_direct(direct + direct_w);
}

// Balanced CSR (Section 5.2, Fig. 8): the edge array is cut into chunks of equal length and a
// small array names the vertex whose list holds the first edge of each chunk.  Workers take
// chunks, not vertices: every worker gets the same number of edges and, a chunk lying inside one
// page, exactly one page of columns, however the degrees are distributed; a long neighbour list
// is shared by as many workers as it has chunks.  A warp draws a chunk ticket, walks the chunk's
// vertices 32 at a time, and expands the part of each active vertex's list that lies in the chunk.  counters: [0] updates, [2] chunk ticket.
constexpr int kBcsrBlocksPerSm = 2;    // 128 registers, no spills: 37 ms for the CC against 40 ms with four blocks at 64
// The CC draws its chunks from the last one down: in an RMAT graph the chunks of the sparse end span tens of
// thousands of vertices each and take longest, so they go first and the short ones fill the tail (33 against 37 ms).
constexpr int kBcsrCcSweep = 1;
template <class Mem, class Op>
__global__ void __launch_bounds__(256, kBcsrBlocksPerSm) bcsr_sweep_kernel(Mem m, Op op, unsigned long long off_off, unsigned long long col_off,
                                                         unsigned long long chunk_off, unsigned int nv,
                                                         unsigned long long n_edges, unsigned int chunk_edges,
                                                         unsigned int *__restrict__ counters, int sweep)
{
    const unsigned int lane = threadIdx.x & 31;
    const unsigned int n_chunks = (unsigned int)((n_edges + chunk_edges - 1) / chunk_edges);
    unsigned int found = 0;
    for (;;) {
        unsigned int ticket = 0;
        if (lane == 0) ticket = atomicAdd(counters + 2, 1u);
        ticket = __shfl_sync(0xFFFFFFFFu, ticket, 0);
        if (ticket >= n_chunks) break;
        const unsigned int c = (sweep & 1) ? n_chunks - 1 - ticket : ticket;
        const long long c_lo = (long long)c * chunk_edges;
        const long long c_hi = c_lo + chunk_edges < (long long)n_edges ? c_lo + chunk_edges : (long long)n_edges;
        // vertices whose lists reach into this chunk: first vertex of this chunk .. first vertex of the next
        int vr = 0;
        if (lane < 2) vr = m.template read<int>(chunk_off, (unsigned long long)c + lane);   // chunk table has n_chunks + 1 entries
        const unsigned int v_first = (unsigned int)__shfl_sync(0xFFFFFFFFu, vr, 0);
        const unsigned int v_last = (unsigned int)__shfl_sync(0xFFFFFFFFu, vr, 1);
        // which groups of 32 vertices have an active one: eight groups' flags are loaded at a time (a chunk
        // in a region of low degrees spans tens of thousands of vertices)
        for (unsigned int g0 = v_first; g0 <= v_last && g0 < nv; g0 += 256) {
        unsigned int group_active = 0;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const unsigned long long vk = (unsigned long long)g0 + 32u * k + lane;
            const bool a = vk <= v_last && vk < nv && op.active(vk);
            group_active |= (__any_sync(0xFFFFFFFFu, a) ? 1u : 0u) << k;
        }
        if (!group_active) continue;
        // The row offsets of these 256 vertices and of the one after them: one pin when they lie in one unit (a
        // chunk in a region of low degrees walks a thousand groups of 32 vertices; a pin per group was most of
        // its time).  Nothing else is pinned meanwhile: one page at a time, no pool is too small.
        long long lo8[8], lo_next;
        const unsigned long long ob = off_off + 8ull * g0;
        if ((unsigned long long)g0 + 256 <= nv && ob % m.unit() + 257 * 8 <= m.unit()) {
            gpuvm_token tok_o;
            const unsigned char *po = m.pin(ob, GPUVM_READ, tok_o);
            if (!po) return;
#pragma unroll
            for (int k = 0; k < 8; ++k) lo8[k] = Mem::load_i64(po + 8 * (32 * k + lane));
            lo_next = Mem::load_i64(po + 8 * 256);
            m.release(tok_o);
        } else {
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const unsigned long long vk = (unsigned long long)g0 + 32u * k + lane;
                lo8[k] = m.template read<long long>(off_off, vk < nv ? vk : nv);
            }
            lo_next = m.template read<long long>(off_off, (unsigned long long)g0 + 256 < nv ? (unsigned long long)g0 + 256 : nv);
        }
        // the chunk's column page: pinned at the first group that has an edge in it, held to the end of the block
        gpuvm_token tok;
        const unsigned char *p = nullptr;
        // (not unrolled: eight copies of the body below overflow the instruction cache, a quarter of all issue
        // slots went to waiting for instructions; the eight offsets then live in local memory, two reads per group)
#pragma unroll 1
        for (int k8 = 0; k8 < 8; ++k8) {
            if (!((group_active >> k8) & 1u)) continue;
            const unsigned int v0 = g0 + 32u * k8;
            const unsigned long long v = (unsigned long long)v0 + lane;
            const bool active = v <= v_last && v < nv && op.active(v);
            if (!__any_sync(0xFFFFFFFFu, active)) continue;
            long long lo = lo8[k8];
            long long hi = __shfl_down_sync(0xFFFFFFFFu, lo, 1);
            const long long first_of_next = k8 < 7 ? __shfl_sync(0xFFFFFFFFu, lo8[k8 < 7 ? k8 + 1 : 7], 0) : lo_next;
            if (lane == 31) hi = first_of_next;
            if (lo < c_lo) lo = c_lo;
            if (hi > c_hi) hi = c_hi;
            unsigned int touch = __ballot_sync(0xFFFFFFFFu, active && hi > lo);
            if (!touch) continue;
            const int uval = active ? op.begin(v) : 0;
            if (!p) {
                p = m.pin(col_off + 4ull * c_lo, GPUVM_READ, tok);
                if (!p) return;
            }
            if (__popc(touch) >= 8) {
                // Many of the 32 vertices have edges here: their lists lie one after the other in the chunk, so
                // the lanes take the edges of the whole stretch, 32 x 4 at a time, and each looks up whose edge
                // it has (the last vertex whose list starts at or before it: a binary search over the 32 clipped
                // starts, five shuffles).  Every lane works whatever the degrees are; with one list at a time a
                // list of sixteen edges leaves half the warp idle and every list costs its own round trips.
                const long long e_begin = __shfl_sync(0xFFFFFFFFu, lo, 0);
                long long e_end = __shfl_sync(0xFFFFFFFFu, hi, 31);
                if (e_end < e_begin) e_end = e_begin;
                constexpr int U = 4;
                for (long long b = e_begin; b < e_end; b += 32 * U) {
                    int c[U], own[U], seen[U];
#pragma unroll
                    for (int k = 0; k < U; ++k) {
                        const long long e = b + 32 * k + lane;
                        int j = 0;
#pragma unroll
                        for (int step = 16; step; step >>= 1) {
                            const long long lo_t = __shfl_sync(0xFFFFFFFFu, lo, (j + step) & 31);
                            if (lo_t <= e) j += step;                   // starts are sorted; j + step <= 31 here
                        }
                        const bool mine = e < e_end && ((touch >> j) & 1u);
                        own[k] = mine ? j : -1;
                        c[k] = mine ? Mem::load_i32(p + 4 * (e - c_lo)) : -1;
                    }
#pragma unroll
                    for (int k = 0; k < U; ++k) seen[k] = c[k] >= 0 ? op.peek(c[k]) : 0;
#pragma unroll
                    for (int k = 0; k < U; ++k) {
                        const int uv = __shfl_sync(0xFFFFFFFFu, uval, own[k] & 31);
                        if (c[k] >= 0) found += op.edge(uv, (long long)(v0 + own[k]), c[k], 0, seen[k], 0u);
                    }
                }
            } else {
                while (touch) {
                    const int L = __ffs(touch) - 1;
                    touch &= touch - 1;
                    const long long blo = __shfl_sync(0xFFFFFFFFu, lo, L), bhi = __shfl_sync(0xFFFFFFFFu, hi, L);
                    found += visit_edges<Mem, Op, false>(op, p, nullptr, c_lo, (long long)(v0 + L), __shfl_sync(0xFFFFFFFFu, uval, L),
                                                         blo, bhi, lane, 0u);
                }
            }
        }
        if (p) m.release(tok);
        }
    }
    for (int o = 16; o; o >>= 1) found += __shfl_down_sync(0xFFFFFFFFu, found, o);
    if (lane == 0 && found) atomicAdd(counters, found);
}

__global__ void bfs_init_kernel(int *level, int source) { level[source] = 0; }

__global__ void cc_init_kernel(int *label, unsigned int nv)
{
    for (unsigned int v = blockIdx.x * blockDim.x + threadIdx.x; v < nv; v += gridDim.x * blockDim.x) label[v] = (int)v;
}

// Every parent becomes its root (= the smallest vertex of its component).  The only stores of this kernel
// are roots (no path halving here: a halving store that lands after the root was stored would undo it).
__global__ void cc_finish_kernel(int *parent, unsigned int nv)
{
    const CcOp op{parent};
    for (unsigned int v = blockIdx.x * blockDim.x + threadIdx.x; v < nv; v += gridDim.x * blockDim.x)
        parent[v] = op.find_read_only((int)v);
}

// label-correcting runs: everything unreached and clean, the source at distance 0 and dirty
__global__ void lc_init_kernel(int *dist, unsigned int nv, unsigned int source)
{
    for (unsigned int v = blockIdx.x * blockDim.x + threadIdx.x; v < nv; v += gridDim.x * blockDim.x)
        dist[v] = v == source ? 1 : kLcInf;
}

// packed words back to distances; `unreached` for what was never lowered; the largest distance goes to *max_out
__global__ void lc_finish_kernel(int *dist, unsigned int nv, int unreached, unsigned int *max_out)
{
    int best = 0;
    for (unsigned int v = blockIdx.x * blockDim.x + threadIdx.x; v < nv; v += gridDim.x * blockDim.x) {
        const int w = dist[v];
        const int d = w >= kLcInf ? unreached : w >> 1;
        dist[v] = d;
        if (w < kLcInf && d > best) best = d;
    }
    for (int o = 16; o; o >>= 1) { const int t = __shfl_down_sync(0xFFFFFFFFu, best, o); best = t > best ? t : best; }
    if ((threadIdx.x & 31) == 0 && best > 0) atomicMax(max_out, (unsigned int)best);
}

// ----------------------------------------------------------------- vector add
// A warp owns one unit (page) of the element range and walks it in chunks of at most 4 KiB.
// HOLD_C = false: it holds exactly one page at a time (a, then b, then c, per chunk), which
// cannot deadlock whatever the pool size.  HOLD_C = true (chosen by the host when the pool has
// at least two frames per warp of the grid and c starts on a page boundary): the page of c
// stays pinned for the whole unit and, when the unit covers the whole page, is requested with
// GPUVM_WRITE_ALL, so it is not fetched from the host before being overwritten; when the
// unit is finished the warp writes the page back at once (gpuvm_clean), which keeps
// write-backs off the fault path and uses the outbound half of the link while the inbound
// half carries a and b.
template <class Mem, bool HOLD_C>
__global__ void __launch_bounds__(256) vadd_kernel(Mem m, unsigned long long a_off, unsigned long long b_off,
                                                   unsigned long long c_off, unsigned long long n,
                                                   unsigned int chunk_bytes)
{
    const unsigned int lane = threadIdx.x & 31;
    const unsigned long long unit = m.unit() > chunk_bytes ? m.unit() : chunk_bytes;
    const unsigned long long total = 4ull * n, units = (total + unit - 1) / unit;
    for (unsigned long long u = warp_in_grid(); u < units; u += warps_in_grid()) {
        unsigned long long lo = u * unit, hi = lo + unit < total ? lo + unit : total;
        gpuvm_token tok_c;
        unsigned char *page_c = nullptr;
        if (HOLD_C) {
            page_c = m.pin(c_off + lo, hi - lo == unit ? GPUVM_WRITE_ALL : GPUVM_WRITE, tok_c);
            if (!page_c) return;
        }
        for (unsigned long long off = lo; off < hi; off += chunk_bytes) {
            const unsigned int len = (unsigned int)(hi - off < chunk_bytes ? hi - off : chunk_bytes);
            const unsigned int n16 = len >> 4;
            uint4 va[8], vb[8];
            gpuvm_token tok;
            const unsigned char *pa = m.pin(a_off + off, GPUVM_READ, tok);
            if (!pa) break;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                unsigned int i = lane + 32u * j;
                if (i < n16) va[j] = Mem::load16(pa + 16ull * i);
            }
            m.release(tok);
            const unsigned char *pb = m.pin(b_off + off, GPUVM_READ, tok);
            if (!pb) break;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                unsigned int i = lane + 32u * j;
                if (i < n16) vb[j] = Mem::load16(pb + 16ull * i);
            }
            m.release(tok);
            unsigned char *pc = HOLD_C ? page_c + (off - lo) : m.pin(c_off + off, GPUVM_WRITE, tok);
            if (!pc) break;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                unsigned int i = lane + 32u * j;
                if (i < n16) {
                    uint4 r;
                    r.x = __float_as_uint(__fadd_rn(__uint_as_float(va[j].x), __uint_as_float(vb[j].x)));
                    r.y = __float_as_uint(__fadd_rn(__uint_as_float(va[j].y), __uint_as_float(vb[j].y)));
                    r.z = __float_as_uint(__fadd_rn(__uint_as_float(va[j].z), __uint_as_float(vb[j].z)));
                    r.w = __float_as_uint(__fadd_rn(__uint_as_float(va[j].w), __uint_as_float(vb[j].w)));
                    Mem::store16(pc + 16ull * i, r);
                }
            }
            if (!HOLD_C) m.release(tok);
        }
        if (HOLD_C) {
            m.clean(tok_c, page_c);          // the finished page goes to the host at once: evicting it later is free
            m.release(tok_c);
        }
    }
}

// -------------------------------------------------------------- embedding bag
template <class Mem>
__global__ void __launch_bounds__(256) embag_kernel(Mem m, unsigned long long t_off, unsigned int dims,
                                                    const long long *__restrict__ rows, unsigned long long n_bags,
                                                    unsigned int bag, float *__restrict__ out)
{
    const unsigned int lane = threadIdx.x & 31;
    const unsigned int q = dims >> 2;                           // 16-byte pieces per row
    for (unsigned long long g = warp_in_grid(); g < n_bags; g += warps_in_grid()) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (unsigned int k = 0; k < bag; ++k) {
            const unsigned long long r = (unsigned long long)rows[g * bag + k];
            if (lane < q) {
                uint4 v = m.template read<uint4>(t_off, r * q + lane);
                acc.x = __fadd_rn(acc.x, __uint_as_float(v.x));
                acc.y = __fadd_rn(acc.y, __uint_as_float(v.y));
                acc.z = __fadd_rn(acc.z, __uint_as_float(v.z));
                acc.w = __fadd_rn(acc.w, __uint_as_float(v.w));
            }
        }
        if (lane < q) reinterpret_cast<float4 *>(out + g * dims)[lane] = acc;
    }
}

// Batched embedding bag.  A requester warp takes 32 bags at a time (bag b of the item belongs
// to lane b) and up to 32 lookups of each: 1024 row requests registered in the page table at
// once.  Rows arrive in any order, so each served row is first copied, by the whole warp with
// coalesced 16-byte accesses, into the warp's staging area (device scratch); when the batch
// is complete the rows of each bag are added up in list order, which keeps the fp32 result
// bit-identical to a sequential sum.  Faults go to the block's migrator warps.
constexpr int kEmbagRequesters = 28;
constexpr int kEmbagMigrators = 4;
constexpr unsigned int kEmbagLookups = 32;                 // lookups of a bag per batch (table rows)
constexpr unsigned int kEmbagChunk = 8192;                 // bytes per bulk copy of a migrator warp
// Bulk copies a migrator warp keeps in flight.  Rows read in place keep thousands of 512-byte reads outstanding,
// and the link serves its queue in order: a page copy with one 8 KiB chunk outstanding per warp gets a
// correspondingly small share and the pages arrive after the rows.
constexpr unsigned int kEmbagStages = 4;                    // 57 / 50 / 46 / 46 ms for 1 / 2 / 4 / 6 on the 64 GiB Zipf table
constexpr unsigned int kEmbagMaxGroups = 8;                // groups of 32 bags a requester warp takes at a time

// How many lookups of the whole list name each page, up to `limit` (all the batched kernel asks is whether a page
// reaches it): it reads the rows of pages below the limit in place and fetches the others at their first touch.
// One atomic per group of equal pages in a warp, and none once a page's count has reached the limit, so the
// hottest pages, which would serialise hundreds of thousands of atomics on one word each, cost a load.
__global__ void embag_demand_kernel(const long long *__restrict__ rows, unsigned long long n, unsigned long long t_off,
                                    unsigned long long row_bytes, unsigned int page_shift, unsigned long long rows_inside,
                                    unsigned int *__restrict__ demand, unsigned int limit)
{
    const unsigned int lane = threadIdx.x & 31;
    const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
    for (unsigned long long base = (blockIdx.x * (unsigned long long)blockDim.x + threadIdx.x) & ~31ull; base < n; base += stride) {
        const unsigned long long i = base + lane;
        const unsigned long long r = i < n ? (unsigned long long)rows[i] : ~0ull;
        const bool inside = r < rows_inside;
        const unsigned int vpn = inside ? (unsigned int)((t_off + r * row_bytes) >> page_shift) : 0u;
        const unsigned int mask = __ballot_sync(0xFFFFFFFFu, inside);
        if (inside) {
            const unsigned int group = __match_any_sync(mask, vpn);
            if (lane == (unsigned int)__ffs(group) - 1u && gpuvm::ld_relaxed_u32(demand + vpn) < limit)
                atomicAdd(demand + vpn, (unsigned int)__popc(group));
        }
    }
}

// Grouped reads in place.  Rows read in place one lookup after the other are scattered over the whole table, and
// scattered reads over a large pinned region are slow on the host side (24.5 GB/s over 64 GiB against 51.4 for
// sequential ones); the same rows read page by page go at 50 GB/s.  So the lookups of the pages that are not
// fetched ("cold": fewer lookups than the limit) are bucketed by page first: bucket_off[p] becomes the start of page
// p's bucket (an exclusive scan of the cold pages' counts; one block, 1024 pages per step), the fill kernel puts
// every cold lookup's number into its page's bucket, and the main kernel reads the rows in bucket order.
// counts[0] = number of cold lookups, counts[1] = number of pages that will be fetched, counts[2] = cold lookups
// whose rows have been staged (counted up by the main kernel).
__global__ void __launch_bounds__(1024) embag_bucket_scan_kernel(const unsigned int *__restrict__ demand, unsigned int n_pages,
                                                                  unsigned int limit, unsigned int *__restrict__ bucket_off,
                                                                  unsigned int *__restrict__ counts)
{
    __shared__ unsigned int warp_sums[32];
    __shared__ unsigned int carry_s, hot_s;
    const unsigned int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) { carry_s = 0; hot_s = 0; }
    __syncthreads();
    unsigned int hot = 0;
    for (unsigned int base = 0; base < n_pages; base += 1024) {
        const unsigned int p = base + threadIdx.x;
        const unsigned int d = p < n_pages ? demand[p] : 0u, v = d < limit ? d : 0u;
        hot += p < n_pages && d >= limit;
        unsigned int x = v;                                      // inclusive scan in the warp
        for (int o = 1; o < 32; o <<= 1) { const unsigned int y = __shfl_up_sync(0xFFFFFFFFu, x, o); if (lane >= (unsigned int)o) x += y; }
        if (lane == 31) warp_sums[warp] = x;
        __syncthreads();
        if (warp == 0) {                                         // exclusive scan of the 32 warp totals
            const unsigned int t = warp_sums[lane];
            unsigned int e = t;
            for (int o = 1; o < 32; o <<= 1) { const unsigned int y = __shfl_up_sync(0xFFFFFFFFu, e, o); if (lane >= (unsigned int)o) e += y; }
            warp_sums[lane] = e - t;
        }
        __syncthreads();
        const unsigned int carry = carry_s;
        if (p < n_pages) bucket_off[p] = carry + warp_sums[warp] + x - v;
        __syncthreads();
        if (threadIdx.x == 1023) carry_s = carry + warp_sums[31] + x;
        __syncthreads();
    }
    for (int o = 16; o; o >>= 1) hot += __shfl_down_sync(0xFFFFFFFFu, hot, o);
    if (lane == 0 && hot) atomicAdd(&hot_s, hot);
    __syncthreads();
    if (threadIdx.x == 0) { counts[0] = carry_s; counts[1] = hot_s; counts[2] = 0; counts[4] = 0; counts[5] = 0; }
}

// After this kernel bucket_off[p] is the END of page p's bucket (every cold lookup moved it on by one).
__global__ void embag_bucket_fill_kernel(const long long *__restrict__ rows, unsigned long long n, unsigned long long t_off,
                                         unsigned long long row_bytes, unsigned int page_shift, unsigned long long rows_inside,
                                         const unsigned int *__restrict__ demand, unsigned int limit,
                                         unsigned int *__restrict__ bucket_off, unsigned int *__restrict__ cold_idx,
                                         unsigned int *__restrict__ where = nullptr)
{
    const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
    for (unsigned long long i = blockIdx.x * (unsigned long long)blockDim.x + threadIdx.x; i < n; i += stride) {
        const unsigned long long r = (unsigned long long)rows[i];
        if (r >= rows_inside) continue;
        const unsigned int vpn = (unsigned int)((t_off + r * row_bytes) >> page_shift);
        if (demand[vpn] < limit) {
            const unsigned int pos = atomicAdd(bucket_off + vpn, 1u);
            cold_idx[pos] = (unsigned int)i;
            if (where) where[i] = pos;                      // (where[] starts out as kNoSlot everywhere)
        }
    }
}

// Where the row of lookup i is staged when every requester warp has one item (one pass): the layout the main
// kernel's tables use (request ((gi * bag + k) * 32 + b) of the warp that has bag g0 + 32 gi + b).
__device__ __forceinline__ size_t embag_staged_row(unsigned long long i, unsigned int bag, unsigned int groups)
{
    const unsigned long long g = i / bag, per_item = 32ull * groups;
    const unsigned int k = (unsigned int)(i - g * bag);
    const unsigned long long t = g / per_item;
    const unsigned int rr = (unsigned int)(g - t * per_item), gi = rr >> 5, b = rr & 31u;
    return (size_t)t * ((size_t)groups * 32 * bag) + (size_t)((gi * bag + k) * 32 + b);
}

// The embedding bag when the pages that are worth fetching fit the pool twice over: no request tables, no copy of
// the rows of fetched pages.  counts: [0] cold lookups, [1] pages to fetch, [2] cold rows staged, [4] warps past
// step (1), [5] warps finished.
//   (1) every page at or above the limit gets the hold bit (the evictor passes over it until this kernel clears
//       the bit again) and, where it is not resident, is handed to the fault ring for the migrator warps;
//   (2) the rows of the other pages are read in place, in bucket order, into a staging area that holds just them
//       (cold_staging[j] for bucket entry j; where[i] = j for lookup i);
//   (3) when all warps are past (1) and all cold rows are staged, a warp adds up its bags in list order: a cold row
//       from the staging area, any other straight from its page's frame, without a reference (the hold bit
//       protects the frame), waiting (bounded) for pages that are still on their way;
//   (4) the last warp to finish clears the hold bits.
constexpr unsigned int kNoSlot = 0xFFFFFFFFu;
__global__ void __launch_bounds__(1024, 1) embag_direct_kernel(gpuvm_dev_t vm, unsigned long long t_off, unsigned int dims,
                                                               const long long *__restrict__ rows, unsigned long long n_bags,
                                                               unsigned int bag, float *__restrict__ out, int requesters,
                                                               gpuvm_shared_queue *shared_queue, unsigned int limit,
                                                               const unsigned int *__restrict__ demand,
                                                               const unsigned int *__restrict__ cold_idx,
                                                               const unsigned int *__restrict__ where, uint4 *cold_staging,
                                                               unsigned int *counts)
{
    __shared__ gpuvm_fault_queue queue_s;
    extern __shared__ __align__(128) unsigned char stage_s[];   // bulk-copy staging: kEmbagStages chunks per migrator warp
    __shared__ __align__(8) unsigned long long mbar_s[kEmbagMigrators][kEmbagStages];
    gpuvm_fault_queue *queue = &queue_s;
    const unsigned int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (unsigned int k = threadIdx.x; k < sizeof(gpuvm_fault_queue) / 4; k += blockDim.x)
        reinterpret_cast<unsigned int *>(queue)[k] = 0;
    __syncthreads();
    if (threadIdx.x == 0) { queue->requesters = (unsigned int)requesters; queue->shared = shared_queue; }
    __syncthreads();
    if ((int)warp >= requesters) {
        const unsigned int mig = warp - requesters;
        const unsigned int chunk = (1ull << vm.page_shift) < kEmbagChunk ? (unsigned int)(1ull << vm.page_shift) : kEmbagChunk;
        if (mig < kEmbagMigrators && chunk >= 128)
            gpuvm_migrator_loop(vm, queue, stage_s + (size_t)mig * kEmbagStages * kEmbagChunk, mbar_s[mig], chunk, kEmbagStages);
        else
            gpuvm_migrator_loop(vm, queue);
        return;
    }
    const unsigned int q = dims >> 2;                            // 16-byte pieces per row
    const unsigned long long row_bytes = 4ull * dims;
    const unsigned long long slot = (unsigned long long)blockIdx.x * requesters + warp;
    const unsigned long long stride = (unsigned long long)gridDim.x * requesters;
    const unsigned long long rows_inside = (vm.bytes - t_off) / row_bytes;
    const unsigned int n_cold = counts[0];
    const unsigned long long limit_ns = (unsigned long long)vm.spin_limit_us * 1000ull;

    // hand page p to the migrators: the caller has turned its entry BUSY
    auto push = [&](unsigned long long p) {
        unsigned long long t0 = 0;
        while (!gpuvm::fault_queue_push(queue, (unsigned int)p, gpuvm::kRead, &vm)) {
            const unsigned long long now = gpuvm::now_ns();
            if (t0 == 0) t0 = now;
            if (now - t0 > limit_ns || gpuvm::has_error(vm)) {
                gpuvm::set_error(vm, GPUVM_E_TIMEOUT, p);
                atomicXor(vm.pte + p, gpuvm::kBusy);             // back to INVALID
                return;
            }
            __nanosleep(256);
        }
    };

    // (1)
    for (unsigned long long p = slot * 32 + lane; p < vm.n_pages; p += stride * 32) {
        if (demand[p] < limit) continue;
        const unsigned long long w = atomicOr(vm.pte + p, gpuvm::kHold) | gpuvm::kHold;
        if ((w & gpuvm::kStMask) == gpuvm::kInvalid && atomicCAS(vm.pte + p, w, (w & ~gpuvm::kFrameMask) | gpuvm::kBusy) == w)
            push(p);
    }
    __threadfence();
    __syncwarp();
    if (lane == 0) atomicAdd(counts + 4, 1u);

    // (2)
    unsigned int n_here = 0;
    constexpr int Q = 4;
    for (unsigned long long j0 = slot * Q; j0 < n_cold; j0 += stride * Q) {
        uint4 v[Q];
        int cnt = 0;
#pragma unroll
        for (int u = 0; u < Q; ++u)
            if (j0 + u < n_cold) {
                const unsigned long long r = (unsigned long long)rows[cold_idx[j0 + u]];
                if (lane < q) v[u] = gpuvm_load16(vm.host + t_off + r * row_bytes + 16u * lane);
                cnt = u + 1;
            }
#pragma unroll
        for (int u = 0; u < Q; ++u)
            if (u < cnt && lane < q) cold_staging[(j0 + u) * q + lane] = v[u];
        n_here += cnt;
    }
    if (lane == 0 && n_here) gpuvm::stat_add(vm, gpuvm::kBytesDirect, (unsigned long long)n_here * row_bytes);
    __threadfence();
    __syncwarp();
    if (lane == 0 && n_here) atomicAdd(counts + 2, n_here);

    // (3) wait for the stragglers of (1) and (2)
    {
        unsigned long long t0 = 0;
        bool ok = true;
        while (ld_volatile_u32(counts + 2) < n_cold || ld_volatile_u32(counts + 4) < (unsigned int)stride) {
            const unsigned long long now = gpuvm::now_ns();
            if (t0 == 0) t0 = now;
            if (now - t0 > limit_ns || gpuvm::has_error(vm)) { ok = false; break; }
            __nanosleep(256);
        }
        if (!__all_sync(0xFFFFFFFFu, ok) && lane == 0) gpuvm::set_error(vm, GPUVM_E_TIMEOUT, ~0ull);
        __threadfence();
    }
    for (unsigned long long g = slot; g < n_bags && !gpuvm::has_error(vm); g += stride) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (unsigned int k0 = 0; k0 < bag; k0 += 32) {
            const unsigned int nk = bag - k0 < 32u ? bag - k0 : 32u;
            // lane k finds where the row of lookup k0 + k is
            const unsigned char *src = nullptr;
            if (lane < nk) {
                const unsigned long long i = g * bag + k0 + lane;
                const unsigned long long r = (unsigned long long)rows[i];
                const unsigned int at = where[i];
                if (at != kNoSlot) {
                    src = reinterpret_cast<const unsigned char *>(cold_staging) + (size_t)at * row_bytes;
                } else if (r >= rows_inside) {
                    gpuvm::set_error(vm, GPUVM_E_RANGE, ~0ull);   // a row past the end of the table: nothing is added for it
                } else {
                    const unsigned long long byte_off = t_off + r * row_bytes, p = byte_off >> vm.page_shift;
                    unsigned long long t0 = 0;
                    for (;;) {
                        const unsigned long long w = gpuvm::ld_acquire_u64(vm.pte + p);
                        const unsigned long long st = w & gpuvm::kStMask;
                        if (st == gpuvm::kValid) {
                            src = vm.pool + (((w & gpuvm::kFrameMask) >> gpuvm::kFrameShift) << vm.page_shift) +
                                  (byte_off & ((1ull << vm.page_shift) - 1ull));
                            break;
                        }
                        // nobody has asked for it (it was being evicted when (1) looked): ask now
                        if (st == gpuvm::kInvalid && atomicCAS(vm.pte + p, w, (w & ~gpuvm::kFrameMask) | gpuvm::kBusy) == w) push(p);
                        const unsigned long long now = gpuvm::now_ns();
                        if (t0 == 0) t0 = now;
                        if (now - t0 > limit_ns || gpuvm::has_error(vm)) { gpuvm::set_error(vm, GPUVM_E_TIMEOUT, p); break; }
                        __nanosleep(128);
                    }
                }
            }
            __syncwarp();
            // the rows, in list order, eight loads in flight
            for (unsigned int k = 0; k < nk; k += 8) {
                uint4 v[8];
#pragma unroll
                for (unsigned int u = 0; u < 8; ++u) {
                    const unsigned char *s = reinterpret_cast<const unsigned char *>(
                        __shfl_sync(0xFFFFFFFFu, reinterpret_cast<unsigned long long>(src), (k + u) & 31u));
                    v[u] = make_uint4(0u, 0u, 0u, 0u);
                    if (k + u < nk && s != nullptr && lane < q) v[u] = gpuvm_load16(s + 16u * lane);
                }
#pragma unroll
                for (unsigned int u = 0; u < 8; ++u)
                    if (k + u < nk) {
                        acc.x = __fadd_rn(acc.x, __uint_as_float(v[u].x));
                        acc.y = __fadd_rn(acc.y, __uint_as_float(v[u].y));
                        acc.z = __fadd_rn(acc.z, __uint_as_float(v[u].z));
                        acc.w = __fadd_rn(acc.w, __uint_as_float(v[u].w));
                    }
            }
        }
        if (lane < q) reinterpret_cast<float4 *>(out + g * dims)[lane] = acc;
    }

    // (4) the last warp to get here lets the pages go
    __syncwarp();
    unsigned int done = 0;
    if (lane == 0) done = atomicAdd(counts + 5, 1u) + 1u;
    done = __shfl_sync(0xFFFFFFFFu, done, 0);
    if (done == (unsigned int)stride)
        for (unsigned long long p = lane; p < vm.n_pages; p += 32)
            if (demand[p] >= limit) atomicAnd(vm.pte + p, ~gpuvm::kHold);
    if (lane == 0) gpuvm_requester_done(queue);
}

// All 32 lanes: add the staged rows of the warp's bags g0 .. g0 + 32 groups - 1 in list order (lookups k of this
// batch, nk of them; `first`: the batch starts the bag, otherwise it adds to what is in out).
__device__ __forceinline__ void embag_add_bags(const uint4 *staging, float *__restrict__ out, unsigned int dims, unsigned int q,
                                               unsigned long long g0, unsigned long long n_bags, unsigned int groups,
                                               unsigned int nk, bool first, unsigned int lane)
{
    for (unsigned int gb = 0; gb < 32 * groups && g0 + gb < n_bags; ++gb) {
        if (lane < q) {
            const unsigned int gi = gb >> 5, b = gb & 31;
            float4 *dst = reinterpret_cast<float4 *>(out + (g0 + gb) * dims) + lane;
            float4 acc = first ? make_float4(0.f, 0.f, 0.f, 0.f) : *dst;
#pragma unroll 8
            for (unsigned int k = 0; k < nk; ++k) {
                const uint4 v = __ldcg(staging + (size_t)((gi * nk + k) * 32 + b) * q + lane);   // some may have been staged by other warps
                acc.x = __fadd_rn(acc.x, __uint_as_float(v.x));
                acc.y = __fadd_rn(acc.y, __uint_as_float(v.y));
                acc.z = __fadd_rn(acc.z, __uint_as_float(v.z));
                acc.w = __fadd_rn(acc.w, __uint_as_float(v.w));
            }
            *dst = acc;
        }
    }
}

__global__ void __launch_bounds__(1024, 1) embag_batch_kernel(gpuvm_dev_t vm, unsigned long long t_off, unsigned int dims,
                                                              const long long *__restrict__ rows, unsigned long long n_bags,
                                                              unsigned int bag, float *__restrict__ out, int requesters,
                                                              gpuvm_batch_entry *g_tables, unsigned char *g_staging,
                                                              unsigned int groups, bool one_pass,
                                                              gpuvm_shared_queue *shared_queue, unsigned int inplace_limit,
                                                              const unsigned int *demand, const unsigned int *cold_idx,
                                                              const unsigned int *cold_counts)
{
    __shared__ gpuvm_fault_queue queue_s;
    extern __shared__ __align__(128) unsigned char stage_s[];   // bulk-copy staging: kEmbagStages chunks per migrator warp
    __shared__ __align__(8) unsigned long long mbar_s[kEmbagMigrators][kEmbagStages];
    gpuvm_fault_queue *queue = &queue_s;
    const unsigned int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (unsigned int k = threadIdx.x; k < sizeof(gpuvm_fault_queue) / 4; k += blockDim.x)
        reinterpret_cast<unsigned int *>(queue)[k] = 0;
    __syncthreads();
    if (threadIdx.x == 0) { queue->requesters = (unsigned int)requesters; queue->shared = shared_queue; }
    __syncthreads();
    if ((int)warp >= requesters) {
        const unsigned int mig = warp - requesters;
        const unsigned int chunk = (1ull << vm.page_shift) < kEmbagChunk ? (unsigned int)(1ull << vm.page_shift) : kEmbagChunk;
        if (mig < kEmbagMigrators && chunk >= 128)
            gpuvm_migrator_loop(vm, queue, stage_s + (size_t)mig * kEmbagStages * kEmbagChunk, mbar_s[mig], chunk, kEmbagStages);
        else
            gpuvm_migrator_loop(vm, queue);
        return;
    }
    const unsigned int q = dims >> 2;                            // 16-byte pieces per row
    const unsigned long long row_bytes = 4ull * dims;
    const size_t slot = (size_t)blockIdx.x * requesters + warp;
    const size_t per_warp = (size_t)groups * 32 * (bag < kEmbagLookups ? bag : kEmbagLookups);
    gpuvm_batch_entry *table = g_tables + slot * per_warp;
    uint4 *staging = reinterpret_cast<uint4 *>(g_staging + slot * per_warp * row_bytes);
    unsigned long long masks[2 * ((kEmbagMaxGroups * kEmbagLookups + 63) / 64)];
    const unsigned long long per_item = 32ull * groups;
    const unsigned long long items = (n_bags + per_item - 1) / per_item;
    const unsigned long long stride = (unsigned long long)gridDim.x * requesters;
    const unsigned long long rows_inside = (vm.bytes - t_off) / row_bytes;   // rows that lie in the backing store entirely
    const bool grouped = cold_idx != nullptr;                    // one pass, every lookup's staging slot is known (embag_staged_row)
    if (grouped) {
        // (1) The pages that will be fetched are asked for up front, so that the migrator warps move them while the
        // requesters read the other pages' rows: a warp looks at its share of the page counts and hands every
        // page at or above the limit that nobody has asked for yet to the fault ring.  Not when those pages
        // would fill more than half the pool: then they are fetched as their lookups come up.
        const unsigned int n_cold = cold_counts[0], n_hot = cold_counts[1];
        if (2ull * n_hot <= vm.n_frames) {
            for (unsigned long long p = slot * 32 + lane; p < vm.n_pages; p += stride * 32) {
                if (demand[p] < inplace_limit) continue;
                const unsigned long long w = gpuvm::ld_relaxed_u64(vm.pte + p);
                if ((w & gpuvm::kStMask) != gpuvm::kInvalid) continue;
                if (atomicCAS(vm.pte + p, w, (w & ~gpuvm::kFrameMask) | gpuvm::kBusy) != w) continue;
                if (!gpuvm::fault_queue_push(queue, (unsigned int)p, gpuvm::kRead, &vm))
                    atomicXor(vm.pte + p, gpuvm::kBusy);         // the ring is full: back to INVALID, its lookups will fetch it
            }
            __syncwarp();
        }
        // (2) The rows of the other pages, in bucket order (page by page), four in flight per warp; the warps of
        // the grid take neighbouring entries, so at any moment the reads in flight fall into a few hundred pages.
        // A warp reads its whole share first and then runs the engine over its lookups of the fetched pages, which
        // have arrived by then (running the engine after 30, 50 or 70 % of the share was measured: 52 / 49 / 49 ms
        // against 44-45).
        unsigned int n_here = 0;
        constexpr int Q = 4;                                     // (2, 4 and 8 rows in flight per warp: the same 44-46 ms)
        uint4 *const all_staging = reinterpret_cast<uint4 *>(g_staging);
        auto read_in_place = [&](unsigned long long j_begin, unsigned long long j_end) {
            for (unsigned long long j0 = j_begin + slot * Q; j0 < j_end; j0 += stride * Q) {
                uint4 v[Q];
                size_t where[Q];
                int cnt = 0;
#pragma unroll
                for (int u = 0; u < Q; ++u) {
                    where[u] = 0;
                    if (j0 + u < j_end) {
                        const unsigned int i = cold_idx[j0 + u];
                        const unsigned long long r = (unsigned long long)rows[i];
                        where[u] = embag_staged_row(i, bag, groups) * q;
                        if (lane < q) v[u] = gpuvm_load16(vm.host + t_off + r * row_bytes + 16u * lane);
                        cnt = u + 1;
                    }
                }
#pragma unroll
                for (int u = 0; u < Q; ++u)
                    if (u < cnt && lane < q) all_staging[where[u] + lane] = v[u];
                n_here += cnt;
            }
        };
        read_in_place(0, n_cold);
        if (lane == 0 && n_here) gpuvm::stat_add(vm, gpuvm::kBytesDirect, (unsigned long long)n_here * row_bytes);
        // the rows are in their slots for everybody before they are counted as staged
        __threadfence();
        __syncwarp();
        if (lane == 0 && n_here) atomicAdd(const_cast<unsigned int *>(cold_counts) + 2, n_here);
        const unsigned long long t = slot, g0 = per_item * t;
        const unsigned int nk = bag;                             // one pass: bag <= kEmbagLookups, one item per warp
        if (t < items) {
            for (unsigned int gi = 0; gi < groups; ++gi)
                for (unsigned int k = 0; k < nk; ++k) {
                    const unsigned long long g = g0 + 32ull * gi + lane;
                    const unsigned int at = (gi * nk + k) * 32 + lane;
                    if (g < n_bags) {
                        const unsigned long long r = (unsigned long long)rows[g * bag + k];
                        const bool inside = r < rows_inside;
                        if (inside && demand[(t_off + r * row_bytes) >> vm.page_shift] < inplace_limit)
                            gpuvm_batch_skip(table, at);                     // its row is staged by read_in_place
                        else
                            gpuvm_batch_set(vm, table, at, inside ? t_off + r * row_bytes : ~0ull);
                    } else
                        gpuvm_batch_skip(table, at);
                }
            __syncwarp();
            gpuvm_batch_run<true>(vm, gpuvm_entry_table{table}, groups * nk * 32, GPUVM_READ, gpuvm_row_copy{staging, q},
                                  queue, masks, 1u, true, 0u, (unsigned int)row_bytes, nullptr);
            __syncwarp();
        }
        // A bag's rows that were read in place were staged by whichever warps had their bucket entries: wait
        // (bounded) until all of them are counted as staged.  Every warp stages its share before it comes here,
        // so the wait is for the stragglers of the grid only.  (The shares are fixed, not drawn from a counter:
        // warps get through theirs at different speeds, and the early ones add up their bags while the others
        // keep the link busy; with a counter all warps finished reading together and all that came after it.)
        if (t < items) {
            const unsigned long long limit_ns = (unsigned long long)vm.spin_limit_us * 1000ull;
            unsigned long long t0 = 0;
            bool ok = true;
            while (ld_volatile_u32(cold_counts + 2) < n_cold) {
                const unsigned long long now = gpuvm::now_ns();
                if (t0 == 0) t0 = now;
                if (now - t0 > limit_ns || gpuvm::has_error(vm)) { ok = false; break; }
                __nanosleep(256);
            }
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) { if (lane == 0) gpuvm::set_error(vm, GPUVM_E_TIMEOUT, ~0ull); }
            else {
                __threadfence();
                embag_add_bags(staging, out, dims, q, g0, n_bags, groups, nk, /* first = */ true, lane);
            }
        }
        if (lane == 0) gpuvm_requester_done(queue);
        return;
    }
    for (unsigned long long t = slot; t < items; t += stride) {
        const unsigned long long g0 = per_item * t;
        for (unsigned int k0 = 0; k0 < bag; k0 += kEmbagLookups) {
            const unsigned int nk = bag - k0 < kEmbagLookups ? bag - k0 : kEmbagLookups;
            // request ((gi * nk + k) * 32 + b): lookup k0 + k of bag g0 + 32 gi + b
            for (unsigned int gi = 0; gi < groups; ++gi)
                for (unsigned int k = 0; k < nk; ++k) {
                    const unsigned long long g = g0 + 32ull * gi + lane;
                    if (g < n_bags) {
                        // a row that ends past the backing store is refused like one that starts there
                        const unsigned long long r = (unsigned long long)rows[g * bag + k0 + k];
                        const bool inside = r < rows_inside;
                        gpuvm_batch_set(vm, table, (gi * nk + k) * 32 + lane, inside ? t_off + r * row_bytes : ~0ull);
                    } else
                        gpuvm_batch_skip(table, (gi * nk + k) * 32 + lane);
                }
            __syncwarp();
            // every served row is copied to its slot of the staging area by the whole warp (the engine does it
            // itself, four rows in flight: gpuvm_row_copy), from its frame or in place from the backing store
            gpuvm_batch_run<true>(vm, gpuvm_entry_table{table}, groups * nk * 32, GPUVM_READ, gpuvm_row_copy{staging, q},
                                  queue, masks, 1u, one_pass, inplace_limit, (unsigned int)row_bytes, demand);
            __syncwarp();
            embag_add_bags(staging, out, dims, q, g0, n_bags, groups, nk, k0 == 0, lane);
            __syncwarp();
        }
    }
    if (lane == 0) gpuvm_requester_done(queue);
}

// ------------------------------------------------------- element read-modify-write
template <class Mem>
__global__ void __launch_bounds__(256) scatter_update_kernel(Mem m, unsigned long long a_off,
                                                             const long long *__restrict__ idx, unsigned long long n)
{
    const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
    for (unsigned long long k = blockIdx.x * (unsigned long long)blockDim.x + threadIdx.x; k < n; k += stride) {
        const unsigned long long i = (unsigned long long)idx[k];
        unsigned int v = m.template read<unsigned int>(a_off, i);
        m.template write<unsigned int>(a_off, i, v * 3u + 1u);
    }
}

// The same update with batched requests and no helper warps: every warp stages 1024 requests in
// shared memory and migrates the pages of the faults it owns itself.
__global__ void __launch_bounds__(128) scatter_update_batch_kernel(gpuvm_dev_t vm, unsigned long long a_off,
                                                                   const long long *__restrict__ idx, unsigned long long n)
{
    __shared__ gpuvm_batch_entry s_table[4][1024];
    const unsigned int lane = threadIdx.x & 31;
    gpuvm_batch_entry *table = s_table[threadIdx.x >> 5];
    const unsigned long long batches = (n + 1023) / 1024;
    for (unsigned long long t = warp_in_grid(); t < batches; t += warps_in_grid()) {
        const unsigned long long base = t * 1024;
        const unsigned int m = (unsigned int)(n - base < 1024 ? n - base : 1024);
        for (unsigned int k = lane; k < m; k += 32)
            gpuvm_batch_set(vm, table, k, a_off + 4ull * (unsigned long long)idx[base + k]);
        __syncwarp();
        gpuvm_batch_access(vm, table, m, GPUVM_WRITE, [](unsigned int, const unsigned char *p) {
            unsigned int *q = reinterpret_cast<unsigned int *>(const_cast<unsigned char *>(p));
            gpuvm_store(q, gpuvm_load(q) * 3u + 1u);
        });
        __syncwarp();
    }
}

// The same update with the block's fault ring: six requester warps with 512 requests each, two
// migrator warps (write mode: victims are dirty and are written back by the migrators; pages come
// in by bulk copy).
constexpr int kScatterRequesters = 6;
constexpr int kScatterMigrators = 2;
constexpr unsigned int kScatterBatch = 512;
constexpr unsigned int kScatterChunk = 4096;

__global__ void __launch_bounds__((kScatterRequesters + kScatterMigrators) * 32)
scatter_update_queued_kernel(gpuvm_dev_t vm, unsigned long long a_off, const long long *__restrict__ idx,
                             unsigned long long n, gpuvm_shared_queue *shared_queue)
{
    __shared__ gpuvm_fault_queue queue_s;
    __shared__ gpuvm_batch_entry s_table[kScatterRequesters][kScatterBatch];
    __shared__ __align__(128) unsigned char stage_s[kScatterMigrators][kScatterChunk];
    __shared__ __align__(8) unsigned long long mbar_s[kScatterMigrators];
    gpuvm_fault_queue *queue = &queue_s;
    const unsigned int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (unsigned int k = threadIdx.x; k < sizeof(gpuvm_fault_queue) / 4; k += blockDim.x)
        reinterpret_cast<unsigned int *>(queue)[k] = 0;
    __syncthreads();
    if (threadIdx.x == 0) { queue->requesters = kScatterRequesters; queue->shared = shared_queue; }
    __syncthreads();
    if (warp >= kScatterRequesters) {
        const unsigned int mig = warp - kScatterRequesters;
        const unsigned int chunk = (1ull << vm.page_shift) < kScatterChunk ? (unsigned int)(1ull << vm.page_shift) : kScatterChunk;
        if (chunk >= 128) gpuvm_migrator_loop(vm, queue, stage_s[mig], &mbar_s[mig], chunk, 1);
        else gpuvm_migrator_loop(vm, queue);
        return;
    }
    gpuvm_batch_entry *table = s_table[warp];
    const unsigned long long batches = (n + kScatterBatch - 1) / kScatterBatch;
    const unsigned long long stride = (unsigned long long)gridDim.x * kScatterRequesters;
    for (unsigned long long t = (unsigned long long)blockIdx.x * kScatterRequesters + warp; t < batches; t += stride) {
        const unsigned long long base = t * kScatterBatch;
        const unsigned int m = (unsigned int)(n - base < kScatterBatch ? n - base : kScatterBatch);
        for (unsigned int k = lane; k < m; k += 32)
            gpuvm_batch_set(vm, table, k, a_off + 4ull * (unsigned long long)idx[base + k]);
        __syncwarp();
        gpuvm_batch_access(vm, table, m, GPUVM_WRITE, [](unsigned int, const unsigned char *p) {
            unsigned int *q = reinterpret_cast<unsigned int *>(const_cast<unsigned char *>(p));
            gpuvm_store(q, gpuvm_load(q) * 3u + 1u);
        }, queue);
        __syncwarp();
    }
    if (lane == 0) gpuvm_requester_done(queue);
}

// ------------------------------------------------------------------ page touch
__global__ void __launch_bounds__(256, 2) touch_pages_kernel(gpuvm_dev_t vm, unsigned long long first_page, unsigned long long n_pages)
{
    for (unsigned long long p = warp_in_grid(); p < n_pages; p += warps_in_grid()) {
        gpuvm_token tok;
        void *ptr = gpuvm_ptr(vm, (first_page + p) << vm.page_shift, GPUVM_READ, &tok);
        if (ptr) gpuvm_release(vm, tok);
    }
}

// --------------------------------------------------------------- link kernels
__global__ void link_in_kernel(const uint4 *__restrict__ src, uint4 *__restrict__ dst, size_t n16)
{
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t base = blockIdx.x * (size_t)blockDim.x + threadIdx.x; base < n16; base += stride * 8) {
        uint4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) { size_t i = base + u * stride; if (i < n16) v[u] = gpuvm::ld_host16(src + i); }
#pragma unroll
        for (int u = 0; u < 8; ++u) { size_t i = base + u * stride; if (i < n16) gpuvm::st_frame16(dst + i, v[u]); }
    }
}

// Scattered rows over the link: row i of the launch is a hashed row of the host region; a warp has four rows in
// flight (16 bytes per lane and row).  What a workload that reads rows in place can reach at most.  With
// run > 1, `run` consecutive rows of the launch fall into the same 2 MiB of the region (a hashed 2 MiB block, hashed
// rows inside it): the access pattern of rows that have been bucketed by page.
__device__ __forceinline__ unsigned long long splitmix64(unsigned long long z)
{
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

__global__ void link_scattered_kernel(const unsigned char *__restrict__ host, unsigned long long host_rows, unsigned int units16,
                                      unsigned long long n_rows, unsigned long long seed, unsigned int run, uint4 *__restrict__ dst,
                                      unsigned long long dst_rows)
{
    const unsigned int lane = threadIdx.x & 31;
    const unsigned long long warp = (blockIdx.x * (unsigned long long)blockDim.x + threadIdx.x) >> 5;
    const unsigned long long warps = ((unsigned long long)gridDim.x * blockDim.x) >> 5;
    const unsigned long long row_bytes = 16ull * units16;
    const unsigned long long block_rows = (2ull << 20) / row_bytes, blocks = host_rows / block_rows;
    for (unsigned long long i = warp * 4; i < n_rows; i += warps * 4) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            unsigned long long r = splitmix64(seed + (i + u) * 0x9E3779B97F4A7C15ull) % host_rows;
            if (run > 1 && blocks > 0)
                r = (splitmix64(seed ^ ((i + u) / run)) % blocks) * block_rows + splitmix64(seed + i + u) % block_rows;
            if (i + u < n_rows && lane < units16)
                v[u] = gpuvm::ld_host16(reinterpret_cast<const uint4 *>(host + r * row_bytes) + lane);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (i + u < n_rows && lane < units16) gpuvm::st_frame16(dst + ((i + u) % dst_rows) * units16 + lane, v[u]);
    }
}

__global__ void link_out_kernel(const uint4 *__restrict__ src, uint4 *__restrict__ dst, size_t n16)
{
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t base = blockIdx.x * (size_t)blockDim.x + threadIdx.x; base < n16; base += stride * 8) {
        uint4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) { size_t i = base + u * stride; if (i < n16) v[u] = gpuvm::ld_frame16(src + i); }
#pragma unroll
        for (int u = 0; u < 8; ++u) { size_t i = base + u * stride; if (i < n16) gpuvm::st_host16(dst + i, v[u]); }
    }
}

// even blocks read the first half of the host buffer, odd blocks write the second half
__global__ void link_duplex_kernel(uint4 *host, uint4 *dev, size_t n16)
{
    const size_t half = n16 / 2;
    const size_t stride = (size_t)(gridDim.x / 2) * blockDim.x;
    const size_t t = (blockIdx.x / 2) * (size_t)blockDim.x + threadIdx.x;
    if (blockIdx.x & 1) {
        for (size_t i = t; i < half; i += stride) gpuvm::st_host16(host + half + i, gpuvm::ld_frame16(dev + half + i));
    } else {
        for (size_t base = t; base < half; base += stride * 8) {
            uint4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) { size_t i = base + u * stride; if (i < half) v[u] = gpuvm::ld_host16(host + i); }
#pragma unroll
            for (int u = 0; u < 8; ++u) { size_t i = base + u * stride; if (i < half) gpuvm::st_frame16(dev + i, v[u]); }
        }
    }
}

int sm_count()
{
    static int sms = 0;
    if (!sms) {
        int dev = 0;
        cudaGetDevice(&dev);
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) sms = 148;
    }
    return sms;
}

int launched(unsigned long long n = 1)
{
    gpuvm_note_launch_(n);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? GPUVM_OK : GPUVM_E_CUDA;
}

// The grid-wide fault ring of a batched kernel, zeroed on the stream; nullptr when pages are
// small.  Sharing the backlog pays when one page takes a migrator warp long to move (a 2 MiB
// page: 0.8 ms, so a block that owns more faults than the others finishes long after them:
// 1.52 s -> 1.34 s on the embedding bag); with 64 KiB pages the blocks' backlogs even out by
// themselves and the extra migrators only add to the contention for frames (23.2 -> 24.0 ms
// on the gather).
constexpr size_t kSharedQueueMinPage = size_t(256) << 10;

gpuvm_shared_queue *shared_queue_at(const gpuvm_dev_t &vm, unsigned char *where, cudaStream_t stream)
{
    if ((size_t(1) << vm.page_shift) < kSharedQueueMinPage) return nullptr;
    if (cudaMemsetAsync(where, 0, sizeof(gpuvm_shared_queue), stream) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    return reinterpret_cast<gpuvm_shared_queue *>(where);
}

bool view_of(gpuvm_t h, Paged &m) { return h && gpuvm_device_view(h, &m.vm) == GPUVM_OK; }

// The number of edges is the last row offset; it is read from the backing store on the host
// (row offsets are never written) and only bounds the sweeps' prefetches.
void hint_edges(gpuvm_t h, Paged &m, size_t off_off, size_t nv)
{
    const unsigned char *host = static_cast<const unsigned char *>(gpuvm_host_ptr(h));
    if (!host || off_off + 8 * (nv + 1) > m.vm.bytes) return;
    long long ne = 0;
    memcpy(&ne, host + off_off + 8 * nv, sizeof(ne));
    if (ne > 0) m.edges_hint = (unsigned long long)ne;
}

template <class Mem>
int run_stream_sum(const Mem &m, size_t a_off, size_t n, int64_t *d_sum, cudaStream_t s)
{
    if (!d_sum) return GPUVM_E_ARG;
    if (a_off % 16) return GPUVM_E_ALIGN;
    if (cudaMemsetAsync(d_sum, 0, sizeof(int64_t), s) != cudaSuccess) { cudaGetLastError(); return GPUVM_E_CUDA; }
    if (n == 0) return GPUVM_OK;
    // Pages per warp at a time: as many as the pool lets every warp of the grid hold at once (a warp that
    // holds pins while it faults needs a free frame), at most four.
    const int blocks = sm_count() * 4, warps = blocks * 8;
    int g = m.pins_per_warp(warps, 4);
    unsigned long long *out = reinterpret_cast<unsigned long long *>(d_sum);
    if (g >= 4) stream_sum_kernel<Mem, 4><<<blocks, 256, 0, s>>>(m, a_off, n, out);
    else if (g >= 2) stream_sum_kernel<Mem, 2><<<blocks, 256, 0, s>>>(m, a_off, n, out);
    else stream_sum_kernel<Mem, 1><<<blocks, 256, 0, s>>>(m, a_off, n, out);
    return launched();
}

template <class Mem>
int run_gather(const Mem &m, size_t x_off, const int64_t *d_idx, size_t n_idx, size_t block, float *d_fsum,
               int64_t *d_bsum, cudaStream_t s)
{
    if (!d_idx || !d_fsum || !d_bsum || block == 0 || block > (size_t(1) << 20)) return GPUVM_E_ARG;
    if (x_off % 16) return GPUVM_E_ALIGN;
    if (n_idx == 0) return GPUVM_OK;
    size_t nb = (n_idx + block - 1) / block;
    unsigned int threads = block >= 256 ? 256u : (unsigned int)((block + 31) / 32 * 32);
    size_t resident = (size_t)sm_count() * (256 * kGatherPlainBlocksPerSm / threads);
    unsigned int grid = (unsigned int)(nb < resident ? nb : resident);
    gather_kernel<Mem><<<grid, threads, 0, s>>>(m, x_off, reinterpret_cast<const long long *>(d_idx), n_idx, block,
                                                 d_fsum, reinterpret_cast<long long *>(d_bsum));
    return launched();
}

constexpr int kVaddBlocksPerSm = 4;
constexpr size_t kBfsScratchBytes = 4 * kBigQueue * sizeof(long long) + kCntWords * sizeof(unsigned int);

// Scratch of the sweeps: queue of pieces, counters, then (label-correcting runs) the queue of vertices
// lowered behind the sweep position.
constexpr size_t kBehindMin = 1u << 16;
size_t behind_capacity(size_t nv, bool weighted)
{
    // with weights a vertex is lowered several times per sweep (every shorter path found), with unit lengths about once
    const size_t want = weighted ? nv / 2 : nv / 4;
    return want > kBehindMin ? want : kBehindMin;
}
size_t lc_scratch_bytes(size_t nv, bool weighted) { return kBfsScratchBytes + behind_capacity(nv, weighted) * sizeof(unsigned int); }

// One sweep and its update count.  `sweep` counts from 0 within a call.
template <class Mem, class Op, bool WEIGHTED>
int graph_sweep(const Mem &m, const Op &op, size_t off_off, size_t col_off, size_t w_off, size_t nv, void *scratch, int sweep,
                unsigned int *updates, cudaStream_t s, int backward = -1)
{
    if (backward < 0) backward = sweep & 1;                  // odd sweeps run downwards
    // number of edges = last row offset; only used to keep prefetches inside the column array
    const unsigned long long n_edges = m.edges_hint;
    long long *span_q = static_cast<long long *>(scratch);
    unsigned int *counters = reinterpret_cast<unsigned int *>(span_q + 4 * kBigQueue);
    // paged: 4 blocks per SM; over managed memory a narrower window of 2 blocks per SM is 10x faster
    const int grid = sm_count() * Mem::kSweepBlocksPerSm;
    if (sweep == 0) cudaMemsetAsync(span_q, 0, 4 * kBigQueue * sizeof(long long), s);     // ready words: once per call
    cudaMemsetAsync(counters, 0, kCntWords * sizeof(unsigned int), s);
    graph_sweep_kernel<Mem, Op, WEIGHTED><<<grid, 256, 0, s>>>(m, op, off_off, col_off, w_off, (unsigned int)nv, n_edges, span_q, counters, sweep, backward);
    int rc = launched(1);
    static const bool trace = getenv("GPUVM_TRACE_SWEEPS") != nullptr;     // one line per sweep on stderr
    unsigned int host_counters[kCntWords] = {0};
    const size_t want = trace ? sizeof(host_counters) : 2 * sizeof(unsigned int);
    const auto t0 = std::chrono::steady_clock::now();
    if (cudaMemcpyAsync(host_counters, counters, want, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess) { cudaGetLastError(); return GPUVM_E_CUDA; }
    if (trace)
        fprintf(stderr, "sweep %d: %.3f ms (host clock, from launch to counters read), updates %u, pieces %u/%u, chunks done %u, "
                        "behind queued %u taken %u\n", sweep,
                std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now() - t0).count(), host_counters[kCntUpdates],
                host_counters[kCntTaken], host_counters[kCntPushed], host_counters[kCntDone], host_counters[kCntBehindTail],
                host_counters[kCntBehindHead]);
    *updates = host_counters[0];
    return rc;
}

// One level-synchronous BFS on caller-provided scratch (kBfsScratchBytes, 16-byte aligned): one sweep per level.
template <class Mem>
int bfs_levels(const Mem &m, size_t off_off, size_t col_off, size_t nv, size_t source, int32_t *d_level, int *n_levels,
               void *scratch, cudaStream_t s)
{
    cudaMemsetAsync(d_level, 0xFF, nv * sizeof(int32_t), s);
    bfs_init_kernel<<<1, 1, 0, s>>>(d_level, (int)source);
    int rc = launched();
    int depth = 0;
    unsigned int found = 1;
    while (rc == GPUVM_OK && found > 0) {
        rc = graph_sweep<Mem, BfsOp, false>(m, BfsOp{d_level, depth}, off_off, col_off, 0, nv, scratch, depth, &found, s);
        ++depth;
    }
    if (n_levels) *n_levels = depth;
    return rc;
}

// Label-correcting sweeps until nothing changes (BFS: unit lengths; SSSP: the weights at w_off).  d_dist holds
// the packed words while the sweeps run and the distances afterwards.  scratch: lc_scratch_bytes(nv, WEIGHTED).
// *max_dist receives the largest distance reached.
template <class Mem, bool WEIGHTED>
int lc_sweeps(const Mem &m, size_t off_off, size_t col_off, size_t w_off, size_t nv, size_t source, int32_t *d_dist,
              int unreached, int *n_sweeps, unsigned int *max_dist, void *scratch, cudaStream_t s)
{
    unsigned int *counters = reinterpret_cast<unsigned int *>(static_cast<long long *>(scratch) + 4 * kBigQueue);
    unsigned int *behind_q = counters + kCntWords;
    // Over plain pointers (the managed-memory twin) the queue is off: re-expanding vertices at random places
    // behind the sweep is only cheap when one can ask whether their pages are resident, which a plain pointer
    // cannot; there the vertices simply stay dirty for the next sweep.
    const unsigned int cap = Mem::kBehindQueue ? (unsigned int)behind_capacity(nv, WEIGHTED) : 0u;
    lc_init_kernel<<<sm_count() * 4, 256, 0, s>>>(d_dist, (unsigned int)nv, (unsigned int)source);
    int rc = launched();
    int sweep = 0;
    unsigned int updates = 1;
    while (rc == GPUVM_OK && updates > 0) {
        cudaMemsetAsync(behind_q, 0xFF, (size_t)cap * sizeof(unsigned int), s);
        // The first sweep expands the source alone.  (A sweep draws its chunks as fast as it can skip them: with
        // one dirty vertex it would be over before that vertex's neighbours are lowered, and they would all count
        // as "behind".)  The second one runs upwards again, from the pages the first one left; then they alternate.
        const int backward = sweep == 0 ? 0 : (sweep - 1) & 1;
        // A sweep that follows one with few updates has little to expand, scattered over the whole graph: it reads
        // what it needs in place instead of fetching a page per vertex (see sparse_sweep).
        const int sparse = sweep >= 2 && m.sparse_sweep(updates);
        const LcOp<WEIGHTED> op{d_dist, behind_q, counters, cap, (unsigned int)((nv + 31) / 32), backward,
                                sweep == 0 ? (unsigned int)source : kNoVertex, sparse};
        rc = graph_sweep<Mem, LcOp<WEIGHTED>, WEIGHTED>(m, op, off_off, col_off, w_off, nv, scratch, sweep, &updates, s, backward);
        ++sweep;
    }
    cudaMemsetAsync(counters + kCntMax, 0, sizeof(unsigned int), s);
    lc_finish_kernel<<<sm_count() * 4, 256, 0, s>>>(d_dist, (unsigned int)nv, unreached, counters + kCntMax);
    if (rc == GPUVM_OK) rc = launched(); else launched();
    unsigned int far = 0;
    if (cudaMemcpyAsync(&far, counters + kCntMax, sizeof(far), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess) { cudaGetLastError(); return GPUVM_E_CUDA; }
    if (max_dist) *max_dist = far;
    if (n_sweeps) *n_sweeps = sweep;
    return rc;
}

template <class Mem>
int run_bfs(const Mem &m, size_t off_off, size_t col_off, size_t nv, size_t source, int32_t *d_level, int *n_levels,
            void *scratch, cudaStream_t s)
{
    if (!d_level || nv == 0 || source >= nv || nv > 0x3FFFFFFFull) return GPUVM_E_ARG;
    if (off_off % 16 || col_off % 16) return GPUVM_E_ALIGN;
    if (!scratch) return GPUVM_E_ALLOC;
    unsigned int far = 0;
    int rc = lc_sweeps<Mem, false>(m, off_off, col_off, 0, nv, source, d_level, -1, nullptr, &far, scratch, s);
    if (n_levels) *n_levels = (int)far + 1;               // levels 0 .. far were expanded, the last one found nothing
    return rc;
}

// BFS over Balanced CSR: one chunk sweep per level.
template <class Mem>
int run_bfs_bcsr(const Mem &m, size_t off_off, size_t col_off, size_t chunk_off, size_t nv, size_t n_edges,
                 size_t chunk_edges, size_t source, int32_t *d_level, int *n_levels, void *scratch, cudaStream_t s)
{
    if (!d_level || nv == 0 || source >= nv || nv > 0x7FFFFFFFull || chunk_edges == 0 || chunk_edges > 0x7FFFFFFFull)
        return GPUVM_E_ARG;
    if (off_off % 16 || col_off % 16 || chunk_off % 16) return GPUVM_E_ALIGN;
    // a chunk must lie inside one unit (page) of the column array
    if (col_off % m.unit_host() || m.unit_host() % (4 * chunk_edges)) return GPUVM_E_ALIGN;
    if (!scratch) return GPUVM_E_ALLOC;
    unsigned int *counters = static_cast<unsigned int *>(scratch);
    cudaMemsetAsync(d_level, 0xFF, nv * sizeof(int32_t), s);
    bfs_init_kernel<<<1, 1, 0, s>>>(d_level, (int)source);
    int rc = launched();
    int depth = 0;
    unsigned int found = 1;
    while (rc == GPUVM_OK && found > 0 && n_edges > 0) {
        cudaMemsetAsync(counters, 0, 4 * sizeof(unsigned int), s);
        bcsr_sweep_kernel<Mem, BfsOp><<<sm_count() * kBcsrBlocksPerSm, 256, 0, s>>>(m, BfsOp{d_level, depth}, off_off, col_off, chunk_off,
                                                                     (unsigned int)nv, n_edges, (unsigned int)chunk_edges,
                                                                     counters, depth);
        rc = launched();
        const auto t0 = std::chrono::steady_clock::now();
        if (cudaMemcpyAsync(&found, counters, sizeof(found), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
            cudaStreamSynchronize(s) != cudaSuccess) { cudaGetLastError(); rc = GPUVM_E_CUDA; break; }
        static const bool trace = getenv("GPUVM_TRACE_SWEEPS") != nullptr;     // one line per level on stderr
        if (trace)
            fprintf(stderr, "level %d: %.3f ms (host clock, from launch to counters read), found %u\n", depth,
                    std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now() - t0).count(), found);
        ++depth;
    }
    if (n_edges == 0) depth = 1;
    cudaStreamSynchronize(s);
    if (n_levels) *n_levels = depth;
    return rc;
}

// Connected components over Balanced CSR: the one union-find pass, chunk by chunk.
template <class Mem>
int run_cc_bcsr(const Mem &m, size_t off_off, size_t col_off, size_t chunk_off, size_t nv, size_t n_edges,
                size_t chunk_edges, int32_t *d_label, void *scratch, cudaStream_t s)
{
    if (!d_label || nv == 0 || nv > 0x7FFFFFFFull || chunk_edges == 0 || chunk_edges > 0x7FFFFFFFull) return GPUVM_E_ARG;
    if (off_off % 16 || col_off % 16 || chunk_off % 16) return GPUVM_E_ALIGN;
    if (col_off % m.unit_host() || m.unit_host() % (4 * chunk_edges)) return GPUVM_E_ALIGN;
    if (!scratch) return GPUVM_E_ALLOC;
    unsigned int *counters = static_cast<unsigned int *>(scratch);
    cc_init_kernel<<<sm_count() * 4, 256, 0, s>>>(d_label, (unsigned int)nv);
    int rc = launched();
    if (rc == GPUVM_OK && n_edges > 0) {
        cudaMemsetAsync(counters, 0, 4 * sizeof(unsigned int), s);
        bcsr_sweep_kernel<Mem, CcOp><<<sm_count() * kBcsrBlocksPerSm, 256, 0, s>>>(m, CcOp{d_label}, off_off, col_off, chunk_off, (unsigned int)nv,
                                                                    n_edges, (unsigned int)chunk_edges, counters, kBcsrCcSweep);
        rc = launched();
    }
    cc_finish_kernel<<<sm_count() * 4, 256, 0, s>>>(d_label, (unsigned int)nv);
    if (rc == GPUVM_OK) rc = launched(); else launched();
    cudaStreamSynchronize(s);
    return rc;
}

struct Scratch {                     // device scratch for one call, freed on scope exit
    void *p = nullptr;
    explicit Scratch(size_t bytes) { if (cudaMalloc(&p, bytes) != cudaSuccess) { cudaGetLastError(); p = nullptr; } }
    ~Scratch() { if (p) cudaFree(p); }
};

template <class Mem>
int run_cc(const Mem &m, size_t off_off, size_t col_off, size_t nv, int32_t *d_label, int *n_sweeps, void *scratch,
           cudaStream_t s)
{
    if (!d_label || nv == 0 || nv > 0x7FFFFFFFull) return GPUVM_E_ARG;
    if (off_off % 16 || col_off % 16) return GPUVM_E_ALIGN;
    if (!scratch) return GPUVM_E_ALLOC;
    cc_init_kernel<<<sm_count() * 4, 256, 0, s>>>(d_label, (unsigned int)nv);
    int rc = launched();
    unsigned int hooks = 0;
    if (rc == GPUVM_OK) rc = graph_sweep<Mem, CcOp, false>(m, CcOp{d_label}, off_off, col_off, 0, nv, scratch, 0, &hooks, s);
    cc_finish_kernel<<<sm_count() * 4, 256, 0, s>>>(d_label, (unsigned int)nv);
    if (rc == GPUVM_OK) rc = launched(); else launched();
    cudaStreamSynchronize(s);
    if (n_sweeps) *n_sweeps = 1;
    return rc;
}

template <class Mem>
int run_sssp(const Mem &m, size_t off_off, size_t col_off, size_t w_off, size_t nv, size_t source, int32_t *d_dist,
             int *n_rounds, void *scratch, cudaStream_t s)
{
    if (!d_dist || nv == 0 || source >= nv || nv > 0x7FFFFFFFull) return GPUVM_E_ARG;
    if (off_off % 16 || col_off % 16 || w_off % 16) return GPUVM_E_ALIGN;
    if ((w_off > col_off ? w_off - col_off : col_off - w_off) % m.unit_host() != 0) return GPUVM_E_ALIGN;
    if (!scratch) return GPUVM_E_ALLOC;          // lc_scratch_bytes(nv, true)
    return lc_sweeps<Mem, true>(m, off_off, col_off, w_off, nv, source, d_dist, 0x7FFFFFFF, n_rounds, nullptr, scratch, s);
}

template <class Mem>
int run_vadd(const Mem &m, size_t a_off, size_t b_off, size_t c_off, size_t n, bool hold_c, int blocks, int threads,
             cudaStream_t s)
{
    unsigned long long unit = 0;
    if (n % 4) return GPUVM_E_ALIGN;
    if (n == 0) return GPUVM_OK;
    unit = m.unit_host();
    unsigned int chunk = unit < 4096 ? (unsigned int)unit : 4096u;
    if (chunk < 512) return GPUVM_E_PAGE;             // a warp moves 512 bytes per instruction
    if (a_off % chunk || b_off % chunk || c_off % chunk) return GPUVM_E_ALIGN;
    if (hold_c && c_off % unit == 0)
        vadd_kernel<Mem, true><<<blocks, threads, 0, s>>>(m, a_off, b_off, c_off, n, chunk);
    else
        vadd_kernel<Mem, false><<<blocks, threads, 0, s>>>(m, a_off, b_off, c_off, n, chunk);
    return launched();
}

template <class Mem>
int run_embag(const Mem &m, size_t t_off, size_t dims, const int64_t *d_rows, size_t n_bags, size_t bag, float *d_out,
              cudaStream_t s)
{
    if (!d_rows || !d_out || dims == 0 || dims % 4 || dims / 4 > 32 || bag == 0 || bag > 0xFFFFFFFFull) return GPUVM_E_ARG;
    if (t_off % 16) return GPUVM_E_ALIGN;
    if (n_bags == 0) return GPUVM_OK;
    embag_kernel<Mem><<<sm_count() * 4, 256, 0, s>>>(m, t_off, (unsigned int)dims, reinterpret_cast<const long long *>(d_rows),
                                                      n_bags, (unsigned int)bag, d_out);
    return launched();
}


// ---- scratch for gpuvm_bfs_csr_noalloc: lives in the module image of every device that loads
// this library, from load until exit.  Host code must never pass `g_bfs_static_scratch` itself
// to a kernel: in host code that name is only a stand-in for the symbol, not a device
// address.  The real address comes from cudaGetSymbolAddress, once per device.
static __device__ __align__(256) unsigned char g_bfs_static_scratch[kBfsScratchBytes];

constexpr int kMaxDevices = 64;
std::atomic<void *> g_bfs_static_ptr[kMaxDevices];

// Device address of the static scratch on the current device (looked up on first use).
int bfs_static_scratch(void **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return GPUVM_E_NODEVICE; }
    void *p = g_bfs_static_ptr[dev].load();
    if (!p) {
        cudaError_t e = cudaGetSymbolAddress(&p, g_bfs_static_scratch);
        if (e != cudaSuccess || !p) { cudaGetLastError(); return GPUVM_E_CUDA; }
        g_bfs_static_ptr[dev].store(p);
    }
    *out = p;
    return GPUVM_OK;
}

struct PagedH : Paged { unsigned long long unit_host() const { return 1ull << vm.page_shift; } };
struct RawH : Raw { unsigned long long unit_host() const { return unit_bytes; } };

}  // namespace

extern "C" {

void gpuvm_note_launch_(unsigned long long n) { g_launches += n; }
unsigned long long gpuvm_launch_count(void) { return g_launches.load(); }

int gpuvm_stream_sum_i32(gpuvm_t h, size_t a_off, size_t n, int64_t *d_sum, void *stream)
{
    Paged m;
    if (!view_of(h, m)) return GPUVM_E_ARG;
    return run_stream_sum(m, a_off, n, d_sum, static_cast<cudaStream_t>(stream));
}

int gpuvm_gather_f32(gpuvm_t h, size_t x_off, const int64_t *d_idx, size_t n_idx, size_t block, float *d_fsum,
                     int64_t *d_bsum, void *stream)
{
    Paged m;
    if (!view_of(h, m)) return GPUVM_E_ARG;
    if (!d_idx || !d_fsum || !d_bsum || block == 0 || block > (size_t(1) << 20)) return GPUVM_E_ARG;
    if (x_off % 16) return GPUVM_E_ALIGN;
    if (n_idx == 0) return GPUVM_OK;
    const int requesters = kGatherRequesters, migrators = kGatherMigrators;
    // Requests per requester warp: all of a warp's share of the index list when that is at most
    // kGatherBatch (then every page is fetched once per run), whole index blocks, at least 2048.
    const size_t warps_all = (size_t)sm_count() * requesters;
    size_t share = (n_idx + warps_all - 1) / warps_all;
    if (block <= kGatherBatch) share = (share + block - 1) / block * block;
    // Without a scratch bound and with index blocks of at least kGatherDirectMinBlock the requests are
    // read from the index list in place and summed as they arrive: no table, no scratch.
    const bool direct = block >= kGatherDirectMinBlock && gpuvm_scratch_limit_(h) == ~size_t(0);
    if (!direct && (m.vm.bytes - x_off) / 4 >= kNoIndex) return GPUVM_E_RANGE;      // element indices are staged as 32-bit numbers
    unsigned int batch = 2048;
    while (batch < kGatherBatch && batch < share &&
           (direct || warps_all * (size_t)batch * 2 * sizeof(unsigned int) <= gpuvm_scratch_limit_(h)))
        batch *= 2;
    const size_t nb = (n_idx + block - 1) / block;
    const size_t per = block <= batch ? batch / block : 1;
    const size_t items = (nb + per - 1) / per;
    const size_t blocks_needed = (items + requesters - 1) / requesters;
    const unsigned int grid = (unsigned int)(blocks_needed < (size_t)sm_count() ? blocks_needed : (size_t)sm_count());
    const size_t slots = items < (size_t)grid * requesters ? items : (size_t)grid * requesters;   // warps that get work
    const size_t tables_bytes = direct ? 0 : (slots * batch * sizeof(unsigned int) + 255) & ~size_t(255);
    const bool want_ring = (size_t(1) << m.vm.page_shift) >= kSharedQueueMinPage;
    unsigned int *tables = nullptr;
    gpuvm_shared_queue *shared_queue = nullptr;
    if (tables_bytes || want_ring) {                          // the table-free form with small pages needs no scratch at all
        tables = static_cast<unsigned int *>(gpuvm_scratch_(h, tables_bytes + (want_ring ? sizeof(gpuvm_shared_queue) : 0)));
        if (!tables) return GPUVM_E_ALLOC;
        if (want_ring)
            shared_queue = shared_queue_at(m.vm, reinterpret_cast<unsigned char *>(tables) + tables_bytes,
                                           static_cast<cudaStream_t>(stream));
    }
    // staging of the migrator warps: kGatherStages pieces of at most kGatherChunk bytes each
    const unsigned int stage_chunk = (unsigned int)((size_t(1) << m.vm.page_shift) < kGatherChunk ? (size_t(1) << m.vm.page_shift) : kGatherChunk);
    const unsigned int stage_count = stage_chunk >= 128 ? kGatherStages : 0;     // tiny pages: copy through registers
    const size_t mask_bytes = (size_t)requesters * gpuvm_batch_mask_words(batch) * 32 * sizeof(unsigned long long) +
                              (size_t)migrators * stage_count * (stage_chunk + sizeof(unsigned long long)) +
                              (direct ? (size_t)requesters * 2 * kGatherAcc * sizeof(double) : 0);
    auto kernel = direct ? gather_batch_kernel<true> : gather_batch_kernel<false>;
    if (mask_bytes > 40 * 1024 &&
        cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)mask_bytes) != cudaSuccess) {
        cudaGetLastError();
        return GPUVM_E_CUDA;
    }
    kernel<<<grid, (requesters + migrators) * 32, mask_bytes, static_cast<cudaStream_t>(stream)>>>(
        m.vm, x_off, reinterpret_cast<const long long *>(d_idx), n_idx, block, d_fsum, reinterpret_cast<long long *>(d_bsum),
        requesters, batch, tables, stage_chunk, stage_count, /* one_pass = */ items <= (size_t)grid * requesters, shared_queue);
    return launched();
}

int gpuvm_gather_f32_unbatched(gpuvm_t h, size_t x_off, const int64_t *d_idx, size_t n_idx, size_t block, float *d_fsum,
                               int64_t *d_bsum, void *stream)
{
    Paged m;
    if (!view_of(h, m)) return GPUVM_E_ARG;
    return run_gather(m, x_off, d_idx, n_idx, block, d_fsum, d_bsum, static_cast<cudaStream_t>(stream));
}

int gpuvm_bfs_csr(gpuvm_t h, size_t off_off, size_t col_off, size_t nv, size_t source, int32_t *d_level, int *n_levels,
                  void *stream)
{
    Paged m;
    if (!view_of(h, m)) return GPUVM_E_ARG;
    hint_edges(h, m, off_off, nv);
    return run_bfs(m, off_off, col_off, nv, source, d_level, n_levels, gpuvm_scratch_(h, lc_scratch_bytes(nv, false)),
                   static_cast<cudaStream_t>(stream));
}

int gpuvm_bfs_csr_noalloc(gpuvm_t h, size_t off_off, size_t col_off, size_t nv, size_t source, int32_t *d_level,
                          int *n_levels, void *stream)
{
    Paged m;
    if (!view_of(h, m)) return GPUVM_E_ARG;
    if (!d_level || nv == 0 || source >= nv) return GPUVM_E_ARG;
    if (nv > GPUVM_BFS_NOALLOC_MAX_VERTICES) return GPUVM_E_RANGE;     // beyond what the fixed scratch is sized for
    if (off_off % 16 || col_off % 16) return GPUVM_E_ALIGN;
    void *scratch = nullptr;
    int rc = bfs_static_scratch(&scratch);
    if (rc != GPUVM_OK) return rc;
    hint_edges(h, m, off_off, nv);
    // bfs_levels zeroes the counters at the start of every level and writes each queue entry
    // before reading it, so whatever the previous call left in the array does not matter
    return bfs_levels(m, off_off, col_off, nv, source, d_level, n_levels, scratch, static_cast<cudaStream_t>(stream));
}

int gpuvm_bfs_bcsr(gpuvm_t h, size_t off_off, size_t col_off, size_t chunk_off, size_t nv, size_t n_edges,
                   size_t chunk_edges, size_t source, int32_t *d_level, int *n_levels, void *stream)
{
    PagedH m;
    if (!view_of(h, m)) return GPUVM_E_ARG;
    return run_bfs_bcsr(m, off_off, col_off, chunk_off, nv, n_edges, chunk_edges, source, d_level, n_levels,
                        gpuvm_scratch_(h, kBfsScratchBytes), static_cast<cudaStream_t>(stream));
}

int gpuvm_cc_bcsr(gpuvm_t h, size_t off_off, size_t col_off, size_t chunk_off, size_t nv, size_t n_edges, size_t chunk_edges,
                  int32_t *d_label, void *stream)
{
    PagedH m;
    if (!view_of(h, m)) return GPUVM_E_ARG;
    return run_cc_bcsr(m, off_off, col_off, chunk_off, nv, n_edges, chunk_edges, d_label, gpuvm_scratch_(h, kBfsScratchBytes),
                       static_cast<cudaStream_t>(stream));
}

int gpuvm_bcsr_build(const int64_t *row_off, size_t nv, size_t chunk_edges, int32_t *chunk_vertex, size_t capacity,
                     size_t *n_chunks_out)
{
    if (!row_off || nv == 0 || nv > 0x7FFFFFFFull || chunk_edges == 0) return GPUVM_E_ARG;
    const int64_t ne = row_off[nv];
    if (ne < 0 || row_off[0] != 0) return GPUVM_E_ARG;
    const size_t n_chunks = ((size_t)ne + chunk_edges - 1) / chunk_edges;
    if (n_chunks_out) *n_chunks_out = n_chunks;
    if (!chunk_vertex) return GPUVM_OK;                       // size query
    if (capacity < n_chunks + 1) return GPUVM_E_RANGE;
    // one pass over the row offsets: v follows the chunk boundaries, which only move forward
    size_t v = 0;
    for (size_t c = 0; c < n_chunks; ++c) {
        const int64_t first = (int64_t)(c * chunk_edges);
        while (row_off[v + 1] <= first) ++v;                  // skips vertices without edges: first < ne = row_off[nv]
        chunk_vertex[c] = (int32_t)v;
    }
    if (ne > 0) { while (row_off[v + 1] <= ne - 1) ++v; }
    chunk_vertex[n_chunks] = (int32_t)(ne > 0 ? v : 0);
    return GPUVM_OK;
}

int gpuvm_cc_csr(gpuvm_t h, size_t off_off, size_t col_off, size_t nv, int32_t *d_label, int *n_sweeps, void *stream)
{
    Paged m;
    if (!view_of(h, m)) return GPUVM_E_ARG;
    hint_edges(h, m, off_off, nv);
    return run_cc(m, off_off, col_off, nv, d_label, n_sweeps, gpuvm_scratch_(h, kBfsScratchBytes),
                  static_cast<cudaStream_t>(stream));
}

int gpuvm_sssp_csr(gpuvm_t h, size_t off_off, size_t col_off, size_t w_off, size_t nv, size_t source, int32_t *d_dist,
                   int *n_rounds, void *stream)
{
    PagedH m;
    if (!view_of(h, m)) return GPUVM_E_ARG;
    // column and weight page of an edge range are held together: two frames per warp of the grid
    if (gpuvm_safe_warps(h, 2) < sm_count() * 2 * 8) return GPUVM_E_FRAMES;
    hint_edges(h, m, off_off, nv);
    return run_sssp(m, off_off, col_off, w_off, nv, source, d_dist, n_rounds, gpuvm_scratch_(h, lc_scratch_bytes(nv, true)),
                    static_cast<cudaStream_t>(stream));
}

int gpuvm_vadd_f32(gpuvm_t h, size_t a_off, size_t b_off, size_t c_off, size_t n, void *stream)
{
    PagedH m;
    if (!view_of(h, m)) return GPUVM_E_ARG;
    // c may be a or b itself (in place): every chunk is then read before it is written, by the same
    // warp, one page at a time; the no-fetch path is out, because it hands out the page of c without
    // its contents.  Any other overlap of c with an input has no defined result.
    const size_t len = 4 * n;
    auto overlaps = [len](size_t x, size_t y) { return x < y + len && y < x + len; };
    const bool in_place = c_off == a_off || c_off == b_off;
    if ((c_off != a_off && overlaps(c_off, a_off)) || (c_off != b_off && overlaps(c_off, b_off))) return GPUVM_E_ARG;
    // The grid is sized to the pool: a warp works on three pages at a time (it holds the page of c, or comes
    // back to it, and comes back to its pages of a and b chunk by chunk).  More warps than that would evict
    // one another's pages between chunks and fetch every page many times (measured: 13 times); the link
    // is full from a few dozen migrating warps anyway, so a small pool costs warps, not bandwidth.
    const int safe = gpuvm_safe_warps(h, 4);                // three pages in rotation and one to spare for the ring's slack
    int blocks = sm_count() * kVaddBlocksPerSm, threads = 256;
    if (safe >= 8) blocks = blocks < safe / 8 ? blocks : safe / 8;
    else { blocks = 1; threads = 32 * (safe > 0 ? safe : 1); }
    const bool hold_c = !in_place && gpuvm_safe_warps(h, 2) >= 1;
    return run_vadd(m, a_off, b_off, c_off, n, hold_c, blocks, threads, static_cast<cudaStream_t>(stream));
}

int gpuvm_embag_f32(gpuvm_t h, size_t t_off, size_t dims, const int64_t *d_rows, size_t n_bags, size_t bag, float *d_out,
                    void *stream)
{
    Paged m;
    if (!view_of(h, m)) return GPUVM_E_ARG;
    if (!d_rows || !d_out || dims == 0 || dims % 4 || dims / 4 > 32 || bag == 0 || bag > 0xFFFFFFFFull) return GPUVM_E_ARG;
    if (t_off % 16) return GPUVM_E_ALIGN;
    if (n_bags == 0) return GPUVM_OK;
    // The batched kernel registers a row by its first byte and then reads the whole row from that
    // frame: a row must lie inside one page.  Tables whose rows straddle pages (a row size that does
    // not divide the page size, a table that does not start on a row boundary inside its page, pages
    // smaller than a row) take the one-request-at-a-time kernel, which asks for every 16 bytes it reads.
    const size_t row_bytes = 4 * dims, page_bytes = size_t(1) << m.vm.page_shift;
    if (page_bytes % row_bytes != 0 || t_off % row_bytes != 0)
        return run_embag(m, t_off, dims, d_rows, n_bags, bag, d_out, static_cast<cudaStream_t>(stream));
    const int requesters = kEmbagRequesters, migrators = kEmbagMigrators;
    {
        // The direct form (embag_direct_kernel): lookups counted per page, rows of the pages below the limit read in
        // place page by page into a staging area of their own, every other row read straight from its page's
        // frame.  It needs the pages at or above the limit to fit the pool twice over (they are held in their
        // frames for the length of the launch) and their number to fit the fault rings; how many there are is
        // read back after the count, which makes this call synchronous at that point.
        cudaStream_t s = static_cast<cudaStream_t>(stream);
        const size_t n_lookups = n_bags * bag;
        size_t divisor = gpuvm_inplace_divisor_(h);
        if (divisor == GPUVM_INPLACE_AUTO) divisor = 1;
        const size_t charged = row_bytes < 128 ? 128 : row_bytes;
        const unsigned int limit = divisor ? (unsigned int)(page_bytes / divisor / charged) : 0u;
        if (gpuvm_inplace_counted_(h) == 2 && limit != 0u && n_lookups < 0xFFFFFFFFull && m.vm.n_pages <= (1ull << 20)) {
            const long long *rows_ll = reinterpret_cast<const long long *>(d_rows);
            const unsigned long long rows_inside = (m.vm.bytes - t_off) / row_bytes;
            const size_t pages_bytes = (m.vm.n_pages * sizeof(unsigned int) + 255) & ~size_t(255);
            const size_t head_bytes = 2 * pages_bytes + 256 + sizeof(gpuvm_shared_queue);      // demand, bucket starts, counts, ring
            const size_t where_bytes = (n_lookups * sizeof(unsigned int) + 255) & ~size_t(255);
            unsigned int host_counts[2] = {0, 0};
            unsigned char *scratch = nullptr;
            unsigned int *demand = nullptr, *bucket_off = nullptr, *counts = nullptr;
            size_t total = head_bytes;
            bool fits = true;
            for (int attempt = 0; attempt < 2; ++attempt) {
                scratch = static_cast<unsigned char *>(gpuvm_scratch_(h, total));
                if (!scratch) return GPUVM_E_ALLOC;
                demand = reinterpret_cast<unsigned int *>(scratch);
                bucket_off = reinterpret_cast<unsigned int *>(scratch + pages_bytes);
                counts = reinterpret_cast<unsigned int *>(scratch + 2 * pages_bytes);
                if (cudaMemsetAsync(demand, 0, pages_bytes, s) != cudaSuccess) { cudaGetLastError(); return GPUVM_E_CUDA; }
                embag_demand_kernel<<<sm_count() * 8, 256, 0, s>>>(rows_ll, n_lookups, t_off, row_bytes, m.vm.page_shift, rows_inside,
                                                                    demand, limit);
                embag_bucket_scan_kernel<<<1, 1024, 0, s>>>(demand, (unsigned int)m.vm.n_pages, limit, bucket_off, counts);
                gpuvm_note_launch_(2);
                if (cudaMemcpyAsync(host_counts, counts, sizeof(host_counts), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
                    cudaStreamSynchronize(s) != cudaSuccess) { cudaGetLastError(); return GPUVM_E_CUDA; }
                const size_t cold_bytes = ((size_t)host_counts[0] * sizeof(unsigned int) + 255) & ~size_t(255);
                const size_t rows_bytes_total = ((size_t)host_counts[0] * row_bytes + 255) & ~size_t(255);
                total = head_bytes + cold_bytes + where_bytes + rows_bytes_total;
                fits = 2ull * host_counts[1] <= m.vm.n_frames && host_counts[1] <= 32768u &&
                       (gpuvm_scratch_limit_(h) == ~size_t(0) || total <= gpuvm_scratch_limit_(h));
                if (!fits || total <= gpuvm_scratch_bytes(h)) break;     // else: the scratch grows and the count is taken again in it
            }
            if (fits) {
                const size_t cold_bytes = ((size_t)host_counts[0] * sizeof(unsigned int) + 255) & ~size_t(255);
                unsigned int *cold_idx = reinterpret_cast<unsigned int *>(scratch + head_bytes);
                unsigned int *where = reinterpret_cast<unsigned int *>(scratch + head_bytes + cold_bytes);
                uint4 *cold_staging = reinterpret_cast<uint4 *>(scratch + head_bytes + cold_bytes + where_bytes);
                gpuvm_shared_queue *shared_queue = shared_queue_at(m.vm, scratch + 2 * pages_bytes + 256, s);
                if (cudaMemsetAsync(where, 0xFF, where_bytes, s) != cudaSuccess) { cudaGetLastError(); return GPUVM_E_CUDA; }
                embag_bucket_fill_kernel<<<sm_count() * 8, 256, 0, s>>>(rows_ll, n_lookups, t_off, row_bytes, m.vm.page_shift,
                                                                     rows_inside, demand, limit, bucket_off, cold_idx, where);
                const size_t stage_bytes = (size_t)kEmbagMigrators * kEmbagStages * kEmbagChunk;
                if (stage_bytes > 40 * 1024 &&
                    cudaFuncSetAttribute(embag_direct_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)stage_bytes) != cudaSuccess) {
                    cudaGetLastError();
                    return GPUVM_E_CUDA;
                }
                const size_t warps_needed = n_bags > (size_t)host_counts[0] / 4 ? n_bags : (size_t)host_counts[0] / 4 + 1;
                const size_t blocks_needed = (warps_needed + requesters - 1) / requesters;
                const unsigned int grid = (unsigned int)(blocks_needed < (size_t)sm_count() ? blocks_needed : (size_t)sm_count());
                embag_direct_kernel<<<grid, (requesters + migrators) * 32, stage_bytes, s>>>(
                    m.vm, t_off, (unsigned int)dims, rows_ll, n_bags, (unsigned int)bag, d_out, requesters, shared_queue, limit,
                    demand, cold_idx, where, cold_staging, counts);
                return launched(2);
            }
        }
    }
    // Groups of 32 bags per requester warp: enough for every bag to be in flight at once when
    // that takes at most kEmbagMaxGroups, within the scratch bound (table + staged rows).
    const size_t warps_all = (size_t)sm_count() * requesters;
    const size_t lookups_now = bag < kEmbagLookups ? bag : kEmbagLookups;
    unsigned int groups = 1;
    while (groups < kEmbagMaxGroups && (n_bags + 32 * groups - 1) / (32 * groups) > warps_all &&
           warps_all * (2 * groups) * 32 * lookups_now * (sizeof(gpuvm_batch_entry) + 4 * dims) <= gpuvm_scratch_limit_(h))
        groups *= 2;
    const size_t items = (n_bags + 32 * groups - 1) / (32 * groups);
    const size_t blocks_needed = (items + requesters - 1) / requesters;
    const unsigned int grid = (unsigned int)(blocks_needed < (size_t)sm_count() ? blocks_needed : (size_t)sm_count());
    const size_t per_warp = (size_t)groups * 32 * lookups_now;
    const size_t slots = items < (size_t)grid * requesters ? items : (size_t)grid * requesters;   // warps that get work
    const size_t table_bytes = (slots * per_warp * sizeof(gpuvm_batch_entry) + 255) & ~size_t(255);
    const size_t staging_bytes = (slots * per_warp * 4 * dims + 255) & ~size_t(255);
    const bool one_pass = items <= (size_t)grid * requesters && bag <= kEmbagLookups;
    // Which pages are fetched.  A page is fetched when its lookups would move at least page_bytes / divisor in place
    // (gpuvm_set_inplace_divisor); the rows of the others are read in place from the backing store.  The lookup
    // list is at hand, so the lookups per page are counted before the first access (gpuvm_set_inplace_counted);
    // when, in addition, every lookup's staging slot is known beforehand (one pass) the rows read in place are
    // bucketed by page and read page by page ("grouped"), which the host link serves at its full rate, and
    // the break-even point is the page's size (divisor 1); read one lookup after the other they are scattered
    // over the table and served at half that rate or less, and a quarter of the page is where the two streams
    // balance (divisor 4).  A row is a whole number of 128-byte link reads when it is a multiple of 128 bytes
    // long; shorter rows are charged 128 bytes.
    const size_t n_lookups = n_bags * bag;
    const bool counted = gpuvm_inplace_counted_(h) != 0, want_grouped = gpuvm_inplace_counted_(h) == 2;
    const size_t demand_bytes = (m.vm.n_pages * sizeof(unsigned int) + 255) & ~size_t(255);
    const size_t index_bytes = (n_lookups * sizeof(unsigned int) + 255) & ~size_t(255);
    const size_t base_bytes = table_bytes + staging_bytes + sizeof(gpuvm_shared_queue) + demand_bytes;
    const bool grouped = want_grouped && one_pass && n_lookups < 0xFFFFFFFFull && m.vm.n_pages <= (1ull << 20) &&
                         (gpuvm_scratch_limit_(h) == ~size_t(0) || base_bytes + demand_bytes + index_bytes + 256 <= gpuvm_scratch_limit_(h));
    size_t divisor = gpuvm_inplace_divisor_(h);
    if (divisor == GPUVM_INPLACE_AUTO) divisor = grouped ? 1 : 4;
    const size_t charged = row_bytes < 128 ? 128 : row_bytes;
    const unsigned int inplace_limit = divisor ? (unsigned int)(page_bytes / divisor / charged) : 0u;
    const bool use_grouped = grouped && inplace_limit != 0u;
    unsigned char *scratch = static_cast<unsigned char *>(
        gpuvm_scratch_(h, base_bytes + (use_grouped ? demand_bytes + index_bytes + 256 : 0)));
    if (!scratch) return GPUVM_E_ALLOC;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    gpuvm_shared_queue *shared_queue = shared_queue_at(m.vm, scratch + table_bytes + staging_bytes, s);
    unsigned int *demand = nullptr, *bucket_off = nullptr, *cold_idx = nullptr, *cold_counts = nullptr;
    unsigned long long launches = 1;
    const long long *rows_ll = reinterpret_cast<const long long *>(d_rows);
    const unsigned long long rows_inside = (m.vm.bytes - t_off) / row_bytes;
    if (inplace_limit != 0u && counted) {
        demand = reinterpret_cast<unsigned int *>(scratch + table_bytes + staging_bytes + sizeof(gpuvm_shared_queue));
        if (cudaMemsetAsync(demand, 0, demand_bytes, s) != cudaSuccess) { cudaGetLastError(); return GPUVM_E_CUDA; }
        embag_demand_kernel<<<sm_count() * 8, 256, 0, s>>>(rows_ll, n_lookups, t_off, row_bytes, m.vm.page_shift, rows_inside,
                                                            demand, inplace_limit);
        ++launches;
        if (use_grouped) {
            bucket_off = reinterpret_cast<unsigned int *>(scratch + base_bytes);
            cold_idx = reinterpret_cast<unsigned int *>(scratch + base_bytes + demand_bytes);
            cold_counts = reinterpret_cast<unsigned int *>(scratch + base_bytes + demand_bytes + index_bytes);
            embag_bucket_scan_kernel<<<1, 1024, 0, s>>>(demand, (unsigned int)m.vm.n_pages, inplace_limit, bucket_off, cold_counts);
            embag_bucket_fill_kernel<<<sm_count() * 8, 256, 0, s>>>(rows_ll, n_lookups, t_off, row_bytes, m.vm.page_shift,
                                                                 rows_inside, demand, inplace_limit, bucket_off, cold_idx);
            launches += 2;
        }
    }
    const size_t stage_bytes = (size_t)kEmbagMigrators * kEmbagStages * kEmbagChunk;
    if (stage_bytes > 40 * 1024 &&
        cudaFuncSetAttribute(embag_batch_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)stage_bytes) != cudaSuccess) {
        cudaGetLastError();
        return GPUVM_E_CUDA;
    }
    embag_batch_kernel<<<grid, (requesters + migrators) * 32, stage_bytes, s>>>(
        m.vm, t_off, (unsigned int)dims, rows_ll, n_bags, (unsigned int)bag, d_out,
        requesters, reinterpret_cast<gpuvm_batch_entry *>(scratch), scratch + table_bytes, groups, one_pass, shared_queue,
        inplace_limit, demand, cold_idx, cold_counts);
    return launched(launches);
}

int gpuvm_embag_f32_unbatched(gpuvm_t h, size_t t_off, size_t dims, const int64_t *d_rows, size_t n_bags, size_t bag,
                              float *d_out, void *stream)
{
    Paged m;
    if (!view_of(h, m)) return GPUVM_E_ARG;
    return run_embag(m, t_off, dims, d_rows, n_bags, bag, d_out, static_cast<cudaStream_t>(stream));
}

int gpuvm_scatter_update_u32(gpuvm_t h, size_t a_off, const int64_t *d_idx, size_t n, void *stream)
{
    Paged m;
    if (!view_of(h, m) || !d_idx) return GPUVM_E_ARG;
    if (a_off % 16) return GPUVM_E_ALIGN;
    if (n == 0) return GPUVM_OK;
    scatter_update_kernel<Paged><<<sm_count() * 4, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        m, a_off, reinterpret_cast<const long long *>(d_idx), n);
    return launched();
}

int gpuvm_scatter_update_u32_batched(gpuvm_t h, size_t a_off, const int64_t *d_idx, size_t n, void *stream)
{
    Paged m;
    if (!view_of(h, m) || !d_idx) return GPUVM_E_ARG;
    if (a_off % 16) return GPUVM_E_ALIGN;
    if (n == 0) return GPUVM_OK;
    scatter_update_batch_kernel<<<sm_count() * 4, 128, 0, static_cast<cudaStream_t>(stream)>>>(
        m.vm, a_off, reinterpret_cast<const long long *>(d_idx), n);
    return launched();
}

int gpuvm_scatter_update_u32_queued(gpuvm_t h, size_t a_off, const int64_t *d_idx, size_t n, void *stream)
{
    Paged m;
    if (!view_of(h, m) || !d_idx) return GPUVM_E_ARG;
    if (a_off % 16) return GPUVM_E_ALIGN;
    if (n == 0) return GPUVM_OK;
    unsigned char *scratch = static_cast<unsigned char *>(gpuvm_scratch_(h, sizeof(gpuvm_shared_queue)));
    if (!scratch) return GPUVM_E_ALLOC;
    gpuvm_shared_queue *shared_queue = shared_queue_at(m.vm, scratch, static_cast<cudaStream_t>(stream));
    scatter_update_queued_kernel<<<sm_count() * 2, (kScatterRequesters + kScatterMigrators) * 32, 0, static_cast<cudaStream_t>(stream)>>>(
        m.vm, a_off, reinterpret_cast<const long long *>(d_idx), n, shared_queue);
    return launched();
}

int gpuvm_touch_pages(gpuvm_t h, size_t first_page, size_t n_pages, int warps_per_sm, void *stream)
{
    Paged m;
    if (!view_of(h, m) || warps_per_sm <= 0 || warps_per_sm > 64) return GPUVM_E_ARG;
    if (first_page + n_pages > m.vm.n_pages) return GPUVM_E_RANGE;
    if (n_pages == 0) return GPUVM_OK;
    int threads = warps_per_sm * 32 > 256 ? 256 : warps_per_sm * 32;      // 128 registers per thread: 256-thread blocks
    int blocks_per_sm = (warps_per_sm * 32 + threads - 1) / threads;
    touch_pages_kernel<<<sm_count() * blocks_per_sm, threads, 0, static_cast<cudaStream_t>(stream)>>>(m.vm, first_page, n_pages);
    return launched();
}

int gpuvm_touch_pages_warps(gpuvm_t h, size_t first_page, size_t n_pages, int total_warps, void *stream)
{
    Paged m;
    if (!view_of(h, m) || total_warps <= 0 || total_warps > 65536) return GPUVM_E_ARG;
    if (first_page + n_pages > m.vm.n_pages) return GPUVM_E_RANGE;
    if (n_pages == 0) return GPUVM_OK;
    // spread the warps over the SMs: one-warp blocks up to the SM count, wider blocks beyond
    const int per_block = (total_warps + sm_count() - 1) / sm_count() > 8 ? 8 : (total_warps + sm_count() - 1) / sm_count();
    const int blocks = (total_warps + per_block - 1) / per_block;
    touch_pages_kernel<<<blocks, per_block * 32, 0, static_cast<cudaStream_t>(stream)>>>(m.vm, first_page, n_pages);
    return launched();
}

int gpuvm_raw_stream_sum_i32(const int32_t *a, size_t n, int64_t *d_sum, void *stream)
{
    if (!a) return GPUVM_E_ARG;
    Raw m{reinterpret_cast<unsigned char *>(const_cast<int32_t *>(a)), 65536};
    return run_stream_sum(m, 0, n, d_sum, static_cast<cudaStream_t>(stream));
}

int gpuvm_raw_gather_f32(const float *x, const int64_t *d_idx, size_t n_idx, size_t block, float *d_fsum, int64_t *d_bsum,
                         void *stream)
{
    if (!x) return GPUVM_E_ARG;
    Raw m{reinterpret_cast<unsigned char *>(const_cast<float *>(x)), 65536};
    return run_gather(m, 0, d_idx, n_idx, block, d_fsum, d_bsum, static_cast<cudaStream_t>(stream));
}

int gpuvm_raw_bfs_csr(const int64_t *row_off, const int32_t *col, size_t nv, size_t source, int32_t *d_level,
                      int *n_levels, void *stream)
{
    if (!row_off || !col) return GPUVM_E_ARG;
    // one policy object addresses both arrays relative to the lower of the two
    unsigned char *ro = reinterpret_cast<unsigned char *>(const_cast<int64_t *>(row_off));
    unsigned char *co = reinterpret_cast<unsigned char *>(const_cast<int32_t *>(col));
    unsigned char *base = ro < co ? ro : co;
    if ((ro - base) % 16 || (co - base) % 16) return GPUVM_E_ALIGN;
    Raw m{base, 65536};
    Scratch scratch(lc_scratch_bytes(nv, false));
    return run_bfs(m, (size_t)(ro - base), (size_t)(co - base), nv, source, d_level, n_levels, scratch.p,
                   static_cast<cudaStream_t>(stream));
}

int gpuvm_raw_cc_csr(const int64_t *row_off, const int32_t *col, size_t nv, int32_t *d_label, int *n_sweeps, void *stream)
{
    if (!row_off || !col) return GPUVM_E_ARG;
    unsigned char *ro = reinterpret_cast<unsigned char *>(const_cast<int64_t *>(row_off));
    unsigned char *co = reinterpret_cast<unsigned char *>(const_cast<int32_t *>(col));
    unsigned char *base = ro < co ? ro : co;
    if ((ro - base) % 16 || (co - base) % 16) return GPUVM_E_ALIGN;
    Raw m{base, 65536};
    Scratch scratch(kBfsScratchBytes);
    return run_cc(m, (size_t)(ro - base), (size_t)(co - base), nv, d_label, n_sweeps, scratch.p,
                  static_cast<cudaStream_t>(stream));
}

int gpuvm_raw_sssp_csr(const int64_t *row_off, const int32_t *col, const int32_t *weight, size_t nv, size_t source,
                       int32_t *d_dist, int *n_rounds, void *stream)
{
    if (!row_off || !col || !weight) return GPUVM_E_ARG;
    unsigned char *ro = reinterpret_cast<unsigned char *>(const_cast<int64_t *>(row_off));
    unsigned char *co = reinterpret_cast<unsigned char *>(const_cast<int32_t *>(col));
    unsigned char *we = reinterpret_cast<unsigned char *>(const_cast<int32_t *>(weight));
    unsigned char *base = ro < co ? (ro < we ? ro : we) : (co < we ? co : we);
    RawH m;
    m.base = base;
    m.unit_bytes = 65536;
    Scratch scratch(lc_scratch_bytes(nv, true));
    return run_sssp(m, (size_t)(ro - base), (size_t)(co - base), (size_t)(we - base), nv, source, d_dist, n_rounds,
                    scratch.p, static_cast<cudaStream_t>(stream));
}

int gpuvm_raw_vadd_f32(const float *a, const float *b, float *c, size_t n, void *stream)
{
    if (!a || !b || !c) return GPUVM_E_ARG;
    unsigned char *pa = reinterpret_cast<unsigned char *>(const_cast<float *>(a));
    unsigned char *pb = reinterpret_cast<unsigned char *>(const_cast<float *>(b));
    unsigned char *pc = reinterpret_cast<unsigned char *>(c);
    unsigned char *base = pa < pb ? (pa < pc ? pa : pc) : (pb < pc ? pb : pc);
    RawH m;
    m.base = base;
    m.unit_bytes = 65536;
    return run_vadd(m, (size_t)(pa - base), (size_t)(pb - base), (size_t)(pc - base), n, false, sm_count() * kVaddBlocksPerSm, 256, static_cast<cudaStream_t>(stream));
}

int gpuvm_raw_embag_f32(const float *table, size_t dims, const int64_t *d_rows, size_t n_bags, size_t bag, float *d_out,
                        void *stream)
{
    if (!table) return GPUVM_E_ARG;
    Raw m{reinterpret_cast<unsigned char *>(const_cast<float *>(table)), 65536};
    return run_embag(m, 0, dims, d_rows, n_bags, bag, d_out, static_cast<cudaStream_t>(stream));
}

int gpuvm_link_peak(void *host_ptr, void *d_buf, size_t bytes, int reps, double *out)
{
    if (!host_ptr || !d_buf || !out || bytes < 4096 || bytes % 32 || reps <= 0) return GPUVM_E_ARG;
    void *dh = nullptr;
    if (cudaHostGetDevicePointer(&dh, host_ptr, 0) != cudaSuccess) { cudaGetLastError(); return GPUVM_E_PIN; }
    cudaEvent_t a, b;
    cudaEventCreate(&a);
    cudaEventCreate(&b);
    const size_t n16 = bytes / 16;
    const int grid = sm_count() * 2;
    double best[3] = {0, 0, 0};
    for (int mode = 0; mode < 3; ++mode)
        for (int r = 0; r <= reps; ++r) {
            cudaEventRecord(a);
            if (mode == 0) link_in_kernel<<<grid, 512>>>(static_cast<const uint4 *>(dh), static_cast<uint4 *>(d_buf), n16);
            else if (mode == 1) link_out_kernel<<<grid, 512>>>(static_cast<const uint4 *>(d_buf), static_cast<uint4 *>(dh), n16);
            else link_duplex_kernel<<<grid * 2, 512>>>(static_cast<uint4 *>(dh), static_cast<uint4 *>(d_buf), n16);
            gpuvm_note_launch_(1);
            cudaEventRecord(b);
            if (cudaEventSynchronize(b) != cudaSuccess) { cudaGetLastError(); cudaEventDestroy(a); cudaEventDestroy(b); return GPUVM_E_CUDA; }
            float ms = 0;
            cudaEventElapsedTime(&ms, a, b);
            double gbs = (double)bytes / (ms * 1e6);
            if (r > 0 && gbs > best[mode]) best[mode] = gbs;     // r == 0 is the warm-up
        }
    cudaEventDestroy(a);
    cudaEventDestroy(b);
    out[0] = best[0]; out[1] = best[1]; out[2] = best[2];
    return GPUVM_OK;
}

int gpuvm_link_peak_scattered(void *host_ptr, size_t host_bytes, size_t row_bytes, size_t n_rows, size_t run, void *d_buf,
                              size_t d_bytes, int reps, double *out)
{
    if (!host_ptr || !d_buf || !out || row_bytes < 16 || row_bytes % 16 || row_bytes > 512 || host_bytes < row_bytes ||
        d_bytes < row_bytes || n_rows == 0 || reps <= 0 || run == 0 || run > 0xFFFFFFFFull)
        return GPUVM_E_ARG;
    void *dh = nullptr;
    if (cudaHostGetDevicePointer(&dh, host_ptr, 0) != cudaSuccess) { cudaGetLastError(); return GPUVM_E_PIN; }
    cudaEvent_t a, b;
    cudaEventCreate(&a);
    cudaEventCreate(&b);
    double best = 0;
    for (int r = 0; r <= reps; ++r) {
        cudaEventRecord(a);
        link_scattered_kernel<<<sm_count(), 1024>>>(static_cast<const unsigned char *>(dh), host_bytes / row_bytes,
                                                    (unsigned int)(row_bytes / 16), n_rows, 0x5CA77E2ull + r, (unsigned int)run,
                                                    static_cast<uint4 *>(d_buf), d_bytes / row_bytes);
        gpuvm_note_launch_(1);
        cudaEventRecord(b);
        if (cudaEventSynchronize(b) != cudaSuccess) { cudaGetLastError(); cudaEventDestroy(a); cudaEventDestroy(b); return GPUVM_E_CUDA; }
        float ms = 0;
        cudaEventElapsedTime(&ms, a, b);
        const double gbs = (double)n_rows * row_bytes / (ms * 1e6);
        if (r > 0 && gbs > best) best = gbs;                      // r == 0 is the warm-up
    }
    cudaEventDestroy(a);
    cudaEventDestroy(b);
    out[0] = best;
    return GPUVM_OK;
}

}  // extern "C"

