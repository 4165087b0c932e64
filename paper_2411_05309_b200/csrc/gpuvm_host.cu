// Host side of the demand-paging runtime: handle life cycle, flush, reset, counters
// and the invariant kernel.  Everything a kernel needs travels in gpuvm_dev_t.
#include <cuda_runtime.h>

#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "gpuvm.h"
#include "gpuvm_device.cuh"
#include "gpuvm_internal.h"

struct gpuvm_handle {
    gpuvm_dev_t dev;
    void *host_user;        // host pointer of the backing store
    bool host_registered;   // we called cudaHostRegister on it
    bool host_allocated;    // we called cudaHostAlloc for it
    int device;
    int sms;                // SMs of that device
    int last_cuda;
    unsigned long long *check_buf;   // device, 8 words
    void *scratch;                   // device scratch for workload kernels (request tables)
    size_t scratch_bytes;
    size_t scratch_limit;      /* 0: none */
    unsigned int inplace_divisor;
    unsigned long long kept_pages;   // pages with the keep advice (gpuvm_advise_keep)
    int inplace_counted;    // 0: online; 1: lookups counted per page first; 2: counted, and rows in place read page by page
};

namespace {

using namespace gpuvm;

int fail(gpuvm_handle *h, cudaError_t e, int code)
{
    if (h) h->last_cuda = (int)e;
    cudaGetLastError();   // clear the non-sticky error state
    return code;
}

// A11: one warp per frame; dirty resident pages go back to the host.
__global__ void flush_kernel(gpuvm_dev_t vm)
{
    const unsigned int warps = (gridDim.x * blockDim.x) >> 5;
    const unsigned int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const unsigned int lane = threadIdx.x & 31;
    for (unsigned int f = warp; f < vm.n_frames; f += warps) {
        unsigned int e = vm.frame_vpn[f];
        if (e == kFrameFree || (e & kFrameLock)) continue;
        unsigned long long w = vm.pte[e];
        if ((w & kStMask) != kValid || !(w & kDirty)) continue;
        if ((unsigned int)((w & kFrameMask) >> kFrameShift) != f) continue;
        unsigned int len = page_len(vm, e);
        warp_copy<8, true>(vm.host + ((unsigned long long)e << vm.page_shift),
                           vm.pool + ((unsigned long long)f << vm.page_shift), len >> 4, lane, 32);
        __threadfence_system();
        __syncwarp();
        if (lane == 0) {
            atomicAnd(vm.pte + e, ~kDirty);
            stat_add(vm, kFlushWritebacks, 1);
            stat_add(vm, kBytesOut, len);
        }
    }
}

// A13: structural invariants of page table and frame ring.
// out: resident, frames_used, bad_state, bad_refcount, bad_backref, bad_range, dirty
__global__ void check_kernel(gpuvm_dev_t vm, unsigned long long *out)
{
    unsigned long long tid = blockIdx.x * (unsigned long long)blockDim.x + threadIdx.x;
    unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
    unsigned long long c[7] = {0, 0, 0, 0, 0, 0, 0};
    for (unsigned long long v = tid; v < vm.n_pages; v += stride) {
        unsigned long long w = vm.pte[v];
        unsigned long long st = w & kStMask;
        if (w & kRcMask) c[3]++;
        if (st == kValid) {
            c[0]++;
            if (w & kDirty) c[6]++;
            unsigned long long f = (w & kFrameMask) >> kFrameShift;
            if (f >= vm.n_frames) c[5]++;
            else if (vm.frame_vpn[f] != (unsigned int)v) c[4]++;
            if (w & ~(kStMask | kDirty | kRef | kKeep | kFrameMask | kRcMask)) c[2]++;
        } else if (st == kInvalid) {
            if (w & ~(kRcMask | kFrameMask | kKeep)) c[2]++;   // (the frame field counts in-place reads while INVALID)
        } else {
            c[2]++;
        }
    }
    for (unsigned long long f = tid; f < vm.n_frames; f += stride) {
        unsigned int e = vm.frame_vpn[f];
        if (e == kFrameFree) continue;
        c[1]++;
        if (e & kFrameLock) { c[2]++; continue; }
        if (e >= vm.n_pages) { c[5]++; continue; }
        unsigned long long w = vm.pte[e];
        if ((w & kStMask) != kValid || ((w & kFrameMask) >> kFrameShift) != f) c[4]++;
    }
    for (int k = 0; k < 7; ++k) {
        unsigned long long v = c[k];
        for (int o = 16; o; o >>= 1) v += __shfl_down_sync(0xFFFFFFFFu, v, o);
        if ((threadIdx.x & 31) == 0 && v) atomicAdd(out + k, v);
    }
}

__global__ void reset_keep_kernel(unsigned long long *pte, unsigned long long n_pages)
{
    for (unsigned long long v = blockIdx.x * (unsigned long long)blockDim.x + threadIdx.x; v < n_pages;
         v += (unsigned long long)gridDim.x * blockDim.x)
        pte[v] &= kKeep;
}

// Sets or clears the keep bit of the pages [first, first + n); *changed counts the entries whose bit changed.
__global__ void advise_keep_kernel(unsigned long long *pte, unsigned long long first, unsigned long long n, int keep,
                                   unsigned long long *changed)
{
    unsigned long long c = 0;
    for (unsigned long long v = blockIdx.x * (unsigned long long)blockDim.x + threadIdx.x; v < n;
         v += (unsigned long long)gridDim.x * blockDim.x) {
        const unsigned long long old = keep ? atomicOr(pte + first + v, kKeep) : atomicAnd(pte + first + v, ~kKeep);
        c += ((old & kKeep) != 0ull) != (keep != 0);
    }
    if (c) atomicAdd(changed, c);
}

// Number of SMs of the handle's device (grids are sized in multiples of it).
int sm_count_of(int device)
{
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sms <= 0) {
        cudaGetLastError();
        sms = 148;
    }
    return sms;
}

bool is_pow2(size_t x) { return x && !(x & (x - 1)); }

int ilog2(size_t x)
{
    int s = 0;
    while ((size_t(1) << s) < x) ++s;
    return s;
}

}  // namespace

extern "C" {

int gpuvm_create(gpuvm_t *out, void *host_backing, size_t bytes, size_t page_bytes, size_t pool_bytes)
{
    if (!out) return GPUVM_E_ARG;
    *out = nullptr;
    if (bytes == 0) return GPUVM_E_ARG;
    if (!is_pow2(page_bytes) || page_bytes < 16 || page_bytes > (size_t(1) << 30)) return GPUVM_E_PAGE;
    if ((bytes + page_bytes - 1) / page_bytes > 0x7FFFFFFEull) return GPUVM_E_PAGE;
    if (pool_bytes == 0 || pool_bytes % page_bytes != 0 || pool_bytes / page_bytes > 0x7FFFFFFEull)
        return GPUVM_E_POOL;
    if (bytes % 16 != 0 || (reinterpret_cast<uintptr_t>(host_backing) & 15u)) return GPUVM_E_ALIGN;

    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0) { cudaGetLastError(); return GPUVM_E_NODEVICE; }

    gpuvm_handle *h = new (std::nothrow) gpuvm_handle();
    if (!h) return GPUVM_E_ALLOC;
    memset(h, 0, sizeof(*h));
    cudaGetDevice(&h->device);
    h->sms = sm_count_of(h->device);
    h->inplace_divisor = GPUVM_INPLACE_AUTO;
    h->inplace_counted = 2;
    cudaError_t e;

    // backing store: pinned and mapped (Section 4: the host region is registered before
    // the application starts; here with the CUDA driver instead of a NIC)
    void *dev_host = nullptr;
    if (!host_backing) {
        e = cudaHostAlloc(&host_backing, bytes, cudaHostAllocMapped | cudaHostAllocPortable);
        if (e != cudaSuccess) { int rc = fail(h, e, GPUVM_E_PIN); delete h; return rc; }
        h->host_allocated = true;
    } else {
        cudaPointerAttributes attr;
        e = cudaPointerGetAttributes(&attr, host_backing);
        bool pinned = (e == cudaSuccess && attr.type == cudaMemoryTypeHost);
        cudaGetLastError();
        if (e == cudaSuccess && (attr.type == cudaMemoryTypeDevice || attr.type == cudaMemoryTypeManaged)) {
            delete h;
            return GPUVM_E_PIN;     // the backing store must be host memory
        }
        if (!pinned) {
            e = cudaHostRegister(host_backing, bytes, cudaHostRegisterMapped | cudaHostRegisterPortable);
            if (e != cudaSuccess) { int rc = fail(h, e, GPUVM_E_PIN); delete h; return rc; }
            h->host_registered = true;
        }
    }
    h->host_user = host_backing;
    e = cudaHostGetDevicePointer(&dev_host, host_backing, 0);
    if (e != cudaSuccess) {
        int rc = fail(h, e, GPUVM_E_PIN);
        if (h->host_registered) cudaHostUnregister(host_backing);
        if (h->host_allocated) cudaFreeHost(host_backing);
        delete h;
        return rc;
    }

    gpuvm_dev_t &d = h->dev;
    d.host = static_cast<unsigned char *>(dev_host);
    d.bytes = bytes;
    d.page_shift = (unsigned int)ilog2(page_bytes);
    d.n_pages = (bytes + page_bytes - 1) / page_bytes;
    d.n_frames = (unsigned int)(pool_bytes / page_bytes);
    d.policy = GPUVM_POLICY_CLOCK;
    d.spin_limit_us = 10u * 1000u * 1000u;
    d.clean_ahead = 0;                              // write-back off the fault path is opt-in: gpuvm_set_clean_ahead

    bool ok = cudaMalloc(&d.pte, d.n_pages * sizeof(unsigned long long)) == cudaSuccess &&
              cudaMalloc(&d.frame_vpn, d.n_frames * sizeof(unsigned int)) == cudaSuccess &&
              cudaMalloc(&d.ctl, kCtlWords * sizeof(unsigned long long)) == cudaSuccess &&
              cudaMalloc(&h->check_buf, 8 * sizeof(unsigned long long)) == cudaSuccess &&
              cudaMalloc(&d.pool, pool_bytes) == cudaSuccess;
    if (!ok) {
        fail(h, cudaGetLastError(), GPUVM_E_ALLOC);
        cudaFree(d.pte); cudaFree(d.frame_vpn); cudaFree(d.ctl); cudaFree(h->check_buf); cudaFree(d.pool);
        if (h->host_registered) cudaHostUnregister(host_backing);
        if (h->host_allocated) cudaFreeHost(host_backing);
        cudaGetLastError();
        delete h;
        return GPUVM_E_ALLOC;
    }
    *out = h;
    int rc = gpuvm_reset(h);
    if (rc != GPUVM_OK) { gpuvm_destroy(h); *out = nullptr; }
    return rc;
}

int gpuvm_reset_on(gpuvm_t h, void *stream)
{
    if (!h) return GPUVM_E_ARG;
    gpuvm_dev_t &d = h->dev;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaSuccess;
    if (h->kept_pages == 0) {
        e = cudaMemsetAsync(d.pte, 0, d.n_pages * sizeof(unsigned long long), s);
    } else {                                                  // advice survives a reset
        reset_keep_kernel<<<h->sms * 4, 256, 0, s>>>(d.pte, d.n_pages);
        gpuvm_note_launch_(1);
        e = cudaGetLastError();
    }
    if (e == cudaSuccess) e = cudaMemsetAsync(d.frame_vpn, 0xFF, d.n_frames * sizeof(unsigned int), s);
    if (e == cudaSuccess) e = cudaMemsetAsync(d.ctl, 0, kCtlWords * sizeof(unsigned long long), s);
    return e == cudaSuccess ? GPUVM_OK : fail(h, e, GPUVM_E_CUDA);
}

int gpuvm_reset(gpuvm_t h)
{
    if (!h) return GPUVM_E_ARG;
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return fail(h, e, GPUVM_E_CUDA);
    int rc = gpuvm_reset_on(h, nullptr);
    if (rc != GPUVM_OK) return rc;
    e = cudaDeviceSynchronize();
    return e == cudaSuccess ? GPUVM_OK : fail(h, e, GPUVM_E_CUDA);
}

int gpuvm_flush(gpuvm_t h, void *stream)
{
    if (!h) return GPUVM_E_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const unsigned int all = (unsigned int)h->sms * 32u;      // one warp per frame, up to 32 warps per SM
    unsigned int warps = h->dev.n_frames < all ? h->dev.n_frames : all;
    unsigned int blocks = (warps + 7) / 8;
    flush_kernel<<<blocks, 256, 0, s>>>(h->dev);
    gpuvm_note_launch_(1);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    return e == cudaSuccess ? GPUVM_OK : fail(h, e, GPUVM_E_CUDA);
}

int gpuvm_destroy(gpuvm_t h)
{
    if (!h) return GPUVM_E_ARG;
    int rc = gpuvm_flush(h, nullptr);
    cudaFree(h->dev.pte); cudaFree(h->dev.frame_vpn); cudaFree(h->dev.ctl);
    cudaFree(h->check_buf); cudaFree(h->dev.pool); cudaFree(h->scratch);
    if (h->host_registered) cudaHostUnregister(h->host_user);
    if (h->host_allocated) cudaFreeHost(h->host_user);
    cudaGetLastError();
    delete h;
    return rc;
}

int gpuvm_check_on(gpuvm_t h, gpuvm_check_t *out, void *stream)
{
    if (!h || !out) return GPUVM_E_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemsetAsync(h->check_buf, 0, 8 * sizeof(unsigned long long), s);
    if (e != cudaSuccess) return fail(h, e, GPUVM_E_CUDA);
    check_kernel<<<h->sms, 256, 0, s>>>(h->dev, h->check_buf);
    gpuvm_note_launch_(1);
    unsigned long long c[8];
    e = cudaMemcpyAsync(c, h->check_buf, sizeof(c), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return fail(h, e, GPUVM_E_CUDA);
    out->resident = c[0]; out->frames_used = c[1]; out->bad_state = c[2]; out->bad_refcount = c[3];
    out->bad_backref = c[4]; out->bad_range = c[5]; out->dirty = c[6];
    bool bad = c[2] || c[3] || c[4] || c[5] || c[0] != c[1] || c[0] > h->dev.n_frames;
    return bad ? GPUVM_E_INVARIANT : GPUVM_OK;
}

int gpuvm_check(gpuvm_t h, gpuvm_check_t *out) { return gpuvm_check_on(h, out, nullptr); }

int gpuvm_stats_on(gpuvm_t h, gpuvm_stats_t *out, void *stream)
{
    if (!h || !out) return GPUVM_E_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    unsigned long long local[kCtlWords];
    cudaError_t e = cudaMemcpyAsync(local, h->dev.ctl, sizeof(local), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return fail(h, e, GPUVM_E_CUDA);
    unsigned long long sum[kNumStats] = {0};
    for (int k = 0; k < kStatSlots; ++k)
        for (int j = 0; j < kNumStats; ++j) sum[j] += local[kCtlCounters + k * 16 + j];
    memset(out, 0, sizeof(*out));
    out->faults = sum[kFaults]; out->hits = sum[kHits]; out->waits = sum[kWaits];
    out->lanes_coalesced = sum[kLanes]; out->evictions = sum[kEvictions];
    out->writebacks = sum[kWritebacks]; out->flush_writebacks = sum[kFlushWritebacks];
    out->bytes_in = sum[kBytesIn]; out->bytes_out = sum[kBytesOut];
    out->hand_steps = sum[kHandSteps]; out->retries = sum[kRetries];
    out->ring_drops = sum[kRingDrops];
    out->cleaned = sum[kCleaned];
    out->bytes_direct = sum[kBytesDirect];
    out->resident = out->faults - out->evictions;
    out->error = (int32_t)(long long)local[kCtlErr];
    out->error_page = local[kCtlErrPage];
    return out->error;
}

int gpuvm_stats(gpuvm_t h, gpuvm_stats_t *out)
{
    if (!h || !out) return GPUVM_E_ARG;
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return fail(h, e, GPUVM_E_CUDA);
    return gpuvm_stats_on(h, out, nullptr);
}

void *gpuvm_scratch_(gpuvm_handle *h, size_t bytes)
{
    if (!h) return nullptr;
    if (bytes <= h->scratch_bytes) return h->scratch;
    cudaDeviceSynchronize();
    cudaFree(h->scratch);
    h->scratch = nullptr;
    h->scratch_bytes = 0;
    if (cudaMalloc(&h->scratch, bytes) != cudaSuccess) { h->last_cuda = (int)cudaGetLastError(); h->scratch = nullptr; return nullptr; }
    h->scratch_bytes = bytes;
    return h->scratch;
}

size_t gpuvm_scratch_limit_(gpuvm_handle *h) { return h && h->scratch_limit ? h->scratch_limit : ~size_t(0); }

int gpuvm_set_scratch_limit(gpuvm_t h, size_t bytes)
{
    if (!h) return GPUVM_E_ARG;
    h->scratch_limit = bytes;
    return GPUVM_OK;
}

size_t gpuvm_scratch_bytes(gpuvm_t h) { return h ? h->scratch_bytes : 0; }

size_t gpuvm_inplace_divisor_(gpuvm_handle *h) { return h ? h->inplace_divisor : 0; }
int gpuvm_inplace_counted_(gpuvm_handle *h) { return h ? h->inplace_counted : 0; }

int gpuvm_set_inplace_divisor(gpuvm_t h, unsigned int divisor)
{
    if (!h) return GPUVM_E_ARG;
    h->inplace_divisor = divisor;
    return GPUVM_OK;
}

int gpuvm_advise_keep(gpuvm_t h, size_t byte_off, size_t bytes, int keep)
{
    if (!h || bytes == 0) return GPUVM_E_ARG;
    gpuvm_dev_t &d = h->dev;
    if (byte_off >= d.bytes || bytes > d.bytes - byte_off) return GPUVM_E_RANGE;
    const unsigned long long first = byte_off >> d.page_shift, last = (byte_off + bytes - 1) >> d.page_shift;
    const unsigned long long n = last - first + 1;
    // pages that may never be evicted must leave room for the others: at most half the pool
    if (keep && h->kept_pages + n > d.n_frames / 2) return GPUVM_E_FRAMES;
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return fail(h, e, GPUVM_E_CUDA);
    unsigned long long *changed = h->check_buf;               // (device scratch of the checker, free between calls)
    e = cudaMemset(changed, 0, sizeof(unsigned long long));
    if (e != cudaSuccess) return fail(h, e, GPUVM_E_CUDA);
    advise_keep_kernel<<<h->sms * 4, 256>>>(d.pte, first, n, keep, changed);
    gpuvm_note_launch_(1);
    unsigned long long c = 0;
    e = cudaMemcpy(&c, changed, sizeof(c), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return fail(h, e, GPUVM_E_CUDA);
    if (keep) h->kept_pages += c; else h->kept_pages -= c < h->kept_pages ? c : h->kept_pages;
    return GPUVM_OK;
}

int gpuvm_set_inplace_counted(gpuvm_t h, int counted)
{
    if (!h || counted < 0 || counted > 2) return GPUVM_E_ARG;
    h->inplace_counted = counted;
    return GPUVM_OK;
}

int gpuvm_device_view(gpuvm_t h, gpuvm_dev_t *out)
{
    if (!h || !out) return GPUVM_E_ARG;
    *out = h->dev;
    return GPUVM_OK;
}

void *gpuvm_host_ptr(gpuvm_t h) { return h ? h->host_user : nullptr; }

int gpuvm_set_policy(gpuvm_t h, int policy)
{
    if (!h || (policy != GPUVM_POLICY_FIFO && policy != GPUVM_POLICY_CLOCK)) return GPUVM_E_ARG;
    h->dev.policy = (unsigned int)policy;
    return GPUVM_OK;
}

int gpuvm_set_debug(gpuvm_t h, unsigned int flags)
{
    if (!h || (flags & ~(unsigned int)(GPUVM_DEBUG_POISON | GPUVM_DEBUG_FENCED_RELEASE))) return GPUVM_E_ARG;
    h->dev.debug = flags;
    return GPUVM_OK;
}

int gpuvm_set_clean_ahead(gpuvm_t h, unsigned int frames)
{
    if (!h) return GPUVM_E_ARG;
    h->dev.clean_ahead = frames < h->dev.n_frames ? frames : h->dev.n_frames;
    return GPUVM_OK;
}

int gpuvm_set_spin_limit_us(gpuvm_t h, unsigned int us)
{
    if (!h || us == 0) return GPUVM_E_ARG;
    h->dev.spin_limit_us = us;
    return GPUVM_OK;
}

int gpuvm_safe_warps(gpuvm_t h, int pins_per_warp)
{
    if (!h || pins_per_warp <= 0) return GPUVM_E_ARG;
    unsigned int w = h->dev.n_frames / (unsigned int)pins_per_warp;
    return w > 0x7FFFFFFFu ? 0x7FFFFFFF : (int)w;
}

double gpuvm_inflight_pages(double latency_s, double bytes_per_s, double page_bytes)
{
    return page_bytes > 0 ? latency_s * bytes_per_s / page_bytes : 0.0;
}

int gpuvm_debug_poke_pte(gpuvm_t h, uint64_t page, uint64_t value)
{
    if (!h || page >= h->dev.n_pages) return GPUVM_E_ARG;
    cudaError_t e = cudaMemcpy(h->dev.pte + page, &value, sizeof(value), cudaMemcpyHostToDevice);
    return e == cudaSuccess ? GPUVM_OK : fail(h, e, GPUVM_E_CUDA);
}

int gpuvm_debug_peek_pte(gpuvm_t h, uint64_t page, uint64_t *value)
{
    if (!h || !value || page >= h->dev.n_pages) return GPUVM_E_ARG;
    cudaError_t e = cudaMemcpy(value, h->dev.pte + page, sizeof(*value), cudaMemcpyDeviceToHost);
    return e == cudaSuccess ? GPUVM_OK : fail(h, e, GPUVM_E_CUDA);
}

const char *gpuvm_strerror(int status)
{
    switch (status) {
    case GPUVM_OK: return "ok";
    case GPUVM_E_ARG: return "bad argument";
    case GPUVM_E_PAGE: return "page size must be a power of two between 16 bytes and 1 GiB, with fewer than 2^31 pages";
    case GPUVM_E_POOL: return "pool size must be a non-zero multiple of the page size";
    case GPUVM_E_ALIGN: return "backing store must be 16-byte aligned and a multiple of 16 bytes long";
    case GPUVM_E_PIN: return "cannot pin and map the host backing store";
    case GPUVM_E_ALLOC: return "device allocation failed";
    case GPUVM_E_CUDA: return "CUDA runtime error";
    case GPUVM_E_TIMEOUT: return "a device-side wait ran out";
    case GPUVM_E_RANGE: return "offset past the end of the paged array";
    case GPUVM_E_INVARIANT: return "page-table invariant violated";
    case GPUVM_E_NODEVICE: return "no CUDA device";
    case GPUVM_E_PINS: return "too many simultaneous references to one page";
    case GPUVM_E_FRAMES: return "the pool has too few frames for the pages this workload pins at once";
    default: return "unknown status";
    }
}

int gpuvm_last_cuda_error(gpuvm_t h) { return h ? h->last_cuda : 0; }

}  // extern "C"
