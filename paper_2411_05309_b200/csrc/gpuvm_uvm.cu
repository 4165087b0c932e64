// Managed-memory helpers for the UVM comparison runs (not part of the paged path).
#include <cuda_runtime.h>

#include "gpuvm_uvm.h"

namespace {
int status(cudaError_t e, int code)
{
    if (e == cudaSuccess) return GPUVM_OK;
    cudaGetLastError();
    return code;
}
}  // namespace

extern "C" {

int gpuvm_uvm_alloc(void **out, size_t bytes)
{
    if (!out || bytes == 0) return GPUVM_E_ARG;
    *out = nullptr;
    return status(cudaMallocManaged(out, bytes, cudaMemAttachGlobal), GPUVM_E_ALLOC);
}

int gpuvm_uvm_free(void *p) { return p ? status(cudaFree(p), GPUVM_E_CUDA) : GPUVM_E_ARG; }

int gpuvm_uvm_advise_read_mostly(void *p, size_t bytes, int on)
{
    if (!p || bytes == 0) return GPUVM_E_ARG;
    int dev = 0;
    cudaGetDevice(&dev);
    return status(cudaMemAdvise(p, bytes, on ? cudaMemAdviseSetReadMostly : cudaMemAdviseUnsetReadMostly, dev),
                  GPUVM_E_CUDA);
}

int gpuvm_uvm_evict_to_host(void *p, size_t bytes)
{
    if (!p || bytes == 0) return GPUVM_E_ARG;
    cudaError_t e = cudaMemPrefetchAsync(p, bytes, cudaCpuDeviceId, nullptr);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    return status(e, GPUVM_E_CUDA);
}

int gpuvm_mem_info(size_t *free_bytes, size_t *total_bytes)
{
    if (!free_bytes || !total_bytes) return GPUVM_E_ARG;
    return status(cudaMemGetInfo(free_bytes, total_bytes), GPUVM_E_CUDA);
}

int gpuvm_balloon_alloc(void **out, size_t leave_free)
{
    if (!out) return GPUVM_E_ARG;
    *out = nullptr;
    size_t free_b = 0, total_b = 0;
    if (cudaMemGetInfo(&free_b, &total_b) != cudaSuccess) { cudaGetLastError(); return GPUVM_E_CUDA; }
    if (free_b <= leave_free) return GPUVM_OK;
    size_t take = (free_b - leave_free) & ~((size_t(2) << 20) - 1);
    if (take == 0) return GPUVM_OK;
    return status(cudaMalloc(out, take), GPUVM_E_ALLOC);
}

int gpuvm_balloon_free(void *p) { return p ? status(cudaFree(p), GPUVM_E_CUDA) : GPUVM_OK; }

}  // extern "C"
