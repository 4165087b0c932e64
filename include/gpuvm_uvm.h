/*
 * gpuvm_uvm.h -- helpers for the comparison runs over CUDA managed memory (the
 * paper's UVM baseline, Section 5: the same kernels on cudaMallocManaged data with
 * the GPU memory artificially limited, with and without cudaMemAdviseSetReadMostly).
 * Not part of the paged path.  All functions return 0 or a negative gpuvm_status.
 */
#ifndef GPUVM_UVM_H
#define GPUVM_UVM_H

#include "gpuvm.h"

#ifdef __cplusplus
extern "C" {
#endif

/* cudaMallocManaged / cudaFree.  *out: host pointer to the result (valid on host and device). */
int gpuvm_uvm_alloc(void **out, size_t bytes);
int gpuvm_uvm_free(void *p);

/* cudaMemAdviseSetReadMostly (on != 0) or Unset on [p, p + bytes) for the current device. */
int gpuvm_uvm_advise_read_mostly(void *p, size_t bytes, int on);

/* Send every page of [p, p + bytes) back to host memory and wait: a cold start. */
int gpuvm_uvm_evict_to_host(void *p, size_t bytes);

/* Free and total device memory in bytes (host pointers). */
int gpuvm_mem_info(size_t *free_bytes, size_t *total_bytes);

/* "Balloon": one cudaMalloc that leaves only `leave_free` bytes of device memory
 * free, so that managed memory is oversubscribed the way the paper limits GPU
 * memory (Section 5.4).  *out receives the device pointer (NULL if nothing needed
 * to be taken).  gpuvm_balloon_free releases it. */
int gpuvm_balloon_alloc(void **out, size_t leave_free);
int gpuvm_balloon_free(void *p);

#ifdef __cplusplus
}
#endif
#endif /* GPUVM_UVM_H */
