// Shared by the translation units of libgpuvm: launch accounting and handle-owned scratch.
#ifndef GPUVM_INTERNAL_H
#define GPUVM_INTERNAL_H
#include <stddef.h>
#ifdef __cplusplus
extern "C" {
#endif
void gpuvm_note_launch_(unsigned long long n);

/* Device scratch owned by the handle: at least `bytes` long, 256-byte aligned, contents
 * undefined.  Grown (never shrunk) on demand, freed by gpuvm_destroy.  NULL if the
 * allocation fails.  Growing synchronises the device. */
struct gpuvm_handle;
void *gpuvm_scratch_(struct gpuvm_handle *h, size_t bytes);
/* bound set with gpuvm_set_scratch_limit, SIZE_MAX when there is none */
size_t gpuvm_scratch_limit_(struct gpuvm_handle *h);
/* divisor set with gpuvm_set_inplace_divisor (default GPUVM_INPLACE_AUTO; 0: requests are never served in place) and
 * whether lookups are counted per page first (gpuvm_set_inplace_counted, default yes) */
size_t gpuvm_inplace_divisor_(struct gpuvm_handle *h);
int gpuvm_inplace_counted_(struct gpuvm_handle *h);
#ifdef __cplusplus
}
#endif
#endif
