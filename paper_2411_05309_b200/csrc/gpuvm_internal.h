// Shared by the translation units of libgpuvm: launch accounting only.
#ifndef GPUVM_INTERNAL_H
#define GPUVM_INTERNAL_H
#ifdef __cplusplus
extern "C" {
#endif
void gpuvm_note_launch_(unsigned long long n);
#ifdef __cplusplus
}
#endif
#endif
