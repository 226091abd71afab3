// Checked build (-DEDGELORA_CHECKED): the library's own device buffers get a zone of 256 bytes in
// front and behind, filled with a fixed byte, and edgelora_check_guards() compares every zone with
// that byte; kernels check the indices they take from device memory (see EL_CHECK in internal.cuh).
// In the normal build el_malloc / el_free are cudaMalloc / cudaFree and nothing is registered.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>

namespace edgelora {

#ifdef EDGELORA_CHECKED
cudaError_t el_malloc_impl(void **ptr, size_t bytes);
cudaError_t el_free(void *ptr);
#else
inline cudaError_t el_malloc_impl(void **ptr, size_t bytes) { return cudaMalloc(ptr, bytes); }
inline cudaError_t el_free(void *ptr) { return cudaFree(ptr); }
#endif
template <typename T>
inline cudaError_t el_malloc(T **ptr, size_t bytes) {
  return el_malloc_impl(reinterpret_cast<void **>(ptr), bytes);
}

// 0 = every zone intact (always, in the normal build); otherwise the 1-based number of the first
// damaged buffer in allocation order, with its size in *bytes_out and -1 / +1 in *side_out for the
// zone in front of / behind it.  Synchronises the device.
int guards_check(size_t *bytes_out, int *side_out);

}  // namespace edgelora
