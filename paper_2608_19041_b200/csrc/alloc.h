// Device allocations of the library, with a process-wide byte count for umlmd_query.
#pragma once

#include <cuda_runtime.h>

#include <cstdint>

namespace umd {

cudaError_t dev_malloc(void** p, size_t bytes);
void dev_free(void* p);
int64_t dev_bytes_held();

// Grow-only typed buffer: reallocates (contents lost) when `need` exceeds the capacity.
template <typename T>
cudaError_t dev_ensure(T** p, int64_t* cap, int64_t need, double growth = 1.0) {
    if (*p && need <= *cap) return cudaSuccess;
    if (*p) dev_free(*p);
    *p = nullptr;
    *cap = 0;
    const int64_t n = (int64_t)(need * growth) + 16;
    cudaError_t e = dev_malloc((void**)p, (size_t)n * sizeof(T));
    if (e == cudaSuccess) *cap = n;
    return e;
}

}  // namespace umd
