#include "alloc.h"

#include <mutex>
#include <unordered_map>

namespace umd {

namespace {
std::mutex g_mu;
std::unordered_map<void*, size_t> g_sizes;
int64_t g_total = 0;
}  // namespace

cudaError_t dev_malloc(void** p, size_t bytes) {
    *p = nullptr;
    if (bytes == 0) bytes = 16;
    cudaError_t e = cudaMalloc(p, bytes);
    if (e != cudaSuccess) { *p = nullptr; return e; }
    std::lock_guard<std::mutex> lk(g_mu);
    g_sizes[*p] = bytes;
    g_total += (int64_t)bytes;
    return cudaSuccess;
}

void dev_free(void* p) {
    if (!p) return;
    {
        std::lock_guard<std::mutex> lk(g_mu);
        auto it = g_sizes.find(p);
        if (it != g_sizes.end()) { g_total -= (int64_t)it->second; g_sizes.erase(it); }
    }
    cudaFree(p);
}

int64_t dev_bytes_held() {
    std::lock_guard<std::mutex> lk(g_mu);
    return g_total;
}

}  // namespace umd
