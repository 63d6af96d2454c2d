// Stand-alone top-k chunk selection kernel: one CTA per KV head (see select.cuh).
#include "internal.h"
#include "select.cuh"

namespace chunkkv {

namespace {

constexpr int kSelThreads = 512;
constexpr int kSelKeyCap = 40960;     // keys staged in dynamic shared memory (160 KB)

__global__ void __launch_bounds__(kSelThreads)
select_kernel(const float* __restrict__ scores, int L, int w, int c, int C, int k, int n_max,
              int32_t* __restrict__ out_idx, int key_cap) {
    __shared__ SelectSmem sm;
    extern __shared__ uint32_t sel_keys[];
    const int h = blockIdx.x;
    select_head(scores + static_cast<size_t>(h) * C, L, w, c, C, k, n_max,
                out_idx + static_cast<size_t>(h) * n_max, sm, sel_keys, key_cap);
}

}  // namespace

cudaError_t launch_select(const float* scores, int L, int Hkv, int w, int c, int C, int k, int n_max,
                          int32_t* out_idx, cudaStream_t stream) {
    static int attr_set[64] = {0};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const int key_cap = C <= kSelKeyCap ? C : 0;          // too many keys: re-read them from memory
    const int dyn = key_cap * static_cast<int>(sizeof(uint32_t));
    if (dev < 0 || dev >= 64 || attr_set[dev] < dyn) {
        e = cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kSelKeyCap * static_cast<int>(sizeof(uint32_t)));
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set[dev] = kSelKeyCap * static_cast<int>(sizeof(uint32_t));
    }
    select_kernel<<<Hkv, kSelThreads, dyn, stream>>>(scores, L, w, c, C, k, n_max, out_idx, key_cap);
    return cudaGetLastError();
}

}  // namespace chunkkv
