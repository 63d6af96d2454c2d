// Stand-alone top-k chunk selection kernel: one CTA per KV head (see select.cuh).
#include "internal.h"
#include "select.cuh"

namespace chunkkv {

namespace {

constexpr int kSelThreads = 512;

template <bool IN_REGS>
__global__ void __launch_bounds__(kSelThreads)
select_kernel(const float* __restrict__ scores, int L, int w, int c, int C, int k, int n_max,
              int32_t* __restrict__ out_idx) {
    __shared__ SelectSmem sm;
    const int h = blockIdx.x;
    select_head<IN_REGS>(scores + static_cast<size_t>(h) * C, L, w, c, C, k, n_max,
                         out_idx + static_cast<size_t>(h) * n_max, sm);
}

}  // namespace

cudaError_t launch_select(const float* scores, int L, int Hkv, int w, int c, int C, int k, int n_max,
                          int32_t* out_idx, cudaStream_t stream) {
    if (C <= kSelThreads * kSelPerThread)
        select_kernel<true><<<Hkv, kSelThreads, 0, stream>>>(scores, L, w, c, C, k, n_max, out_idx);
    else
        select_kernel<false><<<Hkv, kSelThreads, 0, stream>>>(scores, L, w, c, C, k, n_max, out_idx);
    return cudaGetLastError();
}

}  // namespace chunkkv
