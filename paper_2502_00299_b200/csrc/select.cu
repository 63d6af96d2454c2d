// Stand-alone top-k chunk selection kernel: one CTA per KV head (see select.cuh).
#include "internal.h"
#include "select.cuh"

namespace chunkkv {

namespace {

constexpr int kSelThreads = 512;

template <int KPT>
__global__ void __launch_bounds__(kSelThreads)
select_kernel(const float* __restrict__ scores, int L, int w, int c, int C, int k, int n_max,
              int32_t* __restrict__ out_idx) {
    __shared__ SelectSmem sm;
    const int h = blockIdx.x;
    select_head<KPT>(scores + static_cast<size_t>(h) * C, nullptr, L, w, c, C, k, n_max,
                     out_idx + static_cast<size_t>(h) * n_max, sm);
}

}  // namespace

cudaError_t launch_select(const float* scores, int L, int Hkv, int w, int c, int C, int k, int n_max,
                          int32_t* out_idx, cudaStream_t stream) {
    // fewest registers per thread that still hold every key
    if (C <= kSelThreads * 4)
        select_kernel<4><<<Hkv, kSelThreads, 0, stream>>>(scores, L, w, c, C, k, n_max, out_idx);
    else if (C <= kSelThreads * 8)
        select_kernel<8><<<Hkv, kSelThreads, 0, stream>>>(scores, L, w, c, C, k, n_max, out_idx);
    else if (C <= kSelThreads * kSelPerThread)
        select_kernel<kSelPerThread><<<Hkv, kSelThreads, 0, stream>>>(scores, L, w, c, C, k, n_max, out_idx);
    else if (C <= kSelThreads * kSelPerThreadMax)
        select_kernel<kSelPerThreadMax><<<Hkv, kSelThreads, 0, stream>>>(scores, L, w, c, C, k, n_max, out_idx);
    else
        select_kernel<0><<<Hkv, kSelThreads, 0, stream>>>(scores, L, w, c, C, k, n_max, out_idx);
    return cudaGetLastError();
}

}  // namespace chunkkv
