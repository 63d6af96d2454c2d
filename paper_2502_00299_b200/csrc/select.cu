// Stand-alone top-k chunk selection kernel: one CTA per KV head (see select.cuh).
#include "internal.h"
#include "select.cuh"

namespace chunkkv {

namespace {

constexpr int kSelThreads = 512;

// KPT > 0: keys in registers (C <= kSelThreads * KPT). KPT = 0: keys in key_bytes of dynamic
// shared memory, or recomputed from the scores on every use if key_bytes is 0.
template <int KPT>
__global__ void __launch_bounds__(kSelThreads)
select_kernel(const float* __restrict__ scores, int L, int w, int c, int C, int k, int n_max,
              int32_t* __restrict__ out_idx, int key_bytes, int tok_cap) {
    __shared__ SelectSmem sm;
    extern __shared__ uint32_t key_buf[];
    const int h = blockIdx.x;
    const float* sc = scores + static_cast<size_t>(h) * C;
    int32_t* out = out_idx + static_cast<size_t>(h) * n_max;
    if constexpr (KPT > 0)
        select_head_regs<KPT>(sc, nullptr, L, w, c, C, k, n_max, out, sm, tok_cap);
    else if (key_bytes > 0)
        select_head_smem(sc, nullptr, L, w, c, C, k, n_max, out, sm, key_buf, tok_cap);
    else
        select_head_rows(sc, nullptr, L, w, c, C, k, n_max, out, sm, nullptr, tok_cap);
}

}  // namespace

cudaError_t launch_select(const float* scores, int L, int Hkv, int w, int c, int C, int k, int n_max,
                          int32_t* out_idx, cudaStream_t stream, int tok_cap) {
    // thousands of chunks per head: eight CTAs per head
    if (select_cluster_applies(C, k)) return launch_select_cluster(scores, L, Hkv, w, c, C, k, n_max, out_idx, stream, tok_cap);
    // a few keys per thread: registers (the fewest that hold every key)
    if (C <= kSelThreads * 4) {
        select_kernel<4><<<Hkv, kSelThreads, 0, stream>>>(scores, L, w, c, C, k, n_max, out_idx, 0, tok_cap);
        return cudaGetLastError();
    }
    if (C <= kSelThreads * 8) {
        select_kernel<8><<<Hkv, kSelThreads, 0, stream>>>(scores, L, w, c, C, k, n_max, out_idx, 0, tok_cap);
        return cudaGetLastError();
    }
    // more: the keys of a head live in dynamic shared memory if they fit beside the static scratch
    // (beyond the 48 KB every kernel may use, so the kernel opts in), else they are recomputed
    const size_t want = static_cast<size_t>(C) * 4;
    int key_bytes = 0, dev = 0, optin = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    const long room = static_cast<long>(optin) - static_cast<long>(sizeof(SelectSmem)) - 1024;
    if (room > 0 && want <= static_cast<size_t>(room)) {
        if (cudaFuncSetAttribute(select_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(room)) == cudaSuccess)
            key_bytes = static_cast<int>(want);
        else
            cudaGetLastError();
    }
    select_kernel<0><<<Hkv, kSelThreads, key_bytes, stream>>>(scores, L, w, c, C, k, n_max, out_idx, key_bytes, tok_cap);
    return cudaGetLastError();
}

}  // namespace chunkkv
