// Index-similarity diagnostic: Jaccard similarity of the kept-index rows of two layers, per KV
// head (the layer-wise index reuse section of the ChunkKV paper measures it between adjacent layers
// to justify sharing indices; on device it lets a caller pick the reuse depth while prefilling).
//
// Rows are as chunkkv_select / chunkkv_compress_layer write them: valid token positions in
// ascending order without repeats, then -1 padding. One CTA per head: every valid entry of row A is
// looked up in row B by binary search; |A u B| = |A| + |B| - |A n B|.
#include "internal.h"

namespace chunkkv {

namespace {

constexpr int kJacThreads = 256;

__global__ void __launch_bounds__(kJacThreads)
jaccard_kernel(const int32_t* __restrict__ idx_a, const int32_t* __restrict__ idx_b, int n_a, int n_b,
               float* __restrict__ out_ratio, int32_t* __restrict__ out_counts) {
    __shared__ int s_cnt[3];            // |A n B|, |A|, |B|
    const int h = blockIdx.x;
    const int32_t* a = idx_a + static_cast<size_t>(h) * n_a;
    const int32_t* b = idx_b + static_cast<size_t>(h) * n_b;
    if (threadIdx.x < 3) s_cnt[threadIdx.x] = 0;
    __syncthreads();
    // valid lengths: padding is a suffix, so the first negative entry ends the row
    int inter = 0, va = 0, vb = 0;
    for (int i = threadIdx.x; i < n_b; i += kJacThreads) vb += b[i] >= 0;
    // (row B's valid prefix length is needed for the searches: reduce it first)
    for (int off = 16; off > 0; off >>= 1) vb += __shfl_xor_sync(0xffffffffu, vb, off);
    if ((threadIdx.x & 31) == 0) atomicAdd(&s_cnt[2], vb);
    __syncthreads();
    const int len_b = s_cnt[2];
    for (int i = threadIdx.x; i < n_a; i += kJacThreads) {
        const int v = a[i];
        if (v < 0) continue;
        ++va;
        int lo = 0, hi = len_b;         // first position with b[pos] >= v
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (b[mid] < v) lo = mid + 1;
            else hi = mid;
        }
        inter += (lo < len_b && b[lo] == v);
    }
    for (int off = 16; off > 0; off >>= 1) {
        inter += __shfl_xor_sync(0xffffffffu, inter, off);
        va += __shfl_xor_sync(0xffffffffu, va, off);
    }
    if ((threadIdx.x & 31) == 0) {
        atomicAdd(&s_cnt[0], inter);
        atomicAdd(&s_cnt[1], va);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const int i_n = s_cnt[0], a_n = s_cnt[1], b_n = s_cnt[2];
        const int u_n = a_n + b_n - i_n;
        out_ratio[h] = u_n > 0 ? static_cast<float>(static_cast<double>(i_n) / static_cast<double>(u_n)) : 1.0f;
        if (out_counts != nullptr) {
            out_counts[h * 3 + 0] = i_n;
            out_counts[h * 3 + 1] = a_n;
            out_counts[h * 3 + 2] = b_n;
        }
    }
}

}  // namespace

cudaError_t launch_jaccard(const int32_t* idx_a, const int32_t* idx_b, int Hkv, int n_a, int n_b,
                           float* out_ratio, int32_t* out_counts_or_null, cudaStream_t stream) {
    if (Hkv <= 0) return cudaSuccess;
    jaccard_kernel<<<Hkv, kJacThreads, 0, stream>>>(idx_a, idx_b, n_a, n_b, out_ratio, out_counts_or_null);
    return cudaGetLastError();
}

}  // namespace chunkkv
