// Stand-alone K/V row gather and compaction kernel (see gather.cuh). With indices taken from
// another layer this is the whole work of an index-reuse layer (ChunkKV Algorithm 2).
#include "gather.cuh"
#include "internal.h"

namespace chunkkv {

namespace {

constexpr int kGatherThreads = 256;

template <int VPR>
__global__ void __launch_bounds__(kGatherThreads)
gather_kernel(const uint4* __restrict__ K, const uint4* __restrict__ V, const int32_t* __restrict__ idx,
              int L, int n_max, uint4* __restrict__ out_K, uint4* __restrict__ out_V,
              int32_t* __restrict__ idx_copy) {
    const int h = blockIdx.y;
    const uint4* Kh = K + static_cast<size_t>(h) * L * VPR;
    const uint4* Vh = V + static_cast<size_t>(h) * L * VPR;
    const int32_t* ih = idx + static_cast<size_t>(h) * n_max;
    uint4* oK = out_K + static_cast<size_t>(h) * n_max * VPR;
    uint4* oV = out_V + static_cast<size_t>(h) * n_max * VPR;
    int32_t* ic = idx_copy ? idx_copy + static_cast<size_t>(h) * n_max : nullptr;
    const int rows_per_block = (kGatherThreads / VPR) * kGatherRowsPerThread;
    for (int n0 = blockIdx.x * rows_per_block; n0 < n_max; n0 += gridDim.x * rows_per_block)
        gather_rows<VPR, false>(Kh, Vh, ih, L, n_max, n0, threadIdx.x, kGatherThreads, oK, oV, ic);
}

}  // namespace

cudaError_t launch_gather(const void* K, const void* V, const int32_t* idx, int L, int Hkv, int d,
                          int n_max, void* out_K, void* out_V, int32_t* idx_copy_or_null,
                          int num_sms, cudaStream_t stream) {
    if (n_max <= 0 || Hkv <= 0) return cudaSuccess;
    const int vpr = d / 8;
    const int rows_per_block = (kGatherThreads / vpr) * kGatherRowsPerThread;
    int bx = (n_max + rows_per_block - 1) / rows_per_block;
    const int cap = (16 * num_sms + Hkv - 1) / Hkv;
    if (bx > cap) bx = cap;
    if (bx < 1) bx = 1;
    dim3 grid(bx, Hkv);
    if (vpr == 16)
        gather_kernel<16><<<grid, kGatherThreads, 0, stream>>>(
            static_cast<const uint4*>(K), static_cast<const uint4*>(V), idx, L, n_max,
            static_cast<uint4*>(out_K), static_cast<uint4*>(out_V), idx_copy_or_null);
    else
        gather_kernel<8><<<grid, kGatherThreads, 0, stream>>>(
            static_cast<const uint4*>(K), static_cast<const uint4*>(V), idx, L, n_max,
            static_cast<uint4*>(out_K), static_cast<uint4*>(out_V), idx_copy_or_null);
    return cudaGetLastError();
}

}  // namespace chunkkv
