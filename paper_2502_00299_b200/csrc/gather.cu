// Stand-alone K/V row gather and compaction kernel (see gather.cuh). With indices taken from
// another layer this is the whole work of an index-reuse layer (ChunkKV Algorithm 2).
#include "gather.cuh"
#include "internal.h"

namespace chunkkv {

namespace {

constexpr int kGatherThreads = 256;
// A CTA small enough (64 threads x 64 registers) to share an SM with a resident layer-kernel CTA
// (576 threads x 96 registers leave room for 10240 registers).
constexpr int kGatherThreadsSmall = 64;

template <int VPR, int THREADS>
__global__ void __launch_bounds__(THREADS)
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
    const int rows_per_block = (THREADS / VPR) * kGatherRowsPerThread;
    for (int n0 = blockIdx.x * rows_per_block; n0 < n_max; n0 += gridDim.x * rows_per_block)
        gather_rows<VPR, false>(Kh, Vh, ih, L, n_max, n0, threadIdx.x, THREADS, oK, oV, ic);
}

}  // namespace

template <int THREADS>
static cudaError_t launch_gather_t(const void* K, const void* V, const int32_t* idx, int L, int Hkv, int d, int n_max,
                                   void* out_K, void* out_V, int32_t* idx_copy_or_null, int max_blocks,
                                   cudaStream_t stream) {
    const int vpr = d / 8;
    const int rows_per_block = (THREADS / vpr) * kGatherRowsPerThread;
    int bx = (n_max + rows_per_block - 1) / rows_per_block;
    const int cap = (max_blocks + Hkv - 1) / Hkv;
    if (bx > cap) bx = cap;
    if (bx < 1) bx = 1;
    dim3 grid(bx, Hkv);
    if (vpr == 16)
        gather_kernel<16, THREADS><<<grid, THREADS, 0, stream>>>(
            static_cast<const uint4*>(K), static_cast<const uint4*>(V), idx, L, n_max,
            static_cast<uint4*>(out_K), static_cast<uint4*>(out_V), idx_copy_or_null);
    else
        gather_kernel<8, THREADS><<<grid, THREADS, 0, stream>>>(
            static_cast<const uint4*>(K), static_cast<const uint4*>(V), idx, L, n_max,
            static_cast<uint4*>(out_K), static_cast<uint4*>(out_V), idx_copy_or_null);
    return cudaGetLastError();
}

cudaError_t launch_gather(const void* K, const void* V, const int32_t* idx, int L, int Hkv, int d,
                          int n_max, void* out_K, void* out_V, int32_t* idx_copy_or_null,
                          int num_sms, cudaStream_t stream) {
    if (n_max <= 0 || Hkv <= 0) return cudaSuccess;
    return launch_gather_t<kGatherThreads>(K, V, idx, L, Hkv, d, n_max, out_K, out_V, idx_copy_or_null, 16 * num_sms,
                                           stream);
}

// The same gather in CTAs of 64 threads spread over the whole GPU: such a CTA fits on an SM
// beside a resident CTA of the layer kernel, so the row traffic of one lane's layer can use every
// SM's load/store path while the other lanes keep scoring.
cudaError_t launch_gather_shared_sms(const void* K, const void* V, const int32_t* idx, int L, int Hkv, int d,
                                     int n_max, void* out_K, void* out_V, int num_sms, cudaStream_t stream) {
    if (n_max <= 0 || Hkv <= 0) return cudaSuccess;
    return launch_gather_t<kGatherThreadsSmall>(K, V, idx, L, Hkv, d, n_max, out_K, out_V, nullptr, 4 * num_sms, stream);
}

}  // namespace chunkkv
