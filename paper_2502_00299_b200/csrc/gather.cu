// K/V row gather and compaction (ChunkKV Algorithm 3 "index_select(K, indices)" /
// "index_select(V, indices)"; with indices taken from another layer this is the whole work of
// an index-reuse layer, Algorithm 2).
//
// Rows are d bf16 = 128 or 256 bytes. Each thread moves 16 bytes of a row; a row is covered by
// d/8 adjacent threads, so every warp request is a set of fully used 128-byte lines. Each
// thread handles kRowsPerThread rows of K and of V with all loads issued before the stores.
#include "internal.h"

namespace chunkkv {

namespace {

constexpr int kGatherThreads = 256;
constexpr int kRowsPerThread = 4;

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream(uint4* p, const uint4& v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z),
                 "r"(v.w)
                 : "memory");
}

template <int VPR>   // 16-byte vectors per row: 8 (d = 64) or 16 (d = 128)
__global__ void __launch_bounds__(kGatherThreads)
gather_kernel(const uint4* __restrict__ K, const uint4* __restrict__ V, const int32_t* __restrict__ idx,
              int L, int n_max, uint4* __restrict__ out_K, uint4* __restrict__ out_V,
              int32_t* __restrict__ idx_copy) {
    constexpr int ROWS_PER_PASS = kGatherThreads / VPR;
    const int h = blockIdx.y;
    const int vec = threadIdx.x % VPR;
    const int sub = threadIdx.x / VPR;
    const uint4* Kh = K + static_cast<size_t>(h) * L * VPR;
    const uint4* Vh = V + static_cast<size_t>(h) * L * VPR;
    const int32_t* ih = idx + static_cast<size_t>(h) * n_max;
    uint4* oK = out_K + static_cast<size_t>(h) * n_max * VPR;
    uint4* oV = out_V + static_cast<size_t>(h) * n_max * VPR;
    const int rows_per_block = ROWS_PER_PASS * kRowsPerThread;
    for (int n0 = blockIdx.x * rows_per_block; n0 < n_max; n0 += gridDim.x * rows_per_block) {
        int src[kRowsPerThread];
        uint4 kv[kRowsPerThread], vv[kRowsPerThread];
#pragma unroll
        for (int u = 0; u < kRowsPerThread; ++u) {
            const int n = n0 + u * ROWS_PER_PASS + sub;
            src[u] = (n < n_max) ? ih[n] : -1;
        }
#pragma unroll
        for (int u = 0; u < kRowsPerThread; ++u) {
            const bool ok = static_cast<unsigned>(src[u]) < static_cast<unsigned>(L);
            kv[u] = ok ? ld_stream(Kh + static_cast<size_t>(src[u]) * VPR + vec) : make_uint4(0, 0, 0, 0);
            vv[u] = ok ? ld_stream(Vh + static_cast<size_t>(src[u]) * VPR + vec) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < kRowsPerThread; ++u) {
            const int n = n0 + u * ROWS_PER_PASS + sub;
            if (n < n_max) {
                st_stream(oK + static_cast<size_t>(n) * VPR + vec, kv[u]);
                st_stream(oV + static_cast<size_t>(n) * VPR + vec, vv[u]);
                if (idx_copy != nullptr && vec == 0) idx_copy[static_cast<size_t>(h) * n_max + n] = src[u];
            }
        }
    }
}

}  // namespace

cudaError_t launch_gather(const void* K, const void* V, const int32_t* idx, int L, int Hkv, int d,
                          int n_max, void* out_K, void* out_V, int32_t* idx_copy_or_null,
                          int num_sms, cudaStream_t stream) {
    if (n_max <= 0 || Hkv <= 0) return cudaSuccess;
    const int vpr = d / 8;
    const int rows_per_block = (kGatherThreads / vpr) * kRowsPerThread;
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
