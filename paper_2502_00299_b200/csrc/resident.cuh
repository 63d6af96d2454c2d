// Pieces shared by the kernels that keep their chunk partial sums in tensor memory
// (layer_resident.cu: one layer per launch; model_kernel.cu: many layers per launch).
#pragma once
#include "ptx.cuh"

#include <cuda_runtime.h>
#include <stdint.h>

namespace chunkkv {

constexpr int kRTile = 120;                  // keys per accumulator tile
constexpr int kRUmmaN = 128;                 // UMMA N (a multiple of 16): the last 8 columns are never read
constexpr int kRPanel = 60;                  // keys per epilogue panel (half a tile)
constexpr int kRStageBytes = kRTile * 128;   // one stage = 120 keys x 64 dims, 128-byte swizzled rows
constexpr int kRMaxStages = 14;
constexpr int kRPartCol0 = 256;              // tensor-memory column of the first chunk partial sum
constexpr int kRPartCols = 256;
constexpr int kRQTileBytes = 128 * 128;

template <int SPP>
__device__ __forceinline__ void part_store(uint32_t taddr, const float (&p)[SPP]) {
    static_assert(SPP == 6 || SPP == 3, "chunk slots per 60-key panel");
    if constexpr (SPP == 6) { tmem_st_x4(taddr, &p[0]); tmem_st_x2(taddr + 4, &p[4]); }
    else { tmem_st_x2(taddr, &p[0]); tmem_st_x1(taddr + 2, &p[2]); }
}
template <int SPP>
__device__ __forceinline__ void part_load(uint32_t taddr, float* p) {
    if constexpr (SPP == 6) { tmem_ld_x4(taddr, p); tmem_ld_x2(taddr + 4, p + 4); }
    else { tmem_ld_x2(taddr, p); tmem_ld_x1(taddr + 2, p + 2); }
}

// Sum of 32 values per lane over the 32 lanes of a warp, transposed: lane j returns the sum over
// all lanes of their v[j]. 31 shuffles instead of 32 x 5 (each step halves the values a lane holds).
__device__ __forceinline__ float warp_transpose_reduce(float (&v)[32], int lane) {
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        const bool up = (lane & off) != 0;
#pragma unroll
        for (int i = 0; i < off; ++i) {
            const float send = up ? v[i] : v[i + off];
            const float keep = up ? v[i + off] : v[i];
            v[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
        }
    }
    return v[0];
}

// Named barrier for a subset of the CTA's warps (id 1..15; id 0 is __syncthreads).
__device__ __forceinline__ void named_barrier(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// The same, returning to every participating thread whether any of them passed a true predicate.
__device__ __forceinline__ bool named_barrier_or(int id, int nthreads, bool pred) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 p, %3, 0;\n\t"
        "barrier.cta.red.or.pred q, %1, %2, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(out)
        : "r"(id), "r"(nthreads), "r"(static_cast<uint32_t>(pred))
        : "memory");
    return out != 0;
}

// Merge (max, sum-of-exp2) pairs: (M, S) <- (M, S) (+) (m, s), all in the log2 domain.
__device__ __forceinline__ void merge_ml(float& M, float& S, float m, float s) {
    const float nm = fmaxf(M, m);
    const float so = (M == __int_as_float(0xff800000)) ? 0.f : S * ex2_approx(M - nm);
    const float sn = (m == __int_as_float(0xff800000)) ? 0.f : s * ex2_approx(m - nm);
    M = nm;
    S = so + sn;
}

}  // namespace chunkkv
