// Device-side body of the K/V row gather (ChunkKV Algorithm 3 "index_select(K, indices)" /
// "index_select(V, indices)"), shared by the stand-alone gather kernel and the fused layer kernel.
//
// Rows are d bf16 = 128 or 256 bytes. Each thread moves 16 bytes of a row; a row is covered by
// d/8 adjacent threads, so every warp request is a set of fully used 128-byte lines. Each
// thread handles kGatherRowsPerThread rows of K and of V with all loads issued before the stores.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace chunkkv {

constexpr int kGatherRowsPerThread = 4;

// Rows are read once: no L1 allocation, first in line for eviction from L2.
__device__ __forceinline__ unsigned long long gather_policy() {
    unsigned long long p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint4 gather_ld(const uint4* p, unsigned long long policy) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.u32 {%0, %1, %2, %3}, [%4], %5;"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p), "l"(policy));
    return v;
}
__device__ __forceinline__ void gather_st(uint4* p, const uint4& v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z),
                 "r"(v.w)
                 : "memory");
}

// Destination rows in a paged cache [num_pages, page_size, Hkv, d]: compacted position n of head h goes to
// page block_table[n / page_size], slot n % page_size; pages outside [0, num_pages) are skipped.
// block_table == nullptr: packed outputs.
struct PagedDst {
    const int32_t* block_table;
    int page_size, num_pages, Hkv, h;
};

// Work item `item` of `n_items` (a CTA-sized slab of rows of one head); threads = nthreads
// (a multiple of VPR). VPR = 16-byte vectors per row: 8 (d = 64) or 16 (d = 128).
// FRESH_IDX: the indices were written earlier in the same kernel launch, so they must not be
// read through the non-coherent path. k_row_vecs / v_row_vecs: 16-byte vectors between consecutive
// source rows of a head (VPR for packed rows; more for a token-major cache).
template <int VPR, bool FRESH_IDX>
__device__ __forceinline__ void gather_rows(const uint4* __restrict__ Kh, const uint4* __restrict__ Vh,
                                            const int32_t* ih, int L, int n_max, int n0, int tid, int nthreads,
                                            uint4* __restrict__ oK, uint4* __restrict__ oV, int32_t* idx_copy,
                                            long long k_row_vecs = VPR, long long v_row_vecs = VPR,
                                            PagedDst pg = PagedDst{nullptr, 0, 0, 0, 0}) {
    const int rows_per_pass = nthreads / VPR;
    const int vec = tid % VPR, sub = tid / VPR;
    const unsigned long long policy = gather_policy();
    int src[kGatherRowsPerThread];
    uint4 kv[kGatherRowsPerThread], vv[kGatherRowsPerThread];
#pragma unroll
    for (int u = 0; u < kGatherRowsPerThread; ++u) {
        const int n = n0 + u * rows_per_pass + sub;
        if (n < n_max) src[u] = FRESH_IDX ? __ldcg(ih + n) : ih[n];
        else src[u] = -1;
    }
#pragma unroll
    for (int u = 0; u < kGatherRowsPerThread; ++u) {
        const bool ok = static_cast<unsigned>(src[u]) < static_cast<unsigned>(L);
        kv[u] = ok ? gather_ld(Kh + static_cast<size_t>(src[u]) * k_row_vecs + vec, policy) : make_uint4(0, 0, 0, 0);
        vv[u] = ok ? gather_ld(Vh + static_cast<size_t>(src[u]) * v_row_vecs + vec, policy) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int u = 0; u < kGatherRowsPerThread; ++u) {
        const int n = n0 + u * rows_per_pass + sub;
        if (n < n_max) {
            if (pg.block_table == nullptr) {
                gather_st(oK + static_cast<size_t>(n) * VPR + vec, kv[u]);
                gather_st(oV + static_cast<size_t>(n) * VPR + vec, vv[u]);
            } else {                                    // (oK / oV are the bases of the paged caches)
                const int page = pg.block_table[n / pg.page_size];
                if (static_cast<unsigned>(page) < static_cast<unsigned>(pg.num_pages)) {
                    const size_t row = (static_cast<size_t>(page) * pg.page_size + n % pg.page_size) * pg.Hkv + pg.h;
                    gather_st(oK + row * VPR + vec, kv[u]);
                    gather_st(oV + row * VPR + vec, vv[u]);
                }
            }
            if (idx_copy != nullptr && vec == 0) idx_copy[n] = src[u];
        }
    }
}

}  // namespace chunkkv
