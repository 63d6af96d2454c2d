// Top-k chunk selection and kept-index emission (ChunkKV Algorithm 3: "Top-K(chunk_scores, k)",
// the selection mask, "always keep most recent tokens", "nonzero(mask)").
//
// One CTA per KV head. The k-th largest score is found by an exact 4-pass radix select on
// order-preserving 32-bit keys; a single ordered sweep then keeps every chunk above the
// threshold plus the lowest-numbered chunks equal to it until k are kept, and writes their token
// positions directly in ascending order - no mask, no sort and no compaction of a mask.
#include "internal.h"

namespace chunkkv {

namespace {

constexpr int kSelThreads = 1024;

__device__ __forceinline__ uint32_t order_key(float x) {
    const uint32_t b = __float_as_uint(x + 0.0f);          // -0 and +0 compare equal
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);   // larger float <=> larger key
}

// Exclusive prefix sum of one int per thread across the CTA; also returns the CTA total.
// warp_sums must hold 33 ints. Ends with a barrier, so warp_sums can be reused at once.
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_sums, int* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, inc, off);
        if (lane >= off) inc += n;
    }
    if (lane == 31) warp_sums[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        const int s = warp_sums[lane];
        int sinc = s;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int n = __shfl_up_sync(0xffffffffu, sinc, off);
            if (lane >= off) sinc += n;
        }
        warp_sums[lane] = sinc - s;            // exclusive warp offsets
        if (lane == 31) warp_sums[32] = sinc;  // total
    }
    __syncthreads();
    const int res = warp_sums[warp] + inc - v;
    *total = warp_sums[32];
    __syncthreads();
    return res;
}

__global__ void __launch_bounds__(kSelThreads)
select_kernel(const float* __restrict__ scores, int L, int w, int c, int C, int k, int n_max,
              int32_t* __restrict__ out_idx) {
    __shared__ int hist[256];
    __shared__ int warp_sums[33];
    __shared__ uint32_t s_prefix;
    __shared__ int s_need;
    __shared__ int s_last_kept;
    const int h = blockIdx.x;
    const int P = L - w;
    const float* sc = scores + static_cast<size_t>(h) * C;
    int32_t* out = out_idx + static_cast<size_t>(h) * n_max;
    const int tid = threadIdx.x;

    if (tid == 0) s_last_kept = 0;
    uint32_t thresh = 0;   // key of the k-th largest score
    int need_eq = 0;       // how many chunks equal to the threshold are kept
    const bool keep_all = (k >= C);
    if (!keep_all && k > 0) {
        uint32_t prefix = 0;
        int need = k;
        for (int pass = 0; pass < 4; ++pass) {
            const int shift = 24 - 8 * pass;
            if (tid < 256) hist[tid] = 0;
            __syncthreads();
            const uint32_t himask = (pass == 0) ? 0u : (0xFFFFFFFFu << (shift + 8));
            for (int i = tid; i < C; i += blockDim.x) {
                const uint32_t key = order_key(sc[i]);
                if ((key & himask) == prefix) atomicAdd(&hist[(key >> shift) & 0xFF], 1);
            }
            __syncthreads();
            if (tid == 0) {
                int b = 255, above = 0;
                while (b > 0 && above + hist[b] < need) { above += hist[b]; --b; }
                s_prefix = prefix | (static_cast<uint32_t>(b) << shift);
                s_need = need - above;
            }
            __syncthreads();
            prefix = s_prefix;
            need = s_need;
        }
        thresh = prefix;
        need_eq = need;
    }
    __syncthreads();

    // Ordered sweep over chunk ids: running counts of kept chunks and of threshold ties.
    if (k > 0) {
        int kept_before = 0, eq_before = 0;
        for (int base = 0; base < C; base += blockDim.x) {
            const int ch = base + tid;
            bool gt = false, eq = false;
            if (ch < C) {
                if (keep_all) gt = true;
                else {
                    const uint32_t key = order_key(sc[ch]);
                    gt = key > thresh;
                    eq = key == thresh;
                }
            }
            int eq_total;
            const int eq_rank = eq_before + block_exclusive_scan(eq ? 1 : 0, warp_sums, &eq_total);
            const bool keep = gt || (eq && eq_rank < need_eq);
            int keep_total;
            const int rank = kept_before + block_exclusive_scan(keep ? 1 : 0, warp_sums, &keep_total);
            if (keep) {
                const int j0 = ch * c;
                const int len = min(c, P - j0);                        // only chunk C-1 can be short
                int32_t* dst = out + static_cast<size_t>(rank) * c;    // and it is the last one kept
                for (int t = 0; t < len; ++t) dst[t] = j0 + t;
                if (ch == C - 1) s_last_kept = 1;
            }
            kept_before += keep_total;
            eq_before += eq_total;
        }
    }
    __syncthreads();
    const int kk = min(k, C);
    const int tail = (C > 0) ? (P - (C - 1) * c) : 0;            // length of chunk C-1
    const int n_tok = kk * c - ((s_last_kept && kk > 0) ? (c - tail) : 0);
    for (int i = tid; i < w; i += blockDim.x) out[n_tok + i] = P + i;
    for (int i = n_tok + w + tid; i < n_max; i += blockDim.x) out[i] = -1;
}

}  // namespace

cudaError_t launch_select(const float* scores, int L, int Hkv, int w, int c, int C, int k, int n_max,
                          int32_t* out_idx, cudaStream_t stream) {
    select_kernel<<<Hkv, kSelThreads, 0, stream>>>(scores, L, w, c, C, k, n_max, out_idx);
    return cudaGetLastError();
}

}  // namespace chunkkv
