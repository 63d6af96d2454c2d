// Top-k chunk selection and kept-index emission (ChunkKV Algorithm 3: "Top-K(chunk_scores, k)",
// the selection mask, "always keep most recent tokens", "nonzero(mask)").
//
// One CTA per KV head. Each thread owns a contiguous run of chunk ids and keeps their
// order-preserving 32-bit keys in registers. The k-th largest key is found by an exact 4-pass
// radix select; every warp counts into its own 16-bit histogram row (lanes that hit the same
// bin add once), so no two warps ever touch the same counter. One block-wide prefix sum over
// (#above threshold, #equal to threshold) then gives every chunk its rank among the kept ones:
// rank = #above before it + min(#equal before it, ties to keep) - ties go to the lower chunk
// id. Token positions are written directly in ascending order: no mask, no sort.
#include "internal.h"

namespace chunkkv {

namespace {

constexpr int kSelThreads = 1024;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kPerThread = 8;                         // chunk keys held in registers per thread
constexpr int kRegCap = kSelThreads * kPerThread;     // more chunks than this are re-read from memory
constexpr int kSelCap = 4096;                         // kept-chunk ids staged for coalesced index writes

__device__ __forceinline__ uint32_t order_key(float x) {
    const uint32_t b = __float_as_uint(x + 0.0f);          // -0 and +0 compare equal
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);     // larger float <=> larger key
}

template <bool IN_REGS>
__global__ void __launch_bounds__(kSelThreads)
select_kernel(const float* __restrict__ scores, int L, int w, int c, int C, int k, int n_max,
              int32_t* __restrict__ out_idx) {
    __shared__ unsigned short whist[kSelWarps][256];
    __shared__ int sel_s[kSelCap];
    __shared__ int hist[256];
    __shared__ unsigned long long warp_sums[33];
    __shared__ uint32_t s_prefix;
    __shared__ int s_need;
    __shared__ int s_last_kept;
    const int h = blockIdx.x;
    const int P = L - w;
    const float* sc = scores + static_cast<size_t>(h) * C;
    int32_t* out = out_idx + static_cast<size_t>(h) * n_max;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool keep_all = (k >= C);
    const int kk = min(k, C);

    // thread t owns chunk ids [c0, c1)
    const int per = (C + kSelThreads - 1) / kSelThreads;
    const int c0 = min(tid * per, C), c1 = min(c0 + per, C);
    uint32_t keys[kPerThread];
    if (IN_REGS && kk > 0 && !keep_all) {
#pragma unroll
        for (int u = 0; u < kPerThread; ++u) keys[u] = (c0 + u < c1) ? order_key(sc[c0 + u]) : 0u;
    }
    if (tid == 0) s_last_kept = 0;

    uint32_t thresh = 0;   // key of the k-th largest score
    int need_eq = 0;       // how many chunks equal to the threshold are kept
    if (!keep_all && kk > 0) {
        uint32_t prefix = 0;
        int need = k;
        for (int pass = 0; pass < 4; ++pass) {
            const int shift = 24 - 8 * pass;
            {   // clear this warp's histogram row (256 x 16 bit = 128 words)
                uint32_t* row = reinterpret_cast<uint32_t*>(whist[warp]);
#pragma unroll
                for (int q = 0; q < 4; ++q) row[lane + 32 * q] = 0u;
            }
            __syncwarp();
            const uint32_t himask = (pass == 0) ? 0u : (0xFFFFFFFFu << (shift + 8));
            auto count_one = [&](bool have, uint32_t key) {
                const bool in = have && (key & himask) == prefix;
                const int bin = in ? static_cast<int>((key >> shift) & 0xFF) : -1;
                const unsigned peers = __match_any_sync(0xffffffffu, bin);
                if (in && lane == __ffs(peers) - 1) whist[warp][bin] += static_cast<unsigned short>(__popc(peers));
                __syncwarp();
            };
            if (IN_REGS) {
#pragma unroll
                for (int u = 0; u < kPerThread; ++u)
                    if (u < per) count_one(c0 + u < c1, keys[u]);      // `per` is uniform: no divergence
            } else {
                for (int u = 0; u < per; ++u) count_one(c0 + u < c1, (c0 + u < c1) ? order_key(sc[c0 + u]) : 0u);
            }
            __syncthreads();
            if (tid < 256) {
                int sum = 0;
#pragma unroll 8
                for (int wv = 0; wv < kSelWarps; ++wv) sum += whist[wv][tid];
                hist[tid] = sum;
            }
            __syncthreads();
            if (warp == 0) {
                // lane t owns bins 255-8t .. 248-8t (descending), so a prefix over lanes counts from the top
                int cnt[8], sum = 0;
#pragma unroll
                for (int q = 0; q < 8; ++q) { cnt[q] = hist[255 - 8 * lane - q]; sum += cnt[q]; }
                int inc = sum;
#pragma unroll
                for (int off = 1; off < 32; off <<= 1) {
                    const int n = __shfl_up_sync(0xffffffffu, inc, off);
                    if (lane >= off) inc += n;
                }
                const unsigned reach = __ballot_sync(0xffffffffu, inc >= need);
                const int owner = reach ? (__ffs(reach) - 1) : 31;
                if (lane == owner) {
                    int above = inc - sum, q = 0;
                    while (q < 7 && above + cnt[q] < need) { above += cnt[q]; ++q; }
                    s_prefix = prefix | (static_cast<uint32_t>(255 - 8 * lane - q) << shift);
                    s_need = need - above;
                }
            }
            __syncthreads();
            prefix = s_prefix;
            need = s_need;
        }
        thresh = prefix;
        need_eq = need;
    }

    // Ordered sweep over the chunk ids.
    const bool stage_sel = kk <= kSelCap;
    if (kk > 0) {
        unsigned gt_n = 0, eq_n = 0;
        if (keep_all) gt_n = c1 - c0;
        else if (IN_REGS) {
#pragma unroll
            for (int u = 0; u < kPerThread; ++u)
                if (c0 + u < c1) { gt_n += keys[u] > thresh; eq_n += keys[u] == thresh; }
        } else {
            for (int ch = c0; ch < c1; ++ch) {
                const uint32_t key = order_key(sc[ch]);
                gt_n += key > thresh;
                eq_n += key == thresh;
            }
        }
        // block-wide exclusive prefix of the packed pair (eq in the high half, gt in the low half)
        const unsigned long long mine = (static_cast<unsigned long long>(eq_n) << 32) | gt_n;
        unsigned long long inc = mine;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned long long n = __shfl_up_sync(0xffffffffu, inc, off);
            if (lane >= off) inc += n;
        }
        if (lane == 31) warp_sums[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            const unsigned long long s = warp_sums[lane];
            unsigned long long sinc = s;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const unsigned long long n = __shfl_up_sync(0xffffffffu, sinc, off);
                if (lane >= off) sinc += n;
            }
            warp_sums[lane] = sinc - s;
        }
        __syncthreads();
        const unsigned long long excl = warp_sums[warp] + inc - mine;
        int gt_before = static_cast<int>(excl & 0xffffffffu), eq_before = static_cast<int>(excl >> 32);
        auto visit = [&](int ch, uint32_t key) {
            const bool gt = keep_all || key > thresh;
            const bool eq = !keep_all && key == thresh;
            if (gt || (eq && eq_before < need_eq)) {
                const int rank = gt_before + min(eq_before, need_eq);
                if (stage_sel) sel_s[rank] = ch;
                else {
                    const int j0 = ch * c, len = min(c, P - j0);
                    int32_t* dst = out + static_cast<size_t>(rank) * c;
                    for (int t = 0; t < len; ++t) dst[t] = j0 + t;
                }
                if (ch == C - 1) s_last_kept = 1;
            }
            gt_before += gt;
            eq_before += eq;
        };
        if (IN_REGS && !keep_all) {
#pragma unroll
            for (int u = 0; u < kPerThread; ++u)
                if (c0 + u < c1) visit(c0 + u, keys[u]);
        } else {
            for (int ch = c0; ch < c1; ++ch) visit(ch, keep_all ? 0u : order_key(sc[ch]));
        }
    }
    __syncthreads();
    // Every kept chunk is full except possibly chunk C-1, which can only be the last kept one.
    const int tail = (C > 0) ? (P - (C - 1) * c) : 0;
    const int n_tok = kk * c - ((s_last_kept && kk > 0) ? (c - tail) : 0);
    if (stage_sel)
        for (int n = tid; n < n_tok; n += kSelThreads) {
            const int rank = n / c;
            out[n] = sel_s[rank] * c + (n - rank * c);
        }
    for (int i = tid; i < w; i += kSelThreads) out[n_tok + i] = P + i;
    for (int i = n_tok + w + tid; i < n_max; i += kSelThreads) out[i] = -1;
}

}  // namespace

cudaError_t launch_select(const float* scores, int L, int Hkv, int w, int c, int C, int k, int n_max,
                          int32_t* out_idx, cudaStream_t stream) {
    if (C <= kRegCap)
        select_kernel<true><<<Hkv, kSelThreads, 0, stream>>>(scores, L, w, c, C, k, n_max, out_idx);
    else
        select_kernel<false><<<Hkv, kSelThreads, 0, stream>>>(scores, L, w, c, C, k, n_max, out_idx);
    return cudaGetLastError();
}

}  // namespace chunkkv
