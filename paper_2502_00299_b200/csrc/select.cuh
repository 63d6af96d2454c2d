// Device-side body of the top-k chunk selection (ChunkKV Algorithm 3: "Top-K(chunk_scores, k)",
// the selection mask, "always keep most recent tokens", "nonzero(mask)"), shared by the
// stand-alone select kernel and the fused layer kernel.
//
// One CTA works on one KV head. Each thread owns a contiguous run of chunk ids and keeps their
// order-preserving 32-bit keys in registers. The k-th largest key is found by an exact 4-pass
// radix select; every warp counts into its own 16-bit histogram row (lanes that hit the same
// bin add once), so no two warps ever touch the same counter. One block-wide prefix sum over
// (#above threshold, #equal to threshold) then gives every chunk its rank among the kept ones:
// rank = #above before it + min(#equal before it, ties to keep) - ties go to the lower chunk
// id. Token positions are written directly in ascending order: no mask, no sort.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace chunkkv {

constexpr int kSelMaxWarps = 32;
constexpr int kSelPerThread = 16;     // chunk keys per thread of the usual register variant
constexpr int kSelPerThreadMax = 64;  // the largest register variant (token-level selection: tens of thousands of keys per head)
constexpr int kSelCap = 4096;         // kept-chunk ids staged for coalesced index writes

struct SelectSmem {
    unsigned short whist[kSelMaxWarps][256];
    int sel[kSelCap];
    int hist[256];
    unsigned long long warp_sums[kSelMaxWarps + 1];
    uint32_t prefix;
    int need;
    int last_kept;
};

__device__ __forceinline__ uint32_t select_order_key(float x) {
    const uint32_t b = __float_as_uint(x + 0.0f);          // -0 and +0 compare equal
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);     // larger float <=> larger key
}

// All threads of the CTA must call this (it uses __syncthreads); blockDim.x must be a multiple
// of 32 and at most 1024. KPT > 0: every thread keeps up to KPT keys in registers, which needs
// C <= blockDim.x * KPT; KPT = 0: keys are re-read from memory on every use.
// sc2 != NULL: the head's scores are sc[ch] + sc2[ch] (a KV head scored as two heads of half the rows).
template <int KPT>
__device__ __forceinline__ void select_head(const float* __restrict__ sc, const float* __restrict__ sc2, int L, int w, int c,
                                            int C, int k, int n_max, int32_t* __restrict__ out, SelectSmem& sm) {
    auto score_at = [&](int ch) { return sc2 != nullptr ? sc[ch] + sc2[ch] : sc[ch]; };
    const int P = L - w;
    const int nt = blockDim.x, nwarps = nt >> 5;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool keep_all = (k >= C);
    const int kk = min(k, C);

    // thread t owns chunk ids [c0, c1)
    const int per = (C + nt - 1) / nt;
    const int c0 = min(tid * per, C), c1 = min(c0 + per, C);
    constexpr bool IN_REGS = KPT > 0;
    constexpr int KR = IN_REGS ? KPT : 1;
    uint32_t keys[KR];
    if (IN_REGS && kk > 0 && !keep_all) {
#pragma unroll
        for (int u = 0; u < KR; ++u) keys[u] = (c0 + u < c1) ? select_order_key(score_at(c0 + u)) : 0u;
    }
    if (tid == 0) sm.last_kept = 0;

    uint32_t thresh = 0;   // key of the k-th largest score
    int need_eq = 0;       // how many chunks equal to the threshold are kept
    if (!keep_all && kk > 0) {
        uint32_t prefix = 0;
        int need = k;
        for (int pass = 0; pass < 4; ++pass) {
            const int shift = 24 - 8 * pass;
            // Pass 0 sees the sign and exponent bits, which are nearly the same for all scores:
            // lanes that hit the same bin are grouped with a match and add once to the warp's own
            // histogram row. Later passes see spread-out digits of the few keys that still carry
            // the prefix: there one atomic add per key into the shared histogram is cheaper.
            const bool grouped = (pass == 0);
            if (grouped) {   // clear this warp's histogram row (256 x 16 bit = 128 words)
                uint32_t* row = reinterpret_cast<uint32_t*>(sm.whist[warp]);
#pragma unroll
                for (int q = 0; q < 4; ++q) row[lane + 32 * q] = 0u;
                __syncwarp();
            } else {
                if (tid < 256) sm.hist[tid] = 0;
                __syncthreads();
            }
            const uint32_t himask = (pass == 0) ? 0u : (0xFFFFFFFFu << (shift + 8));
            auto count_one = [&](bool have, uint32_t key) {
                const bool in = have && (key & himask) == prefix;
                const int bin = in ? static_cast<int>((key >> shift) & 0xFF) : -1;
                if (grouped) {
                    const unsigned peers = __match_any_sync(0xffffffffu, bin);
                    if (in && lane == __ffs(peers) - 1)
                        sm.whist[warp][bin] += static_cast<unsigned short>(__popc(peers));
                    __syncwarp();
                } else if (in) {
                    atomicAdd(&sm.hist[bin], 1);
                }
            };
            if (IN_REGS) {
#pragma unroll
                for (int u = 0; u < KR; ++u)
                    if (u < per) count_one(c0 + u < c1, keys[u]);      // `per` is uniform: no divergence
            } else {
                for (int u = 0; u < per; ++u)
                    count_one(c0 + u < c1, (c0 + u < c1) ? select_order_key(score_at(c0 + u)) : 0u);
            }
            __syncthreads();
            if (grouped) {
                if (tid < 256) {
                    int sum = 0;
                    for (int wv = 0; wv < nwarps; ++wv) sum += sm.whist[wv][tid];
                    sm.hist[tid] = sum;
                }
                __syncthreads();
            }
            if (warp == 0) {
                // lane t owns bins 255-8t .. 248-8t (descending), so a prefix over lanes counts from the top
                int cnt[8], sum = 0;
#pragma unroll
                for (int q = 0; q < 8; ++q) { cnt[q] = sm.hist[255 - 8 * lane - q]; sum += cnt[q]; }
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
                    sm.prefix = prefix | (static_cast<uint32_t>(255 - 8 * lane - q) << shift);
                    sm.need = need - above;
                }
            }
            __syncthreads();
            prefix = sm.prefix;
            need = sm.need;
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
            for (int u = 0; u < KR; ++u)
                if (c0 + u < c1) { gt_n += keys[u] > thresh; eq_n += keys[u] == thresh; }
        } else {
            for (int ch = c0; ch < c1; ++ch) {
                const uint32_t key = select_order_key(score_at(ch));
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
        if (lane == 31) sm.warp_sums[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            const unsigned long long s = (lane < nwarps) ? sm.warp_sums[lane] : 0ull;
            unsigned long long sinc = s;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const unsigned long long n = __shfl_up_sync(0xffffffffu, sinc, off);
                if (lane >= off) sinc += n;
            }
            sm.warp_sums[lane] = sinc - s;
        }
        __syncthreads();
        const unsigned long long excl = sm.warp_sums[warp] + inc - mine;
        int gt_before = static_cast<int>(excl & 0xffffffffu), eq_before = static_cast<int>(excl >> 32);
        auto visit = [&](int ch, uint32_t key) {
            const bool gt = keep_all || key > thresh;
            const bool eq = !keep_all && key == thresh;
            if (gt || (eq && eq_before < need_eq)) {
                const int rank = gt_before + min(eq_before, need_eq);
                if (stage_sel) sm.sel[rank] = ch;
                else {
                    const int j0 = ch * c, len = min(c, P - j0);
                    int32_t* dst = out + static_cast<size_t>(rank) * c;
                    for (int t = 0; t < len; ++t) dst[t] = j0 + t;
                }
                if (ch == C - 1) sm.last_kept = 1;
            }
            gt_before += gt;
            eq_before += eq;
        };
        if (IN_REGS && !keep_all) {
#pragma unroll
            for (int u = 0; u < KR; ++u)
                if (c0 + u < c1) visit(c0 + u, keys[u]);
        } else {
            for (int ch = c0; ch < c1; ++ch) visit(ch, keep_all ? 0u : select_order_key(score_at(ch)));
        }
    }
    __syncthreads();
    // Every kept chunk is full except possibly chunk C-1, which can only be the last kept one.
    const int tail = (C > 0) ? (P - (C - 1) * c) : 0;
    const int n_tok = kk * c - ((sm.last_kept && kk > 0) ? (c - tail) : 0);
    if (stage_sel)
        for (int n = tid; n < n_tok; n += nt) {
            const int rank = n / c;
            out[n] = sm.sel[rank] * c + (n - rank * c);
        }
    for (int i = tid; i < w; i += nt) out[n_tok + i] = P + i;
    for (int i = n_tok + w + tid; i < n_max; i += nt) out[i] = -1;
    __syncthreads();     // shared state may be reused by the caller
}

}  // namespace chunkkv
