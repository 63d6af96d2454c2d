// Top-k chunk selection for heads with thousands of chunks (token-level layers, long contexts),
// ChunkKV Algorithm 3 "Top-K(chunk_scores, k)" and the ordered "nonzero(mask)": the same exact
// adaptive radix select as select.cuh, spread over a thread-block cluster of eight CTAs per KV
// head. A CTA keeps an eighth of the head's keys in registers; histograms, candidate keys and
// counts travel between the CTAs through distributed shared memory and cluster barriers (hardware
// barriers among co-scheduled CTAs: no spin-waits). Results are identical to the one-CTA kernels:
// the k-th largest key is found exactly, ties go to the lower chunk id, positions are ascending.
#include "internal.h"
#include "select.cuh"

#include <cooperative_groups.h>

namespace cg = cooperative_groups;

namespace chunkkv {

namespace {

constexpr int kCsCtas = 8;            // CTAs per cluster (the portable maximum)
constexpr int kCsKpt = 8;             // keys per thread
constexpr int kCsBinsPerCta = kSelBins / kCsCtas;

struct ClusterSel {
    int hist[kSelBins];
    uint32_t cand[kSelCandCap];
    unsigned long long minmax[kCsCtas];     // written by every CTA of the cluster
    int slice_tot[kCsCtas];                 // keys in a CTA's 256 bins (all CTAs' histograms added)
    unsigned long long cta_cnt[kCsCtas];    // (#equal << 32 | #above) per CTA
    unsigned long long warp_sums[33];
    int warp_tot[32];
    int n_cand;
    uint32_t bin;
    int need;
    int bin_count;
    uint32_t thresh;
    int need_eq;
    int last_kept;
};

// kCsThreads = 512 (every thread may use 128 registers: no spills) or 1024 (twice the keys per cluster)
template <int kCsThreads>
__global__ void __cluster_dims__(kCsCtas, 1, 1) __launch_bounds__(kCsThreads, 1)
select_cluster_kernel(const float* __restrict__ scores, int L, int w, int c, int C, int k, int n_max,
                      int32_t* __restrict__ out_idx, int tok_cap) {
    constexpr unsigned kFull = 0xffffffffu;
    __shared__ ClusterSel cs;
    cg::cluster_group cluster = cg::this_cluster();
    const int r = static_cast<int>(cluster.block_rank());
    const int h = blockIdx.x / kCsCtas;
    const float* sc = scores + static_cast<size_t>(h) * C;
    int32_t* out = out_idx + static_cast<size_t>(h) * n_max;
    const int P = L - w;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int nwarps = kCsThreads / 32;

    // CTA r owns chunk ids [r S, (r + 1) S); thread t of it a contiguous run of at most kCsKpt ids
    const int S = (C + kCsCtas - 1) / kCsCtas;
    const int s0 = min(r * S, C), s1 = min(s0 + S, C);
    const int per = (S + kCsThreads - 1) / kCsThreads;
    const int c0 = min(s0 + tid * per, s1), c1 = min(c0 + per, s1);
    uint32_t keys[kCsKpt];
#pragma unroll
    for (int u = 0; u < kCsKpt; ++u) keys[u] = (c0 + u < c1) ? select_order_key(__ldcg(sc + c0 + u)) : 0u;

    // ---- smallest and largest key of the head
    uint32_t lo = 0xffffffffu, hi = 0u;
#pragma unroll
    for (int u = 0; u < kCsKpt; ++u)
        if (c0 + u < c1) { lo = min(lo, keys[u]); hi = max(hi, keys[u]); }
    lo = __reduce_min_sync(kFull, lo);
    hi = __reduce_max_sync(kFull, hi);
    if (lane == 0) cs.warp_sums[warp] = (static_cast<unsigned long long>(hi) << 32) | lo;
    for (int i = tid; i < kSelBins; i += kCsThreads) cs.hist[i] = 0;
    if (tid == 0) { cs.n_cand = 0; cs.last_kept = 0; }
    __syncthreads();
    if (warp == 0) {
        const unsigned long long v = (lane < nwarps) ? cs.warp_sums[lane] : 0x00000000ffffffffull;
        uint32_t l2 = __reduce_min_sync(kFull, static_cast<uint32_t>(v));
        uint32_t h2 = __reduce_max_sync(kFull, static_cast<uint32_t>(v >> 32));
        if (lane < kCsCtas) *cluster.map_shared_rank(&cs.minmax[r], lane) = (static_cast<unsigned long long>(h2) << 32) | l2;
    }
    cluster.sync();
    uint32_t base = 0xffffffffu, top = 0u;
#pragma unroll
    for (int q = 0; q < kCsCtas; ++q) {
        const unsigned long long v = cs.minmax[q];
        base = min(base, static_cast<uint32_t>(v));
        top = max(top, static_cast<uint32_t>(v >> 32));
    }
    uint32_t span = top - base;          // the keys of interest lie in [base, base + span]
    int need = k;                        // the need-th largest of them is the threshold
    uint32_t thresh = 0;
    int need_eq = 0;
    for (int round = 0;; ++round) {
        if (span == 0u) { thresh = base; need_eq = need; break; }
        const int shift = max(0, 21 - __clz(span));      // (span >> shift) < kSelBins
        if (round > 0) {
            // every CTA has read this histogram (the cluster barriers of the previous round lie behind)
            for (int i = tid; i < kSelBins; i += kCsThreads) cs.hist[i] = 0;
            __syncthreads();
        }
#pragma unroll
        for (int u = 0; u < kCsKpt; ++u) {
            const uint32_t dlt = keys[u] - base;
            if (c0 + u < c1 && keys[u] >= base && dlt <= span) atomicAdd(&cs.hist[dlt >> shift], 1);
        }
        cluster.sync();
        // CTA r adds up bins [256 r, 256 r + 256) of the eight histograms; thread t < 256 takes bin
        // 256 r + 255 - t, so a prefix over the threads counts from the top of the slice
        int tot = 0;
        if (tid < kCsBinsPerCta) {
            const int b = kCsBinsPerCta * r + kCsBinsPerCta - 1 - tid;
#pragma unroll
            for (int q = 0; q < kCsCtas; ++q) tot += *cluster.map_shared_rank(&cs.hist[b], q);
        }
        int inc = tot;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int n = __shfl_up_sync(kFull, inc, off);
            if (lane >= off) inc += n;
        }
        if (lane == 31) cs.warp_tot[warp] = inc;
        __syncthreads();
        int before = 0;
        for (int wv = 0; wv < warp && wv < kCsBinsPerCta / 32; ++wv) before += cs.warp_tot[wv];
        inc += before;
        if (tid == kCsBinsPerCta - 1) {
#pragma unroll
            for (int q = 0; q < kCsCtas; ++q) *cluster.map_shared_rank(&cs.slice_tot[r], q) = inc;
        }
        cluster.sync();
        int above = 0;                   // keys in the bins above this CTA's slice
        for (int q = r + 1; q < kCsCtas; ++q) above += cs.slice_tot[q];
        if (tid < kCsBinsPerCta && above + inc - tot < need && need <= above + inc) {     // exactly one thread of the cluster
            const uint32_t b = static_cast<uint32_t>(kCsBinsPerCta * r + kCsBinsPerCta - 1 - tid);
            const int nd = need - (above + inc - tot);
#pragma unroll
            for (int q = 0; q < kCsCtas; ++q) {
                *cluster.map_shared_rank(&cs.bin, q) = b;
                *cluster.map_shared_rank(&cs.need, q) = nd;
                *cluster.map_shared_rank(&cs.bin_count, q) = tot;
            }
        }
        cluster.sync();
        const uint32_t bin = cs.bin;
        const int n_bin = cs.bin_count;
        need = cs.need;
        const uint32_t sub = bin << shift;
        const uint32_t width = (shift >= 32) ? 0xffffffffu : ((1u << shift) - 1u);
        base += sub;
        span = min(width, span - sub);
        if (n_bin <= kSelCandCap) {
            // few keys left: gather them in CTA 0, then every CTA ranks its own copy of them
            ClusterSel* lead = cluster.map_shared_rank(&cs, 0);
#pragma unroll
            for (int u = 0; u < kCsKpt; ++u) {
                const uint32_t dlt = keys[u] - base;
                if (c0 + u < c1 && keys[u] >= base && dlt <= span) lead->cand[atomicAdd(&lead->n_cand, 1)] = keys[u];
            }
            cluster.sync();
            if (r != 0)
                for (int j = tid; j < n_bin; j += kCsThreads) cs.cand[j] = lead->cand[j];
            __syncthreads();
            for (int j = tid; j < n_bin; j += kCsThreads) {
                const uint32_t v = cs.cand[j];
                int gt = 0, ge = 0;
                for (int i = 0; i < n_bin; ++i) { gt += cs.cand[i] > v; ge += cs.cand[i] >= v; }
                if (gt < need && need <= ge) { cs.thresh = v; cs.need_eq = need - gt; }   // same values from every writer
            }
            __syncthreads();
            thresh = cs.thresh;
            need_eq = cs.need_eq;
            break;
        }
    }

    // ---- ordered sweep over the chunk ids
    unsigned gt_n = 0, eq_n = 0;
#pragma unroll
    for (int u = 0; u < kCsKpt; ++u)
        if (c0 + u < c1) { gt_n += keys[u] > thresh; eq_n += keys[u] == thresh; }
    const unsigned long long mine = (static_cast<unsigned long long>(eq_n) << 32) | gt_n;
    unsigned long long inc = mine;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const unsigned long long n = __shfl_up_sync(kFull, inc, off);
        if (lane >= off) inc += n;
    }
    __syncthreads();                      // warp_sums was read above (first round) by warp 0 only; be safe
    if (lane == 31) cs.warp_sums[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        const unsigned long long s = (lane < nwarps) ? cs.warp_sums[lane] : 0ull;
        unsigned long long sinc = s;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned long long n = __shfl_up_sync(kFull, sinc, off);
            if (lane >= off) sinc += n;
        }
        cs.warp_sums[lane] = sinc - s;
        const unsigned long long total = __shfl_sync(kFull, sinc, 31);
        if (lane < kCsCtas) *cluster.map_shared_rank(&cs.cta_cnt[r], lane) = total;
    }
    cluster.sync();                       // (also the CTA-wide barrier for warp_sums)
    unsigned long long excl = cs.warp_sums[warp] + inc - mine;
    for (int q = 0; q < r; ++q) excl += cs.cta_cnt[q];
    int gt_before = static_cast<int>(excl & 0xffffffffu), eq_before = static_cast<int>(excl >> 32);
#pragma unroll
    for (int u = 0; u < kCsKpt; ++u) {
        if (c0 + u < c1) {
            const int ch = c0 + u;
            const bool gt = keys[u] > thresh, eq = keys[u] == thresh;
            if (gt || (eq && eq_before < need_eq)) {
                const int rank = gt_before + min(eq_before, need_eq);
                const int j0 = ch * c, len = min(c, P - j0);
                int32_t* dst = out + static_cast<size_t>(rank) * c;
                for (int t = 0; t < len; ++t)
                    if (rank * c + t < tok_cap) dst[t] = j0 + t;
                if (ch == C - 1) cs.last_kept = 1;
            }
            gt_before += gt;
            eq_before += eq;
        }
    }
    // the CTA that owns the last chunk writes the window positions and the padding: every kept chunk
    // is full except possibly chunk C - 1, which can only be the last kept one
    if (r == (C - 1) / S) {
        __syncthreads();
        const int tail = P - (C - 1) * c;
        const int n_tok = min(k * c - (cs.last_kept ? (c - tail) : 0), tok_cap);
        for (int i = tid; i < w; i += kCsThreads) out[n_tok + i] = P + i;
        for (int i = n_tok + w + tid; i < n_max; i += kCsThreads) out[i] = -1;
    }
}

}  // namespace

bool select_cluster_applies(int C, int k) {
    return C > 4096 && C <= kCsCtas * 1024 * kCsKpt && k > 0 && k < C;
}

cudaError_t launch_select_cluster(const float* scores, int L, int Hkv, int w, int c, int C, int k, int n_max,
                                  int32_t* out_idx, cudaStream_t stream, int tok_cap) {
    if (C <= kCsCtas * 512 * kCsKpt)
        select_cluster_kernel<512><<<Hkv * kCsCtas, 512, 0, stream>>>(scores, L, w, c, C, k, n_max, out_idx, tok_cap);
    else
        select_cluster_kernel<1024><<<Hkv * kCsCtas, 1024, 0, stream>>>(scores, L, w, c, C, k, n_max, out_idx, tok_cap);
    return cudaGetLastError();
}

}  // namespace chunkkv
