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
constexpr int kCsCandCap = 512;       // at most this many keys are ranked against each other directly

struct ClusterSel {
    alignas(16) int hist[kSelBins];
    uint32_t cand[kCsCandCap];
    unsigned long long minmax[kCsCtas];     // written by every CTA of the cluster
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
    // (launched as a programmatic dependent of the kernel that wrote the scores)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
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
            for (int i = tid; i < kSelBins; i += kCsThreads) cs.hist[i] = 0;
            __syncthreads();
        }
#pragma unroll
        for (int u = 0; u < kCsKpt; ++u) {
            const uint32_t dlt = keys[u] - base;
            if (c0 + u < c1 && keys[u] >= base && dlt <= span) atomicAdd(&cs.hist[dlt >> shift], 1);
        }
        cluster.sync();
        // every CTA adds up the eight histograms itself (thread t < 512 takes bins 2047 - 4t .. 2044 - 4t,
        // so a prefix over the threads counts from the top) and finds the bin of the need-th largest
        // key on its own: same answer everywhere, no further exchange
        int cnt[4] = {0, 0, 0, 0}, sum = 0;
        if (tid < kSelBins / 4) {
#pragma unroll
            for (int q = 0; q < kCsCtas; ++q) {
                const int4 v = *reinterpret_cast<const int4*>(cluster.map_shared_rank(&cs.hist[kSelBins - 4 - 4 * tid], q));
                cnt[0] += v.w; cnt[1] += v.z; cnt[2] += v.y; cnt[3] += v.x;
            }
            sum = (cnt[0] + cnt[1]) + (cnt[2] + cnt[3]);
        }
        int inc = sum;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int n = __shfl_up_sync(kFull, inc, off);
            if (lane >= off) inc += n;
        }
        if (lane == 31) cs.warp_tot[warp] = inc;
        __syncthreads();
        int before = 0;
        for (int wv = 0; wv < warp; ++wv) before += cs.warp_tot[wv];
        inc += before;
        if (tid < kSelBins / 4 && inc - sum < need && need <= inc) {     // exactly one thread of the CTA
            int above = inc - sum, q = 0, cq = cnt[0];
#pragma unroll
            for (int t = 0; t < 3; ++t)          // (unrolled: cnt stays in registers)
                if (q == t && above + cnt[t] < need) { above += cnt[t]; q = t + 1; cq = cnt[t + 1]; }
            cs.bin = static_cast<uint32_t>(kSelBins - 1 - 4 * tid - q);
            cs.need = need - above;
            cs.bin_count = cq;
        }
        __syncthreads();
        const uint32_t bin = cs.bin;
        const int n_bin = cs.bin_count;
        need = cs.need;
        const uint32_t sub = bin << shift;
        const uint32_t width = (shift >= 32) ? 0xffffffffu : ((1u << shift) - 1u);
        base += sub;
        span = min(width, span - sub);
        if (n_bin <= kCsCandCap) {
            // few keys left: every CTA gets a copy of all of them (positions handed out by a counter in
            // CTA 0)
            int* lead_count = cluster.map_shared_rank(&cs.n_cand, 0);
#pragma unroll
            for (int u = 0; u < kCsKpt; ++u) {
                const uint32_t dlt = keys[u] - base;
                if (c0 + u < c1 && keys[u] >= base && dlt <= span) {
                    const int pos = atomicAdd(lead_count, 1);
#pragma unroll
                    for (int q = 0; q < kCsCtas; ++q) *cluster.map_shared_rank(&cs.cand[pos], q) = keys[u];
                }
            }
            cluster.sync();
            // the CTAs share the candidates out; a warp per candidate, its lanes striding over the others.
            // The warp that holds the need-th largest tells every CTA.
            for (int j = r + kCsCtas * warp; j < n_bin; j += kCsCtas * nwarps) {
                const uint32_t v = cs.cand[j];
                int gt = 0, ge = 0;
                for (int i = lane; i < n_bin; i += 32) {
                    const uint32_t x = cs.cand[i];
                    gt += x > v;
                    ge += x >= v;
                }
                gt = __reduce_add_sync(kFull, gt);
                ge = __reduce_add_sync(kFull, ge);
                if (lane < kCsCtas && gt < need && need <= ge) {       // (same values from every writer)
                    *cluster.map_shared_rank(&cs.thresh, lane) = v;
                    *cluster.map_shared_rank(&cs.need_eq, lane) = need - gt;
                }
            }
            cluster.sync();
            thresh = cs.thresh;
            need_eq = cs.need_eq;
            break;
        }
        cluster.sync();      // another round: every CTA has read this histogram before it is cleared
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
    const bool small = C <= kCsCtas * 512 * kCsKpt;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(Hkv * kCsCtas);
    cfg.blockDim = dim3(small ? 512 : 1024);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (small) return cudaLaunchKernelEx(&cfg, select_cluster_kernel<512>, scores, L, w, c, C, k, n_max, out_idx, tok_cap);
    return cudaLaunchKernelEx(&cfg, select_cluster_kernel<1024>, scores, L, w, c, C, k, n_max, out_idx, tok_cap);
}

}  // namespace chunkkv
