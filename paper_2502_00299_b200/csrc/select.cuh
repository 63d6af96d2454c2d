// Device-side bodies of the top-k chunk selection (ChunkKV Algorithm 3: "Top-K(chunk_scores, k)",
// the selection mask, "always keep most recent tokens", "nonzero(mask)"), shared by the
// stand-alone select kernel and the fused layer kernel. One CTA works on one KV head.
//
// Both bodies find the k-th largest of the order-preserving 32-bit keys exactly and then rank
// every chunk among the kept ones: rank = #above before it + min(#equal before it, ties to keep) -
// ties go to the lower chunk id. Token positions are written directly in ascending order: no
// mask, no sort.
//
// select_head_regs (a few chunks per thread): each thread owns a contiguous run of chunk ids and
// keeps their keys in registers; the threshold comes from an adaptive radix select (2048 equal
// sub-intervals of [min key, max key], repeated on the sub-interval that holds the k-th largest
// until few enough keys remain to rank directly). One block-wide prefix sum over the threads'
// (#above, #equal) gives the ranks.
//
// select_head_rows (many chunks per thread, e.g. token-level selection of tens of thousands of
// keys): unrolled code over registers would spill and spend its time fetching instructions that
// run once, so this body is short rolled loops over a key buffer (shared memory where it fits).
// Each warp owns a contiguous block of chunk ids and walks it in rows of 32 consecutive ids, one
// per lane: accesses are coalesced and the order inside a row is the lane order. In the first
// pass every lane counts the four bins around the warp's first key in registers and the warp
// adds its totals once; any other bin, and every bin of the later passes, takes one
// shared-memory atomic per key. Ranks come from warp ballots plus one block-wide prefix sum
// over the warps' (#above, #equal) totals.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace chunkkv {

constexpr int kSelMaxWarps = 32;
constexpr int kSelCap = 4096;         // kept-chunk ids staged for coalesced index writes

struct SelectSmem {
    unsigned short whist[kSelMaxWarps][256];
    int sel[kSelCap];
    int hist[256];
    unsigned long long warp_sums[kSelMaxWarps + 1];
    int warp_tot[kSelMaxWarps];
    uint32_t prefix;
    int need;
    int bin_count;
    int n_cand;
    int last_kept;
};

__device__ __forceinline__ uint32_t select_order_key(float x) {
    const uint32_t b = __float_as_uint(x + 0.0f);          // -0 and +0 compare equal
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);     // larger float <=> larger key
}

// Selection for a few chunks per thread. All threads of the CTA must call this (it uses
// __syncthreads); blockDim.x must be a multiple of 32, at least 512 and at most 1024. Every thread
// keeps up to KPT keys in registers, which needs C <= blockDim.x * KPT.
// sc2 != NULL: the head's scores are sc[ch] + sc2[ch] (a KV head scored as two heads of half the rows).
//
// The k-th largest key is found by an adaptive radix select: the keys of interest always lie in a
// known interval [base, base + span]; one round histograms them into 2048 equal sub-intervals,
// finds the sub-interval that holds the k-th largest and makes it the new interval. Chunk scores
// of one head sit in a narrow band of the float range, so the first round (over [min, max] of the
// keys) already leaves a handful of candidates; as soon as at most kSelCandCap keys remain they are
// ranked against each other directly. Ties and degenerate inputs (all keys equal) end with
// span = 0, i.e. a single key value. Exact for any input.
constexpr int kSelBins = 2048;
constexpr int kSelCandCap = 1024;

template <int KPT>
__device__ __forceinline__ void select_head_regs(const float* sc, const float* sc2, int L, int w, int c,
                                            int C, int k, int n_max, int32_t* out, SelectSmem& sm,
                                            int tok_cap = 0x7fffffff) {
    static_assert(KPT > 0, "keys live in registers");
    constexpr unsigned kFull = 0xffffffffu;
    auto score_at = [&](int ch) { return sc2 != nullptr ? __ldcg(sc + ch) + __ldcg(sc2 + ch) : __ldcg(sc + ch); };
    const int P = L - w;
    const int nt = blockDim.x, nwarps = nt >> 5;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool keep_all = (k >= C);
    const int kk = min(k, C);

    // thread t owns chunk ids [c0, c1)
    const int per = (C + nt - 1) / nt;
    const int c0 = min(tid * per, C), c1 = min(c0 + per, C);
    uint32_t keys[KPT];
    if (kk > 0 && !keep_all) {
#pragma unroll
        for (int u = 0; u < KPT; ++u) keys[u] = (c0 + u < c1) ? select_order_key(score_at(c0 + u)) : 0u;
    }
    if (tid == 0) sm.last_kept = 0;

    uint32_t thresh = 0;   // key of the k-th largest score
    int need_eq = 0;       // how many chunks equal to the threshold are kept
    if (!keep_all && kk > 0) {
        int* hist = reinterpret_cast<int*>(&sm.whist[0][0]);            // kSelBins counters
        uint32_t* cand = reinterpret_cast<uint32_t*>(&sm.sel[0]);       // kSelCandCap keys (sel is written later)
        // smallest and largest key of the head
        uint32_t lo = 0xffffffffu, hi = 0u;
#pragma unroll
        for (int u = 0; u < KPT; ++u)
            if (c0 + u < c1) { lo = min(lo, keys[u]); hi = max(hi, keys[u]); }
        lo = __reduce_min_sync(kFull, lo);
        hi = __reduce_max_sync(kFull, hi);
        if (lane == 0) sm.warp_sums[warp] = (static_cast<unsigned long long>(hi) << 32) | lo;
        for (int i = tid; i < kSelBins; i += nt) hist[i] = 0;
        if (tid == 0) sm.n_cand = 0;
        __syncthreads();
        uint32_t base = 0xffffffffu, top = 0u;
        for (int wv = 0; wv < nwarps; ++wv) {
            const unsigned long long v = sm.warp_sums[wv];
            base = min(base, static_cast<uint32_t>(v));
            top = max(top, static_cast<uint32_t>(v >> 32));
        }
        uint32_t span = top - base;          // the keys of interest lie in [base, base + span]
        int need = k;                        // the need-th largest of them is the threshold
        for (int round = 0;; ++round) {
            if (span == 0u) { thresh = base; need_eq = need; break; }
            const int shift = max(0, 21 - __clz(span));      // (span >> shift) < kSelBins
            if (round > 0) {
                for (int i = tid; i < kSelBins; i += nt) hist[i] = 0;
                __syncthreads();
            }
#pragma unroll
            for (int u = 0; u < KPT; ++u) {
                const uint32_t dlt = keys[u] - base;
                if (c0 + u < c1 && keys[u] >= base && dlt <= span) atomicAdd(&hist[dlt >> shift], 1);
            }
            __syncthreads();
            // thread t < 512 owns bins 2047 - 4t .. 2044 - 4t, so a prefix over threads counts from the top
            int cnt[4] = {0, 0, 0, 0}, sum = 0;
            if (tid < kSelBins / 4) {
#pragma unroll
                for (int q = 0; q < 4; ++q) { cnt[q] = hist[kSelBins - 1 - 4 * tid - q]; sum += cnt[q]; }
            }
            int inc = sum;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int n = __shfl_up_sync(kFull, inc, off);
                if (lane >= off) inc += n;
            }
            if (lane == 31) sm.warp_tot[warp] = inc;
            __syncthreads();
            int before = 0;
            for (int wv = 0; wv < warp; ++wv) before += sm.warp_tot[wv];
            inc += before;
            if (tid < kSelBins / 4 && inc - sum < need && need <= inc) {     // exactly one thread
                int above = inc - sum, q = 0, cq = cnt[0];
#pragma unroll
                for (int t = 0; t < 3; ++t)          // (unrolled: cnt stays in registers)
                    if (q == t && above + cnt[t] < need) { above += cnt[t]; q = t + 1; cq = cnt[t + 1]; }
                sm.prefix = static_cast<uint32_t>(kSelBins - 1 - 4 * tid - q);
                sm.need = need - above;
                sm.bin_count = cq;
            }
            __syncthreads();
            const uint32_t bin = sm.prefix;
            const int n_bin = sm.bin_count;
            need = sm.need;
            const uint32_t sub = bin << shift;
            const uint32_t width = (shift >= 32) ? 0xffffffffu : ((1u << shift) - 1u);
            base += sub;
            span = min(width, span - sub);
            if (n_bin <= kSelCandCap) {
                // few keys left: rank them against each other
#pragma unroll
                for (int u = 0; u < KPT; ++u) {
                    const uint32_t dlt = keys[u] - base;
                    if (c0 + u < c1 && keys[u] >= base && dlt <= span) cand[atomicAdd(&sm.n_cand, 1)] = keys[u];
                }
                __syncthreads();
                for (int j = tid; j < n_bin; j += nt) {
                    const uint32_t v = cand[j];
                    int gt = 0, ge = 0;
                    for (int i = 0; i < n_bin; ++i) { gt += cand[i] > v; ge += cand[i] >= v; }
                    if (gt < need && need <= ge) { sm.prefix = v; sm.need = need - gt; }   // same values from every writer
                }
                __syncthreads();
                thresh = sm.prefix;
                need_eq = sm.need;
                break;
            }
        }
        __syncthreads();       // cand (= sel) and the shared words are reused below
    }

    // Ordered sweep over the chunk ids.
    const bool stage_sel = kk <= kSelCap;
    if (kk > 0) {
        unsigned gt_n = 0, eq_n = 0;
        if (keep_all) gt_n = c1 - c0;
        else {
#pragma unroll
            for (int u = 0; u < KPT; ++u)
                if (c0 + u < c1) { gt_n += keys[u] > thresh; eq_n += keys[u] == thresh; }
        }
        // block-wide exclusive prefix of the packed pair (eq in the high half, gt in the low half)
        const unsigned long long mine = (static_cast<unsigned long long>(eq_n) << 32) | gt_n;
        unsigned long long inc = mine;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned long long n = __shfl_up_sync(kFull, inc, off);
            if (lane >= off) inc += n;
        }
        if (lane == 31) sm.warp_sums[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            const unsigned long long s = (lane < nwarps) ? sm.warp_sums[lane] : 0ull;
            unsigned long long sinc = s;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const unsigned long long n = __shfl_up_sync(kFull, sinc, off);
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
                    for (int t = 0; t < len; ++t)
                        if (rank * c + t < tok_cap) dst[t] = j0 + t;
                }
                if (ch == C - 1) sm.last_kept = 1;
            }
            gt_before += gt;
            eq_before += eq;
        };
        if (!keep_all) {
#pragma unroll
            for (int u = 0; u < KPT; ++u)
                if (c0 + u < c1) visit(c0 + u, keys[u]);
        } else {
            for (int ch = c0; ch < c1; ++ch) visit(ch, 0u);
        }
    }
    __syncthreads();
    // Every kept chunk is full except possibly chunk C-1, which can only be the last kept one.
    const int tail = (C > 0) ? (P - (C - 1) * c) : 0;
    // tok_cap: at most this many tokens of the kept chunks are emitted, lowest positions first
    // (Algorithm 1 keeps the first L_max - w selected tokens); no cap by default
    const int n_tok = min(kk * c - ((sm.last_kept && kk > 0) ? (c - tail) : 0), tok_cap);
    if (stage_sel)
        for (int r = tid; r < kk; r += nt) {            // one kept chunk per thread: its c positions
            const int j0 = sm.sel[r] * c, n0 = r * c;
            for (int t = 0; t < c; ++t)
                if (n0 + t < n_tok) out[n0 + t] = j0 + t;
        }
    for (int i = tid; i < w; i += nt) out[n_tok + i] = P + i;
    for (int i = n_tok + w + tid; i < n_max; i += nt) out[i] = -1;
    __syncthreads();     // shared state may be reused by the caller
}

// The same selection with the keys of the head in a shared-memory buffer (kbuf, room for C keys)
// instead of registers: for heads with many chunks per thread (token-level selection: tens of
// thousands of keys). Same adaptive radix select and ordered sweep as select_head_regs; the passes
// over the keys are strided loops (coalesced, conflict-free), the sweep walks thread-contiguous runs.
// All threads of the CTA must call it; blockDim.x a multiple of 32, at least 512, at most 1024.
__device__ __forceinline__ void select_head_smem(const float* sc, const float* sc2, int L, int w, int c, int C, int k,
                                                 int n_max, int32_t* out, SelectSmem& sm, uint32_t* kbuf,
                                                 int tok_cap = 0x7fffffff) {
    constexpr unsigned kFull = 0xffffffffu;
    const int P = L - w;
    const int nt = blockDim.x, nwarps = nt >> 5;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool keep_all = (k >= C);
    const int kk = min(k, C);
    if (tid == 0) sm.last_kept = 0;
    uint32_t thresh = 0;
    int need_eq = 0;
    if (!keep_all && kk > 0) {
        int* hist = reinterpret_cast<int*>(&sm.whist[0][0]);
        uint32_t* cand = reinterpret_cast<uint32_t*>(&sm.sel[0]);
        uint32_t lo = 0xffffffffu, hi = 0u;
        constexpr int kB = 16;                             // loads in flight per thread
#pragma unroll 1
        for (int ch0 = tid; ch0 < C; ch0 += kB * nt) {
            float v[kB];
#pragma unroll
            for (int q = 0; q < kB; ++q) v[q] = __ldcg(sc + min(ch0 + q * nt, C - 1));
            if (sc2 != nullptr) {
#pragma unroll
                for (int q = 0; q < kB; ++q) v[q] += __ldcg(sc2 + min(ch0 + q * nt, C - 1));
            }
#pragma unroll
            for (int q = 0; q < kB; ++q)
                if (ch0 + q * nt < C) {
                    const uint32_t key = select_order_key(v[q]);
                    kbuf[ch0 + q * nt] = key;
                    lo = min(lo, key);
                    hi = max(hi, key);
                }
        }
        lo = __reduce_min_sync(kFull, lo);
        hi = __reduce_max_sync(kFull, hi);
        if (lane == 0) sm.warp_sums[warp] = (static_cast<unsigned long long>(hi) << 32) | lo;
        for (int i = tid; i < kSelBins; i += nt) hist[i] = 0;
        if (tid == 0) sm.n_cand = 0;
        __syncthreads();
        uint32_t base = 0xffffffffu, top = 0u;
        for (int wv = 0; wv < nwarps; ++wv) {
            const unsigned long long v = sm.warp_sums[wv];
            base = min(base, static_cast<uint32_t>(v));
            top = max(top, static_cast<uint32_t>(v >> 32));
        }
        uint32_t span = top - base;
        int need = k;
        for (int round = 0;; ++round) {
            if (span == 0u) { thresh = base; need_eq = need; break; }
            const int shift = max(0, 21 - __clz(span));
            if (round > 0) {
                for (int i = tid; i < kSelBins; i += nt) hist[i] = 0;
                __syncthreads();
            }
#pragma unroll 4
            for (int ch = tid; ch < C; ch += nt) {
                const uint32_t key = kbuf[ch], dlt = key - base;
                if (key >= base && dlt <= span) atomicAdd(&hist[dlt >> shift], 1);
            }
            __syncthreads();
            int cnt[4] = {0, 0, 0, 0}, sum = 0;
            if (tid < kSelBins / 4) {
#pragma unroll
                for (int q = 0; q < 4; ++q) { cnt[q] = hist[kSelBins - 1 - 4 * tid - q]; sum += cnt[q]; }
            }
            int inc = sum;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int n = __shfl_up_sync(kFull, inc, off);
                if (lane >= off) inc += n;
            }
            if (lane == 31) sm.warp_tot[warp] = inc;
            __syncthreads();
            int before = 0;
            for (int wv = 0; wv < warp; ++wv) before += sm.warp_tot[wv];
            inc += before;
            if (tid < kSelBins / 4 && inc - sum < need && need <= inc) {
                int above = inc - sum, q = 0, cq = cnt[0];
#pragma unroll
                for (int t = 0; t < 3; ++t)
                    if (q == t && above + cnt[t] < need) { above += cnt[t]; q = t + 1; cq = cnt[t + 1]; }
                sm.prefix = static_cast<uint32_t>(kSelBins - 1 - 4 * tid - q);
                sm.need = need - above;
                sm.bin_count = cq;
            }
            __syncthreads();
            const uint32_t bin = sm.prefix;
            const int n_bin = sm.bin_count;
            need = sm.need;
            const uint32_t sub = bin << shift;
            base += sub;
            span = min((1u << shift) - 1u, span - sub);
            if (n_bin <= kSelCandCap) {
#pragma unroll 4
                for (int ch = tid; ch < C; ch += nt) {
                    const uint32_t key = kbuf[ch], dlt = key - base;
                    if (key >= base && dlt <= span) cand[atomicAdd(&sm.n_cand, 1)] = key;
                }
                __syncthreads();
                for (int j = tid; j < n_bin; j += nt) {
                    const uint32_t v = cand[j];
                    int gt = 0, ge = 0;
                    for (int i = 0; i < n_bin; ++i) { gt += cand[i] > v; ge += cand[i] >= v; }
                    if (gt < need && need <= ge) { sm.prefix = v; sm.need = need - gt; }
                }
                __syncthreads();
                thresh = sm.prefix;
                need_eq = sm.need;
                break;
            }
        }
        __syncthreads();
    }
    // ordered sweep: warp v owns the contiguous ids [v * rows * 32, (v + 1) * rows * 32) and walks them in
    // rows of 32 consecutive ids, one per lane; ballots give a row's (#above, #equal) in lane order
    const bool stage_sel = kk <= kSelCap;
    if (kk > 0) {
        const unsigned lt_mask = (1u << lane) - 1u;
        const int rows = (C + nt - 1) / nt;
        const int base_id = warp * rows * 32 + lane;
        unsigned gt_n = 0, eq_n = 0;
#pragma unroll 4
        for (int u = 0; u < rows; ++u) {
            const int ch = base_id + 32 * u;
            const uint32_t key = (ch < C && !keep_all) ? kbuf[ch] : 0u;
            gt_n += __popc(__ballot_sync(kFull, ch < C && (keep_all || key > thresh)));
            eq_n += __popc(__ballot_sync(kFull, ch < C && !keep_all && key == thresh));
        }
        if (lane == 0) sm.warp_sums[warp] = (static_cast<unsigned long long>(eq_n) << 32) | gt_n;
        __syncthreads();
        if (warp == 0) {
            const unsigned long long s = (lane < nwarps) ? sm.warp_sums[lane] : 0ull;
            unsigned long long sinc = s;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const unsigned long long n = __shfl_up_sync(kFull, sinc, off);
                if (lane >= off) sinc += n;
            }
            sm.warp_sums[lane] = sinc - s;
        }
        __syncthreads();
        const unsigned long long excl = sm.warp_sums[warp];
        int gt_run = static_cast<int>(excl & 0xffffffffu), eq_run = static_cast<int>(excl >> 32);
#pragma unroll 2
        for (int u = 0; u < rows; ++u) {
            const int ch = base_id + 32 * u;
            const uint32_t key = (ch < C && !keep_all) ? kbuf[ch] : 0u;
            const bool gt = ch < C && (keep_all || key > thresh);
            const bool eq = ch < C && !keep_all && key == thresh;
            const unsigned gtm = __ballot_sync(kFull, gt), eqm = __ballot_sync(kFull, eq);
            const int gt_before = gt_run + __popc(gtm & lt_mask);
            const int eq_before = eq_run + __popc(eqm & lt_mask);
            if (gt || (eq && eq_before < need_eq)) {
                const int rank = gt_before + min(eq_before, need_eq);
                if (stage_sel) sm.sel[rank] = ch;
                else {
                    const int j0 = ch * c, len = min(c, P - j0);
                    int32_t* dst = out + static_cast<size_t>(rank) * c;
                    for (int t = 0; t < len; ++t)
                        if (rank * c + t < tok_cap) dst[t] = j0 + t;
                }
                if (ch == C - 1) sm.last_kept = 1;
            }
            gt_run += __popc(gtm);
            eq_run += __popc(eqm);
        }
    }
    __syncthreads();
    const int tail = (C > 0) ? (P - (C - 1) * c) : 0;
    const int n_tok = min(kk * c - ((sm.last_kept && kk > 0) ? (c - tail) : 0), tok_cap);
    if (stage_sel)
        for (int r = tid; r < kk; r += nt) {
            const int j0 = sm.sel[r] * c, n0 = r * c;
            for (int t = 0; t < c; ++t)
                if (n0 + t < n_tok) out[n0 + t] = j0 + t;
        }
    for (int i = tid; i < w; i += nt) out[n_tok + i] = P + i;
    for (int i = n_tok + w + tid; i < n_max; i += nt) out[i] = -1;
    __syncthreads();
}

// Selection for many chunks per thread. All threads of the CTA must call this (it uses
// __syncthreads); blockDim.x must be a multiple of 32 and at most 1024. kbuf: room for C keys
// (shared or global memory; it may be the score array itself, which is then overwritten), or
// NULL: keys are then recomputed from the scores on every use. sc2 != NULL: the head's scores are sc[ch] + sc2[ch] (a KV head scored as two
// heads of half the rows).
__device__ __forceinline__ void select_head_rows(const float* sc, const float* sc2, int L, int w, int c, int C, int k,
                                            int n_max, int32_t* __restrict__ out, SelectSmem& sm, uint32_t* kbuf,
                                            int tok_cap = 0x7fffffff) {
    auto score_at = [&](int ch) { return sc2 != nullptr ? __ldcg(sc + ch) + __ldcg(sc2 + ch) : __ldcg(sc + ch); };
    constexpr unsigned kFull = 0xffffffffu;
    const int P = L - w;
    const int nt = blockDim.x, nwarps = nt >> 5;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned lt_mask = (1u << lane) - 1u;
    const bool keep_all = (k >= C);
    const int kk = min(k, C);

    // warp v owns chunk ids [v * rows * 32, (v + 1) * rows * 32); row u of it holds base + 32 u (+ lane)
    const int rows = (C + nt - 1) / nt;
    const int base = warp * rows * 32 + lane;
    const bool need_keys = kk > 0 && !keep_all;
    if (need_keys && kbuf != nullptr) {
        // kB loads in flight per thread, no control flow between them (ids past the end are clamped)
        constexpr int kB = 16;
#pragma unroll 1
        for (int ch0 = tid; ch0 < C; ch0 += kB * nt) {
            float v[kB];
#pragma unroll
            for (int q = 0; q < kB; ++q) v[q] = __ldcg(sc + min(ch0 + q * nt, C - 1));
            if (sc2 != nullptr) {
#pragma unroll
                for (int q = 0; q < kB; ++q) v[q] += __ldcg(sc2 + min(ch0 + q * nt, C - 1));
            }
#pragma unroll
            for (int q = 0; q < kB; ++q)
                if (ch0 + q * nt < C) kbuf[ch0 + q * nt] = select_order_key(v[q]);
        }
    }
    if (tid == 0) sm.last_kept = 0;
    __syncthreads();                                         // kbuf complete
    auto key_at = [&](int ch) -> uint32_t { return kbuf != nullptr ? kbuf[ch] : select_order_key(score_at(ch)); };

    uint32_t thresh = 0;   // key of the k-th largest score
    int need_eq = 0;       // how many chunks equal to the threshold are kept
    if (need_keys) {
        uint32_t prefix = 0;
        int need = k;
#pragma unroll 1
        for (int pass = 0; pass < 4; ++pass) {
            const int shift = 24 - 8 * pass;
            if (tid < 256) sm.hist[tid] = 0;
            __syncthreads();
            if (pass == 0) {
                // bins b0 - 1 .. b0 + 2 around the bin of the warp's first key are counted in
                // registers (two 16-bit counters per register; a lane sees at most `rows` keys)
                const int ch_first = warp * rows * 32;
                const int b0 = (ch_first < C) ? static_cast<int>(key_at(ch_first) >> 24) : 0;
                const bool packed = rows < 65536;
                uint32_t lo = 0u, hi = 0u;
#pragma unroll 4
                for (int u = 0; u < rows; ++u) {
                    const int ch = base + 32 * u;
                    if (ch < C) {
                        const int bin = static_cast<int>(key_at(ch) >> 24);
                        const unsigned d = static_cast<unsigned>(bin - b0 + 1);
                        if (packed && d < 4u) {
                            const uint32_t inc = 1u << ((d & 1u) * 16u);
                            lo += (d < 2u) ? inc : 0u;
                            hi += (d < 2u) ? 0u : inc;
                        } else {
                            atomicAdd(&sm.hist[bin], 1);
                        }
                    }
                }
                const unsigned c0 = __reduce_add_sync(kFull, lo & 0xffffu), c1 = __reduce_add_sync(kFull, lo >> 16);
                const unsigned c2 = __reduce_add_sync(kFull, hi & 0xffffu), c3 = __reduce_add_sync(kFull, hi >> 16);
                if (lane == 0) {   // a non-zero count belongs to a bin some key fell into: 0 <= bin <= 255
                    if (c0) atomicAdd(&sm.hist[b0 - 1], static_cast<int>(c0));
                    if (c1) atomicAdd(&sm.hist[b0], static_cast<int>(c1));
                    if (c2) atomicAdd(&sm.hist[b0 + 1], static_cast<int>(c2));
                    if (c3) atomicAdd(&sm.hist[b0 + 2], static_cast<int>(c3));
                }
            } else {
                const uint32_t himask = 0xFFFFFFFFu << (shift + 8);
#pragma unroll 4
                for (int u = 0; u < rows; ++u) {
                    const int ch = base + 32 * u;
                    if (ch < C) {
                        const uint32_t key = key_at(ch);
                        if ((key & himask) == prefix) atomicAdd(&sm.hist[(key >> shift) & 0xFFu], 1);
                    }
                }
            }
            __syncthreads();
            if (warp == 0) {
                // lane t owns bins 255-8t .. 248-8t (descending), so a prefix over lanes counts from the top
                int cnt[8], sum = 0;
#pragma unroll
                for (int q = 0; q < 8; ++q) { cnt[q] = sm.hist[255 - 8 * lane - q]; sum += cnt[q]; }
                int inc = sum;
#pragma unroll
                for (int off = 1; off < 32; off <<= 1) {
                    const int n = __shfl_up_sync(kFull, inc, off);
                    if (lane >= off) inc += n;
                }
                const unsigned reach = __ballot_sync(kFull, inc >= need);
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

    // Ordered sweep over the chunk ids: ballots give a row's (#above, #equal) in lane order.
    const bool stage_sel = kk <= kSelCap;
    if (kk > 0) {
        auto row_flags = [&](int ch, unsigned& gtm, unsigned& eqm, bool& gt, bool& eq) {
            const bool valid = ch < C;
            uint32_t key = 0u;
            if (!keep_all && valid) key = key_at(ch);
            gt = valid && (keep_all || key > thresh);
            eq = valid && !keep_all && key == thresh;
            gtm = __ballot_sync(kFull, gt);
            eqm = __ballot_sync(kFull, eq);
        };
        unsigned gt_n = 0, eq_n = 0;                         // the warp's totals (same in every lane)
#pragma unroll 4
        for (int u = 0; u < rows; ++u) {
            unsigned gtm, eqm;
            bool gt, eq;
            row_flags(base + 32 * u, gtm, eqm, gt, eq);
            gt_n += __popc(gtm);
            eq_n += __popc(eqm);
        }
        // block-wide exclusive prefix of the packed pair (eq in the high half, gt in the low half)
        if (lane == 0) sm.warp_sums[warp] = (static_cast<unsigned long long>(eq_n) << 32) | gt_n;
        __syncthreads();
        if (warp == 0) {
            const unsigned long long s = (lane < nwarps) ? sm.warp_sums[lane] : 0ull;
            unsigned long long sinc = s;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const unsigned long long n = __shfl_up_sync(kFull, sinc, off);
                if (lane >= off) sinc += n;
            }
            sm.warp_sums[lane] = sinc - s;
        }
        __syncthreads();
        const unsigned long long excl = sm.warp_sums[warp];
        int gt_run = static_cast<int>(excl & 0xffffffffu), eq_run = static_cast<int>(excl >> 32);
#pragma unroll 2
        for (int u = 0; u < rows; ++u) {
            const int ch = base + 32 * u;
            unsigned gtm, eqm;
            bool gt, eq;
            row_flags(ch, gtm, eqm, gt, eq);
            const int gt_before = gt_run + __popc(gtm & lt_mask);
            const int eq_before = eq_run + __popc(eqm & lt_mask);
            if (gt || (eq && eq_before < need_eq)) {
                const int rank = gt_before + min(eq_before, need_eq);
                if (stage_sel) sm.sel[rank] = ch;
                else {
                    const int j0 = ch * c, len = min(c, P - j0);
                    int32_t* dst = out + static_cast<size_t>(rank) * c;
                    for (int t = 0; t < len; ++t)
                        if (rank * c + t < tok_cap) dst[t] = j0 + t;
                }
                if (ch == C - 1) sm.last_kept = 1;
            }
            gt_run += __popc(gtm);
            eq_run += __popc(eqm);
        }
    }
    __syncthreads();
    // Every kept chunk is full except possibly chunk C-1, which can only be the last kept one.
    const int tail = (C > 0) ? (P - (C - 1) * c) : 0;
    // tok_cap: at most this many tokens of the kept chunks are emitted, lowest positions first
    // (Algorithm 1 keeps the first L_max - w selected tokens); no cap by default
    const int n_tok = min(kk * c - ((sm.last_kept && kk > 0) ? (c - tail) : 0), tok_cap);
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
