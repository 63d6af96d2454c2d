// Device-side bodies of the top-k chunk selection (ChunkKV Algorithm 3: "Top-K(chunk_scores, k)",
// the selection mask, "always keep most recent tokens", "nonzero(mask)"), shared by the
// stand-alone select kernel and the fused layer kernel. One CTA works on one KV head.
//
// Both bodies find the k-th largest of the order-preserving 32-bit keys by an exact 4-pass radix
// select and then rank every chunk among the kept ones: rank = #above before it + min(#equal
// before it, ties to keep) - ties go to the lower chunk id. Token positions are written directly
// in ascending order: no mask, no sort.
//
// select_head_regs (a few chunks per thread): each thread owns a contiguous run of chunk ids and
// keeps their keys in registers. In the first radix pass, whose digit (sign and high exponent
// bits) is nearly constant, every warp counts into its own 16-bit histogram row (lanes that hit
// the same bin add once); later passes add one shared-memory atomic per surviving key. One
// block-wide prefix sum over the threads' (#above, #equal) gives the ranks. Fully unrolled.
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
    uint32_t prefix;
    int need;
    int last_kept;
};

__device__ __forceinline__ uint32_t select_order_key(float x) {
    const uint32_t b = __float_as_uint(x + 0.0f);          // -0 and +0 compare equal
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);     // larger float <=> larger key
}

// Selection for a few chunks per thread. All threads of the CTA must call this (it uses
// __syncthreads); blockDim.x must be a multiple of 32 and at most 1024. Every thread keeps up to
// KPT keys in registers, which needs C <= blockDim.x * KPT (KPT = 0 re-reads keys from memory
// on every use instead).
// sc2 != NULL: the head's scores are sc[ch] + sc2[ch] (a KV head scored as two heads of half the rows).
template <int KPT>
__device__ __forceinline__ void select_head_regs(const float* __restrict__ sc, const float* __restrict__ sc2, int L, int w, int c,
                                            int C, int k, int n_max, int32_t* __restrict__ out, SelectSmem& sm,
                                            int tok_cap = 0x7fffffff) {
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
                    for (int t = 0; t < len; ++t)
                        if (rank * c + t < tok_cap) dst[t] = j0 + t;
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
