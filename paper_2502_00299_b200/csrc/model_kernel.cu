// Many layers in one launch (ChunkKV Algorithm 2: "for l = 0 .. N_layers - 1", with Algorithm 3 per
// computed layer): a persistent version of the layer kernel of layer_resident.cu in which the
// steps of successive layers overlap inside every CTA.
//
// A CTA belongs to one scoring head and one key range for the whole launch. Its warps have roles:
//   warp 0         TMA producer: streams the Q tile and the CTA's K tiles of layer after layer
//                  through the shared-memory ring, as far ahead as the ring allows
//   warp 1         tcgen05.mma issuer
//   warps 2..17    epilogue: one exponential per score element, chunk sums into tensor memory;
//                  at the end of a layer they publish the CTA's per-row (max, sum), wait for the
//                  head's other CTAs (bounded), merge the row statistics, contract the partial
//                  sums over the rows into the chunk scores of the CTA's key range (global memory),
//                  announce them on the head's second counter and go on with the next layer
//   warps 18..19   tail: for each computed layer, once the head's chunk scores are complete, run
//                  the exact top-k (every CTA of a head computes the same kept-chunk list), write
//                  out_idx (one CTA per head) and move this CTA's share of the kept K/V rows with
//                  bulk asynchronous copies (global -> shared -> global, whole chunks at a time) -
//                  for the computed layer and for every following layer that reuses its indices
//
// So while the tail warps select and gather layer l, the other warps already score layer l + 1: the
// latency-bound steps cost no memory bandwidth and the copies ride along with the K stream.
// Hand-over counters only grow during a launch (layer l waits for (l + 1) x CTAs arrivals); the
// last CTA to leave clears them. Every wait is bounded and reports through the device status word.
#include "internal.h"
#include "panels.cuh"
#include "ptx.cuh"
#include "resident.cuh"
#include "select.cuh"

#include <math_constants.h>

namespace chunkkv {

namespace {

constexpr int kMThreads = 640;
constexpr int kMEpiThreads = 512;
constexpr int kMTailThreads = 64;
constexpr int kMMiscBytes = 14336;      // epilogue: group records, slices, m_i, 1 / l_i, row sums per lane quarter
constexpr int kMSlots = 8;              // staging slots of the row copies
constexpr int kMSelBins = 2048;
constexpr int kMCandCap = 1024;
constexpr int kBarEpi = 1, kBarTail = 2;

struct ModelCtl {
    unsigned long long full[kRMaxStages];
    unsigned long long empty[kRMaxStages];
    unsigned long long tfull[2];
    unsigned long long tempty[2];
    unsigned long long qfull;
    unsigned long long qempty;
    unsigned long long gfull[kMSlots];
    unsigned long long sfull;          // the head's chunk scores have landed in shared memory (tail warps)
    uint32_t tmem_base;
    int abort_flag;
    int epi_ok;
    // tail warps
    int tail_ok;
    unsigned long long t_pair[2];
    int t_tot[2];
    uint32_t t_prefix;
    int t_need, t_bin_count, t_ncand, t_last_kept;
};

struct ModelLayer {
    const uint4* K;
    const uint4* V;
    uint4* out_K;
    uint4* out_V;
    int32_t* out_idx;
    int slot;          // computed layer: its slot (0 .. n_compute - 1); reuse layer: the slot of its source layer
    int computes;      // 1: scored and selected here; 0: gathered with the slot's indices
};

struct ModelParams {
    CUtensorMap tm_q[kModelMaxCompute];
    CUtensorMap tm_k[kModelMaxCompute];
    ModelLayer layer[kModelMaxLayers];
    int n_layers, n_compute;
    int L, P, w, R, Hs, d, kv_shift;
    float sl2;
    int cph, n_tiles, n_stages, q_box_rows, k_box_rows;
    int C, k, n_max, Hkv;
    int Cpad;              // row stride of the chunk scores (C rounded up to a multiple of 4: rows stay 16-byte aligned)
    int off_ring, off_pmax, off_misc, off_tail, stage_slot_bytes;
    float* cta_stat;       // [2 (slot parity)][grid][{max, sum}][128]
    float* scores;         // [n_compute][Hs][Cpad]
    unsigned* cnt_a;       // [Hs]
    unsigned* cnt_b;       // [Hs]
    unsigned* exits;
    int* status;
};

// ---- bulk asynchronous copies (no multicast): global -> this CTA's shared memory with byte-counted
//      completion on an mbarrier, and shared -> global in bulk groups
__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_smem),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void bulk_store(void* dst, uint32_t src_smem, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src_smem), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// Bounded wait of one thread on a counter that only grows.
__device__ __forceinline__ bool wait_counter(const unsigned* counter, unsigned target, volatile int* abort_flag,
                                             unsigned sleep_ns) {
    unsigned cur;
    asm volatile("ld.acquire.gpu.u32 %0, [%1];" : "=r"(cur) : "l"(counter) : "memory");
    if (cur >= target) return true;
    const long long t0 = clock64();
    for (;;) {
        if (sleep_ns) __nanosleep(sleep_ns);
        asm volatile("ld.acquire.gpu.u32 %0, [%1];" : "=r"(cur) : "l"(counter) : "memory");
        if (cur >= target) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > kWaitLimitClocks) { *abort_flag = 1; return false; }
    }
}

// Exact top-k of one head's chunk scores by the 64 tail threads (same adaptive radix select as
// select_head_regs in select.cuh, with the keys in shared memory): fills sel[0 .. kk) with the kept
// chunk ids in ascending order and returns whether the clipped last chunk is among them.
// Two warps have little latency hiding of their own, so every pass walks the keys four at a time
// (16-byte shared-memory accesses) with several independent accesses in flight per thread.
// keys: Cpad = C rounded up to a multiple of 4 entries; entries at or past C are ignored.
__device__ __forceinline__ int tail_select(const float* row2, int C, int Cpad, int k, uint32_t* keys, int* hist,
                                           int* sel, ModelCtl& ctl, int tt) {
    // keys[0 .. C) holds the head's chunk scores as floats on entry (row2 != NULL: to be added to a
    // second row, the other half of the head's query rows) and their order-preserving keys afterwards
    constexpr unsigned kFull = 0xffffffffu;
    const int lane = tt & 31, tw = tt >> 5;
    if (tt == 0) { ctl.t_last_kept = 0; ctl.t_ncand = 0; }
    if (k >= C) {                      // everything is kept
        for (int ch = tt; ch < C; ch += kMTailThreads) sel[ch] = ch;
        named_barrier(kBarTail, kMTailThreads);
        return C > 0 ? 1 : 0;
    }
    const int nv = Cpad >> 2;          // 16-byte groups of keys
    uint4* kv = reinterpret_cast<uint4*>(keys);
    const float4* r2 = reinterpret_cast<const float4*>(row2);
    uint32_t lo = 0xffffffffu, hi = 0u;
#pragma unroll 4
    for (int v = tt; v < nv; v += kMTailThreads) {
        const uint4 raw = kv[v];
        float4 f = make_float4(__uint_as_float(raw.x), __uint_as_float(raw.y), __uint_as_float(raw.z), __uint_as_float(raw.w));
        if (row2 != nullptr) { const float4 g = r2[v]; f.x += g.x; f.y += g.y; f.z += g.z; f.w += g.w; }
        uint4 key = make_uint4(select_order_key(f.x), select_order_key(f.y), select_order_key(f.z), select_order_key(f.w));
        const int ch = 4 * v;
        if (ch + 1 >= C) key.y = key.x;      // entries past C copy a valid key: they never widen [min, max]
        if (ch + 2 >= C) key.z = key.x;
        if (ch + 3 >= C) key.w = key.x;
        kv[v] = key;
        lo = min(min(lo, key.x), min(min(key.y, key.z), key.w));
        hi = max(max(hi, key.x), max(max(key.y, key.z), key.w));
    }
    lo = __reduce_min_sync(kFull, lo);
    hi = __reduce_max_sync(kFull, hi);
    if (lane == 0) ctl.t_pair[tw] = (static_cast<unsigned long long>(hi) << 32) | lo;
    {
        int4* hv = reinterpret_cast<int4*>(hist);
#pragma unroll
        for (int i = 0; i < kMSelBins / 4 / kMTailThreads; ++i) hv[tt + i * kMTailThreads] = make_int4(0, 0, 0, 0);
    }
    named_barrier(kBarTail, kMTailThreads);
    uint32_t base = min(static_cast<uint32_t>(ctl.t_pair[0]), static_cast<uint32_t>(ctl.t_pair[1]));
    const uint32_t top = max(static_cast<uint32_t>(ctl.t_pair[0] >> 32), static_cast<uint32_t>(ctl.t_pair[1] >> 32));
    uint32_t span = top - base;
    int need = k;
    uint32_t thresh = 0;
    int need_eq = 0;
    for (int round = 0;; ++round) {
        if (span == 0u) { thresh = base; need_eq = need; break; }
        const int shift = max(0, 21 - __clz(span));
        if (round > 0) {
            int4* hv = reinterpret_cast<int4*>(hist);
#pragma unroll
            for (int i = 0; i < kMSelBins / 4 / kMTailThreads; ++i) hv[tt + i * kMTailThreads] = make_int4(0, 0, 0, 0);
            named_barrier(kBarTail, kMTailThreads);
        }
#pragma unroll 4
        for (int v = tt; v < nv; v += kMTailThreads) {
            const uint4 key = kv[v];
            const int ch = 4 * v;
            const uint32_t d0 = key.x - base, d1 = key.y - base, d2 = key.z - base, d3 = key.w - base;
            if (key.x >= base && d0 <= span) atomicAdd(&hist[d0 >> shift], 1);
            if (ch + 1 < C && key.y >= base && d1 <= span) atomicAdd(&hist[d1 >> shift], 1);
            if (ch + 2 < C && key.z >= base && d2 <= span) atomicAdd(&hist[d2 >> shift], 1);
            if (ch + 3 < C && key.w >= base && d3 <= span) atomicAdd(&hist[d3 >> shift], 1);
        }
        named_barrier(kBarTail, kMTailThreads);
        // thread t owns bins 2047 - 32 t .. 2016 - 32 t (descending): eight 16-byte loads
        const int b_lo = kMSelBins - 32 - 32 * tt;
        const int4* hb = reinterpret_cast<const int4*>(hist + b_lo);
        int4 hq[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) hq[i] = hb[i];
        int sum = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) sum += (hq[i].x + hq[i].y) + (hq[i].z + hq[i].w);
        int inc = sum;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int n = __shfl_up_sync(kFull, inc, off);
            if (lane >= off) inc += n;
        }
        if (lane == 31) ctl.t_tot[tw] = inc;
        named_barrier(kBarTail, kMTailThreads);
        if (tw == 1) inc += ctl.t_tot[0];
        if (inc - sum < need && need <= inc) {          // exactly one thread
            int above = inc - sum, q = 0;
            const int b_hi = b_lo + 31;
            while (q < 31 && above + hist[b_hi - q] < need) { above += hist[b_hi - q]; ++q; }
            ctl.t_prefix = static_cast<uint32_t>(b_hi - q);
            ctl.t_need = need - above;
            ctl.t_bin_count = hist[b_hi - q];
        }
        named_barrier(kBarTail, kMTailThreads);
        const uint32_t bin = ctl.t_prefix;
        const int n_bin = ctl.t_bin_count;
        need = ctl.t_need;
        const uint32_t sub = bin << shift;
        base += sub;
        span = min((1u << shift) - 1u, span - sub);
        if (n_bin <= kMCandCap) {
            uint32_t* cand = reinterpret_cast<uint32_t*>(hist);      // the histogram is no longer needed
            named_barrier(kBarTail, kMTailThreads);                   // ... once every thread has read it
#pragma unroll 4
            for (int v = tt; v < nv; v += kMTailThreads) {
                const uint4 key = kv[v];
                const int ch = 4 * v;
                if (key.x >= base && key.x - base <= span) cand[atomicAdd(&ctl.t_ncand, 1)] = key.x;
                if (ch + 1 < C && key.y >= base && key.y - base <= span) cand[atomicAdd(&ctl.t_ncand, 1)] = key.y;
                if (ch + 2 < C && key.z >= base && key.z - base <= span) cand[atomicAdd(&ctl.t_ncand, 1)] = key.z;
                if (ch + 3 < C && key.w >= base && key.w - base <= span) cand[atomicAdd(&ctl.t_ncand, 1)] = key.w;
            }
            named_barrier(kBarTail, kMTailThreads);
            for (int j = tt; j < n_bin; j += kMTailThreads) {
                const uint32_t v = cand[j];
                int gt = 0, ge = 0;
                for (int i = 0; i < n_bin; ++i) { gt += cand[i] > v; ge += cand[i] >= v; }
                if (gt < need && need <= ge) { ctl.t_prefix = v; ctl.t_need = need - gt; }
            }
            named_barrier(kBarTail, kMTailThreads);
            thresh = ctl.t_prefix;
            need_eq = ctl.t_need;
            break;
        }
    }
    // ordered sweep: thread t owns the contiguous 16-byte groups [v0, v1)
    const int pv = (nv + kMTailThreads - 1) / kMTailThreads;
    const int v0 = min(tt * pv, nv), v1 = min(v0 + pv, nv);
    unsigned gt_n = 0, eq_n = 0;
#pragma unroll 4
    for (int v = v0; v < v1; ++v) {
        const uint4 key = kv[v];
        const int ch = 4 * v;
        gt_n += (key.x > thresh) + (ch + 1 < C && key.y > thresh) + (ch + 2 < C && key.z > thresh) + (ch + 3 < C && key.w > thresh);
        eq_n += (key.x == thresh) + (ch + 1 < C && key.y == thresh) + (ch + 2 < C && key.z == thresh) + (ch + 3 < C && key.w == thresh);
    }
    const unsigned long long mine = (static_cast<unsigned long long>(eq_n) << 32) | gt_n;
    unsigned long long inc = mine;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const unsigned long long n = __shfl_up_sync(kFull, inc, off);
        if (lane >= off) inc += n;
    }
    named_barrier(kBarTail, kMTailThreads);           // t_pair was read above by every thread
    if (lane == 31) ctl.t_pair[tw] = inc;
    named_barrier(kBarTail, kMTailThreads);
    const unsigned long long excl = (tw == 1 ? ctl.t_pair[0] : 0ull) + inc - mine;
    int gt_before = static_cast<int>(excl & 0xffffffffu), eq_before = static_cast<int>(excl >> 32);
    auto visit = [&](int ch, uint32_t key) {
        const bool gt = key > thresh, eq = key == thresh;
        if (gt || (eq && eq_before < need_eq)) {
            sel[gt_before + min(eq_before, need_eq)] = ch;
            if (ch == C - 1) ctl.t_last_kept = 1;
        }
        gt_before += gt;
        eq_before += eq;
    };
#pragma unroll 2
    for (int v = v0; v < v1; ++v) {
        const uint4 key = kv[v];
        const int ch = 4 * v;
        visit(ch, key.x);
        if (ch + 1 < C) visit(ch + 1, key.y);
        if (ch + 2 < C) visit(ch + 2, key.z);
        if (ch + 3 < C) visit(ch + 3, key.w);
    }
    named_barrier(kBarTail, kMTailThreads);
    return ctl.t_last_kept;
}

template <int C_STATIC>
__global__ void __launch_bounds__(kMThreads, 1)
model_kernel(const __grid_constant__ ModelParams p) {
    constexpr int SPP = kRPanel / C_STATIC;
    constexpr uint32_t IDESC = umma_idesc_bf16(128, kRUmmaN);

    extern __shared__ uint8_t smem_raw[];
    __shared__ ModelCtl ctl;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int KB = p.d >> 6;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* dyn = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t q_base = smem_base;
    const uint32_t k_base = smem_base + static_cast<uint32_t>(p.off_ring);
    float* pmax = reinterpret_cast<float*>(dyn + p.off_pmax);
    float* misc = reinterpret_cast<float*>(dyn + p.off_misc);
    float* rec = misc;                 // [4 groups][{max, sum}][128]
    float* slice = misc + 1024;        // [4 slices][{max, sum}][128]
    float* gm = misc + 2048;
    float* ginv = misc + 2176;
    float* red = misc + 2304;          // [4 lane quarters][256 chunk slots]
    volatile int* abort_flag = &ctl.abort_flag;
    const uint32_t n_stages = static_cast<uint32_t>(p.n_stages);

    const int hs = blockIdx.x / p.cph, part = blockIdx.x - hs * p.cph;
    const int hkv = hs >> p.kv_shift;
    const int t_begin = p.n_tiles * part / p.cph, t_end = p.n_tiles * (part + 1) / p.cph;
    const int nt = t_end - t_begin;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.n_stages; ++s) {
            mbar_init(smem_u32(&ctl.full[s]), 1);
            mbar_init(smem_u32(&ctl.empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&ctl.tfull[b]), 1);
            mbar_init(smem_u32(&ctl.tempty[b]), 8);
        }
        mbar_init(smem_u32(&ctl.qfull), 1);
        mbar_init(smem_u32(&ctl.qempty), 1);
        for (int s = 0; s < kMSlots; ++s) mbar_init(smem_u32(&ctl.gfull[s]), 1);
        mbar_init(smem_u32(&ctl.sfull), 1);
        ctl.abort_flag = 0;
        ctl.epi_ok = 1;
        ctl.tail_ok = 1;
        fence_mbar_init();
        fence_proxy_async();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&ctl.tmem_base), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl.tmem_base;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (elect_one() && nt > 0) {
            const uint32_t qbar = smem_u32(&ctl.qfull);
            const uint32_t q_bytes = static_cast<uint32_t>(KB * p.q_box_rows) * 128u;
            const uint32_t k_bytes = static_cast<uint32_t>(p.k_box_rows) * 128u;
            uint32_t st = 0, st_par = 1;
            int issued = 0;
            bool ok = true;
            for (int s = 0; s < p.n_compute && ok; ++s) {
                prefetch_tmap(&p.tm_q[s]);
                prefetch_tmap(&p.tm_k[s]);
                // the Q tile is free again once the last UMMA of the previous layer has read it
                if (s > 0) ok = mbar_wait(smem_u32(&ctl.qempty), (s - 1) & 1, abort_flag);
                if (!ok) break;
                mbar_arrive_expect_tx(qbar, q_bytes);
                for (int kb = 0; kb < KB; ++kb)
                    tma_load_3d(q_base + static_cast<uint32_t>(kb) * kRQTileBytes, &p.tm_q[s], qbar, kb * 64, 0, hs);
                for (int t = t_begin; t < t_end && ok; ++t) {
                    for (int kb = 0; kb < KB; ++kb) {
                        ok = mbar_wait(smem_u32(&ctl.empty[st]), st_par, abort_flag);
                        if (!ok) break;
                        const uint32_t bar = smem_u32(&ctl.full[st]);
                        mbar_arrive_expect_tx(bar, k_bytes);
                        tma_load_3d(k_base + st * kRStageBytes, &p.tm_k[s], bar, kb * 64, t * kRTile, hkv);
                        ++issued;
                        if (++st == n_stages) { st = 0; st_par ^= 1u; }
                    }
                }
            }
            if (!ok) {
                const int back = min(issued, p.n_stages);
                for (int i = 1; i <= back; ++i) {
                    const int cc = issued - i, s = cc % p.n_stages;
                    const long long t0 = clock64();
                    while (!mbar_try_wait(smem_u32(&ctl.full[s]), (cc / p.n_stages) & 1) &&
                           clock64() - t0 < kWaitLimitClocks / 8) {
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ UMMA issuer
        if (elect_one() && nt > 0) {
            uint32_t st = 0, st_par = 0;
            int tg = 0;                  // tiles issued so far (all layers): buffer = tg & 1
            bool ok = true;
            for (int s = 0; s < p.n_compute && ok; ++s) {
                ok = mbar_wait(smem_u32(&ctl.qfull), s & 1, abort_flag);
                for (int ti = 0; ti < nt && ok; ++ti, ++tg) {
                    const int buf = tg & 1, use = tg >> 1;
                    ok = mbar_wait(smem_u32(&ctl.tempty[buf]), (use & 1) ^ 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t d_addr = tmem_base + static_cast<uint32_t>(buf * kRUmmaN);
#pragma unroll
                    for (int kb = 0; kb < 2; ++kb) {
                        if (kb >= KB || !ok) break;
                        ok = mbar_wait(smem_u32(&ctl.full[st]), st_par, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                        const uint64_t b_desc = umma_desc_sw128(k_base + st * kRStageBytes);
                        const uint64_t a_desc = umma_desc_sw128(q_base + static_cast<uint32_t>(kb) * kRQTileBytes);
#pragma unroll
                        for (int k4 = 0; k4 < 4; ++k4)
                            umma_bf16(d_addr, a_desc + 2u * k4, b_desc + 2u * k4, IDESC, (kb > 0 || k4 > 0) ? 1u : 0u);
                        umma_commit(smem_u32(&ctl.empty[st]));
                        if (++st == n_stages) { st = 0; st_par ^= 1u; }
                    }
                    if (ok) umma_commit(smem_u32(&ctl.tfull[buf]));
                }
                if (ok) umma_commit(smem_u32(&ctl.qempty));       // every UMMA of this layer has read the Q tile
            }
        }
    } else if (warp < 18) {
        // ------------------------------------------------------------------ epilogue
        const int et = threadIdx.x - 64;                 // 0 .. 511
        const int grp = (warp - 2) >> 2, quarter = warp & 3;
        const int pair = grp >> 1, half = grp & 1;
        const int row = quarter * 32 + lane;
        const bool active = row < p.R;
        const int last_visible = p.P + (row % p.w);
        const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        const int n_pl = 2 * nt;
        const int n_local = nt * (kRTile / C_STATIC);
        const int ch0 = t_begin * (kRTile / C_STATIC);
        bool ok = true;
        int tg0 = 0;                                      // global index of the layer's first tile
        for (int s = 0; s < p.n_compute && ok; ++s, tg0 += nt) {
            float run_m = -CUDART_INF_F, run_l = 0.f;
            // this pair's tiles: global tile index tg with (tg & 1) == pair
            for (int ti = (pair - (tg0 & 1)) & 1; ti < nt; ti += 2) {
                const int tg = tg0 + ti, use = tg >> 1;
                bool ready = true;
                if (lane == 0) ready = mbar_wait(smem_u32(&ctl.tfull[pair]), use & 1, abort_flag);
                if (!__shfl_sync(0xffffffffu, ready, 0)) { ok = false; break; }
                tc_fence_after();
                float v[kRPanel];
                load_panel<kRPanel>(lane_addr + static_cast<uint32_t>(pair * kRUmmaN + half * kRPanel), v);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctl.tempty[pair]));
                const int pl = ti * 2 + half;
                const int j0 = (t_begin + ti) * kRTile + half * kRPanel;
                float pr[SPP], m2, l;
                auto emit = [&](int ch, float acc) { pr[ch] = acc; };
                if (j0 + kRPanel <= p.P)
                    panel_fast<C_STATIC, kRPanel>(v, p.sl2, emit, &m2, &l);
                else
                    panel_static_tail<C_STATIC, kRPanel>(v, p.sl2, emit, j0, p.P, last_visible, &m2, &l);
                part_store<SPP>(lane_addr + static_cast<uint32_t>(kRPartCol0 + pl * SPP), pr);
                pmax[pl * 128 + row] = m2;
                const float nm = fmaxf(run_m, m2);
                const float s_old = (run_m == -CUDART_INF_F) ? 0.f : ex2_approx(run_m - nm);
                const float s_new = (m2 == -CUDART_INF_F) ? 0.f : ex2_approx(m2 - nm);
                run_l = run_l * s_old + l * s_new;
                run_m = nm;
            }
            tmem_st_wait();
            rec[(grp * 2 + 0) * 128 + row] = active ? run_m : -CUDART_INF_F;
            rec[(grp * 2 + 1) * 128 + row] = active ? run_l : 0.f;
            tc_fence_before();
            named_barrier(kBarEpi, kMEpiThreads);
            tc_fence_after();
            if (ctl.abort_flag) { ok = false; break; }
            // ---- publish this CTA's (max, sum) per row; wait for the head's other CTAs
            if (et < 128) {
                float M = -CUDART_INF_F, Ls = 0.f;
#pragma unroll
                for (int g = 0; g < 4; ++g) merge_ml(M, Ls, rec[(g * 2) * 128 + et], rec[(g * 2 + 1) * 128 + et]);
                float* dst = p.cta_stat + (static_cast<size_t>(s & 1) * gridDim.x + blockIdx.x) * 256;
                dst[et] = M;
                dst[128 + et] = Ls;
            }
            named_barrier(kBarEpi, kMEpiThreads);
            if (et == 0) {
                unsigned old;
                asm volatile("atom.add.release.gpu.u32 %0, [%1], 1;" : "=r"(old) : "l"(p.cnt_a + hs) : "memory");
                const bool w_ok = wait_counter(p.cnt_a + hs, static_cast<unsigned>(s + 1) * p.cph, abort_flag, 0);
                asm volatile("fence.acq_rel.gpu;" ::: "memory");
                ctl.epi_ok = w_ok ? 1 : 0;
            }
            named_barrier(kBarEpi, kMEpiThreads);
            if (!ctl.epi_ok) { ok = false; break; }
            // ---- row statistics of the head
            {
                const int i = et & 127, sl = et >> 7;
                const float* src = p.cta_stat + (static_cast<size_t>(s & 1) * gridDim.x + static_cast<size_t>(hs) * p.cph) * 256 + i;
                float M = -CUDART_INF_F, Ls = 0.f;
                for (int j0 = sl; j0 < p.cph; j0 += 16) {
                    float rm[4], rl[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int j = j0 + 4 * u;
                        rm[u] = (j < p.cph) ? __ldcg(src + static_cast<size_t>(j) * 256) : -CUDART_INF_F;
                        rl[u] = (j < p.cph) ? __ldcg(src + static_cast<size_t>(j) * 256 + 128) : 0.f;
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) merge_ml(M, Ls, rm[u], rl[u]);
                }
                slice[(sl * 2 + 0) * 128 + i] = M;
                slice[(sl * 2 + 1) * 128 + i] = Ls;
            }
            named_barrier(kBarEpi, kMEpiThreads);
            if (et < 128) {
                float M = -CUDART_INF_F, Ls = 0.f;
#pragma unroll
                for (int q = 0; q < 4; ++q) merge_ml(M, Ls, slice[(q * 2) * 128 + et], slice[(q * 2 + 1) * 128 + et]);
                gm[et] = M;
                ginv[et] = 1.0f / Ls;
            }
            named_barrier(kBarEpi, kMEpiThreads);
            // ---- chunk scores of this CTA's key range (see layer_resident.cu)
            {
                const float mi = gm[row], li = ginv[row];
                constexpr int PPB = 30 / SPP;
                for (int b0 = 0; grp + 4 * b0 < n_pl; b0 += PPB) {
                    float v[32];
#pragma unroll
                    for (int u = 0; u < PPB; ++u) {
                        const int pl = min(grp + 4 * (b0 + u), n_pl - 1);
                        part_load<SPP>(lane_addr + static_cast<uint32_t>(kRPartCol0 + pl * SPP), &v[u * SPP]);
                    }
                    tmem_ld_wait();
                    v[30] = 0.f;
                    v[31] = 0.f;
#pragma unroll
                    for (int u = 0; u < PPB; ++u) {
                        const int pl = grp + 4 * (b0 + u);
                        const bool have = active && pl < n_pl;
                        const float f = have ? ex2_approx(pmax[min(pl, n_pl - 1) * 128 + row] - mi) * li : 0.f;
#pragma unroll
                        for (int q = 0; q < SPP; ++q) v[u * SPP + q] = have ? v[u * SPP + q] * f : 0.f;
                    }
                    const float tot = warp_transpose_reduce(v, lane);
                    const int pl = grp + 4 * (b0 + lane / SPP);
                    if (lane < 30 && pl < n_pl) red[quarter * 256 + pl * SPP + lane % SPP] = tot;
                }
            }
            tc_fence_before();
            named_barrier(kBarEpi, kMEpiThreads);
            tc_fence_after();
            float* sc_out = p.scores + (static_cast<size_t>(s) * p.Hs + hs) * p.Cpad;
            for (int lc = et; lc < n_local; lc += kMEpiThreads)
                if (ch0 + lc < p.C) sc_out[ch0 + lc] = (red[lc] + red[256 + lc]) + (red[512 + lc] + red[768 + lc]);
            named_barrier(kBarEpi, kMEpiThreads);
            if (et == 0) {
                unsigned old;     // release: the scores written above (ordered by the barrier) are visible to whoever sees the count
                asm volatile("atom.add.release.gpu.u32 %0, [%1], 1;" : "=r"(old) : "l"(p.cnt_b + hs) : "memory");
            }
        }
        if (!ok && lane == 0) ctl.abort_flag = 1;
    } else {
        // ------------------------------------------------------------------ tail: select + row copies
        const int tt = threadIdx.x - 576;                // 0 .. 63
        uint8_t* tbase = dyn + p.off_tail;
        int* hist = reinterpret_cast<int*>(tbase);                                   // 2048 bins (8 KB)
        uint32_t* keys = reinterpret_cast<uint32_t*>(tbase + 8192);                  // [1 or 2][Cpad] scores, then C keys
        const size_t keys_bytes = ((static_cast<size_t>(p.Cpad) * 4 << p.kv_shift) + 127) & ~size_t(127);
        int* sel = reinterpret_cast<int*>(tbase + 8192 + keys_bytes);                // kept chunk ids
        const size_t sel_bytes = (static_cast<size_t>(min(p.k, p.C)) * 4 + 127) & ~size_t(127);
        const uint32_t stage0 = smem_u32(tbase + 8192 + keys_bytes + sel_bytes);     // kMSlots x stage_slot_bytes, 128-byte aligned
        const int Q = p.cph << p.kv_shift;               // CTAs of this KV head
        const int q = static_cast<int>(blockIdx.x) - (hkv << p.kv_shift) * p.cph;
        const int kk = min(p.k, p.C);
        const int wu = (p.w + C_STATIC - 1) / C_STATIC;  // the window as pseudo-chunks of up to c rows
        const int U = kk + wu;                           // copy units of the head
        const int u_begin = static_cast<int>(static_cast<long long>(U) * q / Q);
        const int u_end = static_cast<int>(static_cast<long long>(U) * (q + 1) / Q);
        const uint32_t row_bytes = static_cast<uint32_t>(p.d) * 2u;
        const int tail_rows = (p.C > 0) ? (p.P - (p.C - 1) * C_STATIC) : 0;      // rows of the clipped last chunk
        uint32_t g_issued = 0;                           // units loaded so far (all layers): slot = g % kMSlots
        bool ok = true;
        for (int li = 0; li < p.n_layers && ok;) {
            const int s = p.layer[li].slot;
            // ---- the head's chunk scores of slot s are complete once every CTA of its scoring heads has
            //      announced them; one bulk copy per row brings them into shared memory
            if (tt == 0) {
                const unsigned target = static_cast<unsigned>(s + 1) * p.cph;
                bool w_ok = wait_counter(p.cnt_b + (hkv << p.kv_shift), target, abort_flag, 200);
                if (w_ok && p.kv_shift) w_ok = wait_counter(p.cnt_b + (hkv << p.kv_shift) + 1, target, abort_flag, 200);
                asm volatile("fence.acq_rel.gpu;" ::: "memory");
                if (w_ok) {
                    const float* sc = p.scores + (static_cast<size_t>(s) * p.Hs + (hkv << p.kv_shift)) * p.Cpad;
                    const uint32_t bytes = static_cast<uint32_t>(p.Cpad) * 4u << p.kv_shift;     // the rows are adjacent
                    const uint32_t bar = smem_u32(&ctl.sfull);
                    mbar_arrive_expect_tx(bar, bytes);
                    // the scores were written with ordinary stores by other CTAs: order them before the bulk copy's reads
                    asm volatile("fence.proxy.async.global;" ::: "memory");
                    bulk_load(smem_u32(keys), sc, bytes, bar);
                }
                ctl.tail_ok = w_ok ? 1 : 0;
            }
            named_barrier(kBarTail, kMTailThreads);
            if (!ctl.tail_ok) { ok = false; break; }
            if (!mbar_wait(smem_u32(&ctl.sfull), static_cast<uint32_t>(s) & 1u, abort_flag)) { ok = false; }
            // (every tail thread waits by itself; a thread that gave up has raised the abort flag, which the
            //  others see in their own wait)
            named_barrier(kBarTail, kMTailThreads);
            if (ctl.abort_flag) { ok = false; break; }
            const float* row2 = p.kv_shift ? reinterpret_cast<const float*>(keys) + p.Cpad : nullptr;
            const int last_kept = tail_select(row2, p.C, p.Cpad, p.k, keys, hist, sel, ctl, tt);
            const int n_tok = kk * C_STATIC - ((last_kept && kk > 0) ? (C_STATIC - tail_rows) : 0);
            // ---- this layer and the layers after it that reuse its indices
            int lj = li;
            do {
                const ModelLayer& ly = p.layer[lj];
                if (q == 0) {        // one CTA per head writes the kept positions
                    int32_t* dst = ly.out_idx + static_cast<size_t>(hkv) * p.n_max;
                    for (int r = tt; r < kk; r += kMTailThreads) {
                        const int j0 = sel[r] * C_STATIC, n0 = r * C_STATIC;
#pragma unroll
                        for (int t = 0; t < C_STATIC; ++t)
                            if (n0 + t < n_tok) dst[n0 + t] = j0 + t;
                    }
                    for (int i = tt; i < p.w; i += kMTailThreads) dst[n_tok + i] = p.P + i;
                    for (int i = n_tok + p.w + tt; i < p.n_max; i += kMTailThreads) dst[i] = -1;
                    // rows past the kept ones (only when the clipped last chunk is kept) are zero rows
                    const int vpr = p.d >> 3;
                    uint4* zk = ly.out_K + (static_cast<size_t>(hkv) * p.n_max + n_tok + p.w) * vpr;
                    uint4* zv = ly.out_V + (static_cast<size_t>(hkv) * p.n_max + n_tok + p.w) * vpr;
                    const int nz = (p.n_max - n_tok - p.w) * vpr;
                    for (int i = tt; i < nz; i += kMTailThreads) { zk[i] = make_uint4(0, 0, 0, 0); zv[i] = make_uint4(0, 0, 0, 0); }
                }
                // ---- this CTA's units: whole chunks (and window pieces) through the staging slots
                if (tt == 0) {
                    const char* Kh = reinterpret_cast<const char*>(ly.K) + static_cast<size_t>(hkv) * p.L * row_bytes;
                    const char* Vh = reinterpret_cast<const char*>(ly.V) + static_cast<size_t>(hkv) * p.L * row_bytes;
                    char* oK = reinterpret_cast<char*>(ly.out_K) + static_cast<size_t>(hkv) * p.n_max * row_bytes;
                    char* oV = reinterpret_cast<char*>(ly.out_V) + static_cast<size_t>(hkv) * p.n_max * row_bytes;
                    const uint32_t half_slot = static_cast<uint32_t>(p.stage_slot_bytes) / 2u;
                    auto unit = [&](int u, int& src_row, int& dst_row, int& rows) {
                        if (u < kk) {
                            src_row = sel[u] * C_STATIC;
                            dst_row = u * C_STATIC;
                            rows = min(C_STATIC, p.P - src_row);
                        } else {
                            const int j = u - kk;
                            src_row = p.P + j * C_STATIC;
                            dst_row = n_tok + j * C_STATIC;
                            rows = min(C_STATIC, p.L - src_row);
                        }
                    };
                    const int n_units = u_end - u_begin;
                    // loads run kMSlots - 1 units ahead of the stores
                    int loaded = 0;
                    auto issue_load = [&](int idx) {
                        int sr, dr, rows;
                        unit(u_begin + idx, sr, dr, rows);
                        const uint32_t slot = (g_issued + idx) % kMSlots;
                        const uint32_t bytes = static_cast<uint32_t>(rows) * row_bytes;
                        const uint32_t bar = smem_u32(&ctl.gfull[slot]);
                        mbar_arrive_expect_tx(bar, 2u * bytes);
                        bulk_load(stage0 + slot * p.stage_slot_bytes, Kh + static_cast<size_t>(sr) * row_bytes, bytes, bar);
                        bulk_load(stage0 + slot * p.stage_slot_bytes + half_slot, Vh + static_cast<size_t>(sr) * row_bytes, bytes, bar);
                    };
                    for (; loaded < n_units && loaded < kMSlots - 1; ++loaded) issue_load(loaded);
                    bool c_ok = true;
                    for (int idx = 0; idx < n_units && c_ok; ++idx) {
                        const uint32_t gi = g_issued + idx;
                        const uint32_t slot = gi % kMSlots;
                        c_ok = mbar_wait(smem_u32(&ctl.gfull[slot]), (gi / kMSlots) & 1u, abort_flag);
                        if (!c_ok) break;
                        int sr, dr, rows;
                        unit(u_begin + idx, sr, dr, rows);
                        const uint32_t bytes = static_cast<uint32_t>(rows) * row_bytes;
                        bulk_store(oK + static_cast<size_t>(dr) * row_bytes, stage0 + slot * p.stage_slot_bytes, bytes);
                        bulk_store(oV + static_cast<size_t>(dr) * row_bytes, stage0 + slot * p.stage_slot_bytes + half_slot, bytes);
                        bulk_commit();
                        if (loaded < n_units) {
                            // the slot the next load takes was stored one unit ago: all but the newest group have been read
                            bulk_wait_read<1>();
                            issue_load(loaded);
                            ++loaded;
                        }
                    }
                    bulk_wait_read<0>();          // the slots are reused by the next layer's first loads
                    g_issued += static_cast<uint32_t>(n_units);
                    ctl.tail_ok = c_ok ? 1 : 0;
                }
                named_barrier(kBarTail, kMTailThreads);
                if (!ctl.tail_ok) { ok = false; break; }
                ++lj;
            } while (lj < p.n_layers && !p.layer[lj].computes);
            li = lj;
        }
        if (tt == 0) bulk_wait_all();
        if (!ok && tt == 0) ctl.abort_flag = 1;
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
    if (threadIdx.x == 0) {
        if (ctl.abort_flag) atomicExch(p.status, 1);
        const unsigned old = atomicAdd(p.exits, 1u);
        if (old + 1u == gridDim.x) {
            for (int h = 0; h < p.Hs; ++h) { p.cnt_a[h] = 0u; p.cnt_b[h] = 0u; }
            *p.exits = 0u;
            __threadfence();
        }
    }
}

}  // namespace

bool make_model_plan(int L, int Rs, int Hs, int kv_shift, int d, int c, int C, int k, int max_ctas, int smem_limit,
                     ModelPlan* plan) {
    if (c != 10 && c != 20) return false;
    if (Rs < 1 || Rs > 128 || (d != 64 && d != 128) || L < 1 || C < 1 || k < 1 || Hs < 1 || Hs > kResidentMaxHeads)
        return false;
    if (max_ctas < Hs) return false;
    ModelPlan p{};
    p.c_static = c;
    p.cph = max_ctas / Hs;
    p.grid = p.cph * Hs;
    p.n_tiles = (L + kRTile - 1) / kRTile;
    p.t_max = (p.n_tiles + p.cph - 1) / p.cph;
    if (p.t_max * (kRTile / c) > kRPartCols) return false;
    const int KB = d / 64;
    const int q_bytes = KB * kRQTileBytes;
    const int pmax_bytes = p.t_max * 2 * 128 * 4;
    const int kk = k < C ? k : C;
    p.stage_slot_bytes = 2 * c * d * 2;                        // K rows and V rows of one chunk
    const int cpad = (C + 3) & ~3;
    const int tail_bytes = 8192 + (((cpad * 4 << kv_shift) + 127) & ~127) + ((kk * 4 + 127) & ~127) +
                           kMSlots * p.stage_slot_bytes + 128;
    const int fixed = 1024 + q_bytes + 1024 + pmax_bytes + kMMiscBytes + tail_bytes;
    int ns = (smem_limit - 512 - fixed) / kRStageBytes;           // (the control block is larger than the layer kernel's)
    if (ns > kRMaxStages) ns = kRMaxStages;
    if (ns < 2 * KB + 1) return false;
    p.n_stages = ns;
    p.off_ring = q_bytes;
    p.off_pmax = p.off_ring + ns * kRStageBytes + 1024;
    p.off_misc = p.off_pmax + pmax_bytes;
    p.off_tail = p.off_misc + kMMiscBytes;
    p.smem_bytes = 1024 + p.off_tail + tail_bytes;
    *plan = p;
    return true;
}

size_t model_scratch_floats(const ModelPlan& plan, int Hs, int C, int n_compute) {
    return static_cast<size_t>(2) * plan.grid * 256 + static_cast<size_t>(n_compute) * Hs * ((C + 3) & ~3) + 64;
}

cudaError_t launch_model(const ModelPlan& plan, const ModelIO& io, const CUtensorMap* tm_q, const CUtensorMap* tm_k,
                         const ModelLayerIO* layers, int n_layers, cudaStream_t stream) {
    ModelParams* pp = new ModelParams();        // too large for the host stack frame of every caller; copied at launch
    ModelParams& p = *pp;
    int n_compute = 0;
    for (int i = 0; i < n_layers; ++i) {
        ModelLayer& ly = p.layer[i];
        ly.K = static_cast<const uint4*>(layers[i].K);
        ly.V = static_cast<const uint4*>(layers[i].V);
        ly.out_K = static_cast<uint4*>(layers[i].out_K);
        ly.out_V = static_cast<uint4*>(layers[i].out_V);
        ly.out_idx = layers[i].out_idx;
        ly.computes = layers[i].computes ? 1 : 0;
        if (ly.computes) {
            p.tm_q[n_compute] = tm_q[n_compute];
            p.tm_k[n_compute] = tm_k[n_compute];
            ++n_compute;
        }
        ly.slot = n_compute - 1;
    }
    p.n_layers = n_layers;
    p.n_compute = n_compute;
    p.L = io.L; p.P = io.L - io.w; p.w = io.w; p.R = io.Rs; p.Hs = io.Hs; p.d = io.d; p.kv_shift = io.kv_shift;
    p.sl2 = io.sl2;
    p.cph = plan.cph; p.n_tiles = plan.n_tiles; p.n_stages = plan.n_stages;
    p.q_box_rows = io.Rs < 128 ? io.Rs : 128;
    p.k_box_rows = io.L < kRTile ? io.L : kRTile;
    p.C = io.C; p.k = io.k; p.n_max = io.n_max; p.Hkv = io.Hs >> io.kv_shift;
    p.Cpad = (io.C + 3) & ~3;
    p.off_ring = plan.off_ring; p.off_pmax = plan.off_pmax; p.off_misc = plan.off_misc; p.off_tail = plan.off_tail;
    p.stage_slot_bytes = plan.stage_slot_bytes;
    p.cta_stat = io.scratch;
    p.scores = io.scratch + static_cast<size_t>(2) * plan.grid * 256;
    p.exits = io.counters;
    p.cnt_a = io.counters + 16;
    p.cnt_b = io.counters + 16 + kResidentMaxHeads;
    p.status = io.status;
    const void* kern = plan.c_static == 10 ? reinterpret_cast<const void*>(model_kernel<10>)
                                           : reinterpret_cast<const void*>(model_kernel<20>);
    static int smem_set[2][64] = {{0}};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    const int v = plan.c_static == 10 ? 0 : 1;
    if (e == cudaSuccess && (dev < 0 || dev >= 64 || smem_set[v][dev] < plan.smem_bytes)) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, plan.smem_bytes);
        if (e == cudaSuccess && dev >= 0 && dev < 64) smem_set[v][dev] = plan.smem_bytes;
    }
    if (e == cudaSuccess) {
        void* params[] = {&p};
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(plan.grid);
        cfg.blockDim = dim3(kMThreads);
        cfg.dynamicSmemBytes = static_cast<size_t>(plan.smem_bytes);
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeCooperative;      // the CTAs of a head wait for one another: all must be resident
        attr[0].val.cooperative = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        e = cudaLaunchKernelExC(&cfg, kern, params);
    }
    delete pp;
    return e;
}

}  // namespace chunkkv
