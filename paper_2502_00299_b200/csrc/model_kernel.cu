// Many layers in one launch (ChunkKV Algorithm 2: "for l = 0 .. N_layers - 1", with Algorithm 3 per
// computed layer): a persistent version of the layer kernel of layer_resident.cu in which the
// steps of successive layers overlap inside every CTA.
//
// A CTA belongs to one scoring head and one key range for the whole launch. Its warps have roles:
//   warp 0         TMA producer: streams the Q tile and the CTA's K tiles of layer after layer
//                  through the shared-memory ring, as far ahead as the ring allows
//   warp 1         tcgen05.mma issuer
//   warps 2..17    epilogue, four groups of four warps: one exponential per score element, chunk sums
//                  into a ring of tensor-memory columns that holds more than one layer; at the end
//                  of a layer a group leaves its per-row (max, sum) in shared memory and goes straight
//                  on with the next layer; when the head's row statistics have arrived (normally long
//                  before they are needed) it contracts the partial sums it wrote itself over the rows
//                  into chunk scores of the CTA's key range (global memory)
//   warp 18        one thread: for each computed layer, once a selector CTA has published the head's
//                  kept-chunk list, moves this CTA's share of the kept K/V rows with bulk asynchronous
//                  copies (global -> shared -> global, whole chunks at a time) - for the computed
//                  layer and for every following layer that reuses its indices
//   warp 19        row statistics: merges the groups' records, stores and announces the CTA's record,
//                  waits (bounded) for the head's other CTAs, merges their records into m_i and 1 / l_i
//                  for the contraction, and announces the CTA's chunk scores when they are stored
// The CTAs after the scoring CTAs are selectors: exact top-k per head, out_idx, kept-chunk lists.
//
// So while the selectors and copy threads work on layer l, the other warps already score layer l + 1:
// the latency-bound steps cost no memory bandwidth and the copies ride along with the K stream.
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

constexpr int kMThreads = 640;          // warp 0: TMA, warp 1: UMMA issue, warps 2..17: epilogue, warp 18: row copies, warp 19: row statistics
                                        // (five warps per scheduler: a sixth would cut every thread to 80 registers)
constexpr int kMMiscBytes = 18432;      // epilogue: group records (two slots), m_i, 1 / l_i, row sums per lane quarter
constexpr int kMSlots = 8;              // staging slots of the row copies
// Tensor memory: three 64-column accumulators (one 60-key panel of a tile each, in rotation; the
// second panel of a tile is computed on keys 56 .. 119 so that its operand starts on a swizzle-atom
// boundary, and begins at column 4), and 320 columns of chunk partial sums: a ring that holds one
// layer and two thirds of the next at c = 10, so the statistics of a layer have most of the next
// layer's scoring time to travel before its contraction needs them.
constexpr int kMAccN = 64;
constexpr int kMAccBufs = 3;
constexpr int kMAccSlots = 12;                     // (buffer, epilogue group) pairs: lcm(3 buffers, 4 groups)
constexpr int kMAcc1Row = 56;
constexpr int kMPartCol0 = kMAccBufs * kMAccN;
constexpr int kMPartCols = 512 - kMPartCol0;
// Ring sizes are multiples of the four epilogue groups: a panel's ring slot is its number (since the
// start of the launch) modulo the ring size and its group is that number modulo 4, so a ring slot
// is only ever reused by the group that wrote and contracted its previous contents.
constexpr int kMRingPanels10 = kMPartCols / 6 / 4 * 4;   // c = 10: 6 chunk columns per panel
constexpr int kMRingPanels20 = 84;                       // c = 20: 3 per panel; more would only cost shared memory
static_assert(kMRingPanels10 % 4 == 0 && kMRingPanels20 % 4 == 0 && kMRingPanels20 * 3 <= kMPartCols, "ring sizes");
constexpr int kBarGroup = 2;                       // named barriers 2 .. 5: the four warps of an epilogue group

struct ModelCtl {
    unsigned long long full[kRMaxStages];
    unsigned long long empty[kRMaxStages];
    unsigned long long tfull[kMAccSlots];      // by panel number modulo 12: one (accumulator, epilogue group) pair each
    unsigned long long tempty[kMAccSlots];
    unsigned long long qfull;
    unsigned long long qempty;
    unsigned long long gfull[kMSlots];
    unsigned long long sfull;          // a kept-chunk list has landed in shared memory (copy thread)
    unsigned long long stat_full[2];   // m_i and 1 / l_i of a slot are in shared memory (statistics warps -> epilogue)
    unsigned long long pub_done[2];    // every epilogue warp has stored its part of the slot's record (-> statistics warp)
    unsigned long long sc_done[2];     // every epilogue warp has stored its chunk scores of the slot (-> statistics warp)
    uint32_t tmem_base;
    int abort_flag;
    int sel_flag[2];                   // selector CTAs: wait result, abort flag
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
    int n_score, n_sel;    // scoring CTAs (Hs * cph) and selector CTAs (the rest of the grid)
    int sel_row_bytes;     // bytes of one kept-chunk list: 4 header ints + the kept chunk ids, padded to 16 bytes
    int sel_keys_fit;      // selector: the keys of a head fit its shared memory (many chunks per thread)
    int off_ring, off_pmax, off_misc, off_tail, stage_slot_bytes;
    // bytes between consecutive rows of a head and between heads of K and of V (packed: d * 2 and L * d * 2)
    long long k_row_bytes, k_head_bytes, v_row_bytes, v_head_bytes;
    float* cta_stat;       // [2 (slot parity)][grid][{max, sum}][128]
    float* scores;         // [n_compute][Hs][Cpad]
    unsigned* cnt_a;       // [Hs]
    unsigned* cnt_b;       // [Hs]   chunk scores of a slot announced by the scoring CTAs
    unsigned* cnt_c;       // [Hkv]  kept-chunk lists announced by the selector CTAs
    int* sel_rows;         // [n_compute][Hkv][sel_row_bytes / 4]
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

// Fold N (max, sum-of-exp2) records into (M, S), one row each of four rows at a time: the new maximum
// first, then N independent exponentials (a short dependency chain, unlike N merges in sequence).
template <int N>
__device__ __forceinline__ void merge_batch(float (&M)[4], float (&S)[4], const float4 (&m)[N], const float4 (&l)[N], int n) {
    const float ninf = -CUDART_INF_F;
    float nm[4] = {M[0], M[1], M[2], M[3]};
#pragma unroll
    for (int j = 0; j < N; ++j)
        if (j < n) {
            nm[0] = fmaxf(nm[0], m[j].x);
            nm[1] = fmaxf(nm[1], m[j].y);
            nm[2] = fmaxf(nm[2], m[j].z);
            nm[3] = fmaxf(nm[3], m[j].w);
        }
#pragma unroll
    for (int r = 0; r < 4; ++r) S[r] = (M[r] == ninf) ? 0.f : S[r] * ex2_approx(M[r] - nm[r]);
#pragma unroll
    for (int j = 0; j < N; ++j)
        if (j < n) {
            S[0] += (m[j].x == ninf) ? 0.f : l[j].x * ex2_approx(m[j].x - nm[0]);
            S[1] += (m[j].y == ninf) ? 0.f : l[j].y * ex2_approx(m[j].y - nm[1]);
            S[2] += (m[j].z == ninf) ? 0.f : l[j].z * ex2_approx(m[j].z - nm[2]);
            S[3] += (m[j].w == ninf) ? 0.f : l[j].w * ex2_approx(m[j].w - nm[3]);
        }
#pragma unroll
    for (int r = 0; r < 4; ++r) M[r] = nm[r];
}

// Bounded wait of a whole warp on a counter that only grows: every lane performs the acquire load, so
// each lane's later loads are ordered behind the arrivals it has seen. Lane 0 keeps the time limit.
__device__ __forceinline__ bool wait_counter_warp(const unsigned* counter, unsigned target, volatile int* abort_flag) {
    const long long t0 = clock64();
    for (;;) {
        unsigned cur;
        asm volatile("ld.acquire.gpu.u32 %0, [%1];" : "=r"(cur) : "l"(counter) : "memory");
        if (__all_sync(0xffffffffu, cur >= target)) return true;
        int bad = 0;
        if ((threadIdx.x & 31) == 0) {
            if (*abort_flag) bad = 1;
            else if (clock64() - t0 > kWaitLimitClocks) { *abort_flag = 1; bad = 1; }
        }
        if (__shfl_sync(0xffffffffu, bad, 0)) return false;
    }
}

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

// Selector CTA (the CTAs after the scoring CTAs; they run on SMs the scoring grid leaves free): for
// every slot and each of its KV heads, once the head's chunk scores are complete, the whole CTA
// runs the exact top-k (select.cuh), writes the kept positions to out_idx of the computed layer
// and of every layer that reuses its indices (and zero rows behind the kept rows, which exist
// only when the clipped last chunk is kept), publishes the kept-chunk list for the scoring CTAs'
// copy threads and announces it on the head's third counter.
template <int C_STATIC>
__device__ __forceinline__ bool selector_loop(const ModelParams& p, uint8_t* dyn, int* flag_smem) {
    SelectSmem& ss = *reinterpret_cast<SelectSmem*>(dyn);
    constexpr size_t kSelBytes = (sizeof(SelectSmem) + 127) & ~size_t(127);
    int32_t* sidx = reinterpret_cast<int32_t*>(dyn + kSelBytes);                  // [n_max] kept positions
    const size_t idx_bytes = (static_cast<size_t>(p.n_max) * 4 + 127) & ~size_t(127);
    uint32_t* kbuf = reinterpret_cast<uint32_t*>(dyn + kSelBytes + idx_bytes);    // keys, when there are many chunks per thread
    const int sid = static_cast<int>(blockIdx.x) - p.n_score;
    const int kk = min(p.k, p.C);
    const int tail_rows = (p.C > 0) ? (p.P - (p.C - 1) * C_STATIC) : 0;
    const int row_ints = p.sel_row_bytes / 4;
    volatile int* flag = flag_smem;
    for (int li = 0; li < p.n_layers;) {
        const int s = p.layer[li].slot;
        int lj_end = li + 1;
        while (lj_end < p.n_layers && !p.layer[lj_end].computes) ++lj_end;
        for (int hkv = sid; hkv < p.Hkv; hkv += p.n_sel) {
            if (threadIdx.x == 0) {
                const unsigned target = static_cast<unsigned>(s + 1) * p.cph;
                bool w_ok = wait_counter(p.cnt_b + (hkv << p.kv_shift), target, flag + 1, 100);
                if (w_ok && p.kv_shift) w_ok = wait_counter(p.cnt_b + (hkv << p.kv_shift) + 1, target, flag + 1, 100);
                asm volatile("fence.acq_rel.gpu;" ::: "memory");
                flag[0] = w_ok ? 1 : 0;
            }
            __syncthreads();
            if (!flag[0]) return false;
            const float* sc = p.scores + (static_cast<size_t>(s) * p.Hs + (hkv << p.kv_shift)) * p.Cpad;
            const float* sc2 = p.kv_shift ? sc + p.Cpad : nullptr;
            if (p.C <= kMThreads * 8)
                select_head_regs<8>(sc, sc2, p.L, p.w, C_STATIC, p.C, p.k, p.n_max, sidx, ss);
            else
{
                if (p.sel_keys_fit)
                    select_head_smem(sc, sc2, p.L, p.w, C_STATIC, p.C, p.k, p.n_max, sidx, ss, kbuf);
                else
                    select_head_rows(sc, sc2, p.L, p.w, C_STATIC, p.C, p.k, p.n_max, sidx, ss, nullptr);
            }
            const int n_tok = kk * C_STATIC - ((ss.last_kept && kk > 0) ? (C_STATIC - tail_rows) : 0);
            // the kept-chunk list for the copy threads: [n_tok, -, -, -, chunk ids]
            int* row = p.sel_rows + (static_cast<size_t>(s) * p.Hkv + hkv) * row_ints;
            if (threadIdx.x == 0) row[0] = n_tok;
            for (int r = threadIdx.x; r < kk; r += kMThreads) row[4 + r] = ss.sel[r];
            const int vpr = p.d >> 3;
            for (int lj = li; lj < lj_end; ++lj) {
                const ModelLayer& ly = p.layer[lj];
                int32_t* dst = ly.out_idx + static_cast<size_t>(hkv) * p.n_max;
                for (int n = threadIdx.x; n < p.n_max; n += kMThreads) dst[n] = sidx[n];
                uint4* zk = ly.out_K + (static_cast<size_t>(hkv) * p.n_max + n_tok + p.w) * vpr;
                uint4* zv = ly.out_V + (static_cast<size_t>(hkv) * p.n_max + n_tok + p.w) * vpr;
                const int nz = (p.n_max - n_tok - p.w) * vpr;
                for (int i = threadIdx.x; i < nz; i += kMThreads) { zk[i] = make_uint4(0, 0, 0, 0); zv[i] = make_uint4(0, 0, 0, 0); }
            }
            __syncthreads();
            if (threadIdx.x == 0) {
                unsigned old;   // release: the list and the positions written above are visible to whoever sees the count
                asm volatile("atom.add.release.gpu.u32 %0, [%1], 1;" : "=r"(old) : "l"(p.cnt_c + hkv) : "memory");
            }
        }
        li = lj_end;
    }
    return true;
}

// STRIDED: the rows of a head are not adjacent in memory (e.g. token-major caches): the copy thread moves
// kept rows one at a time. A variant of its own, so that the packed kernel's code is exactly what it was.
template <int C_STATIC, bool STRIDED>
__global__ void __launch_bounds__(kMThreads, 1)
model_kernel(const __grid_constant__ ModelParams p) {
    constexpr int SPP = kRPanel / C_STATIC;
    constexpr uint32_t IDESC = umma_idesc_bf16(128, kMAccN);

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
    float* rec = misc;                 // [4 groups][{max, sum}][128]; the odd slots' copy sits at misc + 3584
    float* gstat = misc + 1024;        // [2 (slot parity)][{m_i, 1 / l_i}][128]
    float* red = misc + 2304;          // [4 lane quarters][256 chunk slots]
    volatile int* abort_flag = &ctl.abort_flag;
    const uint32_t n_stages = static_cast<uint32_t>(p.n_stages);

    if (static_cast<int>(blockIdx.x) >= p.n_score) {
        // ------------------------------------------------------------------ selector CTA
        if (threadIdx.x == 0) { ctl.sel_flag[0] = 1; ctl.sel_flag[1] = 0; }
        __syncthreads();
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
        asm volatile("griddepcontrol.wait;" ::: "memory");
        const bool s_ok = selector_loop<C_STATIC>(p, dyn, ctl.sel_flag);
        __syncthreads();
        if (threadIdx.x == 0) {
            if (!s_ok) atomicExch(p.status, 1);
            const unsigned old = atomicAdd(p.exits, 1u);
            if (old + 1u == gridDim.x) {
                for (int h = 0; h < p.Hs; ++h) { p.cnt_a[h] = 0u; p.cnt_b[h] = 0u; }
                for (int h = 0; h < p.Hkv; ++h) p.cnt_c[h] = 0u;
                *p.exits = 0u;
                __threadfence();
            }
        }
        return;
    }
    const int hs = blockIdx.x / p.cph, part = blockIdx.x - hs * p.cph;
    const int hkv = hs >> p.kv_shift;
    // tiles are dealt out rounding up, so the head's last CTA - whose last panels take the slow, masked path -
    // is never one of those that get an extra tile
    const int t_begin = (p.n_tiles * part + p.cph - 1) / p.cph, t_end = (p.n_tiles * (part + 1) + p.cph - 1) / p.cph;
    const int nt = t_end - t_begin;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.n_stages; ++s) {
            mbar_init(smem_u32(&ctl.full[s]), 1);
            mbar_init(smem_u32(&ctl.empty[s]), 1);
        }
        for (int b = 0; b < kMAccSlots; ++b) {
            mbar_init(smem_u32(&ctl.tfull[b]), 1);
            mbar_init(smem_u32(&ctl.tempty[b]), 4);
        }
        mbar_init(smem_u32(&ctl.qfull), 1);
        mbar_init(smem_u32(&ctl.qempty), 1);
        for (int s = 0; s < kMSlots; ++s) mbar_init(smem_u32(&ctl.gfull[s]), 1);
        mbar_init(smem_u32(&ctl.sfull), 1);
        mbar_init(smem_u32(&ctl.stat_full[0]), 1);
        mbar_init(smem_u32(&ctl.stat_full[1]), 1);
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&ctl.pub_done[b]), 16);
            mbar_init(smem_u32(&ctl.sc_done[b]), 16);
        }
        ctl.abort_flag = 0;
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
            int tg = 0;                  // tiles issued so far (all layers); the epilogue pair tg & 1 reads tile tg
            bool ok = true;
            for (int s = 0; s < p.n_compute && ok; ++s) {
                ok = mbar_wait(smem_u32(&ctl.qfull), s & 1, abort_flag);
                for (int ti = 0; ti < nt && ok; ++ti, ++tg) {
                    uint32_t st_kb[2] = {0u, 0u};
#pragma unroll
                    for (int kb = 0; kb < 2; ++kb) {
                        if (kb >= KB || !ok) break;
                        ok = mbar_wait(smem_u32(&ctl.full[st]), st_par, abort_flag);
                        st_kb[kb] = st;
                        if (++st == n_stages) { st = 0; st_par ^= 1u; }
                    }
                    if (!ok) break;
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        // panel pc goes to accumulator pc % 3, which panel pc - 3 used last
                        const int pc = 2 * tg + half;
                        if (pc >= kMAccBufs) {
                            const int prev = pc - kMAccBufs;
                            ok = mbar_wait(smem_u32(&ctl.tempty[prev % kMAccSlots]), (prev / kMAccSlots) & 1, abort_flag);
                        }
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t d_addr = tmem_base + static_cast<uint32_t>((pc % kMAccBufs) * kMAccN);
#pragma unroll
                        for (int kb = 0; kb < 2; ++kb) {
                            if (kb >= KB) break;
                            const uint64_t b_desc =
                                umma_desc_sw128(k_base + st_kb[kb] * kRStageBytes + static_cast<uint32_t>(half * kMAcc1Row * 128));
                            const uint64_t a_desc = umma_desc_sw128(q_base + static_cast<uint32_t>(kb) * kRQTileBytes);
#pragma unroll
                            for (int k4 = 0; k4 < 4; ++k4)
                                umma_bf16(d_addr, a_desc + 2u * k4, b_desc + 2u * k4, IDESC, (kb > 0 || k4 > 0) ? 1u : 0u);
                        }
                        umma_commit(smem_u32(&ctl.tfull[pc % kMAccSlots]));
                    }
                    if (!ok) break;
#pragma unroll
                    for (int kb = 0; kb < 2; ++kb)
                        if (kb < KB) umma_commit(smem_u32(&ctl.empty[st_kb[kb]]));
                }
                if (ok) umma_commit(smem_u32(&ctl.qempty));       // every UMMA of this layer has read the Q tile
            }
        }
    } else if (warp < 18) {
        // ------------------------------------------------------------------ epilogue
        // The chunk partial sums and panel maxima of a layer live in rings (tensor-memory columns,
        // shared memory) that hold more than one layer's worth, so after its last tile of layer s a
        // thread only publishes the CTA's row records and goes straight on with the first `ahead`
        // tiles of layer s + 1; the chunk scores of layer s are formed after those, when the other
        // CTAs' records have long arrived and the statistics warp has merged them.
        const int grp = (warp - 2) >> 2, quarter = warp & 3;
        const int gt = threadIdx.x - 64 - grp * 128;    // 0 .. 127 within the group
        const int pair = grp >> 1, half = grp & 1;
        const int row = quarter * 32 + lane;
        const bool active = row < p.R;
        const int last_visible = p.P + (row % p.w);
        const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        const int n_pl = 2 * nt;
        constexpr int PR = (C_STATIC == 10) ? kMRingPanels10 : kMRingPanels20;     // panels in the rings
        const int ahead = max(0, min(nt, (PR - n_pl) / 2));   // tiles of the next layer scored before the contraction
        const int ch0 = t_begin * (kRTile / C_STATIC);
        bool ok = true;
        float run_m = -CUDART_INF_F, run_l = 0.f;
        // tiles [ti_lo, ti_hi) of slot s that belong to this thread's pair
        auto do_tiles = [&](int s, int ti_lo, int ti_hi) {
            if (!ok) return;
            const int tg0 = s * nt, pbase = (s * n_pl) % PR;
            for (int ti = ti_lo + ((pair - ((tg0 + ti_lo) & 1)) & 1); ti < ti_hi; ti += 2) {
                const int pc = 2 * (tg0 + ti) + half;        // panel number since the start of the launch
                const int aslot = pc % kMAccSlots;
                bool ready = true;
                if (lane == 0) ready = mbar_wait(smem_u32(&ctl.tfull[aslot]), (pc / kMAccSlots) & 1, abort_flag);
                if (!__shfl_sync(0xffffffffu, ready, 0)) { ok = false; break; }
                tc_fence_after();
                float v[kRPanel];
                load_panel<kRPanel>(lane_addr + static_cast<uint32_t>((pc % kMAccBufs) * kMAccN + half * (kRPanel - kMAcc1Row)), v);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctl.tempty[aslot]));
                const int pl = ti * 2 + half;
                int slot = pbase + pl;
                slot -= (slot >= PR) ? PR : 0;
                const int j0 = (t_begin + ti) * kRTile + half * kRPanel;
                float pr[SPP], m2, l;
                auto emit = [&](int ch, float acc) { pr[ch] = acc; };
                if (j0 + kRPanel <= p.P)
                    panel_fast<C_STATIC, kRPanel>(v, p.sl2, emit, &m2, &l);
                else
                    panel_static_tail<C_STATIC, kRPanel>(v, p.sl2, emit, j0, p.P, last_visible, &m2, &l);
                part_store<SPP>(lane_addr + static_cast<uint32_t>(kMPartCol0 + slot * SPP), pr);
                pmax[slot * 128 + row] = m2;
                const float nm = fmaxf(run_m, m2);
                const float s_old = (run_m == -CUDART_INF_F) ? 0.f : ex2_approx(run_m - nm);
                const float s_new = (m2 == -CUDART_INF_F) ? 0.f : ex2_approx(m2 - nm);
                run_l = run_l * s_old + l * s_new;
                run_m = nm;
            }
        };
        // end of slot s: this group's (max, sum) per row -> shared memory; the statistics warp merges the four
        // groups, stores the CTA's record and announces it (no block-wide barrier on the scoring warps' path)
        auto publish = [&](int s) {
            float* rc = rec + (s & 1) * 3584;
            rc[(grp * 2 + 0) * 128 + row] = active ? run_m : -CUDART_INF_F;
            rc[(grp * 2 + 1) * 128 + row] = active ? run_l : 0.f;
            run_m = -CUDART_INF_F;
            run_l = 0.f;
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl.pub_done[s & 1]));
        };
        // Chunk scores of slot s from the partial sums in the rings. A group contracts the panels it
        // scored itself - every thread reads back the tensor-memory columns and panel maxima it wrote -
        // so the only synchronisation is among the group's four warps (the four lane quarters of a sum).
        auto contract = [&](int s) -> bool {
            const int tg0 = s * nt, pbase = (s * n_pl) % PR;
            // first panel of the slot that this group scored; its others follow every fourth panel
            const int g1 = 2 * (((grp >> 1) - tg0) & 1) + half;
            bool ready = true;
            if (lane == 0) ready = mbar_wait(smem_u32(&ctl.stat_full[s & 1]), (s >> 1) & 1, abort_flag);
            if (!__shfl_sync(0xffffffffu, ready, 0)) ok = false;   // (the failed wait has raised the abort flag)
            tmem_st_wait();
            // the group's previous sums have been read by all its warps; and a uniform decision to go on
            if (named_barrier_or(kBarGroup + grp, 128, !ok || ctl.abort_flag != 0)) return false;
            const float* gm = gstat + (s & 1) * 256;
            const float mi = gm[row], li = gm[128 + row];
            constexpr int PPB = 30 / SPP;
            for (int b0 = 0; g1 + 4 * b0 < n_pl; b0 += PPB) {
                float v[32];
                int slot_of[PPB];
#pragma unroll
                for (int u = 0; u < PPB; ++u) {
                    const int pl = min(g1 + 4 * (b0 + u), n_pl - 1);
                    int slot = pbase + pl;
                    slot -= (slot >= PR) ? PR : 0;
                    slot_of[u] = slot;
                    part_load<SPP>(lane_addr + static_cast<uint32_t>(kMPartCol0 + slot * SPP), &v[u * SPP]);
                }
                tmem_ld_wait();
                v[30] = 0.f;
                v[31] = 0.f;
#pragma unroll
                for (int u = 0; u < PPB; ++u) {
                    const int pl = g1 + 4 * (b0 + u);
                    const bool have = active && pl < n_pl;
                    const float f = have ? ex2_approx(pmax[slot_of[u] * 128 + row] - mi) * li : 0.f;
#pragma unroll
                    for (int q = 0; q < SPP; ++q) v[u * SPP + q] = have ? v[u * SPP + q] * f : 0.f;
                }
                const float tot = warp_transpose_reduce(v, lane);
                const int pl = g1 + 4 * (b0 + lane / SPP);
                if (lane < 30 && pl < n_pl) red[quarter * 256 + pl * SPP + lane % SPP] = tot;
            }
            named_barrier(kBarGroup + grp, 128);
            float* sc_out = p.scores + (static_cast<size_t>(s) * p.Hs + hs) * p.Cpad;
            const int n_own = (n_pl - g1 + 3) / 4 * SPP;     // chunk slots of this group's panels
            for (int i = gt; i < n_own; i += 128) {
                const int lc = (g1 + 4 * (i / SPP)) * SPP + i % SPP;
                if (ch0 + lc < p.C) sc_out[ch0 + lc] = (red[lc] + red[256 + lc]) + (red[512 + lc] + red[768 + lc]);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl.sc_done[s & 1]));      // announced by the statistics warp
            return true;
        };
        for (int s = 0; s <= p.n_compute; ++s) {
            if (s < p.n_compute) do_tiles(s, 0, ahead);
            if (s > 0 && !contract(s - 1)) break;
            if (s < p.n_compute) {
                do_tiles(s, ahead, nt);
                publish(s);
            }
        }
        if (!ok && lane == 0) ctl.abort_flag = 1;
    } else if (warp == 19) {
        // ------------------------------------------------------------------ statistics warp
        // Per slot: merge the groups' records into the CTA's record, store and announce it, wait (bounded)
        // until every CTA of the scoring head has done the same, read their records from the L2, merge
        // them into m_i and 1 / l_i - four rows per lane - and hand the result to the epilogue; then
        // announce the CTA's chunk scores once the epilogue has stored them.
        const int r0 = 4 * lane;
        bool ok = true;
        for (int s = 0; s < p.n_compute && ok; ++s) {
            bool w_ok = true;
            if (lane == 0)
                w_ok = mbar_wait(smem_u32(&ctl.pub_done[s & 1]), static_cast<uint32_t>(s >> 1) & 1u, abort_flag);
            if (!__shfl_sync(0xffffffffu, w_ok, 0)) break;
            {
                // every epilogue warp has left its group's (max, sum) per row in shared memory: merge the
                // four groups (this lane: rows 4 lane .. 4 lane + 3), store the CTA's record and announce it.
                // release: the record stores of the whole warp, ordered by __syncwarp, are visible to whoever
                // sees the count
                const float* rc = rec + (s & 1) * 3584;
                float Mo[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F}, So[4] = {0.f, 0.f, 0.f, 0.f};
                float4 m[4], l[4];
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    m[g] = *reinterpret_cast<const float4*>(rc + (g * 2) * 128 + r0);
                    l[g] = *reinterpret_cast<const float4*>(rc + (g * 2 + 1) * 128 + r0);
                }
                merge_batch<4>(Mo, So, m, l, 4);
                float* dst = p.cta_stat + (static_cast<size_t>(s & 1) * gridDim.x + blockIdx.x) * 256;
                *reinterpret_cast<float4*>(dst + r0) = make_float4(Mo[0], Mo[1], Mo[2], Mo[3]);
                *reinterpret_cast<float4*>(dst + 128 + r0) = make_float4(So[0], So[1], So[2], So[3]);
                __syncwarp();
            }
            if (lane == 0) asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p.cnt_a + hs) : "memory");
            if (!wait_counter_warp(p.cnt_a + hs, static_cast<unsigned>(s + 1) * p.cph, abort_flag)) break;
            const float* src = p.cta_stat + (static_cast<size_t>(s & 1) * gridDim.x + static_cast<size_t>(hs) * p.cph) * 256;
            float M[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F}, S[4] = {0.f, 0.f, 0.f, 0.f};
            // the head's records straight from the L2 (they were written by other SMs; every lane has
            // acquired the counter), six CTAs' worth of loads in flight per lane
            for (int j0 = 0; j0 < p.cph; j0 += 6) {
                float4 m[6], l[6];
#pragma unroll
                for (int j = 0; j < 6; ++j) {
                    const int jj = min(j0 + j, p.cph - 1);
                    m[j] = __ldcg(reinterpret_cast<const float4*>(src + static_cast<size_t>(jj) * 256 + r0));
                    l[j] = __ldcg(reinterpret_cast<const float4*>(src + static_cast<size_t>(jj) * 256 + 128 + r0));
                }
                merge_batch<6>(M, S, m, l, p.cph - j0);
            }
            if (!ok) break;
            float* gm = gstat + (s & 1) * 256;
            *reinterpret_cast<float4*>(gm + r0) = make_float4(M[0], M[1], M[2], M[3]);
            *reinterpret_cast<float4*>(gm + 128 + r0) = make_float4(1.0f / S[0], 1.0f / S[1], 1.0f / S[2], 1.0f / S[3]);
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(smem_u32(&ctl.stat_full[s & 1]));
                // the epilogue forms the slot's chunk scores next; announce them when they are stored
                if (mbar_wait(smem_u32(&ctl.sc_done[s & 1]), static_cast<uint32_t>(s >> 1) & 1u, abort_flag))
                    asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p.cnt_b + hs) : "memory");
                else
                    ok = false;
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
        }
    } else if (warp == 18) {
        // ------------------------------------------------------------------ tail: row copies
        // One thread: waits until the selector CTA has published the head's kept-chunk list of a
        // slot, fetches the list, and moves this CTA's share of the rows - whole chunks and window
        // pieces - through the staging slots with bulk copies, for the computed layer and for every
        // layer that reuses its indices. (Strided variant: the whole warp runs this loop in step - lane 0 waits,
        // stores and keeps the books, every lane issues the copy of one source row.)
        if (STRIDED || lane == 0) {
            uint8_t* tbase = dyn + p.off_tail;
            int* row = reinterpret_cast<int*>(tbase);        // [4 + kkpad]: n_tok, -, -, -, kept chunk ids
            const uint32_t stage0 = smem_u32(tbase + p.sel_row_bytes);
            const int* sel = row + 4;
            const int Q = p.cph << p.kv_shift;               // CTAs of this KV head
            const int q = static_cast<int>(blockIdx.x) - (hkv << p.kv_shift) * p.cph;
            const int kk = min(p.k, p.C);
            const int wu = (p.w + C_STATIC - 1) / C_STATIC;  // the window as pseudo-chunks of up to c rows
            const int U = kk + wu;                           // copy units of the head
            const int u_begin = static_cast<int>(static_cast<long long>(U) * q / Q);
            const int u_end = static_cast<int>(static_cast<long long>(U) * (q + 1) / Q);
            const int n_units = u_end - u_begin;
            const uint32_t row_bytes = static_cast<uint32_t>(p.d) * 2u;
            const uint32_t half_slot = static_cast<uint32_t>(p.stage_slot_bytes) / 2u;
            uint32_t g_issued = 0;                           // units loaded so far (all layers): slot = g % kMSlots
            bool ok = true;
            for (int li = 0; li < p.n_layers && ok;) {
                const int s = p.layer[li].slot;
                if (lane == 0) {
                    ok = wait_counter(p.cnt_c + hkv, static_cast<unsigned>(s + 1), abort_flag, 200);
                    if (ok) {
                        asm volatile("fence.acq_rel.gpu;" ::: "memory");
                        const uint32_t bar = smem_u32(&ctl.sfull);
                        mbar_arrive_expect_tx(bar, static_cast<uint32_t>(p.sel_row_bytes));
                        // the list was written with ordinary stores by the selector CTA
                        asm volatile("fence.proxy.async.global;" ::: "memory");
                        bulk_load(smem_u32(row), p.sel_rows + (static_cast<size_t>(s) * p.Hkv + hkv) * (p.sel_row_bytes / 4),
                                  static_cast<uint32_t>(p.sel_row_bytes), bar);
                    }
                }
                if constexpr (STRIDED) ok = __shfl_sync(0xffffffffu, ok, 0);
                // (every lane that reads the list waits for it itself)
                if (ok) ok = mbar_wait(smem_u32(&ctl.sfull), static_cast<uint32_t>(s) & 1u, abort_flag);
                if constexpr (STRIDED) ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                const int n_tok = row[0];
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
                int lj = li;
                do {
                    const ModelLayer& ly = p.layer[lj];
                    const char* Kh = reinterpret_cast<const char*>(ly.K) +
                                     (STRIDED ? static_cast<size_t>(hkv) * p.k_head_bytes : static_cast<size_t>(hkv) * p.L * row_bytes);
                    const char* Vh = reinterpret_cast<const char*>(ly.V) +
                                     (STRIDED ? static_cast<size_t>(hkv) * p.v_head_bytes : static_cast<size_t>(hkv) * p.L * row_bytes);
                    char* oK = reinterpret_cast<char*>(ly.out_K) + static_cast<size_t>(hkv) * p.n_max * row_bytes;
                    char* oV = reinterpret_cast<char*>(ly.out_V) + static_cast<size_t>(hkv) * p.n_max * row_bytes;
                    int loaded = 0;
                    auto issue_load = [&](int idx) {
                        int sr, dr, rows;
                        unit(u_begin + idx, sr, dr, rows);
                        const uint32_t slot = (g_issued + idx) % kMSlots;
                        const uint32_t bytes = static_cast<uint32_t>(rows) * row_bytes;
                        const uint32_t bar = smem_u32(&ctl.gfull[slot]);
                        if (lane == 0) mbar_arrive_expect_tx(bar, 2u * bytes);
                        if constexpr (!STRIDED) {
                            bulk_load(stage0 + slot * p.stage_slot_bytes, Kh + static_cast<size_t>(sr) * row_bytes, bytes, bar);
                            bulk_load(stage0 + slot * p.stage_slot_bytes + half_slot, Vh + static_cast<size_t>(sr) * row_bytes, bytes, bar);
                        } else {
                            // rows of a chunk are not adjacent in memory (e.g. a token-major cache): lane r copies row r
                            __syncwarp();             // the byte count is on the barrier before any copy can complete
                            if (lane < rows) {
                                bulk_load(stage0 + slot * p.stage_slot_bytes + static_cast<uint32_t>(lane) * row_bytes,
                                          Kh + static_cast<size_t>(sr + lane) * p.k_row_bytes, row_bytes, bar);
                                bulk_load(stage0 + slot * p.stage_slot_bytes + half_slot + static_cast<uint32_t>(lane) * row_bytes,
                                          Vh + static_cast<size_t>(sr + lane) * p.v_row_bytes, row_bytes, bar);
                            }
                        }
                    };
                    // loads run kMSlots - 1 units ahead of the stores
                    for (; loaded < n_units && loaded < kMSlots - 1; ++loaded) issue_load(loaded);
                    for (int idx = 0; idx < n_units && ok; ++idx) {
                        const uint32_t gi = g_issued + idx;
                        const uint32_t slot = gi % kMSlots;
                        if (lane == 0) ok = mbar_wait(smem_u32(&ctl.gfull[slot]), (gi / kMSlots) & 1u, abort_flag);
                        if constexpr (STRIDED) ok = __shfl_sync(0xffffffffu, ok, 0);
                        if (!ok) break;
                        int sr, dr, rows;
                        unit(u_begin + idx, sr, dr, rows);
                        const uint32_t bytes = static_cast<uint32_t>(rows) * row_bytes;
                        if (lane == 0) {
                            bulk_store(oK + static_cast<size_t>(dr) * row_bytes, stage0 + slot * p.stage_slot_bytes, bytes);
                            bulk_store(oV + static_cast<size_t>(dr) * row_bytes, stage0 + slot * p.stage_slot_bytes + half_slot, bytes);
                            bulk_commit();
                        }
                        if (loaded < n_units) {
                            // the slot the next load takes was stored one unit ago: all but the newest group have been read
                            if (lane == 0) bulk_wait_read<1>();
                            if constexpr (STRIDED) __syncwarp();
                            issue_load(loaded);
                            ++loaded;
                        }
                    }
                    if (lane == 0) bulk_wait_read<0>();          // the slots are reused by the next layer's first loads
                    if constexpr (STRIDED) __syncwarp();
                    g_issued += static_cast<uint32_t>(n_units);
                    ++lj;
                } while (ok && lj < p.n_layers && !p.layer[lj].computes);
                li = lj;
            }
            if (lane == 0) bulk_wait_all();
            if (!ok && lane == 0) ctl.abort_flag = 1;
        }
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
            for (int h = 0; h < p.Hkv; ++h) p.cnt_c[h] = 0u;
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
    const int Hkv = Hs >> kv_shift;
    const int kk = k < C ? k : C;
    if (kk > kSelCap) return false;                          // the selector stages the kept chunk ids in shared memory
    if (max_ctas < Hs + 1) return false;
    ModelPlan p{};
    p.c_static = c;
    // a few CTAs do nothing but select (they take the SMs the scoring grid would leave idle anyway)
    p.n_sel = Hkv < 4 ? Hkv : 4;
    if (max_ctas - p.n_sel < Hs) p.n_sel = max_ctas - Hs;
    p.cph = (max_ctas - p.n_sel) / Hs;
    p.n_score = p.cph * Hs;
    p.grid = p.n_score + p.n_sel;
    p.n_tiles = (L + kRTile - 1) / kRTile;
    p.t_max = (p.n_tiles + p.cph - 1) / p.cph;
    const int ring_panels = c == 10 ? kMRingPanels10 : kMRingPanels20;
    // a layer's chunk scores are summed in a 4 x 256-float buffer, its panels must fit the rings
    if (p.t_max * (kRTile / c) > 252 || 2 * p.t_max > ring_panels) return false;
    const int KB = d / 64;
    const int q_bytes = KB * kRQTileBytes;
    const int pmax_bytes = ring_panels * 128 * 4;            // the panel-maxima ring: one row set per ring panel
    p.stage_slot_bytes = 2 * c * d * 2;                        // K rows and V rows of one chunk
    p.sel_row_bytes = ((4 + kk) * 4 + 127) & ~127;
    const int tail_bytes = p.sel_row_bytes + kMSlots * p.stage_slot_bytes + 128;
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
    // the selector CTAs use the same allocation for their scratch, the kept positions and (many chunks) the keys
    const size_t n_max = static_cast<size_t>(kk) * c + 4096;      // (w <= 256 rows; generous)
    const size_t sel_need = ((sizeof(SelectSmem) + 127) & ~size_t(127)) + ((n_max * 4 + 127) & ~size_t(127));
    if (sel_need + 1024 > static_cast<size_t>(p.smem_bytes)) return false;
    p.sel_keys_fit = (sel_need + static_cast<size_t>(C) * 4 + 1024 <= static_cast<size_t>(p.smem_bytes)) ? 1 : 0;
    *plan = p;
    return true;
}

size_t model_scratch_floats(const ModelPlan& plan, int Hs, int kv_shift, int C, int n_compute) {
    return static_cast<size_t>(2) * plan.grid * 256 + static_cast<size_t>(n_compute) * Hs * ((C + 3) & ~3) +
           static_cast<size_t>(n_compute) * (Hs >> kv_shift) * (plan.sel_row_bytes / 4) + 64;
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
    p.k_row_bytes = 2 * (io.k_row_elems ? io.k_row_elems : io.d);
    p.v_row_bytes = 2 * (io.v_row_elems ? io.v_row_elems : io.d);
    p.k_head_bytes = 2 * (io.k_head_elems ? io.k_head_elems : static_cast<long long>(io.L) * io.d);
    p.v_head_bytes = 2 * (io.v_head_elems ? io.v_head_elems : static_cast<long long>(io.L) * io.d);
    p.cph = plan.cph; p.n_tiles = plan.n_tiles; p.n_stages = plan.n_stages;
    p.q_box_rows = io.Rs < 128 ? io.Rs : 128;
    p.k_box_rows = io.L < kRTile ? io.L : kRTile;
    p.C = io.C; p.k = io.k; p.n_max = io.n_max; p.Hkv = io.Hs >> io.kv_shift;
    p.Cpad = (io.C + 3) & ~3;
    p.n_score = plan.n_score; p.n_sel = plan.n_sel;
    p.sel_row_bytes = plan.sel_row_bytes; p.sel_keys_fit = plan.sel_keys_fit;
    p.off_ring = plan.off_ring; p.off_pmax = plan.off_pmax; p.off_misc = plan.off_misc; p.off_tail = plan.off_tail;
    p.stage_slot_bytes = plan.stage_slot_bytes;
    p.cta_stat = io.scratch;
    p.scores = io.scratch + static_cast<size_t>(2) * plan.grid * 256;
    p.sel_rows = reinterpret_cast<int*>(p.scores + static_cast<size_t>(n_compute) * io.Hs * p.Cpad);   // 16-byte aligned: Cpad % 4 == 0
    p.exits = io.counters;
    p.cnt_a = io.counters + 16;
    p.cnt_b = io.counters + 16 + kResidentMaxHeads;
    p.cnt_c = io.counters + 16 + 2 * kResidentMaxHeads;
    p.status = io.status;
    const bool strided = io.k_row_elems != 0 || io.v_row_elems != 0 || io.k_head_elems != 0 || io.v_head_elems != 0;
    const void* kern = plan.c_static == 10
                           ? (strided ? reinterpret_cast<const void*>(model_kernel<10, true>) : reinterpret_cast<const void*>(model_kernel<10, false>))
                           : (strided ? reinterpret_cast<const void*>(model_kernel<20, true>) : reinterpret_cast<const void*>(model_kernel<20, false>));
    static int smem_set[4][64] = {{0}};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    const int v = (plan.c_static == 10 ? 0 : 1) + (strided ? 2 : 0);
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
