// The whole layer in one cooperative launch with the chunk partial sums kept on chip
// (ChunkKV Algorithm 3: observe-window scores, chunk scores, top-k, index_select on K and V).
//
// Every CTA belongs to one scoring head (a KV head, or one half of its query rows when a KV head
// has more than 128 of them) and owns a contiguous range of that head's keys. While it streams its
// keys through the tensor cores it keeps, per query row and chunk, the sum of exp2(s - m_panel) in
// TENSOR MEMORY (lane = query row, column = chunk of the CTA's range, 256 columns beside the two
// accumulator buffers) and the panel maxima in shared memory, so nothing but a (max, sum) pair per
// row and CTA ever goes to global memory before the chunk scores themselves:
//
//   1. score      TMA -> tcgen05.mma (128 rows x 120 keys per accumulator tile) -> epilogue
//                 warps: one exponential per score element, chunk sums to tensor memory
//   2. hand-over  the CTAs of a scoring head publish their per-row (max, sum) and wait for one
//                 another on a per-head counter (bounded wait)
//   3. contract   every CTA merges the head's records into m_i and 1 / l_i and contracts its own
//                 partial sums over the rows: chunk scores of its key range -> global memory
//   4. hand-over  per KV head, until all of its chunk scores are there (bounded wait)
//   5. select     every CTA of the head runs the same exact top-k over the head's chunk scores
//                 and so holds the kept token positions in shared memory without a third wait;
//                 one of them writes out_idx
//   6. gather     the head's output rows are split evenly over its CTAs
//
// Heads never wait for each other. The launch is cooperative only so that all CTAs are resident
// while they wait for their head's other CTAs; every wait gives up after a clock limit, raises the
// device status word and lets the CTA leave.
#include "gather.cuh"
#include "internal.h"
#include "panels.cuh"
#include "ptx.cuh"
#include "resident.cuh"
#include "select.cuh"

#include <math_constants.h>

namespace chunkkv {

namespace {

constexpr int kRThreads = 576;               // warp 0: TMA, warp 1: UMMA issue, warps 2..17: epilogue
constexpr int kRMiscBytes = 14336;           // records of the four epilogue groups, slices, m_i, 1 / l_i, row sums per lane quarter

struct ResCtl {
    unsigned long long full[kRMaxStages];
    unsigned long long empty[kRMaxStages];
    unsigned long long tfull[2];
    unsigned long long tempty[2];
    unsigned long long qfull;
    uint32_t tmem_base;
    int abort_flag;
    int wait_ok;
};

struct ResArgs {
    int L, P, w, R, Hs, d, kv_shift;   // R rows per scoring head, Hs scoring heads
    float sl2;                         // log2(e) / sqrt(d)
    int cph;                           // CTAs per scoring head (grid = Hs * cph)
    int n_tiles;                       // accumulator tiles per head
    int n_stages;
    int q_box_rows, k_box_rows;
    int C, k, n_max, Hkv;
    int off_ring, ring_bytes, off_pmax, off_misc;   // dynamic shared memory layout (bytes from the aligned base)
    const uint4* K;
    const uint4* V;
    long long k_row, k_head, v_row, v_head;   // 16-byte vectors between rows of a head / between heads
    const int32_t* block_table;              // non-null: out_K / out_V are paged caches
    int page_size, num_pages;
    int tok_cap;                             // Algorithm 1: tokens of the kept chunks that are emitted
    uint4* out_K;
    uint4* out_V;
    int32_t* out_idx;
    float* cta_stat;                   // [grid, {max, sum}, 128]
    float* scores;                     // [Hs, C]
    unsigned* cnt_a;                   // [Hs]  hand-over 2, zero between launches
    unsigned* cnt_b;                   // [Hkv] hand-over 4
    unsigned* exits;                   // CTAs that left; the last one clears the counters
    int* status;
};

// One thread publishes this CTA's arrival on `counter` and waits until `target` CTAs have arrived.
// Block-wide: every thread calls it; returns false if the wait was abandoned.
__device__ __forceinline__ bool head_handover(unsigned* counter, unsigned target, ResCtl& ctl) {
    __syncthreads();
    if (threadIdx.x == 0) {
        bool ok = true;
        unsigned old;
        // release: what this CTA wrote before the barrier above becomes visible to the others
        asm volatile("atom.add.release.gpu.u32 %0, [%1], 1;" : "=r"(old) : "l"(counter) : "memory");
        if (old + 1u < target) {
            const long long t0 = clock64();
            unsigned cur;
            for (;;) {
                asm volatile("ld.acquire.gpu.u32 %0, [%1];" : "=r"(cur) : "l"(counter) : "memory");
                if (cur >= target) break;
                if (clock64() - t0 > kWaitLimitClocks) { ok = false; break; }
            }
        }
        asm volatile("fence.acq_rel.gpu;" ::: "memory");
        ctl.wait_ok = ok ? 1 : 0;
    }
    __syncthreads();
    return ctl.wait_ok != 0;
}

template <int C_STATIC>
__global__ void __launch_bounds__(kRThreads, 1)
layer_resident_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                      const ResArgs a) {
    constexpr int SPP = kRPanel / C_STATIC;          // chunk slots per panel
    constexpr uint32_t IDESC = umma_idesc_bf16(128, kRUmmaN);
    static_assert(kRPanel % C_STATIC == 0, "the chunk size must divide the panel");

    extern __shared__ uint8_t smem_raw[];
    __shared__ ResCtl ctl;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int KB = a.d >> 6;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* dyn = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t q_base = smem_base;
    const uint32_t k_base = smem_base + static_cast<uint32_t>(a.off_ring);
    float* pmax = reinterpret_cast<float*>(dyn + a.off_pmax);      // [panel of this CTA][128] panel maxima (log2 domain)
    float* misc = reinterpret_cast<float*>(dyn + a.off_misc);
    float* rec = misc;                 // [4 groups][{max, sum}][128]
    float* slice = misc + 1024;        // [4 slices][{max, sum}][128]
    float* gm = misc + 2048;           // [128] row maxima of the head
    float* ginv = misc + 2176;         // [128] 1 / row sums of the head
    uint8_t* ring = dyn + a.off_ring;  // reused after scoring
    volatile int* abort_flag = &ctl.abort_flag;
    const uint32_t n_stages = static_cast<uint32_t>(a.n_stages);

    const int hs = blockIdx.x / a.cph, part = blockIdx.x - hs * a.cph;
    const int hkv = hs >> a.kv_shift;
    // tiles are dealt out rounding up, so the head's last CTA - whose last panels take the slow, masked path -
    // is never one of those that get an extra tile
    const int t_begin = (a.n_tiles * part + a.cph - 1) / a.cph, t_end = (a.n_tiles * (part + 1) + a.cph - 1) / a.cph;
    const int nt = t_end - t_begin;

    if (threadIdx.x == 0) {
        for (int s = 0; s < a.n_stages; ++s) {
            mbar_init(smem_u32(&ctl.full[s]), 1);
            mbar_init(smem_u32(&ctl.empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&ctl.tfull[b]), 1);
            mbar_init(smem_u32(&ctl.tempty[b]), 8);      // one arrival per warp of the pair that reads the buffer
        }
        mbar_init(smem_u32(&ctl.qfull), 1);
        ctl.abort_flag = 0;
        ctl.wait_ok = 1;
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
    // Programmatic dependent launch (used when the launch asks for it, otherwise both are no-ops):
    // the next kernel of the stream may be set up while this one runs, and this one touches no
    // global memory before everything queued ahead of it has completed.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (elect_one() && nt > 0) {
            prefetch_tmap(&tm_q);
            prefetch_tmap(&tm_k);
            const uint32_t qbar = smem_u32(&ctl.qfull);
            mbar_arrive_expect_tx(qbar, static_cast<uint32_t>(KB * a.q_box_rows) * 128u);
            for (int kb = 0; kb < KB; ++kb)
                tma_load_3d(q_base + static_cast<uint32_t>(kb) * kRQTileBytes, &tm_q, qbar, kb * 64, 0, hs);
            const uint32_t k_bytes = static_cast<uint32_t>(a.k_box_rows) * 128u;
            uint32_t st = 0, st_par = 1;
            int issued = 0;
            bool ok = true;
            for (int t = t_begin; t < t_end && ok; ++t) {
                for (int kb = 0; kb < KB; ++kb) {
                    ok = mbar_wait(smem_u32(&ctl.empty[st]), st_par, abort_flag);
                    if (!ok) break;
                    const uint32_t bar = smem_u32(&ctl.full[st]);
                    mbar_arrive_expect_tx(bar, k_bytes);
                    tma_load_3d(k_base + st * kRStageBytes, &tm_k, bar, kb * 64, t * kRTile, hkv);
                    ++issued;
                    if (++st == n_stages) { st = 0; st_par ^= 1u; }
                }
            }
            if (!ok) {
                // Give copies already in flight a bounded chance to land before the CTA exits.
                const int back = min(issued, a.n_stages);
                for (int i = 1; i <= back; ++i) {
                    const int cc = issued - i, s = cc % a.n_stages;
                    const long long t0 = clock64();
                    while (!mbar_try_wait(smem_u32(&ctl.full[s]), (cc / a.n_stages) & 1) &&
                           clock64() - t0 < kWaitLimitClocks / 8) {
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ UMMA issuer
        if (elect_one() && nt > 0) {
            bool ok = mbar_wait(smem_u32(&ctl.qfull), 0, abort_flag);
            uint32_t st = 0, st_par = 0;
            for (int ti = 0; ti < nt && ok; ++ti) {
                const int buf = ti & 1, use = ti >> 1;
                ok = mbar_wait(smem_u32(&ctl.tempty[buf]), (use & 1) ^ 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_addr = tmem_base + static_cast<uint32_t>(buf * kRUmmaN);
#pragma unroll
                for (int kb = 0; kb < 2; ++kb) {          // d is 64 or 128: one or two 64-element blocks
                    if (kb >= KB || !ok) break;
                    ok = mbar_wait(smem_u32(&ctl.full[st]), st_par, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t b_desc = umma_desc_sw128(k_base + st * kRStageBytes);
                    const uint64_t a_desc = umma_desc_sw128(q_base + static_cast<uint32_t>(kb) * kRQTileBytes);
#pragma unroll
                    for (int k4 = 0; k4 < 4; ++k4)      // k-steps advance the start address by 32 bytes
                        umma_bf16(d_addr, a_desc + 2u * k4, b_desc + 2u * k4, IDESC, (kb > 0 || k4 > 0) ? 1u : 0u);
                    umma_commit(smem_u32(&ctl.empty[st]));
                    if (++st == n_stages) { st = 0; st_par ^= 1u; }
                }
                if (ok) umma_commit(smem_u32(&ctl.tfull[buf]));
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue
        // Four groups of four warps (a group's warps cover the four tensor-memory lane quarters =
        // the 128 query rows). The groups form two pairs that take alternate accumulator tiles;
        // inside a pair each group takes one 60-key half of the tile.
        const int grp = (warp - 2) >> 2, quarter = warp & 3;
        const int pair = grp >> 1, half = grp & 1;
        const int row = quarter * 32 + lane;
        const bool active = row < a.R;
        const int last_visible = a.P + (row % a.w);      // this row sees keys j <= P + r (all < L)
        const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        float run_m = -CUDART_INF_F, run_l = 0.f;
        for (int ti = pair; ti < nt; ti += 2) {
            const int use = ti >> 1;
            bool ready = true;                           // one lane polls, the warp follows
            if (lane == 0) ready = mbar_wait(smem_u32(&ctl.tfull[pair]), use & 1, abort_flag);
            if (!__shfl_sync(0xffffffffu, ready, 0)) break;
            tc_fence_after();
            float v[kRPanel];
            load_panel<kRPanel>(lane_addr + static_cast<uint32_t>(pair * kRUmmaN + half * kRPanel), v);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl.tempty[pair]));   // the buffer may be overwritten now
            const int pl = ti * 2 + half;                // panel of this CTA
            const int j0 = (t_begin + ti) * kRTile + half * kRPanel;
            float pr[SPP], m2, l;
            auto emit = [&](int ch, float acc) { pr[ch] = acc; };
            if (j0 + kRPanel <= a.P)
                panel_fast<C_STATIC, kRPanel>(v, a.sl2, emit, &m2, &l);
            else
                panel_static_tail<C_STATIC, kRPanel>(v, a.sl2, emit, j0, a.P, last_visible, &m2, &l);
            part_store<SPP>(lane_addr + static_cast<uint32_t>(kRPartCol0 + pl * SPP), pr);
            pmax[pl * 128 + row] = m2;
            // fold into the running record: l is relative to m2, run_l to run_m
            const float nm = fmaxf(run_m, m2);
            const float s_old = (run_m == -CUDART_INF_F) ? 0.f : ex2_approx(run_m - nm);
            const float s_new = (m2 == -CUDART_INF_F) ? 0.f : ex2_approx(m2 - nm);
            run_l = run_l * s_old + l * s_new;
            run_m = nm;
        }
        tmem_st_wait();
        rec[(grp * 2 + 0) * 128 + row] = active ? run_m : -CUDART_INF_F;
        rec[(grp * 2 + 1) * 128 + row] = active ? run_l : 0.f;
    }

    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    bool ok = ctl.abort_flag == 0;

    // ---- 2. this CTA's (max, sum) per row -> global memory; wait for the head's other CTAs
    if (ok) {
        if (threadIdx.x < 128) {
            const int i = threadIdx.x;
            float M = -CUDART_INF_F, Ls = 0.f;
#pragma unroll
            for (int g = 0; g < 4; ++g) M = fmaxf(M, rec[(g * 2) * 128 + i]);
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                const float m = rec[(g * 2) * 128 + i];
                Ls += (m == -CUDART_INF_F) ? 0.f : rec[(g * 2 + 1) * 128 + i] * ex2_approx(m - M);
            }
            float* dst = a.cta_stat + static_cast<size_t>(blockIdx.x) * 256;
            dst[i] = M;
            dst[128 + i] = Ls;
        }
        ok = head_handover(a.cnt_a + hs, static_cast<unsigned>(a.cph), ctl);
    }

    // ---- 3. row statistics of the head, then this CTA's chunk scores
    if (ok) {
        if (threadIdx.x < 512) {
            const int i = threadIdx.x & 127, sl = threadIdx.x >> 7;
            const float* src = a.cta_stat + static_cast<size_t>(hs) * a.cph * 256 + i;
            float M = -CUDART_INF_F, Ls = 0.f;
            for (int j0 = sl; j0 < a.cph; j0 += 16) {     // four records in flight per thread
                float rm[4], rl[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int j = j0 + 4 * u;
                    rm[u] = (j < a.cph) ? __ldcg(src + static_cast<size_t>(j) * 256) : -CUDART_INF_F;
                    rl[u] = (j < a.cph) ? __ldcg(src + static_cast<size_t>(j) * 256 + 128) : 0.f;
                }
                float bm = M;
#pragma unroll
                for (int u = 0; u < 4; ++u) bm = fmaxf(bm, rm[u]);
                float acc = (M == -CUDART_INF_F) ? 0.f : Ls * ex2_approx(M - bm);
#pragma unroll
                for (int u = 0; u < 4; ++u) acc += (rm[u] == -CUDART_INF_F) ? 0.f : rl[u] * ex2_approx(rm[u] - bm);
                M = bm;
                Ls = acc;
            }
            slice[(sl * 2 + 0) * 128 + i] = M;
            slice[(sl * 2 + 1) * 128 + i] = Ls;
        }
        __syncthreads();
        if (threadIdx.x < 128) {
            const int i = threadIdx.x;
            float M = -CUDART_INF_F, Ls = 0.f;
#pragma unroll
            for (int s = 0; s < 4; ++s) M = fmaxf(M, slice[(s * 2) * 128 + i]);
#pragma unroll
            for (int s = 0; s < 4; ++s) {
                const float m = slice[(s * 2) * 128 + i];
                Ls += (m == -CUDART_INF_F) ? 0.f : slice[(s * 2 + 1) * 128 + i] * ex2_approx(m - M);
            }
            gm[i] = M;
            ginv[i] = 1.0f / Ls;       // rows >= R are never used
        }
        __syncthreads();
        // chunk scores of this CTA's key range: partial sums x exp2(m_panel - m_i) / l_i, summed over
        // the rows. A thread holds one row of up to 30 chunk slots at a time (PPB panels of its
        // group: panels grp, grp + 4, ...); a transposing warp reduction leaves lane j with the sum
        // over the warp's 32 rows of slot j; the four lane quarters are added through shared memory.
        float* red = misc + 2304;      // [4 lane quarters][256 chunk slots of this CTA]
        const int n_pl = 2 * nt;
        if (warp >= 2) {
            const int grp = (warp - 2) >> 2, quarter = warp & 3;
            const int row = quarter * 32 + lane;
            const bool active = row < a.R;
            const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
            const float mi = gm[row], li = ginv[row];
            constexpr int PPB = 30 / SPP;                // panels per block of 32 values (30 used)
            for (int b0 = 0; grp + 4 * b0 < n_pl; b0 += PPB) {
                float v[32];
#pragma unroll
                for (int u = 0; u < PPB; ++u) {
                    const int pl = min(grp + 4 * (b0 + u), n_pl - 1);   // clamped: every lane issues the same loads
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
                    for (int s = 0; s < SPP; ++s) v[u * SPP + s] = have ? v[u * SPP + s] * f : 0.f;
                }
                const float tot = warp_transpose_reduce(v, lane);
                const int pl = grp + 4 * (b0 + lane / SPP);
                if (lane < 30 && pl < n_pl) red[quarter * 256 + pl * SPP + lane % SPP] = tot;
            }
        }
        tc_fence_before();
        __syncthreads();
        const int n_local = nt * (kRTile / C_STATIC);    // chunk slots of this CTA
        const int ch0 = t_begin * (kRTile / C_STATIC);   // its first chunk
        for (int lc = threadIdx.x; lc < n_local; lc += kRThreads)
            if (ch0 + lc < a.C)
                a.scores[static_cast<size_t>(hs) * a.C + ch0 + lc] =
                    (red[lc] + red[256 + lc]) + (red[512 + lc] + red[768 + lc]);
    }
    // ---- 4. wait for the KV head's other CTAs, 5. select, 6. gather
    if (ok) ok = head_handover(a.cnt_b + hkv, static_cast<unsigned>(a.cph) << a.kv_shift, ctl);
    if (ok) {
        SelectSmem& ss = *reinterpret_cast<SelectSmem*>(ring);
        constexpr size_t kSelBytes = (sizeof(SelectSmem) + 127) & ~size_t(127);
        int32_t* sidx = reinterpret_cast<int32_t*>(ring + kSelBytes);          // [n_max] kept positions of the head
        const float* sc = a.scores + (static_cast<size_t>(hkv) << a.kv_shift) * a.C;
        const float* sc2 = a.kv_shift ? sc + a.C : nullptr;
        if (a.C <= kRThreads * 6) {
            select_head_regs<6>(sc, sc2, a.L, a.w, C_STATIC, a.C, a.k, a.n_max, sidx, ss, a.tok_cap);
        } else {
            const size_t idx_bytes = (static_cast<size_t>(a.n_max) * 4 + 127) & ~size_t(127);
            uint32_t* kbuf = reinterpret_cast<uint32_t*>(ring + kSelBytes + idx_bytes);
            const bool fits = kSelBytes + idx_bytes + static_cast<size_t>(a.C) * 4 <= static_cast<size_t>(a.ring_bytes);
            if (fits)
                select_head_smem(sc, sc2, a.L, a.w, C_STATIC, a.C, a.k, a.n_max, sidx, ss, kbuf, a.tok_cap);
            else
                select_head_rows(sc, sc2, a.L, a.w, C_STATIC, a.C, a.k, a.n_max, sidx, ss, nullptr);
        }
        const int Q = a.cph << a.kv_shift;               // CTAs of this KV head
        const int q = static_cast<int>(blockIdx.x) - (hkv << a.kv_shift) * a.cph;
        if (q == 0) {
            int32_t* dst = a.out_idx + static_cast<size_t>(hkv) * a.n_max;
            for (int n = threadIdx.x; n < a.n_max; n += kRThreads) dst[n] = sidx[n];
        }
        const int r_begin = static_cast<int>(static_cast<long long>(a.n_max) * q / Q);
        const int r_end = static_cast<int>(static_cast<long long>(a.n_max) * (q + 1) / Q);
        const int vpr = a.d >> 3;
        const int rows_per_pass = (kRThreads / vpr) * kGatherRowsPerThread;
        // packed outputs: this head's block; paged outputs: the cache base (rows are placed through the block table)
        const PagedDst pg{a.block_table, a.page_size, a.num_pages, a.Hkv, hkv};
        const size_t head_out = a.block_table ? 0 : static_cast<size_t>(hkv) * a.n_max;
        for (int n0 = r_begin; n0 < r_end; n0 += rows_per_pass) {
            if (vpr == 16)
                gather_rows<16, false>(a.K + static_cast<size_t>(hkv) * a.k_head, a.V + static_cast<size_t>(hkv) * a.v_head,
                                       sidx, a.L, r_end, n0, threadIdx.x, kRThreads, a.out_K + head_out * 16,
                                       a.out_V + head_out * 16, nullptr, a.k_row, a.v_row, pg);
            else
                gather_rows<8, false>(a.K + static_cast<size_t>(hkv) * a.k_head, a.V + static_cast<size_t>(hkv) * a.v_head,
                                      sidx, a.L, r_end, n0, threadIdx.x, kRThreads, a.out_K + head_out * 8,
                                      a.out_V + head_out * 8, nullptr, a.k_row, a.v_row, pg);
        }
    }
    // tensor memory has not been read since the barrier after the contraction (or after scoring)
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
    if (threadIdx.x == 0) {
        if (!ok) atomicExch(a.status, 1);
        // The last CTA to leave clears the hand-over counters for the next launch. (After an
        // abandoned wait the counters are left as they are; chunkkv_device_status clears them.)
        const unsigned old = atomicAdd(a.exits, 1u);
        if (old + 1u == gridDim.x) {
            for (int h = 0; h < a.Hs; ++h) a.cnt_a[h] = 0u;
            for (int h = 0; h < a.Hkv; ++h) a.cnt_b[h] = 0u;
            *a.exits = 0u;
            __threadfence();
        }
    }
}

}  // namespace

size_t resident_scratch_floats(const ResidentPlan& plan, int Hs, int C) {
    return static_cast<size_t>(plan.grid) * 256 + ((static_cast<size_t>(Hs) * C + 63) & ~static_cast<size_t>(63));
}

bool make_resident_plan(int L, int Rs, int Hs, int kv_shift, int d, int c, int C, int n_max, int max_ctas,
                        int smem_limit, ResidentPlan* plan) {
    if (c != 10 && c != 20) return false;
    if (Rs < 1 || Rs > 128 || (d != 64 && d != 128) || L < 1 || C < 1 || Hs < 1 || Hs > kResidentMaxHeads) return false;
    if (max_ctas < Hs) return false;
    ResidentPlan p{};
    p.c_static = c;
    p.cph = max_ctas / Hs;
    p.grid = p.cph * Hs;
    p.n_tiles = (L + kRTile - 1) / kRTile;
    p.t_max = (p.n_tiles + p.cph - 1) / p.cph;
    if (p.t_max * (kRTile / c) > kRPartCols) return false;          // the chunk partial sums must fit tensor memory
    const int KB = d / 64;
    const int q_bytes = KB * kRQTileBytes;
    const int pmax_bytes = p.t_max * 2 * 128 * 4;
    const int fixed = 1024 /* alignment */ + q_bytes + 1024 /* tail of the last stage's UMMA read */ + pmax_bytes + kRMiscBytes;
    int ns = (smem_limit - fixed) / kRStageBytes;
    if (ns > kRMaxStages) ns = kRMaxStages;
    if (ns < 2 * KB) return false;
    p.n_stages = ns;
    p.off_ring = q_bytes;
    p.ring_bytes = ns * kRStageBytes + 1024;
    p.off_pmax = p.off_ring + p.ring_bytes;
    p.off_misc = p.off_pmax + pmax_bytes;
    p.smem_bytes = 1024 + p.off_misc + kRMiscBytes;
    // after scoring the ring holds the selection scratch and the kept positions
    const size_t sel_bytes = ((sizeof(SelectSmem) + 127) & ~size_t(127)) + ((static_cast<size_t>(n_max) * 4 + 127) & ~size_t(127));
    if (sel_bytes > static_cast<size_t>(p.ring_bytes)) return false;
    *plan = p;
    return true;
}

cudaError_t launch_layer_resident(const ResidentPlan& plan, const CUtensorMap& tm_q, const CUtensorMap& tm_k,
                                  const ResidentIO& io, cudaStream_t stream) {
    ResArgs a{};
    a.L = io.L; a.P = io.L - io.w; a.w = io.w; a.R = io.Rs; a.Hs = io.Hs; a.d = io.d; a.kv_shift = io.kv_shift;
    a.sl2 = io.sl2;
    a.cph = plan.cph; a.n_tiles = plan.n_tiles; a.n_stages = plan.n_stages;
    a.q_box_rows = io.Rs < 128 ? io.Rs : 128;
    a.k_box_rows = io.L < kRTile ? io.L : kRTile;
    a.C = io.C; a.k = io.k; a.n_max = io.n_max; a.Hkv = io.Hs >> io.kv_shift;
    a.off_ring = plan.off_ring; a.ring_bytes = plan.ring_bytes; a.off_pmax = plan.off_pmax; a.off_misc = plan.off_misc;
    a.K = static_cast<const uint4*>(io.K); a.V = static_cast<const uint4*>(io.V);
    a.block_table = io.block_table; a.page_size = io.page_size; a.num_pages = io.num_pages;
    a.tok_cap = io.tok_cap;
    {
        const long long vpr = io.d / 8;
        a.k_row = io.k_row_elems ? io.k_row_elems / 8 : vpr;
        a.v_row = io.v_row_elems ? io.v_row_elems / 8 : vpr;
        a.k_head = io.k_head_elems ? io.k_head_elems / 8 : static_cast<long long>(io.L) * vpr;
        a.v_head = io.v_head_elems ? io.v_head_elems / 8 : static_cast<long long>(io.L) * vpr;
    }
    a.out_K = static_cast<uint4*>(io.out_K); a.out_V = static_cast<uint4*>(io.out_V); a.out_idx = io.out_idx;
    a.cta_stat = io.scratch;
    a.scores = io.scratch + static_cast<size_t>(plan.grid) * 256;
    a.exits = io.counters;
    a.cnt_a = io.counters + 16;
    a.cnt_b = io.counters + 16 + kResidentMaxHeads;
    a.status = io.status;
    const void* kern = plan.c_static == 10 ? reinterpret_cast<const void*>(layer_resident_kernel<10>)
                                           : reinterpret_cast<const void*>(layer_resident_kernel<20>);
    static int smem_set[2][64] = {{0}};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const int v = plan.c_static == 10 ? 0 : 1;
    if (dev < 0 || dev >= 64 || smem_set[v][dev] < plan.smem_bytes) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, plan.smem_bytes);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) smem_set[v][dev] = plan.smem_bytes;
    }
    void* params[] = {const_cast<CUtensorMap*>(&tm_q), const_cast<CUtensorMap*>(&tm_k), &a};
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(plan.grid);
    cfg.blockDim = dim3(kRThreads);
    cfg.dynamicSmemBytes = static_cast<size_t>(plan.smem_bytes);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    if (io.cooperative) {
        // several such launches may share the GPU (lanes): each must have all of its CTAs resident
        attr[0].id = cudaLaunchAttributeCooperative;
        attr[0].val.cooperative = 1;
    } else {
        // One launch at a time on the device (the calls share one scratch buffer and are ordered): at
        // most one CTA per SM and no more CTAs than SMs, so every CTA becomes resident without
        // waiting for another CTA of this grid. Launched as a programmatic dependent of the
        // preceding kernel, the set-up of this one overlaps the end of that one.
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
    }
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelExC(&cfg, kern, params);
}

}  // namespace chunkkv
