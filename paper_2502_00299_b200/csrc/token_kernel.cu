// Token scores (ChunkKV Algorithm 3 with chunk size 1, the token-level selection of the paper's
// hybrid experiment; also chunkkv_score's token-score output): t[j] = sum over the window rows of
// softmax(q k^T / sqrt(d))[i, j] for every prefix key j.
//
// With one chunk per key the per-(chunk, row) partial sums of the other kernels would be the whole
// score matrix, so this kernel walks its keys twice instead, in one launch: pass 1 only folds the
// per-row (max, sum) of the CTA's key range; the CTAs of a head exchange those records (one
// bounded hand-over per head); pass 2 recomputes the same tiles (the keys come back from L2),
// normalises every element with the final row statistics and sums over the 128 rows with a
// transposing warp reduction, so only the token scores are written. Same tiling, producer / issuer
// / epilogue roles and bounded waits as layer_resident.cu.
#include "internal.h"
#include "panels.cuh"
#include "ptx.cuh"
#include "resident.cuh"

#include <math_constants.h>

namespace chunkkv {

namespace {

constexpr int kTThreads = 576;
constexpr int kTMiscBytes = 20480;     // group records, slices, m_i, 1 / l_i, per-group column sums (two buffers)

struct TokCtl {
    unsigned long long full[kRMaxStages];
    unsigned long long empty[kRMaxStages];
    unsigned long long tfull[2];
    unsigned long long tempty[2];
    unsigned long long qfull;
    uint32_t tmem_base;
    int abort_flag;
    int wait_ok;
};

struct TokArgs {
    int L, P, w, R, Hs, d, kv_shift;
    float sl2;
    int cph, n_tiles, n_tiles_prefix, n_stages, q_box_rows, k_box_rows;
    int off_ring, off_misc;
    float* cta_stat;       // [grid][{max, sum}][128]
    float* token_scores;   // [Hs][P]
    unsigned* cnt_a;       // [Hs]
    unsigned* exits;
    int* status;
};

__global__ void __launch_bounds__(kTThreads, 1)
token_scores_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const TokArgs a) {
    constexpr uint32_t IDESC = umma_idesc_bf16(128, kRUmmaN);
    extern __shared__ uint8_t smem_raw[];
    __shared__ TokCtl ctl;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int KB = a.d >> 6;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* dyn = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t q_base = smem_base;
    const uint32_t k_base = smem_base + static_cast<uint32_t>(a.off_ring);
    float* misc = reinterpret_cast<float*>(dyn + a.off_misc);
    float* rec = misc;                 // [4 groups][{max, sum}][128]
    float* slice = misc + 1024;        // [4 slices][{max, sum}][128]
    float* gm = misc + 2048;           // [128]
    float* ginv = misc + 2176;         // [128]
    float* qsum = misc + 2304;         // [4 groups][2 buffers][4 lane quarters][64]
    volatile int* abort_flag = &ctl.abort_flag;
    const uint32_t n_stages = static_cast<uint32_t>(a.n_stages);

    const int hs = blockIdx.x / a.cph, part = blockIdx.x - hs * a.cph;
    const int hkv = hs >> a.kv_shift;
    const int t_begin = a.n_tiles * part / a.cph, t_end = a.n_tiles * (part + 1) / a.cph;
    const int nt = t_end - t_begin;
    const int nt2 = max(0, min(t_end, a.n_tiles_prefix) - t_begin);   // tiles of pass 2: those that hold prefix keys

    if (threadIdx.x == 0) {
        for (int s = 0; s < a.n_stages; ++s) {
            mbar_init(smem_u32(&ctl.full[s]), 1);
            mbar_init(smem_u32(&ctl.empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&ctl.tfull[b]), 1);
            mbar_init(smem_u32(&ctl.tempty[b]), 8);
        }
        mbar_init(smem_u32(&ctl.qfull), 1);
        ctl.abort_flag = 0;
        ctl.wait_ok = 1;
        fence_mbar_init();
        fence_proxy_async();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&ctl.tmem_base), 256);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl.tmem_base;
    // the selection that follows is a programmatic dependent: its CTAs may be scheduled as this grid's retire;
    // this grid itself touches no global memory before its predecessor is complete
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer: the key range, twice
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
            for (int pass = 0; pass < 2 && ok; ++pass) {
                // pass 2 walks the tiles backwards: the keys read last in pass 1 are the ones still in L2
                const int n_pass = pass == 0 ? nt : nt2;
                for (int i = 0; i < n_pass && ok; ++i) {
                    const int t = pass == 0 ? t_begin + i : t_begin + nt2 - 1 - i;
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
            }
            if (!ok) {
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
            for (int tg = 0; tg < nt + nt2 && ok; ++tg) {
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
        }
    } else {
        // ------------------------------------------------------------------ epilogue
        const int et = threadIdx.x - 64;
        const int grp = (warp - 2) >> 2, quarter = warp & 3;
        const int pair = grp >> 1, half = grp & 1;
        const int row = quarter * 32 + lane;
        const bool active = row < a.R;
        const int last_visible = a.P + (row % a.w);
        const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        // ---- pass 1: (max, sum of exp2) per row over this CTA's keys
        float run_m = -CUDART_INF_F, run_l = 0.f;
        for (int ti = pair; ti < nt; ti += 2) {
            const int use = ti >> 1;
            bool ready = true;
            if (lane == 0) ready = mbar_wait(smem_u32(&ctl.tfull[pair]), use & 1, abort_flag);
            if (!__shfl_sync(0xffffffffu, ready, 0)) break;
            tc_fence_after();
            float v[kRPanel];
            load_panel<kRPanel>(lane_addr + static_cast<uint32_t>(pair * kRUmmaN + half * kRPanel), v);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl.tempty[pair]));
            const int j0 = (t_begin + ti) * kRTile + half * kRPanel;
            float m2, l;
            auto emit = [](int, float) {};
            if (j0 + kRPanel <= a.P)
                panel_fast<10, kRPanel>(v, a.sl2, emit, &m2, &l);
            else
                panel_static_tail<10, kRPanel>(v, a.sl2, emit, j0, a.P, last_visible, &m2, &l);
            const float nm = fmaxf(run_m, m2);
            const float s_old = (run_m == -CUDART_INF_F) ? 0.f : ex2_approx(run_m - nm);
            const float s_new = (m2 == -CUDART_INF_F) ? 0.f : ex2_approx(m2 - nm);
            run_l = run_l * s_old + l * s_new;
            run_m = nm;
        }
        rec[(grp * 2 + 0) * 128 + row] = active ? run_m : -CUDART_INF_F;
        rec[(grp * 2 + 1) * 128 + row] = active ? run_l : 0.f;
        named_barrier(1, 512);
        bool ok = ctl.abort_flag == 0;               // same answer in every epilogue thread
        // ---- the head's row statistics: publish, wait for the head's other CTAs, merge
        if (ok) {
            if (et < 128) {
                float M = -CUDART_INF_F, Ls = 0.f;
#pragma unroll
                for (int g = 0; g < 4; ++g) merge_ml(M, Ls, rec[(g * 2) * 128 + et], rec[(g * 2 + 1) * 128 + et]);
                float* dst = a.cta_stat + static_cast<size_t>(blockIdx.x) * 256;
                dst[et] = M;
                dst[128 + et] = Ls;
            }
            named_barrier(1, 512);
            if (et == 0) {
                unsigned old;
                asm volatile("atom.add.release.gpu.u32 %0, [%1], 1;" : "=r"(old) : "l"(a.cnt_a + hs) : "memory");
                bool w_ok = true;
                if (old + 1u < static_cast<unsigned>(a.cph)) {
                    const long long t0 = clock64();
                    unsigned cur;
                    for (;;) {
                        asm volatile("ld.acquire.gpu.u32 %0, [%1];" : "=r"(cur) : "l"(a.cnt_a + hs) : "memory");
                        if (cur >= static_cast<unsigned>(a.cph)) break;
                        if (clock64() - t0 > kWaitLimitClocks) { w_ok = false; ctl.abort_flag = 1; break; }
                    }
                }
                asm volatile("fence.acq_rel.gpu;" ::: "memory");
                ctl.wait_ok = w_ok ? 1 : 0;
            }
            named_barrier(1, 512);
            ok = ctl.wait_ok != 0;
        }
        if (ok) {
            const int i = et & 127, sl = et >> 7;
            const float* src = a.cta_stat + static_cast<size_t>(hs) * a.cph * 256 + i;
            float M = -CUDART_INF_F, Ls = 0.f;
            for (int j0 = sl; j0 < a.cph; j0 += 16) {
                float rm[4], rl[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int j = j0 + 4 * u;
                    rm[u] = (j < a.cph) ? __ldcg(src + static_cast<size_t>(j) * 256) : -CUDART_INF_F;
                    rl[u] = (j < a.cph) ? __ldcg(src + static_cast<size_t>(j) * 256 + 128) : 0.f;
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) merge_ml(M, Ls, rm[u], rl[u]);
            }
            slice[(sl * 2 + 0) * 128 + i] = M;
            slice[(sl * 2 + 1) * 128 + i] = Ls;
            named_barrier(1, 512);
            if (et < 128) {
                float M2 = -CUDART_INF_F, L2 = 0.f;
#pragma unroll
                for (int q = 0; q < 4; ++q) merge_ml(M2, L2, slice[(q * 2) * 128 + et], slice[(q * 2 + 1) * 128 + et]);
                gm[et] = M2;
                ginv[et] = log2f(L2);          // the normaliser goes into the exponent: exp2(s - m_i - log2 l_i)
            }
            named_barrier(1, 512);
            // ---- pass 2: the same tiles again, normalised, summed over the rows
            const float nm = active ? -(gm[row] + ginv[row]) : 0.f;
            float* out = a.token_scores + static_cast<size_t>(hs) * a.P;
            int mine = 0;                                  // tiles this group has taken in pass 2 (column-sum buffer = mine & 1)
            for (int ti = (pair - (nt & 1)) & 1; ti < nt2; ti += 2, ++mine) {
                const int tg = nt + ti, use = tg >> 1;
                bool ready = true;
                if (lane == 0) ready = mbar_wait(smem_u32(&ctl.tfull[pair]), use & 1, abort_flag);
                ready = __shfl_sync(0xffffffffu, ready, 0);
                float* qs = qsum + ((grp * 2 + (mine & 1)) * 4 + quarter) * 64;
                if (ready) {
                    tc_fence_after();
                    float v[kRPanel];
                    load_panel<kRPanel>(lane_addr + static_cast<uint32_t>(pair * kRUmmaN + half * kRPanel), v);
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&ctl.tempty[pair]));
#pragma unroll
                    for (int b = 0; b < 2; ++b) {
                        float x[32];
#pragma unroll
                        for (int u = 0; u < 30; ++u)      // (an inactive row holds garbage: select, do not multiply)
                            x[u] = active ? ex2_approx(fmaf(v[b * 30 + u], a.sl2, nm)) : 0.f;
                        x[30] = 0.f;
                        x[31] = 0.f;
                        const float tot = warp_transpose_reduce(x, lane);
                        if (lane < 30) qs[b * 30 + lane] = tot;
                    }
                }
                named_barrier(2 + grp, 128);               // the four lane quarters of this panel are in shared memory
                if (ctl.abort_flag) break;                 // same answer in the four warps of the group
                const int gt = threadIdx.x - 64 - grp * 128;   // 0 .. 127 within the group
                const int j = (t_begin + nt2 - 1 - ti) * kRTile + half * kRPanel + gt;      // (pass 2 runs backwards)
                if (gt < kRPanel && j < a.P) {
                    const float* q0 = qsum + ((grp * 2 + (mine & 1)) * 4) * 64 + gt;
                    out[j] = (q0[0] + q0[64]) + (q0[128] + q0[192]);
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 256);
    }
    if (threadIdx.x == 0) {
        if (ctl.abort_flag) atomicExch(a.status, 1);
        const unsigned old = atomicAdd(a.exits, 1u);
        if (old + 1u == gridDim.x) {
            for (int h = 0; h < a.Hs; ++h) a.cnt_a[h] = 0u;
            *a.exits = 0u;
            __threadfence();
        }
    }
}

}  // namespace

bool make_token_plan(int L, int w, int Rs, int Hs, int d, int max_ctas, int smem_limit, TokenPlan* plan) {
    if (Rs < 1 || Rs > 128 || (d != 64 && d != 128) || L < 1 || L - w < 1 || Hs < 1 || Hs > kResidentMaxHeads) return false;
    if (max_ctas < Hs) return false;
    TokenPlan p{};
    p.cph = max_ctas / Hs;
    p.grid = p.cph * Hs;
    p.n_tiles = (L + kRTile - 1) / kRTile;
    p.n_tiles_prefix = (L - w + kRTile - 1) / kRTile;
    const int KB = d / 64;
    const int q_bytes = KB * kRQTileBytes;
    const int fixed = 1024 + q_bytes + 1024 + kTMiscBytes;
    int ns = (smem_limit - fixed) / kRStageBytes;
    if (ns > kRMaxStages) ns = kRMaxStages;
    if (ns < 2 * KB) return false;
    p.n_stages = ns;
    p.off_ring = q_bytes;
    p.off_misc = p.off_ring + ns * kRStageBytes + 1024;
    p.smem_bytes = 1024 + p.off_misc + kTMiscBytes;
    *plan = p;
    return true;
}

cudaError_t launch_token_scores(const TokenPlan& plan, const CUtensorMap& tm_q, const CUtensorMap& tm_k,
                                const TokenIO& io, cudaStream_t stream) {
    TokArgs a{};
    a.L = io.L; a.P = io.L - io.w; a.w = io.w; a.R = io.Rs; a.Hs = io.Hs; a.d = io.d; a.kv_shift = io.kv_shift;
    a.sl2 = io.sl2;
    a.cph = plan.cph; a.n_tiles = plan.n_tiles; a.n_tiles_prefix = plan.n_tiles_prefix; a.n_stages = plan.n_stages;
    a.q_box_rows = io.Rs < 128 ? io.Rs : 128;
    a.k_box_rows = io.L < kRTile ? io.L : kRTile;
    a.off_ring = plan.off_ring; a.off_misc = plan.off_misc;
    a.cta_stat = io.scratch;
    a.token_scores = io.token_scores;
    a.exits = io.counters;
    a.cnt_a = io.counters + 16;
    a.status = io.status;
    static int smem_set[64] = {0};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || smem_set[dev] < plan.smem_bytes) {
        e = cudaFuncSetAttribute(token_scores_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, plan.smem_bytes);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) smem_set[dev] = plan.smem_bytes;
    }
    void* params[] = {const_cast<CUtensorMap*>(&tm_q), const_cast<CUtensorMap*>(&tm_k), &a};
    // The CTAs of a head wait for one another, so all must be resident: the plan allows at most one CTA
    // per SM (its shared memory) and no more CTAs than SMs, and this path is only taken with the whole
    // GPU, so every CTA becomes resident without waiting for another CTA of this grid. Launched as a
    // programmatic dependent of the preceding kernel, the set-up of this one overlaps the end of that one.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(plan.grid);
    cfg.blockDim = dim3(kTThreads);
    cfg.dynamicSmemBytes = static_cast<size_t>(plan.smem_bytes);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelExC(&cfg, reinterpret_cast<const void*>(token_scores_kernel), params);
}

}  // namespace chunkkv
