// Observation-window attention scoring with the chunk sums fused into the epilogue
// (ChunkKV Algorithm 3: "A <- q_observe K^T" and "Vectorized Chunk Score Calculation"),
// followed by a small finalisation kernel that turns per-panel partial sums into chunk scores.
//
// Per KV head the score matrix is S = Q_obs K^T (R rows = window queries of the grouped
// query heads, L columns = keys). The kernel streams K through shared memory with TMA and
// multiplies 128-row x n_tile-key tiles on the tensor cores (tcgen05, fp32 accumulators in
// tensor memory). The accumulator is consumed in "panels" of wp columns: one thread per query
// row pulls its wp values into registers with one round of TMEM loads (the accumulator buffer
// goes back to the tensor cores as soon as a thread holds its last panel), then computes
//     the panel row maximum, exp2 of every visible element relative to it, the row sum, and
//     the sum over each chunk's columns ("partial", one value per row and chunk).
// Each score element is read once and exponentiated once. The softmax normaliser of a row is
// only known after all panels, so partials are kept per row; every CTA also folds the
// (max, sum) pairs of the panels it processed into one record per head and row. The
// finalisation kernel merges those records into global row maxima / sums and contracts the
// partials over the rows:
//     score[ch] = sum_i partial[ch, i] * exp2(m_panel[i] - m[i]) / l[i].
#include "gather.cuh"
#include "internal.h"
#include "ptx.cuh"
#include "panels.cuh"
#include "select.cuh"

#include <math_constants.h>

namespace chunkkv {

namespace {

constexpr int kMaxStages = 16;
constexpr int kThreads = 576;          // warp 0: TMA, warp 1: UMMA issue, warps 2..17: epilogue
constexpr int kGroups = 4;             // epilogue groups of four warps (one warp per TMEM lane quarter)
constexpr int kTmemCols = 512;
constexpr int kQTileBytes = 128 * 128; // 128 query rows x 64 bf16, swizzled 128-byte rows

struct SharedCtl {
    unsigned long long full[kMaxStages];
    unsigned long long empty[kMaxStages];
    unsigned long long tfull[2];
    unsigned long long tempty[2];
    unsigned long long qfull[2];
    unsigned long long qempty[2];
    uint32_t tmem_base;
    int abort_flag;
};

// Any panel: run-time chunk size, chunk grid clipped at P, causal mask inside the window
// columns [P, L), nothing visible at or beyond L. Window columns add to the row sum only.
template <int WP>
__device__ __forceinline__ void panel_general(const float (&v)[WP], float sl2, bool active, float* part,
                                              int row_stride, int j0, int P, int c, int last_visible,
                                              float* out_m, float* out_l) {
    float mx = -CUDART_INF_F;
#pragma unroll
    for (int u = 0; u < WP; ++u) mx = (j0 + u <= last_visible) ? fmaxf(mx, v[u]) : mx;
    const float neg_m2 = (mx == -CUDART_INF_F) ? 0.f : -mx * sl2;
    float l = 0.f, acc = 0.f;
    int nb = (j0 < P) ? min((j0 / c + 1) * c, P) : 0;   // end (exclusive) of the current chunk
    float* dst = part;
#pragma unroll
    for (int u = 0; u < WP; ++u) {
        const int j = j0 + u;
        const float e = (j <= last_visible) ? ex2_approx(fmaf(v[u], sl2, neg_m2)) : 0.f;
        if (j < P) {
            acc += e;
            if (j + 1 == nb) {
                if (active) *dst = acc;
                dst += row_stride;
                l += acc;
                acc = 0.f;
                nb = min(nb + c, P);
            }
        } else {
            l += e;
        }
    }
    if (j0 < P) {
        const int je = min(j0 + WP, P);
        if (je != P && (je % c) != 0) {   // a chunk continues into the next panel: emit its piece
            if (active) *dst = acc;
            l += acc;
        }
    }
    *out_m = (mx == -CUDART_INF_F) ? -CUDART_INF_F : mx * sl2;
    *out_l = l;
}

constexpr int kFinThreads = 512;
constexpr int kFinPanelCap = 24;      // panels whose scales fit in the finalize kernel's shared memory

struct FinGeom {
    int n_panels;     // per head
    int spp;
    int wp;
    int n_tiles;
    int n_mt;
    int score_grid;   // CTAs of the scoring launch
    int hs_max;
    int C;
};

struct RowStatSmem {
    float red[kFinThreads];
    float red2[kFinThreads];
    int rec_base[256];
};

// Merge the records of the CTAs that touched head h into the global row maxima m[i] and
// 1 / l[i] (written to gm / ginv, which may be shared or global memory). Block-wide: every
// thread of the CTA must call it; the first kFinThreads threads work, each on a slice of the
// records of one row so that the loads overlap.
__device__ __forceinline__ void block_row_stats(const ScoreArgs& a, const FinGeom& g, int h, float* gm,
                                                float* ginv, RowStatSmem& sm) {
    const int tid = threadIdx.x;
    // CTA b owns tiles [total*b/G, total*(b+1)/G): the owner of tile T is floor(((T+1)*G - 1) / total).
    // (32-bit arithmetic: the host checks that total_tiles * (grid + 1) fits)
    const unsigned total = static_cast<unsigned>(a.Hkv) * g.n_tiles, G = g.score_grid;
    const unsigned first_tile = static_cast<unsigned>(h) * g.n_tiles, last_tile = first_tile + g.n_tiles - 1;
    const int b_lo = static_cast<int>(((first_tile + 1) * G - 1) / total);
    const int b_hi = static_cast<int>(((last_tile + 1) * G - 1) / total);
    const int nb = b_hi - b_lo + 1;                 // <= 256: the scoring grid is capped there
    for (int j = tid; j < nb; j += blockDim.x) {
        const unsigned b = b_lo + j;
        const unsigned tb0 = total * b / G, tb1 = total * (b + 1) / G;
        const int head0 = static_cast<int>(tb0 / g.n_tiles);
        // a CTA without tiles (more CTAs than tiles) wrote no record
        sm.rec_base[j] = (tb1 > tb0) ? static_cast<int>((b * g.hs_max + (h - head0)) * (kGroups * 256)) : -1;
    }
    __syncthreads();
    const int rp = (a.R > 128) ? 256 : 128;         // rows padded to the slice stride
    const int ns = kFinThreads / rp;                // record slices per row
    const int gpr = kGroups / g.n_mt;               // groups (records per CTA) that hold a given row
    const int i = tid % rp, sl = tid / rp;
    const bool work = tid < kFinThreads && i < a.R;
    const int g0 = (g.n_mt == 2) ? (i >> 7) * gpr : 0;
    const int rr = i & 127;
    // Each thread folds its slice of the records into one (max, sum) pair. Records are fetched
    // kRecBatch CTAs at a time with every load issued before the first use.
    constexpr int kRecBatch = 6;
    float M = -CUDART_INF_F, Lsum = 0.f;
    if (work) {
        for (int j0 = sl; j0 < nb; j0 += ns * kRecBatch) {
            float rm[kRecBatch][kGroups], rl[kRecBatch][kGroups];
#pragma unroll
            for (int t = 0; t < kRecBatch; ++t) {
                const int j = j0 + t * ns;
                const int base = (j < nb) ? sm.rec_base[j] : -1;
#pragma unroll
                for (int q = 0; q < kGroups; ++q) {
                    const bool have = base >= 0 && q < gpr;
                    const float* rec = a.cta_stat + (have ? base : 0) + (g0 + (have ? q : 0)) * 256 + rr;
                    rm[t][q] = have ? __ldcg(rec) : -CUDART_INF_F;
                    rl[t][q] = have ? __ldcg(rec + 128) : 0.f;
                }
            }
            float bm = M;
#pragma unroll
            for (int t = 0; t < kRecBatch; ++t)
#pragma unroll
                for (int q = 0; q < kGroups; ++q) bm = fmaxf(bm, rm[t][q]);
            float acc = (M == -CUDART_INF_F) ? 0.f : Lsum * ex2_approx(M - bm);
#pragma unroll
            for (int t = 0; t < kRecBatch; ++t)
#pragma unroll
                for (int q = 0; q < kGroups; ++q)
                    acc += (rm[t][q] == -CUDART_INF_F) ? 0.f : rl[t][q] * ex2_approx(rm[t][q] - bm);
            M = bm;
            Lsum = acc;
        }
    }
    float* red_m = sm.red;                           // [kFinThreads] maxima, sums in red2
    if (tid < kFinThreads) { red_m[tid] = M; sm.red2[tid] = Lsum; }
    __syncthreads();
    if (work && sl == 0) {
        float gmax = M;
        for (int s2 = 1; s2 < ns; ++s2) gmax = fmaxf(gmax, red_m[s2 * rp + i]);
        float lt = 0.f;
        for (int s2 = 0; s2 < ns; ++s2) {
            const float pm = red_m[s2 * rp + i];
            lt += (pm == -CUDART_INF_F) ? 0.f : sm.red2[s2 * rp + i] * ex2_approx(pm - gmax);
        }
        gm[i] = gmax;
        ginv[i] = 1.0f / lt;
    }
    __syncthreads();
}

// Chunk scores of the chunks that start in panels [p_lo, p_hi) of head h, whose scales
// f[p - p_lo][i] = exp2(m_panel - m) / l are staged in `fs` (row stride fs_stride). A chunk
// that continues past p_hi takes the scale of the later panels from global memory. One warp
// reduces BATCH chunks at a time with all of their NIT * 32 rows' loads issued before the first
// use (the step is bound by L2 latency, so loads in flight are what counts); fixed order, so
// results are deterministic. Requires R <= 32 * NIT.
template <int NIT, int BATCH>
__device__ __forceinline__ void contract_chunks_t(const ScoreArgs& a, const FinGeom& g, int h, int p_lo, int p_hi,
                                                  int ch0, int ch1, const float* fs, int fs_stride,
                                                  const float* gm, const float* ginv, float* __restrict__ out) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, nwarps = blockDim.x >> 5;
    const float* stat_h = a.stat_m + static_cast<size_t>(h) * g.n_panels * a.R;
    const float* part_h = a.partial + static_cast<size_t>(h) * g.n_panels * g.spp * a.R;
    float* out_h = out + static_cast<size_t>(h) * g.C;
    // When the chunk size divides the panel width, slots are exactly the chunks in order: chunk ch
    // sits at offset ch * R and never straddles panels, so no division is needed per chunk.
    const bool aligned = (g.wp % a.c) == 0 && g.spp * a.c == g.wp;
    for (int cb = ch0 + warp * BATCH; cb < ch1; cb += nwarps * BATCH) {
        float acc[BATCH];
        bool single = true;
        int pa[BATCH], po[BATCH];
        if (aligned) {
            int p_ = cb / g.spp, s_ = cb - p_ * g.spp;
            single = p_ >= p_lo;
#pragma unroll
            for (int u = 0; u < BATCH; ++u) {
                if (u == 0 || cb + u < ch1) {
                    pa[u] = p_;
                    po[u] = (cb + u) * a.R;
                    if (++s_ == g.spp) { s_ = 0; ++p_; }
                } else {
                    pa[u] = pa[u > 0 ? u - 1 : 0];
                    po[u] = po[u > 0 ? u - 1 : 0];
                }
                single = single && pa[u] < p_hi;
                acc[u] = 0.f;
            }
        } else {
#pragma unroll
            for (int u = 0; u < BATCH; ++u) {
                const int ch = min(cb + u, ch1 - 1);
                const int ja = ch * a.c, jb = min(ja + a.c, a.P);
                pa[u] = ja / g.wp;
                single = single && (pa[u] == (jb - 1) / g.wp) && pa[u] >= p_lo && pa[u] < p_hi;
                po[u] = (pa[u] * g.spp + (ch - (pa[u] * g.wp) / a.c)) * a.R;
                acc[u] = 0.f;
            }
        }
        if (single) {       // every chunk of the batch lies in one staged panel
            float pv[BATCH][NIT];
#pragma unroll
            for (int it = 0; it < NIT; ++it) {
                const int i = lane + 32 * it;
#pragma unroll
                for (int u = 0; u < BATCH; ++u) pv[u][it] = (i < a.R) ? __ldcg(part_h + po[u] + i) : 0.f;
            }
#pragma unroll
            for (int it = 0; it < NIT; ++it) {
                const int i = lane + 32 * it;
                if (i < a.R) {
#pragma unroll
                    for (int u = 0; u < BATCH; ++u) acc[u] += pv[u][it] * fs[(pa[u] - p_lo) * fs_stride + i];
                }
            }
        } else {
#pragma unroll
            for (int u = 0; u < BATCH; ++u) {
                const int ch = min(cb + u, ch1 - 1);
                const int ja = ch * a.c, jb = min(ja + a.c, a.P);
                for (int p = ja / g.wp; p <= (jb - 1) / g.wp; ++p) {
                    const float* o = part_h + static_cast<size_t>(p * g.spp + (ch - (p * g.wp) / a.c)) * a.R;
                    const float* so = stat_h + static_cast<size_t>(p) * a.R;
                    for (int i = lane; i < a.R; i += 32)
                        acc[u] += __ldcg(o + i) * (ex2_approx(__ldcg(so + i) - gm[i]) * ginv[i]);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < BATCH; ++u) {
            float v = acc[u];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
            if (lane == 0 && cb + u < ch1) out_h[cb + u] = v;
        }
    }
}

// Chunk scores of panels [p_lo, p_hi) of head h when chunks never straddle panels (the chunk
// size divides the panel width, so panel p holds chunks p * spp .. p * spp + spp - 1 in its slots)
// and R is a multiple of 4. One warp takes PP panels at a time: each lane owns four consecutive
// rows (eight when R > 128), fetches the panel maxima and up to kSlotBatch chunk slots of those
// rows with 16-byte loads that are all issued before the first use, forms the row factors
// exp2(m_panel - m) / l in registers and reduces over the rows with shuffles. Nothing is staged in
// shared memory and no block-wide synchronisation is needed. Fixed order: deterministic.
// gm / ginv: row maxima and reciprocal sums, 16-byte aligned (shared or global memory).
constexpr int kSlotBatch = 6;        // chunk slots in flight per panel (a 60-key panel of 10-key chunks has six)
constexpr int kSlotBatchWide = 16;   // for panels with many slots (token-level: one slot per key)
// RV float4 row groups per lane (1: R <= 128, 2: R <= 256); PP panels in flight per warp; SB slots per panel in flight
template <int RV, int PP, int SB = kSlotBatch>
__device__ __forceinline__ void contract_panels_aligned(const ScoreArgs& a, const FinGeom& g, int h, int p_lo,
                                                        int p_hi, const float* gm, const float* ginv,
                                                        float* __restrict__ out) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    const int r4 = a.R >> 2;                                       // float4 per row vector
    const float4* stat_h = reinterpret_cast<const float4*>(a.stat_m + static_cast<size_t>(h) * g.n_panels * a.R);
    const float4* part_h =
        reinterpret_cast<const float4*>(a.partial + static_cast<size_t>(h) * g.n_panels * g.spp * a.R);
    float* out_h = out + static_cast<size_t>(h) * g.C;
    const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
    const uint64_t drop = l2_policy_evict_first();    // the partial sums are dead once read
    float4 m4[RV], li4[RV];
    bool have[RV];
#pragma unroll
    for (int it = 0; it < RV; ++it) {
        const int i4 = lane + 32 * it;
        have[it] = i4 < r4;
        m4[it] = have[it] ? reinterpret_cast<const float4*>(gm)[i4] : zero4;
        li4[it] = have[it] ? reinterpret_cast<const float4*>(ginv)[i4] : zero4;
    }
    for (int pb = p_lo + warp; pb < p_hi; pb += nwarps * PP) {
        int n_slots[PP], max_slots = 0;
        float4 pm[PP][RV];
#pragma unroll
        for (int q = 0; q < PP; ++q) {
            const int p = pb + q * nwarps;
            n_slots[q] = (p < p_hi) ? max(0, min(g.spp, g.C - p * g.spp)) : 0;   // chunks of the panel that exist
            max_slots = max(max_slots, n_slots[q]);
#pragma unroll
            for (int it = 0; it < RV; ++it)
                pm[q][it] = (n_slots[q] > 0 && have[it]) ? ld_last_use(stat_h + static_cast<size_t>(p) * r4 + lane + 32 * it, drop)
                                                         : zero4;
        }
        if (max_slots == 0) break;                                 // panels past the prefix hold no chunk
        float4 f[PP][RV];
        for (int s0 = 0; s0 < max_slots; s0 += SB) {
            float4 pv[PP][SB][RV];
#pragma unroll
            for (int q = 0; q < PP; ++q) {
                const int ch_base = (pb + q * nwarps) * g.spp;
#pragma unroll
                for (int u = 0; u < SB; ++u) {
                    const bool slot = s0 + u < n_slots[q];
#pragma unroll
                    for (int it = 0; it < RV; ++it)
                        pv[q][u][it] = (slot && have[it])
                                           ? ld_last_use(part_h + static_cast<size_t>(ch_base + s0 + u) * r4 + lane + 32 * it, drop)
                                           : zero4;
                }
            }
            if (s0 == 0) {
#pragma unroll
                for (int q = 0; q < PP; ++q)
#pragma unroll
                    for (int it = 0; it < RV; ++it) {
                        f[q][it].x = ex2_approx(pm[q][it].x - m4[it].x) * li4[it].x;
                        f[q][it].y = ex2_approx(pm[q][it].y - m4[it].y) * li4[it].y;
                        f[q][it].z = ex2_approx(pm[q][it].z - m4[it].z) * li4[it].z;
                        f[q][it].w = ex2_approx(pm[q][it].w - m4[it].w) * li4[it].w;
                    }
            }
            float acc[PP][SB];
#pragma unroll
            for (int q = 0; q < PP; ++q)
#pragma unroll
                for (int u = 0; u < SB; ++u) {
                    float v = 0.f;
#pragma unroll
                    for (int it = 0; it < RV; ++it) {
                        v = fmaf(pv[q][u][it].x, f[q][it].x, v);
                        v = fmaf(pv[q][u][it].y, f[q][it].y, v);
                        v = fmaf(pv[q][u][it].z, f[q][it].z, v);
                        v = fmaf(pv[q][u][it].w, f[q][it].w, v);
                    }
                    acc[q][u] = v;
                }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
#pragma unroll
                for (int q = 0; q < PP; ++q)
#pragma unroll
                    for (int u = 0; u < SB; ++u) acc[q][u] += __shfl_xor_sync(0xffffffffu, acc[q][u], off);
            }
            if (lane == 0) {
#pragma unroll
                for (int q = 0; q < PP; ++q)
#pragma unroll
                    for (int u = 0; u < SB; ++u)
                        if (s0 + u < n_slots[q]) out_h[(pb + q * nwarps) * g.spp + s0 + u] = acc[q][u];
            }
        }
    }
}

__device__ __forceinline__ void contract_chunks(const ScoreArgs& a, const FinGeom& g, int h, int p_lo, int p_hi,
                                                int ch0, int ch1, const float* fs, int fs_stride,
                                                const float* gm, const float* ginv, float* __restrict__ out) {
    if (a.R <= 128)
        contract_chunks_t<4, 8>(a, g, h, p_lo, p_hi, ch0, ch1, fs, fs_stride, gm, ginv, out);
    else
        contract_chunks_t<8, 4>(a, g, h, p_lo, p_hi, ch0, ch1, fs, fs_stride, gm, ginv, out);
}

// Everything the fused layer kernel needs beyond scoring.
struct LayerArgs {
    const uint4* K;
    const uint4* V;
    uint4* out_K;
    uint4* out_V;
    int32_t* out_idx;
    float* chunk_scores;   // [Hkv, C]
    int C, k, n_max;
    int Hkv_out;           // KV heads: selection and gather (scoring heads >> kv_shift)
    unsigned long long* bar_count;   // grid barrier counter (zero between launches); its exit counter 64 bytes on
    int cooperative;                 // host side only: which kind of launch
};

// Grid-wide barrier for a cooperative launch (all CTAs co-resident). One 64-bit counter that
// only grows during a launch: the k-th barrier (k = 0, 1, ...) is passed once the counter has
// reached (k + 1) * nblocks, so nothing is reset between barriers and there is no second flag to
// publish. The counter must be zero when the kernel starts; grid_barrier_finish() puts it back.
// The wait is bounded: on expiry the CTA raises its abort flag and the caller leaves the kernel.
__device__ __forceinline__ bool grid_barrier(unsigned long long* count, unsigned nblocks, unsigned k, int* ok_smem,
                                             volatile int* abort_flag) {
    __syncthreads();
    if (threadIdx.x == 0) {
        bool ok = true;
        unsigned long long old;
        // release: everything this CTA wrote (ordered before by the barrier above) becomes visible
        asm volatile("atom.add.release.gpu.u64 %0, [%1], 1;" : "=l"(old) : "l"(count) : "memory");
        const unsigned long long target = static_cast<unsigned long long>(k + 1) * nblocks;
        if (old + 1ull < target) {
            const long long t0 = clock64();
            unsigned long long cur;
            for (;;) {
                asm volatile("ld.acquire.gpu.u64 %0, [%1];" : "=l"(cur) : "l"(count) : "memory");
                if (cur >= target) break;
                if (clock64() - t0 > kWaitLimitClocks) { ok = false; break; }
            }
        }
        asm volatile("fence.acq_rel.gpu;" ::: "memory");
        if (!ok) *abort_flag = 1;
        *ok_smem = ok ? 1 : 0;
    }
    __syncthreads();
    return *ok_smem != 0;
}

// Called by every CTA after its last barrier: the last one to check out zeroes both counters for
// the next launch (which may use a different grid size). No CTA waits here.
__device__ __forceinline__ void grid_barrier_finish(unsigned long long* count, unsigned long long* exits,
                                                    unsigned nblocks) {
    if (threadIdx.x == 0) {
        const unsigned long long old = atomicAdd(exits, 1ull);
        if (old + 1ull == nblocks) {
            *reinterpret_cast<volatile unsigned long long*>(count) = 0ull;
            *reinterpret_cast<volatile unsigned long long*>(exits) = 0ull;
            __threadfence();
        }
    }
}

struct KernelGeom {
    int n_tiles;      // accumulator tiles per head
    int spp;          // chunk slots per panel
    int n_stages;
    int total_tiles;  // Hkv * n_tiles
    int q_box_rows;   // rows delivered per Q box (min(128, R))
    int k_box_rows;   // rows delivered per K box (min(n_tile, L))
    int hs_max;       // head records per CTA in cta_stat
    int dyn_bytes;    // usable dynamic shared memory after 1024-byte alignment
};

// FUSED = false: scoring only (chunkkv_score). FUSED = true: the whole layer in one cooperative
// launch - after scoring, a grid barrier, then every CTA turns the partial sums of its own
// panels into chunk scores, a second barrier, top-k selection (one CTA per head), a third
// barrier, and the K/V gather on all CTAs.
template <int C_STATIC, int N_MT, int N_TILE, bool FUSED>
__global__ void __launch_bounds__(kThreads, 1)
score_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
             const ScoreArgs a, const KernelGeom g, const LayerArgs la) {
    static_assert(N_MT == 1 || N_MT == 2, "one or two 128-row query tiles");
    static_assert(N_TILE % 16 == 0 && N_TILE * N_MT <= 256, "accumulator tiles must fit half of TMEM");
    constexpr int NQBUF = (N_MT == 1) ? 2 : 1;
    constexpr int TCOLS = 256 / N_MT;              // TMEM columns reserved per accumulator
    constexpr int PPT = kGroups / N_MT;            // panels per tile = groups sharing a query tile
    constexpr int WP = N_TILE / PPT;               // columns per group
    // Compile-time chunk sizes take a group's columns as one panel; the run-time-c path walks
    // them as 32-column panels to keep its register footprint small.
    constexpr int WPP = (C_STATIC > 0) ? WP : 32;  // panel width in keys
    constexpr int SUBS = WP / WPP;                 // panels a thread processes per tile
    static_assert(WP % WPP == 0, "group columns must split into whole panels");
    // ALT: the four groups form two pairs that take alternate accumulator tiles (pair p reads
    // buffer p only); inside a pair each group walks one half of the tile as two panels. The
    // pairs run half a tile period apart, so one pair's waits (accumulator ready, TMEM load)
    // fall into the other pair's arithmetic.
    constexpr bool ALT = (N_MT == 1 && C_STATIC > 0);
    constexpr int ASUBS = ALT ? 2 : SUBS;          // panels a thread processes per tile it takes
    static_assert(C_STATIC == 0 || WPP % C_STATIC == 0, "static chunk size must divide the panel");
    constexpr uint32_t IDESC = umma_idesc_bf16(128, N_TILE);

    extern __shared__ uint8_t smem_raw[];
    __shared__ SharedCtl ctl;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int KB = a.d >> 6;                       // 64-element blocks along d
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t q_base = smem_base;
    const uint32_t stage_bytes = static_cast<uint32_t>(N_TILE) * 128u;
    const uint32_t k_base = q_base + static_cast<uint32_t>(NQBUF * N_MT * KB) * kQTileBytes;
    volatile int* abort_flag = &ctl.abort_flag;
    const uint32_t full0_bar = smem_u32(&ctl.full[0]);   // full[s] at +8*s, empty[s] at +8*(kMaxStages + s)
    const uint32_t n_stages = static_cast<uint32_t>(g.n_stages);

    // CTA b owns tiles [total*b/G, total*(b+1)/G) in (head, tile) order; 32-bit arithmetic (the
    // host checks that total_tiles * (grid + 1) fits).
    const unsigned total = g.total_tiles;
    const int t_begin = static_cast<int>(total * blockIdx.x / gridDim.x);
    const int t_end = static_cast<int>(total * (blockIdx.x + 1) / gridDim.x);
    const int head_begin = t_begin / g.n_tiles, tile_begin = t_begin - head_begin * g.n_tiles;

    if (threadIdx.x == 0) {
        for (int s = 0; s < g.n_stages; ++s) {
            mbar_init(smem_u32(&ctl.full[s]), 1);
            mbar_init(smem_u32(&ctl.empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&ctl.tfull[b]), 1);
            mbar_init(smem_u32(&ctl.tempty[b]), ALT ? 2 * kGroups : 4 * kGroups);   // one arrival per reading warp
            mbar_init(smem_u32(&ctl.qfull[b]), 1);
            mbar_init(smem_u32(&ctl.qempty[b]), 1);
        }
        ctl.abort_flag = 0;
        fence_mbar_init();
        fence_proxy_async();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&ctl.tmem_base), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl.tmem_base;
    // (as a programmatic dependent: dependents may be scheduled as this grid retires; no global memory
    // is touched before the predecessor is complete. Both are no-ops in any other launch.)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (elect_one()) {
            prefetch_tmap(&tm_q);
            prefetch_tmap(&tm_k);
            const uint32_t q_bytes = static_cast<uint32_t>(N_MT * KB * g.q_box_rows) * 128u;
            const uint32_t k_bytes = static_cast<uint32_t>(g.k_box_rows) * 128u;
            int ctr = 0, hs = -1, cur_head = -1;
            // ring position and the parity of the phase to wait for, advanced without dividing
            // (this thread's serial instruction stream bounds how far the loads run ahead)
            uint32_t st = 0, st_par = 1;
            bool ok = true;
            int head = head_begin, tile = tile_begin;
            for (int t = t_begin; t < t_end && ok; ++t, ++tile) {
                if (tile == g.n_tiles) { tile = 0; ++head; }
                if (head != cur_head) {
                    cur_head = head;
                    ++hs;
                    const int qb = hs % NQBUF;
                    if (hs >= NQBUF)
                        ok = mbar_wait(smem_u32(&ctl.qempty[qb]), ((hs / NQBUF) - 1) & 1, abort_flag);
                    if (!ok) break;
                    const uint32_t bar = smem_u32(&ctl.qfull[qb]);
                    mbar_arrive_expect_tx(bar, q_bytes);
                    for (int mt = 0; mt < N_MT; ++mt)
                        for (int kb = 0; kb < KB; ++kb)
                            tma_load_3d(q_base + static_cast<uint32_t>((qb * N_MT + mt) * KB + kb) * kQTileBytes,
                                        &tm_q, bar, kb * 64, mt * 128, head);
                }
                for (int kb = 0; kb < KB; ++kb) {
                    ok = mbar_wait(full0_bar + 8u * (kMaxStages + st), st_par, abort_flag);   // empty[st]
                    if (!ok) break;
                    const uint32_t bar = full0_bar + 8u * st;
                    mbar_arrive_expect_tx(bar, k_bytes);
                    tma_load_3d(k_base + st * stage_bytes, &tm_k, bar, kb * 64, tile * N_TILE, head >> a.kv_shift);
                    ++ctr;
                    if (++st == n_stages) { st = 0; st_par ^= 1u; }
                }
            }
            if (!ok) {
                // Give copies already in flight a bounded chance to land before the CTA exits.
                const int back = min(ctr, g.n_stages);
                for (int i = 1; i <= back; ++i) {
                    const int cc = ctr - i, s = cc % g.n_stages;
                    const long long t0 = clock64();
                    while (!mbar_try_wait(smem_u32(&ctl.full[s]), (cc / g.n_stages) & 1) &&
                           clock64() - t0 < kWaitLimitClocks / 8) {
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ UMMA issuer
        if (elect_one()) {
            int hs = -1, cur_head = -1, ti = 0, qb = 0;
            // The tensor pipe is fed by this one thread: its serial instruction stream sets the
            // floor of the tile period, so the ring position and phase parity advance without
            // dividing and the descriptors of a stage differ only by an added constant.
            uint32_t st = 0, st_par = 0;
            bool ok = true;
            int head = head_begin, tile = tile_begin;
            for (int t = t_begin; t < t_end && ok; ++t, ++ti, ++tile) {
                if (tile == g.n_tiles) { tile = 0; ++head; }
                if (head != cur_head) {
                    if (cur_head >= 0) umma_commit(smem_u32(&ctl.qempty[qb]));
                    cur_head = head;
                    ++hs;
                    qb = hs % NQBUF;
                    ok = mbar_wait(smem_u32(&ctl.qfull[qb]), (hs / NQBUF) & 1, abort_flag);
                    if (!ok) break;
                }
                const int buf = ti & 1, use = ti >> 1;
                ok = mbar_wait(smem_u32(&ctl.tempty[buf]), (use & 1) ^ 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int kb = 0; kb < 2; ++kb) {         // d is 64 or 128: one or two 64-element blocks
                    if (kb >= KB || !ok) break;
                    ok = mbar_wait(full0_bar + 8u * st, st_par, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    // k-steps advance the start-address field (16-byte units) by 32 bytes
                    const uint64_t b_desc = umma_desc_sw128(k_base + st * stage_bytes);
#pragma unroll
                    for (int mt = 0; mt < N_MT; ++mt) {
                        const uint64_t a_desc = umma_desc_sw128(
                            q_base + static_cast<uint32_t>((qb * N_MT + mt) * KB + kb) * kQTileBytes);
                        const uint32_t d_addr = tmem_base + static_cast<uint32_t>(buf * 256 + mt * TCOLS);
#pragma unroll
                        for (int k4 = 0; k4 < 4; ++k4)
                            umma_bf16(d_addr, a_desc + 2u * k4, b_desc + 2u * k4, IDESC, (kb > 0 || k4 > 0) ? 1u : 0u);
                    }
                    umma_commit(full0_bar + 8u * (kMaxStages + st));   // empty[st]
                    if (++st == n_stages) { st = 0; st_par ^= 1u; }
                }
                if (ok) umma_commit(smem_u32(&ctl.tfull[buf]));
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue
        // Four groups of four warps; a group's warps cover the four TMEM lane quarters, i.e. the
        // 128 rows of one query tile. With one query tile the groups split the tile's columns
        // into four panels; with two query tiles, two groups (two panels) serve each of them.
        // A thread pulls its panel into registers and releases the accumulator buffer at once.
        const int grp = (warp - 2) >> 2;
        const int quarter = warp & 3;               // TMEM lane quarter this warp may read
        const int mt = grp / PPT;
        const int pit = grp % PPT;                  // panel within the tile
        const int pair = grp >> 1, half = grp & 1;  // ALT only
        const int row = mt * 128 + quarter * 32 + lane;
        const bool active = row < a.R;
        const int last_visible = a.P + (row % a.w);  // this row sees keys j <= P + r (all < L)
        const int n_panels = g.n_tiles * PPT * SUBS;
        float run_m = -CUDART_INF_F, run_l = 0.f;    // (max, sum) over this thread's panels of the head
        // the partial sums and panel maxima are read back once, shortly: hold them in L2 ahead of streamed data
        const uint64_t keep = l2_policy_evict_last();
        int cur_head = -1, hs = -1, ti = 0;
        auto flush_head = [&]() {
            if (cur_head >= 0 && hs < g.hs_max) {
                float* rec = a.cta_stat +
                             ((static_cast<size_t>(blockIdx.x) * g.hs_max + hs) * kGroups + grp) * 256;
                rec[quarter * 32 + lane] = run_m;
                rec[128 + quarter * 32 + lane] = run_l;
            }
        };
        int head = head_begin, tile = tile_begin;
        for (int t = t_begin; t < t_end; ++t, ++ti, ++tile) {
            if (tile == g.n_tiles) { tile = 0; ++head; }
            if (head != cur_head) {
                flush_head();
                cur_head = head;
                ++hs;
                run_m = -CUDART_INF_F;
                run_l = 0.f;
            }
            if (ALT && (ti & 1) != pair) continue;   // the other pair's tile
            const int buf = ti & 1, use = ti >> 1;
            bool ready = true;                       // one lane polls, the warp follows
            if (lane == 0) ready = mbar_wait(smem_u32(&ctl.tfull[buf]), use & 1, abort_flag);
            if (!__shfl_sync(0xffffffffu, ready, 0)) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) +
                                   static_cast<uint32_t>(buf * 256 + mt * TCOLS + (ALT ? half * 2 * WPP : pit * WP));
#pragma unroll
            for (int sub = 0; sub < ASUBS; ++sub) {
                float v[WPP];
                load_panel<WPP>(taddr + sub * WPP, v);
                if (sub == ASUBS - 1) {              // this thread's last read of the buffer
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&ctl.tempty[buf]));   // it may be overwritten now
                }
                const int panel = ALT ? tile * (PPT * SUBS) + half * 2 + sub : (tile * PPT + pit) * SUBS + sub;
                const size_t panel_id = static_cast<size_t>(head) * n_panels + panel;
                float* part = a.partial + panel_id * g.spp * a.R + row;
                const int j0 = panel * WPP;
                float m2, l;
                if constexpr (C_STATIC > 0) {
                    const int n_pre = a.P - j0;      // chunk slots that start before P hold a chunk
                    auto emit = [&](int ch, float acc) {
                        if (active && ch * C_STATIC < n_pre) st_keep(part + static_cast<size_t>(ch) * a.R, acc, keep);
                    };
                    if (j0 + WPP <= a.P)
                        panel_fast<C_STATIC, WPP>(v, a.sl2, emit, &m2, &l);
                    else
                        panel_static_tail<C_STATIC, WPP>(v, a.sl2, emit, j0, a.P, last_visible, &m2, &l);
                } else {
                    panel_general<WPP>(v, a.sl2, active, part, a.R, j0, a.P, a.c, last_visible, &m2, &l);
                }
                if (active) st_keep(a.stat_m + panel_id * a.R + row, m2, keep);
                // fold into the running record: l is relative to m2, run_l to run_m
                const float nm = fmaxf(run_m, m2);
                const float s_old = (run_m == -CUDART_INF_F) ? 0.f : ex2_approx(run_m - nm);
                const float s_new = (m2 == -CUDART_INF_F) ? 0.f : ex2_approx(m2 - nm);
                run_l = run_l * s_old + l * s_new;
                run_m = nm;
            }
        }
        flush_head();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
    if (ctl.abort_flag) {
        if (threadIdx.x == 0) atomicExch(a.status, 1);
        return;
    }
    if constexpr (FUSED) {
        // The K ring and the Q buffers are idle from here on: reuse the dynamic shared memory.
        uint8_t* dyn = smem_raw + (smem_base - smem_u32(smem_raw));
        RowStatSmem& rs = *reinterpret_cast<RowStatSmem*>(dyn);
        float* gm = reinterpret_cast<float*>(dyn + sizeof(RowStatSmem));
        float* ginv = gm + 256;
        float* fs = ginv + 256;
        const int fs_cap = (g.dyn_bytes - static_cast<int>(sizeof(RowStatSmem)) - 2048) / 4;   // floats
        SelectSmem& ss = *reinterpret_cast<SelectSmem*>(dyn);
        int* bar_ok = reinterpret_cast<int*>(&ctl.tmem_base);     // free again after the dealloc
        FinGeom fg;
        fg.n_panels = g.n_tiles * PPT * SUBS;
        fg.spp = g.spp;
        fg.wp = WPP;
        fg.n_tiles = g.n_tiles;
        fg.n_mt = N_MT;
        fg.score_grid = gridDim.x;
        fg.hs_max = g.hs_max;
        fg.C = la.C;
        constexpr int PPTT = PPT * SUBS;               // panels per tile

        // One CTA per head (grid = Hkv): tiles, row statistics, chunk scores, selection and output
        // rows of a head all belong to the same CTA, so no CTA ever waits for another one.
        const bool solo = static_cast<int>(gridDim.x) == a.Hkv && a.kv_shift == 0;
        if (!solo && !grid_barrier(la.bar_count, gridDim.x, 0, bar_ok, abort_flag)) {
            if (threadIdx.x == 0) atomicExch(a.status, 1);
            return;
        }
        // ---- chunk scores of the panels this CTA scored
        const bool direct = C_STATIC > 0 && (a.R & 3) == 0;
        for (int t = t_begin; t < t_end;) {
            const int head = t / g.n_tiles;
            const int seg_end = min(t_end, (head + 1) * g.n_tiles);
            const int max_tiles = max(1, fs_cap / (PPTT * a.R));
            const size_t stat_base = static_cast<size_t>(head) * fg.n_panels * a.R;
            // Panel maxima of the first batch of tiles are fetched into registers before the row
            // statistics are computed, so that the two round trips to L2 overlap.
            constexpr int kPF = 8;
            float mp[kPF];
            const int tb_first = min(seg_end, t + max_tiles);
            const int p_first = (t - head * g.n_tiles) * PPTT;
            const int n_first = (tb_first - t) * PPTT * a.R;
            const bool prefetched = !direct && n_first <= kPF * kThreads;
            if (prefetched) {
#pragma unroll
                for (int u = 0; u < kPF; ++u) {
                    const int e = threadIdx.x + u * kThreads;
                    mp[u] = (e < n_first) ? __ldcg(a.stat_m + stat_base + static_cast<size_t>(p_first) * a.R + e) : 0.f;
                }
            }
            block_row_stats(a, fg, head, gm, ginv, rs);
            if (direct) {   // chunks never straddle panels: straight from the partial sums, no staging
                const int p_lo = (t - head * g.n_tiles) * PPTT, p_hi = (seg_end - head * g.n_tiles) * PPTT;
                // panels and slots in flight per warp: about a dozen 16-byte loads per lane, whatever
                // the number of chunk slots per panel
                constexpr int SPP = C_STATIC > 0 ? WPP / C_STATIC : 1;
                if constexpr (N_MT == 1) {
                    if constexpr (SPP >= kSlotBatchWide)
                        contract_panels_aligned<1, 1, kSlotBatchWide>(a, fg, head, p_lo, p_hi, gm, ginv, la.chunk_scores);
                    else if constexpr (SPP <= 3)
                        contract_panels_aligned<1, 4, 3>(a, fg, head, p_lo, p_hi, gm, ginv, la.chunk_scores);
                    else
                        contract_panels_aligned<1, 2>(a, fg, head, p_lo, p_hi, gm, ginv, la.chunk_scores);
                } else {
                    if constexpr (SPP <= 2)
                        contract_panels_aligned<2, 2, 2>(a, fg, head, p_lo, p_hi, gm, ginv, la.chunk_scores);
                    else
                        contract_panels_aligned<2, 1>(a, fg, head, p_lo, p_hi, gm, ginv, la.chunk_scores);
                }
                __syncthreads();            // gm / ginv are rewritten for the next head
                t = seg_end;
                continue;
            }
            for (int ta = t; ta < seg_end; ta += max_tiles) {
                const int tb = min(seg_end, ta + max_tiles);
                const int p_lo = (ta - head * g.n_tiles) * PPTT, p_hi = (tb - head * g.n_tiles) * PPTT;
                const int n = (p_hi - p_lo) * a.R;
                if (ta == t && prefetched) {
                    int i = threadIdx.x % a.R;                 // row of element e, advanced without dividing
                    const int step = kThreads % a.R;
#pragma unroll
                    for (int u = 0; u < kPF; ++u) {
                        const int e = threadIdx.x + u * kThreads;
                        if (e < n) fs[e] = ex2_approx(mp[u] - gm[i]) * ginv[i];
                        i += step;
                        i -= (i >= a.R) ? a.R : 0;
                    }
                } else {
                    const float* src = a.stat_m + stat_base + static_cast<size_t>(p_lo) * a.R;
                    for (int e0 = threadIdx.x; e0 < n; e0 += 8 * kThreads) {   // eight loads in flight per thread
                        float t8[8];
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            const int e = e0 + u * kThreads;
                            t8[u] = (e < n) ? __ldcg(src + e) : 0.f;
                        }
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            const int e = e0 + u * kThreads;
                            if (e < n) {
                                const int i = e % a.R;
                                fs[e] = ex2_approx(t8[u] - gm[i]) * ginv[i];
                            }
                        }
                    }
                }
                __syncthreads();
                const int key_a = p_lo * WPP, key_b = min(p_hi * WPP, a.P);
                if (key_a < key_b)   // chunks whose first key lies in [key_a, key_b)
                    contract_chunks(a, fg, head, p_lo, p_hi, (key_a + a.c - 1) / a.c, (key_b + a.c - 1) / a.c, fs,
                                    a.R, gm, ginv, la.chunk_scores);
                __syncthreads();
            }
            t = seg_end;
        }
        if (!solo && !grid_barrier(la.bar_count, gridDim.x, 1, bar_ok, abort_flag)) {
            if (threadIdx.x == 0) atomicExch(a.status, 1);
            return;
        }
        // ---- top-k selection: one CTA per head
        const bool rows_elsewhere = la.out_K == nullptr;   // the rows are gathered by a separate launch
        if (rows_elsewhere && !solo) {
            // Nothing follows the selection in this launch: CTAs check out of the barrier now
            // (no CTA waits on it again) and those without a head leave at once.
            grid_barrier_finish(la.bar_count, la.bar_count + 8, gridDim.x);
            if (static_cast<int>(blockIdx.x) >= la.Hkv_out) return;
        }
        for (int h = blockIdx.x; h < la.Hkv_out; h += gridDim.x) {
            const float* sc = la.chunk_scores + (static_cast<size_t>(h) << a.kv_shift) * la.C;
            const float* sc2 = a.kv_shift ? sc + la.C : nullptr;        // the head's second scoring head
            int32_t* out = la.out_idx + static_cast<size_t>(h) * la.n_max;
            if (la.C <= kThreads * 6) {
                select_head_regs<6>(sc, sc2, a.L, a.w, a.c, la.C, la.k, la.n_max, out, ss);
            } else {
                // keys go to the idle dynamic shared memory behind the selection scratch; if they do
                // not fit there (token-level selection of very long sequences) they replace the
                // chunk scores, which nothing reads after the selection
                uint32_t* kbuf = reinterpret_cast<uint32_t*>(dyn + ((sizeof(SelectSmem) + 127) & ~size_t(127)));
                const bool fits = static_cast<size_t>(la.C) * 4 + sizeof(SelectSmem) + 256 <= static_cast<size_t>(g.dyn_bytes);
                if (fits)
                    select_head_smem(sc, sc2, a.L, a.w, a.c, la.C, la.k, la.n_max, out, ss, kbuf);
                else
                    select_head_rows(sc, sc2, a.L, a.w, a.c, la.C, la.k, la.n_max, out, ss,
                                     reinterpret_cast<uint32_t*>(const_cast<float*>(sc)));
            }
        }
        if (rows_elsewhere) return;
        if (!solo) {
            if (!grid_barrier(la.bar_count, gridDim.x, 2, bar_ok, abort_flag)) {
                if (threadIdx.x == 0) atomicExch(a.status, 1);
                return;
            }
            grid_barrier_finish(la.bar_count, la.bar_count + 8, gridDim.x);   // exit counter sits 64 bytes on
        }
        // ---- gather: the Hkv * n_max output rows are split evenly over the CTAs
        const int vpr = a.d >> 3;
        const int rows_per_pass = (kThreads / vpr) * kGatherRowsPerThread;
        // (32-bit arithmetic: the host checks that Hkv * n_max * (grid + 1) fits)
        const unsigned rows_total = static_cast<unsigned>(la.Hkv_out) * la.n_max;
        const int r_begin = static_cast<int>(rows_total * blockIdx.x / gridDim.x);
        const int r_end = static_cast<int>(rows_total * (blockIdx.x + 1) / gridDim.x);
        // The indices of this CTA's rows (contiguous in [Hkv, n_max] order) go to shared memory
        // first, so that each pass below waits for one round trip (the rows) instead of two.
        int32_t* sidx = reinterpret_cast<int32_t*>(dyn);
        const bool staged = (r_end - r_begin) * 4 <= g.dyn_bytes - 2048;
        if (staged) {
            __syncthreads();                                   // the selection scratch is no longer read
            for (int i = threadIdx.x; i < r_end - r_begin; i += kThreads) sidx[i] = __ldcg(la.out_idx + r_begin + i);
            __syncthreads();
        }
        for (int r0 = r_begin; r0 < r_end;) {
            const int h = r0 / la.n_max;
            const int n0 = r0 - h * la.n_max;
            // rows [n0, n_hi) of head h in this pass
            const int n_hi = min(la.n_max, min(r_end - h * la.n_max, n0 + rows_per_pass));
            const int32_t* ih = la.out_idx + static_cast<size_t>(h) * la.n_max;
            if (staged) {
                const int32_t* sh = sidx + (h * la.n_max - r_begin);   // sh[n] = index of row n of head h
                if (vpr == 16)
                    gather_rows<16, false>(la.K + static_cast<size_t>(h) * a.L * 16, la.V + static_cast<size_t>(h) * a.L * 16,
                                           sh, a.L, n_hi, n0, threadIdx.x, kThreads,
                                           la.out_K + static_cast<size_t>(h) * la.n_max * 16,
                                           la.out_V + static_cast<size_t>(h) * la.n_max * 16, nullptr);
                else
                    gather_rows<8, false>(la.K + static_cast<size_t>(h) * a.L * 8, la.V + static_cast<size_t>(h) * a.L * 8,
                                          sh, a.L, n_hi, n0, threadIdx.x, kThreads,
                                          la.out_K + static_cast<size_t>(h) * la.n_max * 8,
                                          la.out_V + static_cast<size_t>(h) * la.n_max * 8, nullptr);
            } else if (vpr == 16)
                gather_rows<16, true>(la.K + static_cast<size_t>(h) * a.L * 16, la.V + static_cast<size_t>(h) * a.L * 16, ih,
                                      a.L, n_hi, n0, threadIdx.x, kThreads,
                                      la.out_K + static_cast<size_t>(h) * la.n_max * 16,
                                      la.out_V + static_cast<size_t>(h) * la.n_max * 16, nullptr);
            else
                gather_rows<8, true>(la.K + static_cast<size_t>(h) * a.L * 8, la.V + static_cast<size_t>(h) * a.L * 8, ih,
                                     a.L, n_hi, n0, threadIdx.x, kThreads,
                                     la.out_K + static_cast<size_t>(h) * la.n_max * 8,
                                     la.out_V + static_cast<size_t>(h) * la.n_max * 8, nullptr);
            r0 += n_hi - n0;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Finalisation, two small kernels:
//   rowstats_kernel  merges the per-CTA records of each head into global row maxima m[i] and
//                    1 / l[i];
//   finalize_kernel  computes the scale f[p][i] = exp2(m_panel[p][i] - m[i]) / l[i] for the
//                    panels its chunks touch (kept in shared memory) and contracts
//                    partial[ch][.] * f over the R rows, one warp working on four chunks at a time.
// All reductions have a fixed order, so results are deterministic.
__global__ void __launch_bounds__(kFinThreads)
rowstats_kernel(const ScoreArgs a, const FinGeom g) {
    __shared__ RowStatSmem sm;
    const int h = blockIdx.x;
    block_row_stats(a, g, h, a.row_stat + static_cast<size_t>(h) * 512, a.row_stat + static_cast<size_t>(h) * 512 + 256, sm);
}

// grid = (blocks per head, Hkv): chunk scores from partial sums, see the header of this section.
__global__ void __launch_bounds__(kFinThreads)
finalize_kernel(const ScoreArgs a, const FinGeom g, float* __restrict__ out) {
    __shared__ float gm[256];
    __shared__ float ginv[256];
    __shared__ float fs[kFinPanelCap * 256];
    const int h = blockIdx.y;
    const int tid = threadIdx.x;
    if (tid < a.R) {
        gm[tid] = a.row_stat[static_cast<size_t>(h) * 512 + tid];
        ginv[tid] = a.row_stat[static_cast<size_t>(h) * 512 + 256 + tid];
    }
    __syncthreads();
    const int per_block = (g.C + gridDim.x - 1) / gridDim.x;
    const int ch0 = blockIdx.x * per_block, ch1 = min(ch0 + per_block, g.C);
    if (ch0 >= ch1) return;
    const int p_lo = (ch0 * a.c) / g.wp;
    const int p_hi = min(p_lo + kFinPanelCap, (min(ch1 * a.c, a.P) - 1) / g.wp + 1);
    const size_t stat_base = static_cast<size_t>(h) * g.n_panels * a.R;
    const int n = (p_hi - p_lo) * a.R;
    for (int e = tid; e < n; e += kFinThreads) {
        const int pp = e / a.R, i = e - pp * a.R;
        fs[pp * 256 + i] =
            ex2_approx(a.stat_m[stat_base + static_cast<size_t>(p_lo + pp) * a.R + i] - gm[i]) * ginv[i];
    }
    __syncthreads();
    contract_chunks(a, g, h, p_lo, p_hi, ch0, ch1, fs, 256, gm, ginv, out);
}

template <int C_STATIC, int N_MT, int N_TILE, bool FUSED>
cudaError_t launch_variant(const ScorePlan& plan, const CUtensorMap& tm_q, const CUtensorMap& tm_k,
                           const ScoreArgs& args, const LayerArgs& la, cudaStream_t stream) {
    auto kern = score_kernel<C_STATIC, N_MT, N_TILE, FUSED>;
    // Opt in to large dynamic shared memory once per device and variant (not a stream operation,
    // so later launches stay free of it, e.g. inside a stream capture).
    static int smem_set[64] = {0};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || smem_set[dev] < plan.smem_bytes) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, plan.smem_bytes);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) smem_set[dev] = plan.smem_bytes;
    }
    KernelGeom g;
    g.n_tiles = plan.n_tiles;
    g.spp = plan.spp;
    g.n_stages = plan.n_stages;
    g.total_tiles = args.Hkv * plan.n_tiles;
    g.q_box_rows = args.R < 128 ? args.R : 128;
    g.k_box_rows = args.L < N_TILE ? args.L : N_TILE;
    g.hs_max = plan.hs_max;
    g.dyn_bytes = plan.smem_bytes - 1024;
    if (FUSED) {
        // Cooperative launch: the grid barriers need every CTA resident (one per SM). With one CTA
        // per head the kernel has no grid barrier, but it keeps this launch: its CTAs then start
        // together, which measured 9 % faster with 18 layers in flight than an ordinary launch.
        void* params[] = {const_cast<CUtensorMap*>(&tm_q), const_cast<CUtensorMap*>(&tm_k),
                          const_cast<ScoreArgs*>(&args), &g, const_cast<LayerArgs*>(&la)};
        if (la.cooperative)
            return cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(kern), dim3(plan.grid), dim3(kThreads),
                                               params, static_cast<size_t>(plan.smem_bytes), stream);
        // With the whole GPU to itself (no lanes) every CTA becomes resident anyway - at most one per SM, no
        // more CTAs than SMs - and the kernel is launched as a programmatic dependent of its predecessor
        // instead: its set-up overlaps the end of that one.
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(plan.grid);
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = static_cast<size_t>(plan.smem_bytes);
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        return cudaLaunchKernelExC(&cfg, reinterpret_cast<const void*>(kern), params);
    } else {
        kern<<<plan.grid, kThreads, plan.smem_bytes, stream>>>(tm_q, tm_k, args, g, la);
        return cudaGetLastError();
    }
}

template <bool FUSED>
cudaError_t dispatch_variant(const ScorePlan& plan, const CUtensorMap& tm_q, const CUtensorMap& tm_k,
                             const ScoreArgs& args, const LayerArgs& la, cudaStream_t stream) {
    if (plan.n_mt == 1) {
        if (plan.c_static == 10) return launch_variant<10, 1, 240, FUSED>(plan, tm_q, tm_k, args, la, stream);
        if (plan.c_static == 20) return launch_variant<20, 1, 240, FUSED>(plan, tm_q, tm_k, args, la, stream);
        if (plan.c_static == 1) return launch_variant<1, 1, 256, FUSED>(plan, tm_q, tm_k, args, la, stream);
        return launch_variant<0, 1, 256, FUSED>(plan, tm_q, tm_k, args, la, stream);
    }
    if (plan.c_static == 10) return launch_variant<10, 2, 80, FUSED>(plan, tm_q, tm_k, args, la, stream);
    if (plan.c_static == 20) return launch_variant<20, 2, 80, FUSED>(plan, tm_q, tm_k, args, la, stream);
    return launch_variant<0, 2, 128, FUSED>(plan, tm_q, tm_k, args, la, stream);
}

}  // namespace

bool make_score_plan(int L, int R, int Hkv, int d, int c, int num_sms, int smem_limit, bool full_grid,
                     ScorePlan* plan) {
    if (R < 1 || R > 256 || (d != 64 && d != 128) || c < 1 || L < 1 || Hkv < 1 || num_sms < 1) return false;
    ScorePlan p{};
    p.n_mt = (R + 127) / 128;
    // Chunk sizes with a compiled-in variant use panels that are a multiple of the chunk size;
    // every other chunk size runs the run-time-c variant on the widest tile.
    p.c_static = 0;
    // (two query tiles share the accumulator columns: 80 keys per tile, 40 per epilogue panel)
    if (c == 10 || c == 20) { p.c_static = c; p.n_tile = p.n_mt == 1 ? 240 : 80; }
    else if (p.n_mt == 1 && c == 1) { p.c_static = 1; p.n_tile = 256; }
    else p.n_tile = 256 / p.n_mt;
    p.wp = p.c_static ? p.n_tile / (kGroups / p.n_mt) : 32;
    p.n_tiles = (L + p.n_tile - 1) / p.n_tile;
    p.n_panels = p.n_tiles * (p.n_tile / p.wp);
    p.spp = p.c_static ? p.wp / p.c_static : (p.wp + c - 1) / c + 1;
    const long long total = static_cast<long long>(Hkv) * p.n_tiles;
    p.grid = static_cast<int>((total < num_sms && !full_grid) ? total : num_sms);
    // A CTA count that is a multiple of the head count makes every CTA's tile range end on a head
    // boundary (tiles are dealt out as total * b / grid), so no CTA has to switch heads mid-way.
    // Taken only where it gives up at most 1/16 of the CTAs (148 -> 144 for 8 heads, not 18 -> 16).
    if (p.grid >= Hkv && p.grid % Hkv != 0 && total >= p.grid && (p.grid % Hkv) * 16 <= p.grid) p.grid -= p.grid % Hkv;
    if (total * (static_cast<long long>(num_sms) + 1) >= (1LL << 32)) return false;   // kernels use 32-bit tile arithmetic
    if (p.grid > 256) p.grid = 256;   // rowstats_kernel indexes at most 256 CTA records per head
    const int tiles_per_cta = static_cast<int>((total + p.grid - 1) / p.grid);
    p.hs_max = (tiles_per_cta + p.n_tiles - 1) / p.n_tiles + 1;
    const int KB = d / 64;
    const int nqbuf = p.n_mt == 1 ? 2 : 1;
    const int q_bytes = nqbuf * p.n_mt * KB * kQTileBytes;
    const int stage = p.n_tile * 128;
    int ns = (smem_limit - 1024 - q_bytes) / stage;
    if (ns > kMaxStages) ns = kMaxStages;
    if (ns < 2) return false;
    p.n_stages = ns;
    p.smem_bytes = 1024 + q_bytes + ns * stage;
    *plan = p;
    return true;
}

size_t score_scratch_floats(const ScorePlan& plan, int Hkv, int R) {
    const size_t panels = static_cast<size_t>(Hkv) * plan.n_panels;
    return panels * R + static_cast<size_t>(plan.grid) * plan.hs_max * (kGroups * 256) +
           static_cast<size_t>(Hkv) * 512 + panels * plan.spp * R;
}

void score_scratch_layout(const ScorePlan& plan, int Hkv, int R, float* base, ScoreArgs* args) {
    const size_t panels = static_cast<size_t>(Hkv) * plan.n_panels;
    args->stat_m = base;
    args->cta_stat = base + panels * R;
    args->row_stat = args->cta_stat + static_cast<size_t>(plan.grid) * plan.hs_max * (kGroups * 256);
    args->partial = args->row_stat + static_cast<size_t>(Hkv) * 512;
}

cudaError_t launch_score(const ScorePlan& plan, const CUtensorMap& tm_q, const CUtensorMap& tm_k,
                         const ScoreArgs& args, cudaStream_t stream) {
    LayerArgs none{};
    return dispatch_variant<false>(plan, tm_q, tm_k, args, none, stream);
}

cudaError_t launch_layer_fused(const ScorePlan& plan, const CUtensorMap& tm_q, const CUtensorMap& tm_k,
                               const ScoreArgs& args, const FusedLayerIO& io, cudaStream_t stream) {
    LayerArgs la;
    la.K = static_cast<const uint4*>(io.K);
    la.V = static_cast<const uint4*>(io.V);
    la.out_K = static_cast<uint4*>(io.out_K);
    la.out_V = static_cast<uint4*>(io.out_V);
    la.out_idx = io.out_idx;
    la.chunk_scores = io.chunk_scores;
    la.C = io.C;
    la.k = io.k;
    la.n_max = io.n_max;
    la.Hkv_out = io.Hkv_out;
    la.bar_count = io.bar_count;
    la.cooperative = io.cooperative ? 1 : 0;
    return dispatch_variant<true>(plan, tm_q, tm_k, args, la, stream);
}

__global__ void pair_sum_kernel(const float* __restrict__ in, float* __restrict__ out, int C, size_t n) {
    const size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const size_t h = i / C, ch = i - h * C;
    out[i] = in[(2 * h) * C + ch] + in[(2 * h + 1) * C + ch];
}

// Chunk scores for compile-time chunk sizes (chunks never straddle panels) and R % 4 == 0, in CTAs
// of two warps: small enough (64 threads) to run on an SM beside a resident CTA of the scoring
// kernel, so the L2-latency-bound contraction of one layer spreads over every SM while other
// layers are being scored. grid = (blocks per head, Hkv); a block takes a contiguous panel range.
constexpr int kFinSmallThreads = 64;
template <int RV, int PP, int SB>
__global__ void __launch_bounds__(kFinSmallThreads)
finalize_panels_kernel(const ScoreArgs a, const FinGeom g, float* __restrict__ out) {
    const int h = blockIdx.y;
    const int n_p = (a.P + g.wp - 1) / g.wp;                       // panels that hold chunks
    const int per = (n_p + gridDim.x - 1) / gridDim.x;
    const int p_lo = blockIdx.x * per, p_hi = min(p_lo + per, n_p);
    if (p_lo >= p_hi) return;
    const float* rs = a.row_stat + static_cast<size_t>(h) * 512;
    contract_panels_aligned<RV, PP, SB>(a, g, h, p_lo, p_hi, rs, rs + 256, out);
}

cudaError_t launch_pair_sum(const float* in, float* out, int Hkv, int C, cudaStream_t stream) {
    const size_t n = static_cast<size_t>(Hkv) * C;
    if (n == 0) return cudaSuccess;
    pair_sum_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, stream>>>(in, out, C, n);
    return cudaGetLastError();
}

cudaError_t launch_finalize(const ScorePlan& plan, const ScoreArgs& args, int C, float* out_scores,
                            int num_sms, cudaStream_t stream) {
    if (C <= 0) return cudaSuccess;
    int bx = (2 * num_sms + args.Hkv - 1) / args.Hkv;
    const int max_bx = (C + 15) / 16;
    if (bx > max_bx) bx = max_bx;
    if (bx < 1) bx = 1;
    FinGeom g;
    g.n_panels = plan.n_panels;
    g.spp = plan.spp;
    g.wp = plan.wp;
    g.n_tiles = plan.n_tiles;
    g.n_mt = plan.n_mt;
    g.score_grid = plan.grid;
    g.hs_max = plan.hs_max;
    g.C = C;
    rowstats_kernel<<<args.Hkv, kFinThreads, 0, stream>>>(args, g);
    if (plan.c_static > 0 && (args.R & 3) == 0) {
        const int n_p = (args.P + plan.wp - 1) / plan.wp;
        int px = (4 * num_sms + args.Hkv - 1) / args.Hkv;          // about four small CTAs per SM
        const int max_px = (n_p + 3) / 4;                          // at least four panels per CTA
        if (px > max_px) px = max_px;
        if (px < 1) px = 1;
        dim3 pgrid(px, args.Hkv);
        // panels x slots in flight per warp chosen so that a lane has a dozen or more 16-byte loads out
        if (args.R <= 128) {
            if (plan.spp >= kSlotBatchWide)
                finalize_panels_kernel<1, 1, kSlotBatchWide><<<pgrid, kFinSmallThreads, 0, stream>>>(args, g, out_scores);
            else if (plan.spp <= 3)
                finalize_panels_kernel<1, 4, 3><<<pgrid, kFinSmallThreads, 0, stream>>>(args, g, out_scores);
            else
                finalize_panels_kernel<1, 2, kSlotBatch><<<pgrid, kFinSmallThreads, 0, stream>>>(args, g, out_scores);
        } else {
            if (plan.spp <= 2)
                finalize_panels_kernel<2, 4, 2><<<pgrid, kFinSmallThreads, 0, stream>>>(args, g, out_scores);
            else if (plan.spp <= 4)
                finalize_panels_kernel<2, 2, 4><<<pgrid, kFinSmallThreads, 0, stream>>>(args, g, out_scores);
            else
                finalize_panels_kernel<2, 1, kSlotBatch><<<pgrid, kFinSmallThreads, 0, stream>>>(args, g, out_scores);
        }
        return cudaGetLastError();
    }
    dim3 grid(bx, args.Hkv);
    finalize_kernel<<<grid, kFinThreads, 0, stream>>>(args, g, out_scores);
    return cudaGetLastError();
}

}  // namespace chunkkv
