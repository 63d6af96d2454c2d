// Observation-window attention scoring with the chunk sums fused into the epilogue
// (ChunkKV Algorithm 3: "A <- q_observe K^T" and "Vectorized Chunk Score Calculation"),
// followed by a small finalisation kernel that turns per-tile partial sums into chunk scores.
//
// Per KV head the score matrix is S = Q_obs K^T (R rows = window queries of the grouped
// query heads, L columns = keys). The kernel streams K through shared memory with TMA,
// multiplies 128-row x n_tile-key tiles on the tensor cores (tcgen05, fp32 accumulators in
// tensor memory) and lets one thread per query row reduce its row of the tile:
//     tile row maximum, exp2 of every visible element relative to it, row sum, and the sum
//     over each chunk's columns ("partial", one value per row and chunk).
// Each score element is exponentiated exactly once. Because the softmax normaliser of a row
// is only known after all tiles, partials are kept per row; the finalisation kernel combines
// tile statistics into global row maxima / sums and contracts partials over the rows:
//     score[ch] = sum_i partial[ch, i] * exp2(m_tile[i] - m[i]) / l[i].
#include "internal.h"
#include "ptx.cuh"

#include <math_constants.h>

namespace chunkkv {

namespace {

constexpr int kMaxStages = 16;
constexpr int kThreads = 320;          // warp 0: TMA, warp 1: UMMA issue, warps 2..9: epilogue
constexpr int kTmemCols = 512;
constexpr int kQTileBytes = 128 * 128; // 128 query rows x 64 bf16, swizzled 128-byte rows

struct KernelGeom {
    int n_tiles;      // tiles per head
    int spt;          // chunk slots per tile
    int n_stages;
    int total_tiles;  // Hkv * n_tiles
    int q_box_rows;   // rows delivered per Q box (min(128, R))
    int k_box_rows;   // rows delivered per K box (min(n_tile, L))
};

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

// One thread owns one query row of the tile. `taddr` points at the thread's lane quarter and
// the first column of the accumulator. All reads use 32- or 16-column TMEM loads.
// UNROLL_BLOCKS: unroll across the 32-column blocks too, so that column numbers are
// compile-time constants in `f` (the fast path needs that; the general path does not).
template <int N_TILE, bool UNROLL_BLOCKS, typename F>
__device__ __forceinline__ void for_each_column(uint32_t taddr, F&& f) {
    constexpr int FULL = N_TILE / 32;
    if constexpr (UNROLL_BLOCKS) {
#pragma unroll
        for (int b = 0; b < FULL; ++b) {
            float v[32];
            tmem_ld_x32(taddr + b * 32, v);
            tmem_ld_wait();
#pragma unroll
            for (int u = 0; u < 32; ++u) f(b * 32 + u, v[u]);
        }
    } else {
#pragma unroll 1
        for (int b = 0; b < FULL; ++b) {
            float v[32];
            tmem_ld_x32(taddr + b * 32, v);
            tmem_ld_wait();
#pragma unroll
            for (int u = 0; u < 32; ++u) f(b * 32 + u, v[u]);
        }
    }
    if constexpr (N_TILE % 32 != 0) {
        float v[16];
        tmem_ld_x16(taddr + FULL * 32, v);
        tmem_ld_wait();
#pragma unroll
        for (int u = 0; u < 16; ++u) f(FULL * 32 + u, v[u]);
    }
}

// Tile that lies wholly inside the prefix and starts on a chunk boundary, chunk size known at
// compile time: every branch below folds away after unrolling.
template <int C, int N_TILE>
__device__ __forceinline__ void tile_fast(uint32_t taddr, float sl2, bool active, float* part,
                                          int row_stride, float* out_m, float* out_l) {
    float mx = -CUDART_INF_F;
#pragma unroll
    for (int cb = 0; cb < N_TILE; cb += 32) {
        if (cb + 32 <= N_TILE) {
            float v[32];
            tmem_ld_x32(taddr + cb, v);
            tmem_ld_wait();
#pragma unroll
            for (int u = 0; u < 32; u += 2) mx = fmax3(mx, v[u], v[u + 1]);
        } else {
            float v[16];
            tmem_ld_x16(taddr + cb, v);
            tmem_ld_wait();
#pragma unroll
            for (int u = 0; u < 16; u += 2) mx = fmax3(mx, v[u], v[u + 1]);
        }
    }
    const float neg_m2 = -mx * sl2;
    float l = 0.f, acc = 0.f;
    for_each_column<N_TILE, true>(taddr, [&](int j, float x) {
        const float e = ex2_approx(fmaf(x, sl2, neg_m2));
        acc += e;
        if ((j + 1) % C == 0) {
            if (active) part[static_cast<size_t>((j + 1) / C - 1) * row_stride] = acc;
            l += acc;
            acc = 0.f;
        }
    });
    *out_m = mx * sl2;
    *out_l = l;
}

// Any tile: run-time chunk size, chunk grid clipped at P, causal mask inside the window
// columns [P, L), nothing visible at or beyond L. Window columns add to the row sum only.
template <int N_TILE>
__device__ __forceinline__ void tile_general(uint32_t taddr, float sl2, bool active, float* part,
                                             int row_stride, int j0, int P, int L, int c, int r,
                                             float* out_m, float* out_l) {
    const int last_visible = min(P + r, L - 1);   // this row sees keys j <= P + r
    float mx = -CUDART_INF_F;
    for_each_column<N_TILE, false>(taddr, [&](int u, float x) {
        const bool vis = (j0 + u) <= last_visible;
        mx = vis ? fmaxf(mx, x) : mx;
    });
    const float neg_m2 = (mx == -CUDART_INF_F) ? 0.f : -mx * sl2;
    float l = 0.f, acc = 0.f;
    int slot = 0;
    int nb = (j0 < P) ? min((j0 / c + 1) * c, P) : 0;   // end (exclusive) of the current chunk
    for_each_column<N_TILE, false>(taddr, [&](int u, float x) {
        const int j = j0 + u;
        const bool vis = j <= last_visible;
        const float e = vis ? ex2_approx(fmaf(x, sl2, neg_m2)) : 0.f;
        if (j < P) {
            acc += e;
            if (j + 1 == nb) {
                if (active) part[static_cast<size_t>(slot) * row_stride] = acc;
                l += acc;
                acc = 0.f;
                ++slot;
                nb = min(nb + c, P);
            }
        } else {
            l += e;
        }
    });
    if (j0 < P) {
        const int je = min(j0 + N_TILE, P);
        if (je != P && (je % c) != 0) {   // a chunk continues into the next tile: emit its piece
            if (active) part[static_cast<size_t>(slot) * row_stride] = acc;
            l += acc;
        }
    }
    *out_m = (mx == -CUDART_INF_F) ? -CUDART_INF_F : mx * sl2;
    *out_l = l;
}

template <int C_STATIC, int N_MT, int N_TILE>
__global__ void __launch_bounds__(kThreads, 1)
score_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
             const ScoreArgs a, const KernelGeom g) {
    static_assert(N_MT == 1 || N_MT == 2, "one or two 128-row query tiles");
    static_assert(N_TILE % 16 == 0 && N_TILE * N_MT <= 256, "accumulator tiles must fit half of TMEM");
    static_assert(C_STATIC == 0 || N_TILE % C_STATIC == 0, "static chunk size must divide the tile");
    constexpr int NQBUF = (N_MT == 1) ? 2 : 1;
    constexpr int TCOLS = 256 / N_MT;              // TMEM columns reserved per accumulator
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

    const long long total = g.total_tiles;
    const int t_begin = static_cast<int>(total * blockIdx.x / gridDim.x);
    const int t_end = static_cast<int>(total * (blockIdx.x + 1) / gridDim.x);

    if (threadIdx.x == 0) {
        for (int s = 0; s < g.n_stages; ++s) {
            mbar_init(smem_u32(&ctl.full[s]), 1);
            mbar_init(smem_u32(&ctl.empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&ctl.tfull[b]), 1);
            mbar_init(smem_u32(&ctl.tempty[b]), 128 * N_MT);
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

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (elect_one()) {
            prefetch_tmap(&tm_q);
            prefetch_tmap(&tm_k);
            const uint32_t q_bytes = static_cast<uint32_t>(N_MT * KB * g.q_box_rows) * 128u;
            const uint32_t k_bytes = static_cast<uint32_t>(g.k_box_rows) * 128u;
            int ctr = 0, hs = -1, cur_head = -1;
            bool ok = true;
            for (int t = t_begin; t < t_end && ok; ++t) {
                const int head = t / g.n_tiles, tile = t - head * g.n_tiles;
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
                    const int s = ctr % g.n_stages;
                    ok = mbar_wait(smem_u32(&ctl.empty[s]), ((ctr / g.n_stages) & 1) ^ 1, abort_flag);
                    if (!ok) break;
                    const uint32_t bar = smem_u32(&ctl.full[s]);
                    mbar_arrive_expect_tx(bar, k_bytes);
                    tma_load_3d(k_base + static_cast<uint32_t>(s) * stage_bytes, &tm_k, bar, kb * 64,
                                tile * N_TILE, head);
                    ++ctr;
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
            int ctr = 0, hs = -1, cur_head = -1, ti = 0, qb = 0;
            bool ok = true;
            for (int t = t_begin; t < t_end && ok; ++t, ++ti) {
                const int head = t / g.n_tiles;
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
                for (int kb = 0; kb < KB && ok; ++kb) {
                    const int s = ctr % g.n_stages;
                    ok = mbar_wait(smem_u32(&ctl.full[s]), (ctr / g.n_stages) & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t b_addr = k_base + static_cast<uint32_t>(s) * stage_bytes;
#pragma unroll
                    for (int mt = 0; mt < N_MT; ++mt) {
                        const uint32_t a_addr =
                            q_base + static_cast<uint32_t>((qb * N_MT + mt) * KB + kb) * kQTileBytes;
                        const uint32_t d_addr = tmem_base + static_cast<uint32_t>(buf * 256 + mt * TCOLS);
#pragma unroll
                        for (int k4 = 0; k4 < 4; ++k4) {
                            umma_bf16(d_addr, umma_desc_sw128(a_addr + k4 * 32),
                                      umma_desc_sw128(b_addr + k4 * 32), IDESC,
                                      (kb > 0 || k4 > 0) ? 1u : 0u);
                        }
                    }
                    umma_commit(smem_u32(&ctl.empty[s]));
                    ++ctr;
                }
                if (ok) umma_commit(smem_u32(&ctl.tfull[buf]));
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue
        const int grp = (warp - 2) >> 2;            // 0 or 1
        const int quarter = warp & 3;               // TMEM lane quarter this warp may read
        const int mt = (N_MT == 2) ? grp : 0;
        const int row = mt * 128 + quarter * 32 + lane;
        const bool active = row < a.R;
        const int r = row % a.w;
        int ti = 0;
        for (int t = t_begin; t < t_end; ++t, ++ti) {
            if (N_MT == 1 && (ti & 1) != grp) continue;
            const int head = t / g.n_tiles, tile = t - head * g.n_tiles;
            const int buf = ti & 1, use = ti >> 1;
            if (!mbar_wait(smem_u32(&ctl.tfull[buf]), use & 1, abort_flag)) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) +
                                   static_cast<uint32_t>(buf * 256 + mt * TCOLS);
            const size_t tile_id = static_cast<size_t>(head) * g.n_tiles + tile;
            float* part = a.partial + tile_id * g.spt * a.R + row;
            const int j0 = tile * N_TILE;
            float m2, l;
            if (C_STATIC > 0 && j0 + N_TILE <= a.P) {
                tile_fast<(C_STATIC > 0 ? C_STATIC : 1), N_TILE>(taddr, a.sl2, active, part, a.R, &m2, &l);
            } else {
                tile_general<N_TILE>(taddr, a.sl2, active, part, a.R, j0, a.P, a.L, a.c, r, &m2, &l);
            }
            tc_fence_before();
            mbar_arrive(smem_u32(&ctl.tempty[buf]));
            if (active) {
                a.stat_m[tile_id * a.R + row] = m2;
                a.stat_l[tile_id * a.R + row] = l;
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
    if (threadIdx.x == 0 && ctl.abort_flag) atomicExch(a.status, 1);
}

// ---------------------------------------------------------------------------------------------
// Finalisation: global row statistics from tile statistics, then one warp per chunk contracts
// the chunk's partial sums over the R rows. Fixed reduction order, so results are deterministic.
constexpr int kFinThreads = 256;

__global__ void __launch_bounds__(kFinThreads)
finalize_kernel(const ScoreArgs a, int n_tiles, int spt, int n_tile, int C, float* __restrict__ out) {
    __shared__ float gm[256];
    __shared__ float ginv[256];
    const int h = blockIdx.y;
    const size_t stat_base = static_cast<size_t>(h) * n_tiles * a.R;
    for (int i = threadIdx.x; i < a.R; i += blockDim.x) {
        float m = -CUDART_INF_F;
        for (int t = 0; t < n_tiles; ++t) m = fmaxf(m, a.stat_m[stat_base + static_cast<size_t>(t) * a.R + i]);
        float l = 0.f;
        for (int t = 0; t < n_tiles; ++t) {
            const size_t o = stat_base + static_cast<size_t>(t) * a.R + i;
            l += a.stat_l[o] * ex2_approx(a.stat_m[o] - m);
        }
        gm[i] = m;
        ginv[i] = 1.0f / l;
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    const int per_block = (C + gridDim.x - 1) / gridDim.x;
    const int ch0 = blockIdx.x * per_block, ch1 = min(ch0 + per_block, C);
    for (int ch = ch0 + warp; ch < ch1; ch += nwarps) {
        const int ja = ch * a.c, jb = min(ja + a.c, a.P);
        const int t0 = ja / n_tile, t1 = (jb - 1) / n_tile;
        float acc = 0.f;
        for (int t = t0; t <= t1; ++t) {
            const int slot = ch - (t * n_tile) / a.c;
            const size_t so = stat_base + static_cast<size_t>(t) * a.R;
            const size_t po = ((static_cast<size_t>(h) * n_tiles + t) * spt + slot) * a.R;
            for (int i = lane; i < a.R; i += 32)
                acc += a.partial[po + i] * ex2_approx(a.stat_m[so + i] - gm[i]) * ginv[i];
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        if (lane == 0) out[static_cast<size_t>(h) * C + ch] = acc;
    }
}

template <int C_STATIC, int N_MT, int N_TILE>
cudaError_t launch_variant(const ScorePlan& plan, const CUtensorMap& tm_q, const CUtensorMap& tm_k,
                           const ScoreArgs& args, int num_sms, cudaStream_t stream) {
    auto kern = score_kernel<C_STATIC, N_MT, N_TILE>;
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
    g.spt = plan.spt;
    g.n_stages = plan.n_stages;
    g.total_tiles = args.Hkv * plan.n_tiles;
    g.q_box_rows = args.R < 128 ? args.R : 128;
    g.k_box_rows = args.L < N_TILE ? args.L : N_TILE;
    const int grid = g.total_tiles < num_sms ? g.total_tiles : num_sms;
    kern<<<grid, kThreads, plan.smem_bytes, stream>>>(tm_q, tm_k, args, g);
    return cudaGetLastError();
}

}  // namespace

bool make_score_plan(int L, int R, int d, int c, int smem_limit, ScorePlan* plan) {
    if (R < 1 || R > 256 || (d != 64 && d != 128) || c < 1 || L < 1) return false;
    ScorePlan p{};
    p.n_mt = (R + 127) / 128;
    // Chunk sizes with a compiled-in variant use a tile that is a multiple of lcm(c, 16);
    // every other chunk size runs the run-time-c variant on the widest tile.
    p.c_static = 0;
    if (p.n_mt == 1 && (c == 10 || c == 20)) { p.c_static = c; p.n_tile = 240; }
    else if (p.n_mt == 1 && c == 1) { p.c_static = 1; p.n_tile = 256; }
    else p.n_tile = 256 / p.n_mt;
    p.n_tiles = (L + p.n_tile - 1) / p.n_tile;
    p.spt = p.c_static ? p.n_tile / p.c_static : (p.n_tile + c - 1) / c + 1;
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
    const size_t tiles = static_cast<size_t>(Hkv) * plan.n_tiles;
    return tiles * R * 2 + tiles * plan.spt * R;
}

cudaError_t launch_score(const ScorePlan& plan, const CUtensorMap& tm_q, const CUtensorMap& tm_k,
                         const ScoreArgs& args, int num_sms, cudaStream_t stream) {
    if (plan.n_mt == 1) {
        if (plan.c_static == 10) return launch_variant<10, 1, 240>(plan, tm_q, tm_k, args, num_sms, stream);
        if (plan.c_static == 20) return launch_variant<20, 1, 240>(plan, tm_q, tm_k, args, num_sms, stream);
        if (plan.c_static == 1) return launch_variant<1, 1, 256>(plan, tm_q, tm_k, args, num_sms, stream);
        return launch_variant<0, 1, 256>(plan, tm_q, tm_k, args, num_sms, stream);
    }
    return launch_variant<0, 2, 128>(plan, tm_q, tm_k, args, num_sms, stream);
}

cudaError_t launch_finalize(const ScorePlan& plan, const ScoreArgs& args, int C, float* out_scores,
                            int num_sms, cudaStream_t stream) {
    if (C <= 0) return cudaSuccess;
    int bx = (2 * num_sms + args.Hkv - 1) / args.Hkv;
    const int max_bx = (C + 7) / 8;
    if (bx > max_bx) bx = max_bx;
    if (bx < 1) bx = 1;
    dim3 grid(bx, args.Hkv);
    finalize_kernel<<<grid, kFinThreads, 0, stream>>>(args, plan.n_tiles, plan.spt, plan.n_tile, C, out_scores);
    return cudaGetLastError();
}

}  // namespace chunkkv
