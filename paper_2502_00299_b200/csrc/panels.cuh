// Epilogue panels of the scoring kernels: one thread owns one query row of a panel of WP score
// columns (keys), pulled from tensor memory into registers. For that row it takes the panel
// maximum, exponentiates every visible element once relative to it, and sums the exponentials per
// chunk of C keys (ChunkKV Algorithm 3, "Vectorized Chunk Score Calculation", before the softmax
// normaliser is known). What happens to a chunk's partial sum is the caller's business: `emit(ch,
// value)` is called once per chunk slot of the panel with a compile-time-unrolled `ch`.
#pragma once
#include "ptx.cuh"

#include <math_constants.h>

namespace chunkkv {

// Pull WP consecutive accumulator columns of this thread's row into registers.
template <int WP>
__device__ __forceinline__ void load_panel(uint32_t taddr, float (&v)[WP]) {
    static_assert(WP % 4 == 0, "panel width must be a multiple of 4 columns");
    int o = 0;
#pragma unroll
    for (int b = 0; b < WP / 32; ++b, o += 32) tmem_ld_x32(taddr + o, &v[o]);
    if constexpr ((WP & 16) != 0) { tmem_ld_x16(taddr + o, &v[o]); o += 16; }
    if constexpr ((WP & 8) != 0) { tmem_ld_x8(taddr + o, &v[o]); o += 8; }
    if constexpr ((WP & 4) != 0) { tmem_ld_x4(taddr + o, &v[o]); o += 4; }
    tmem_ld_wait();
}

// Panel that lies wholly inside the prefix and starts on a chunk boundary, chunk size known at
// compile time: all control flow below folds away after unrolling.
template <int C, int WP, class Emit>
__device__ __forceinline__ void panel_fast(float (&v)[WP], float sl2, Emit emit, float* out_m, float* out_l) {
    static_assert(WP % 4 == 0 && WP >= 8, "panel width");
    // row max with three-input max instructions, two independent chains
    float m0 = fmaxf(v[0], v[1]), m1 = fmaxf(v[2], v[3]);
#pragma unroll
    for (int u = 4; u + 3 < WP; u += 4) {
        m0 = fmax3(m0, v[u], v[u + 1]);
        m1 = fmax3(m1, v[u + 2], v[u + 3]);
    }
    const float mx = fmaxf(m0, m1);
    const float neg_m2 = -mx * sl2;
    float l = 0.f;
    if constexpr (C % 2 == 0) {
        // Two columns per instruction: scale-and-shift and the chunk sums run on packed pairs
        // (same arithmetic, fewer instructions issued).
        const unsigned long long s2 = pack2(sl2, sl2), n2 = pack2(neg_m2, neg_m2);
        unsigned long long e[WP / 2];
#pragma unroll
        for (int u = 0; u < WP / 2; ++u) {
            float x0, x1;
            unpack2(fma2(pack2(v[2 * u], v[2 * u + 1]), s2, n2), x0, x1);
            e[u] = pack2(ex2_approx(x0), ex2_approx(x1));
        }
        constexpr int H = C / 2;     // pairs per chunk
#pragma unroll
        for (int ch = 0; ch < WP / C; ++ch) {
            unsigned long long s0 = e[ch * H];
            unsigned long long s1 = (H > 1) ? e[ch * H + 1] : 0ull;
#pragma unroll
            for (int t = 2; t < H; t += 2) {
                s0 = add2(s0, e[ch * H + t]);
                if (t + 1 < H) s1 = add2(s1, e[ch * H + t + 1]);
            }
            if (H > 1) s0 = add2(s0, s1);
            float lo, hi;
            unpack2(s0, lo, hi);
            const float acc = lo + hi;
            emit(ch, acc);
            l += acc;
        }
    } else {
        // exponentials first, in place: WP independent operations the scheduler can overlap freely
#pragma unroll
        for (int u = 0; u < WP; ++u) v[u] = ex2_approx(fmaf(v[u], sl2, neg_m2));
        // chunk sums as balanced trees (short dependency chains), one store per chunk
#pragma unroll
        for (int ch = 0; ch < WP / C; ++ch) {
            float s0 = 0.f, s1 = 0.f;
#pragma unroll
            for (int t = 0; t < C; t += 2) {
                s0 += v[ch * C + t];
                if (t + 1 < C) s1 += v[ch * C + t + 1];
            }
            const float acc = s0 + s1;
            emit(ch, acc);
            l += acc;
        }
    }
    *out_m = mx * sl2;
    *out_l = l;
}

// Panel of a compile-time chunk size that starts on a chunk boundary but reaches past the
// prefix: chunk positions are still static; columns at or past P only feed the row sum, and
// columns the row cannot see (causal mask in the window, or past L) contribute nothing.
template <int C, int WP, class Emit>
__device__ __forceinline__ void panel_static_tail(const float (&v)[WP], float sl2, Emit emit, int j0, int P,
                                                  int last_visible, float* out_m, float* out_l) {
    const int n_vis = last_visible - j0 + 1;     // columns u < n_vis are visible
    const int n_pre = P - j0;                    // columns u < n_pre belong to the prefix
    if (n_vis <= 0) {                            // the row sees nothing of this panel (e.g. a panel past L)
#pragma unroll
        for (int ch = 0; ch < WP / C; ++ch) emit(ch, 0.f);
        *out_m = -CUDART_INF_F;
        *out_l = 0.f;
        return;
    }
    // two independent chains each for the maximum and the row sum
    float mx0 = -CUDART_INF_F, mx1 = -CUDART_INF_F;
#pragma unroll
    for (int u = 0; u + 1 < WP; u += 2) {
        mx0 = (u < n_vis) ? fmaxf(mx0, v[u]) : mx0;
        mx1 = (u + 1 < n_vis) ? fmaxf(mx1, v[u + 1]) : mx1;
    }
    if constexpr (WP % 2 == 1) mx0 = (WP - 1 < n_vis) ? fmaxf(mx0, v[WP - 1]) : mx0;
    const float mx = fmaxf(mx0, mx1);
    const float neg_m2 = (mx == -CUDART_INF_F) ? 0.f : -mx * sl2;
    float l0 = 0.f, l1 = 0.f, acc = 0.f;
#pragma unroll
    for (int u = 0; u < WP; ++u) {
        const float e = (u < n_vis) ? ex2_approx(fmaf(v[u], sl2, neg_m2)) : 0.f;
        if (u & 1) l1 += e; else l0 += e;
        const float pe = (u < n_pre) ? e : 0.f;
        acc = (u % C == 0) ? pe : acc + pe;
        if ((u + 1) % C == 0) {
            // a slot whose chunk starts at or past P holds no chunk: it receives 0
            emit((u + 1) / C - 1, ((u + 1 - C) < n_pre) ? acc : 0.f);
        }
    }
    const float l = l0 + l1;
    *out_m = (mx == -CUDART_INF_F) ? -CUDART_INF_F : mx * sl2;
    *out_l = l;
}

}  // namespace chunkkv
