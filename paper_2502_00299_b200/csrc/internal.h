// Declarations shared by the translation units of libchunkkv (host side).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace chunkkv {

// Every scratch buffer (device workspace, lane, pipe) starts with a header of this many bytes that is
// zero between launches: device status word at +0, the grid barrier's ticket and exit counters at
// +64 / +128, and from +192 the counters of the layer kernel with on-chip partial sums (exit
// counter, then one hand-over counter per scoring head and one per KV head).
constexpr size_t kHeaderBytes = 2048;
constexpr size_t kResidentCountersOffset = 192;
constexpr int kResidentMaxHeads = 148;   // three counter arrays of this length follow the exit counter

// Geometry of one scoring launch, fixed on the host.
struct ScorePlan {
    int c_static;   // chunk size baked into the kernel (0 = run-time chunk size)
    int n_mt;       // 128-row query tiles per KV head (1 or 2)
    int n_tile;     // keys per accumulator tile (one UMMA N)
    int wp;         // keys per epilogue panel (a quarter or half tile; 32 for run-time chunk sizes)
    int n_tiles;    // accumulator tiles per head = ceil(L / n_tile)
    int n_panels;   // panels per head
    int spp;        // chunk slots per panel in the partial-sum scratch
    int grid;       // CTAs of the scoring launch
    int hs_max;     // per-CTA head records in the CTA statistics scratch
    int n_stages;   // shared-memory stages in the K ring (one stage = n_tile keys x 64 dims)
    int smem_bytes; // dynamic shared memory of the launch
};

struct ScoreArgs {
    int L, P, w, c, R, Hkv, d;   // R rows per scoring head, Hkv scoring heads (see kv_shift)
    int kv_shift;         // scoring head v reads the keys of KV head v >> kv_shift: 1 when the rows of a KV head
                          // are scored as two heads of half the rows (rows are independent, sums add up)
    float sl2;            // log2(e) / sqrt(d)
    float* stat_m;        // [Hkv, n_panels, R] panel row maxima (log2 domain)
    float* cta_stat;      // [grid, hs_max, 4 groups, {max, sum}, 128] per-CTA folded row statistics
    float* row_stat;      // [Hkv, {max, 1 / sum}, 256] global row statistics
    float* partial;       // [Hkv, n_panels, spp, R] chunk partial sums relative to the panel maximum
    int* status;          // device status word
};

// Head-count and size limits shared by every entry point that scores (CHUNKKV_OK or CHUNKKV_EINVAL_SHAPE).
int check_heads(int L, int Hq, int Hkv, int d, int w);

// Chooses kernel variant and tile geometry for a shape. Returns false if unsupported.
// full_grid: launch one CTA per SM even if there are fewer tiles (the fused layer kernel wants
// every SM for its later phases).
bool make_score_plan(int L, int R, int Hkv, int d, int c, int num_sms, int smem_limit, bool full_grid,
                     ScorePlan* plan);

// Scratch floats needed for a plan (panel maxima + CTA records + partial sums), per layer.
size_t score_scratch_floats(const ScorePlan& plan, int Hkv, int R);

// Points the scratch pointers of `args` into `base` (score_scratch_floats floats).
void score_scratch_layout(const ScorePlan& plan, int Hkv, int R, float* base, ScoreArgs* args);

cudaError_t launch_score(const ScorePlan& plan, const CUtensorMap& tm_q, const CUtensorMap& tm_k,
                         const ScoreArgs& args, cudaStream_t stream);

// Inputs and outputs of the fused layer kernel beyond scoring.
struct FusedLayerIO {
    const void* K;
    const void* V;
    void* out_K;
    void* out_V;
    int32_t* out_idx;
    float* chunk_scores;   // [scoring heads, C] scratch
    int C, k, n_max;
    int Hkv_out;           // KV heads (selection and gather), = scoring heads >> kv_shift
    unsigned long long* bar_count;   // grid barrier ticket counter in the scratch header
    bool cooperative = true;         // lanes: cooperative launch; the whole GPU: programmatic dependent launch
};

// The whole layer in one cooperative launch (plan made with full_grid = true, C > 0, k > 0).
cudaError_t launch_layer_fused(const ScorePlan& plan, const CUtensorMap& tm_q, const CUtensorMap& tm_k,
                               const ScoreArgs& args, const FusedLayerIO& io, cudaStream_t stream);

// The layer kernel that keeps its chunk partial sums in tensor memory (layer_resident.cu): every CTA
// belongs to one scoring head, `cph` CTAs per head.
struct ResidentPlan {
    int c_static;     // 10 or 20
    int grid, cph;
    int n_tiles;      // 120-key accumulator tiles per head
    int t_max;        // most tiles any CTA takes
    int n_stages;
    int smem_bytes;
    int off_ring, ring_bytes, off_pmax, off_misc;
};

struct ResidentIO {
    int L, w, Rs, Hs, d, kv_shift;   // Rs rows per scoring head, Hs scoring heads, KV head = scoring head >> kv_shift
    float sl2;
    int C, k, n_max;
    const void* K;
    const void* V;
    void* out_K;
    void* out_V;
    int32_t* out_idx;
    float* scratch;       // resident_scratch_floats() floats
    unsigned* counters;   // header + kResidentCountersOffset
    int* status;
    bool cooperative;     // cooperative launch (lanes: several launches share the GPU) instead of a programmatic dependent one
    // elements between consecutive rows of a head and between heads of K and of V; 0 = packed [Hkv, L, d]
    long long k_row_elems = 0, k_head_elems = 0, v_row_elems = 0, v_head_elems = 0;
    // out_K / out_V are paged caches [num_pages, page_size, Hkv, d] addressed through this block table (else packed)
    const int32_t* block_table = nullptr;
    int page_size = 0, num_pages = 0;
    // Algorithm 1's budget rule: at most this many tokens of the kept chunks are emitted (lowest positions first)
    int tok_cap = 0x7fffffff;
};

// false when the shape does not fit this kernel (chunk size other than 10 / 20, more than 128 rows
// per scoring head, more chunks per CTA than tensor memory holds, fewer CTAs than scoring heads).
bool make_resident_plan(int L, int Rs, int Hs, int kv_shift, int d, int c, int C, int n_max, int max_ctas,
                        int smem_limit, ResidentPlan* plan);
size_t resident_scratch_floats(const ResidentPlan& plan, int Hs, int C);
cudaError_t launch_layer_resident(const ResidentPlan& plan, const CUtensorMap& tm_q, const CUtensorMap& tm_k,
                                  const ResidentIO& io, cudaStream_t stream);

// The persistent kernel that runs many layers per launch (model_kernel.cu). Same tiling as the
// layer kernel above, plus two tail warps per CTA that select and copy rows behind the scoring.
constexpr int kModelMaxLayers = 32;     // layers per launch (computed + reusing)
constexpr int kModelMaxCompute = 32;    // computed layers per launch

struct ModelPlan {
    int c_static, grid, cph, n_tiles, t_max, n_stages, smem_bytes;
    int n_score, n_sel;          // scoring CTAs, selector CTAs (grid = n_score + n_sel)
    int sel_row_bytes, sel_keys_fit;
    int off_ring, off_pmax, off_misc, off_tail, stage_slot_bytes;
};

struct ModelIO {
    int L, w, Rs, Hs, d, kv_shift;
    float sl2;
    int C, k, n_max;
    float* scratch;       // model_scratch_floats() floats
    unsigned* counters;   // header + kResidentCountersOffset
    int* status;
    // elements between consecutive rows of a head and between heads of K and of V (all layers); 0 = packed
    long long k_row_elems = 0, k_head_elems = 0, v_row_elems = 0, v_head_elems = 0;
};

struct ModelLayerIO {
    const void* K;
    const void* V;
    void* out_K;
    void* out_V;
    int32_t* out_idx;
    bool computes;        // false: gather with the indices of the nearest computed layer before it
};

bool make_model_plan(int L, int Rs, int Hs, int kv_shift, int d, int c, int C, int k, int max_ctas, int smem_limit,
                     ModelPlan* plan);
size_t model_scratch_floats(const ModelPlan& plan, int Hs, int kv_shift, int C, int n_compute);
// layers[0] must compute; tm_q / tm_k hold one tensor map per computed layer, in order.
cudaError_t launch_model(const ModelPlan& plan, const ModelIO& io, const CUtensorMap* tm_q, const CUtensorMap* tm_k,
                         const ModelLayerIO* layers, int n_layers, cudaStream_t stream);

// Token scores in one launch, two passes over the keys (token_kernel.cu).
struct TokenPlan {
    int grid, cph, n_tiles, n_tiles_prefix, n_stages, smem_bytes, off_ring, off_misc;
};
struct TokenIO {
    int L, w, Rs, Hs, d, kv_shift;
    float sl2;
    float* token_scores;  // [Hs][P]
    float* scratch;       // grid * 256 floats
    unsigned* counters;   // header + kResidentCountersOffset
    int* status;
};
bool make_token_plan(int L, int w, int Rs, int Hs, int d, int max_ctas, int smem_limit, TokenPlan* plan);
cudaError_t launch_token_scores(const TokenPlan& plan, const CUtensorMap& tm_q, const CUtensorMap& tm_k,
                                const TokenIO& io, cudaStream_t stream);

cudaError_t launch_finalize(const ScorePlan& plan, const ScoreArgs& args, int C, float* out_scores,
                            int num_sms, cudaStream_t stream);

// tok_cap: at most this many tokens of the kept chunks are emitted (lowest positions first)
// Selection over a cluster of eight CTAs per head (select_cluster.cu): for heads with thousands of chunks.
bool select_cluster_applies(int C, int k);
cudaError_t launch_select_cluster(const float* scores, int L, int Hkv, int w, int c, int C, int k, int n_max,
                                  int32_t* out_idx, cudaStream_t stream, int tok_cap);
cudaError_t launch_select(const float* scores, int L, int Hkv, int w, int c, int C, int k, int n_max,
                          int32_t* out_idx, cudaStream_t stream, int tok_cap = 0x7fffffff);

cudaError_t launch_gather(const void* K, const void* V, const int32_t* idx, int L, int Hkv, int d,
                          int n_max, void* out_K, void* out_V, int32_t* idx_copy_or_null,
                          int num_sms, cudaStream_t stream);
// The gather into a paged cache [page, slot, head, d] through a block table (device int32).
cudaError_t launch_gather_strided(const void* K, const void* V, const int32_t* idx, int L, int Hkv, int d, int n_max,
                                  long long k_token_stride, long long k_head_stride, long long v_token_stride,
                                  long long v_head_stride, void* out_K, void* out_V, int32_t* idx_copy_or_null,
                                  int num_sms, cudaStream_t stream);
cudaError_t launch_gather_paged(const void* K, const void* V, const int32_t* idx, int L, int Hkv, int d, int n_max,
                                const int32_t* block_table, int page_size, int num_pages, void* cache_K, void* cache_V,
                                int num_sms, cudaStream_t stream);
// Window queries from a fused QKV activation, rotary embedding applied (see gather.cu).
cudaError_t launch_window_queries(const void* qkv, long long row_elems, int T, int Hq, int d, int w, const float* cos_t,
                                  const float* sin_t, void* q_obs, cudaStream_t stream);
// Jaccard similarity of two kept-index matrices, one CTA per head (diagnostics.cu).
cudaError_t launch_jaccard(const int32_t* idx_a, const int32_t* idx_b, int Hkv, int n_a, int n_b,
                           float* out_ratio, int32_t* out_counts_or_null, cudaStream_t stream);

// out[h][ch] = in[2h][ch] + in[2h + 1][ch]: chunk scores of KV heads from their two scoring heads.
cudaError_t launch_pair_sum(const float* in, float* out, int Hkv, int C, cudaStream_t stream);

// The gather in small CTAs that can share SMs with resident layer-kernel CTAs (lanes).
cudaError_t launch_gather_shared_sms(const void* K, const void* V, const int32_t* idx, int L, int Hkv, int d,
                                     int n_max, void* out_K, void* out_V, int num_sms, cudaStream_t stream);

// Scoring (score + finalisation kernels) into caller-supplied scratch: a 256-byte header whose
// first word is the device status word, then the payload. Returns a CHUNKKV_* status;
// CHUNKKV_ETOOLARGE if scratch_bytes is too small. Allocates nothing.
int score_with_scratch(const void* q_obs, const void* K, int L, int Hq, int Hkv, int d, int w, int c,
                       float* out_scores, void* scratch, size_t scratch_bytes, cudaStream_t stream);

}  // namespace chunkkv
