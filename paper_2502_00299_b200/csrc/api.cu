// C ABI of libchunkkv: argument checks, scratch management, tensor-map encoding and the
// launch sequence of each entry point. Every step of the method runs in the kernels of
// score.cu / select.cu / gather.cu; this file only validates and dispatches.
#include "../../include/chunkkv.h"
#include "internal.h"

#include <math.h>
#include <mutex>
#include <vector>

using namespace chunkkv;

namespace {

constexpr int kMaxDevices = 64;

thread_local int g_last_cuda_error = 0;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

struct ProfileRec {
    cudaEvent_t start, stop;
    int slot;
};

struct DeviceCtx {
    bool init = false;
    int num_sms = 0;
    int smem_optin = 0;
    void* ws = nullptr;        // scratch handed over with chunkkv_set_workspace (header + payload)
    size_t ws_bytes = 0;
    std::vector<ProfileRec> recs;
    float prof_ms[CHUNKKV_PROFILE_SLOTS] = {0, 0, 0, 0};
    int prof_n[CHUNKKV_PROFILE_SLOTS] = {0, 0, 0, 0};
};

std::mutex g_mu;

// Host side of a pipe (chunkkv_pipe_*): caller-owned lane scratch, a side stream for the row gathers
// and the two events that order it against the caller's stream.
struct Pipe {
    int device = 0;
    char* scratch = nullptr;
    size_t bytes = 0;
    int max_ctas = 0;
    cudaStream_t side = nullptr;
    cudaEvent_t scored = nullptr;    // the layer kernel of the latest layer, on the caller's stream
    cudaEvent_t posted = nullptr;    // the row gather of the latest layer, on the side stream
    bool pending = false;            // a gather was queued since the last join
};
DeviceCtx g_ctx[kMaxDevices];
EncodeTiledFn g_encode = nullptr;
bool g_profile = false;

int cuda_fail(cudaError_t e) {
    g_last_cuda_error = static_cast<int>(e);
    return CHUNKKV_ECUDA;
}

// Caller holds g_mu.
int get_ctx(DeviceCtx** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev < 0 || dev >= kMaxDevices) return CHUNKKV_EINVAL_SHAPE;
    DeviceCtx& c = g_ctx[dev];
    if (!c.init) {
        e = cudaDeviceGetAttribute(&c.num_sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return cuda_fail(e);
        e = cudaDeviceGetAttribute(&c.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
        if (e != cudaSuccess) return cuda_fail(e);
        c.init = true;
    }
    if (g_encode == nullptr) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess) return cuda_fail(e);
        if (fn == nullptr || qres != cudaDriverEntryPointSuccess) return cuda_fail(cudaErrorNotSupported);
        g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    *out = &c;
    return CHUNKKV_OK;
}

// Shared-memory budget for the dynamic part of the score kernel (static control block excluded).
int smem_budget(const DeviceCtx& c) { return c.smem_optin - 1024; }

// The library never allocates: the scratch is whatever chunkkv_set_workspace was given.
int ensure_workspace(DeviceCtx& c, size_t payload_bytes) {
    const size_t need = kHeaderBytes + payload_bytes;
    if (c.ws != nullptr && c.ws_bytes >= need) return CHUNKKV_OK;
    return CHUNKKV_ENOWORKSPACE;
}

// How the R = w * Hq / Hkv window rows of a KV head are scored. Rows are independent (each has its
// own softmax) and chunk scores are sums over rows, so more than 128 rows of an even number of
// query heads are scored as two heads of R / 2 rows each that read the same keys: every scoring
// head then fits one 128-row query tile and takes the faster single-tile kernel; its two chunk
// score vectors are added before the selection.
struct ScoreShape {
    int Hs;      // scoring heads
    int Rs;      // rows per scoring head
    int shift;   // scoring head v belongs to KV head v >> shift
};
ScoreShape score_shape(int Hq, int Hkv, int w) {
    const int G = Hq / Hkv, R = w * G;
    if (R > 128 && G % 2 == 0) return {2 * Hkv, R / 2, 1};
    return {Hkv, R, 0};
}
size_t round64(size_t n) { return (n + 63) & ~static_cast<size_t>(63); }

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_sizes(int L, int w, int c, int budget) {
    if (w < 1 || c < 1 || L < w || budget < w) return CHUNKKV_EINVAL_SHAPE;
    return CHUNKKV_OK;
}

// row_elems / head_elems: elements between consecutive rows of a head and between heads; 0 = packed [heads, rows, d]
int encode_bf16_3d(CUtensorMap* tm, const void* base, int d, long long rows, int heads, int box_rows,
                   CUtensorMapL2promotion promo, long long row_elems = 0, long long head_elems = 0) {
    cuuint64_t dims[3] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(rows),
                          static_cast<cuuint64_t>(heads)};
    if (row_elems == 0) row_elems = d;
    if (head_elems == 0) head_elems = rows * d;
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(row_elems) * 2, static_cast<cuuint64_t>(head_elems) * 2};
    cuuint32_t box[3] = {64, static_cast<cuuint32_t>(box_rows), 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = g_encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides,
                          box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, promo,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        g_last_cuda_error = 100000 + static_cast<int>(r);
        return CHUNKKV_ECUDA;
    }
    return CHUNKKV_OK;
}

struct Timer {
    DeviceCtx* c;
    cudaStream_t s;
    bool on;
    ProfileRec rec;
    Timer(DeviceCtx* ctx, cudaStream_t st, int slot) : c(ctx), s(st), on(g_profile) {
        if (!on) return;
        rec.slot = slot;
        if (cudaEventCreate(&rec.start) != cudaSuccess || cudaEventCreate(&rec.stop) != cudaSuccess) {
            on = false;
            return;
        }
        cudaEventRecord(rec.start, s);
    }
    ~Timer() {
        if (!on) return;
        cudaEventRecord(rec.stop, s);
        c->recs.push_back(rec);
    }
};

// Score + finalise for chunk size c. Chunk scores go to `out_scores`, or - when that is NULL -
// to the first `extra_payload_floats` floats of the scratch payload; `*resolved` receives the
// address used. Caller holds g_mu and has validated the arguments.
int run_score(DeviceCtx& ctx, const void* q_obs, const void* K, int L, int Hq, int Hkv, int d, int w,
              int c, float* out_scores, size_t extra_payload_floats, float** resolved,
              cudaStream_t stream, long long k_row_elems = 0, long long k_head_elems = 0) {
    const int P = L - w;
    const int C = (P + c - 1) / c;
    if (C <= 0) return CHUNKKV_OK;
    const ScoreShape sh = score_shape(Hq, Hkv, w);
    const int R = sh.Rs;
    // with two scoring heads per KV head their chunk scores go to scratch first and are added into the output
    const size_t pair_floats = sh.shift ? round64(static_cast<size_t>(sh.Hs) * C) : 0;
    TokenPlan tplan;
    if (c == 1 && make_token_plan(L, w, R, sh.Hs, d, ctx.num_sms, smem_budget(ctx), &tplan)) {
        // token scores: two passes over the keys in one launch, nothing but row records in scratch
        const size_t tfloats = extra_payload_floats + pair_floats + static_cast<size_t>(tplan.grid) * 256;
        int st2 = ensure_workspace(ctx, tfloats * sizeof(float));
        if (st2 != CHUNKKV_OK) return st2;
        float* payload = reinterpret_cast<float*>(static_cast<char*>(ctx.ws) + kHeaderBytes);
        if (out_scores == nullptr) out_scores = payload;
        if (resolved != nullptr) *resolved = out_scores;
        float* head_scores = sh.shift ? payload + extra_payload_floats : out_scores;
        CUtensorMap tq, tk;
        st2 = encode_bf16_3d(&tq, q_obs, d, R, sh.Hs, R < 128 ? R : 128, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
        if (st2 != CHUNKKV_OK) return st2;
        st2 = encode_bf16_3d(&tk, K, d, L, Hkv, L < 120 ? L : 120, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, k_row_elems, k_head_elems);
        if (st2 != CHUNKKV_OK) return st2;
        TokenIO io;
        io.L = L; io.w = w; io.Rs = R; io.Hs = sh.Hs; io.d = d; io.kv_shift = sh.shift;
        io.sl2 = static_cast<float>(1.4426950408889634 / sqrt(static_cast<double>(d)));
        io.token_scores = head_scores;
        io.scratch = payload + extra_payload_floats + pair_floats;
        io.counters = reinterpret_cast<unsigned*>(static_cast<char*>(ctx.ws) + kResidentCountersOffset);
        io.status = static_cast<int*>(ctx.ws);
        cudaError_t e2;
        {
            Timer t(&ctx, stream, 0);
            e2 = launch_token_scores(tplan, tq, tk, io, stream);
            if (e2 == cudaSuccess && sh.shift) e2 = launch_pair_sum(head_scores, out_scores, Hkv, C, stream);
        }
        if (e2 != cudaSuccess) return cuda_fail(e2);
        return CHUNKKV_OK;
    }
    ScorePlan plan;
    if (!make_score_plan(L, R, sh.Hs, d, c, ctx.num_sms, smem_budget(ctx), false, &plan)) return CHUNKKV_EINVAL_SHAPE;
    const size_t floats = score_scratch_floats(plan, sh.Hs, R) + extra_payload_floats + pair_floats;
    int st = ensure_workspace(ctx, floats * sizeof(float));
    if (st != CHUNKKV_OK) return st;
    float* payload = reinterpret_cast<float*>(static_cast<char*>(ctx.ws) + kHeaderBytes);
    if (out_scores == nullptr) out_scores = payload;
    if (resolved != nullptr) *resolved = out_scores;
    float* head_scores = sh.shift ? payload + extra_payload_floats : out_scores;
    ScoreArgs a;
    a.L = L; a.P = P; a.w = w; a.c = c; a.R = R; a.Hkv = sh.Hs; a.d = d; a.kv_shift = sh.shift;
    a.sl2 = static_cast<float>(1.4426950408889634 / sqrt(static_cast<double>(d)));
    score_scratch_layout(plan, sh.Hs, R, payload + extra_payload_floats + pair_floats, &a);
    a.status = static_cast<int*>(ctx.ws);
    CUtensorMap tm_q, tm_k;
    st = encode_bf16_3d(&tm_q, q_obs, d, R, sh.Hs, R < 128 ? R : 128, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
    if (st != CHUNKKV_OK) return st;
    st = encode_bf16_3d(&tm_k, K, d, L, Hkv, L < plan.n_tile ? L : plan.n_tile,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, k_row_elems, k_head_elems);
    if (st != CHUNKKV_OK) return st;
    cudaError_t e;
    {
        Timer t(&ctx, stream, 0);
        e = launch_score(plan, tm_q, tm_k, a, stream);
    }
    if (e != cudaSuccess) return cuda_fail(e);
    {
        Timer t(&ctx, stream, 1);
        e = launch_finalize(plan, a, C, head_scores, ctx.num_sms, stream);
        if (e == cudaSuccess && sh.shift) e = launch_pair_sum(head_scores, out_scores, Hkv, C, stream);
    }
    if (e != cudaSuccess) return cuda_fail(e);
    return CHUNKKV_OK;
}

// Scratch floats of the scoring kernels for a shape: the larger of the score-only launch and the
// fused layer launch (which always uses one CTA per SM and so may keep more per-CTA records).
size_t scratch_floats_for(const DeviceCtx& ctx, int L, int R, int Hkv, int d, int c) {
    ScorePlan plan;
    size_t n = 0;
    for (int full = 0; full < 2; ++full) {
        if (!make_score_plan(L, R, Hkv, d, c, ctx.num_sms, smem_budget(ctx), full != 0, &plan)) return 0;
        const size_t f = score_scratch_floats(plan, Hkv, R);
        n = f > n ? f : n;
    }
    return n;
}

}  // namespace

namespace chunkkv {

int check_heads(int L, int Hq, int Hkv, int d, int w) {
    if (Hkv < 1 || Hq < Hkv || Hq % Hkv != 0) return CHUNKKV_EINVAL_SHAPE;
    if (d != 64 && d != 128) return CHUNKKV_EINVAL_SHAPE;
    const long long R = static_cast<long long>(w) * (Hq / Hkv);
    if (R > 256) return CHUNKKV_EINVAL_SHAPE;
    if (static_cast<long long>(Hkv) * L * d >= (1LL << 40)) return CHUNKKV_EINVAL_SHAPE;
    if (Hkv > 65535) return CHUNKKV_EINVAL_SHAPE;
    if (static_cast<long long>(Hkv) * L >= (1LL << 23)) return CHUNKKV_EINVAL_SHAPE;   // 32-bit row arithmetic in the kernels
    return CHUNKKV_OK;
}

// Scoring into caller-supplied scratch (256-byte header + payload). Used by the fixed-scratch
// entry point; allocates nothing and records no profiling events.
int score_with_scratch(const void* q_obs, const void* K, int L, int Hq, int Hkv, int d, int w, int c,
                       float* out_scores, void* scratch, size_t scratch_bytes, cudaStream_t stream) {
    std::lock_guard<std::mutex> lk(g_mu);
    DeviceCtx* ctx;
    int st = get_ctx(&ctx);
    if (st != CHUNKKV_OK) return st;
    const int P = L - w;
    const int C = (P + c - 1) / c;
    if (C <= 0) return CHUNKKV_OK;
    const ScoreShape sh = score_shape(Hq, Hkv, w);
    const int R = sh.Rs;
    ScorePlan plan;
    if (!make_score_plan(L, R, sh.Hs, d, c, ctx->num_sms, smem_budget(*ctx), false, &plan)) return CHUNKKV_EINVAL_SHAPE;
    const size_t pair_floats = sh.shift ? round64(static_cast<size_t>(sh.Hs) * C) : 0;
    if (kHeaderBytes + (score_scratch_floats(plan, sh.Hs, R) + pair_floats) * sizeof(float) > scratch_bytes)
        return CHUNKKV_ETOOLARGE;
    float* payload = reinterpret_cast<float*>(static_cast<char*>(scratch) + kHeaderBytes);
    float* head_scores = sh.shift ? payload : out_scores;
    ScoreArgs a;
    a.L = L; a.P = P; a.w = w; a.c = c; a.R = R; a.Hkv = sh.Hs; a.d = d; a.kv_shift = sh.shift;
    a.sl2 = static_cast<float>(1.4426950408889634 / sqrt(static_cast<double>(d)));
    score_scratch_layout(plan, sh.Hs, R, payload + pair_floats, &a);
    a.status = static_cast<int*>(scratch);
    CUtensorMap tm_q, tm_k;
    st = encode_bf16_3d(&tm_q, q_obs, d, R, sh.Hs, R < 128 ? R : 128, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
    if (st != CHUNKKV_OK) return st;
    st = encode_bf16_3d(&tm_k, K, d, L, Hkv, L < plan.n_tile ? L : plan.n_tile, CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
    if (st != CHUNKKV_OK) return st;
    cudaError_t e = launch_score(plan, tm_q, tm_k, a, stream);
    if (e != cudaSuccess) return cuda_fail(e);
    e = launch_finalize(plan, a, C, head_scores, ctx->num_sms, stream);
    if (e == cudaSuccess && sh.shift) e = launch_pair_sum(head_scores, out_scores, Hkv, C, stream);
    if (e != cudaSuccess) return cuda_fail(e);
    return CHUNKKV_OK;
}

}  // namespace chunkkv

extern "C" {

const char* chunkkv_strerror(int status) {
    switch (status) {
        case CHUNKKV_OK: return "ok";
        case CHUNKKV_EINVAL_NULL: return "a required pointer is NULL";
        case CHUNKKV_EINVAL_SHAPE: return "a size is outside the supported range";
        case CHUNKKV_EINVAL_ALIGN: return "a tensor pointer is not 16-byte aligned";
        case CHUNKKV_ENOWORKSPACE: return "no scratch workspace was set, or it is too small for this shape";
        case CHUNKKV_ECUDA: return "a CUDA call failed";
        case CHUNKKV_EDEVICE: return "a kernel abandoned a bounded wait";
        case CHUNKKV_ETOOLARGE: return "the problem needs more scratch than the fixed-size variant provides";
        default: return "unknown status";
    }
}

int chunkkv_last_cuda_error(void) { return g_last_cuda_error; }

int chunkkv_num_chunks(int L, int w, int c) {
    if (w < 1 || c < 1 || L < w) return CHUNKKV_EINVAL_SHAPE;
    return (L - w + c - 1) / c;
}

int chunkkv_num_kept_chunks(int L, int w, int c, int budget) {
    int st = check_sizes(L, w, c, budget);
    if (st != CHUNKKV_OK) return st;
    const int C = (L - w + c - 1) / c;
    const int k = (budget - w) / c;
    return k < C ? k : C;
}

int chunkkv_out_len(int L, int w, int c, int budget) {
    const int k = chunkkv_num_kept_chunks(L, w, c, budget);
    if (k < 0) return k;
    const long long n = static_cast<long long>(k) * c + w;
    if (n > 0x7fffffffLL) return CHUNKKV_EINVAL_SHAPE;
    return static_cast<int>(n);
}

size_t chunkkv_workspace_bytes(int L, int Hq, int Hkv, int d, int w, int c) {
    if (w < 1 || c < 1 || L < w) return 0;
    if (check_heads(L, Hq, Hkv, d, w) != CHUNKKV_OK) return 0;
    std::lock_guard<std::mutex> lk(g_mu);
    DeviceCtx* ctx;
    if (get_ctx(&ctx) != CHUNKKV_OK) return 0;
    const ScoreShape sh = score_shape(Hq, Hkv, w);
    const int C = (L - w + c - 1) / c;
    // chunk scores of the KV heads, those of the scoring heads, and the scoring kernels' scratch
    size_t floats = scratch_floats_for(*ctx, L, sh.Rs, sh.Hs, d, c) + round64(static_cast<size_t>(Hkv) * C) +
                    round64(static_cast<size_t>(sh.Hs) * C);
    ResidentPlan rplan;
    if (C > 0 && make_resident_plan(L, sh.Rs, sh.Hs, sh.shift, d, c, C, 0, ctx->num_sms, smem_budget(*ctx), &rplan)) {
        const size_t rf = resident_scratch_floats(rplan, sh.Hs, C);
        floats = rf > floats ? rf : floats;
    }
    return kHeaderBytes + floats * sizeof(float);
}

int chunkkv_set_workspace(void* dev_ptr, size_t bytes) {
    std::lock_guard<std::mutex> lk(g_mu);
    DeviceCtx* ctx;
    int st = get_ctx(&ctx);
    if (st != CHUNKKV_OK) return st;
    // set-up call: work queued earlier may still use the previous scratch
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev_ptr == nullptr) {
        ctx->ws = nullptr;
        ctx->ws_bytes = 0;
        return CHUNKKV_OK;
    }
    if ((reinterpret_cast<uintptr_t>(dev_ptr) & 255u) != 0) return CHUNKKV_EINVAL_ALIGN;
    if (bytes < kHeaderBytes) return CHUNKKV_ENOWORKSPACE;
    e = cudaMemset(dev_ptr, 0, kHeaderBytes);
    if (e != cudaSuccess) return cuda_fail(e);
    e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return cuda_fail(e);
    ctx->ws = dev_ptr;
    ctx->ws_bytes = bytes;
    return CHUNKKV_OK;
}

int chunkkv_device_status(void* stream) {
    std::lock_guard<std::mutex> lk(g_mu);
    DeviceCtx* ctx;
    int st = get_ctx(&ctx);
    if (st != CHUNKKV_OK) return st;
    cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(e);
    if (ctx->ws == nullptr) return CHUNKKV_OK;
    int flag = 0;
    e = cudaMemcpy(&flag, ctx->ws, sizeof(int), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(e);
    if (flag != 0) {
        cudaMemset(ctx->ws, 0, kHeaderBytes);   // status word and grid-barrier words
        return CHUNKKV_EDEVICE;
    }
    return CHUNKKV_OK;
}

int chunkkv_score(const void* q_obs, const void* K, int L, int Hq, int Hkv, int d, int w, int c,
                  float* out_token_scores, float* out_chunk_scores, void* stream) {
    if (w < 1 || c < 1 || L < w) return CHUNKKV_EINVAL_SHAPE;
    int st = check_heads(L, Hq, Hkv, d, w);
    if (st != CHUNKKV_OK) return st;
    if (q_obs == nullptr || K == nullptr || out_chunk_scores == nullptr) return CHUNKKV_EINVAL_NULL;
    if (!aligned16(q_obs) || !aligned16(K) || !aligned16(out_chunk_scores) ||
        (out_token_scores != nullptr && !aligned16(out_token_scores)))
        return CHUNKKV_EINVAL_ALIGN;
    std::lock_guard<std::mutex> lk(g_mu);
    DeviceCtx* ctx;
    st = get_ctx(&ctx);
    if (st != CHUNKKV_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    st = run_score(*ctx, q_obs, K, L, Hq, Hkv, d, w, c, out_chunk_scores, 0, nullptr, s);
    if (st != CHUNKKV_OK) return st;
    if (out_token_scores != nullptr)
        st = run_score(*ctx, q_obs, K, L, Hq, Hkv, d, w, 1, out_token_scores, 0, nullptr, s);
    return st;
}

int chunkkv_select(const float* chunk_scores, int L, int Hkv, int w, int c, int budget,
                   int32_t* out_idx, void* stream) {
    int st = check_sizes(L, w, c, budget);
    if (st != CHUNKKV_OK) return st;
    if (Hkv < 1 || Hkv > 65535) return CHUNKKV_EINVAL_SHAPE;
    const int C = chunkkv_num_chunks(L, w, c);
    const int k = chunkkv_num_kept_chunks(L, w, c, budget);
    const int n_max = chunkkv_out_len(L, w, c, budget);
    if (n_max < 0) return n_max;
    if (out_idx == nullptr || (C > 0 && k > 0 && chunk_scores == nullptr)) return CHUNKKV_EINVAL_NULL;
    if (!aligned16(out_idx) || !aligned16(chunk_scores)) return CHUNKKV_EINVAL_ALIGN;
    std::lock_guard<std::mutex> lk(g_mu);
    DeviceCtx* ctx;
    st = get_ctx(&ctx);
    if (st != CHUNKKV_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    {
        Timer t(ctx, s, 2);
        e = launch_select(chunk_scores, L, Hkv, w, c, C, k, n_max, out_idx, s);
    }
    if (e != cudaSuccess) return cuda_fail(e);
    return CHUNKKV_OK;
}

int chunkkv_gather(const void* K, const void* V, const int32_t* idx, int L, int Hkv, int d,
                   int n_max, void* out_K, void* out_V, void* stream) {
    if (L < 1 || Hkv < 1 || Hkv > 65535 || n_max < 0 || (d != 64 && d != 128)) return CHUNKKV_EINVAL_SHAPE;
    if (static_cast<long long>(Hkv) * L * d >= (1LL << 40)) return CHUNKKV_EINVAL_SHAPE;
    if (K == nullptr || V == nullptr || idx == nullptr || out_K == nullptr || out_V == nullptr)
        return CHUNKKV_EINVAL_NULL;
    if (!aligned16(K) || !aligned16(V) || !aligned16(idx) || !aligned16(out_K) || !aligned16(out_V))
        return CHUNKKV_EINVAL_ALIGN;
    std::lock_guard<std::mutex> lk(g_mu);
    DeviceCtx* ctx;
    int st = get_ctx(&ctx);
    if (st != CHUNKKV_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    {
        Timer t(ctx, s, 3);
        e = launch_gather(K, V, idx, L, Hkv, d, n_max, out_K, out_V, nullptr, ctx->num_sms, s);
    }
    if (e != cudaSuccess) return cuda_fail(e);
    return CHUNKKV_OK;
}

// Shared body of chunkkv_compress_layer and chunkkv_compress_layer_lane. `lane` = caller-owned
// scratch (NULL: the device-wide scratch), `max_ctas` = CTA budget of the launch (0: every SM).
// rows_elsewhere != NULL (pipes): the caller gathers the rows itself after this call, so the layer
// kernel always runs without its gather phase and no gather is launched here.
static int compress_impl(const void* q_obs, const void* K, const void* V, int L, int Hq, int Hkv, int d, int w,
                         int c, int budget, const int32_t* reuse_idx, void* out_K, void* out_V,
                         int32_t* out_idx, void* lane, size_t lane_bytes, int max_ctas, void* stream,
                         const void* rows_elsewhere = nullptr) {
    int st = check_sizes(L, w, c, budget);
    if (st != CHUNKKV_OK) return st;
    st = check_heads(L, Hq, Hkv, d, w);
    if (st != CHUNKKV_OK) return st;
    if (K == nullptr || V == nullptr || out_K == nullptr || out_V == nullptr || out_idx == nullptr)
        return CHUNKKV_EINVAL_NULL;
    if (reuse_idx == nullptr && q_obs == nullptr) return CHUNKKV_EINVAL_NULL;
    if (!aligned16(q_obs) || !aligned16(K) || !aligned16(V) || !aligned16(out_K) || !aligned16(out_V) ||
        !aligned16(out_idx) || !aligned16(reuse_idx))
        return CHUNKKV_EINVAL_ALIGN;
    if (max_ctas < 0) return CHUNKKV_EINVAL_SHAPE;
    const int C = chunkkv_num_chunks(L, w, c);
    const int k = chunkkv_num_kept_chunks(L, w, c, budget);
    const int n_max = chunkkv_out_len(L, w, c, budget);
    if (n_max < 0) return n_max;
    std::lock_guard<std::mutex> lk(g_mu);
    DeviceCtx* ctx;
    st = get_ctx(&ctx);
    if (st != CHUNKKV_OK) return st;
    const int ctas = (max_ctas > 0 && max_ctas < ctx->num_sms) ? max_ctas : ctx->num_sms;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    if (reuse_idx != nullptr) {
        Timer t(ctx, s, 3);
        e = launch_gather(K, V, reuse_idx, L, Hkv, d, n_max, out_K, out_V,
                          reuse_idx == out_idx ? nullptr : out_idx, ctas, s);
        if (e != cudaSuccess) return cuda_fail(e);
        return CHUNKKV_OK;
    }
    float* chunk_scores = nullptr;
    if (C > 0 && k > 0) {
        const ScoreShape sh = score_shape(Hq, Hkv, w);
        const int R = sh.Rs;
        // chunk scores (of the scoring heads) sit at the start of the scratch payload, the score
        // kernels' scratch after them
        const size_t cs_floats = round64(static_cast<size_t>(sh.Hs) * C);
        // A lane that owns at most half of the SMs leaves the row gather to a second launch of
        // small CTAs that spread over every SM (they fit beside the other lanes' resident
        // CTAs), instead of moving the rows through its own few SMs.
        const bool split = rows_elsewhere != nullptr || (lane != nullptr && 2 * ctas <= ctx->num_sms);
        ResidentPlan rplan;
        if (!split && make_resident_plan(L, R, sh.Hs, sh.shift, d, c, C, n_max, ctas, smem_budget(*ctx), &rplan)) {
            // One cooperative launch; the chunk partial sums never leave the SMs.
            const size_t need = resident_scratch_floats(rplan, sh.Hs, C) * sizeof(float);
            char* base;
            if (lane != nullptr) {
                if (kHeaderBytes + need > lane_bytes) return CHUNKKV_ENOWORKSPACE;
                base = static_cast<char*>(lane);
            } else {
                st = ensure_workspace(*ctx, need);
                if (st != CHUNKKV_OK) return st;
                base = static_cast<char*>(ctx->ws);
            }
            CUtensorMap tm_q, tm_k;
            st = encode_bf16_3d(&tm_q, q_obs, d, R, sh.Hs, R < 128 ? R : 128, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
            if (st != CHUNKKV_OK) return st;
            st = encode_bf16_3d(&tm_k, K, d, L, Hkv, L < 120 ? L : 120, CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
            if (st != CHUNKKV_OK) return st;
            ResidentIO io;
            io.L = L; io.w = w; io.Rs = R; io.Hs = sh.Hs; io.d = d; io.kv_shift = sh.shift;
            io.sl2 = static_cast<float>(1.4426950408889634 / sqrt(static_cast<double>(d)));
            io.C = C; io.k = k; io.n_max = n_max;
            io.K = K; io.V = V; io.out_K = out_K; io.out_V = out_V; io.out_idx = out_idx;
            io.scratch = reinterpret_cast<float*>(base + kHeaderBytes);
            io.counters = reinterpret_cast<unsigned*>(base + kResidentCountersOffset);
            io.status = reinterpret_cast<int*>(base);
            io.cooperative = lane != nullptr;
            {
                Timer t(ctx, s, 0);
                e = launch_layer_resident(rplan, tm_q, tm_k, io, s);
            }
            if (e != cudaSuccess) return cuda_fail(e);
            return CHUNKKV_OK;
        }
        ScorePlan plan;
        TokenPlan tplan;
        // token-level layers on the whole GPU: the two-pass token-score kernel, then select and gather
        const bool token_path = c == 1 && lane == nullptr && rows_elsewhere == nullptr &&
                                make_token_plan(L, w, R, sh.Hs, d, ctx->num_sms, smem_budget(*ctx), &tplan);
        if (!token_path && make_score_plan(L, R, sh.Hs, d, c, ctas, smem_budget(*ctx), true, &plan)) {
            // One cooperative launch for the whole layer.
            const size_t need = (cs_floats + score_scratch_floats(plan, sh.Hs, R)) * sizeof(float);
            char* base;
            if (lane != nullptr) {
                if (kHeaderBytes + need > lane_bytes) return CHUNKKV_ENOWORKSPACE;
                base = static_cast<char*>(lane);
            } else {
                st = ensure_workspace(*ctx, need);
                if (st != CHUNKKV_OK) return st;
                base = static_cast<char*>(ctx->ws);
            }
            float* payload = reinterpret_cast<float*>(base + kHeaderBytes);
            ScoreArgs a;
            a.L = L; a.P = L - w; a.w = w; a.c = c; a.R = R; a.Hkv = sh.Hs; a.d = d; a.kv_shift = sh.shift;
            a.sl2 = static_cast<float>(1.4426950408889634 / sqrt(static_cast<double>(d)));
            score_scratch_layout(plan, sh.Hs, R, payload + cs_floats, &a);
            a.status = reinterpret_cast<int*>(base);
            CUtensorMap tm_q, tm_k;
            st = encode_bf16_3d(&tm_q, q_obs, d, R, sh.Hs, R < 128 ? R : 128, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
            if (st != CHUNKKV_OK) return st;
            st = encode_bf16_3d(&tm_k, K, d, L, Hkv, L < plan.n_tile ? L : plan.n_tile,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
            if (st != CHUNKKV_OK) return st;
            FusedLayerIO io;
            io.K = K; io.V = V; io.out_K = split ? nullptr : out_K; io.out_V = out_V; io.out_idx = out_idx;
            io.chunk_scores = payload;
            io.C = C; io.k = k; io.n_max = n_max; io.Hkv_out = Hkv;
            io.bar_count = reinterpret_cast<unsigned long long*>(base + 64);
            io.cooperative = lane != nullptr;
            {
                Timer t(ctx, s, 0);
                e = launch_layer_fused(plan, tm_q, tm_k, a, io, s);
            }
            if (e != cudaSuccess) return cuda_fail(e);
            if (split && rows_elsewhere == nullptr) {
                e = launch_gather_shared_sms(K, V, out_idx, L, Hkv, d, n_max, out_K, out_V, ctx->num_sms, s);
                if (e != cudaSuccess) return cuda_fail(e);
            }
            return CHUNKKV_OK;
        }
        if (lane != nullptr) return CHUNKKV_EINVAL_SHAPE;
        st = run_score(*ctx, q_obs, K, L, Hq, Hkv, d, w, c, nullptr, round64(static_cast<size_t>(Hkv) * C), &chunk_scores, s);
        if (st != CHUNKKV_OK) return st;
    }
    {
        Timer t(ctx, s, 2);
        e = launch_select(chunk_scores, L, Hkv, w, c, C, k, n_max, out_idx, s);
    }
    if (e != cudaSuccess) return cuda_fail(e);
    if (rows_elsewhere == nullptr) {
        Timer t(ctx, s, 3);
        e = launch_gather(K, V, out_idx, L, Hkv, d, n_max, out_K, out_V, nullptr, ctas, s);
    }
    if (e != cudaSuccess) return cuda_fail(e);
    return CHUNKKV_OK;
}

int chunkkv_jaccard(const int32_t* idx_a, const int32_t* idx_b, int Hkv, int n_a, int n_b,
                    float* out_ratio, int32_t* out_counts, void* stream) {
    if (Hkv < 1 || Hkv > 65535 || n_a < 0 || n_b < 0) return CHUNKKV_EINVAL_SHAPE;
    if (idx_a == nullptr || idx_b == nullptr || out_ratio == nullptr) return CHUNKKV_EINVAL_NULL;
    cudaError_t e = launch_jaccard(idx_a, idx_b, Hkv, n_a, n_b, out_ratio, out_counts, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(e);
    return CHUNKKV_OK;
}

int chunkkv_compress_layer(const void* q_obs, const void* K, const void* V, int L, int Hq, int Hkv,
                           int d, int w, int c, int budget, const int32_t* reuse_idx,
                           void* out_K, void* out_V, int32_t* out_idx, void* stream) {
    return compress_impl(q_obs, K, V, L, Hq, Hkv, d, w, c, budget, reuse_idx, out_K, out_V, out_idx, nullptr, 0, 0,
                         stream);
}

// The whole layer on keys and values that are not packed [Hkv, L, d]: e.g. a token-major cache [L, Hkv, d]
// (token stride Hkv * d, head stride d). Scores through tensor maps with those strides, selection, and a
// gather that reads rows by stride and writes packed outputs: separate launches.
int chunkkv_compress_layer_strided(const void* q_obs, const void* K, const void* V, int L, int Hq, int Hkv, int d,
                                   int w, int c, int budget, long long k_token_stride, long long k_head_stride,
                                   long long v_token_stride, long long v_head_stride, const int32_t* reuse_idx,
                                   void* out_K, void* out_V, int32_t* out_idx, void* stream) {
    if (k_token_stride == d && v_token_stride == d && k_head_stride == static_cast<long long>(L) * d &&
        v_head_stride == static_cast<long long>(L) * d)
        return chunkkv_compress_layer(q_obs, K, V, L, Hq, Hkv, d, w, c, budget, reuse_idx, out_K, out_V, out_idx, stream);
    int st = check_heads(L, Hq, Hkv, d, w);
    if (st != CHUNKKV_OK) return st;
    st = check_sizes(L, w, c, budget);
    if (st != CHUNKKV_OK) return st;
    if (K == nullptr || V == nullptr || out_K == nullptr || out_V == nullptr || out_idx == nullptr) return CHUNKKV_EINVAL_NULL;
    if (reuse_idx == nullptr && q_obs == nullptr) return CHUNKKV_EINVAL_NULL;
    // rows are moved and loaded 16 bytes at a time; a row may not overlap the next one
    const long long strides[4] = {k_token_stride, k_head_stride, v_token_stride, v_head_stride};
    for (long long sdv : strides)
        if (sdv < d || (sdv & 7) != 0) return CHUNKKV_EINVAL_SHAPE;
    if (!aligned16(q_obs) || !aligned16(K) || !aligned16(V) || !aligned16(out_K) || !aligned16(out_V))
        return CHUNKKV_EINVAL_ALIGN;
    const int C = chunkkv_num_chunks(L, w, c);
    const int k = chunkkv_num_kept_chunks(L, w, c, budget);
    const int n_max = chunkkv_out_len(L, w, c, budget);
    if (n_max < 0) return n_max;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    std::lock_guard<std::mutex> lk(g_mu);
    DeviceCtx* ctx = nullptr;
    st = get_ctx(&ctx);
    if (st != CHUNKKV_OK) return st;
    cudaError_t e;
    const int32_t* idx = reuse_idx;
    if (reuse_idx == nullptr && C > 0 && k > 0) {
        // the one-launch layer kernel takes strided keys and values as they are (tensor map and gather strides)
        const ScoreShape sh = score_shape(Hq, Hkv, w);
        ResidentPlan rplan;
        if (make_resident_plan(L, sh.Rs, sh.Hs, sh.shift, d, c, C, n_max, ctx->num_sms, smem_budget(*ctx), &rplan)) {
            st = ensure_workspace(*ctx, resident_scratch_floats(rplan, sh.Hs, C) * sizeof(float));
            if (st != CHUNKKV_OK) return st;
            char* base = static_cast<char*>(ctx->ws);
            CUtensorMap tm_q, tm_k;
            st = encode_bf16_3d(&tm_q, q_obs, d, sh.Rs, sh.Hs, sh.Rs < 128 ? sh.Rs : 128, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
            if (st != CHUNKKV_OK) return st;
            st = encode_bf16_3d(&tm_k, K, d, L, Hkv, L < 120 ? L : 120, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, k_token_stride,
                                k_head_stride);
            if (st != CHUNKKV_OK) return st;
            ResidentIO io;
            io.L = L; io.w = w; io.Rs = sh.Rs; io.Hs = sh.Hs; io.d = d; io.kv_shift = sh.shift;
            io.sl2 = static_cast<float>(1.4426950408889634 / sqrt(static_cast<double>(d)));
            io.C = C; io.k = k; io.n_max = n_max;
            io.K = K; io.V = V; io.out_K = out_K; io.out_V = out_V; io.out_idx = out_idx;
            io.scratch = reinterpret_cast<float*>(base + kHeaderBytes);
            io.counters = reinterpret_cast<unsigned*>(base + kResidentCountersOffset);
            io.status = reinterpret_cast<int*>(base);
            io.cooperative = false;
            io.k_row_elems = k_token_stride; io.k_head_elems = k_head_stride;
            io.v_row_elems = v_token_stride; io.v_head_elems = v_head_stride;
            e = launch_layer_resident(rplan, tm_q, tm_k, io, s);
            if (e != cudaSuccess) return cuda_fail(e);
            return CHUNKKV_OK;
        }
    }
    if (reuse_idx == nullptr) {
        float* chunk_scores = nullptr;
        if (C > 0 && k > 0) {
            st = run_score(*ctx, q_obs, K, L, Hq, Hkv, d, w, c, nullptr, round64(static_cast<size_t>(Hkv) * C), &chunk_scores, s,
                           k_token_stride, k_head_stride);
            if (st != CHUNKKV_OK) return st;
        }
        e = launch_select(chunk_scores, L, Hkv, w, c, C, k, n_max, out_idx, s);
        if (e != cudaSuccess) return cuda_fail(e);
        idx = out_idx;
    }
    e = launch_gather_strided(K, V, idx, L, Hkv, d, n_max, k_token_stride, k_head_stride, v_token_stride, v_head_stride,
                              out_K, out_V, idx == out_idx ? nullptr : out_idx, ctx->num_sms, s);
    if (e != cudaSuccess) return cuda_fail(e);
    return CHUNKKV_OK;
}

// ---- Adapters to the steps either side of the path: window queries out of a fused QKV activation
//      (with rotary embedding), and kept rows into a paged decode cache.
int chunkkv_window_queries(const void* qkv, long long row_elems, int T, int Hq, int Hkv, int d, int w,
                           const float* cos_rows, const float* sin_rows, void* out_q_obs, void* stream) {
    if (Hkv < 1 || Hq < Hkv || Hq % Hkv != 0 || (d != 64 && d != 128) || w < 1 || T < w) return CHUNKKV_EINVAL_SHAPE;
    if (row_elems < static_cast<long long>(Hq + 2 * Hkv) * d) return CHUNKKV_EINVAL_SHAPE;
    if (qkv == nullptr || cos_rows == nullptr || sin_rows == nullptr || out_q_obs == nullptr) return CHUNKKV_EINVAL_NULL;
    if (!aligned16(out_q_obs) || (reinterpret_cast<uintptr_t>(qkv) & 1u) != 0 || (row_elems & 7) != 0)
        return CHUNKKV_EINVAL_ALIGN;
    cudaError_t e = launch_window_queries(qkv, row_elems, T, Hq, d, w, cos_rows, sin_rows, out_q_obs,
                                          static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(e);
    return CHUNKKV_OK;
}

static int check_paged(int n_max, int page_size, int num_pages, const int32_t* block_table, const void* cache_K,
                       const void* cache_V) {
    if (page_size < 1 || num_pages < 1 || n_max < 0) return CHUNKKV_EINVAL_SHAPE;
    if (block_table == nullptr || cache_K == nullptr || cache_V == nullptr) return CHUNKKV_EINVAL_NULL;
    if (!aligned16(cache_K) || !aligned16(cache_V) || (reinterpret_cast<uintptr_t>(block_table) & 3u) != 0)
        return CHUNKKV_EINVAL_ALIGN;
    return CHUNKKV_OK;
}

int chunkkv_gather_paged(const void* K, const void* V, const int32_t* idx, int L, int Hkv, int d, int n_max,
                         const int32_t* block_table, int page_size, int num_pages, void* cache_K, void* cache_V,
                         void* stream) {
    if (L < 1 || Hkv < 1 || Hkv > 65535 || n_max < 0 || (d != 64 && d != 128)) return CHUNKKV_EINVAL_SHAPE;
    if (static_cast<long long>(Hkv) * L * d >= (1LL << 40)) return CHUNKKV_EINVAL_SHAPE;
    int st = check_paged(n_max, page_size, num_pages, block_table, cache_K, cache_V);
    if (st != CHUNKKV_OK) return st;
    if (K == nullptr || V == nullptr || idx == nullptr) return CHUNKKV_EINVAL_NULL;
    if (!aligned16(K) || !aligned16(V) || !aligned16(idx)) return CHUNKKV_EINVAL_ALIGN;
    std::lock_guard<std::mutex> lk(g_mu);
    DeviceCtx* ctx;
    st = get_ctx(&ctx);
    if (st != CHUNKKV_OK) return st;
    cudaError_t e = launch_gather_paged(K, V, idx, L, Hkv, d, n_max, block_table, page_size, num_pages, cache_K, cache_V,
                                        ctx->num_sms, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(e);
    return CHUNKKV_OK;
}

int chunkkv_compress_layer_paged(const void* q_obs, const void* K, const void* V, int L, int Hq, int Hkv, int d, int w,
                                 int c, int budget, const int32_t* reuse_idx, const int32_t* block_table, int page_size,
                                 int num_pages, void* cache_K, void* cache_V, int32_t* out_idx, void* stream) {
    int st = check_sizes(L, w, c, budget);
    if (st != CHUNKKV_OK) return st;
    st = check_heads(L, Hq, Hkv, d, w);
    if (st != CHUNKKV_OK) return st;
    const int C = chunkkv_num_chunks(L, w, c);
    const int k = chunkkv_num_kept_chunks(L, w, c, budget);
    const int n_max = chunkkv_out_len(L, w, c, budget);
    if (n_max < 0) return n_max;
    st = check_paged(n_max, page_size, num_pages, block_table, cache_K, cache_V);
    if (st != CHUNKKV_OK) return st;
    if (K == nullptr || V == nullptr || out_idx == nullptr || (reuse_idx == nullptr && q_obs == nullptr))
        return CHUNKKV_EINVAL_NULL;
    if (!aligned16(q_obs) || !aligned16(K) || !aligned16(V) || !aligned16(out_idx) || !aligned16(reuse_idx))
        return CHUNKKV_EINVAL_ALIGN;
    std::lock_guard<std::mutex> lk(g_mu);
    DeviceCtx* ctx;
    st = get_ctx(&ctx);
    if (st != CHUNKKV_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    if (reuse_idx != nullptr) {
        if (reuse_idx != out_idx) {
            e = cudaMemcpyAsync(out_idx, reuse_idx, static_cast<size_t>(Hkv) * n_max * sizeof(int32_t),
                                cudaMemcpyDeviceToDevice, s);
            if (e != cudaSuccess) return cuda_fail(e);
        }
    } else {
        if (C > 0 && k > 0) {
            // the one-launch layer kernel places the kept rows through the block table itself
            const ScoreShape sh = score_shape(Hq, Hkv, w);
            ResidentPlan rplan;
            if (make_resident_plan(L, sh.Rs, sh.Hs, sh.shift, d, c, C, n_max, ctx->num_sms, smem_budget(*ctx), &rplan)) {
                st = ensure_workspace(*ctx, resident_scratch_floats(rplan, sh.Hs, C) * sizeof(float));
                if (st != CHUNKKV_OK) return st;
                char* base = static_cast<char*>(ctx->ws);
                CUtensorMap tm_q, tm_k;
                st = encode_bf16_3d(&tm_q, q_obs, d, sh.Rs, sh.Hs, sh.Rs < 128 ? sh.Rs : 128, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
                if (st != CHUNKKV_OK) return st;
                st = encode_bf16_3d(&tm_k, K, d, L, Hkv, L < 120 ? L : 120, CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
                if (st != CHUNKKV_OK) return st;
                ResidentIO io;
                io.L = L; io.w = w; io.Rs = sh.Rs; io.Hs = sh.Hs; io.d = d; io.kv_shift = sh.shift;
                io.sl2 = static_cast<float>(1.4426950408889634 / sqrt(static_cast<double>(d)));
                io.C = C; io.k = k; io.n_max = n_max;
                io.K = K; io.V = V; io.out_K = cache_K; io.out_V = cache_V; io.out_idx = out_idx;
                io.scratch = reinterpret_cast<float*>(base + kHeaderBytes);
                io.counters = reinterpret_cast<unsigned*>(base + kResidentCountersOffset);
                io.status = reinterpret_cast<int*>(base);
                io.cooperative = false;
                io.block_table = block_table; io.page_size = page_size; io.num_pages = num_pages;
                e = launch_layer_resident(rplan, tm_q, tm_k, io, s);
                if (e != cudaSuccess) return cuda_fail(e);
                return CHUNKKV_OK;
            }
        }
        float* chunk_scores = nullptr;
        if (C > 0 && k > 0) {
            st = run_score(*ctx, q_obs, K, L, Hq, Hkv, d, w, c, nullptr, round64(static_cast<size_t>(Hkv) * C),
                           &chunk_scores, s);
            if (st != CHUNKKV_OK) return st;
        }
        e = launch_select(chunk_scores, L, Hkv, w, c, C, k, n_max, out_idx, s);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    e = launch_gather_paged(K, V, out_idx, L, Hkv, d, n_max, block_table, page_size, num_pages, cache_K, cache_V,
                            ctx->num_sms, s);
    if (e != cudaSuccess) return cuda_fail(e);
    return CHUNKKV_OK;
}

// ---- Algorithm 2 over a whole model: every reuse_depth-th layer computes indices, the layers
//      between gather with them. Where the shape fits the persistent kernel the layers go through
//      it in launches of up to kModelMaxLayers; otherwise layer by layer.
static int model_args_ok(int n_layers, int reuse_depth) {
    if (n_layers < 1 || reuse_depth < 1) return CHUNKKV_EINVAL_SHAPE;
    return CHUNKKV_OK;
}

size_t chunkkv_model_workspace_bytes(int n_layers, int L, int Hq, int Hkv, int d, int w, int c, int budget,
                                     int reuse_depth) {
    if (model_args_ok(n_layers, reuse_depth) != CHUNKKV_OK || check_sizes(L, w, c, budget) != CHUNKKV_OK) return 0;
    const size_t per_layer = chunkkv_workspace_bytes(L, Hq, Hkv, d, w, c);
    if (per_layer == 0) return 0;
    std::lock_guard<std::mutex> lk(g_mu);
    DeviceCtx* ctx;
    if (get_ctx(&ctx) != CHUNKKV_OK) return 0;
    const ScoreShape sh = score_shape(Hq, Hkv, w);
    const int C = (L - w + c - 1) / c;
    const int k = chunkkv_num_kept_chunks(L, w, c, budget);
    ModelPlan mp;
    size_t need = per_layer;
    if (C > 0 && k > 0 && make_model_plan(L, sh.Rs, sh.Hs, sh.shift, d, c, C, k, ctx->num_sms, smem_budget(*ctx), &mp)) {
        const int per_launch = n_layers < kModelMaxLayers ? n_layers : kModelMaxLayers;
        const int n_compute = (per_launch + reuse_depth - 1) / reuse_depth + 1;
        const size_t m = kHeaderBytes + model_scratch_floats(mp, sh.Hs, sh.shift, C, n_compute) * sizeof(float);
        need = m > need ? m : need;
    }
    return need;
}

// kt / kh / vt / vh: elements between consecutive rows of a head and between heads of K and of V; 0 = packed
static int compress_model_impl(int n_layers, const void* const* q_obs, const void* const* K, const void* const* V,
                               int L, int Hq, int Hkv, int d, int w, int c, int budget, int reuse_depth,
                               void* const* out_K, void* const* out_V, int32_t* const* out_idx, void* stream,
                               long long kt, long long kh, long long vt, long long vh,
                               const int32_t* const* block_tables = nullptr, int page_size = 0, int num_pages = 0) {
    const bool strided = kt != 0;
    const bool paged = page_size > 0;      // out_K / out_V are then the layers' paged caches
    int st = model_args_ok(n_layers, reuse_depth);
    if (st != CHUNKKV_OK) return st;
    st = check_sizes(L, w, c, budget);
    if (st != CHUNKKV_OK) return st;
    st = check_heads(L, Hq, Hkv, d, w);
    if (st != CHUNKKV_OK) return st;
    if (q_obs == nullptr || K == nullptr || V == nullptr || out_K == nullptr || out_V == nullptr || out_idx == nullptr)
        return CHUNKKV_EINVAL_NULL;
    for (int l = 0; l < n_layers; ++l) {
        const bool computes = (l % reuse_depth) == 0;
        if (K[l] == nullptr || V[l] == nullptr || out_K[l] == nullptr || out_V[l] == nullptr || out_idx[l] == nullptr ||
            (computes && q_obs[l] == nullptr))
            return CHUNKKV_EINVAL_NULL;
        if (!aligned16(K[l]) || !aligned16(V[l]) || !aligned16(out_K[l]) || !aligned16(out_V[l]) ||
            !aligned16(out_idx[l]) || (computes && !aligned16(q_obs[l])))
            return CHUNKKV_EINVAL_ALIGN;
    }
    const int C = chunkkv_num_chunks(L, w, c);
    const int k = chunkkv_num_kept_chunks(L, w, c, budget);
    const int n_max = chunkkv_out_len(L, w, c, budget);
    if (n_max < 0) return n_max;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    ModelPlan mp;
    bool persistent = false;
    DeviceCtx* ctx = nullptr;
    ScoreShape sh = score_shape(Hq, Hkv, w);
    {
        std::lock_guard<std::mutex> lk(g_mu);
        st = get_ctx(&ctx);
        if (st != CHUNKKV_OK) return st;
        // paged outputs run layer by layer: the one-launch layer kernel places rows through the block table with all
        // its threads, which measured faster (35 us per layer) than the persistent kernel's copy warp doing it (41 us)
        persistent = !paged && C > 0 && k > 0 &&
                     make_model_plan(L, sh.Rs, sh.Hs, sh.shift, d, c, C, k, ctx->num_sms, smem_budget(*ctx), &mp);
    }
    if (!persistent) {
        // layer by layer: Algorithm 2's call sequence over chunkkv_compress_layer
        for (int l = 0; l < n_layers; ++l) {
            const int src = (l / reuse_depth) * reuse_depth;
            if (paged)
                st = chunkkv_compress_layer_paged(l == src ? q_obs[l] : nullptr, K[l], V[l], L, Hq, Hkv, d, w, c, budget,
                                                  l == src ? nullptr : out_idx[src], block_tables[l], page_size, num_pages,
                                                  out_K[l], out_V[l], out_idx[l], stream);
            else if (strided)
                st = chunkkv_compress_layer_strided(l == src ? q_obs[l] : nullptr, K[l], V[l], L, Hq, Hkv, d, w, c, budget, kt, kh,
                                                    vt, vh, l == src ? nullptr : out_idx[src], out_K[l], out_V[l], out_idx[l],
                                                    stream);
            else
                st = chunkkv_compress_layer(l == src ? q_obs[l] : nullptr, K[l], V[l], L, Hq, Hkv, d, w, c, budget,
                                        l == src ? nullptr : out_idx[src], out_K[l], out_V[l], out_idx[l], stream);
            if (st != CHUNKKV_OK) return st;
        }
        return CHUNKKV_OK;
    }
    std::lock_guard<std::mutex> lk(g_mu);
    std::vector<CUtensorMap> tm_q(kModelMaxCompute), tm_k(kModelMaxCompute);
    std::vector<ModelLayerIO> lay(kModelMaxLayers);
    for (int l0 = 0; l0 < n_layers;) {
        // a launch takes whole reuse groups, at most kModelMaxLayers layers
        int l1 = l0;
        int n_compute = 0;
        while (l1 < n_layers) {
            const int group_end = (l1 + reuse_depth < n_layers) ? l1 + reuse_depth : n_layers;
            if (group_end - l0 > kModelMaxLayers && l1 > l0) break;
            if (group_end - l0 > kModelMaxLayers) {         // a single reuse group longer than a launch: split it
                l1 = l0 + kModelMaxLayers;
                if (n_compute == 0) n_compute = 1;
                break;
            }
            l1 = group_end;
            ++n_compute;
        }
        const int n = l1 - l0;
        const size_t need = model_scratch_floats(mp, sh.Hs, sh.shift, C, n_compute) * sizeof(float);
        st = ensure_workspace(*ctx, need);
        if (st != CHUNKKV_OK) return st;
        char* base = static_cast<char*>(ctx->ws);
        int nc = 0;
        for (int i = 0; i < n; ++i) {
            const int l = l0 + i;
            const bool computes = (l % reuse_depth) == 0;
            lay[i].K = K[l]; lay[i].V = V[l]; lay[i].out_K = out_K[l]; lay[i].out_V = out_V[l]; lay[i].out_idx = out_idx[l];
            lay[i].computes = computes;
            if (computes) {
                st = encode_bf16_3d(&tm_q[nc], q_obs[l], d, sh.Rs, sh.Hs, sh.Rs < 128 ? sh.Rs : 128,
                                    CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
                if (st != CHUNKKV_OK) return st;
                st = encode_bf16_3d(&tm_k[nc], K[l], d, L, Hkv, L < 120 ? L : 120, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, kt, kh);
                if (st != CHUNKKV_OK) return st;
                ++nc;
            }
        }
        if (!lay[0].computes) {
            // the launch starts inside a reuse group (a group longer than a launch): these layers gather
            // with indices computed by an earlier launch
            int i = 0;
            for (; i < n && !lay[i].computes; ++i) {
                const int l = l0 + i, src = (l / reuse_depth) * reuse_depth;
                cudaError_t e = paged   ? launch_gather_paged(K[l], V[l], out_idx[src], L, Hkv, d, n_max, block_tables[l], page_size,
                                                              num_pages, out_K[l], out_V[l], ctx->num_sms, s)
                                : strided ? launch_gather_strided(K[l], V[l], out_idx[src], L, Hkv, d, n_max, kt, kh, vt, vh, out_K[l],
                                                                out_V[l], out_idx[l], ctx->num_sms, s)
                                        : launch_gather(K[l], V[l], out_idx[src], L, Hkv, d, n_max, out_K[l], out_V[l], out_idx[l],
                                                        ctx->num_sms, s);
                if (e != cudaSuccess) return cuda_fail(e);
                if (paged && out_idx[l] != out_idx[src]) {      // (the paged gather does not copy the indices)
                    e = cudaMemcpyAsync(out_idx[l], out_idx[src], static_cast<size_t>(Hkv) * n_max * sizeof(int32_t),
                                        cudaMemcpyDeviceToDevice, s);
                    if (e != cudaSuccess) return cuda_fail(e);
                }
            }
            l0 += i;
            continue;
        }
        ModelIO io;
        io.L = L; io.w = w; io.Rs = sh.Rs; io.Hs = sh.Hs; io.d = d; io.kv_shift = sh.shift;
        io.sl2 = static_cast<float>(1.4426950408889634 / sqrt(static_cast<double>(d)));
        io.C = C; io.k = k; io.n_max = n_max;
        io.scratch = reinterpret_cast<float*>(base + kHeaderBytes);
        io.counters = reinterpret_cast<unsigned*>(base + kResidentCountersOffset);
        io.status = reinterpret_cast<int*>(base);
        io.k_row_elems = kt; io.k_head_elems = kh; io.v_row_elems = vt; io.v_head_elems = vh;
        cudaError_t e;
        {
            Timer t(ctx, s, 0);
            e = launch_model(mp, io, tm_q.data(), tm_k.data(), lay.data(), n, s);
        }
        if (e != cudaSuccess) return cuda_fail(e);
        l0 = l1;
    }
    return CHUNKKV_OK;
}

int chunkkv_compress_model(int n_layers, const void* const* q_obs, const void* const* K, const void* const* V,
                           int L, int Hq, int Hkv, int d, int w, int c, int budget, int reuse_depth,
                           void* const* out_K, void* const* out_V, int32_t* const* out_idx, void* stream) {
    return compress_model_impl(n_layers, q_obs, K, V, L, Hq, Hkv, d, w, c, budget, reuse_depth, out_K, out_V, out_idx, stream,
                               0, 0, 0, 0);
}

int chunkkv_compress_model_paged(int n_layers, const void* const* q_obs, const void* const* K, const void* const* V,
                                 int L, int Hq, int Hkv, int d, int w, int c, int budget, int reuse_depth,
                                 const int32_t* const* block_tables, int page_size, int num_pages, void* const* cache_K,
                                 void* const* cache_V, int32_t* const* out_idx, void* stream) {
    int st = model_args_ok(n_layers, reuse_depth);
    if (st != CHUNKKV_OK) return st;
    st = check_sizes(L, w, c, budget);
    if (st != CHUNKKV_OK) return st;
    if (block_tables == nullptr || cache_K == nullptr || cache_V == nullptr) return CHUNKKV_EINVAL_NULL;
    const int n_max = chunkkv_out_len(L, w, c, budget);
    if (n_max < 0) return n_max;
    for (int l = 0; l < n_layers; ++l) {
        st = check_paged(n_max, page_size, num_pages, block_tables[l], cache_K[l], cache_V[l]);
        if (st != CHUNKKV_OK) return st;
    }
    return compress_model_impl(n_layers, q_obs, K, V, L, Hq, Hkv, d, w, c, budget, reuse_depth, cache_K, cache_V, out_idx, stream,
                               0, 0, 0, 0, block_tables, page_size, num_pages);
}

int chunkkv_compress_model_strided(int n_layers, const void* const* q_obs, const void* const* K, const void* const* V,
                                   int L, int Hq, int Hkv, int d, int w, int c, int budget, int reuse_depth,
                                   long long k_token_stride, long long k_head_stride, long long v_token_stride,
                                   long long v_head_stride, void* const* out_K, void* const* out_V,
                                   int32_t* const* out_idx, void* stream) {
    if (k_token_stride == d && v_token_stride == d && k_head_stride == static_cast<long long>(L) * d &&
        v_head_stride == static_cast<long long>(L) * d)
        return chunkkv_compress_model(n_layers, q_obs, K, V, L, Hq, Hkv, d, w, c, budget, reuse_depth, out_K, out_V, out_idx,
                                      stream);
    const long long strides[4] = {k_token_stride, k_head_stride, v_token_stride, v_head_stride};
    for (long long sdv : strides)
        if (sdv < d || (sdv & 7) != 0) return CHUNKKV_EINVAL_SHAPE;
    return compress_model_impl(n_layers, q_obs, K, V, L, Hq, Hkv, d, w, c, budget, reuse_depth, out_K, out_V, out_idx, stream,
                               k_token_stride, k_head_stride, v_token_stride, v_head_stride);
}

// ---- Algorithm 1's budget rule: k = floor(L_max / c) chunks, their tokens cut to the first
//      L_max - w, the window last. Scoring and gathering are the calls above; only the number of
//      kept chunks, the output length and the cut differ.
int chunkkv_budget_from_ratio(int L, double ratio) {
    if (L < 0 || !(ratio >= 0.0 && ratio <= 1.0)) return CHUNKKV_EINVAL_SHAPE;
    return static_cast<int>(floor(ratio * static_cast<double>(L)));
}

int chunkkv_num_kept_chunks_alg1(int L, int w, int c, int budget) {
    int st = check_sizes(L, w, c, budget);
    if (st != CHUNKKV_OK) return st;
    const int C = (L - w + c - 1) / c;
    const int k = budget / c;
    return k < C ? k : C;
}

int chunkkv_out_len_alg1(int L, int w, int c, int budget) {
    const int k = chunkkv_num_kept_chunks_alg1(L, w, c, budget);
    if (k < 0) return k;
    const long long full = static_cast<long long>(k) * c, cap = budget - w;
    return static_cast<int>((full < cap ? full : cap) + w);
}

int chunkkv_select_alg1(const float* chunk_scores, int L, int Hkv, int w, int c, int budget,
                        int32_t* out_idx, void* stream) {
    int st = check_sizes(L, w, c, budget);
    if (st != CHUNKKV_OK) return st;
    if (Hkv < 1 || Hkv > 65535) return CHUNKKV_EINVAL_SHAPE;
    const int C = chunkkv_num_chunks(L, w, c);
    const int k = chunkkv_num_kept_chunks_alg1(L, w, c, budget);
    const int n_max = chunkkv_out_len_alg1(L, w, c, budget);
    if (out_idx == nullptr || (C > 0 && k > 0 && chunk_scores == nullptr)) return CHUNKKV_EINVAL_NULL;
    if (!aligned16(out_idx) || !aligned16(chunk_scores)) return CHUNKKV_EINVAL_ALIGN;
    std::lock_guard<std::mutex> lk(g_mu);
    DeviceCtx* ctx;
    st = get_ctx(&ctx);
    if (st != CHUNKKV_OK) return st;
    cudaError_t e = launch_select(chunk_scores, L, Hkv, w, c, C, k, n_max, out_idx,
                                  static_cast<cudaStream_t>(stream), budget - w);
    if (e != cudaSuccess) return cuda_fail(e);
    return CHUNKKV_OK;
}

int chunkkv_compress_layer_alg1(const void* q_obs, const void* K, const void* V, int L, int Hq, int Hkv,
                                int d, int w, int c, int budget, void* out_K, void* out_V, int32_t* out_idx,
                                void* stream) {
    int st = check_sizes(L, w, c, budget);
    if (st != CHUNKKV_OK) return st;
    st = check_heads(L, Hq, Hkv, d, w);
    if (st != CHUNKKV_OK) return st;
    if (q_obs == nullptr || K == nullptr || V == nullptr || out_K == nullptr || out_V == nullptr || out_idx == nullptr)
        return CHUNKKV_EINVAL_NULL;
    if (!aligned16(q_obs) || !aligned16(K) || !aligned16(V) || !aligned16(out_K) || !aligned16(out_V) ||
        !aligned16(out_idx))
        return CHUNKKV_EINVAL_ALIGN;
    const int C = chunkkv_num_chunks(L, w, c);
    const int k = chunkkv_num_kept_chunks_alg1(L, w, c, budget);
    const int n_max = chunkkv_out_len_alg1(L, w, c, budget);
    std::lock_guard<std::mutex> lk(g_mu);
    DeviceCtx* ctx;
    st = get_ctx(&ctx);
    if (st != CHUNKKV_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (C > 0 && k > 0) {
        // the one-launch layer kernel with Algorithm 1's chunk count and token cap
        const ScoreShape sh = score_shape(Hq, Hkv, w);
        ResidentPlan rplan;
        if (make_resident_plan(L, sh.Rs, sh.Hs, sh.shift, d, c, C, n_max, ctx->num_sms, smem_budget(*ctx), &rplan)) {
            st = ensure_workspace(*ctx, resident_scratch_floats(rplan, sh.Hs, C) * sizeof(float));
            if (st != CHUNKKV_OK) return st;
            char* base = static_cast<char*>(ctx->ws);
            CUtensorMap tm_q, tm_k;
            st = encode_bf16_3d(&tm_q, q_obs, d, sh.Rs, sh.Hs, sh.Rs < 128 ? sh.Rs : 128, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
            if (st != CHUNKKV_OK) return st;
            st = encode_bf16_3d(&tm_k, K, d, L, Hkv, L < 120 ? L : 120, CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
            if (st != CHUNKKV_OK) return st;
            ResidentIO io;
            io.L = L; io.w = w; io.Rs = sh.Rs; io.Hs = sh.Hs; io.d = d; io.kv_shift = sh.shift;
            io.sl2 = static_cast<float>(1.4426950408889634 / sqrt(static_cast<double>(d)));
            io.C = C; io.k = k; io.n_max = n_max;
            io.K = K; io.V = V; io.out_K = out_K; io.out_V = out_V; io.out_idx = out_idx;
            io.scratch = reinterpret_cast<float*>(base + kHeaderBytes);
            io.counters = reinterpret_cast<unsigned*>(base + kResidentCountersOffset);
            io.status = reinterpret_cast<int*>(base);
            io.cooperative = false;
            io.tok_cap = budget - w;
            cudaError_t e2 = launch_layer_resident(rplan, tm_q, tm_k, io, s);
            if (e2 != cudaSuccess) return cuda_fail(e2);
            return CHUNKKV_OK;
        }
    }
    float* chunk_scores = nullptr;
    if (C > 0 && k > 0) {
        st = run_score(*ctx, q_obs, K, L, Hq, Hkv, d, w, c, nullptr, round64(static_cast<size_t>(Hkv) * C), &chunk_scores, s);
        if (st != CHUNKKV_OK) return st;
    }
    cudaError_t e = launch_select(chunk_scores, L, Hkv, w, c, C, k, n_max, out_idx, s, budget - w);
    if (e != cudaSuccess) return cuda_fail(e);
    e = launch_gather(K, V, out_idx, L, Hkv, d, n_max, out_K, out_V, nullptr, ctx->num_sms, s);
    if (e != cudaSuccess) return cuda_fail(e);
    return CHUNKKV_OK;
}

size_t chunkkv_lane_bytes(int L, int Hq, int Hkv, int d, int w, int c, int max_ctas) {
    if (w < 1 || c < 1 || L < w || max_ctas < 0) return 0;
    if (check_heads(L, Hq, Hkv, d, w) != CHUNKKV_OK) return 0;
    std::lock_guard<std::mutex> lk(g_mu);
    DeviceCtx* ctx;
    if (get_ctx(&ctx) != CHUNKKV_OK) return 0;
    const int ctas = (max_ctas > 0 && max_ctas < ctx->num_sms) ? max_ctas : ctx->num_sms;
    const ScoreShape sh = score_shape(Hq, Hkv, w);
    const int C = (L - w + c - 1) / c;
    ScorePlan plan;
    if (!make_score_plan(L, sh.Rs, sh.Hs, d, c, ctas, smem_budget(*ctx), true, &plan)) return 0;
    size_t floats = score_scratch_floats(plan, sh.Hs, sh.Rs) + round64(static_cast<size_t>(sh.Hs) * C);
    ResidentPlan rplan;
    if (C > 0 && make_resident_plan(L, sh.Rs, sh.Hs, sh.shift, d, c, C, 0, ctas, smem_budget(*ctx), &rplan)) {
        const size_t rf = resident_scratch_floats(rplan, sh.Hs, C);
        floats = rf > floats ? rf : floats;
    }
    return kHeaderBytes + floats * sizeof(float);
}

int chunkkv_lane_init(void* lane, size_t bytes, void* stream) {
    if (lane == nullptr) return CHUNKKV_EINVAL_NULL;
    if ((reinterpret_cast<uintptr_t>(lane) & 255u) != 0) return CHUNKKV_EINVAL_ALIGN;
    if (bytes < kHeaderBytes) return CHUNKKV_ENOWORKSPACE;
    cudaError_t e = cudaMemsetAsync(lane, 0, kHeaderBytes, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(e);
    return CHUNKKV_OK;
}

int chunkkv_lane_status(void* lane, void* stream) {
    if (lane == nullptr) return CHUNKKV_EINVAL_NULL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail(e);
    int flag = 0;
    e = cudaMemcpy(&flag, lane, sizeof(int), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(e);
    if (flag != 0) {
        cudaMemset(lane, 0, kHeaderBytes);
        return CHUNKKV_EDEVICE;
    }
    return CHUNKKV_OK;
}

int chunkkv_compress_layer_lane(const void* q_obs, const void* K, const void* V, int L, int Hq, int Hkv,
                                int d, int w, int c, int budget, const int32_t* reuse_idx,
                                void* out_K, void* out_V, int32_t* out_idx,
                                void* lane, size_t lane_bytes, int max_ctas, void* stream) {
    if (lane == nullptr) return CHUNKKV_EINVAL_NULL;
    if ((reinterpret_cast<uintptr_t>(lane) & 255u) != 0) return CHUNKKV_EINVAL_ALIGN;
    return compress_impl(q_obs, K, V, L, Hq, Hkv, d, w, c, budget, reuse_idx, out_K, out_V, out_idx, lane, lane_bytes,
                         max_ctas, stream);
}

size_t chunkkv_pipe_bytes(int L, int Hq, int Hkv, int d, int w, int c, int max_ctas) {
    return chunkkv_lane_bytes(L, Hq, Hkv, d, w, c, max_ctas);
}

int chunkkv_pipe_open(void* scratch, size_t bytes, int max_ctas, void** pipe_out) {
    if (scratch == nullptr || pipe_out == nullptr) return CHUNKKV_EINVAL_NULL;
    *pipe_out = nullptr;
    if ((reinterpret_cast<uintptr_t>(scratch) & 255u) != 0) return CHUNKKV_EINVAL_ALIGN;
    if (max_ctas < 0) return CHUNKKV_EINVAL_SHAPE;
    if (bytes < kHeaderBytes) return CHUNKKV_ENOWORKSPACE;
    Pipe* p = new Pipe();
    cudaError_t e = cudaGetDevice(&p->device);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&p->side, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p->scored, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p->posted, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaMemset(scratch, 0, kHeaderBytes);
    if (e != cudaSuccess) {
        if (p->scored) cudaEventDestroy(p->scored);
        if (p->posted) cudaEventDestroy(p->posted);
        if (p->side) cudaStreamDestroy(p->side);
        delete p;
        return cuda_fail(e);
    }
    p->scratch = static_cast<char*>(scratch);
    p->bytes = bytes;
    p->max_ctas = max_ctas;
    *pipe_out = p;
    return CHUNKKV_OK;
}

int chunkkv_pipe_layer(void* pipe, const void* q_obs, const void* K, const void* V, int L, int Hq, int Hkv,
                       int d, int w, int c, int budget, void* out_K, void* out_V, int32_t* out_idx,
                       void* stream) {
    if (pipe == nullptr) return CHUNKKV_EINVAL_NULL;
    Pipe* p = static_cast<Pipe*>(pipe);
    if (q_obs == nullptr) return CHUNKKV_EINVAL_NULL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // scoring, chunk scores and selection on the caller's stream (the lane's layer kernel without
    // its gather phase), ...
    int st = compress_impl(q_obs, K, V, L, Hq, Hkv, d, w, c, budget, nullptr, out_K, out_V, out_idx, p->scratch,
                           p->bytes, p->max_ctas, stream, /*rows_on=*/&p->side);
    if (st != CHUNKKV_OK) return st;
    std::lock_guard<std::mutex> lk(g_mu);
    // ... the row gather on the pipe's stream, after it
    cudaError_t e = cudaEventRecord(p->scored, s);
    if (e != cudaSuccess) return cuda_fail(e);
    e = cudaStreamWaitEvent(p->side, p->scored, 0);
    if (e != cudaSuccess) return cuda_fail(e);
    DeviceCtx* ctx;
    st = get_ctx(&ctx);
    if (st != CHUNKKV_OK) return st;
    const int n_max = chunkkv_out_len(L, w, c, budget);
    e = launch_gather_shared_sms(K, V, out_idx, L, Hkv, d, n_max, out_K, out_V, ctx->num_sms, p->side);
    if (e != cudaSuccess) return cuda_fail(e);
    e = cudaEventRecord(p->posted, p->side);
    if (e != cudaSuccess) return cuda_fail(e);
    p->pending = true;
    return CHUNKKV_OK;
}

int chunkkv_pipe_join(void* pipe, void* stream) {
    if (pipe == nullptr) return CHUNKKV_EINVAL_NULL;
    Pipe* p = static_cast<Pipe*>(pipe);
    std::lock_guard<std::mutex> lk(g_mu);
    if (p->pending) {
        cudaError_t e = cudaStreamWaitEvent(static_cast<cudaStream_t>(stream), p->posted, 0);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    p->pending = false;
    return CHUNKKV_OK;
}

int chunkkv_pipe_status(void* pipe, void* stream) {
    int st = chunkkv_pipe_join(pipe, stream);
    if (st != CHUNKKV_OK) return st;
    return chunkkv_lane_status(static_cast<Pipe*>(pipe)->scratch, stream);
}

int chunkkv_pipe_close(void* pipe) {
    if (pipe == nullptr) return CHUNKKV_EINVAL_NULL;
    Pipe* p = static_cast<Pipe*>(pipe);
    std::lock_guard<std::mutex> lk(g_mu);
    cudaError_t e = cudaStreamSynchronize(p->side);
    cudaEventDestroy(p->scored);
    cudaEventDestroy(p->posted);
    cudaStreamDestroy(p->side);
    delete p;
    if (e != cudaSuccess) return cuda_fail(e);
    return CHUNKKV_OK;
}

int chunkkv_compress_layer_host(const void* host_q_obs, const void* host_K, const void* host_V,
                                int L, int Hq, int Hkv, int d, int w, int c, int budget,
                                void* dev_q_obs, void* dev_K, void* dev_V,
                                void* dev_out_K, void* dev_out_V, int32_t* dev_out_idx,
                                void* host_out_K, void* host_out_V, int32_t* host_out_idx,
                                void* stream) {
    int st = check_sizes(L, w, c, budget);
    if (st != CHUNKKV_OK) return st;
    st = check_heads(L, Hq, Hkv, d, w);
    if (st != CHUNKKV_OK) return st;
    if (!host_q_obs || !host_K || !host_V || !dev_q_obs || !dev_K || !dev_V || !dev_out_K || !dev_out_V ||
        !dev_out_idx || !host_out_K || !host_out_V || !host_out_idx)
        return CHUNKKV_EINVAL_NULL;
    const int n_max = chunkkv_out_len(L, w, c, budget);
    if (n_max < 0) return n_max;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t q_bytes = static_cast<size_t>(Hq) * w * d * 2;
    const size_t kv_bytes = static_cast<size_t>(Hkv) * L * d * 2;
    const size_t o_bytes = static_cast<size_t>(Hkv) * n_max * d * 2;
    const size_t i_bytes = static_cast<size_t>(Hkv) * n_max * sizeof(int32_t);
    cudaError_t e;
    if ((e = cudaMemcpyAsync(dev_q_obs, host_q_obs, q_bytes, cudaMemcpyHostToDevice, s)) != cudaSuccess ||
        (e = cudaMemcpyAsync(dev_K, host_K, kv_bytes, cudaMemcpyHostToDevice, s)) != cudaSuccess ||
        (e = cudaMemcpyAsync(dev_V, host_V, kv_bytes, cudaMemcpyHostToDevice, s)) != cudaSuccess)
        return cuda_fail(e);
    st = chunkkv_compress_layer(dev_q_obs, dev_K, dev_V, L, Hq, Hkv, d, w, c, budget, nullptr, dev_out_K,
                                dev_out_V, dev_out_idx, stream);
    if (st != CHUNKKV_OK) return st;
    if ((e = cudaMemcpyAsync(host_out_K, dev_out_K, o_bytes, cudaMemcpyDeviceToHost, s)) != cudaSuccess ||
        (e = cudaMemcpyAsync(host_out_V, dev_out_V, o_bytes, cudaMemcpyDeviceToHost, s)) != cudaSuccess ||
        (e = cudaMemcpyAsync(host_out_idx, dev_out_idx, i_bytes, cudaMemcpyDeviceToHost, s)) != cudaSuccess)
        return cuda_fail(e);
    return CHUNKKV_OK;
}

int chunkkv_profile_enable(int on) {
    std::lock_guard<std::mutex> lk(g_mu);
    g_profile = (on != 0);
    return CHUNKKV_OK;
}

int chunkkv_profile_read(float* ms_per_slot, int* launches_per_slot) {
    if (ms_per_slot == nullptr || launches_per_slot == nullptr) return CHUNKKV_EINVAL_NULL;
    std::lock_guard<std::mutex> lk(g_mu);
    DeviceCtx* ctx;
    int st = get_ctx(&ctx);
    if (st != CHUNKKV_OK) return st;
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return cuda_fail(e);
    for (ProfileRec& r : ctx->recs) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, r.start, r.stop) == cudaSuccess) {
            ctx->prof_ms[r.slot] += ms;
            ctx->prof_n[r.slot] += 1;
        }
        cudaEventDestroy(r.start);
        cudaEventDestroy(r.stop);
    }
    ctx->recs.clear();
    for (int i = 0; i < CHUNKKV_PROFILE_SLOTS; ++i) {
        ms_per_slot[i] = ctx->prof_ms[i];
        launches_per_slot[i] = ctx->prof_n[i];
        ctx->prof_ms[i] = 0.f;
        ctx->prof_n[i] = 0;
    }
    return CHUNKKV_OK;
}

}  // extern "C"
