// Stand-alone K/V row gather and compaction kernel (see gather.cuh). With indices taken from
// another layer this is the whole work of an index-reuse layer (ChunkKV Algorithm 2).
#include "gather.cuh"
#include "internal.h"

namespace chunkkv {

namespace {

constexpr int kGatherThreads = 256;
// A CTA small enough (64 threads x 64 registers) to share an SM with a resident layer-kernel CTA
// (576 threads x 96 registers leave room for 10240 registers).
constexpr int kGatherThreadsSmall = 64;

template <int VPR, int THREADS>
__global__ void __launch_bounds__(THREADS)
gather_kernel(const uint4* __restrict__ K, const uint4* __restrict__ V, const int32_t* __restrict__ idx,
              int L, int n_max, uint4* __restrict__ out_K, uint4* __restrict__ out_V,
              int32_t* __restrict__ idx_copy) {
    // launched as a programmatic dependent of the preceding kernel: let the next kernel's CTAs be
    // scheduled as this one's retire, and touch no global memory before the predecessor is complete
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int h = blockIdx.y;
    const uint4* Kh = K + static_cast<size_t>(h) * L * VPR;
    const uint4* Vh = V + static_cast<size_t>(h) * L * VPR;
    const int32_t* ih = idx + static_cast<size_t>(h) * n_max;
    uint4* oK = out_K + static_cast<size_t>(h) * n_max * VPR;
    uint4* oV = out_V + static_cast<size_t>(h) * n_max * VPR;
    int32_t* ic = idx_copy ? idx_copy + static_cast<size_t>(h) * n_max : nullptr;
    const int rows_per_block = (THREADS / VPR) * kGatherRowsPerThread;
    for (int n0 = blockIdx.x * rows_per_block; n0 < n_max; n0 += gridDim.x * rows_per_block)
        gather_rows<VPR, false>(Kh, Vh, ih, L, n_max, n0, threadIdx.x, THREADS, oK, oV, ic);
}

// The same gather with a paged destination: compacted position n of head h goes to page
// block_table[n / page_size], slot n % page_size of a cache laid out [page, slot, head, d]
// (zero rows where idx is outside [0, L)). Positions whose page number is outside [0, num_pages)
// are skipped, never dereferenced.
template <int VPR>
__global__ void __launch_bounds__(kGatherThreads)
gather_paged_kernel(const uint4* __restrict__ K, const uint4* __restrict__ V, const int32_t* __restrict__ idx,
                    int L, int Hkv, int n_max, const int32_t* __restrict__ block_table, int page_size, int num_pages,
                    uint4* __restrict__ cache_K, uint4* __restrict__ cache_V) {
    const int h = blockIdx.y;
    const uint4* Kh = K + static_cast<size_t>(h) * L * VPR;
    const uint4* Vh = V + static_cast<size_t>(h) * L * VPR;
    const int32_t* ih = idx + static_cast<size_t>(h) * n_max;
    const int rows_per_pass = kGatherThreads / VPR;
    const int vec = threadIdx.x % VPR, sub = threadIdx.x / VPR;
    const unsigned long long policy = gather_policy();
    for (int n0 = blockIdx.x * rows_per_pass * kGatherRowsPerThread; n0 < n_max;
         n0 += gridDim.x * rows_per_pass * kGatherRowsPerThread) {
        int src[kGatherRowsPerThread], page[kGatherRowsPerThread];
        uint4 kv[kGatherRowsPerThread], vv[kGatherRowsPerThread];
#pragma unroll
        for (int u = 0; u < kGatherRowsPerThread; ++u) {
            const int n = n0 + u * rows_per_pass + sub;
            src[u] = (n < n_max) ? ih[n] : -1;
            page[u] = (n < n_max) ? block_table[n / page_size] : -1;
        }
#pragma unroll
        for (int u = 0; u < kGatherRowsPerThread; ++u) {
            const bool ok = static_cast<unsigned>(src[u]) < static_cast<unsigned>(L);
            kv[u] = ok ? gather_ld(Kh + static_cast<size_t>(src[u]) * VPR + vec, policy) : make_uint4(0, 0, 0, 0);
            vv[u] = ok ? gather_ld(Vh + static_cast<size_t>(src[u]) * VPR + vec, policy) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < kGatherRowsPerThread; ++u) {
            const int n = n0 + u * rows_per_pass + sub;
            if (n < n_max && static_cast<unsigned>(page[u]) < static_cast<unsigned>(num_pages)) {
                const size_t row = (static_cast<size_t>(page[u]) * page_size + n % page_size) * Hkv + h;
                gather_st(cache_K + row * VPR + vec, kv[u]);
                gather_st(cache_V + row * VPR + vec, vv[u]);
            }
        }
    }
}

}  // namespace

cudaError_t launch_gather_paged(const void* K, const void* V, const int32_t* idx, int L, int Hkv, int d, int n_max,
                                const int32_t* block_table, int page_size, int num_pages, void* cache_K, void* cache_V,
                                int num_sms, cudaStream_t stream) {
    if (n_max <= 0 || Hkv <= 0) return cudaSuccess;
    const int vpr = d / 8;
    const int rows_per_block = (kGatherThreads / vpr) * kGatherRowsPerThread;
    int bx = (n_max + rows_per_block - 1) / rows_per_block;
    const int cap = (16 * num_sms + Hkv - 1) / Hkv;
    if (bx > cap) bx = cap;
    dim3 grid(bx, Hkv);
    if (vpr == 16)
        gather_paged_kernel<16><<<grid, kGatherThreads, 0, stream>>>(
            static_cast<const uint4*>(K), static_cast<const uint4*>(V), idx, L, Hkv, n_max, block_table, page_size,
            num_pages, static_cast<uint4*>(cache_K), static_cast<uint4*>(cache_V));
    else
        gather_paged_kernel<8><<<grid, kGatherThreads, 0, stream>>>(
            static_cast<const uint4*>(K), static_cast<const uint4*>(V), idx, L, Hkv, n_max, block_table, page_size,
            num_pages, static_cast<uint4*>(cache_K), static_cast<uint4*>(cache_V));
    return cudaGetLastError();
}

// q_obs [Hq, w, d] bf16 from the last w rows of a fused QKV activation [T, row_elems] bf16 (query
// heads first), rotated by the rotary embedding of the rows' positions (rotate-half pairing;
// cos / sin [w, d / 2] f32). The arithmetic is fp64 without contraction and the result is rounded
// to fp32 and then to bf16 (nearest even), so that it equals the fp64 statement of the same
// rotation bit for bit.
namespace {
__global__ void window_queries_kernel(const unsigned short* __restrict__ qkv, long long row_elems, int T, int Hq, int d,
                                      int w, const float* __restrict__ cos_t, const float* __restrict__ sin_t,
                                      unsigned short* __restrict__ q_obs) {
    const int half = d >> 1;
    const int total = Hq * w * half;
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < total; e += gridDim.x * blockDim.x) {
        const int i = e % half, r = (e / half) % w, g = e / (half * w);
        const unsigned short* src = qkv + static_cast<size_t>(T - w + r) * row_elems + static_cast<size_t>(g) * d;
        const double x1 = static_cast<double>(__uint_as_float(static_cast<unsigned>(src[i]) << 16));
        const double x2 = static_cast<double>(__uint_as_float(static_cast<unsigned>(src[i + half]) << 16));
        const double c = static_cast<double>(cos_t[r * half + i]), s = static_cast<double>(sin_t[r * half + i]);
        const double y1 = __dsub_rn(__dmul_rn(x1, c), __dmul_rn(x2, s));
        const double y2 = __dadd_rn(__dmul_rn(x2, c), __dmul_rn(x1, s));
        auto to_bf16 = [](double y) {
            const unsigned u = __float_as_uint(__double2float_rn(y));
            return static_cast<unsigned short>((u + 0x7FFFu + ((u >> 16) & 1u)) >> 16);
        };
        unsigned short* dst = q_obs + (static_cast<size_t>(g) * w + r) * d;
        dst[i] = to_bf16(y1);
        dst[i + half] = to_bf16(y2);
    }
}
}  // namespace

cudaError_t launch_window_queries(const void* qkv, long long row_elems, int T, int Hq, int d, int w, const float* cos_t,
                                  const float* sin_t, void* q_obs, cudaStream_t stream) {
    const int total = Hq * w * (d / 2);
    if (total <= 0) return cudaSuccess;
    window_queries_kernel<<<(total + 255) / 256, 256, 0, stream>>>(static_cast<const unsigned short*>(qkv), row_elems, T,
                                                                 Hq, d, w, cos_t, sin_t,
                                                                 static_cast<unsigned short*>(q_obs));
    return cudaGetLastError();
}

// The same gather from keys and values that are not packed [Hkv, L, d]: source rows are found by a token
// stride and a head stride (in 16-byte vectors); the outputs are packed.
template <int VPR>
__global__ void __launch_bounds__(kGatherThreads)
gather_strided_kernel(const uint4* __restrict__ K, const uint4* __restrict__ V, const int32_t* __restrict__ idx,
                      int L, int n_max, long long k_tok, long long k_head, long long v_tok, long long v_head,
                      uint4* __restrict__ out_K, uint4* __restrict__ out_V, int32_t* __restrict__ idx_copy) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int h = blockIdx.y;
    const uint4* Kh = K + static_cast<size_t>(h) * k_head;
    const uint4* Vh = V + static_cast<size_t>(h) * v_head;
    const int32_t* ih = idx + static_cast<size_t>(h) * n_max;
    uint4* oK = out_K + static_cast<size_t>(h) * n_max * VPR;
    uint4* oV = out_V + static_cast<size_t>(h) * n_max * VPR;
    int32_t* ic = idx_copy ? idx_copy + static_cast<size_t>(h) * n_max : nullptr;
    const int rows_per_block = (kGatherThreads / VPR) * kGatherRowsPerThread;
    for (int n0 = blockIdx.x * rows_per_block; n0 < n_max; n0 += gridDim.x * rows_per_block)
        gather_rows<VPR, false>(Kh, Vh, ih, L, n_max, n0, threadIdx.x, kGatherThreads, oK, oV, ic, k_tok, v_tok);
}

template <int THREADS>
static cudaError_t launch_gather_t(const void* K, const void* V, const int32_t* idx, int L, int Hkv, int d, int n_max,
                                   void* out_K, void* out_V, int32_t* idx_copy_or_null, int max_blocks,
                                   cudaStream_t stream) {
    const int vpr = d / 8;
    const int rows_per_block = (THREADS / vpr) * kGatherRowsPerThread;
    int bx = (n_max + rows_per_block - 1) / rows_per_block;
    const int cap = (max_blocks + Hkv - 1) / Hkv;
    if (bx > cap) bx = cap;
    if (bx < 1) bx = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(bx, Hkv);
    cfg.blockDim = dim3(THREADS);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const uint4* Kp = static_cast<const uint4*>(K);
    const uint4* Vp = static_cast<const uint4*>(V);
    uint4* oK = static_cast<uint4*>(out_K);
    uint4* oV = static_cast<uint4*>(out_V);
    if (vpr == 16) return cudaLaunchKernelEx(&cfg, gather_kernel<16, THREADS>, Kp, Vp, idx, L, n_max, oK, oV, idx_copy_or_null);
    return cudaLaunchKernelEx(&cfg, gather_kernel<8, THREADS>, Kp, Vp, idx, L, n_max, oK, oV, idx_copy_or_null);
}

cudaError_t launch_gather(const void* K, const void* V, const int32_t* idx, int L, int Hkv, int d,
                          int n_max, void* out_K, void* out_V, int32_t* idx_copy_or_null,
                          int num_sms, cudaStream_t stream) {
    if (n_max <= 0 || Hkv <= 0) return cudaSuccess;
    return launch_gather_t<kGatherThreads>(K, V, idx, L, Hkv, d, n_max, out_K, out_V, idx_copy_or_null, 16 * num_sms,
                                           stream);
}

cudaError_t launch_gather_strided(const void* K, const void* V, const int32_t* idx, int L, int Hkv, int d, int n_max,
                                  long long k_token_stride, long long k_head_stride, long long v_token_stride,
                                  long long v_head_stride, void* out_K, void* out_V, int32_t* idx_copy_or_null,
                                  int num_sms, cudaStream_t stream) {
    if (n_max <= 0 || Hkv <= 0) return cudaSuccess;
    const int vpr = d / 8;
    const int rows_per_block = (kGatherThreads / vpr) * kGatherRowsPerThread;
    int bx = (n_max + rows_per_block - 1) / rows_per_block;
    const int cap = (16 * num_sms + Hkv - 1) / Hkv;
    if (bx > cap) bx = cap;
    if (bx < 1) bx = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(bx, Hkv);
    cfg.blockDim = dim3(kGatherThreads);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const uint4* Kp = static_cast<const uint4*>(K);
    const uint4* Vp = static_cast<const uint4*>(V);
    uint4* oK = static_cast<uint4*>(out_K);
    uint4* oV = static_cast<uint4*>(out_V);
    // strides in 16-byte vectors (8 bf16 elements)
    const long long kt = k_token_stride / 8, kh = k_head_stride / 8, vt = v_token_stride / 8, vh = v_head_stride / 8;
    if (vpr == 16)
        return cudaLaunchKernelEx(&cfg, gather_strided_kernel<16>, Kp, Vp, idx, L, n_max, kt, kh, vt, vh, oK, oV, idx_copy_or_null);
    return cudaLaunchKernelEx(&cfg, gather_strided_kernel<8>, Kp, Vp, idx, L, n_max, kt, kh, vt, vh, oK, oV, idx_copy_or_null);
}

// The same gather in CTAs of 64 threads spread over the whole GPU: such a CTA fits on an SM
// beside a resident CTA of the layer kernel, so the row traffic of one lane's layer can use every
// SM's load/store path while the other lanes keep scoring.
cudaError_t launch_gather_shared_sms(const void* K, const void* V, const int32_t* idx, int L, int Hkv, int d,
                                     int n_max, void* out_K, void* out_V, int num_sms, cudaStream_t stream) {
    if (n_max <= 0 || Hkv <= 0) return cudaSuccess;
    return launch_gather_t<kGatherThreadsSmall>(K, V, idx, L, Hkv, d, n_max, out_K, out_V, nullptr, 4 * num_sms, stream);
}

}  // namespace chunkkv
