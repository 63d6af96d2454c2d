// chunkkv_score_noalloc: the scoring step for callers that must not allocate.
//
// Some users of this library cannot call cudaMalloc once they are running: an inference server
// that gave all free HBM to its KV-cache pool at start-up has nothing left for a driver
// allocation, and a latency-critical loop cannot afford the device-wide synchronisation that
// cudaMalloc and cudaFree bring with them. For them the scratch of the scoring kernels lives in
// a fixed array inside this translation unit's device image instead of in an allocated buffer.
//
// Consequences a caller has to know (also stated in chunkkv.h):
//   * every GPU that loads this part of the library carries the array (kScratchBytes) until the
//     process exits. The CUDA runtime loads device code lazily: the array takes its memory when
//     this entry point is first called on a device, so that first call belongs at start-up,
//     before the process gives its free memory away, and outside any stream capture;
//   * shapes that need more scratch are refused, nothing is launched;
//   * all calls on a device share the array and it keeps the previous call's contents. Nothing in
//     it has to start at zero except the device status word, which starts at zero when the array
//     is loaded and is only cleared again by chunkkv_score_noalloc_status (so a failure is not
//     lost when another call follows); calls that overlap on the GPU would race on the rest, so
//     they must be ordered.
#include "../../include/chunkkv.h"
#include "internal.h"

#include <mutex>

namespace {

constexpr size_t kScratchBytes = 8u << 20;   // 8 MiB per GPU
constexpr int kMaxDevices = 64;

// In host code this name is only a handle for the symbol, not a device address: the address a
// kernel can use comes from cudaGetSymbolAddress (below), once per device.
static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

std::mutex g_setup_mu;
void* g_scratch_addr[kMaxDevices] = {nullptr};

// Device address of the array on the current device (set-up on first use, with that device current).
int scratch_address(void** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return CHUNKKV_ECUDA;
    std::lock_guard<std::mutex> lk(g_setup_mu);
    if (g_scratch_addr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_scratch) != cudaSuccess || p == nullptr) return CHUNKKV_ECUDA;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return CHUNKKV_OK;
}

}  // namespace

extern "C" int chunkkv_score_noalloc(const void* q_obs, const void* K, int L, int Hq, int Hkv, int d, int w,
                                     int c, float* out_chunk_scores, void* stream) {
    if (w < 1 || c < 1 || L < w) return CHUNKKV_EINVAL_SHAPE;
    int st = chunkkv::check_heads(L, Hq, Hkv, d, w);
    if (st != CHUNKKV_OK) return st;
    if (q_obs == nullptr || K == nullptr || out_chunk_scores == nullptr) return CHUNKKV_EINVAL_NULL;
    if (((reinterpret_cast<uintptr_t>(q_obs) | reinterpret_cast<uintptr_t>(K) |
          reinterpret_cast<uintptr_t>(out_chunk_scores)) & 15u) != 0)
        return CHUNKKV_EINVAL_ALIGN;
    // The documented limit is phrased in terms of the public size query, so callers can test it.
    const size_t need = chunkkv_workspace_bytes(L, Hq, Hkv, d, w, c);
    if (need == 0) return CHUNKKV_EINVAL_SHAPE;
    if (need > kScratchBytes) return CHUNKKV_ETOOLARGE;
    void* scratch = nullptr;
    st = scratch_address(&scratch);
    if (st != CHUNKKV_OK) return st;
    return chunkkv::score_with_scratch(q_obs, K, L, Hq, Hkv, d, w, c, out_chunk_scores, scratch, kScratchBytes,
                                       static_cast<cudaStream_t>(stream));
}

extern "C" int chunkkv_score_noalloc_status(void* stream) {
    void* scratch = nullptr;
    int st = scratch_address(&scratch);
    if (st != CHUNKKV_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaStreamSynchronize(s) != cudaSuccess) return CHUNKKV_ECUDA;
    int flag = 0;
    if (cudaMemcpyAsync(&flag, scratch, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess)
        return CHUNKKV_ECUDA;
    if (flag == 0) return CHUNKKV_OK;
    if (cudaMemsetAsync(scratch, 0, sizeof(int), s) != cudaSuccess || cudaStreamSynchronize(s) != cudaSuccess)
        return CHUNKKV_ECUDA;
    return CHUNKKV_EDEVICE;
}
