// chunkkv_score_noalloc: the scoring step for callers that must not allocate.
//
// Some users of this library cannot call cudaMalloc once they are running: an inference server
// that gave all free HBM to its KV-cache pool at start-up has nothing left for a driver
// allocation, and a latency-critical loop cannot afford the device-wide synchronisation that
// cudaMalloc and cudaFree bring with them. For them the scratch of the scoring kernels lives in
// a fixed array inside this translation unit's device image instead of in an allocated buffer.
//
// Consequences a caller has to know (also stated in chunkkv.h):
//   * every GPU that loads the library carries the array (kScratchBytes) until the process exits;
//   * shapes that need more scratch are refused, nothing is launched;
//   * all calls on a device share the array and it keeps the previous call's contents; the one
//     word that must start at zero (the device status word) is cleared on every call, and calls
//     that overlap on the GPU would race on the rest, so they must be ordered;
//   * the first call on a device resolves the array's device address and should therefore happen
//     outside any stream capture.
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

}  // namespace

extern "C" int chunkkv_score_noalloc(const void* q_obs, const void* K, int L, int Hq, int Hkv, int d, int w,
                                     int c, float* out_chunk_scores, void* stream) {
    if (w < 1 || c < 1 || L < w) return CHUNKKV_EINVAL_SHAPE;
    if (Hkv < 1 || Hkv > 65535 || Hq < Hkv || Hq % Hkv != 0 || (d != 64 && d != 128)) return CHUNKKV_EINVAL_SHAPE;
    if (static_cast<long long>(w) * (Hq / Hkv) > 256) return CHUNKKV_EINVAL_SHAPE;
    if (static_cast<long long>(Hkv) * L * d >= (1LL << 40)) return CHUNKKV_EINVAL_SHAPE;
    if (q_obs == nullptr || K == nullptr || out_chunk_scores == nullptr) return CHUNKKV_EINVAL_NULL;
    if (((reinterpret_cast<uintptr_t>(q_obs) | reinterpret_cast<uintptr_t>(K) |
          reinterpret_cast<uintptr_t>(out_chunk_scores)) & 15u) != 0)
        return CHUNKKV_EINVAL_ALIGN;
    // The documented limit is phrased in terms of the public size query, so callers can test it.
    if (chunkkv_workspace_bytes(L, Hq, Hkv, d, w, c) > kScratchBytes) return CHUNKKV_ETOOLARGE;

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return CHUNKKV_ECUDA;
    void* scratch = nullptr;
    {
        std::lock_guard<std::mutex> lk(g_setup_mu);
        if (g_scratch_addr[dev] == nullptr) {
            // set-up, once per device, with that device current
            void* p = nullptr;
            if (cudaGetSymbolAddress(&p, g_scratch) != cudaSuccess || p == nullptr) return CHUNKKV_ECUDA;
            g_scratch_addr[dev] = p;
        }
        scratch = g_scratch_addr[dev];
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // The array keeps the last call's contents; only the status word has to start at zero.
    if (cudaMemsetAsync(scratch, 0, 256, s) != cudaSuccess) return CHUNKKV_ECUDA;
    return chunkkv::score_with_scratch(q_obs, K, L, Hq, Hkv, d, w, c, out_chunk_scores, scratch, kScratchBytes, s);
}
