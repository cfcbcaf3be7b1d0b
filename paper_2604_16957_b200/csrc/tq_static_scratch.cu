// tq_sdpa_int4_attend_static: fused int4 attention (phase 1 + Eq. 5 reduction) for callers that
// must not allocate device memory.  The split partials, which every other entry point expects in a
// caller-provided buffer, live here in a fixed array inside the library image.
#include <mutex>

#include "tq_internal.cuh"

namespace tq {
namespace {

// The scratch itself.  In host code this name is only a handle for the runtime, not a device
// address: the address is looked up once per device with cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_scratch[TQ_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_ptr[kMaxDevices] = {};

inline size_t align256(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }

size_t partial_bytes(size_t B, size_t H_q, size_t d, size_t C) {
  const size_t n = B * H_q * C;
  return align256(n * d * sizeof(float)) + 2 * align256(n * sizeof(float));
}

// Device address of the scratch array on the current device (set up on first use).
cudaError_t scratch_address(void** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return cudaSuccess;
}

}  // namespace
}  // namespace tq

using namespace tq;

extern "C" int tq_sdpa_int4_attend_static(const tq_kv_cache* cache, const void* q, int32_t H_q, float attn_scale,
                                          void* out, int32_t out_is_fp32, int32_t* status, void* stream) {
  // the host-side checks of tq_sdpa_int4_decode and tq_sdpa_int4_combine (contiguous and paged caches,
  // every head dimension), before anything is launched
  if (int r = check_cache(cache)) return r;
  if (!q || !out) return TQ_ERR_NULL;
  if (int r = check_heads(cache, H_q)) return r;
  if (int r = check_decode_grid(cache, H_q, 1)) return r;
  if (static_cast<long long>(cache->B) * H_q > 0x7fffffffLL) return TQ_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(q) & 15u) || (reinterpret_cast<uintptr_t>(out) & 15u) ||
      (reinterpret_cast<uintptr_t>(status) & 3u))
    return TQ_ERR_ALIGN;
  const int d = cache->d;

  // largest split count, not above the library's usual choice, whose partials fit the fixed scratch
  int C = tq_auto_splits(cache->B, cache->H_kv, H_q, d, cache->S_cap);
  while (C > 1 && partial_bytes(cache->B, H_q, d, C) > TQ_STATIC_SCRATCH_BYTES) --C;
  if (partial_bytes(cache->B, H_q, d, C) > TQ_STATIC_SCRATCH_BYTES) return TQ_ERR_WORKSPACE;  // B * H_q * d too large

  void* base = nullptr;
  if (int r = finish(scratch_address(&base))) return r;
  const size_t n = static_cast<size_t>(cache->B) * H_q * C;
  char* p = static_cast<char*>(base);
  float* o_part = reinterpret_cast<float*>(p);
  float* m_part = reinterpret_cast<float*>(p + align256(n * d * sizeof(float)));
  float* l_part = reinterpret_cast<float*>(reinterpret_cast<char*>(m_part) + align256(n * sizeof(float)));
  auto st = static_cast<cudaStream_t>(stream);
  // Every partial of every (sequence, head, split) is written by phase 1, empty splits included, so
  // nothing in the scratch has to be cleared between calls.
  if (int r = finish(launch_decode_mma(*cache, static_cast<const __half*>(q), H_q, 1, attn_scale, 0, C, o_part, m_part,
                                       l_part, status, st)))
    return r;
  return finish(launch_combine(o_part, m_part, l_part, cache->B, H_q, d, C, out, out_is_fp32 != 0, st));
}
