// Internal declarations shared by the translation units of libtq (not part of the ABI).
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "tq.h"

namespace tq {

constexpr int kGroup = TQ_GROUP;
constexpr int kQuantum = TQ_SPLIT_QUANTUM;

// Split partition shared by host and device: split c of C over the attended tokens [begin, len) of a
// sequence (begin = 0 without a sliding window, max(0, len - window) with one).  Boundaries fall on
// multiples of 16 tokens except the two ends.
__host__ __device__ inline void split_range(int begin, int len, int C, int c, int& t0, int& t1) {
  if (len < 0) len = 0;
  if (begin < 0) begin = 0;
  if (begin > len) begin = len;
  const long long nb0 = begin / kQuantum, nb1 = (len + kQuantum - 1) / kQuantum;
  const long long n = nb1 - nb0;
  const long long b0 = nb0 + (n * c) / C, b1 = nb0 + (n * (c + 1)) / C;
  long long s = b0 * kQuantum, e = b1 * kQuantum;
  if (s < begin) s = begin;
  if (e > len) e = len;
  if (e < s) e = s;
  t0 = (int)s;
  t1 = (int)e;
}
// Partition of the overlapped decode: the first stable_tokens / 16 blocks are cut into C equal runs of blocks,
// whatever the length; the last split also takes every token from there to len.
__host__ __device__ inline void split_range_stable(int len, int stable_tokens, int C, int c, int& t0, int& t1) {
  const long long sb = stable_tokens > 0 ? stable_tokens / kQuantum : 0;
  t0 = static_cast<int>((sb * c) / C) * kQuantum;
  t1 = static_cast<int>((sb * (c + 1)) / C) * kQuantum;
  if (c == C - 1 && len > t1) t1 = len;
}
__host__ __device__ inline int window_begin(int len, int window) {
  return (window > 0 && window < len) ? len - window : 0;
}

// Several query tokens per sequence (S_q >= 1): query token s is the (S_q - 1 - s)-th newest cached token and
// attends causally the tokens [query_lo, query_hi).
__host__ __device__ inline int query_hi(int len, int S_q, int s) {
  const int hi = len - (S_q - 1 - s);
  return hi > 0 ? hi : 0;
}
__host__ __device__ inline int query_lo(int len, int S_q, int s, int window) {
  return window_begin(query_hi(len, S_q, s), window);
}

// ---- block layout of the cache (see tq.h).  d is 64, 128 or 256.
__host__ __device__ inline int block_bytes(int d) { return 16 * (d + d / 4); }
__host__ __device__ inline int swizzle_term(int d, int t) {
  const int ng = d >> 5;
  return (t >> (ng == 2 ? 2 : (ng == 4 ? 1 : 0))) & (ng - 1);
}
// byte offset inside a block of code byte `byte` of token t (which: 0 = K, 1 = V)
__host__ __device__ inline int code_offset(int d, int which, int t, int byte) {
  const int rowb = d >> 1;
  return which * 16 * rowb + t * rowb + ((((byte >> 4) ^ swizzle_term(d, t))) << 4) + (byte & 15);
}
// byte offset inside a block of the scale (is_zero = 0) or zero (1) of group g, token t
__host__ __device__ inline int meta_offset(int d, int which, int is_zero, int g, int t) {
  const int ng = d >> 5;
  return 16 * d + (2 * which + is_zero) * (ng * 32) + (g * 16 + t) * 2;
}
// Index (in units of blocks) of the block that holds logical 16-token block j of (sequence b, KV head kvh),
// contiguous or paged (see tq.h).  ok = false (paged only) when the page-table entry is outside the pool;
// the index returned then refers to page 0.
__device__ inline long long cache_block_index(const tq_kv_cache& c, int b, int kvh, int j, bool& ok) {
  ok = true;
  if (c.page_table == nullptr) return (static_cast<long long>(b) * c.H_kv + kvh) * (c.S_cap >> 4) + j;
  const int bpp = c.page_tokens >> 4;
  const int i = j / bpp;
  int p = c.page_table[static_cast<long long>(b) * c.max_pages + i];
  if (p < 0 || p >= c.num_pages) {
    ok = false;
    p = 0;
  }
  return (static_cast<long long>(p) * c.H_kv + kvh) * bpp + (j - i * bpp);
}
// The same from bh = b * H_kv + kvh (what the quantiser has at hand); the contiguous case stays three instructions.
__device__ inline uint8_t* cache_block_bh(const tq_kv_cache& c, long long bh, int b, int tok, int32_t* status, bool& ok) {
  if (c.page_table == nullptr) {
    ok = true;
    return c.blocks + (bh * (c.S_cap >> 4) + (tok >> 4)) * block_bytes(c.d);
  }
  const long long idx = cache_block_index(c, b, static_cast<int>(bh - static_cast<long long>(b) * c.H_kv), tok >> 4, ok);
  if (!ok && status) atomicOr(status, TQ_STATUS_BAD_PAGE);
  return c.blocks + idx * block_bytes(c.d);
}
__device__ inline uint8_t* cache_block(const tq_kv_cache& c, int b, int kvh, int tok, int32_t* status, bool& ok) {
  const long long idx = cache_block_index(c, b, kvh, tok >> 4, ok);
  if (!ok && status) atomicOr(status, TQ_STATUS_BAD_PAGE);
  return c.blocks + idx * block_bytes(c.d);
}

// Clamp a device-side sequence length into [0, S_cap], flagging bad or empty values.
__device__ inline int checked_len(const int32_t* seq_lens, int b, int S_cap, int32_t* status) {
  int len = seq_lens[b];
  if (len < 0 || len > S_cap) {
    if (status && threadIdx.x == 0) atomicOr(status, TQ_STATUS_BAD_LEN);
    len = len < 0 ? 0 : S_cap;
  }
  if (len == 0 && status && threadIdx.x == 0) atomicOr(status, TQ_STATUS_EMPTY_SEQ);
  return len;
}

// Programmatic dependent launch.  The three kernels of a decode step (append, phase 1, reduction) are
// launched with the programmatic-stream-serialization attribute, so the launch latency of each one
// overlaps the tail of the kernel before it in the stream.  Every kernel first calls
// pdl_launch_dependents(), which lets the next kernel's blocks be scheduled as soon as there is room for
// them, and then pdl_wait() before its first global access (that wait returns once the preceding kernel
// has completed and its writes are visible, so ordering is exactly stream order; it holds transitively,
// since the preceding kernel itself waited for the one before it).  The one exception is the overlapped
// decode (tq_sdpa_int4_decode_overlapped), which reads what its caller promised to be final before it
// waits.  Both calls are no-ops when the kernel was launched the ordinary way.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory"); }

bool pdl_enabled();  // false when the environment has TQ_PDL=0

template <typename... KArgs, typename... Args>
cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// host-side launchers (each returns the launch error, if any)
long long run_division_check();  // tq_quantize.cu: test support, see division_check_kernel
cudaError_t launch_quantize_append(const tq_kv_cache& c, const __half* k_new, const __half* v_new, int T,
                                   int32_t* status, cudaStream_t st);
cudaError_t launch_decode_mma(const tq_kv_cache& c, const __half* q, int H_q, int S_q, float attn_scale, int window,
                              int C, float* o_part, float* m_part, float* l_part, int32_t* status, cudaStream_t st,
                              int stable_tokens = 0);
cudaError_t launch_decode_step(const tq_kv_cache& c, const __half* k_new, const __half* v_new, const __half* q, int H_q,
                               int S_q, float attn_scale, int window, int C, int stable_tokens, float* o_part,
                               float* m_part, float* l_part, int32_t* counters, void* out, bool out_fp32,
                               int32_t* status, cudaStream_t st, const int32_t* stable_lens = nullptr);
cudaError_t launch_decode_simple(const tq_kv_cache& c, const __half* q, int H_q, int S_q, float attn_scale, int window,
                                 int C, float* o_part, float* m_part, float* l_part, int32_t* status, cudaStream_t st);
cudaError_t launch_combine(const float* o_part, const float* m_part, const float* l_part, int B, int H_q, int d, int C,
                           void* out, bool out_fp32, cudaStream_t st);
cudaError_t launch_dequant(const tq_kv_cache& c, void* k_mat, void* v_mat, bool fp32, cudaStream_t st);
cudaError_t launch_attend_mat_mma(const tq_kv_cache& c, const void* k_mat, const void* v_mat, bool fp32, const __half* q,
                                  int H_q, float attn_scale, int C, float* o_part, float* m_part, float* l_part,
                                  int32_t* status, cudaStream_t st);  // tq_attend_mat.cu; cudaErrorNotSupported: use the scalar kernel
cudaError_t launch_attend_materialized(const tq_kv_cache& c, const void* k_mat, const void* v_mat, bool fp32,
                                       const __half* q, int H_q, float attn_scale, int C, float* o_part, float* m_part,
                                       float* l_part, int32_t* status, cudaStream_t st);
cudaError_t launch_attend_mixed(const tq_kv_cache& c, const __half* k_fp16, const __half* v_fp16, const __half* q, int H_q,
                                float attn_scale, int C, float* o_part, float* m_part, float* l_part, int32_t* status,
                                cudaStream_t st);
// Knobs for the library's own tests, set through tq_internal_test_hook (exported from the shared object for
// the test suite but not declared in tq.h: not part of the ABI).  Read with relaxed loads on the call path.
struct TestHooks {
  std::atomic<int> decode_impl{0};   // key 0: 0 = tensor-core kernel, 1 = the scalar Algorithm-1 kernel of tq_attend_simple.cu
  std::atomic<int> spin_limit{0};    // key 1: > 0 = poll limit of the decode kernel's stage waits (instrumented instantiation)
  std::atomic<int> fault_block{-1};  // key 2: >= 0 = the copy of this 16-token block announces 16 bytes that never arrive
};
TestHooks& test_hooks();
extern "C" int tq_internal_test_hook(int key, int value);

int device_sm_count();  // SM count of the current device (looked up once per device)

// Host-side argument checks shared by every entry point (tq_api.cu).  Each returns a tq_result.
int check_cache(const tq_kv_cache* c);                       // pointers, sizes, alignment, paging fields
int check_heads(const tq_kv_cache* c, int H_q);              // GQA shape
int check_decode_grid(const tq_kv_cache* c, int H_q, int S_q);  // blockIdx.y limit of the decode kernel
int finish(cudaError_t e);                                   // records a CUDA error for tq_last_cuda_error()

}  // namespace tq
