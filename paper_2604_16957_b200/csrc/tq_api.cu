// extern "C" entry points of libtq: argument validation and dispatch.  See include/tq.h.
#include <atomic>
#include <cstdlib>
#include <cstring>

#include <algorithm>

#include "tq_internal.cuh"

namespace tq {

static thread_local int g_last_cuda_error = 0;

int device_sm_count() {
  // one attribute query per device and process; 148 (B200) when no device can be asked
  constexpr int kMaxDevices = 64;
  static std::atomic<int> cached[kMaxDevices];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    (void)cudaGetLastError();
    return 148;
  }
  int n = cached[dev].load(std::memory_order_relaxed);
  if (n > 0) return n;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
    (void)cudaGetLastError();
    return 148;
  }
  cached[dev].store(n, std::memory_order_relaxed);
  return n;
}

TestHooks& test_hooks() {
  static TestHooks h;
  return h;
}

bool pdl_enabled() {
  static const bool on = [] {
    const char* e = std::getenv("TQ_PDL");
    return !(e && e[0] == '0');
  }();
  return on;
}

namespace {
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
}  // namespace

int check_cache(const tq_kv_cache* c) {
  if (!c) return TQ_ERR_NULL;
  if (!c->blocks || !c->seq_lens) return TQ_ERR_NULL;
  if (!(c->d == 64 || c->d == 128 || c->d == 256 || c->d == 512)) return TQ_ERR_SHAPE;
  if (c->B < 1 || c->B > 65535 || c->H_kv < 1 || c->H_kv > 4096 || c->S_cap < 16 || (c->S_cap % 16) != 0)
    return TQ_ERR_SHAPE;
  if (!aligned16(c->blocks) || (reinterpret_cast<uintptr_t>(c->seq_lens) & 3u)) return TQ_ERR_ALIGN;
  if (c->page_table) {
    if (c->page_tokens < 16 || (c->page_tokens & (c->page_tokens - 1)) != 0 || c->max_pages < 1 || c->num_pages < 1 ||
        static_cast<long long>(c->page_tokens) * c->max_pages != c->S_cap ||
        static_cast<long long>(c->num_pages) * c->H_kv * (c->page_tokens / 16) > 0x7fffffffLL)
      return TQ_ERR_SHAPE;
    if (reinterpret_cast<uintptr_t>(c->page_table) & 3u) return TQ_ERR_ALIGN;
  }
  return TQ_OK;
}

int check_heads(const tq_kv_cache* c, int H_q) {
  if (H_q < 1 || (H_q % c->H_kv) != 0 || H_q / c->H_kv > 64) return TQ_ERR_SHAPE;
  return TQ_OK;
}

int check_decode_grid(const tq_kv_cache* c, int H_q, int S_q) {
  const long long tiles = (static_cast<long long>(H_q / c->H_kv) * S_q + 7) / 8;
  return static_cast<long long>(c->H_kv) * tiles > 65535 ? TQ_ERR_SHAPE : TQ_OK;
}

int finish(cudaError_t e) {
  if (e == cudaSuccess) return TQ_OK;
  (void)cudaGetLastError();  // clear the sticky-free launch error so that it is reported once, here
  g_last_cuda_error = static_cast<int>(e);
  return TQ_ERR_CUDA;
}

namespace {

size_t align256(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }

}  // namespace
}  // namespace tq

using namespace tq;

extern "C" {

int tq_kv_quantize_append(const tq_kv_cache* cache, const void* k_new, const void* v_new, int32_t T, int32_t* status,
                          void* stream) {
  if (int r = check_cache(cache)) return r;
  if (!k_new || !v_new) return TQ_ERR_NULL;
  if (T < 1 || T > cache->S_cap) return TQ_ERR_SHAPE;
  if (!aligned16(k_new) || !aligned16(v_new) || (reinterpret_cast<uintptr_t>(status) & 3u)) return TQ_ERR_ALIGN;
  return finish(launch_quantize_append(*cache, static_cast<const __half*>(k_new), static_cast<const __half*>(v_new), T,
                                       status, static_cast<cudaStream_t>(stream)));
}

// waves2: thread-block waves of a batch launch, in halves (8 = four waves)
static int32_t auto_splits(int32_t B, int32_t H_kv, int32_t H_q, int32_t max_seq_len, int waves2) {
  if (B < 1 || H_kv < 1 || H_q < H_kv || max_seq_len < 1) return 1;
  const long long G = H_q / H_kv;
  const long long base = static_cast<long long>(B) * H_kv * ((G + 7) / 8);
  const long long slots = 2LL * device_sm_count();  // two resident thread blocks per SM
  long long C, min_tokens;
  if (4 * base <= slots) {
    // few (sequence, KV head) pairs: one wave of equal splits fills the GPU (37 splits at B = 1, 8 KV heads)
    C = slots / base;
    min_tokens = 512;
  } else {
    // a batch: several waves of blocks, so that sequences of different lengths even out (measured on
    // 16 sequences of 4K..64K tokens: 216 us with one wave of 2 splits, 158 us with 10 splits)
    C = waves2 == 8 ? (waves2 * slots + 2 * base - 1) / (2 * base) : (waves2 * slots) / (2 * base);  // (four waves: rounded up)
    min_tokens = 2048;
  }
  const long long by_len = max_seq_len / min_tokens;  // keep splits from getting too short
  if (C > by_len) C = by_len;
  if (C > TQ_MAX_SPLITS) C = TQ_MAX_SPLITS;
  if (C < 1) C = 1;
  return static_cast<int32_t>(C);
}

int32_t tq_auto_splits(int32_t B, int32_t H_kv, int32_t H_q, int32_t d, int32_t max_seq_len) {
  (void)d;
  return auto_splits(B, H_kv, H_q, max_seq_len, 8);  // separate launches: about four waves for a batch
}

int32_t tq_auto_splits_step(int32_t B, int32_t H_kv, int32_t H_q, int32_t d, int32_t max_seq_len) {
  (void)d;
  // Launches of these entry points overlap their predecessor, which fills the tail of a batch launch: fewer, longer
  // thread blocks do better (16 sequences, 296 slots: ragged 4K..64K 134.0 us with 10 splits, 132.6 with 8; equal
  // 32K 120.0 and 118.7; 6 splits: 134.9 and 114.5).
  const int32_t C = auto_splits(B, H_kv, H_q, max_seq_len, 7);
  if (B < 1 || H_kv < 1 || H_q < H_kv) return C;
  // up to 1K tokens one split does best: its thread block writes the result itself (no partials, no second pass)
  if (max_seq_len <= 1024) return 1;
  const long long base = static_cast<long long>(B) * H_kv * ((H_q / H_kv + 7) / 8);
  const long long slots = 2LL * device_sm_count();
  // One wave that would take every slot: leave an eighth of the slots (at least one per (sequence, KV head)) free,
  // so that the first thread blocks of the next launch are resident, streaming its stable part, while the last
  // ones of this launch finish.  Measured on 8 KV heads and 296 slots (us per step, 128K / 32K): C = 37: 34.7 / -;
  // 36: 30.2 / 11.9; 32: 29.9 / 11.6; 28: 29.9 / 11.8; 24: 30.5 / 11.9.
  if (32 * base <= slots && C > 1) {
    const long long spare = std::max(base, slots / 8);
    const long long cap = std::max(1LL, (slots - spare) / base);
    if (C > cap) return static_cast<int32_t>(cap);
  }
  return C;
}

void tq_split_range(int32_t len, int32_t C, int32_t c, int32_t* t0, int32_t* t1) {
  tq_split_range_window(len, 0, C, c, t0, t1);
}

void tq_split_range_window(int32_t len, int32_t window, int32_t C, int32_t c, int32_t* t0, int32_t* t1) {
  int a = 0, b = 0;
  if (C >= 1 && c >= 0 && c < C) split_range(window_begin(len, window), len, C, c, a, b);
  if (t0) *t0 = a;
  if (t1) *t1 = b;
}

int tq_sdpa_int4_decode(const tq_kv_cache* cache, const void* q, int32_t H_q, float attn_scale, int32_t num_splits,
                        float* o_part, float* m_part, float* l_part, int32_t* status, void* stream) {
  return tq_sdpa_int4_decode_window(cache, q, H_q, attn_scale, 0, num_splits, o_part, m_part, l_part, status, stream);
}

void tq_split_range_stable(int32_t len, int32_t stable_tokens, int32_t C, int32_t c, int32_t* t0, int32_t* t1) {
  int a = 0, b = 0;
  if (C >= 1 && c >= 0 && c < C) {
    if (stable_tokens / kQuantum >= C) split_range_stable(len, stable_tokens, C, c, a, b);
    else split_range(0, len, C, c, a, b);
  }
  if (t0) *t0 = a;
  if (t1) *t1 = b;
}

int tq_sdpa_int4_decode_overlapped(const tq_kv_cache* cache, const void* q, int32_t H_q, float attn_scale,
                                   int32_t num_splits, int32_t stable_tokens, float* o_part, float* m_part,
                                   float* l_part, int32_t* status, void* stream) {
  if (int r = check_cache(cache)) return r;
  if (stable_tokens < 0 || stable_tokens > cache->S_cap) return TQ_ERR_SHAPE;
  if (!q || !o_part || !m_part || !l_part) return TQ_ERR_NULL;
  if (int r = check_heads(cache, H_q)) return r;
  if (num_splits < 0 || num_splits > TQ_MAX_SPLITS) return TQ_ERR_SHAPE;
  if (!aligned16(q) || !aligned16(o_part) || (reinterpret_cast<uintptr_t>(m_part) & 3u) ||
      (reinterpret_cast<uintptr_t>(l_part) & 3u) || (reinterpret_cast<uintptr_t>(status) & 3u))
    return TQ_ERR_ALIGN;
  if (int r = check_decode_grid(cache, H_q, 1)) return r;
  const int C = num_splits ? num_splits : tq_auto_splits_step(cache->B, cache->H_kv, H_q, cache->d, cache->S_cap);
  const bool overlapped = stable_tokens / kQuantum >= C &&
                          test_hooks().decode_impl.load(std::memory_order_relaxed) == 0;
  if (!overlapped)
    return tq_sdpa_int4_decode(cache, q, H_q, attn_scale, C, o_part, m_part, l_part, status, stream);
  return finish(launch_decode_mma(*cache, static_cast<const __half*>(q), H_q, 1, attn_scale, 0, C, o_part, m_part, l_part,
                                  status, static_cast<cudaStream_t>(stream), stable_tokens));
}

size_t tq_step_counter_bytes(int32_t B, int32_t H_kv) {
  if (B < 1 || H_kv < 1) return 0;
  return align256((static_cast<size_t>(B) * H_kv + B) * sizeof(int32_t));
}

size_t tq_step_workspace_bytes(int32_t B, int32_t H_kv, int32_t H_q, int32_t d, int32_t num_splits) {
  if (B < 1 || H_kv < 1 || H_q < 1 || d < 1 || num_splits < 1) return 0;
  return tq_step_counter_bytes(B, H_kv) + tq_partials_bytes(B, H_q, d, num_splits);
}

// Both forms of the fused step: one stable part for the whole batch, or one per sequence (device array).
static int step_common(const tq_kv_cache* cache, const void* k_new, const void* v_new, const void* q, int32_t H_q,
                       float attn_scale, int32_t num_splits, int32_t stable_tokens, const int32_t* stable_lens,
                       void* workspace, size_t workspace_bytes, void* out, int32_t out_is_fp32, int32_t* status,
                       void* stream, int32_t window = 0) {
  if (int r = check_cache(cache)) return r;
  if (!q || !workspace || !out || ((k_new == nullptr) != (v_new == nullptr))) return TQ_ERR_NULL;
  if (int r = check_heads(cache, H_q)) return r;
  if (H_q / cache->H_kv > 8) return TQ_ERR_SHAPE;
  if (window < 0 || (window > 0 && cache->page_table != nullptr)) return TQ_ERR_SHAPE;  // windowed step: contiguous caches
  if (stable_tokens < 0 || stable_tokens > cache->S_cap || num_splits < 0 || num_splits > TQ_MAX_SPLITS) return TQ_ERR_SHAPE;
  if (!aligned16(q) || !aligned16(workspace) || !aligned16(out) || !aligned16(k_new) || !aligned16(v_new) ||
      (reinterpret_cast<uintptr_t>(status) & 3u) || (reinterpret_cast<uintptr_t>(stable_lens) & 3u))
    return TQ_ERR_ALIGN;
  const int span = (window > 0 && window < cache->S_cap) ? window : cache->S_cap;
  const int C = num_splits ? num_splits
                           : (window > 0 ? tq_auto_splits(cache->B, cache->H_kv, H_q, cache->d, span)
                                         : tq_auto_splits_step(cache->B, cache->H_kv, H_q, cache->d, cache->S_cap));
  if (workspace_bytes < tq_step_workspace_bytes(cache->B, cache->H_kv, H_q, cache->d, C)) return TQ_ERR_WORKSPACE;
  char* ws = static_cast<char*>(workspace);
  int32_t* counters = reinterpret_cast<int32_t*>(ws);
  const size_t n = static_cast<size_t>(cache->B) * H_q * C;
  float* o_part = reinterpret_cast<float*>(ws + tq_step_counter_bytes(cache->B, cache->H_kv));
  float* m_part = reinterpret_cast<float*>(reinterpret_cast<char*>(o_part) + align256(n * cache->d * sizeof(float)));
  float* l_part = reinterpret_cast<float*>(reinterpret_cast<char*>(m_part) + align256(n * sizeof(float)));
  int stable = stable_tokens / kQuantum >= C ? stable_tokens : 0;
  if (window > 0 && stable > 0) {
    // windowed step: the early region (see the kernel) must hold at least one block per split, else the general form
    const long long sb = stable / kQuantum, lo = sb * kQuantum + TQ_WINDOW_SLACK - window;
    const long long early0 = lo > 0 ? std::min((lo + kQuantum - 1) / kQuantum, sb) : 0;
    if (sb - early0 < C) stable = 0;
  }
  return finish(launch_decode_step(*cache, static_cast<const __half*>(k_new), static_cast<const __half*>(v_new),
                                   static_cast<const __half*>(q), H_q, 1, attn_scale, window, C, stable, o_part, m_part, l_part,
                                   counters, out, out_is_fp32 != 0, status, static_cast<cudaStream_t>(stream), stable_lens));
}

int tq_sdpa_int4_step(const tq_kv_cache* cache, const void* k_new, const void* v_new, const void* q, int32_t H_q,
                      float attn_scale, int32_t num_splits, int32_t stable_tokens, void* workspace,
                      size_t workspace_bytes, void* out, int32_t out_is_fp32, int32_t* status, void* stream) {
  return step_common(cache, k_new, v_new, q, H_q, attn_scale, num_splits, stable_tokens, nullptr, workspace,
                     workspace_bytes, out, out_is_fp32, status, stream);
}

int tq_sdpa_int4_step_window(const tq_kv_cache* cache, const void* k_new, const void* v_new, const void* q, int32_t H_q,
                             float attn_scale, int32_t window, int32_t num_splits, int32_t stable_tokens, void* workspace,
                             size_t workspace_bytes, void* out, int32_t out_is_fp32, int32_t* status, void* stream) {
  if (window < 1) return TQ_ERR_SHAPE;
  return step_common(cache, k_new, v_new, q, H_q, attn_scale, num_splits, stable_tokens, nullptr, workspace,
                     workspace_bytes, out, out_is_fp32, status, stream, window);
}

int tq_sdpa_int4_step_ragged(const tq_kv_cache* cache, const void* k_new, const void* v_new, const void* q, int32_t H_q,
                             float attn_scale, int32_t num_splits, const int32_t* stable_lens, void* workspace,
                             size_t workspace_bytes, void* out, int32_t out_is_fp32, int32_t* status, void* stream) {
  if (!stable_lens) return TQ_ERR_NULL;
  return step_common(cache, k_new, v_new, q, H_q, attn_scale, num_splits, 0, stable_lens, workspace, workspace_bytes, out,
                     out_is_fp32, status, stream);
}

int tq_sdpa_int4_decode_window(const tq_kv_cache* cache, const void* q, int32_t H_q, float attn_scale, int32_t window,
                               int32_t num_splits, float* o_part, float* m_part, float* l_part, int32_t* status,
                               void* stream) {
  return tq_sdpa_int4_decode_multi(cache, q, H_q, 1, attn_scale, window, num_splits, o_part, m_part, l_part, status,
                                   stream);
}

int tq_sdpa_int4_decode_multi(const tq_kv_cache* cache, const void* q, int32_t H_q, int32_t S_q, float attn_scale,
                              int32_t window, int32_t num_splits, float* o_part, float* m_part, float* l_part,
                              int32_t* status, void* stream) {
  if (int r = check_cache(cache)) return r;
  if (!q || !o_part || !m_part || !l_part) return TQ_ERR_NULL;
  if (int r = check_heads(cache, H_q)) return r;
  if (num_splits < 0 || num_splits > TQ_MAX_SPLITS) return TQ_ERR_SHAPE;
  if (!aligned16(q) || !aligned16(o_part) || (reinterpret_cast<uintptr_t>(m_part) & 3u) ||
      (reinterpret_cast<uintptr_t>(l_part) & 3u) || (reinterpret_cast<uintptr_t>(status) & 3u))
    return TQ_ERR_ALIGN;
  if (window < 0 || S_q < 1 || S_q > TQ_MAX_QUERY_TOKENS) return TQ_ERR_SHAPE;
  if (int r = check_decode_grid(cache, H_q, S_q)) return r;
  const int span = (window > 0 && window < cache->S_cap) ? window : cache->S_cap;  // most tokens a sequence attends
  const int C = num_splits ? num_splits : tq_auto_splits(cache->B, cache->H_kv, H_q * S_q, cache->d, span);
  auto st = static_cast<cudaStream_t>(stream);
  auto qh = static_cast<const __half*>(q);
  if (test_hooks().decode_impl.load(std::memory_order_relaxed) == 1)
    return finish(launch_decode_simple(*cache, qh, H_q, S_q, attn_scale, window, C, o_part, m_part, l_part, status, st));
  return finish(launch_decode_mma(*cache, qh, H_q, S_q, attn_scale, window, C, o_part, m_part, l_part, status, st));
}

int tq_sdpa_int4_combine(const float* o_part, const float* m_part, const float* l_part, int32_t B, int32_t H_q,
                         int32_t d, int32_t num_splits, void* out, int32_t out_is_fp32, void* stream) {
  if (!o_part || !m_part || !l_part || !out) return TQ_ERR_NULL;
  if (B < 1 || H_q < 1 || num_splits < 1 || num_splits > TQ_MAX_SPLITS || d < 32 || d > 512 || (d % 32) != 0 ||
      static_cast<long long>(B) * H_q > 0x7fffffffLL)
    return TQ_ERR_SHAPE;
  if (!aligned16(o_part) || !aligned16(out) || (reinterpret_cast<uintptr_t>(m_part) & 3u) ||
      (reinterpret_cast<uintptr_t>(l_part) & 3u))
    return TQ_ERR_ALIGN;
  return finish(launch_combine(o_part, m_part, l_part, B, H_q, d, num_splits, out, out_is_fp32 != 0,
                               static_cast<cudaStream_t>(stream)));
}

size_t tq_partials_bytes(int32_t B, int32_t H_q, int32_t d, int32_t num_splits) {
  if (B < 1 || H_q < 1 || d < 1 || num_splits < 1) return 0;
  const size_t n = static_cast<size_t>(B) * H_q * num_splits;
  return align256(n * d * sizeof(float)) + 2 * align256(n * sizeof(float));
}

size_t tq_dequant_workspace_bytes(int32_t B, int32_t H_kv, int32_t H_q, int32_t S_cap, int32_t d, int32_t ws_is_fp32) {
  if (B < 1 || H_kv < 1 || H_q < 1 || S_cap < 1 || d < 1) return 0;
  const size_t mat = align256(static_cast<size_t>(B) * H_kv * S_cap * d * (ws_is_fp32 ? 4 : 2));
  const int C = tq_auto_splits(B, H_kv, H_q, d, S_cap);
  return 2 * mat + tq_partials_bytes(B, H_q, d, C);
}

int tq_sdpa_dequant_then_attend(const tq_kv_cache* cache, const void* q, int32_t H_q, float attn_scale, void* workspace,
                                size_t workspace_bytes, int32_t ws_is_fp32, void* out, int32_t out_is_fp32,
                                int32_t* status, void* stream) {
  if (int r = check_cache(cache)) return r;
  if (!q || !workspace || !out) return TQ_ERR_NULL;
  if (int r = check_heads(cache, H_q)) return r;
  if (!aligned16(q) || !aligned16(workspace) || !aligned16(out) || (reinterpret_cast<uintptr_t>(status) & 3u))
    return TQ_ERR_ALIGN;
  if (workspace_bytes < tq_dequant_workspace_bytes(cache->B, cache->H_kv, H_q, cache->S_cap, cache->d, ws_is_fp32))
    return TQ_ERR_WORKSPACE;
  const bool f32 = ws_is_fp32 != 0;
  const int d = cache->d;
  const int C = tq_auto_splits(cache->B, cache->H_kv, H_q, d, cache->S_cap);
  const size_t mat = align256(static_cast<size_t>(cache->B) * cache->H_kv * cache->S_cap * d * (f32 ? 4 : 2));
  const size_t n = static_cast<size_t>(cache->B) * H_q * C;
  char* ws = static_cast<char*>(workspace);
  void* k_mat = ws;
  void* v_mat = ws + mat;
  float* o_part = reinterpret_cast<float*>(ws + 2 * mat);
  float* m_part = reinterpret_cast<float*>(ws + 2 * mat + align256(n * d * sizeof(float)));
  float* l_part = reinterpret_cast<float*>(reinterpret_cast<char*>(m_part) + align256(n * sizeof(float)));
  auto st = static_cast<cudaStream_t>(stream);
  if (int r = finish(launch_dequant(*cache, k_mat, v_mat, f32, st))) return r;
  if (int r = finish(launch_attend_materialized(*cache, k_mat, v_mat, f32, static_cast<const __half*>(q), H_q,
                                                attn_scale, C, o_part, m_part, l_part, status, st)))
    return r;
  return finish(launch_combine(o_part, m_part, l_part, cache->B, H_q, d, C, out, out_is_fp32 != 0, st));
}

int tq_sdpa_mixed_precision_attend(const tq_kv_cache* cache, const void* k_fp16, const void* v_fp16, const void* q,
                                   int32_t H_q, float attn_scale, int32_t num_splits, float* o_part, float* m_part,
                                   float* l_part, int32_t* status, void* stream) {
  if (int r = check_cache(cache)) return r;
  if (!q || !o_part || !m_part || !l_part) return TQ_ERR_NULL;
  if (int r = check_heads(cache, H_q)) return r;
  if (num_splits < 0 || num_splits > TQ_MAX_SPLITS) return TQ_ERR_SHAPE;
  if (!aligned16(q) || !aligned16(o_part) || !aligned16(k_fp16) || !aligned16(v_fp16) ||
      (reinterpret_cast<uintptr_t>(m_part) & 3u) || (reinterpret_cast<uintptr_t>(l_part) & 3u) ||
      (reinterpret_cast<uintptr_t>(status) & 3u))
    return TQ_ERR_ALIGN;
  const int C = num_splits ? num_splits : tq_auto_splits(cache->B, cache->H_kv, H_q, cache->d, cache->S_cap);
  return finish(launch_attend_mixed(*cache, static_cast<const __half*>(k_fp16), static_cast<const __half*>(v_fp16),
                                    static_cast<const __half*>(q), H_q, attn_scale, C, o_part, m_part, l_part, status,
                                    static_cast<cudaStream_t>(stream)));
}

size_t tq_cache_bytes(int32_t B, int32_t H_kv, int32_t S_cap, int32_t d) {
  if (B < 1 || H_kv < 1 || S_cap < 1 || d < 1) return 0;
  return static_cast<size_t>(B) * H_kv * ((static_cast<size_t>(S_cap) + 15) / 16) * TQ_BLOCK_BYTES(d);
}

size_t tq_cache_code_offset(int32_t d, int32_t which, int32_t t, int32_t byte) {
  return static_cast<size_t>(code_offset(d, which, t, byte));
}

size_t tq_cache_meta_offset(int32_t d, int32_t which, int32_t is_zero, int32_t g, int32_t t) {
  return static_cast<size_t>(meta_offset(d, which, is_zero, g, t));
}

const char* tq_result_string(int r) {
  switch (r) {
    case TQ_OK: return "ok";
    case TQ_ERR_NULL: return "null pointer";
    case TQ_ERR_SHAPE: return "unsupported or inconsistent shape";
    case TQ_ERR_ALIGN: return "pointer not 16-byte aligned";
    case TQ_ERR_WORKSPACE: return "workspace too small";
    case TQ_ERR_CUDA: return "CUDA error";
    default: return "unknown";
  }
}

int tq_last_cuda_error(void) { return g_last_cuda_error; }

const char* tq_version(void) {
#if defined(TQ_PROBE_COPIES_ONLY)
  return "libtq 0.2 (sm_100a) TIMING PROBE: copies only, results are meaningless";
#elif defined(TQ_PROBE_MATH_ONLY)
  return "libtq 0.2 (sm_100a) TIMING PROBE: arithmetic only, results are meaningless";
#else
  return "libtq 0.2 (sm_100a)";
#endif
}

// Test hook (tq_internal.cuh); deliberately absent from tq.h.
int tq_internal_test_hook(int key, int value) {
  TestHooks& h = test_hooks();
  switch (key) {
    case 0: h.decode_impl.store(value, std::memory_order_relaxed); return 0;
    case 1: h.spin_limit.store(value, std::memory_order_relaxed); return 0;
    case 2: h.fault_block.store(value, std::memory_order_relaxed); return 0;
    case 3: return static_cast<int>(run_division_check());  // mismatches of the quantiser's division shortcut (-1: CUDA error)
    default: return -1;
  }
}

}  // extern "C"
