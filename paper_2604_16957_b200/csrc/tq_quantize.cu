// int4 quantise-and-append of new K/V tokens (Sec. 2.1, Eq. 2-3), written in place into a
// pre-allocated cache.
//
// Mapping: one thread owns 8 consecutive elements (one 16-byte load, one packed 32-bit store);
// the 4 threads of a lane quad own one quantisation group of 32, so min/max need two shuffles.
// A warp covers 256 consecutive elements.  Destinations follow the block layout of the cache
// (swizzled code chunks, scales and zeros per group of 16 tokens), see tq.h.
//
// All arithmetic is IEEE binary32 with explicit round-to-nearest intrinsics so that the result
// is bit-identical on any machine that follows the same operation order:
//   s = fp16((max - min) / 15);  z = fp16((0 - min) / s);  q = clamp(rint(x / s + z), 0, 15).
#include "tq_internal.cuh"

namespace tq {
namespace {


// Redo the flagged elements with the defining arithmetic (true division).  Kept out of line so that the
// common path carries no division code.
__device__ __noinline__ uint32_t exact_codes(const float (&x)[8], float sf, float zf, uint32_t word, uint32_t unsure) {
  for (int i = 0; i < 8; ++i) {
    if (unsure & (1u << i)) {
      const float u = fminf(fmaxf(__fadd_rn(__fdiv_rn(x[i], sf), zf), 0.0f), 15.0f);
      const uint32_t q = __float_as_uint(u + 12582912.0f) & 0xFu;
      word = (word & ~(0xFu << (4 * i))) | (q << (4 * i));
    }
  }
  return word;
}

// Quantise the 8 elements held by this thread (quad = one group).  All 32 lanes must call.
__device__ __forceinline__ void quantize_chunk(const uint4 raw, bool active, uint32_t& word, __half& s_out,
                                               __half& z_out) {
  const __half2* h2 = reinterpret_cast<const __half2*>(&raw);
  float x[8];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float2 f = __half22float2(h2[i]);
    x[2 * i] = f.x;
    x[2 * i + 1] = f.y;
  }
  float mn = x[0], mx = x[0];
#pragma unroll
  for (int i = 1; i < 8; ++i) {
    mn = fminf(mn, x[i]);
    mx = fmaxf(mx, x[i]);
  }
#pragma unroll
  for (int off = 1; off <= 2; off <<= 1) {
    mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, off));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
  }
  (void)active;
  const float range = __fsub_rn(mx, mn);
  const float s32 = __fdiv_rn(range, 15.0f);
  __half s16 = __float2half_rn(s32);
  word = 0u;
  if ((__half_as_ushort(s16) & 0x7FFFu) == 0) {  // scale rounds to zero: constant (or nearly constant) group
    s_out = __ushort_as_half(0x3C00u);            // 1.0
    z_out = __float2half_rn(__fsub_rn(0.0f, mn));
    return;
  }
  const float sf = __half2float(s16);
  float z32 = __fdiv_rn(__fsub_rn(0.0f, mn), sf);
  z32 = fminf(fmaxf(z32, -65504.0f), 65504.0f);
  const __half z16 = __float2half_rn(z32);
  const float zf = __half2float(z16);
  // Codes.  The defining arithmetic is u = fl(fl(x / s) + z) with a true division, q = clamp(rint(u), 0, 15)
  // = rint(clamp(u, 0, 15)) (rint is monotone).  A true division, a round and a float-to-int conversion per
  // element make this kernel bound by the special-function pipe, so the common case avoids all three:
  //   ua = fl(x * (1/s) + z) with the correctly rounded reciprocal differs from u by at most
  //        (|x/s| + |u|) * 2^-23 <= tol (a per-group bound, with a 4x margin);
  //   y = clamp(ua) + 1.5 * 2^23 rounds to nearest-even in the addition and leaves the code in the low
  //        mantissa bits.
  // Only when clamp(ua) lies within tol of a rounding boundary k + 1/2 could the two disagree, and exactly
  // those elements are redone with the division.  The result is bit-identical to the defining arithmetic.
  const float rs = __frcp_rn(sf);
  const float tol = (2.0f * fmaxf(fabsf(mn), fabsf(mx)) * rs + fabsf(zf) + 17.0f) * 4.76837158203125e-7f;  // 2^-21
  constexpr float kMagic = 12582912.0f;  // 1.5 * 2^23
  uint32_t unsure = 0;  // elements whose fast result sits within tol of a rounding boundary
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float u = fminf(fmaxf(fmaf(x[i], rs, zf), 0.0f), 15.0f);  // fmaxf also turns NaN into 0
    const float y = u + kMagic;
    if (fabsf(fabsf(u - (y - kMagic)) - 0.5f) <= tol) unsure |= 1u << i;
    word |= (__float_as_uint(y) & 0xFu) << (4 * i);
  }
  if (unsure) word = exact_codes(x, sf, zf, word, unsure);  // rare
  s_out = s16;
  z_out = z16;
}

// chunk index -> (b, h, t, c) of a [B][H_kv][T][d] tensor and the destination row in the cache
__device__ __forceinline__ void process_chunk(const tq_kv_cache& c, const __half* src, int which, int T,
                                              long long chunk, bool in_range, int b, int len, int32_t* status) {
  const int d = c.d;
  const int cpr = d >> 3;  // chunks per row
  uint4 raw = make_uint4(0, 0, 0, 0);
  long long row_in = 0;
  int cc = 0;
  if (in_range) {
    row_in = chunk / cpr;  // (b * H_kv + h) * T + t
    cc = static_cast<int>(chunk - row_in * cpr);
    raw = *reinterpret_cast<const uint4*>(src + row_in * d + cc * 8);
  }
  uint32_t word;
  __half s, z;
  quantize_chunk(raw, in_range, word, s, z);
  if (in_range) {
    const long long bh = row_in / T;
    const int t = static_cast<int>(row_in - bh * T);
    const int tok = len + t;
    bool ok;
    uint8_t* blk = cache_block_bh(c, bh, b, tok, status, ok);
    if (!ok) return;  // a page outside the pool: nothing is written
    *reinterpret_cast<uint32_t*>(blk + code_offset(d, which, tok & 15, cc * 4)) = word;
    if ((cc & 3) == 0) {
      *reinterpret_cast<__half*>(blk + meta_offset(d, which, 0, cc >> 2, tok & 15)) = s;
      *reinterpret_cast<__half*>(blk + meta_offset(d, which, 1, cc >> 2, tok & 15)) = z;
    }
  }
}

// Bulk variant: one thread block per destination cache block (16 tokens of one KV head, K or V), so the
// codes leave as one contiguous kilobyte and the block's scales and zeros, gathered in shared memory,
// as 16-byte vectors (written one by one they were four times as many memory transactions as the codes).
// grid: (blocks touched per sequence, B * H_kv, {K, V}); 2 * d threads (one per 8 elements).
// seq_lens is read only here and bumped by bump_lens_kernel afterwards, so that no block can observe a
// length that another block of the same launch has already advanced.
// THREADS = the largest block this instantiation is launched with (1024 only for d = 512, so that the
// common head dimensions keep the register budget of a 512-thread block).
template <int THREADS>
__global__ void __launch_bounds__(THREADS) quantize_bulk_kernel(tq_kv_cache c, const __half* k_new, const __half* v_new,
                                                                int T, int32_t* status) {
  __shared__ __align__(16) __half sm_meta[2][16][16];  // [scale | zero][group][token], up to d = 512
  pdl_wait();
  pdl_launch_dependents();
  const int d = c.d, cpr = d >> 3, ng = d >> 5;
  const long long bh = blockIdx.y;
  const int b = static_cast<int>(bh / c.H_kv);
  const int len = c.seq_lens[b];
  if (len < 0 || len + T > c.S_cap) return;  // flagged by bump_lens_kernel
  const int which = blockIdx.z;
  const int j = (len >> 4) + blockIdx.x;                       // destination block
  const int tok_lo = max(16 * j, len), tok_hi = min(16 * j + 16, len + T);
  if (tok_lo >= tok_hi) return;
  const int t = threadIdx.x / cpr, cc = threadIdx.x - t * cpr;  // token in the block, 8-element chunk in the row
  const int tok = 16 * j + t;
  const bool active = tok >= tok_lo && tok < tok_hi;
  uint4 raw = make_uint4(0, 0, 0, 0);
  if (active) raw = *reinterpret_cast<const uint4*>((which ? v_new : k_new) + (bh * T + (tok - len)) * d + cc * 8);
  uint32_t word;
  __half s, z;
  quantize_chunk(raw, active, word, s, z);
  bool page_ok;
  uint8_t* blk = cache_block_bh(c, bh, b, 16 * j, threadIdx.x == 0 ? status : nullptr, page_ok);
  if (!page_ok) return;  // a page outside the pool: nothing is written (uniform over the block)
  if (active) *reinterpret_cast<uint32_t*>(blk + code_offset(d, which, t, cc * 4)) = word;
  const bool whole = tok_lo == 16 * j && tok_hi == 16 * j + 16;
  if ((cc & 3) == 0) {
    if (whole) {
      sm_meta[0][cc >> 2][t] = s;
      sm_meta[1][cc >> 2][t] = z;
    } else if (active) {  // a block only partly covered by this append: write the few values directly
      *reinterpret_cast<__half*>(blk + meta_offset(d, which, 0, cc >> 2, t)) = s;
      *reinterpret_cast<__half*>(blk + meta_offset(d, which, 1, cc >> 2, t)) = z;
    }
  }
  if (!whole) return;  // uniform over the block
  __syncthreads();
  // scales [ng][16] then zeros [ng][16] are adjacent in the cache block: 2 * ng * 32 bytes
  const int vecs = ng * 2;  // 16-byte vectors per array
  if (threadIdx.x < 2 * vecs) {
    const int arr = threadIdx.x / vecs, v = threadIdx.x - arr * vecs;
    const uint4 val = reinterpret_cast<const uint4*>(&sm_meta[arr][0][0])[v];
    reinterpret_cast<uint4*>(blk + meta_offset(d, which, arr, 0, 0))[v] = val;
  }
}

__global__ void bump_lens_kernel(tq_kv_cache c, int T, int32_t* status) {
  pdl_wait();
  pdl_launch_dependents();
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= c.B) return;
  const int len = c.seq_lens[b];
  if (len < 0 || len + T > c.S_cap) {
    if (status) atomicOr(status, TQ_STATUS_CACHE_FULL);
    return;
  }
  c.seq_lens[b] = len + T;
}

// Decode-step variant (small T): one block per sequence quantises K and V of all its KV heads,
// then advances the length itself -- a single launch, and no block reads another's length.
__global__ void __launch_bounds__(256) quantize_step_kernel(tq_kv_cache c, const __half* k_new, const __half* v_new,
                                                            int T, int32_t* status) {
  pdl_wait();
  pdl_launch_dependents();
  const int b = blockIdx.x;
  const int len = c.seq_lens[b];
  if (len < 0 || len + T > c.S_cap) {
    if (status && threadIdx.x == 0) atomicOr(status, TQ_STATUS_CACHE_FULL);
    return;
  }
  const long long per_seq = static_cast<long long>(c.H_kv) * T * (c.d >> 3);
  for (long long base = 0; base < 2 * per_seq; base += blockDim.x) {  // per_seq is a multiple of 4: quads stay whole
    const long long i = base + threadIdx.x;
    const bool is_v = i >= per_seq;
    const long long local = is_v ? i - per_seq : i;
    const bool in_range = i < 2 * per_seq;
    process_chunk(c, is_v ? v_new : k_new, is_v ? 1 : 0, T, static_cast<long long>(b) * per_seq + local, in_range, b, len,
                  status);
  }
  __syncthreads();
  if (threadIdx.x == 0) c.seq_lens[b] = len + T;
}

}  // namespace

cudaError_t launch_quantize_append(const tq_kv_cache& c, const __half* k_new, const __half* v_new, int T,
                                   int32_t* status, cudaStream_t st) {
  const long long per_seq = static_cast<long long>(c.H_kv) * T * (c.d >> 3);
  if (2 * per_seq <= 8192) {
    return launch_kernel(quantize_step_kernel, dim3(c.B), dim3(256), 0, st, c, k_new, v_new, T, status);
  } else {
    dim3 grid(static_cast<unsigned>((T + 15) / 16 + 1), static_cast<unsigned>(c.B * c.H_kv), 2);
    const cudaError_t e =
        c.d > 256 ? launch_kernel(quantize_bulk_kernel<1024>, grid, dim3(2 * c.d), 0, st, c, k_new, v_new, T, status)
                  : launch_kernel(quantize_bulk_kernel<512>, grid, dim3(2 * c.d), 0, st, c, k_new, v_new, T, status);
    if (e != cudaSuccess) return e;
    return launch_kernel(bump_lens_kernel, dim3((c.B + 127) / 128), dim3(128), 0, st, c, T, status);
  }
}

}  // namespace tq
