// Scalar split attention kernels and the dequantise-to-matrix kernel.
//
//  * attend_simple_kernel<D, Src>: Algorithm 1 run per split on CUDA cores, one warp per token
//    stream, one lane per D/32 consecutive channels, warp-shuffle dot products, fp32 online
//    softmax.  Src selects where a K/V row comes from:
//      SrcInt4  -- the packed cache, dequantised in registers (a plain reference variant of the
//                  fused kernel, selected by the test hook of tq_internal.cuh; the tensor-core kernel in
//                  tq_decode_mma.cu is the production path)
//      SrcF32 / SrcF16 -- a materialised [B][H_kv][S_cap][D] matrix: the attention half of the
//                  dequantize-then-attend comparison path (Sec. 3.1 first paragraph, Table 2).
//  * dequant_kernel: the other half of that comparison path, x^ = (q - z) * s for every valid
//    row (Eq. 3), written to the materialised matrix.
#include "tq_internal.cuh"

namespace tq {
namespace {

constexpr int kWarps = 4;
// (query token, head) pairs per thread block: 8, or 4 at d = 512 where a pair's registers double
template <int D>
struct HeadTile {
  static constexpr int value = D > 256 ? 4 : 8;
};
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

template <int D>
struct SrcInt4 {
  static constexpr int EPL = D / 32;  // elements per lane
  tq_kv_cache c;
  // row = (b * H_kv + kvh) * S_cap + token
  __device__ void load(bool is_v, long long row, int lane, float (&x)[EPL]) const {
    const long long bh = row / c.S_cap;
    const int tok = static_cast<int>(row - bh * c.S_cap);
    const int b = static_cast<int>(bh / c.H_kv);
    bool ok;
    const uint8_t* blk = cache_block(c, b, static_cast<int>(bh - static_cast<long long>(b) * c.H_kv), tok, nullptr, ok);
    const int g = (lane * EPL) / 32;
    const float s = __half2float(*reinterpret_cast<const __half*>(blk + meta_offset(D, is_v, 0, g, tok & 15)));
    const float z = __half2float(*reinterpret_cast<const __half*>(blk + meta_offset(D, is_v, 1, g, tok & 15)));
#pragma unroll
    for (int i = 0; i < EPL / 2; ++i) {
      const uint32_t byte = blk[code_offset(D, is_v, tok & 15, lane * (EPL / 2) + i)];
      x[2 * i] = (static_cast<float>(byte & 0xF) - z) * s;
      x[2 * i + 1] = (static_cast<float>(byte >> 4) - z) * s;
    }
  }
};

template <int D, typename T>
struct SrcMat {
  static constexpr int EPL = D / 32;
  const T *k, *v;
  __device__ void load(bool is_v, long long row, int lane, float (&x)[EPL]) const {
    const T* p = (is_v ? v : k) + row * D + lane * EPL;
#pragma unroll
    for (int i = 0; i < EPL; ++i) {
      if constexpr (sizeof(T) == 4) x[i] = p[i];
      else x[i] = __half2float(p[i]);
    }
  }
};

// K and V from different places: each either the int4 cache or an unquantised fp16 matrix
// [B][H_kv][S_cap][D].  This is the K-versus-V precision ablation of Sec. 5 (int4 K with full-precision
// V against full-precision K with int4 V).
template <int D>
struct SrcMixed {
  static constexpr int EPL = D / 32;
  SrcInt4<D> cache;
  SrcMat<D, __half> mat;  // a null k or v means "take that side from the cache"
  __device__ void load(bool is_v, long long row, int lane, float (&x)[EPL]) const {
    if ((is_v ? mat.v : mat.k) != nullptr) mat.load(is_v, row, lane, x);
    else cache.load(is_v, row, lane, x);
  }
};

// grid: (C, H_kv * head_tiles, B); block: kWarps warps.
// GEN = sliding window and / or several query tokens: per-pair token ranges are checked inside the token loop.
template <int D, typename Src, bool GEN>
__global__ void __launch_bounds__(kWarps * 32) attend_simple_kernel(Src src, const int32_t* seq_lens, int H_kv,
                                                                    int S_cap, const __half* q, int H_q, int S_q,
                                                                    float attn_scale, int window, int C, float* o_part,
                                                                    float* m_part, float* l_part, int32_t* status) {
  constexpr int EPL = D / 32;
  constexpr int kHeadTile = HeadTile<D>::value;
  const int G = H_q / H_kv;
  const int GV = G * S_q;  // (query token, head) pairs of one KV head: v = s * G + g
  const int tiles = (GV + kHeadTile - 1) / kHeadTile;
  const int c = blockIdx.x, kvh = blockIdx.y / tiles, tile = blockIdx.y % tiles, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  pdl_launch_dependents();
  pdl_wait();
  const int len = checked_len(seq_lens, b, S_cap, (c == 0 && blockIdx.y == 0) ? status : nullptr);
  int t0, t1;
  split_range(query_lo(len, S_q, 0, window), len, C, c, t0, t1);
  const int v0 = tile * kHeadTile;
  const int nh = min(kHeadTile, GV - v0);
  auto q_row = [&](int v) -> long long {  // row of pair v in q and in the partial arrays, [B][S_q][H_q]
    const int s = v / G;
    return (static_cast<long long>(b) * S_q + s) * H_q + kvh * G + (v - s * G);
  };

  float qr[kHeadTile][EPL], o[kHeadTile][EPL], m[kHeadTile], l[kHeadTile];
  int lo[kHeadTile], hi[kHeadTile];  // tokens each pair attends (causal among the S_q query tokens)
#pragma unroll
  for (int h = 0; h < kHeadTile; ++h) {
    m[h] = -INFINITY;
    l[h] = 0.f;
    const int s = min((v0 + h) / G, S_q - 1);
    hi[h] = query_hi(len, S_q, s);
    lo[h] = window_begin(hi[h], window);
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      o[h][e] = 0.f;
      qr[h][e] = h < nh ? __half2float(q[q_row(v0 + h) * D + lane * EPL + e]) : 0.f;
    }
  }
  const long long row0 = (static_cast<long long>(b) * H_kv + kvh) * S_cap;
  const float sc = attn_scale * kLog2e;
  for (int i = t0 + warp; i < t1; i += kWarps) {
    float kx[EPL], vx[EPL];
    src.load(false, row0 + i, lane, kx);
    src.load(true, row0 + i, lane, vx);
#pragma unroll
    for (int h = 0; h < kHeadTile; ++h) {
      if (GEN && (i < lo[h] || i >= hi[h])) continue;
      float dot = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) dot = fmaf(qr[h][e], kx[e], dot);
#pragma unroll
      for (int off = 16; off; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
      const float a = dot * sc;  // log2 units
      const float mn = fmaxf(m[h], a);
      const float corr = exp2f(m[h] - mn);  // exp2(-inf) = 0 on the first token
      const float p = exp2f(a - mn);
      l[h] = l[h] * corr + p;
#pragma unroll
      for (int e = 0; e < EPL; ++e) o[h][e] = o[h][e] * corr + p * vx[e];
      m[h] = mn;
    }
  }
  // merge the warps' (m, l, o) through shared memory, then write the normalised partial
  __shared__ float sm_m[kWarps][kHeadTile], sm_l[kWarps][kHeadTile];
  __shared__ float sm_o[kWarps][kHeadTile][D];
#pragma unroll
  for (int h = 0; h < kHeadTile; ++h) {
    if (lane == 0) {
      sm_m[warp][h] = m[h];
      sm_l[warp][h] = l[h];
    }
#pragma unroll
    for (int e = 0; e < EPL; ++e) sm_o[warp][h][lane * EPL + e] = o[h][e];
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < nh * D; idx += blockDim.x) {
    const int h = idx / D, x = idx % D;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) M = fmaxf(M, sm_m[w][h]);
    float num = 0.f, den = 0.f;
    if (M > -INFINITY) {
#pragma unroll
      for (int w = 0; w < kWarps; ++w) {
        const float f = exp2f(sm_m[w][h] - M);
        num += f * sm_o[w][h][x];
        den += f * sm_l[w][h];
      }
    }
    const long long pidx = q_row(v0 + h) * C + c;
    o_part[pidx * D + x] = den > 0.f ? num / den : 0.f;
    if (x == 0) {
      m_part[pidx] = M * kLn2;  // back to natural-log units of attn_scale * q.k
      l_part[pidx] = den;
    }
  }
}

template <int D, typename Src>
cudaError_t launch_simple(const Src& src, const tq_kv_cache& c, const __half* q, int H_q, int S_q, float attn_scale,
                          int window, int C, float* o_part, float* m_part, float* l_part, int32_t* status,
                          cudaStream_t st) {
  constexpr int kHeadTile = HeadTile<D>::value;
  const int GV = (H_q / c.H_kv) * S_q;
  const int tiles = (GV + kHeadTile - 1) / kHeadTile;
  dim3 grid(C, c.H_kv * tiles, c.B);
  if (S_q > 1 || window > 0)
    attend_simple_kernel<D, Src, true><<<grid, kWarps * 32, 0, st>>>(src, c.seq_lens, c.H_kv, c.S_cap, q, H_q, S_q,
                                                                     attn_scale, window, C, o_part, m_part, l_part, status);
  else
    attend_simple_kernel<D, Src, false><<<grid, kWarps * 32, 0, st>>>(src, c.seq_lens, c.H_kv, c.S_cap, q, H_q, 1,
                                                                      attn_scale, 0, C, o_part, m_part, l_part, status);
  return cudaGetLastError();
}

// x^ = (q - z) * s for every valid row, in binary32 (fsub then fmul, each rounded to nearest).  One thread per
// quantisation group: a 16-byte load of 32 codes, the group's scale and zero, 128 (fp32) or 64 (fp16) bytes
// stored.  The codes become floats without an integer conversion: (w & 0x000F000F) | 0x64006400 is the half2
// (1024 + n_0, 1024 + n_4), and 1024 + 16 n for the nibbles one position up; fma(f, 1, -1024) and
// fma(f, 1/16, -64) are exactly n.  A warp's 32 groups are one contiguous run of the output (4 KB of fp32):
// the lanes park their pieces in shared memory and the warp stores them as contiguous 512-byte rows.
// grid = (groups of a head's rows, sequence, 2 * H_kv: K then V per head).
template <typename T>
__global__ void __launch_bounds__(256) dequant_kernel(tq_kv_cache c, T* k_mat, T* v_mat) {
  pdl_launch_dependents();
  pdl_wait();
  const int d = c.d, ng = d >> 5, sh = 31 - __clz(ng);  // groups per row (a power of two)
  const int b = blockIdx.y;
  int len = c.seq_lens[b];
  len = len < 0 ? 0 : (len > c.S_cap ? c.S_cap : len);
  const bool is_v = (blockIdx.z & 1) != 0;
  const int h = blockIdx.z >> 1;
  const long long idx = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  constexpr int kPiece = 32 * sizeof(T), kPitch = kPiece + 16;  // a lane's output bytes; its pitch in shared memory
  __shared__ __align__(16) uint8_t park[8][32 * kPitch];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t = static_cast<int>(idx >> sh), g = static_cast<int>(idx) & (ng - 1);
  const bool valid = t < len;
  const int tr = valid ? t : 0;  // (lanes past the end compute row 0 and store nothing)
  bool ok;
  const uint8_t* blk = cache_block(c, b, h, tr, nullptr, ok);
  const uint4 w4 = *reinterpret_cast<const uint4*>(blk + code_offset(d, is_v, tr & 15, g * 16));
  const float s = __half2float(*reinterpret_cast<const __half*>(blk + meta_offset(d, is_v, 0, g, tr & 15)));
  const float z = __half2float(*reinterpret_cast<const __half*>(blk + meta_offset(d, is_v, 1, g, tr & 15)));
  const uint32_t words[4] = {w4.x, w4.y, w4.z, w4.w};
  uint8_t* const mine = park[warp] + lane * kPitch;
#pragma unroll
  for (int j = 0; j < 4; ++j) {  // word j: elements 8j .. 8j+7, nibble i at bits 4i
    float x[8];
#pragma unroll
    for (int half = 0; half < 2; ++half) {  // bytes 0 / 2 of the word, then bytes 1 / 3
      const uint32_t w = half ? words[j] >> 8 : words[j];
      const uint32_t lo = (w & 0x000F000Fu) | 0x64006400u, hi = (w & 0x00F000F0u) | 0x64006400u;
      const float2 fl = __half22float2(*reinterpret_cast<const __half2*>(&lo));  // 1024 + n of nibbles 2*half, 2*half + 4
      const float2 fh = __half22float2(*reinterpret_cast<const __half2*>(&hi));  // 1024 + 16 n of nibbles 2*half + 1, + 5
      x[2 * half] = __fmul_rn(__fsub_rn(__fmaf_rn(fl.x, 1.0f, -1024.0f), z), s);
      x[2 * half + 4] = __fmul_rn(__fsub_rn(__fmaf_rn(fl.y, 1.0f, -1024.0f), z), s);
      x[2 * half + 1] = __fmul_rn(__fsub_rn(__fmaf_rn(fh.x, 0.0625f, -64.0f), z), s);
      x[2 * half + 5] = __fmul_rn(__fsub_rn(__fmaf_rn(fh.y, 0.0625f, -64.0f), z), s);
    }
    if constexpr (sizeof(T) == 4) {
      reinterpret_cast<float4*>(mine)[2 * j] = make_float4(x[0], x[1], x[2], x[3]);
      reinterpret_cast<float4*>(mine)[2 * j + 1] = make_float4(x[4], x[5], x[6], x[7]);
    } else {
      __half2 h2[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) h2[i] = __floats2half2_rn(x[2 * i], x[2 * i + 1]);
      reinterpret_cast<uint4*>(mine)[j] = *reinterpret_cast<uint4*>(h2);
    }
  }
  __syncwarp();
  // the warp's groups idx0 .. idx0 + 31 are consecutive in the output: element offset (row0 * ng + idx0) * 32
  const long long idx0 = idx - lane;
  uint8_t* const out0 = reinterpret_cast<uint8_t*>((is_v ? v_mat : k_mat) +
                                                   ((static_cast<long long>(b) * c.H_kv + h) * c.S_cap * ng + idx0) * 32);
#pragma unroll
  for (int i = 0; i < kPiece / 16; ++i) {
    const int o = i * 512 + 16 * lane, src = o / kPiece;
    if (static_cast<int>((idx0 + src) >> sh) < len)
      *reinterpret_cast<uint4*>(out0 + o) = *reinterpret_cast<const uint4*>(park[warp] + src * kPitch + (o % kPiece));
  }
}

}  // namespace

cudaError_t launch_decode_simple(const tq_kv_cache& c, const __half* q, int H_q, int S_q, float attn_scale, int window,
                                 int C, float* o_part, float* m_part, float* l_part, int32_t* status, cudaStream_t st) {
  auto run = [&](auto dtag) {
    constexpr int D = decltype(dtag)::value;
    SrcInt4<D> src{c};
    return launch_simple<D>(src, c, q, H_q, S_q, attn_scale, window, C, o_part, m_part, l_part, status, st);
  };
  switch (c.d) {
    case 64: return run(std::integral_constant<int, 64>{});
    case 128: return run(std::integral_constant<int, 128>{});
    case 512: return run(std::integral_constant<int, 512>{});
    default: return run(std::integral_constant<int, 256>{});
  }
}

cudaError_t launch_attend_materialized(const tq_kv_cache& c, const void* k_mat, const void* v_mat, bool fp32,
                                       const __half* q, int H_q, float attn_scale, int C, float* o_part, float* m_part,
                                       float* l_part, int32_t* status, cudaStream_t st) {
  // the tensor-core kernel where it applies (d = 128, at most 8 query heads per KV head), else the scalar one
  const cudaError_t fast = launch_attend_mat_mma(c, k_mat, v_mat, fp32, q, H_q, attn_scale, C, o_part, m_part, l_part, status, st);
  if (fast != cudaErrorNotSupported) return fast;
  auto run = [&](auto dtag, auto ttag) {
    constexpr int D = decltype(dtag)::value;
    using T = decltype(ttag);
    SrcMat<D, T> src{static_cast<const T*>(k_mat), static_cast<const T*>(v_mat)};
    return launch_simple<D>(src, c, q, H_q, 1, attn_scale, 0, C, o_part, m_part, l_part, status, st);
  };
  auto by_d = [&](auto ttag) {
    switch (c.d) {
      case 64: return run(std::integral_constant<int, 64>{}, ttag);
      case 128: return run(std::integral_constant<int, 128>{}, ttag);
      case 512: return run(std::integral_constant<int, 512>{}, ttag);
      default: return run(std::integral_constant<int, 256>{}, ttag);
    }
  };
  return fp32 ? by_d(float{}) : by_d(__half{});
}

cudaError_t launch_attend_mixed(const tq_kv_cache& c, const __half* k_fp16, const __half* v_fp16, const __half* q, int H_q,
                                float attn_scale, int C, float* o_part, float* m_part, float* l_part, int32_t* status,
                                cudaStream_t st) {
  auto run = [&](auto dtag) {
    constexpr int D = decltype(dtag)::value;
    SrcMixed<D> src{SrcInt4<D>{c}, SrcMat<D, __half>{k_fp16, v_fp16}};
    return launch_simple<D>(src, c, q, H_q, 1, attn_scale, 0, C, o_part, m_part, l_part, status, st);
  };
  switch (c.d) {
    case 64: return run(std::integral_constant<int, 64>{});
    case 128: return run(std::integral_constant<int, 128>{});
    case 512: return run(std::integral_constant<int, 512>{});
    default: return run(std::integral_constant<int, 256>{});
  }
}

cudaError_t launch_dequant(const tq_kv_cache& c, void* k_mat, void* v_mat, bool fp32, cudaStream_t st) {
  const long long per_head = static_cast<long long>(c.S_cap) * (c.d >> 5);
  dim3 grid(static_cast<unsigned>((per_head + 255) / 256), c.B, 2 * c.H_kv);
  if (fp32)
    dequant_kernel<float><<<grid, 256, 0, st>>>(c, static_cast<float*>(k_mat), static_cast<float*>(v_mat));
  else
    dequant_kernel<__half><<<grid, 256, 0, st>>>(c, static_cast<__half*>(k_mat), static_cast<__half*>(v_mat));
  return cudaGetLastError();
}

}  // namespace tq
