// Comparison path, second half (Sec. 3.1 first paragraph, Table 2): split attention over MATERIALISED K^, V^
// matrices [B][H_kv][S_cap][128] in fp16 or fp32 -- the decode kernel's structure minus the unpacking, so that
// "dequantize-then-attend" is limited by the bytes it moves (160 + 2 * 1024 per token and KV head with an fp32
// workspace) and not by scalar arithmetic.  d = 128 and at most 8 query heads per KV head; every other shape
// stays with the scalar kernel of tq_attend_simple.cu.
//
// One warp per 16-token block, operands straight from global memory in the register layout of
// mma.sync.m16n8k16 (no shared-memory staging: 16 resident warps per SM keep enough loads in flight):
//   scores  S[token][head] = K^[token][:] . q[head][:]   A = K^ rows (each lane loads 16-byte chunks of rows
//           gid and gid + 8; which channel sits in which k slot is free as long as q is loaded the same way),
//           B = q.  fp32 matrices are split into fp16 hi + lo parts and cost two MMAs per k step.
//   output  O^T[channel][head] += V^^T[channel][token] . P[token][head]   A = V^ with two tokens side by side
//           in one register (byte permutes of the rows of tokens 2*tid4, 2*tid4+1, ...), B = fp16(P)
//           transposed by movmatrix.  fp32 V^ is rounded to fp16 here, like P.
// Online softmax in the log2 domain (Algorithm 1); the eight warps merge through shared memory and write the
// normalised partial (o_c, m_c, l_c) of Eq. 5.
#include "tq_internal.cuh"

namespace tq {
namespace {

constexpr int kD = 128;
constexpr int kWarpsMat = 8;
constexpr float kLog2eM = 1.4426950408889634f;
constexpr float kLn2M = 0.6931471805599453f;
constexpr float kNoMaxM = -1.0e30f;

__device__ __forceinline__ void mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                        uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t movm_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(d) : "r"(a));
  return d;
}
__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_h2(float a, float b) {
  const __half2 h = __floats2half2_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// Eight consecutive channels of one row as four half2 registers; fp32 rows are rounded (hi) and, for K^, the
// remainders kept (lo).
template <typename T, bool LO>
__device__ __forceinline__ void load_chunk(const T* p, uint32_t (&hi)[4], uint32_t (&lo)[4]) {
  if constexpr (sizeof(T) == 2) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(p));
    hi[0] = v.x; hi[1] = v.y; hi[2] = v.z; hi[3] = v.w;
    lo[0] = lo[1] = lo[2] = lo[3] = 0u;
  } else {
    const float4 a = __ldg(reinterpret_cast<const float4*>(p)), b = __ldg(reinterpret_cast<const float4*>(p) + 1);
    const float x[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const __half2 h = __floats2half2_rn(x[2 * r], x[2 * r + 1]);
      hi[r] = *reinterpret_cast<const uint32_t*>(&h);
      if (LO) {
        const float2 f = __half22float2(h);
        lo[r] = pack_h2(x[2 * r] - f.x, x[2 * r + 1] - f.y);
      } else {
        lo[r] = 0u;
      }
    }
  }
}

template <typename T>
__global__ void __launch_bounds__(kWarpsMat * 32, 2)
    attend_mat_kernel(const T* __restrict__ k_mat, const T* __restrict__ v_mat, const int32_t* seq_lens, int H_kv, int S_cap,
                      const __half* __restrict__ q, int H_q, float attn_scale, int C, float* __restrict__ o_part,
                      float* __restrict__ m_part, float* __restrict__ l_part, int32_t* status) {
  constexpr bool F32 = sizeof(T) == 4;
  __shared__ float sm_ml[kWarpsMat][16];         // per warp: m of 8 heads, l of 8 heads
  __shared__ float sm_o[kWarpsMat][8][kD + 4];   // per warp: unnormalised output [head][channel]
  pdl_launch_dependents();
  pdl_wait();
  const int c = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, gid = lane >> 2, t4 = lane & 3;
  const int G = H_q / H_kv;
  const int len = checked_len(seq_lens, b, S_cap, (c == 0 && kvh == 0) ? status : nullptr);
  int t0, t1;
  split_range(0, len, C, c, t0, t1);

  // q as B fragments: head gid of this KV head, 16-byte chunk t4 + 4j of its row (k slots follow the chunks)
  uint32_t qf[4][4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    uint4 v = make_uint4(0, 0, 0, 0);
    if (gid < G) v = *reinterpret_cast<const uint4*>(q + (static_cast<long long>(b) * H_q + kvh * G + gid) * kD + (t4 + 4 * j) * 8);
    qf[j][0] = v.x; qf[j][1] = v.y; qf[j][2] = v.z; qf[j][3] = v.w;
  }
  float oacc[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i) oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f;
  float m0 = kNoMaxM, m1 = kNoMaxM, l0 = 0.f, l1 = 0.f;  // heads 2*t4, 2*t4+1; l: this lane's tokens only
  const float cs = attn_scale * kLog2eM;
  const T* const kb = k_mat + (static_cast<long long>(b) * H_kv + kvh) * S_cap * kD;
  const T* const vb = v_mat + (static_cast<long long>(b) * H_kv + kvh) * S_cap * kD;
  const int last = t1 - 1;  // rows past the end of the split are never read: their loads go to this row, their weights are 0

#pragma unroll 1
  for (int first = t0 + 16 * warp; first < t1; first += 16 * kWarpsMat) {
    // ---------------- scores of 16 tokens x 8 heads
    const long long ra = static_cast<long long>(min(first + gid, last)) * kD;
    const long long rb = static_cast<long long>(min(first + gid + 8, last)) * kD;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      uint32_t ah[4], al[4], bh[4], bl[4];
      load_chunk<T, true>(kb + ra + (t4 + 4 * j) * 8, ah, al);
      load_chunk<T, true>(kb + rb + (t4 + 4 * j) * 8, bh, bl);
#pragma unroll
      for (int p = 0; p < 2; ++p) {
        mma_f16(acc, ah[2 * p], bh[2 * p], ah[2 * p + 1], bh[2 * p + 1], qf[j][2 * p], qf[j][2 * p + 1]);
        if (F32) mma_f16(acc, al[2 * p], bl[2 * p], al[2 * p + 1], bl[2 * p + 1], qf[j][2 * p], qf[j][2 * p + 1]);
      }
    }
    // ---------------- online softmax, log2 domain: acc[0], acc[1] = token gid, acc[2], acc[3] = token gid + 8
    const bool on0 = first + gid < t1, on8 = first + gid + 8 < t1;
    const float a0 = on0 ? acc[0] * cs : -INFINITY, a1 = on0 ? acc[1] * cs : -INFINITY;
    const float a2 = on8 ? acc[2] * cs : -INFINITY, a3 = on8 ? acc[3] * cs : -INFINITY;
    float bm0 = fmaxf(a0, a2), bm1 = fmaxf(a1, a3);
#pragma unroll
    for (int off = 4; off <= 16; off <<= 1) {
      bm0 = fmaxf(bm0, __shfl_xor_sync(0xffffffffu, bm0, off));
      bm1 = fmaxf(bm1, __shfl_xor_sync(0xffffffffu, bm1, off));
    }
    if (bm0 > m0 || bm1 > m1) {  // (the same for every lane of a quad column; lanes of other columns rescale on their own maxima)
      const float n0 = fmaxf(m0, bm0), n1 = fmaxf(m1, bm1);
      const float f0 = ex2f(m0 - n0), f1 = ex2f(m1 - n1);
      m0 = n0; m1 = n1;
      l0 *= f0; l1 *= f1;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        oacc[i][0] *= f0; oacc[i][1] *= f1; oacc[i][2] *= f0; oacc[i][3] *= f1;
      }
    }
    const float p0 = ex2f(a0 - m0), p1 = ex2f(a1 - m1), p2 = ex2f(a2 - m0), p3 = ex2f(a3 - m1);
    l0 += p0 + p2;
    l1 += p1 + p3;
    const uint32_t pt0 = movm_trans(pack_h2(p0, p1)), pt1 = movm_trans(pack_h2(p2, p3));

    // ---------------- O^T += V^^T . P: rows of tokens 2*t4, 2*t4+1, 2*t4+8, 2*t4+9, chunks gid and gid + 8
    long long tv[4];
    tv[0] = static_cast<long long>(min(first + 2 * t4, last)) * kD;
    tv[1] = static_cast<long long>(min(first + 2 * t4 + 1, last)) * kD;
    tv[2] = static_cast<long long>(min(first + 2 * t4 + 8, last)) * kD;
    tv[3] = static_cast<long long>(min(first + 2 * t4 + 9, last)) * kD;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      uint32_t v[4][4], unused[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) load_chunk<T, false>(vb + tv[i] + (gid + 8 * h) * 8, v[i], unused);
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        // rows gid / gid + 8 of this M tile are channels 8 * (gid + 8h) + 2r and + 2r + 1
        mma_f16(oacc[4 * h + r], __byte_perm(v[0][r], v[1][r], 0x5410), __byte_perm(v[0][r], v[1][r], 0x7632),
                __byte_perm(v[2][r], v[3][r], 0x5410), __byte_perm(v[2][r], v[3][r], 0x7632), pt0, pt1);
      }
    }
  }

  // ---------------- merge the eight warps, write the normalised partial (o_c, m_c, l_c)
#pragma unroll
  for (int off = 4; off <= 16; off <<= 1) {
    l0 += __shfl_xor_sync(0xffffffffu, l0, off);
    l1 += __shfl_xor_sync(0xffffffffu, l1, off);
  }
  if (gid == 0) {
    sm_ml[warp][2 * t4] = m0;
    sm_ml[warp][2 * t4 + 1] = m1;
    sm_ml[warp][8 + 2 * t4] = l0;
    sm_ml[warp][8 + 2 * t4 + 1] = l1;
  }
#pragma unroll
  for (int mt = 0; mt < 8; ++mt) {
    const int ch = 8 * (gid + 8 * (mt >> 2)) + 2 * (mt & 3);
    sm_o[warp][2 * t4][ch] = oacc[mt][0];
    sm_o[warp][2 * t4 + 1][ch] = oacc[mt][1];
    sm_o[warp][2 * t4][ch + 1] = oacc[mt][2];
    sm_o[warp][2 * t4 + 1][ch + 1] = oacc[mt][3];
  }
  __syncthreads();
  const int head = warp;  // warp w finishes head w: lane l owns channels 4l .. 4l+3
  if (head < G) {
    float M = kNoMaxM;
#pragma unroll
    for (int w = 0; w < kWarpsMat; ++w) M = fmaxf(M, sm_ml[w][head]);
    float den = 0.f;
    float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int w = 0; w < kWarpsMat; ++w) {  // a warp that saw no token has m = -1e30, l = 0, o = 0
      const float f = ex2f(sm_ml[w][head] - M);
      den = fmaf(f, sm_ml[w][8 + head], den);
      const float4 x = *reinterpret_cast<const float4*>(&sm_o[w][head][4 * lane]);
      o.x = fmaf(f, x.x, o.x); o.y = fmaf(f, x.y, o.y); o.z = fmaf(f, x.z, o.z); o.w = fmaf(f, x.w, o.w);
    }
    const float inv = den > 0.f ? 1.f / den : 0.f;
    const long long pidx = (static_cast<long long>(b) * H_q + kvh * G + head) * C + c;
    reinterpret_cast<float4*>(o_part + pidx * kD)[lane] = make_float4(o.x * inv, o.y * inv, o.z * inv, o.w * inv);
    if (lane == 0) {
      m_part[pidx] = den > 0.f ? M * kLn2M : -INFINITY;  // natural-log units of attn_scale * q.k^
      l_part[pidx] = den;
    }
  }
}

}  // namespace

// d = 128, at most 8 query heads per KV head: the tensor-core kernel above.  Returns cudaErrorNotSupported for
// every other shape (the caller then uses the scalar kernel).
cudaError_t launch_attend_mat_mma(const tq_kv_cache& c, const void* k_mat, const void* v_mat, bool fp32, const __half* q,
                                  int H_q, float attn_scale, int C, float* o_part, float* m_part, float* l_part,
                                  int32_t* status, cudaStream_t st) {
  if (c.d != kD || H_q / c.H_kv > 8) return cudaErrorNotSupported;
  dim3 grid(C, c.H_kv, c.B);
  if (fp32)
    return launch_kernel(attend_mat_kernel<float>, grid, dim3(kWarpsMat * 32), 0, st, static_cast<const float*>(k_mat),
                         static_cast<const float*>(v_mat), c.seq_lens, c.H_kv, c.S_cap, q, H_q, attn_scale, C, o_part, m_part,
                         l_part, status);
  return launch_kernel(attend_mat_kernel<__half>, grid, dim3(kWarpsMat * 32), 0, st, static_cast<const __half*>(k_mat),
                       static_cast<const __half*>(v_mat), c.seq_lens, c.H_kv, c.S_cap, q, H_q, attn_scale, C, o_part, m_part,
                       l_part, status);
}

}  // namespace tq
