// Split reduction of Eq. 5:  o = sum_c l_c e^{m_c - m_g} o_c / sum_c l_c e^{m_c - m_g}.
// One 256-thread block per (sequence, query head).  The C split weights are computed once into
// shared memory; the weighted sum over splits is spread over the block (each thread owns one
// float4 of channels and every nsl-th split) so that the loads of a row of partials are
// independent and in flight together, then folded through shared memory.
#include "tq_internal.cuh"

namespace tq {
namespace {

constexpr int kThreads = 256;

__global__ void __launch_bounds__(kThreads) combine_kernel(const float* __restrict__ o_part,
                                                           const float* __restrict__ m_part,
                                                           const float* __restrict__ l_part, int d, int C,
                                                           void* __restrict__ out, int out_fp32) {
  __shared__ float w[TQ_MAX_SPLITS];
  __shared__ float red[kThreads / 32];
  __shared__ float4 acc[kThreads];
  pdl_launch_dependents();
  pdl_wait();
  const long long bh = blockIdx.x;
  const float* m = m_part + bh * C;
  const float* l = l_part + bh * C;
  const int tid = threadIdx.x;
  const int nchunk = d >> 2;            // float4 chunks per row (8 .. 64)
  const int nsl = kThreads / nchunk;    // split lanes
  const int chunk = tid % nchunk, sl = tid / nchunk;
  const float4* o = reinterpret_cast<const float4*>(o_part + bh * C * d) + chunk;

  // The partial outputs do not depend on the weights: fetch this thread's first kPre of them now, so
  // that their latency overlaps the (m, l) loads and the weight computation below.
  constexpr int kPre = 8;
  float4 pre[kPre];
#pragma unroll
  for (int i = 0; i < kPre; ++i) {
    const int c = sl + i * nsl;
    pre[i] = (sl < nsl && c < C) ? o[static_cast<long long>(c) * nchunk] : make_float4(0.f, 0.f, 0.f, 0.f);
  }

  // global maximum over non-empty splits (C <= 256: one split per thread)
  const float lc = tid < C ? l[tid] : 0.f;
  const float mc = (tid < C && lc > 0.f) ? m[tid] : -INFINITY;
  float mg = mc;
#pragma unroll
  for (int off = 16; off; off >>= 1) mg = fmaxf(mg, __shfl_xor_sync(0xffffffffu, mg, off));
  if ((tid & 31) == 0) red[tid >> 5] = mg;
  __syncthreads();
  mg = red[0];
#pragma unroll
  for (int i = 1; i < kThreads / 32; ++i) mg = fmaxf(mg, red[i]);
  if (tid < C) w[tid] = lc > 0.f ? lc * __expf(mc - mg) : 0.f;
  __syncthreads();

  float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
  float den = 0.f;
  if (sl < nsl) {
#pragma unroll
    for (int i = 0; i < kPre; ++i) {
      const int c = sl + i * nsl;
      const float wc = c < C ? w[c] : 0.f;  // an empty split has weight 0 and o = 0
      a.x = fmaf(wc, pre[i].x, a.x);
      a.y = fmaf(wc, pre[i].y, a.y);
      a.z = fmaf(wc, pre[i].z, a.z);
      a.w = fmaf(wc, pre[i].w, a.w);
    }
    for (int c = sl + kPre * nsl; c < C; c += nsl) {
      const float wc = w[c];
      const float4 v = o[static_cast<long long>(c) * nchunk];
      a.x = fmaf(wc, v.x, a.x);
      a.y = fmaf(wc, v.y, a.y);
      a.z = fmaf(wc, v.z, a.z);
      a.w = fmaf(wc, v.w, a.w);
    }
  }
  acc[tid] = a;
  __syncthreads();
  if (tid < nchunk) {
    for (int c = 0; c < C; ++c) den += w[c];
    float4 s = acc[tid];
    for (int j = 1; j < nsl; ++j) {
      const float4 v = acc[j * nchunk + tid];
      s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
    }
    const float inv = den > 0.f ? 1.f / den : 0.f;
    s.x *= inv; s.y *= inv; s.z *= inv; s.w *= inv;
    if (out_fp32) {
      reinterpret_cast<float4*>(static_cast<float*>(out) + bh * d)[tid] = s;
    } else {
      __half2 h[2] = {__floats2half2_rn(s.x, s.y), __floats2half2_rn(s.z, s.w)};
      reinterpret_cast<uint2*>(static_cast<__half*>(out) + bh * d)[tid] = *reinterpret_cast<uint2*>(h);
    }
  }
}

}  // namespace

cudaError_t launch_combine(const float* o_part, const float* m_part, const float* l_part, int B, int H_q, int d, int C,
                           void* out, bool out_fp32, cudaStream_t st) {
  return launch_kernel(combine_kernel, dim3(B * H_q), dim3(kThreads), 0, st, o_part, m_part, l_part, d, C, out,
                       out_fp32 ? 1 : 0);
}

}  // namespace tq
