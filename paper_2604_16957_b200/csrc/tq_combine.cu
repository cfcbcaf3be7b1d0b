// Split reduction of Eq. 5:  o = sum_c l_c e^{m_c - m_g} o_c / sum_c l_c e^{m_c - m_g}.
// One block per (sequence, query head), one thread per output channel; the C weights are
// computed once per block into shared memory.
#include "tq_internal.cuh"

namespace tq {
namespace {

__global__ void __launch_bounds__(256) combine_kernel(const float* __restrict__ o_part, const float* __restrict__ m_part,
                                                      const float* __restrict__ l_part, int d, int C,
                                                      void* __restrict__ out, int out_fp32) {
  __shared__ float w[TQ_MAX_SPLITS];
  __shared__ float red[8];
  const long long bh = blockIdx.x;
  const float* m = m_part + bh * C;
  const float* l = l_part + bh * C;
  // global maximum over non-empty splits
  float mg = -INFINITY;
  for (int c = threadIdx.x; c < C; c += blockDim.x)
    if (l[c] > 0.f) mg = fmaxf(mg, m[c]);
#pragma unroll
  for (int off = 16; off; off >>= 1) mg = fmaxf(mg, __shfl_xor_sync(0xffffffffu, mg, off));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = mg;
  __syncthreads();
  mg = red[0];
  for (int i = 1; i < (blockDim.x >> 5); ++i) mg = fmaxf(mg, red[i]);
  for (int c = threadIdx.x; c < C; c += blockDim.x) w[c] = l[c] > 0.f ? l[c] * __expf(m[c] - mg) : 0.f;
  __syncthreads();
  const int x = threadIdx.x;
  if (x >= d) return;
  float num = 0.f, den = 0.f;
  const float* o = o_part + bh * C * d + x;
  for (int c = 0; c < C; ++c) {
    const float wc = w[c];
    den += wc;
    if (wc > 0.f) num = fmaf(wc, o[static_cast<long long>(c) * d], num);
  }
  const float r = den > 0.f ? num / den : 0.f;
  if (out_fp32) static_cast<float*>(out)[bh * d + x] = r;
  else static_cast<__half*>(out)[bh * d + x] = __float2half_rn(r);
}

}  // namespace

cudaError_t launch_combine(const float* o_part, const float* m_part, const float* l_part, int B, int H_q, int d, int C,
                           void* out, bool out_fp32, cudaStream_t st) {
  const int threads = ((d + 31) / 32) * 32;
  combine_kernel<<<B * H_q, threads, 0, st>>>(o_part, m_part, l_part, d, C, out, out_fp32 ? 1 : 0);
  return cudaGetLastError();
}

}  // namespace tq
