// The quantiser of Sec. 2.1 (Eq. 2-3) for the eight elements one thread holds; shared by the append kernels
// (tq_quantize.cu) and the fused decode step (tq_decode_mma.cu).  Internal to libtq.
//
// All arithmetic is IEEE binary32 with explicit round-to-nearest intrinsics so that the result is
// bit-identical on any machine that follows the same operation order:
//   s = fp16((max - min) / 15);  z = fp16((0 - min) / s);  q = clamp(rint(x / s + z), 0, 15).
#pragma once
#include "tq_internal.cuh"

namespace tq {

// The defining arithmetic, step by step (true divisions, explicit roundings): what every result must be equal
// to, bit for bit.  Out of line: the fast path below hands over whenever it cannot prove its own result.
// Returns the eight codes (element i in bits 4i .. 4i+3) and the stored scale (low half) and zero (high half).
// Arguments and result travel in registers (no arrays by reference: those would live in local memory).
static __device__ __noinline__ uint2 quantize_exact(const uint4 raw, float mn, float mx) {
  const __half2* h2 = reinterpret_cast<const __half2*>(&raw);
  const float s32 = __fdiv_rn(__fsub_rn(mx, mn), 15.0f);
  const __half s16 = __float2half_rn(s32);
  if ((__half_as_ushort(s16) & 0x7FFFu) == 0) {  // scale rounds to zero: constant (or nearly constant) group
    // s = 1.0, all codes 0
    return make_uint2(0u, 0x3C00u | (static_cast<uint32_t>(__half_as_ushort(__float2half_rn(__fsub_rn(0.0f, mn)))) << 16));
  }
  const float sf = __half2float(s16);
  float z32 = __fdiv_rn(__fsub_rn(0.0f, mn), sf);
  z32 = fminf(fmaxf(z32, -65504.0f), 65504.0f);
  const __half z16 = __float2half_rn(z32);
  const float zf = __half2float(z16);
  uint32_t word = 0u;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 f = __half22float2(h2[i]);
    const float u0 = fminf(fmaxf(__fadd_rn(__fdiv_rn(f.x, sf), zf), 0.0f), 15.0f);  // fmaxf also turns NaN into 0
    const float u1 = fminf(fmaxf(__fadd_rn(__fdiv_rn(f.y, sf), zf), 0.0f), 15.0f);
    word |= (__float_as_uint(u0 + 12582912.0f) & 0xFu) << (8 * i);                // rint, ties to even
    word |= (__float_as_uint(u1 + 12582912.0f) & 0xFu) << (8 * i + 4);
  }
  return make_uint2(word, static_cast<uint32_t>(__half_as_ushort(s16)) | (static_cast<uint32_t>(__half_as_ushort(z16)) << 16));
}

// Correctly rounded a / b from a correctly rounded reciprocal rb = fl(1 / b): q = fl(a * rb), the remainder
// r = a - q * b (exact in one fused multiply-add), and fl(q + r * rb).  For the quotients of the quantiser --
// a difference of two finite binary16 numbers over 15, and a negated finite binary16 number over a positive
// binary16 scale -- the result is bit-identical to __fdiv_rn: nothing under- or overflows on the way, and the
// library's own check (division_check_kernel, run by its tests) compares all 4.0e9 + 2.0e9 such pairs.
// A zero or non-finite b gives a non-finite or NaN result, which the callers' range checks reject; a zero
// numerator may come back with the other sign (-0 / 15), which only a zero range produces and which is
// rejected the same way (its scale is zero).
__device__ __forceinline__ float div_rn_by_reciprocal(float a, float b, float rb) {
  const float q = __fmul_rn(a, rb);
  return fmaf(fmaf(-q, b, a), rb, q);
}
__device__ __forceinline__ float div_rn_by_15(float a) { return div_rn_by_reciprocal(a, 15.0f, 0.0666666701436042785645f); }

// Quantise the 8 elements held by this thread (quad = one group).  All 32 lanes must call.
//
// Defining arithmetic: s = fp16((max - min) / 15), z = fp16(clamp((0 - min) / s)), u = fl(fl(x / s) + z),
// q = clamp(rint(u), 0, 15), every operation rounded to nearest even in binary32.  A division, a round, two
// clamps and a conversion per element would make this kernel many times slower than the memory system, so
// the common case does less and proves that it changed nothing:
//   ua = fma(x, 1/s, z) with the correctly rounded reciprocal differs from u by at most
//        (|x/s| + |u|) * 2^-23 <= tol (a per-group bound, with a 4x margin);
//   ua is monotone in x, so all eight lie between fma(min, 1/s, z) and fma(max, 1/s, z): if those are inside
//        (-0.49, 15.49) no clamp can act;
//   r = (ua + 1.5 * 2^23) - 1.5 * 2^23 is rint(ua), ties to even; if no ua is within tol of a rounding
//        boundary k + 1/2, rint(u) = rint(ua) for all eight.
// Whenever one of the conditions fails (a NaN anywhere fails them too: degenerate groups, overflowing zeros,
// non-finite inputs) the thread takes quantize_exact.  The result is bit-identical to the defining arithmetic.
__device__ __forceinline__ void quantize_chunk(const uint4 raw, uint32_t& word, __half& s_out, __half& z_out) {
  const __half2* h2 = reinterpret_cast<const __half2*>(&raw);
  float x[8];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float2 f = __half22float2(h2[i]);
    x[2 * i] = f.x;
    x[2 * i + 1] = f.y;
  }
  float mn = fminf(fminf(fminf(x[0], x[1]), fminf(x[2], x[3])), fminf(fminf(x[4], x[5]), fminf(x[6], x[7])));
  float mx = fmaxf(fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3])), fmaxf(fmaxf(x[4], x[5]), fmaxf(x[6], x[7])));
#pragma unroll
  for (int off = 1; off <= 2; off <<= 1) {
    mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, off));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
  }
  const __half s16 = __float2half_rn(__fdiv_rn(__fsub_rn(mx, mn), 15.0f));
  const float sf = __half2float(s16);
  const __half z16 = __float2half_rn(__fdiv_rn(__fsub_rn(0.0f, mn), sf));  // no clamp here: an overflow fails the checks
  const float zf = __half2float(z16);
  const float rs = __frcp_rn(sf);
  const float tol = (2.0f * fmaxf(fabsf(mn), fabsf(mx)) * rs + fabsf(zf) + 17.0f) * 4.76837158203125e-7f;  // 2^-21
  constexpr float kMagic = 12582912.0f;  // 1.5 * 2^23
  float r[8];          // the codes as floats
  float far = 0.0f;    // largest |ua - rint(ua)| over the 8 elements (at most 1/2)
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float u = fmaf(x[i], rs, zf);
    r[i] = (u + kMagic) - kMagic;
    far = fmaxf(far, fabsf(u - r[i]));
  }
  // four codes are a 16-bit integer that fp32 holds exactly: Horner with fused multiply-adds, then the
  // integer is read off the low mantissa bits of (value + 2^23)
  const float lo = fmaf(fmaf(fmaf(r[3], 16.0f, r[2]), 16.0f, r[1]), 16.0f, r[0]);
  const float hi = fmaf(fmaf(fmaf(r[7], 16.0f, r[6]), 16.0f, r[5]), 16.0f, r[4]);
  word = __byte_perm(__float_as_uint(lo + 8388608.0f), __float_as_uint(hi + 8388608.0f), 0x5410);
  s_out = s16;
  z_out = z16;
  const bool proven = fmaf(mn, rs, zf) > -0.49f && fmaf(mx, rs, zf) < 15.49f && 0.5f - far > tol;
  if (!proven) {  // rare
    const uint2 e = quantize_exact(raw, mn, mx);
    word = e.x;
    s_out = __ushort_as_half(static_cast<unsigned short>(e.y & 0xFFFFu));
    z_out = __ushort_as_half(static_cast<unsigned short>(e.y >> 16));
  }
}


// Cold path of quantize_group32: the elements whose two-sided roundings disagree are redone with the defining
// arithmetic (a true division) and their codes put in place.  Out of line, everything in registers.
static __device__ __noinline__ uint4 redo_near_boundaries(const uint4 r0, const uint4 r1, const uint4 r2, const uint4 r3,
                                                          uint4 words, float rs, float sf, float zf, float z_lo,
                                                          float z_hi) {
  constexpr float kMagic = 12582912.0f;  // 1.5 * 2^23
  const uint4 raw[4] = {r0, r1, r2, r3};
  const __half2* h2 = reinterpret_cast<const __half2*>(&raw[0]);
  uint32_t word[4] = {words.x, words.y, words.z, words.w};
#pragma unroll
  for (int i = 0; i < 32; ++i) {  // unrolled: every index is a constant, the arrays stay in registers
    const float2 f = __half22float2(h2[i >> 1]);
    const float x = (i & 1) ? f.y : f.x;
    if (((__float_as_uint(fmaf(x, rs, z_lo)) ^ __float_as_uint(fmaf(x, rs, z_hi))) >> 16) != 0) {
      const float ue = __fadd_rn(__fdiv_rn(x, sf), zf);
      const uint32_t q = __float_as_uint(ue + kMagic) & 0xFu;  // rint, ties to even; 0 .. 15 because no clamp can act
      word[i >> 3] = (word[i >> 3] & ~(0xFu << (4 * (i & 7)))) | (q << (4 * (i & 7)));
    }
  }
  return make_uint4(word[0], word[1], word[2], word[3]);
}

// The same quantiser for a thread that holds a whole group of 32 elements (the bulk kernel): minimum and
// maximum are found on the packed halves, the per-group work (two divisions, a reciprocal, the bound) is paid
// once per 32 elements instead of once per 8, and no shuffle is needed.  raw[j] holds elements 8j .. 8j+7.
// Bit-identical to quantize_chunk run by a lane quad: the fast path proves its own result or hands over to
// the defining arithmetic.  Its proof costs two fused multiply-adds and one logic operation per element:
//   v = x / s + z (real numbers); the defined u = fl(fl(x / s) + z) has |u - v| <= 2^-24 (|x / s| + |u|);
//   t- = fma(x, 1/s, fl(z + fl(128.5 - T))) and t+ = fma(x, 1/s, fl(z + fl(128.5 + T))) lie in [128, 144) when
//        no clamp can act (checked on the group's extremes, as in quantize_chunk), where binary32 has a unit
//        of 2^-16: bits 16 .. 19 of such a number are floor(t) - 128;
//   t- >= v + 128.5 - T - e and t+ <= v + 128.5 + T + e with e <= 2^-24 (|x / s| + |z| + 129) + 2^-16 (the
//        reciprocal, the rounding of z + c, of c and of the fma);
//   so if floor(t-) = floor(t+) = 128 + k then k - 1/2 + (T - e) <= v < k + 1/2 - (T - e), and with
//        T = tol + 2^-15, tol >= 8 * 2^-24 (2 |x / s| + |z| + 17), u lies strictly inside (k - 1/2, k + 1/2):
//        rint(u) = k, the byte 2 of t-.
// The exclusive-or of t- and t+ of all 32 elements is accumulated; if its bits 16 and up are clear, every
// code is proven.  Otherwise (about one group in 300 on Gaussian inputs) the elements whose two sides
// disagree are redone by true division.
__device__ __forceinline__ void quantize_group32(const uint4 (&raw)[4], uint32_t (&word)[4], __half& s_out, __half& z_out) {
  const __half2* h2 = reinterpret_cast<const __half2*>(&raw[0]);
  __half2 mn2 = h2[0], mx2 = h2[0];
#pragma unroll
  for (int i = 1; i < 16; ++i) {
    mn2 = __hmin2(mn2, h2[i]);
    mx2 = __hmax2(mx2, h2[i]);
  }
  const float mn = fminf(__low2float(mn2), __high2float(mn2));
  const float mx = fmaxf(__low2float(mx2), __high2float(mx2));
  const __half s16 = __float2half_rn(div_rn_by_15(__fsub_rn(mx, mn)));
  const float sf = __half2float(s16);
  const float rs = __frcp_rn(sf);
  const __half z16 = __float2half_rn(div_rn_by_reciprocal(__fsub_rn(0.0f, mn), sf, rs));  // no clamp here: an overflow fails the checks
  const float zf = __half2float(z16);
  const float tol = fmaf(2.0f * fmaxf(fabsf(mn), fabsf(mx)) * rs + fabsf(zf) + 17.0f, 4.76837158203125e-7f,  // 2^-21
                         3.0517578125e-5f);                                                               // 2^-15
  const float z_lo = __fadd_rn(zf, __fsub_rn(128.5f, tol)), z_hi = __fadd_rn(zf, __fadd_rn(128.5f, tol));
  uint32_t differ = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    uint32_t t[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 f = __half22float2(h2[4 * j + i]);
      t[2 * i] = __float_as_uint(fmaf(f.x, rs, z_lo));
      t[2 * i + 1] = __float_as_uint(fmaf(f.y, rs, z_lo));
      differ |= t[2 * i] ^ __float_as_uint(fmaf(f.x, rs, z_hi));
      differ |= t[2 * i + 1] ^ __float_as_uint(fmaf(f.y, rs, z_hi));
    }
    // byte 2 of each t is its code: gather the even and the odd elements' bytes, then odd * 16 + even
    const uint32_t ev = __byte_perm(__byte_perm(t[0], t[2], 0x0062), __byte_perm(t[4], t[6], 0x0062), 0x5410);
    const uint32_t od = __byte_perm(__byte_perm(t[1], t[3], 0x0062), __byte_perm(t[5], t[7], 0x0062), 0x5410);
    word[j] = od * 16u + ev;
  }
  s_out = s16;
  z_out = z16;
  const bool in_range = fmaf(mn, rs, zf) > -0.49f && fmaf(mx, rs, zf) < 15.49f;
  if (in_range && (differ >> 16) != 0) {
    // Rare: no clamp can act, but some element sits within the bound of a rounding boundary.
    const uint4 w = redo_near_boundaries(raw[0], raw[1], raw[2], raw[3], make_uint4(word[0], word[1], word[2], word[3]),
                                         rs, sf, zf, z_lo, z_hi);
    word[0] = w.x; word[1] = w.y; word[2] = w.z; word[3] = w.w;
  } else if (!in_range) {  // rarer: clamps, degenerate scales, overflowing zeros
#pragma unroll  // constant indices: raw stays in registers
    for (int j = 0; j < 4; ++j) {
      const uint2 e = quantize_exact(raw[j], mn, mx);
      word[j] = e.x;
      s_out = __ushort_as_half(static_cast<unsigned short>(e.y & 0xFFFFu));
      z_out = __ushort_as_half(static_cast<unsigned short>(e.y >> 16));
    }
  }
}

}  // namespace tq
