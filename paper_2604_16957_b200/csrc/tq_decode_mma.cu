// Fused int4 decode attention, phase 1 (Sec. 3.1 Algorithm 1 per split, Sec. 3.2), for sm_100a.
//
// One thread block handles one (sequence, KV head, tile of up to 8 query heads, split).  The
// query heads that share the KV head are packed into the N = 8 dimension of
// mma.sync.m16n8k16, so every byte of the cache is read from HBM once per head tile.
// The path is HBM-bound: operands stream global -> shared with 16-byte cp.async into a
// per-warp ring of 16-token stages (each warp owns its tokens end to end, so the main loop has
// no block-wide barrier), and the tensor cores only take the G-packed q.K^T and P.V
// contractions off the CUDA cores, which could not keep up with the memory system otherwise.
//
// Dequantisation in registers (the paper's dequant4, and its Eq. 4 idea of folding the nibble
// position into the other operand):
//   * A 4-bit code n masked in place inside a 16-bit lane IS an fp16 number: bits 0-3 give the
//     subnormal n * 2^-24, bits 4-7 give n * 2^-20.  So `w & 0x000F000F` and `w & 0x00F000F0`
//     are ready-made half2 MMA operands holding exact codes; the factor 16 between the two is
//     folded into q (K side, exactly Eq. 4) or into the output row (V side), and 2^-24 into
//     the final scale.  No int->float conversion, no multiply per element.
//   * K: each pair of MMAs covers one quantisation group (k = 32 channels), so the per-token,
//     per-group scale is applied to the fp32 accumulator:
//        q.k^ = sum_g s_g * (sum_{c in g} q_c n_c  -  z_g * sum_{c in g} q_c).
//   * V: the scale varies along the contraction (token) axis, so it is folded into the other
//     operand: B_g = fp16(p * s_g) per group, o = sum_tok B_g * n - sum_tok B_g * z_g, the
//     second sum produced by one extra MMA per group whose A rows all hold z_g.
// Softmax is online in the log2 domain with a lazily updated running maximum (the maximum is
// raised only when a score exceeds it by more than 2^4, which keeps P <= 16 in fp16 and makes
// the rescale of the accumulators rare).
//
// Shared-memory layout of one stage (16 tokens of one KV head):
//   K codes [16][D/2] | V codes [16][D/2] | K scale [16][D/32] | K zero | V scale | V zero
// Code rows are padded by 16 bytes (pitch D/2 + 16) so that both access patterns below are
// bank-conflict free while every address is one per-lane base plus a compile-time offset:
//   K: lane (gid, tid4) reads word tid4 of group g of token gid      (8 tokens x 16 B per load)
//   V: lane (gid, tid4) reads word gid%4 of group g of token 2*tid4  (4 tokens x 16 B per load)
#include "tq_internal.cuh"

namespace tq {
namespace {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kBlk = 16;              // tokens per stage = MMA M (scores) = MMA K (P.V)
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 4.0f;  // log2 units
constexpr uint32_t kMaskLo = 0x000F000Fu;  // nibbles 0 / 4 of a 32-bit word: n * 2^-24 as fp16
constexpr uint32_t kMaskHi = 0x00F000F0u;  // nibbles 1 / 5: n * 2^-20 as fp16

template <int D>
struct Cfg {
  static constexpr int NG = D / 32;                 // groups per row == 16-byte chunks per code row
  static constexpr int ROWB = D / 2;                // bytes per code row in global memory
  static constexpr int PITCH = ROWB + 16;           // bytes per code row in shared memory
  static constexpr int PK = kBlk * PITCH;           // code bytes per stage, K or V
  static constexpr int SZ = kBlk * NG * 2;          // bytes of one scale or zero array per stage
  static constexpr int STAGE = 2 * PK + 4 * SZ;     // 1792 / 3072 / 5632 bytes
  static constexpr int NST = D == 64 ? 6 : 4;       // stages in the per-warp ring
  static constexpr int MINB = D == 256 ? 1 : 2;     // resident blocks per SM
  static constexpr int PIPE = kWarps * NST * STAGE; // 84 KB (D = 64), 96 KB (128), 176 KB (256)
  static constexpr int MERGE = kWarps * (8 * D + 16) * 4;
  static constexpr int SMEM = (PIPE > MERGE ? PIPE : MERGE) + 8 * NG * 4;
  // loader geometry
  static constexpr int TOK_PER_PASS = 32 / NG;      // tokens covered by one warp-wide pass of 16-byte chunks
  static constexpr int CODE_PASSES = kBlk / TOK_PER_PASS;
  static constexpr int LPA = NG == 2 ? 4 : 8;       // lanes per scale/zero array
  static constexpr int SZ_PASSES = (SZ / 16) / LPA;
};

__device__ __forceinline__ void mma16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(d) : "r"(a));
  return d;
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}

__device__ __forceinline__ uint32_t h2_as_u32(__half2 h) { return *reinterpret_cast<uint32_t*>(&h); }
__device__ __forceinline__ __half2 u32_as_h2(uint32_t u) { return *reinterpret_cast<__half2*>(&u); }

// Per-lane source pointers of the next token block to fetch, and the per-lane destination
// offsets inside a stage.  Advancing to the warp's next block is three pointer additions.
template <int D>
struct Loader {
  using C = Cfg<D>;
  const uint8_t *pk, *pv, *psz;  // psz points into one of the four scale / zero arrays, chosen by lane
  uint32_t dst_code, dst_sz;
  bool sz_lane;                  // this lane copies scale / zero chunks (all lanes unless D = 64)

  __device__ __forceinline__ void init(const tq_kv_cache& cache, long long row0, int first_blk, int lane) {
    const long long tok0 = static_cast<long long>(first_blk) * kBlk;
    pk = cache.k_packed + (row0 + tok0) * C::ROWB + lane * 16;
    pv = cache.v_packed + (row0 + tok0) * C::ROWB + lane * 16;
    dst_code = (lane / C::NG) * C::PITCH + (lane % C::NG) * 16;
    const int arr = lane / C::LPA, ch = lane % C::LPA;
    const uint16_t* base = arr == 0 ? cache.k_scale : (arr == 1 ? cache.k_zero : (arr == 2 ? cache.v_scale : cache.v_zero));
    sz_lane = arr < 4;
    psz = reinterpret_cast<const uint8_t*>(base) + (row0 + tok0) * (C::NG * 2) + ch * 16;
    dst_sz = 2 * C::PK + arr * C::SZ + ch * 16;
  }
  // copy one 16-token block into the stage at shared address `stage`, then step to the block kWarps further on
  __device__ __forceinline__ void issue(uint32_t stage) {
#pragma unroll
    for (int j = 0; j < C::CODE_PASSES; ++j) {
      cp_async16(stage + dst_code + j * C::TOK_PER_PASS * C::PITCH, pk + j * 512);
      cp_async16(stage + C::PK + dst_code + j * C::TOK_PER_PASS * C::PITCH, pv + j * 512);
    }
    if (C::LPA * 4 == 32 || sz_lane) {
#pragma unroll
      for (int j = 0; j < C::SZ_PASSES; ++j) cp_async16(stage + dst_sz + j * C::LPA * 16, psz + j * C::LPA * 16);
    }
    pk += kWarps * kBlk * C::ROWB;
    pv += kWarps * kBlk * C::ROWB;
    psz += kWarps * kBlk * C::NG * 2;
  }
};

template <int D>
__global__ void __launch_bounds__(kThreads, Cfg<D>::MINB)
    decode_mma_kernel(tq_kv_cache cache, const __half* __restrict__ q, int H_q, float attn_scale, int C,
                      float* __restrict__ o_part, float* __restrict__ m_part, float* __restrict__ l_part,
                      int32_t* status) {
  using Cf = Cfg<D>;
  constexpr int NG = Cf::NG;
  extern __shared__ __align__(128) uint8_t smem[];
  float* sm_qs = reinterpret_cast<float*>(smem + (Cf::SMEM - 8 * NG * 4));  // [8 heads][NG] group sums of q

  const int G = H_q / cache.H_kv;
  const int tiles = (G + 7) >> 3;
  const int c = blockIdx.x, kvh = blockIdx.y / tiles, tile = blockIdx.y - kvh * tiles, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, gid = lane >> 2, tid4 = lane & 3;
  const int h0 = kvh * G + tile * 8;         // first query head of this tile
  const int nh = min(8, G - tile * 8);       // heads in the tile; the rest of N = 8 is zero padding
  const int len = checked_len(cache.seq_lens, b, cache.S_cap, (c == 0 && blockIdx.y == 0) ? status : nullptr);
  int t0, t1;
  split_range(len, C, c, t0, t1);

  // ---- group sums of q (for the zero-point term), scaled by 2^-24 like the code operands
  {
    const int pair = threadIdx.x >> 2, part = threadIdx.x & 3;  // pair = head * NG + group
    float s = 0.f;
    if (pair < 8 * NG) {
      const int h = pair / NG, g = pair - h * NG;
      if (h < nh) {
        const uint4 raw = *reinterpret_cast<const uint4*>(q + (static_cast<long long>(b) * H_q + h0 + h) * D + g * 32 + part * 8);
        const __half2* h2 = reinterpret_cast<const __half2*>(&raw);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 f = __half22float2(h2[i]);
          s += f.x + f.y;
        }
      }
    }
    s += __shfl_xor_sync(0xffffffffu, s, 1);
    s += __shfl_xor_sync(0xffffffffu, s, 2);
    if (pair < 8 * NG && part == 0) sm_qs[pair] = s * 5.9604644775390625e-8f;  // 2^-24
  }
  __syncthreads();

  // ---- q as MMA B fragments: column n = gid is head h0 + gid; k slots follow the nibble order
  uint32_t qf[NG][4];
  float qs[NG][2];
#pragma unroll
  for (int g = 0; g < NG; ++g) {
    uint4 raw = make_uint4(0, 0, 0, 0);
    if (gid < nh)
      raw = *reinterpret_cast<const uint4*>(q + (static_cast<long long>(b) * H_q + h0 + gid) * D + g * 32 + tid4 * 8);
    const __half2 sixteenth = __float2half2_rn(0.0625f);
    qf[g][0] = __byte_perm(raw.x, raw.z, 0x5410);                                            // (c0, c4)
    qf[g][1] = h2_as_u32(__hmul2(u32_as_h2(__byte_perm(raw.x, raw.z, 0x7632)), sixteenth));  // (c1, c5) / 16
    qf[g][2] = __byte_perm(raw.y, raw.w, 0x5410);                                            // (c2, c6)
    qf[g][3] = h2_as_u32(__hmul2(u32_as_h2(__byte_perm(raw.y, raw.w, 0x7632)), sixteenth));  // (c3, c7) / 16
    qs[g][0] = sm_qs[(2 * tid4) * NG + g];
    qs[g][1] = sm_qs[(2 * tid4 + 1) * NG + g];
  }

  // ---- this warp's token blocks: blk0 + warp, blk0 + warp + kWarps, ...
  const int blk0 = t0 / kBlk, blk1 = (t1 + kBlk - 1) / kBlk;
  const int nblk = blk1 - blk0 > warp ? (blk1 - blk0 - warp + kWarps - 1) / kWarps : 0;
  const long long row0 = (static_cast<long long>(b) * cache.H_kv + kvh) * cache.S_cap;
  Loader<D> ld;
  ld.init(cache, row0, blk0 + warp, lane);

  uint8_t* const ring = smem + warp * (Cf::NST * Cf::STAGE);
  const uint32_t ring_s = static_cast<uint32_t>(__cvta_generic_to_shared(ring));

  float oacc[D / 16][4];  // [M tile][c0..c3]: rows = channels, cols = heads 2*tid4, 2*tid4+1
  float zacc[NG][4];      // sum_tok B_g * z_g  (rows identical; [0], [1] are used)
#pragma unroll
  for (int i = 0; i < D / 16; ++i) oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f;
#pragma unroll
  for (int g = 0; g < NG; ++g) zacc[g][0] = zacc[g][1] = zacc[g][2] = zacc[g][3] = 0.f;
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
  const float cs = attn_scale * kLog2e * 16777216.0f;  // scores carry 2^-24 from the code operands

  // per-lane byte offsets inside a stage (everything else is a compile-time offset from these)
  const uint32_t k_lane = gid * Cf::PITCH + tid4 * 4;                          // K codes: token gid, word tid4
  const uint32_t v_lane = Cf::PK + (2 * tid4) * Cf::PITCH + (gid & 3) * 4;     // V codes: token 2*tid4, word gid%4
  const uint32_t ksz_lane = 2 * Cf::PK + gid * (NG * 2);                       // K scale row of token gid
  const uint32_t vsz_lane = 2 * Cf::PK + 2 * Cf::SZ + (2 * tid4) * (NG * 2);   // V scale rows of tokens 2*tid4, +1
  const uint32_t bsel0 = gid >> 2, bsel1 = 2 + (gid >> 2);  // byte of the word used for M-tile half 0 / 1
  const uint32_t sel0 = bsel0 | (bsel0 << 4) | ((4 + bsel0) << 8) | ((4 + bsel0) << 12);
  const uint32_t sel1 = bsel1 | (bsel1 << 4) | ((4 + bsel1) << 8) | ((4 + bsel1) << 12);

#pragma unroll
  for (int s = 0; s < Cf::NST - 1; ++s) {
    if (s < nblk) ld.issue(ring_s + s * Cf::STAGE);
    cp_async_commit();
  }

  int stage = 0;                    // stage consumed in this iteration
  int fill = Cf::NST - 1;           // stage filled in this iteration
  for (int k = 0; k < nblk; ++k) {
    cp_async_wait<Cf::NST - 2>();
    __syncwarp();
    if (k + Cf::NST - 1 < nblk) ld.issue(ring_s + fill * Cf::STAGE);
    cp_async_commit();
    fill = fill + 1 == Cf::NST ? 0 : fill + 1;
    const uint8_t* st = ring + stage * Cf::STAGE;
    stage = stage + 1 == Cf::NST ? 0 : stage + 1;
    const int valid = t1 - (blk0 + warp + k * kWarps) * kBlk;  // >= 16 except in the block holding the sequence end
    const bool tail = valid < kBlk;
    if (tail) {
      // rows past the end hold unspecified bytes: give them scale = zero = 0 so they dequantise to 0
      __half* sz = reinterpret_cast<__half*>(const_cast<uint8_t*>(st) + 2 * Cf::PK);
      for (int i = lane; i < 4 * kBlk * NG; i += 32) {
        const int tok = (i / NG) % kBlk;
        if (tok >= valid) sz[i] = __ushort_as_half(0);
      }
      __syncwarp();
    }

    // ---------------- scores: S[token][head] over this block's 16 tokens
    float sc[4] = {0.f, 0.f, 0.f, 0.f};
    {
      const uint8_t* kp = st + k_lane;
      // scales and zeros of tokens gid and gid + 8, all groups
      __half2 ks_lo[NG / 2], kz_lo[NG / 2], ks_hi[NG / 2], kz_hi[NG / 2];
      {
        const uint32_t* r = reinterpret_cast<const uint32_t*>(st + ksz_lane);
#pragma unroll
        for (int i = 0; i < NG / 2; ++i) {
          ks_lo[i] = u32_as_h2(r[i]);
          kz_lo[i] = u32_as_h2(r[Cf::SZ / 4 + i]);
          ks_hi[i] = u32_as_h2(r[8 * NG / 2 + i]);
          kz_hi[i] = u32_as_h2(r[Cf::SZ / 4 + 8 * NG / 2 + i]);
        }
      }
#pragma unroll
      for (int g = 0; g < NG; ++g) {
        const uint32_t w0 = *reinterpret_cast<const uint32_t*>(kp + g * 16);
        const uint32_t w8 = *reinterpret_cast<const uint32_t*>(kp + 8 * Cf::PITCH + g * 16);
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        mma16816(acc, w0 & kMaskLo, w8 & kMaskLo, w0 & kMaskHi, w8 & kMaskHi, qf[g][0], qf[g][1]);
        const uint32_t y0 = w0 >> 8, y8 = w8 >> 8;
        mma16816(acc, y0 & kMaskLo, y8 & kMaskLo, y0 & kMaskHi, y8 & kMaskHi, qf[g][2], qf[g][3]);
        const float s_lo = (g & 1) ? __high2float(ks_lo[g >> 1]) : __low2float(ks_lo[g >> 1]);
        const float z_lo = (g & 1) ? __high2float(kz_lo[g >> 1]) : __low2float(kz_lo[g >> 1]);
        const float s_hi = (g & 1) ? __high2float(ks_hi[g >> 1]) : __low2float(ks_hi[g >> 1]);
        const float z_hi = (g & 1) ? __high2float(kz_hi[g >> 1]) : __low2float(kz_hi[g >> 1]);
        sc[0] = fmaf(s_lo, fmaf(-z_lo, qs[g][0], acc[0]), sc[0]);
        sc[1] = fmaf(s_lo, fmaf(-z_lo, qs[g][1], acc[1]), sc[1]);
        sc[2] = fmaf(s_hi, fmaf(-z_hi, qs[g][0], acc[2]), sc[2]);
        sc[3] = fmaf(s_hi, fmaf(-z_hi, qs[g][1], acc[3]), sc[3]);
      }
    }
    // ---------------- online softmax (log2 domain)
    float a0 = sc[0] * cs, a1 = sc[1] * cs, a2 = sc[2] * cs, a3 = sc[3] * cs;
    if (tail) {
      if (gid >= valid) a0 = a1 = -INFINITY;
      if (gid + 8 >= valid) a2 = a3 = -INFINITY;
    }
    float bm0 = fmaxf(a0, a2), bm1 = fmaxf(a1, a3);
    const bool need = (bm0 > m0 + kRescaleThreshold) || (bm1 > m1 + kRescaleThreshold);
    if (__any_sync(0xffffffffu, need)) {
#pragma unroll
      for (int off = 4; off <= 16; off <<= 1) {
        bm0 = fmaxf(bm0, __shfl_xor_sync(0xffffffffu, bm0, off));
        bm1 = fmaxf(bm1, __shfl_xor_sync(0xffffffffu, bm1, off));
      }
      const float n0 = fmaxf(m0, bm0), n1 = fmaxf(m1, bm1);  // finite: every block has a valid token
      const float f0 = ex2(m0 - n0), f1 = ex2(m1 - n1);      // ex2(-inf) = 0 on the first block
      m0 = n0;
      m1 = n1;
      l0 *= f0;
      l1 *= f1;
#pragma unroll
      for (int i = 0; i < D / 16; ++i) {
        oacc[i][0] *= f0; oacc[i][1] *= f1; oacc[i][2] *= f0; oacc[i][3] *= f1;
      }
#pragma unroll
      for (int g = 0; g < NG; ++g) {
        zacc[g][0] *= f0; zacc[g][1] *= f1; zacc[g][2] *= f0; zacc[g][3] *= f1;
      }
    }
    const float p0 = ex2(a0 - m0), p1 = ex2(a1 - m1), p2 = ex2(a2 - m0), p3 = ex2(a3 - m1);  // ex2(-inf) = 0
    l0 += p0 + p2;
    l1 += p1 + p3;
    // P^T as B fragments: (tokens 2*tid4, 2*tid4+1 | head gid) and (tokens 8+2*tid4, 9+2*tid4 | head gid)
    const uint32_t pt0 = movmatrix_trans(h2_as_u32(__floats2half2_rn(p0, p1)));
    const uint32_t pt1 = movmatrix_trans(h2_as_u32(__floats2half2_rn(p2, p3)));

    // ---------------- P.V: O^T[channel][head] += V^T[channel][token] * (P * s)[token][head]
    {
      const uint8_t* vp = st + v_lane;
      // scales / zeros of tokens (2*tid4, 2*tid4+1) and (2*tid4+8, 2*tid4+9): NG halves per token
      uint32_t sAB[NG], sCD[NG], zAB[NG], zCD[NG];  // [0, NG/2) first token, [NG/2, NG) second token
      {
        const uint32_t* r = reinterpret_cast<const uint32_t*>(st + vsz_lane);
#pragma unroll
        for (int i = 0; i < NG; ++i) {
          sAB[i] = r[i];
          sCD[i] = r[8 * NG / 2 + i];
          zAB[i] = r[Cf::SZ / 4 + i];
          zCD[i] = r[Cf::SZ / 4 + 8 * NG / 2 + i];
        }
      }
#pragma unroll
      for (int g = 0; g < NG; ++g) {
        const uint32_t psel = (g & 1) ? 0x7632u : 0x5410u;
        const uint32_t b0 = h2_as_u32(__hmul2(u32_as_h2(pt0), u32_as_h2(__byte_perm(sAB[g >> 1], sAB[NG / 2 + (g >> 1)], psel))));
        const uint32_t b1 = h2_as_u32(__hmul2(u32_as_h2(pt1), u32_as_h2(__byte_perm(sCD[g >> 1], sCD[NG / 2 + (g >> 1)], psel))));
        const uint32_t zab = __byte_perm(zAB[g >> 1], zAB[NG / 2 + (g >> 1)], psel);
        const uint32_t zcd = __byte_perm(zCD[g >> 1], zCD[NG / 2 + (g >> 1)], psel);
        mma16816(zacc[g], zab, zab, zcd, zcd, b0, b1);
        const uint32_t wA = *reinterpret_cast<const uint32_t*>(vp + g * 16);
        const uint32_t wB = *reinterpret_cast<const uint32_t*>(vp + Cf::PITCH + g * 16);
        const uint32_t wC = *reinterpret_cast<const uint32_t*>(vp + 8 * Cf::PITCH + g * 16);
        const uint32_t wD = *reinterpret_cast<const uint32_t*>(vp + 9 * Cf::PITCH + g * 16);
        uint32_t u = __byte_perm(wA, wB, sel0), u2 = __byte_perm(wC, wD, sel0);
        mma16816(oacc[2 * g], u & kMaskLo, u & kMaskHi, u2 & kMaskLo, u2 & kMaskHi, b0, b1);
        u = __byte_perm(wA, wB, sel1);
        u2 = __byte_perm(wC, wD, sel1);
        mma16816(oacc[2 * g + 1], u & kMaskLo, u & kMaskHi, u2 & kMaskLo, u2 & kMaskHi, b0, b1);
      }
    }
  }
  cp_async_wait<0>();

  // ---------------- per-warp result -> shared, merge the warps, write the normalised partial
#pragma unroll
  for (int off = 4; off <= 16; off <<= 1) {
    l0 += __shfl_xor_sync(0xffffffffu, l0, off);
    l1 += __shfl_xor_sync(0xffffffffu, l1, off);
  }
  __syncthreads();  // every warp is done with its ring; the memory is reused below
  float* mo = reinterpret_cast<float*>(smem) + warp * (8 * D + 16);  // [D channels][8 heads] then m[8], l[8]
#pragma unroll
  for (int mt = 0; mt < D / 16; ++mt) {
    const int g = mt >> 1;
    const int ch = 32 * g + 8 * (gid & 3) + 2 * (2 * (mt & 1) + (gid >> 2));
    // even channel: codes carried 2^-24; odd channel (high nibble): 2^-20
    *reinterpret_cast<float2*>(mo + ch * 8 + 2 * tid4) =
        make_float2(oacc[mt][0] * 16777216.0f - zacc[g][0], oacc[mt][1] * 16777216.0f - zacc[g][1]);
    *reinterpret_cast<float2*>(mo + (ch + 1) * 8 + 2 * tid4) =
        make_float2(oacc[mt][2] * 1048576.0f - zacc[g][0], oacc[mt][3] * 1048576.0f - zacc[g][1]);
  }
  if (gid == 0) {
    mo[8 * D + 2 * tid4] = m0;
    mo[8 * D + 2 * tid4 + 1] = m1;
    mo[8 * D + 8 + 2 * tid4] = l0;
    mo[8 * D + 8 + 2 * tid4 + 1] = l1;
  }
  __syncthreads();
  const float* all = reinterpret_cast<const float*>(smem);
  for (int idx = threadIdx.x; idx < 8 * D; idx += kThreads) {
    const int x = idx >> 3, h = idx & 7;  // consecutive threads take consecutive heads of one channel
    if (h >= nh) continue;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) M = fmaxf(M, all[w * (8 * D + 16) + 8 * D + h]);
    float num = 0.f, den = 0.f;
    if (M > -INFINITY) {
#pragma unroll
      for (int w = 0; w < kWarps; ++w) {
        const float* wb = all + w * (8 * D + 16);
        const float f = ex2(wb[8 * D + h] - M);  // ex2(-inf) = 0 for a warp that saw no token
        num = fmaf(f, wb[idx], num);
        den = fmaf(f, wb[8 * D + 8 + h], den);
      }
    }
    const long long pidx = (static_cast<long long>(b) * H_q + h0 + h) * C + c;
    o_part[pidx * D + x] = den > 0.f ? num / den : 0.f;
    if (x == 0) {
      m_part[pidx] = M * kLn2;  // natural-log units of attn_scale * q.k^
      l_part[pidx] = den;
    }
  }
}

template <int D>
cudaError_t launch(const tq_kv_cache& c, const __half* q, int H_q, float attn_scale, int C, float* o_part,
                   float* m_part, float* l_part, int32_t* status, cudaStream_t st) {
  const cudaError_t attr = cudaFuncSetAttribute(decode_mma_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                Cfg<D>::SMEM);
  if (attr != cudaSuccess) return attr;
  const int G = H_q / c.H_kv;
  dim3 grid(C, c.H_kv * ((G + 7) / 8), c.B);
  decode_mma_kernel<D><<<grid, kThreads, Cfg<D>::SMEM, st>>>(c, q, H_q, attn_scale, C, o_part, m_part, l_part, status);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_decode_mma(const tq_kv_cache& c, const __half* q, int H_q, float attn_scale, int C, float* o_part,
                              float* m_part, float* l_part, int32_t* status, cudaStream_t st) {
  switch (c.d) {
    case 64: return launch<64>(c, q, H_q, attn_scale, C, o_part, m_part, l_part, status, st);
    case 128: return launch<128>(c, q, H_q, attn_scale, C, o_part, m_part, l_part, status, st);
    default: return launch<256>(c, q, H_q, attn_scale, C, o_part, m_part, l_part, status, st);
  }
}

}  // namespace tq
