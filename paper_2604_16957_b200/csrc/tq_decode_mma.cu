// Fused int4 decode attention, phase 1 (Sec. 3.1 Algorithm 1 per split, Sec. 3.2), for sm_100a.
//
// One thread block handles one (sequence, KV head, tile of up to 8 query heads, split); with several
// query tokens per sequence the tile holds (query token, head) pairs.  The query heads that share the
// KV head are packed into the N = 8 dimension of mma.sync.m16n8k16, so every byte of the cache is read
// from HBM once per head tile.  The path is HBM-bound.  The cache is stored in 16-token blocks that are
// already in the shared-memory layout this kernel wants (tq.h), so a stage is filled by ONE bulk
// asynchronous copy (cp.async.bulk, the TMA unit) of a contiguous 2560-byte block (d = 128) issued by
// one lane and completing on the stage's mbarrier.  Each warp owns a ring of 4 stages (3 in the second
// shared-memory layout, see Layout) and its tokens end to end, so the main loop has no block-wide barrier.  (Head dimensions 256 and 512 are split over
// teams of 2 and 4 warps that share a ring and exchange their partial scores once per token block.)
// Measured on the 128K Llama-shaped layer, the copies alone take 27.9 us with bulk copies against
// 30.2 us with 16-byte cp.async.  The tensor cores only take the G-packed q.K^T and P.V contractions
// off the CUDA cores, which could not keep up with the memory system otherwise.
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
//   * Warps that own 128 channels (d >= 128) do both zero-point terms with ONE MMA each, on exact fp16
//     (hi, lo) pairs of s * z (block_scores, block_softmax_pv); a spare row of the P.V one yields the softmax
//     denominator; the upper byte of a V code word enters as one operand, n2 + 16 n3, beside n2 alone.
// Timing probes (evidence for where a launch's time goes; never used by the library itself): compiling this
// file with -DTQ_PROBE_COPIES_ONLY leaves the copies and their waits but drops the arithmetic of the full
// blocks; -DTQ_PROBE_MATH_ONLY keeps the arithmetic but stops waiting for and issuing copies after the first
// three.  `python -m paper_2604_16957_b200.build --probe copies|math` builds them as separate libraries whose
// results are meaningless and whose version string says "probe".
//
// Softmax is online in the log2 domain with a lazily updated running maximum (the maximum is
// raised only when a score exceeds it by more than 2^4, which keeps P <= 16 in fp16 and makes
// the rescale of the accumulators rare).
//
// Shared-memory layout of one stage (16 tokens of one KV head):
//   K codes [16][D/2] | V codes [16][D/2] | K scale [D/32][16] | K zero | V scale | V zero
// The 16-byte chunks of the code rows are XOR-swizzled with the token index, which makes the
// fragment loads conflict free (a padded layout was measured too: it costs 3-4x the shared-memory
// wavefronts on the way in).  Fragments come from ldmatrix, whose 8x8 b16 "matrix" is here 8 tokens x
// one 16-byte chunk (32 codes of one group):
//   K: plain ldmatrix  -> lane (gid, tid4) holds word tid4 of token gid: 8 codes of one token,
//      the A operand rows of the score MMA;
//   V: ldmatrix.trans  -> lane (gid, tid4) holds 16-bit lane gid of tokens 2*tid4 and 2*tid4+1
//      side by side: the token-pair interleave the P.V MMA needs (k = tokens), done by the
//      load itself, so V needs no byte permutes.
#include "tq_async.cuh"
#include "tq_internal.cuh"
#include "tq_quantize_core.cuh"

namespace tq {
namespace {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kBlk = 16;              // tokens per stage = MMA M (scores) = MMA K (P.V)
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 4.0f;  // log2 units
constexpr int kWinSlack = TQ_WINDOW_SLACK;  // tokens a windowed overlapped step may find beyond its stable part
constexpr float kNoMax = -1.0e30f;         // running reference before any token was seen
constexpr uint32_t kMaskLo = 0x000F000Fu;  // nibbles 0 / 4 of a 32-bit word: n * 2^-24 as fp16
constexpr uint32_t kMaskHi = 0x00F000F0u;  // nibbles 1 / 5: n * 2^-20 as fp16

template <int D>
struct Cfg {
  static constexpr int NG = D / 32;                 // groups per row == 16-byte chunks per code row
  static constexpr int ROWB = D / 2;                // bytes per code row in global memory
  static constexpr int PK = kBlk * ROWB;            // code bytes per stage, K or V
  static constexpr int SWZ_SHIFT = NG == 2 ? 2 : (NG == 4 ? 1 : 0);  // chunk' = chunk ^ ((tok >> SHIFT) & (NG - 1))
  static constexpr int SZ = kBlk * NG * 2;          // bytes of one scale or zero array per stage
  static constexpr int STAGE = 2 * PK + 4 * SZ;     // 1280 / 2560 / 5120 / 10240 bytes
  // Head dimensions above 128 are split over DS warps (a "team") that work on the same token block, each
  // on DW = 128 channels: the accumulators of one warp stay within 128 registers per thread, so two
  // blocks fit an SM at every head dimension.  A team owns one ring; the kernel has NTEAM teams.
  static constexpr int DS = D <= 128 ? 1 : D / 128;
  static constexpr int DW = D / DS;                 // channels per warp
  static constexpr int NGW = DW / 32;               // groups per warp
  static constexpr int NTEAM = kWarps / DS;
  static constexpr int MINB = 2;                    // resident blocks per SM
  static_assert(STAGE == TQ_BLOCK_BYTES(D), "a stage is one cache block");
  static_assert(kWarps % DS == 0, "teams tile the block");
  __host__ __device__ static constexpr int swz(int tok) { return (tok >> SWZ_SHIFT) & (NG - 1); }
};

// Shared memory of one thread block.  Two layouts:
//  * SEP = false: rings of four stages; the merge arrays of the epilogue and the weights of the fused step's
//    reduction reuse the rings' memory once every warp is done with its ring (80 KB at d >= 128).
//  * SEP = true (d = 128): rings of three stages and merge arrays of their own beside them (93 KB; only the
//    reduction's weights still reuse the rings), so a warp that has finished its blocks stores its rows without
//    first waiting for the other warps' rings to drain.  Measured: 0.3 - 0.5 us less per 128K layer and per 32K
//    step; but three stages cost a batch that runs in several waves 1.5 %, and a footprint above 98 KB (two
//    blocks then need the largest shared-memory carve-out) costs a short step 0.5 us, so the weights stay in the
//    rings and the launch takes this layout only for long splits that run in one wave.
template <int D, bool SEP>
struct Layout {
  using Cf = Cfg<D>;
  static_assert(!SEP || D == 128, "the separate merge arrays fit beside the rings at d = 128 only");
  static constexpr int NTEAM = Cf::NTEAM, DS = Cf::DS;
  static constexpr int NST = SEP ? 3 : 4;           // stages in a ring
  static constexpr int PIPE = NTEAM * NST * Cf::STAGE;  // 40 KB (D = 64), 60 or 80 KB (D = 128), 80 KB otherwise
  static constexpr int MERGE = (NTEAM * 16 + NTEAM * 8 * D) * 4;  // merge arrays of the epilogue
  static constexpr int BARS = SEP ? PIPE : (PIPE > MERGE ? PIPE : MERGE);  // offset of the mbarriers: [NTEAM][NST] x 8 bytes
  static constexpr int XCH = BARS + NTEAM * NST * 8;        // score exchange of the teams: [NTEAM][2][DS][32] float4 + flags
  static constexpr int XCH_TEAM = DS > 1 ? 2 * DS * 32 * 16 + 2 * DS * 4 : 0;
  static constexpr int MERGE_OFF = SEP ? XCH + NTEAM * XCH_TEAM : 0;
  static constexpr int WTS = SEP ? 0 : (MERGE + 15) & ~15;  // weights of the fused step's reduction (inside the rings)
  static constexpr int WTS_BYTES = 8 * TQ_MAX_SPLITS * 4 + 16 + 8 * 4;  // [8 heads][splits] + ticket + 1 / denominators
  static constexpr int SMEM = SEP ? MERGE_OFF + MERGE : XCH + NTEAM * XCH_TEAM;
  static_assert(XCH % 16 == 0 && SMEM % 8 == 0, "alignment of the exchange arrays and the page addresses");
  static_assert(WTS + WTS_BYTES <= PIPE, "the weights fit the rings");
};

__device__ __forceinline__ void mma16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// d = a * b + z where z is a quad of registers that hold zero (kept apart from d so that no
// accumulator has to be cleared)
__device__ __forceinline__ void mma16816_first(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1, const float (&z)[4]) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%11,%12,%13};\n"
      : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(z[0]), "f"(z[1]), "f"(z[2]), "f"(z[3]));
}

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(d) : "r"(a));
  return d;
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}

// bytes 1 and 3 of w moved to bytes 0 and 2, the others cleared: (w >> 8) & 0x00FF00FF in one instruction
__device__ __forceinline__ uint32_t upper_bytes(uint32_t w) { return __byte_perm(w, 0u, 0x4341); }
__device__ __forceinline__ uint32_t h2_as_u32(__half2 h) { return *reinterpret_cast<uint32_t*>(&h); }
__device__ __forceinline__ __half2 u32_as_h2(uint32_t u) { return *reinterpret_cast<__half2*>(&u); }

template <int D>
struct WarpCtx {
  uint32_t kaddr[Cfg<D>::NGW / 2];  // ldmatrix row address this lane supplies (slot 0 of the warp's ring), per K load; V: + PK
  uint32_t ksz_lane, vsz_lane;
  uint32_t vz_lane, vs2_lane;  // row addresses of the V scale / zero load of the zero-point MMA and of the scale loads
  uint32_t kz_lane;            // row address of the scale / zero load that feeds the zero-point MMA of the scores
  uint32_t keep;               // all ones, except 0 in the lanes of row 4 of the P.V zero-point MMA (see block_softmax_pv)
  float cs0, cs1;              // score -> log2 units of the softmax for the thread's two columns (heads 2*tid4, 2*tid4+1)
  int gid;
};
template <int D> struct KZ { static constexpr bool on = Cfg<D>::NGW == 4; };  // every warp that works on 128 channels

// Which tokens of a block count, as rows relative to the block's first token.  Rows >= zrow lie past the
// end of the sequence and hold unspecified bytes; column j (j = 0, 1: the thread's two score columns, i.e.
// query heads 2*tid4 + j of the tile) attends rows lo[j] <= row < hi[j].
struct RowMask {
  int zrow, lo0, hi0, lo1, hi1;
};

// First half of one 16-token block: this warp's share of the scores S[token][head] (over its DW channels;
// they carry a factor 2^-24).  TAIL = a block in which some token does not count for some column.
template <int D, bool TAIL>
__device__ __forceinline__ void block_scores(const WarpCtx<D>& cx, const uint8_t* st, uint32_t st_off, const RowMask& mk,
                                             const uint32_t (&qf)[Cfg<D>::NGW][4], const float (&qs)[Cfg<D>::NGW][2],
                                             const uint32_t (&qz)[2],
                                             const float (&zero4)[4], float (&sc)[4]) {
  using Cf = Cfg<D>;
  constexpr int NGW = Cf::NGW;
  if (TAIL) {
    // rows past the end hold unspecified bytes: give them scale = zero = 0 so they dequantise to 0
    // (every warp of a team clears all of them before its own reads; the stores are idempotent)
    __half* sz = reinterpret_cast<__half*>(const_cast<uint8_t*>(st) + 2 * Cf::PK);
    const int lane = threadIdx.x & 31;
    for (int i = lane; i < 4 * kBlk * Cf::NG; i += 32) {
      if ((i % kBlk) >= mk.zrow) sz[i] = __ushort_as_half(0);  // arrays are [group][16 tokens]
    }
    __syncwarp();
  }
  // matrix j = 4 * i + m of load i is (group j / 2 of this warp, tokens 8 * (j % 2) ..), as for V below
  uint32_t kw[NGW / 2][4], ksz[4];
#pragma unroll
  for (int i = 0; i < NGW / 2; ++i) ldmatrix_x4(kw[i], cx.kaddr[i] + st_off);
  if constexpr (KZ<D>::on) {
    // Zero-point term of the scores by one MMA: sum_g (s_g z_g) * qsum_g with the product s * z split
    // exactly into an fp16 pair (hi = rn(s z), lo = s z - hi by a fused multiply-add) and qsum into
    // hi + lo as well.  k slots 0-7 carry the hi parts of groups 0 1 2 3 0 1 2 3, slots 8-15 the lo parts in
    // the same order; the B rows (qz, the same register for both halves) hold the hi parts of the group sums in
    // slots 0-3 and 8-11 and their lo parts in 4-7 and 12-15: hi x hi + hi x lo + lo x hi + lo x lo.
    // The transposing load hands lane (gid, tid4) the half2 (x[g][token], x[g+1][token]) of groups
    // g = 2 * (tid4 & 1): scales of tokens gid, gid + 8, then zeros of the same.
    uint32_t r[4];
    ldmatrix_x4_trans(r, cx.kz_lane + st_off);
    const __half2 pa = __hmul2(u32_as_h2(r[0]), u32_as_h2(r[2])), pb = __hmul2(u32_as_h2(r[1]), u32_as_h2(r[3]));
    const uint32_t la = h2_as_u32(__hfma2(u32_as_h2(r[0]), u32_as_h2(r[2]), __hneg2(pa)));
    const uint32_t lb = h2_as_u32(__hfma2(u32_as_h2(r[1]), u32_as_h2(r[3]), __hneg2(pb)));
    float accz[4];
    mma16816_first(accz, h2_as_u32(pa), h2_as_u32(pb), la, lb, qz[0], qz[0], zero4);
    // scales of all four groups for tokens gid, gid + 8: matrices (g0 g1 | tokens 0-7), (g0 g1 | 8-15), (g2 g3 | ..)
    ldmatrix_x4_trans(ksz, cx.ksz_lane + st_off);
    // (q was scaled so that this term and the code terms below carry the same power of two: no multiply here)
    sc[0] = accz[0]; sc[1] = accz[1]; sc[2] = accz[2]; sc[3] = accz[3];
#pragma unroll
    for (int g = 0; g < NGW; ++g) {
      const uint32_t w0 = kw[g / 2][2 * (g % 2)];                // token gid
      const uint32_t w8 = kw[g / 2][2 * (g % 2) + 1];            // token gid + 8
      float acc[4];
      mma16816_first(acc, w0 & kMaskLo, w8 & kMaskLo, w0 & kMaskHi, w8 & kMaskHi, qf[g][0], qf[g][1], zero4);
      // (The whole-byte operand of the P.V side is not used here: paired with q3 / 16 it needs q2 - q3 / 16 for
      // nibble 2, whose fp16 rounding reaches the scores -- measured 1e-3 relative L2 at 64K, 1.8e-3 worst head.)
      const uint32_t y0 = w0 >> 8, y8 = w8 >> 8;
      mma16816(acc, y0 & kMaskLo, y8 & kMaskLo, y0 & kMaskHi, y8 & kMaskHi, qf[g][2], qf[g][3]);
      const __half2 slo = u32_as_h2(ksz[2 * (g / 2)]), shi = u32_as_h2(ksz[2 * (g / 2) + 1]);
      const float s_lo = (g & 1) ? __high2float(slo) : __low2float(slo);
      const float s_hi = (g & 1) ? __high2float(shi) : __low2float(shi);
      sc[0] = fmaf(s_lo, acc[0], sc[0]); sc[1] = fmaf(s_lo, acc[1], sc[1]);
      sc[2] = fmaf(s_hi, acc[2], sc[2]); sc[3] = fmaf(s_hi, acc[3], sc[3]);
    }
  } else {
#pragma unroll
  for (int g = 0; g < NGW; ++g) {
    const uint32_t w0 = kw[g / 2][2 * (g % 2)];                // token gid
    const uint32_t w8 = kw[g / 2][2 * (g % 2) + 1];            // token gid + 8
    float acc[4];
    mma16816_first(acc, w0 & kMaskLo, w8 & kMaskLo, w0 & kMaskHi, w8 & kMaskHi, qf[g][0], qf[g][1], zero4);
    const uint32_t y0 = w0 >> 8, y8 = w8 >> 8;
    mma16816(acc, y0 & kMaskLo, y8 & kMaskLo, y0 & kMaskHi, y8 & kMaskHi, qf[g][2], qf[g][3]);
    // Scales and zeros of tokens gid and gid + 8 for groups g, g+1 by one transposing ldmatrix: its
    // matrices are (scale | tokens 0-7), (scale | 8-15), (zero | 0-7), (zero | 8-15), each with rows
    // alternating between the 16-byte chunks of groups g and g+1, so every lane receives element gid
    // of both chunks: half2 (x[g][token], x[g+1][token]).
    if ((g & 1) == 0) ldmatrix_x4_trans(ksz, cx.ksz_lane + st_off + 32 * g);
    const float s_lo = (g & 1) ? __high2float(u32_as_h2(ksz[0])) : __low2float(u32_as_h2(ksz[0]));
    const float s_hi = (g & 1) ? __high2float(u32_as_h2(ksz[1])) : __low2float(u32_as_h2(ksz[1]));
    const float z_lo = (g & 1) ? __high2float(u32_as_h2(ksz[2])) : __low2float(u32_as_h2(ksz[2]));
    const float z_hi = (g & 1) ? __high2float(u32_as_h2(ksz[3])) : __low2float(u32_as_h2(ksz[3]));
    const float t0 = fmaf(-z_lo, qs[g][0], acc[0]), t1 = fmaf(-z_lo, qs[g][1], acc[1]);
    const float t2 = fmaf(-z_hi, qs[g][0], acc[2]), t3 = fmaf(-z_hi, qs[g][1], acc[3]);
    if (g == 0) {
      sc[0] = s_lo * t0; sc[1] = s_lo * t1; sc[2] = s_hi * t2; sc[3] = s_hi * t3;
    } else {
      sc[0] = fmaf(s_lo, t0, sc[0]); sc[1] = fmaf(s_lo, t1, sc[1]);
      sc[2] = fmaf(s_hi, t2, sc[2]); sc[3] = fmaf(s_hi, t3, sc[3]);
    }
  }
  }
}

// A operand of the zero-point MMA of P.V (see block_softmax_pv): does not depend on the scores, so a team
// computes it while it waits for its partner's partial scores.
template <int D>
__device__ __forceinline__ void pv_zero_operands(const WarpCtx<D>& cx, uint32_t st_off, uint32_t (&zop)[4]) {
  uint32_t r[4];
  ldmatrix_x4(r, cx.vz_lane + st_off);
  const __half2 pa = __hmul2(u32_as_h2(r[0]), u32_as_h2(r[2])), pb = __hmul2(u32_as_h2(r[1]), u32_as_h2(r[3]));
  zop[1] = h2_as_u32(__hfma2(u32_as_h2(r[0]), u32_as_h2(r[2]), __hneg2(pa)));
  zop[3] = h2_as_u32(__hfma2(u32_as_h2(r[1]), u32_as_h2(r[3]), __hneg2(pb)));
  // Rows 4-7 repeat the groups of rows 0-3 and are not read back, so row 4 is given ones instead: its
  // accumulators become sum_tok fp16(P)[tok][head], the softmax denominator (of exactly the weights the
  // numerator uses), at no instruction beyond the two selects.
  constexpr uint32_t kOnes = 0x3C003C00u;  // half2 (1, 1)
  zop[0] = (h2_as_u32(pa) & cx.keep) | (~cx.keep & kOnes);
  zop[2] = (h2_as_u32(pb) & cx.keep) | (~cx.keep & kOnes);
}

// Second half: online softmax on the complete scores, then P.V for this warp's DW output channels.
// PRE: the zero-point operands were computed by the caller (pv_zero_operands).
template <int D, bool TAIL, bool PRE = false>
__device__ __forceinline__ void block_softmax_pv(const WarpCtx<D>& cx, uint32_t st_off, const RowMask& mk,
                                                 const float (&sc)[4], float (&oacc)[Cfg<D>::DW / 16][4],
                                                 float (&zacc)[Cfg<D>::NGW][4], float& m0, float& m1, float& l0,
                                                 float& l1, const uint32_t* pre = nullptr) {
  constexpr int NGW = Cfg<D>::NGW;
  // ---------------- online softmax in the log2 domain.  d = score - running reference m; the
  // reference is raised only when some d exceeds the threshold, so the common path is 4 FMAs.
  float d0 = fmaf(sc[0], cx.cs0, -m0), d1 = fmaf(sc[1], cx.cs1, -m1);
  float d2 = fmaf(sc[2], cx.cs0, -m0), d3 = fmaf(sc[3], cx.cs1, -m1);
  // rows gid (d0, d1) and gid + 8 (d2, d3); columns 0 (d0, d2) and 1 (d1, d3)
  const bool off0 = TAIL && (cx.gid < mk.lo0 || cx.gid >= mk.hi0), off1 = TAIL && (cx.gid < mk.lo1 || cx.gid >= mk.hi1);
  const bool off2 = TAIL && (cx.gid + 8 < mk.lo0 || cx.gid + 8 >= mk.hi0);
  const bool off3 = TAIL && (cx.gid + 8 < mk.lo1 || cx.gid + 8 >= mk.hi1);
  if (TAIL) {
    if (off0) d0 = -INFINITY;
    if (off1) d1 = -INFINITY;
    if (off2) d2 = -INFINITY;
    if (off3) d3 = -INFINITY;
  }
  const bool need = fmaxf(fmaxf(d0, d2), fmaxf(d1, d3)) > kRescaleThreshold;
  if (__any_sync(0xffffffffu, need)) {
    float a0 = sc[0] * cx.cs0, a1 = sc[1] * cx.cs1, a2 = sc[2] * cx.cs0, a3 = sc[3] * cx.cs1;
    if (TAIL) {
      if (off0) a0 = -INFINITY;
      if (off1) a1 = -INFINITY;
      if (off2) a2 = -INFINITY;
      if (off3) a3 = -INFINITY;
    }
    float bm0 = fmaxf(a0, a2), bm1 = fmaxf(a1, a3);
#pragma unroll
    for (int off = 4; off <= 16; off <<= 1) {
      bm0 = fmaxf(bm0, __shfl_xor_sync(0xffffffffu, bm0, off));
      bm1 = fmaxf(bm1, __shfl_xor_sync(0xffffffffu, bm1, off));
    }
    const float n0 = fmaxf(m0, bm0), n1 = fmaxf(m1, bm1);
    const float f0 = ex2(m0 - n0), f1 = ex2(m1 - n1);  // m starts at -1e30: the first factor underflows to 0
    m0 = n0;
    m1 = n1;
    if constexpr (!KZ<D>::on) {
      l0 *= f0;
      l1 *= f1;
    }
#pragma unroll
    for (int i = 0; i < Cfg<D>::DW / 16; ++i) {
      oacc[i][0] *= f0; oacc[i][1] *= f1; oacc[i][2] *= f0; oacc[i][3] *= f1;
    }
    if constexpr (KZ<D>::on) {  // one accumulator quad for all groups: hi sums in [0], [1], lo sums in [2], [3]
      zacc[0][0] *= f0; zacc[0][1] *= f1; zacc[0][2] *= f0; zacc[0][3] *= f1;
    } else {
#pragma unroll
      for (int g = 0; g < NGW; ++g) {
        zacc[g][0] *= f0; zacc[g][1] *= f1;
      }
    }
    d0 = a0 - m0; d1 = a1 - m1; d2 = a2 - m0; d3 = a3 - m1;
  }
  const float p0 = ex2(d0), p1 = ex2(d1), p2 = ex2(d2), p3 = ex2(d3);  // ex2(-inf) = 0 for masked tokens
  if constexpr (!KZ<D>::on) {  // (otherwise the denominator comes out of the zero-point MMA below)
    l0 += p0 + p2;
    l1 += p1 + p3;
  }
  // P^T as B fragments: (tokens 2*tid4, 2*tid4+1 | head gid) and (tokens 8+2*tid4, 9+2*tid4 | head gid)
  const uint32_t pt0 = movmatrix_trans(h2_as_u32(__floats2half2_rn(p0, p1)));
  const uint32_t pt1 = movmatrix_trans(h2_as_u32(__floats2half2_rn(p2, p3)));

  // ---------------- P.V: O^T[channel][head] += V^T[channel][token] * (P * s)[token][head]
  // matrix j = 4 * i + m of load i is (group j / 2 of this warp, tokens 8 * (j % 2) ..)
  uint32_t vw[4];
  if constexpr (KZ<D>::on) {
    // Zero-point term of all four groups by ONE MMA (instead of one per group): sum_tok (s z)[tok][g] * P[tok][head]
    // with the product s * z split exactly into an fp16 pair -- hi = rn(s z) in rows 0-7 (row r: group r & 3),
    // lo = fma(s, z, -hi) in rows 8-15, so the accumulator quad holds the hi sums in [0], [1] and the lo sums
    // in [2], [3] -- and B = fp16(P), the operand the scaled B_g below are made from.  (The code term sees fp16(fp16(P) * s), the
    // zero term the unrounded product: the two no longer cancel rounding for rounding, which costs about a
    // factor 1.6 in output error, inside the tolerance; it saves three MMAs and eight shared-memory wavefronts
    // per block, 1.2 us per 128K layer when the kernel runs against the power limit.)
    uint32_t zop[4];
    if constexpr (PRE) {
      zop[0] = pre[0]; zop[1] = pre[1]; zop[2] = pre[2]; zop[3] = pre[3];
    } else {
      pv_zero_operands<D>(cx, st_off, zop);
    }
    mma16816(zacc[0], zop[0], zop[1], zop[2], zop[3], pt0, pt1);
    uint32_t vs[4];
#pragma unroll
    for (int g = 0; g < NGW; ++g) {
      // scales of token pairs (2*tid4, +1) and (2*tid4+8, +9) for groups g, g+1 by one load of four matrices
      // whose eight rows are each one and the same 16-byte chunk
      if ((g & 1) == 0) ldmatrix_x4(vs, cx.vs2_lane + st_off + 32 * g);
      const uint32_t b0 = h2_as_u32(__hmul2(u32_as_h2(pt0), u32_as_h2(vs[2 * (g & 1)])));
      const uint32_t b1 = h2_as_u32(__hmul2(u32_as_h2(pt1), u32_as_h2(vs[2 * (g & 1) + 1])));
      if ((g & 1) == 0) ldmatrix_x4_trans(vw, cx.kaddr[g / 2] + st_off + Cfg<D>::PK);
      const uint32_t r1 = vw[2 * (g % 2)], r2 = vw[2 * (g % 2) + 1];
      mma16816(oacc[2 * g], r1 & kMaskLo, r1 & kMaskHi, r2 & kMaskLo, r2 & kMaskHi, b0, b1);
      // upper bytes: rows 0-7 take nibble 2 alone, rows 8-15 the whole byte n2 + 16 n3 (still an exact fp16
      // subnormal); the epilogue takes the difference of the two fp32 accumulators.  One permute and one
      // mask per register instead of a shift and two masks.
      const uint32_t y1 = upper_bytes(r1), y2 = upper_bytes(r2);
      mma16816(oacc[2 * g + 1], y1 & kMaskLo, y1, y2 & kMaskLo, y2, b0, b1);
    }
  } else {
#pragma unroll
  for (int g = 0; g < NGW; ++g) {
    // Scales / zeros of token pairs (2*tid4, 2*tid4+1) and (2*tid4+8, 2*tid4+9) of group g: an ldmatrix
    // whose eight row addresses are equal hands every lane word tid4 of that 16-byte chunk; the four
    // matrices are (zero | tokens 0-7), (scale | 0-7), (zero | 8-15), (scale | 8-15).  In that order the
    // four result registers are, as they stand, the A operand of the zero-point MMA: rows 0-7 hold z_g
    // (c0, c1 accumulate sum_tok z_g * B_g), rows 8-15 hold the scales and produce values never read.
    uint32_t vsz[4];
    ldmatrix_x4(vsz, cx.vsz_lane + st_off + 32 * g);
    const uint32_t b0 = h2_as_u32(__hmul2(u32_as_h2(pt0), u32_as_h2(vsz[1])));
    const uint32_t b1 = h2_as_u32(__hmul2(u32_as_h2(pt1), u32_as_h2(vsz[3])));
    mma16816(zacc[g], vsz[0], vsz[1], vsz[2], vsz[3], b0, b1);
    // r1 = (tokens 2*tid4, 2*tid4+1), r2 = (tokens 2*tid4+8, +9): 16-bit lane gid of chunk g, i.e. codes of
    // channels 32g + 4*gid .. +3 of two tokens side by side
    if ((g & 1) == 0) ldmatrix_x4_trans(vw, cx.kaddr[g / 2] + st_off + Cfg<D>::PK);
    const uint32_t r1 = vw[2 * (g % 2)], r2 = vw[2 * (g % 2) + 1];
    mma16816(oacc[2 * g], r1 & kMaskLo, r1 & kMaskHi, r2 & kMaskLo, r2 & kMaskHi, b0, b1);
    const uint32_t y1 = upper_bytes(r1), y2 = upper_bytes(r2);  // see the four-group form above
    mma16816(oacc[2 * g + 1], y1 & kMaskLo, y1, y2 & kMaskLo, y2, b0, b1);
  }
  }
}

// Row mask of a block that holds an end of some column's token range (general form).  Masked blocks are
// rare, so this is a real call: whatever it needs is recomputed from the launch arguments instead of
// being kept in registers across the block loop.  `col` = the thread's first score column in the KV head,
// `first` = the block's first token.
__device__ __noinline__ RowMask general_row_mask(const int32_t* seq_lens, int b, int S_cap, int S_q, int window, int C,
                                                 int c, int G, int col, int first, int len_known) {
  // (the fused step passes the length it works with: the one in memory is advanced by another thread block meanwhile)
  const int n = len_known >= 0 ? len_known : checked_len(seq_lens, b, S_cap, nullptr);
  int a, e;  // this split's token range, as at the top of the kernel
  split_range(query_lo(n, S_q, 0, window), n, C, c, a, e);
  const int s0 = min(col / G, S_q - 1), s1 = min((col + 1) / G, S_q - 1);
  const int hi0 = query_hi(n, S_q, s0), hi1 = query_hi(n, S_q, s1);
  return RowMask{e - first, window_begin(hi0, window) - first, min(hi0, e) - first, window_begin(hi1, window) - first,
                 min(hi1, e) - first};
}

// What the fused decode step (tq_sdpa_int4_step) adds to phase 1; all null for the plain calls.
struct StepArgs {
  const __half* k_new;  // [B][H_kv][1][D]: quantised and appended by the last split of each KV head (null: no append)
  const __half* v_new;
  void* out;            // [B][H_q][D]: written by the last block to finish of each (sequence, KV head) (null: no reduction)
  int out_fp32;
  int32_t* counters;    // [B * H_kv] arrivals, then [B] length readers; zero between launches
  const int32_t* stable_lens;  // [B] device: per-sequence stable part in tokens, instead of the launch argument (null: not used)
  // instrumented instantiation only (the library's own tests, see TestHooks): poll limit of the stage waits in
  // SM cycles, and the 16-token block of each (sequence, KV head) whose copy announces 16 bytes too many, so
  // that its barrier never completes although the data lands
  int wait_cycles, fault_blk;
};

// Fused step: one warp quantises the new token's K and V rows of one KV head (Eq. 2-3) into row `row` of the
// cache block `blk`.  Out of line: its registers are not the block loop's.
template <int D>
__device__ __noinline__ void quantize_new_row(uint8_t* blk, int row, const __half* k_row, const __half* v_row) {
  const int lane = threadIdx.x & 31;
  constexpr int CPR = D / 8;  // 8-element chunks per row; K chunks first, then V
#pragma unroll
  for (int i0 = 0; i0 < 2 * CPR; i0 += 32) {
    const int i = i0 + lane;
    const bool on = i < 2 * CPR;
    const int which = i >= CPR ? 1 : 0, cc = i - which * CPR;
    uint4 raw = make_uint4(0, 0, 0, 0);
    if (on) raw = *reinterpret_cast<const uint4*>((which ? v_row : k_row) + cc * 8);
    uint32_t word;
    __half sq, zq;
    quantize_chunk(raw, word, sq, zq);
    if (on) {
      *reinterpret_cast<uint32_t*>(blk + code_offset(D, which, row, cc * 4)) = word;
      if ((cc & 3) == 0) {
        *reinterpret_cast<__half*>(blk + meta_offset(D, which, 0, cc >> 2, row)) = sq;
        *reinterpret_cast<__half*>(blk + meta_offset(D, which, 1, cc >> 2, row)) = zq;
      }
    }
  }
  // the row is fetched back by this block's bulk copies (asynchronous proxy): order them after the stores
  __threadfence();
  asm volatile("fence.proxy.async;\n" ::: "memory");
}

// GEN = the general form: a sliding window (Appendix A) and / or several query tokens per sequence
// (S_q > 1, the grid's S_q factor in Appendix A).  With S_q query tokens the "heads" of a KV head are its
// G * S_q (query token, head) pairs, v = s * G + g, packed into MMA columns like plain heads; query token s
// is the (S_q - 1 - s)-th newest cached token and attends causally: tokens [lo_s, hi_s) with
// hi_s = len - (S_q - 1 - s), lo_s = max(0, hi_s - window).  The plain instantiation carries none of this
// arithmetic into the block loop.  MODE: 0 plain, 1 general, 2 general over a paged cache (tq.h), 3 overlapped /
// fused step, 4 the same over a paged cache, 5 the fused step with a sliding window (general form, contiguous), 6 the
// overlapped fused step with a sliding window: the block
// addresses then come from the page table through a per-thread-block table of page addresses.
template <int D, int MODE, bool HOOK = false, bool SEP = false>
__global__ void __launch_bounds__(kThreads, Cfg<D>::MINB)
    decode_mma_kernel(tq_kv_cache cache, const __half* __restrict__ q, int H_q, int S_q, float attn_scale, int window,
                      int C, float* __restrict__ o_part, float* __restrict__ m_part, float* __restrict__ l_part,
                      int32_t* status, int stable_blocks_arg, StepArgs sa) {
  using Cf = Cfg<D>;
  using Ly = Layout<D, SEP>;
  constexpr int NGW = Cf::NGW, DS = Cf::DS, NTEAM = Cf::NTEAM;
  constexpr bool GEN = MODE == 1 || MODE == 2 || MODE == 5, PAGED = MODE == 2 || MODE == 4;
  constexpr bool OVL = MODE == 3 || MODE == 4 || MODE == 6, WIN = MODE == 6;  // WIN: overlapped step over a sliding window
  constexpr bool STEP = OVL || MODE == 5;  // the forms that can append the new token and reduce the partials themselves
  const long long wait_limit = HOOK ? static_cast<long long>(sa.wait_cycles) : kMaxWaitCycles;
  extern __shared__ __align__(1024) uint8_t smem[];

  const int G = H_q / cache.H_kv;
  const int GV = GEN ? G * S_q : G;  // columns of this KV head
  const int tiles = (GV + 7) >> 3;
  const int c = blockIdx.x, kvh = blockIdx.y / tiles, tile = blockIdx.y - kvh * tiles, b = blockIdx.z;
  // the warp index through a broadcast, so that the compiler keeps what derives from it (ring, barrier and
  // block addresses) in uniform registers
  const int warp = __shfl_sync(0xffffffffu, static_cast<int>(threadIdx.x >> 5), 0);
  const int lane = threadIdx.x & 31, gid = lane >> 2, tid4 = lane & 3;
  const int team = warp / DS, sub = warp - team * DS;  // this warp works on channels [sub * DW, (sub + 1) * DW)
  const int v0 = tile * 8;                   // first column of this tile
  const int nh = min(8, GV - v0);            // columns in the tile; the rest of N = 8 is zero padding
  // row of column v in q and in the partial arrays: [B][S_q][H_q]
  auto q_row = [&](int v) -> long long {
    const int s = GEN ? v / G : 0;
    return (static_cast<long long>(b) * (GEN ? S_q : 1) + s) * H_q + kvh * G + (v - s * G);
  };
  // The next kernel in the stream may be scheduled from here on (it waits for this one where it must).
  pdl_launch_dependents();
  // Overlapped form (MODE 3): the splits partition the `stable_blocks` oldest 16-token blocks, which nothing
  // still running writes, and q is final too (the caller's promise, tq.h); so this kernel streams and
  // computes without waiting for the kernel before it, waits once the stable part is done, reads the length
  // and lets its last split take the tokens beyond the stable part.  Every other form waits here, before its
  // first global access.
  // the stable part of this sequence in 16-token blocks: the launch argument, or the caller's per-sequence array
  // (final before the preceding work starts, like what it describes; fewer blocks than splits: no early start)
  int stable_blocks = stable_blocks_arg;
  if (OVL && sa.stable_lens != nullptr) {
    const int st = min(max(sa.stable_lens[blockIdx.z], 0), cache.S_cap) / kBlk;
    stable_blocks = st >= C ? st : 0;
  }
  const bool ovl = OVL && stable_blocks > 0;
  if (!ovl) pdl_wait();
  const long long row0 = (static_cast<long long>(b) * cache.H_kv + kvh) * cache.S_cap;
  const uint8_t* const head_blocks = cache.blocks + (row0 >> 4) * Cf::STAGE;  // contiguous cache
  // Paged cache: the address of this KV head's part of the page that table entry `entry` of the sequence names
  // (a page outside the pool is flagged and page 0 read instead).
  const int pshift = PAGED ? 31 - __clz(cache.page_tokens >> 4) : 0;
  auto page_base = [&](int entry) -> const uint8_t* {
    int pg = cache.page_table[static_cast<long long>(b) * cache.max_pages + entry];
    if (static_cast<uint32_t>(pg) >= static_cast<uint32_t>(cache.num_pages)) {
      if (status) atomicOr(status, TQ_STATUS_BAD_PAGE);
      pg = 0;
    }
    // block index in the pool (fits 32 bits: the pool is checked to hold fewer than 2^31 blocks)
    const uint32_t idx = (static_cast<uint32_t>(pg) * cache.H_kv + kvh) << pshift;
    return cache.blocks + static_cast<size_t>(idx) * Cf::STAGE;
  };
  auto block_addr = [&](int blk) -> const uint8_t* {  // any block of this (sequence, KV head), by a table lookup if paged
    if (PAGED) return page_base(blk >> pshift) + static_cast<size_t>(blk & ((1 << pshift) - 1)) * Cf::STAGE;
    return head_blocks + static_cast<size_t>(blk) * Cf::STAGE;
  };
  // The length of this sequence; in the fused step also the place where the new token is quantised and
  // written (by the block of the last split of this KV head, which is the only one to read that row: it
  // issues its copies of the newest blocks after this) and where the length is advanced (by whichever block
  // of the sequence is the last to have read the old one).  Every block of the grid calls it once, after the
  // wait for the preceding kernel.
  auto read_len = [&]() -> int {
    int n = checked_len(cache.seq_lens, b, cache.S_cap, (c == 0 && blockIdx.y == 0) ? status : nullptr);
    if (STEP && sa.k_new != nullptr) {
      const int old = n;
      if (old < cache.S_cap) n = old + 1;
      else if (c == 0 && blockIdx.y == 0 && threadIdx.x == 0 && status) atomicOr(status, TQ_STATUS_CACHE_FULL);
      if (c == C - 1 && n > old) {  // one head tile per KV head in this form (checked on the host)
        bool writable = true;  // paged: a table entry outside the pool is flagged (by block_addr) and nothing is written
        if (PAGED) {
          const int pg = cache.page_table[static_cast<long long>(b) * cache.max_pages + ((old >> 4) >> pshift)];
          writable = static_cast<uint32_t>(pg) < static_cast<uint32_t>(cache.num_pages);
        }
        uint8_t* const dst = const_cast<uint8_t*>(block_addr(old >> 4));
        if (warp == 0 && writable)
          quantize_new_row<D>(dst, old & 15,
                              sa.k_new + (static_cast<long long>(b) * cache.H_kv + kvh) * D,
                              sa.v_new + (static_cast<long long>(b) * cache.H_kv + kvh) * D);
        __syncthreads();
      }
      if (threadIdx.x == 0) {
        const int readers = cache.H_kv * C;
        int32_t* const cnt = sa.counters + static_cast<long long>(cache.B) * cache.H_kv + b;
        if (atomicAdd(cnt, 1) == readers - 1) {  // every block of the sequence has read the old length
          cache.seq_lens[b] = n;
          *cnt = 0;
        }
      }
    }
    return n;
  };
  // Windowed overlapped step (WIN): the caller promises stable_tokens <= length <= stable_tokens + kWinSlack, so
  // the blocks from `early0` up to the end of the stable part lie inside the window whatever the length turns
  // out to be, and are final: the splits partition those and stream them before the wait.  The few blocks at
  // the two ends (the window's start, the newest tokens) are attended by the last split after the wait, with
  // row masks.  (The host sends shapes with fewer early blocks than splits to the general form instead.)
  int early0 = 0;
  if (WIN) {
    const int lo = stable_blocks * kBlk + kWinSlack - window;
    early0 = lo > 0 ? min((lo + kBlk - 1) / kBlk, stable_blocks) : 0;
  }
  int len = 0, t0, t1;
  if (ovl) {
    const long long ne = stable_blocks - early0;
    t0 = (early0 + static_cast<int>((ne * c) / C)) * kBlk;
    t1 = (early0 + static_cast<int>((ne * (c + 1)) / C)) * kBlk;
  } else {
    len = STEP ? read_len() : checked_len(cache.seq_lens, b, cache.S_cap, (c == 0 && blockIdx.y == 0) ? status : nullptr);
    split_range(GEN ? query_lo(len, S_q, 0, window) : 0, len, C, c, t0, t1);  // attended tokens of this split
  }

  // ---- q first (a handful of loads that must not queue behind the cache stream), used further down
  uint4 qraw[NGW];
#pragma unroll
  for (int g = 0; g < NGW; ++g) {
    qraw[g] = make_uint4(0, 0, 0, 0);
    if (gid < nh)
      qraw[g] = *reinterpret_cast<const uint4*>(q + q_row(v0 + gid) * D + (sub * NGW + g) * 32 + tid4 * 8);
  }

  // ---- this team's token blocks: blk0 + team, blk0 + team + NTEAM, ...
  int blk0 = t0 / kBlk;
  // windowed overlapped step: a second run of blocks behind the first (see the phase after the wait)
  int seg_n = 0x7fffffff, blk0b = 0, strideb = NTEAM;
  (void)seg_n; (void)blk0b; (void)strideb;
  const int blk1 = t1 > t0 ? (t1 + kBlk - 1) / kBlk : blk0;  // an empty split owns no block
  int nblk = blk1 - blk0 > team ? (blk1 - blk0 - team + NTEAM - 1) / NTEAM : 0;
  uint8_t* const ring = smem + team * (Ly::NST * Cf::STAGE);
  const uint32_t ring_s = static_cast<uint32_t>(__cvta_generic_to_shared(ring));
  const uint32_t bars = static_cast<uint32_t>(__cvta_generic_to_shared(smem + Ly::BARS)) + team * (Ly::NST * 8);
  if (sub == 0 && lane == 0) {
#pragma unroll
    for (int s = 0; s < Ly::NST; ++s) mbar_init(bars + 8 * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    if (DS > 1) {  // the team's two timeout flags (see the score exchange below)
      int* const xf = reinterpret_cast<int*>(smem + Ly::XCH + team * Ly::XCH_TEAM + 2 * DS * 32 * 16);
      xf[0] = xf[1] = 0;
    }
  }
  // The team's n-th block is block blk0 + team + n * NTEAM of this (sequence, KV head); one lane of the team
  // copies it into ring slot n mod NST.  Contiguous cache: it starts at head_blocks + block * STAGE.
  // Paged: page_tokens is a power of two, so block j sits in table entry j >> pshift at offset j & (bpp - 1);
  // the thread block first turns the table entries of its split into addresses of this KV head's part of each
  // page (checked against the pool once), kept in shared memory behind everything else, so that issuing a copy
  // costs a shift, a shared-memory load and a multiply-add.
  // (In the overlapped form the table entries of the stable part are read before the wait for the preceding
  // kernel: they belong to what the caller declared final.  The few blocks the last split attends beyond
  // the stable part are looked up one by one after the wait.)
  const int page0 = blk0 >> pshift;
  const uint8_t** const page_ptr = reinterpret_cast<const uint8_t**>(smem + Ly::SMEM);
  const int npages = (PAGED && blk1 > blk0) ? ((blk1 - 1) >> pshift) - page0 + 1 : 0;
  if (PAGED) {
    for (int i = threadIdx.x; i < npages; i += kThreads) page_ptr[i] = page_base(page0 + i);
  }
  if (DS > 1 || PAGED) __syncthreads();  // a team's warps wait on the same barriers; everybody reads the page addresses
  else __syncwarp();
  auto issue_to = [&](int n, int slot) {
    if (sub == 0 && lane == 0) {
      const int blk = (WIN && n >= seg_n) ? blk0b + team + n * strideb : blk0 + team + n * NTEAM;
      const uint8_t* src;
      if (PAGED) {
        const int pi = (blk >> pshift) - page0;
        src = (!OVL || pi < npages) ? page_ptr[pi] + static_cast<size_t>(blk & ((1 << pshift) - 1)) * Cf::STAGE : block_addr(blk);
      } else {
        src = head_blocks + static_cast<size_t>(blk) * Cf::STAGE;
      }
      const uint32_t bar = bars + 8 * slot;
      mbar_expect_tx(bar, Cf::STAGE + ((HOOK && blk == sa.fault_blk) ? 16 : 0));
      bulk_g2s(ring_s + slot * Cf::STAGE, src, Cf::STAGE, bar);
    }
  };

  auto issue = [&](int n) { issue_to(n, n % Ly::NST); };

  // start streaming: the first stages are in flight while q is turned into fragments
#pragma unroll
  for (int s = 0; s < Ly::NST - 1; ++s)
    if (s < nblk) issue(s);
  // issue the team's n-th block, if it has one
  auto refill = [&](int n) {
    if (n < nblk) issue(n);
  };

  // ---- q as MMA B fragments: column n = gid is column v0 + gid of the tile; k slots follow the nibble order.
  // qs[g][j] = 2^-24 * sum of q over group g for heads 2*tid4 + j (the zero-point term of the scores).
  uint32_t qf[NGW][4];
  float qs[NGW][2];
#pragma unroll
  for (int g = 0; g < NGW; ++g) {
    const uint4 raw = qraw[g];
    const __half2 sixteenth = __float2half2_rn(0.0625f);
    qf[g][0] = __byte_perm(raw.x, raw.z, 0x5410);                                            // (c0, c4)
    qf[g][1] = h2_as_u32(__hmul2(u32_as_h2(__byte_perm(raw.x, raw.z, 0x7632)), sixteenth));  // (c1, c5) / 16
    qf[g][2] = __byte_perm(raw.y, raw.w, 0x5410);                                            // (c2, c6)
    qf[g][3] = h2_as_u32(__hmul2(u32_as_h2(__byte_perm(raw.y, raw.w, 0x7632)), sixteenth));  // (c3, c7) / 16
    const __half2* h2 = reinterpret_cast<const __half2*>(&raw);
    float sum = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 f = __half22float2(h2[i]);
      sum += f.x + f.y;
    }
    sum += __shfl_xor_sync(0xffffffffu, sum, 1);
    sum += __shfl_xor_sync(0xffffffffu, sum, 2);  // every lane of quad gid: sum over group g of head gid
    sum *= 5.9604644775390625e-8f;                // 2^-24, like the code operands
    qs[g][0] = __shfl_sync(0xffffffffu, sum, (2 * tid4) * 4);
    qs[g][1] = __shfl_sync(0xffffffffu, sum, (2 * tid4 + 1) * 4);
  }

  // B operand of the zero-point MMA of the scores (see block_scores) and the softmax scale of the thread's columns
  uint32_t qz[2] = {0u, 0u};
  float cs0 = attn_scale * kLog2e * 16777216.0f, cs1 = cs0;  // scores carry 2^-24 from the code operands
  if constexpr (KZ<D>::on) {
    // Head gid's row is scaled by a power of two, 2^(14 - e) with e = floor(log2(largest magnitude)), so that it
    // fills the fp16 range whatever the size of q: the code terms then carry 2^(-24 + 14 - e), and the group sums
    // of q are given the same factor, 2^(-10 - e) (they stay below 2^-3 and are split into an fp16 pair), so
    // that the zero-point MMA's result adds to the code terms as it stands.  The factor goes into the softmax
    // scale of the column.  A team agrees on e over the whole row.
    float mx = 0.f, sumg[NGW];
#pragma unroll
    for (int g = 0; g < NGW; ++g) {
      const __half2* h2 = reinterpret_cast<const __half2*>(&qraw[g]);
      float sum = 0.f;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 f = __half22float2(h2[i]);
        sum += f.x + f.y;
        mx = fmaxf(mx, fmaxf(fabsf(f.x), fabsf(f.y)));
      }
      sum += __shfl_xor_sync(0xffffffffu, sum, 1);
      sum += __shfl_xor_sync(0xffffffffu, sum, 2);
      sumg[g] = sum;
    }
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
    if constexpr (DS > 1) {  // through the half of the exchange buffer that block 1 is the first to use
      float* const qmx = reinterpret_cast<float*>(smem + Ly::XCH + team * Ly::XCH_TEAM + DS * 32 * 16);
      qmx[sub * 32 + lane] = mx;
      // (named barriers 9 + team: 1 .. 8 belong to the score exchange of the block loop)
      asm volatile("bar.sync %0, %1;\n" ::"r"(9 + team), "r"(32 * DS) : "memory");
#pragma unroll
      for (int w = 0; w < DS; ++w) mx = fmaxf(mx, qmx[w * 32 + lane]);
      asm volatile("bar.sync %0, %1;\n" ::"r"(9 + team), "r"(32 * DS) : "memory");
    }
    int e = ((__float_as_int(mx) >> 23) & 0xff) - 127;  // floor(log2(max)); an all-zero row gives -127
    e = max(-24, min(e, 15));
    const float up = __int_as_float((127 + 14 - e) << 23);     // 2^(14 - e)
    const float dn = __int_as_float((127 - 10 - e) << 23);     // 2^(-10 - e)
    const float back = __int_as_float((127 + 10 + e) << 23);   // 2^(10 + e): what the scores carry
#pragma unroll
    for (int g = 0; g < NGW; ++g) {
      const __half2* h2 = reinterpret_cast<const __half2*>(&qraw[g]);
      uint32_t w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 f = __half22float2(h2[i]);
        w[i] = h2_as_u32(__floats2half2_rn(f.x * up, f.y * up));  // exact: a power of two, inside the fp16 range
      }
      const __half2 sixteenth = __float2half2_rn(0.0625f);
      qf[g][0] = __byte_perm(w[0], w[2], 0x5410);
      qf[g][1] = h2_as_u32(__hmul2(u32_as_h2(__byte_perm(w[0], w[2], 0x7632)), sixteenth));
      qf[g][2] = __byte_perm(w[1], w[3], 0x5410);
      qf[g][3] = h2_as_u32(__hmul2(u32_as_h2(__byte_perm(w[1], w[3], 0x7632)), sixteenth));
    }
    const float sa = -(tid4 & 1 ? sumg[2] : sumg[0]) * dn, sb = -(tid4 & 1 ? sumg[3] : sumg[1]) * dn;
    const __half2 hi = __floats2half2_rn(sa, sb);
    const float2 hf = __half22float2(hi);
    const __half2 lo = __floats2half2_rn(sa - hf.x, sb - hf.y);
    qz[0] = qz[1] = tid4 < 2 ? h2_as_u32(hi) : h2_as_u32(lo);
    const float csh = attn_scale * kLog2e * back;
    cs0 = __shfl_sync(0xffffffffu, csh, (2 * tid4) * 4);
    cs1 = __shfl_sync(0xffffffffu, csh, (2 * tid4 + 1) * 4);
  }

  float oacc[Cf::DW / 16][4];  // [M tile][c0..c3]: rows = channels, cols = heads 2*tid4, 2*tid4+1
  float zacc[NGW][4];          // sum_tok B_g * z_g: [0], [1] are heads 2*tid4, 2*tid4+1; [2], [3] are not used
  float zero4[4];              // four registers holding 0, opaque to the compiler: the C operand of accumulator-less MMAs
#pragma unroll
  for (int i = 0; i < 4; ++i) asm volatile("mov.f32 %0, 0f00000000;\n" : "=f"(zero4[i]));
#pragma unroll
  for (int i = 0; i < Cf::DW / 16; ++i) oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f;
#pragma unroll
  for (int g = 0; g < NGW; ++g) zacc[g][0] = zacc[g][1] = zacc[g][2] = zacc[g][3] = 0.f;
  float m0 = kNoMax, m1 = kNoMax, l0 = 0.f, l1 = 0.f;

  // Blocks in which every token counts for every column go through the plain step, the others through the
  // masking one.  Plain decode: only the block holding the end of the sequence is partial.  General form:
  // blocks that reach beyond the oldest query's end, or begin before the newest query's window start.
  int rem_last = t1 - (blk0 + team + (nblk - 1) * NTEAM) * kBlk;  // tokens in this team's last block
  int nfull = (nblk > 0 && rem_last < kBlk) ? nblk - 1 : nblk;    // this team's blocks k < nfull are full
  int nhead = 0;                                                        // ... and blocks k < nhead are masked
  if (GEN) {
    const int full_end = min(t1, query_hi(len, S_q, 0)) >> 4;                   // blocks below it end inside every range
    const int full_begin = (query_lo(len, S_q, S_q - 1, window) + kBlk - 1) >> 4;  // blocks from it on begin inside
    const int first_blk = blk0 + team;
    nfull = full_end > first_blk ? min(nblk, (full_end - first_blk + NTEAM - 1) / NTEAM) : 0;
    nhead = full_begin > first_blk ? min(nblk, (full_begin - first_blk + NTEAM - 1) / NTEAM) : 0;
  }
  const unsigned nplain = nfull > nhead ? nfull - nhead : 0;  // general form: blocks nhead <= k < nhead + nplain are full
  const int plain_lo = GEN ? nhead : 0, plain_hi = GEN ? nhead + static_cast<int>(nplain) : nfull;  // (of the first phase)
  // per-lane byte offsets inside a stage: ldmatrix row addresses of the code, scale and zero fragments of
  // this warp's channel groups sub * NGW .. (see block_scores / block_softmax_pv)
  WarpCtx<D> cx;
  cx.cs0 = cs0; cx.cs1 = cs1; cx.gid = gid; cx.keep = gid == 4 ? 0u : 0xFFFFFFFFu;
  cx.ksz_lane = ring_s + 2 * Cf::PK + (lane >> 4) * Cf::SZ + ((lane >> 3) & 1) * 16 + (lane & 1) * 32 + sub * NGW * 32;
  if constexpr (KZ<D>::on) {
    cx.ksz_lane = ring_s + 2 * Cf::PK + (2 * (lane >> 4) + (lane & 1)) * 32 + ((lane >> 3) & 1) * 16 + sub * NGW * 32;
    cx.kz_lane = ring_s + 2 * Cf::PK + (lane >> 4) * Cf::SZ + ((lane >> 3) & 1) * 16 + (lane & 3) * 32 + sub * NGW * 32;
  } else {
    cx.kz_lane = 0;
  }
  cx.vsz_lane = ring_s + 2 * Cf::PK + (3 - ((lane >> 3) & 1)) * Cf::SZ + (lane >> 4) * 16 + sub * NGW * 32;
  cx.vz_lane = ring_s + 2 * Cf::PK + (2 + (lane >> 4)) * Cf::SZ + ((lane >> 3) & 1) * 16 + (lane & 3) * 32 + sub * NGW * 32;
  cx.vs2_lane = ring_s + 2 * Cf::PK + 2 * Cf::SZ + ((lane >> 3) & 1) * 16 + (lane >> 4) * 32 + sub * NGW * 32;
#pragma unroll
  for (int i = 0; i < NGW / 2; ++i) {
    const int j = 4 * i + (lane >> 3);
    const int tok = (lane & 7) + 8 * (j % 2), grp = sub * NGW + j / 2;
    cx.kaddr[i] = ring_s + tok * Cf::ROWB + ((grp ^ Cf::swz(tok)) << 4);
  }
  // Score exchange of a team: [2 (parity of k)][DS][32 lanes] float4, then two timeout flags (parity of k).
  // The warps of a team each hold the scores over their own channels: they exchange and add them in a fixed
  // order, so that every warp of the team continues with bit-identical scores.  The barrier of block k also
  // tells that every warp is done with the slot of block k - 1, which is refilled after it.  A warp whose
  // wait ran out raises the flag of that block's parity before the barrier (the flags start at 0 and are
  // never lowered: nothing runs after a timeout), and the whole team stops together.
  float4* const xch = reinterpret_cast<float4*>(smem + Ly::XCH + team * Ly::XCH_TEAM);
  volatile int* const xflag = reinterpret_cast<volatile int*>(smem + Ly::XCH + team * Ly::XCH_TEAM + 2 * DS * 32 * 16);
  // Two-warp teams split the barrier in two: a warp announces its partial on its own barrier (bar.arrive, does
  // not wait) and later waits on its partner's (bar.sync), so whatever does not depend on the scores can be
  // issued in between.  Barrier 1 + 2 * team + sub belongs to warp `sub` of the team: 32 arrivals from its owner
  // and 32 from the partner's wait complete a phase.  Four-warp teams keep one barrier per team.
  auto exchange_post = [&](const float (&sc)[4], int par01, bool arrived) {
    float4* const xb = xch + par01 * (DS * 32);
    xb[sub * 32 + lane] = make_float4(sc[0], sc[1], sc[2], sc[3]);
    if (!arrived && lane == 0) xflag[par01] = 1;
    if (DS == 2) asm volatile("bar.arrive %0, 64;\n" ::"r"(1 + 2 * team + sub) : "memory");
  };
  auto exchange_wait = [&](float (&sc)[4], int par01) -> bool {
    float4* const xb = xch + par01 * (DS * 32);
    if (DS == 2) {  // a + b in either order is the same number
      asm volatile("bar.sync %0, 64;\n" ::"r"(1 + 2 * team + (sub ^ 1)) : "memory");
      const float4 part = xb[(sub ^ 1) * 32 + lane];
      sc[0] += part.x; sc[1] += part.y; sc[2] += part.z; sc[3] += part.w;
    } else {
      asm volatile("bar.sync %0, %1;\n" ::"r"(1 + team), "r"(32 * DS) : "memory");
      sc[0] = sc[1] = sc[2] = sc[3] = 0.f;
#pragma unroll
      for (int w = 0; w < DS; ++w) {
        const float4 part = xb[w * 32 + lane];
        sc[0] += part.x; sc[1] += part.y; sc[2] += part.z; sc[3] += part.w;
      }
    }
    return xflag[par01] == 0;
  };
  auto exchange = [&](float (&sc)[4], int par01, bool arrived) -> bool {
    exchange_post(sc, par01, arrived);
    return exchange_wait(sc, par01);
  };

  bool timed_out = false;
  int k = 0, kf = 0;  // kf: the block whose wait ran out
#pragma unroll 1
  for (int phase = 0; phase < (ovl ? 2 : 1); ++phase) {
  if (ovl && phase == 1) {
    // the stable part is done: from here on this kernel is ordered after the one before it
    pdl_wait();
    len = read_len();
    const int stable_tokens = stable_blocks * kBlk;
    if ((len < stable_tokens || (WIN && len > stable_tokens + kWinSlack)) && c == 0 && blockIdx.y == 0 && threadIdx.x == 0 &&
        status)
      atomicOr(status, TQ_STATUS_BAD_LEN);  // the promise did not hold: tokens outside the attended range were attended
    int next = 0;
    if (c == C - 1 && len > stable_tokens && !timed_out) {
      const int eb1 = (len + kBlk - 1) / kBlk;
      next = eb1 - stable_blocks > team ? (eb1 - stable_blocks - team + NTEAM - 1) / NTEAM : 0;
    }
    // the ring goes on where it stood: block number n >= nblk of this team is now stable_blocks + team + (n - nblk) * NTEAM
    blk0 = stable_blocks - nblk * NTEAM;
    nblk += next;
    rem_last = next > 0 ? len - (blk0 + team + (nblk - 1) * NTEAM) * kBlk : kBlk;
    nfull = rem_last < kBlk ? nblk - 1 : nblk;
    if (WIN) {
      // Windowed step: every block from here on goes through the masking step.  Behind the newest blocks come the
      // blocks between the window's start and the early region, dealt out over all the teams of all the splits of
      // this KV head (nothing still running writes them), so that no thread block has more than one or two; they
      // are issued together with the newest ones: one memory latency, not two.  Blocks n >= seg_n of this team
      // are blk0b + team + n * strideb.
      nfull = k;
      const int hb0 = max(0, len - window) / kBlk, mine = c * NTEAM + team;
      strideb = C * NTEAM;
      seg_n = nblk;
      int more = 0;
      if (early0 - hb0 > mine && !timed_out) more = (early0 - hb0 - mine + strideb - 1) / strideb;
      blk0b = hb0 + c * NTEAM - nblk * strideb;
      nblk += more;
      next += more;
    }
    if (next > 0) {
      for (int n = k; n < k + Ly::NST - 1; ++n)
        if (n < nblk) issue(n);
    }
  }
  fast_blocks:
  if constexpr (DS == 1) {
   // Full blocks one ring (NST blocks) at a time: ring slot, barrier and stage offsets are constants of each of
   // the NST copies of the block step, so the loop carries no slot arithmetic.  It starts on a block whose number
   // is a multiple of NST (plain decode: block 0; general form: the first such block behind the masked ones
   // at the old end of the attended range, reached by the one-block loop below).
   constexpr int NST = Ly::NST;
   if (phase == 0 && k % NST == 0 && k >= plain_lo && k + NST <= plain_hi) {
    const RowMask all{kBlk, 0, kBlk, 0, kBlk};
    uint32_t par = (k / NST) & 1;
    // The barrier of the next block is probed one block ahead (the probe's latency then hides behind a block
    // of arithmetic); only a probe that came back negative is followed by the blocking wait.  No warp-wide
    // synchronisation is needed before a slot is refilled: its last readers were the warp-collective loads
    // of the previous block, whose results the MMAs issued since then have already consumed.
    bool ready = mbar_test_wait(bars, par);
#ifdef TQ_PROBE_MATH_ONLY
    // Timing probe (results are meaningless): the three copies issued above are awaited here, the fourth
    // slot is cleared, and the unrolled loop then runs its arithmetic on whatever the ring holds without
    // waiting for or issuing any copy; the blocks it leaves over are skipped.
    for (int s = 0; s < Ly::NST - 1; ++s)
      if (s < nblk) wait_stage(bars + 8 * s, 0);
    for (int i = lane; i < Cf::STAGE / 4; i += 32) reinterpret_cast<uint32_t*>(ring + (NST - 1) * Cf::STAGE)[i] = 0;
    __syncwarp();
    ready = true;
#endif
    for (; k + NST <= plain_hi; k += NST) {
#pragma unroll
      for (int S = 0; S < NST; ++S) {
        if (!ready && !wait_stage(bars + 8 * S, par, wait_limit)) {  // cold: leave the loops, keep the phase order
          timed_out = true;
          kf = k + S;
          goto phase_done;
        }
#ifndef TQ_PROBE_MATH_ONLY
        if (k + S + NST - 1 < nblk) issue_to(k + S + NST - 1, (S + NST - 1) % NST);
        ready = mbar_test_wait(bars + 8 * ((S + 1) % NST), S == NST - 1 ? par ^ 1 : par);
#endif
#ifndef TQ_PROBE_COPIES_ONLY
        float sc[4];
        block_scores<D, false>(cx, nullptr, S * Cf::STAGE, all, qf, qs, qz, zero4, sc);
        block_softmax_pv<D, false>(cx, S * Cf::STAGE, all, sc, oacc, zacc, m0, m1, l0, l1);
#endif
      }
      par ^= 1;
    }
#ifdef TQ_PROBE_MATH_ONLY
    k = nblk;
#endif
   }
  }
  if constexpr (DS > 1) {
   if (phase == 0 && k % Ly::NST == 0 && k >= plain_lo && k + Ly::NST <= plain_hi) {
    // The same four-block step for a team: the scores of each block are exchanged before its softmax.
    static_assert(Ly::NST == 4, "the unrolled loop walks a ring of four slots");
    const RowMask all{kBlk, 0, kBlk, 0, kBlk};
    uint32_t par = (k / Ly::NST) & 1;
    bool ready = mbar_test_wait(bars, par);
    for (; k + 4 <= plain_hi; k += 4) {
#pragma unroll
      for (int S = 0; S < 4; ++S) {
        const bool arrived = ready || wait_stage(bars + 8 * S, par, wait_limit);
        float sc[4];
        block_scores<D, false>(cx, nullptr, S * Cf::STAGE, all, qf, qs, qz, zero4, sc);
        exchange_post(sc, S & 1, arrived);
        // what does not depend on the scores goes between the announcement and the wait (hoisting the first V
        // scale and code loads as well was measured: it spills and is slower)
        uint32_t zop[4];
        pv_zero_operands<D>(cx, S * Cf::STAGE, zop);
        ready = mbar_test_wait(bars + 8 * ((S + 1) & 3), S == 3 ? par ^ 1 : par);
        if (!exchange_wait(sc, S & 1)) {
          timed_out = true;
          kf = k + S;
          goto phase_done;
        }
        if (k + S + 3 < nblk) issue_to(k + S + 3, (S + 3) & 3);
        block_softmax_pv<D, false, true>(cx, S * Cf::STAGE, all, sc, oacc, zacc, m0, m1, l0, l1, zop);
      }
      par ^= 1;
    }
   }
  }
#pragma unroll 1
  for (; k < nblk && !timed_out; ++k) {
    // Wait for this block's bytes.  The wait is bounded: if the copy never completes (which would take
    // a bad pointer), the warp flags the status word and stops consuming.
    const bool arrived = wait_stage(bars + 8 * (k % Ly::NST), (k / Ly::NST) & 1, wait_limit);
    if (DS == 1) {
      if (!arrived) { timed_out = true; kf = k; break; }
      __syncwarp();  // every lane is done with the slot consumed in the previous iteration: refill it
      refill(k + Ly::NST - 1);
    }
    const uint32_t st_s = (k % Ly::NST) * Cf::STAGE;
    const uint8_t* st = ring + (k % Ly::NST) * Cf::STAGE;
    const bool plain = GEN ? static_cast<unsigned>(k - nhead) < nplain : k < nfull;
    auto mask_of_block = [&]() {
      RowMask mk{rem_last, 0, rem_last, 0, rem_last};
      if (WIN) {  // rows of the block inside [max(0, len - window), len)
        const int first = (k >= seg_n ? blk0b + team + k * strideb : blk0 + team + k * NTEAM) * kBlk;
        const int lo = max(0, len - window) - first, hi = len - first;
        mk = RowMask{hi, lo, hi, lo, hi};
      }
      if (GEN) {
        mk = general_row_mask(cache.seq_lens, blockIdx.z, cache.S_cap, S_q, window, C, blockIdx.x, H_q / cache.H_kv,
                              (blockIdx.y % tiles) * 8 + 2 * (threadIdx.x & 3), (blk0 + team + k * NTEAM) * kBlk,
                              STEP ? len : -1);
      }
      return mk;
    };
    const RowMask all{kBlk, 0, kBlk, 0, kBlk};
    float sc[4];
    if (DS == 1) {
      if (plain) {
        block_scores<D, false>(cx, st, st_s, all, qf, qs, qz, zero4, sc);
        block_softmax_pv<D, false>(cx, st_s, all, sc, oacc, zacc, m0, m1, l0, l1);
      } else {
        const RowMask mk = mask_of_block();
        block_scores<D, true>(cx, st, st_s, mk, qf, qs, qz, zero4, sc);
        block_softmax_pv<D, true>(cx, st_s, mk, sc, oacc, zacc, m0, m1, l0, l1);
      }
      if (GEN && phase == 0 && (k + 1) % Ly::NST == 0 && k + 1 >= plain_lo && k + 1 + Ly::NST <= plain_hi) {
        ++k;  // behind the masked blocks of the old end: the four-block loop takes the full ones
        goto fast_blocks;
      }
    } else {
      const RowMask mk = plain ? all : mask_of_block();
      if (plain) block_scores<D, false>(cx, st, st_s, mk, qf, qs, qz, zero4, sc);
      else block_scores<D, true>(cx, st, st_s, mk, qf, qs, qz, zero4, sc);
      if (!exchange(sc, k & 1, arrived)) { timed_out = true; kf = k; break; }
      refill(k + Ly::NST - 1);
      if (plain) block_softmax_pv<D, false>(cx, st_s, mk, sc, oacc, zacc, m0, m1, l0, l1);
      else block_softmax_pv<D, true>(cx, st_s, mk, sc, oacc, zacc, m0, m1, l0, l1);
      if (GEN && phase == 0 && (k + 1) % Ly::NST == 0 && k + 1 >= plain_lo && k + 1 + Ly::NST <= plain_hi) {
        ++k;
        goto fast_blocks;
      }
    }
  }
  phase_done:;
  }  // phase
  if (timed_out) {
    // The copies of blocks kf, kf + 1, kf + 2 of this team may still be in flight into its ring: give each the
    // full bounded time to land before the block reuses the memory, then report.  The partial written below
    // is not valid in that case.
    for (int n = kf; n < kf + Ly::NST - 1 && n < nblk; ++n)
      wait_stage(bars + 8 * (n % Ly::NST), (n / Ly::NST) & 1);
    if (lane == 0 && status) atomicOr(status, TQ_STATUS_TIMEOUT);
  }

  // ---------------- merge the teams and write the normalised partial (o_c, m_c, l_c)
  if constexpr (KZ<D>::on) {  // row 4 of the zero-point accumulator holds the denominators of heads 2*tid4, 2*tid4+1
    l0 = __shfl_sync(0xffffffffu, zacc[0][0], 16 + tid4);
    l1 = __shfl_sync(0xffffffffu, zacc[0][1], 16 + tid4);
  } else {
#pragma unroll
    for (int off = 4; off <= 16; off <<= 1) {
      l0 += __shfl_xor_sync(0xffffffffu, l0, off);
      l1 += __shfl_xor_sync(0xffffffffu, l1, off);
    }
  }
  if constexpr (!SEP) __syncthreads();  // every warp is done with its ring; the memory is reused below
  // layout (floats): wml[NTEAM][16] = each team's m[8], l[8] | slab[NTEAM][8 heads][D] = each team's unnormalised
  // output rows.  The 16-byte chunks of a row are XOR-swizzled inside every run of 8 chunks by the head's pair
  // index, which makes both the fragment stores below and the row reads after them conflict free.
  float* const wml = reinterpret_cast<float*>(smem + Ly::MERGE_OFF);
  float* const slab = wml + NTEAM * 16;
  if (gid == 0 && sub == 0) {  // the warps of a team hold identical m and l
    wml[team * 16 + 2 * tid4] = m0;
    wml[team * 16 + 2 * tid4 + 1] = m1;
    wml[team * 16 + 8 + 2 * tid4] = l0;
    wml[team * 16 + 8 + 2 * tid4 + 1] = l1;
  }
  if constexpr (KZ<D>::on) {  // the single zero-point accumulator: hi + lo sums of group r & 3 in the lanes of row r
    const float z0 = zacc[0][0] + zacc[0][2], z1 = zacc[0][1] + zacc[0][3];
#pragma unroll
    for (int g = 0; g < NGW; ++g) {
      zacc[g][0] = __shfl_sync(0xffffffffu, z0, g * 4 + tid4);
      zacc[g][1] = __shfl_sync(0xffffffffu, z1, g * 4 + tid4);
    }
  }
#pragma unroll
  for (int g = 0; g < NGW; ++g) {
    // channels sub * DW + 32 g + 4 gid + {0, 1, 2, 3} of heads 2*tid4 + j: M tile 2g holds channels +0 (rows 0-7:
    // codes carried 2^-24) and +1 (rows 8-15, high nibble: 2^-20), M tile 2g + 1 channels +2 and +3, where
    // rows 8-15 accumulated the whole upper byte n2 + 16 n3 and rows 0-7 hold the n2 part
    const int chunk = sub * (Cf::DW / 4) + 8 * g + (gid ^ (2 * tid4));  // swizzled position of the 16-byte chunk
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const float z = zacc[g][j];
      float4 v;
      v.x = oacc[2 * g][j] * 16777216.0f - z;
      v.y = oacc[2 * g][2 + j] * 1048576.0f - z;
      v.z = oacc[2 * g + 1][j] * 16777216.0f - z;
      v.w = (oacc[2 * g + 1][2 + j] - oacc[2 * g + 1][j]) * 1048576.0f - z;
      *reinterpret_cast<float4*>(slab + ((team * 8 + 2 * tid4 + j) * D + 4 * chunk)) = v;
    }
  }
  __syncthreads();
  // warp h merges head h: reference M over the teams, weights, denominator, then the weighted sum of the rows
  const bool direct = STEP && sa.out != nullptr && C == 1;  // one split: its partial is the result (Eq. 5 with one term)
  if (warp < nh) {
    const int h = warp;
    float fw[NTEAM], M = kNoMax, den = 0.f;
#pragma unroll
    for (int w = 0; w < NTEAM; ++w) M = fmaxf(M, wml[w * 16 + h]);
#pragma unroll
    for (int w = 0; w < NTEAM; ++w) {  // a team that saw no token has m = -1e30 and l = 0
      fw[w] = ex2(wml[w * 16 + h] - M);
      den = fmaf(fw[w], wml[w * 16 + 8 + h], den);
    }
    const float inv = den > 0.f ? 1.f / den : 0.f;
    const long long pidx = q_row(v0 + h) * C + c;
    for (int qd = lane; qd < D / 4; qd += 32) {
      const int phys = (qd & ~7) | ((qd & 7) ^ (h & 6));
      float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int w = 0; w < NTEAM; ++w) {
        const float4 v = *reinterpret_cast<const float4*>(slab + ((w * 8 + h) * D + 4 * phys));
        a.x = fmaf(fw[w], v.x, a.x); a.y = fmaf(fw[w], v.y, a.y); a.z = fmaf(fw[w], v.z, a.z); a.w = fmaf(fw[w], v.w, a.w);
      }
      a.x *= inv; a.y *= inv; a.z *= inv; a.w *= inv;
      if (direct) {  // no partials, no arrival counter, no second pass: the step of a short context ends here
        const long long orow = q_row(v0 + h) * D + 4 * qd;
        if (sa.out_fp32) {
          *reinterpret_cast<float4*>(static_cast<float*>(sa.out) + orow) = a;
        } else {
          __half2 hh[2] = {__floats2half2_rn(a.x, a.y), __floats2half2_rn(a.z, a.w)};
          *reinterpret_cast<uint2*>(static_cast<__half*>(sa.out) + orow) = *reinterpret_cast<uint2*>(hh);
        }
      } else {
        *reinterpret_cast<float4*>(o_part + pidx * D + 4 * qd) = a;
      }
    }
    if (lane == 0 && !direct) {
      m_part[pidx] = den > 0.f ? M * kLn2 : -INFINITY;  // natural-log units of attn_scale * q.k^
      l_part[pidx] = den;
    }
  }
  if (direct) return;

  // ---------------- fused step: Eq. 5 by the last block of this (sequence, KV head) to get here
  if (STEP && sa.out != nullptr) {
    constexpr int kWts = Ly::WTS;  // in the rings' memory: every warp is past the barrier below before they are written
    float* const wts = reinterpret_cast<float*>(smem + kWts) + warp * TQ_MAX_SPLITS;
    int* const ticket = reinterpret_cast<int*>(smem + kWts + kWarps * TQ_MAX_SPLITS * 4);
    float* const inv_den = reinterpret_cast<float*>(smem + kWts + kWarps * TQ_MAX_SPLITS * 4 + 16);
    __threadfence();  // this block's partial is visible before its arrival is
    __syncthreads();
    if (threadIdx.x == 0) *ticket = atomicAdd(sa.counters + static_cast<long long>(b) * cache.H_kv + kvh, 1);
    __syncthreads();
    if (*ticket == C - 1) {
      __threadfence();
      if (warp < nh) {  // weights: one warp per query head; the partials of other blocks come from L2 (ld.cg)
        const long long prow = q_row(v0 + warp) * C;
        // weights: every lane fetches (m, l) of up to 8 splits at once, one round trip to L2
        constexpr int kPer = TQ_MAX_SPLITS / 32;
        float lv[kPer], mv[kPer];
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
          const int cc = lane + 32 * i;
          lv[i] = cc < C ? __ldcg(l_part + prow + cc) : 0.f;
          mv[i] = cc < C ? __ldcg(m_part + prow + cc) : -INFINITY;
        }
        float mg = -INFINITY;
#pragma unroll
        for (int i = 0; i < kPer; ++i)
          if (lv[i] > 0.f) mg = fmaxf(mg, mv[i]);
#pragma unroll
        for (int off = 16; off; off >>= 1) mg = fmaxf(mg, __shfl_xor_sync(0xffffffffu, mg, off));
        float den = 0.f;
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
          const int cc = lane + 32 * i;
          const float wc = lv[i] > 0.f ? lv[i] * __expf(mv[i] - mg) : 0.f;
          if (cc < C) wts[cc] = wc;
          den += wc;
        }
#pragma unroll
        for (int off = 16; off; off >>= 1) den += __shfl_xor_sync(0xffffffffu, den, off);
        if (lane == 0) inv_den[warp] = den > 0.f ? 1.f / den : 0.f;
      }
      __syncthreads();
      // one float4 of one head's output per thread, the heads' rows spread over all the warps
      for (int item = threadIdx.x; item < nh * (D / 4); item += kThreads) {
        const int h = item / (D / 4), ch = item - h * (D / 4);
        const float* const wh = reinterpret_cast<const float*>(smem + kWts) + h * TQ_MAX_SPLITS;
        const float4* const op = reinterpret_cast<const float4*>(o_part + q_row(v0 + h) * C * D);
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
        constexpr int kBatch = 16;  // partial outputs in flight per thread
        for (int c0 = 0; c0 < C; c0 += kBatch) {
          float4 v[kBatch];
#pragma unroll
          for (int i = 0; i < kBatch; ++i)
            v[i] = c0 + i < C ? __ldcg(op + static_cast<long long>(c0 + i) * (D / 4) + ch) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
          for (int i = 0; i < kBatch; ++i) {
            const float wc = c0 + i < C ? wh[c0 + i] : 0.f;
            a.x = fmaf(wc, v[i].x, a.x); a.y = fmaf(wc, v[i].y, a.y); a.z = fmaf(wc, v[i].z, a.z); a.w = fmaf(wc, v[i].w, a.w);
          }
        }
        const float inv = inv_den[h];
        a.x *= inv; a.y *= inv; a.z *= inv; a.w *= inv;
        const long long orow = q_row(v0 + h) * D;
        if (sa.out_fp32) {
          reinterpret_cast<float4*>(static_cast<float*>(sa.out) + orow)[ch] = a;
        } else {
          __half2 hh[2] = {__floats2half2_rn(a.x, a.y), __floats2half2_rn(a.z, a.w)};
          reinterpret_cast<uint2*>(static_cast<__half*>(sa.out) + orow)[ch] = *reinterpret_cast<uint2*>(hh);
        }
      }
      if (threadIdx.x == 0) sa.counters[static_cast<long long>(b) * cache.H_kv + kvh] = 0;  // ready for the next launch
    }
  }
}

template <int D, int MODE, bool HOOK = false, bool SEP = false>
cudaError_t launch_layout(const tq_kv_cache& c, const __half* q, int H_q, int S_q, float attn_scale, int window, int C,
                          float* o_part, float* m_part, float* l_part, int32_t* status, int stable_blocks, const StepArgs& sa,
                          cudaStream_t st) {
  size_t smem = Layout<D, SEP>::SMEM;
  if (MODE == 2 || MODE == 4) {
    // room for the page addresses of the longest split: its blocks, rounded out to whole pages
    const long long span = (window > 0 && window < c.S_cap) ? static_cast<long long>(window) + S_q + 15 : c.S_cap;
    const long long blocks = (span + 15) / 16 + 1, per_split = (blocks + C - 1) / C + 1;
    smem += 8 * static_cast<size_t>(per_split / (c.page_tokens / 16) + 2);
    if (smem > 227 * 1024) return cudaErrorInvalidConfiguration;  // tiny pages and too few splits for this capacity
  }
  const cudaError_t attr = cudaFuncSetAttribute(decode_mma_kernel<D, MODE, HOOK, SEP>,
                                                cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (attr != cudaSuccess) return attr;
  const int GV = (H_q / c.H_kv) * S_q;
  dim3 grid(C, c.H_kv * ((GV + 7) / 8), c.B);
  return launch_kernel(decode_mma_kernel<D, MODE, HOOK, SEP>, grid, dim3(kThreads), smem, st, c, q, H_q, S_q, attn_scale,
                       window, C, o_part, m_part, l_part, status, stable_blocks, sa);
}

template <int D, int MODE, bool HOOK = false>
cudaError_t launch(const tq_kv_cache& c, const __half* q, int H_q, int S_q, float attn_scale, int window, int C,
                   float* o_part, float* m_part, float* l_part, int32_t* status, int stable_blocks, const StepArgs& sa,
                   cudaStream_t st) {
  if constexpr (D == 128 && !HOOK && (MODE == 0 || MODE == 3)) {
    // Separate merge arrays (see Layout) where they were measured to pay: every split at least 48 token blocks
    // of capacity (six per warp) and the whole grid resident at once.
    const long long blocks = static_cast<long long>(c.B) * c.H_kv * ((H_q / c.H_kv + 7) / 8) * C;
    if (c.S_cap / C >= 48 * kBlk && blocks <= Cfg<D>::MINB * device_sm_count())
      return launch_layout<D, MODE, false, true>(c, q, H_q, S_q, attn_scale, window, C, o_part, m_part, l_part, status,
                                                 stable_blocks, sa, st);
  }
  return launch_layout<D, MODE, HOOK, false>(c, q, H_q, S_q, attn_scale, window, C, o_part, m_part, l_part, status,
                                             stable_blocks, sa, st);
}

template <int D>
cudaError_t launch(const tq_kv_cache& c, const __half* q, int H_q, int S_q, float attn_scale, int window, int C,
                   float* o_part, float* m_part, float* l_part, int32_t* status, int stable_blocks, const StepArgs& sa,
                   bool step, cudaStream_t st) {
  const StepArgs none = {nullptr, nullptr, nullptr, 0, nullptr, nullptr, 0, -1};
  if (step && window > 0 && stable_blocks > 0)
    return launch<D, 6>(c, q, H_q, 1, attn_scale, window, C, o_part, m_part, l_part, status, stable_blocks, sa, st);
  if (step && window > 0)
    return launch<D, 5>(c, q, H_q, 1, attn_scale, window, C, o_part, m_part, l_part, status, 0, sa, st);
  if (step && c.page_table != nullptr)
    return launch<D, 4>(c, q, H_q, 1, attn_scale, 0, C, o_part, m_part, l_part, status, stable_blocks, sa, st);
  if (step) return launch<D, 3>(c, q, H_q, 1, attn_scale, 0, C, o_part, m_part, l_part, status, stable_blocks, sa, st);
  if (c.page_table != nullptr) return launch<D, 2>(c, q, H_q, S_q, attn_scale, window, C, o_part, m_part, l_part, status, 0, none, st);
  if (window > 0 || S_q > 1) return launch<D, 1>(c, q, H_q, S_q, attn_scale, window, C, o_part, m_part, l_part, status, 0, none, st);
  if constexpr (D == 128 || D == 256) {
    // the library's own tests can shorten the stage waits or make one copy's barrier never complete (TestHooks):
    // served by an instrumented instantiation, so that the production kernels carry none of it
    const int lim = test_hooks().spin_limit.load(std::memory_order_relaxed);
    const int fb = test_hooks().fault_block.load(std::memory_order_relaxed);
    if (lim > 0 || fb >= 0) {
      const StepArgs hook = {nullptr, nullptr, nullptr, 0, nullptr, nullptr, lim > 0 ? lim : static_cast<int>(kMaxWaitCycles), fb};
      return launch<D, 0, true>(c, q, H_q, 1, attn_scale, 0, C, o_part, m_part, l_part, status, 0, hook, st);
    }
  }
  return launch<D, 0>(c, q, H_q, 1, attn_scale, 0, C, o_part, m_part, l_part, status, 0, none, st);
}

}  // namespace

// Plain decode; stable_tokens > 0 selects the overlapped form (contiguous cache, one query token, no window).
cudaError_t launch_decode_mma(const tq_kv_cache& c, const __half* q, int H_q, int S_q, float attn_scale, int window,
                              int C, float* o_part, float* m_part, float* l_part, int32_t* status, cudaStream_t st,
                              int stable_tokens) {
  return launch_decode_step(c, nullptr, nullptr, q, H_q, S_q, attn_scale, window, C, stable_tokens, o_part, m_part, l_part,
                            nullptr, nullptr, false, status, st, nullptr);
}

// The fused step (tq_sdpa_int4_step): k_new / v_new non-null appends one token, out non-null reduces in the
// same launch (counters then points at B * H_kv + B zeroed ints).  Both null with stable_tokens > 0 is the
// overlapped decode.
cudaError_t launch_decode_step(const tq_kv_cache& c, const __half* k_new, const __half* v_new, const __half* q, int H_q,
                               int S_q, float attn_scale, int window, int C, int stable_tokens, float* o_part,
                               float* m_part, float* l_part, int32_t* counters, void* out, bool out_fp32,
                               int32_t* status, cudaStream_t st, const int32_t* stable_lens) {
  const int sb = stable_tokens > 0 ? stable_tokens / kBlk : 0;
  const StepArgs sa = {k_new, v_new, out, out_fp32 ? 1 : 0, counters, stable_lens, 0, -1};
  // (a window with the step's extras selects the windowed step form: contiguous caches, checked by the caller)
  const bool step = S_q == 1 && (k_new != nullptr || out != nullptr || (window == 0 && (sb > 0 || stable_lens != nullptr)));
  switch (c.d) {
    case 64: return launch<64>(c, q, H_q, S_q, attn_scale, window, C, o_part, m_part, l_part, status, sb, sa, step, st);
    case 128: return launch<128>(c, q, H_q, S_q, attn_scale, window, C, o_part, m_part, l_part, status, sb, sa, step, st);
    case 512: return launch<512>(c, q, H_q, S_q, attn_scale, window, C, o_part, m_part, l_part, status, sb, sa, step, st);
    default: return launch<256>(c, q, H_q, S_q, attn_scale, window, C, o_part, m_part, l_part, status, sb, sa, step, st);
  }
}

}  // namespace tq
