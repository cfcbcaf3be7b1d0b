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
#include "tq_quantize_core.cuh"

namespace tq {
namespace {


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
  quantize_chunk(raw, word, s, z);
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

// Bulk variant: a thread block of 2 * D threads (one per 8 elements) walks over kBulkBlocks consecutive
// destination cache blocks (16 tokens of one KV head, K or V each), so the codes of a block leave as one
// contiguous kilobyte and its scales and zeros, gathered in shared memory, as 16-byte vectors (written one by
// one they were four times as many memory transactions as the codes).  The head dimension is a template
// parameter: every offset inside a block is a compile-time constant per thread.
// grid: (ceil(blocks touched per sequence / kBulkBlocks), B * H_kv, {K, V}).  Registers are capped for 1536
// resident threads per SM: the kernel waits on its loads, and more warps in flight measured faster (203 -> 195 us).
// seq_lens is read only here and bumped by bump_lens_kernel afterwards, so that no block can observe a
// length that another block of the same launch has already advanced.
#ifndef TQ_BULK_BLOCKS
#define TQ_BULK_BLOCKS 8
#endif
constexpr int kBulkBlocks = TQ_BULK_BLOCKS;

template <int D>
__global__ void __launch_bounds__(2 * D, 1536 / (2 * D)) quantize_bulk_kernel(tq_kv_cache c, const __half* k_new, const __half* v_new,
                                                              int T, int32_t* status, int runs) {
  constexpr int CPR = D / 8, NG = D / 32;
  __shared__ __align__(16) __half sm_meta[kBulkBlocks][2][NG][16];  // [block][scale | zero][group][token]
  pdl_launch_dependents();
  pdl_wait();
  const long long bh = blockIdx.y;
  const int b = static_cast<int>(bh / c.H_kv);
  const int len = c.seq_lens[b];
  if (len < 0 || len > c.S_cap - T) return;  // flagged by bump_lens_kernel
  const int which = blockIdx.z;
  const int t = threadIdx.x / CPR, cc = threadIdx.x % CPR;  // token in the block, 8-element chunk in the row
  const int code_off = code_offset(D, which, t, cc * 4);
  const __half* const src = which ? v_new : k_new;
  const long long row_base = bh * T - len;  // row of token `tok` in the input is row_base + tok
  // `runs` > 0 (contiguous cache): quantize_group_kernel does every destination block that lies wholly inside
  // the append; this kernel is then launched with two thread blocks per (sequence, KV head, K | V) for the
  // runs that hold the first and the last block of the append, and writes only partly covered blocks.
  const bool partial_only = runs > 0;
  int run = blockIdx.x;
  if (partial_only && run == 1) {
    run = (((len + T) >> 4) - (len >> 4)) / kBulkBlocks;  // the run of the append's last block
    if (run == 0) return;                                 // same run as the first block
  }
  const int j0 = (len >> 4) + run * kBulkBlocks;
  auto fetch = [&](int j) {
    const int tok = 16 * j + t;
    return (tok >= len && tok < len + T) ? *reinterpret_cast<const uint4*>(src + (row_base + tok) * D + cc * 8)
                                         : make_uint4(0, 0, 0, 0);
  };
  // Interior of the append (every block of this thread block lies entirely inside the new tokens, contiguous
  // cache): no per-thread conditions, and the scales and zeros of all its blocks leave after ONE barrier.
  uint4 raw = fetch(j0);
#pragma unroll 1
  for (int jj = 0; jj < kBulkBlocks; ++jj) {
    const int j = j0 + jj;                                    // destination block
    const int tok_lo = max(16 * j, len), tok_hi = min(16 * j + 16, len + T);
    if (tok_lo >= tok_hi) return;                             // past the end (uniform over the block)
    const uint4 cur = raw;
    if (jj + 1 < kBulkBlocks) raw = fetch(j + 1);             // next block's elements are in flight during the arithmetic
    const int tok = 16 * j + t;
    const bool whole_blk = tok_lo == 16 * j && tok_hi == 16 * j + 16;
    if (partial_only && whole_blk) continue;                  // the group kernel's (uniform over the block)
    const bool active = tok >= tok_lo && tok < tok_hi;
    uint32_t word;
    __half s, z;
    quantize_chunk(cur, word, s, z);
    bool page_ok;
    uint8_t* blk = cache_block_bh(c, bh, b, 16 * j, threadIdx.x == 0 ? status : nullptr, page_ok);
    if (!page_ok) continue;  // a page outside the pool: nothing is written (uniform over the block)
    if (active) *reinterpret_cast<uint32_t*>(blk + code_off) = word;
    const bool whole = tok_lo == 16 * j && tok_hi == 16 * j + 16;
    if ((cc & 3) == 0) {
      if (whole) {
        sm_meta[jj][0][cc >> 2][t] = s;
        sm_meta[jj][1][cc >> 2][t] = z;
      } else if (active) {  // a block only partly covered by this append: write the few values directly
        *reinterpret_cast<__half*>(blk + meta_offset(D, which, 0, cc >> 2, t)) = s;
        *reinterpret_cast<__half*>(blk + meta_offset(D, which, 1, cc >> 2, t)) = z;
      }
    }
    if (!whole) continue;  // uniform over the block
    __syncthreads();       // one barrier per block: each block has its own buffer
    // scales [NG][16] then zeros [NG][16] are adjacent in the cache block: 2 * NG * 32 bytes
    constexpr int kVecs = NG * 2;  // 16-byte vectors per array
    if (threadIdx.x < 2 * kVecs) {
      const int arr = threadIdx.x / kVecs, v = threadIdx.x % kVecs;
      const uint4 val = reinterpret_cast<const uint4*>(&sm_meta[jj][arr][0][0])[v];
      reinterpret_cast<uint4*>(blk + meta_offset(D, which, arr, 0, 0))[v] = val;
    }
  }
}

// Full blocks of a bulk append (contiguous cache): every destination cache block that lies wholly inside the
// new tokens.  One THREAD per quantisation group of 32 elements: the per-group work (two divisions, a
// reciprocal, the bound) is paid once per 32 elements instead of once per 8 by each lane of a quad, and no
// shuffle is needed -- 430 instead of 650 instructions per 32 elements.  A warp owns 32 / (D/32) token rows of K
// or of V of a destination block: 2 KB of input, contiguous, read as four 16-byte loads per lane with the next
// block's loads in flight during the arithmetic; each lane stores its 16-byte code chunk straight to the
// cache block (eight neighbouring lanes fill one 128-byte line); the warp's 128 bytes of scales and zeros are
// gathered in shared memory and leave as one 4-byte store per lane.  No block-wide barrier.  A thread block
// walks over group_run consecutive destination blocks of one (sequence, KV head); the host picks group_run so
// that the grid is a whole number of waves.  Partly covered blocks, and
// paged caches, are left to quantize_bulk_kernel.  (Staging the input through bulk asynchronous copies was
// measured and is slower here: 200 - 250 us per 128K layer against 178.)
#ifndef TQ_QG_WARPS
#define TQ_QG_WARPS 24  // resident warps per SM the kernel is compiled for (80 registers per thread)
#endif
template <int D>
__global__ void __launch_bounds__(D, TQ_QG_WARPS * 32 / D) quantize_group_kernel(tq_kv_cache c, const __half* k_new, const __half* v_new, int T,
                                                            int32_t* status, int group_run) {
  constexpr int NG = D / 32, NW = NG;        // groups per row; warps per thread block
  constexpr int TPW = 32 / NG;               // token rows per warp
  constexpr int kBlock = 16 * (D + D / 4);
  constexpr int VW = 2 * TPW;                // bytes of one (array, group) run of this warp's scales or zeros
  __shared__ __align__(16) uint8_t meta_all[NW * 128];
  (void)status;
  pdl_launch_dependents();
  pdl_wait();
  const long long bh = blockIdx.y;
  const int b = static_cast<int>(bh / c.H_kv);
  const int len = c.seq_lens[b];
  if (len < 0 || len > c.S_cap - T || c.page_table != nullptr) return;
  const int jf0 = (len + 15) >> 4, jf1 = (len + T) >> 4;  // full blocks of the append: [jf0, jf1)
  const int j0 = jf0 + blockIdx.x * group_run;
  const int nrun = min(group_run, jf1 - j0);
  if (nrun <= 0) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int which = warp / (NW / 2), tok0 = (warp % (NW / 2)) * TPW;  // K or V; first token row of this warp
  const int tok = tok0 + lane / NG, g = lane % NG;
  uint8_t* const meta = meta_all + warp * 128;
  // lane order is row order: this lane's 64 bytes of the warp's 2 KB
  const uint4* src = reinterpret_cast<const uint4*>((which ? v_new : k_new) + (bh * T - len + 16LL * j0 + tok0) * D) + lane * 4;
  uint8_t* const dst0 = c.blocks + (bh * (c.S_cap >> 4) + j0) * static_cast<long long>(kBlock);
  const uint32_t code_at = code_offset(D, which, tok, g * 16);
  // scales and zeros of the warp in shared memory: [scale | zero][group][TPW tokens] halves = 128 bytes;
  // lane l later stores bytes 4l .. 4l+3 of it, which belong to array a_l, group g_l
  const uint32_t s_at = (g * TPW + (tok - tok0)) * 2, z_at = 64 + s_at;
  const int a_l = (4 * lane) / 64, g_l = ((4 * lane) % 64) / VW, off_l = (4 * lane) % VW;
  const uint32_t meta_dst = meta_offset(D, which, a_l, g_l, tok0) + off_l;
  constexpr int kStep = 16 * D * 2 / 16;  // 16-byte units from one block's rows to the next block's
  auto fetch = [&](uint4 (&r)[4], const uint4* p) {
#pragma unroll
    for (int i = 0; i < 4; ++i) r[i] = __ldg(p + i);
  };
  auto emit = [&](const uint4 (&raw)[4], int jj) {
    uint32_t w[4];
    __half sq, zq;
    quantize_group32(raw, w, sq, zq);
    uint8_t* const blk = dst0 + static_cast<long long>(jj) * kBlock;
    *reinterpret_cast<uint4*>(blk + code_at) = make_uint4(w[0], w[1], w[2], w[3]);
    *reinterpret_cast<__half*>(meta + s_at) = sq;
    *reinterpret_cast<__half*>(meta + z_at) = zq;
    __syncwarp();
    *reinterpret_cast<uint32_t*>(blk + meta_dst) = *reinterpret_cast<const uint32_t*>(meta + 4 * lane);
    __syncwarp();  // the 128 bytes are read before the next block overwrites them
  };
  // two register buffers taken in turn: the next block's loads are in flight during the arithmetic and no
  // register is copied
#ifndef TQ_QG_PF
#define TQ_QG_PF 2  // blocks ahead of the register loads that are prefetched into L2 (0: none; measured 128.7 / 125.6 / 129.5 / 140.0 us for 0 / 2 / 3 / 5)
#endif
  auto ahead = [&](const uint4* p) {  // this lane's 64 bytes of a later block, into L2
    if (TQ_QG_PF > 0) asm volatile("prefetch.global.L2 [%0];\n" ::"l"(p));
  };
  uint4 ra[4], rb[4];
  fetch(ra, src);
  if (TQ_QG_PF > 1) {
#pragma unroll
    for (int a = 2; a <= TQ_QG_PF; ++a)
      if (a < nrun) ahead(src + a * kStep);
  }
#pragma unroll 1
  for (int jj = 0; jj < nrun; jj += 2) {
    if (jj + 1 < nrun) fetch(rb, src + kStep);
    if (jj + 1 + TQ_QG_PF < nrun) ahead(src + (1 + TQ_QG_PF) * kStep);
    emit(ra, jj);
    if (jj + 1 >= nrun) break;
    if (jj + 2 < nrun) fetch(ra, src + 2 * kStep);
    if (jj + 2 + TQ_QG_PF < nrun) ahead(src + (2 + TQ_QG_PF) * kStep);
    emit(rb, jj + 1);
    src += 2 * kStep;
  }
}

// Compares div_rn_by_reciprocal with the true division on every quotient the quantiser can form: block x
// takes the finite binary16 number a with index x, its threads walk over every finite b.  (i) fl(a - b) / 15
// for a > b; (ii) (0 - a) / b for b > 0.  Mismatches are counted in *bad.  Test support.
__device__ __forceinline__ float finite_half(int idx) {  // 0 .. 31743: +0 .. 65504; 31744 .. 63487: -0 .. -65504
  const unsigned short bits = idx < 31744 ? idx : 0x8000 + (idx - 31744);
  return __half2float(__ushort_as_half(bits));
}
__global__ void division_check_kernel(unsigned long long* bad) {
  const float a = finite_half(blockIdx.x);
  unsigned long long n = 0;
  for (int j = threadIdx.x; j < 63488; j += blockDim.x) {
    const float b = finite_half(j);
    if (a > b) {  // (a zero range never uses the shortcut's result: its scale is zero and the defining arithmetic takes over)
      const float d = __fsub_rn(a, b);
      n += __float_as_uint(__fdiv_rn(d, 15.0f)) != __float_as_uint(div_rn_by_15(d));
    }
    if (b > 0.0f) {
      const float num = __fsub_rn(0.0f, a);
      n += __float_as_uint(__fdiv_rn(num, b)) != __float_as_uint(div_rn_by_reciprocal(num, b, __frcp_rn(b)));
    }
  }
  if (n) atomicAdd(bad, n);
}

__global__ void bump_lens_kernel(tq_kv_cache c, int T, int32_t* status) {
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= c.B) return;
  const int len = c.seq_lens[b];
  if (len < 0 || len > c.S_cap - T) {
    if (status) atomicOr(status, TQ_STATUS_CACHE_FULL);
    return;
  }
  c.seq_lens[b] = len + T;
}

// Decode-step variant (small T): one block per sequence quantises K and V of all its KV heads,
// then advances the length itself -- a single launch, and no block reads another's length.
__global__ void __launch_bounds__(256) quantize_step_kernel(tq_kv_cache c, const __half* k_new, const __half* v_new,
                                                            int T, int32_t* status) {
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.x;
  const int len = c.seq_lens[b];
  if (len < 0 || len > c.S_cap - T) {
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

template <int D>
cudaError_t launch_group(dim3 grid, cudaStream_t st, const tq_kv_cache& c, const __half* k_new, const __half* v_new, int T,
                         int32_t* status, int group_run) {
  return launch_kernel(quantize_group_kernel<D>, grid, dim3(D), 0, st, c, k_new, v_new, T, status, group_run);
}

}  // namespace

cudaError_t launch_quantize_append(const tq_kv_cache& c, const __half* k_new, const __half* v_new, int T,
                                   int32_t* status, cudaStream_t st) {
  const long long per_seq = static_cast<long long>(c.H_kv) * T * (c.d >> 3);
  if (2 * per_seq <= 8192) {
    return launch_kernel(quantize_step_kernel, dim3(c.B), dim3(256), 0, st, c, k_new, v_new, T, status);
  } else {
    const int touched = (T + 15) / 16 + 1;  // destination blocks a sequence's new tokens can reach
    const int runs = (touched + kBulkBlocks - 1) / kBulkBlocks;
    const bool paged = c.page_table != nullptr;
    // partly covered blocks (and all of a paged cache) by the general kernel, full blocks by the group kernel;
    // the two write disjoint cache blocks
    dim3 grid(static_cast<unsigned>(paged ? runs : 2), static_cast<unsigned>(c.B * c.H_kv), 2);
    const int edge_runs = paged ? 0 : runs;
    cudaError_t e;
    switch (c.d) {
      case 64: e = launch_kernel(quantize_bulk_kernel<64>, grid, dim3(128), 0, st, c, k_new, v_new, T, status, edge_runs); break;
      case 128: e = launch_kernel(quantize_bulk_kernel<128>, grid, dim3(256), 0, st, c, k_new, v_new, T, status, edge_runs); break;
      case 256: e = launch_kernel(quantize_bulk_kernel<256>, grid, dim3(512), 0, st, c, k_new, v_new, T, status, edge_runs); break;
      default: e = launch_kernel(quantize_bulk_kernel<512>, grid, dim3(1024), 0, st, c, k_new, v_new, T, status, edge_runs); break;
    }
    if (e != cudaSuccess) return e;
    if (!paged && T >= 16) {
      // Run length: about 32 blocks per thread block, adjusted so that the thread blocks (TQ_QG_WARPS warps' worth
      // of them are resident per SM) make a whole number of waves.
      const long long bhn = static_cast<long long>(c.B) * c.H_kv, nb = T / 16;
      const long long slots = static_cast<long long>(device_sm_count()) * (TQ_QG_WARPS * 32) / c.d;
      const long long waves = std::max(1LL, (bhn * nb + 32 * slots - 1) / (32 * slots));
      const long long per_bh = std::max(1LL, waves * slots / bhn);  // thread blocks per (sequence, KV head)
      const int group_run = static_cast<int>(std::max(1LL, (nb + per_bh - 1) / per_bh));
      dim3 ggrid(static_cast<unsigned>((nb + group_run - 1) / group_run), static_cast<unsigned>(bhn));
      switch (c.d) {
        case 64: e = launch_group<64>(ggrid, st, c, k_new, v_new, T, status, group_run); break;
        case 128: e = launch_group<128>(ggrid, st, c, k_new, v_new, T, status, group_run); break;
        case 256: e = launch_group<256>(ggrid, st, c, k_new, v_new, T, status, group_run); break;
        default: e = launch_group<512>(ggrid, st, c, k_new, v_new, T, status, group_run); break;
      }
      if (e != cudaSuccess) return e;
    }
    return launch_kernel(bump_lens_kernel, dim3((c.B + 127) / 128), dim3(128), 0, st, c, T, status);
  }
}

// Runs division_check_kernel on the current device; returns the number of mismatches, or -1 on a CUDA error.
long long run_division_check() {
  unsigned long long* bad = nullptr;
  unsigned long long host = 0;
  if (cudaMalloc(&bad, sizeof(*bad)) != cudaSuccess) return -1;
  cudaError_t e = cudaMemset(bad, 0, sizeof(*bad));
  if (e == cudaSuccess) {
    division_check_kernel<<<63488, 256>>>(bad);
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaMemcpy(&host, bad, sizeof(host), cudaMemcpyDeviceToHost);
  cudaFree(bad);
  return e == cudaSuccess ? static_cast<long long>(host > 0x7fffffffULL ? 0x7fffffffULL : host) : -1;
}

}  // namespace tq
