/*
 * tq.h -- C ABI of libtq: fused int4 compressed-domain decode attention for NVIDIA B200 (sm_100a).
 *
 * The library implements the decode-time hot path of "Open-TQ-Metal": the KV cache is kept in
 * per-group asymmetric int4 (Sec. 2.1, Eq. 2-3), new tokens are quantised and appended in
 * place, and single-query attention is computed directly on the packed cache (Sec. 3.1,
 * Algorithm 1) with split-K over the sequence (Sec. 3.2) followed by the reduction of Eq. 5.
 *
 * General rules
 *   - Every pointer named below is a DEVICE pointer unless it says "host".  The caller owns all
 *     memory; the library allocates nothing, keeps no state between calls and never
 *     synchronises.  Work is enqueued on `stream` (a cudaStream_t passed as void*; NULL is the
 *     default stream) and is ordered by it.
 *   - All device pointers must be 16-byte aligned (m_part, l_part, seq_lens, page_table and status: 4-byte).
 *   - Every entry point returns a tq_result.  Errors that the host can see (null pointer, bad
 *     shape, bad alignment, workspace too small) are returned before anything is launched.
 *   - Conditions only the device can see (a full cache, an empty sequence) OR bits into the
 *     caller's `status` word (int32 in device memory, may be NULL) and the offending piece of
 *     work is skipped; kernels never trap and every wait inside them is bounded.
 *   - fp16 means IEEE binary16; such buffers are declared `void*` / `uint16_t*` (bit patterns).
 *
 * Data format (Sec. 2.1).  A K or V vector of `d` elements (one token, one KV head) is cut into
 * d/32 groups of 32 consecutive elements.  Each group stores
 *     scale s = fp16((max - min) / 15),   zero z = fp16(-min / s)   (z is real-valued, not an integer)
 *     code  q = clamp(round_half_even(x / s + z), 0, 15)            (s the stored fp16 value)
 * and reconstructs x^ = (q - z) * s.  Codes are packed two per byte, element 2b in the low nibble
 * of byte b and element 2b+1 in the high nibble (the order implied by the masks of Eq. 4).  That
 * is 20 bytes per 32 elements, 3.2x smaller than fp16.  The quantiser is evaluated in IEEE
 * binary32 with one rounding per operation (true division, no fused multiply-add); a group whose
 * scale rounds to zero in fp16 stores s = 1, z = -min and all codes 0; z is clamped to +-65504.
 */
#ifndef TQ_H_
#define TQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum tq_result {
  TQ_OK = 0,
  TQ_ERR_NULL = 1,      /* a required pointer is NULL */
  TQ_ERR_SHAPE = 2,     /* unsupported or inconsistent sizes (see each function) */
  TQ_ERR_ALIGN = 3,     /* a device pointer is not 16-byte aligned */
  TQ_ERR_WORKSPACE = 4, /* workspace_bytes smaller than tq_dequant_workspace_bytes() */
  TQ_ERR_CUDA = 5       /* a CUDA call failed; tq_last_cuda_error() has the code */
} tq_result;

/* bits OR-ed into the device status word */
#define TQ_STATUS_CACHE_FULL 1 /* quantize_append: seq_lens[b] + T > S_cap; that sequence was skipped */
#define TQ_STATUS_EMPTY_SEQ 2  /* attention over a sequence with seq_lens[b] <= 0; its output is zero */
#define TQ_STATUS_BAD_LEN 4    /* seq_lens[b] outside [0, S_cap]; treated as clamped to that range */
#define TQ_STATUS_TIMEOUT 8    /* a bounded wait for an asynchronous copy ran out; that call's results are not valid */
#define TQ_STATUS_BAD_PAGE 16  /* a page-table entry outside [0, num_pages) was met */

#define TQ_GROUP 32         /* quantisation group size g (fixed) */
#define TQ_SPLIT_QUANTUM 16 /* split boundaries fall on multiples of this many tokens */

/*
 * The int4 KV cache of ONE layer.  The paper fixes the values (codes, fp16 scale, fp16 zero per
 * group of 32) but not how they are laid out; the layout here is built for the decode kernel, which
 * fetches a whole 16-token block of one KV head with a single bulk copy.
 *
 * `blocks` is an array [B][H_kv][S_cap / 16] of blocks, each TQ_BLOCK_BYTES(d) = 16 * (d + d/4) bytes
 * (2560 at d = 128).  Block j of (sequence b, KV head h) holds tokens 16j .. 16j+15 as
 *     K codes | V codes | K scales | K zeros | V scales | V zeros
 *   codes (16 * d/2 bytes each): token t of the block is the d/2-byte row t; inside a row the 16-byte
 *     chunks (32 codes = one group each) are stored in XOR-swizzled order: group g of token t sits at
 *     chunk position g ^ ((t >> shift) & (d/32 - 1)), shift = 2, 1, 0, 0 for d = 64, 128, 256, 512 -- the
 *     bank-conflict-free shared-memory layout, kept in global memory so that no rearrangement is
 *     needed on the way in.  Within a chunk, element 2i is the low nibble of byte i.
 *   scales, zeros (d/32 * 16 fp16 each): value of (group g, token t) at index g * 16 + t.
 * Use tq_cache_code_offset / tq_cache_meta_offset to address single elements from the host.
 * Rows at or beyond seq_lens[b] are unspecified.
 * Requirements: d in {64, 128, 256, 512} (512: the paper's Gemma global layers, Table 7); S_cap a
 * positive multiple of 16; B, H_kv >= 1.
 */
#define TQ_BLOCK_TOKENS 16
#define TQ_BLOCK_BYTES(d) (16 * ((d) + (d) / 4))
typedef struct tq_kv_cache {
  uint8_t* blocks;    /* [B][H_kv][S_cap/16][TQ_BLOCK_BYTES(d)]; with paging: the page pool, see below */
  int32_t* seq_lens;  /* [B] number of valid tokens per sequence (device memory, updated by append) */
  int32_t B, H_kv, S_cap, d;
  /*
   * Paging (optional; the paper's cache is one growing tensor per layer and it names cache management as its
   * end-to-end overhead, Sec. 5 and 6.3; pages are the usual way to serve ragged batches from one pool).
   * page_table == NULL: the contiguous layout above, the three integers are ignored.  Otherwise `blocks` is a
   * pool [num_pages][H_kv][page_tokens/16][TQ_BLOCK_BYTES(d)], page_table is device memory
   * [B][max_pages] int32, entry (b, i) names the pool page that holds tokens i*page_tokens ..
   * (i+1)*page_tokens - 1 of sequence b (for all KV heads), and S_cap must equal max_pages * page_tokens.
   * Only the entries below ceil(seq_lens[b] / page_tokens) (after an append: of the new length) are read.
   * An entry outside [0, num_pages) sets TQ_STATUS_BAD_PAGE and is treated as page 0 by readers and
   * skipped by writers.  page_tokens is a power of two, at least 16.  Every entry point takes either form.
   */
  const int32_t* page_table;
  int32_t page_tokens, max_pages, num_pages;
} tq_kv_cache;

/* Byte offset inside a block of code byte `byte` (0 .. d/2-1) of token `t` (0 .. 15); which = 0 for K, 1 for V. */
size_t tq_cache_code_offset(int32_t d, int32_t which, int32_t t, int32_t byte);
/* Byte offset inside a block of the fp16 scale (is_zero = 0) or zero (1) of group g, token t; which = 0 K, 1 V. */
size_t tq_cache_meta_offset(int32_t d, int32_t which, int32_t is_zero, int32_t g, int32_t t);

/*
 * Quantise T new tokens per sequence and append them in place (Sec. 2.1, Eq. 2-3; Sec. 1 describes the
 * cache as quantised while tokens are generated).  The paper's implementation appends by concatenation and names
 * that as its main end-to-end overhead; here the cache is pre-allocated and rows are written at
 * positions seq_lens[b] .. seq_lens[b] + T - 1.
 *   k_new, v_new : [B][H_kv][T][d] fp16, read only.
 *   T >= 1.  On return (in stream order) seq_lens[b] has grown by T for every sequence that had
 *   room; a sequence with seq_lens[b] + T > S_cap is left untouched and TQ_STATUS_CACHE_FULL is
 *   set.  T = S with seq_lens = 0 is the bulk quantisation of a prefilled cache.
 * Errors: TQ_ERR_NULL, TQ_ERR_SHAPE (cache requirements, T < 1), TQ_ERR_ALIGN, TQ_ERR_CUDA.
 */
int tq_kv_quantize_append(const tq_kv_cache* cache /* host */, const void* k_new, const void* v_new, int32_t T,
                          int32_t* status, void* stream);

/*
 * Number of sequence splits C the library would pick for a decode step over sequences of up to
 * `max_seq_len` tokens (host function; it launches nothing, but the first call on a device asks the CUDA
 * runtime for the SM count of the current device and remembers it per device).  Chosen from the SM count: with few
 * (sequence, KV head) pairs, B * H_kv * ceil(G / 8) * C thread blocks fill the GPU in one wave of
 * equal splits (at least 512 tokens each); with a batch, in about four waves (splits of at least
 * 2048 tokens), so that sequences of different lengths even out.  Always in [1, TQ_MAX_SPLITS].
 */
#define TQ_MAX_SPLITS 256
int32_t tq_auto_splits(int32_t B, int32_t H_kv, int32_t H_q, int32_t d, int32_t max_seq_len);

/*
 * Token range of split c of a sequence of `len` tokens cut into C splits (host function): with
 * nb = ceil(len / 16), split c covers tokens [16 * floor(c * nb / C), min(len, 16 * floor((c + 1) * nb / C))).
 * This is the partition tq_sdpa_int4_decode uses; exposed so that partials can be checked.  With a
 * sliding window the same rule applies to the blocks that overlap [len - window, len), and the first
 * split starts at len - window.
 */
void tq_split_range(int32_t len, int32_t C, int32_t c, int32_t* t0 /* host */, int32_t* t1 /* host */);

/*
 * Phase 1 of the fused int4 attention (Sec. 3.1 Algorithm 1 run per split, Sec. 3.2): for every
 * sequence b, query head h and split c, attend over the split's tokens reading packed codes,
 * scales and zeros straight from the cache, dequantising in registers, and write the partial
 * triple of Sec. 3.2:
 *   o_part [B][H_q][C][d] fp32   partial output, already divided by l_part (as Eq. 5 expects)
 *   m_part [B][H_q][C]    fp32   maximum of attn_scale * q.k^ over the split (natural-log units)
 *   l_part [B][H_q][C]    fp32   sum over the split of exp(score - m_part)
 * An empty split writes o = 0, m = -inf, l = 0.
 *   q          : [B][H_q][d] fp16.  Query head h reads KV head h / (H_q / H_kv) (Sec. 3.1, GQA).
 *   attn_scale : the factor alpha in alpha * q.k (1/sqrt(d) for Llama, 1.0 for Gemma-style models).
 *   num_splits : C >= 1, or 0 for tq_auto_splits(B, H_kv, H_q, d, S_cap).
 * All seq_lens[b] cached tokens are attended (no mask).  Requirements: H_q a multiple of H_kv,
 * H_q / H_kv <= 64, C <= TQ_MAX_SPLITS.
 * Errors: TQ_ERR_NULL, TQ_ERR_SHAPE, TQ_ERR_ALIGN, TQ_ERR_CUDA.  Status: TQ_STATUS_EMPTY_SEQ, TQ_STATUS_BAD_LEN,
 * TQ_STATUS_TIMEOUT (a bulk copy did not complete within the bound: that call's partials are not valid), and
 * TQ_STATUS_BAD_PAGE with a paged cache.
 */
int tq_sdpa_int4_decode(const tq_kv_cache* cache /* host */, const void* q, int32_t H_q, float attn_scale,
                        int32_t num_splits, float* o_part, float* m_part, float* l_part, int32_t* status,
                        void* stream);

/*
 * Phase 1 overlapped with the work before it in the stream (the paper's Sec. 3.2 two-phase attention, unchanged
 * in what it computes; the paper orders its two Metal dispatches through the framework's graph, here the
 * ordering against the preceding kernel is relaxed where the data allows it).  The ordinary call starts by
 * waiting for everything enqueued before it, because the quantize-append just before it may still be writing
 * the newest tokens and the length.  A decode step, however, reads almost only tokens that were written
 * steps ago.  The caller states how many:
 *   stable_tokens : every sequence's cached tokens [0, stable_tokens) -- rounded down to a multiple of 16 --
 *                   and all of q are FINAL before the preceding work in the stream starts: nothing that can
 *                   still be running when this call's kernel starts writes them.  (Typically the shortest
 *                   sequence length before this step's append.  libtq's own kernels let their successor be
 *                   scheduled as soon as they start, so "the preceding work" reaches back to the last kernel
 *                   that was not launched with programmatic dependent launch, or to the last synchronisation.)
 * The kernel then streams and attends the stable tokens at once, waits for the preceding kernel only after
 * that, reads seq_lens[b], and lets its last split attend the tokens [stable_tokens, seq_lens[b]).  The splits
 * therefore partition the stable part, not the whole sequence: tq_split_range_stable gives the partition; keep
 * stable_tokens close to the lengths or the last split grows (inside a replayed CUDA graph the value is fixed at
 * capture time: re-capture, or update the node, every few hundred steps).
 * seq_lens[b] < stable_tokens breaks the promise: TQ_STATUS_BAD_LEN is set and that sequence's result is not valid.
 * With stable_tokens / 16 below the split count the call is exactly tq_sdpa_int4_decode.  With a paged cache the
 * promise also covers the page-table entries of the stable tokens' pages (they are read before the wait too).
 * num_splits = 0 picks tq_auto_splits_step(B, H_kv, H_q, d, S_cap).
 * Everything else (arguments, partial layout, errors, status) as tq_sdpa_int4_decode; stable_tokens < 0 or
 * > S_cap is TQ_ERR_SHAPE.  On the 128K Llama-shaped layer the overlap is worth about 3 us per launch.
 */
int tq_sdpa_int4_decode_overlapped(const tq_kv_cache* cache /* host */, const void* q, int32_t H_q, float attn_scale,
                                   int32_t num_splits, int32_t stable_tokens, float* o_part, float* m_part,
                                   float* l_part, int32_t* status, void* stream);
/* Token range of split c under tq_sdpa_int4_decode_overlapped (host function): with sb = stable_tokens / 16 >= C,
 * split c covers tokens [16 * floor(c * sb / C), 16 * floor((c + 1) * sb / C)), and the last one reaches to len;
 * with sb < C it is tq_split_range(len, C, c). */
void tq_split_range_stable(int32_t len, int32_t stable_tokens, int32_t C, int32_t c, int32_t* t0 /* host */,
                           int32_t* t1 /* host */);

/*
 * One decode step of one layer in a single launch: the quantize-append of the new token (Sec. 2.1), the fused
 * int4 attention over the cache including it (Sec. 3.1, 3.2) and the reduction of Eq. 5.  The paper runs these as
 * separate dispatches chained through its framework; here one kernel does all three, so a step costs one
 * launch (what short contexts are made of) and consecutive layers' steps follow each other without the two
 * hand-overs in between.  The result is that of tq_kv_quantize_append (T = 1), tq_sdpa_int4_decode_overlapped
 * and tq_sdpa_int4_combine called in that order, up to the summation order of the reduction.
 *   k_new, v_new : [B][H_kv][1][d] fp16, or both NULL for a step that appends nothing.  The row of KV head h is
 *                  quantised by the thread block of that head's last split, written to the cache, and read
 *                  back by the same block; seq_lens[b] is advanced by the last block of the sequence to have
 *                  read the old value.  A full cache sets TQ_STATUS_CACHE_FULL and attends the old tokens only.
 *   stable_tokens: as in tq_sdpa_int4_decode_overlapped (the promise covers q and the first stable_tokens cached
 *                  tokens; k_new / v_new are read after the wait for the preceding kernel).  0 or a value below
 *                  16 * C: nothing is read early and the splits partition the whole sequence.
 *   workspace    : tq_step_workspace_bytes(...) bytes, 16-byte aligned: counters, then the split partials.
 *                  ZERO the first tq_step_counter_bytes(B, H_kv) bytes once before the first use (cudaMemsetAsync);
 *                  every launch leaves them zero again.  After a TQ_STATUS_TIMEOUT zero them again.  Launches that may
 *                  overlap on the GPU (other streams) need workspaces of their own.
 *   out          : [B][H_q][d] fp16 or fp32, written by the last thread block of each (sequence, KV head) to finish.
 *   num_splits   : C >= 1, or 0 for tq_auto_splits_step(B, H_kv, H_q, d, S_cap).
 * Contiguous and paged caches alike (paged: the page that the new token falls into must be in the table; an entry
 * outside the pool sets TQ_STATUS_BAD_PAGE and that row is not written).  Restriction: H_q / H_kv <= 8; otherwise
 * TQ_ERR_SHAPE -- use the three calls.  Errors: TQ_ERR_NULL, TQ_ERR_SHAPE, TQ_ERR_ALIGN, TQ_ERR_WORKSPACE, TQ_ERR_CUDA.  Status as the three calls.
 */
int tq_sdpa_int4_step(const tq_kv_cache* cache /* host */, const void* k_new, const void* v_new, const void* q,
                      int32_t H_q, float attn_scale, int32_t num_splits, int32_t stable_tokens, void* workspace,
                      size_t workspace_bytes, void* out, int32_t out_is_fp32, int32_t* status, void* stream);
/*
 * The same step with one stable part PER SEQUENCE, for batches of unequal lengths (the ragged batch of decode
 * steps): stable_lens is a DEVICE array of B int32, stable_lens[b] = the number of oldest cached tokens of sequence
 * b that are final before the preceding work in the stream starts; the array itself and q are covered by the same
 * promise (the kernel reads them before it waits for its predecessor).  Values are clamped to [0, S_cap] and
 * rounded down to a multiple of 16; a sequence whose stable part holds fewer 16-token blocks than there are splits
 * starts nothing early.  seq_lens[b] < stable_lens[b] sets TQ_STATUS_BAD_LEN.  Everything else as
 * tq_sdpa_int4_step; stable_lens == NULL is TQ_ERR_NULL.  The paper has no counterpart (its batches are single
 * sequences).
 */
int tq_sdpa_int4_step_ragged(const tq_kv_cache* cache /* host */, const void* k_new, const void* v_new, const void* q,
                             int32_t H_q, float attn_scale, int32_t num_splits, const int32_t* stable_lens /* device */,
                             void* workspace, size_t workspace_bytes, void* out, int32_t out_is_fp32, int32_t* status,
                             void* stream);
/*
 * The same step over a sliding window (Appendix A: Gemma's sliding-attention layers, w = 1024): append, attention
 * over the last `window` tokens of every sequence (the new one included) and the reduction in one launch.  A
 * window layer's step is made of latencies more than of bytes (5 MB at w = 1024 with 16 KV heads of d = 256), so
 * what counts is one launch instead of three and not waiting for the preceding kernel before streaming:
 *   stable_tokens : 0, or a promise as in tq_sdpa_int4_decode_overlapped, here with an upper bound too: every
 *                   sequence's length when the kernel reads it lies in [stable_tokens, stable_tokens +
 *                   TQ_WINDOW_SLACK], the tokens below stable_tokens and q are final.  The blocks that are inside
 *                   the window for every such length (from stable_tokens + TQ_WINDOW_SLACK - window up to
 *                   stable_tokens) are then attended before the wait for the preceding kernel, split evenly; the
 *                   last split attends the few tokens at the two ends after it.  A length outside the promised
 *                   range sets TQ_STATUS_BAD_LEN.  0, or fewer such blocks than splits: nothing is read early
 *                   (the general windowed form).
 * window >= 1; num_splits = 0 picks tq_auto_splits(B, H_kv, H_q, d, window); contiguous caches only (a paged cache
 * is TQ_ERR_SHAPE: use the three calls); everything else as tq_sdpa_int4_step.
 */
#define TQ_WINDOW_SLACK 128
int tq_sdpa_int4_step_window(const tq_kv_cache* cache /* host */, const void* k_new, const void* v_new, const void* q,
                             int32_t H_q, float attn_scale, int32_t window, int32_t num_splits, int32_t stable_tokens,
                             void* workspace, size_t workspace_bytes, void* out, int32_t out_is_fp32, int32_t* status,
                             void* stream);
size_t tq_step_workspace_bytes(int32_t B, int32_t H_kv, int32_t H_q, int32_t d, int32_t num_splits);
/*
 * Split count that tq_sdpa_int4_step and tq_sdpa_int4_decode_overlapped pick for num_splits = 0 (host function).
 * Like tq_auto_splits, but when one wave of thread blocks would fill the GPU it leaves an eighth of the resident
 * slots (at least one per (sequence, KV head)) unused: launches of these entry points overlap their predecessor,
 * and with every slot taken the blocks that finish a launch last (those that also reduce the partials) hold up
 * the first blocks of the next one.  Measured on the 128K Llama-shaped step (8 KV heads, 296 slots), us per layer
 * by number of splits: 37: 34.7, 36: 30.2, 32: 29.9, 28: 29.9, 24: 30.5; the 32K step: 36: 11.9, 32: 11.6, 28: 11.8.
 * (A step that declares no stable part overlaps nothing: there every slot is worth taking, 35.8 us per layer with
 * 37 splits against 37.5 with 32, and tq_auto_splits gives the better count.)
 * The slots are left only where (sequences x KV heads) is at most 1/32 of them (with 16 KV heads the d = 256
 * shape measured 39.0 us with one spare slot per KV head and 37.4 us without).  For a batch (more than a quarter of the slots per split) it picks about
 * three and a half waves of thread blocks instead of tq_auto_splits' four: the overlap fills a launch's tail.
 * Up to 1024 tokens it picks one split: with num_splits = 1 the step's thread blocks write `out` themselves
 * (Eq. 5 with a single term), without partials, arrival counter or second pass.
 */
int32_t tq_auto_splits_step(int32_t B, int32_t H_kv, int32_t H_q, int32_t d, int32_t max_seq_len);
size_t tq_step_counter_bytes(int32_t B, int32_t H_kv);

/*
 * Phase 1 restricted to a sliding window (Appendix A: Gemma's sliding-attention layers, w = 1024, which
 * the paper's kernel serves by skipping tokens inside its loop): sequence b attends only its last `window`
 * tokens, [max(0, seq_lens[b] - window), seq_lens[b]).  Here the skip is not per token: the splits
 * partition the window only, so tokens outside it are never fetched.  window = 0 means no window
 * (identical to tq_sdpa_int4_decode); window < 0 is TQ_ERR_SHAPE.  num_splits = 0 picks
 * tq_auto_splits(B, H_kv, H_q, d, min(window, S_cap)).  Everything else as tq_sdpa_int4_decode; combine
 * with tq_sdpa_int4_combine.  tq_split_range_window gives the partition.
 */
int tq_sdpa_int4_decode_window(const tq_kv_cache* cache /* host */, const void* q, int32_t H_q, float attn_scale,
                               int32_t window, int32_t num_splits, float* o_part, float* m_part, float* l_part,
                               int32_t* status, void* stream);
void tq_split_range_window(int32_t len, int32_t window, int32_t C, int32_t c, int32_t* t0 /* host */,
                           int32_t* t1 /* host */);

/*
 * Phase 1 for several query tokens per sequence (the S_q factor of the grid in Appendix A; speculative or
 * chunked decode).  The S_q query tokens are the S_q newest tokens of each sequence and must already be in
 * the cache (one tq_kv_quantize_append with T = S_q).  The paper does not say what each of them attends; here
 * it is causal: query token s (0 = oldest) attends cached tokens [lo_s, hi_s) with
 *   hi_s = seq_lens[b] - (S_q - 1 - s),   lo_s = max(0, hi_s - window)   (window = 0: lo_s = 0),
 * each through its quantised K/V.  A query token with hi_s <= 0 attends nothing and gives o = 0, l = 0.
 *   q       : device, fp16 [B][S_q][H_q][d]
 *   o_part  : device, fp32 [B][S_q][H_q][C][d];  m_part, l_part : device, fp32 [B][S_q][H_q][C]
 * i.e. the layouts of tq_sdpa_int4_decode with S_q * H_q in place of H_q, so tq_sdpa_int4_combine with
 * H_q' = S_q * H_q reduces them to out [B][S_q][H_q][d].  The (query token, head) pairs that share a KV head
 * are packed eight to a thread block like plain GQA heads, so S_q * (H_q / H_kv) <= 8 costs one pass over the
 * cache.  Splits partition the tokens [lo_0, seq_lens[b]); num_splits = 0 picks
 * tq_auto_splits(B, H_kv, S_q * H_q, d, span).  S_q = 1 is tq_sdpa_int4_decode_window.
 * Errors as tq_sdpa_int4_decode, plus TQ_ERR_SHAPE for S_q outside 1..TQ_MAX_QUERY_TOKENS.
 */
#define TQ_MAX_QUERY_TOKENS 64
int tq_sdpa_int4_decode_multi(const tq_kv_cache* cache /* host */, const void* q, int32_t H_q, int32_t S_q,
                              float attn_scale, int32_t window, int32_t num_splits, float* o_part, float* m_part,
                              float* l_part, int32_t* status, void* stream);

/*
 * Phase 2, the reduction of Eq. 5:
 *   out[b][h][:] = sum_c w_c * o_part[b][h][c][:] / sum_c w_c,   w_c = l_c * exp(m_c - max_c m_c),
 * skipping splits with l_c = 0; if all are empty the output row is zero.
 *   out : [B][H_q][d], fp16 (out_is_fp32 = 0) or fp32 (out_is_fp32 = 1).
 * Errors: TQ_ERR_NULL, TQ_ERR_SHAPE (B, H_q, num_splits < 1, d not a multiple of 32 or > 512), TQ_ERR_ALIGN,
 * TQ_ERR_CUDA.
 */
int tq_sdpa_int4_combine(const float* o_part, const float* m_part, const float* l_part, int32_t B, int32_t H_q,
                         int32_t d, int32_t num_splits, void* out, int32_t out_is_fp32, void* stream);

/* Bytes needed for o_part + m_part + l_part when laid out back to back (host function). */
size_t tq_partials_bytes(int32_t B, int32_t H_q, int32_t d, int32_t num_splits);

/*
 * Comparison path: the "dequantize-then-attend" baseline the paper measures against (Sec. 3.1 first
 * paragraph, Table 2).  Dequantises all valid rows of K and V into a materialised
 * [B][H_kv][S_cap][d] matrix in `workspace` (fp32 as in the paper when ws_is_fp32 = 1, fp16
 * otherwise), then runs split attention and the Eq. 5 reduction on the materialised matrices.
 * Same result as decode + combine up to rounding.  Built to be limited by the bytes it moves, like the
 * fused path (d = 128 with at most 8 query heads per KV head: tensor-core attention over the matrices, an fp32
 * K^ entering as fp16 hi + lo parts, V^ and the softmax weights as fp16; other shapes: a scalar kernel), so
 * that the ratio between the two paths is the ratio of their bytes.
 *   workspace_bytes >= tq_dequant_workspace_bytes(...), 16-byte aligned, contents destroyed.
 */
int tq_sdpa_dequant_then_attend(const tq_kv_cache* cache /* host */, const void* q, int32_t H_q, float attn_scale,
                                void* workspace, size_t workspace_bytes, int32_t ws_is_fp32, void* out,
                                int32_t out_is_fp32, int32_t* status, void* stream);

size_t tq_dequant_workspace_bytes(int32_t B, int32_t H_kv, int32_t H_q, int32_t S_cap, int32_t d,
                                  int32_t ws_is_fp32);

/*
 * K-versus-V precision ablation (Sec. 5: int4 K with full-precision V loses less than full-precision K
 * with int4 V, because key errors pass through the softmax while value errors reach the output
 * directly).  Phase 1 with each of K and V taken either from the int4 cache or from an unquantised
 * matrix: k_fp16 / v_fp16 are device fp16 [B][H_kv][S_cap][d] (rows below seq_lens[b] are read), or
 * NULL to take that side from the cache.  Both NULL is the plain fused attention; both given ignores
 * the cache's contents (its lengths still apply) and is full-precision attention.  Same partials as
 * tq_sdpa_int4_decode (combine with tq_sdpa_int4_combine).  A scalar kernel meant for the experiment,
 * not for speed.  num_splits = 0 picks tq_auto_splits(B, H_kv, H_q, d, S_cap).
 * Errors and status as tq_sdpa_int4_decode.
 */
int tq_sdpa_mixed_precision_attend(const tq_kv_cache* cache /* host */, const void* k_fp16, const void* v_fp16,
                                   const void* q, int32_t H_q, float attn_scale, int32_t num_splits, float* o_part,
                                   float* m_part, float* l_part, int32_t* status, void* stream);

/*
 * Fused attention for callers that cannot allocate (the paper has no counterpart for this entry
 * point; it exists for integration, not for the method).  Some hosts of this library may not call
 * cudaMalloc at the point where attention runs: an inference server that hands all device memory
 * to its own pool at start-up, code running while a stream is being captured into a CUDA graph
 * (where an allocation is illegal), or a latency-critical decode loop where cudaMalloc / cudaFree
 * would serialise the whole device.  They have nowhere to put the split partials that
 * tq_sdpa_int4_decode writes and tq_sdpa_int4_combine reads.  This call runs both phases in one go
 * and keeps the partials in a fixed TQ_STATIC_SCRATCH_BYTES array that is part of the library image
 * (every GPU on which the library is used holds those bytes until the process exits).
 *   Result: out[b][h][:] as tq_sdpa_int4_decode followed by tq_sdpa_int4_combine would give it
 *   (the split count may differ, so agreement is to rounding, not bit for bit).
 *   It calls no cudaMalloc / cudaFree nor any routine that allocates.  The caller still provides
 *   q, the cache (contiguous or paged, any supported head dimension) and out; the arguments are
 *   checked exactly as tq_sdpa_int4_decode and tq_sdpa_int4_combine check theirs.
 *   Limit: the partials of the chosen split count, B * H_q * C * (d + 2) * 4 bytes (plus padding),
 *   must fit the array.  The split count is lowered as far as 1 to make them fit; if they still
 *   do not, nothing is launched and TQ_ERR_WORKSPACE is returned.
 *   First use on a device looks up the array's device address (with that device current; the
 *   device of `stream` must be the current device).  Make that first call outside any stream
 *   capture; later calls do no set-up.
 *   All calls share the one array and it keeps the previous call's contents.  Nothing needs
 *   clearing (every partial is rewritten by each call), but two calls whose kernels overlap on
 *   the GPU -- different streams, or graphs launched concurrently -- race on it: serialise them.
 * Errors: TQ_ERR_NULL, TQ_ERR_SHAPE, TQ_ERR_ALIGN, TQ_ERR_WORKSPACE (see Limit), TQ_ERR_CUDA.
 * Status: as tq_sdpa_int4_decode.
 */
#define TQ_STATIC_SCRATCH_BYTES (8u << 20)
int tq_sdpa_int4_attend_static(const tq_kv_cache* cache /* host */, const void* q, int32_t H_q, float attn_scale,
                               void* out, int32_t out_is_fp32, int32_t* status, void* stream);

/* Bytes of one layer's cache arrays (packed + scales + zeros, K and V), i.e. Eq. 1 with the int4 format. */
size_t tq_cache_bytes(int32_t B, int32_t H_kv, int32_t S_cap, int32_t d);

const char* tq_result_string(int result);
int tq_last_cuda_error(void); /* cudaError_t of the most recent failing CUDA call of this thread, 0 if none */
const char* tq_version(void);

#ifdef __cplusplus
}
#endif
#endif /* TQ_H_ */
