"""Timings of the secondary workloads (everything except the headline 128K Llama-shaped step, which
bench.py at the repository root measures): short contexts, the d = 256 Gemma-style shape, the ragged
batch, sliding-window and multi-query decode, bulk quantisation and the dequantize-then-attend path.

    python -m paper_2604_16957_b200.workloads [--only NAME] [--steps K] [--warmup W]

Prints one JSON line per workload: microseconds per call (CUDA events around replays of a CUDA graph
that walks over enough distinct caches to exceed L2), the algorithmic bytes of the call and the
resulting GB/s.  Inputs are seeded device-side normals (K with 4 outlier channels x10 per KV head
where the Llama shape is used), quantised by tq_kv_quantize_append.  Needs a CUDA device.
"""
import argparse
import json

import numpy as np
import torch

from . import tq

L2_BYTES = 126 << 20
IDENTITY_PAGES = False  # --identity-pages: page i of a paged cache is pool page i (default: a random assignment)
FUSED_EVERYWHERE = False  # --fused: the one-launch step wherever it applies
NO_STABLE = False  # --no-stable: the fused step declares no stable part (every step waits for the one before it: latency, not throughput)
SEPARATE_CALLS = False  # --calls: time append / decode / combine as separate launches even where the fused step applies


def _fill(B, H_kv, S_cap, d, n_caches, seed, outliers, sigma=1.0, lens=None, page_tokens=0):
    """n_caches quantised caches filled to S_cap tokens; lens (if given) then overrides the lengths.
    page_tokens > 0: paged caches, each with a seeded random page assignment."""
    gen = torch.Generator(device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    caches = []
    chunk = max(1, min(S_cap, (256 << 20) // (B * H_kv * d * 4)))  // 16 * 16 or 16
    for i in range(n_caches):
        gen.manual_seed(seed + i)
        if page_tokens:
            mp = S_cap // page_tokens
            cache = tq.PagedKVCache(B, H_kv, page_tokens, mp, B * mp, d)
            perm = torch.randperm(B * mp, generator=torch.Generator().manual_seed(seed + i)).int()
            if IDENTITY_PAGES:
                perm = torch.arange(B * mp, dtype=torch.int32)
            cache.page_table.copy_(perm.view(B, mp))
        else:
            cache = tq.KVCache(B, H_kv, S_cap, d)
        ch = torch.randperm(d, generator=torch.Generator().manual_seed(seed))[:4].cuda()
        for t0 in range(0, S_cap, chunk):
            T = min(chunk, S_cap - t0)
            k = torch.randn((B, H_kv, T, d), generator=gen, device="cuda") * sigma
            if outliers:
                k[..., ch] *= 10.0
            v = torch.randn((B, H_kv, T, d), generator=gen, device="cuda")
            tq.tq_kv_quantize_append(cache, k.half(), v.half(), status)
        if lens is not None:
            cache.seq_lens.copy_(torch.as_tensor(lens, dtype=torch.int32))
        caches.append(cache)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return caches


def _time(enqueue, steps, warmup, before=None):
    """enqueue() launches one pass over all caches; returns seconds per pass."""
    enqueue()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        enqueue()
    for _ in range(warmup):
        if before: before()
        g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    total = 0.0
    for _ in range(steps):
        if before: before()
        e0.record()
        g.replay()
        e1.record()
        torch.cuda.synchronize()
        total += e0.elapsed_time(e1) / 1e3
    return total / steps


def _n_caches(bytes_per_cache):
    return max(2, min(256, -(-3 * L2_BYTES // bytes_per_cache)))


def _emit(name, us, alg_bytes, **kw):
    print(json.dumps({"workload": name, "us_per_call": round(us, 3), "algorithmic_bytes": int(alg_bytes),
                      "GBps": round(alg_bytes / us / 1e3, 1), **kw}), flush=True)


def decode_workload(name, B, H_q, H_kv, d, S, alpha, steps, warmup, outliers, sigma=1.0, window=0, S_q=1, lens=None,
                    with_append=False, compare=False, splits=0, page_tokens=0):
    """Times decode + combine (optionally preceded by a T = S_q append) over rotating caches."""
    per_tok = 2 * (d // 2 + d // 8)
    S_cap = (S + 15) // 16 * 16 + (64 if with_append else 0)
    if page_tokens:
        S_cap = -(-S_cap // page_tokens) * page_tokens
    cache_bytes = B * H_kv * S_cap * per_tok
    n = _n_caches(cache_bytes)
    caches = _fill(B, H_kv, S_cap, d, n, 31, outliers, sigma, lens if lens is not None else [S] * B, page_tokens)
    base_lens = torch.as_tensor(lens if lens is not None else [S] * B, dtype=torch.int32).cuda()
    span = window or S
    # one launch per step (tq_sdpa_int4_step) wherever it applies: plain decode (contiguous or paged cache), at most 8
    # query heads per KV head; the tokens present before the timed steps are its stable part
    # (measured: it wins on 1K to 128K Llama-shaped contexts, the d = 256 shape, and by 2 % on batches, where the
    # ragged one gives every sequence its own stable part)
    ragged = lens is not None and min(lens) != max(lens)
    windowed = window > 0 and window < S_cap and not page_tokens and lens is None  # tq_sdpa_int4_step_window
    fused = (not SEPARATE_CALLS) and S_q == 1 and (window == 0 or windowed) and H_q // H_kv <= 8 and (
        FUSED_EVERYWHERE or d <= 256)
    C = splits or (tq.tq_auto_splits_step if fused and not window else tq.tq_auto_splits)(B, H_kv, H_q * S_q, d, span)
    o, m, l = tq.alloc_partials(B, H_q * S_q, d, C)
    ws = tq.alloc_step_workspace(B, H_kv, H_q, d, C) if fused else None
    # (the stable part is one number for the whole batch: with ragged lengths the last split of the longer
    # sequences would get everything beyond it, so the ragged batch declares none)
    stable = base_lens.clone() if ragged else S  # ragged: one stable part per sequence (tq_sdpa_int4_step_ragged)
    if NO_STABLE:
        stable = 0
    gen = torch.Generator(device="cuda").manual_seed(5)
    q = (torch.randn((B, S_q, H_q, d), generator=gen, device="cuda") * sigma).half()
    kn = (torch.randn((B, H_kv, S_q, d), generator=gen, device="cuda") * sigma).half()
    vn = torch.randn((B, H_kv, S_q, d), generator=gen, device="cuda").half()
    out = torch.empty((B, S_q * H_q, d), dtype=torch.float16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def reset():
        for c in caches:
            c.seq_lens.copy_(base_lens)

    def enqueue():
        for c in caches:
            if fused and window:
                tq.tq_sdpa_int4_step_window(c, kn if with_append else None, vn if with_append else None, q[:, 0], alpha,
                                            window, C, S, ws, out, status)
                continue
            if fused:
                tq.tq_sdpa_int4_step(c, kn if with_append else None, vn if with_append else None, q[:, 0], alpha, C, stable,
                                     ws, out, status)
                continue
            if with_append:
                tq.tq_kv_quantize_append(c, kn, vn, status)
            if S_q == 1 and window == 0:
                tq.tq_sdpa_int4_decode(c, q[:, 0], alpha, C, o, m, l, status)
            else:
                tq.tq_sdpa_int4_decode_multi(c, q, alpha, window, C, o, m, l, status)
            tq.tq_sdpa_int4_combine(o, m, l, out)

    us = _time(enqueue, steps, warmup, before=reset if with_append else None) / n * 1e6
    assert int(status.item()) == 0
    L = np.asarray(lens if lens is not None else [S] * B, dtype=np.int64) + (S_q if with_append else 0)
    attended = np.minimum(L, window + S_q - 1) if window else L
    alg = int(attended.sum()) * H_kv * per_tok
    extra = {}
    if compare:
        need = tq.tq_dequant_workspace_bytes(B, H_kv, H_q, S_cap, d, True)
        ws = torch.empty(need, dtype=torch.uint8, device="cuda")
        reset()

        def enqueue_cmp():
            for c in caches:
                tq.tq_sdpa_dequant_then_attend(c, q[:, 0], alpha, ws, True, out, status)

        extra["dequant_then_attend_us"] = round(_time(enqueue_cmp, max(2, steps // 4), 1) / n * 1e6, 1)
    _emit(name, us, alg, B=B, H_q=H_q, H_kv=H_kv, d=d, S=S if lens is None else "ragged", S_q=S_q, window=window,
          num_splits=C, caches_rotated=n, page_tokens=page_tokens,
          includes="append+decode+combine" if with_append else "decode+combine",
          entry="tq_sdpa_int4_step (one launch)" if fused else "separate calls", **extra)


def bulk_quantize_workload(steps, warmup):
    H_kv, d, S = 8, 128, 131072
    gen = torch.Generator(device="cuda").manual_seed(3)
    k = torch.randn((1, H_kv, S, d), generator=gen, device="cuda").half()
    v = torch.randn((1, H_kv, S, d), generator=gen, device="cuda").half()
    cache = tq.KVCache(1, H_kv, S, d)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def enqueue():
        cache.seq_lens.zero_()
        tq.tq_kv_quantize_append(cache, k, v, status)

    us = _time(enqueue, steps, warmup) * 1e6
    assert int(status.item()) == 0
    _emit("bulk quantise, one 128K Llama-shaped layer (T = S)", us, 2 * H_kv * S * d * 2 + H_kv * S * 160,
          note="537 MB of fp16 read + 168 MB written; includes a 4-byte memset")


def ragged_lengths():
    # same draw as the parity tests' generator for the ragged configuration
    from .inputs import ragged_lengths as rl
    return rl(16, 4096, 65536, 5).tolist()


WORKLOADS = {
    "llama_1k": lambda a: decode_workload("llama shape, 1K context", 1, 64, 8, 128, 1024, 128 ** -0.5, a.steps, a.warmup, True, splits=a.splits),
    "llama_4k": lambda a: decode_workload("llama shape, 4K context", 1, 64, 8, 128, 4096, 128 ** -0.5, a.steps, a.warmup, True, splits=a.splits),
    "llama_8k": lambda a: decode_workload("llama shape, 8K context", 1, 64, 8, 128, 8192, 128 ** -0.5, a.steps, a.warmup, True, splits=a.splits),
    "llama_32k": lambda a: decode_workload("llama shape, 32K context", 1, 64, 8, 128, 32768, 128 ** -0.5, a.steps, a.warmup, True, splits=a.splits),
    "gemma_32k": lambda a: decode_workload("gemma-style d=256, 32K context", 1, 32, 16, 256, 32768, 1.0, a.steps, a.warmup,
                                           False, sigma=0.25, splits=a.splits),
    "gemma_32k_window": lambda a: decode_workload("gemma-style d=256, 32K context, window 1024", 1, 32, 16, 256, 32768, 1.0,
                                                  a.steps, a.warmup, False, sigma=0.25, window=1024, splits=a.splits),
    "gemma_32k_sq4": lambda a: decode_workload("gemma-style d=256, 32K context, 4 query tokens", 1, 32, 16, 256, 32768, 1.0,
                                               a.steps, a.warmup, False, sigma=0.25, S_q=4),
    "llama_32k_sq4": lambda a: decode_workload("llama shape, 32K context, 4 query tokens", 1, 64, 8, 128, 32768,
                                               128 ** -0.5, a.steps, a.warmup, True, S_q=4),
    "ragged_b16": lambda a: decode_workload("ragged batch B=16, lengths U{4096..65536}", 16, 64, 8, 128, 65536,
                                            128 ** -0.5, a.steps, a.warmup, True, lens=ragged_lengths(),
                                            with_append=True, compare=a.splits == 0, splits=a.splits),
    "ragged_b16_paged": lambda a: decode_workload("ragged batch B=16, lengths U{4096..65536}, 256-token pages", 16, 64, 8,
                                                  128, 65536, 128 ** -0.5, a.steps, a.warmup, True,
                                                  lens=ragged_lengths(), with_append=True, splits=a.splits,
                                                  page_tokens=256),
    "llama_32k_paged": lambda a: decode_workload("llama shape, 32K context, 64-token pages", 1, 64, 8, 128, 32768,
                                                 128 ** -0.5, a.steps, a.warmup, True, page_tokens=64),
    "ragged_b16_general": lambda a: decode_workload("ragged batch B=16, general kernel (window 2^30)", 16, 64, 8, 128, 65536,
                                                    128 ** -0.5, a.steps, a.warmup, True, lens=ragged_lengths(),
                                                    with_append=True, splits=a.splits or 10, window=1 << 30),
    "batch16_32k": lambda a: decode_workload("batch B=16, equal lengths 32K", 16, 64, 8, 128, 32768, 128 ** -0.5, a.steps,
                                             a.warmup, True, with_append=True, splits=a.splits),
    "bulk_quantize": lambda a: bulk_quantize_workload(a.steps, a.warmup),
}


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--only", default=None, choices=sorted(WORKLOADS))
    ap.add_argument("--splits", type=int, default=0, help="sequence splits (batch, short-context and window workloads (0 = library default)")
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--identity-pages", action="store_true", help="paged workloads: pool page i holds page i")
    ap.add_argument("--calls", action="store_true", help="separate append / decode / combine launches everywhere")
    ap.add_argument("--no-stable", action="store_true", help="fused steps declare no stable part: each step waits for its predecessor before reading anything")
    ap.add_argument("--fused", action="store_true", help="tq_sdpa_int4_step wherever it applies (default: one sequence, d <= 256)")
    args = ap.parse_args()
    global IDENTITY_PAGES, SEPARATE_CALLS, FUSED_EVERYWHERE, NO_STABLE
    IDENTITY_PAGES = args.identity_pages
    SEPARATE_CALLS = args.calls
    NO_STABLE = args.no_stable
    FUSED_EVERYWHERE = args.fused
    assert torch.cuda.is_available(), "needs a CUDA device (there is no CPU path)"
    for name, fn in WORKLOADS.items():
        if args.only in (None, name):
            fn(args)
            torch.cuda.empty_cache()


if __name__ == "__main__":
    main()
