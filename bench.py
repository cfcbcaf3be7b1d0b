#!/usr/bin/env python
"""Benchmark of the int4 compressed-domain decode-attention hot path on B200.

Workload (N = 1): the Llama-3.1-70B-shaped long-context configuration -- 64 query heads, 8 KV
heads, d = 128, 131072 cached tokens, all 80 layers' int4 KV caches resident (13.4 GB).  One
step is one decode step run layer by layer: for each of the 80 layers, quantize-append of the
new token's K/V, fused int4 attention (split-K partials) and the split reduction.  The metric
is microseconds per layer-step; the roofline object reports the fused kernel's algorithmic
HBM bytes per second against the measured copy bandwidth of this GPU pool.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--context S] [--layers L]

Prints ONE JSON line on stdout (rank 0).  All inputs are seeded and synthetic.
"""
import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

H_Q, H_KV, D, LAYERS, CONTEXT = 64, 8, 128, 80, 131072
ALPHA = D ** -0.5
BYTES_PER_TOKEN_HEAD = 2 * (D // 2 + 2 * (D // 32) * 2)  # K + V: codes + fp16 scale + fp16 zero = 160 B
HBM_NOMINAL_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
PAPER_CONTEXT = {"hardware": "Apple M1 Max 64 GB (Metal)", "fused_ms_at_128K": 9.9,
                 "dequant_then_attend_ms_at_128K": 480.6, "speedup_at_128K": 48,
                 "note": "paper Table 2; another machine and API, context only"}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--context", type=int, default=CONTEXT)
    ap.add_argument("--layers", type=int, default=LAYERS)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-compare", action="store_true", help="skip the dequantize-then-attend timing")
    ap.add_argument("--splits", type=int, default=0, help="sequence splits C of the fused kernel (0 = library default)")
    ap.add_argument("--classic", action="store_true",
                    help="time the step as three calls (append, tq_sdpa_int4_decode, combine) instead of the fused step")
    ap.add_argument("--lib", default=None,
                    help="time another build of the library (a timing probe from `build.py --probe`); implies --no-parity")
    ap.add_argument("--no-parity", action="store_true", help="skip the oracle check of sampled layers of the timed state")
    return ap.parse_args()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json, device copy)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (earlier measurement on this pool)"


# ------------------------------------------------------------------ clocks (read-only NVML sampling)
class ClockSampler:
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap",
               0x80: "hw_power_brake", 0x2: "applications_clocks_setting", 0x100: "display_clock_setting"}

    def __init__(self, index):
        self.samples, self.reasons, self.max_mhz, self.power_w, self.mem_mhz = [], set(), None, [], []
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    self.power_w.append(nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0)
                    self.mem_mhz.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_MEM)))
                except Exception:
                    pass
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.005)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"]}
        out = {"sm_mhz": int(statistics.median(self.samples)), "sm_min_mhz": min(self.samples), "sm_max_mhz": self.max_mhz,
               "reasons": sorted(self.reasons), "samples": len(self.samples)}
        if self.power_w:
            out["power_w_median"] = round(statistics.median(self.power_w), 1)
            out["power_w_max"] = round(max(self.power_w), 1)
            out["mem_mhz"] = int(statistics.median(self.mem_mhz))
        return out


# ------------------------------------------------------------------ CPU oracle leg
def oracle_sample_us_per_layer(context, repeats=1, kv_heads=1):
    """Time the CPU oracle as it stands on a bounded sample of the workload: `kv_heads` of the 8 KV
    heads (with their 8 query heads each) of one `context`-token layer, quantised by the oracle
    itself; the time is scaled by 8 / kv_heads to a full layer.
    Returns (us_per_layer list, seconds list, threads)."""
    import numpy as np
    from oracle import tq_oracle as O
    from paper_2604_16957_b200 import inputs as I
    sh = I.Shape("llama-sample", 1, (H_Q // H_KV) * kv_heads, kv_heads, D, ALPHA, k_outlier_channels=4)
    k, v = I.make_kv(sh, context, seed=1000)
    q = I.make_q(sh, seed=1000)
    cache = O.Cache(1, kv_heads, context, D)
    cache.append(k, v)
    del k, v
    secs = []
    for _ in range(repeats):
        t = time.perf_counter()
        out = O.attention(cache, q, ALPHA)
        secs.append(time.perf_counter() - t)
    assert np.all(np.isfinite(out))
    return [s * (H_KV / kv_heads) * 1e6 for s in secs], secs, O.num_threads()


def run_reference(args, rank):
    """--impl reference: the oracle, timed on the host cores, same metric and config."""
    if rank != 0:
        return
    # one cache build, then warmup + steps timed repetitions on it
    # (a step is one full layer, all 64 query heads, so the oracle's thread pool is used as in the GPU arm's
    # cpu_baseline; 80 layers per step would take minutes per step)
    per, secs, threads = oracle_sample_us_per_layer(args.context, repeats=args.warmup + args.steps, kv_heads=H_KV)
    timed = per[args.warmup:]
    value = sum(timed) / len(timed)
    sample = (f"one full {args.context}-token layer (all {H_Q} query heads, {H_KV} KV heads) per step instead of "
              f"{args.layers}, fp64 oracle on the oracle-quantised cache")
    line = {"impl": "reference", "metric": "int4 decode-attn us/layer @128K (Llama-70B shape)", "value": value,
            "unit": "us/layer", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": value / 1e3, "layers_per_step": 1, "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict(args),
            "cpu_baseline": {"value": value, "unit": "us/layer", "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "us/layer", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def config_dict(args):
    return {"workload": f"llama70b-shape long context: B=1, H_q={H_Q}, H_kv={H_KV}, d={D}, context={args.context}, "
                        f"{args.layers} layers resident, int4 KV group 32, attn_scale=1/sqrt(d), one decode step "
                        f"layer by layer (quantize-append + fused int4 attention + split combine per layer)",
            "context": args.context, "layers": args.layers, "H_q": H_Q, "H_kv": H_KV, "d": D,
            "l2": "inputs larger than L2: every layer's cache (168 MB at 128K) is a distinct buffer, 13.4 GB in all"}


def max_over_ranks(seconds, world, device):
    """Replicas only: every rank times its own replica; the job's time is the slowest rank's."""
    if world <= 1:
        return seconds
    import torch
    import torch.distributed as dist
    t = torch.tensor([seconds], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_us_per_layer(seconds_for_steps, steps, layers, world):
    """N independent replicas complete N * layers layer-steps per step in the time of the slowest."""
    return seconds_for_steps / steps / layers / world * 1e6


# ------------------------------------------------------------------ GPU arm
def main():
    args = parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
        return

    if args.lib:
        os.environ["TQ_LIBRARY"] = os.path.abspath(args.lib)
        args.no_parity = True
    import torch
    from paper_2604_16957_b200 import tq  # fails loudly if libtq.so is missing
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    L, S = args.layers, args.context
    total_appends = 2 * (args.warmup + args.steps) + 8
    S_cap = (S + total_appends + 15) // 16 * 16
    C = args.splits or (tq.tq_auto_splits if args.classic else tq.tq_auto_splits_step)(1, H_KV, H_Q, D, S)

    # ---- resident state: L quantised layer caches, filled from seeded device-side normals.
    # K gets 4 seeded outlier channels x10 per KV head, like the parity-test generator.
    caches = []
    gen = torch.Generator(device=dev)
    ch_rng = torch.Generator().manual_seed(4242)
    outlier_channels = [[torch.randperm(D, generator=ch_rng)[:4] for _ in range(H_KV)] for _ in range(L)]
    status = torch.zeros(1, dtype=torch.int32, device=dev)

    def layer_kv(layer):
        """The seeded fp16 K, V that layer's cache was quantised from (regenerated for the parity check)."""
        gen.manual_seed(7000 + layer + 1000 * rank)
        k = torch.randn((1, H_KV, S, D), generator=gen, device=dev, dtype=torch.float32)
        for h in range(H_KV):
            k[0, h, :, outlier_channels[layer][h].to(dev)] *= 10.0
        k = k.to(torch.float16)
        v = torch.randn((1, H_KV, S, D), generator=gen, device=dev, dtype=torch.float32).to(torch.float16)
        return k, v

    for layer in range(L):
        k, v = layer_kv(layer)
        cache = tq.KVCache(1, H_KV, S_cap, D, device=dev)
        tq.tq_kv_quantize_append(cache, k, v, status)
        caches.append(cache)
        del k, v
    torch.cuda.synchronize()
    assert int(status.item()) == 0, f"device status word set while filling the caches: {int(status.item())}"

    # per-layer step inputs (q, k_new, v_new) in one buffer, outputs in another
    per_layer_in = H_Q * D + 2 * H_KV * D
    gen.manual_seed(99 + rank)
    inp = torch.randn((L, per_layer_in), generator=gen, device=dev, dtype=torch.float32).to(torch.float16)
    out = torch.zeros((L, H_Q, D), dtype=torch.float16, device=dev)
    o_part, m_part, l_part = tq.alloc_partials(1, H_Q, D, C, device=dev)
    q_l = [inp[i, :H_Q * D].view(1, H_Q, D) for i in range(L)]
    kn_l = [inp[i, H_Q * D:H_Q * D + H_KV * D].view(1, H_KV, 1, D) for i in range(L)]
    vn_l = [inp[i, H_Q * D + H_KV * D:].view(1, H_KV, 1, D) for i in range(L)]
    out_l = [out[i].view(1, H_Q, D) for i in range(L)]

    def reset_lens():
        for cch in caches:
            cch.seq_lens.fill_(S)

    # The S tokens of the fill were written long before any step: they are the stable part that the fused
    # step / the overlapped decode may attend without waiting for the kernel before it (tq.h).
    ws = tq.alloc_step_workspace(1, H_KV, H_Q, D, C, device=dev)

    def enqueue(append=True, decode=True, combine=True, classic=args.classic, stable=S):
        fused = append and decode and combine and not classic
        for i in range(L):
            if fused:   # one launch: quantize-append + fused int4 attention + split reduction
                tq.tq_sdpa_int4_step(caches[i], kn_l[i], vn_l[i], q_l[i], ALPHA, C, stable, ws, out_l[i], status)
                continue
            if append:
                tq.tq_kv_quantize_append(caches[i], kn_l[i], vn_l[i], status)
            if decode and classic:
                tq.tq_sdpa_int4_decode(caches[i], q_l[i], ALPHA, C, o_part, m_part, l_part, status)
            elif decode:
                tq.tq_sdpa_int4_decode_overlapped(caches[i], q_l[i], ALPHA, C, S, o_part, m_part, l_part, status)
            if combine:
                tq.tq_sdpa_int4_combine(o_part, m_part, l_part, out_l[i])

    def make_graph(**kw):
        enqueue(**kw)  # eager once (also sets function attributes outside capture)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            enqueue(**kw)
        return g

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def time_graph(g, warmup, steps, pre=None, post=None):
        """K replays bracketed by events on the current stream; returns seconds for the K steps."""
        reset_lens()
        for _ in range(warmup):
            if pre: pre()
            g.replay()
            if post: post()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            if pre: pre()
            g.replay()
            if post: post()
        e1.record()
        barrier()
        return max_over_ranks(e0.elapsed_time(e1) / 1e3, world, dev)

    g_step = make_graph()
    g_decode = make_graph(append=False, combine=False)
    g_attn = make_graph(append=False)
    g_append = make_graph(decode=False, combine=False)
    g_decode_classic = make_graph(append=False, combine=False, classic=True)
    g_three = make_graph(classic=True)
    g_step_dependent = make_graph(stable=0)   # the fused step with no stable part: every launch waits for its predecessor

    W, K = args.warmup, args.steps
    with ClockSampler(local_rank) as clocks:
        t_step = time_graph(g_step, W, K)
    us_per_layer = job_us_per_layer(t_step, K, L, 1)

    # per-kernel figures (same graph-replay timing, decode launches back to back over the L distinct layers)
    t_decode = time_graph(g_decode, W, K)
    t_attn = time_graph(g_attn, W, K)
    t_append = time_graph(g_append, W, K)
    decode_us = t_decode / K / L * 1e6
    decode_classic_us = time_graph(g_decode_classic, W, K) / K / L * 1e6
    three_us = time_graph(g_three, W, K) / K / L * 1e6
    step_dependent_us = time_graph(g_step_dependent, W, K) / K / L * 1e6

    # ---- end to end through host buffers: pinned host inputs -> device, the step, outputs -> pinned host
    h_in = torch.empty_like(inp, device="cpu").pin_memory()
    h_in.copy_(inp)
    h_out = torch.empty_like(out, device="cpu").pin_memory()
    t_e2e = time_graph(g_step, W, K, pre=lambda: inp.copy_(h_in, non_blocking=True),
                       post=lambda: (h_out.copy_(out, non_blocking=True), torch.cuda.current_stream().synchronize()))
    e2e_us = t_e2e / K / L * 1e6
    assert int(status.item()) == 0, f"device status word set during the benchmark: {int(status.item())}"

    # ---- what was timed is also what is right: one more replay of the timed graph from the initial lengths,
    # then sampled layers of that very state against the CPU oracle (outside every timed region)
    parity = None
    if rank == 0 and not args.no_parity:
        reset_lens()
        g_step.replay()
        torch.cuda.synchronize()
        parity = check_sampled_layers(torch, caches, layer_kv, inp, out, S, S_cap, sorted({0, L // 2 - 1 if L > 1 else 0, L - 1}))

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel (fused decode)
    peak, peak_src = measured_peak()
    alg_bytes = H_KV * S * BYTES_PER_TOKEN_HEAD
    # the timed step is one launch of the fused kernel per layer, so its per-layer time is that kernel's average
    # launch-to-launch duration; with --classic the fused-attention kernel is timed in a graph of its own
    kernel_us = decode_classic_us if args.classic else us_per_layer
    achieved = alg_bytes / (kernel_us * 1e-6) / 1e9
    roofline = {"bound": "hbm", "kernel": "decode_mma_kernel<128, 0, 0, 1>" if args.classic else
                "decode_mma_kernel<128, 3, 0, 1> (append + attention + reduction in one launch)", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_source": peak_src, "traffic": ncu_traffic_bytes() if S == CONTEXT else None,
                "algorithmic_bytes_per_launch": alg_bytes, "us_per_launch": kernel_us,
                "frac_of_nominal_8TBs": achieved / HBM_NOMINAL_GBS}

    line = {"metric": "int4 decode-attn us/layer @128K (Llama-70B shape)", "value": job_us_per_layer(t_step, K, L, world),
            "unit": "us/layer", "n_gpus": world, "steps": K, "warmup": W, "ms_per_step": t_step / K * 1e3,
            "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f16 codes->f32 accum",
            "data": "synthetic", "config": config_dict(args), "clocks": clocks.summary(),
            "e2e": {"value": e2e_us / world, "unit": "us/layer", "h2d_bytes_per_step": inp.numel() * 2,
                    "d2h_bytes_per_step": out.numel() * 2},
            "gpu_launches": (3 if args.classic else 1) * L * K, "roofline": roofline,
            "breakdown_us_per_layer": {"append+decode+combine": us_per_layer, "decode+combine": t_attn / K / L * 1e6,
                                       "decode": decode_us, "append": t_append / K / L * 1e6,
                                       "decode_waiting_for_predecessor": decode_classic_us,
                                       "append+decode+combine waiting for predecessor (stable_tokens=0)": step_dependent_us,
                                       "append+decode+combine as three calls": three_us},
            "step_entry": ("tq_kv_quantize_append + tq_sdpa_int4_decode + tq_sdpa_int4_combine" if args.classic else
                           f"tq_sdpa_int4_step(stable_tokens={S}): one launch per layer"),
            "hbm_gbs_whole_step": alg_bytes / (us_per_layer * 1e-6) / 1e9, "num_splits": C,
            "paper_context": PAPER_CONTEXT, "device": device_info(torch, dev), "library": tq.tq_version()}
    if parity is not None:
        line["parity"] = parity
    if world > 1:
        line["config"]["replicas"] = "independent replicas, no collective (the path does not shard in this build)"

    if not args.no_compare:
        line["dequant_then_attend_us_per_layer"] = time_dequant_then_attend(tq, torch, caches, q_l, out, S, S_cap, dev)
    if not args.no_cpu_baseline:
        per, secs, threads = oracle_sample_us_per_layer(S, repeats=2, kv_heads=H_KV)
        line["cpu_baseline"] = {"value": min(per), "unit": "us/layer", "cores": threads, "kind": "oracle",
                                "sample": f"one full {S}-token layer (all {H_Q} query heads, {H_KV} KV heads) of the "
                                          f"{L}-layer step, oracle-quantised, best of 2 runs ({min(secs):.2f} s wall on "
                                          f"{threads} threads)"}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def check_sampled_layers(torch, caches, layer_kv, inp, out, S, S_cap, layers):
    """Oracle check of the state the benchmark timed.  For each sampled layer: the oracle quantises the same
    seeded fp16 K, V (and the step's new token) on the host; the device cache must equal it bit for bit over
    the S + 1 valid tokens; the step's output must match the oracle's fp64 attention over that cache within
    max-abs 2e-3 (+ half an fp16 ulp, the output being fp16) and relative L2 1e-3 (+ 2^-11 for the fp16
    rounding).  Raises if not."""
    import numpy as np
    from oracle import tq_oracle as O
    res = {"layers": layers, "max_abs": 0.0, "rel_l2": 0.0, "cache_bits_equal": True,
           "tolerance": {"max_abs": 2e-3, "rel_l2": 1e-3, "fp16_output_allowance": "half ulp / 2^-11"}}
    for i in layers:
        k, v = layer_kv(i)
        host = O.Cache(1, H_KV, S_cap, D)
        host.append(k.cpu().numpy(), v.cpu().numpy())
        del k, v
        row = inp[i].cpu().numpy()
        q = row[:H_Q * D].reshape(1, H_Q, D)
        host.append(row[H_Q * D:H_Q * D + H_KV * D].reshape(1, H_KV, 1, D), row[H_Q * D + H_KV * D:].reshape(1, H_KV, 1, D))
        n = S + 1
        assert int(caches[i].seq_lens.item()) == n == int(host.lens[0])
        for d_arr, h_arr in zip(caches[i].arrays_token_major(), host.arrays()):
            dv, hv = d_arr[:, :, :n].cpu().numpy(), h_arr[:, :, :n]
            if dv.dtype == np.float16:
                dv, hv = dv.view(np.uint16), hv.view(np.uint16)
            if not np.array_equal(dv, hv):
                res["cache_bits_equal"] = False
        ref = O.attention(host, q, ALPHA)
        got = out[i].float().cpu().numpy().astype(np.float64).reshape(ref.shape)
        diff = np.abs(got - ref)
        rel = float(np.sqrt((diff ** 2).sum() / max((ref ** 2).sum(), 1e-300)))
        res["max_abs"] = max(res["max_abs"], float(diff.max()))
        res["rel_l2"] = max(res["rel_l2"], rel)
        ok = bool(np.all(diff <= 2e-3 + np.abs(ref) * 2.0 ** -11) and rel <= 1e-3 + 2.0 ** -11)
        if not (ok and res["cache_bits_equal"]):
            raise AssertionError(f"benchmark state fails the oracle check at layer {i}: {res}")
        del host
    return res


def device_info(torch, dev):
    """What the budgets assume about the GPU, as the driver reports it."""
    p = torch.cuda.get_device_properties(dev)
    return {"name": p.name, "sms": p.multi_processor_count, "l2_bytes": getattr(p, "L2_cache_size", None),
            "smem_per_sm_bytes": getattr(p, "shared_memory_per_multiprocessor", None),
            "hbm_bytes": p.total_memory}


def ncu_traffic_bytes():
    """DRAM bytes (read + write) of one fused-decode launch, from the committed ncu summary."""
    import re
    path = os.path.join(ROOT, "profiles", "decode_mma_llama128k.md")
    try:
        with open(path) as f:
            m = re.search(r"^dram_bytes_per_launch:\s*(\d+)", f.read(), re.M)
        return int(m.group(1)) if m else None
    except Exception:
        return None


def time_dequant_then_attend(tq, torch, caches, q_l, out, S, S_cap, dev):
    """The comparison path on the same GPU and inputs, one layer at a time (its matrix workspace is
    1 GB in fp32), rotating over distinct layers."""
    res = {}
    for name, f32 in (("fp32_workspace", True), ("fp16_workspace", False)):
        nbytes = tq.tq_dequant_workspace_bytes(1, H_KV, H_Q, S_cap, D, f32)
        ws = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        o = out[0].view(1, H_Q, D)
        n = min(len(caches), 8)
        for i in range(2):
            tq.tq_sdpa_dequant_then_attend(caches[i % n], q_l[i % n], ALPHA, ws, f32, o)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(n):
            tq.tq_sdpa_dequant_then_attend(caches[i], q_l[i], ALPHA, ws, f32, o)
        e1.record()
        torch.cuda.synchronize()
        res[name] = e0.elapsed_time(e1) / n * 1e3
        del ws
    return res


if __name__ == "__main__":
    main()
