"""GPU parity of the fused int4 decode attention (decode + combine), its partials, the Eq. 5
reduction alone and the dequantize-then-attend comparison path, against the CPU oracle.

Tolerance (stated by the benchmark spec for outputs computed from the same dequantised values):
max-abs <= 2e-3 and relative L2 <= 1e-3 on the fp32 output.
"""
import os

import numpy as np
import pytest

from paper_2604_16957_b200 import inputs as I
from util import (MAX_ABS_TOL, REL_L2_TOL, assert_attention_close, assert_cache_bits_equal, device_cache, errors,
                  fused_attention, oracle_cache)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gpu():
    import torch
    from paper_2604_16957_b200 import tq
    assert torch.cuda.is_available()
    return tq, torch


def _both(gpu, oracle, shape, S, seed, S_cap=None, lens=None, fill_byte=None):
    tq, torch = gpu
    k, v = I.make_kv(shape, S, seed)
    S_cap = S_cap or (S + 15) // 16 * 16
    host = oracle_cache(oracle, shape, k, v, S_cap, lens)
    dev = device_cache(tq, torch, shape, k, v, S_cap, lens, fill_byte)
    return host, dev


def test_config1_tiny_then_append_one_token(gpu, oracle):
    tq, torch = gpu
    sh = I.TINY
    host, dev = _both(gpu, oracle, sh, 256, 1, S_cap=272, fill_byte=0xFF)
    q = I.make_q(sh, 1)
    out, _, _ = fused_attention(tq, torch, dev, q, sh.alpha)
    assert_attention_close(out, oracle.attention(host, q, sh.alpha), "tiny/256")
    k1, v1 = I.make_kv(sh, 1, 1, stream=1)
    host.append(k1, v1)
    tq.tq_kv_quantize_append(dev, torch.from_numpy(k1).cuda(), torch.from_numpy(v1).cuda())
    assert_cache_bits_equal(dev, host)
    q1 = I.make_q(sh, 1, stream=1)
    for C in (0, 1, 3, 17, 256):  # up to the largest split count: nearly all splits are empty
        out, _, _ = fused_attention(tq, torch, dev, q1, sh.alpha, num_splits=C)
        assert_attention_close(out, oracle.attention(host, q1, sh.alpha), f"tiny/257 C={C}")


def test_both_shared_memory_layouts_give_the_same_bits(gpu, oracle):
    """At d = 128 the launch picks between two shared-memory layouts of the decode kernel by the cache's capacity
    per split (rings of four stages whose memory the merge reuses, or three stages beside separate merge arrays).
    Both hand the same token blocks to the same warps and merge in the same order, so the same sequence in a small
    and in a large cache must give bit-equal partials; both are checked against the oracle as well."""
    tq, torch = gpu
    sh, S, C = I.LLAMA, 4096 + 37, 8
    q = I.make_q(sh, 21)
    partials = []
    for S_cap in (4608, 8 * 1024):  # 576 and 1024 tokens of capacity per split: below and above the 768 of the rule
        host, dev = _both(gpu, oracle, sh, S, 21, S_cap=S_cap)
        out, (o, m, l), _ = fused_attention(tq, torch, dev, q, sh.alpha, num_splits=C)
        assert_attention_close(out, oracle.attention(host, q, sh.alpha), f"S_cap={S_cap}")
        partials.append((o.cpu().numpy(), m.cpu().numpy(), l.cpu().numpy()))
    for a, b in zip(*partials):
        assert np.array_equal(a, b)


@pytest.mark.parametrize("S,seed", [(1024, 2), (4096, 3), (8192, 4)])
def test_config2_llama_shape_short_contexts(gpu, oracle, S, seed):
    tq, torch = gpu
    host, dev = _both(gpu, oracle, I.LLAMA, S, seed)
    assert_cache_bits_equal(dev, host)
    q = I.make_q(I.LLAMA, seed)
    ref = oracle.attention(host, q, I.LLAMA.alpha)
    out, _, _ = fused_attention(tq, torch, dev, q, I.LLAMA.alpha)
    mx, rel = assert_attention_close(out, ref, f"llama/{S}")
    print(f"llama S={S}: max-abs {mx:.2e} rel-L2 {rel:.2e}")
    out16, _, _ = fused_attention(tq, torch, dev, q, I.LLAMA.alpha, out_dtype=torch.float16)
    assert np.abs(out16 - ref).max() <= MAX_ABS_TOL + np.abs(ref).max() * 2.0 ** -11


def test_config4_gemma_style_d256_scale_one(gpu, oracle):
    tq, torch = gpu
    host, dev = _both(gpu, oracle, I.GEMMA, 32768, 5)
    q = I.make_q(I.GEMMA, 5)
    ref = oracle.attention(host, q, I.GEMMA.alpha)
    out, _, C = fused_attention(tq, torch, dev, q, I.GEMMA.alpha, out_dtype=torch.float16)
    mx, rel = errors(out, ref)
    print(f"gemma 32K C={C}: max-abs {mx:.2e} rel-L2 {rel:.2e}")
    assert mx <= MAX_ABS_TOL + np.abs(ref).max() * 2.0 ** -11
    out32, _, _ = fused_attention(tq, torch, dev, q, I.GEMMA.alpha)
    assert_attention_close(out32, ref, "gemma/32K")


@pytest.mark.parametrize("d,H_q,H_kv", [(64, 4, 1), (64, 16, 2), (128, 2, 2), (128, 6, 2), (128, 32, 2), (256, 8, 4),
                                        (256, 24, 1)])
def test_head_layouts_and_ragged_lengths(gpu, oracle, d, H_q, H_kv):
    """GQA factors 1, 3, 4, 8, 16, 24 (more than one tile of 8 heads), ragged lengths including
    1, non-multiples of 16 and a full cache, junk bytes past the end of each sequence."""
    tq, torch = gpu
    sh = I.Shape("x", 5, H_q, H_kv, d, d ** -0.5, k_outlier_channels=2)
    lens = [1, 15, 333, 1000, 1008]
    host, dev = _both(gpu, oracle, sh, 1008, 11, S_cap=1008, lens=lens, fill_byte=0xFF)
    q = I.make_q(sh, 11)
    ref = oracle.attention(host, q, sh.alpha)
    for C in (1, 4, 64):
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        out, _, _ = fused_attention(tq, torch, dev, q, sh.alpha, num_splits=C, status=status)
        assert int(status.item()) == 0
        assert_attention_close(out, ref, f"d={d} Hq={H_q} Hkv={H_kv} C={C}")


def test_partials_match_oracle_partials(gpu, oracle):
    tq, torch = gpu
    sh = I.Shape("x", 2, 16, 2, 128, 128 ** -0.5)
    lens = [700, 50]
    host, dev = _both(gpu, oracle, sh, 704, 12, lens=lens)
    q = I.make_q(sh, 12)
    C = 7
    _, (o, m, l), _ = fused_attention(tq, torch, dev, q, sh.alpha, num_splits=C)
    bounds = np.zeros((2, C + 1), np.int32)
    for b in range(2):
        for c in range(C):
            bounds[b, c], bounds[b, c + 1] = tq.tq_split_range(lens[b], C, c)
    ro, rm, rl = oracle.attention_partials(host, q, sh.alpha, bounds)
    o, m, l = o.cpu().numpy(), m.cpu().numpy(), l.cpu().numpy()
    empty = rl == 0
    assert empty.any()  # 50 tokens are 4 blocks of 16: cut into 7 splits, some are empty
    assert np.all(l[empty] == 0) and np.all(np.isneginf(m[empty])) and np.all(o[empty] == 0)
    ne = ~empty
    # (m, l) may be reported relative to a slightly different reference than the exact maximum,
    # what is unique is m + log(l) and the normalised output
    assert np.abs((m[ne] + np.log(l[ne])) - (rm[ne] + np.log(rl[ne]))).max() < 1e-3
    assert np.all(m[ne] <= rm[ne] + 1e-4) and np.all(m[ne] >= rm[ne] - 4 * np.log(2) - 1e-4)
    assert_attention_close(o[ne], ro[ne], "partials")
    # and they recombine through the oracle's Eq. 5 to the oracle's answer
    assert_attention_close(oracle.combine(o, m, l), oracle.attention(host, q, sh.alpha), "oracle-combined")


def test_combine_alone_matches_eq5(gpu, oracle):
    tq, torch = gpu
    rng = np.random.default_rng(13)
    B, H, Cn, d = 2, 5, 9, 128
    o = rng.standard_normal((B, H, Cn, d))
    m = rng.standard_normal((B, H, Cn)) * 20
    l = rng.uniform(0.5, 500, (B, H, Cn))
    l[0, 0, 3] = 0; m[0, 0, 3] = -np.inf; o[0, 0, 3] = 0           # one empty split
    l[1, 2, :] = 0; m[1, 2, :] = -np.inf; o[1, 2, :] = 0           # a row whose splits are all empty
    ref = oracle.combine(o, m, l)
    to = lambda a: torch.from_numpy(a.astype(np.float32)).cuda()
    ref = oracle.combine(o.astype(np.float32), m.astype(np.float32), l.astype(np.float32))
    for dt in (torch.float32, torch.float16):
        # guard bands around the output catch out-of-bounds writes
        buf = torch.full((B * H * d + 64,), 7.0, dtype=dt, device="cuda")
        out = buf[32:32 + B * H * d].view(B, H, d)
        tq.tq_sdpa_int4_combine(to(o), to(m), to(l), out)
        torch.cuda.synchronize()
        got = out.float().cpu().numpy()
        tol = 1e-5 if dt == torch.float32 else 2e-3
        assert np.abs(got - ref).max() <= tol * max(1.0, np.abs(ref).max())
        assert np.all(got[1, 2] == 0)
        assert torch.all(buf[:32] == 7.0) and torch.all(buf[32 + B * H * d:] == 7.0)


@pytest.mark.parametrize("ws_fp32", [True, False])
def test_dequant_then_attend_matches_oracle(gpu, oracle, ws_fp32):
    tq, torch = gpu
    sh = I.Shape("x", 2, 16, 2, 128, 128 ** -0.5, k_outlier_channels=2)
    lens = [2048, 777]
    host, dev = _both(gpu, oracle, sh, 2048, 14, lens=lens)
    q = I.make_q(sh, 14)
    ref = oracle.attention(host, q, sh.alpha)
    nbytes = tq.tq_dequant_workspace_bytes(sh.B, sh.H_kv, sh.H_q, 2048, sh.d, ws_fp32)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    out = torch.empty((sh.B, sh.H_q, sh.d), dtype=torch.float32, device="cuda")
    tq.tq_sdpa_dequant_then_attend(dev, torch.from_numpy(q).cuda(), sh.alpha, ws, ws_fp32, out)
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    if ws_fp32:
        assert_attention_close(got, ref, "dequant-then-attend fp32")
    else:  # an fp16 matrix rounds every k^, v^ to 11 bits: looser, reported not gated at 1e-3
        mx, rel = errors(got, ref)
        assert mx <= MAX_ABS_TOL and rel <= 3e-3
    # the materialised matrix itself: fp32 rounding of (q - z) * s
    if ws_fp32:
        kmat = ws[:sh.B * sh.H_kv * 2048 * sh.d * 4].view(torch.float32).view(sh.B, sh.H_kv, 2048, sh.d).cpu().numpy()
        kd = oracle.dequant_rows(host.k_packed, host.k_scale, host.k_zero)
        for b in range(2):
            assert np.abs(kmat[b, :, :lens[b]] - kd[b, :, :lens[b]]).max() <= 2.0 ** -22 * np.abs(kd).max()


@pytest.mark.parametrize("H_q,H_kv", [(2, 2), (8, 2), (16, 2), (24, 2)])
@pytest.mark.parametrize("ws_fp32", [True, False])
def test_dequant_then_attend_head_groups_and_ragged_ends(gpu, oracle, H_q, H_kv, ws_fp32):
    """The comparison path at d = 128 with 1, 4, 8 query heads per KV head (tensor-core attention over the
    materialised matrices) and 12 (the scalar kernel), lengths that end inside a 16-token block, a
    one-token and an empty sequence."""
    tq, torch = gpu
    sh = I.Shape("x", 4, H_q, H_kv, 128, 128 ** -0.5, k_outlier_channels=2)
    lens = [1000, 1, 0, 4113]
    host, dev = _both(gpu, oracle, sh, 4113, 16, S_cap=4128, lens=lens)
    q = I.make_q(sh, 16)
    ref = oracle.attention(host, q, sh.alpha)
    nbytes = tq.tq_dequant_workspace_bytes(sh.B, sh.H_kv, sh.H_q, 4128, sh.d, ws_fp32)
    ws = torch.full((nbytes,), 0xFF, dtype=torch.uint8, device="cuda")     # rows nobody wrote are NaN patterns
    out = torch.full((sh.B, sh.H_q, sh.d), 7.0, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    tq.tq_sdpa_dequant_then_attend(dev, torch.from_numpy(q).cuda(), sh.alpha, ws, ws_fp32, out, status)
    torch.cuda.synchronize()
    assert int(status.item()) == tq.TQ_STATUS_EMPTY_SEQ
    got = out.cpu().numpy()
    assert not got[2].any()                                                  # the empty sequence: zeros
    keep = [0, 1, 3]
    if ws_fp32:
        assert_attention_close(got[keep], ref[keep], f"dequant-then-attend {H_q}/{H_kv}")
    else:
        # an fp16 matrix rounds every v^ to 11 bits: the one-token sequence returns fp16(v^_0), half an fp16 ulp off
        mx, rel = errors(got[keep], ref[keep])
        assert mx <= MAX_ABS_TOL + np.abs(ref).max() * 2.0 ** -11 and rel <= 3e-3


def test_simple_reference_kernel_matches_oracle(gpu, oracle):
    tq, torch = gpu
    sh = I.Shape("x", 2, 24, 2, 128, 128 ** -0.5)
    host, dev = _both(gpu, oracle, sh, 512, 15, lens=[512, 100])
    q = I.make_q(sh, 15)
    tq._test_hook(tq.HOOK_DECODE_IMPL, 1)
    try:
        out, _, _ = fused_attention(tq, torch, dev, q, sh.alpha, num_splits=5)
    finally:
        tq._test_hook(tq.HOOK_DECODE_IMPL, 0)
    assert_attention_close(out, oracle.attention(host, q, sh.alpha), "simple")


def test_empty_sequence_sets_status_and_returns_zero(gpu, oracle):
    tq, torch = gpu
    sh = I.Shape("x", 2, 8, 2, 128, 0.1)
    host, dev = _both(gpu, oracle, sh, 64, 16, lens=[0, 64], fill_byte=0xFF)
    q = I.make_q(sh, 16)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out, _, _ = fused_attention(tq, torch, dev, q, sh.alpha, num_splits=2, status=status)
    assert int(status.item()) == tq.TQ_STATUS_EMPTY_SEQ
    assert np.all(out[0] == 0)
    assert_attention_close(out[1:], oracle.attention(host, q, sh.alpha)[1:], "non-empty sequence")


def test_outputs_stay_inside_their_buffers(gpu, oracle):
    tq, torch = gpu
    sh = I.Shape("x", 1, 8, 1, 128, 0.1)
    host, dev = _both(gpu, oracle, sh, 200, 17, S_cap=208)
    q = torch.from_numpy(I.make_q(sh, 17)).cuda()
    C = 3
    n = sh.B * sh.H_q * C
    bo = torch.full((n * sh.d + 128,), 3.0, device="cuda")
    bm = torch.full((n + 128,), 3.0, device="cuda")
    bl = torch.full((n + 128,), 3.0, device="cuda")
    tq.tq_sdpa_int4_decode(dev, q, sh.alpha, C, bo[64:], bm[64:], bl[64:])
    torch.cuda.synchronize()
    for buf, size in ((bo, n * sh.d), (bm, n), (bl, n)):
        assert torch.all(buf[:64] == 3.0) and torch.all(buf[64 + size:] == 3.0)
        assert not torch.any(buf[64:64 + size] == 3.0)


def test_constant_v_and_single_token(gpu, oracle):
    tq, torch = gpu
    sh = I.Shape("x", 1, 8, 1, 128, 128 ** -0.5)
    k, _ = I.make_kv(sh, 320, 18)
    v = np.full_like(k, np.float16(-2.75))
    host = oracle_cache(oracle, sh, k, v, 320)
    dev = device_cache(tq, torch, sh, k, v, 320)
    q = I.make_q(sh, 18)
    out, _, _ = fused_attention(tq, torch, dev, q, sh.alpha, num_splits=3)
    assert np.abs(out + 2.75).max() <= 1e-3
    dev.seq_lens.fill_(1)
    host.lens[:] = 1
    out1, _, _ = fused_attention(tq, torch, dev, q, sh.alpha, num_splits=2)
    assert np.abs(out1 + 2.75).max() <= 1e-3


def test_full_size_128k_llama_layer_in_bench_configuration(gpu, oracle):
    """One 128K-token Llama-70B-shaped layer, default split count (the launch the benchmark
    times), every query head checked against the oracle."""
    tq, torch = gpu
    S = 131072
    host, dev = _both(gpu, oracle, I.LLAMA, S, 20)
    assert_cache_bits_equal(dev, host)
    q = I.make_q(I.LLAMA, 20)
    ref = oracle.attention(host, q, I.LLAMA.alpha)
    out, _, C = fused_attention(tq, torch, dev, q, I.LLAMA.alpha)
    mx, rel = assert_attention_close(out, ref, "llama/128K")
    print(f"llama 128K C={C}: max-abs {mx:.2e} rel-L2 {rel:.2e}")


@pytest.mark.parametrize("entry", ["calls", "step"])
def test_config5_ragged_batch_64_decode_steps(gpu, oracle, entry):
    """Batched ragged decode: B = 16, Llama-70B head shapes, context lengths uniform in [4096, 65536],
    64 consecutive steps of quantize-append followed by fused attention, as three calls per step or as one
    launch per step (tq_sdpa_int4_step_ragged, every sequence's length before the steps as its stable part).  The shortest and the longest
    sequence carry seeded data and are checked against the oracle at the first and the last step (cache
    bit-exact, attention within tolerance); the other sequences hold zeros but have their drawn lengths,
    so the launch has the real ragged work distribution."""
    tq, torch = gpu
    sh = I.RAGGED
    lens = I.ragged_lengths(sh.B, 4096, 65536, seed=5)
    S_cap = 65536 + 64
    picked = [int(np.argmin(lens)), int(np.argmax(lens))]
    one = I.Shape("ragged-1seq", 1, sh.H_q, sh.H_kv, sh.d, sh.alpha, k_outlier_channels=sh.k_outlier_channels)
    dev = tq.KVCache(sh.B, sh.H_kv, S_cap, sh.d)
    host = {}
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for b in picked:  # prefill the two sampled sequences through the CUDA quantiser, one sequence at a time
        k, v = I.make_kv(one, int(lens[b]), seed=500 + b)
        host[b] = oracle.Cache(1, sh.H_kv, S_cap, sh.d)
        host[b].append(k, v)
        view = tq.tq_kv_cache(dev.blocks[b].data_ptr(), dev.seq_lens[b:b + 1].data_ptr(), 1, sh.H_kv, S_cap, sh.d)
        tq.tq_kv_quantize_append(view, torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda(), status)
    dev.seq_lens.copy_(torch.from_numpy(lens))
    C = (tq.tq_auto_splits if entry == "calls" else tq.tq_auto_splits_step)(sh.B, sh.H_kv, sh.H_q, sh.d, S_cap)
    o, m, l = tq.alloc_partials(sh.B, sh.H_q, sh.d, C)
    ws = tq.alloc_step_workspace(sh.B, sh.H_kv, sh.H_q, sh.d, C)
    stable = torch.from_numpy(lens.astype(np.int32)).cuda()
    out = torch.empty((sh.B, sh.H_q, sh.d), dtype=torch.float32, device="cuda")
    for step in range(64):
        k_new = np.zeros((sh.B, sh.H_kv, 1, sh.d), np.float16)
        v_new = np.zeros_like(k_new)
        q = np.zeros((sh.B, sh.H_q, sh.d), np.float16)
        for b in picked:
            kb, vb = I.make_kv(one, 1, seed=500 + b, stream=1 + step)
            k_new[b], v_new[b] = kb[0], vb[0]
            q[b] = I.make_q(one, seed=500 + b, stream=step)[0]
            host[b].append(kb, vb)
        if entry == "calls":
            tq.tq_kv_quantize_append(dev, torch.from_numpy(k_new).cuda(), torch.from_numpy(v_new).cuda(), status)
            tq.tq_sdpa_int4_decode(dev, torch.from_numpy(q).cuda(), sh.alpha, C, o, m, l, status)
            tq.tq_sdpa_int4_combine(o, m, l, out)
        else:
            tq.tq_sdpa_int4_step(dev, torch.from_numpy(k_new).cuda(), torch.from_numpy(v_new).cuda(),
                                 torch.from_numpy(q).cuda(), sh.alpha, C, stable, ws, out, status)
        if step in (0, 63):
            torch.cuda.synchronize()
            got = out.cpu().numpy()
            for b in picked:
                n = int(lens[b]) + step + 1
                assert int(host[b].lens[0]) == n
                for d_arr, h_arr in zip(dev.arrays_token_major(), host[b].arrays()):
                    assert np.array_equal(d_arr[b, :, :n].cpu().numpy().view(np.uint8), h_arr[0, :, :n].view(np.uint8))
                ref = oracle.attention(host[b], q[b:b + 1], sh.alpha)
                mx, rel = assert_attention_close(got[b:b + 1], ref, f"ragged step {step} seq {b}")
                print(f"ragged step {step} seq {b} len {n}: max-abs {mx:.2e} rel-L2 {rel:.2e}")
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert dev.seq_lens.cpu().tolist() == [int(x) + 64 for x in lens]


@pytest.mark.parametrize("d,H_q,H_kv", [(256, 32, 16), (128, 16, 2), (64, 4, 1)])
def test_sliding_window_decode(gpu, oracle, d, H_q, H_kv):
    """Appendix A: sliding-window layers (w = 1024 in the paper).  Windows that start inside a 16-token
    block, are longer than the sequence, are a single token, plus ragged lengths and several split
    counts; partial ranges are also checked against tq_split_range_window."""
    tq, torch = gpu
    sh = I.Shape("x", 4, H_q, H_kv, d, d ** -0.5 if d != 256 else 1.0, sigma_qk=1.0 if d != 256 else 0.25)
    lens = [3000, 1024, 1029, 7]
    host, dev = _both(gpu, oracle, sh, 3008, 51, S_cap=3008, lens=lens, fill_byte=0xFF)
    q = I.make_q(sh, 51)
    qd = torch.from_numpy(q).cuda()
    for window, C in ((1024, 0), (1024, 5), (1000, 3), (1, 2), (17, 1), (5000, 4), (0, 2)):
        ref = oracle.attention_window(host, q, sh.alpha, window)
        Cn = C or tq.tq_auto_splits(sh.B, sh.H_kv, sh.H_q, sh.d, window or 3008)
        o, m, l = tq.alloc_partials(sh.B, sh.H_q, sh.d, Cn)
        out = torch.empty((sh.B, sh.H_q, sh.d), dtype=torch.float32, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        tq.tq_sdpa_int4_decode_window(dev, qd, sh.alpha, window, C, o, m, l, status)
        tq.tq_sdpa_int4_combine(o, m, l, out)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert_attention_close(out.cpu().numpy(), ref, f"window {window} C {C}")
    # the partition covers exactly the window
    for length, window, Cn in ((3000, 1024, 5), (1029, 1024, 3), (7, 1024, 2), (100, 1, 4)):
        prev = max(0, length - window)
        for c in range(Cn):
            t0, t1 = tq.tq_split_range_window(length, window, Cn, c)
            assert t0 == prev and t1 >= t0
            prev = t1
        assert prev == length


@pytest.mark.parametrize("d,H_q,H_kv,S_q", [(256, 32, 16, 4), (128, 64, 8, 3), (64, 4, 1, 5), (128, 8, 4, 16)])
@pytest.mark.parametrize("impl", ["mma", "simple"])
def test_multi_query_decode(gpu, oracle, d, H_q, H_kv, S_q, impl):
    """Several query tokens per sequence (the S_q factor of Appendix A), causal among themselves, with and
    without a sliding window: one tile (G * S_q = 8), several tiles, a partly filled last tile; lengths
    whose newest S_q tokens straddle a 16-token block, and a sequence shorter than S_q."""
    tq, torch = gpu
    sh = I.Shape("x", 4, H_q, H_kv, d, d ** -0.5 if d != 256 else 1.0, sigma_qk=1.0 if d != 256 else 0.25)
    lens = [2000, 1026, 2, 48]
    host, dev = _both(gpu, oracle, sh, 2000, 61, S_cap=2000, lens=lens, fill_byte=0xFF)
    q = np.ascontiguousarray(np.stack([I.make_q(sh, 61, stream=s) for s in range(S_q)], axis=1))
    qd = torch.from_numpy(q).cuda()
    if impl == "simple":
        tq._test_hook(tq.HOOK_DECODE_IMPL, 1)
    try:
        for window, C in ((0, 0), (0, 3), (1024, 0), (20, 2), (1, 1)):
            ref = oracle.attention_multi(host, q, sh.alpha, window)
            Cn = C or tq.tq_auto_splits(sh.B, sh.H_kv, sh.H_q * S_q, sh.d, window or 2000)
            o, m, l = tq.alloc_partials(sh.B, sh.H_q * S_q, sh.d, Cn)
            out = torch.empty((sh.B, S_q, sh.H_q, sh.d), dtype=torch.float32, device="cuda")
            status = torch.zeros(1, dtype=torch.int32, device="cuda")
            tq.tq_sdpa_int4_decode_multi(dev, qd, sh.alpha, window, C, o, m, l, status)
            tq.tq_sdpa_int4_combine(o, m, l, out.view(sh.B, S_q * sh.H_q, sh.d))
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            got = out.cpu().numpy()
            for s in range(S_q):  # query tokens older than the sequence attend nothing
                if 2 - (S_q - 1 - s) <= 0:
                    assert not got[2, s].any() and not ref[2, s].any()
            assert_attention_close(got.reshape(sh.B, -1, sh.d), ref.reshape(sh.B, -1, sh.d), f"S_q {S_q} window {window} C {C}")
    finally:
        tq._test_hook(tq.HOOK_DECODE_IMPL, 0)


@pytest.mark.parametrize("d,H_q,H_kv", [(128, 16, 2), (256, 8, 4)])
@pytest.mark.parametrize("paged", [False, True])
def test_general_forms_on_long_ranges(gpu, oracle, d, H_q, H_kv, paged):
    """Sliding windows and several query tokens over ranges long enough that every warp (team) first walks the
    masked blocks at the old end of its range one by one and then enters the four-block loop, with few splits,
    window starts inside a block and lengths that end inside one; contiguous and from a page pool."""
    tq, torch = gpu
    sh = I.Shape("x", 2, H_q, H_kv, d, d ** -0.5 if d != 256 else 1.0, sigma_qk=1.0 if d != 256 else 0.25)
    lens = [9000, 5531]
    k, v = I.make_kv(sh, 9000, 71)
    if paged:
        host = oracle.Cache(sh.B, sh.H_kv, 9024, sh.d)
        dev = _paged(tq, torch, sh, 64, 9024 // 64, 71)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        host.append(k[:, :, :5531], v[:, :, :5531])
        tq.tq_kv_quantize_append(dev, torch.from_numpy(np.ascontiguousarray(k[:, :, :5531])).cuda(),
                                 torch.from_numpy(np.ascontiguousarray(v[:, :, :5531])).cuda(), status)
        assert int(status.item()) == 0          # (both sequences 5531 tokens: the last block holds 11)
    else:
        host, dev = _both(gpu, oracle, sh, 9000, 71, S_cap=9008, lens=lens, fill_byte=0xFF)
    for S_q, window, C in ((1, 5000, 1), (1, 777, 2), (3, 0, 1), (3, 4100, 2), (1, 8999, 3)):
        q = np.ascontiguousarray(np.stack([I.make_q(sh, 71, stream=s) for s in range(S_q)], axis=1))
        ref = oracle.attention_multi(host, q, sh.alpha, window)
        o, m, l = tq.alloc_partials(sh.B, sh.H_q * S_q, sh.d, C)
        out = torch.empty((sh.B, S_q, sh.H_q, sh.d), dtype=torch.float32, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        tq.tq_sdpa_int4_decode_multi(dev, torch.from_numpy(q).cuda(), sh.alpha, window, C, o, m, l, status)
        tq.tq_sdpa_int4_combine(o, m, l, out.view(sh.B, S_q * sh.H_q, sh.d))
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert_attention_close(out.cpu().numpy().reshape(sh.B, -1, sh.d), ref.reshape(sh.B, -1, sh.d),
                               f"S_q {S_q} window {window} C {C} paged {paged}")


@pytest.mark.parametrize("impl", ["mma", "simple"])
def test_head_dim_512(gpu, oracle, impl):
    """Table 7's Gemma global layers: d = 512, 32 query heads per KV head (four head tiles).  Decode after a
    bulk fill and a T = 1 append, with ragged lengths, explicit and automatic splits, a window and several
    query tokens."""
    tq, torch = gpu
    sh = I.Shape("global512", 2, 64, 2, 512, 1.0, sigma_qk=0.2)
    lens = [1500, 333]
    host, dev = _both(gpu, oracle, sh, 1500, 71, S_cap=1520, lens=lens, fill_byte=0xFF)
    k1, v1 = I.make_kv(sh, 1, 71, stream=1)
    host.append(k1, v1)
    tq.tq_kv_quantize_append(dev, torch.from_numpy(k1).cuda(), torch.from_numpy(v1).cuda())
    assert_cache_bits_equal(dev, host)
    q = I.make_q(sh, 71)
    if impl == "simple":
        tq._test_hook(tq.HOOK_DECODE_IMPL, 1)
    try:
        for C in (0, 1, 5):
            out, _, _ = fused_attention(tq, torch, dev, q, sh.alpha, num_splits=C)
            assert_attention_close(out, oracle.attention(host, q, sh.alpha), f"d512 C={C}")
        q3 = np.ascontiguousarray(np.stack([I.make_q(sh, 71, stream=s) for s in range(3)], axis=1))
        for window in (0, 100):
            o, m, l = tq.alloc_partials(sh.B, sh.H_q * 3, sh.d, 4)
            out = torch.empty((sh.B, 3, sh.H_q, sh.d), dtype=torch.float32, device="cuda")
            tq.tq_sdpa_int4_decode_multi(dev, torch.from_numpy(q3).cuda(), sh.alpha, window, 4, o, m, l)
            tq.tq_sdpa_int4_combine(o, m, l, out.view(sh.B, 3 * sh.H_q, sh.d))
            torch.cuda.synchronize()
            ref = oracle.attention_multi(host, q3, sh.alpha, window)
            assert_attention_close(out.cpu().numpy().reshape(sh.B, -1, sh.d), ref.reshape(sh.B, -1, sh.d), f"d512 w={window}")
    finally:
        tq._test_hook(tq.HOOK_DECODE_IMPL, 0)


def test_mixed_precision_attend_matches_oracle(gpu, oracle):
    """Sec. 5 ablation path: K and V each from the int4 cache or from the unquantised fp16 values."""
    tq, torch = gpu
    sh = I.Shape("x", 2, 16, 2, 128, 128 ** -0.5, k_outlier_channels=4)
    k, v = I.make_kv(sh, 600, 81)
    lens = [600, 77]
    host = oracle_cache(oracle, sh, k, v, 608, lens)
    dev = device_cache(tq, torch, sh, k, v, 608, lens)
    pad = lambda a: np.ascontiguousarray(np.pad(a, ((0, 0), (0, 0), (0, 8), (0, 0))))
    kf, vf = torch.from_numpy(pad(k)).cuda(), torch.from_numpy(pad(v)).cuda()
    q = I.make_q(sh, 81)
    qd = torch.from_numpy(q).cuda()
    for use_k, use_v in ((False, False), (True, False), (False, True), (True, True)):
        o, m, l = tq.alloc_partials(sh.B, sh.H_q, sh.d, 3)
        out = torch.empty((sh.B, sh.H_q, sh.d), dtype=torch.float32, device="cuda")
        tq.tq_sdpa_mixed_precision_attend(dev, kf if use_k else None, vf if use_v else None, qd, sh.alpha, 3, o, m, l)
        tq.tq_sdpa_int4_combine(o, m, l, out)
        torch.cuda.synchronize()
        ref = oracle.attention_mixed(host, k if use_k else None, v if use_v else None, q, sh.alpha)
        assert_attention_close(out.cpu().numpy(), ref, f"mixed k_fp16={use_k} v_fp16={use_v}")


def _paged(tq, torch, sh, page_tokens, max_pages, seed):
    """A paged cache whose page table is a seeded random assignment of distinct pool pages."""
    num_pages = sh.B * max_pages + 3
    cache = tq.PagedKVCache(sh.B, sh.H_kv, page_tokens, max_pages, num_pages, sh.d)
    perm = np.random.default_rng(seed).permutation(num_pages)[:sh.B * max_pages].astype(np.int32)
    cache.page_table.copy_(torch.from_numpy(perm.reshape(sh.B, max_pages)))
    cache.blocks.fill_(0xFF)
    return cache


@pytest.mark.parametrize("d,H_q,H_kv,page_tokens", [(128, 16, 2, 64), (256, 8, 4, 16), (64, 4, 1, 128), (512, 32, 1, 32)])
def test_paged_cache_append_and_decode(gpu, oracle, d, H_q, H_kv, page_tokens):
    """The cache served from a pool of pages through a page table (random page assignment): bulk and
    single-token appends are bit-exact against the oracle, decode (plain, windowed, several query tokens)
    and the comparison path match it, and the result equals the contiguous cache's bit for bit."""
    tq, torch = gpu
    sh = I.Shape("x", 3, H_q, H_kv, d, d ** -0.5 if d < 256 else 1.0, sigma_qk=1.0 if d < 256 else 0.25)
    S = 700
    max_pages = (S + 40 + page_tokens - 1) // page_tokens
    k, v = I.make_kv(sh, S, 91)
    host = oracle.Cache(sh.B, sh.H_kv, page_tokens * max_pages, sh.d)
    host.append(k, v)
    dev = _paged(tq, torch, sh, page_tokens, max_pages, 91)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    tq.tq_kv_quantize_append(dev, torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda(), status)
    for step in range(3):
        k1, v1 = I.make_kv(sh, 1, 91, stream=1 + step)
        host.append(k1, v1)
        tq.tq_kv_quantize_append(dev, torch.from_numpy(k1).cuda(), torch.from_numpy(v1).cuda(), status)
    assert_cache_bits_equal(dev, host)
    flat = dev.contiguous()
    q = I.make_q(sh, 91)
    for C in (0, 3):
        out, o_p, _ = fused_attention(tq, torch, dev, q, sh.alpha, num_splits=C)
        assert_attention_close(out, oracle.attention(host, q, sh.alpha), f"paged C={C}")
        out_flat, o_f, _ = fused_attention(tq, torch, flat, q, sh.alpha, num_splits=C)
        assert np.array_equal(out, out_flat)
    q3 = np.ascontiguousarray(np.stack([I.make_q(sh, 91, stream=s) for s in range(3)], axis=1))
    for window in (0, 100):
        o, m, l = tq.alloc_partials(sh.B, sh.H_q * 3, sh.d, 2)
        out = torch.empty((sh.B, 3, sh.H_q, sh.d), dtype=torch.float32, device="cuda")
        tq.tq_sdpa_int4_decode_multi(dev, torch.from_numpy(q3).cuda(), sh.alpha, window, 2, o, m, l, status)
        tq.tq_sdpa_int4_combine(o, m, l, out.view(sh.B, 3 * sh.H_q, sh.d))
        ref = oracle.attention_multi(host, q3, sh.alpha, window)
        assert_attention_close(out.cpu().numpy().reshape(sh.B, -1, sh.d), ref.reshape(sh.B, -1, sh.d), f"paged w={window}")
    # comparison path through the page table
    need = tq.tq_dequant_workspace_bytes(sh.B, sh.H_kv, sh.H_q, dev.S_cap, sh.d, False)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    out = torch.empty((sh.B, sh.H_q, sh.d), dtype=torch.float32, device="cuda")
    tq.tq_sdpa_dequant_then_attend(dev, torch.from_numpy(q).cuda(), sh.alpha, ws, False, out, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert_attention_close(out.cpu().numpy(), oracle.attention(host, q, sh.alpha), "paged dequant-then-attend")


def test_paged_cache_bad_page_is_flagged_not_followed(gpu, oracle):
    tq, torch = gpu
    sh = I.Shape("x", 2, 8, 2, 128, 0.1)
    dev = _paged(tq, torch, sh, 32, 4, 5)
    k, v = I.make_kv(sh, 100, 5)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    tq.tq_kv_quantize_append(dev, torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda(), status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    before = dev.blocks.clone()
    dev.page_table[1, 1] = dev.num_pages + 7   # tokens 32..63 of sequence 1
    dev.page_table[0, 3] = -1                  # tokens 96..127 of sequence 0 (the next append lands there)
    q = I.make_q(sh, 5)
    out, _, _ = fused_attention(tq, torch, dev, q, sh.alpha, num_splits=2, status=status)
    assert int(status.item()) & 16                 # flagged; the reads went to pool page 0, not out of bounds
    assert np.all(np.isfinite(out[0]))             # sequence 0's bad entry lies beyond its length and is never read
    status.zero_()
    k1, v1 = I.make_kv(sh, 1, 5, stream=1)
    tq.tq_kv_quantize_append(dev, torch.from_numpy(k1).cuda(), torch.from_numpy(v1).cuda(), status)
    torch.cuda.synchronize()
    assert int(status.item()) & 16
    changed = (dev.blocks != before).flatten(1).any(dim=1).cpu().numpy()
    assert changed.sum() == 1 and changed[int(dev.page_table[1, 3])]  # only sequence 1's page was written


def test_decode_step_replays_as_a_cuda_graph(gpu, oracle):
    """The whole step (append, decode, combine) is captured once and replayed: lengths live in device memory,
    so every replay appends at the next position and attends one token more; each replay matches the oracle
    and the eager calls bit for bit."""
    tq, torch = gpu
    sh = I.Shape("x", 2, 16, 2, 128, 128 ** -0.5, k_outlier_channels=4)
    lens = [500, 90]
    host, dev = _both(gpu, oracle, sh, 500, 97, S_cap=512, lens=lens)
    eager = tq.KVCache(sh.B, sh.H_kv, 512, sh.d)
    eager.blocks.copy_(dev.blocks)
    eager.seq_lens.copy_(dev.seq_lens)
    C = 3
    o, m, l = tq.alloc_partials(sh.B, sh.H_q, sh.d, C)
    out = torch.empty((sh.B, sh.H_q, sh.d), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    k_in = torch.empty((sh.B, sh.H_kv, 1, sh.d), dtype=torch.float16, device="cuda")
    v_in = torch.empty_like(k_in)
    q_in = torch.empty((sh.B, sh.H_q, sh.d), dtype=torch.float16, device="cuda")

    def step(cache):
        tq.tq_kv_quantize_append(cache, k_in, v_in, status)
        tq.tq_sdpa_int4_decode(cache, q_in, sh.alpha, C, o, m, l, status)
        tq.tq_sdpa_int4_combine(o, m, l, out)

    k1, v1 = I.make_kv(sh, 1, 97, stream=1)
    k_in.copy_(torch.from_numpy(k1)); v_in.copy_(torch.from_numpy(v1)); q_in.copy_(torch.from_numpy(I.make_q(sh, 97)))
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step(eager)                       # warm-up outside the capture (sets function attributes), on the eager copy
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    host.append(k1, v1)
    eager_out = [out.clone()]
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        step(dev)
    for i in range(3):
        kn, vn = I.make_kv(sh, 1, 97, stream=1 + i)
        qn = I.make_q(sh, 97, stream=i)
        k_in.copy_(torch.from_numpy(kn)); v_in.copy_(torch.from_numpy(vn)); q_in.copy_(torch.from_numpy(qn))
        if i > 0:
            host.append(kn, vn)
            step(eager)
            torch.cuda.synchronize()
            eager_out.append(out.clone())
        g.replay()
        torch.cuda.synchronize()
        assert dev.seq_lens.tolist() == [lens[0] + i + 1, lens[1] + i + 1]
        assert_attention_close(out.cpu().numpy(), oracle.attention(host, qn, sh.alpha), f"graph replay {i}")
        assert torch.equal(out, eager_out[i])
    assert int(status.item()) == 0
    assert_cache_bits_equal(dev, host)


def test_offsets_beyond_4_gib(gpu, oracle):
    """A 4M-token cache (5.4 GB) whose only tokens sit at its very end: bulk append, single-token append and
    windowed decode address blocks more than 2^32 bytes into the buffer."""
    tq, torch = gpu
    sh = I.Shape("x", 1, 64, 8, 128, 128 ** -0.5, k_outlier_channels=4)
    S_cap = 1 << 22
    start = S_cap - 208
    dev = tq.KVCache(sh.B, sh.H_kv, S_cap, sh.d)
    assert dev.blocks.numel() > (1 << 32)
    dev.seq_lens.fill_(start)
    k, v = I.make_kv(sh, 150, 103)
    k1, v1 = I.make_kv(sh, 1, 103, stream=1)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    tq.tq_kv_quantize_append(dev, torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda(), status)
    tq.tq_kv_quantize_append(dev, torch.from_numpy(k1).cuda(), torch.from_numpy(v1).cuda(), status)
    host = oracle.Cache(sh.B, sh.H_kv, 160, sh.d)
    host.append(k, v)
    host.append(k1, v1)
    q = I.make_q(sh, 103)
    for window, C in ((120, 1), (151, 3), (40, 0)):
        o, m, l = tq.alloc_partials(sh.B, sh.H_q, sh.d, C or tq.tq_auto_splits(sh.B, sh.H_kv, sh.H_q, sh.d, window))
        out = torch.empty((sh.B, sh.H_q, sh.d), dtype=torch.float32, device="cuda")
        tq.tq_sdpa_int4_decode_window(dev, torch.from_numpy(q).cuda(), sh.alpha, window, C, o, m, l, status)
        tq.tq_sdpa_int4_combine(o, m, l, out)
        torch.cuda.synchronize()
        assert_attention_close(out.cpu().numpy(), oracle.attention_window(host, q, sh.alpha, window), f"4GiB w={window}")
    assert int(status.item()) == 0 and dev.seq_lens.tolist() == [start + 151]
    # the rows written are the oracle's, bit for bit (read back through the offset helpers)
    blocks = dev.blocks[0, :, (start >> 4):].cpu()
    tail = tq.KVCache(1, sh.H_kv, blocks.shape[1] * 16, sh.d, device="cpu")
    tail.blocks.copy_(blocks.unsqueeze(0))
    for d_arr, h_arr in zip(tail.arrays_token_major(), host.arrays()):
        assert np.array_equal(d_arr[0, :, :151].numpy().view(np.uint8), h_arr[0, :, :151].view(np.uint8))


def test_many_sequences_and_the_widest_gqa(gpu, oracle):
    """B = 96 short sequences (grid z) and 64 query heads on one KV head (eight head tiles)."""
    tq, torch = gpu
    sh = I.Shape("x", 96, 2, 1, 64, 0.125)
    lens = [1 + (7 * i) % 80 for i in range(96)]
    host, dev = _both(gpu, oracle, sh, 80, 111, lens=lens, fill_byte=0xFF)
    q = I.make_q(sh, 111)
    out, _, _ = fused_attention(tq, torch, dev, q, sh.alpha)
    assert_attention_close(out, oracle.attention(host, q, sh.alpha), "B=96")
    sh = I.Shape("x", 1, 64, 1, 128, 128 ** -0.5)
    host, dev = _both(gpu, oracle, sh, 1000, 112, fill_byte=0xFF)
    q = I.make_q(sh, 112)
    for C in (0, 2):
        out, _, _ = fused_attention(tq, torch, dev, q, sh.alpha, num_splits=C)
        assert_attention_close(out, oracle.attention(host, q, sh.alpha), f"G=64 C={C}")
