"""tq_sdpa_int4_attend_static: the entry point for callers that cannot allocate device memory (a
server whose memory pool owns the whole GPU, code inside a stream capture, a decode loop that
cannot afford the device-wide stall of cudaMalloc).  Its split partials sit in a fixed array inside
the library, so the test checks what matters for such a caller: same answer as the two-call path
that uses caller-provided partials and as the CPU oracle, on calls in a row with different inputs
and cache forms (the array keeps the previous call's contents), and a clean refusal when the
partials cannot fit."""
import ctypes as C

import numpy as np
import pytest

from paper_2604_16957_b200 import inputs as I
from util import MAX_ABS_TOL, REL_L2_TOL, assert_attention_close, device_cache, errors, fused_attention, oracle_cache

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gpu():
    import torch
    from paper_2604_16957_b200 import tq
    assert torch.cuda.is_available()
    return tq, torch


def _static(tq, torch, cache, q_np, alpha, dtype):
    q = torch.from_numpy(q_np).cuda()
    out = torch.full(q.shape, 7.0, dtype=dtype, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    tq.tq_sdpa_int4_attend_static(cache, q, alpha, out, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return out.float().cpu().numpy()


def test_two_calls_in_a_row_match_the_two_call_path(gpu, oracle):
    tq, torch = gpu
    # call 1: Llama-shaped heads, ragged batch;  call 2: other shape, other data, fewer partials --
    # whatever call 1 left in the shared array must not show up in call 2's result
    cases = [(I.Shape("a", 3, 64, 8, 128, 128 ** -0.5, k_outlier_channels=4), [4096, 1000, 17], 4096, 31),
             (I.Shape("b", 1, 8, 2, 256, 1.0, sigma_qk=0.25), [777], 784, 32)]
    for sh, lens, S, seed in cases:
        k, v = I.make_kv(sh, S, seed)
        cache = device_cache(tq, torch, sh, k, v, S, lens=lens, fill_byte=0xFF)
        q = I.make_q(sh, seed)
        ref, _, _ = fused_attention(tq, torch, cache, q, sh.alpha)           # existing entry points
        want = oracle.attention(oracle_cache(oracle, sh, k, v, S, lens=lens), q, sh.alpha)   # and the CPU oracle
        for dtype in (torch.float32, torch.float16):
            got = _static(tq, torch, cache, q, sh.alpha, dtype)
            assert np.all(np.isfinite(got))
            if dtype == torch.float32:
                assert_attention_close(got, want, f"static entry vs oracle, shape {sh.name}")
            mx, rel = errors(got, ref.astype(np.float64))
            slack = 0.0 if dtype == torch.float32 else np.abs(ref).max() * 2.0 ** -11
            assert mx <= MAX_ABS_TOL + slack and rel <= REL_L2_TOL + (0 if dtype == torch.float32 else 1e-3), (mx, rel)


def test_paged_cache_and_head_dim_512_through_the_static_entry(gpu, oracle):
    """The static entry serves every cache form the other entry points serve: a paged pool (random page
    assignment) and the 512-wide heads, each against the oracle and the two-call path."""
    tq, torch = gpu
    for sh, S, page_tokens, seed in ((I.Shape("paged", 2, 16, 2, 128, 128 ** -0.5), 700, 64, 41),
                                     (I.Shape("wide", 1, 32, 1, 512, 1.0, sigma_qk=0.2), 300, 0, 42)):
        k, v = I.make_kv(sh, S, seed)
        q = I.make_q(sh, seed)
        if page_tokens:
            max_pages = (S + page_tokens - 1) // page_tokens
            num_pages = sh.B * max_pages + 3
            cache = tq.PagedKVCache(sh.B, sh.H_kv, page_tokens, max_pages, num_pages, sh.d)
            perm = np.random.default_rng(seed).permutation(num_pages)[:sh.B * max_pages].astype(np.int32)
            cache.page_table.copy_(torch.from_numpy(perm.reshape(sh.B, max_pages)))
            cache.blocks.fill_(0xFF)
            S_cap = page_tokens * max_pages
        else:
            S_cap = (S + 15) // 16 * 16
            cache = tq.KVCache(sh.B, sh.H_kv, S_cap, sh.d)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        tq.tq_kv_quantize_append(cache, torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda(), status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        want = oracle.attention(oracle_cache(oracle, sh, k, v, S_cap), q, sh.alpha)
        ref, _, _ = fused_attention(tq, torch, cache, q, sh.alpha)
        got = _static(tq, torch, cache, q, sh.alpha, torch.float32)
        assert_attention_close(got, want, f"static entry vs oracle, {sh.name}")
        assert_attention_close(got, ref.astype(np.float64), f"static entry vs two-call path, {sh.name}")


def test_sizes_beyond_the_fixed_array_are_refused(gpu):
    tq, torch = gpu
    # B * H_q * (d + 2) * 4 bytes for a single split already exceeds the array: nothing may be launched
    B, H_q, H_kv, d = 64, 256, 4, 256
    assert B * H_q * (d + 2) * 4 > tq.TQ_STATIC_SCRATCH_BYTES
    cache = tq.KVCache(B, H_kv, 16, d)
    q = torch.zeros((B, H_q, d), dtype=torch.float16, device="cuda")
    out = torch.full((B, H_q, d), 7.0, dtype=torch.float32, device="cuda")
    with pytest.raises(tq.TqError) as e:
        tq.tq_sdpa_int4_attend_static(cache, q, 1.0, out)
    assert e.value.code == tq.TQ_ERR_WORKSPACE
    torch.cuda.synchronize()
    assert torch.all(out == 7.0)
    assert tq._lib.tq_sdpa_int4_attend_static(None, None, 8, 1.0, None, 1, None, None) == tq.TQ_ERR_NULL
