"""The C-ABI library loads, exports every symbol the header declares, and rejects bad arguments
on the host before touching a GPU (CPU only: no kernel is launched here)."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2604_16957_b200 import build
    return C.CDLL(build.build())


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "tq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tq_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_symbols()
    assert {"tq_kv_quantize_append", "tq_sdpa_int4_decode", "tq_sdpa_int4_combine",
            "tq_sdpa_dequant_then_attend"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    from paper_2604_16957_b200 import tq
    assert sorted(tq.SYMBOLS) == names
    assert {"TQ_STATUS_TIMEOUT", "TQ_STATUS_BAD_PAGE"} <= set(dir(tq)) and tq.TQ_STATUS_TIMEOUT == 8
    assert tq._lib.tq_internal_test_hook(99, 0) == -1   # the test knob is exported but is not in the header
    assert "tq_internal_test_hook" not in names


def test_host_side_helpers(lib):
    from paper_2604_16957_b200 import tq
    assert tq.tq_cache_bytes(1, 8, 131072, 128) * 80 == int(12.5 * 2 ** 30)       # Table 4, 128K row
    assert tq.tq_partials_bytes(1, 64, 128, 37) >= 64 * 37 * 130 * 4
    # split ranges tile [0, len) in order, on multiples of 16 except the end
    for length, Cn in ((0, 3), (1, 4), (257, 5), (131072, 37), (4097, 256)):
        prev = 0
        for c in range(Cn):
            t0, t1 = tq.tq_split_range(length, Cn, c)
            assert t0 == prev and t1 >= t0 and (t0 % 16 == 0)
            prev = t1
        assert prev == length
    # block layout: 2560 bytes per 16 tokens at d = 128; the offset helpers cover a block exactly once
    for d in (64, 128, 256, 512):
        nbytes = tq.TQ_BLOCK_BYTES(d)
        assert nbytes == 16 * 2 * tq.tq_cache_bytes(1, 1, 16, d) // 32 == 16 * (d + d // 4)
        seen = set()
        for which in (0, 1):
            for t in range(16):
                for byte in range(d // 2):
                    seen.add(tq._lib.tq_cache_code_offset(d, which, t, byte))
                for g in range(d // 32):
                    for is_zero in (0, 1):
                        o = tq._lib.tq_cache_meta_offset(d, which, is_zero, g, t)
                        seen.update((o, o + 1))
        assert seen == set(range(nbytes))
    assert tq._lib.tq_cache_code_offset(128, 0, 0, 5) == 5 and tq._lib.tq_cache_code_offset(128, 1, 0, 0) == 1024
    assert tq._lib.tq_cache_code_offset(128, 0, 2, 0) == 2 * 64 + 16   # token 2: chunks XOR 1
    c = tq.tq_auto_splits(1, 8, 64, 128, 131072)
    assert 1 <= c <= 256
    assert tq.tq_auto_splits(1, 8, 64, 128, 100) == 1


def test_split_policy_of_the_step(lib):
    """tq_auto_splits_step on a machine that cannot be asked (no device: 148 SMs, 296 resident slots assumed):
    within [1, TQ_MAX_SPLITS], never splits shorter than the stated minimum, one split up to 1K tokens, and an
    eighth of the slots left free where (sequences x KV heads) is at most 1/32 of them."""
    from paper_2604_16957_b200 import tq
    slots = 296
    for B, H_kv, H_q in ((1, 8, 64), (1, 4, 32), (1, 1, 8), (1, 2, 16), (1, 16, 32), (2, 8, 64), (16, 8, 64), (64, 8, 64)):
        base = B * H_kv * ((H_q // H_kv + 7) // 8)
        for n in (1, 100, 1024, 1025, 4096, 8192, 32768, 131072, 1 << 20):
            c = tq.tq_auto_splits_step(B, H_kv, H_q, 128, n)
            plain = tq.tq_auto_splits(B, H_kv, H_q, 128, n)
            assert 1 <= c <= 256 and c <= max(1, plain)
            if n <= 1024:
                assert c == 1
            else:
                assert c <= max(1, n // 512)
            if 32 * base <= slots and c > 1:
                assert c * base <= slots - max(base, slots // 8)
    assert tq.tq_auto_splits_step(1, 8, 64, 128, 131072) == 32 and tq.tq_auto_splits(1, 8, 64, 128, 131072) == 37
    assert tq.tq_auto_splits_step(1, 16, 32, 256, 32768) == 18       # 16 KV heads: no spare slots
    assert tq.tq_auto_splits_step(1, 0, 8, 128, 4096) == 1           # nonsense shapes give 1, not a crash


def test_argument_validation_without_gpu(lib):
    from paper_2604_16957_b200 import tq
    lib.tq_result_string.restype = C.c_char_p
    assert lib.tq_result_string(0) == b"ok"
    assert tq._lib.tq_kv_quantize_append(None, None, None, 1, None, None) == tq.TQ_ERR_NULL
    fake = 0x1000  # never dereferenced: validation fails first
    cs = tq.tq_kv_cache(fake, fake, 1, 1, 64, 100)   # d = 100
    assert tq._lib.tq_kv_quantize_append(C.byref(cs), fake, fake, 1, None, None) == tq.TQ_ERR_SHAPE
    cs = tq.tq_kv_cache(fake, fake, 1, 1, 60, 128)   # S_cap % 16 != 0
    assert tq._lib.tq_sdpa_int4_decode(C.byref(cs), fake, 8, 1.0, 1, fake, fake, fake, None, None) == tq.TQ_ERR_SHAPE
    cs = tq.tq_kv_cache(fake + 8, fake, 1, 1, 64, 128)
    assert tq._lib.tq_kv_quantize_append(C.byref(cs), fake, fake, 1, None, None) == tq.TQ_ERR_ALIGN
    cs = tq.tq_kv_cache(fake, fake, 1, 2, 64, 128)
    assert tq._lib.tq_sdpa_int4_decode(C.byref(cs), fake, 7, 1.0, 1, fake, fake, fake, None, None) == tq.TQ_ERR_SHAPE
    assert tq._lib.tq_sdpa_int4_decode(C.byref(cs), fake, 8, 1.0, 300, fake, fake, fake, None, None) == tq.TQ_ERR_SHAPE
    assert tq._lib.tq_sdpa_int4_decode(C.byref(cs), None, 8, 1.0, 1, fake, fake, fake, None, None) == tq.TQ_ERR_NULL
    assert tq._lib.tq_kv_quantize_append(C.byref(cs), fake, fake, 0, None, None) == tq.TQ_ERR_SHAPE
    assert tq._lib.tq_sdpa_int4_combine(fake, fake, fake, 1, 8, 100, 4, fake, 1, None) == tq.TQ_ERR_SHAPE
    assert tq._lib.tq_sdpa_int4_combine(fake, fake, fake, 1, 8, 128, 0, fake, 1, None) == tq.TQ_ERR_SHAPE
    need = tq.tq_dequant_workspace_bytes(1, 2, 8, 64, 128, 1)
    assert need >= 2 * 2 * 64 * 128 * 4
    assert tq._lib.tq_sdpa_dequant_then_attend(C.byref(cs), fake, 8, 1.0, fake, need - 1, 1, fake, 1, None,
                                               None) == tq.TQ_ERR_WORKSPACE
    # the secondary entry points validate the same way
    assert tq._lib.tq_sdpa_int4_decode_window(C.byref(cs), fake, 8, 1.0, -1, 1, fake, fake, fake, None, None) == tq.TQ_ERR_SHAPE
    assert tq._lib.tq_sdpa_int4_decode_multi(C.byref(cs), fake, 8, 0, 1.0, 0, 1, fake, fake, fake, None, None) == tq.TQ_ERR_SHAPE
    assert tq._lib.tq_sdpa_int4_decode_multi(C.byref(cs), fake, 8, 65, 1.0, 0, 1, fake, fake, fake, None, None) == tq.TQ_ERR_SHAPE
    assert tq._lib.tq_sdpa_mixed_precision_attend(C.byref(cs), fake + 2, None, fake, 8, 1.0, 1, fake, fake, fake, None,
                                                  None) == tq.TQ_ERR_ALIGN
    assert tq._lib.tq_sdpa_int4_attend_static(None, fake, 8, 1.0, fake, 1, None, None) == tq.TQ_ERR_NULL
    # ... including the entry point with the built-in scratch: same shape, alignment and grid checks
    assert tq._lib.tq_sdpa_int4_attend_static(C.byref(cs), fake, 7, 1.0, fake, 1, None, None) == tq.TQ_ERR_SHAPE
    assert tq._lib.tq_sdpa_int4_attend_static(C.byref(cs), fake, 8, 1.0, None, 1, None, None) == tq.TQ_ERR_NULL
    assert tq._lib.tq_sdpa_int4_attend_static(C.byref(cs), fake + 4, 8, 1.0, fake, 1, None, None) == tq.TQ_ERR_ALIGN
    assert tq._lib.tq_sdpa_int4_attend_static(C.byref(cs), fake, 8, 1.0, fake, 1, fake + 2, None) == tq.TQ_ERR_ALIGN
    for bad in (dict(d=100), dict(S_cap=60), dict(H_kv=5000), dict(B=70000), dict(blocks=fake + 8)):
        bs = tq.tq_kv_cache(**{**dict(blocks=fake, seq_lens=fake, B=1, H_kv=2, S_cap=64, d=128), **bad})
        r = tq._lib.tq_sdpa_int4_attend_static(C.byref(bs), fake, 2 * bs.H_kv, 1.0, fake, 1, None, None)
        assert r == (tq.TQ_ERR_ALIGN if "blocks" in bad else tq.TQ_ERR_SHAPE), bad
    big = tq.tq_kv_cache(fake, fake, 1, 4096, 64, 128)
    # 4096 KV heads x 8 head tiles fit the grid, but the partials of one split exceed the built-in scratch;
    # with 4 query tokens the 32 head tiles per KV head exceed the grid's y limit
    assert tq._lib.tq_sdpa_int4_attend_static(C.byref(big), fake, 4096 * 64, 1.0, fake, 1, None, None) == tq.TQ_ERR_WORKSPACE
    assert tq._lib.tq_sdpa_int4_decode_multi(C.byref(big), fake, 4096 * 64, 4, 1.0, 0, 1, fake, fake, fake, None,
                                             None) == tq.TQ_ERR_SHAPE
    # paged caches: page size a power of two >= 16, capacity = pages * page size, table aligned
    ok_paged = dict(blocks=fake, seq_lens=fake, B=1, H_kv=2, S_cap=128, d=128, page_table=fake, page_tokens=32,
                    max_pages=4, num_pages=9)
    for bad in (dict(page_tokens=48), dict(page_tokens=8), dict(max_pages=3), dict(num_pages=0), dict(S_cap=96)):
        cs = tq.tq_kv_cache(**{**ok_paged, **bad})
        assert tq._lib.tq_sdpa_int4_decode(C.byref(cs), fake, 8, 1.0, 1, fake, fake, fake, None, None) == tq.TQ_ERR_SHAPE, bad
        # a page size below 16 used to reach a host-side division by zero through this entry point
        assert tq._lib.tq_sdpa_int4_attend_static(C.byref(cs), fake, 8, 1.0, fake, 1, None, None) == tq.TQ_ERR_SHAPE, bad
    cs = tq.tq_kv_cache(**{**ok_paged, "page_table": fake + 2})
    assert tq._lib.tq_kv_quantize_append(C.byref(cs), fake, fake, 1, None, None) == tq.TQ_ERR_ALIGN
    assert tq._lib.tq_sdpa_int4_attend_static(C.byref(cs), fake, 8, 1.0, fake, 1, None, None) == tq.TQ_ERR_ALIGN
    # the one-launch step and its per-sequence form: same checks, plus their own arguments
    cs = tq.tq_kv_cache(fake, fake, 1, 2, 64, 128)
    wsb = tq._lib.tq_step_workspace_bytes(1, 2, 8, 128, 2)
    step, ragged = tq._lib.tq_sdpa_int4_step, tq._lib.tq_sdpa_int4_step_ragged
    assert step(C.byref(cs), fake, None, fake, 8, 1.0, 2, 0, fake, wsb, fake, 1, None, None) == tq.TQ_ERR_NULL
    assert step(C.byref(cs), None, None, fake, 8, 1.0, 2, 65, fake, wsb, fake, 1, None, None) == tq.TQ_ERR_SHAPE
    assert step(C.byref(cs), None, None, fake, 24, 1.0, 2, 0, fake, wsb, fake, 1, None, None) == tq.TQ_ERR_SHAPE   # 12 heads per KV head
    assert step(C.byref(cs), None, None, fake, 8, 1.0, 2, 0, fake, wsb - 1, fake, 1, None, None) == tq.TQ_ERR_WORKSPACE
    assert ragged(C.byref(cs), None, None, fake, 8, 1.0, 2, None, fake, wsb, fake, 1, None, None) == tq.TQ_ERR_NULL
    assert ragged(C.byref(cs), None, None, fake, 8, 1.0, 2, fake + 2, fake, wsb, fake, 1, None, None) == tq.TQ_ERR_ALIGN
    assert ragged(C.byref(cs), None, None, fake, 8, 1.0, 300, fake, fake, wsb, fake, 1, None, None) == tq.TQ_ERR_SHAPE
    # split ranges under a window tile exactly the window
    for length, window, Cn in ((3000, 1024, 5), (1029, 1024, 3), (7, 1024, 2), (100, 1, 4), (0, 5, 2)):
        prev = max(0, length - window)
        for c in range(Cn):
            t0, t1 = tq.tq_split_range_window(length, window, Cn, c)
            assert t0 == prev and t1 >= t0
            prev = t1
        assert prev == length
    # split policy: one wave for few heads, several for a batch, never shorter than the stated minimum
    assert tq.tq_auto_splits(16, 8, 64, 128, 65536) >= 4
    assert tq.tq_auto_splits(16, 8, 64, 128, 2048) == 1
