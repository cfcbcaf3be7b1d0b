"""ctypes binding of libtq.so -- same names as include/tq.h, argument marshalling only.

Tensors are torch CUDA tensors (torch supplies device memory and streams, nothing else); every
function forwards data pointers and sizes to the C entry point and raises TqError on a non-zero
result.  There is no CPU fallback: importing this module fails if the library has not been
built (python -m paper_2604_16957_b200.build), and calls fail without a CUDA device.
"""
import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# TQ_LIBRARY names another build of the same library (the timing probes of build.py); never a fallback
LIB_PATH = os.environ.get("TQ_LIBRARY") or os.path.join(_HERE, "libtq.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2604_16957_b200.build`")

_lib = C.CDLL(LIB_PATH)

TQ_OK, TQ_ERR_NULL, TQ_ERR_SHAPE, TQ_ERR_ALIGN, TQ_ERR_WORKSPACE, TQ_ERR_CUDA = range(6)
TQ_STATUS_CACHE_FULL, TQ_STATUS_EMPTY_SEQ, TQ_STATUS_BAD_LEN, TQ_STATUS_TIMEOUT, TQ_STATUS_BAD_PAGE = 1, 2, 4, 8, 16
TQ_GROUP, TQ_SPLIT_QUANTUM, TQ_MAX_SPLITS = 32, 16, 256
TQ_STATIC_SCRATCH_BYTES = 8 << 20

# every symbol include/tq.h declares
SYMBOLS = ("tq_kv_quantize_append", "tq_auto_splits", "tq_split_range", "tq_sdpa_int4_decode", "tq_sdpa_int4_combine",
           "tq_partials_bytes", "tq_sdpa_dequant_then_attend", "tq_dequant_workspace_bytes", "tq_cache_bytes",
           "tq_result_string", "tq_last_cuda_error", "tq_version", "tq_sdpa_int4_attend_static",
           "tq_cache_code_offset", "tq_cache_meta_offset", "tq_sdpa_int4_decode_window", "tq_split_range_window",
           "tq_sdpa_int4_decode_multi", "tq_sdpa_mixed_precision_attend", "tq_sdpa_int4_decode_overlapped",
           "tq_split_range_stable", "tq_sdpa_int4_step", "tq_sdpa_int4_step_ragged", "tq_sdpa_int4_step_window", "tq_step_workspace_bytes", "tq_step_counter_bytes", "tq_auto_splits_step")


class tq_kv_cache(C.Structure):
    _fields_ = [("blocks", C.c_void_p), ("seq_lens", C.c_void_p), ("B", C.c_int32), ("H_kv", C.c_int32),
                ("S_cap", C.c_int32), ("d", C.c_int32), ("page_table", C.c_void_p), ("page_tokens", C.c_int32),
                ("max_pages", C.c_int32), ("num_pages", C.c_int32)]


def TQ_BLOCK_BYTES(d):
    return 16 * (d + d // 4)


_vp, _i32, _f32, _sz = C.c_void_p, C.c_int32, C.c_float, C.c_size_t
_cache_p = C.POINTER(tq_kv_cache)
_lib.tq_kv_quantize_append.argtypes = [_cache_p, _vp, _vp, _i32, _vp, _vp]
_lib.tq_kv_quantize_append.restype = C.c_int
_lib.tq_auto_splits.argtypes = [_i32] * 5
_lib.tq_auto_splits.restype = _i32
_lib.tq_auto_splits_step.argtypes = [_i32] * 5
_lib.tq_auto_splits_step.restype = _i32
_lib.tq_split_range.argtypes = [_i32, _i32, _i32, C.POINTER(_i32), C.POINTER(_i32)]
_lib.tq_split_range.restype = None
_lib.tq_sdpa_int4_decode.argtypes = [_cache_p, _vp, _i32, _f32, _i32, _vp, _vp, _vp, _vp, _vp]
_lib.tq_sdpa_int4_decode.restype = C.c_int
_lib.tq_sdpa_int4_decode_overlapped.argtypes = [_cache_p, _vp, _i32, _f32, _i32, _i32, _vp, _vp, _vp, _vp, _vp]
_lib.tq_sdpa_int4_decode_overlapped.restype = C.c_int
_lib.tq_split_range_stable.argtypes = [_i32, _i32, _i32, _i32, C.POINTER(_i32), C.POINTER(_i32)]
_lib.tq_split_range_stable.restype = None
_lib.tq_sdpa_int4_step.argtypes = [_cache_p, _vp, _vp, _vp, _i32, _f32, _i32, _i32, _vp, _sz, _vp, _i32, _vp, _vp]
_lib.tq_sdpa_int4_step.restype = C.c_int
_lib.tq_sdpa_int4_step_ragged.argtypes = [_cache_p, _vp, _vp, _vp, _i32, _f32, _i32, _vp, _vp, _sz, _vp, _i32, _vp, _vp]
_lib.tq_sdpa_int4_step_ragged.restype = C.c_int
_lib.tq_sdpa_int4_step_window.argtypes = [_cache_p, _vp, _vp, _vp, _i32, _f32, _i32, _i32, _i32, _vp, _sz, _vp, _i32, _vp, _vp]
_lib.tq_sdpa_int4_step_window.restype = C.c_int
_lib.tq_step_workspace_bytes.argtypes = [_i32] * 5
_lib.tq_step_workspace_bytes.restype = _sz
_lib.tq_step_counter_bytes.argtypes = [_i32] * 2
_lib.tq_step_counter_bytes.restype = _sz
_lib.tq_sdpa_int4_decode_window.argtypes = [_cache_p, _vp, _i32, _f32, _i32, _i32, _vp, _vp, _vp, _vp, _vp]
_lib.tq_sdpa_int4_decode_window.restype = C.c_int
_lib.tq_sdpa_int4_decode_multi.argtypes = [_cache_p, _vp, _i32, _i32, _f32, _i32, _i32, _vp, _vp, _vp, _vp, _vp]
_lib.tq_sdpa_int4_decode_multi.restype = C.c_int
_lib.tq_sdpa_mixed_precision_attend.argtypes = [_cache_p, _vp, _vp, _vp, _i32, _f32, _i32, _vp, _vp, _vp, _vp, _vp]
_lib.tq_sdpa_mixed_precision_attend.restype = C.c_int
_lib.tq_split_range_window.argtypes = [_i32, _i32, _i32, _i32, C.POINTER(_i32), C.POINTER(_i32)]
_lib.tq_split_range_window.restype = None
_lib.tq_sdpa_int4_combine.argtypes = [_vp, _vp, _vp, _i32, _i32, _i32, _i32, _vp, _i32, _vp]
_lib.tq_sdpa_int4_combine.restype = C.c_int
_lib.tq_partials_bytes.argtypes = [_i32] * 4
_lib.tq_partials_bytes.restype = _sz
_lib.tq_sdpa_dequant_then_attend.argtypes = [_cache_p, _vp, _i32, _f32, _vp, _sz, _i32, _vp, _i32, _vp, _vp]
_lib.tq_sdpa_dequant_then_attend.restype = C.c_int
_lib.tq_dequant_workspace_bytes.argtypes = [_i32] * 6
_lib.tq_dequant_workspace_bytes.restype = _sz
_lib.tq_sdpa_int4_attend_static.argtypes = [_cache_p, _vp, _i32, _f32, _vp, _i32, _vp, _vp]
_lib.tq_sdpa_int4_attend_static.restype = C.c_int
_lib.tq_cache_bytes.argtypes = [_i32] * 4
_lib.tq_cache_bytes.restype = _sz
_lib.tq_cache_code_offset.argtypes = [_i32] * 4
_lib.tq_cache_code_offset.restype = _sz
_lib.tq_cache_meta_offset.argtypes = [_i32] * 5
_lib.tq_cache_meta_offset.restype = _sz
_lib.tq_result_string.argtypes = [C.c_int]
_lib.tq_result_string.restype = C.c_char_p
_lib.tq_last_cuda_error.restype = C.c_int
_lib.tq_version.restype = C.c_char_p
# knob of the library's own tests (exported by the shared object, not declared in tq.h, not part of the ABI)
_lib.tq_internal_test_hook.argtypes = [C.c_int, C.c_int]
_lib.tq_internal_test_hook.restype = C.c_int
HOOK_DECODE_IMPL, HOOK_SPIN_LIMIT, HOOK_FAULT_BLOCK = 0, 1, 2


def _test_hook(key, value):
    """Set a test knob of the library (see TestHooks in csrc/tq_internal.cuh); used only by tests/."""
    if _lib.tq_internal_test_hook(int(key), int(value)) != 0:
        raise ValueError(f"unknown test hook {key}")


def _division_self_check():
    """Mismatches between the quantiser's reciprocal-based divisions and true division over every quotient it can
    form (runs a kernel on the current device; -1 on a CUDA error); used only by tests/."""
    return int(_lib.tq_internal_test_hook(3, 0))


class TqError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        msg = _lib.tq_result_string(code).decode()
        if code == TQ_ERR_CUDA:
            msg += f" (cudaError {_lib.tq_last_cuda_error()})"
        super().__init__(f"{where}: {msg} [{code}]")


def _check(code, where):
    if code != TQ_OK:
        raise TqError(code, where)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


class KVCache:
    """Device buffer of one layer's int4 KV cache (16-token blocks, see tq.h) plus the C struct that
    describes it."""

    def __init__(self, B, H_kv, S_cap, d, device="cuda"):
        assert S_cap % 16 == 0 and d in (64, 128, 256, 512)
        self.B, self.H_kv, self.S_cap, self.d = B, H_kv, S_cap, d
        self.blocks = torch.zeros((B, H_kv, S_cap // 16, TQ_BLOCK_BYTES(d)), dtype=torch.uint8, device=device)
        self.seq_lens = torch.zeros((B,), dtype=torch.int32, device=device)

    def struct(self):
        return tq_kv_cache(self.blocks.data_ptr(), self.seq_lens.data_ptr(), self.B, self.H_kv, self.S_cap, self.d,
                           None, 0, 0, 0)

    def arrays_token_major(self):
        """Decode the blocks into plain token-major arrays (copies, for inspection and tests):
        (k_packed [B][H_kv][S_cap][d/2] u8, k_scale, k_zero [B][H_kv][S_cap][d/32] f16, v_packed, v_scale, v_zero)."""
        B, H, S, d = self.B, self.H_kv, self.S_cap, self.d
        ng, rowb, nb = d // 32, d // 2, S // 16
        pk, sz = 16 * rowb, ng * 32
        shift = {2: 2, 4: 1, 8: 0, 16: 0}[ng]
        t = torch.arange(16, device=self.blocks.device)
        g = torch.arange(ng, device=self.blocks.device)
        pos = g[None, :] ^ ((t[:, None] >> shift) & (ng - 1))          # [16][ng]: chunk position of group g of token t
        idx = pos[None, None, None, :, :, None].expand(B, H, nb, 16, ng, 16)
        out = []
        for which in (0, 1):
            codes = self.blocks[..., which * pk:(which + 1) * pk].reshape(B, H, nb, 16, ng, 16)
            out.append(torch.gather(codes, 4, idx).reshape(B, H, S, rowb))
            for is_zero in (0, 1):
                a = 2 * which + is_zero
                m = self.blocks[..., 16 * d + a * sz:16 * d + (a + 1) * sz].contiguous().view(torch.float16)
                out.append(m.reshape(B, H, nb, ng, 16).permute(0, 1, 2, 4, 3).reshape(B, H, S, ng))
        return tuple(out)


class PagedKVCache:
    """The same cache served from a pool of pages: `blocks` is [num_pages][H_kv][page_tokens/16][block bytes],
    `page_table` [B][max_pages] int32 names the pool page of every page_tokens-token stretch of a sequence."""

    def __init__(self, B, H_kv, page_tokens, max_pages, num_pages, d, device="cuda"):
        assert page_tokens >= 16 and page_tokens & (page_tokens - 1) == 0 and d in (64, 128, 256, 512)
        self.B, self.H_kv, self.d = B, H_kv, d
        self.page_tokens, self.max_pages, self.num_pages = page_tokens, max_pages, num_pages
        self.S_cap = page_tokens * max_pages
        self.blocks = torch.zeros((num_pages, H_kv, page_tokens // 16, TQ_BLOCK_BYTES(d)), dtype=torch.uint8, device=device)
        self.page_table = torch.zeros((B, max_pages), dtype=torch.int32, device=device)
        self.seq_lens = torch.zeros((B,), dtype=torch.int32, device=device)

    def struct(self):
        return tq_kv_cache(self.blocks.data_ptr(), self.seq_lens.data_ptr(), self.B, self.H_kv, self.S_cap, self.d,
                           self.page_table.data_ptr(), self.page_tokens, self.max_pages, self.num_pages)

    def contiguous(self):
        """A KVCache holding the same logical contents (a copy gathered through the page table)."""
        out = KVCache(self.B, self.H_kv, self.S_cap, self.d, device=self.blocks.device)
        pages = self.blocks[self.page_table.long().clamp(0, self.num_pages - 1)]  # [B][max_pages][H_kv][bpp][bytes]
        out.blocks.copy_(pages.permute(0, 2, 1, 3, 4).reshape(out.blocks.shape))
        out.seq_lens.copy_(self.seq_lens)
        return out

    def arrays_token_major(self):
        return self.contiguous().arrays_token_major()


def _cs(cache):
    return cache if isinstance(cache, tq_kv_cache) else cache.struct()


def tq_kv_quantize_append(cache, k_new, v_new, status=None, stream=None):
    """k_new, v_new: [B][H_kv][T][d] float16 CUDA tensors (contiguous)."""
    assert k_new.is_contiguous() and v_new.is_contiguous() and k_new.dtype == torch.float16 == v_new.dtype
    assert k_new.shape == v_new.shape and k_new.dim() == 4
    cs = _cs(cache)
    _check(_lib.tq_kv_quantize_append(C.byref(cs), _ptr(k_new), _ptr(v_new), k_new.shape[2], _ptr(status),
                                      _stream(stream)), "tq_kv_quantize_append")


def tq_auto_splits(B, H_kv, H_q, d, max_seq_len):
    return int(_lib.tq_auto_splits(B, H_kv, H_q, d, max_seq_len))


def tq_auto_splits_step(B, H_kv, H_q, d, max_seq_len):
    return int(_lib.tq_auto_splits_step(B, H_kv, H_q, d, max_seq_len))


def tq_split_range(length, C_, c):
    t0, t1 = _i32(), _i32()
    _lib.tq_split_range(length, C_, c, C.byref(t0), C.byref(t1))
    return t0.value, t1.value


def tq_partials_bytes(B, H_q, d, num_splits):
    return int(_lib.tq_partials_bytes(B, H_q, d, num_splits))


def tq_dequant_workspace_bytes(B, H_kv, H_q, S_cap, d, ws_is_fp32):
    return int(_lib.tq_dequant_workspace_bytes(B, H_kv, H_q, S_cap, d, int(ws_is_fp32)))


def tq_cache_bytes(B, H_kv, S_cap, d):
    return int(_lib.tq_cache_bytes(B, H_kv, S_cap, d))


def tq_version():
    return _lib.tq_version().decode()


def tq_sdpa_int4_decode(cache, q, attn_scale, num_splits, o_part, m_part, l_part, status=None, stream=None):
    """q: [B][H_q][d] float16; o_part [B][H_q][C][d], m_part / l_part [B][H_q][C] float32."""
    assert q.is_contiguous() and q.dtype == torch.float16 and q.dim() == 3
    cs = _cs(cache)
    _check(_lib.tq_sdpa_int4_decode(C.byref(cs), _ptr(q), q.shape[1], float(attn_scale), int(num_splits), _ptr(o_part),
                                    _ptr(m_part), _ptr(l_part), _ptr(status), _stream(stream)), "tq_sdpa_int4_decode")


def tq_sdpa_int4_decode_overlapped(cache, q, attn_scale, num_splits, stable_tokens, o_part, m_part, l_part, status=None,
                                   stream=None):
    """Phase 1 that does not wait for the preceding kernel before attending the first stable_tokens tokens."""
    cs = _cs(cache)
    _check(_lib.tq_sdpa_int4_decode_overlapped(C.byref(cs), _ptr(q), q.shape[1], float(attn_scale), int(num_splits),
                                               int(stable_tokens), _ptr(o_part), _ptr(m_part), _ptr(l_part),
                                               _ptr(status), _stream(stream)), "tq_sdpa_int4_decode_overlapped")


def alloc_step_workspace(B, H_kv, H_q, d, num_splits, device="cuda"):
    """Zeroed workspace of tq_sdpa_int4_step (counters, then partials) as a uint8 tensor."""
    return torch.zeros(int(_lib.tq_step_workspace_bytes(B, H_kv, H_q, d, num_splits)), dtype=torch.uint8, device=device)


def tq_sdpa_int4_step(cache, k_new, v_new, q, attn_scale, num_splits, stable_tokens, workspace, out, status=None,
                      stream=None):
    """append (k_new, v_new: [B][H_kv][1][d] fp16 or None) + fused int4 attention + split reduction, one launch."""
    assert q.is_contiguous() and q.dtype == torch.float16 and q.dim() == 3
    assert out.is_contiguous() and out.shape == q.shape and out.dtype in (torch.float16, torch.float32)
    for t in (k_new, v_new):
        assert t is None or (t.is_contiguous() and t.dtype == torch.float16 and t.shape == (cache.B, cache.H_kv, 1, cache.d))
    cs = _cs(cache)
    if isinstance(stable_tokens, torch.Tensor):  # one stable part per sequence: a device int32 [B]
        assert stable_tokens.is_cuda and stable_tokens.dtype == torch.int32 and stable_tokens.shape == (cache.B,)
        _check(_lib.tq_sdpa_int4_step_ragged(C.byref(cs), _ptr(k_new), _ptr(v_new), _ptr(q), q.shape[1], float(attn_scale),
                                             int(num_splits), _ptr(stable_tokens), _ptr(workspace), workspace.numel(),
                                             _ptr(out), int(out.dtype == torch.float32), _ptr(status), _stream(stream)),
               "tq_sdpa_int4_step_ragged")
        return
    _check(_lib.tq_sdpa_int4_step(C.byref(cs), _ptr(k_new), _ptr(v_new), _ptr(q), q.shape[1], float(attn_scale),
                                  int(num_splits), int(stable_tokens), _ptr(workspace), workspace.numel(), _ptr(out),
                                  int(out.dtype == torch.float32), _ptr(status), _stream(stream)), "tq_sdpa_int4_step")


def tq_sdpa_int4_step_window(cache, k_new, v_new, q, attn_scale, window, num_splits, stable_tokens, workspace, out,
                             status=None, stream=None):
    """append + attention over the last `window` tokens + split reduction, one launch (contiguous caches)."""
    assert q.is_contiguous() and q.dtype == torch.float16 and q.dim() == 3
    assert out.is_contiguous() and out.shape == q.shape and out.dtype in (torch.float16, torch.float32)
    for t in (k_new, v_new):
        assert t is None or (t.is_contiguous() and t.dtype == torch.float16 and t.shape == (cache.B, cache.H_kv, 1, cache.d))
    cs = _cs(cache)
    _check(_lib.tq_sdpa_int4_step_window(C.byref(cs), _ptr(k_new), _ptr(v_new), _ptr(q), q.shape[1], float(attn_scale),
                                         int(window), int(num_splits), int(stable_tokens), _ptr(workspace), workspace.numel(), _ptr(out),
                                         int(out.dtype == torch.float32), _ptr(status), _stream(stream)),
           "tq_sdpa_int4_step_window")


def tq_split_range_stable(length, stable_tokens, C_, c):
    t0, t1 = _i32(), _i32()
    _lib.tq_split_range_stable(length, stable_tokens, C_, c, C.byref(t0), C.byref(t1))
    return t0.value, t1.value


def tq_sdpa_int4_decode_window(cache, q, attn_scale, window, num_splits, o_part, m_part, l_part, status=None,
                               stream=None):
    """Phase 1 over the last `window` tokens of every sequence (0 = no window)."""
    assert q.is_contiguous() and q.dtype == torch.float16 and q.dim() == 3
    cs = _cs(cache)
    _check(_lib.tq_sdpa_int4_decode_window(C.byref(cs), _ptr(q), q.shape[1], float(attn_scale), int(window),
                                           int(num_splits), _ptr(o_part), _ptr(m_part), _ptr(l_part), _ptr(status),
                                           _stream(stream)), "tq_sdpa_int4_decode_window")


def tq_sdpa_int4_decode_multi(cache, q, attn_scale, window, num_splits, o_part, m_part, l_part, status=None,
                              stream=None):
    """Phase 1 for q [B][S_q][H_q][d]: the S_q newest cached tokens as queries, causal among themselves.
    Partials are [B][S_q * H_q][C][...]."""
    assert q.is_contiguous() and q.dtype == torch.float16 and q.dim() == 4
    cs = _cs(cache)
    _check(_lib.tq_sdpa_int4_decode_multi(C.byref(cs), _ptr(q), q.shape[2], q.shape[1], float(attn_scale),
                                          int(window), int(num_splits), _ptr(o_part), _ptr(m_part), _ptr(l_part),
                                          _ptr(status), _stream(stream)), "tq_sdpa_int4_decode_multi")


def tq_sdpa_mixed_precision_attend(cache, k_fp16, v_fp16, q, attn_scale, num_splits, o_part, m_part, l_part,
                                   status=None, stream=None):
    """Phase 1 with K and / or V from unquantised fp16 [B][H_kv][S_cap][d] (None: from the int4 cache)."""
    assert q.is_contiguous() and q.dtype == torch.float16 and q.dim() == 3
    for t in (k_fp16, v_fp16):
        assert t is None or (t.is_contiguous() and t.dtype == torch.float16 and
                             tuple(t.shape) == (cache.B, cache.H_kv, cache.S_cap, cache.d))
    cs = _cs(cache)
    _check(_lib.tq_sdpa_mixed_precision_attend(C.byref(cs), _ptr(k_fp16), _ptr(v_fp16), _ptr(q), q.shape[1],
                                               float(attn_scale), int(num_splits), _ptr(o_part), _ptr(m_part),
                                               _ptr(l_part), _ptr(status), _stream(stream)),
           "tq_sdpa_mixed_precision_attend")


def tq_split_range_window(length, window, C_, c):
    t0, t1 = _i32(), _i32()
    _lib.tq_split_range_window(length, window, C_, c, C.byref(t0), C.byref(t1))
    return t0.value, t1.value


def tq_sdpa_int4_combine(o_part, m_part, l_part, out, stream=None):
    B, H_q, Cn, d = o_part.shape
    assert out.shape == (B, H_q, d) and out.dtype in (torch.float16, torch.float32) and out.is_contiguous()
    _check(_lib.tq_sdpa_int4_combine(_ptr(o_part), _ptr(m_part), _ptr(l_part), B, H_q, d, Cn, _ptr(out),
                                     int(out.dtype == torch.float32), _stream(stream)), "tq_sdpa_int4_combine")


def tq_sdpa_dequant_then_attend(cache, q, attn_scale, workspace, ws_is_fp32, out, status=None, stream=None):
    assert q.is_contiguous() and q.dtype == torch.float16 and workspace.dtype == torch.uint8
    cs = _cs(cache)
    _check(_lib.tq_sdpa_dequant_then_attend(C.byref(cs), _ptr(q), q.shape[1], float(attn_scale), _ptr(workspace),
                                            workspace.numel(), int(ws_is_fp32), _ptr(out),
                                            int(out.dtype == torch.float32), _ptr(status), _stream(stream)),
           "tq_sdpa_dequant_then_attend")


def tq_sdpa_int4_attend_static(cache, q, attn_scale, out, status=None, stream=None):
    """Decode + combine in one call for callers that cannot allocate: the split partials live in a
    fixed array inside the library instead of caller memory.  q: [B][H_q][d] float16; out: [B][H_q][d]
    float16 or float32.  Raises TqError(TQ_ERR_WORKSPACE) when B * H_q * d is too large for that array."""
    assert q.is_contiguous() and q.dtype == torch.float16 and q.dim() == 3
    assert out.shape == q.shape and out.dtype in (torch.float16, torch.float32) and out.is_contiguous()
    cs = _cs(cache)
    _check(_lib.tq_sdpa_int4_attend_static(C.byref(cs), _ptr(q), q.shape[1], float(attn_scale), _ptr(out),
                                           int(out.dtype == torch.float32), _ptr(status), _stream(stream)),
           "tq_sdpa_int4_attend_static")


def alloc_partials(B, H_q, d, num_splits, device="cuda"):
    o = torch.empty((B, H_q, num_splits, d), dtype=torch.float32, device=device)
    m = torch.empty((B, H_q, num_splits), dtype=torch.float32, device=device)
    l = torch.empty((B, H_q, num_splits), dtype=torch.float32, device=device)
    return o, m, l
