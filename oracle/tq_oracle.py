"""numpy-facing wrapper of the C oracle (test infrastructure only; see tq_oracle.c).

All fp16 data crosses this boundary as numpy float16 arrays (viewed as uint16 bit patterns on
the C side); attention results are float64.
"""
import ctypes as C

import numpy as np

from . import build as _build

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _lib.tqo_half_to_float.restype = C.c_float
        _lib.tqo_half_to_float.argtypes = [C.c_uint16]
        _lib.tqo_float_to_half.restype = C.c_uint16
        _lib.tqo_float_to_half.argtypes = [C.c_float]
        for name in ("tqo_int4_vector_bytes",):
            getattr(_lib, name).restype = C.c_int64
            getattr(_lib, name).argtypes = [C.c_int64]
        for name in ("tqo_fp16_cache_bytes", "tqo_int4_cache_bytes"):
            getattr(_lib, name).restype = C.c_int64
            getattr(_lib, name).argtypes = [C.c_int64] * 4
        _lib.tqo_quantize_append.restype = C.c_int
        _lib.tqo_num_threads.restype = C.c_int
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


def _i64(v):
    return C.c_int64(int(v))


def num_threads() -> int:
    return int(lib().tqo_num_threads())


def half_to_float(bits: int) -> float:
    return float(lib().tqo_half_to_float(int(bits)))


def float_to_half(f) -> int:
    return int(lib().tqo_float_to_half(C.c_float(float(np.float32(f)))))


def int4_vector_bytes(d):
    return int(lib().tqo_int4_vector_bytes(d))


def fp16_cache_bytes(L, H_kv, S, d):
    return int(lib().tqo_fp16_cache_bytes(L, H_kv, S, d))


def int4_cache_bytes(L, H_kv, S, d):
    return int(lib().tqo_int4_cache_bytes(L, H_kv, S, d))


def pack_nibbles(codes: np.ndarray) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    out = np.empty(codes.shape[:-1] + (codes.shape[-1] // 2,), dtype=np.uint8)
    lib().tqo_pack_nibbles(_p(codes), _i64(codes.size), _p(out))
    return out


def unpack_nibbles(packed: np.ndarray) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    out = np.empty(packed.shape[:-1] + (packed.shape[-1] * 2,), dtype=np.uint8)
    lib().tqo_unpack_nibbles(_p(packed), _i64(out.size), _p(out))
    return out


def quantize_rows(x: np.ndarray):
    """x: [..., d] float16 -> (packed [..., d/2] u8, scale [..., d/32] f16, zero [..., d/32] f16)."""
    x = np.ascontiguousarray(x, dtype=np.float16)
    d = x.shape[-1]
    assert d % 32 == 0
    n = x.size // d
    packed = np.empty(x.shape[:-1] + (d // 2,), dtype=np.uint8)
    scale = np.empty(x.shape[:-1] + (d // 32,), dtype=np.float16)
    zero = np.empty(x.shape[:-1] + (d // 32,), dtype=np.float16)
    lib().tqo_quantize_rows(_p(x), _i64(n), _i64(d), _p(packed), _p(scale), _p(zero))
    return packed, scale, zero


def dequant_rows(packed, scale, zero) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    scale = np.ascontiguousarray(scale, dtype=np.float16)
    zero = np.ascontiguousarray(zero, dtype=np.float16)
    d = packed.shape[-1] * 2
    n = packed.size // (d // 2)
    out = np.empty(packed.shape[:-1] + (d,), dtype=np.float64)
    lib().tqo_dequant_rows(_p(packed), _p(scale), _p(zero), _i64(n), _i64(d), _p(out))
    return out


class Cache:
    """Host-side int4 KV cache in the layout the paper's kernel consumes: packed codes plus
    per-group fp16 scale and zero, [B][H_kv][S_cap][...], and per-sequence lengths."""

    def __init__(self, B, H_kv, S_cap, d):
        self.B, self.H_kv, self.S_cap, self.d = B, H_kv, S_cap, d
        g = d // 32
        self.k_packed = np.zeros((B, H_kv, S_cap, d // 2), np.uint8)
        self.v_packed = np.zeros((B, H_kv, S_cap, d // 2), np.uint8)
        self.k_scale = np.zeros((B, H_kv, S_cap, g), np.float16)
        self.k_zero = np.zeros((B, H_kv, S_cap, g), np.float16)
        self.v_scale = np.zeros((B, H_kv, S_cap, g), np.float16)
        self.v_zero = np.zeros((B, H_kv, S_cap, g), np.float16)
        self.lens = np.zeros((B,), np.int32)

    def arrays(self):
        return (self.k_packed, self.k_scale, self.k_zero, self.v_packed, self.v_scale, self.v_zero)

    def append(self, k_new: np.ndarray, v_new: np.ndarray) -> int:
        """k_new, v_new: [B][H_kv][T][d] float16.  Returns the number of sequences skipped
        because they would overflow S_cap (those are left untouched)."""
        k_new = np.ascontiguousarray(k_new, dtype=np.float16)
        v_new = np.ascontiguousarray(v_new, dtype=np.float16)
        T = k_new.shape[2]
        assert k_new.shape == (self.B, self.H_kv, T, self.d) and v_new.shape == k_new.shape
        f = lib().tqo_quantize_append
        args = (_i64(self.B), _i64(self.H_kv), _i64(self.S_cap), _i64(self.d))
        sk = f(_p(self.k_packed), _p(self.k_scale), _p(self.k_zero), _p(self.lens), *args, _p(k_new), _i64(T),
               C.c_int(0))
        sv = f(_p(self.v_packed), _p(self.v_scale), _p(self.v_zero), _p(self.lens), *args, _p(v_new), _i64(T),
               C.c_int(1))
        assert sk == sv
        return int(sk)

    def _cargs(self):
        return [_p(a) for a in self.arrays()] + [_p(self.lens), _i64(self.B), _i64(self.H_kv), _i64(self.S_cap),
                                                 _i64(self.d)]


def attention(cache: Cache, q: np.ndarray, alpha: float, heads=None) -> np.ndarray:
    """softmax(alpha q K^T) V on the dequantised cache, fp64.  q: [B][H_q][d] float16.
    heads=(h0, h1) restricts the computation to query heads [h0, h1); other rows stay zero."""
    q = np.ascontiguousarray(q, dtype=np.float16)
    B, H_q, d = q.shape
    out = np.zeros((B, H_q, d), np.float64)
    h0, h1 = (0, H_q) if heads is None else heads
    lib().tqo_attention(*cache._cargs(), _p(q), _i64(H_q), C.c_double(alpha), _i64(h0), _i64(h1), _p(out))
    return out


def attention_window(cache: Cache, q: np.ndarray, alpha: float, window: int) -> np.ndarray:
    """Attention over the last `window` tokens of every sequence (window <= 0: all tokens), fp64."""
    q = np.ascontiguousarray(q, dtype=np.float16)
    B, H_q, d = q.shape
    out = np.zeros((B, H_q, d), np.float64)
    lib().tqo_attention_window(*cache._cargs(), _p(q), _i64(H_q), C.c_double(alpha), _i64(window), _p(out))
    return out


def attention_multi(cache: Cache, q: np.ndarray, alpha: float, window: int = 0) -> np.ndarray:
    """Several query tokens per sequence, q [B][S_q][H_q][d]: the S_q newest cached tokens as queries.
    The paper only names the S_q factor (Appendix A); the reading here is causal attention: query token s
    sees the cache as it was when that token was the newest one, i.e. the first
    lens[b] - (S_q - 1 - s) tokens (and of those the last `window`, if a window is set).
    Returns [B][S_q][H_q][d] fp64."""
    q = np.ascontiguousarray(q, dtype=np.float16)
    B, S_q, H_q, d = q.shape
    out = np.zeros((B, S_q, H_q, d), np.float64)
    full = cache.lens.copy()
    try:
        for s in range(S_q):
            cache.lens[:] = np.maximum(full - (S_q - 1 - s), 0)
            out[:, s] = attention_window(cache, q[:, s], alpha, window)
    finally:
        cache.lens[:] = full
    return out


def attention_mixed(cache: Cache, k16, v16, q: np.ndarray, alpha: float) -> np.ndarray:
    """K-versus-V precision ablation (Sec. 5): softmax(alpha q K^T) V in fp64 with K and V each either the
    dequantised cache (argument None) or the given unquantised fp16 values [B][H_kv][>= len][d].
    Returns [B][H_q][d]."""
    q = np.asarray(q, dtype=np.float16).astype(np.float64)
    B, H_q, d = q.shape
    G = H_q // cache.H_kv
    kd = dequant_rows(cache.k_packed, cache.k_scale, cache.k_zero) if k16 is None else None
    vd = dequant_rows(cache.v_packed, cache.v_scale, cache.v_zero) if v16 is None else None
    out = np.zeros((B, H_q, d), np.float64)
    for b in range(B):
        n = int(cache.lens[b])
        if n == 0:
            continue
        for h in range(H_q):
            kv = h // G
            K = (kd[b, kv, :n] if k16 is None else np.asarray(k16[b, kv, :n], dtype=np.float16).astype(np.float64))
            V = (vd[b, kv, :n] if v16 is None else np.asarray(v16[b, kv, :n], dtype=np.float16).astype(np.float64))
            a = alpha * (K @ q[b, h])
            w = np.exp(a - a.max())
            out[b, h] = (w / w.sum()) @ V
    return out


def attention_weights(cache: Cache, q, alpha, b, h) -> np.ndarray:
    q = np.ascontiguousarray(q, dtype=np.float16)
    w = np.zeros((int(cache.lens[b]),), np.float64)
    lib().tqo_attention_weights(*cache._cargs(), _p(q), _i64(q.shape[1]), C.c_double(alpha), _i64(b), _i64(h), _p(w))
    return w


def attention_partials(cache: Cache, q, alpha, bounds: np.ndarray):
    """bounds: [B][C+1] int32 token boundaries.  Returns (o_part [B][H_q][C][d], m_part, l_part)."""
    q = np.ascontiguousarray(q, dtype=np.float16)
    bounds = np.ascontiguousarray(bounds, dtype=np.int32)
    B, H_q, d = q.shape
    Cn = bounds.shape[1] - 1
    o = np.zeros((B, H_q, Cn, d), np.float64)
    m = np.zeros((B, H_q, Cn), np.float64)
    l = np.zeros((B, H_q, Cn), np.float64)
    lib().tqo_attention_partials(*cache._cargs(), _p(q), _i64(H_q), C.c_double(alpha), _i64(Cn), _p(bounds), _p(o),
                                 _p(m), _p(l))
    return o, m, l


def combine(o_part, m_part, l_part) -> np.ndarray:
    o_part = np.ascontiguousarray(o_part, dtype=np.float64)
    m_part = np.ascontiguousarray(m_part, dtype=np.float64)
    l_part = np.ascontiguousarray(l_part, dtype=np.float64)
    B, H_q, Cn, d = o_part.shape
    out = np.zeros((B, H_q, d), np.float64)
    lib().tqo_combine(_p(o_part), _p(m_part), _p(l_part), _i64(B), _i64(H_q), _i64(Cn), _i64(d), _p(out))
    return out
