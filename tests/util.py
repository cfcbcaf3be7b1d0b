"""Shared helpers of the GPU parity tests: build the same cache on the host (oracle quantiser)
and on the device (CUDA quantiser) from one set of seeded fp16 inputs, and compare results."""
import numpy as np

MAX_ABS_TOL = 2e-3   # attention output against the fp64 oracle on the same dequantised values
REL_L2_TOL = 1e-3


def errors(got: np.ndarray, ref: np.ndarray):
    got = got.astype(np.float64)
    diff = np.abs(got - ref)
    rel = np.sqrt((diff ** 2).sum() / max((ref ** 2).sum(), 1e-300))
    return float(diff.max()), float(rel)


def assert_attention_close(got, ref, what=""):
    assert np.all(np.isfinite(got)), f"{what}: non-finite output"
    mx, rel = errors(got, ref)
    assert mx <= MAX_ABS_TOL and rel <= REL_L2_TOL, f"{what}: max-abs {mx:.3e} rel-L2 {rel:.3e}"
    return mx, rel


def oracle_cache(oracle, shape, k, v, S_cap, lens=None):
    """Quantise k, v ([B][H_kv][S][d] fp16) with the oracle into a host cache of capacity S_cap."""
    cache = oracle.Cache(shape.B, shape.H_kv, S_cap, shape.d)
    cache.append(k, v)
    if lens is not None:
        cache.lens[:] = lens
    return cache


def device_cache(tq, torch, shape, k, v, S_cap, lens=None, fill_byte=None):
    """Quantise the same k, v on the GPU through tq_kv_quantize_append.  With fill_byte the
    arrays are pre-filled with that byte so rows past the end hold junk (0xFF -> NaN scales)."""
    cache = tq.KVCache(shape.B, shape.H_kv, S_cap, shape.d)
    if fill_byte is not None:
        cache.blocks.fill_(fill_byte)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    tq.tq_kv_quantize_append(cache, torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda(), status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    if lens is not None:
        cache.seq_lens.copy_(torch.as_tensor(np.asarray(lens, dtype=np.int32)))
    return cache


def assert_cache_bits_equal(dev_cache, host_cache, lens=None):
    """Bit-exact comparison of the valid rows of all six arrays."""
    B = host_cache.B
    lens = host_cache.lens if lens is None else lens
    for name, d_arr, h_arr in zip(("k_packed", "k_scale", "k_zero", "v_packed", "v_scale", "v_zero"),
                                  dev_cache.arrays_token_major(), host_cache.arrays()):
        d_np = d_arr.cpu().numpy()
        for b in range(B):
            n = int(lens[b])
            dv, hv = d_np[b, :, :n], h_arr[b, :, :n]
            if dv.dtype == np.float16:
                dv, hv = dv.view(np.uint16), hv.view(np.uint16)
            assert np.array_equal(dv, hv), f"{name} differs for sequence {b}: {np.count_nonzero(dv != hv)} elements"


def fused_attention(tq, torch, cache, q_np, alpha, num_splits=0, out_dtype=None, status=None):
    """decode + combine through the C ABI; returns (out numpy, (o_part, m_part, l_part) tensors, C)."""
    out_dtype = out_dtype or torch.float32
    q = torch.from_numpy(q_np).cuda()
    B, H_q, d = q.shape
    C = num_splits or tq.tq_auto_splits(B, cache.H_kv, H_q, d, cache.S_cap)
    o, m, l = tq.alloc_partials(B, H_q, d, C)
    out = torch.empty((B, H_q, d), dtype=out_dtype, device="cuda")
    tq.tq_sdpa_int4_decode(cache, q, alpha, C, o, m, l, status)
    tq.tq_sdpa_int4_combine(o, m, l, out)
    torch.cuda.synchronize()
    return out.float().cpu().numpy(), (o, m, l), C
