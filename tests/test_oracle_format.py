"""Pins for the oracle's number formats, packing and size model (CPU only)."""
import numpy as np
import pytest


def test_half_to_float_all_65536(oracle):
    bits = np.arange(65536, dtype=np.uint16)
    ref = bits.view(np.float16).astype(np.float32)
    got = np.array([oracle.half_to_float(int(b)) for b in bits], dtype=np.float32)
    nan = np.isnan(ref)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan].view(np.uint32), ref[~nan].view(np.uint32))


def test_float_to_half_round_to_nearest_even(oracle):
    rng = np.random.default_rng(11)
    # random bit patterns over the whole binary32 range, plus values dense around the fp16 range
    cand = [rng.integers(0, 2 ** 32, size=40000, dtype=np.uint64).astype(np.uint32).view(np.float32),
            (rng.standard_normal(40000) * 10.0 ** rng.uniform(-9, 5, 40000)).astype(np.float32)]
    # exact ties: midpoints between neighbouring halves (normal and subnormal), both signs
    h = np.arange(0, 0x7BFF, dtype=np.uint16)
    lo = h.view(np.float16).astype(np.float64)
    hi = (h + 1).astype(np.uint16).view(np.float16).astype(np.float64)
    mid = ((lo + hi) / 2).astype(np.float32)
    assert np.array_equal(mid.astype(np.float64), (lo + hi) / 2)  # midpoints are exact in binary32
    cand += [mid, -mid, np.nextafter(mid, np.float32(np.inf)), np.nextafter(mid, np.float32(-np.inf))]
    cand += [np.array([0.0, -0.0, 65504.0, 65519.99, 65520.0, 1e30, -1e30, np.inf, -np.inf, 2.0 ** -25,
                       np.nextafter(np.float32(2.0 ** -25), np.float32(1)), 2.0 ** -24, 5.96e-8, 1e-45],
                      dtype=np.float32)]
    x = np.concatenate(cand)
    x = x[~np.isnan(x)]
    with np.errstate(over="ignore"):
        ref = x.astype(np.float16).view(np.uint16)
    got = np.array([oracle.float_to_half(v) for v in x], dtype=np.uint16)
    assert np.array_equal(got, ref)
    assert oracle.float_to_half(np.float32(np.nan)) & 0x7C00 == 0x7C00


def test_pack_unpack_roundtrip_and_nibble_order(oracle):
    # every byte value: low nibble is the even element, high nibble the odd one
    allb = np.arange(256, dtype=np.uint8)
    codes = oracle.unpack_nibbles(allb)
    assert np.array_equal(codes[0::2], allb & 0xF)
    assert np.array_equal(codes[1::2], allb >> 4)
    assert np.array_equal(oracle.pack_nibbles(codes), allb)
    rng = np.random.default_rng(3)
    c = rng.integers(0, 16, size=(7, 128), dtype=np.uint8)
    assert np.array_equal(oracle.unpack_nibbles(oracle.pack_nibbles(c)), c)


def test_eq4_masked_dot_identity_all_words(oracle):
    """Eq. 4: sum_j (q_j / 16^j) * (w & mask_j) equals sum_j q_j * nibble_j for every 16-bit word w,
    where nibble_j is element j of the four codes the oracle packs into that word (little endian)."""
    w = np.arange(65536, dtype=np.uint32)
    bytes_le = np.stack([(w & 0xFF).astype(np.uint8), (w >> 8).astype(np.uint8)], axis=1)  # [65536][2]
    codes = oracle.unpack_nibbles(bytes_le).astype(np.float64)  # [65536][4]
    q = np.array([0.75, -1.5, 2.25, -0.625])  # exactly representable, so both sides are exact
    masks = np.array([0x000F, 0x00F0, 0x0F00, 0xF000], dtype=np.uint32)
    q_pre = q / 16.0 ** np.arange(4)
    lhs = ((w[:, None] & masks[None, :]).astype(np.float64) * q_pre[None, :]).sum(1)
    rhs = (codes * q[None, :]).sum(1)
    assert np.array_equal(lhs, rhs)


def test_group_storage_is_20_bytes_per_32_elements(oracle):
    assert oracle.int4_vector_bytes(32) == 20
    assert oracle.int4_vector_bytes(128) == 80
    assert oracle.int4_vector_bytes(256) == 160
    # Sec. 2.1: 3.2x against fp16 at g = 32
    assert 128 * 2 / oracle.int4_vector_bytes(128) == pytest.approx(3.2, abs=1e-12)


def test_cache_size_model_matches_paper_table(oracle):
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "kv_cache_sizes.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    assert len(rows) == 4
    GiB = 2.0 ** 30
    for S, fp16_g, int4_g in rows:
        S = int(S)
        assert abs(oracle.fp16_cache_bytes(80, 8, S, 128) / GiB - float(fp16_g)) <= 0.05 + 1e-9
        assert abs(oracle.int4_cache_bytes(80, 8, S, 128) / GiB - float(int4_g)) <= 0.05 + 1e-9
    # Eq. 1 exactly: 2 * 80 * 8 * 128K * 128 * 2 bytes = 40 GiB
    assert oracle.fp16_cache_bytes(80, 8, 131072, 128) == 40 * 2 ** 30
    assert oracle.int4_cache_bytes(80, 8, 131072, 128) * 3.2 == pytest.approx(40 * 2 ** 30)
