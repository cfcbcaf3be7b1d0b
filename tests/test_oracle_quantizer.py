"""Pins for the oracle's int4 quantiser (Eq. 2-3) -- invariants, bounds and brute force (CPU only).

Everything is evaluated in float64 from the STORED numbers (codes, fp16 scale, fp16 zero), so a
mistake anywhere in the float32 recipe (wrong sign of z, scale from the unrounded range, a
transposed nibble, truncation instead of rounding) breaks at least one check.
"""
import numpy as np
import pytest

from paper_2604_16957_b200 import inputs as I


def _groups(x):
    return x.reshape(-1, 32)


def _quant(oracle, x):
    p, s, z = oracle.quantize_rows(x)
    codes = oracle.unpack_nibbles(p)
    return codes, s.astype(np.float64), z.astype(np.float64)


@pytest.mark.parametrize("maker", ["normal", "outlier", "gemma_k", "shifted"])
def test_error_bound_and_code_range(oracle, maker):
    rng = np.random.default_rng(5)
    if maker == "normal":
        x = rng.standard_normal((4096, 128)).astype(np.float16)
    elif maker == "outlier":
        x = I.make_kv(I.LLAMA, 512, seed=2)[0].reshape(-1, 128)
    elif maker == "gemma_k":
        x = I.make_kv(I.GEMMA, 128, seed=4)[0].reshape(-1, 256)
    else:  # all-positive / all-negative groups: zero-point outside [0, 15]
        x = (rng.standard_normal((2048, 128)) + rng.choice([-6.0, 6.0], size=(2048, 1))).astype(np.float16)
    codes, s, z = _quant(oracle, x)
    assert codes.min() >= 0 and codes.max() <= 15
    xg = _groups(x.astype(np.float64))
    cg = _groups(codes.astype(np.float64))
    sg, zg = s.reshape(-1, 1), z.reshape(-1, 1)
    xhat = (cg - zg) * sg
    # stored scale is the fp16 rounding of range / 15
    rng_ = xg.max(1) - xg.min(1)
    assert np.all(np.abs(sg[:, 0] - rng_ / 15) <= np.abs(rng_ / 15) * 2.0 ** -10 + 1e-12)
    # zero-point: (0 - z) * s reproduces the group's minimum up to the fp16 rounding of z
    assert np.all(np.abs(-zg[:, 0] * sg[:, 0] - xg.min(1)) <= sg[:, 0] * np.maximum(np.abs(zg[:, 0]), 1) * 2.0 ** -10)
    # |x - x^| <= s/2 (+ the fp16 spacing of z and of s*15, valid while |z| <= 2048)
    assert np.abs(zg).max() < 2048
    assert np.all(np.abs(xg - xhat) <= sg * (0.5 + 2.0 ** -9) * (1 + np.abs(zg) * 2.0 ** -9))
    # the minimum maps to code 0, the maximum to code 15
    imin, imax = xg.argmin(1), xg.argmax(1)
    r = np.arange(len(xg))
    assert np.all(cg[r, imin] == 0)
    assert np.all(cg[r, imax] == 15)
    # monotone within a group
    order = np.argsort(xg, axis=1, kind="stable")
    assert np.all(np.diff(np.take_along_axis(cg, order, 1), axis=1) >= 0)


def test_chosen_code_is_nearest_by_brute_force(oracle):
    rng = np.random.default_rng(6)
    x = (rng.standard_normal((512, 64)) * rng.uniform(0.01, 30, size=(512, 1))).astype(np.float16)
    codes, s, z = _quant(oracle, x)
    xg, cg = _groups(x.astype(np.float64)), _groups(codes.astype(np.int64))
    sg, zg = s.reshape(-1, 1, 1), z.reshape(-1, 1, 1)
    cand = (np.arange(16, dtype=np.float64)[None, None, :] - zg) * sg  # every code's reconstruction
    err = np.abs(xg[:, :, None] - cand)
    chosen = np.take_along_axis(err, cg[:, :, None], 2)[:, :, 0]
    # nearest up to float32 rounding of x/s + z (a few ulp of a number below 32 -> 1e-5 * s)
    assert np.all(chosen <= err.min(2) + 1e-5 * sg[:, :, 0])


def test_rounding_is_half_to_even_on_exact_ties(oracle):
    # s = 1 exactly (range 15), z = 0 (min 0): x = k + 0.5 is an exact tie in binary32
    x = np.zeros((1, 32), np.float16)
    x[0, :16] = np.arange(16)                 # 0..15 -> codes 0..15, fixes min = 0 and max = 15
    x[0, 16:31] = np.arange(15) + 0.5          # 0.5, 1.5, ..., 14.5
    codes, s, z = _quant(oracle, x)
    assert s[0, 0] == 1.0 and z[0, 0] == 0.0
    assert list(codes[0, :16]) == list(range(16))
    expect = [int(np.rint(k + 0.5)) for k in range(15)]  # numpy rint is half-to-even: 0,2,2,4,4,...
    assert expect[:4] == [0, 2, 2, 4]
    assert list(codes[0, 16:31]) == expect


def test_constant_and_tiny_range_groups_reconstruct_exactly(oracle):
    vals = np.array([0.0, -0.0, 1.0, -3.5, 65504.0, -65504.0, 6.1e-5, 5.96e-8], dtype=np.float16)
    x = np.repeat(vals[:, None], 32, axis=1)
    p, s, z = oracle.quantize_rows(x)
    assert np.all(p == 0)
    assert np.all(s == np.float16(1.0))
    xhat = oracle.dequant_rows(p, s, z)
    assert np.array_equal(xhat, x.astype(np.float64))
    # +0 and -0 give the same stored zero-point bits
    assert z.view(np.uint16)[0, 0] == z.view(np.uint16)[1, 0] == 0
    # a range so small that range/15 underflows fp16: every element reconstructs to the minimum
    y = np.full((1, 32), 1.0, np.float16)
    y[0, 5] = np.nextafter(np.float16(1.0), np.float16(0))  # 1 - 2^-11 ; range/15 = 3.3e-5 (subnormal, nonzero)
    y2 = np.zeros((1, 32), np.float16)
    y2[0, 3] = np.float16(5.96e-8)  # range 2^-24, range/15 rounds to 0 in fp16
    p2, s2, z2 = oracle.quantize_rows(y2)
    assert s2[0, 0] == np.float16(1.0) and np.all(p2 == 0)
    assert np.abs(oracle.dequant_rows(p2, s2, z2) - y2.astype(np.float64)).max() <= 2.0 ** -24
    p1, s1, z1 = oracle.quantize_rows(y)
    assert np.all(np.isfinite(oracle.dequant_rows(p1, s1, z1)))


def test_huge_zero_point_is_clamped_not_nan(oracle):
    x = np.full((1, 32), 1000.0, np.float16)
    x[0, 0] = np.float16(1000.5)  # range 0.5, s = 0.0333, z = -30000 (finite); dequant finite
    p, s, z = oracle.quantize_rows(x)
    assert np.all(np.isfinite(z.astype(np.float64)))
    assert np.all(np.isfinite(oracle.dequant_rows(p, s, z)))


def test_statistics_on_standard_normal(oracle):
    """Drift alarm: on N(0,1) with g = 32, E[range] = 4.14 so E[s] is about 0.276; the
    quantisation error is close to uniform on [-s/2, s/2]; cosine(x, x^) is about 0.997
    (the paper reports 0.998 / 0.992 on real activations, Table 1)."""
    rng = np.random.default_rng(7)
    x = rng.standard_normal((8192, 128)).astype(np.float16)
    p, s, z = oracle.quantize_rows(x)
    xhat = oracle.dequant_rows(p, s, z)
    xd = x.astype(np.float64)
    assert s.astype(np.float64).mean() == pytest.approx(0.276, abs=0.004)
    e = (xhat - xd) / np.repeat(s.astype(np.float64), 32, axis=1)
    assert e.std() == pytest.approx(12 ** -0.5, abs=0.01)
    cos = (xd * xhat).sum() / np.sqrt((xd ** 2).sum() * (xhat ** 2).sum())
    assert cos == pytest.approx(0.9970, abs=0.0008)


def test_append_positions_lengths_and_overflow(oracle):
    sh = I.Shape("t", 3, 4, 2, 64, 0.125)
    cache = oracle.Cache(sh.B, sh.H_kv, 40, sh.d)
    cache.lens[:] = [0, 7, 38]
    k, v = I.make_kv(sh, 3, seed=9)
    before = [a.copy() for a in cache.arrays()]
    skipped = cache.append(k, v)
    assert skipped == 1                          # sequence 2 would overflow (38 + 3 > 40)
    assert list(cache.lens) == [3, 10, 38]
    kp, ks, kz = oracle.quantize_rows(k)
    vp, vs, vz = oracle.quantize_rows(v)
    for b, start in ((0, 0), (1, 7)):
        assert np.array_equal(cache.k_packed[b, :, start:start + 3], kp[b])
        assert np.array_equal(cache.v_zero[b, :, start:start + 3], vz[b])
        assert np.array_equal(cache.k_scale[b, :, start:start + 3], ks[b])
        assert np.array_equal(cache.v_packed[b, :, start:start + 3], vp[b])
    # nothing else was touched
    mask = np.ones((3, 2, 40), bool)
    mask[0, :, 0:3] = False
    mask[1, :, 7:10] = False
    for a, a0 in zip(cache.arrays(), before):
        assert np.array_equal(a[mask], a0[mask])
