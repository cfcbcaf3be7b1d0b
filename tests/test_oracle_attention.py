"""Pins for the oracle's attention, split partials and Eq. 5 reduction (CPU only)."""
import numpy as np
import pytest

from paper_2604_16957_b200 import inputs as I


def _cache(oracle, shape, S, seed, S_cap=None, lens=None):
    k, v = I.make_kv(shape, S, seed)
    cache = oracle.Cache(shape.B, shape.H_kv, S_cap or S, shape.d)
    cache.append(k, v)
    if lens is not None:
        cache.lens[:] = lens
    return cache


def _dequant(oracle, cache):
    return (oracle.dequant_rows(cache.k_packed, cache.k_scale, cache.k_zero),
            oracle.dequant_rows(cache.v_packed, cache.v_scale, cache.v_zero))


def test_softmax_weights_sum_to_one(oracle):
    cache = _cache(oracle, I.TINY, 256, 1)
    q = I.make_q(I.TINY, 1)
    for h in range(4):
        w = oracle.attention_weights(cache, q, I.TINY.alpha, 0, h)
        assert w.shape == (256,) and w.min() >= 0
        assert abs(w.sum() - 1.0) < 1e-12


def test_matches_library_attention_on_dequantised_values(oracle):
    """The definition, evaluated by a library routine (torch fp64 SDPA) on the dequantised K, V."""
    import torch
    sh = I.Shape("t", 2, 8, 2, 64, 0.37, k_outlier_channels=2)
    cache = _cache(oracle, sh, 100, 21)
    q = I.make_q(sh, 21)
    got = oracle.attention(cache, q, sh.alpha)
    kd, vd = _dequant(oracle, cache)
    G = sh.H_q // sh.H_kv
    kt = torch.from_numpy(kd).repeat_interleave(G, dim=1)  # consecutive query heads share a KV head
    vt = torch.from_numpy(vd).repeat_interleave(G, dim=1)
    qt = torch.from_numpy(q.astype(np.float64))[:, :, None, :]
    ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, scale=sh.alpha)[:, :, 0, :].numpy()
    assert np.abs(got - ref).max() < 1e-12


def test_brute_force_tiny_python_loops(oracle):
    """Pure-Python evaluation from the unpacked codes: softmax(alpha q.k^) weighted sum of v^."""
    import math
    sh = I.Shape("t", 1, 2, 1, 32, 0.5)
    cache = _cache(oracle, sh, 5, 33)
    q = I.make_q(sh, 33).astype(np.float64)
    kc, vc = oracle.unpack_nibbles(cache.k_packed), oracle.unpack_nibbles(cache.v_packed)
    got = oracle.attention(cache, q.astype(np.float16), sh.alpha)
    for h in range(2):
        scores, vrows = [], []
        for i in range(5):
            sk, zk = float(cache.k_scale[0, 0, i, 0]), float(cache.k_zero[0, 0, i, 0])
            sv, zv = float(cache.v_scale[0, 0, i, 0]), float(cache.v_zero[0, 0, i, 0])
            scores.append(sh.alpha * sum(float(q[0, h, c]) * (int(kc[0, 0, i, c]) - zk) * sk for c in range(32)))
            vrows.append([(int(vc[0, 0, i, c]) - zv) * sv for c in range(32)])
        mx = max(scores)
        p = [math.exp(a - mx) for a in scores]
        out = [sum(p[i] * vrows[i][c] for i in range(5)) / sum(p) for c in range(32)]
        assert np.abs(got[0, h] - np.array(out)).max() < 1e-13


def test_blocked_log_sum_exp_evaluation_equals_two_pass_definition(oracle):
    """The same attention evaluated another way: tokens cut into uneven blocks, each block reduced to its
    log-sum-exp and its softmax-weighted value mean, the blocks then merged by their log-sum-exps.  A
    mistake in the oracle's maximum, exponent or normalisation shows up against this."""
    sh = I.Shape("t", 2, 4, 2, 64, 0.125)
    lens = [300, 17]
    cache = _cache(oracle, sh, 300, 8, lens=lens)
    q = I.make_q(sh, 8)
    full = oracle.attention(cache, q, sh.alpha)
    kd, vd = _dequant(oracle, cache)
    G = sh.H_q // sh.H_kv
    for b in range(2):
        n = lens[b]
        cuts = [0] + sorted(set(np.random.default_rng(b).integers(1, n, 6).tolist())) + [n]
        for h in range(4):
            a = sh.alpha * (kd[b, h // G, :n] @ q[b, h].astype(np.float64))
            lses, means = [], []
            for i0, i1 in zip(cuts[:-1], cuts[1:]):
                lse = np.logaddexp.reduce(a[i0:i1])
                lses.append(lse)
                means.append(np.exp(a[i0:i1] - lse) @ vd[b, h // G, i0:i1])
            w = np.exp(np.array(lses) - np.logaddexp.reduce(lses))
            assert abs(w.sum() - 1) < 1e-12
            assert np.abs(w @ np.array(means) - full[b, h]).max() < 1e-12


def test_constant_v_returns_v(oracle):
    sh = I.Shape("t", 1, 4, 2, 64, 0.125)
    k, _ = I.make_kv(sh, 64, 12)
    # (a) every token has the same V row: output is that row's dequantised value
    row = I.make_kv(sh, 1, 13)[1]
    v = np.repeat(row, 64, axis=2)
    cache = oracle.Cache(1, 2, 64, 64)
    cache.append(k, v)
    out = oracle.attention(cache, I.make_q(sh, 12), sh.alpha)
    vd = oracle.dequant_rows(cache.v_packed, cache.v_scale, cache.v_zero)
    for h in range(4):
        assert np.abs(out[0, h] - vd[0, h // 2, 0]).max() < 1e-12
    # (b) all elements equal (degenerate groups): output equals the constant exactly
    v2 = np.full_like(v, np.float16(-2.75))
    cache2 = oracle.Cache(1, 2, 64, 64)
    cache2.append(k, v2)
    out2 = oracle.attention(cache2, I.make_q(sh, 12), sh.alpha)
    assert np.abs(out2 - (-2.75)).max() < 1e-12


def test_single_token_zero_query_and_permutation(oracle):
    sh = I.Shape("t", 1, 4, 2, 64, 0.125)
    cache = _cache(oracle, sh, 50, 14)
    kd, vd = _dequant(oracle, cache)
    q = I.make_q(sh, 14)
    # S = 1: the output is v^_0
    c1 = _cache(oracle, sh, 50, 14, lens=[1])
    o1 = oracle.attention(c1, q, sh.alpha)
    for h in range(4):
        assert np.array_equal(o1[0, h], vd[0, h // 2, 0])
    # q = 0: uniform weights -> mean of v^
    o0 = oracle.attention(cache, np.zeros_like(q), sh.alpha)
    for h in range(4):
        assert np.abs(o0[0, h] - vd[0, h // 2].mean(0)).max() < 1e-12
    # permuting the tokens of the cache leaves the output unchanged
    perm = np.random.default_rng(1).permutation(50)
    pc = oracle.Cache(1, 2, 50, 64)
    for dst, src in zip(pc.arrays(), cache.arrays()):
        dst[:] = src[:, :, perm]
    pc.lens[:] = 50
    assert np.abs(oracle.attention(pc, q, sh.alpha) - oracle.attention(cache, q, sh.alpha)).max() < 1e-12


def test_gqa_head_mapping(oracle):
    sh = I.Shape("t", 1, 8, 2, 64, 0.125)
    cache = _cache(oracle, sh, 40, 15)
    q = I.make_q(sh, 15)
    q[0, :] = q[0, 0]  # identical queries: heads 0..3 share KV head 0, heads 4..7 share KV head 1
    out = oracle.attention(cache, q, sh.alpha)
    for h in range(1, 4):
        assert np.array_equal(out[0, h], out[0, 0])
    for h in range(5, 8):
        assert np.array_equal(out[0, h], out[0, 4])
    assert np.abs(out[0, 0] - out[0, 4]).max() > 1e-3
    # heads restriction computes the same rows
    part = oracle.attention(cache, q, sh.alpha, heads=(4, 6))
    assert np.array_equal(part[0, 4:6], out[0, 4:6]) and np.all(part[0, :4] == 0) and np.all(part[0, 6:] == 0)


def test_attn_scale_is_a_plain_multiplier(oracle):
    sh = I.Shape("t", 1, 4, 2, 64, 0.25)
    cache = _cache(oracle, sh, 40, 16)
    q = I.make_q(sh, 16)
    a = oracle.attention(cache, q, 0.25)
    b = oracle.attention(cache, (q.astype(np.float32) * 0.25).astype(np.float16), 1.0)  # exact: power of two
    assert np.abs(a - b).max() < 1e-12
    assert np.abs(a - oracle.attention(cache, q, 1.0)).max() > 1e-3


@pytest.mark.parametrize("bounds", [[0, 300], [0, 1, 300], [0, 0, 150, 150, 299, 300], [0, 64, 128, 192, 256, 300],
                                    [0, 300, 300]])
def test_split_partials_recombine_by_eq5(oracle, bounds):
    sh = I.Shape("t", 2, 4, 2, 64, 0.125)
    cache = _cache(oracle, sh, 300, 17, lens=[300, 200])
    q = I.make_q(sh, 17)
    b2 = np.array([bounds, [min(x, 200) for x in bounds]], np.int32)
    o, m, l = oracle.attention_partials(cache, q, sh.alpha, b2)
    full = oracle.attention(cache, q, sh.alpha)
    assert np.abs(oracle.combine(o, m, l) - full).max() < 1e-12
    # empty splits report (0, -inf, 0)
    empty = np.diff(b2, axis=1) == 0
    for b in range(2):
        for c in np.nonzero(empty[b])[0]:
            assert np.all(l[b, :, c] == 0) and np.all(np.isneginf(m[b, :, c])) and np.all(o[b, :, c] == 0)
    # partial outputs are normalised: a one-token split returns that token's v^
    if bounds[:2] == [0, 1]:
        vd = oracle.dequant_rows(cache.v_packed, cache.v_scale, cache.v_zero)
        assert np.array_equal(o[0, 0, 0], vd[0, 0, 0]) and l[0, 0, 0] == 1.0


def test_zero_length_sequence_gives_zero(oracle):
    sh = I.Shape("t", 2, 4, 2, 64, 0.125)
    cache = _cache(oracle, sh, 10, 18, lens=[0, 10])
    out = oracle.attention(cache, I.make_q(sh, 18), sh.alpha)
    assert np.all(out[0] == 0) and np.abs(out[1]).max() > 0


def test_sliding_window_equals_attention_over_the_last_w_tokens(oracle):
    sh = I.Shape("t", 2, 4, 2, 64, 0.125)
    lens = [100, 37]
    cache = _cache(oracle, sh, 100, 19, lens=lens)
    q = I.make_q(sh, 19)
    full = oracle.attention(cache, q, sh.alpha)
    # a window at least as long as the sequence, or none, changes nothing
    assert np.array_equal(oracle.attention_window(cache, q, sh.alpha, 0), full)
    assert np.array_equal(oracle.attention_window(cache, q, sh.alpha, 100), full)
    assert np.array_equal(oracle.attention_window(cache, q, sh.alpha, 5000), full)
    vd = oracle.dequant_rows(cache.v_packed, cache.v_scale, cache.v_zero)
    # window 1: the last token's v^
    w1 = oracle.attention_window(cache, q, sh.alpha, 1)
    for b in range(2):
        for h in range(4):
            assert np.array_equal(w1[b, h], vd[b, h // 2, lens[b] - 1])
    # window w: the same as full attention over a cache that holds only the last w tokens
    for w in (7, 16, 40):
        cut = oracle.Cache(sh.B, sh.H_kv, 100, sh.d)
        for b in range(2):
            n = min(w, lens[b])
            for dst, src in zip(cut.arrays(), cache.arrays()):
                dst[b, :, :n] = src[b, :, lens[b] - n:lens[b]]
            cut.lens[b] = n
        assert np.abs(oracle.attention_window(cache, q, sh.alpha, w) - oracle.attention(cut, q, sh.alpha)).max() < 1e-12
        assert np.abs(oracle.attention_window(cache, q, sh.alpha, w) - full).max() > 1e-4


def test_multi_query_is_causal_attention_of_each_query_token(oracle):
    sh = I.Shape("t", 2, 4, 2, 64, 0.125)
    lens = [60, 2]
    cache = _cache(oracle, sh, 64, 23, lens=lens)
    S_q = 3
    q = np.stack([I.make_q(sh, 23, stream=s) for s in range(S_q)], axis=1)  # [B][S_q][H_q][d]
    out = oracle.attention_multi(cache, q, sh.alpha)
    assert np.array_equal(cache.lens, np.array(lens, np.int32))  # the lengths are restored
    # the newest query token sees everything; one query token is plain attention
    assert np.array_equal(out[:, S_q - 1], oracle.attention(cache, q[:, S_q - 1], sh.alpha))
    assert np.array_equal(oracle.attention_multi(cache, q[:, :1], sh.alpha)[:, 0], oracle.attention(cache, q[:, 0], sh.alpha))
    # query token s: brute force over the first len - (S_q - 1 - s) tokens from the dequantised cache
    kd = oracle.dequant_rows(cache.k_packed, cache.k_scale, cache.k_zero)
    vd = oracle.dequant_rows(cache.v_packed, cache.v_scale, cache.v_zero)
    for b in range(2):
        for s in range(S_q):
            n = max(lens[b] - (S_q - 1 - s), 0)
            for h in range(4):
                if n == 0:
                    assert not out[b, s, h].any()
                    continue
                a = sh.alpha * kd[b, h // 2, :n] @ q[b, s, h].astype(np.float64)
                w = np.exp(a - a.max())
                ref = (w / w.sum()) @ vd[b, h // 2, :n]
                assert np.abs(out[b, s, h] - ref).max() < 1e-12
    # with a window, the same over the last w of those tokens
    outw = oracle.attention_multi(cache, q, sh.alpha, window=10)
    a = sh.alpha * kd[0, 1, 48:58] @ q[0, 0, 3].astype(np.float64)
    w = np.exp(a - a.max())
    assert np.abs(outw[0, 0, 3] - (w / w.sum()) @ vd[0, 1, 48:58]).max() < 1e-12


def test_mixed_precision_attention_reduces_to_its_two_ends(oracle):
    sh = I.Shape("t", 2, 4, 2, 64, 0.125)
    k, v = I.make_kv(sh, 80, 29)
    cache = oracle.Cache(sh.B, sh.H_kv, 80, sh.d)
    cache.append(k, v)
    cache.lens[:] = [80, 33]
    q = I.make_q(sh, 29)
    # both sides from the cache: the C implementation of the definition
    assert np.abs(oracle.attention_mixed(cache, None, None, q, sh.alpha) - oracle.attention(cache, q, sh.alpha)).max() < 1e-12
    # both sides unquantised: attention on the fp16 inputs, independent of the cache contents
    full = oracle.attention_mixed(cache, k, v, q, sh.alpha)
    other = oracle.Cache(sh.B, sh.H_kv, 80, sh.d)
    other.lens[:] = cache.lens
    assert np.array_equal(oracle.attention_mixed(other, k, v, q, sh.alpha), full)
    # one side each: equal to plain attention over a cache whose other side is exact, which is the case
    # for values that int4 represents exactly (here V in {0..15}/4 per group with min 0 and max 15/4)
    rng = np.random.default_rng(3)
    v_exact = (rng.integers(0, 16, size=v.shape) / 4.0).astype(np.float16)
    v_exact[..., 0::32] = 0.0
    v_exact[..., 1::32] = 3.75
    c2 = oracle.Cache(sh.B, sh.H_kv, 80, sh.d)
    c2.append(k, v_exact)
    vd = oracle.dequant_rows(c2.v_packed, c2.v_scale, c2.v_zero)
    assert np.array_equal(vd, v_exact.astype(np.float64))
    assert np.abs(oracle.attention_mixed(c2, None, v_exact, q, sh.alpha) - oracle.attention(c2, q, sh.alpha)).max() < 1e-12
    # and the ablation's ordering is measurable: each variant differs from the unquantised result
    for kk, vv in ((None, v), (k, None)):
        assert np.abs(oracle.attention_mixed(cache, kk, vv, q, sh.alpha) - full).max() > 1e-4
