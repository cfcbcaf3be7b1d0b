"""GPU parity of tq_kv_quantize_append against the CPU oracle: bit-exact codes, scales, zeros."""
import numpy as np
import pytest

from paper_2604_16957_b200 import inputs as I
from util import assert_cache_bits_equal, device_cache, oracle_cache

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gpu():
    import torch
    from paper_2604_16957_b200 import tq
    assert torch.cuda.is_available()
    return tq, torch


@pytest.mark.parametrize("shape,S,seed", [(I.TINY, 256, 1), (I.LLAMA, 1024, 2), (I.LLAMA, 4096 + 48, 3),
                                          (I.GEMMA, 512, 4), (I.Shape("b3", 3, 8, 2, 64, 0.125), 100, 6),
                                          (I.Shape("global512", 2, 32, 1, 512, 1.0, sigma_qk=0.25), 300, 7)])
def test_bulk_quantise_bit_exact(gpu, oracle, shape, S, seed):
    tq, torch = gpu
    k, v = I.make_kv(shape, S, seed)
    S_cap = (S + 15) // 16 * 16 + 16
    host = oracle_cache(oracle, shape, k, v, S_cap)
    dev = device_cache(tq, torch, shape, k, v, S_cap)
    assert dev.seq_lens.cpu().tolist() == [S] * shape.B
    assert_cache_bits_equal(dev, host)


def test_adversarial_groups_bit_exact(gpu, oracle):
    tq, torch = gpu
    rng = np.random.default_rng(40)
    rows = []
    consts = np.array([0.0, -0.0, 1.0, -3.5, 65504.0, -65504.0, 6.1e-5, 5.96e-8], np.float16)
    rows.append(np.repeat(consts[:, None], 128, 1))                                   # constant groups, signed zeros
    t = np.zeros((4, 128), np.float16); t[:, 3] = np.float16(5.96e-8); t[1] += np.float16(1.0)
    t[2, 40] = np.float16(-6e-8); t[3, 100] = np.float16(2e-4)
    rows.append(t)                                                                    # ranges that underflow fp16
    tie = np.zeros((1, 128), np.float16); tie[0, :16] = np.arange(16); tie[0, 16:31] = np.arange(15) + 0.5
    tie[0, 32:64] = tie[0, :32] * 2; tie[0, 64:96] = -tie[0, :32]; tie[0, 96:] = tie[0, :32] + 1000
    rows.append(tie)                                                                  # exact .5 ties
    rows.append(np.clip(rng.standard_normal((64, 128)) * 10.0 ** rng.uniform(-6, 4.5, (64, 1)), -65504, 65504).astype(np.float16))  # finite only: Inf / NaN inputs are undefined
    rows.append((rng.standard_normal((64, 128)) + rng.choice([-300.0, 300.0, 2000.0], (64, 1))).astype(np.float16))
    big = rng.choice(np.array([65504, -65504, 0, 1, 30000], np.float16), (16, 128))
    rows.append(big)                                                                  # full fp16 range
    sub = (rng.integers(0, 1024, (16, 128)).astype(np.uint16)).view(np.float16)       # subnormal inputs
    rows.append(sub)
    # a few thousand groups over many magnitudes and offsets (offset / spread up to ~1e4: the zero-point leaves
    # the range in which the kernel's shortcut is provably exact and the step-by-step arithmetic takes over)
    spread = 10.0 ** rng.uniform(-4, 3, (2048, 1))
    offset = spread * rng.choice([0.0, 1.0, -1.0, 30.0, -30.0, 600.0, -600.0, 1e4], (2048, 1))
    rows.append(np.clip(rng.standard_normal((2048, 128)) * spread + offset, -65504, 65504).astype(np.float16))
    x = np.concatenate(rows, 0)
    n = x.shape[0]
    shape = I.Shape("adv", 1, 1, 1, 128, 1.0)
    k = x.reshape(1, 1, n, 128)
    v = k[:, :, ::-1].copy()
    S_cap = (n + 15) // 16 * 16
    host = oracle_cache(oracle, shape, k, v, S_cap)
    dev = device_cache(tq, torch, shape, k, v, S_cap)
    assert_cache_bits_equal(dev, host)


def test_decode_step_appends_and_overflow(gpu, oracle):
    """T = 1 and T = 3 appends on ragged lengths, several steps in a row, with one sequence that
    runs out of room: its rows and length stay untouched and the status bit is set."""
    tq, torch = gpu
    shape = I.Shape("r", 4, 8, 2, 128, 0.1)
    S_cap = 64
    lens0 = [0, 17, 61, 40]
    k0, v0 = I.make_kv(shape, S_cap, 7)
    host = oracle_cache(oracle, shape, k0, v0, S_cap, lens=lens0)
    dev = device_cache(tq, torch, shape, k0, v0, S_cap, lens=lens0)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for step, T in enumerate([1, 3, 1, 1]):
        k, v = I.make_kv(shape, T, 7, stream=step + 1)
        before = [a.clone() for a in dev.arrays_token_major()]
        lens_before = dev.seq_lens.cpu().numpy().copy()
        skipped = host.append(k, v)
        tq.tq_kv_quantize_append(dev, torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda(), status)
        torch.cuda.synchronize()
        assert dev.seq_lens.cpu().tolist() == host.lens.tolist()
        assert_cache_bits_equal(dev, host)
        assert (int(status.item()) & tq.TQ_STATUS_CACHE_FULL != 0) == (skipped > 0 or step > 1)
        # rows outside [len, len + T) of every sequence are untouched
        for a, a0 in zip(dev.arrays_token_major(), before):
            an, a0n = a.cpu().numpy(), a0.cpu().numpy()
            for b in range(shape.B):
                lo = int(lens_before[b])
                hi = int(host.lens[b])
                assert np.array_equal(an[b, :, :lo].view(np.uint8), a0n[b, :, :lo].view(np.uint8))
                assert np.array_equal(an[b, :, hi:].view(np.uint8), a0n[b, :, hi:].view(np.uint8))
    assert host.lens.tolist() == [6, 23, 64, 46]


def test_lengths_near_int_max_are_refused_not_wrapped(gpu):
    """A caller-owned length close to INT_MAX must not wrap around in the capacity test: the sequence is
    skipped and flagged, its length and every byte of the cache stay as they were (small and bulk paths)."""
    tq, torch = gpu
    shape = I.Shape("m", 2, 4, 2, 128, 0.1)
    for T in (1, 3, 600):
        dev = tq.KVCache(shape.B, shape.H_kv, 1024, shape.d)
        dev.blocks.fill_(0xA5)
        dev.seq_lens.copy_(torch.tensor([2 ** 31 - 1, 2 ** 31 - 2], dtype=torch.int32))
        before = dev.blocks.clone()
        k, v = I.make_kv(shape, T, 9)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        tq.tq_kv_quantize_append(dev, torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda(), status)
        torch.cuda.synchronize()
        assert int(status.item()) & tq.TQ_STATUS_CACHE_FULL
        assert dev.seq_lens.cpu().tolist() == [2 ** 31 - 1, 2 ** 31 - 2]
        assert torch.equal(dev.blocks, before)


def test_bulk_path_with_ragged_lengths_and_overflow(gpu, oracle):
    tq, torch = gpu
    shape = I.Shape("r", 3, 8, 2, 128, 0.1)
    S_cap, T = 4096, 1500     # large enough to take the multi-block path
    k0, v0 = I.make_kv(shape, 16, 8)
    lens0 = [0, 1000, 3000]   # the last one overflows (3000 + 1500 > 4096)
    host = oracle_cache(oracle, shape, k0, v0, S_cap, lens=lens0)
    dev = device_cache(tq, torch, shape, k0, v0, S_cap, lens=lens0)
    k, v = I.make_kv(shape, T, 8, stream=1)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    assert host.append(k, v) == 1
    tq.tq_kv_quantize_append(dev, torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda(), status)
    torch.cuda.synchronize()
    assert int(status.item()) == tq.TQ_STATUS_CACHE_FULL
    assert dev.seq_lens.cpu().tolist() == [1500, 2500, 3000]
    # compare only rows that were ever written on both sides
    assert_cache_bits_equal(dev, host, lens=[1500, 0, 0])
    for name, d_arr, h_arr in zip("abcdef", dev.arrays_token_major(), host.arrays()):
        assert np.array_equal(d_arr.cpu().numpy()[1, :, 1000:2500].view(np.uint8), h_arr[1, :, 1000:2500].view(np.uint8))


def test_division_shortcut_equals_true_division_everywhere(gpu):
    """The group quantiser forms (max - min) / 15 and (0 - min) / scale from a reciprocal and one remainder
    correction; the library compares both with the correctly rounded division over all finite binary16
    (max, min) pairs and all (min, positive scale) pairs."""
    tq, torch = gpu
    assert tq._division_self_check() == 0
