"""The bounded waits of the decode kernel.  Every wait for an asynchronous copy has a limit; when it runs out the
warp flags TQ_STATUS_TIMEOUT, gives the copies still in flight their time to land and returns.  A test cannot
make a real copy fail without a bad pointer, so the library's instrumented instantiation (test hook, not part
of the ABI) makes one chosen block's barrier expect 16 bytes that never arrive -- the data itself lands -- and
can shorten the limit.  Nothing here faults, traps or waits without a bound."""
import numpy as np
import pytest

from paper_2604_16957_b200 import inputs as I
from util import assert_attention_close, device_cache, fused_attention, oracle_cache

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gpu():
    import torch
    from paper_2604_16957_b200 import tq
    assert torch.cuda.is_available()
    return tq, torch


def _guarded(torch, n, dtype=None):
    """n elements with 64 canary elements on each side."""
    buf = torch.full((n + 128,), 12345.0, dtype=dtype or torch.float32, device="cuda")
    return buf, buf[64:64 + n]


@pytest.mark.parametrize("d,H_q,H_kv", [(128, 16, 2), (256, 8, 2)])   # one warp per token block; two-warp teams
def test_wait_that_cannot_complete_is_flagged_and_the_call_returns(gpu, oracle, d, H_q, H_kv):
    tq, torch = gpu
    sh = I.Shape("x", 2, H_q, H_kv, d, d ** -0.5 if d < 256 else 1.0, sigma_qk=1.0 if d < 256 else 0.25)
    lens = [2000, 700]
    k, v = I.make_kv(sh, 2000, 121)
    host = oracle_cache(oracle, sh, k, v, 2000, lens)
    dev = device_cache(tq, torch, sh, k, v, 2000, lens)
    q_np = I.make_q(sh, 121)
    q = torch.from_numpy(q_np).cuda()
    C = 3
    n = sh.B * sh.H_q * C
    ob, o = _guarded(torch, n * sh.d)
    mb, m = _guarded(torch, n)
    lb, l = _guarded(torch, n)
    o, m, l = o.view(sh.B, sh.H_q, C, sh.d), m.view(sh.B, sh.H_q, C), l.view(sh.B, sh.H_q, C)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    tq._test_hook(tq.HOOK_FAULT_BLOCK, 40)      # tokens 640 .. 655 of every (sequence, KV head)
    tq._test_hook(tq.HOOK_SPIN_LIMIT, 200000)   # 0.1 ms instead of 2 ms for the stage waits (the drain keeps the full limit)
    try:
        tq.tq_sdpa_int4_decode(dev, q, sh.alpha, C, o, m, l, status)
        torch.cuda.synchronize()                # returns: the wait gave up
    finally:
        tq._test_hook(tq.HOOK_FAULT_BLOCK, -1)
        tq._test_hook(tq.HOOK_SPIN_LIMIT, 0)
    assert int(status.item()) & tq.TQ_STATUS_TIMEOUT
    for buf in (ob, mb, lb):                    # nothing was written outside the partial arrays
        assert torch.all(buf[:64] == 12345.0) and torch.all(buf[-64:] == 12345.0)
    # the context is intact: the same call without the hook is correct, on the same stream
    status.zero_()
    out, _, _ = fused_attention(tq, torch, dev, q_np, sh.alpha, num_splits=C, status=status)
    assert int(status.item()) == 0
    assert_attention_close(out, oracle.attention(host, q_np, sh.alpha), "after the timeout")


def test_shortened_wait_either_completes_or_flags(gpu, oracle):
    """A limit of one clock cycle: a wait whose copy has not landed yet gives up at once.  Whether any wait is
    caught that early depends on timing; the call must return either way, and a clean status means a correct
    result."""
    tq, torch = gpu
    sh = I.Shape("x", 1, 64, 8, 128, 128 ** -0.5)
    k, v = I.make_kv(sh, 8192, 122)
    host = oracle_cache(oracle, sh, k, v, 8192)
    dev = device_cache(tq, torch, sh, k, v, 8192)
    q_np = I.make_q(sh, 122)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    tq._test_hook(tq.HOOK_SPIN_LIMIT, 1)
    try:
        out, _, _ = fused_attention(tq, torch, dev, q_np, sh.alpha, num_splits=8, status=status)
    finally:
        tq._test_hook(tq.HOOK_SPIN_LIMIT, 0)
    st = int(status.item())
    assert st in (0, tq.TQ_STATUS_TIMEOUT)
    if st == 0:
        assert_attention_close(out, oracle.attention(host, q_np, sh.alpha), "short limit, no timeout")
    status.zero_()
    out, _, _ = fused_attention(tq, torch, dev, q_np, sh.alpha, num_splits=8, status=status)
    assert int(status.item()) == 0
    assert_attention_close(out, oracle.attention(host, q_np, sh.alpha), "afterwards")
