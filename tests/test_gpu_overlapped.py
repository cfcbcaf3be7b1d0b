"""tq_sdpa_int4_decode_overlapped: phase 1 that attends the caller-declared stable part of the cache without
waiting for the kernel before it, then waits, reads the lengths and finishes with the newest tokens.  Checked
against the oracle (outputs and per-split partials under tq_split_range_stable), across head dimensions,
ragged lengths, stable parts that end on and off a block boundary, the fallbacks, a broken promise, and
back-to-back steps (eager and as a replayed CUDA graph) in which the call really overlaps its predecessors."""
import numpy as np
import pytest

from paper_2604_16957_b200 import inputs as I
from util import assert_attention_close, device_cache, oracle_cache

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gpu():
    import torch
    from paper_2604_16957_b200 import tq
    assert torch.cuda.is_available()
    return tq, torch


def _run(tq, torch, cache, q_np, alpha, C, stable, status=None, out_dtype=None):
    q = torch.from_numpy(q_np).cuda()
    B, H_q, d = q.shape
    o, m, l = tq.alloc_partials(B, H_q, d, C)
    out = torch.empty((B, H_q, d), dtype=out_dtype or torch.float32, device="cuda")
    tq.tq_sdpa_int4_decode_overlapped(cache, q, alpha, C, stable, o, m, l, status)
    tq.tq_sdpa_int4_combine(o, m, l, out)
    torch.cuda.synchronize()
    return out.float().cpu().numpy(), (o.cpu().numpy(), m.cpu().numpy(), l.cpu().numpy())


@pytest.mark.parametrize("d,H_q,H_kv", [(128, 16, 2), (64, 4, 1), (256, 8, 4), (512, 32, 1), (128, 24, 2)])
def test_matches_oracle_across_shapes_and_stable_parts(gpu, oracle, d, H_q, H_kv):
    tq, torch = gpu
    sh = I.Shape("x", 3, H_q, H_kv, d, d ** -0.5 if d < 256 else 1.0, sigma_qk=1.0 if d < 256 else 0.25,
                 k_outlier_channels=4 if d == 128 else 0)
    lens = [1500, 1203, 1216]
    k, v = I.make_kv(sh, 1500, 101)
    host = oracle_cache(oracle, sh, k, v, 1504, lens)
    dev = device_cache(tq, torch, sh, k, v, 1504, lens, fill_byte=0xFF)
    q = I.make_q(sh, 101)
    ref = oracle.attention(host, q, sh.alpha)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    # stable part: the shortest length, on and off a block boundary, far shorter, fewer blocks than splits
    # (falls back to the ordinary partition), zero (ordinary decode)
    for C, stable in ((5, 1203), (5, 1200), (3, 1216 - 16), (7, 480), (37, 1203), (1, 1203), (9, 100), (4, 0)):
        out, (o, m, l) = _run(tq, torch, dev, q, sh.alpha, C, stable, status)
        assert int(status.item()) == 0, (C, stable)
        assert_attention_close(out, ref, f"d={d} C={C} stable={stable}")
        bounds = np.zeros((sh.B, C + 1), np.int32)
        for b in range(sh.B):
            for c in range(C):
                bounds[b, c], bounds[b, c + 1] = tq.tq_split_range_stable(lens[b], stable, C, c)
            assert bounds[b, 0] == 0 and bounds[b, C] == lens[b]
        ro, rm, rl = oracle.attention_partials(host, q, sh.alpha, bounds)
        ne = rl > 0
        assert np.all(l[~ne] == 0) and np.all(o[~ne] == 0)
        assert np.abs((m[ne] + np.log(l[ne])) - (rm[ne] + np.log(rl[ne]))).max() < 1e-3
        assert_attention_close(o[ne], ro[ne], f"partials d={d} C={C} stable={stable}")


def test_partition_helper(gpu):
    tq, _ = gpu
    for length, stable, C in ((1000, 640, 5), (1000, 1000, 3), (131089, 131072, 37), (77, 64, 4), (5000, 40, 7)):
        prev = 0
        for c in range(C):
            t0, t1 = tq.tq_split_range_stable(length, stable, C, c)
            assert t0 == prev and t1 >= t0 and t0 % 16 == 0
            prev = t1
        assert prev == length
        if stable // 16 >= C:    # all but the last split depend on the stable part only
            assert [tq.tq_split_range_stable(length, stable, C, c) for c in range(C - 1)] == \
                   [tq.tq_split_range_stable(length + 999, stable, C, c) for c in range(C - 1)]
        else:
            assert [tq.tq_split_range_stable(length, stable, C, c) for c in range(C)] == \
                   [tq.tq_split_range(length, C, c) for c in range(C)]


def test_paged_cache_and_bad_arguments(gpu, oracle):
    tq, torch = gpu
    sh = I.Shape("x", 1, 8, 2, 128, 128 ** -0.5)
    k, v = I.make_kv(sh, 400, 102)
    q = I.make_q(sh, 102)
    host = oracle_cache(oracle, sh, k, v, 448)
    paged = tq.PagedKVCache(1, 2, 64, 7, 9, 128)
    paged.page_table.copy_(torch.tensor([[8, 1, 5, 0, 3, 7, 2]], dtype=torch.int32))
    tq.tq_kv_quantize_append(paged, torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda())
    out, _ = _run(tq, torch, paged, q, sh.alpha, 3, 384)          # paged: served by the ordinary decode
    assert_attention_close(out, oracle.attention(host, q, sh.alpha), "paged")
    dev = device_cache(tq, torch, sh, k, v, 448)
    o, m, l = tq.alloc_partials(1, 8, 128, 3)
    for bad in (-1, 449):
        with pytest.raises(tq.TqError) as e:
            tq.tq_sdpa_int4_decode_overlapped(dev, torch.from_numpy(q).cuda(), sh.alpha, 3, bad, o, m, l)
        assert e.value.code == tq.TQ_ERR_SHAPE


def test_length_below_the_stable_part_is_flagged(gpu):
    tq, torch = gpu
    sh = I.Shape("x", 2, 8, 2, 128, 0.1)
    k, v = I.make_kv(sh, 640, 103)
    dev = device_cache(tq, torch, sh, k, v, 640, lens=[640, 300])
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out, _ = _run(tq, torch, dev, I.make_q(sh, 103), sh.alpha, 4, 512, status)
    assert int(status.item()) == tq.TQ_STATUS_BAD_LEN
    assert np.all(np.isfinite(out))


@pytest.mark.parametrize("use_graph", [False, True])
def test_back_to_back_steps_overlap_their_predecessors(gpu, oracle, use_graph):
    """Twenty decode steps enqueued without any synchronisation between them (append, overlapped decode,
    combine, the next step's append, ...), so that each decode kernel starts while the kernels before it are
    still running; the stable part is the length before the first step.  Lengths cross a block boundary on
    the way.  Every step's output, kept in its own buffer, matches the oracle; as a replayed CUDA graph too."""
    tq, torch = gpu
    sh = I.Shape("x", 2, 64, 8, 128, 128 ** -0.5, k_outlier_channels=4)
    lens = [6000, 4107]
    steps, C, stable = 20, 9, 4096
    k, v = I.make_kv(sh, 6000, 104)
    host = oracle_cache(oracle, sh, k, v, 6032, lens)
    dev = device_cache(tq, torch, sh, k, v, 6032, lens, fill_byte=0xFF)
    kn = [I.make_kv(sh, 1, 104, stream=1 + i) for i in range(steps)]
    qn = [I.make_q(sh, 104, stream=i) for i in range(steps)]
    k_in = torch.stack([torch.from_numpy(a[0]) for a in kn]).cuda()
    v_in = torch.stack([torch.from_numpy(a[1]) for a in kn]).cuda()
    q_in = torch.stack([torch.from_numpy(a) for a in qn]).cuda()
    outs = torch.zeros((steps, sh.B, sh.H_q, sh.d), dtype=torch.float32, device="cuda")
    o, m, l = tq.alloc_partials(sh.B, sh.H_q, sh.d, C)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def enqueue():
        for i in range(steps):
            tq.tq_kv_quantize_append(dev, k_in[i], v_in[i], status)
            tq.tq_sdpa_int4_decode_overlapped(dev, q_in[i], sh.alpha, C, stable, o, m, l, status)
            tq.tq_sdpa_int4_combine(o, m, l, outs[i])

    if use_graph:
        warm = tq.KVCache(sh.B, sh.H_kv, 6032, sh.d)      # function attributes are set outside the capture
        warm.blocks.copy_(dev.blocks); warm.seq_lens.copy_(dev.seq_lens)
        tq.tq_sdpa_int4_decode_overlapped(warm, q_in[0], sh.alpha, C, stable, o, m, l, status)
        tq.tq_kv_quantize_append(warm, k_in[0], v_in[0], status)
        tq.tq_sdpa_int4_combine(o, m, l, outs[0])
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            enqueue()
        g.replay()
    else:
        enqueue()
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got = outs.cpu().numpy()
    for i in range(steps):
        host.append(*kn[i])
        if i in (0, 1, 4, 5, 10, steps - 1):       # lengths 4107 + i + 1: the second sequence crosses 4112 = 257 * 16 at i = 4
            assert_attention_close(got[i], oracle.attention(host, qn[i], sh.alpha), f"step {i}")
    assert dev.seq_lens.cpu().tolist() == [lens[0] + steps, lens[1] + steps]
