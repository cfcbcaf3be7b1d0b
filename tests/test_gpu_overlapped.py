"""tq_sdpa_int4_decode_overlapped: phase 1 that attends the caller-declared stable part of the cache without
waiting for the kernel before it, then waits, reads the lengths and finishes with the newest tokens.  Checked
against the oracle (outputs and per-split partials under tq_split_range_stable), across head dimensions,
ragged lengths, stable parts that end on and off a block boundary, the fallbacks, a broken promise, and
back-to-back steps (eager and as a replayed CUDA graph) in which the call really overlaps its predecessors."""
import numpy as np
import pytest

from paper_2604_16957_b200 import inputs as I
from util import MAX_ABS_TOL, assert_attention_close, device_cache, oracle_cache

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
    for stable in (384, 128, 0):                                  # paged caches take the overlapped form too
        out, _ = _run(tq, torch, paged, q, sh.alpha, 3, stable)
        assert_attention_close(out, oracle.attention(host, q, sh.alpha), f"paged stable={stable}")
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


# ------------------------------------------------------------------------------------------------ fused step
def _step_setup(tq, torch, oracle, sh, S, S_cap, lens, seed):
    k, v = I.make_kv(sh, S, seed)
    host = oracle_cache(oracle, sh, k, v, S_cap, lens)
    dev = device_cache(tq, torch, sh, k, v, S_cap, lens, fill_byte=0xFF)
    return host, dev


@pytest.mark.parametrize("d,H_q,H_kv", [(128, 16, 2), (64, 4, 1), (256, 4, 2), (512, 8, 1), (128, 64, 8)])
def test_fused_step_matches_three_calls_and_oracle(gpu, oracle, d, H_q, H_kv):
    """tq_sdpa_int4_step against the oracle: the appended rows bit for bit, the lengths, and the outputs, over
    several steps, stable parts (none, exact, short), split counts, both output types; lengths pass a block
    boundary, one sequence is one token short of its capacity at the start."""
    from util import assert_cache_bits_equal
    tq, torch = gpu
    sh = I.Shape("x", 3, H_q, H_kv, d, d ** -0.5 if d < 256 else 1.0, sigma_qk=1.0 if d < 256 else 0.25,
                 k_outlier_channels=4 if d == 128 else 0)
    lens = [900, 13, 1039]
    S_cap = 1040
    host, dev = _step_setup(tq, torch, oracle, sh, 1039, S_cap, lens, 111)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for step, (C, stable, dt) in enumerate(((4, 0, torch.float32), (4, 0, torch.float32), (3, 896, torch.float32),
                                            (1, 0, torch.float16), (7, 16, torch.float32), (37, 900, torch.float32))):
        ws = tq.alloc_step_workspace(sh.B, sh.H_kv, sh.H_q, sh.d, C)
        kn, vn = I.make_kv(sh, 1, 111, stream=1 + step)
        qn = I.make_q(sh, 111, stream=step)
        out = torch.full((sh.B, sh.H_q, sh.d), 7.0, dtype=dt, device="cuda")
        st_stable = min(stable, 13 // 16 * 16) if stable else 0    # the promise must hold for every sequence
        tq.tq_sdpa_int4_step(dev, torch.from_numpy(kn).cuda(), torch.from_numpy(vn).cuda(), torch.from_numpy(qn).cuda(),
                             sh.alpha, C, st_stable, ws, out, status)
        torch.cuda.synchronize()
        skipped = host.append(kn, vn)
        full = int(status.item()) & tq.TQ_STATUS_CACHE_FULL
        assert bool(full) == (skipped > 0) and int(status.item()) & ~tq.TQ_STATUS_CACHE_FULL == 0
        status.zero_()
        assert dev.seq_lens.cpu().tolist() == host.lens.tolist()
        assert_cache_bits_equal(dev, host)
        assert not ws[:tq._lib.tq_step_counter_bytes(sh.B, sh.H_kv)].any()     # counters are left zero
        ref = oracle.attention(host, qn, sh.alpha)
        got = out.float().cpu().numpy()
        if dt == torch.float32:
            assert_attention_close(got, ref, f"step {step} C={C} stable={st_stable}")
        else:
            assert np.abs(got - ref).max() <= 2e-3 + np.abs(ref).max() * 2.0 ** -11
    assert host.lens.tolist() == [906, 19, 1040]


def test_fused_step_with_a_real_stable_part_and_no_append(gpu, oracle):
    tq, torch = gpu
    sh = I.Shape("x", 2, 64, 8, 128, 128 ** -0.5, k_outlier_channels=4)
    lens = [5000, 4100]
    host, dev = _step_setup(tq, torch, oracle, sh, 5000, 5008, lens, 112)
    q = I.make_q(sh, 112)
    ref = oracle.attention(host, q, sh.alpha)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for C, stable in ((9, 4096), (0, 4100), (16, 0)):
        Cn = C or tq.tq_auto_splits_step(sh.B, sh.H_kv, sh.H_q, sh.d, 5008)
        ws = tq.alloc_step_workspace(sh.B, sh.H_kv, sh.H_q, sh.d, Cn)
        out = torch.empty((sh.B, sh.H_q, sh.d), dtype=torch.float32, device="cuda")
        tq.tq_sdpa_int4_step(dev, None, None, torch.from_numpy(q).cuda(), sh.alpha, C, stable, ws, out, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0 and dev.seq_lens.cpu().tolist() == lens
        assert_attention_close(out.cpu().numpy(), ref, f"no append C={C} stable={stable}")


def test_fused_step_argument_checks(gpu):
    tq, torch = gpu
    dev = tq.KVCache(1, 2, 64, 128)
    q = torch.zeros((1, 32, 128), dtype=torch.float16, device="cuda")       # 16 query heads per KV head
    out = torch.zeros((1, 32, 128), dtype=torch.float32, device="cuda")
    ws = tq.alloc_step_workspace(1, 2, 32, 128, 2)
    with pytest.raises(tq.TqError) as e:
        tq.tq_sdpa_int4_step(dev, None, None, q, 1.0, 2, 0, ws, out)
    assert e.value.code == tq.TQ_ERR_SHAPE
    q, out = q[:, :16].contiguous(), out[:, :16].contiguous()
    with pytest.raises(tq.TqError) as e:
        tq.tq_sdpa_int4_step(dev, None, None, q, 1.0, 2, 0, ws[:1024], out)
    assert e.value.code == tq.TQ_ERR_WORKSPACE


@pytest.mark.parametrize("use_graph", [False, True])
def test_fused_steps_back_to_back(gpu, oracle, use_graph):
    """Twenty fused steps on one cache enqueued without synchronisation (each kernel overlaps the tail of the
    one before it), eager and as a replayed CUDA graph: every output matches the oracle, the cache ends up
    bit-identical to the oracle's."""
    from util import assert_cache_bits_equal
    tq, torch = gpu
    sh = I.Shape("x", 2, 64, 8, 128, 128 ** -0.5, k_outlier_channels=4)
    lens = [6000, 4107]
    steps, C, stable = 20, 9, 4096
    host, dev = _step_setup(tq, torch, oracle, sh, 6000, 6032, lens, 113)
    kn = [I.make_kv(sh, 1, 113, stream=1 + i) for i in range(steps)]
    qn = [I.make_q(sh, 113, stream=i) for i in range(steps)]
    k_in = torch.stack([torch.from_numpy(a[0]) for a in kn]).cuda()
    v_in = torch.stack([torch.from_numpy(a[1]) for a in kn]).cuda()
    q_in = torch.stack([torch.from_numpy(a) for a in qn]).cuda()
    outs = torch.zeros((steps, sh.B, sh.H_q, sh.d), dtype=torch.float32, device="cuda")
    ws = tq.alloc_step_workspace(sh.B, sh.H_kv, sh.H_q, sh.d, C)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def enqueue(cache):
        for i in range(steps):
            tq.tq_sdpa_int4_step(cache, k_in[i], v_in[i], q_in[i], sh.alpha, C, stable, ws, outs[i], status)

    if use_graph:
        warm = tq.KVCache(sh.B, sh.H_kv, 6032, sh.d)      # function attributes are set outside the capture
        warm.blocks.copy_(dev.blocks); warm.seq_lens.copy_(dev.seq_lens)
        tq.tq_sdpa_int4_step(warm, k_in[0], v_in[0], q_in[0], sh.alpha, C, stable, ws, outs[0], status)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            enqueue(dev)
        g.replay()
    else:
        enqueue(dev)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got = outs.cpu().numpy()
    for i in range(steps):
        host.append(*kn[i])
        if i in (0, 1, 4, 5, 10, steps - 1):
            assert_attention_close(got[i], oracle.attention(host, qn[i], sh.alpha), f"step {i}")
    assert dev.seq_lens.cpu().tolist() == host.lens.tolist()
    assert_cache_bits_equal(dev, host)


@pytest.mark.parametrize("S", [32768, 131072])
def test_config3_long_context_layer_through_the_one_launch_step(gpu, oracle, S):
    """One Llama-70B-shaped layer at 32K and at 128K tokens through tq_sdpa_int4_step exactly as the benchmark
    launches it (library-chosen split count, the tokens present before the step declared stable, the new token
    appended by the same launch; fp32 output on the first step, fp16 on the second): the cache bit for bit, then every query head against the oracle."""
    from util import assert_cache_bits_equal
    tq, torch = gpu
    sh = I.LLAMA
    S_cap = S + 16
    host, dev = _step_setup(tq, torch, oracle, sh, S, S_cap, [S], 30 + S // 32768)
    C = tq.tq_auto_splits_step(sh.B, sh.H_kv, sh.H_q, sh.d, S_cap)
    ws = tq.alloc_step_workspace(sh.B, sh.H_kv, sh.H_q, sh.d, C)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for step, dt in enumerate((torch.float32, torch.float16)):   # the second step's stable part ends inside the block the first wrote to
        out = torch.zeros((sh.B, sh.H_q, sh.d), dtype=dt, device="cuda")
        kn, vn = I.make_kv(sh, 1, 31, stream=1 + step)
        qn = I.make_q(sh, 31, stream=step)
        tq.tq_sdpa_int4_step(dev, torch.from_numpy(kn).cuda(), torch.from_numpy(vn).cuda(), torch.from_numpy(qn).cuda(),
                             sh.alpha, C, S, ws, out, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        host.append(kn, vn)
        assert dev.seq_lens.cpu().tolist() == [S + step + 1]
        ref = oracle.attention(host, qn, sh.alpha)
        got = out.float().cpu().numpy()
        if dt == torch.float32:
            mx, rel = assert_attention_close(got, ref, f"S={S} step {step}")
            print(f"llama {S} + 1 through the step entry, C={C}: max-abs {mx:.2e} rel-L2 {rel:.2e}")
        else:
            assert np.abs(got - ref).max() <= MAX_ABS_TOL + np.abs(ref).max() * 2.0 ** -11, f"S={S} step {step}"
    assert_cache_bits_equal(dev, host)


@pytest.mark.parametrize("d,H_q,H_kv,page_tokens", [(128, 16, 2, 64), (256, 8, 4, 16), (64, 4, 1, 128), (512, 8, 1, 32)])
def test_fused_step_on_a_paged_cache(gpu, oracle, d, H_q, H_kv, page_tokens):
    """tq_sdpa_int4_step over a page pool (random page assignment): steps that append into the last page, cross
    into the next one, and run with stable parts that end inside a page, at a page boundary and at zero; rows bit
    for bit, lengths, outputs against the oracle; then a table entry outside the pool for the page the new token
    falls into: flagged, nothing written."""
    from util import assert_cache_bits_equal
    tq, torch = gpu
    sh = I.Shape("x", 2, H_q, H_kv, d, d ** -0.5 if d < 256 else 1.0, sigma_qk=1.0 if d < 256 else 0.25,
                 k_outlier_channels=4 if d == 128 else 0)
    S = 2 * page_tokens * 3 - 2                    # two tokens short of a page boundary
    max_pages = S // page_tokens + 3
    num_pages = sh.B * max_pages + 2
    dev = tq.PagedKVCache(sh.B, sh.H_kv, page_tokens, max_pages, num_pages, sh.d)
    perm = np.random.default_rng(5).permutation(num_pages)[:sh.B * max_pages].astype(np.int32)
    dev.page_table.copy_(torch.from_numpy(perm.reshape(sh.B, max_pages)))
    dev.blocks.fill_(0xFF)
    host = oracle.Cache(sh.B, sh.H_kv, page_tokens * max_pages, sh.d)
    k, v = I.make_kv(sh, S, 121)
    host.append(k, v)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    tq.tq_kv_quantize_append(dev, torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda(), status)
    for step, (C, stable) in enumerate(((3, S // 16 * 16), (2, 0), (4, S - page_tokens), (1, 16), (5, S))):
        ws = tq.alloc_step_workspace(sh.B, sh.H_kv, sh.H_q, sh.d, C)
        kn, vn = I.make_kv(sh, 1, 121, stream=1 + step)
        qn = I.make_q(sh, 121, stream=step)
        out = torch.full((sh.B, sh.H_q, sh.d), 7.0, dtype=torch.float32, device="cuda")
        tq.tq_sdpa_int4_step(dev, torch.from_numpy(kn).cuda(), torch.from_numpy(vn).cuda(), torch.from_numpy(qn).cuda(),
                             sh.alpha, C, stable, ws, out, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        host.append(kn, vn)
        assert dev.seq_lens.cpu().tolist() == host.lens.tolist()
        assert_cache_bits_equal(dev, host)
        assert_attention_close(out.cpu().numpy(), oracle.attention(host, qn, sh.alpha), f"paged step {step} C={C} stable={stable}")
    # the next token of sequence 1 falls into a page whose table entry is outside the pool
    entry = int(host.lens[1]) // page_tokens
    before = dev.blocks.clone()
    dev.page_table[1, entry] = num_pages + 7
    kn, vn = I.make_kv(sh, 1, 121, stream=99)
    ws = tq.alloc_step_workspace(sh.B, sh.H_kv, sh.H_q, sh.d, 2)
    out = torch.zeros((sh.B, sh.H_q, sh.d), dtype=torch.float32, device="cuda")
    tq.tq_sdpa_int4_step(dev, torch.from_numpy(kn).cuda(), torch.from_numpy(vn).cuda(), torch.from_numpy(I.make_q(sh, 121)).cuda(),
                         sh.alpha, 2, 0, ws, out, status)
    torch.cuda.synchronize()
    assert int(status.item()) & tq.TQ_STATUS_BAD_PAGE
    per_page = dev.blocks.numel() // num_pages
    changed = (dev.blocks != before).view(num_pages, per_page).any(dim=1).nonzero().flatten().tolist()
    assert set(changed) <= {int(perm.reshape(sh.B, max_pages)[0, int(host.lens[0]) // page_tokens])}   # only sequence 0's row


@pytest.mark.parametrize("paged", [False, True])
def test_fused_step_with_one_stable_part_per_sequence(gpu, oracle, paged):
    """tq_sdpa_int4_step_ragged: a batch of unequal lengths, each sequence with its own stable part (its length
    before the steps; one sequence too short to start early, one with a stable part of zero, one with a value
    beyond its capacity that is clamped), several steps, against the oracle; then a stable part longer than a
    sequence: flagged."""
    from util import assert_cache_bits_equal
    tq, torch = gpu
    sh = I.Shape("x", 5, 16, 2, 128, 128 ** -0.5, k_outlier_channels=4)
    lens = [3000, 517, 40, 2049, 1200]
    S_cap = 3072
    k, v = I.make_kv(sh, 3000, 131)
    if paged:
        dev = tq.PagedKVCache(sh.B, sh.H_kv, 64, S_cap // 64, sh.B * (S_cap // 64) + 1, sh.d)
        perm = np.random.default_rng(6).permutation(dev.num_pages)[:sh.B * dev.max_pages].astype(np.int32)
        dev.page_table.copy_(torch.from_numpy(perm.reshape(sh.B, dev.max_pages)))
        host = oracle_cache(oracle, sh, k, v, S_cap, lens)
        flat = device_cache(tq, torch, sh, k, v, S_cap, lens)     # the ragged fill, then moved into the pool page by page
        pages = flat.blocks.view(sh.B, sh.H_kv, S_cap // 64, 4, -1).permute(0, 2, 1, 3, 4).reshape(sh.B * (S_cap // 64), sh.H_kv, 4, -1)
        dev.blocks[torch.from_numpy(perm).long()] = pages
        dev.seq_lens.copy_(flat.seq_lens)
    else:
        host = oracle_cache(oracle, sh, k, v, S_cap, lens)
        dev = device_cache(tq, torch, sh, k, v, S_cap, lens, fill_byte=0xFF)
    stable = torch.tensor([3000, 517, 40, 0, 99999], dtype=torch.int32, device="cuda")   # 99999 clamps to S_cap > 1200
    stable[4] = 1200
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for step, C in enumerate((4, 7, 1)):
        ws = tq.alloc_step_workspace(sh.B, sh.H_kv, sh.H_q, sh.d, C)
        kn, vn = I.make_kv(sh, 1, 131, stream=1 + step)
        qn = I.make_q(sh, 131, stream=step)
        out = torch.full((sh.B, sh.H_q, sh.d), 7.0, dtype=torch.float32, device="cuda")
        tq.tq_sdpa_int4_step(dev, torch.from_numpy(kn).cuda(), torch.from_numpy(vn).cuda(), torch.from_numpy(qn).cuda(),
                             sh.alpha, C, stable, ws, out, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        host.append(kn, vn)
        assert dev.seq_lens.cpu().tolist() == host.lens.tolist()
        assert_cache_bits_equal(dev, host)
        assert_attention_close(out.cpu().numpy(), oracle.attention(host, qn, sh.alpha), f"ragged step {step} C={C}")
    stable[1] = 1024                               # longer than sequence 1 (520 tokens now): a broken promise
    ws = tq.alloc_step_workspace(sh.B, sh.H_kv, sh.H_q, sh.d, 4)
    tq.tq_sdpa_int4_step(dev, None, None, torch.from_numpy(I.make_q(sh, 131)).cuda(), sh.alpha, 4, stable, ws, out, status)
    torch.cuda.synchronize()
    assert int(status.item()) & tq.TQ_STATUS_BAD_LEN


@pytest.mark.parametrize("d,H_q,H_kv", [(256, 32, 16), (128, 16, 2), (64, 4, 1), (512, 8, 1)])
def test_fused_step_with_a_sliding_window(gpu, oracle, d, H_q, H_kv):
    """tq_sdpa_int4_step_window: append + attention over the last `window` tokens + reduction in one launch, over
    several steps (lengths pass a block boundary, one sequence is shorter than the window, one is full), windows that
    start inside a block, split counts from 1 up; rows bit for bit, lengths, outputs against the oracle.  First
    without a stable part (the general windowed form), then with one (the overlapped form: lengths from the stable
    part itself up to TQ_WINDOW_SLACK beyond it), then a length beyond the promised range: flagged."""
    from util import assert_cache_bits_equal
    tq, torch = gpu
    sh = I.Shape("x", 4, H_q, H_kv, d, d ** -0.5 if d < 256 else 1.0, sigma_qk=1.0 if d < 256 else 0.25,
                 k_outlier_channels=4 if d == 128 else 0)
    lens = [3000, 1024, 30, 3055]
    S_cap = 3056
    host, dev = _step_setup(tq, torch, oracle, sh, 3055, S_cap, lens, 141)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def run(step, window, C, stable, append=True):
        Cn = C or tq.tq_auto_splits(sh.B, sh.H_kv, sh.H_q, sh.d, window)
        ws = tq.alloc_step_workspace(sh.B, sh.H_kv, sh.H_q, sh.d, Cn)
        kn, vn = I.make_kv(sh, 1, 141, stream=1 + step)
        qn = I.make_q(sh, 141, stream=step)
        out = torch.full((sh.B, sh.H_q, sh.d), 7.0, dtype=torch.float32, device="cuda")
        tq.tq_sdpa_int4_step_window(dev, torch.from_numpy(kn).cuda() if append else None,
                                    torch.from_numpy(vn).cuda() if append else None, torch.from_numpy(qn).cuda(),
                                    sh.alpha, window, C, stable, ws, out, status)
        torch.cuda.synchronize()
        skipped = host.append(kn, vn) if append else 0
        return out.cpu().numpy(), qn, skipped

    for step, (window, C) in enumerate(((1024, 0), (1000, 3), (17, 1), (5000, 4), (1, 2), (1024, 7))):
        got, qn, skipped = run(step, window, C, 0)
        full = int(status.item()) & tq.TQ_STATUS_CACHE_FULL
        assert bool(full) == (skipped > 0) and int(status.item()) & ~tq.TQ_STATUS_CACHE_FULL == 0
        status.zero_()
        assert dev.seq_lens.cpu().tolist() == host.lens.tolist()
        assert_cache_bits_equal(dev, host)
        assert_attention_close(got, oracle.attention_window(host, qn, sh.alpha, window), f"window step {step} w={window} C={C}")

    # overlapped form: every sequence between `stable` and `stable` + 128 tokens long
    lens2 = [2000, 2001, 2120, 2064]
    host, dev = _step_setup(tq, torch, oracle, sh, 2120, S_cap, lens2, 142)
    for step, (window, C) in enumerate(((1024, 0), (1000, 3), (1024, 7), (400, 2), (2500, 5))):
        stable = 2000 if step < 4 else 2010          # (2010: not a multiple of 16; rounded down by the library)
        got, qn, _ = run(10 + step, window, C, stable, append=step != 2)
        assert int(status.item()) == 0
        assert dev.seq_lens.cpu().tolist() == host.lens.tolist()
        assert_cache_bits_equal(dev, host)
        assert_attention_close(got, oracle.attention_window(host, qn, sh.alpha, window), f"overlapped window step {step} w={window} C={C}")
    run(20, 1024, 2, 1856, append=False)             # sequence 2 holds 2124 tokens now: more than 1856 + 128
    assert int(status.item()) & tq.TQ_STATUS_BAD_LEN
    status.zero_()
    paged = tq.PagedKVCache(1, sh.H_kv, 32, 2, 3, sh.d)
    q1 = torch.zeros((1, sh.H_q, sh.d), dtype=torch.float16, device="cuda")
    with pytest.raises(tq.TqError) as e:
        tq.tq_sdpa_int4_step_window(paged, None, None, q1, 1.0, 16, 1, 0, tq.alloc_step_workspace(1, sh.H_kv, sh.H_q, sh.d, 1),
                                    torch.zeros_like(q1, dtype=torch.float32), status)
    assert e.value.code == tq.TQ_ERR_SHAPE
