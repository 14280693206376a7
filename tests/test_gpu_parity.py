"""GPU-vs-oracle parity through the C ABI (run with -m gpu on a B200).

Bit-exact: gathered rows, counts, ready / expired ID lists, emission numbers after sorting by (id, seq),
timestamps, procedural table fill.  Within tolerance (normwise, 1e-5 for fp32 configurations, 1e-2 where
DFVs or head operands are bfloat16): head input, probabilities, loss, head gradients, dX, embedding
gradients and updated tables, open-group sums, averaged gradients.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_1806_03925_b200 import workloads
from paper_1806_03925_b200.workloads import BF16, F32, PRESETS, Batch, BatchSource

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gb():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_1806_03925_b200 import binding
    binding.load()
    return binding


def _pair(*a, **k):
    from gpu_harness import Pair
    return Pair(*a, **k)


# ------------------------------------------------------------------ procedural fill
def test_procedural_fill_is_bit_identical(gb):
    for dtype, np_dt, dim, rows in ((torch.float32, np.float32, 20, 1000), (torch.bfloat16, np.uint16, 24, 777),
                                    (torch.float32, np.float32, 3, 5)):
        t = torch.empty((rows, dim), dtype=dtype, device="cuda")
        gb.gear_fill_uniform(t, seed=11, tag=gb.GEAR_TAG_DFV)
        want = oracle.fill_rows(11, oracle.TAG_DFV, dim, None, rows, np_dt)
        got = t.view(torch.int16).cpu().numpy().view(np.uint16) if dtype == torch.bfloat16 else t.cpu().numpy()
        assert np.array_equal(got, want)


# ------------------------------------------------------------------ whole step, every configuration (reduced where needed)
def _run_steps(p, steps, seed=0, want_emb_grad=False, B=None, dense=None, fused=False):
    src = BatchSource(p, seed)
    batches = [src.batch(s, B) for s in range(steps)]
    pair = _pair(p, batches, seed=seed, want_emb_grad=want_emb_grad, dense=dense, fused=fused)
    out = []
    try:
        for s, b in enumerate(batches):
            out.append(pair.step_and_compare(b, now=s + 1))
    finally:
        pair.close()
    return out


@pytest.mark.parametrize("fused", [False, True])
def test_tiny_config_all_steps(gb, fused):
    p = PRESETS["tiny"]
    out = _run_steps(p, p.steps, fused=fused)
    assert all(o["status"] == 0 for o in out)
    assert sum(o["n_ready"] for o in out) > 0 and sum(o["n_expired"] for o in out) > 0


def test_tiny_config_embedding_gradients(gb):
    _run_steps(PRESETS["tiny"], 3, want_emb_grad=True)


def test_medium_config_two_steps(gb):
    # full medium shapes (1M-row tables, bf16 DFVs, 192-256-128-1 head); the oracle keeps the touched rows only
    p = PRESETS["medium"]
    out = _run_steps(p, 2, dense=False)
    assert out[-1]["n_ready"] > 0


def test_medium_config_two_steps_events_5_and_6_in_one_call(gb):
    out = _run_steps(PRESETS["medium"], 2, dense=False, fused=True)
    assert out[-1]["n_ready"] > 0


@pytest.mark.parametrize("head", [F32, BF16])
def test_split_image_workload_with_a_dense_input_on_the_fast_side(gb, head):
    """The shape of the paper's CIFAR100 experiment (Section 4): half of every image (1536 values) stays on the Fastgear
    side as a dense input of its own, appended to the head input; the other half is the cached DFV."""
    p = PRESETS["split_image"].scaled(head_dtype=head, dfv_dtype=head)
    out = _run_steps(p, 3, want_emb_grad=True)
    assert out[-1]["n_ready"] > 0
    _run_steps(p, 2, B=333, fused=True)


def test_medium_shapes_ragged_batch(gb):
    p = PRESETS["medium"].scaled(user_vocab=50_000, url_vocab=30_000, img_vocab=20_000)
    _run_steps(p, 2, B=1237, want_emb_grad=True)


def test_skew_shapes_ragged_batch(gb):
    # fp32 head of 192-256-128-1 (the 128 x 128 product kernel) on a batch that ends inside a tile and inside a
    # 16-byte piece of the batch-long reductions
    p = PRESETS["skew"].scaled(M=8, img_vocab=50_000, user_vocab=50_000, url_vocab=50_000)
    _run_steps(p, 2, B=1237, want_emb_grad=True)


@pytest.mark.parametrize("head,hidden,E,D,dfv,B", [
    (BF16, (1024, 64), 4, 256, BF16, 3000),     # widest layer, narrowest layer, a batch that ends inside a row tile
    (BF16, (192, 448), 64, 256, F32, 1),        # widths that are no multiple of a 256-column tile; one view
    (BF16, (320,), 20, 200, BF16, 129),         # head input 240 wide: a partial reduction block and partial column tiles
    (F32, (264,), 32, 8, F32, 2049),            # fp32 head: 128 x 128 product tiles with ragged edges on every side
    (F32, (64, 96), 16, 8, F32, 33),            # fp32 head below the large-tile threshold
    # DFV widths on either side of the row widths the gather and the reduce pass are instantiated for
    # (1, 2, 4 or 8 sixteen-byte chunks per lane): 3, 5, 6 and 7 chunks per lane take the guarded path of the next
    # instantiation up; 4 and 8 chunks per lane the unguarded one
    (F32, (64,), 16, 384, F32, 257),
    (F32, (64,), 16, 640, F32, 130),
    (BF16, (128,), 32, 768, BF16, 300),
    (F32, (64,), 16, 896, F32, 65),
    (F32, (64,), 8, 512, F32, 100),
    (F32, (64,), 8, 1024, F32, 40),
    (BF16, (64,), 8, 1024, BF16, 40),
    # a 1024-wide layer on top of a 320-wide one, 3000 views: thousands of units inside the ReLU rounding band
    (BF16, (320, 1024), 20, 512, BF16, 3000),
])
def test_odd_head_shapes(gb, head, hidden, E, D, dfv, B):
    p = PRESETS["medium"].scaled(emb_dim=E, dfv_dim=D, dfv_dtype=dfv, head_dtype=head, hidden=hidden, M=3,
                                 user_vocab=30_000, url_vocab=20_000, img_vocab=40_000, expire=2)
    _run_steps(p, 2, B=B, want_emb_grad=True)


def _soak_case(case: int):
    """A random but reproducible configuration: head type and widths, embedding and DFV widths, DFV type, batch
    size, M, image vocabulary and expiry time are all drawn from (case)."""
    rng = np.random.default_rng(1000 + case)
    bf = rng.random() < 0.65
    if bf:
        hidden = tuple(int(rng.choice([64, 128, 192, 256, 320, 448, 512, 1024])) for _ in range(int(rng.integers(1, 3))))
        E = int(rng.choice([4, 8, 20, 32, 64]))
        D = int(rng.choice([8, 24, 64, 128, 200, 256, 384, 512, 768]))
        dfv_dtype = BF16 if rng.random() < 0.7 else F32
    else:
        hidden = tuple(int(rng.choice([8, 24, 64, 96, 136, 256, 264])) for _ in range(int(rng.integers(1, 3))))
        E = int(rng.choice([4, 12, 16, 32]))
        D = int(rng.choice([8, 40, 64, 128, 256, 640]))
        dfv_dtype = F32
    B = int(rng.choice([1, 7, 33, 129, 500, 1237, 2049, 3000]))
    p = PRESETS["medium"].scaled(emb_dim=E, dfv_dim=D, dfv_dtype=dfv_dtype, head_dtype=BF16 if bf else F32,
                                 hidden=hidden, M=int(rng.choice([1, 2, 5, 16])), user_vocab=30_000, url_vocab=20_000,
                                 img_vocab=int(rng.choice([5_000, 40_000])), expire=int(rng.choice([0, 2, 50])))
    return p, B, bool(rng.random() < 0.5)


@pytest.mark.parametrize("case", range(24))
def test_random_shapes(gb, case):
    p, B, want_emb_grad = _soak_case(case)
    _run_steps(p, 2, seed=case, B=B, want_emb_grad=want_emb_grad, fused=bool(case % 2))


@pytest.mark.parametrize("M", [1, 64, 1024])
def test_skew_config_reduced(gb, M):
    # skew shapes with a smaller batch and image table; Zipf 1.3 keeps most rows on a handful of images
    p = PRESETS["skew"].scaled(M=M, img_vocab=100_000, user_vocab=100_000, url_vocab=100_000)
    out = _run_steps(p, 3, B=4096)
    if M == 1:
        assert out[0]["n_ready"] > 4096


@pytest.mark.parametrize("M", [1, 64])
def test_skew_config_reduced_atomic_mode(gb, M):
    # GEAR_ACC_ATOMIC under the same contention: counts, emission (id, seq) pairs exact; averages and kept sums
    # against the oracle's order-free store (the order of the fp32 reductions is the hardware's)
    p = PRESETS["skew"].scaled(M=M, img_vocab=100_000, user_vocab=100_000, url_vocab=100_000)
    src = BatchSource(p, 0)
    batches = [src.batch(s, 4096) for s in range(3)]
    pair = _pair(p, batches, seed=0, atomic=True)
    try:
        out = [pair.step_and_compare(b, now=s + 1) for s, b in enumerate(batches)]
    finally:
        pair.close()
    assert sum(o["n_ready"] for o in out) > 0


def test_large_shapes_reduced(gb):
    # large-table head (384-512-256-1, bf16 DFV dim 256, E 64, M 32) on small tables and 1536 views
    p = PRESETS["large"].scaled(user_vocab=80_000, url_vocab=60_000, img_vocab=40_000)
    _run_steps(p, 2, B=1536)


# ------------------------------------------------------------------ accumulate-only (micro-benchmark shapes, reduced)
@pytest.mark.parametrize("zipf_s,M,atomic", [(0.0, 8, False), (1.1, 8, False), (1.1, 64, False), (1.1, 8, True)])
def test_accumulate_only_reduced(gb, zipf_s, M, atomic):
    from gpu_harness import assert_close, _np
    V, D, n = 50_000, 128, 200_003
    p = PRESETS["skew"].scaled(img_vocab=V, dfv_dim=D, M=M, user_vocab=16, url_vocab=16, expire=1 << 40)
    mp = workloads.MicroPreset("t", n, V, D, M, zipf_s)
    ids = workloads.micro_ids(mp, seed=3)
    pair = _pair(p, [], seed=3, dense=True, extra_img_ids=ids, ready_cap=2 * n, atomic=atomic)
    try:
        g = torch.empty((n, D), dtype=torch.float32, device="cuda")
        gb.gear_fill_uniform(g, seed=3, tag=gb.GEAR_TAG_GRAD, amp=1.0)
        g_cpu = oracle.fill_rows(3, oracle.TAG_GRAD, D, None, n, np.float32, amp=1.0).astype(np.float64)
        ids_t = torch.from_numpy(ids).cuda()
        half = n // 2 + 1
        for lo, hi in ((0, half), (half, n)):       # two calls before one collect: emission numbers continue
            pair.gpu.accumulate_rows(ids_t[lo:hi], g[lo:hi])
            pair.cpu.accumulate(ids[lo:hi], g_cpu[lo:hi], pooled=atomic)
            pair.compare_store()
        n_ready = pair.collect_and_compare()
        k = np.bincount(ids, minlength=V)
        assert n_ready == int((k // M).sum())
        pair.status()
        assert pair.status_bits == 0
    finally:
        pair.close()


# ------------------------------------------------------------------ edge cases
def _tiny_pair(batches, **kw):
    p = PRESETS["tiny"].scaled(user_vocab=500, url_vocab=400, img_vocab=300, **kw.pop("preset", {}))
    return p, _pair(p, batches, dense=True, **kw)


def _manual_batch(uid, hid, imgs, labels):
    n = [len(v) for v in imgs]
    off = np.concatenate([[0], np.cumsum(n)]).astype(np.int32)
    flat = np.array([i for v in imgs for i in v], dtype=np.int32)
    return Batch(np.array(uid, np.int32), np.array(hid, np.int32), off, flat, np.array(labels, np.float32))


def test_empty_views_repeated_images_and_bad_ids(gb):
    b = _manual_batch([1, 2, 2, 499, 7], [0, 399, 5, 5, 1000],          # url 1000 is out of range
                      [[5, 5, 5], [], [299], [-3, 10, 10, 7], [12]],    # empty view, repeats, a negative image id
                      [1, 0, 0, 1, 0])
    p, pair = _tiny_pair([b], preset=dict(M=2))
    try:
        out = pair.step_and_compare(b, now=1)
        assert out["bad"] == 2
        assert out["status"] & 1 and out["rc"] == -3        # GEAR_DEV_BAD_ID, GEAR_ERR_BAD_ID
        assert pair.gpu.status()[1] == 0                    # the status word is cleared once read
    finally:
        pair.close()


def test_single_view_and_batch_of_one_image(gb):
    b = _manual_batch([3], [4], [[8]], [1])
    p, pair = _tiny_pair([b], preset=dict(M=1))
    try:
        out = pair.step_and_compare(b, now=1)
        assert out["n_ready"] == 1
    finally:
        pair.close()


def test_plan_made_ahead_is_dropped_when_other_calls_come_first(gb):
    """gear_forward_backward prepares the plan of the accumulate call that usually follows.  Calls that change what the
    plan was made from (another accumulate, a collect) in between must not be able to make that plan go stale."""
    from paper_1806_03925_b200.session import DeviceBatch
    p = PRESETS["tiny"].scaled(user_vocab=500, url_vocab=400, img_vocab=300, M=2)
    src = BatchSource(p, 3)
    b = src.batch(0, 200)
    extra_ids = src.batch(1, 64).img_id
    pair = _pair(p, [b], seed=3, dense=True, extra_img_ids=extra_ids)
    try:
        g, cpu = pair.gpu, pair.cpu
        db = DeviceBatch.from_host(b)
        g.forward_backward(db)
        r = cpu.forward_backward(pair.params.astype(np.float64), pair.ru(b.user_id), pair.rh(b.url_id), b.img_off,
                                 pair.ri(b.img_id), b.label)
        # another accumulate call and a collect come between the step and its own accumulate
        rows = torch.ones((len(extra_ids), p.dfv_dim), device="cuda") * 0.5
        g.accumulate_rows(torch.from_numpy(extra_ids).cuda(), rows)
        cpu.accumulate(pair.ri(extra_ids), np.full((len(extra_ids), p.dfv_dim), 0.5))
        pair.compare_store()
        pair.collect_and_compare()
        g.accumulate_from_step(db)
        cpu.accumulate(pair.ri(b.img_id), cpu.dfv_grad_rows(b.img_off, r.dX))
        pair.compare_store()
        assert pair.collect_and_compare() > 0
        pair.status()
        assert pair.status_bits == 0
    finally:
        pair.close()


def test_fused_call_on_a_non_empty_queue_and_with_a_short_list(gb):
    """gear_accumulate_collect must give the results of accumulate + collect also where it cannot bypass the queue:
    when averages of an earlier call are still waiting, and when the caller's lists are shorter than the row count."""
    from gpu_harness import _np, assert_close
    p = PRESETS["tiny"].scaled(user_vocab=16, url_vocab=16, img_vocab=300, M=2)
    rng = np.random.default_rng(11)
    ids_a = rng.integers(0, 40, 500).astype(np.int32)
    ids_b = rng.integers(0, 40, 300).astype(np.int32)
    ga = rng.normal(0, 1, (500, p.dfv_dim)).astype(np.float32)
    gb_ = rng.normal(0, 1, (300, p.dfv_dim)).astype(np.float32)
    for cap in (None, 260):          # None: lists as long as the row count; 260 < 300 rows, but enough for the groups
        pair = _pair(p, [], dense=True, extra_img_ids=np.concatenate([ids_a, ids_b]), ready_cap=cap or 0)
        try:
            g, cpu = pair.gpu, pair.cpu
            if cap is None:
                g.accumulate_rows(torch.from_numpy(ids_a).cuda(), torch.from_numpy(ga).cuda())     # stays in the queue
                cpu.accumulate(ids_a, ga.astype(np.float64))
            n = g.accumulate_collect_rows(torch.from_numpy(ids_b).cuda(), torch.from_numpy(gb_).cuda())
            cpu.accumulate(ids_b, gb_.astype(np.float64))
            pair.compare_store()
            eid, eseq, eavg = oracle.sort_emissions(*cpu.collect_ready())
            assert n == len(eid) and n > 0
            assert np.array_equal(_np(g.ready_ids[:n]), eid) and np.array_equal(_np(g.ready_seq[:n]), eseq)
            assert_close(_np(g.ready_avg[:n]), eavg, 1e-5, "averaged gradients")
            assert g.status()[1:] == (0, 0) and g.guards_intact()
            # and straight after, with the queue empty again, the same call bypasses the queue
            n2 = g.accumulate_collect_rows(torch.from_numpy(ids_a[:200]).cuda(), torch.from_numpy(ga[:200]).cuda())
            cpu.accumulate(ids_a[:200], ga[:200].astype(np.float64))
            pair.compare_store()
            eid, eseq, eavg = oracle.sort_emissions(*cpu.collect_ready())
            assert n2 == len(eid)
            assert np.array_equal(_np(g.ready_ids[:n2]), eid) and np.array_equal(_np(g.ready_seq[:n2]), eseq)
            assert_close(_np(g.ready_avg[:n2]), eavg, 1e-5, "averaged gradients")
            assert g.status()[1:] == (0, 0) and g.guards_intact()
        finally:
            pair.close()


def test_fused_call_whose_lists_cannot_take_the_completed_groups(gb):
    """Lists shorter than what the call completes: the reduce pass must notice on the device, leave the averages in the
    ready queue, report the required count and hand nothing over; a later hand-over into long enough lists gets all."""
    from gpu_harness import _np, assert_close
    p = PRESETS["tiny"].scaled(user_vocab=16, url_vocab=16, img_vocab=300, M=1)
    rng = np.random.default_rng(12)
    ids = rng.integers(0, 300, 500).astype(np.int32)
    g_rows = rng.normal(0, 1, (500, p.dfv_dim)).astype(np.float32)
    pair = _pair(p, [], dense=True, extra_img_ids=ids, ready_cap=1000)
    try:
        g, cpu = pair.gpu, pair.cpu
        d_ids, d_rows = torch.from_numpy(ids).cuda(), torch.from_numpy(g_rows).cuda()
        with pytest.raises(gb.GearError) as e:          # M = 1: 500 groups, lists of 100
            gb.gear_accumulate_collect(g.ctx, d_ids, d_rows.data_ptr(), p.dfv_dim, None, None, 500, g.ready_ids, g.ready_seq,
                                       g.ready_avg, 100, d_n=g.d_counts[0:1])
        assert e.value.code == gb.GEAR_ERR_CAPACITY and int(g.d_counts[0].item()) == 500
        rc, bits, pending = g.status()
        assert pending == 500 and bits & gb.GEAR_DEV_OUT_CAPACITY
        cpu.accumulate(ids, g_rows.astype(np.float64))
        pair.compare_store()
        # a second fused call with lists of 100 that DO suffice (2 new groups) must not bypass the non-empty queue
        with pytest.raises(gb.GearError):
            gb.gear_accumulate_collect(g.ctx, d_ids[:2], d_rows.data_ptr(), p.dfv_dim, None, None, 2, g.ready_ids, g.ready_seq,
                                       g.ready_avg, 100, d_n=g.d_counts[0:1])
        assert int(g.d_counts[0].item()) == 502
        g.status()
        cpu.accumulate(ids[:2], g_rows[:2].astype(np.float64))
        n = g.collect_ready()
        eid, eseq, eavg = oracle.sort_emissions(*cpu.collect_ready())
        assert n == 502 == len(eid)
        assert np.array_equal(_np(g.ready_ids[:n]), eid) and np.array_equal(_np(g.ready_seq[:n]), eseq)
        assert_close(_np(g.ready_avg[:n]), eavg, 1e-5, "averaged gradients")
        assert g.status()[1:] == (0, 0) and g.guards_intact()
    finally:
        pair.close()


def test_zero_sized_calls_are_accepted(gb):
    b = _manual_batch([3], [4], [[8]], [1])
    p, pair = _tiny_pair([b])
    try:
        g = pair.gpu
        empty_i = torch.zeros(0, dtype=torch.int32, device="cuda")
        g.accumulate_rows(empty_i, torch.zeros((0, p.dfv_dim), device="cuda"))
        assert g.collect_ready() == 0
        from paper_1806_03925_b200.session import DeviceBatch
        eb = Batch(np.zeros(0, np.int32), np.zeros(0, np.int32), np.zeros(1, np.int32), np.zeros(0, np.int32),
                   np.zeros(0, np.float32))
        g.forward_backward(DeviceBatch.from_host(eb))
        assert g.status()[0] == 0
        assert float(g.loss.item()) == 0.0 and not g.head_grad.any().item()
    finally:
        pair.close()


def test_ready_capacity_too_small_consumes_nothing(gb):
    from gpu_harness import _np
    rng = np.random.default_rng(5)
    b = _manual_batch(rng.integers(0, 500, 64), rng.integers(0, 400, 64), [[int(i)] for i in rng.integers(0, 20, 64)],
                      rng.integers(0, 2, 64))
    p, pair = _tiny_pair([b], preset=dict(M=2))
    try:
        g, c = pair.gpu, pair.cpu
        from paper_1806_03925_b200.session import DeviceBatch
        db = DeviceBatch.from_host(b)
        g.forward_backward(db)
        g.accumulate_from_step(db)
        pending = g.status()[2]
        assert pending > 1
        with pytest.raises(gb.GearError) as e:
            gb.gear_collect_ready(g.ctx, g.ready_ids, g.ready_seq, g.ready_avg, pending - 1)
        assert e.value.code == gb.GEAR_ERR_CAPACITY
        rc, status, still = g.status()
        assert still == pending and status & gb.GEAR_DEV_OUT_CAPACITY
        assert g.collect_ready() == pending                 # a large enough list gets everything
    finally:
        pair.close()


def test_expired_capacity_too_small_lists_and_restamps_nothing(gb):
    b = _manual_batch([3], [4], [[8]], [1])
    p, pair = _tiny_pair([b], preset=dict(expire=10))
    try:
        g = pair.gpu
        before = g.dfv_ts.clone()
        with pytest.raises(gb.GearError) as e:
            gb.gear_collect_expired(g.ctx, 5, True, g.expired_ids, 3)
        assert e.value.code == gb.GEAR_ERR_CAPACITY
        assert torch.equal(before, g.dfv_ts)
        g.status()
        pair.expire_and_compare(5)
        pair.expire_and_compare(5)                          # restamped: nothing is expired any more
        pair.expire_and_compare(14, restamp=False)
        pair.expire_and_compare(15, restamp=False)
    finally:
        pair.close()


def test_ready_queue_overflow_drops_the_call(gb):
    p = PRESETS["tiny"].scaled(user_vocab=16, url_vocab=16, img_vocab=64, M=1)
    ids = np.arange(40, dtype=np.int32) % 64
    pair = _pair(p, [], dense=True, extra_img_ids=ids, ready_cap=50)
    try:
        g = pair.gpu
        rows = torch.ones((40, p.dfv_dim), device="cuda")
        ids_t = torch.from_numpy(ids).cuda()
        g.accumulate_rows(ids_t, rows)
        g.accumulate_rows(ids_t, rows)                      # 80 > 50: dropped whole
        rc, status, pending = g.status()
        assert pending == 40 and status & gb.GEAR_DEV_READY_OVERFLOW and rc == gb.GEAR_ERR_CAPACITY
        assert g.collect_ready() == 40
    finally:
        pair.close()


def test_bad_arguments_are_refused_on_the_host(gb):
    p = PRESETS["tiny"]
    cfg = gb.make_config(p.user_vocab, p.url_vocab, p.img_vocab, 15, p.dfv_dim, 0, 0, [64], 4, 0, 16, 64)
    with pytest.raises(gb.GearError) as e:
        gb.gear_workspace_bytes(cfg)
    assert e.value.code == gb.GEAR_ERR_ARG
    b = _manual_batch([3], [4], [[8]], [1])
    _, pair = _tiny_pair([b])
    try:
        g = pair.gpu
        from paper_1806_03925_b200.session import DeviceBatch
        big = BatchSource(PRESETS["tiny"].scaled(user_vocab=500, url_vocab=400, img_vocab=300), 0).batch(0, 64)
        with pytest.raises(gb.GearError):
            g.forward_backward(DeviceBatch.from_host(big))          # B > max_batch
    finally:
        pair.close()


# ------------------------------------------------------------------ full size: the large-table configuration
def test_large_tables_full_size_sampled(gb):
    """The 48.9 GB large-table configuration as bench.py runs it.  The oracle cannot run 65536 views
    through the head in seconds, so it checks (a) the gather, forward and per-view backward of a sample
    of views (per-view results do not depend on the other views except through the 1/B factor),
    (b) the full-size accumulate / collect on procedurally generated gradient rows, (c) the expiry scan."""
    from gpu_harness import assert_close, _np, Remap, TOL_BF16
    from oracle import GearOracle
    from paper_1806_03925_b200.session import DeviceBatch, GearSession
    free, _ = torch.cuda.mem_get_info()
    if free < 70 * 2**30:
        pytest.skip("needs about 60 GB of device memory")
    p = PRESETS["large"]
    src = BatchSource(p, 0)
    b = src.batch(0)
    params = workloads.head_params(p, 0)
    g = GearSession(p, params, seed=0, fill=True, now=0, want_debug=True)
    try:
        db = DeviceBatch.from_host(b)
        g.forward_backward(db, lr=0.0)                      # lr 0: tables stay as generated
        # (a) sample of views
        rng = np.random.default_rng(0)
        views = np.sort(rng.choice(b.B, 384, replace=False))
        n_b = np.diff(b.img_off)
        off_s = np.concatenate([[0], np.cumsum(n_b[views])]).astype(np.int32)
        img_s = np.concatenate([b.img_id[b.img_off[v]:b.img_off[v + 1]] for v in views])
        ru, rh, ri = (Remap(b.user_id[views], p.user_vocab, False), Remap(b.url_id[views], p.url_vocab, False),
                      Remap(img_s, p.img_vocab, False))
        cpu = GearOracle(oracle.fill_rows(0, oracle.TAG_USER, p.emb_dim, ru.rows, ru.n, np.float32),
                         oracle.fill_rows(0, oracle.TAG_URL, p.emb_dim, rh.rows, rh.n, np.float32),
                         oracle.fill_rows(0, oracle.TAG_DFV, p.dfv_dim, ri.rows, ri.n, np.uint16),
                         p.hidden, p.M, p.expire, round_bf16=True)
        r = cpu.forward_backward(params.astype(np.float64), ru(b.user_id[views]), rh(b.url_id[views]), off_s,
                                 ri(img_s), b.label[views])
        vt = torch.from_numpy(views).cuda()
        X = _np(g.x_debug[vt])
        E = p.emb_dim
        assert np.array_equal(X[:, :2 * E].astype(np.float64), r.X[:, :2 * E])
        one = n_b[views] == 1
        assert np.array_equal(X[one, 2 * E:].astype(np.float64), r.X[one, 2 * E:])
        assert_close(X, r.X, TOL_BF16, "head input")
        assert_close(_np(g.prob[vt]), r.prob, TOL_BF16, "prob")
        assert_close(_np(g.dX[vt]) * (b.B / len(views)), r.dX, TOL_BF16, "dX of the sampled views")
        assert np.isfinite(g.loss.item()) and abs(g.loss.item() - np.log(2)) < 0.5
        # (b) full-size accumulate on procedural rows, twice, then collect
        n, D = b.nnz, p.dfv_dim
        grads = torch.empty((n, D), dtype=torch.float32, device="cuda")
        gb.gear_fill_uniform(grads, seed=9, tag=gb.GEAR_TAG_GRAD, amp=1.0)
        g_cpu = oracle.fill_rows(9, oracle.TAG_GRAD, D, None, n, np.float32, amp=1.0).astype(np.float64)
        ria = Remap(b.img_id, p.img_vocab, False)
        acc = GearOracle(np.zeros((1, 4), np.float32), np.zeros((1, 4), np.float32), np.zeros((ria.n, D), np.float32),
                         (8,), p.M, p.expire, ts=oracle.fill_ts(0, p.expire, 0, None, p.img_vocab))
        ids_c = ria(b.img_id)
        rows_t = torch.from_numpy(ria.rows).cuda()
        for _ in range(2):
            g.accumulate_rows(db.img_id, grads)
            acc.accumulate(ids_c, g_cpu)
            assert np.array_equal(_np(g.dfv_gcnt[rows_t]), acc.gcnt)
        assert int(g.dfv_gcnt.sum().item()) == int(acc.gcnt.sum())
        assert_close(_np(g.dfv_gsum[rows_t]), acc.gsum, 1e-5, "open-group sums")
        n_ready = g.collect_ready()
        eid, eseq, eavg = oracle.sort_emissions(*acc.collect_ready())
        assert n_ready == len(eid)
        assert np.array_equal(ria(_np(g.ready_ids[:n_ready])), eid)
        assert np.array_equal(_np(g.ready_seq[:n_ready]), eseq)
        assert_close(_np(g.ready_avg[:n_ready]), eavg, 1e-5, "averaged gradients")
        # (c) expiry over all 20M timestamps
        for now in (1, 2, 60):
            k = g.collect_expired(now, True)
            want = acc.collect_expired(now, True)
            assert k == len(want) and np.array_equal(_np(g.expired_ids[:k]), want)
        assert g.status()[1] == 0
    finally:
        g.close()


# ------------------------------------------------------------------ the whole step, expiry scan on a second stream
def test_step_with_expiry_on_its_own_stream_matches_step_on_one_stream(gb):
    """GearSession.step forks the expiry scan onto a stream of its own and joins it at the step's end; the
    results must be those of the same calls issued one after the other on one stream.  With every timestamp 0
    and expire 3 the scan must list every image at now = 3 and, after the restamp, again at now = 6."""
    from gpu_harness import assert_close, _np
    from paper_1806_03925_b200.session import DeviceBatch, GearSession
    p = PRESETS["medium"].scaled(batch=2048, user_vocab=50_000, url_vocab=50_000, img_vocab=300_001, expire=3, M=4)
    src = BatchSource(p, 3)
    batches = [src.batch(s) for s in range(7)]
    max_nnz = max(b.nnz for b in batches)
    sessions = [GearSession(p, workloads.head_params(p, 3), max_batch=p.batch, max_nnz=max_nnz, seed=3, fill=True, now=0,
                            expired_cap=p.img_vocab) for _ in range(2)]
    try:
        for sess in sessions:
            sess.dfv_ts.zero_()
        torch.cuda.synchronize()
        for s, b in enumerate(batches):
            now = s + 1
            out = []
            for sess, beside in zip(sessions, (False, True)):
                n_ready, n_exp = sess.step(DeviceBatch.from_host(b), now, sync=True, expiry_beside=beside)
                torch.cuda.synchronize()
                out.append((n_ready, n_exp, _np(sess.ready_ids[:n_ready]), _np(sess.ready_seq[:n_ready]),
                            _np(sess.ready_avg[:n_ready]), _np(sess.expired_ids[:n_exp]), _np(sess.loss)))
            a, c = out
            assert a[0] == c[0] and a[1] == c[1], (now, a[:2], c[:2])
            assert np.array_equal(a[2], c[2]) and np.array_equal(a[3], c[3]) and np.array_equal(a[5], c[5])
            assert_close(c[4], a[4], 1e-5, "averaged gradients")
            assert_close(c[6], a[6], 1e-5, "loss")
            want_all = now in (3, 6)
            assert c[1] == (p.img_vocab if want_all else 0), (now, c[1])
            if want_all:
                assert np.array_equal(c[5], np.arange(p.img_vocab, dtype=np.int32))
        assert torch.equal(sessions[0].dfv_ts, sessions[1].dfv_ts)
        assert int(sessions[1].dfv_ts.min().item()) == 6 and int(sessions[1].dfv_ts.max().item()) == 6
        for sess in sessions:
            assert sess.status()[1] == 0
    finally:
        for sess in sessions:
            sess.close()


def test_profiling_modes_leave_the_results_alone(gb):
    """Per-kernel timing (every kernel alone on the caller's stream) and the timeline mode (the side stream stays)
    bracket the same launches with events: the step's outputs are those of an unprofiled step, bit for bit where the
    sums are taken in a fixed order, and the timeline lists every launch once, each with stop >= start >= 0."""
    from gpu_harness import assert_close, _np
    from paper_1806_03925_b200.session import DeviceBatch, GearSession
    p = PRESETS["medium"].scaled(batch=2048, user_vocab=50_000, url_vocab=50_000, img_vocab=300_001, M=4)
    src = BatchSource(p, 5)
    batches = [src.batch(s) for s in range(3)]
    max_nnz = max(b.nnz for b in batches)
    sessions = [GearSession(p, workloads.head_params(p, 5), max_batch=p.batch, max_nnz=max_nnz, seed=5, fill=True, now=0,
                            expired_cap=p.img_vocab) for _ in range(3)]
    try:
        gb.gear_profile_enable(sessions[1].ctx, True)
        gb.gear_profile_enable(sessions[2].ctx, 2)
        for s, b in enumerate(batches):
            out = []
            before = [gb.gear_launch_count(sess.ctx) for sess in sessions]
            for sess in sessions:
                n_ready, n_exp = sess.step(DeviceBatch.from_host(b), s + 1, sync=True, expiry_beside=False)
                torch.cuda.synchronize()
                out.append((n_ready, n_exp, _np(sess.ready_ids[:n_ready]), _np(sess.ready_seq[:n_ready]),
                            _np(sess.ready_avg[:n_ready]), _np(sess.loss), _np(sess.head_grad), _np(sess.prob)))
            launches = [gb.gear_launch_count(sess.ctx) - n0 for sess, n0 in zip(sessions, before)]
            assert launches[0] == launches[1] == launches[2] > 0
            for c in out[1:]:
                a = out[0]
                assert a[0] == c[0] and a[1] == c[1]
                assert np.array_equal(a[2], c[2]) and np.array_equal(a[3], c[3]) and np.array_equal(a[7], c[7])
                assert_close(c[4], a[4], 1e-5, "averaged gradients")
                assert_close(c[5], a[5], 1e-5, "loss")
                assert_close(c[6], a[6], 1e-4, "head gradient")          # split sums arrive in any order
            per_kernel = gb.gear_profile_read(sessions[1].ctx, 64)
            assert sum(v[1] for v in per_kernel.values()) == launches[1]
            assert all(v[0] >= 0.0 for v in per_kernel.values())
            timeline = gb.gear_profile_timeline(sessions[2].ctx, 256)
            assert len(timeline) == launches[2]
            assert sorted(k for k, _, _ in timeline) == sorted(k for k, v in per_kernel.items() for _ in range(v[1]))
            assert all(t1 >= t0 >= 0.0 for _, t0, t1 in timeline)
            assert gb.gear_profile_timeline(sessions[2].ctx, 256) == []         # reading clears the records
        for sess in sessions:
            assert sess.status()[1] == 0
    finally:
        for sess in sessions:
            sess.close()


# ------------------------------------------------------------------ refresh of cached DFVs
@pytest.mark.parametrize("name", ["tiny", "medium"])
def test_refresh_dfv_matches_oracle(gb, name):
    """Rows, timestamps and the skipped-ID flag, bit for bit; fp32 table (tiny) and bf16 table (medium); source rows
    with a leading dimension wider than the row; the device-side count bounds the call."""
    from gpu_harness import _np
    p = PRESETS[name].scaled(img_vocab=60_000) if name == "medium" else PRESETS[name]
    rng = np.random.default_rng(5)
    n = 3000
    ids = rng.choice(p.img_vocab, n, replace=False).astype(np.int32)
    ids[17], ids[1234] = -3, p.img_vocab                     # skipped, flagged
    rows = rng.normal(0, 1, (n + 100, p.dfv_dim + 12)).astype(np.float32)
    rows[5, :4] = [1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -0.0, 3.0e38]      # bf16 ties and edge values
    pair = _pair(p, [], seed=2, dense=True)
    g, cpu = pair.gpu, pair.cpu
    try:
        d_ids, d_rows = torch.from_numpy(ids).cuda(), torch.from_numpy(rows).cuda()
        view = d_rows[:, :p.dfv_dim]                                          # ld = dfv_dim + 12
        # first call: everything; second call: capacity n, the device count says 1000 (other rows, other time)
        g.refresh_dfv(d_ids, view, now=77)
        assert cpu.refresh_dfv(ids, rows[:n, :p.dfv_dim], now=77) == 2
        d_n = torch.tensor([1000], dtype=torch.int64, device="cuda")
        g.refresh_dfv(d_ids, view[100:], now=90, n=n, d_n=d_n)
        assert cpu.refresh_dfv(ids[:1000], rows[100:1100, :p.dfv_dim], now=90) == 1
        got = g.dfv.view(torch.int16).cpu().numpy().view(np.uint16) if p.dfv_dtype == BF16 else _np(g.dfv)
        assert np.array_equal(got, cpu.dfv)
        assert np.array_equal(_np(g.dfv_ts), cpu.ts)
        assert not g.dfv_gsum.any().item() and not g.dfv_gcnt.any().item()
        rc, bits, _ = g.status()
        assert bits & gb.GEAR_DEV_BAD_ID
        # argument checks: misaligned rows, short leading dimension
        with pytest.raises(gb.GearError):
            gb.gear_refresh_dfv(g.ctx, d_ids, d_rows[:, 1:1 + p.dfv_dim], n, 5)
        # a refreshed image is gathered in its new form and not listed by the scan before now + expire
        k = g.collect_expired(90 + p.expire - 1, restamp=False)
        listed = set(_np(g.expired_ids[:k]).tolist())
        assert not (set(ids[:1000].tolist()) - {-3, p.img_vocab}) & listed
    finally:
        g.close()


def test_gear_loop_on_the_gpu_path_trains_a_linear_dense_part(gb):
    """The whole loop of the paper's Section 3 on the device, with the smallest Dense Part there is (DFV_i = raw_i . Wd):
    M = 1 and expiry 0, so every step the scan lists every image, gear_dense_forward recomputes every DFV from the current
    Wd, gear_refresh_dfv stores them, the step's averaged gradients go back through the Dense Part
    (gear_dense_backward: Eq. 1) and Wd takes an Adam step (gear_adam_dense, Section 4).  Three steps against the same
    loop on the oracle; no product, sum or optimiser arithmetic happens in the test."""
    from gpu_harness import _np, assert_close
    from oracle import AdamConfig
    from paper_1806_03925_b200.session import DeviceBatch
    p = PRESETS["tiny"].scaled(M=1, expire=0, img_vocab=512, batch=128)
    R = 24
    rng = np.random.default_rng(9)
    raw = rng.normal(0, 1, (p.img_vocab, R)).astype(np.float32)
    Wd0 = rng.normal(0, 0.3, (R, p.dfv_dim)).astype(np.float32)
    src = BatchSource(p, 4)
    batches = [src.batch(s) for s in range(3)]
    pair = _pair(p, batches, seed=4, dense=True)
    g, cpu = pair.gpu, pair.cpu
    acfg = AdamConfig(lr=2e-2, beta1=0.9, beta2=0.99, eps=1e-8)
    adam = gb.make_adam(acfg.lr, acfg.beta1, acfg.beta2, acfg.eps)
    try:
        d_raw = torch.from_numpy(raw).cuda()
        Wd = torch.from_numpy(Wd0.copy()).cuda()
        Wd_m, Wd_v, Wd_grad = torch.zeros_like(Wd), torch.zeros_like(Wd), torch.zeros_like(Wd)
        rows = torch.zeros((p.img_vocab, p.dfv_dim), device="cuda")
        Wc, mc, vc = Wd0.astype(np.float64), np.zeros(Wd0.shape), np.zeros(Wd0.shape)
        for step, b in enumerate(batches):
            now, t = step + 1, step + 1
            # --- device
            k = g.collect_expired(now, restamp=True)
            assert k == p.img_vocab
            g.dense_forward(d_raw, Wd, g.expired_ids, rows, n=p.img_vocab, d_n=g.d_counts[1:2])
            g.refresh_dfv(g.expired_ids, rows, now, n=p.img_vocab, d_n=g.d_counts[1:2])
            db = DeviceBatch.from_host(b)
            g.forward_backward(db, lr=0.0)
            n_ready = g.accumulate_collect_from_step(db)
            assert n_ready == b.nnz                                    # M = 1: every gradient row is handed over
            Wd_grad.zero_()
            g.dense_backward(d_raw, b.nnz, Wd_grad, d_n=g.d_counts[0:1])
            gb.gear_adam_dense(Wd, Wd_grad, Wd_m, Wd_v, t, adam)
            # --- oracle
            exp_c = cpu.collect_expired(now, restamp=True)
            cpu.refresh_dfv(exp_c, oracle.dense_forward(raw, Wc, exp_c).astype(np.float32), now)
            r = cpu.forward_backward(pair.params.astype(np.float64), b.user_id, b.url_id, b.img_off, b.img_id, b.label)
            cpu.accumulate(b.img_id, cpu.dfv_grad_rows(b.img_off, r.dX))
            cid, _, cavg = cpu.collect_ready()
            G_c = oracle.dense_backward(raw, cid, cavg)
            assert_close(_np(Wd_grad), G_c, 1e-5, "dense-part gradient of step %d" % step)
            oracle.adam_step(Wc, G_c, mc, vc, t, acfg)
            assert_close(_np(Wd) - Wd0, Wc - Wd0, 1e-4, "movement of the dense-part weights after step %d" % step)
            assert_close(_np(Wd_m), mc, 1e-5, "first moments")
            assert_close(_np(Wd_v), vc, 1e-5, "second moments")
            got = _np(g.dfv)
            assert_close(got, cpu.dfv, 1e-5, "refreshed DFV table")
        assert np.abs(Wc - Wd0).max() > 1e-2                           # the steps did move the weights
        assert g.status()[1] == 0
    finally:
        g.close()


def test_dense_part_calls_edge_cases(gb):
    """Ragged sizes on every side of the tiles, a device-side count below the capacity, a leading dimension wider than
    the row, an out-of-range ID (zero row / skipped, flagged), repeated IDs in the emission list."""
    from gpu_harness import _np, assert_close
    p = PRESETS["tiny"].scaled(user_vocab=64, url_vocab=64, img_vocab=1000, dfv_dim=72)
    pair = _pair(p, [], dense=True)
    g = pair.gpu
    try:
        rng = np.random.default_rng(31)
        R, n = 37, 333
        raw = rng.normal(0, 1, (p.img_vocab, R)).astype(np.float32)
        Wd = rng.normal(0, 0.3, (R, p.dfv_dim)).astype(np.float32)
        ids = rng.integers(0, p.img_vocab, n).astype(np.int32)
        ids[5] = p.img_vocab + 3
        ids[77] = ids[78] = ids[200]
        d_raw, d_Wd, d_ids = torch.from_numpy(raw).cuda(), torch.from_numpy(Wd).cuda(), torch.from_numpy(ids).cuda()
        rows = torch.full((n, p.dfv_dim + 8), 7.0, device="cuda")
        d_n = torch.tensor([300], dtype=torch.int64, device="cuda")
        gb.gear_dense_forward(g.ctx, d_raw, d_Wd, d_ids, n, rows[:, :p.dfv_dim], d_n=d_n)
        want = oracle.dense_forward(raw, Wd.astype(np.float64), ids[:300])
        assert_close(_np(rows[:300, :p.dfv_dim]), want, 1e-5, "dense forward")
        assert not _np(rows[5, :p.dfv_dim]).any()
        assert (_np(rows[300:]) == 7.0).all() and (_np(rows[:, p.dfv_dim:]) == 7.0).all()       # nothing beyond the count / the row
        rc, bits, _ = g.status()
        assert bits & gb.GEAR_DEV_BAD_ID
        avg = rng.normal(0, 1, (n, p.dfv_dim)).astype(np.float32)
        G = torch.zeros((R, p.dfv_dim), device="cuda")
        gb.gear_dense_backward(g.ctx, d_raw, d_ids, torch.from_numpy(avg).cuda(), n, G, d_n=d_n)
        assert_close(_np(G), oracle.dense_backward(raw, ids[:300], avg[:300].astype(np.float64)), 1e-5, "dense backward")
        gb.gear_dense_backward(g.ctx, d_raw, d_ids, torch.from_numpy(avg).cuda(), n, G)          # adds to what is there
        want2 = oracle.dense_backward(raw, ids[:300], avg[:300].astype(np.float64)) + oracle.dense_backward(raw, ids, avg.astype(np.float64))
        assert_close(_np(G), want2, 1e-5, "dense backward, accumulated")
        g.status()
    finally:
        pair.close()


@pytest.mark.parametrize("name", ["tiny", "medium"])
def test_adam_on_the_embedding_rows_and_the_head(gb, name):
    """Section 4's optimiser through the library: the embedding rows a step touches (the adam fields of gear_step_out)
    and the head's parameters (gear_adam_dense on head_grad) against the oracle, three steps, so that the second and
    third start from non-zero moments and revisit rows.  Tables, both moment tables and the parameters are compared.

    The moments are linear / quadratic in the gradient and are held to the configuration's tolerance.  The step itself
    divides by sqrt(v) + eps, which turns a gradient entry's RELATIVE error into an error of the step: an entry far
    below the largest one carries an absolute error of tol * max|g| like every other, so its sign and size, and with
    them its step, are only as good as tol * max|g| / (|g| + eps).  The fp32 configuration runs with the usual
    eps = 1e-8 (entry errors around 1e-10: steps good to 1e-2 of the learning rate in the worst entry); the bf16
    configuration, whose gradient entries are good to about 1e-6, with eps = 1e-4, which keeps the same bound."""
    from gpu_harness import _np, _rows, assert_close, Remap, tol_of
    from oracle import AdamConfig, GearOracle
    from paper_1806_03925_b200.session import DeviceBatch, GearSession
    p = PRESETS[name].scaled(user_vocab=3000, url_vocab=2000, img_vocab=5000, batch=1500)
    tol = tol_of(p)
    acfg = AdamConfig(lr=1e-2, beta1=0.9, beta2=0.99, eps=1e-8 if p.head_dtype == F32 else 1e-4)
    step_tol = 2e-2 if p.head_dtype == F32 else 5e-2          # of the largest movement, which is about lr
    adam = gb.make_adam(acfg.lr, acfg.beta1, acfg.beta2, acfg.eps)
    src = BatchSource(p, 6)
    batches = [src.batch(s) for s in range(3)]
    params = workloads.head_params(p, 6)
    g = GearSession(p, params, max_batch=p.batch, max_nnz=max(b.nnz for b in batches), seed=6, fill=True, adam=adam)
    dfv_np = np.uint16 if p.dfv_dtype == BF16 else np.float32
    cpu = GearOracle(oracle.fill_rows(6, oracle.TAG_USER, p.emb_dim, None, p.user_vocab, np.float32),
                     oracle.fill_rows(6, oracle.TAG_URL, p.emb_dim, None, p.url_vocab, np.float32),
                     oracle.fill_rows(6, oracle.TAG_DFV, p.dfv_dim, None, p.img_vocab, dfv_np),
                     p.hidden, p.M, p.expire, round_bf16=(p.head_dtype == BF16))
    try:
        u0, h0 = cpu.user_emb.copy(), cpu.url_emb.copy()
        mom = {k: np.zeros(t.shape) for k, t in (("um", u0), ("uv", u0), ("hm", h0), ("hv", h0))}
        pc, pm, pv = params.astype(np.float64), np.zeros(len(params)), np.zeros(len(params))
        hp_m, hp_v = torch.zeros_like(g.head_params), torch.zeros_like(g.head_params)
        for step, b in enumerate(batches):
            t = step + 1
            g.forward_backward(DeviceBatch.from_host(b))
            gb.gear_adam_dense(g.head_params, g.head_grad, hp_m, hp_v, t, adam)
            r = cpu.forward_backward(pc.copy(), b.user_id, b.url_id, b.img_off, b.img_id, b.label)
            assert_close(_np(g.head_grad), r.head_grad, tol, "head_grad of step %d" % step)
            oracle.emb_adam(cpu.user_emb, mom["um"], mom["uv"], b.user_id, r.dX, 0, t, acfg)
            oracle.emb_adam(cpu.url_emb, mom["hm"], mom["hv"], b.url_id, r.dX, p.emb_dim, t, acfg)
            oracle.adam_step(pc, r.head_grad, pm, pv, t, acfg)
            # what moved, against what should have moved (the tables themselves are 0.17 wide, a step 0.01)
            assert_close(_np(g.user_emb) - u0, cpu.user_emb.astype(np.float64) - u0, step_tol, "user table movement")
            assert_close(_np(g.url_emb) - h0, cpu.url_emb.astype(np.float64) - h0, step_tol, "url table movement")
            assert_close(_np(g.user_m), mom["um"], tol, "user first moments")
            assert_close(_np(g.user_v), mom["uv"], tol, "user second moments")
            assert_close(_np(g.url_m), mom["hm"], tol, "url first moments")
            assert_close(_np(g.url_v), mom["hv"], tol, "url second moments")
            assert_close(_np(g.head_params) - params, pc - params, step_tol, "head parameter movement")
            # rows no view named stay bit for bit, moments included
            idle = np.setdiff1d(np.arange(p.user_vocab), np.concatenate([x.user_id for x in batches[:step + 1]]))
            assert np.array_equal(_np(g.user_emb)[idle], u0[idle]) and not _np(g.user_m)[idle].any() and not _np(g.user_v)[idle].any()
        assert g.status()[1] == 0
    finally:
        g.close()


# ------------------------------------------------------------------ tables partitioned by ID over several ranks
@pytest.mark.parametrize("name,world", [("tiny", 2), ("tiny", 3), ("medium", 2)])
def test_step_with_tables_partitioned_by_id(gb, name, world):
    """Every rank holds the table rows whose ID is congruent to its rank and works on its own page views: IDs travel
    to the owners, rows come back, gradient rows travel to the owners (paper, Section 3: "by partition of Image ID").
    All ranks run in this process, one after the other, over an in-process exchange (no kernel of one rank waits for
    another's), and the result is compared with the oracle doing the same thing on whole tables: every worker's
    forward and backward pass on the tables as they stood at the start of the step, then all embedding gradients
    applied, then all (Image ID, gradient) pairs fed to the store rank by rank in row order.  Two steps."""
    from gpu_harness import _np, assert_close, tol_of
    from oracle import GearOracle
    from paper_1806_03925_b200.sharded import LoopbackExchange, ShardedGear
    p = PRESETS[name].scaled(user_vocab=1501, url_vocab=1200, img_vocab=2003, batch=700, expire=3)
    tol = tol_of(p)
    dfv_np = np.uint16 if p.dfv_dtype == BF16 else np.float32
    tables = dict(user_emb=oracle.fill_rows(2, oracle.TAG_USER, p.emb_dim, None, p.user_vocab, np.float32),
                  url_emb=oracle.fill_rows(2, oracle.TAG_URL, p.emb_dim, None, p.url_vocab, np.float32),
                  dfv=oracle.fill_rows(2, oracle.TAG_DFV, p.dfv_dim, None, p.img_vocab, dfv_np),
                  ts=oracle.fill_ts(2, p.expire, 0, None, p.img_vocab))
    params = workloads.head_params(p, 2)
    src = BatchSource(p, 2)
    # rank r takes batches r, world + r, ... ; the ranks' batches differ in size
    sizes = [p.batch - 37 * r for r in range(world)]
    steps = [[src.batch(s * world + r, sizes[r]) for r in range(world)] for s in range(2)]
    sg = ShardedGear(p, params, LoopbackExchange(world), max_batch_local=p.batch, max_nnz_local=p.batch * p.img_hi,
                     tables=tables)
    cpu = GearOracle(tables["user_emb"].copy(), tables["url_emb"].copy(), tables["dfv"].copy(), p.hidden, p.M, p.expire,
                     round_bf16=(p.head_dtype == BF16), ts=tables["ts"].copy())

    def gather_shards(attr):
        out = None
        for r, ow in enumerate(sg.owners):
            t = _np(getattr(ow, attr))
            if out is None:
                out = np.zeros((getattr(p, {"user_emb": "user_vocab", "url_emb": "url_vocab"}.get(attr, "img_vocab")),) + t.shape[1:], t.dtype)
            out[r::world] = t
        return out
    try:
        for s, batches in enumerate(steps):
            now = s + 1
            out = sg.step(batches, now, mean_head_grad=False)
            res = [cpu.forward_backward(params.astype(np.float64), b.user_id, b.url_id, b.img_off, b.img_id, b.label)
                   for b in batches]
            for wk, b, r in zip(sg.workers, batches, res):
                assert_close(_np(wk.loss), [r.loss], tol, "loss")
                assert_close(_np(wk.prob[:b.B]), r.prob, tol, "prob")
                assert_close(_np(wk.dX[:b.B]), r.dX, tol, "dX")
                assert_close(_np(wk.head_grad), r.head_grad, tol, "head_grad")
            uid = np.concatenate([b.user_id for b in batches]); hid = np.concatenate([b.url_id for b in batches])
            dX = np.concatenate([r.dX for r in res])
            cpu.emb_apply("user", uid, dX, -p.lr)
            cpu.emb_apply("url", hid, dX, -p.lr)
            assert_close(gather_shards("user_emb"), cpu.user_emb, tol, "user table")
            assert_close(gather_shards("url_emb"), cpu.url_emb, tol, "url table")
            img = np.concatenate([b.img_id for b in batches])
            rows = np.concatenate([cpu.dfv_grad_rows(b.img_off, r.dX) for b, r in zip(batches, res)])
            cpu.accumulate(img, rows)
            assert np.array_equal(gather_shards("dfv_gcnt"), cpu.gcnt), "open-group counts"
            assert_close(gather_shards("dfv_gsum"), cpu.gsum, tol, "open-group sums")
            eid, eseq, eavg = oracle.sort_emissions(*cpu.collect_ready())
            got = []
            for r, (ow, (n_ready, _)) in enumerate(zip(sg.owners, out)):
                got.append((_np(ow.ready_ids[:n_ready]).astype(np.int64) * world + r, _np(ow.ready_seq[:n_ready]),
                            _np(ow.ready_avg[:n_ready])))
            gid = np.concatenate([g[0] for g in got]); gseq = np.concatenate([g[1] for g in got])
            gavg = np.concatenate([g[2] for g in got])
            order = np.lexsort((gseq, gid))
            assert np.array_equal(gid[order], eid) and np.array_equal(gseq[order], eseq), "emitted (id, seq) pairs"
            assert_close(gavg[order], eavg, tol, "averaged gradients")
            want_exp = cpu.collect_expired(now, True)
            got_exp = np.sort(np.concatenate([_np(ow.expired_ids[:n_exp]).astype(np.int64) * world + r
                                              for r, (ow, (_, n_exp)) in enumerate(zip(sg.owners, out))]))
            assert np.array_equal(got_exp, want_exp), "expired ids"
            assert np.array_equal(gather_shards("dfv_ts"), cpu.ts)
        assert sum(n for n, _ in out) > 0
        for s_ in sg.owners + sg.workers:
            assert s_.status()[1] == 0
        # the head's gradient averaged over the ranks, as the collective would leave it on every rank
        want = np.mean([r.head_grad for r in res], axis=0)
        sg.ex.mean_over_ranks([wk.head_grad for wk in sg.workers])
        for wk in sg.workers:
            assert_close(_np(wk.head_grad), want, tol, "head_grad, mean over the ranks")
    finally:
        sg.close()
