"""GPU-vs-oracle parity at the full sizes of the large-table, skew-stress and accumulate-only configurations,
through the C ABI, in the launch configuration the benchmark times (run with -m gpu on a B200).

The oracle works on a compact problem where the tables are too large for the host: only the rows the batches touch
are generated (each side from its own implementation of the procedural fill) and IDs are renumbered; GPU results are
read back at those rows.  Tolerances and bit-exact items are those of test_gpu_parity.py.
"""
import numpy as np
import pytest
import torch

import oracle
from oracle import GearOracle
from paper_1806_03925_b200 import workloads
from paper_1806_03925_b200.workloads import MICRO_PRESETS, PRESETS, BatchSource

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gb():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_1806_03925_b200 import binding
    binding.load()
    return binding


def _need_device_memory(gib: float):
    free, _ = torch.cuda.mem_get_info()
    if free < gib * 2**30:
        pytest.skip("needs about %.0f GiB of free device memory" % gib)


# ------------------------------------------------------------------ large tables: the whole 65536-view batch
def test_large_tables_whole_batch_two_steps(gb):
    """Every output of two consecutive steps of the 48.9 GB configuration against the oracle run on all 65536 views:
    head input, probabilities, loss, head gradients, dX; step 0 with the embedding gradients exported (tables
    untouched), step 1 with the in-place update (lr != 0); in both the accumulate call fed by the step's own dX
    through the plan made ahead during gear_forward_backward, the hand-over of the completed groups and the expiry
    scan of all 20M timestamps.  Step 1 starts from the sums and counts step 0 left."""
    from gpu_harness import Pair, max_views_with_flips
    _need_device_memory(95)
    p = PRESETS["large"]
    src = BatchSource(p, 0)
    batches = [src.batch(0), src.batch(1)]
    pair = Pair(p, batches, seed=0, dense=False, want_emb_grad=True, fused=True)    # the calls bench.py times
    try:
        out0 = pair.step_and_compare(batches[0], now=1)
        # from here on the library updates the tables in place
        g = pair.gpu
        g.user_grad = g.url_grad = None
        g._step_out = None
        pair.want_emb_grad = False
        torch.cuda.empty_cache()
        out1 = pair.step_and_compare(batches[1], now=2)
        for out in (out0, out1):
            assert out["status"] == 0 and out["n_ready"] > 1000 and out["n_expired"] > 0
            assert out["relu"]["views"] <= max_views_with_flips(p.batch)
        assert out1["n_ready"] > out0["n_ready"]            # open groups of step 0 complete in step 1
    finally:
        pair.close()


# ------------------------------------------------------------------ skew stress at full size
@pytest.mark.parametrize("M", [1, 64, 1024])
@pytest.mark.parametrize("atomic", [False, True])
def test_skew_config_full_size(gb, M, atomic):
    """B = 32768, 4M images, Zipf 1.3 (the top image alone receives about a quarter of the gradient rows), fp32
    DFVs and head; sorted and atomic accumulation; two steps."""
    from gpu_harness import Pair
    _need_device_memory(12)
    p = PRESETS["skew"].scaled(M=M)
    src = BatchSource(p, 0)
    batches = [src.batch(s) for s in range(2)]
    pair = Pair(p, batches, seed=0, dense=False, atomic=atomic, fused=(M == 64))
    try:
        outs = [pair.step_and_compare(b, now=s + 1) for s, b in enumerate(batches)]
        assert all(o["status"] == 0 for o in outs)
        top = np.bincount(pair.ri(batches[0].img_id)).max()
        assert top > 0.15 * batches[0].nnz                  # the contention the configuration is about
        if M == 1:
            assert outs[0]["n_ready"] == batches[0].nnz
        if M == 64:
            assert outs[0]["n_ready"] >= top // 64
    finally:
        pair.close()


# ------------------------------------------------------------------ accumulate-only micro-benchmark at full size
def _assert_close_chunked(get_rows, want: np.ndarray, tol: float, what: str, step: int = 1 << 18):
    """max |got - want| <= tol * max |want| over a tall array, read back from the device in pieces."""
    scale = max(float(np.abs(want).max()), 1e-30) if want.size else 1.0
    for lo in range(0, want.shape[0], step):
        hi = min(lo + step, want.shape[0])
        err = float(np.abs(get_rows(lo, hi).astype(np.float64) - want[lo:hi]).max())
        assert err <= tol * scale, "%s rows %d..%d: max abs error %.3e > %.1e * %.3e" % (what, lo, hi, err, tol, scale)


@pytest.mark.parametrize("name", sorted(MICRO_PRESETS))
def test_accumulate_only_full_size(gb, name):
    """2^24 gradient rows of 128 floats into a 2^22-image store, then the hand-over of the completed groups: counts,
    emitted IDs and emission numbers bit for bit, open-group sums and averages to 1e-5.  The oracle takes the rows in
    pieces of 2^20 (same arrival order), so that the host never holds all 8.6 GB of them."""
    from paper_1806_03925_b200.session import GearSession
    _need_device_memory(20)
    mp = MICRO_PRESETS[name]
    n, V, D, M = mp.n_rows, mp.img_vocab, mp.dfv_dim, mp.M
    ids = workloads.micro_ids(mp, seed=0)
    k = np.bincount(ids, minlength=V)
    n_emit = int((k // M).sum())
    p = PRESETS["skew"].scaled(img_vocab=V, dfv_dim=D, M=M, user_vocab=64, url_vocab=64, expire=1 << 40)
    g = GearSession(p, np.zeros(p.n_params, np.float32), max_batch=8, max_nnz=n, ready_cap=n_emit + 8, fill=True,
                    expired_cap=1)
    # the oracle's store; its DFV table is never read here (bf16 zeros: untouched pages cost nothing)
    cpu = GearOracle(np.zeros((1, 4), np.float32), np.zeros((1, 4), np.float32), np.zeros((V, D), np.uint16), (8,), M,
                     p.expire)
    try:
        grads = torch.empty((n, D), dtype=torch.float32, device="cuda")
        gb.gear_fill_uniform(grads, seed=5, tag=gb.GEAR_TAG_GRAD, amp=1.0)
        g.accumulate_rows(torch.from_numpy(ids).cuda(), grads)
        del grads
        step = 1 << 20
        for lo in range(0, n, step):
            hi = min(lo + step, n)
            rows = oracle.fill_rows(5, oracle.TAG_GRAD, D, np.arange(lo, hi, dtype=np.int64), hi - lo, np.float32, amp=1.0)
            cpu.accumulate(ids[lo:hi], rows.astype(np.float64))
        assert np.array_equal(g.dfv_gcnt.cpu().numpy(), cpu.gcnt), "open-group counts"
        _assert_close_chunked(lambda lo, hi: g.dfv_gsum[lo:hi].cpu().numpy(), cpu.gsum, 1e-5, "open-group sums")
        rc, status, pending = g.status()
        assert status == 0 and pending == n_emit == cpu.pending_ready
        assert g.collect_ready() == n_emit
        eid, eseq, eavg = oracle.sort_emissions(*cpu.collect_ready())
        assert np.array_equal(g.ready_ids[:n_emit].cpu().numpy(), eid), "emitted ids"
        assert np.array_equal(g.ready_seq[:n_emit].cpu().numpy(), eseq), "emission numbers"
        _assert_close_chunked(lambda lo, hi: g.ready_avg[lo:hi].cpu().numpy(), eavg, 1e-5, "averaged gradients")
        assert g.guards_intact()
        # conservation: M * emissions + what stays open = arrivals
        assert M * n_emit + int(g.dfv_gcnt.sum().item()) == n
        assert g.status()[1] == 0
    finally:
        g.close()
