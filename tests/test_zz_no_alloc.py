"""gear_collect_expired_static: the expiry scan for callers that cannot allocate device memory.

Some users of libgear run where cudaMalloc is not theirs to call (a serving process with a fixed memory
plan, a plug-in that is only handed buffers), so they cannot give a gear_ctx its workspace.  This entry
point keeps its scratch in a fixed array inside the library instead.  The test calls it through the C ABI,
twice in a row on the same table, and checks each result against the ctx-based gear_collect_expired on an
identical copy of the table and against the CPU oracle's scan of the same timestamps: ID lists and restamped
timestamps must be bit-identical (integer work, so the tolerance is zero, as in the other expiry tests).  The
second call runs on whatever the first one left in the shared scratch and finds a different, smaller set of
expired images.

This file sorts last on purpose: a run that stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

from paper_1806_03925_b200 import workloads
from paper_1806_03925_b200.workloads import PRESETS

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gb():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_1806_03925_b200 import binding
    binding.load()
    return binding


def test_static_expiry_scan_matches_the_ctx_based_scan_twice_in_a_row(gb):
    from paper_1806_03925_b200.session import GearSession
    V, T = 300_007, 50                                     # several 8192-entry tiles and a ragged tail
    p = PRESETS["tiny"].scaled(user_vocab=64, url_vocab=64, img_vocab=V, expire=T)
    ts0 = workloads.timestamps(V, T, seed=4, now=0)
    tables = dict(user_emb=np.zeros((64, p.emb_dim), np.float32), url_emb=np.zeros((64, p.emb_dim), np.float32),
                  dfv=np.zeros((V, p.dfv_dim), np.float32), ts=ts0.copy())
    ref = GearSession(p, workloads.head_params(p, 0), max_batch=8, max_nnz=32, tables=tables)
    from oracle import GearOracle
    cpu = GearOracle(tables["user_emb"], tables["url_emb"], np.zeros((1, p.dfv_dim), np.float32), p.hidden, p.M, T,
                     ts=ts0.copy())
    try:
        ts = torch.from_numpy(ts0.copy()).cuda()
        ids = torch.full((V,), -1, dtype=torch.int32, device="cuda")
        d_n = torch.zeros(1, dtype=torch.int64, device="cuda")
        seen = []
        for now in (7, 30):                                # two calls in a row share the library's scratch
            n_ref = ref.collect_expired(now, restamp=True)
            n = gb.gear_collect_expired_static(ts, T, now, True, ids, V, d_n=d_n)
            assert n == n_ref and int(d_n.item()) == n_ref
            assert torch.equal(ids[:n], ref.expired_ids[:n])
            assert torch.equal(ts, ref.dfv_ts)
            want = cpu.collect_expired(now, restamp=True)
            assert n == len(want) and np.array_equal(ids[:n].cpu().numpy(), want)
            assert np.array_equal(ts.cpu().numpy(), cpu.ts)
            seen.append(n)
        assert seen[0] > 0 and seen[1] > 0 and seen[0] != seen[1]
        # without restamping, and with the count read from the device only
        n_ref = ref.collect_expired(60, restamp=False)
        assert gb.gear_collect_expired_static(ts, T, 60, False, ids, V, d_n=d_n, sync=False) is None
        assert int(d_n.item()) == n_ref and torch.equal(ids[:n_ref], ref.expired_ids[:n_ref])
        assert torch.equal(ts, ref.dfv_ts)
        assert np.array_equal(ids[:n_ref].cpu().numpy(), cpu.collect_expired(60, restamp=False))
    finally:
        ref.close()


def test_static_expiry_scan_limits(gb):
    ts = torch.zeros(1000, dtype=torch.int64, device="cuda")
    ids = torch.zeros(1000, dtype=torch.int32, device="cuda")
    # a table beyond the fixed scratch is refused on the host, before any kernel is enqueued
    with pytest.raises(gb.GearError) as e:
        gb.gear_collect_expired_static(ts, 0, 5, True, ids, 1000, img_vocab=gb.GEAR_STATIC_EXPIRY_MAX_VOCAB + 1)
    assert e.value.code == gb.GEAR_ERR_CAPACITY
    # a list that is too short: nothing listed, nothing restamped, the required count is reported
    before = ts.clone()
    d_n = torch.zeros(1, dtype=torch.int64, device="cuda")
    with pytest.raises(gb.GearError) as e:
        gb.gear_collect_expired_static(ts, 0, 5, True, ids, 10, d_n=d_n)
    assert e.value.code == gb.GEAR_ERR_CAPACITY and int(d_n.item()) == 1000
    assert torch.equal(ts, before)
    assert gb.gear_collect_expired_static(ts, 0, 5, True, ids, 1000) == 1000     # the next call is unaffected
    assert torch.equal(ids, torch.arange(1000, dtype=torch.int32, device="cuda"))
