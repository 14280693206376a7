"""Pins for the CPU oracle: every check here compares the oracle with something
other than itself -- finite differences, a reverse-mode autodiff library,
closed forms, a literal keep-every-gradient store, invariants the paper's
rules imply, and a published known-answer vector for the table-fill generator.

The paper (arXiv 1806.03925) prints no worked numeric example for this path.
"""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from oracle import GearOracle, sort_emissions

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------
# helpers
# ----------------------------------------------------------------------------
def small_problem(seed=0, B=4, E=3, D=4, hidden=(5,), Vu=6, Vh=5, Vi=7, max_imgs=3, dtype=np.float64):
    rng = np.random.default_rng(seed)
    user = rng.normal(0, 0.5, (Vu, E)).astype(dtype)
    url = rng.normal(0, 0.5, (Vh, E)).astype(dtype)
    dfv = rng.normal(0, 0.5, (Vi, D)).astype(dtype)
    n = rng.integers(1, max_imgs + 1, B)
    off = np.concatenate([[0], np.cumsum(n)]).astype(np.int32)
    batch = dict(user_id=rng.integers(0, Vu, B).astype(np.int32),
                 url_id=rng.integers(0, Vh, B).astype(np.int32),
                 img_off=off, img_id=rng.integers(0, Vi, off[-1]).astype(np.int32),
                 label=(rng.random(B) < 0.4).astype(np.float64))
    orc = GearOracle(user, url, dfv, hidden, M=1, expire=0)
    params = rng.normal(0, 0.6, orc.n_params)
    return orc, params, batch


def split_params(params, d_in, hidden):
    out, pos, fan = [], 0, d_in
    for h in hidden:
        out.append((params[pos:pos + fan * h].reshape(fan, h), params[pos + fan * h:pos + fan * h + h]))
        pos += fan * h + h
        fan = h
    return out, params[pos:pos + fan], params[pos + fan]


def loss_of(orc, params, batch):
    return orc.forward_backward(params, **batch, backward=False).loss


def central_diff(f, x, idx, h=1e-6):
    old = x.flat[idx]
    x.flat[idx] = old + h
    fp = f()
    x.flat[idx] = old - h
    fm = f()
    x.flat[idx] = old
    return (fp - fm) / (2 * h)


# ----------------------------------------------------------------------------
# table-fill generator and bf16 rounding
# ----------------------------------------------------------------------------
def test_splitmix64_known_answers():
    want = [int(l) for l in open(os.path.join(GOLDEN, "splitmix64_seed1234567.txt")) if l[0] != "#"]
    gamma, mask = 0x9E3779B97F4A7C15, (1 << 64) - 1
    got = [oracle.lib().orc_mix64((1234567 + (i + 1) * gamma) & mask) for i in range(len(want))]
    assert got == want


def test_fill_is_counter_based_and_in_range():
    full = oracle.fill_rows(7, oracle.TAG_DFV, 8, None, 50)
    rows = np.array([49, 3, 3, 17], dtype=np.int64)
    some = oracle.fill_rows(7, oracle.TAG_DFV, 8, rows, len(rows))
    assert np.array_equal(some, full[rows])                       # any row regenerates alone
    other = oracle.fill_rows(7, oracle.TAG_USER, 8, None, 50)
    assert not np.array_equal(full, other)                        # tables are independent streams
    big = oracle.fill_rows(1, oracle.TAG_USER, 64, None, 4096).astype(np.float64)
    assert np.all(np.abs(big) <= oracle.FILL_AMP)
    assert abs(big.std() - 0.1) < 2e-3 and abs(big.mean()) < 2e-3  # the paper's initial std 0.1
    # value = (top 24 bits - 2^23) * float(amp / 2^23), recomputed from the raw draw
    d = oracle.draw(7, oracle.TAG_DFV, 5 * 8 + 2)
    want = np.float32((d >> 40) - (1 << 23)) * np.float32(oracle.FILL_AMP / 8388608.0)
    assert full[5, 2] == want


def test_fill_ts_window():
    ts = oracle.fill_ts(3, expire=10, now=100, rows=None, n_rows=5000)
    assert ts.min() == 91 and ts.max() == 100
    counts = np.bincount(100 - ts, minlength=10)
    assert counts.min() > 400                                      # roughly uniform over the window
    assert np.array_equal(oracle.fill_ts(3, 0, 100, None, 10), np.full(10, 100))


def test_bf16_rounding_matches_library():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.normal(0, 1, 2000), rng.normal(0, 1e-3, 500), [0.0, 1.0, -1.0, 3.0],
                        # exact ties between two bf16 neighbours (round to even)
                        [1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -(2.0 + 2.0 ** -7)]]).astype(np.float32)
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()
    got = np.array([oracle.round_bf16(float(v)) for v in x])
    assert np.array_equal(got, want)
    # and the storage path: a bf16 table is read back exactly
    bits = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    orc = GearOracle(np.zeros((1, 1)), np.zeros((1, 1)), bits.reshape(-1, 1), (2,), 1, 0)
    params = np.zeros(orc.n_params)
    r = orc.forward_backward(params, [0], [0], [0, 1], [5], [0.0], backward=False)
    assert r.X[0, 2] == want[5]


# ----------------------------------------------------------------------------
# gather / pool
# ----------------------------------------------------------------------------
def test_gather_is_a_copy_and_single_image_pool_is_the_row():
    rng = np.random.default_rng(1)
    user = rng.normal(size=(9, 4)).astype(np.float32)
    url = rng.normal(size=(8, 4)).astype(np.float32)
    dfv = rng.normal(size=(11, 6)).astype(np.float32)
    orc = GearOracle(user, url, dfv, (3,), 1, 0)
    uid = np.array([8, 0, 3, 3], dtype=np.int32)
    hid = np.array([1, 7, 7, 2], dtype=np.int32)
    off = np.array([0, 1, 2, 3, 4], dtype=np.int32)
    img = np.array([10, 0, 4, 4], dtype=np.int32)
    r = orc.forward_backward(np.zeros(orc.n_params), uid, hid, off, img, np.zeros(4), backward=False)
    assert np.array_equal(r.X[:, 0:4], user[uid].astype(np.float64))
    assert np.array_equal(r.X[:, 4:8], url[hid].astype(np.float64))
    assert np.array_equal(r.X[:, 8:], dfv[img].astype(np.float64))


def test_pool_is_the_mean_with_repeats_and_empty_views():
    rng = np.random.default_rng(2)
    dfv = rng.normal(size=(5, 3))
    orc = GearOracle(np.zeros((2, 2)), np.zeros((2, 2)), dfv, (2,), 1, 0)
    off = np.array([0, 3, 3, 5], dtype=np.int32)          # view 1 has no image
    img = np.array([4, 4, 1, 0, 2], dtype=np.int32)       # image 4 twice in view 0
    r = orc.forward_backward(np.zeros(orc.n_params), [0, 1, 0], [1, 1, 0], off, img, np.zeros(3),
                             backward=False)
    np.testing.assert_allclose(r.X[0, 4:], (2 * dfv[4] + dfv[1]) / 3, rtol=1e-15)
    assert np.all(r.X[1, 4:] == 0.0)
    np.testing.assert_allclose(r.X[2, 4:], (dfv[0] + dfv[2]) / 2, rtol=1e-15)


def test_out_of_range_ids_are_counted_and_skipped():
    orc, params, batch = small_problem()
    batch["user_id"][1] = 99
    batch["img_id"][0] = -1
    r = orc.forward_backward(params, **batch)
    assert r.bad_ids == 2
    assert np.all(r.X[1, 0:3] == 0.0)


# ----------------------------------------------------------------------------
# head forward / backward
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("hidden", [(5,), (5, 4)])
def test_head_gradients_by_finite_differences(hidden):
    orc, params, batch = small_problem(seed=3, hidden=hidden)
    r = orc.forward_backward(params, **batch)
    f = lambda: loss_of(orc, params, batch)
    # every head parameter
    for i in range(orc.n_params):
        assert abs(central_diff(f, params, i) - r.head_grad[i]) < 1e-8, i
    # every table entry: chain through gather / mean-pool
    E, D = orc.E, orc.D
    gu = orc.emb_grad("user", batch["user_id"], r.dX)
    gh = orc.emb_grad("url", batch["url_id"], r.dX)
    for i in range(orc.user_emb.size):
        assert abs(central_diff(f, orc.user_emb, i) - gu.flat[i]) < 1e-8
    for i in range(orc.url_emb.size):
        assert abs(central_diff(f, orc.url_emb, i) - gh.flat[i]) < 1e-8
    rows = orc.dfv_grad_rows(batch["img_off"], r.dX)
    gd = np.zeros_like(orc.dfv)
    np.add.at(gd, batch["img_id"], rows)
    for i in range(orc.dfv.size):
        assert abs(central_diff(f, orc.dfv, i) - gd.flat[i]) < 1e-8


@pytest.mark.parametrize("hidden", [(6,), (7, 3)])
def test_head_against_autodiff_library(hidden):
    orc, params, batch = small_problem(seed=4, B=9, E=4, D=6, hidden=hidden, Vi=5)
    r = orc.forward_backward(params, **batch)
    X = torch.tensor(r.X, requires_grad=True)
    p = torch.tensor(params, requires_grad=True)
    layers, w_out, b_out = split_params(p, orc.d_in, hidden)
    h = X
    for W, b in layers:
        h = torch.relu(h @ W + b)
    z = h @ w_out + b_out
    y = torch.tensor(batch["label"])
    loss = torch.nn.functional.binary_cross_entropy_with_logits(z, y, reduction="mean")
    loss.backward()
    assert abs(loss.item() - r.loss) < 1e-13
    np.testing.assert_allclose(r.prob, torch.sigmoid(z).detach().numpy(), atol=1e-14)
    np.testing.assert_allclose(r.head_grad, p.grad.numpy(), atol=1e-14)
    np.testing.assert_allclose(r.dX, X.grad.numpy(), atol=1e-14)


def test_closed_form_with_zero_hidden_weights():
    orc, params, batch = small_problem(seed=5, B=8, hidden=(4, 3))
    params[:] = 0.0
    params[-1] = 0.7                                       # only the output bias is non-zero
    r = orc.forward_backward(params, **batch)
    p = 1.0 / (1.0 + math.exp(-0.7))
    ybar = batch["label"].mean()
    assert abs(r.loss + (ybar * math.log(p) + (1 - ybar) * math.log(1 - p))) < 1e-14
    np.testing.assert_allclose(r.prob, p, rtol=1e-15)
    assert abs(r.head_grad[-1] - (p - ybar)) < 1e-15       # d loss / d b_out = mean(p - y)
    assert np.all(r.head_grad[:-1] == 0.0) and np.all(r.dX == 0.0)


def test_two_view_batch_by_hand():
    # one hidden unit, everything positive so the ReLU is active: z = w_o * (x . w) + b_o
    user = np.array([[1.0], [2.0]]); url = np.array([[0.5]]); dfv = np.array([[2.0], [4.0]])
    orc = GearOracle(user, url, dfv, (1,), 1, 0)
    params = np.array([0.1, 0.2, 0.3, 0.05, 2.0, -0.4])   # W(3x1), b, w_out, b_out
    r = orc.forward_backward(params, [0, 1], [0, 0], [0, 2, 3], [0, 1, 1], [1.0, 0.0])
    x0 = np.array([1.0, 0.5, 3.0]); x1 = np.array([2.0, 0.5, 4.0])
    a0 = 0.1 * 1 + 0.2 * 0.5 + 0.3 * 3 + 0.05
    a1 = 0.1 * 2 + 0.2 * 0.5 + 0.3 * 4 + 0.05
    z0, z1 = 2 * a0 - 0.4, 2 * a1 - 0.4
    p0, p1 = 1 / (1 + math.exp(-z0)), 1 / (1 + math.exp(-z1))
    assert abs(r.loss - 0.5 * (-math.log(p0) - math.log(1 - p1))) < 1e-14
    dz0, dz1 = (p0 - 1) / 2, p1 / 2
    np.testing.assert_allclose(r.dX[0], dz0 * 2.0 * np.array([0.1, 0.2, 0.3]), rtol=1e-13)
    np.testing.assert_allclose(r.head_grad[0:3], 2.0 * (dz0 * x0 + dz1 * x1), rtol=1e-13)
    assert abs(r.head_grad[4] - (dz0 * a0 + dz1 * a1)) < 1e-14
    rows = orc.dfv_grad_rows([0, 2, 3], r.dX)
    np.testing.assert_allclose(rows[:, 0], [r.dX[0, 2] / 2, r.dX[0, 2] / 2, r.dX[1, 2]], rtol=1e-15)


def test_relu_derivative_is_zero_at_zero():
    orc = GearOracle(np.array([[1.0]]), np.array([[1.0]]), np.array([[2.0]]), (1,), 1, 0)
    params = np.array([1.0, 1.0, -1.0, 0.0, 1.0, 0.0])    # pre-activation 1 + 1 - 2 = 0 exactly
    r = orc.forward_backward(params, [0], [0], [0, 1], [0], [1.0])
    assert np.all(r.dX == 0.0) and np.all(r.head_grad[0:4] == 0.0)


def test_view_permutation_leaves_loss_and_gradients_unchanged():
    orc, params, batch = small_problem(seed=6, B=12, Vu=4, Vh=3, max_imgs=1)
    r = orc.forward_backward(params, **batch)
    perm = np.random.default_rng(0).permutation(12)
    pb = dict(user_id=batch["user_id"][perm], url_id=batch["url_id"][perm], img_off=batch["img_off"],
              img_id=batch["img_id"][perm], label=batch["label"][perm])
    q = orc.forward_backward(params, **pb)
    assert abs(r.loss - q.loss) < 1e-15
    np.testing.assert_allclose(r.head_grad, q.head_grad, atol=1e-15)
    np.testing.assert_allclose(orc.emb_grad("user", batch["user_id"], r.dX),
                               orc.emb_grad("user", pb["user_id"], q.dX), atol=1e-15)


def test_mean_pool_backward_rows_sum_to_dpooled():
    orc, params, batch = small_problem(seed=7, B=6, max_imgs=4)
    r = orc.forward_backward(params, **batch)
    rows = orc.dfv_grad_rows(batch["img_off"], r.dX)
    off = batch["img_off"]
    for b in range(6):
        np.testing.assert_allclose(rows[off[b]:off[b + 1]].sum(0), r.dX[b, 2 * orc.E:], rtol=1e-14)


class _RoundBoth(torch.autograd.Function):
    """bf16 rounding of an activation and of the gradient that flows back through it."""
    @staticmethod
    def forward(ctx, x):
        return x.float().bfloat16().double()

    @staticmethod
    def backward(ctx, g):
        return g.float().bfloat16().double()


class _RoundFwd(torch.autograd.Function):
    """bf16 rounding of an operand; the gradient passes through unrounded."""
    @staticmethod
    def forward(ctx, x):
        return x.float().bfloat16().double()

    @staticmethod
    def backward(ctx, g):
        return g


def test_bf16_operand_rounding_points_against_autodiff_library():
    rng = np.random.default_rng(8)
    B, E, D, hidden = 16, 4, 8, (12, 6)
    user = rng.normal(0, 0.3, (5, E)).astype(np.float32)
    url = rng.normal(0, 0.3, (5, E)).astype(np.float32)
    dfv = torch.from_numpy(rng.normal(0, 0.3, (9, D)).astype(np.float32)).bfloat16()
    dfv_bits = dfv.view(torch.int16).numpy().view(np.uint16)
    orc = GearOracle(user, url, dfv_bits, hidden, 1, 0, round_bf16=True)
    params = rng.normal(0, 0.4, orc.n_params).astype(np.float32).astype(np.float64)
    n = rng.integers(1, 4, B)
    off = np.concatenate([[0], np.cumsum(n)]).astype(np.int32)
    uid, hid = rng.integers(0, 5, B), rng.integers(0, 5, B)
    img = rng.integers(0, 9, off[-1])
    y = (rng.random(B) < 0.5).astype(np.float64)
    r = orc.forward_backward(params, uid, hid, off, img, y)
    # head input before rounding, built with library ops
    pooled = np.stack([dfv.double().numpy()[img[off[b]:off[b + 1]]].sum(0) / n[b] for b in range(B)])
    X0 = torch.tensor(np.concatenate([user[uid], url[hid], pooled], 1), dtype=torch.float64, requires_grad=True)
    p = torch.tensor(params, requires_grad=True)
    layers, w_out, b_out = split_params(p, orc.d_in, hidden)
    h = _RoundFwd.apply(X0)
    for W, b in layers:
        h = _RoundBoth.apply(torch.relu(h @ _RoundFwd.apply(W) + b))
    z = h @ w_out + b_out
    loss = torch.nn.functional.binary_cross_entropy_with_logits(z, torch.tensor(y), reduction="mean")
    loss.backward()
    np.testing.assert_array_equal(r.X, _RoundFwd.apply(X0).detach().numpy())
    assert abs(loss.item() - r.loss) < 1e-12
    np.testing.assert_allclose(r.head_grad, p.grad.numpy(), atol=1e-12)
    np.testing.assert_allclose(r.dX, X0.grad.numpy(), atol=1e-12)


def test_bf16_mode_is_exact_on_bf16_representable_problem():
    # small integers / powers of two everywhere: no rounding can occur, both modes must agree
    user = np.array([[1.0, -2.0], [0.5, 4.0]], dtype=np.float32)
    url = np.array([[2.0, 1.0]], dtype=np.float32)
    dfv = np.array([[1.0, 3.0], [3.0, 1.0]], dtype=np.float32)
    params = np.array([1, 0, 0, 1, 1, -1, 0.5, 0.5, -1, 1, 0.5, 2,  0, 0,  1, -1, 0], dtype=np.float64)
    args = ([0, 1], [0, 0], [0, 2, 3], [0, 1, 1], [1.0, 0.0])
    a = GearOracle(user, url, dfv, (2,), 1, 0, round_bf16=False).forward_backward(params, *args)
    b = GearOracle(user, url, dfv, (2,), 1, 0, round_bf16=True).forward_backward(params, *args)
    assert a.loss == b.loss and np.array_equal(a.X, b.X) and np.array_equal(a.prob, b.prob)


# ----------------------------------------------------------------------------
# embedding apply
# ----------------------------------------------------------------------------
def test_emb_apply_sums_duplicates_and_updates_once():
    rng = np.random.default_rng(9)
    user = rng.normal(size=(4, 3))
    orc = GearOracle(user.copy(), np.zeros((1, 3)), np.zeros((1, 2)), (2,), 1, 0)
    dX = rng.normal(size=(5, 8))
    ids = np.array([2, 2, 0, 2, 3], dtype=np.int32)
    G = orc.emb_grad("user", ids, dX)
    np.testing.assert_allclose(G[2], dX[[0, 1, 3], 0:3].sum(0), rtol=1e-15)
    assert np.all(G[1] == 0.0)
    orc.emb_apply("user", ids, dX, alpha=-0.5)
    np.testing.assert_allclose(orc.user_emb, user - 0.5 * G, rtol=1e-15)
    # the url table reads its own column block
    orc2 = GearOracle(np.zeros((1, 3)), np.zeros((4, 3)), np.zeros((1, 2)), (2,), 1, 0)
    np.testing.assert_allclose(orc2.emb_grad("url", ids, dX)[0], dX[2, 3:6], rtol=1e-15)


# ----------------------------------------------------------------------------
# accumulate-to-M and emit
# ----------------------------------------------------------------------------
def literal_gradient_store(V, D, M, calls):
    """The paper's own wording: keep every gradient of an image; when M are
    stored, average them, hand the average on, and start over."""
    store = {i: [] for i in range(V)}
    seq = {}
    per_collect = []
    for ids, g in calls:
        for r, i in enumerate(ids):
            store[i].append(g[r])
            if len(store[i]) == M:
                k = seq.get(i, 0)
                per_collect.append((i, k, np.mean(np.stack(store[i]), axis=0)))
                seq[i] = k + 1
                store[i] = []
    return per_collect, store


@pytest.mark.parametrize("M", [1, 2, 3, 5])
def test_accumulate_against_literal_store(M):
    rng = np.random.default_rng(10 + M)
    V, D = 6, 3
    orc = GearOracle(np.zeros((1, 1)), np.zeros((1, 1)), np.zeros((V, D)), (1,), M, 0)
    calls = []
    for _ in range(4):
        n = int(rng.integers(0, 25))
        ids = np.minimum(rng.geometric(0.45, n) - 1, V - 1).astype(np.int32)   # skewed ids
        calls.append((ids, rng.normal(size=(n, D))))
    for ids, g in calls:
        orc.accumulate(ids, g)
    eid, eseq, eavg = orc.collect_ready()
    want, store = literal_gradient_store(V, D, M, calls)
    assert [w[0] for w in want] == list(eid)               # same emissions, same (arrival) order
    assert [w[1] for w in want] == list(eseq)
    np.testing.assert_allclose(eavg, np.stack([w[2] for w in want]) if want else np.zeros((0, D)), atol=1e-15)
    for i in range(V):                                     # what is left in the store
        assert orc.gcnt[i] == len(store[i])
        np.testing.assert_allclose(orc.gsum[i], np.sum(store[i], axis=0) if store[i] else 0.0, atol=1e-15)


def test_accumulate_invariants_on_zipf_stream():
    from paper_1806_03925_b200 import workloads
    M, V, D, n = 4, 300, 8, 5000
    rng = np.random.default_rng(11)
    ids = workloads.ZipfIds(V, 1.1).sample(rng, n)
    g = rng.normal(size=(n, D))
    orc = GearOracle(np.zeros((1, 1)), np.zeros((1, 1)), np.zeros((V, D)), (1,), M, 0)
    halves = [(ids[:2000], g[:2000]), (ids[2000:], g[2000:])]
    members = []
    for hi, hg in halves:
        _, mem = orc.accumulate(hi, hg, want_members=True)
        members.append(mem)
    eid, eseq, eavg = orc.collect_ready()
    # conservation: every arrival is either in an emitted group or still counted
    assert M * len(eid) + orc.gcnt.sum() == n
    k = np.bincount(ids, minlength=V)
    assert np.array_equal(np.bincount(eid, minlength=V), k // M)   # floor(k / M) emissions per image
    assert np.array_equal(orc.gcnt, k % M)
    # emission numbers of an image are 0, 1, 2, ... in arrival order
    for i in np.unique(eid):
        assert list(eseq[eid == i]) == list(range(k[i] // M))
    # M * average == sum of the group's members (second call: groups made only of its arrivals)
    mem = members[1]
    for e in np.unique(mem[mem >= 0]):
        rows = np.where(mem == e)[0]
        if len(rows) == M:
            np.testing.assert_allclose(M * eavg[e], halves[1][1][rows].sum(0), atol=1e-12)
            assert np.all(halves[1][0][rows] == eid[e])
    # per image: M * (sum of its averages) + residual == sum of all its gradients
    tot = np.zeros((V, D)); np.add.at(tot, ids, g)
    emitted = np.zeros((V, D)); np.add.at(emitted, eid, M * eavg)
    np.testing.assert_allclose(emitted + orc.gsum, tot, atol=1e-10)


def test_M1_emits_every_row_in_order_and_keeps_the_table_empty():
    rng = np.random.default_rng(12)
    ids = rng.integers(0, 5, 40).astype(np.int32)
    g = rng.normal(size=(40, 4))
    orc = GearOracle(np.zeros((1, 1)), np.zeros((1, 1)), np.zeros((5, 4)), (1,), 1, 0)
    orc.accumulate(ids, g)
    eid, eseq, eavg = orc.collect_ready()
    assert np.array_equal(eid, ids) and np.array_equal(eavg, g)
    assert not orc.gsum.any() and not orc.gcnt.any()
    assert orc.pending_ready == 0
    orc.accumulate(ids[:3], g[:3])                          # numbering restarts after a collect
    assert list(orc.collect_ready()[1]) == [0] * 3 or len(set(ids[:3])) < 3


def test_pooled_store_conserves_sums_and_matches_the_ordered_store_where_order_cannot_matter():
    """The order-free store (asynchronous arrivals): same counts and emission counts as the ordered one,
    M * (sum of averages) + kept sum == pooled sum, every emission of an image is the pooled mean; where an
    image receives exactly M gradients into an empty store, or identical gradients, both stores agree."""
    from paper_1806_03925_b200 import workloads
    M, V, D, n = 4, 200, 6, 3000
    rng = np.random.default_rng(21)
    ids = workloads.ZipfIds(V, 1.1).sample(rng, n)
    g = rng.normal(size=(n, D))
    mk = lambda: GearOracle(np.zeros((1, 1)), np.zeros((1, 1)), np.zeros((V, D)), (1,), M, 0)
    a, b = mk(), mk()
    tot = np.zeros((V, D)); cnt = np.zeros(V, dtype=np.int64)
    for lo, hi in ((0, 1200), (1200, n)):
        before_sum, before_cnt = b.gsum.copy(), b.gcnt.copy()
        a.accumulate(ids[lo:hi], g[lo:hi])
        b.accumulate(ids[lo:hi], g[lo:hi], pooled=True)
        assert np.array_equal(a.gcnt, b.gcnt)                       # counts are order-free
        np.add.at(tot, ids[lo:hi], g[lo:hi]); np.add.at(cnt, ids[lo:hi], 1)
        # every emission of this call is the mean of what the image held plus what arrived
        k_call = np.bincount(ids[lo:hi], minlength=V) + before_cnt
        pooled = before_sum.copy(); np.add.at(pooled, ids[lo:hi], g[lo:hi])
        new = slice(len(b._emit_id) - int((k_call // M).sum()), len(b._emit_id))
        for i, avg in zip(b._emit_id[new], b._emit_avg[new]):
            np.testing.assert_allclose(avg, pooled[i] / k_call[i], atol=1e-12)
    ea, eb = a.collect_ready(), b.collect_ready()
    assert np.array_equal(np.bincount(ea[0], minlength=V), np.bincount(eb[0], minlength=V))
    assert np.array_equal(np.bincount(eb[0], minlength=V), cnt // M)
    sa, sb = oracle.sort_emissions(*ea), oracle.sort_emissions(*eb)
    assert np.array_equal(sa[0], sb[0]) and np.array_equal(sa[1], sb[1])    # same (id, seq) pairs
    emitted = np.zeros((V, D)); np.add.at(emitted, eb[0], M * eb[2])
    np.testing.assert_allclose(emitted + b.gsum, tot, atol=1e-10)           # nothing lost, nothing counted twice
    # exactly M gradients into an empty store: one group either way
    c, d = mk(), mk()
    ids2 = np.repeat(np.arange(5, dtype=np.int32), M); g2 = rng.normal(size=(5 * M, D))
    perm = rng.permutation(5 * M)
    c.accumulate(ids2[perm], g2[perm]); d.accumulate(ids2[perm], g2[perm], pooled=True)
    sc, sd = oracle.sort_emissions(*c.collect_ready()), oracle.sort_emissions(*d.collect_ready())
    np.testing.assert_allclose(sc[2], sd[2], atol=1e-12)
    assert not d.gcnt.any() and np.abs(d.gsum).max() == 0.0
    # identical gradients: any grouping gives the same averages and residual
    e, f = mk(), mk()
    ids3 = np.zeros(11, dtype=np.int32); g3 = np.tile(rng.normal(size=(1, D)), (11, 1))
    e.accumulate(ids3, g3); f.accumulate(ids3, g3, pooled=True)
    np.testing.assert_allclose(e.gsum, f.gsum, atol=1e-12)
    np.testing.assert_allclose(e.collect_ready()[2], f.collect_ready()[2], atol=1e-12)


def test_bad_image_ids_are_ignored_by_accumulate():
    orc = GearOracle(np.zeros((1, 1)), np.zeros((1, 1)), np.zeros((3, 2)), (1,), 2, 0)
    bad = orc.accumulate(np.array([0, 7, -1, 0], dtype=np.int32), np.ones((4, 2)))
    assert bad == 2
    eid, _, eavg = orc.collect_ready()
    assert list(eid) == [0] and np.all(eavg == 1.0)


# ----------------------------------------------------------------------------
# Eq. 1: gear training with M = 1 and zero expiry is ordinary back-propagation
# ----------------------------------------------------------------------------
def _linear_dense_setup(seed, M):
    rng = np.random.default_rng(seed)
    B, E, D, R, Vi = 6, 2, 3, 4, 5
    raw = rng.normal(size=(Vi, R))                         # "raw images"
    Wd = rng.normal(0, 0.5, (R, D))                        # linear Dense Part: DFV_i = raw_i @ Wd
    user, url = rng.normal(size=(4, E)), rng.normal(size=(4, E))
    n = rng.integers(1, 4, B)
    off = np.concatenate([[0], np.cumsum(n)]).astype(np.int32)
    batch = dict(user_id=rng.integers(0, 4, B).astype(np.int32), url_id=rng.integers(0, 4, B).astype(np.int32),
                 img_off=off, img_id=rng.integers(0, Vi, off[-1]).astype(np.int32),
                 label=(rng.random(B) < 0.5).astype(np.float64))
    orc = GearOracle(user, url, raw @ Wd, (4,), M, expire=0)
    params = rng.normal(0, 0.6, orc.n_params)
    return orc, params, batch, raw, Wd


def _dense_grad_by_finite_differences(orc, params, batch, raw, Wd):
    def f():
        orc.dfv[:] = raw @ Wd                              # zero expiry: the cache is refreshed every step
        return loss_of(orc, params, batch)
    return np.array([central_diff(f, Wd, i) for i in range(Wd.size)]).reshape(Wd.shape)


def test_eq1_M1_zero_expiry_equals_direct_backprop():
    orc, params, batch, raw, Wd = _linear_dense_setup(13, M=1)
    assert len(orc.collect_expired(now=5)) == orc.V        # expiry 0: every cached DFV is always stale
    want = _dense_grad_by_finite_differences(orc, params, batch, raw, Wd)
    r = orc.forward_backward(params, **batch)
    orc.accumulate(batch["img_id"], orc.dfv_grad_rows(batch["img_off"], r.dX))
    eid, _, eavg = orc.collect_ready()
    got = oracle.dense_backward(raw, eid, eavg)              # dLoss/dDFV . dDFV/dW_dense, event 6's second half
    np.testing.assert_allclose(got, want, atol=1e-8)


def test_eq1_total_gradient_is_conserved_for_M3():
    orc, params, batch, raw, Wd = _linear_dense_setup(14, M=3)
    want = _dense_grad_by_finite_differences(orc, params, batch, raw, Wd)
    r = orc.forward_backward(params, **batch)
    orc.accumulate(batch["img_id"], orc.dfv_grad_rows(batch["img_off"], r.dX))
    eid, _, eavg = orc.collect_ready()
    got = oracle.dense_backward(raw, eid, 3 * eavg)
    got = got + oracle.dense_backward(raw, np.arange(orc.V), orc.gsum)      # what is still waiting in the store
    np.testing.assert_allclose(got, want, atol=1e-8)


# ----------------------------------------------------------------------------
# expiry
# ----------------------------------------------------------------------------
def _expiry_oracle(ts, T):
    return GearOracle(np.zeros((1, 1)), np.zeros((1, 1)), np.zeros((len(ts), 1)), (1,), 1, T, ts=ts)


def test_expiry_special_cases():
    ts = np.array([5, -3, 0, 9, 2, 2], dtype=np.int64)
    assert list(_expiry_oracle(ts, 0).collect_expired(now=9)) == [0, 1, 2, 3, 4, 5]     # T = 0: all
    assert len(_expiry_oracle(ts, 13).collect_expired(now=9)) == 0                     # T > now - min(ts): none
    assert list(_expiry_oracle(ts, 12).collect_expired(now=9)) == [1]                  # boundary is inclusive
    assert list(_expiry_oracle(ts, 7).collect_expired(now=9)) == [1, 2, 4, 5]          # ascending ids


def test_restamp_makes_an_id_reappear_exactly_T_later():
    T = 4
    orc = _expiry_oracle(np.array([0, 1, 2, 3], dtype=np.int64), T)
    seen = {i: [] for i in range(4)}
    for now in range(0, 20):
        for i in orc.collect_expired(now, restamp=True):
            seen[int(i)].append(now)
    for i in range(4):
        assert seen[i] == list(range(i + T, 20, T))
    keep = _expiry_oracle(np.array([0], dtype=np.int64), 2)
    assert [len(keep.collect_expired(now, restamp=False)) for now in range(4)] == [0, 0, 1, 1]


# ----------------------------------------------------------------------------
# refresh of cached inference results
# ----------------------------------------------------------------------------
def test_refresh_replaces_rows_rounds_to_the_table_dtype_and_restarts_the_clock():
    rng = np.random.default_rng(3)
    Vi, D = 9, 5
    for dt in (np.float64, np.float32, np.uint16):
        table = (rng.normal(size=(Vi, D)).astype(dt) if dt != np.uint16
                 else (rng.integers(0, 2 ** 15, (Vi, D))).astype(np.uint16))
        before = table.copy()
        orc = GearOracle(np.zeros((1, 1)), np.zeros((1, 1)), table, (1,), 1, 3, ts=np.arange(Vi, dtype=np.int64))
        ids = np.array([7, 2, -1, 4, Vi], dtype=np.int32)          # two of them out of range
        rows = rng.normal(size=(len(ids), D)).astype(np.float32)
        rows[1, 0] = 1.0 + 2.0 ** -8                               # a tie between two bfloat16 values: goes to even (1.0)
        rows[1, 1] = 1.0 + 3 * 2.0 ** -8                           # ... and this one up (1.015625)
        assert orc.refresh_dfv(ids, rows, now=40) == 2
        for k, i in enumerate(ids):
            if not 0 <= i < Vi:
                continue
            if dt == np.uint16:                                    # bit patterns, against torch's own rounding
                want = torch.from_numpy(rows[k]).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
                assert np.array_equal(orc.dfv[i], want)
            else:
                assert np.array_equal(orc.dfv[i], rows[k].astype(dt))
        if dt == np.uint16:
            assert orc.dfv[2, 0] == 0x3f80 and orc.dfv[2, 1] == 0x3f82
        untouched = [i for i in range(Vi) if i not in (7, 2, 4)]
        assert np.array_equal(orc.dfv[untouched], before[untouched])
        assert list(orc.ts) == [0, 1, 40, 3, 40, 5, 6, 40, 8]
        assert not orc.gsum.any() and not orc.gcnt.any()           # the gradient store is left alone
        # a refreshed image is not listed again before now + T, the others are
        assert list(orc.collect_expired(now=42, restamp=False)) == [0, 1, 3, 5, 6, 8]
        assert list(orc.collect_expired(now=43, restamp=False)) == list(range(Vi))


def test_refresh_in_index_order_last_row_wins_and_ts_ids_may_differ():
    table = np.zeros((3, 2), dtype=np.float32)
    orc = GearOracle(np.zeros((1, 1)), np.zeros((1, 1)), table, (1,), 1, 1, ts=np.zeros(10, dtype=np.int64))
    rows = np.array([[1, 1], [2, 2], [3, 3]], dtype=np.float32)
    assert orc.refresh_dfv([1, 0, 1], rows, now=7, ts_ids=[9, 4, 9]) == 0
    assert np.array_equal(orc.dfv, [[2, 2], [3, 3], [0, 0]])
    assert list(np.nonzero(orc.ts)[0]) == [4, 9] and orc.ts[9] == 7


def test_gear_loop_with_refresh_every_step_is_ordinary_training_of_the_dense_part():
    """M = 1, expiry 0, linear Dense Part: every step the expired list is everything, the refreshed DFVs are
    raw @ Wd for the current Wd, and the emitted averages give dLoss/dWd exactly (Eq. 1).  Two SGD steps on Wd
    through the loop must equal two SGD steps with the gradient taken by finite differences."""
    orc, params, batch, raw, Wd = _linear_dense_setup(15, M=1)
    Wd_loop, Wd_ref, lr = Wd.copy(), Wd.copy(), 0.3
    for step in range(2):
        expired = orc.collect_expired(now=step, restamp=True)
        assert len(expired) == orc.V
        orc.refresh_dfv(expired, oracle.dense_forward(raw, Wd_loop, expired).astype(np.float32), now=step)
        orc.dfv[:] = raw @ Wd_loop                                 # keep the fp64 table exact (refresh rows are fp32)
        r = orc.forward_backward(params, **batch)
        orc.accumulate(batch["img_id"], orc.dfv_grad_rows(batch["img_off"], r.dX))
        eid, _, eavg = orc.collect_ready()
        Wd_loop = Wd_loop - lr * oracle.dense_backward(raw, eid, eavg)
        Wd_ref = Wd_ref - lr * _dense_grad_by_finite_differences(orc, params, batch, raw, Wd_ref)
        orc.dfv[:] = raw @ Wd_loop
    np.testing.assert_allclose(Wd_loop, Wd_ref, atol=1e-7)


# ----------------------------------------------------------------------------
# units whose ReLU decision is within rounding distance of zero
# ----------------------------------------------------------------------------
def test_near_zero_units_are_listed_and_can_take_the_other_branch():
    from oracle import decode_unit
    orc = GearOracle(np.array([[1.0]]), np.array([[1.0]]), np.array([[2.0]]), (2,), 1, 0)
    # unit 0: pre-activation 1 + 1 - 2 = 0 exactly; unit 1: clearly active
    params = np.array([1.0, 0.5, 1.0, 0.5, -1.0, 0.5, 0.0, 0.25, 1.0, -2.0, 0.3])
    args = ([0], [0], [0, 1], [0], [1.0])
    r = orc.forward_backward(params, *args, relu_margin=1e-12)
    assert [decode_unit(c, 1) for c in r.near_units] == [(0, 0, 0)]
    flipped = orc.forward_backward(params, *args, flip_units=r.near_units)
    assert flipped.loss == r.loss and np.array_equal(flipped.prob, r.prob)
    # the other branch is the network whose ReLU has derivative 1 at 0: check against the autodiff library
    X = torch.tensor(r.X, requires_grad=True)
    p = torch.tensor(params, requires_grad=True)
    (W, b), = split_params(p, 3, (2,))[0]
    a = X @ W + b
    h = torch.where(a >= 0, a, torch.zeros_like(a))
    z = h @ p[8:10] + p[10]
    loss = torch.nn.functional.binary_cross_entropy_with_logits(z, torch.tensor([1.0], dtype=torch.float64))
    loss.backward()
    np.testing.assert_allclose(flipped.head_grad, p.grad.numpy(), atol=1e-15)
    np.testing.assert_allclose(flipped.dX, X.grad.numpy(), atol=1e-15)
    assert np.any(flipped.dX != r.dX)
    assert len(orc.forward_backward(params, *args, relu_margin=0.5).near_units) == 1      # |0.25 + ...| unit stays out
    # the relative form of the margin: |a| <= rel * max|input row| * max|weights| = rel * 2 * 1; unit 1 has a = 2.25
    wide = orc.forward_backward(params, *args, relu_margin=0.0, relu_margin_rel=1.2)
    assert [decode_unit(c, 1) for c in wide.near_units] == [(0, 0, 0), (0, 0, 1)]
    assert wide.near_abs.tolist() == [0.0, 2.25]
    assert len(orc.forward_backward(params, *args, relu_margin=0.0, relu_margin_rel=1.1).near_units) == 1
    assert np.array_equal(wide.dX, r.dX) and np.array_equal(wide.head_grad, r.head_grad)   # listing changes no result


# ----------------------------------------------------------------------------
# the linear Dense Part and the optimiser
# ----------------------------------------------------------------------------
def test_dense_forward_special_cases():
    raw = np.array([[1.0, 0.0, 0.0], [0.0, 0.0, 1.0], [2.0, -1.0, 0.5]])
    Wd = np.array([[1.0, 2.0], [3.0, 4.0], [5.0, 6.0]])
    rows = oracle.dense_forward(raw, Wd, [0, 1, 2, 1, 7])
    assert rows[0].tolist() == [1.0, 2.0] and rows[1].tolist() == [5.0, 6.0]      # unit rows pick rows of Wd
    assert rows[2].tolist() == [2 - 3 + 2.5, 4 - 4 + 3.0]                          # by hand
    assert np.array_equal(rows[3], rows[1]) and not rows[4].any()                  # repeats; out-of-range id: zeros
    assert np.array_equal(oracle.dense_forward(raw, np.eye(3), [2, 0]), raw[[2, 0]])   # identity Wd: the raw rows
    # float32 storage is read exactly
    assert np.array_equal(oracle.dense_forward(raw.astype(np.float32), Wd, [2]), rows[2:3])


def test_dense_backward_is_the_gradient_of_the_dense_forward():
    # L(Wd) = sum_e <avg_e, raw[id_e] . Wd> is linear in Wd, so its gradient is exact by finite differences
    rng = np.random.default_rng(21)
    raw, Wd = rng.normal(size=(6, 4)), rng.normal(size=(4, 3))
    ids, avg = np.array([5, 0, 5, 2], np.int32), rng.normal(size=(4, 3))
    G = oracle.dense_backward(raw, ids, avg)
    f = lambda: float((oracle.dense_forward(raw, Wd, ids) * avg).sum())
    want = np.array([central_diff(f, Wd, i, h=1e-3) for i in range(Wd.size)]).reshape(Wd.shape)
    np.testing.assert_allclose(G, want, atol=1e-9)
    # a repeated image counts once per emission; an out-of-range id is skipped
    one = oracle.dense_backward(raw, np.array([5], np.int32), avg[:1] + avg[2:3])
    two = oracle.dense_backward(raw, np.array([5, 5, 9], np.int32), np.vstack([avg[:1], avg[2:3], avg[:1]]))
    np.testing.assert_allclose(one, two, atol=1e-15)


def test_adam_matches_the_optimiser_library_and_the_closed_form_of_its_first_step():
    from oracle import AdamConfig
    rng = np.random.default_rng(22)
    cfg = AdamConfig(lr=1e-2, beta1=0.8, beta2=0.95, eps=1e-6)
    p0 = rng.normal(size=17)
    p, m, v = p0.copy(), np.zeros(17), np.zeros(17)
    tp = torch.tensor(p0.copy(), requires_grad=True)
    opt = torch.optim.Adam([tp], lr=cfg.lr, betas=(cfg.beta1, cfg.beta2), eps=cfg.eps)
    for t in range(1, 6):
        g = rng.normal(size=17) * (10.0 ** rng.integers(-3, 2))
        oracle.adam_step(p, g, m, v, t, cfg)
        tp.grad = torch.tensor(g.copy())
        opt.step()
        np.testing.assert_allclose(p, tp.detach().numpy(), rtol=0, atol=1e-13)
    # first step from zero moments: m_hat = g, v_hat = g^2, so the step is -lr * g / (|g| + eps), about -lr * sign(g)
    g = np.array([3.0, -0.2, 1e-3, -50.0])
    p, m, v = np.zeros(4), np.zeros(4), np.zeros(4)
    oracle.adam_step(p, g, m, v, 1, cfg)
    np.testing.assert_allclose(p, -cfg.lr * g / (np.abs(g) + cfg.eps), rtol=1e-12)
    np.testing.assert_allclose(m, (1 - cfg.beta1) * g, rtol=1e-15)
    np.testing.assert_allclose(v, (1 - cfg.beta2) * g * g, rtol=1e-15)
    # a zero gradient with zero moments moves nothing
    p, m, v = np.ones(3), np.zeros(3), np.zeros(3)
    oracle.adam_step(p, np.zeros(3), m, v, 4, cfg)
    assert p.tolist() == [1.0, 1.0, 1.0]


def test_embedding_adam_steps_each_touched_row_once_with_the_summed_gradient():
    from oracle import AdamConfig
    rng = np.random.default_rng(23)
    cfg = AdamConfig(lr=1e-2)
    V, E = 6, 3
    table = rng.normal(size=(V, E))
    m, v = rng.normal(0, 0.1, (V, E)), rng.random((V, E)) * 0.01
    ids = np.array([4, 1, 4, 9, 4], np.int32)                 # id 4 three times, id 9 out of range
    dX = rng.normal(size=(5, 8))
    t0, m0, v0 = table.copy(), m.copy(), v.copy()
    assert oracle.emb_adam(table, m, v, ids, dX, col0=2, t=3, cfg=cfg) == 1
    for i in (0, 2, 3, 5):                                    # untouched rows and their moments stay
        assert np.array_equal(table[i], t0[i]) and np.array_equal(m[i], m0[i]) and np.array_equal(v[i], v0[i])
    for i, views in ((4, [0, 2, 4]), (1, [1])):               # one step with the sum, not one step per view
        g = dX[views, 2:5].sum(0)
        pr, mr, vr = t0[i].copy(), m0[i].copy(), v0[i].copy()
        oracle.adam_step(pr, g, mr, vr, 3, cfg)
        np.testing.assert_allclose(table[i], pr, atol=1e-15)
        np.testing.assert_allclose(m[i], mr, atol=1e-15)
        np.testing.assert_allclose(v[i], vr, atol=1e-15)


# ----------------------------------------------------------------------------
# a dense input of the view's own (the Fastgear side's share of the image)
# ----------------------------------------------------------------------------
def test_fast_side_dense_input_is_appended_to_the_head_input():
    rng = np.random.default_rng(41)
    B, E, D, F, Vi = 4, 2, 3, 5, 6
    orc = GearOracle(rng.normal(size=(3, E)), rng.normal(size=(3, E)), rng.normal(size=(Vi, D)), (4, 3), 1, 0, fast_dim=F)
    assert orc.d_in == 2 * E + D + F
    params = rng.normal(0, 0.5, orc.n_params)
    n = np.array([2, 1, 0, 3])
    off = np.concatenate([[0], np.cumsum(n)]).astype(np.int32)
    fast = rng.normal(size=(B, F))
    batch = dict(user_id=rng.integers(0, 3, B).astype(np.int32), url_id=rng.integers(0, 3, B).astype(np.int32), img_off=off,
                 img_id=rng.integers(0, Vi, off[-1]).astype(np.int32), label=np.array([1.0, 0.0, 0.0, 1.0]), fast=fast)
    r = orc.forward_backward(params, **batch)
    assert np.array_equal(r.X[:, 2 * E + D:], fast)                       # a copy, after the pooled DFV
    assert np.array_equal(r.X[2, 2 * E:2 * E + D], np.zeros(D))          # the empty view still pools to zeros
    # dLoss/d(fast) and dLoss/d(DFV table) by central differences: the new columns moved nothing else
    want = np.array([central_diff(lambda: loss_of(orc, params, batch), fast, i) for i in range(fast.size)]).reshape(fast.shape)
    np.testing.assert_allclose(r.dX[:, 2 * E + D:], want, atol=1e-8)
    g_tab = np.zeros_like(orc.dfv)
    rows = orc.dfv_grad_rows(off, r.dX)
    for k, i in enumerate(batch["img_id"]):
        g_tab[i] += rows[k]
    want_tab = np.array([central_diff(lambda: loss_of(orc, params, batch), orc.dfv, i) for i in range(orc.dfv.size)]).reshape(orc.dfv.shape)
    np.testing.assert_allclose(g_tab, want_tab, atol=1e-8)
    # with zero weights on the new columns the network is the one without them
    plain = GearOracle(orc.user_emb, orc.url_emb, orc.dfv, (4, 3), 1, 0)
    W1 = params[:orc.d_in * 4].reshape(orc.d_in, 4).copy()
    p0 = params.copy(); p0[:orc.d_in * 4] = np.vstack([W1[:2 * E + D], np.zeros((F, 4))]).ravel()
    pp = np.concatenate([W1[:2 * E + D].ravel(), params[orc.d_in * 4:]])
    b2 = {k: v for k, v in batch.items() if k != "fast"}
    assert abs(orc.forward_backward(p0, **batch).loss - plain.forward_backward(pp, **b2).loss) < 1e-15
