"""Pins of the oracle's three workload steps: special cases, closed forms and finite differences.

The loss functions used for the finite differences are the textbook definitions written with
numpy in fp64; they are themselves tied down by special cases (zero scores give log 2 per term,
ComplEx without imaginary parts is the trilinear product, exact low-rank data has zero error).
"""
import numpy as np
import pytest

from oracle import Oracle, CONFORM, REPLICATE


@pytest.fixture(params=[4, 8], ids=["fp32", "fp64"], autouse=True)
def both_value_types(request, monkeypatch):
    """Every pin of this file runs against both builds of the oracle: 4-byte and 8-byte values."""
    import oracle
    init = oracle.Oracle.__init__

    def patched(self, *a, **kw):
        kw.setdefault("value_bytes", request.param)
        init(self, *a, **kw)
    monkeypatch.setattr(oracle.Oracle, "__init__", patched)
    return request.param



def softplus(x):
    return np.logaddexp(0.0, x)


def test_sgns_zero_scores_give_log2_per_term():
    V, L, K = 20, 8, 3
    o = Oracle(2 * V, L, workers=2)
    o.table()[:V] = 0.0                      # centre vectors zero: every score is 0
    o.table()[V:] = 1.0
    d = o.register_distribution(V, None, V, CONFORM, seed=0)
    loss = o.step_sgns(np.arange(4, dtype=np.uint32), np.arange(4, dtype=np.uint32) + V, d, K, 0.1)
    assert abs(loss - (K + 1) * np.log(2.0)) < 1e-6


def sgns_loss(T, c, o_key, negs):
    v = T[c]
    return softplus(-(v @ T[o_key])) + sum(softplus(v @ T[k]) for k in negs)


def test_sgns_single_item_is_textbook_sgd_by_finite_differences():
    V, L, K, lr = 12, 5, 3, 0.05
    rng = np.random.default_rng(0)
    init = rng.normal(0, 0.5, size=(2 * V, L)).astype(np.float32)
    o = Oracle(2 * V, L, workers=1)
    o.table()[:] = init
    d = o.register_distribution(V, None, V, CONFORM, seed=3)
    c, ctx = 4, V + 7
    loss, negs = o.step_sgns(np.array([c], np.uint32), np.array([ctx], np.uint32), d, K, lr, return_negatives=True)
    T = init.astype(np.float64)
    assert abs(loss - sgns_loss(T, c, ctx, negs)) < 1e-6
    grad = np.zeros_like(T)
    h = 1e-6
    for k in set([c, ctx] + list(negs)):
        for e in range(L):
            Tp, Tm = T.copy(), T.copy()
            Tp[k, e] += h
            Tm[k, e] -= h
            grad[k, e] = (sgns_loss(Tp, c, ctx, negs) - sgns_loss(Tm, c, ctx, negs)) / (2 * h)
    np.testing.assert_allclose(o.table() - init, -lr * grad, rtol=2e-4, atol=2e-7)
    assert np.abs(grad).max() > 0.01


def test_sgns_batch_uses_snapshot_and_sums_duplicates():
    # two identical items in one batch: both gradients come from the same start values
    V, L, lr = 6, 4, 0.1
    rng = np.random.default_rng(1)
    init = rng.normal(0, 0.5, size=(2 * V, L)).astype(np.float32)
    one = Oracle(2 * V, L, workers=1)
    one.table()[:] = init
    d1 = one.register_distribution(V, None, V, CONFORM, seed=0)
    one.step_sgns(np.array([2], np.uint32), np.array([V + 3], np.uint32), d1, 0, lr)
    two = Oracle(2 * V, L, workers=1)
    two.table()[:] = init
    d2 = two.register_distribution(V, None, V, CONFORM, seed=0)
    two.step_sgns(np.array([2, 2], np.uint32), np.array([V + 3, V + 3], np.uint32), d2, 0, lr)
    np.testing.assert_allclose(two.table() - init, 2 * (one.table() - init), rtol=1e-6, atol=1e-8)


def complex_score(T, h, r, t):
    d = T.shape[1] // 2
    H, R, Tt = (T[h, :d] + 1j * T[h, d:]), (T[r, :d] + 1j * T[r, d:]), (T[t, :d] + 1j * T[t, d:])
    return float(np.real(np.sum(H * R * np.conj(Tt))))


def complex_loss(T, h, r, t, negs):
    loss = softplus(-complex_score(T, h, r, t))
    for j, e in enumerate(negs):
        loss += softplus(complex_score(T, e, r, t) if j % 2 == 0 else complex_score(T, h, r, e))
    return loss


def test_complex_without_imaginary_parts_is_trilinear_product():
    E, Rl, L = 10, 3, 8
    rng = np.random.default_rng(2)
    o = Oracle(E + Rl, L, workers=1, with_adagrad=True)
    init = rng.normal(0, 0.5, size=(E + Rl, L)).astype(np.float32)
    init[:, L // 2:] = 0.0
    o.table()[:] = init
    d = o.register_distribution(0, None, E, CONFORM, seed=0)
    loss = o.step_complex(np.array([1], np.uint32), np.array([E + 2], np.uint32), np.array([5], np.uint32),
                          d, 0, 0.1, 1e-10)
    tri = float(np.sum(init[1, :4].astype(np.float64) * init[E + 2, :4] * init[5, :4]))
    assert abs(loss - softplus(-tri)) < 1e-6


def test_complex_adagrad_first_step_by_finite_differences():
    E, Rl, L, K, lr, eps = 9, 2, 6, 4, 0.1, 1e-10
    rng = np.random.default_rng(3)
    init = rng.normal(0, 0.7, size=(E + Rl, L)).astype(np.float32)
    acc0 = rng.uniform(0.5, 1.5, size=(E + Rl, L)).astype(np.float32)
    o = Oracle(E + Rl, L, workers=1, with_adagrad=True)
    o.table(0)[:] = init
    o.table(1)[:] = acc0
    d = o.register_distribution(0, None, E, CONFORM, seed=5)
    h, r, t = 3, E + 1, 6
    loss, negs = o.step_complex(np.array([h], np.uint32), np.array([r], np.uint32), np.array([t], np.uint32),
                                d, K, lr, eps, return_negatives=True)
    T = init.astype(np.float64)
    assert abs(loss - complex_loss(T, h, r, t, negs)) < 1e-6
    # per-role gradients: a key that plays several roles in the item gets one update per role
    roles = [h, r, t] + list(negs)
    dval = np.zeros_like(T)
    dacc = np.zeros_like(T)
    hstep = 1e-6
    base = np.vstack([T, np.zeros((len(roles), L))])        # give every role its own row copy
    idx = list(range(E + Rl, E + Rl + len(roles)))
    for j, k in enumerate(roles):
        base[idx[j]] = T[k]

    def loss_roles(B):
        return complex_loss(B, idx[0], idx[1], idx[2], idx[3:])
    for j, k in enumerate(roles):
        for e in range(L):
            Bp, Bm = base.copy(), base.copy()
            Bp[idx[j], e] += hstep
            Bm[idx[j], e] -= hstep
            g = (loss_roles(Bp) - loss_roles(Bm)) / (2 * hstep)
            dacc[k, e] += g * g
            dval[k, e] += -lr * g / (np.sqrt(acc0[k, e] + g * g) + eps)
    np.testing.assert_allclose(o.table(0) - init, dval, rtol=5e-4, atol=1e-6)
    np.testing.assert_allclose(o.table(1) - acc0, dacc, rtol=5e-4, atol=1e-7)
    assert np.abs(dval).max() > 1e-3


def test_adagrad_closed_form_on_constant_gradient():
    # after t steps of a constant gradient g the accumulator is t*g^2 and the t-th step has size
    # lr/sqrt(t); driven through pull2/push2 exactly as a step does it
    o = Oracle(1, 1, workers=1, with_adagrad=True)
    g, lr = 0.5, 0.1
    for t in range(1, 6):
        v, a = o.pull(np.array([0], np.uint32), with_acc=True)
        assert abs(a[0, 0] - (t - 1) * g * g) < 1e-6
        step = -lr * g / np.sqrt(a[0, 0] + g * g)
        assert abs(step + lr / np.sqrt(t)) < 1e-6
        o.push(np.array([0], np.uint32), np.array([[step]], np.float32), np.array([[g * g]], np.float32))
    assert abs(o.table(0)[0, 0] + lr * sum(1 / np.sqrt(t) for t in range(1, 6))) < 1e-6


def test_complex_one_step_closed_form():
    # d = 1, real embeddings: phi = h*r*t, so d(phi)/d(r) = h*t and g_r = (sigmoid(phi) - 1) * h * t;
    # the first AdaGrad step with a zero accumulator and eps = 0 has size lr exactly.
    o = Oracle(3, 2, workers=1, with_adagrad=True)
    o.table(0)[:] = np.array([[1.0, 0.0], [0.5, 0.0], [2.0, 0.0]], np.float32)   # h, r, t
    d = o.register_distribution(0, None, 1, CONFORM, seed=0)
    o.step_complex(np.array([0], np.uint32), np.array([1], np.uint32), np.array([2], np.uint32), d, 0, 0.1, 0.0)
    phi = 1.0 * 0.5 * 2.0
    coef = 1 / (1 + np.exp(-phi)) - 1
    g_r = coef * 2.0                                        # h_re * t_re
    assert abs(o.table(1)[1, 0] - g_r ** 2) < 1e-7
    assert abs(o.table(0)[1, 0] - (0.5 - 0.1 * g_r / abs(g_r))) < 1e-6   # first AdaGrad step is lr * sign(g)


def test_mf_zero_gradient_at_true_factors_and_fd():
    M, N, L = 6, 5, 4
    rng = np.random.default_rng(4)
    Wt = rng.normal(size=(M, L))
    Ht = rng.normal(size=(N, L))
    o = Oracle(M + N, L, workers=2)
    o.table()[:M] = Wt.astype(np.float32)
    o.table()[M:] = Ht.astype(np.float32)
    T0 = o.table().copy()
    rows = np.array([0, 3, 5], np.uint32)
    cols = np.array([M + 1, M + 4, M + 0], np.uint32)
    x = np.array([T0[r].astype(np.float64) @ T0[c] for r, c in zip(rows, cols)], np.float32)
    loss = o.step_mf(rows, cols, x, 0.1, 0.0)
    assert loss < 1e-10
    np.testing.assert_allclose(o.table(), T0, atol=1e-6)
    # general point: update = -lr * d/dparam [ 1/2 e^2 + 1/2 l2 (|w|^2 + |h|^2) ], by finite differences
    lr, l2 = 0.05, 0.01
    xx = np.array([0.3], np.float32)
    o2 = Oracle(M + N, L, workers=1)
    o2.table()[:] = T0
    loss2 = o2.step_mf(np.array([2], np.uint32), np.array([M + 3], np.uint32), xx, lr, l2)
    T = T0.astype(np.float64)

    def obj(B):
        e = float(xx[0]) - B[2] @ B[M + 3]
        return 0.5 * e * e + 0.5 * l2 * (B[2] @ B[2] + B[M + 3] @ B[M + 3])
    assert abs(loss2 - (float(xx[0]) - T[2] @ T[M + 3]) ** 2) < 1e-5
    grad = np.zeros_like(T)
    for k in (2, M + 3):
        for e in range(L):
            Bp, Bm = T.copy(), T.copy()
            Bp[k, e] += 1e-6
            Bm[k, e] -= 1e-6
            grad[k, e] = (obj(Bp) - obj(Bm)) / 2e-6
    np.testing.assert_allclose(o2.table() - T0, -lr * grad, rtol=2e-4, atol=1e-7)


def test_steps_sync_interval_and_replicated_keys():
    V, L, K = 30, 4, 2
    rng = np.random.default_rng(6)
    init = rng.normal(0, 0.3, size=(2 * V, L)).astype(np.float32)
    c = rng.integers(0, V, 40).astype(np.uint32)
    ctx = (rng.integers(0, V, 40) + V).astype(np.uint32)
    outs = []
    for hot, interval in (([], 1), ([0, 1, 2, V, V + 1], 1), ([0, 1, 2, V, V + 1], 2)):
        o = Oracle(2 * V, L, workers=4, sync_interval=interval)
        o.table()[:] = init
        if hot:
            o.set_management(np.array(hot, np.uint32), REPLICATE)
        d = o.register_distribution(V, None, V, CONFORM, seed=1)
        losses = [o.step_sgns(c[i:i + 10], ctx[i:i + 10], d, K, 0.05) for i in range(0, 40, 10)]
        o.sync()
        outs.append((o.table().copy(), losses, o.stats()))
    np.testing.assert_allclose(outs[1][0], outs[0][0], rtol=1e-5, atol=1e-6)   # technique is transparent
    np.testing.assert_allclose(outs[1][1], outs[0][1], rtol=1e-6)
    assert outs[1][2]["syncs"] == 4 + 1 and outs[2][2]["syncs"] == 2 + 1   # automatic + the final one
    assert not np.allclose(outs[2][0], outs[0][0], rtol=1e-7, atol=1e-9)       # stale replicas differ a little
    np.testing.assert_allclose(outs[2][0], outs[0][0], rtol=0.2, atol=0.02)


def test_tiny_sgns_loss_decreases():
    from paper_2104_00501_b200 import inputs
    V, L, K = 200, 16, 3
    c, ctx, counts = inputs.sgns_batch_stream(V, 3000, 1.1, 0)
    w = inputs.integer_weights(counts).numpy().astype(np.uint32)
    o = Oracle(2 * V, L, workers=4)
    o.table()[:] = inputs.normal_init(2 * V, L, 0.1, 0)
    d = o.register_distribution(V, w, V, CONFORM, seed=0)
    c, ctx = inputs.u32(c), inputs.u32(ctx)
    losses = [o.step_sgns(c[i:i + 64], ctx[i:i + 64], d, K, 0.025) for i in range(0, 64 * 400, 64)]
    assert np.mean(losses[-50:]) < 0.9 * np.mean(losses[:50])


# ---------------------------------------------------------------------------------------------------------
# gradient-norm clipping for replicated keys (Section 5.1): pinned by a worked case with a closed form
# ---------------------------------------------------------------------------------------------------------
def _mf_clip_store(L=4):
    # rows 0..9 start at zero and are replicated; column key 10 holds h and is not replicated.  With w = 0 and
    # l2 = 0 a cell (i, 10, x) gives dw = lr * x * h (norm lr * |x| * |h|) and dh = lr * x * w = 0: h never moves.
    o = Oracle(11, L, workers=2)
    h = np.array([3.0, 0.0, 4.0, 0.0], np.float32)[:L]
    o.table()[10] = h
    o.set_management(np.arange(10, dtype=np.uint32), REPLICATE)
    return o, h


def test_clipping_closed_form_on_matrix_factorization_cells():
    lr = 0.5
    o, h = _mf_clip_store()
    o.set_clipping(2.0)
    hn = float(np.linalg.norm(h))                           # 5
    # step 1: nothing to compare with yet -> applied as it is; the mean norm becomes lr * 1 * 5 = 2.5
    o.step_mf([0], [10], [1.0], lr, 0.0)
    assert o.clip_stats() == (pytest.approx(lr * hn), 1)
    # step 2: two cells of one batch with x = 10 and x = -40: norms 25 and 100, both above 2 * 2.5 = 5 and both
    # judged against the same bound (the batch does not see itself): each becomes 5 long, direction kept
    o.step_mf([1, 2], [10, 10], [10.0, -40.0], lr, 0.0)
    s, c = o.clip_stats()
    assert c == 3 and s == pytest.approx(2.5 + 5.0 + 5.0)
    # step 3: mean is 12.5 / 3, bound 8.33: x = 3 (norm 7.5) passes, x = 4 (norm 10) is cut to 8.33
    o.step_mf([3, 4], [10, 10], [3.0, 4.0], lr, 0.0)
    o.sync()
    t = o.table()
    np.testing.assert_allclose(t[0], lr * 1.0 * h, rtol=1e-6)
    np.testing.assert_allclose(t[1], 5.0 * h / hn, rtol=1e-6)
    np.testing.assert_allclose(t[2], -5.0 * h / hn, rtol=1e-6)
    np.testing.assert_allclose(t[3], lr * 3.0 * h, rtol=1e-6)
    np.testing.assert_allclose(t[4], (2.0 * 12.5 / 3.0) * h / hn, rtol=1e-6)
    np.testing.assert_array_equal(t[10], h)                  # the column row never moved (w was zero)
    s, c = o.clip_stats()
    assert c == 5 and s == pytest.approx(12.5 + 7.5 + 2.0 * 12.5 / 3.0)


def test_clipping_leaves_non_replicated_keys_and_unclipped_runs_alone():
    rng = np.random.default_rng(5)
    V, L, K, n = 60, 8, 2, 64
    init = rng.normal(0, 0.5, (2 * V, L)).astype(np.float32)
    c, ctx = rng.integers(0, V, n).astype(np.uint32), (V + rng.integers(0, V, n)).astype(np.uint32)
    w = rng.integers(1, 50, V).astype(np.uint32)

    def run(hot, factor):
        o = Oracle(2 * V, L, workers=3)
        o.table()[:] = init
        if len(hot):
            o.set_management(np.asarray(hot, np.uint32), REPLICATE)
        o.set_clipping(factor)
        d = o.register_distribution(V, w, V, CONFORM, seed=4)
        for _ in range(4):
            o.step_sgns(c, ctx, d, K, 0.5)
        return o.table().copy(), o.clip_stats()

    plain, st0 = run([], 0.0)
    same, st1 = run([], 2.0)                                 # nothing replicated: nothing to clip, nothing counted
    assert np.array_equal(plain, same) and st0 == (0.0, 0) and st1 == (0.0, 0)
    hot = np.arange(0, 2 * V, 3)
    base, _ = run(hot, 0.0)
    huge, st = run(hot, 1e9)                                 # a bound nobody reaches: same values, norms still counted
    assert np.array_equal(base, huge) and st[1] > 0
    tight, _ = run(hot, 0.5)                                 # a tight bound changes replicated rows only through
    assert not np.array_equal(base, tight)                   # what was pushed to them; every update got shorter:
    d_base, d_tight = np.abs(base - init).sum(), np.abs(tight - init).sum()
    assert d_tight < d_base


def test_scores_beyond_thirty_are_clamped_in_skip_gram():
    # a positive pair whose score is 50: the clamp makes it 30, so loss = softplus(-30) (9.4e-14, not the
    # 1.9e-22 of an unclamped 50) and the gradient factor is sigmoid(30) - 1; the centre component that starts
    # at zero shows the update -lr * g * u exactly
    V, L, lr = 4, 4, 0.5
    o = Oracle(2 * V, L, workers=1)
    o.table()[1] = [5.0, 0.0, 0.0, 0.0]                     # centre v
    o.table()[V + 2] = [10.0, 1.0, 0.0, 0.0]                # context u: v.u = 50
    d = o.register_distribution(V, None, 1, CONFORM, seed=0)
    loss = o.step_sgns(np.array([1], np.uint32), np.array([V + 2], np.uint32), d, 0, lr)
    g = 1.0 / (1.0 + np.exp(-30.0)) - 1.0
    assert loss == pytest.approx(softplus(-30.0), rel=1e-5)
    assert loss > 1e-15                                     # softplus(-50) would be 1.9e-22
    assert o.table()[1, 1] == pytest.approx(-lr * g * 1.0, rel=1e-5)
    # a negative sample whose score is 50 (the distribution has one key, so the negative is known): loss term
    # softplus(30), not 50; a score of -50 for the positive pair: softplus(30) as well
    o2 = Oracle(2 * V, L, workers=1)
    o2.table()[1] = [5.0, 0.0, 0.0, 0.0]
    o2.table()[V] = [10.0, 1.0, 0.0, 0.0]                   # the only key negatives can be
    o2.table()[V + 3] = [-10.0, 0.0, 0.0, 0.0]              # context: v.u = -50
    d2 = o2.register_distribution(V, None, 1, CONFORM, seed=0)
    loss2, negs = o2.step_sgns(np.array([1], np.uint32), np.array([V + 3], np.uint32), d2, 1, lr, return_negatives=True)
    assert list(negs) == [V]
    assert loss2 == pytest.approx(2 * softplus(30.0), rel=1e-6)
    # the gradient factor of the clamped negative is sigmoid(30): u_neg -= lr * sigmoid(30) * v
    assert o2.table()[V, 0] == pytest.approx(10.0 - lr * (1.0 / (1.0 + np.exp(-30.0))) * 5.0, rel=1e-6)


def test_scores_beyond_thirty_are_clamped_in_complex():
    # d = 1, real parts only: phi = h r t = 50 -> clamped to 30.  With a zero accumulator the first AdaGrad step is
    # -lr g / (|g| + eps): for g = (sigmoid(30) - 1) * 10 = -9.4e-13 and eps = 1e-10 that is lr * 0.0093, where an
    # unclamped score of 50 (g = -1.9e-21) would give lr * 1.9e-11
    o = Oracle(3, 2, workers=1, with_adagrad=True)
    o.table(0)[:] = np.array([[5.0, 0.0], [1.0, 0.0], [10.0, 0.0]], np.float32)   # h, r, t
    d = o.register_distribution(0, None, 1, CONFORM, seed=0)
    lr, eps = 0.1, 1e-10
    loss = o.step_complex(np.array([0], np.uint32), np.array([1], np.uint32), np.array([2], np.uint32), d, 0, lr, eps)
    coef = 1.0 / (1.0 + np.exp(-30.0)) - 1.0
    assert loss == pytest.approx(softplus(-30.0), rel=1e-5)
    g_r = coef * 5.0 * 10.0                                 # d(phi)/d(r) = h t
    assert o.table(1)[1, 0] == pytest.approx(g_r ** 2, rel=1e-5)
    assert o.table(0)[1, 0] - 1.0 == pytest.approx(-lr * g_r / (abs(g_r) + eps), rel=1e-3)
    assert o.table(0)[1, 0] - 1.0 > 1e-4                    # an unclamped score would move it by 2e-12
