"""CUDA path vs oracle on the degenerate and extreme cases of the method."""
import numpy as np
import pytest
import torch

from oracle import BOUNDED, CONFORM, REPLICATE
from paper_2104_00501_b200 import binding, inputs
from tests.common import dev_f32, dev_keys, host_keys, make_pair, tables_close, tables_equal

pytestmark = pytest.mark.gpu


def test_empty_calls_are_noops_and_bad_sizes_are_refused():
    o, s = make_pair(50, 8, init=np.ones((50, 8), np.float32))
    empty_k = torch.zeros(0, dtype=torch.int32, device="cuda")
    empty_v = torch.zeros((0, 8), dtype=torch.float32, device="cuda")
    before = s.stats()["launches"]
    assert s.pull(empty_k).shape == (0, 8)
    s.push(empty_k, empty_v)
    s.count_accesses(empty_k)
    s.localize(empty_k)
    s.set_management(empty_k, REPLICATE)
    assert s.stats()["launches"] == before
    tables_equal(o, s)
    d = s.register_distribution(0, None, 50, CONFORM)
    for call in (lambda: s.prepare_sample(d, 0), lambda: s.step_sgns(empty_k, empty_k, d, 3, 0.1),
                 lambda: s.step_mf(empty_k, empty_k, torch.zeros(0, device="cuda"), 0.1, 0.1),
                 lambda: s.register_distribution(0, None, 0, CONFORM), lambda: s.prepare_sample(99, 5)):
        with pytest.raises(binding.NupsError) as e:
            call()
        assert e.value.code == binding.EINVAL
    with pytest.raises(binding.NupsError):
        binding.Store(10, 6)                       # rows must be multiples of 16 bytes
    with pytest.raises(binding.NupsError):
        binding.Store(10, 8, workers=255)


@pytest.mark.parametrize("K", [0, 30])
def test_sgns_extreme_negative_counts_and_widest_rows(K):
    V, L, n = 90, 512, 70
    c, ctx, counts = inputs.sgns_batch_stream(V, 40, 1.1, 3)
    c, ctx = inputs.u32(c)[:n], inputs.u32(ctx)[:n]
    w = inputs.integer_weights(counts).numpy().astype(np.uint32)
    init = inputs.normal_init(2 * V, L, 0.05, 3)
    o, s = make_pair(2 * V, L, R=3, init=init, deterministic=True, count_accesses=True)
    hot = np.array([0, 1, V, V + 1], np.uint32)
    o.set_management(hot, REPLICATE)
    s.set_management(dev_keys(hot), REPLICATE)
    do = o.register_distribution(V, w, V, CONFORM, seed=1)
    ds = s.register_distribution(V, dev_keys(w), V, CONFORM, seed=1)
    lb = torch.zeros(1, device="cuda")
    lo, negs = o.step_sgns(c, ctx, do, K, 0.05, return_negatives=True)
    s.step_sgns(dev_keys(c), dev_keys(ctx), ds, K, 0.05, lb)
    assert np.array_equal(host_keys(s.last_negatives()), negs)
    assert abs(lb.item() - lo) <= 1e-5 * abs(lo)
    o.sync()
    s.sync()
    tables_close(o, s)
    assert np.array_equal(s.counts().cpu().numpy().astype(np.uint64), o.counts())
    with pytest.raises(binding.NupsError):
        s.step_sgns(dev_keys(c), dev_keys(ctx), ds, 31, 0.05, lb)


def test_complex_thirty_negatives_widest_rows():
    E, Rl, L, K, n = 60, 4, 512, 30, 40
    h, r, t = [inputs.u32(x) for x in inputs.kge_triples(n, E, Rl, 0.9, 1.2, 1)]
    rng = np.random.default_rng(1)
    init = rng.normal(0, 0.05, size=(E + Rl, L)).astype(np.float32)
    acc0 = rng.uniform(0.1, 0.2, size=(E + Rl, L)).astype(np.float32)
    o, s = make_pair(E + Rl, L, R=2, init=init, acc_init=acc0, deterministic=True, with_adagrad=True)
    do = o.register_distribution(0, None, E, CONFORM, seed=2)
    ds = s.register_distribution(0, None, E, CONFORM, seed=2)
    lb = torch.zeros(1, device="cuda")
    lo, negs = o.step_complex(h, r, t, do, K, 0.1, 1e-10, return_negatives=True)
    s.step_complex(dev_keys(h), dev_keys(r), dev_keys(t), ds, K, 0.1, 1e-10, lb)
    assert np.array_equal(host_keys(s.last_negatives()), negs)
    assert abs(lb.item() - lo) <= 1e-5 * abs(lo)
    tables_close(o, s, 0)
    tables_close(o, s, 1)


@pytest.mark.parametrize("R", [1, 254])
def test_one_and_many_workers(R):
    nk, L = 300, 8
    rng = np.random.default_rng(R)
    o, s = make_pair(nk, L, R=R, init=rng.normal(size=(nk, L)).astype(np.float32), deterministic=True,
                     track_ownership=True)
    hot = np.arange(0, nk, 7, dtype=np.uint32)
    o.set_management(hot, REPLICATE)
    s.set_management(dev_keys(hot), REPLICATE)
    for n in (5, 1000):                                   # fewer items than workers, and more
        keys = rng.integers(0, nk, n).astype(np.uint32)
        d = rng.normal(size=(n, L)).astype(np.float32)
        o.push(keys, d)
        s.push(dev_keys(keys), dev_f32(d))
        assert np.array_equal(s.pull(dev_keys(keys)).cpu().numpy(), o.pull(keys))
    do = o.register_distribution(0, None, nk, BOUNDED, U=2, G=9, seed=5)
    ds = s.register_distribution(0, None, nk, BOUNDED, U=2, G=9, seed=5)
    for N in (3, 700):
        ko, vo = o.pull_sample(o.prepare_sample(do, N), N)
        ks, vs = s.pull_sample(s.prepare_sample(ds, N), N)
        assert np.array_equal(host_keys(ks), ko) and np.array_equal(vs.cpu().numpy(), vo)
    o.sync()
    s.sync()
    tables_equal(o, s)


def test_everything_replicated_one_hot_key_and_a_one_key_store():
    # every key replicated
    nk, L = 64, 16
    rng = np.random.default_rng(0)
    o, s = make_pair(nk, L, R=4, init=rng.normal(size=(nk, L)).astype(np.float32), deterministic=True)
    allk = np.arange(nk, dtype=np.uint32)
    o.set_management(allk, REPLICATE)
    s.set_management(dev_keys(allk), REPLICATE)
    # a batch in which every item hits the same key
    keys = np.full(5000, 17, np.uint32)
    d = rng.normal(size=(5000, L)).astype(np.float32)
    o.push(keys, d)
    s.push(dev_keys(keys), dev_f32(d))
    o.sync()
    s.sync()
    tables_equal(o, s)
    # the same in fast mode: conservation within rounding
    _, f = make_pair(nk, L, R=4, deterministic=False)
    f.push(dev_keys(np.tile(keys, 8)), dev_f32(np.tile(d, (8, 1))))
    got = f.read_table().cpu().numpy()[17]
    want = 8 * d.astype(np.float64).sum(0)
    assert np.abs(got - want).max() < 1e-4 * np.abs(want).max() + 1e-3
    # a store with a single key
    o1, s1 = make_pair(1, 4, R=2, deterministic=True)
    k1 = np.zeros(33, np.uint32)
    o1.push(k1, np.ones((33, 4), np.float32))
    s1.push(dev_keys(k1), dev_f32(np.ones((33, 4), np.float32)))
    tables_equal(o1, s1)
    d1o = o1.register_distribution(0, None, 1, CONFORM)
    d1s = s1.register_distribution(0, None, 1, CONFORM)
    assert np.array_equal(host_keys(s1.pull_sample(s1.prepare_sample(d1s, 9), 9, values=False)),
                          o1.pull_sample(o1.prepare_sample(d1o, 9), 9, values=False))


def test_scores_beyond_thirty_are_clamped_like_the_oracles():
    # rows long enough for scores far beyond +-30 on both sides of zero: loss and updates follow the oracle's clamp
    V, L, K, n = 40, 16, 3, 64
    rng = np.random.default_rng(4)
    init = rng.normal(0, 2.5, size=(2 * V, L)).astype(np.float32)            # |v.u| is typically ~25, often > 30
    c = rng.integers(0, V, n).astype(np.uint32)
    ctx = (V + rng.integers(0, V, n)).astype(np.uint32)
    scores = np.einsum("ij,ij->i", init[c].astype(np.float64), init[ctx].astype(np.float64))
    assert (scores > 35).sum() >= 2 and (scores < -35).sum() >= 2
    o, s = make_pair(2 * V, L, R=2, init=init, deterministic=True)
    do = o.register_distribution(V, None, V, CONFORM, seed=2)
    ds = s.register_distribution(V, None, V, CONFORM, seed=2)
    lb = torch.zeros(1, device="cuda")
    lo = o.step_sgns(c, ctx, do, K, 0.01)
    s.step_sgns(dev_keys(c), dev_keys(ctx), ds, K, 0.01, lb)
    assert abs(lb.item() - lo) <= 1e-5 * abs(lo)
    tables_close(o, s)
    # ComplEx: the same with trilinear scores
    E, Rl, Lc = 30, 3, 8
    init = rng.normal(0, 2.2, size=(E + Rl, Lc)).astype(np.float32)
    acc0 = np.full((E + Rl, Lc), 0.5, np.float32)
    h, r, t = [inputs.u32(x) for x in inputs.kge_triples(48, E, Rl, 0.9, 1.2, 4)]
    oc, sc = make_pair(E + Rl, Lc, R=2, init=init, acc_init=acc0, deterministic=True, with_adagrad=True)
    dco = oc.register_distribution(0, None, E, CONFORM, seed=3)
    dcs = sc.register_distribution(0, None, E, CONFORM, seed=3)
    lo = oc.step_complex(h, r, t, dco, 4, 0.05, 1e-10)
    sc.step_complex(dev_keys(h), dev_keys(r), dev_keys(t), dcs, 4, 0.05, 1e-10, lb)
    assert lo > 30.0                                                        # clamped scores dominate the loss
    assert abs(lb.item() - lo) <= 1e-5 * abs(lo)
    tables_close(oc, sc, 0)
    tables_close(oc, sc, 1)


@pytest.mark.parametrize("deterministic", [True, False])
def test_calls_see_what_the_streams_earlier_kernels_wrote(deterministic):
    """The kernels may become resident before the stream's previous kernel has ended (they are launched as programmatic
    dependents) but wait before they read: keys and update rows written by the caller's kernels just before a call, with
    no synchronization in between, are the ones the call uses, and a call's results are there for the caller's next kernel."""
    nk, L, n = 4000, 32, 3000
    init = inputs.normal_init(nk, L, 0.1, 5)
    o, s = make_pair(nk, L, R=4, init=init, deterministic=deterministic)
    hot = np.arange(0, 64, dtype=np.uint32)
    o.set_management(hot, REPLICATE)
    s.set_management(dev_keys(hot), REPLICATE)
    rng = np.random.default_rng(7)
    k0 = rng.integers(0, nk, n).astype(np.uint32)
    d0 = rng.standard_normal((n, L)).astype(np.float32)
    keys = dev_keys(k0)
    delta = dev_f32(d0)
    out = torch.empty((n, L), device="cuda")
    total = torch.zeros((), device="cuda", dtype=torch.float64)
    want_total = 0.0
    for it in range(12):
        keys.copy_((keys.long() * 7 + it) % nk)              # the caller's kernels write keys and rows ...
        delta.mul_(-0.5).add_(float(it))
        s.push(keys, delta)                                  # ... which the very next launches read
        s.pull(keys, out)
        total += out.double().sum()                          # and the caller's next kernel reads the result
        k0 = ((k0.astype(np.int64) * 7 + it) % nk).astype(np.uint32)
        d0 = (d0 * np.float32(-0.5) + np.float32(it)).astype(np.float32)
        o.push(k0, d0)
        want_total += float(o.pull(k0).astype(np.float64).sum())
    if deterministic:
        tables_equal(o, s)
        assert abs(total.item() - want_total) <= 1e-9 * max(1.0, abs(want_total))
    else:                                                    # additions in another order: rounding only
        tables_close(o, s, rtol=1e-4, atol=1e-4)
        assert abs(total.item() - want_total) <= 1e-5 * max(1.0, abs(want_total))
