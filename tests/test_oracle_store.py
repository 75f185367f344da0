"""Pins of the oracle's direct-access path: pull, push, sync, counting, hot-set choice, management."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from oracle import Oracle, REPLICATE, SINGLE


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



def brute_tables(nk, L, seed=0):
    rng = np.random.default_rng(seed)
    return rng.normal(size=(nk, L)).astype(np.float32)


def test_pull_is_plain_indexing_on_tiny_table():
    o = Oracle(10, 4, workers=3)
    t = brute_tables(10, 4)
    o.table()[:] = t
    keys = np.array([9, 0, 3, 3, 7, 0, 5], np.uint32)
    out = o.pull(keys)
    for i, k in enumerate(keys):                      # brute force, row by row
        assert np.array_equal(out[i], t[k])
    assert o.pull(np.zeros(0, np.uint32)).shape == (0, 4)


def test_out_of_range_key_is_skipped_and_flagged():
    o = Oracle(10, 4)
    o.table()[:] = 1.0
    out = o.pull(np.array([1, 10, 2], np.uint32))
    assert np.array_equal(out[1], np.zeros(4)) and out[0, 0] == 1.0
    assert o.status() == oracle.EKEY and o.status() == 0
    o.push(np.array([11], np.uint32), np.ones((1, 4), np.float32))
    assert o.status() == oracle.EKEY
    assert np.all(o.table() == 1.0)


@pytest.mark.parametrize("R,hot", [(1, []), (4, []), (4, [3, 7, 1]), (8, list(range(10)))])
def test_conservation_value_is_init_plus_all_pushed_deltas(R, hot):
    # pin: after sync, value = init + sum of pushed deltas, whatever the hot set
    nk, L = 10, 6
    rng = np.random.default_rng(1)
    o = Oracle(nk, L, workers=R)
    init = brute_tables(nk, L)
    o.table()[:] = init
    if hot:
        o.set_management(np.array(hot, np.uint32), REPLICATE)
    exact = init.astype(np.float64)
    for _ in range(5):
        keys = rng.integers(0, nk, 37).astype(np.uint32)
        d = rng.normal(size=(37, L)).astype(np.float32)
        o.push(keys, d)
        np.add.at(exact, keys, d.astype(np.float64))
        if hot:                                        # pending updates are not visible in the table yet
            assert np.array_equal(o.table()[hot], init[hot]) or _ > 0
    o.sync()
    np.testing.assert_allclose(o.table(), exact, rtol=1e-5, atol=1e-5)
    # a dropped or doubled delta would be far outside this tolerance
    assert np.abs(o.table() - init).max() > 1.0


def test_replica_read_sees_own_pending_updates_only():
    o = Oracle(4, 2, workers=2)
    o.set_management(np.array([1], np.uint32), REPLICATE)
    # 2 items: item 0 -> worker 0, item 1 -> worker 1
    o.push(np.array([1, 2], np.uint32), np.array([[1, 1], [5, 5]], np.float32))
    got = o.pull(np.array([1, 1], np.uint32))          # worker 0 then worker 1 read key 1
    assert np.array_equal(got, [[1, 1], [0, 0]])
    assert np.array_equal(o.table()[1], [0, 0])        # stored row untouched until the merge
    assert np.array_equal(o.table()[2], [5, 5])        # a single key is updated in place
    o.sync()
    assert np.array_equal(o.pull(np.array([1, 1], np.uint32)), [[1, 1], [1, 1]])
    assert np.array_equal(o.table()[1], [1, 1])


def test_technique_is_transparent_at_sync_every_step():
    nk, L = 50, 8
    rng = np.random.default_rng(3)
    init = brute_tables(nk, L)
    results = []
    for hot in ([], [0, 1, 2, 3, 4, 5], list(range(nk))):
        o = Oracle(nk, L, workers=4)
        o.table()[:] = init
        if hot:
            o.set_management(np.array(hot, np.uint32), REPLICATE)
        r2 = np.random.default_rng(4)
        for _ in range(10):
            keys = r2.integers(0, nk, 64).astype(np.uint32)
            o.push(keys, r2.normal(size=(64, L)).astype(np.float32))
            o.sync()
        results.append(o.table().copy())
    np.testing.assert_allclose(results[1], results[0], rtol=1e-5, atol=1e-5)
    np.testing.assert_allclose(results[2], results[0], rtol=1e-5, atol=1e-5)


def test_no_replicated_key_means_no_sync_work():
    o = Oracle(10, 2)
    o.push(np.array([1], np.uint32), np.ones((1, 2), np.float32))
    o.sync()
    assert o.stats()["syncs"] == 0


def test_push_applies_duplicates_in_item_order(both_value_types):
    # three adds whose result in the table's precision depends on the order: 2^24 + 1 + 1 in fp32, 2^53 + 1 + 1 in fp64
    ft, big = (np.float32, 2.0 ** 24) if both_value_types == 4 else (np.float64, 2.0 ** 53)
    big, small = ft(big), ft(1.0)
    o = Oracle(2, 1, workers=1)
    o.push(np.array([0, 0, 0], np.uint32), np.array([[big], [small], [small]], ft))
    assert o.table().dtype == ft
    assert o.table()[0, 0] == ft(ft(big + small) + small) == big
    o2 = Oracle(2, 1, workers=1)
    o2.push(np.array([0, 0, 0], np.uint32), np.array([[small], [small], [big]], ft))
    assert o2.table()[0, 0] == big + 2


def test_adagrad_table_pushes_both():
    o = Oracle(5, 3, workers=2, with_adagrad=True)
    o.set_management(np.array([4], np.uint32), REPLICATE)
    keys = np.array([4, 0, 4], np.uint32)
    dv = np.ones((3, 3), np.float32)
    da = np.full((3, 3), 2.0, np.float32)
    o.push(keys, dv, da)
    v, a = o.pull(np.array([4, 4, 0, 0], np.uint32), with_acc=True)   # workers 0,0,1,1
    assert v[0, 0] == 1 and a[0, 0] == 2 and v[2, 0] == 1 and a[3, 0] == 2
    o.sync()
    assert np.all(o.table(0)[4] == 2) and np.all(o.table(1)[4] == 4)
    assert np.all(o.table(1)[0] == 2)


def test_counts_and_selection_brute_force():
    nk = 200
    rng = np.random.default_rng(5)
    o = Oracle(nk, 1)
    stream = (rng.zipf(1.3, 20000) % nk).astype(np.uint32)
    o.count_accesses(stream)
    cnt = o.counts()
    assert cnt.sum() == len(stream)
    assert np.array_equal(cnt, np.bincount(stream, minlength=nk))
    order = sorted(range(nk), key=lambda k: (-int(cnt[k]), k))
    for k in (0, 1, 7, 50, nk, nk + 5):
        assert list(o.select_hot(True, k)) == order[:k]
    total = int(cnt.sum())
    for factor in (1, 2, 10, 100):
        want = [k for k in order if Fraction(int(cnt[k])) > factor * Fraction(total, nk)]
        assert list(o.select_hot(False, factor)) == want
    assert len(o.select_hot(False, 10)) > 0


def test_threshold_rule_is_strict():
    o = Oracle(4, 1)
    o.count_accesses(np.array([0, 0, 1, 2], np.uint32))     # mean = 1; cnt = 2,1,1,0
    assert list(o.select_hot(False, 1)) == [0]               # 1 > 1 is false
    assert list(o.select_hot(False, 2)) == []                # 2 > 2 is false


def test_access_counting_flag_counts_every_access():
    o = Oracle(6, 2, count_accesses=True)
    o.pull(np.array([1, 1, 2], np.uint32))
    o.push(np.array([2, 3], np.uint32), np.zeros((2, 2), np.float32))
    d = o.register_distribution(0, None, 6, oracle.CONFORM, seed=0)
    ks = o.pull_sample(o.prepare_sample(d, 5), 5, values=False)
    want = np.bincount([1, 1, 2, 2, 3] + list(ks), minlength=6)
    assert np.array_equal(o.counts(), want)


def test_set_management_order_dedup_and_demotion():
    o = Oracle(10, 2, workers=2)
    o.table()[:] = 1.0
    o.set_management(np.array([5, 2, 5, 9], np.uint32), REPLICATE)
    assert list(o.hot_keys()) == [5, 2, 9]
    o.set_management(np.array([2, 7], np.uint32), REPLICATE)
    assert list(o.hot_keys()) == [5, 2, 9, 7]
    o.push(np.array([5, 9], np.uint32), np.ones((2, 2), np.float32))
    o.set_management(np.array([5, 3], np.uint32), SINGLE)   # merges pending updates first
    assert list(o.hot_keys()) == [2, 9, 7]
    assert np.all(o.table()[5] == 2.0) and np.all(o.table()[9] == 2.0)
    o.push(np.array([9], np.uint32), np.ones((1, 2), np.float32))
    o.sync()
    assert np.all(o.table()[9] == 3.0)


def test_init_uniform_range_mean_and_determinism():
    o = Oracle(1000, 8)
    o.init_uniform(0, 42, 0.5)
    t = o.table().copy()
    assert t.min() >= -0.5 and t.max() < 0.5 and abs(t.mean()) < 0.01
    assert abs(t.std() - 0.5 / np.sqrt(3)) < 0.01
    o2 = Oracle(1000, 8)
    o2.init_uniform(0, 42, 0.5)
    assert np.array_equal(t, o2.table())
    o2.init_uniform(0, 43, 0.5)
    assert not np.array_equal(t, o2.table())


def test_merge_mean_adds_the_mean_over_the_workers_that_pushed():
    # closed form: a replicated key that two of four workers push to receives (d1 + d2) / 2 at the merge, a key that
    # one worker pushes to twice receives both updates in full (one worker: mean = sum), a key that is not replicated
    # is updated in place as always
    from oracle import Oracle, REPLICATE
    L, R = 4, 4
    o = Oracle(8, L, workers=R)
    o.set_merge_mean(True)
    o.set_management(np.array([1, 2], np.uint32), REPLICATE)
    d = np.array([[1.0, 2.0, 4.0, 8.0], [3.0, 2.0, 0.0, -8.0], [0.5, 0.5, 0.5, 0.5], [0.25, 0.0, 0.0, 0.0]], np.float32)
    # four items, one per worker: workers 0 and 1 push to key 1, workers 2 and 3 to key 5 (not replicated)
    o.push(np.array([1, 1, 5, 5], np.uint32), d)
    # eight items, two per worker: worker 0 pushes twice to key 2
    o.push(np.array([2, 2, 7, 7, 7, 7, 7, 7], np.uint32), np.concatenate([d[:2], np.zeros((6, L), np.float32)]))
    assert not o.table()[1].any() and not o.table()[2].any()        # still pending in the replicas
    o.sync()
    np.testing.assert_array_equal(o.table()[1], (d[0] + d[1]) / 2)
    np.testing.assert_array_equal(o.table()[2], d[0] + d[1])
    np.testing.assert_array_equal(o.table()[5], d[2] + d[3])
    # the flags were cleared: a second merge changes nothing, and a later single push counts one worker
    o.sync()
    np.testing.assert_array_equal(o.table()[1], (d[0] + d[1]) / 2)
    o.push(np.array([1], np.uint32), d[3:4])
    o.sync()
    np.testing.assert_array_equal(o.table()[1], (d[0] + d[1]) / 2 + d[3])


def test_fp64_build_keeps_what_fp32_rounds_away():
    # conservation in the 8-byte build: value = init + sum of pushed deltas to 1e-15 relative (fp64 additions of a few
    # dozen terms), and an update of 1e-12 to a value of 1 is kept, which the 4-byte build cannot do
    nk, L, R = 12, 5, 3
    rng = np.random.default_rng(7)
    o = Oracle(nk, L, workers=R, value_bytes=8)
    init = rng.normal(size=(nk, L))
    o.table()[:] = init
    o.set_management(np.array([2, 3, 11], np.uint32), REPLICATE)
    exact = [[Fraction(float(x)) for x in row] for row in init]
    for _ in range(4):
        keys = rng.integers(0, nk, 29).astype(np.uint32)
        d = rng.normal(size=(29, L)) * 1e-6
        o.push(keys, d)
        for i, k in enumerate(keys):
            for e in range(L):
                exact[k][e] += Fraction(float(d[i, e]))
    o.sync()
    want = np.array([[float(x) for x in row] for row in exact])
    np.testing.assert_allclose(o.table(), want, rtol=1e-14, atol=0)
    assert np.abs(o.table() - init).max() > 1e-7
    one = Oracle(2, 1, workers=1, value_bytes=8)
    one.table()[:] = 1.0
    one.push(np.array([0], np.uint32), np.array([[1e-12]]))
    assert one.table()[0, 0] == 1.0 + 1e-12 and one.table()[1, 0] == 1.0
    four = Oracle(2, 1, workers=1, value_bytes=4)
    four.table()[:] = 1.0
    four.push(np.array([0], np.uint32), np.array([[1e-12]], np.float32))
    assert four.table()[0, 0] == 1.0
