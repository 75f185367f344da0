"""CUDA path vs oracle: direct access, replica merge, counting, hot-set choice, management."""
import numpy as np
import pytest
import torch

from oracle import REPLICATE, SINGLE
from tests.common import dev_f32, dev_keys, host_keys, make_pair, tables_close, tables_equal

pytestmark = pytest.mark.gpu


def rand_table(nk, L, seed=0):
    return np.random.default_rng(seed).normal(size=(nk, L)).astype(np.float32)


@pytest.mark.parametrize("L", [4, 64, 100, 128, 300, 500])
@pytest.mark.parametrize("n", [0, 1, 31, 33, 1000, 4097])
def test_pull_bit_exact(L, n):
    nk = 977
    o, s = make_pair(nk, L, R=3, init=rand_table(nk, L))
    keys = np.random.default_rng(n).integers(0, nk, n).astype(np.uint32)
    got = s.pull(dev_keys(keys)).cpu().numpy()
    assert np.array_equal(got, o.pull(keys))


@pytest.mark.parametrize("L", [8, 64, 128, 256, 300])
@pytest.mark.parametrize("n", [1, 33, 4097])
def test_pull_with_replicated_keys_and_unmerged_updates_is_bit_exact(L, n):
    # rows of 64, 128 and 256 floats take the 256-bit copy kernel once keys are replicated; a replicated key reads as
    # stored row + the pulling worker's own unmerged updates
    nk, R = 977, 3
    rng = np.random.default_rng(L + n)
    o, s = make_pair(nk, L, R=R, init=rand_table(nk, L))
    hot = rng.choice(nk, 60, replace=False).astype(np.uint32)
    o.set_management(hot, REPLICATE)
    s.set_management(dev_keys(hot), REPLICATE)
    pk = np.where(rng.random(500) < 0.5, rng.choice(hot, 500), rng.integers(0, nk, 500)).astype(np.uint32)
    d = rng.normal(size=(500, L)).astype(np.float32)
    o.push(pk, d)
    s.push(dev_keys(pk), dev_f32(d))
    keys = np.where(rng.random(n) < 0.5, rng.choice(hot, n), rng.integers(0, nk, n)).astype(np.uint32)
    got = s.pull(dev_keys(keys)).cpu().numpy()
    assert np.array_equal(got, o.pull(keys))
    # an output buffer that starts 16 bytes into an allocation (not 32-byte aligned) takes the 128-bit kernel
    buf = torch.empty(n * L + 4, device="cuda")
    out = buf[4:].view(n, L)
    s.pull(dev_keys(keys), out)
    assert np.array_equal(out.cpu().numpy(), o.pull(keys))


def test_init_uniform_bit_exact():
    o, s = make_pair(1003, 12, with_adagrad=True)
    for which, seed, scale in ((0, 5, 0.25), (1, 6, 1e-3)):
        o.init_uniform(which, seed, scale)
        s.init_uniform(which, seed, scale)
        tables_equal(o, s, which)


def test_out_of_range_keys_are_skipped_and_reported():
    o, s = make_pair(50, 8, init=rand_table(50, 8))
    keys = np.array([1, 50, 2, 4000000000, 49], np.uint32)
    got = s.pull(dev_keys(keys)).cpu().numpy()
    assert np.array_equal(got, o.pull(keys))
    assert s.status_check() == -4 and s.status_check() == 0 and o.status() == -4
    d = rand_table(5, 8, 1)
    s.push(dev_keys(keys), dev_f32(d))
    o.push(keys, d)
    tables_equal(o, s)
    assert s.status_check() == -4


@pytest.mark.parametrize("hot_n", [0, 7, 200])
@pytest.mark.parametrize("L,R", [(8, 1), (64, 4), (300, 8)])
def test_push_sync_deterministic_is_bit_exact(L, R, hot_n):
    nk = 500
    rng = np.random.default_rng(L + hot_n)
    o, s = make_pair(nk, L, R=R, init=rand_table(nk, L), deterministic=True)
    if hot_n:
        hot = rng.permutation(nk)[:hot_n].astype(np.uint32)
        o.set_management(hot, REPLICATE)
        s.set_management(dev_keys(hot), REPLICATE)
    for it in range(4):
        n = [3000, 1, 4099, 257][it]
        keys = (rng.zipf(1.2, n) % nk).astype(np.uint32)
        d = rng.normal(size=(n, L)).astype(np.float32)
        o.push(keys, d)
        s.push(dev_keys(keys), dev_f32(d))
        # a worker reads its own pending updates
        pk = rng.integers(0, nk, 777).astype(np.uint32)
        assert np.array_equal(s.pull(dev_keys(pk)).cpu().numpy(), o.pull(pk))
        if it % 2 == 1:
            o.sync()
            s.sync()
            tables_equal(o, s)
    o.sync()
    s.sync()
    tables_equal(o, s)


@pytest.mark.parametrize("hot_n", [0, 50])
def test_push_fast_mode_conserves_updates(hot_n):
    nk, L, R = 300, 128, 4
    rng = np.random.default_rng(9)
    init = rand_table(nk, L)
    o, s = make_pair(nk, L, R=R, init=init, deterministic=False)
    if hot_n:
        hot = np.arange(hot_n, dtype=np.uint32)
        o.set_management(hot, REPLICATE)
        s.set_management(dev_keys(hot), REPLICATE)
    exact = init.astype(np.float64)
    for n in (5000, 33, 70000):
        keys = (rng.zipf(1.3, n) % nk).astype(np.uint32)
        d = rng.normal(size=(n, L)).astype(np.float32)
        o.push(keys, d)
        s.push(dev_keys(keys), dev_f32(d))
        np.add.at(exact, keys, d.astype(np.float64))
    o.sync()
    s.sync()
    got = s.read_table().cpu().numpy()
    scale = np.abs(exact).max()
    assert np.abs(got - exact).max() < 2e-5 * scale           # fp32 sums of thousands of terms, any order
    np.testing.assert_allclose(got, o.table(), rtol=1e-3, atol=2e-5 * scale)


def test_adagrad_two_table_push_and_pull():
    nk, L, R = 200, 20, 4
    rng = np.random.default_rng(2)
    o, s = make_pair(nk, L, R=R, init=rand_table(nk, L), acc_init=np.abs(rand_table(nk, L, 1)), with_adagrad=True)
    hot = np.array([3, 5, 150], np.uint32)
    o.set_management(hot, REPLICATE)
    s.set_management(dev_keys(hot), REPLICATE)
    keys = (rng.zipf(1.5, 2000) % nk).astype(np.uint32)
    dv, da = rng.normal(size=(2000, L)).astype(np.float32), rng.random((2000, L)).astype(np.float32)
    o.push(keys, dv, da)
    s.push(dev_keys(keys), dev_f32(dv), dev_f32(da))
    pk = rng.integers(0, nk, 500).astype(np.uint32)
    gv, ga = s.pull(dev_keys(pk), with_acc=True)
    ov, oa = o.pull(pk, with_acc=True)
    assert np.array_equal(gv.cpu().numpy(), ov) and np.array_equal(ga.cpu().numpy(), oa)
    o.sync()
    s.sync()
    tables_equal(o, s, 0)
    tables_equal(o, s, 1)


def test_no_replicated_key_launches_no_sync():
    o, s = make_pair(100, 8)
    before = s.stats()
    s.sync()
    after = s.stats()
    assert after["launches"] == before["launches"] and after["syncs"] == 0


def test_counts_and_hot_selection_bit_exact():
    nk = 5000
    rng = np.random.default_rng(4)
    o, s = make_pair(nk, 4)
    for n in (1, 100000, 4097):
        stream = (rng.zipf(1.2, n) % nk).astype(np.uint32)
        o.count_accesses(stream)
        s.count_accesses(dev_keys(stream))
    assert np.array_equal(s.counts().cpu().numpy().astype(np.uint64), o.counts())
    for k in (0, 1, 10, 999, nk, nk + 10):
        assert np.array_equal(host_keys(s.select_hot(True, k)), o.select_hot(True, k))
    for factor in (1, 5, 100, 10 ** 9):
        assert np.array_equal(host_keys(s.select_hot(False, factor)), o.select_hot(False, factor))
    assert len(o.select_hot(False, 100)) > 0


def test_access_counting_flag_counts_pull_push_and_samples():
    nk = 300
    rng = np.random.default_rng(5)
    o, s = make_pair(nk, 8, count_accesses=True, deterministic=True)
    hot = np.arange(10, dtype=np.uint32)
    o.set_management(hot, REPLICATE)
    s.set_management(dev_keys(hot), REPLICATE)
    k1 = (rng.zipf(1.3, 3000) % nk).astype(np.uint32)
    o.pull(k1)
    s.pull(dev_keys(k1))
    d = rng.normal(size=(3000, 8)).astype(np.float32)
    o.push(k1, d)
    s.push(dev_keys(k1), dev_f32(d))
    do = o.register_distribution(0, None, nk, 1, seed=3)
    ds = s.register_distribution(0, None, nk, 1, seed=3)
    o.pull_sample(o.prepare_sample(do, 1000), 1000)
    s.pull_sample(s.prepare_sample(ds, 1000), 1000)
    assert np.array_equal(s.counts().cpu().numpy().astype(np.uint64), o.counts())
    st, so = s.stats(), o.stats()
    assert st["hot"] == so["hot"] and st["cold"] == so["cold"]


def test_set_management_order_dedup_demotion():
    nk, L = 400, 8
    rng = np.random.default_rng(6)
    o, s = make_pair(nk, L, R=4, init=rand_table(nk, L), deterministic=True)
    lists = [np.array([5, 2, 5, 9, 399, 2], np.uint32), rng.integers(0, nk, 300).astype(np.uint32)]
    for ks in lists:
        o.set_management(ks, REPLICATE)
        s.set_management(dev_keys(ks), REPLICATE)
        assert np.array_equal(host_keys(s.hot_keys()), o.hot_keys())
    keys = rng.integers(0, nk, 2000).astype(np.uint32)
    d = rng.normal(size=(2000, L)).astype(np.float32)
    o.push(keys, d)
    s.push(dev_keys(keys), dev_f32(d))
    drop = np.concatenate([o.hot_keys()[::3], np.array([1, 7], np.uint32)])
    o.set_management(drop, SINGLE)
    s.set_management(dev_keys(drop), SINGLE)          # merges the pending updates first
    assert np.array_equal(host_keys(s.hot_keys()), o.hot_keys())
    tables_equal(o, s)
    o.push(keys, d)
    s.push(dev_keys(keys), dev_f32(d))
    o.sync()
    s.sync()
    tables_equal(o, s)


def test_localize_and_owner_map():
    nk, R = 1000, 5
    rng = np.random.default_rng(7)
    o, s = make_pair(nk, 4, R=R, track_ownership=True)
    hot = np.array([0, 10, 20], np.uint32)
    o.set_management(hot, REPLICATE)
    s.set_management(dev_keys(hot), REPLICATE)
    for n in (1, 333, 5000):
        ks = rng.integers(0, nk, n).astype(np.uint32)
        o.localize(ks)
        s.localize(dev_keys(ks))
    allk = np.arange(nk, dtype=np.uint32)
    got = s.owner_of(dev_keys(allk)).cpu().numpy()
    want = np.array([o.owner_of(k) for k in allk])
    assert np.array_equal(got, want)


@pytest.mark.parametrize("L", [4, 128, 300, 500])
@pytest.mark.parametrize("hot_n", [0, 300])
def test_large_calls_take_the_staged_path_and_stay_exact(L, hot_n):
    # calls of 16384 keys and more run as persistent blocks that stage rows through shared memory;
    # ragged tail, keys out of range and replicated keys with pending updates included
    nk, R = 20000, 5
    rng = np.random.default_rng(L + hot_n)
    init = rand_table(nk, L)
    o, s = make_pair(nk, L, R=R, init=init, deterministic=False, count_accesses=True)
    if hot_n:
        hot = rng.permutation(nk)[:hot_n].astype(np.uint32)
        o.set_management(hot, REPLICATE)
        s.set_management(dev_keys(hot), REPLICATE)
    exact = init.astype(np.float64)
    for n in (16384, 70001):
        keys = (rng.zipf(1.15, n) % nk).astype(np.uint32)
        keys[rng.integers(0, n, 5)] = nk + 7                      # bad keys: skipped, output zero-filled
        d = rng.normal(size=(n, L)).astype(np.float32)
        o.push(keys, d)
        s.push(dev_keys(keys), dev_f32(d))
        ok = keys < nk
        np.add.at(exact, keys[ok], d[ok].astype(np.float64))
        got = s.pull(dev_keys(keys)).cpu().numpy()
        want = o.pull(keys)
        scale = max(1.0, np.abs(want).max())
        assert np.abs(got - want).max() < 3e-5 * scale            # pending updates were added in another order
        assert np.all(got[~ok] == 0)
        assert s.status_check() == -4
    o.sync()
    s.sync()
    got = s.read_table().cpu().numpy()
    assert np.abs(got - exact).max() < 3e-5 * np.abs(exact).max()
    # a pull with nothing pending is an exact copy
    keys = rng.integers(0, nk, 50000).astype(np.uint32)
    assert np.array_equal(s.pull(dev_keys(keys)).cpu().numpy(), got[keys])
    o.pull(keys)
    assert np.array_equal(s.counts().cpu().numpy().astype(np.uint64), o.counts())
    st, so = s.stats(), o.stats()
    assert st["hot"] == so["hot"] and st["cold"] == so["cold"]
