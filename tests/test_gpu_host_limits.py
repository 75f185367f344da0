"""The store's own memory limit (every path that allocates), the wrap-around of the 24-bit counter of key-moving
calls, and the mean-instead-of-sum merge, on the device against the oracle."""
import numpy as np
import pytest
import torch

from oracle import BOUNDED, CONFORM, LONGTERM, Oracle, REPLICATE
from paper_2104_00501_b200 import binding, inputs
from tests.common import dev_f32, dev_keys, host_keys, make_pair, tables_close, tables_equal

pytestmark = pytest.mark.gpu


def _enomem(call):
    with pytest.raises(binding.NupsError) as e:
        call()
    assert e.value.code == binding.ENOMEM


def test_every_allocating_call_respects_the_stores_limit_and_leaves_the_store_usable():
    # 100,000 keys x 8 floats with ownership tracking: tables and maps take ~5.1 MB; limit 8 MiB
    nk, L, R = 100_000, 8, 4
    s = binding.Store(nk, L, workers=R, deterministic=True, track_ownership=True, max_device_mib=8)
    rng = np.random.default_rng(0)
    # replicating 20,000 keys needs 4 workers x 25,016 rows x 32 bytes = 3.2 MB of replicas on top of the scratch of
    # the call: refused, nothing changes
    many = dev_keys(rng.permutation(nk)[:20_000].astype(np.uint32))
    _enomem(lambda: s.set_management(many, binding.REPLICATE))
    assert s.stats()["hot_slots"] == 0
    # an ordered push of 120,000 rows needs ~4.7 MB of sort buffers: refused; a smaller one goes through
    keys = dev_keys(rng.integers(0, nk, 120_000).astype(np.uint32))
    delta = torch.ones((120_000, L), device="cuda")
    _enomem(lambda: s.push(keys, delta))
    assert not s.read_table().any()
    s.push(keys[:2000].contiguous(), delta[:2000].contiguous())
    assert float(s.read_table().sum()) == 2000 * L
    # an alias table over all keys needs ~5 MB of build buffers: refused; one over 1,000 keys is built
    w = torch.ones(nk, dtype=torch.int32, device="cuda")
    _enomem(lambda: s.register_distribution(0, w, nk, binding.CONFORM))
    d = s.register_distribution(0, w[:1000].contiguous(), 1000, binding.LONGTERM, U=2, G=10)
    # a handle of 400,000 samples (keys, postponing lists) does not fit, one of 4,000 does
    _enomem(lambda: s.prepare_sample(d, 400_000))
    ks = s.pull_sample(s.prepare_sample(d, 4000), 4000, values=False)
    assert int(ks.max()) < 1000
    # a step over 150,000 pairs (450,000 negatives, update rows of the ordered mode) does not fit, one over 100 does
    c = dev_keys(rng.integers(0, 500, 150_000).astype(np.uint32))
    _enomem(lambda: s.step_sgns(c, c, d, 3, 0.1))
    s.step_sgns(c[:100].contiguous(), c[:100].contiguous(), d, 3, 0.1)
    assert s.status_check() == 0
    # the agreed copy of the table that merging across GPUs keeps (another 3.2 MB) does not fit either
    _enomem(lambda: s.merge_mark())
    with pytest.raises(binding.NupsError) as e:
        s.merge_export()
    assert e.value.code == binding.ESTATE
    s.close()
    # without a limit the same calls succeed
    s = binding.Store(nk, L, workers=R, deterministic=True, track_ownership=True)
    s.set_management(many, binding.REPLICATE)
    s.push(keys, delta)
    assert s.status_check() == 0
    s.close()


@pytest.mark.parametrize("level", [BOUNDED, LONGTERM])
def test_ownership_survives_the_wrap_of_the_call_counter(level):
    # calls that move keys are numbered with 24 bits inside the ownership words; start three calls before the
    # counter runs out and keep moving keys across the wrap: owners and sampled keys stay the oracle's
    nk, L, R = 4000, 4, 5
    o = Oracle(nk, L, workers=R, track_ownership=True)
    s = binding.Store(nk, L, workers=R, deterministic=True, track_ownership=True, first_epoch=0xFFFFFF - 3)
    hot = np.array([7, 8, 9], np.uint32)
    o.set_management(hot, REPLICATE)
    s.set_management(dev_keys(hot), binding.REPLICATE)
    w = inputs.zipf_integer_weights(nk, 0.9).numpy().astype(np.uint32)
    do = o.register_distribution(0, w, nk, level, U=3, G=40, seed=5)
    ds = s.register_distribution(0, dev_keys(w), nk, level, U=3, G=40, seed=5)
    rng = np.random.default_rng(3)
    allk = np.arange(nk, dtype=np.uint32)
    for call in range(12):
        moved = rng.integers(0, nk, 700).astype(np.uint32)
        o.localize(moved)
        s.localize(dev_keys(moved))
        ho, hs = o.prepare_sample(do, 1500), s.prepare_sample(ds, 1500)
        for cut in (400, 1100):
            assert np.array_equal(host_keys(s.pull_sample(hs, cut, values=False)), o.pull_sample(ho, cut, values=False))
        got = s.owner_of(dev_keys(allk)).cpu().numpy()
        assert np.array_equal(got, np.array([o.owner_of(k) for k in allk])), call
    assert s.status_check() == 0
    s.close()


@pytest.mark.parametrize("deterministic", [True, False])
def test_merge_mean_matches_the_oracle(deterministic):
    # replicated keys pushed to by a varying number of workers per round; updates are multiples of 2^-4 so that the
    # fast mode's sums are exact whatever their order, and the mean's one division rounds the same on both sides
    nk, L, R = 300, 64, 6
    rng = np.random.default_rng(1)
    init = rng.integers(-8, 9, size=(nk, L)).astype(np.float32) / 4
    o = Oracle(nk, L, workers=R)
    o.table()[:] = init
    o.set_merge_mean(True)
    s = binding.Store(nk, L, workers=R, deterministic=deterministic, merge_mean=True)
    s.write_table(0, init)
    hot = rng.permutation(nk)[:25].astype(np.uint32)
    o.set_management(hot, REPLICATE)
    s.set_management(dev_keys(hot), binding.REPLICATE)
    for n in (6, 40_000, 333, 37_001):
        keys = np.where(rng.random(n) < 0.6, hot[rng.integers(0, 25, n)], rng.integers(0, nk, n)).astype(np.uint32)
        if n == 333:
            keys[: n // 2] = hot[3]                          # the first workers only, all on one key
        delta = rng.integers(-8, 9, size=(n, L)).astype(np.float32) / 16
        o.push(keys, delta)
        s.push(dev_keys(keys), dev_f32(delta))
        o.sync()
        s.sync()
        if deterministic:
            tables_equal(o, s)
        else:
            tables_close(o, s)
    assert np.abs(o.table() - init).max() > 1.0
    assert s.status_check() == 0
    s.close()
