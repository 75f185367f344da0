"""CUDA path vs oracle: alias tables and sampled key sequences must match bit for bit."""
import numpy as np
import pytest
import torch

from oracle import BOUNDED, CONFORM, LONGTERM, NONCONFORM, REPLICATE
from paper_2104_00501_b200 import inputs
from tests.common import dev_f32, dev_keys, host_keys, make_pair

pytestmark = pytest.mark.gpu


def weight_cases():
    rng = np.random.default_rng(0)
    yield "ones", np.ones(100, np.uint32)
    yield "single", np.array([7], np.uint32)
    yield "zeros_inside", np.array([10, 0, 0, 1, 0, 7, 3, 3, 0, 100], np.uint32)
    yield "equal_to_mean", np.array([4, 4, 4, 1, 7], np.uint32)
    yield "one_giant", np.concatenate([[10 ** 9], np.ones(4999)]).astype(np.uint32)
    yield "random", rng.integers(0, 1000, 4097).astype(np.uint32)
    yield "zipf_10k", inputs.zipf_integer_weights(10000, 1.0).numpy().astype(np.uint32)
    yield "zipf_300k", inputs.zipf_integer_weights(300000, 1.1).numpy().astype(np.uint32)
    yield "all_equal_big", np.full(3000, 2 ** 20, np.uint32)


@pytest.mark.parametrize("name,w", list(weight_cases()))
def test_alias_table_matches_the_sequential_sweep(name, w):
    import oracle as orc
    n = len(w)
    o, s = make_pair(n + 5, 4)
    d = s.register_distribution(3, dev_keys(w), n, CONFORM, seed=1)
    W, thr, alias = s.alias_table(d, n)
    W0, thr0, alias0 = orc.alias_build(w)
    assert W == W0
    assert np.array_equal(thr.cpu().numpy().astype(np.uint64), thr0)
    assert np.array_equal(host_keys(alias), alias0)


def test_register_rejects_bad_distributions():
    from paper_2104_00501_b200.binding import NupsError
    o, s = make_pair(100, 4)
    with pytest.raises(NupsError):
        s.register_distribution(0, dev_keys(np.zeros(10, np.uint32)), 10, CONFORM)
    with pytest.raises(NupsError):
        s.register_distribution(95, None, 10, CONFORM)
    with pytest.raises(NupsError):
        s.register_distribution(0, None, 10, LONGTERM)          # needs ownership tracking
    with pytest.raises(NupsError):
        s.register_distribution(0, None, 10, BOUNDED, U=2, G=5000)


@pytest.mark.parametrize("level,U,G", [(CONFORM, 1, 1), (BOUNDED, 16, 250), (BOUNDED, 2, 3), (BOUNDED, 3, 1),
                                       (BOUNDED, 2, 700), (NONCONFORM, 1, 1), (LONGTERM, 4, 50)])
@pytest.mark.parametrize("R", [1, 4, 7])
def test_sampled_keys_bit_exact_with_partial_pulls(level, U, G, R):
    nk, L = 3000, 8
    rng = np.random.default_rng(1)
    init = rng.normal(size=(nk, L)).astype(np.float32)
    w = inputs.zipf_integer_weights(2000, 1.0).numpy().astype(np.uint32)
    o, s = make_pair(nk, L, R=R, init=init, track_ownership=True)
    hot = np.array([500, 501, 777], np.uint32)
    o.set_management(hot, REPLICATE)
    s.set_management(dev_keys(hot), REPLICATE)
    do = o.register_distribution(400, w, 2000, level, U=U, G=G, seed=11)
    ds = s.register_distribution(400, dev_keys(w), 2000, level, U=U, G=G, seed=11)
    for N, cuts in ((1, [1]), (5000, [5000]), (4099, [1, 98, 2000, 1500, 500]), (777, [700, 77])):
        ho, hs = o.prepare_sample(do, N), s.prepare_sample(ds, N)
        for c in cuts:
            # other workers relocate keys between partial pulls
            moved = rng.integers(0, nk, 600).astype(np.uint32)
            o.localize(moved)
            s.localize(dev_keys(moved))
            ko, vo = o.pull_sample(ho, c)
            ks, vs = s.pull_sample(hs, c)
            assert np.array_equal(host_keys(ks), ko)
            assert np.array_equal(vs.cpu().numpy(), vo)
    allk = np.arange(nk, dtype=np.uint32)
    assert np.array_equal(s.owner_of(dev_keys(allk)).cpu().numpy(), np.array([o.owner_of(k) for k in allk]))


def test_uniform_distribution_and_overpull():
    from paper_2104_00501_b200.binding import NupsError
    o, s = make_pair(5000, 4, R=3)
    do = o.register_distribution(100, None, 4000, BOUNDED, U=16, G=250, seed=2)
    ds = s.register_distribution(100, None, 4000, BOUNDED, U=16, G=250, seed=2)
    for N in (10000, 12288, 3):
        ko = o.pull_sample(o.prepare_sample(do, N), N, values=False)
        ks = s.pull_sample(s.prepare_sample(ds, N), N, values=False)
        assert np.array_equal(host_keys(ks), ko)
    h = s.prepare_sample(ds, 10)
    s.pull_sample(h, 4, values=False)
    with pytest.raises(NupsError) as e:
        s.pull_sample(h, 7, values=False)
    assert e.value.code == -5
    s.pull_sample(h, 6, values=False)
    with pytest.raises(NupsError):
        s.pull_sample(h, 1, values=False)


def test_large_sample_frequencies_match_target():
    # a property that holds at any size: 2M CONFORM samples follow pi (chi-square), and the
    # oracle agrees on a sampled prefix
    from scipy import stats
    n = 1000
    w = inputs.zipf_integer_weights(n, 1.0).numpy().astype(np.uint32)
    o, s = make_pair(n, 4, R=8)
    do = o.register_distribution(0, w, n, CONFORM, seed=5)
    ds = s.register_distribution(0, dev_keys(w), n, CONFORM, seed=5)
    N = 2_000_000
    ks = host_keys(s.pull_sample(s.prepare_sample(ds, N), N, values=False))
    obs = np.bincount(ks, minlength=n)
    assert stats.chisquare(obs, w / w.sum() * N).pvalue > 1e-4
    for q in (0, 3, 7):
        for i in (0, 1, 12345, N // 8 - 1):
            assert ks[q * (N // 8) + i] == o.draw_iid(do, q, i)


@pytest.mark.parametrize("level", [LONGTERM, NONCONFORM, BOUNDED])
def test_large_handles_with_most_keys_taken_by_other_workers(level):
    # sub-handles longer than one round of the postponing walk; between the partial pulls nearly every key
    # is moved away, so a small pull has to walk far past the stretch whose locality was looked up ahead
    nk, L, R = 150_000, 4, 4
    rng = np.random.default_rng(3)
    w = inputs.zipf_integer_weights(120_000, 0.7).numpy().astype(np.uint32)
    o, s = make_pair(nk, L, R=R, track_ownership=True)
    hot = rng.choice(nk, 50, replace=False).astype(np.uint32)
    o.set_management(hot, REPLICATE)
    s.set_management(dev_keys(hot), REPLICATE)
    do = o.register_distribution(1000, w, 120_000, level, U=4, G=250, seed=21)
    ds = s.register_distribution(1000, dev_keys(w), 120_000, level, U=4, G=250, seed=21)
    N = 400_000
    ho, hs = o.prepare_sample(do, N), s.prepare_sample(ds, N)
    for c in (100, 5_000, 150_000, 1, 244_899):
        moved = rng.permutation(nk).astype(np.uint32)[: nk - 2000]
        o.localize(moved)
        s.localize(dev_keys(moved))
        ko = o.pull_sample(ho, c, values=False)
        ks = s.pull_sample(hs, c, values=False)
        assert np.array_equal(host_keys(ks), ko)
    allk = np.arange(nk, dtype=np.uint32)
    assert np.array_equal(s.owner_of(dev_keys(allk)).cpu().numpy(), np.array([o.owner_of(k) for k in allk]))
    assert s.status_check() == 0


@pytest.mark.parametrize("L", [64, 128, 256])
def test_full_pull_with_values_under_postponing_copies_the_rows_itself(L):
    # rows of 64 / 128 / 256 floats: a full PullSample of a fresh LONG-TERM handle places keys and copies rows in one
    # pass; replicated keys carry unmerged updates, ownership has been stirred, and a second handle is pulled in parts
    # (the separate gather) for comparison with the same oracle
    nk, R, N = 5000, 4, 20_000
    rng = np.random.default_rng(L)
    init = rng.normal(size=(nk, L)).astype(np.float32)
    w = inputs.zipf_integer_weights(4000, 0.9).numpy().astype(np.uint32)
    o, s = make_pair(nk, L, R=R, init=init, track_ownership=True)
    hot = rng.choice(nk, 40, replace=False).astype(np.uint32)
    o.set_management(hot, REPLICATE)
    s.set_management(dev_keys(hot), REPLICATE)
    pk = np.where(rng.random(300) < 0.6, rng.choice(hot, 300), rng.integers(0, nk, 300)).astype(np.uint32)
    d = rng.normal(size=(300, L)).astype(np.float32)
    o.push(pk, d)
    s.push(dev_keys(pk), torch.from_numpy(d).cuda())
    do = o.register_distribution(500, w, 4000, LONGTERM, U=4, G=50, seed=5)
    ds = s.register_distribution(500, dev_keys(w), 4000, LONGTERM, U=4, G=50, seed=5)
    for cuts in ([N], [7000, 13000], [N]):
        moved = rng.integers(0, nk, 3000).astype(np.uint32)
        o.localize(moved)
        s.localize(dev_keys(moved))
        ho, hs = o.prepare_sample(do, N), s.prepare_sample(ds, N)
        for c in cuts:
            ko, vo = o.pull_sample(ho, c)
            ks, vs = s.pull_sample(hs, c)
            assert np.array_equal(host_keys(ks), ko)
            assert np.array_equal(vs.cpu().numpy(), vo)
    allk = np.arange(nk, dtype=np.uint32)
    assert np.array_equal(s.owner_of(dev_keys(allk)).cpu().numpy(), np.array([o.owner_of(k) for k in allk]))


@pytest.mark.parametrize("L,U,G,R", [(128, 16, 250, 8), (64, 4, 100, 3), (256, 16, 250, 8), (512, 3, 250, 2), (1024, 2, 40, 2)])
def test_pooled_reuse_pull_sample_rows_are_what_each_worker_pulls(L, U, G, R):
    # The rows that PullSample returns are exactly what the sub-handle's worker pulls at that moment: the stored row
    # plus that worker's pending replica updates for a replicated key.  Pooled reuse (the same keys come back again and
    # again), rows of 256 bytes to 4 KB, partial pulls cut inside pools and sub-handles, updates pushed (and left
    # pending) between the partial pulls.
    nk = 6000
    rng = np.random.default_rng(L)
    init = rng.standard_normal(size=(nk, L), dtype=np.float32)
    w = inputs.zipf_integer_weights(5000, 1.0).numpy().astype(np.uint32)
    o, s = make_pair(nk, L, R=R, init=init, deterministic=True, sync_interval=0)
    hot = (300 + inputs.u32(inputs.zipf_key_of_rank(5000)[:40])).astype(np.uint32)      # the target's most frequent keys
    o.set_management(hot, REPLICATE)
    s.set_management(dev_keys(hot), REPLICATE)
    do = o.register_distribution(300, w, 5000, BOUNDED, U=U, G=G, seed=21)
    ds = s.register_distribution(300, dev_keys(w), 5000, BOUNDED, U=U, G=G, seed=21)
    for N, cuts in ((20000, [20000]), (9001, [1, 130, 4000, 4870]), (U * G * R + 7, [U * G, U * G * (R - 1) + 7])):
        ho, hs = o.prepare_sample(do, N), s.prepare_sample(ds, N)
        for c in cuts:
            # updates that stay pending in the workers' replicas (no merge): every worker sees its own only
            keys = np.concatenate([hot, rng.integers(0, nk, 200).astype(np.uint32)])
            delta = rng.standard_normal(size=(len(keys), L), dtype=np.float32)
            o.push(keys, delta)
            s.push(dev_keys(keys), dev_f32(delta))
            ko, vo = o.pull_sample(ho, c)
            ks, vs = s.pull_sample(hs, c)
            assert np.array_equal(host_keys(ks), ko)
            assert np.array_equal(vs.cpu().numpy(), vo)
    assert s.status_check() == 0
