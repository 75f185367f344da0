"""Stores with 8-byte values against the oracle's 8-byte build: pull, push, merge and PullSample bit for bit in the
ordered mode, the ComplEx and matrix-factorization steps within 1e-12 relative / 1e-14 absolute (both sides compute
in double; they differ in summation order only), fast-mode pushes conserving every update to 1e-12."""
import numpy as np
import pytest
import torch

from oracle import BOUNDED, CONFORM, Oracle, REPLICATE
from paper_2104_00501_b200 import binding, inputs
from tests.common import dev_keys, host_keys

pytestmark = pytest.mark.gpu

RTOL64, ATOL64 = 1e-12, 1e-14


def pair64(nk, L, R=4, init=None, acc_init=None, **kw):
    o = Oracle(nk, L, workers=R, with_adagrad=kw.get("with_adagrad", False), count_accesses=kw.get("count_accesses", False),
               track_ownership=kw.get("track_ownership", False), sync_interval=kw.get("sync_interval", 1), value_bytes=8)
    s = binding.Store(nk, L, workers=R, sync_interval=kw.get("sync_interval", 1), deterministic=kw.get("deterministic", True),
                      with_adagrad=kw.get("with_adagrad", False), count_accesses=kw.get("count_accesses", False),
                      track_ownership=kw.get("track_ownership", False), merge_mean=kw.get("merge_mean", False), value_bytes=8)
    if kw.get("merge_mean"):
        o.set_merge_mean(True)
    if init is not None:
        o.table(0)[:] = init
        s.write_table(0, init)
    if acc_init is not None:
        o.table(1)[:] = acc_init
        s.write_table(1, acc_init)
    return o, s


def d64(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float64)).cuda()


@pytest.mark.parametrize("L,merge_mean", [(128, False), (6, False), (250, True)])
def test_fp64_pull_push_merge_and_pull_sample_are_bit_exact_in_ordered_mode(L, merge_mean):
    nk, R = 3000, 4
    rng = np.random.default_rng(L)
    init = rng.normal(size=(nk, L))
    o, s = pair64(nk, L, R=R, init=init, deterministic=True, merge_mean=merge_mean)
    assert s.read_table().dtype == torch.float64
    hot = rng.permutation(nk)[:50].astype(np.uint32)
    o.set_management(hot, REPLICATE)
    s.set_management(dev_keys(hot), REPLICATE)
    w = inputs.zipf_integer_weights(2000, 1.0).numpy().astype(np.uint32)
    do = o.register_distribution(500, w, 2000, BOUNDED, U=4, G=50, seed=3)
    ds = s.register_distribution(500, dev_keys(w), 2000, BOUNDED, U=4, G=50, seed=3)
    for n in (1, 4099, 33, 20000):
        keys = (rng.zipf(1.2, n) % nk).astype(np.uint32)
        delta = rng.normal(size=(n, L)) * 1e-9             # far below what single precision keeps of values of size 1
        o.push(keys, delta)
        s.push(dev_keys(keys), d64(delta))
        pk = rng.integers(0, nk, 700).astype(np.uint32)
        assert np.array_equal(s.pull(dev_keys(pk)).cpu().numpy(), o.pull(pk))          # pending replica updates included
        ko, vo = o.pull_sample(o.prepare_sample(do, 900), 900)
        ks, vs = s.pull_sample(s.prepare_sample(ds, 900), 900)
        assert np.array_equal(host_keys(ks), ko) and np.array_equal(vs.cpu().numpy(), vo)
        if n != 33:
            o.sync()
            s.sync()
            assert np.array_equal(s.read_table().cpu().numpy(), o.table())
    assert np.abs(o.table() - init).max() > 1e-9 and np.abs(o.table() - init).max() < 1e-6
    assert s.status_check() == 0


def test_fp64_fast_mode_push_conserves_every_update():
    nk, L, R = 5000, 64, 8
    rng = np.random.default_rng(2)
    init = rng.normal(size=(nk, L))
    o, s = pair64(nk, L, R=R, init=init, deterministic=False)
    hot = rng.permutation(nk)[:30].astype(np.uint32)
    o.set_management(hot, REPLICATE)
    s.set_management(dev_keys(hot), REPLICATE)
    for n in (50_000, 7, 33_333):
        keys = (rng.zipf(1.3, n) % nk).astype(np.uint32)
        delta = rng.normal(size=(n, L)) * 1e-8
        o.push(keys, delta)
        s.push(dev_keys(keys), d64(delta))
    o.sync()
    s.sync()
    got, want = s.read_table().cpu().numpy(), o.table()
    # up to tens of thousands of updates of size 1e-8 per row, added in another order than the oracle's: every addition
    # rounds at 2^-53 of the value (~1), so the two sides agree to 1e-12 of the values, seven orders below the updates
    np.testing.assert_allclose(got, want, rtol=RTOL64, atol=ATOL64)
    assert np.abs(want - init).max() > 1e-6 and np.abs(got - want).max() < 1e-12
    assert s.status_check() == 0


@pytest.mark.parametrize("deterministic", [True, False])
@pytest.mark.parametrize("L,hot_n,K", [(500, 30, 10), (8, 4, 3)])
def test_fp64_complex_step_matches_the_oracle(L, hot_n, K, deterministic):
    # ordered mode: three batches, every element of both tables within the 8-byte tolerance.  Fast mode: one batch in
    # which no two triples share a key (own head, relation and tail; triples whose sampled negatives collide with
    # anybody's keys are left out of the comparison), so nothing can race.
    rng = np.random.default_rng(L + K)
    if deterministic:
        E, Rl, R, batch, nb = 400, 12, 4, 100, 3
        h, r, t = [inputs.u32(x) for x in inputs.kge_triples(nb * batch, E, Rl, 0.9, 1.2, 0)]
        nk = E + Rl
        hot = np.concatenate([np.arange(E, E + Rl), np.unique(h)[:hot_n]]).astype(np.uint32)
    else:
        E, R, batch, nb = 50_000, 4, 128, 1
        perm = rng.permutation(E)[:2 * batch].astype(np.uint32)
        h, t = perm[:batch], perm[batch:]
        r = (E + np.arange(batch)).astype(np.uint32)
        nk = E + batch
        hot = np.concatenate([r[:hot_n], h[:hot_n]]).astype(np.uint32)
    init = rng.normal(0, 0.1, size=(nk, L))
    o, s = pair64(nk, L, R=R, init=init, deterministic=deterministic, with_adagrad=True, sync_interval=1)
    o.set_management(hot, REPLICATE)
    s.set_management(dev_keys(hot), REPLICATE)
    do = o.register_distribution(0, None, E, CONFORM, seed=9)
    ds = s.register_distribution(0, None, E, CONFORM, seed=9)
    lb = torch.zeros(1, dtype=torch.float32, device="cuda")
    for b in range(nb):
        sl = slice(b * batch, (b + 1) * batch)
        lo, negs = o.step_complex(h[sl], r[sl], t[sl], do, K, 0.1, 1e-10, return_negatives=True)
        s.step_complex(dev_keys(h[sl]), dev_keys(r[sl]), dev_keys(t[sl]), ds, K, 0.1, 1e-10, lb)
        assert np.array_equal(host_keys(s.last_negatives()), negs)
        assert abs(lb.item() - lo) <= 2e-5 * abs(lo)
    o.sync()
    s.sync()
    if deterministic:
        rows = np.arange(nk)
    else:
        negs = negs.reshape(batch, K)
        uses = np.bincount(np.concatenate([h, t, negs.ravel()]), minlength=E)
        alone = (uses[negs] == 1).all(axis=1) & (uses[h] == 1) & (uses[t] == 1)
        assert alone.mean() > 0.5
        rows = np.concatenate([h[alone], r[alone], t[alone], negs[alone].ravel()])
    idx = torch.from_numpy(rows.astype(np.int64)).cuda()
    np.testing.assert_allclose(s.read_table(1)[idx].cpu().numpy(), o.table(1)[rows], rtol=RTOL64, atol=ATOL64)
    np.testing.assert_allclose(s.read_table(0)[idx].cpu().numpy(), o.table(0)[rows], rtol=RTOL64, atol=ATOL64)
    assert np.abs(o.table(0)[rows] - init[rows]).max() > 0.05
    assert s.status_check() == 0


@pytest.mark.parametrize("deterministic", [True, False])
@pytest.mark.parametrize("L,hot_n", [(100, 25), (2, 3)])
def test_fp64_mf_step_matches_the_oracle(L, hot_n, deterministic):
    rng = np.random.default_rng(L)
    if deterministic:
        M, N, R, batch, n = 500, 200, 4, 512, 2048
        i, j, x = inputs.mf_cells(n, M, N, 0.8, max(L // 4, 2), 0.1, 0)
        i, j, x = inputs.u32(i), inputs.u32(j), x.numpy()
    else:                                                     # cells that share no row and no column: nothing races
        M, N, R, batch, n = 5000, 5000, 4, 4000, 4000
        i = rng.permutation(M)[:n].astype(np.uint32)
        j = (M + rng.permutation(N)[:n]).astype(np.uint32)
        x = rng.normal(0, 1, n).astype(np.float32)
    init = rng.normal(0, 0.3, size=(M + N, L))
    o, s = pair64(M + N, L, R=R, init=init, deterministic=deterministic, count_accesses=True)
    hot = np.concatenate([i[:hot_n], j[hot_n:2 * hot_n]]).astype(np.uint32)
    o.set_management(hot, REPLICATE)
    s.set_management(dev_keys(hot), REPLICATE)
    lb = torch.zeros(1, dtype=torch.float32, device="cuda")
    for b in range(0, n, batch):
        sl = slice(b, b + batch)
        lo = o.step_mf(i[sl], j[sl], x[sl], 0.01, 0.01)
        s.step_mf(dev_keys(i[sl]), dev_keys(j[sl]), torch.from_numpy(x[sl].copy()).cuda(), 0.01, 0.01, lb)
        assert abs(lb.item() - lo) <= 1e-5 * abs(lo)
    o.sync()
    s.sync()
    np.testing.assert_allclose(s.read_table().cpu().numpy(), o.table(), rtol=RTOL64, atol=ATOL64)
    assert np.array_equal(s.counts().cpu().numpy().astype(np.uint64), o.counts())
    assert np.abs(o.table() - init).max() > 1e-3
    assert s.status_check() == 0


def test_fp64_store_refuses_what_is_single_precision_only():
    s = binding.Store(100, 8, value_bytes=8, deterministic=False)
    k = torch.zeros(4, dtype=torch.int32, device="cuda")
    d = s.register_distribution(0, None, 100, binding.CONFORM)
    with pytest.raises(binding.NupsError) as e:
        s.step_sgns(k, k, d, 3, 0.1)
    assert e.value.code == binding.ESTATE
    with pytest.raises(binding.NupsError) as e:
        s.set_sync_period(1000)
    assert e.value.code == binding.ESTATE
    with pytest.raises(binding.NupsError) as e:
        s.probe_reduction_rate(1 << 10, 1)
    assert e.value.code == binding.ESTATE
    for bad in (dict(value_bytes=2), dict(value_bytes=8, clip_factor=1.0), dict(value_bytes=8, sync_period_us=10)):
        with pytest.raises(binding.NupsError) as e:
            binding.Store(100, 8, **bad)
        assert e.value.code == binding.EINVAL
    with pytest.raises(binding.NupsError):
        binding.Store(100, 3, value_bytes=8)                  # rows must be multiples of 16 bytes
    s.close()
