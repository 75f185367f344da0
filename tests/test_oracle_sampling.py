"""Pins of the oracle's sampling path against what the paper and the mathematics fix."""
import os
from fractions import Fraction

import numpy as np
import pytest
from scipy import stats

import oracle
from oracle import Oracle, CONFORM, BOUNDED, LONGTERM, NONCONFORM, REPLICATE

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLD, "philox4x32_10_kat.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        out = oracle.philox4x32_10(v[0:4], v[4:6])
        assert [int(x) for x in out] == v[6:10]


def test_philox_counter_bijection_small_range():
    # a keyed bijection of the counter: distinct counters give distinct blocks
    seen = set()
    for i in range(2000):
        seen.add(tuple(int(x) for x in oracle.philox4x32_10([i, 0, 0, 0], [1, 2])))
    assert len(seen) == 2000


@pytest.mark.parametrize("w", [
    [1, 1, 1, 1], [5], [1, 2, 3, 4, 5, 6, 7, 8, 9, 10], [10, 0, 0, 1, 0, 7, 3, 3, 0, 100],
    [4, 4, 4, 1, 7], [1000000, 1, 1, 1, 1, 1, 1, 1, 1, 1], [3, 3, 2, 2, 2]])
def test_alias_table_exact_mass(w):
    n = len(w)
    W, thr, alias = oracle.alias_build(w)
    assert W == sum(w)
    mass = [0] * n
    for j in range(n):
        assert 0 <= int(thr[j]) <= W and 0 <= int(alias[j]) < n
        mass[j] += int(thr[j])
        mass[int(alias[j])] += W - int(thr[j])
    assert mass == [n * x for x in w]                      # exact integer invariant
    # implied pmf, in exact rationals, is w / W
    for k in range(n):
        p = sum(Fraction(int(thr[j]), W) * (j == k) + (1 - Fraction(int(thr[j]), W)) * (int(alias[j]) == k)
                for j in range(n)) / n
        assert p == Fraction(w[k], W)


def test_alias_random_tables_mass():
    rng = np.random.default_rng(0)
    for n in [2, 3, 17, 100, 1000]:
        w = rng.integers(0, 1000, n).astype(np.uint32)
        w[rng.integers(0, n)] += 1
        W, thr, alias = oracle.alias_build(w)
        mass = np.zeros(n, dtype=object)
        for j in range(n):
            mass[j] += int(thr[j])
            mass[int(alias[j])] += W - int(thr[j])
        assert all(int(mass[j]) == n * int(w[j]) for j in range(n))


def test_alias_rejects_overflow_and_zero():
    assert oracle.alias_build([0, 0, 0])[0] == 0
    assert oracle.alias_build(np.full(1 << 16, 2 ** 32 - 1, np.uint32))[0] != 0      # 2^16 * 2^48 fits
    big = np.full(1 << 17, 2 ** 32 - 1, np.uint32)
    assert oracle.alias_build(big)[0] == 0                                          # 2^17 * 2^49 does not


def _store(R=4, nk=64, L=4, owner=True):
    return Oracle(nk, L, workers=R, track_ownership=owner)


def chi2_p(keys, probs, base=0):
    obs = np.bincount(keys - base, minlength=len(probs)).astype(float)
    exp = probs * len(keys)
    return stats.chisquare(obs, exp).pvalue


def test_conform_frequencies_and_independence():
    o = _store(R=3, nk=40)
    w = np.array([50, 1, 2, 3, 4, 5, 6, 7, 8, 9, 30, 1, 1, 1, 1, 10, 10, 10, 10, 10], np.uint32)
    d = o.register_distribution(10, w, len(w), CONFORM, seed=7)
    N = 60000
    keys = o.pull_sample(o.prepare_sample(d, N), N, values=False)
    assert keys.min() >= 10 and keys.max() < 30
    assert chi2_p(keys, w / w.sum(), base=10) > 1e-3
    # lag-1 pairs inside one worker's chunk: independence => joint = product
    chunk = keys[: N // 3]
    a, b = chunk[:-1] - 10, chunk[1:] - 10
    joint = np.zeros((20, 20))
    np.add.at(joint, (a, b), 1)
    p = w / w.sum()
    exp = np.outer(p, p) * len(a)
    big = exp > 5
    stat = ((joint[big] - exp[big]) ** 2 / exp[big]).sum()
    assert stats.chi2.sf(stat, big.sum() - 1) > 1e-3
    # a wrong table (uniform) must fail the same test
    assert chi2_p(keys, np.full(20, 1 / 20), base=10) < 1e-6


def test_uniform_distribution_has_no_table():
    o = _store(R=2, nk=100)
    d = o.register_distribution(20, None, 50, CONFORM, seed=3)
    keys = o.pull_sample(o.prepare_sample(d, 20000), 20000, values=False)
    assert keys.min() >= 20 and keys.max() < 70
    assert chi2_p(keys, np.full(50, 1 / 50), base=20) > 1e-3


@pytest.mark.parametrize("level", [CONFORM, BOUNDED])
def test_partial_pulls_concatenate(level):
    w = np.arange(1, 33, dtype=np.uint32)
    full, part = [], []
    for out, cuts in ((full, [1000]), (part, [1, 99, 400, 250, 250])):
        o = _store(R=4)
        d = o.register_distribution(0, w, 32, level, U=3, G=7, seed=11)
        h = o.prepare_sample(d, 1000)
        for c in cuts:
            out.append(o.pull_sample(h, c, values=False))
    assert np.array_equal(np.concatenate(full), np.concatenate(part))


def test_streams_continue_across_handles_and_differ_by_worker():
    w = np.arange(1, 65, dtype=np.uint32)
    o1, o2 = _store(R=2), _store(R=2)
    d1 = o1.register_distribution(0, w, 64, CONFORM, seed=5)
    d2 = o2.register_distribution(0, w, 64, CONFORM, seed=5)
    a = o1.pull_sample(o1.prepare_sample(d1, 200), 200, values=False)
    b1 = o2.pull_sample(o2.prepare_sample(d2, 100), 100, values=False)
    b2 = o2.pull_sample(o2.prepare_sample(d2, 100), 100, values=False)
    # worker 0's stream: first 100 of `a` == first 50 of b1 + first 50 of b2
    assert np.array_equal(a[:100], np.concatenate([b1[:50], b2[:50]]))
    assert np.array_equal(a[100:], np.concatenate([b1[50:], b2[50:]]))
    assert not np.array_equal(a[:100], a[100:])
    # the draw at (worker, position) is a pure function
    assert all(o1.draw_iid(d1, 1, i) == a[100 + i] for i in range(100))


def test_reuse_paper_example_G1():
    # Section 4.4: U = 2, G = 1 gives k1 k1 k2 k2 k3 k3
    line = [l for l in open(os.path.join(GOLD, "reuse_example.txt")) if l.startswith("U=2 G=1")][0]
    pattern = line.split(":")[1].split()
    o = _store(R=1, nk=1000)
    d = o.register_distribution(0, None, 1000, BOUNDED, U=2, G=1, seed=1)
    keys = o.pull_sample(o.prepare_sample(d, 6), 6, values=False)
    iid = [o.draw_iid(d, 0, i) for i in range(3)]
    names = {"k1": iid[0], "k2": iid[1], "k3": iid[2]}
    assert [names[x] for x in pattern] == list(keys)


@pytest.mark.parametrize("U,G", [(2, 3), (16, 250), (3, 1), (4, 5)])
def test_reuse_structure_and_bound(U, G):
    R = 2
    o = _store(R=R, nk=100000)
    d = o.register_distribution(0, None, 100000, BOUNDED, U=U, G=G, seed=9)
    pools = 3
    N = R * pools * U * G
    keys = o.pull_sample(o.prepare_sample(d, N), N, values=False)
    for q in range(R):
        ks = keys[q * N // R:(q + 1) * N // R]
        for p in range(pools):
            pool = sorted(o.draw_iid(d, q, p * G + m) for m in range(G))
            seen_orders = set()
            for t in range(U):
                blk = ks[(p * U + t) * G:(p * U + t + 1) * G]
                assert sorted(blk) == pool          # every pass is a permutation of the pool
                seen_orders.add(tuple(blk))
            if G >= 5:
                assert len(seen_orders) > 1         # every pass freshly shuffled
    # every iid draw is used exactly U times and all uses lie inside one window of U*G samples
    ks = keys[:N // R]
    for p in range(pools):
        win = ks[p * U * G:(p + 1) * U * G]
        vals, cnts = np.unique(win, return_counts=True)
        pool_vals, pool_cnts = np.unique([o.draw_iid(d, 0, p * G + m) for m in range(G)], return_counts=True)
        assert np.array_equal(vals, pool_vals) and np.array_equal(cnts, pool_cnts * U)


def test_reuse_first_order_frequencies_and_shuffle_uniformity():
    o = _store(R=1, nk=64)
    w = np.array([9, 1, 5, 5, 20, 2, 2, 6], np.uint32)
    d = o.register_distribution(0, w, 8, BOUNDED, U=2, G=3, seed=21)
    N = 6 * 20000
    keys = o.pull_sample(o.prepare_sample(d, N), N, values=False)
    # first-order probabilities: thin to one sample per pool so that the sample is iid
    assert chi2_p(keys[::6], w / w.sum()) > 1e-3
    # Fisher-Yates: all 6 orders of a 3-pool equally likely (use pools with 3 distinct keys)
    counts = {}
    for p in range(N // 6):
        pool = [o.draw_iid(d, 0, p * 3 + m) for m in range(3)]
        if len(set(pool)) < 3:
            continue
        for t in range(2):
            blk = keys[p * 6 + t * 3:p * 6 + t * 3 + 3]
            order = tuple(pool.index(x) for x in blk)
            counts[order] = counts.get(order, 0) + 1
    assert len(counts) == 6
    assert stats.chisquare(list(counts.values())).pvalue > 1e-3


def test_longterm_all_local_equals_reuse():
    w = np.arange(1, 41, dtype=np.uint32)
    a = _store(R=1, nk=40)
    b = _store(R=1, nk=40)      # one worker: every key is local
    da = a.register_distribution(0, w, 40, BOUNDED, U=4, G=5, seed=2)
    db = b.register_distribution(0, w, 40, LONGTERM, U=4, G=5, seed=2)
    ka = a.pull_sample(a.prepare_sample(da, 300), 300, values=False)
    hb = b.prepare_sample(db, 300)
    kb = np.concatenate([b.pull_sample(hb, c, values=False) for c in (7, 93, 200)])
    assert np.array_equal(ka, kb)


def test_longterm_postponing_invariants():
    R, nk = 4, 400
    w = np.ones(nk, np.uint32)
    ref = _store(R=R, nk=nk)
    dref = ref.register_distribution(0, w, nk, BOUNDED, U=2, G=10, seed=4)
    slice_ = ref.pull_sample(ref.prepare_sample(dref, 800), 800, values=False)

    o = _store(R=R, nk=nk)
    d = o.register_distribution(0, w, nk, LONGTERM, U=2, G=10, seed=4)
    h = o.prepare_sample(d, 800)
    # another "worker" takes a third of the keys away between PrepareSample and PullSample
    stolen = np.arange(0, nk, 3, dtype=np.uint32)
    o.localize(np.concatenate([stolen, stolen]))     # 2*len items: first half worker 0-1, second 2-3
    owner_at_start = np.array([o.owner_of(k) for k in range(nk)])
    out = o.pull_sample(h, 800, values=False)
    for q in range(R):
        got = out[q * 200:(q + 1) * 200]
        src = slice_[q * 200:(q + 1) * 200]
        assert sorted(got) == sorted(src)            # each sample used exactly once, inside its handle
        local = owner_at_start[src] == q
        # one full pull: locals in their order, then the postponed ones in their order
        assert np.array_equal(got, np.concatenate([src[local], src[~local]]))
        assert (~local).sum() > 0
    # postponed keys were re-localized to the sub-handle's worker when the call ended
    for q in range(R):
        src = slice_[q * 200:(q + 1) * 200]
        for k in src[owner_at_start[src] != q]:
            owners = [qq for qq in range(R) if k in slice_[qq * 200:(qq + 1) * 200]
                      and owner_at_start[k] != qq]
            assert o.owner_of(k) == max(owners)


def test_longterm_partial_pulls_postpone_at_most_once():
    R, nk = 2, 50
    o = _store(R=R, nk=nk)
    d = o.register_distribution(0, None, nk, LONGTERM, U=1, G=4, seed=8)
    h = o.prepare_sample(d, 40)
    bounded = _store(R=R, nk=nk)
    db = bounded.register_distribution(0, None, nk, BOUNDED, U=1, G=4, seed=8)
    src = bounded.pull_sample(bounded.prepare_sample(db, 40), 40, values=False)
    outs = []
    for c in (5, 5, 10, 15, 5):
        # before every partial pull all keys are taken away from both workers' point of view:
        # worker 0's keys go to worker 1 and vice versa
        own = np.array([o.owner_of(k) for k in range(nk)])
        flip = np.concatenate([np.where(own == 1)[0], np.where(own == 0)[0]]).astype(np.uint32)
        # items are split in two contiguous halves: worker 0 gets the first half
        n1 = (own == 1).sum()
        if n1 == len(flip) - n1:
            o.localize(flip)
        outs.append(o.pull_sample(h, c, values=False))
    got = np.concatenate(outs)
    assert sorted(got[:20]) == sorted(src[:20]) and sorted(got[20:]) == sorted(src[20:])


def test_nonconform_local_or_probe_limit():
    R, nk = 4, 1000
    o = _store(R=R, nk=nk)
    w = np.arange(1, nk + 1, dtype=np.uint32)
    d = o.register_distribution(0, w, nk, NONCONFORM, seed=6)
    c = _store(R=R, nk=nk)
    dc = c.register_distribution(0, w, nk, CONFORM, seed=6)
    cand = c.pull_sample(c.prepare_sample(dc, 4000), 4000, values=False)
    got = o.pull_sample(o.prepare_sample(d, 4000), 4000, values=False)
    for q in range(R):
        g, k0 = got[q * 1000:(q + 1) * 1000], cand[q * 1000:(q + 1) * 1000]
        assert np.all(g % R == q)                       # default ownership: key mod R
        assert np.all((g.astype(np.int64) - k0) % nk < R)                # first local key at or after the candidate
    # replicated keys are local everywhere; with every key replicated the scheme is the iid one
    o2 = _store(R=R, nk=nk)
    o2.set_management(np.arange(nk, dtype=np.uint32), REPLICATE)
    d2 = o2.register_distribution(0, w, nk, NONCONFORM, seed=6)
    assert np.array_equal(o2.pull_sample(o2.prepare_sample(d2, 4000), 4000, values=False), cand)
    # nothing local within 64 probes: the candidate itself
    o3 = _store(R=R, nk=nk)
    d3 = o3.register_distribution(0, w, nk, NONCONFORM, seed=6)
    n_items = 4 * nk
    o3.localize(np.concatenate([np.arange(nk, dtype=np.uint32)] * 4)[:n_items])   # last request wins: worker 3
    got3 = o3.pull_sample(o3.prepare_sample(d3, 4000), 4000, values=False)
    assert np.array_equal(got3[:3000], cand[:3000])
    assert np.array_equal(got3[3000:], cand[3000:])      # worker 3 owns everything: candidate is local


def test_nonconform_brute_force_pmf_tiny():
    # 10-key table, 2 workers, default ownership: worker q only ever sees keys = q mod 2 and the
    # probability of key k is pi_k + pi_{k-1} (the candidate one before is not local)
    w = np.array([1, 2, 3, 4, 5, 6, 7, 8, 9, 10], np.uint32)
    o = _store(R=2, nk=10)
    d = o.register_distribution(0, w, 10, NONCONFORM, seed=13)
    keys = o.pull_sample(o.prepare_sample(d, 40000), 40000, values=False)
    p = w / w.sum()
    for q in range(2):
        ks = keys[q * 20000:(q + 1) * 20000]
        exp = np.array([(p[k] + p[(k - 1) % 10]) if k % 2 == q else 0.0 for k in range(10)])
        assert np.all(ks % 2 == q)
        obs = np.bincount(ks, minlength=10)[q::2]
        assert stats.chisquare(obs, exp[q::2] * 20000).pvalue > 1e-3


def test_pull_sample_values_and_overpull():
    o = _store(R=2, nk=30, L=4)
    o.table()[:] = np.arange(120, dtype=np.float32).reshape(30, 4)
    d = o.register_distribution(0, None, 30, CONFORM, seed=1)
    h = o.prepare_sample(d, 10)
    k, v = o.pull_sample(h, 4)
    assert np.array_equal(v, o.table()[k])
    with pytest.raises(oracle.OracleError):
        o.pull_sample(h, 7)
    o.pull_sample(h, 6)
    with pytest.raises(oracle.OracleError):
        o.pull_sample(h, 1)                             # handle is gone once fully pulled
