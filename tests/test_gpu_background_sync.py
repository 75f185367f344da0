"""Time-based replica synchronisation: a background thread merges the replicas while pushes and steps run.

There is no deterministic oracle for merges at arbitrary times; what is fixed regardless of timing is
conservation (after the ticks are stopped and a final merge, every row is its start value plus the sum of
everything pushed to it) and, for training, the loss the oracle reaches with a comparable merge interval.
"""
import time

import numpy as np
import pytest
import torch

from oracle import BOUNDED, REPLICATE
from paper_2104_00501_b200 import binding, inputs
from tests.common import dev_f32, dev_keys, make_pair

pytestmark = pytest.mark.gpu


def test_no_update_is_lost_or_doubled_while_merges_overlap_pushes_and_pulls():
    nk, L, R, n = 4000, 64, 4, 8192
    rng = np.random.default_rng(0)
    s = binding.Store(nk, L, workers=R, sync_interval=0, deterministic=False, sync_period_us=100)
    hot = rng.choice(nk, 300, replace=False).astype(np.uint32)
    s.set_management(dev_keys(hot), binding.REPLICATE)
    # multiples of 2^-6 of small size: every partial sum is exact in fp32, whatever the order of the additions
    total = np.zeros((nk, L), np.int64)
    batches = []
    for b in range(24):
        keys = np.where(rng.random(n) < 0.7, rng.choice(hot, n), rng.integers(0, nk, n)).astype(np.uint32)
        units = rng.integers(-8, 9, (n, L)).astype(np.int64)
        np.add.at(total, keys, units)
        batches.append((dev_keys(keys), dev_f32(units.astype(np.float32) / 64.0)))
    out = torch.empty(n, L, device="cuda")
    t_end = time.time() + 0.25
    rounds = 0
    while time.time() < t_end or rounds < 3:
        for k, d in batches:
            s.push(k, d)
            s.pull(k, out)
        torch.cuda.synchronize()
        rounds += 1
    merges = s.stats()["background_merges"]
    s.set_sync_period(0)
    s.sync()
    got = s.read_table().cpu().numpy()
    assert merges > 0
    assert np.array_equal(got, (total * rounds).astype(np.float32) / 64.0)
    assert s.status_check() == 0
    s.close()


def test_period_can_be_changed_and_management_rebuilt_while_the_thread_runs():
    nk, L = 1000, 8
    s = binding.Store(nk, L, workers=3, sync_interval=0, deterministic=False)
    keys = dev_keys(np.arange(100, dtype=np.uint32))
    ones = torch.ones(100, L, device="cuda")
    s.set_management(keys[:50].contiguous(), binding.REPLICATE)
    s.set_sync_period(50)
    for i in range(50):
        s.push(keys, ones)
        if i % 10 == 5:
            s.set_management(keys[i:i + 20].contiguous(), binding.REPLICATE if i % 20 == 5 else binding.SINGLE)
    s.set_sync_period(2000)
    s.push(keys, ones)
    s.set_sync_period(0)
    before = s.stats()["background_merges"]
    time.sleep(0.02)
    assert s.stats()["background_merges"] == before
    s.sync()
    got = s.read_table().cpu().numpy()
    assert np.array_equal(got[:100], np.full((100, L), 51.0, np.float32))
    assert not got[100:].any()
    s.close()


def test_deterministic_stores_refuse_time_based_merging():
    with pytest.raises(binding.NupsError):
        binding.Store(100, 4, deterministic=True, sync_period_us=100)
    s = binding.Store(100, 4, deterministic=True)
    with pytest.raises(binding.NupsError) as e:
        s.set_sync_period(100)
    assert e.value.code == binding.ESTATE
    s.set_sync_period(0)
    s.close()


def test_sgns_with_time_based_merging_reaches_the_oracles_loss_within_one_percent():
    V, L, K, R, batch = 500, 32, 3, 8, 256
    c, ctx, counts = inputs.sgns_batch_stream(V, 4000, 1.0, 2)
    c, ctx = inputs.u32(c), inputs.u32(ctx)
    w = inputs.integer_weights(counts).numpy().astype(np.uint32)
    init = inputs.normal_init(2 * V, L, 0.1, 2)
    o, _ = make_pair(2 * V, L, R=R, init=init, deterministic=False, sync_interval=4)
    s = binding.Store(2 * V, L, workers=R, sync_interval=0, deterministic=False, sync_period_us=200)
    s.write_table(0, init)
    o.count_accesses(np.concatenate([c, ctx]))
    hot = o.select_hot(True, 20)
    o.set_management(hot, REPLICATE)
    s.set_management(dev_keys(hot), binding.REPLICATE)
    do = o.register_distribution(V, w, V, BOUNDED, U=4, G=50, seed=3)
    ds = s.register_distribution(V, dev_keys(w), V, binding.BOUNDED, U=4, G=50, seed=3)
    lb = torch.zeros(1, device="cuda")
    lo_hist, ls_hist = [], []
    nb = len(c) // batch
    for epoch in range(2):
        for b in range(nb):
            sl = slice(b * batch, (b + 1) * batch)
            lo_hist.append(o.step_sgns(c[sl], ctx[sl], do, K, 0.01))
            s.step_sgns(dev_keys(c[sl]), dev_keys(ctx[sl]), ds, K, 0.01, lb)
            ls_hist.append(lb.item())
    lo, ls = np.mean(lo_hist[-nb:]), np.mean(ls_hist[-nb:])
    assert s.stats()["background_merges"] > 0
    assert abs(ls - lo) <= 0.01 * lo
    assert s.status_check() == 0
    s.close()
