"""The allocation-free ordered push gives what the ordinary ordered push gives.

Some callers cannot allocate device memory while they run (a serving loop that must not hit the
allocator's device-wide synchronisation, a process whose pool was handed out at start-up), so
`nups_push_noalloc` keeps its sort buffers in a fixed array inside the library.  This file is
collected last on purpose: it shares that one array with every other user in the process.
"""
import numpy as np
import pytest
import torch

from oracle import REPLICATE
from paper_2104_00501_b200 import binding
from tests.common import dev_f32, dev_keys, make_pair

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("hot_n", [40, 0])
def test_push_noalloc_matches_push_and_the_oracle_on_two_calls_in_a_row(hot_n):
    # hot_n = 0: a store without replicated keys sorts on fewer bits (an even number of radix passes, so the sorted
    # rows end up in the other pair of buffers of the fixed array)
    nk, L, R = 3000, 64, 4
    rng = np.random.default_rng(0)
    init = rng.normal(size=(nk, L)).astype(np.float32)
    o, a = make_pair(nk, L, R=R, init=init, deterministic=True)        # oracle, ordinary entry point
    _, b = make_pair(nk, L, R=R, init=init, deterministic=True)        # allocation-free entry point
    if hot_n:
        hot = rng.permutation(nk)[:hot_n].astype(np.uint32)
        o.set_management(hot, REPLICATE)
        a.set_management(dev_keys(hot), REPLICATE)
        b.set_management(dev_keys(hot), REPLICATE)
    # the first call on a device looks the array's address up; after it, the calls below must leave the device's free
    # memory as it is (torch's own buffers for keys and updates are made before the reading is taken)
    warm = dev_keys(np.zeros(8, np.uint32))
    b.push_noalloc(warm, dev_f32(np.zeros((8, L), np.float32)))
    # two calls in a row, the second larger than any before it on this store, the third smaller: the array still
    # holds the earlier call's data each time
    batches = []
    for n in (4099, binding.NOALLOC_MAX_ROWS, 1001):
        keys = (rng.zipf(1.2, n) % nk).astype(np.uint32)
        delta = rng.normal(size=(n, L)).astype(np.float32)
        batches.append((keys, delta, dev_keys(keys), dev_f32(delta)))
    pk = rng.integers(0, nk, 1000).astype(np.uint32)
    dpk = dev_keys(pk)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for keys, delta, dkeys, ddelta in batches:
        b.push_noalloc(dkeys, ddelta)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before                 # nothing was allocated on the device
    for keys, delta, dkeys, ddelta in batches:
        o.push(keys, delta)
        a.push(dkeys, ddelta)
    # a second store takes the same calls one by one, with pulls in between (pending replica updates included)
    _, b2 = make_pair(nk, L, R=R, init=init, deterministic=True)
    _, a2 = make_pair(nk, L, R=R, init=init, deterministic=True)
    if hot_n:
        a2.set_management(dev_keys(hot), REPLICATE)
        b2.set_management(dev_keys(hot), REPLICATE)
    for keys, delta, dkeys, ddelta in batches[:2]:
        a2.push(dkeys, ddelta)
        b2.push_noalloc(dkeys, ddelta)
        assert torch.equal(a2.pull(dpk), b2.pull(dpk))
    assert np.array_equal(b.pull(dpk).cpu().numpy(), o.pull(pk))       # what each worker sees before the merge
    o.sync()
    a.sync()
    b.sync()
    # against the existing entry point: both add the same rows in the same order, so the stated tolerance is met
    # with zero error; against the oracle: the ordered push is bit-exact, well inside the stated tolerance
    np.testing.assert_allclose(b.read_table().cpu().numpy(), a.read_table().cpu().numpy(), rtol=1e-5, atol=1e-6)
    assert torch.equal(a.read_table(), b.read_table())
    np.testing.assert_allclose(b.read_table().cpu().numpy(), o.table(), rtol=1e-5, atol=1e-6)
    assert b.status_check() == 0


def test_push_noalloc_rejects_what_it_cannot_serve():
    _, s = make_pair(100, 8, deterministic=True)
    n = binding.NOALLOC_MAX_ROWS + 1
    keys = torch.zeros(n, dtype=torch.int32, device="cuda")
    delta = torch.zeros((n, 8), dtype=torch.float32, device="cuda")
    with pytest.raises(binding.NupsError) as e:
        s.push_noalloc(keys, delta)
    assert e.value.code == binding.EINVAL and "at most" in str(e.value)
    _, fast = make_pair(100, 8, deterministic=False)
    with pytest.raises(binding.NupsError) as e:
        fast.push_noalloc(keys[:10], delta[:10])
    assert e.value.code == binding.ESTATE
    # nothing was enqueued by the refused calls: the table is as it was
    assert not s.read_table().any() and s.status_check() == 0
