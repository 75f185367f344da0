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


def test_push_noalloc_matches_push_on_two_calls_in_a_row():
    nk, L, R = 3000, 64, 4
    rng = np.random.default_rng(0)
    init = rng.normal(size=(nk, L)).astype(np.float32)
    _, a = make_pair(nk, L, R=R, init=init, deterministic=True)        # ordinary entry point
    _, b = make_pair(nk, L, R=R, init=init, deterministic=True)        # allocation-free entry point
    hot = rng.permutation(nk)[:40].astype(np.uint32)
    a.set_management(dev_keys(hot), REPLICATE)
    b.set_management(dev_keys(hot), REPLICATE)
    # two calls in a row, the second smaller than the first: the array still holds the first call's data
    for n in (binding.NOALLOC_MAX_ROWS, 4099):
        keys = dev_keys((rng.zipf(1.2, n) % nk).astype(np.uint32))
        delta = dev_f32(rng.normal(size=(n, L)).astype(np.float32))
        a.push(keys, delta)
        b.push_noalloc(keys, delta)
        pk = dev_keys(rng.integers(0, nk, 1000).astype(np.uint32))
        assert torch.equal(a.pull(pk), b.pull(pk))                     # pending replica updates included
    a.sync()
    b.sync()
    # both paths add the same rows in the same order: the stated tolerance is met with zero error
    np.testing.assert_allclose(b.read_table().cpu().numpy(), a.read_table().cpu().numpy(), rtol=1e-5, atol=1e-6)
    assert torch.equal(a.read_table(), b.read_table())
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
