"""Helpers shared by the GPU parity tests: build an oracle and a CUDA store with the same settings."""
import numpy as np
import torch

from oracle import Oracle
from paper_2104_00501_b200 import binding

RTOL, ATOL = 1e-5, 1e-6          # value tolerance in deterministic mode (the stated bar)


def dev_keys(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.uint32).view(np.int32)).cuda()


def host_keys(t):
    return t.detach().cpu().numpy().view(np.uint32)


def dev_f32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


def make_pair(num_keys, L, R=4, init=None, acc_init=None, **kw):
    """(oracle, store) with identical configuration and start values."""
    o = Oracle(num_keys, L, workers=R, with_adagrad=kw.get("with_adagrad", False),
               count_accesses=kw.get("count_accesses", False), track_ownership=kw.get("track_ownership", False),
               sync_interval=kw.get("sync_interval", 1))
    s = binding.Store(num_keys, L, workers=R, sync_interval=kw.get("sync_interval", 1),
                      deterministic=kw.get("deterministic", True), with_adagrad=kw.get("with_adagrad", False),
                      count_accesses=kw.get("count_accesses", False), track_ownership=kw.get("track_ownership", False))
    if init is not None:
        o.table(0)[:] = init
        s.write_table(0, init)
    if acc_init is not None:
        o.table(1)[:] = acc_init
        s.write_table(1, acc_init)
    return o, s


def tables_close(o, s, which=0, rtol=RTOL, atol=ATOL):
    got = s.read_table(which).cpu().numpy()
    np.testing.assert_allclose(got, o.table(which), rtol=rtol, atol=atol)


def tables_equal(o, s, which=0):
    got = s.read_table(which).cpu().numpy()
    assert np.array_equal(got, o.table(which))
