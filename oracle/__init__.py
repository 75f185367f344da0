"""CPU oracle of the NuPS sparse access path (test infrastructure, never the product path).

`Oracle` is a thin ctypes view of ``nups_oracle.c``: it marshals numpy arrays and
nothing else.  Only tests, the smoke check and the benchmark's CPU-baseline leg
may import this package; it imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "nups_oracle.c")
_LIB = os.path.join(_HERE, "libnups_oracle.so")
_LIB_F64 = os.path.join(_HERE, "libnups_oracle_f64.so")          # the same source with 8-byte values

SINGLE, REPLICATE = 0, 1
CONFORM, BOUNDED, LONGTERM, NONCONFORM = 1, 2, 3, 4
OK, EINVAL, ENOMEM, EKEY, ESTATE = 0, -1, -2, -4, -5


def build(force: bool = False, f64: bool = False) -> str:
    """Compile the oracle with gcc (strict IEEE: no contraction, no fast-math); f64: the build with 8-byte values."""
    out = _LIB_F64 if f64 else _LIB
    if force or not os.path.exists(out) or os.path.getmtime(out) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=gnu11", "-fPIC", "-shared", "-ffp-contract=off", "-fno-fast-math",
               "-Wall", "-Wextra"] + (["-DORC_REAL=double"] if f64 else []) + ["-o", out + ".tmp", _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(out + ".tmp", out)
    return out


_libs = {}

_u32p = C.POINTER(C.c_uint32)
_u64p = C.POINTER(C.c_uint64)


def lib(f64: bool = False):
    """The oracle library with 4-byte (default) or 8-byte values; value buffers cross as untyped pointers."""
    if f64 not in _libs:
        L = C.CDLL(build(f64=f64))
        _f32p = C.c_void_p           # `real*` in the C source: float or double, depending on the build
        sig = {
            "orc_philox4x32_10": (None, [_u32p, _u32p, _u32p]),
            "orc_alias_build": (C.c_uint64, [_u32p, C.c_uint64, _u64p, _u32p]),
            "orc_create": (C.c_void_p, [C.c_uint64, C.c_uint32, C.c_uint32, C.c_int, C.c_int, C.c_int, C.c_uint32]),
            "orc_destroy": (None, [C.c_void_p]),
            "orc_table": (C.c_void_p, [C.c_void_p, C.c_int]),
            "orc_counts": (_u64p, [C.c_void_p]),
            "orc_status": (C.c_int, [C.c_void_p]),
            "orc_num_hot": (C.c_uint64, [C.c_void_p]),
            "orc_hot_keys": (_u32p, [C.c_void_p]),
            "orc_slots": (C.POINTER(C.c_int32), [C.c_void_p]),
            "orc_stats": (None, [C.c_void_p, _u64p]),
            "orc_init_uniform": (None, [C.c_void_p, C.c_int, C.c_uint64, C.c_float]),
            "orc_pull2": (C.c_int, [C.c_void_p, _u32p, C.c_uint64, _f32p, _f32p]),
            "orc_push2": (C.c_int, [C.c_void_p, _u32p, C.c_uint64, _f32p, _f32p]),
            "orc_sync": (C.c_int, [C.c_void_p]),
            "orc_set_clipping": (None, [C.c_void_p, C.c_double]),
            "orc_set_merge_mean": (None, [C.c_void_p, C.c_int]),
            "orc_clip_stats": (None, [C.c_void_p, C.POINTER(C.c_double), _u64p]),
            "orc_count_accesses": (C.c_int, [C.c_void_p, _u32p, C.c_uint64]),
            "orc_select_hot": (C.c_uint64, [C.c_void_p, C.c_int, C.c_uint64, _u32p]),
            "orc_set_management": (C.c_int, [C.c_void_p, _u32p, C.c_uint64, C.c_int]),
            "orc_localize": (C.c_int, [C.c_void_p, _u32p, C.c_uint64]),
            "orc_owner_of": (C.c_int, [C.c_void_p, C.c_uint32]),
            "orc_register_distribution": (C.c_int, [C.c_void_p, C.c_uint32, _u32p, C.c_uint64, C.c_int,
                                                    C.c_uint32, C.c_uint32, C.c_uint64]),
            "orc_dist_thr": (_u64p, [C.c_void_p, C.c_int]),
            "orc_dist_alias": (_u32p, [C.c_void_p, C.c_int]),
            "orc_dist_W": (C.c_uint64, [C.c_void_p, C.c_int]),
            "orc_draw_iid": (C.c_uint32, [C.c_void_p, C.c_int, C.c_uint32, C.c_uint64]),
            "orc_prepare_sample": (C.c_int64, [C.c_void_p, C.c_int, C.c_uint64]),
            "orc_pull_sample": (C.c_int, [C.c_void_p, C.c_int64, C.c_uint64, _u32p, _f32p]),
            "orc_step_sgns": (C.c_int, [C.c_void_p, _u32p, _u32p, C.c_uint64, C.c_int, C.c_uint32, C.c_float,
                                        C.POINTER(C.c_float), _u32p]),
            "orc_step_complex": (C.c_int, [C.c_void_p, _u32p, _u32p, _u32p, C.c_uint64, C.c_int, C.c_uint32,
                                           C.c_float, C.c_float, C.POINTER(C.c_float), _u32p]),
            "orc_step_mf": (C.c_int, [C.c_void_p, _u32p, _u32p, C.POINTER(C.c_float), C.c_uint64, C.c_float, C.c_float,
                                      C.POINTER(C.c_float)]),
        }
        for name, (res, args) in sig.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        L.orc_value_bytes.restype, L.orc_value_bytes.argtypes = C.c_int, []
        assert L.orc_value_bytes() == (8 if f64 else 4)
        _libs[f64] = L
    return _libs[f64]


def _u32(a):
    a = np.ascontiguousarray(a, dtype=np.uint32)
    return a, a.ctypes.data_as(_u32p)


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a, a.ctypes.data_as(C.POINTER(C.c_float))


def philox4x32_10(ctr, key):
    c, cp = _u32(ctr)
    k, kp = _u32(key)
    out = np.zeros(4, np.uint32)
    lib().orc_philox4x32_10(cp, kp, out.ctypes.data_as(_u32p))
    return out


def alias_build(weights):
    w, wp = _u32(weights)
    n = len(w)
    thr = np.zeros(n, np.uint64)
    alias = np.zeros(n, np.uint32)
    W = lib().orc_alias_build(wp, n, thr.ctypes.data_as(_u64p), alias.ctypes.data_as(_u32p))
    return int(W), thr, alias


class OracleError(RuntimeError):
    def __init__(self, code, what):
        super().__init__(f"oracle {what}: status {code}")
        self.code = code


def _chk(code, what):
    if code < 0:
        raise OracleError(code, what)
    return code


class Oracle:
    """One store with R logical workers; mirrors the C-ABI calls one to one."""

    def __init__(self, num_keys, value_len, workers=8, with_adagrad=False, count_accesses=False,
                 track_ownership=False, sync_interval=1, value_bytes=4):
        assert value_bytes in (4, 8)
        self._l = lib(f64=value_bytes == 8)
        self.dtype = np.float64 if value_bytes == 8 else np.float32
        self.num_keys, self.L, self.R = int(num_keys), int(value_len), int(workers)
        self.with_adagrad = bool(with_adagrad)
        self._s = self._l.orc_create(self.num_keys, self.L, self.R, int(with_adagrad), int(count_accesses),
                                     int(track_ownership), int(sync_interval))
        if not self._s:
            raise OracleError(EINVAL, "create")

    def close(self):
        if self._s:
            self._l.orc_destroy(self._s)
            self._s = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- tables -----------------------------------------------------------
    def table(self, which=0):
        """Writable numpy view [num_keys, L] of the value (0) or accumulator (1) table."""
        p = self._l.orc_table(self._s, which)
        ct = C.c_double if self.dtype == np.float64 else C.c_float
        return np.ctypeslib.as_array(C.cast(p, C.POINTER(ct)), shape=(self.num_keys, self.L))

    def init_uniform(self, which, seed, scale):
        self._l.orc_init_uniform(self._s, which, seed, scale)

    def counts(self):
        return np.ctypeslib.as_array(self._l.orc_counts(self._s), shape=(self.num_keys,)).copy()

    def status(self):
        return self._l.orc_status(self._s)

    def stats(self):
        out = np.zeros(4, np.uint64)
        self._l.orc_stats(self._s, out.ctypes.data_as(_u64p))
        return dict(steps=int(out[0]), syncs=int(out[1]), hot=int(out[2]), cold=int(out[3]))

    # -- direct access ----------------------------------------------------
    def pull(self, keys, with_acc=False):
        k, kp = _u32(keys)
        out = np.empty((len(k), self.L), self.dtype)
        out2 = np.empty((len(k), self.L), self.dtype) if with_acc else None
        _chk(self._l.orc_pull2(self._s, kp, len(k), out.ctypes.data, out2.ctypes.data if with_acc else None), "pull")
        return (out, out2) if with_acc else out

    def push(self, keys, delta, delta_acc=None):
        k, kp = _u32(keys)
        d = np.ascontiguousarray(delta, dtype=self.dtype)
        dp = d.ctypes.data
        assert d.shape == (len(k), self.L)
        if delta_acc is not None:
            a = np.ascontiguousarray(delta_acc, dtype=self.dtype)
            ap = a.ctypes.data
        else:
            ap = None
        _chk(self._l.orc_push2(self._s, kp, len(k), dp, ap), "push")

    def sync(self):
        _chk(self._l.orc_sync(self._s), "sync")

    def set_merge_mean(self, on=True):
        """A sync adds the mean of the pending updates over the workers that pushed to a key, not their sum."""
        self._l.orc_set_merge_mean(self._s, int(on))

    # -- management -------------------------------------------------------
    def count_accesses(self, keys):
        k, kp = _u32(keys)
        _chk(self._l.orc_count_accesses(self._s, kp, len(k)), "count")

    def select_hot(self, by_topk, param):
        out = np.zeros(self.num_keys, np.uint32)
        m = self._l.orc_select_hot(self._s, int(by_topk), int(param), out.ctypes.data_as(_u32p))
        return out[:m].copy()

    def set_management(self, keys, technique):
        k, kp = _u32(keys)
        _chk(self._l.orc_set_management(self._s, kp, len(k), technique), "set_management")

    def hot_keys(self):
        h = self._l.orc_num_hot(self._s)
        if h == 0:
            return np.zeros(0, np.uint32)
        return np.ctypeslib.as_array(self._l.orc_hot_keys(self._s), shape=(h,)).copy()

    def localize(self, keys):
        k, kp = _u32(keys)
        _chk(self._l.orc_localize(self._s, kp, len(k)), "localize")

    def owner_of(self, key):
        return self._l.orc_owner_of(self._s, int(key))

    # -- sampling ---------------------------------------------------------
    def register_distribution(self, key_base, weights, n, level, U=16, G=250, seed=0):
        if weights is not None:
            w, wp = _u32(weights)
            assert len(w) == n
        else:
            wp = None
        return _chk(self._l.orc_register_distribution(self._s, key_base, wp, n, level, U, G, seed), "register")

    def alias_table(self, dist):
        n_w = self._l.orc_dist_W(self._s, dist)
        return n_w, self._l.orc_dist_thr(self._s, dist), self._l.orc_dist_alias(self._s, dist)

    def draw_iid(self, dist, worker, pos):
        return self._l.orc_draw_iid(self._s, dist, worker, pos)

    def prepare_sample(self, dist, N):
        return _chk(self._l.orc_prepare_sample(self._s, dist, N), "prepare_sample")

    def pull_sample(self, handle, n, values=True):
        keys = np.zeros(n, np.uint32)
        vals = np.empty((n, self.L), self.dtype) if values else None
        _chk(self._l.orc_pull_sample(self._s, handle, n, keys.ctypes.data_as(_u32p),
                                     vals.ctypes.data if values else None), "pull_sample")
        return (keys, vals) if values else keys

    # -- workload steps ---------------------------------------------------
    def set_clipping(self, factor):
        """Clip updates to replicated keys at `factor` times the mean norm of earlier such updates (0 = off)."""
        self._l.orc_set_clipping(self._s, float(factor))

    def clip_stats(self):
        s, c = C.c_double(0), C.c_uint64(0)
        self._l.orc_clip_stats(self._s, C.byref(s), C.byref(c))
        return s.value, c.value

    def step_sgns(self, center, context, dist, K, lr, return_negatives=False):
        c, cp = _u32(center)
        o, op = _u32(context)
        loss = C.c_float(0)
        neg = np.zeros(len(c) * K, np.uint32)
        _chk(self._l.orc_step_sgns(self._s, cp, op, len(c), dist, K, lr, C.byref(loss),
                                   neg.ctypes.data_as(_u32p)), "step_sgns")
        return (loss.value, neg) if return_negatives else loss.value

    def step_complex(self, h, r, t, dist, K, lr, eps, return_negatives=False):
        hh, hp = _u32(h)
        rr, rp = _u32(r)
        tt, tp = _u32(t)
        loss = C.c_float(0)
        neg = np.zeros(len(hh) * K, np.uint32)
        _chk(self._l.orc_step_complex(self._s, hp, rp, tp, len(hh), dist, K, lr, eps, C.byref(loss),
                                      neg.ctypes.data_as(_u32p)), "step_complex")
        return (loss.value, neg) if return_negatives else loss.value

    def step_mf(self, rows, cols, x, lr, l2):
        r, rp = _u32(rows)
        c, cp = _u32(cols)
        xx, xp = _f32(x)
        loss = C.c_float(0)
        _chk(self._l.orc_step_mf(self._s, rp, cp, xp, len(r), lr, l2, C.byref(loss)), "step_mf")
        return loss.value
