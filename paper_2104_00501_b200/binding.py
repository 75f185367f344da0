"""Thin ctypes binding of ``libnups.so``: argument marshalling only.

Every method maps to the C-ABI call of the same name in ``include/nups.h``; tensors are
torch CUDA tensors used purely as device memory, and the current torch stream is passed
as the call's stream.  There is no CPU fallback: loading fails loudly when the library
is missing or cannot be built.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libnups.so")

OK, EINVAL, ENOMEM, ECUDA, EKEY, ESTATE, ETIMEOUT = 0, -1, -2, -3, -4, -5, -6
SINGLE, REPLICATE = 0, 1
CONFORM, BOUNDED, LONGTERM, NONCONFORM = 1, 2, 3, 4
NOALLOC_MAX_ROWS = 65536

EXPORTS = [
    "nups_create", "nups_destroy", "nups_table_ptr", "nups_table_copy", "nups_init_uniform", "nups_pull", "nups_pull2", "nups_push",
    "nups_push2", "nups_push_noalloc", "nups_set_management", "nups_sync", "nups_count_accesses", "nups_get_counts", "nups_select_hot",
    "nups_get_hot", "nups_localize", "nups_get_owner", "nups_register_distribution", "nups_get_alias_table",
    "nups_prepare_sample", "nups_pull_sample", "nups_step_sgns", "nups_run_sgns", "nups_step_complex", "nups_step_mf", "nups_step_mf_by_column",
    "nups_last_negatives", "nups_status_check", "nups_get_stats", "nups_kernel_timing", "nups_kernel_time", "nups_kernel_times", "nups_probe_reduction_rate", "nups_set_sync_period", "nups_get_clip_stats", "nups_strerror", "nups_last_cuda_error",
    "nups_shard_table_create", "nups_shard_table_destroy", "nups_shard_table_local", "nups_shard_table_copy", "nups_shard_table_export",
    "nups_shard_table_attach", "nups_shard_table_attach_ipc", "nups_shard_pull", "nups_shard_push", "nups_shard_status_check",
    "nups_shard_last_error", "nups_merge_mark", "nups_merge_export", "nups_merge_apply",
]


class Config(C.Structure):
    _fields_ = [("workers", C.c_uint32), ("sync_interval", C.c_uint32), ("deterministic", C.c_uint32),
                ("with_adagrad", C.c_uint32), ("count_accesses", C.c_uint32), ("track_ownership", C.c_uint32),
                ("smem_hot_rows", C.c_uint32), ("sync_period_us", C.c_uint32), ("clip_factor", C.c_float),
                ("max_device_mib", C.c_uint32), ("first_epoch", C.c_uint32), ("merge_mean", C.c_uint32), ("value_bytes", C.c_uint32),
                ("reserved", C.c_uint32 * 3)]


class NupsError(RuntimeError):
    def __init__(self, code, what, detail=""):
        super().__init__(f"{what}: status {code} ({detail})")
        self.code = code


_lib = None


def load(build_if_missing: bool = True):
    """Load libnups.so (building it with nvcc first when it is absent or stale)."""
    global _lib
    if _lib is not None:
        return _lib
    if build_if_missing:
        from . import build as _build
        try:
            _build.build_library()
        except Exception:
            if not os.path.exists(LIB_PATH):
                raise
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2104_00501_b200.build`")
    L = C.CDLL(LIB_PATH)
    vp, u64, u32, i32, f32 = C.c_void_p, C.c_uint64, C.c_uint32, C.c_int32, C.c_float
    sig = {
        "nups_create": [u64, u32, C.POINTER(Config), C.POINTER(vp)],
        "nups_destroy": [vp],
        "nups_table_ptr": [vp, C.c_int, C.POINTER(vp), C.POINTER(u64)],
        "nups_table_copy": [vp, C.c_int, vp, C.c_int, vp],
        "nups_init_uniform": [vp, C.c_int, u64, f32, vp],
        "nups_pull": [vp, vp, u64, vp, vp],
        "nups_pull2": [vp, vp, u64, vp, vp, vp],
        "nups_push": [vp, vp, u64, vp, vp],
        "nups_push2": [vp, vp, u64, vp, vp, vp],
        "nups_push_noalloc": [vp, vp, u64, vp, vp],
        "nups_set_management": [vp, vp, u64, C.c_int, vp],
        "nups_sync": [vp, vp],
        "nups_count_accesses": [vp, vp, u64, vp],
        "nups_get_counts": [vp, vp, vp],
        "nups_select_hot": [vp, C.c_int, u64, vp, C.POINTER(u64), vp],
        "nups_get_hot": [vp, C.POINTER(u64), vp, vp],
        "nups_localize": [vp, vp, u64, vp],
        "nups_get_owner": [vp, vp, u64, vp, vp],
        "nups_register_distribution": [vp, u32, vp, u64, C.c_int, u32, u32, u64, C.POINTER(i32), vp],
        "nups_get_alias_table": [vp, i32, vp, vp, C.POINTER(u64), vp],
        "nups_prepare_sample": [vp, i32, u64, C.POINTER(C.c_int64), vp],
        "nups_pull_sample": [vp, C.c_int64, u64, vp, vp, vp],
        "nups_step_sgns": [vp, vp, vp, u64, i32, u32, f32, vp, vp],
        "nups_run_sgns": [vp, vp, vp, u64, u64, i32, u32, f32, vp, vp],
        "nups_step_complex": [vp, vp, vp, vp, u64, i32, u32, f32, f32, vp, vp],
        "nups_step_mf": [vp, vp, vp, vp, u64, f32, f32, vp, vp],
        "nups_step_mf_by_column": [vp, vp, vp, vp, u64, f32, f32, vp, vp],
        "nups_last_negatives": [vp, C.POINTER(vp), C.POINTER(u64)],
        "nups_status_check": [vp, vp],
        "nups_get_stats": [vp, C.POINTER(u64), vp],
        "nups_kernel_timing": [vp, C.c_int],
        "nups_kernel_time": [vp, C.POINTER(C.c_double), C.POINTER(u64), vp],
        "nups_kernel_times": [vp, C.POINTER(C.c_double), C.POINTER(u64), vp],
        "nups_probe_reduction_rate": [vp, u64, u32, C.POINTER(C.c_double), vp],
        "nups_set_sync_period": [vp, u32],
        "nups_get_clip_stats": [vp, C.POINTER(C.c_double), C.POINTER(u64), vp],
        "nups_shard_table_create": [u64, u32, u32, u32, C.POINTER(vp)],
        "nups_shard_table_local": [vp, C.POINTER(vp), C.POINTER(u64)],
        "nups_shard_table_copy": [vp, vp, C.c_int, vp],
        "nups_shard_table_export": [vp, C.c_char_p],
        "nups_shard_table_attach": [vp, u32, vp],
        "nups_shard_table_attach_ipc": [vp, u32, C.c_char_p],
        "nups_shard_pull": [vp, vp, u64, vp, vp],
        "nups_shard_push": [vp, vp, u64, vp, vp],
        "nups_shard_status_check": [vp, vp],
        "nups_merge_mark": [vp, C.c_int, vp],
        "nups_merge_export": [vp, C.c_int, vp, vp],
        "nups_merge_apply": [vp, C.c_int, vp, vp, vp],
    }
    for name, args in sig.items():
        fn = getattr(L, name)
        fn.restype, fn.argtypes = C.c_int32, args
    L.nups_strerror.restype, L.nups_strerror.argtypes = C.c_char_p, [C.c_int32]
    L.nups_last_cuda_error.restype, L.nups_last_cuda_error.argtypes = C.c_char_p, []
    L.nups_shard_last_error.restype, L.nups_shard_last_error.argtypes = C.c_char_p, [vp]
    L.nups_shard_table_destroy.restype, L.nups_shard_table_destroy.argtypes = None, [vp]
    _lib = L
    return L


def _ptr(t, dtype=None):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device tensors must be contiguous CUDA tensors"
    if dtype is not None:
        assert t.dtype == dtype, f"expected {dtype}, got {t.dtype}"
    return t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


def as_keys(t) -> torch.Tensor:
    """Keys as the library wants them: contiguous CUDA int32 tensor holding uint32 bit patterns."""
    if not torch.is_tensor(t):
        t = torch.as_tensor(t)
    if t.dtype != torch.int32:
        t = t.to(torch.int64).cuda()
        t = torch.where(t >= 2 ** 31, t - 2 ** 32, t).to(torch.int32)
    return t.cuda().contiguous()


class Store:
    """One parameter store on the current CUDA device."""

    def __init__(self, num_keys, value_len, workers=8, sync_interval=1, deterministic=False, with_adagrad=False,
                 count_accesses=False, track_ownership=False, smem_hot_rows=0, sync_period_us=0, clip_factor=0.0,
                 max_device_mib=0, first_epoch=0, merge_mean=False, value_bytes=4):
        self._l = load()
        cfg = Config(workers=workers, sync_interval=sync_interval, deterministic=int(deterministic),
                     with_adagrad=int(with_adagrad), count_accesses=int(count_accesses),
                     track_ownership=int(track_ownership), smem_hot_rows=smem_hot_rows, sync_period_us=sync_period_us,
                     clip_factor=clip_factor, max_device_mib=max_device_mib, first_epoch=first_epoch, merge_mean=int(merge_mean),
                     value_bytes=value_bytes)
        h = C.c_void_p()
        self._s = None
        self._chk(self._l.nups_create(num_keys, value_len, C.byref(cfg), C.byref(h)), "nups_create")
        self._s = h
        self.num_keys, self.L, self.R = int(num_keys), int(value_len), int(workers)
        self.with_adagrad = bool(with_adagrad)
        self.dtype = torch.float64 if value_bytes == 8 else torch.float32       # what every value buffer holds
        self.device = torch.device("cuda", torch.cuda.current_device())

    def _chk(self, code, what):
        if code != OK:
            detail = self._l.nups_strerror(code).decode()
            if code == ECUDA:
                detail += ": " + self._l.nups_last_cuda_error().decode()
            elif code == EINVAL and what == "nups_push_noalloc":
                detail += ": " + self._l.nups_last_cuda_error().decode()
            raise NupsError(code, what, detail)

    def close(self):
        if self._s:
            self._l.nups_destroy(self._s)
            self._s = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- tables -------------------------------------------------------------------------
    def table_ptr(self, which=0):
        p, stride = C.c_void_p(), C.c_uint64()
        self._chk(self._l.nups_table_ptr(self._s, which, C.byref(p), C.byref(stride)), "nups_table_ptr")
        return p.value, stride.value

    def write_table(self, which, values):
        """Copy host (or device) values [num_keys, L] into a table."""
        src = torch.as_tensor(values, dtype=self.dtype).contiguous().cuda()
        assert src.shape == (self.num_keys, self.L)
        self._chk(self._l.nups_table_copy(self._s, which, _ptr(src), 1, _stream()), "nups_table_copy")
        torch.cuda.current_stream().synchronize()

    def read_table(self, which=0, rows=None):
        """Snapshot of a table (or of the given rows of it) as a new CUDA tensor."""
        out = torch.empty((self.num_keys, self.L), dtype=self.dtype, device=self.device)
        self._chk(self._l.nups_table_copy(self._s, which, _ptr(out), 0, _stream()), "nups_table_copy")
        return out if rows is None else out[rows]

    def init_uniform(self, which, seed, scale):
        self._chk(self._l.nups_init_uniform(self._s, which, seed, scale, _stream()), "nups_init_uniform")

    # -- direct access ------------------------------------------------------------------
    def pull(self, keys, out=None, with_acc=False, out_acc=None):
        n = keys.numel()
        if out is None:
            out = torch.empty((n, self.L), dtype=self.dtype, device=self.device)
        assert out.dtype == self.dtype
        if with_acc:
            if out_acc is None:
                out_acc = torch.empty((n, self.L), dtype=self.dtype, device=self.device)
            assert out_acc.dtype == self.dtype
            self._chk(self._l.nups_pull2(self._s, _ptr(keys, torch.int32), n, _ptr(out), _ptr(out_acc), _stream()),
                      "nups_pull2")
            return out, out_acc
        self._chk(self._l.nups_pull(self._s, _ptr(keys, torch.int32), n, _ptr(out), _stream()), "nups_pull")
        return out

    def push(self, keys, delta, delta_acc=None):
        n = keys.numel()
        assert delta is None or (delta.dtype == self.dtype and delta.numel() == n * self.L)
        if delta_acc is None:
            self._chk(self._l.nups_push(self._s, _ptr(keys, torch.int32), n, _ptr(delta), _stream()), "nups_push")
        else:
            assert delta_acc.dtype == self.dtype and delta_acc.numel() == n * self.L
            self._chk(self._l.nups_push2(self._s, _ptr(keys, torch.int32), n, _ptr(delta), _ptr(delta_acc), _stream()),
                      "nups_push2")

    def push_noalloc(self, keys, delta):
        """Ordered push with its sort buffers in the library's fixed device array: for callers that
        may not allocate device memory while they run.  At most NOALLOC_MAX_ROWS rows per call."""
        n = keys.numel()
        assert delta.dtype == self.dtype and delta.numel() == n * self.L
        self._chk(self._l.nups_push_noalloc(self._s, _ptr(keys, torch.int32), n, _ptr(delta), _stream()),
                  "nups_push_noalloc")

    def sync(self):
        self._chk(self._l.nups_sync(self._s, _stream()), "nups_sync")

    # -- management ---------------------------------------------------------------------
    def set_management(self, keys, technique):
        self._chk(self._l.nups_set_management(self._s, _ptr(keys, torch.int32), keys.numel(), technique, _stream()),
                  "nups_set_management")

    def count_accesses(self, keys):
        self._chk(self._l.nups_count_accesses(self._s, _ptr(keys, torch.int32), keys.numel(), _stream()),
                  "nups_count_accesses")

    def counts(self):
        out = torch.empty(self.num_keys, dtype=torch.int64, device=self.device)
        self._chk(self._l.nups_get_counts(self._s, _ptr(out), _stream()), "nups_get_counts")
        return out

    def select_hot(self, by_topk, param):
        cap = min(int(param), self.num_keys) if by_topk else self.num_keys
        out = torch.empty(max(cap, 1), dtype=torch.int32, device=self.device)
        m = C.c_uint64()
        self._chk(self._l.nups_select_hot(self._s, int(by_topk), int(param), _ptr(out), C.byref(m), _stream()),
                  "nups_select_hot")
        return out[:m.value]

    def hot_keys(self):
        m = C.c_uint64()
        self._chk(self._l.nups_get_hot(self._s, C.byref(m), None, _stream()), "nups_get_hot")
        out = torch.empty(max(m.value, 1), dtype=torch.int32, device=self.device)
        if m.value:
            self._chk(self._l.nups_get_hot(self._s, C.byref(m), _ptr(out), _stream()), "nups_get_hot")
        return out[:m.value]

    def localize(self, keys):
        self._chk(self._l.nups_localize(self._s, _ptr(keys, torch.int32), keys.numel(), _stream()), "nups_localize")

    def owner_of(self, keys):
        out = torch.empty(keys.numel(), dtype=torch.int32, device=self.device)
        self._chk(self._l.nups_get_owner(self._s, _ptr(keys, torch.int32), keys.numel(), _ptr(out), _stream()),
                  "nups_get_owner")
        return out

    # -- sampling -----------------------------------------------------------------------
    def register_distribution(self, key_base, weights, n, level, U=16, G=250, seed=0):
        d = C.c_int32()
        if weights is not None:
            assert weights.numel() == n
        self._chk(self._l.nups_register_distribution(self._s, key_base, _ptr(weights, torch.int32), n, level, U, G,
                                                     seed, C.byref(d), _stream()), "nups_register_distribution")
        return d.value

    def alias_table(self, dist, n):
        thr = torch.empty(n, dtype=torch.int64, device=self.device)
        alias = torch.empty(n, dtype=torch.int32, device=self.device)
        W = C.c_uint64()
        self._chk(self._l.nups_get_alias_table(self._s, dist, _ptr(thr), _ptr(alias), C.byref(W), _stream()),
                  "nups_get_alias_table")
        return W.value, thr, alias

    def prepare_sample(self, dist, N):
        h = C.c_int64()
        self._chk(self._l.nups_prepare_sample(self._s, dist, N, C.byref(h), _stream()), "nups_prepare_sample")
        return h.value

    def pull_sample(self, handle, n, values=True, keys_out=None, vals_out=None):
        if keys_out is None:
            keys_out = torch.empty(n, dtype=torch.int32, device=self.device)
        if values and vals_out is None:
            vals_out = torch.empty((n, self.L), dtype=self.dtype, device=self.device)
        assert not values or vals_out.dtype == self.dtype
        self._chk(self._l.nups_pull_sample(self._s, handle, n, _ptr(keys_out), _ptr(vals_out) if values else None,
                                           _stream()), "nups_pull_sample")
        return (keys_out, vals_out) if values else keys_out

    # -- workload steps -----------------------------------------------------------------
    def step_sgns(self, center, context, dist, K, lr, loss_out=None):
        self._chk(self._l.nups_step_sgns(self._s, _ptr(center, torch.int32), _ptr(context, torch.int32),
                                         center.numel(), dist, K, lr, _ptr(loss_out), _stream()), "nups_step_sgns")

    def run_sgns(self, center, context, batch, dist, K, lr, loss_out=None):
        """center.numel() / batch consecutive steps of `batch` pairs; loss_out: one float per step."""
        self._chk(self._l.nups_run_sgns(self._s, _ptr(center, torch.int32), _ptr(context, torch.int32), center.numel(),
                                        batch, dist, K, lr, _ptr(loss_out), _stream()), "nups_run_sgns")

    def step_complex(self, h, r, t, dist, K, lr, eps, loss_out=None):
        self._chk(self._l.nups_step_complex(self._s, _ptr(h, torch.int32), _ptr(r, torch.int32), _ptr(t, torch.int32),
                                            h.numel(), dist, K, lr, eps, _ptr(loss_out), _stream()),
                  "nups_step_complex")

    def step_mf(self, rows, cols, x, lr, l2, loss_out=None, by_column=False):
        """One matrix-factorization step; by_column: the cells arrive column by column (nups_step_mf_by_column)."""
        fn = self._l.nups_step_mf_by_column if by_column else self._l.nups_step_mf
        self._chk(fn(self._s, _ptr(rows, torch.int32), _ptr(cols, torch.int32),
                     _ptr(x, torch.float32), rows.numel(), lr, l2, _ptr(loss_out), _stream()),
                  "nups_step_mf_by_column" if by_column else "nups_step_mf")

    def last_negatives(self):
        p, n = C.c_void_p(), C.c_uint64()
        self._chk(self._l.nups_last_negatives(self._s, C.byref(p), C.byref(n)), "nups_last_negatives")
        if not n.value:
            return torch.empty(0, dtype=torch.int32, device=self.device)

        class _Raw:        # the library's buffer seen through the CUDA array interface, then copied out
            __cuda_array_interface__ = {"shape": (n.value,), "typestr": "<i4", "data": (p.value, False), "version": 2}
        return torch.as_tensor(_Raw(), device=self.device).clone()

    # -- status -------------------------------------------------------------------------
    def status_check(self):
        return self._l.nups_status_check(self._s, _stream())

    def kernel_timing(self, enable):
        self._chk(self._l.nups_kernel_timing(self._s, int(enable)), "nups_kernel_timing")

    def kernel_time(self):
        """(milliseconds, launches) of the main kernels since the last query."""
        ms, n = C.c_double(), C.c_uint64()
        self._chk(self._l.nups_kernel_time(self._s, C.byref(ms), C.byref(n), _stream()), "nups_kernel_time")
        return ms.value, n.value

    KERNEL_KINDS = ("pull", "push", "step", "sample_rows", "draw")

    def kernel_times(self):
        """{kind: (milliseconds, launches)} of the main kernels since the last query, by kind of kernel."""
        ms, n = (C.c_double * 8)(), (C.c_uint64 * 8)()
        self._chk(self._l.nups_kernel_times(self._s, ms, n, _stream()), "nups_kernel_times")
        return {name: (ms[i], n[i]) for i, name in enumerate(self.KERNEL_KINDS)}

    def probe_reduction_rate(self, nbytes, reps=10):
        """GB/s of 128-bit floating-point reductions to streaming addresses (the ceiling of fast-mode updates)."""
        g = C.c_double()
        self._chk(self._l.nups_probe_reduction_rate(self._s, nbytes, reps, C.byref(g), _stream()),
                  "nups_probe_reduction_rate")
        return g.value

    def stats(self):
        out = (C.c_uint64 * 8)()
        self._chk(self._l.nups_get_stats(self._s, out, _stream()), "nups_get_stats")
        return dict(steps=out[0], syncs=out[1], launches=out[2], hot=out[3], cold=out[4], hot_slots=out[5],
                    background_merges=out[6])

    def clip_stats(self):
        """(sum of the norms of the replicated-key updates applied so far, their number)."""
        sm, cnt = C.c_double(0), C.c_uint64(0)
        self._chk(self._l.nups_get_clip_stats(self._s, C.byref(sm), C.byref(cnt), _stream()), "nups_get_clip_stats")
        return sm.value, cnt.value

    def merge_mark(self, which=0):
        """All GPUs hold the same table now: the agreed state that merges across GPUs start from."""
        self._chk(self._l.nups_merge_mark(self._s, which, _stream()), "nups_merge_mark")

    def merge_export(self, which=0, out=None):
        """This GPU's additions since the agreed state, [num_keys, value_len] (its own replicas merged first)."""
        if out is None:
            out = torch.empty((self.num_keys, self.L), dtype=self.dtype, device=self.device)
        self._chk(self._l.nups_merge_export(self._s, which, _ptr(out), _stream()), "nups_merge_export")
        return out

    def merge_apply(self, total, own, which=0):
        """Take over the other GPUs' additions: `total` = sum of every GPU's export, `own` = this GPU's."""
        assert total.dtype == self.dtype and own.dtype == self.dtype and total.numel() == own.numel() == self.num_keys * self.L
        self._chk(self._l.nups_merge_apply(self._s, which, _ptr(total), _ptr(own), _stream()), "nups_merge_apply")

    def set_sync_period(self, period_us):
        """Background merging of the replicas every `period_us` microseconds; 0 stops it."""
        self._chk(self._l.nups_set_sync_period(self._s, period_us), "nups_set_sync_period")


MAX_SHARDS = 16
SHARD_HANDLE_BYTES = 64


class ShardTable:
    """This process's part of a value table partitioned over several GPUs by key range; every shard is reached through
    peer memory by the calling GPU's own kernels (marshalling only: see `nups_shard_*` in include/nups.h)."""

    def __init__(self, num_keys, value_len, n_shards, my_shard):
        self._l = load()
        self.num_keys, self.L, self.n_shards, self.my_shard = num_keys, value_len, n_shards, my_shard
        self.keys_per_shard = -(-num_keys // n_shards)
        self.device = torch.device("cuda", torch.cuda.current_device())
        h = C.c_void_p()
        self._t = None
        self._chk(self._l.nups_shard_table_create(num_keys, value_len, n_shards, my_shard, C.byref(h)), "nups_shard_table_create")
        self._t = h

    def _chk(self, rc, what):
        if rc != 0:
            detail = self._l.nups_strerror(rc).decode()
            if self._t is not None and rc == ECUDA:
                detail += ": " + self._l.nups_shard_last_error(self._t).decode()
            raise NupsError(rc, what, detail)

    def close(self):
        if self._t is not None:
            self._l.nups_shard_table_destroy(self._t)
            self._t = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def local_address(self):
        p, n = C.c_void_p(), C.c_uint64()
        self._chk(self._l.nups_shard_table_local(self._t, C.byref(p), C.byref(n)), "nups_shard_table_local")
        return p.value, n.value

    def write_local(self, rows):
        """Fill the local shard from [keys_per_shard, value_len] fp32 values (host or device)."""
        t = torch.as_tensor(rows, dtype=torch.float32).to(self.device).contiguous()
        assert t.numel() == self.keys_per_shard * self.L
        self._chk(self._l.nups_shard_table_copy(self._t, _ptr(t), 1, _stream()), "nups_shard_table_copy")
        torch.cuda.current_stream().synchronize()

    def read_local(self):
        out = torch.empty((self.keys_per_shard, self.L), dtype=torch.float32, device=self.device)
        self._chk(self._l.nups_shard_table_copy(self._t, _ptr(out), 0, _stream()), "nups_shard_table_copy")
        torch.cuda.current_stream().synchronize()
        return out

    def export_handle(self) -> bytes:
        buf = C.create_string_buffer(SHARD_HANDLE_BYTES)
        self._chk(self._l.nups_shard_table_export(self._t, buf), "nups_shard_table_export")
        return buf.raw

    def attach(self, shard, address):
        self._chk(self._l.nups_shard_table_attach(self._t, shard, C.c_void_p(address)), "nups_shard_table_attach")

    def attach_handle(self, shard, handle: bytes):
        assert len(handle) == SHARD_HANDLE_BYTES
        self._chk(self._l.nups_shard_table_attach_ipc(self._t, shard, handle), "nups_shard_table_attach_ipc")

    def pull(self, keys, out=None):
        n = keys.numel()
        if out is None:
            out = torch.empty((n, self.L), dtype=torch.float32, device=self.device)
        self._chk(self._l.nups_shard_pull(self._t, _ptr(keys, torch.int32), n, _ptr(out, torch.float32), _stream()), "nups_shard_pull")
        return out

    def push(self, keys, delta):
        n = keys.numel()
        assert delta.dtype == torch.float32 and delta.numel() == n * self.L
        self._chk(self._l.nups_shard_push(self._t, _ptr(keys, torch.int32), n, _ptr(delta), _stream()), "nups_shard_push")

    def status_check(self):
        return self._l.nups_shard_status_check(self._t, _stream())
