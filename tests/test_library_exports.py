"""The C-ABI library builds, loads and exports every symbol the public header declares (no GPU needed)."""
import ctypes
import os
import re

from paper_2104_00501_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "nups.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(nups_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build_library()
    lib = ctypes.CDLL(path)
    names = declared_symbols()
    assert len(names) >= 25
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/nups.h but not exported"
    assert sorted(binding.EXPORTS) == names


def test_binding_fails_loudly_without_a_device():
    import pytest
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    with pytest.raises(binding.NupsError) as e:
        binding.Store(10, 4)
    assert e.value.code == binding.ECUDA


def test_strerror_and_argument_checks_need_no_device():
    lib = binding.load()
    assert lib.nups_strerror(0) == b"ok"
    assert b"invalid" in lib.nups_strerror(binding.EINVAL)
    h = ctypes.c_void_p()
    assert lib.nups_create(0, 4, None, ctypes.byref(h)) == binding.EINVAL
    assert lib.nups_create(10, 3, None, ctypes.byref(h)) == binding.EINVAL      # rows must be 16-byte multiples
    assert lib.nups_create(1 << 33, 4, None, ctypes.byref(h)) == binding.EINVAL


def test_binding_config_mirrors_the_header_struct():
    # field for field, in order and width: a drifted mirror would silently hand the library other settings
    text = open(os.path.join(ROOT, "include", "nups.h")).read()
    body = re.search(r"typedef struct nups_config \{(.*?)\} nups_config;", text, flags=re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    header = []
    for ctype, name, dim in re.findall(r"\b(uint32_t|float)\s+([a-z_0-9]+)(?:\[(\d+)\])?;", body):
        header.append((name, ctype, int(dim) if dim else 1))
    mirror = []
    for name, ct in binding.Config._fields_:
        if hasattr(ct, "_length_"):
            mirror.append((name, "uint32_t" if ct._type_ is ctypes.c_uint32 else "float", ct._length_))
        else:
            mirror.append((name, "uint32_t" if ct is ctypes.c_uint32 else "float", 1))
    assert mirror == header
    assert ctypes.sizeof(binding.Config) == 64
    # creation rejects settings that cannot go together, before it looks for a device
    lib = binding.load()
    h = ctypes.c_void_p()
    cfg = binding.Config(deterministic=1, sync_period_us=100)
    assert lib.nups_create(10, 4, ctypes.byref(cfg), ctypes.byref(h)) == binding.EINVAL
    cfg = binding.Config(clip_factor=-1.0)
    assert lib.nups_create(10, 4, ctypes.byref(cfg), ctypes.byref(h)) == binding.EINVAL
    cfg = binding.Config(workers=255)
    assert lib.nups_create(10, 4, ctypes.byref(cfg), ctypes.byref(h)) == binding.EINVAL


def test_the_stores_own_memory_limit_refuses_before_the_device_is_touched():
    # 1000 keys x 64 floats need 256,000 bytes of table alone; with a 1 MiB limit a store of 10,000 keys cannot be
    # created, and that is found out from the sizes alone: NUPS_ENOMEM even on a box without a device
    lib = binding.load()
    h = ctypes.c_void_p()
    cfg = binding.Config(max_device_mib=1)
    assert lib.nups_create(10_000, 64, ctypes.byref(cfg), ctypes.byref(h)) == binding.ENOMEM
    assert not h.value
    cfg = binding.Config(max_device_mib=1, with_adagrad=1)
    assert lib.nups_create(2_000, 64, ctypes.byref(cfg), ctypes.byref(h)) == binding.ENOMEM      # two tables of 512,000 bytes
    cfg = binding.Config(merge_mean=1, sync_period_us=50)
    assert lib.nups_create(10, 4, ctypes.byref(cfg), ctypes.byref(h)) == binding.EINVAL
    cfg = binding.Config(first_epoch=1 << 24)
    assert lib.nups_create(10, 4, ctypes.byref(cfg), ctypes.byref(h)) == binding.EINVAL
