"""The C-ABI shared library builds, loads and exports every symbol include/lossy.h declares.
No compute call is made here (no GPU needed)."""
import ctypes
import os
import re

import pytest

import paper_2507_07114_b200 as L
from paper_2507_07114_b200 import build as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "lossy.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lossy_[a-z0-9_]+|drift_[a-z_]+)\s*\(", text)))


def test_header_symbols_are_exported_and_bound():
    B.build()
    lib = ctypes.CDLL(B.LIB_PATH)
    names = _declared()
    assert "lossy_init" in names and "drift_norms" in names and "lossy_fused_step" in names
    for n in names:
        assert hasattr(lib, n), f"{n} declared in lossy.h but not exported"
        assert n in L.EXPORTS, f"{n} has no Python binding of the same name"
        assert callable(getattr(L, n))
    assert sorted(L.EXPORTS) == names
    # the debug twin (-DLOSSY_DEVCHECK: index checks in the kernels) has the same entry points and says what it is
    chk = ctypes.CDLL(B.CHECK_LIB_PATH)
    for n in names:
        assert hasattr(chk, n), f"{n} missing from the debug build"
    assert lib.lossy_has_device_checks() == 0 and chk.lossy_has_device_checks() == 1


def test_config_struct_layout_matches_the_header():
    # uint32 W, P; uint64 n, base; double x2; uint64 seed; uint32 x4; float x4; uint64 x2
    assert ctypes.sizeof(L.lossy_config) == 4 + 4 + 8 + 8 + 8 + 8 + 8 + 16 + 16 + 8 + 8
    assert L.lossy_config.shard_packet0.offset == 80
    assert L.lossy_config.n.offset == 8 and L.lossy_config.seed.offset == 40 and L.lossy_config.lr.offset == 64


def test_host_only_entry_points_work_without_a_gpu():
    # the delivery-indicator hash is a pure host function of its arguments
    a = L.lossy_hash_u32(1, 2, 3, 4, 5)
    assert a == L.lossy_hash_u32(1, 2, 3, 4, 5) and a != L.lossy_hash_u32(1, 2, 4, 3, 5)
    assert L.lossy_mask(None, 1, 0, 0, 0) == -1
    assert L.lossy_num_packets(None) == 0


def test_missing_library_fails_loudly():
    with pytest.raises(FileNotFoundError):
        L.load_library(os.path.join(ROOT, "no_such_dir", "liblossy_b200.so"))


def test_product_path_never_touches_the_oracle():
    pkg = os.path.join(ROOT, "paper_2507_07114_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.lower(), f"{f} mentions the oracle"
    for f in ("lossy_oracle.c", "oracle.py"):
        src = open(os.path.join(ROOT, "oracle", f)).read()
        assert "paper_2507_07114_b200" not in src and "lossy.h" not in src


def test_configuration_is_validated_on_the_host_before_any_cuda_call():
    """Bad configurations are rejected with LOSSY_EINVAL by plain host code, so this runs without a GPU."""
    lib = L.load_library()
    good = dict(W=8, packet_elems=2048, n=2048 * 10, packet_base=0, p_grad=0.1, p_param=0.1, seed=0,
                grad_dtype=L.LOSSY_BF16, replica_dtype=L.LOSSY_BF16, optimizer=L.LOSSY_ADAM, flags=0,
                lr=3e-4, beta1=0.9, beta2=0.95, eps=1e-8, shard_packet0=0, bucket_packets=0)
    bad = [dict(W=0), dict(W=65), dict(packet_elems=0), dict(packet_elems=100), dict(p_grad=1.0),
           dict(p_param=-1e-9), dict(p_grad=float("nan")), dict(grad_dtype=2), dict(replica_dtype=7),
           dict(optimizer=2), dict(flags=128), dict(n=2 ** 40, packet_elems=8),          # more than 2^31 chunks
           dict(shard_packet0=1), dict(shard_packet0=8, bucket_packets=12),             # range leaves the bucket
           dict(n=2048 * 10 - 8, bucket_packets=20)]                                    # ragged range inside a bucket
    for change in bad:
        kw = dict(good)
        kw.update(change)
        cfg = L.lossy_config(**kw)
        ctx = ctypes.c_void_p()
        assert lib.lossy_init(ctypes.byref(cfg), ctypes.byref(ctx)) == L.LOSSY_EINVAL, change
        assert not ctx.value
    assert lib.lossy_init(None, None) == L.LOSSY_EINVAL
    # entry points refuse a NULL context instead of dereferencing it
    assert lib.lossy_set_lr(None, 0.1) == L.LOSSY_EINVAL
    assert lib.lossy_device_status(None, None) == L.LOSSY_EINVAL
    assert lib.lossy_last_error(None) == b"NULL context"
    lib.lossy_destroy(None)
