"""The C ABI as a binary: the shared library loads without a GPU and exports every function that
include/libra.h declares; host-visible misuse is rejected with a status code."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "libra.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(libra_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert len(names) >= 15
    dll = ctypes.CDLL(lib.LIB_PATH)
    for n in names:
        assert hasattr(dll, n), n
    assert set(names) == set(lib.SIGNATURES), set(names) ^ set(lib.SIGNATURES)


def test_status_strings(lib):
    assert lib.libra_version() >= 100
    seen = {lib.libra_status_string(s) for s in range(7)}
    assert len(seen) == 7 and "unknown status" not in seen
    assert lib.libra_status_string(99) == "unknown status"


def test_create_rejects_bad_shapes_before_touching_cuda(lib):
    H = lib.Handle
    for kwargs, status in [
        (dict(num_q_heads=30, num_kv_heads=8, head_dim=128), lib.INVALID_ARGUMENT),
        (dict(num_q_heads=32, num_kv_heads=8, head_dim=96), lib.UNSUPPORTED_SHAPE),
        (dict(num_q_heads=32, num_kv_heads=1, head_dim=128), lib.UNSUPPORTED_SHAPE),   # group 32 > 16
        (dict(num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=48), lib.UNSUPPORTED_SHAPE),
        (dict(num_q_heads=32, num_kv_heads=8, head_dim=128, kv_strides=(16384, 2048, 100)), lib.INVALID_ARGUMENT),
        (dict(num_q_heads=32, num_kv_heads=8, head_dim=128, sm_scale=-1.0), lib.INVALID_ARGUMENT),
        (dict(num_q_heads=0, num_kv_heads=8, head_dim=128), lib.INVALID_ARGUMENT),
    ]:
        args = dict(num_pages=64, max_batch=4, block_table_ld=8)
        args.update(kwargs)
        with pytest.raises(lib.LibraError) as e:
            H(**args)
        assert e.value.status == status, kwargs


def test_null_handles_are_rejected(lib):
    import ctypes as C
    assert lib.lib.libra_destroy(None) == lib.OK
    n = C.c_size_t(0)
    assert lib.lib.libra_workspace_size(None, C.byref(n)) == lib.INVALID_ARGUMENT
    assert lib.lib.libra_plan(None, None, 0, None, 0, None) == lib.INVALID_ARGUMENT
    assert lib.lib.libra_decode_attn(None, None, None, None, None, None, None, None) == lib.INVALID_ARGUMENT
    assert lib.lib.libra_create(None, None) == lib.INVALID_ARGUMENT
    assert lib.lib.libra_last_cuda_error(None) == 0
