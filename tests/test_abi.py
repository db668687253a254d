"""The C-ABI library loads, exports everything include/d2c.h declares, and rejects bad arguments on
the host before touching a device (none of these calls launches anything)."""
import ctypes as C
import os
import re

import pytest

from paper_2509_23094_b200 import binding, build, inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def _declared():
    text = open(os.path.join(ROOT, "include", "d2c.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(d2c_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert len(names) >= 17
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.SYMBOLS) == names


def test_workspace_bytes_and_config_validation(lib):
    cfg = binding.make_config(inputs.TOY, 1, 128)
    small = binding.d2c_workspace_bytes(cfg)
    assert small > 0 and small % 256 == 0
    # KV cache: 2 * L * N * d values (bf16), plus the rest
    big = binding.d2c_workspace_bytes(binding.make_config(inputs.LLADA_8B, 8, 4096))
    assert big > 2 * 32 * 8 * 4096 * 4096 * 2
    for field, val in [("head_dim", 96), ("d_model", 100), ("n_kv_heads", 3), ("max_seq", 10000), ("vocab", 1001),
                       ("sigma", 0.0), ("flags", 32), ("stage2_candidates", 2)]:
        bad = binding.make_config(inputs.TOY, 1, 128)
        setattr(bad, field, val)
        assert binding.d2c_workspace_bytes(bad) == 0, field
    assert lib.d2c_workspace_bytes(None) == 0


def test_create_rejects_bad_arguments_without_a_device(lib):
    cfg = binding.make_config(inputs.TOY, 1, 128)
    handle = C.c_void_p()
    w = binding.Weights()
    assert lib.d2c_create(C.byref(cfg), None, None, 0, None, C.byref(handle)) == binding.D2C_EINVAL
    assert "null" in binding.last_error()
    bad = binding.make_config(inputs.TOY, 1, 128); bad.head_dim = 80
    assert lib.d2c_create(C.byref(bad), C.byref(w), 256, 1 << 30, None, C.byref(handle)) == binding.D2C_ESHAPE
    assert lib.d2c_create(C.byref(cfg), C.byref(w), 256 + 8, 1 << 30, None, C.byref(handle)) == binding.D2C_EINVAL
    assert lib.d2c_create(C.byref(cfg), C.byref(w), 256, 1024, None, C.byref(handle)) == binding.D2C_ECAPACITY
    assert "workspace" in binding.last_error()
    assert lib.d2c_create(C.byref(cfg), C.byref(w), 256, 1 << 30, None, C.byref(handle)) == binding.D2C_EINVAL
    assert handle.value is None
    assert lib.d2c_destroy(None) == binding.D2C_EINVAL
    assert lib.d2c_step(None, None, None) == binding.D2C_EINVAL


def test_ops_reject_bad_arguments_without_a_device(lib):
    assert lib.d2c_op_select_scratch_bytes(0, 10) == 0
    assert lib.d2c_op_select_scratch_bytes(2, 100) >= 3 * 2 * 100 * 4
    assert lib.d2c_op_lm_head_scratch_bytes(32, 126464) >= 3 * 32 * 988 * 4
    assert lib.d2c_op_rollout_scratch_bytes(1, 1024) > 16 * 1024 * 4
    assert lib.d2c_op_gemm(None, None, None, None, None, 1, 2, 64, 0, None) == binding.D2C_EINVAL
    assert lib.d2c_op_gemm(256, 256, None, 256, 256, 8, 8, 32, 1, None) == binding.D2C_EINVAL
    assert lib.d2c_op_select(None, None, None, None, None, None, 1, 1, 0, 0.5, 10.0, 0, None, None, None, None, None,
                             None, None, 0, None) == binding.D2C_EINVAL
    assert lib.d2c_op_attention(None, 1, 0, None, None, None, 1, 1, 1, 1, 1, 64, None, None, None, 0, None) == binding.D2C_EINVAL
    assert lib.d2c_op_lm_head(None, None, None, 1, 64, 2, None, None, None, None, 0, None) == binding.D2C_EINVAL
    assert lib.d2c_op_rollout(None, 0, 1, None, None, 1, 1, None, None, 0, None) == binding.D2C_EINVAL
    lib.d2c_op_wait_probe.argtypes = [C.c_void_p, C.c_int64, C.c_void_p]
    assert lib.d2c_op_wait_probe(None, 100000, None) == binding.D2C_EINVAL
    assert lib.d2c_op_wait_probe(256, 10, None) == binding.D2C_EINVAL            # limit below 1e3 clocks
