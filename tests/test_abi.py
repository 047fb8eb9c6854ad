"""The shared library loads, exports every symbol the header declares, and its host-only entry points
behave; compute calls are not made here (no GPU needed)."""

import ctypes as C
import os
import re

import pytest
import torch

from paper_2608_05326_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "qevict.h")).read()
    return sorted(set(re.findall(r"QEVICT_API\s+[\w\s\*]+?\b(qevict_\w+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_symbols()
    assert len(names) >= 18
    for n in names:
        assert hasattr(lib, n), n
    # and the binding knows the signature of each
    assert set(names) == set(binding._SIGNATURES)


def test_version_and_status_strings(lib):
    assert re.match(r"^\d+\.\d+$", binding.qevict_version())
    assert lib.qevict_status_string(0) == b"ok"
    assert lib.qevict_status_string(4) == b"unsupported configuration"


def test_budget_from_bytes_matches_closed_form(lib):
    cfg = binding.make_config(1, 1, 32, 8, 128, "bf16", 32, 4, 32, 1, 1, 4096)
    kf, kq, mf, mq = binding.qevict_budget_from_bytes(cfg, 10_000_000, 0.7)
    assert (mf, mq) == (131072, 40960)
    assert (kf, kq) == (22, 170)
    cfg2 = binding.make_config(1, 1, 32, 8, 128, "fp16", 32, 2, 32, 1, 1, 4096)
    _, _, mf2, mq2 = binding.qevict_budget_from_bytes(cfg2, 0, 0.5)
    assert mq2 * 16 == mf2 * 3  # INT2, group 32: 3/16 of a 16-bit window


def test_workspace_and_validation(lib):
    cfg = binding.make_config(1, 1, 32, 8, 128, "bf16", 32, 4, 32, 64, 128, 32768 + 512)
    n = binding.qevict_workspace_bytes(cfg)
    pools = (64 + 2 + 1) * 131072 + (128 + 64) * 40960
    assert pools <= n < pools + (8 << 20)
    bad = binding.make_config(1, 1, 32, 5, 128, "bf16", 32, 4, 32, 64, 128, 32768)
    with pytest.raises(binding.QEvictError) as e:
        binding.qevict_workspace_bytes(bad)
    assert e.value.status == 1
    unsup = binding.make_config(1, 1, 32, 2, 128, "bf16", 32, 4, 32, 64, 128, 32768)  # 16 heads per KV head
    with pytest.raises(binding.QEvictError) as e:
        binding.qevict_workspace_bytes(unsup)
    assert e.value.status == 4
    unsup2 = binding.make_config(1, 1, 8, 8, 96, "bf16", 32, 4, 32, 8, 8, 4096)
    with pytest.raises(binding.QEvictError) as e:
        binding.qevict_workspace_bytes(unsup2)
    assert e.value.status in (1, 4)


def test_shapes_the_kernels_cannot_walk_are_refused_with_a_reason(lib):
    def refused(cfg, word):
        with pytest.raises(binding.QEvictError) as e:
            binding.qevict_workspace_bytes(cfg)
        assert e.value.status == 4 and word in str(e.value), str(e.value)
        assert word in lib.qevict_last_error(None).decode()

    # budgets whose decode work list would exceed 32 entries x 4 warps x 64 splits
    refused(binding.make_config(1, 1, 8, 8, 64, "bf16", 32, 4, 32, 4096, 4100, 8192 * 32), "work-list")
    # routing tables of one sequence beyond the shared memory of an SM
    refused(binding.make_config(1, 1, 8, 8, 64, "bf16", 32, 4, 32, 4000, 4000, 8192 * 32), "shared memory")
    # key-norm ranking stages H_kv * d <= 4096 elements of the token
    refused(binding.make_config(1, 1, 64, 64, 128, "bf16", 32, 4, 32, 8, 8, 4096, rank_mode=3), "key-norm")
    # a failed call does not disturb a good one, and the largest BASELINE shape passes
    ok = binding.make_config(4, 8, 32, 8, 128, "bf16", 64, 4, 64, 64, 256, 131072 + 1024)
    assert binding.qevict_workspace_bytes(ok) > 0


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-device error path")
def test_create_without_a_device_fails_loudly(lib):
    cfg = binding.make_config(1, 1, 4, 2, 64, "fp16", 32, 4, 32, 2, 2, 1024)
    h = C.c_void_p()
    fake = C.c_void_p(256 * 1024)  # never dereferenced on the host; no device to clear it on
    st = lib.qevict_create(C.byref(cfg), fake, 1 << 30, C.byref(h))
    assert st == 5 and not h.value  # QEVICT_ERR_CUDA, no handle, no fallback
    assert b"device" in lib.qevict_last_error(None)
