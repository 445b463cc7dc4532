"""Host-side checks of the C ABI that need no GPU: the library loads, exports what the header
declares, validates arguments before touching CUDA, and agrees with the workload tables."""
import ctypes as C
import os
import re

import pytest

from paper_2107_01460_b200 import binding, build, workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def test_library_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "mava_rollout.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(mava_[a-z_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


@pytest.mark.parametrize("idx", range(5))
def test_params_count_and_record_len(lib, idx):
    w = wl.workload(idx)
    cfg = binding.make_config(w, precision=binding.MAVA_PRECISION_FP32)
    assert lib.mava_params_count(C.byref(cfg)) == wl.params_count(w)
    assert lib.mava_state_record_len(C.byref(cfg)) == 3 * (w["n_agents"] + w["n_food"]) + 3


def test_invalid_configs_are_rejected_before_any_cuda_call(lib):
    w = wl.workload(0)
    bufs = binding.mava_buffers_t(*([16] * 9))  # never dereferenced: validation comes first
    out = C.c_void_p()
    for field, bad in [("grid", 2), ("n_agents", 9), ("n_food", 0), ("max_agent_level", 4), ("episode_cap", 0),
                       ("n_envs", 0), ("max_T", 0), ("net_kind", 7), ("precision", 5)]:
        cfg = binding.make_config(w, precision=binding.MAVA_PRECISION_FP32)
        setattr(cfg, field, bad)
        assert lib.mava_params_count(C.byref(cfg)) == 0
        assert lib.mava_rollout_create(C.byref(cfg), C.byref(bufs), None, C.byref(out)) == binding.MAVA_ERR_INVALID_ARG
        assert not out.value
    cfg = binding.make_config(w, precision=binding.MAVA_PRECISION_FP32)
    assert lib.mava_rollout_create(None, C.byref(bufs), None, C.byref(out)) == binding.MAVA_ERR_INVALID_ARG
    assert lib.mava_rollout_create(C.byref(cfg), None, None, C.byref(out)) == binding.MAVA_ERR_INVALID_ARG
    nullbufs = binding.mava_buffers_t()
    assert lib.mava_rollout_create(C.byref(cfg), C.byref(nullbufs), None, C.byref(out)) == binding.MAVA_ERR_INVALID_ARG
    cfg.view_radius = 1
    assert lib.mava_rollout_create(C.byref(cfg), C.byref(bufs), None, C.byref(out)) == binding.MAVA_ERR_UNSUPPORTED
    cfg = binding.make_config(w, precision=binding.MAVA_PRECISION_FP32)
    cfg.hidden = 96  # not in the compiled shape table
    assert lib.mava_rollout_create(C.byref(cfg), C.byref(bufs), None, C.byref(out)) == binding.MAVA_ERR_UNSUPPORTED


def test_null_handles_are_harmless(lib):
    assert lib.mava_rollout_run(None, None, 1) == binding.MAVA_ERR_INVALID_ARG
    assert lib.mava_gae(None, 0.99, 0.95) == binding.MAVA_ERR_INVALID_ARG
    assert lib.mava_rollout_status(None) == binding.MAVA_ERR_INVALID_ARG
    assert lib.mava_rollout_launch_count(None) == 0
    lib.mava_rollout_destroy(None)
    assert binding.strerror(0) == "ok" and "capacity" in binding.strerror(binding.MAVA_ERR_CAPACITY)


def test_create_without_a_gpu_fails_cleanly(lib):
    import torch

    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    w = wl.workload(0)
    cfg = binding.make_config(w, precision=binding.MAVA_PRECISION_FP32)
    bufs = binding.mava_buffers_t(*([16] * 9))
    out = C.c_void_p()
    assert lib.mava_rollout_create(C.byref(cfg), C.byref(bufs), None, C.byref(out)) == binding.MAVA_ERR_CUDA
    assert not out.value


def test_product_path_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2107_01460_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(import|from)\s+oracle\b|mava_oracle|oracle/|orc_", text, flags=re.M), f
