"""The C-ABI library loads without a GPU and exports every symbol include/rtprune.h declares."""
import ctypes
import os
import re

from paper_2605_00392_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "rtprune.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rtprune_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    names = _declared()
    assert {"rtprune_plan", "rtprune_run", "rtprune_run_host", "rtprune_select",
            "rtprune_query_status", "rtprune_destroy"} <= set(names)
    lib = binding.lib()
    for n in names:
        assert getattr(lib, n) is not None, n


def test_host_only_calls():
    lib = binding.lib()
    assert lib.rtprune_version() >= 100
    assert lib.rtprune_status_string(0) == b"RTPRUNE_OK"
    assert lib.rtprune_status_string(3) == b"RTPRUNE_ERR_WORKSPACE"
    assert lib.rtprune_status_string(99) == b"RTPRUNE_ERR_UNKNOWN"
    p = binding.default_params()
    assert (p.dynamic, p.iters, p.form, p.stop_at_fixed_point) == (0, 100, 0, 1)
    assert abs(p.r_fixed - 0.25) < 1e-7 and abs(p.z - 0.2) < 1e-7 and abs(p.alpha - 0.1) < 1e-7
    assert p.eps == 1.0 and p.tol == 0.0 and p.rho is None
    assert lib.rtprune_default_params(None) == 1
    assert ctypes.sizeof(binding.CParams) == 64      # static_assert-ed in the library too


def test_plan_argument_checks_come_before_any_cuda_call():
    lib = binding.lib()
    h, ws = ctypes.c_void_p(), ctypes.c_size_t()
    args = lambda d, dt, nb, tot, mx: lib.rtprune_plan(ctypes.byref(h), d, dt, nb, tot, mx,
                                                      ctypes.byref(ws))
    assert args(1281, 0, 1, 10, 10) == 2          # d not a multiple of 8
    assert args(1282, 1, 1, 10, 10) == 2          # fp32: d not a multiple of 4
    assert args(8192, 0, 1, 10, 10) == 2          # d too wide
    assert args(1280, 0, 1, 10 ** 6, 9000) == 2   # image too long
    assert args(1280, 5, 1, 10, 10) == 1          # unknown dtype
    assert args(1280, 0, 0, 10, 10) == 1          # empty plan
    assert lib.rtprune_plan(None, 1280, 0, 1, 10, 10, ctypes.byref(ws)) == 1
    assert h.value is None
    lib.rtprune_destroy(None)                     # allowed
    assert lib.rtprune_last_launch_count(None) == 0


def test_no_cpu_fallback():
    import pytest
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(RuntimeError):
        binding.Plan(1280, torch.bfloat16, 1, 64, 64)


def test_shard_images_covers_the_batch():
    for batch, world in [(64, 1), (64, 8), (10, 4), (3, 8), (0, 2)]:
        spans = [binding.shard_images(batch, world, r) for r in range(world)]
        assert spans[0][0] == 0 and spans[-1][1] == batch
        assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
        sizes = [hi - lo for lo, hi in spans]
        assert max(sizes) - min(sizes) <= 1
