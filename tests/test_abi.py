"""The C-ABI library loads and exports every symbol include/trivance.h declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

from paper_2602_17254_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def library():
    build.build()
    return binding.lib()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "trivance.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(trv_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported(library):
    names = _declared_symbols()
    assert len(names) >= 19
    for name in names:
        assert hasattr(library, name), name
    assert sorted(binding.SYMBOLS) == names


def test_strerror_covers_every_status(library):
    seen = set()
    for s in range(9):
        msg = binding.strerror(s)
        assert msg and msg != "unknown status"
        seen.add(msg)
    assert len(seen) == 9
    assert binding.strerror(99) == "unknown status"


def test_plan_create_argument_errors(library):
    P = binding.Plan
    with pytest.raises(binding.TrivanceError) as e:
        P([7], binding.LATENCY_OPTIMAL)
    assert e.value.status == binding.ERR_UNSUPPORTED
    with pytest.raises(binding.TrivanceError) as e:
        P([1], binding.LATENCY_OPTIMAL)
    assert e.value.status == binding.ERR_INVALID_ARG
    with pytest.raises(binding.TrivanceError) as e:
        P([9, 9, 27], binding.LATENCY_OPTIMAL)         # 2187 ranks > TRV_MAX_RANKS
    assert e.value.status == binding.ERR_UNSUPPORTED
    with pytest.raises(binding.TrivanceError) as e:
        P([243], binding.LATENCY_OPTIMAL, binding.ALGO_RECDOUB)
    assert e.value.status == binding.ERR_UNDEFINED_SCHEDULE
    with pytest.raises(binding.TrivanceError) as e:
        P([9], 5)
    assert e.value.status == binding.ERR_INVALID_ARG
    h = ctypes.c_void_p()
    assert library.trv_plan_create(None, 1, 0, ctypes.byref(h)) == binding.ERR_INVALID_ARG
    assert library.trv_plan_destroy(None) == binding.ERR_INVALID_ARG


def test_allreduce_argument_errors_are_found_before_any_launch(library):
    """Host-side validation: none of these reaches a CUDA call, so they run without a GPU."""
    p = binding.Plan([9], binding.LATENCY_OPTIMAL)
    before = binding.launch_count()
    good = [0x1000 + 0x10000 * r for r in range(9)]
    cases = [
        (good[:8] + [0], 16, binding.FLOAT32, binding.ERR_INVALID_ARG),             # NULL buffer
        (good[:8] + [good[8] + 4], 16, binding.FLOAT32, binding.ERR_INVALID_ARG),   # misaligned
        (good[:8] + [good[0] + 32], 16, binding.FLOAT32, binding.ERR_INVALID_ARG),  # overlapping
        (good, 16, 7, binding.ERR_INVALID_ARG),                                      # dtype
    ]
    for ptrs, count, dtype, want in cases:
        with pytest.raises(binding.TrivanceError) as e:
            p.allreduce_ex(ptrs, None, count, dtype)
        assert e.value.status == want
    with pytest.raises(binding.TrivanceError) as e:
        p.allreduce_ex(good, None, 16, binding.FLOAT32, op=3)
    assert e.value.status == binding.ERR_UNSUPPORTED
    with pytest.raises(binding.TrivanceError) as e:
        p.allreduce_ex(good, None, 16, binding.FLOAT32, global_count=8)
    assert e.value.status == binding.ERR_INVALID_ARG
    # separate outputs may not overlap the inputs
    with pytest.raises(binding.TrivanceError) as e:
        p.allreduce_ex(good, [g + 16 for g in good], 16, binding.FLOAT32)
    assert e.value.status == binding.ERR_INVALID_ARG
    # comparator plans run step by step through a wire buffer: without one the call is refused before any launch
    b = binding.Plan([9], binding.LATENCY_OPTIMAL, binding.ALGO_BRUCK)
    with pytest.raises(binding.TrivanceError) as e:
        b.allreduce_ex(good, None, 16, binding.FLOAT32)
    assert e.value.status == binding.ERR_SCRATCH
    with pytest.raises(binding.TrivanceError) as e:
        b.allreduce_ex(good, None, 16, binding.FLOAT32, kernel=binding.KERNEL_FUSED)
    assert e.value.status == binding.ERR_UNSUPPORTED
    # count == 0 is fine and launches nothing
    p.allreduce_ex(good, None, 0, binding.FLOAT32)
    assert binding.launch_count() == before


def test_scratch_and_support_queries(library):
    lat27 = binding.Plan([27], binding.LATENCY_OPTIMAL)
    assert lat27.kernel_supported(binding.KERNEL_FUSED) and lat27.scratch_bytes(1000) == 0
    assert lat27.scratch_bytes(1000, binding.KERNEL_STEP, in_place=True) == 2 * 27 * 1024 * 4     # odd step count
    assert lat27.scratch_bytes(1000, binding.KERNEL_STEP, in_place=False) == 27 * 1024 * 4
    lat9 = binding.Plan([9], binding.LATENCY_OPTIMAL)
    assert lat9.scratch_bytes(64, binding.KERNEL_STEP) == 9 * 64 * 4
    assert binding.Plan([27, 9], binding.LATENCY_OPTIMAL).kernel_supported(binding.KERNEL_FUSED)     # generic line-group kernel
    odd = binding.Plan([243, 3], binding.LATENCY_OPTIMAL)               # a side above 81 off a ring: no fused latency kernel
    assert not odd.kernel_supported(binding.KERNEL_FUSED)
    assert odd.scratch_bytes(64) == odd.scratch_bytes(64, binding.KERNEL_STEP) > 0
    with pytest.raises(binding.TrivanceError):
        odd.scratch_bytes(64, binding.KERNEL_FUSED)
    bw = binding.Plan([9, 9, 9], binding.BANDWIDTH_OPTIMAL)
    assert bw.kernel_supported(binding.KERNEL_FUSED) and bw.scratch_bytes(10 ** 6, binding.KERNEL_STEP) == 0
    assert bw.host_workspace_bytes(1000) == 729 * 4096
