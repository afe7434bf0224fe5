"""Host-side checks of the C ABI that need no GPU: the library builds for sm_100a, loads, exports
every function include/bfq.h declares, the binding lists the same set, and the entry points that
can answer without a device (status strings, argument validation that precedes any CUDA call) do."""
import ctypes
import os
import re

import pytest

from paper_2509_09679_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "bfq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bfq_[a-z0-9_]+)\s*\(", text)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def test_header_functions_are_exported_and_bound(lib):
    names = declared_functions()
    for required in ("bfq_forward_quant", "bfq_inverse", "bfq_backward", "bfq_fold_weights"):
        assert required in names
    for name in names:
        assert hasattr(lib, name), f"{name} declared in bfq.h but not exported by libbfq.so"
    assert sorted(binding.SIGNATURES) == names


def test_status_strings(lib):
    codes = sorted(binding.STATUS_NAMES)
    assert codes == list(range(min(codes), 1))
    seen = {lib.bfq_status_string(c).decode() for c in codes}
    assert len(seen) == len(codes) and "unknown status" not in seen
    assert lib.bfq_status_string(-99).decode() == "unknown status"


def test_validation_that_precedes_any_cuda_call(lib):
    h = ctypes.c_void_p()
    assert lib.bfq_plan_create(None, 256, 0, 0) == -1                      # BFQ_ERR_NULL
    assert lib.bfq_plan_create(ctypes.byref(h), 100, 0, 0) == -2           # not a power of two
    assert lib.bfq_plan_create(ctypes.byref(h), 8, 0, 0) == -2             # below BFQ_MIN_N
    assert lib.bfq_plan_create(ctypes.byref(h), 16384, 0, 0) == -2         # above BFQ_MAX_N
    assert lib.bfq_plan_create(ctypes.byref(h), 256, -1, 0) == -5          # negative max_rows
    assert h.value is None
    assert lib.bfq_plan_destroy(None) == -1
    assert lib.bfq_last_cuda_error(None) == 0
    assert lib.bfq_backward_partials(None) == 0
    assert lib.bfq_forward_quant(None, None, 0, 0, 0, 4, None, None, None) == -1
    assert lib.bfq_forward_quant_host(None, None, 0, 0, 0, 4, None, None, None, 0, None) == -1
    assert lib.bfq_forward_quant_host_workspace(None, 0, 4, 128) == 0
    # the no-allocation backward checks its sizes before it touches the device
    assert lib.bfq_backward_noalloc(2048, None, None, 0, None, 0, 0, 2048, None, 0, None, None) == -10
    assert lib.bfq_backward_noalloc(100, None, None, 0, None, 0, 0, 100, None, 0, None, None) == -2
    assert lib.bfq_backward_noalloc(256, None, None, 0, None, 0, 0, 256, None, 0, None, None) == -1


def _planless(n=256):
    """A Plan object without a device handle: every check below must raise before the library is reached."""
    import torch

    p = object.__new__(binding.Plan)
    p.n, p.L, p.device, p._h = n, n.bit_length() - 1, torch.device("cuda", 0), ctypes.c_void_p()
    return p


def test_binding_rejects_bad_tensors_before_any_launch(monkeypatch):
    import torch

    def no_library():
        raise AssertionError("a bad tensor reached the C ABI")

    monkeypatch.setattr(binding, "lib", no_library)
    p = _planless(256)
    x = torch.zeros((4, 256))
    with pytest.raises(ValueError, match="is on cpu"):
        p.forward_quant(x, 4)                                   # host tensor
    with pytest.raises(ValueError, match="is on cpu"):
        p.backward(x, x)
    with pytest.raises(ValueError):
        p.forward(torch.zeros((4, 128)))                        # wrong row length
    with pytest.raises(ValueError):
        p.forward(torch.zeros((4, 512))[:, ::2])                # inner stride 2
    with pytest.raises(ValueError):
        p.set_angles(torch.zeros((8, 64)))                      # theta of a smaller n
    with pytest.raises(ValueError):
        p.set_angles(torch.zeros((8, 128), dtype=torch.float64))
    # caller-supplied outputs: exact dtype and shape, checked before the device
    with pytest.raises(ValueError, match="codes"):
        p._outputs(4, 256, 4, torch.zeros((4, 64), dtype=torch.uint8), torch.zeros((4,), dtype=torch.float16))
    with pytest.raises(ValueError, match="scales: expected"):
        binding._exact(torch.zeros((3,), dtype=torch.float16), torch.float16, (4,), p.device, "scales")
    with pytest.raises(ValueError, match="codes: tensor is on cpu"):
        p._outputs(4, 256, 4, torch.zeros((4, 128), dtype=torch.uint8), torch.zeros((4,), dtype=torch.float16))
    with pytest.raises(ValueError, match="codes"):
        p._outputs(4, 256, 4, torch.zeros((4, 128), dtype=torch.int8), torch.zeros((4,), dtype=torch.float16))
    # the plan-less entry point sizes theta and dtheta from x
    with pytest.raises(ValueError):
        binding.backward_noalloc(torch.zeros((8, 128)), x, x, None, torch.zeros((8, 128)))
    with pytest.raises(ValueError):
        binding._rows(torch.zeros((4, 300)).as_strided((4, 256), (100, 1)), 256)   # overlapping rows
    with pytest.raises(ValueError, match="expected 4 rows"):
        binding._rows(torch.zeros((5, 256)), 256, None, 4, "out")
