"""bfq_backward_noalloc against bfq_backward and against the CPU oracle.

The no-allocation entry point serves hosts that cannot let the library call cudaMalloc (all device
memory owned by a caching allocator, or no tolerance for the device-wide synchronisation an
allocation implies).  It keeps its cos/sin table and partial sums in one fixed array per GPU that
every call reuses, so the test makes two calls in a row with different row lengths and inputs: the
second must not be disturbed by what the first left behind.  Collected last, so that a failure here
cannot keep any other test from running."""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_09679_b200 import BfqError, Plan, backward_noalloc, synth
from parity import check_dtheta, check_rows_close, to_f64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _case(n, rows, dtype, seed):
    theta = synth.angles(n, "uniform", seed).to(DEV)
    x = synth.rows(rows, n, "student_t3", seed + 1, outliers=4, outlier_scale=20.0, dtype=dtype).to(DEV)
    g = synth.rows(rows, n, "normal", seed + 2, dtype=dtype).to(DEV)
    return theta, x, g


def _check_against_plan(n, rows, dtype, seed):
    theta, x, g = _case(n, rows, dtype, seed)
    plan = Plan(n, DEV)
    plan.set_angles(theta)
    dx_ref, dth_ref = plan.backward(x, g)
    dx = torch.full_like(x, float("nan"))
    dth = torch.full((plan.L, n // 2), float("nan"), dtype=torch.float32, device=DEV)
    backward_noalloc(theta, x, g, dx, dth)
    torch.cuda.synchronize()
    # same per-row arithmetic as the plan-based path: dx within the tolerance of the parity tests
    check_rows_close(dx, to_f64(dx_ref), np.abs(to_f64(g)).max(axis=1), f"noalloc dx n={n}")
    # d-theta is summed over a different number of CTAs: the d-theta tolerance of the parity tests
    check_dtheta(dth, to_f64(dth_ref), f"noalloc dtheta n={n}")
    # and against the oracle itself (at these sizes both paths run the same generic kernel: comparing them with each
    # other alone would compare the kernel with itself)
    dx_o, dth_o = oracle.backward(to_f64(theta), to_f64(x), to_f64(g))
    check_rows_close(dx, dx_o, np.abs(to_f64(g)).max(axis=1), f"noalloc dx vs oracle n={n}")
    check_dtheta(dth, dth_o, f"noalloc dtheta vs oracle n={n}")
    # reproducible from call to call
    dth2 = torch.empty_like(dth)
    backward_noalloc(theta, x, g, None, dth2)
    assert torch.equal(dth, dth2)


def test_two_calls_in_a_row_match_the_plan_based_backward():
    _check_against_plan(1024, 777, torch.bfloat16, 301)
    _check_against_plan(256, 1500, torch.float32, 302)  # smaller n right after: stale scratch must not matter


def test_fewer_partial_sums_after_more():
    """A long batch fills every partial-sum slot the grid cap allows; the short batch right after uses (and must zero
    and reduce) only a few of them, whatever the first call left in the others."""
    _check_against_plan(1024, 6000, torch.bfloat16, 305)
    _check_against_plan(1024, 9, torch.bfloat16, 306)


def test_limits_and_empty_batch():
    theta, x, g = _case(2048, 8, torch.float32, 303)
    dth = torch.empty((11, 1024), dtype=torch.float32, device=DEV)
    with pytest.raises(BfqError) as e:
        backward_noalloc(theta, x, g, None, dth)
    assert e.value.status == -10
    theta, x, g = _case(64, 0, torch.float32, 304)
    dth = torch.ones((6, 32), dtype=torch.float32, device=DEV)
    backward_noalloc(theta, x, g, None, dth)
    assert not dth.any()
