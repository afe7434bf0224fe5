"""GPU parity of the composite transform Q1 (x) Q2 (paper Sec. 3.3) against the CPU oracle: the Cayley factor, the
unquantized rows and the quantized rows, for several (n1, n2) including the paper's 40 x 128."""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_09679_b200 import BfqError, Plan, synth
from parity import check_quant, check_rows_close, to_f64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def setup(n1, n2, rows, dtype, seed=3, std=0.1):
    theta2 = synth.angles(n2, "normal", seed)
    params = synth.cayley_params(n1, seed, std)
    x = synth.rows(rows, n1 * n2, "student_t3", seed + 1, outliers=4, outlier_scale=20.0, dtype=dtype)
    p = Plan(n2, DEV)
    p.set_angles(theta2.to(DEV))
    q1 = p.cayley(params.to(DEV), n1)
    Q1_ref = oracle.cayley(to_f64(params), n1)
    return p, q1, Q1_ref, to_f64(theta2), x


@pytest.mark.parametrize("n1", [2, 3, 17, 40, 64])
@pytest.mark.parametrize("std", [0.05, 1.0])
def test_cayley_factor(n1, std):
    params = synth.cayley_params(n1, 11, std)
    p = Plan(128, DEV)
    q1 = to_f64(p.cayley(params.to(DEV), n1))
    ref = oracle.cayley(to_f64(params), n1)
    assert np.abs(q1 - ref).max() <= 2e-7
    assert np.abs(q1 @ q1.T - np.eye(n1)).max() <= 2e-6


@pytest.mark.parametrize("n1,n2,rows", [(3, 16, 7), (5, 64, 130), (12, 256, 33), (40, 128, 61), (64, 256, 9), (7, 1024, 20)])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_composite_forward(n1, n2, rows, dtype):
    p, q1, Q1_ref, th2, x = setup(n1, n2, rows, dtype)
    if dtype == torch.bfloat16 and (n1, n2) == (40, 128):
        pytest.skip("covered by the tensor-core tests")
    y_ref = oracle.composite_forward(Q1_ref, th2, to_f64(x))
    amax = np.abs(to_f64(x)).max(axis=1)
    y = p.composite_forward(q1, x.to(DEV), out_dtype=torch.float32)
    check_rows_close(y, y_ref, amax, "composite fp32 out")
    yb = p.composite_forward(q1, x.to(DEV), out_dtype=torch.bfloat16)
    check_rows_close(yb, y_ref, amax, "composite bf16 out")
    assert p.device_status() == 0


@pytest.mark.parametrize("n1,n2,rows", [(3, 16, 7), (12, 256, 33), (40, 128, 61)])
@pytest.mark.parametrize("bits", [2, 4, 8])
def test_composite_forward_quant(n1, n2, rows, bits):
    p, q1, Q1_ref, th2, x = setup(n1, n2, rows, torch.float32)
    y_ref = oracle.composite_forward(Q1_ref, th2, to_f64(x))
    codes, scales = p.composite_forward_quant(q1, x.to(DEV), bits)
    check_quant(codes, scales, y_ref, bits, "composite quant")


def test_composite_identity_factor_is_the_butterfly_on_every_run():
    n1, n2, rows = 6, 128, 10
    p, _, _, th2, x = setup(n1, n2, rows, torch.float32)
    eye = torch.eye(n1, dtype=torch.float32, device=DEV)
    y = p.composite_forward(eye, x.to(DEV))
    y_runs = p.forward(x.to(DEV).reshape(rows * n1, n2)).reshape(rows, n1 * n2)
    assert torch.equal(y, y_runs) or (y - y_runs).abs().max() <= 1e-5 * x.abs().max()


def test_composite_argument_validation():
    p = Plan(128, DEV)
    p.set_angles(synth.angles(128, "normal", 1).to(DEV))
    x = torch.zeros((4, 40 * 128), dtype=torch.float32, device=DEV)
    with pytest.raises(BfqError) as e:
        p.composite_forward(torch.eye(65, device=DEV), torch.zeros((1, 65 * 128), device=DEV))
    assert e.value.status == -2
    big = Plan(2048, DEV)
    big.set_angles(synth.angles(2048, "normal", 1).to(DEV))
    with pytest.raises(BfqError) as e:
        big.composite_forward(torch.eye(2, device=DEV), torch.zeros((1, 4096), device=DEV))
    assert e.value.status == -2
    with pytest.raises(BfqError) as e:
        p.composite_forward_quant(torch.eye(40, device=DEV), x, 3)
    assert e.value.status == -3
    fresh = Plan(128, DEV)
    with pytest.raises(BfqError) as e:
        fresh.composite_forward(torch.eye(40, device=DEV), x)
    assert e.value.status == -7
    y = p.composite_forward(torch.eye(40, device=DEV), x[:0])
    assert y.shape == (0, 5120)
