"""Layer-wise calibration of the butterfly angles (paper Sec. 3.4 / "Experimental Setup"): SGD with a cosine
learning-rate schedule from the identity initialisation on the reconstruction loss

    L_recon = mean || W x - Dequant(Quant(W B^T)) . Dequant(Quant(B x)) ||^2 .

Everything runs in the bfq kernels: forward, forward + quantize, weight folding, backward for the angle gradient, and
the dense products (bfq_dequant_gemm: tensor cores, the packed codes dequantized on the fly, fp32 operands split into two
bf16 terms); only element-wise glue (the error, its square, the scaling of the gradient) is torch.  The
quantizers are not differentiable; as usual their gradient is passed straight through (the paper does not
say so explicitly: this is the reading taken here).  With act_bits = None activations stay unquantized
(the paper's W2A16 setting).  Synthetic (W, x) only: the paper's models and calibration set are not here.
"""
from __future__ import annotations

import math

import torch

from .binding import GemmOperand, Plan


def unpack_codes(codes: torch.Tensor, bits: int) -> torch.Tensor:
    """[rows][n*bits/8] packed two's-complement codes -> [rows][n] int32 (element k in bits
    [bits*(k mod 8/bits), +bits) of byte k*bits/8)."""
    per = 8 // bits
    shifts = torch.arange(per, device=codes.device, dtype=torch.int32) * bits
    v = (codes.to(torch.int32).unsqueeze(-1) >> shifts) & ((1 << bits) - 1)
    v = torch.where(v >= (1 << (bits - 1)), v - (1 << bits), v)
    return v.reshape(codes.shape[0], -1)


def dequantize(codes: torch.Tensor, scales: torch.Tensor, bits: int) -> torch.Tensor:
    """Dequant(q) = s * q with the stored fp16 scale, as fp32."""
    return unpack_codes(codes, bits).to(torch.float32) * scales.to(torch.float32).unsqueeze(1)


class LayerCalibrator:
    """Angles of one linear layer y = W x (W: [out][n]) learned so that the rotated, quantized layer
    reproduces it on calibration rows."""

    def __init__(self, W: torch.Tensor, weight_bits: int = 2, act_bits: int | None = None, theta: torch.Tensor | None = None):
        if W.dim() != 2 or not W.is_cuda:
            raise ValueError("W must be a [out][n] CUDA tensor")
        self.W = W.contiguous()
        self.n = W.shape[1]
        self.weight_bits, self.act_bits = int(weight_bits), act_bits
        self.plan = Plan(self.n, W.device)
        L = self.n.bit_length() - 1
        # identity initialisation (all angles zero): the paper's default
        self.theta = torch.zeros((L, self.n // 2), dtype=torch.float32, device=W.device) if theta is None else theta.clone()
        self.plan.set_angles(self.theta)

    def loss_and_grad(self, x: torch.Tensor):
        """x: [tokens][n] calibration rows (same dtype as W); tokens and the layer's output width must be multiples
        of 64 (the K block of the dense products).  Returns (loss, dL/dtheta)."""
        p, W, wb = self.plan, self.W, self.weight_bits
        ref = p.dequant_gemm(GemmOperand(x), GemmOperand(W))                      # W x, the target
        w_codes, w_scales, _ = p.fold_weights(W, wb)                              # Quant(W B^T), codes + scales
        Wq = GemmOperand(w_codes, w_scales, wb)
        if self.act_bits is None:
            y = p.forward(x)                                                      # B x, kept in 16+ bits
            Yq, YqT = GemmOperand(y), GemmOperand(y, transposed=True)
        else:
            a_codes, a_scales = p.forward_quant(x, self.act_bits)                 # Quant(B x)
            Yq = GemmOperand(a_codes, a_scales, self.act_bits)
            YqT = GemmOperand(a_codes, a_scales, self.act_bits, transposed=True)
        err = p.dequant_gemm(Yq, Wq) - ref                                        # [tokens][out]
        loss = (err * err).mean()
        e = err * (2.0 / err.numel())
        # dL/d(B x) = e Wq and dL/d(W B^T) = e^T yq, straight through the two quantizers: the contraction runs across
        # the stored rows of the codes (their scales vary along it) and of e
        g_y = p.dequant_gemm(GemmOperand(e), GemmOperand(w_codes, w_scales, wb, transposed=True))
        g_w = p.dequant_gemm(GemmOperand(e, transposed=True), YqT)
        # row i of W B^T is B w_i: both gradients flow through the same transform, one on the activation rows
        # and one on the weight rows
        _, dth_x = p.backward(x, g_y.to(x.dtype), want_dx=False)
        _, dth_w = p.backward(W, g_w.to(W.dtype), want_dx=False)
        return loss, dth_x + dth_w

    def step(self, grad: torch.Tensor, lr: float):
        self.theta -= lr * grad
        self.plan.set_angles(self.theta)


def cosine_lr(step: int, steps: int, lr0: float) -> float:
    return 0.5 * lr0 * (1.0 + math.cos(math.pi * step / max(1, steps)))


def calibrate(W: torch.Tensor, X: torch.Tensor, steps: int = 200, lr0: float | None = None, batch: int = 2048,
              weight_bits: int = 2, act_bits: int | None = None, seed: int = 0):
    """SGD + cosine schedule from identity.  Returns (calibrator, list of per-step losses).  The paper gives no
    learning rate; lr0 = None takes 0.5 / max|gradient| of the first step (largest first move: half a radian)."""
    cal = LayerCalibrator(W, weight_bits, act_bits)
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    losses = []
    for it in range(steps):
        if batch >= X.shape[0]:
            xb = X  # full batch
        else:
            xb = X[torch.randint(0, X.shape[0], (batch,), generator=gen).to(X.device)]
        loss, grad = cal.loss_and_grad(xb)
        if lr0 is None:
            lr0 = 0.5 / max(float(grad.abs().max()), 1e-30)
        losses.append(float(loss))
        cal.step(grad, cosine_lr(it, steps, lr0))
    return cal, losses
