"""ctypes binding of libbfq.so: the same names as the C ABI, argument marshalling only.

Every step of the path runs in the CUDA kernels behind these calls.  There is no CPU
fallback: if the library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libbfq.so")

BFQ_F32, BFQ_BF16 = 0, 1
BFQ_OK = 0
STATUS_NAMES = {
    0: "BFQ_OK", -1: "BFQ_ERR_NULL", -2: "BFQ_ERR_UNSUPPORTED_N", -3: "BFQ_ERR_BITS", -4: "BFQ_ERR_ALIGN",
    -5: "BFQ_ERR_STRIDE", -6: "BFQ_ERR_DTYPE", -7: "BFQ_ERR_WORKSPACE", -8: "BFQ_ERR_CUDA",
    -9: "BFQ_ERR_DEVICE_TIMEOUT", -10: "BFQ_ERR_TOO_LARGE",
}

# name -> (restype, argtypes); must list every symbol include/bfq.h declares
_i, _i64, _p = ctypes.c_int, ctypes.c_int64, ctypes.c_void_p
SIGNATURES = {
    "bfq_plan_create": (_i, [ctypes.POINTER(_p), _i, _i64, _i]),
    "bfq_plan_destroy": (_i, [_p]),
    "bfq_set_angles": (_i, [_p, _p, _p]),
    "bfq_forward": (_i, [_p, _p, _i, _i64, _i64, _p, _i, _i64, _p]),
    "bfq_forward_quant": (_i, [_p, _p, _i, _i64, _i64, _i, _p, _p, _p]),
    "bfq_forward_quant_stats": (_i, [_p, _p, _i, _i64, _i64, _i, _p, _p, _p, _p, _p]),
    "bfq_inverse": (_i, [_p, _p, _i, _i64, _i64, _p, _i, _i64, _p]),
    "bfq_hadamard": (_i, [_p, _p, _i, _i64, _i64, _p, _i, _i64, _p]),
    "bfq_hadamard_quant": (_i, [_p, _p, _i, _i64, _i64, _i, _p, _p, _p]),
    "bfq_backward": (_i, [_p, _p, _i, _p, _i, _i64, _i64, _p, _i, _p, _p]),
    "bfq_fold_weights": (_i, [_p, _p, _i, _i64, _i64, _i, _p, _p, _p, _i, _p]),
    "bfq_device_status": (_i, [_p]),
    "bfq_last_cuda_error": (_i, [_p]),
    "bfq_status_string": (ctypes.c_char_p, [_i]),
    "bfq_backward_partials": (_i, [_p]),
    "bfq_forward_quant_host": (_i, [_p, _p, _i, _i64, _i64, _i, _p, _p, _p, ctypes.c_size_t, _p]),
    "bfq_forward_quant_host_workspace": (ctypes.c_size_t, [_p, _i, _i, _i64]),
    "bfq_measure_fma_rates": (_i, [_p]),
    "bfq_measure_mma_rates": (_i, [_p]),
    "bfq_dequant_gemm": (_i, [_p, _i64, _i64, _i64, ctypes.c_float, _p, _i, _i, _i64, _p, _p, _i, _i, _i64, _p, _p, _i64, _p]),
    "bfq_stage_form": (_i, [_p]),
    "bfq_test_stuck_wait": (_i, [_p, _i]),
    "bfq_backward_noalloc": (_i, [_i, _p, _p, _i, _p, _i, _i64, _i64, _p, _i, _p, _p]),
    "bfq_cayley": (_i, [_p, _p, _i, _p, _p]),
    "bfq_composite_forward": (_i, [_p, _p, _i, _p, _i, _i64, _i64, _p, _i, _i64, _p]),
    "bfq_composite_forward_quant": (_i, [_p, _p, _i, _p, _i, _i64, _i64, _i, _p, _p, _p]),
    "bfq_composite_inverse": (_i, [_p, _p, _i, _p, _i, _i64, _i64, _p, _i, _i64, _p]),
}

_lib = None


class BfqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().bfq_status_string(status).decode()
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} ({msg})")


def lib() -> ctypes.CDLL:
    """Loads libbfq.so (raises if it has not been built: there is no fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not found: run `python -m paper_2509_09679_b200.build` "
                               "(the CUDA library is the only implementation)")
        L = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def _check(status: int, where: str):
    if status != BFQ_OK:
        raise BfqError(status, where)


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return BFQ_F32
    if t.dtype == torch.bfloat16:
        return BFQ_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _rows(t: torch.Tensor, n: int, device=None, rows=None, what: str = "rows"):
    """Checks a [rows][n] row tensor (unit inner stride; on `device` when given; `rows` rows when given) and returns
    (rows, leading dimension).  Only this layer knows the buffers' sizes: the C ABI takes bare pointers."""
    if not isinstance(t, torch.Tensor) or t.dim() != 2 or t.shape[1] != n or t.stride(1) != 1:
        raise ValueError(f"{what}: expected a [rows][{n}] tensor with unit inner stride, got "
                         f"{tuple(t.shape) if isinstance(t, torch.Tensor) else type(t)}")
    if device is not None:
        _on(t, device, what)
    if rows is not None and t.shape[0] != rows:
        raise ValueError(f"{what}: expected {rows} rows, got {t.shape[0]}")
    if t.shape[0] > 1 and t.stride(0) < n:
        raise ValueError(f"{what}: rows overlap (row stride {t.stride(0)} < {n})")
    return t.shape[0], (t.stride(0) if t.shape[0] > 1 else max(t.stride(0), n))


def _on(t: torch.Tensor, device, what: str):
    if not t.is_cuda or t.device != device:
        raise ValueError(f"{what}: tensor is on {t.device}, the plan works on {device}")


def _exact(t: torch.Tensor, dtype, shape, device, what: str):
    """A contiguous tensor of exactly this dtype and shape on `device` (tables, codes, scales, statistics)."""
    if not isinstance(t, torch.Tensor) or t.dtype != dtype or tuple(t.shape) != tuple(shape) or not t.is_contiguous():
        got = (t.dtype, tuple(t.shape)) if isinstance(t, torch.Tensor) else type(t)
        raise ValueError(f"{what}: expected a contiguous {dtype} tensor of shape {tuple(shape)}, got {got}")
    _on(t, device, what)
    return t


def _stream(t: torch.Tensor):
    return ctypes.c_void_p(torch.cuda.current_stream(t.device).cuda_stream)


class GemmOperand:
    """One operand of Plan.dequant_gemm: rows of fp32 / bf16 numbers, or packed codes with the fp16 scales of their
    stored rows; `transposed` = stored [K][rows] instead of [rows][K]."""

    def __init__(self, data: torch.Tensor, scales: torch.Tensor | None = None, bits: int = 0, transposed: bool = False):
        if data.dim() != 2 or data.stride(1) != 1:
            raise ValueError("operand: expected a 2-D tensor with unit inner stride")
        self.data, self.scales, self.transposed = data, scales, bool(transposed)
        if scales is None:
            self.kind, per = _dt(data), 1
        else:
            if bits not in (2, 4, 8) or data.dtype != torch.uint8:
                raise ValueError("operand: codes are uint8 with bits in {2, 4, 8}")
            self.kind, per = bits, 8 // bits
            _exact(scales, torch.float16, (data.shape[0],), data.device, "operand scales")
        stored_rows, width = data.shape[0], data.shape[1] * per
        self.rows, self.k = (width, stored_rows) if transposed else (stored_rows, width)
        self.ld = (data.stride(0) if stored_rows > 1 else data.shape[1]) * per


class Plan:
    """Owns a bfq_plan for row length n on one CUDA device."""

    def __init__(self, n: int, device=None, max_rows: int = 0):
        dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
        if dev.type != "cuda":
            raise ValueError("bfq runs on CUDA devices only")
        self.n = int(n)
        self.L = self.n.bit_length() - 1
        self.device = torch.device("cuda", dev.index if dev.index is not None else torch.cuda.current_device())
        self._h = ctypes.c_void_p()
        _check(lib().bfq_plan_create(ctypes.byref(self._h), self.n, int(max_rows), self.device.index),
               "bfq_plan_create")

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            lib().bfq_plan_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the C ABI, one method per entry point ------------------------------------------------------
    def set_angles(self, theta: torch.Tensor):
        _exact(theta, torch.float32, (self.L, self.n // 2), self.device, "theta")
        _check(lib().bfq_set_angles(self._h, theta.data_ptr(), _stream(theta)), "bfq_set_angles")

    def forward(self, x: torch.Tensor, out_dtype=None, out: torch.Tensor | None = None) -> torch.Tensor:
        rows, ldx = _rows(x, self.n, self.device, what="x")
        y = out if out is not None else torch.empty((rows, self.n), dtype=out_dtype or x.dtype, device=x.device)
        _, ldy = _rows(y, self.n, self.device, rows, "out")
        _check(lib().bfq_forward(self._h, x.data_ptr(), _dt(x), rows, ldx, y.data_ptr(), _dt(y), ldy, _stream(x)),
               "bfq_forward")
        return y

    def _outputs(self, rows: int, width: int, bits: int, codes, scales):
        """Allocates or checks the codes uint8 [rows][width * bits / 8] and scales fp16 [rows] buffers (the bit width
        itself is the C side's to reject, before any launch)."""
        bits = int(bits)
        if codes is None:
            codes = torch.empty((rows, width * bits // 8), dtype=torch.uint8, device=self.device)
        if scales is None:
            scales = torch.empty((rows,), dtype=torch.float16, device=self.device)
        _exact(codes, torch.uint8, (rows, width * bits // 8), self.device, "codes")
        _exact(scales, torch.float16, (rows,), self.device, "scales")
        return codes, scales

    def forward_quant(self, x: torch.Tensor, bits: int, codes=None, scales=None):
        rows, ldx = _rows(x, self.n, self.device, what="x")
        codes, scales = self._outputs(rows, self.n, bits, codes, scales)
        _check(lib().bfq_forward_quant(self._h, x.data_ptr(), _dt(x), rows, ldx, int(bits), codes.data_ptr(),
                                       scales.data_ptr(), _stream(x)), "bfq_forward_quant")
        return codes, scales

    # -- composite transform Q1 (x) Q2 for d = n1 * n (paper Sec. 3.3); this plan's butterfly is Q2 --------------
    def cayley(self, params: torch.Tensor, n1: int) -> torch.Tensor:
        """Q1 = (I - A)(I + A)^-1 from the n1 (n1 - 1) / 2 upper-triangle entries of the skew A -> fp32 [n1][n1]."""
        if params.dtype != torch.float32 or params.numel() != n1 * (n1 - 1) // 2 or not params.is_contiguous():
            raise ValueError("params must be a contiguous fp32 tensor of n1 (n1 - 1) / 2 entries")
        _on(params, self.device, "params")
        q1 = torch.empty((n1, n1), dtype=torch.float32, device=params.device)
        _check(lib().bfq_cayley(self._h, params.data_ptr(), int(n1), q1.data_ptr(), _stream(params)), "bfq_cayley")
        return q1

    def _q1(self, q1: torch.Tensor) -> int:
        if q1.dtype != torch.float32 or q1.dim() != 2 or q1.shape[0] != q1.shape[1] or not q1.is_contiguous():
            raise ValueError("q1 must be a contiguous fp32 [n1][n1] tensor")
        _on(q1, self.device, "q1")
        return q1.shape[0]

    def composite_forward(self, q1: torch.Tensor, x: torch.Tensor, out_dtype=None, out=None) -> torch.Tensor:
        n1 = self._q1(q1)
        d = n1 * self.n
        rows, ldx = _rows(x, d, self.device, what="x")
        y = out if out is not None else torch.empty((rows, d), dtype=out_dtype or x.dtype, device=x.device)
        if _rows(y, d, self.device, rows, "out")[1] != d:
            raise ValueError("out: rows must be contiguous")
        _check(lib().bfq_composite_forward(self._h, q1.data_ptr(), n1, x.data_ptr(), _dt(x), rows, ldx, y.data_ptr(),
                                           _dt(y), d, _stream(x)), "bfq_composite_forward")
        return y

    def composite_inverse(self, q1: torch.Tensor, y: torch.Tensor, out_dtype=None, out=None) -> torch.Tensor:
        n1 = self._q1(q1)
        d = n1 * self.n
        rows, ldy = _rows(y, d, self.device, what="y")
        x = out if out is not None else torch.empty((rows, d), dtype=out_dtype or y.dtype, device=y.device)
        if _rows(x, d, self.device, rows, "out")[1] != d:
            raise ValueError("out: rows must be contiguous")
        _check(lib().bfq_composite_inverse(self._h, q1.data_ptr(), n1, y.data_ptr(), _dt(y), rows, ldy, x.data_ptr(),
                                           _dt(x), d, _stream(y)), "bfq_composite_inverse")
        return x

    def composite_forward_quant(self, q1: torch.Tensor, x: torch.Tensor, bits: int, codes=None, scales=None):
        n1 = self._q1(q1)
        d = n1 * self.n
        rows, ldx = _rows(x, d, self.device, what="x")
        codes, scales = self._outputs(rows, d, bits, codes, scales)
        _check(lib().bfq_composite_forward_quant(self._h, q1.data_ptr(), n1, x.data_ptr(), _dt(x), rows, ldx, int(bits),
                                                 codes.data_ptr(), scales.data_ptr(), _stream(x)),
               "bfq_composite_forward_quant")
        return codes, scales

    def forward_quant_stats(self, x: torch.Tensor, bits: int):
        """-> (codes, scales, hist int64 [2^bits], rowstats fp32 [rows][2] = (sum y^2, sum y^4))."""
        rows, ldx = _rows(x, self.n, self.device, what="x")
        codes, scales = self._outputs(rows, self.n, bits, None, None)
        hist = torch.empty((1 << bits,), dtype=torch.int64, device=x.device)
        rowstats = torch.empty((rows, 2), dtype=torch.float32, device=x.device)
        _check(lib().bfq_forward_quant_stats(self._h, x.data_ptr(), _dt(x), rows, ldx, int(bits), codes.data_ptr(),
                                             scales.data_ptr(), hist.data_ptr(), rowstats.data_ptr(), _stream(x)),
               "bfq_forward_quant_stats")
        return codes, scales, hist, rowstats

    def hadamard(self, x: torch.Tensor, out_dtype=None, out: torch.Tensor | None = None) -> torch.Tensor:
        rows, ldx = _rows(x, self.n, self.device, what="x")
        y = out if out is not None else torch.empty((rows, self.n), dtype=out_dtype or x.dtype, device=x.device)
        _, ldy = _rows(y, self.n, self.device, rows, "out")
        _check(lib().bfq_hadamard(self._h, x.data_ptr(), _dt(x), rows, ldx, y.data_ptr(), _dt(y), ldy, _stream(x)),
               "bfq_hadamard")
        return y

    def hadamard_quant(self, x: torch.Tensor, bits: int, codes=None, scales=None):
        rows, ldx = _rows(x, self.n, self.device, what="x")
        codes, scales = self._outputs(rows, self.n, bits, codes, scales)
        _check(lib().bfq_hadamard_quant(self._h, x.data_ptr(), _dt(x), rows, ldx, int(bits), codes.data_ptr(),
                                        scales.data_ptr(), _stream(x)), "bfq_hadamard_quant")
        return codes, scales

    def inverse(self, y: torch.Tensor, out_dtype=None, out: torch.Tensor | None = None) -> torch.Tensor:
        rows, ldy = _rows(y, self.n, self.device, what="y")
        x = out if out is not None else torch.empty((rows, self.n), dtype=out_dtype or y.dtype, device=y.device)
        _, ldx = _rows(x, self.n, self.device, rows, "out")
        _check(lib().bfq_inverse(self._h, y.data_ptr(), _dt(y), rows, ldy, x.data_ptr(), _dt(x), ldx, _stream(y)),
               "bfq_inverse")
        return x

    def backward(self, x: torch.Tensor, g: torch.Tensor, dx_dtype=None, want_dx: bool = True, dx=None, dtheta=None):
        rows, ld = _rows(x, self.n, self.device, what="x")
        rows_g, ld_g = _rows(g, self.n, self.device, what="g")
        if rows_g != rows or ld_g != ld:
            raise ValueError("x and g must have the same shape and row stride")
        if want_dx and dx is None:
            dx = torch.empty_strided((rows, self.n), (ld, 1), dtype=dx_dtype or x.dtype, device=x.device)
        if want_dx and _rows(dx, self.n, self.device, rows, "dx")[1] != ld:
            raise ValueError("dx must have the row stride of x")
        if dtheta is None:
            dtheta = torch.empty((self.L, self.n // 2), dtype=torch.float32, device=x.device)
        _exact(dtheta, torch.float32, (self.L, self.n // 2), self.device, "dtheta")
        _check(lib().bfq_backward(self._h, x.data_ptr(), _dt(x), g.data_ptr(), _dt(g), rows, ld,
                                  dx.data_ptr() if want_dx else None, _dt(dx) if want_dx else BFQ_F32,
                                  dtheta.data_ptr(), _stream(x)), "bfq_backward")
        return (dx if want_dx else None), dtheta

    def forward_quant_host_workspace(self, dtype, bits: int, chunk_rows: int) -> int:
        """Bytes of device workspace for forward_quant_host in chunks of chunk_rows rows."""
        xt = BFQ_F32 if dtype == torch.float32 else BFQ_BF16
        return int(lib().bfq_forward_quant_host_workspace(self._h, xt, int(bits), int(chunk_rows)))

    def forward_quant_host(self, x_host: torch.Tensor, bits: int, codes_host: torch.Tensor, scales_host: torch.Tensor,
                           workspace: torch.Tensor):
        """bfq_forward_quant_host: rows, codes and scales in (pinned) host memory, a uint8 device workspace; enqueued on
        the current stream of the plan's device."""
        if x_host.is_cuda or codes_host.is_cuda or scales_host.is_cuda:
            raise ValueError("x_host, codes_host and scales_host must be host tensors")
        if x_host.dim() != 2 or x_host.shape[1] != self.n or x_host.stride(1) != 1:
            raise ValueError(f"x_host must be [rows][{self.n}] with unit inner stride")
        if x_host.dtype not in (torch.float32, torch.bfloat16):
            raise ValueError("x_host must be float32 or bfloat16")
        rows = x_host.shape[0]
        for t, dtype, shape, what in ((codes_host, torch.uint8, (rows, self.n * int(bits) // 8), "codes_host"),
                                      (scales_host, torch.float16, (rows,), "scales_host")):
            if t.dtype != dtype or tuple(t.shape) != shape or not t.is_contiguous():
                raise ValueError(f"{what}: expected a contiguous {dtype} host tensor of shape {shape}")
        if not workspace.is_cuda or workspace.device != self.device or workspace.dtype != torch.uint8 or not workspace.is_contiguous():
            raise ValueError("workspace must be a contiguous uint8 tensor on the plan's device")
        with torch.cuda.device(self.device):
            stream = torch.cuda.current_stream(self.device).cuda_stream
            _check(lib().bfq_forward_quant_host(self._h, x_host.data_ptr(), _dt(x_host), rows, x_host.stride(0), int(bits),
                                                codes_host.data_ptr(), scales_host.data_ptr(), workspace.data_ptr(),
                                                workspace.numel(), stream), "bfq_forward_quant_host")

    def fold_weights(self, W: torch.Tensor, bits: int, want_rotated: bool = False, rotated_dtype=None):
        m, ldw = _rows(W, self.n, self.device, what="W")
        codes, scales = self._outputs(m, self.n, bits, None, None)
        rot = torch.empty((m, self.n), dtype=rotated_dtype or W.dtype, device=W.device) if want_rotated else None
        _check(lib().bfq_fold_weights(self._h, W.data_ptr(), _dt(W), m, ldw, int(bits), codes.data_ptr(),
                                      scales.data_ptr(), rot.data_ptr() if rot is not None else None,
                                      _dt(rot) if rot is not None else BFQ_F32, _stream(W)), "bfq_fold_weights")
        return codes, scales, rot

    def dequant_gemm(self, a: GemmOperand, b: GemmOperand, alpha: float = 1.0, out: torch.Tensor | None = None):
        """C[i][j] = alpha * sum_k A(i, k) B(j, k) on the tensor cores, low-bit operands dequantized on the fly -> fp32."""
        if a.k != b.k:
            raise ValueError(f"operands disagree on K: {a.k} and {b.k}")
        for op, what in ((a, "A"), (b, "B")):
            _on(op.data, self.device, what)
        c = out if out is not None else torch.empty((a.rows, b.rows), dtype=torch.float32, device=self.device)
        _exact(c, torch.float32, (a.rows, b.rows), self.device, "out")
        _check(lib().bfq_dequant_gemm(self._h, a.rows, b.rows, a.k, float(alpha), a.data.data_ptr(), a.kind,
                                      int(a.transposed), a.ld, a.scales.data_ptr() if a.scales is not None else None,
                                      b.data.data_ptr(), b.kind, int(b.transposed), b.ld,
                                      b.scales.data_ptr() if b.scales is not None else None, c.data_ptr(), b.rows,
                                      _stream(c)), "bfq_dequant_gemm")
        return c

    def device_status(self) -> int:
        return int(lib().bfq_device_status(self._h))

    def stage_form(self) -> int:
        """bit 0 / bit 1: the forward / inverse tables of the tuned kernels use the three-shear fallback."""
        r = int(lib().bfq_stage_form(self._h))
        if r < 0:
            raise BfqError(r, "bfq_stage_form")
        return r

    def test_stuck_wait(self, enable: bool):
        _check(lib().bfq_test_stuck_wait(self._h, int(bool(enable))), "bfq_test_stuck_wait")

    def backward_partials(self) -> int:
        return int(lib().bfq_backward_partials(self._h))


def backward_noalloc(theta: torch.Tensor, x: torch.Tensor, g: torch.Tensor, dx: torch.Tensor | None,
                     dtheta: torch.Tensor):
    """bfq_backward_noalloc: the backward pass without a plan and without any device allocation by the
    library (for hosts that must not call cudaMalloc; row length at most 1024).  Every buffer,
    outputs included, is the caller's; pass dx=None to skip dL/dx.  Runs on x's device, which is
    made current for the call.  Calls share one fixed scratch array per GPU: do not overlap them."""
    if not isinstance(x, torch.Tensor) or x.dim() != 2 or not x.is_cuda:
        raise ValueError("x must be a [rows][n] CUDA tensor")
    n = x.shape[1]
    L = n.bit_length() - 1
    if n < 16 or (1 << L) != n:
        raise ValueError("n must be a power of two >= 16")
    rows, ld = _rows(x, n, x.device, what="x")
    rows_g, ld_g = _rows(g, n, x.device, what="g")
    if rows_g != rows or ld_g != ld:
        raise ValueError("x and g must have the same shape and row stride")
    if dx is not None and _rows(dx, n, x.device, rows, "dx") != (rows, ld):
        raise ValueError("dx must have the shape and row stride of x")
    _exact(theta, torch.float32, (L, n // 2), x.device, "theta")
    _exact(dtheta, torch.float32, (L, n // 2), x.device, "dtheta")
    with torch.cuda.device(x.device):
        _check(lib().bfq_backward_noalloc(n, theta.data_ptr(), x.data_ptr(), _dt(x), g.data_ptr(), _dt(g), rows, ld,
                                          dx.data_ptr() if dx is not None else None,
                                          _dt(dx) if dx is not None else BFQ_F32, dtheta.data_ptr(), _stream(x)),
               "bfq_backward_noalloc")
    return dx, dtheta


def measure_fma_rates(device=None):
    """bfq_measure_fma_rates on `device` (default: the current one): SM cycles per FMA instruction per scheduler for
    (packed, three register operands), (packed, two), (scalar, three), (scalar, two)."""
    out = (ctypes.c_float * 4)()
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    with torch.cuda.device(dev):
        _check(lib().bfq_measure_fma_rates(ctypes.cast(out, ctypes.c_void_p)), "bfq_measure_fma_rates")
    return {"packed_3reg": out[0], "packed_2reg": out[1], "scalar_3reg": out[2], "scalar_2reg": out[3]}


def measure_mma_rates(device=None):
    """bfq_measure_mma_rates on `device` (default: the current one): SM cycles per tcgen05.mma (bf16, M = 128, K = 16)
    for N = 16, 64, 128, 256."""
    out = (ctypes.c_float * 4)()
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    with torch.cuda.device(dev):
        _check(lib().bfq_measure_mma_rates(ctypes.cast(out, ctypes.c_void_p)), "bfq_measure_mma_rates")
    return {"n16": out[0], "n64": out[1], "n128": out[2], "n256": out[3]}
