"""numpy front end of the fp64 CPU oracle in ``bcq_ref.c``.

Test infrastructure only: the tests, the smoke check and the CPU-baseline leg of the
benchmark may import this; the CUDA package never does.  Arguments and results are numpy
arrays in host memory.  Each function forwards to the C routine of the same name, which
cites the passage of the paper it follows.

bf16 tensors (X, dY) are passed as ``uint16`` arrays holding the bf16 bit patterns.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bcq_ref.c")
_LIB = os.path.join(_HERE, "libbcq_ref.so")
MAX_Q = 8


def build(force: bool = False) -> str:
    """Compile ``bcq_ref.c`` with gcc (no -ffast-math, no FMA contraction) if needed."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-o", _LIB + ".tmp", _SRC, "-lm"]
        subprocess.run(cmd, check=True, cwd=_HERE)
        os.replace(_LIB + ".tmp", _LIB)
    return _LIB


_lib = None


def _l():
    global _lib
    if _lib is None:
        lib = C.CDLL(build())
        i64, i32, u32, dbl, vp = C.c_int64, C.c_int, C.c_uint32, C.c_double, C.c_void_p
        lib.bcq_ref_pitch_words.restype = i64
        lib.bcq_ref_pitch_words.argtypes = [i64]
        lib.bcq_ref_num_groups.restype = i64
        lib.bcq_ref_num_groups.argtypes = [i64, i64]
        lib.bcq_ref_payload_bits.restype = i64
        lib.bcq_ref_payload_bits.argtypes = [i64] * 4
        lib.bcq_ref_pack.restype = None
        lib.bcq_ref_pack.argtypes = [i64, i64, i32, vp, vp]
        lib.bcq_ref_unpack.restype = None
        lib.bcq_ref_unpack.argtypes = [i64, i64, i32, vp, vp]
        lib.bcq_ref_quantize.restype = i32
        lib.bcq_ref_quantize.argtypes = [i64, i64, i32, i64, vp, i64, i32, vp, vp, vp, vp]
        lib.bcq_ref_dequantize.restype = None
        lib.bcq_ref_dequantize.argtypes = [i64, i64, i32, i64, vp, vp, vp, i64]
        lib.bcq_ref_fwd.restype = None
        lib.bcq_ref_fwd.argtypes = [i64, i64, i32, i64, i64, vp, i64, vp, vp, vp, vp, i64]
        lib.bcq_ref_fwd_at.restype = None
        lib.bcq_ref_fwd_at.argtypes = [i64, i64, i32, i64, vp, i64, vp, vp, vp, i64, vp, vp, vp]
        lib.bcq_ref_bwd_x.restype = None
        lib.bcq_ref_bwd_x.argtypes = [i64, i64, i32, i64, i64, vp, i64, vp, vp, vp, i64]
        lib.bcq_ref_bwd_x_at.restype = None
        lib.bcq_ref_bwd_x_at.argtypes = [i64, i64, i32, i64, vp, i64, vp, vp, i64, vp, vp, vp]
        lib.bcq_ref_bwd_alpha.restype = None
        lib.bcq_ref_bwd_alpha.argtypes = [i64, i64, i32, i64, i64, vp, i64, vp, i64, vp, u32, dbl, vp]
        lib.bcq_ref_bwd_alpha_at.restype = None
        lib.bcq_ref_bwd_alpha_at.argtypes = [i64, i64, i32, i64, i64, vp, i64, vp, i64, vp, dbl,
                                             i64, vp, vp, vp, vp]
        lib.bcq_ref_lr_linear.restype = dbl
        lib.bcq_ref_lr_linear.argtypes = [dbl, i64, i64, i64]
        lib.bcq_ref_adamw.restype = None
        lib.bcq_ref_adamw.argtypes = [i64, vp, vp, vp, vp, i64, dbl, dbl, dbl, dbl, dbl, dbl]
        lib.bcq_ref_num_threads.restype = i32
        lib.bcq_ref_num_threads.argtypes = []
        _lib = lib
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _chk(a, dtype, ndim):
    a = np.ascontiguousarray(a, dtype=dtype)
    assert a.ndim == ndim, (a.shape, ndim)
    return a


def num_threads() -> int:
    return int(_l().bcq_ref_num_threads())


def pitch_words(d_in: int) -> int:
    return int(_l().bcq_ref_pitch_words(d_in))


def num_groups(d_in: int, g: int) -> int:
    return int(_l().bcq_ref_num_groups(d_in, g))


def payload_bytes(d_out: int, d_in: int, q: int, g: int) -> float:
    """Quantized size of one layer as Table 1 counts it (bits + fp32 scales), in bytes."""
    return int(_l().bcq_ref_payload_bits(d_out, d_in, q, g)) / 8.0


def pack(signs: np.ndarray) -> np.ndarray:
    """signs[q][d_out][d_in] in {-1,+1} -> bits[q][d_out][pitch] uint32."""
    signs = _chk(signs, np.int8, 3)
    q, d_out, d_in = signs.shape
    bits = np.empty((q, d_out, pitch_words(d_in)), dtype=np.uint32)
    _l().bcq_ref_pack(d_out, d_in, q, _p(signs), _p(bits))
    return bits


def unpack(bits: np.ndarray, d_in: int) -> np.ndarray:
    bits = _chk(bits, np.uint32, 3)
    q, d_out, pitch = bits.shape
    assert pitch == pitch_words(d_in)
    signs = np.empty((q, d_out, d_in), dtype=np.int8)
    _l().bcq_ref_unpack(d_out, d_in, q, _p(bits), _p(signs))
    return signs


def quantize(W: np.ndarray, q: int, g: int, alt_iters: int = 0):
    """Greedy (alt_iters = 0) or greedy + alternating BCQ of W[d_out][d_in] fp32.

    Returns (bits, alpha[q][d_out][G] fp32, sq_err[d_out][G] fp64, margin[d_out][G] fp64).
    """
    W = _chk(W, np.float32, 2)
    d_out, d_in = W.shape
    if not (1 <= q <= MAX_Q and 1 <= g <= d_in and alt_iters >= 0):
        raise ValueError("bcq_ref_quantize: invalid arguments")
    G = num_groups(d_in, g)
    bits = np.empty((q, d_out, pitch_words(d_in)), dtype=np.uint32)
    alpha = np.empty((q, d_out, G), dtype=np.float32)
    sq_err = np.empty((d_out, G), dtype=np.float64)
    margin = np.empty((d_out, G), dtype=np.float64)
    rc = _l().bcq_ref_quantize(d_out, d_in, q, g, _p(W), d_in, alt_iters, _p(bits), _p(alpha),
                               _p(sq_err), _p(margin))
    if rc != 0:
        raise ValueError("bcq_ref_quantize: invalid arguments")
    return bits, alpha, sq_err, margin


def _shape(bits, alpha, d_in, g):
    bits = _chk(bits, np.uint32, 3)
    alpha = _chk(alpha, np.float32, 3)
    q, d_out, pitch = bits.shape
    assert pitch == pitch_words(d_in), (pitch, d_in)
    assert alpha.shape == (q, d_out, num_groups(d_in, g)), (alpha.shape, q, d_out, d_in, g)
    return bits, alpha, q, d_out


def dequantize(bits, alpha, d_in: int, g: int) -> np.ndarray:
    bits, alpha, q, d_out = _shape(bits, alpha, d_in, g)
    W_hat = np.empty((d_out, d_in), dtype=np.float64)
    _l().bcq_ref_dequantize(d_out, d_in, q, g, _p(bits), _p(alpha), _p(W_hat), d_in)
    return W_hat


def fwd(X_bf16, bits, alpha, d_in: int, g: int, bias=None) -> np.ndarray:
    X = _chk(X_bf16, np.uint16, 2)
    bits, alpha, q, d_out = _shape(bits, alpha, d_in, g)
    n = X.shape[0]
    assert X.shape[1] == d_in
    if bias is not None:
        bias = _chk(bias, np.float32, 1)
        assert bias.shape[0] == d_out
    Y = np.empty((n, d_out), dtype=np.float64)
    _l().bcq_ref_fwd(d_out, d_in, q, g, n, _p(X), d_in, _p(bits), _p(alpha), _p(bias), _p(Y), d_out)
    return Y


def fwd_at(X_bf16, bits, alpha, d_in: int, g: int, t_idx, j_idx, bias=None) -> np.ndarray:
    X = _chk(X_bf16, np.uint16, 2)
    bits, alpha, q, d_out = _shape(bits, alpha, d_in, g)
    t_idx = _chk(t_idx, np.int64, 1)
    j_idx = _chk(j_idx, np.int64, 1)
    if bias is not None:
        bias = _chk(bias, np.float32, 1)
    out = np.empty(t_idx.shape[0], dtype=np.float64)
    _l().bcq_ref_fwd_at(d_out, d_in, q, g, _p(X), d_in, _p(bits), _p(alpha), _p(bias),
                        t_idx.shape[0], _p(t_idx), _p(j_idx), _p(out))
    return out


def bwd_x(dY_bf16, bits, alpha, d_in: int, g: int) -> np.ndarray:
    dY = _chk(dY_bf16, np.uint16, 2)
    bits, alpha, q, d_out = _shape(bits, alpha, d_in, g)
    n = dY.shape[0]
    assert dY.shape[1] == d_out
    dX = np.empty((n, d_in), dtype=np.float64)
    _l().bcq_ref_bwd_x(d_out, d_in, q, g, n, _p(dY), d_out, _p(bits), _p(alpha), _p(dX), d_in)
    return dX


def bwd_x_at(dY_bf16, bits, alpha, d_in: int, g: int, t_idx, k_idx) -> np.ndarray:
    dY = _chk(dY_bf16, np.uint16, 2)
    bits, alpha, q, d_out = _shape(bits, alpha, d_in, g)
    t_idx = _chk(t_idx, np.int64, 1)
    k_idx = _chk(k_idx, np.int64, 1)
    out = np.empty(t_idx.shape[0], dtype=np.float64)
    _l().bcq_ref_bwd_x_at(d_out, d_in, q, g, _p(dY), d_out, _p(bits), _p(alpha),
                          t_idx.shape[0], _p(t_idx), _p(k_idx), _p(out))
    return out


def bwd_alpha(dY_bf16, X_bf16, bits, d_in: int, g: int, plane_mask=None, scale: float = 1.0,
              out=None) -> np.ndarray:
    dY = _chk(dY_bf16, np.uint16, 2)
    X = _chk(X_bf16, np.uint16, 2)
    bits = _chk(bits, np.uint32, 3)
    q, d_out, _ = bits.shape
    n = X.shape[0]
    assert dY.shape == (n, d_out) and X.shape[1] == d_in
    G = num_groups(d_in, g)
    if plane_mask is None:
        plane_mask = (1 << q) - 1
    if out is None:
        out = np.zeros((q, d_out, G), dtype=np.float64)
    assert out.dtype == np.float64 and out.shape == (q, d_out, G) and out.flags.c_contiguous
    _l().bcq_ref_bwd_alpha(d_out, d_in, q, g, n, _p(dY), d_out, _p(X), d_in, _p(bits),
                           plane_mask, scale, _p(out))
    return out


def bwd_alpha_at(dY_bf16, X_bf16, bits, d_in: int, g: int, i_idx, j_idx, c_idx,
                 scale: float = 1.0) -> np.ndarray:
    dY = _chk(dY_bf16, np.uint16, 2)
    X = _chk(X_bf16, np.uint16, 2)
    bits = _chk(bits, np.uint32, 3)
    q, d_out, _ = bits.shape
    n = X.shape[0]
    i_idx = _chk(i_idx, np.int64, 1)
    j_idx = _chk(j_idx, np.int64, 1)
    c_idx = _chk(c_idx, np.int64, 1)
    out = np.empty(i_idx.shape[0], dtype=np.float64)
    _l().bcq_ref_bwd_alpha_at(d_out, d_in, q, g, n, _p(dY), d_out, _p(X), d_in, _p(bits), scale,
                              i_idx.shape[0], _p(i_idx), _p(j_idx), _p(c_idx), _p(out))
    return out


def lr_linear(lr0: float, step: int, warmup: int, total: int) -> float:
    """Learning rate of 0-based step `step`: linear warm-up over `warmup` steps, then linear decay
    to zero at step `total`."""
    return float(_l().bcq_ref_lr_linear(lr0, step, warmup, total))


def adamw(alpha, grad, m, v, step: int, lr: float, beta1: float = 0.9, beta2: float = 0.999,
          eps: float = 1e-8, wd: float = 0.0, grad_scale: float = 1.0):
    """One AdamW step (1-based `step`) in place on the fp32 arrays alpha, m, v; grad is fp32."""
    for a in (alpha, m, v):
        assert a.dtype == np.float32 and a.flags.c_contiguous
    grad = np.ascontiguousarray(grad, dtype=np.float32)
    assert alpha.size == grad.size == m.size == v.size
    _l().bcq_ref_adamw(alpha.size, _p(alpha), _p(grad), _p(m), _p(v), step, lr, beta1, beta2, eps, wd,
                       grad_scale)
    return alpha, m, v
