"""Python binding of the B200 BCQ linear-layer library (``include/bcq.h``).

Argument marshalling only: every function forwards device pointers of torch tensors to the
C-ABI entry point of the same name and raises on a non-zero status.  torch is used for device
memory and streams, nothing else; there is no CPU or eager fallback -- if the CUDA library is
missing or cannot be loaded, the first call raises.
"""
from __future__ import annotations

import ctypes as C
import os

from . import synth  # noqa: F401  (seeded input generators; no BCQ arithmetic)

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libbcq_b200.so")

OK = 0
F32, BF16 = 0, 1
OP_QUANTIZE, OP_FWD, OP_DECODE, OP_BWD_X, OP_BWD_ALPHA, OP_DECODE_PACKED = 0, 1, 2, 3, 4, 5

# every symbol include/bcq.h declares
SYMBOLS = ("bcq_pitch_words", "bcq_bits_bytes", "bcq_num_groups", "bcq_alpha_count",
           "bcq_payload_bits", "bcq_workspace_bytes", "bcq_quantize", "bcq_dequantize",
           "bcq_linear_fwd", "bcq_linear_decode", "bcq_linear_bwd_x", "bcq_linear_bwd_alpha",
           "bcq_status_string", "bcq_last_cuda_error", "bcq_device_timeout_flag",
           "bcq_kernel_launches", "bcq_linear_decode_noalloc", "bcq_decode_pack_bytes",
           "bcq_decode_pack", "bcq_linear_decode_packed", "bcq_lr_linear_decay", "bcq_alpha_adamw",
           "bcq_alpha_pack", "bcq_alpha_unpack", "bcq_prepared_bytes", "bcq_prepare_planes",
           "bcq_linear_fwd_prepared", "bcq_linear_bwd_x_prepared", "bcq_check_device")


class BcqError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__("%s failed: status %d (%s), last CUDA error %d" % (
            what, status, status_string(status), lib().bcq_last_cuda_error()))


_lib = None


def lib() -> C.CDLL:
    """Loads libbcq_b200.so (built in-tree by ``build.build_library``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("CUDA library not built: %s is missing; run "
                               "paper_2210_03858_b200/build.py" % LIB_PATH)
        l = C.CDLL(LIB_PATH)
        i, sz, vp, u32, f32 = C.c_int, C.c_size_t, C.c_void_p, C.c_uint32, C.c_float
        l.bcq_pitch_words.restype = sz
        l.bcq_pitch_words.argtypes = [i]
        l.bcq_bits_bytes.restype = sz
        l.bcq_bits_bytes.argtypes = [i, i, i]
        l.bcq_num_groups.restype = sz
        l.bcq_num_groups.argtypes = [i, i]
        l.bcq_alpha_count.restype = sz
        l.bcq_alpha_count.argtypes = [i, i, i, i]
        l.bcq_payload_bits.restype = sz
        l.bcq_payload_bits.argtypes = [i, i, i, i]
        l.bcq_workspace_bytes.restype = sz
        l.bcq_workspace_bytes.argtypes = [i, i, i, i, i, i]
        l.bcq_quantize.restype = i
        l.bcq_quantize.argtypes = [i, i, i, i, vp, sz, i, vp, vp, vp, vp]
        l.bcq_dequantize.restype = i
        l.bcq_dequantize.argtypes = [i, i, i, i, vp, vp, vp, sz, vp]
        l.bcq_linear_fwd.restype = i
        l.bcq_linear_fwd.argtypes = [i, i, i, i, i, vp, sz, vp, vp, vp, vp, sz, i, vp, sz, vp]
        l.bcq_linear_decode.restype = i
        l.bcq_linear_decode.argtypes = l.bcq_linear_fwd.argtypes
        l.bcq_linear_decode_noalloc.restype = i
        l.bcq_linear_decode_noalloc.argtypes = [i, i, i, i, i, vp, sz, vp, vp, vp, vp, sz, i, vp]
        l.bcq_decode_pack_bytes.restype = sz
        l.bcq_decode_pack_bytes.argtypes = [i, i, i, i]
        l.bcq_decode_pack.restype = i
        l.bcq_decode_pack.argtypes = [i, i, i, i, vp, vp, vp, sz, vp]
        l.bcq_linear_decode_packed.restype = i
        l.bcq_linear_decode_packed.argtypes = [i, i, i, i, i, vp, sz, vp, vp, vp, sz, i, vp, sz, vp]
        l.bcq_linear_bwd_x.restype = i
        l.bcq_linear_bwd_x.argtypes = [i, i, i, i, i, vp, sz, vp, vp, vp, sz, i, vp, sz, vp]
        l.bcq_prepared_bytes.restype = sz
        l.bcq_prepared_bytes.argtypes = [i, i, i, i, i]
        l.bcq_prepare_planes.restype = i
        l.bcq_prepare_planes.argtypes = [i, i, i, i, i, vp, vp, sz, vp]
        l.bcq_linear_fwd_prepared.restype = i
        l.bcq_linear_fwd_prepared.argtypes = l.bcq_linear_fwd.argtypes
        l.bcq_linear_bwd_x_prepared.restype = i
        l.bcq_linear_bwd_x_prepared.argtypes = l.bcq_linear_bwd_x.argtypes
        ll = C.c_longlong
        l.bcq_lr_linear_decay.restype = f32
        l.bcq_lr_linear_decay.argtypes = [f32, ll, ll, ll]
        l.bcq_alpha_adamw.restype = i
        l.bcq_alpha_adamw.argtypes = [ll, i, vp, vp, vp, vp, vp, vp, vp, ll, f32, f32, f32, f32, f32, f32, vp]
        l.bcq_alpha_pack.restype = i
        l.bcq_alpha_pack.argtypes = [ll, i, vp, vp, vp, vp, vp]
        l.bcq_alpha_unpack.restype = i
        l.bcq_alpha_unpack.argtypes = [ll, i, vp, vp, vp, vp, vp]
        l.bcq_linear_bwd_alpha.restype = i
        l.bcq_linear_bwd_alpha.argtypes = [i, i, i, i, i, vp, sz, vp, sz, vp, u32, f32, i, vp, vp, sz, vp]
        l.bcq_status_string.restype = C.c_char_p
        l.bcq_status_string.argtypes = [i]
        l.bcq_last_cuda_error.restype = i
        l.bcq_last_cuda_error.argtypes = []
        l.bcq_kernel_launches.restype = C.c_ulonglong
        l.bcq_kernel_launches.argtypes = []
        l.bcq_check_device.restype = i
        l.bcq_check_device.argtypes = []
        l.bcq_device_timeout_flag.restype = i
        l.bcq_device_timeout_flag.argtypes = [C.POINTER(C.c_int), i]
        _lib = l
    return _lib


def status_string(status: int) -> str:
    return lib().bcq_status_string(status).decode()


# ---------------------------------------------------------------------------- sizes

def pitch_words(d_in: int) -> int:
    return lib().bcq_pitch_words(d_in)


def bits_bytes(d_out: int, d_in: int, q: int) -> int:
    return lib().bcq_bits_bytes(d_out, d_in, q)


def num_groups(d_in: int, g: int) -> int:
    return lib().bcq_num_groups(d_in, g)


def alpha_count(d_out: int, d_in: int, q: int, g: int) -> int:
    return lib().bcq_alpha_count(d_out, d_in, q, g)


def payload_bits(d_out: int, d_in: int, q: int, g: int) -> int:
    return lib().bcq_payload_bits(d_out, d_in, q, g)


def workspace_bytes(op: int, d_out: int, d_in: int, q: int, g: int, n: int = 0) -> int:
    return lib().bcq_workspace_bytes(op, d_out, d_in, q, g, n)


# ---------------------------------------------------------------------------- helpers

def _torch():
    import torch
    return torch


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(_torch().cuda.current_stream().cuda_stream)


def _check(status: int, what: str):
    if status != OK:
        raise BcqError(status, what)


def _ws(op, d_out, d_in, q, g, n, ws, device):
    need = workspace_bytes(op, d_out, d_in, q, g, n)
    if ws is None and need > 0:
        ws = _torch().empty(need, dtype=_torch().uint8, device=device)
    return ws, (0 if ws is None else ws.numel() * ws.element_size())


def _dtype_code(t):
    torch = _torch()
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError("output must be float32 or bfloat16")


# ---------------------------------------------------------------------------- calls

def quantize(W, q: int, g: int, alt_iters: int = 0, want_sq_err: bool = False):
    """bcq_quantize: W [d_out][d_in] fp32 (cuda) -> (bits uint32 [q][d_out][pitch] as int32
    tensor, alpha fp32 [q][d_out][G], sq_err fp64 [d_out][G] or None)."""
    torch = _torch()
    assert W.is_cuda and W.dtype == torch.float32 and W.dim() == 2 and W.stride(1) == 1
    d_out, d_in = W.shape
    G = max(1, num_groups(d_in, g))
    bits = torch.empty((q, d_out, pitch_words(d_in)), dtype=torch.int32, device=W.device)
    alpha = torch.empty((q, d_out, G), dtype=torch.float32, device=W.device)
    sq_err = torch.empty((d_out, G), dtype=torch.float64, device=W.device) if want_sq_err else None
    _check(lib().bcq_quantize(d_out, d_in, q, g, _ptr(W), W.stride(0), alt_iters, _ptr(bits),
                              _ptr(alpha), _ptr(sq_err), _stream()), "bcq_quantize")
    return bits, alpha, sq_err


def dequantize(bits, alpha, d_in: int, g: int):
    torch = _torch()
    q, d_out, _ = bits.shape
    W_hat = torch.empty((d_out, d_in), dtype=torch.float32, device=bits.device)
    _check(lib().bcq_dequantize(d_out, d_in, q, g, _ptr(bits), _ptr(alpha), _ptr(W_hat), d_in,
                                _stream()), "bcq_dequantize")
    return W_hat


class PreparedPlanes:
    """The frozen planes of one layer as written by bcq_prepare_planes for one operation."""

    def __init__(self, op, buf, q, d_out, d_in, g):
        self.op, self.buf, self.q, self.d_out, self.d_in, self.g = op, buf, q, d_out, d_in, g
        self.shape = (q, d_out, pitch_words(d_in))   # shape of the canonical planes it stands for

    def data_ptr(self):
        return self.buf.data_ptr()


def prepare_planes(op: int, bits, d_in: int, g: int) -> PreparedPlanes:
    """bcq_prepare_planes for op = OP_FWD or OP_BWD_X (q <= 4)."""
    torch = _torch()
    q, d_out, _ = bits.shape
    nbytes = lib().bcq_prepared_bytes(op, d_out, d_in, q, g)
    if nbytes == 0:
        raise BcqError(-4, "bcq_prepared_bytes")
    buf = torch.empty(nbytes, dtype=torch.uint8, device=bits.device)
    _check(lib().bcq_prepare_planes(op, d_out, d_in, q, g, _ptr(bits), _ptr(buf), nbytes, _stream()),
           "bcq_prepare_planes")
    return PreparedPlanes(op, buf, q, d_out, d_in, g)


def _fwd(fn, op, name, X, bits, alpha, d_in, g, bias, out, out_dtype, ws):
    torch = _torch()
    assert X.is_cuda and X.dtype == torch.bfloat16 and X.dim() == 2 and X.stride(1) == 1
    if isinstance(bits, PreparedPlanes):
        assert bits.op == OP_FWD and op == OP_FWD
        fn, name = lib().bcq_linear_fwd_prepared, "bcq_linear_fwd_prepared"
    q, d_out, _ = bits.shape
    n = X.shape[0]
    if out is None:
        out = torch.empty((n, d_out), dtype=out_dtype or torch.float32, device=X.device)
    ws, ws_bytes = _ws(op, d_out, d_in, q, g, n, ws, X.device)
    _check(fn(d_out, d_in, q, g, n, _ptr(X), X.stride(0), _ptr(bits), _ptr(alpha), _ptr(bias),
              _ptr(out), out.stride(0), _dtype_code(out), _ptr(ws), ws_bytes, _stream()), name)
    return out


def linear_fwd(X, bits, alpha, d_in: int, g: int, bias=None, out=None, out_dtype=None, ws=None):
    """bcq_linear_fwd: X bf16 [n][d_in] -> Y [n][d_out] (Eq. 2)."""
    return _fwd(lib().bcq_linear_fwd, OP_FWD, "bcq_linear_fwd", X, bits, alpha, d_in, g, bias, out,
                out_dtype, ws)


def linear_decode(X, bits, alpha, d_in: int, g: int, bias=None, out=None, out_dtype=None, ws=None):
    """bcq_linear_decode: same as linear_fwd for 1..16 tokens."""
    return _fwd(lib().bcq_linear_decode, OP_DECODE, "bcq_linear_decode", X, bits, alpha, d_in, g,
                bias, out, out_dtype, ws)


def decode_pack(bits, alpha, d_in: int, g: int):
    """bcq_decode_pack: the frozen (bits, alpha) of a layer rewritten for bcq_linear_decode_packed
    (q <= 4).  Returns the pack as a uint8 tensor."""
    torch = _torch()
    q, d_out, _ = bits.shape
    nbytes = lib().bcq_decode_pack_bytes(d_out, d_in, q, g)
    if nbytes == 0:
        raise BcqError(-4, "bcq_decode_pack_bytes")
    pack = torch.empty(nbytes, dtype=torch.uint8, device=bits.device)
    _check(lib().bcq_decode_pack(d_out, d_in, q, g, _ptr(bits), _ptr(alpha), _ptr(pack), nbytes,
                                 _stream()), "bcq_decode_pack")
    return pack


def linear_decode_packed(X, pack, d_out: int, d_in: int, q: int, g: int, bias=None, out=None,
                         out_dtype=None, ws=None):
    """bcq_linear_decode_packed: X bf16 [n][d_in], n <= 16 -> Y [n][d_out] from a pack."""
    torch = _torch()
    assert X.is_cuda and X.dtype == torch.bfloat16 and X.dim() == 2 and X.stride(1) == 1
    n = X.shape[0]
    if out is None:
        out = torch.empty((n, d_out), dtype=out_dtype or torch.float32, device=X.device)
    ws, ws_bytes = _ws(OP_DECODE_PACKED, d_out, d_in, q, g, n, ws, X.device)
    _check(lib().bcq_linear_decode_packed(d_out, d_in, q, g, n, _ptr(X), X.stride(0), _ptr(pack),
                                          _ptr(bias), _ptr(out), out.stride(0), _dtype_code(out),
                                          _ptr(ws), ws_bytes, _stream()), "bcq_linear_decode_packed")
    return out


NOALLOC_SCRATCH_BYTES = 2 << 20


def linear_decode_noalloc(X, bits, alpha, d_in: int, g: int, bias=None, out=None):
    """bcq_linear_decode_noalloc: decode for callers that cannot provide scratch memory -- the
    library call itself allocates nothing (its partial sums go to a fixed 2 MiB array inside the
    library).  ``out`` must be given by such a caller; it is created here only as a convenience
    for tests."""
    torch = _torch()
    assert X.is_cuda and X.dtype == torch.bfloat16 and X.dim() == 2 and X.stride(1) == 1
    q, d_out, _ = bits.shape
    n = X.shape[0]
    if out is None:
        out = torch.empty((n, d_out), dtype=torch.float32, device=X.device)
    _check(lib().bcq_linear_decode_noalloc(d_out, d_in, q, g, n, _ptr(X), X.stride(0), _ptr(bits),
                                           _ptr(alpha), _ptr(bias), _ptr(out), out.stride(0),
                                           _dtype_code(out), _stream()), "bcq_linear_decode_noalloc")
    return out


def linear_bwd_x(dY, bits, alpha, d_in: int, g: int, out=None, out_dtype=None, ws=None):
    """bcq_linear_bwd_x: dY bf16 [n][d_out] -> dX [n][d_in] (Eq. 3)."""
    torch = _torch()
    assert dY.is_cuda and dY.dtype == torch.bfloat16 and dY.dim() == 2 and dY.stride(1) == 1
    q, d_out, _ = bits.shape
    n = dY.shape[0]
    if out is None:
        out = torch.empty((n, d_in), dtype=out_dtype or torch.float32, device=dY.device)
    ws, ws_bytes = _ws(OP_BWD_X, d_out, d_in, q, g, n, ws, dY.device)
    fn, name = lib().bcq_linear_bwd_x, "bcq_linear_bwd_x"
    if isinstance(bits, PreparedPlanes):
        assert bits.op == OP_BWD_X
        fn, name = lib().bcq_linear_bwd_x_prepared, "bcq_linear_bwd_x_prepared"
    _check(fn(d_out, d_in, q, g, n, _ptr(dY), dY.stride(0), _ptr(bits), _ptr(alpha), _ptr(out),
              out.stride(0), _dtype_code(out), _ptr(ws), ws_bytes, _stream()), name)
    return out


def linear_bwd_alpha(dY, X, bits, d_in: int, g: int, plane_mask=None, scale: float = 1.0,
                     accumulate: bool = False, out=None, ws=None):
    """bcq_linear_bwd_alpha: dalpha fp32 [q][d_out][G] (Eq. 4); planes outside plane_mask are
    left as they are in ``out`` (zeros if ``out`` is created here)."""
    torch = _torch()
    assert dY.is_cuda and dY.dtype == torch.bfloat16 and X.dtype == torch.bfloat16
    q, d_out, _ = bits.shape
    n = X.shape[0]
    G = num_groups(d_in, g)
    if plane_mask is None:
        plane_mask = (1 << q) - 1
    if out is None:
        out = torch.zeros((q, d_out, G), dtype=torch.float32, device=X.device)
    ws, ws_bytes = _ws(OP_BWD_ALPHA, d_out, d_in, q, g, n, ws, X.device)
    _check(lib().bcq_linear_bwd_alpha(d_out, d_in, q, g, n, _ptr(dY), dY.stride(0), _ptr(X),
                                      X.stride(0), _ptr(bits), plane_mask, scale,
                                      1 if accumulate else 0, _ptr(out), _ptr(ws), ws_bytes,
                                      _stream()), "bcq_linear_bwd_alpha")
    return out


# ---------------------------------------------------------------------------- the update

def lr_linear_decay(lr0: float, step: int, warmup_steps: int, total_steps: int) -> float:
    return float(lib().bcq_lr_linear_decay(lr0, step, warmup_steps, total_steps))


class Segments:
    """Device-side description of the trained elements of the flat scale arrays: (begin, count)
    runs -- e.g. AlphaBucket.plane_segments(1) for "alpha_1 of every linear" -- with an optional
    gradient scale per run (1/g_L of Eq. 4)."""

    def __init__(self, runs, device, scales=None):
        torch = _torch()
        self.nseg = len(runs)
        prefix = [0]
        for _, c in runs:
            prefix.append(prefix[-1] + int(c))
        self.count = prefix[-1]
        self.begin = torch.tensor([int(b) for b, _ in runs], dtype=torch.int64, device=device)
        self.prefix = torch.tensor(prefix, dtype=torch.int64, device=device)
        self.scale = None if scales is None else torch.tensor(list(scales), dtype=torch.float32, device=device)


def alpha_adamw(alpha, dalpha, m, v, step: int, lr: float, beta1: float = 0.9, beta2: float = 0.999,
                eps: float = 1e-8, weight_decay: float = 0.0, grad_scale: float = 1.0, segments: Segments = None):
    """bcq_alpha_adamw on flat fp32 tensors (in place).  Without segments the whole arrays are updated."""
    torch = _torch()
    for t in (alpha, dalpha, m, v):
        assert t.is_cuda and t.dtype == torch.float32 and t.is_contiguous() and t.numel() == alpha.numel()
    if segments is None:
        count, nseg, b, pfx, sc = alpha.numel(), 0, None, None, None
    else:
        count, nseg, b, pfx, sc = segments.count, segments.nseg, segments.begin, segments.prefix, segments.scale
    _check(lib().bcq_alpha_adamw(count, nseg, _ptr(b), _ptr(pfx), _ptr(sc), _ptr(alpha), _ptr(dalpha), _ptr(m),
                                 _ptr(v), step, lr, beta1, beta2, eps, weight_decay, grad_scale, _stream()),
           "bcq_alpha_adamw")


def alpha_pack(alpha_flat, segments: Segments):
    """bcq_alpha_pack: the trained scales as one compact fp32 tensor (the per-task checkpoint)."""
    torch = _torch()
    out = torch.empty(segments.count, dtype=torch.float32, device=alpha_flat.device)
    _check(lib().bcq_alpha_pack(segments.count, segments.nseg, _ptr(segments.begin), _ptr(segments.prefix),
                                _ptr(alpha_flat), _ptr(out), _stream()), "bcq_alpha_pack")
    return out


def alpha_unpack(packed, alpha_flat, segments: Segments):
    """bcq_alpha_unpack: writes a checkpoint's scales back into the flat array."""
    assert packed.numel() == segments.count
    _check(lib().bcq_alpha_unpack(segments.count, segments.nseg, _ptr(segments.begin), _ptr(segments.prefix),
                                  _ptr(packed), _ptr(alpha_flat), _stream()), "bcq_alpha_unpack")


def kernel_launches() -> int:
    return int(lib().bcq_kernel_launches())


def check_device() -> None:
    """Synchronises; raises BcqError (status BCQ_ERR_DEVICE_TIMEOUT) if a kernel gave up on a wait."""
    _check(lib().bcq_check_device(), "bcq_check_device")


def device_timeout_flag(reset: bool = False) -> int:
    flag = C.c_int(0)
    _check(lib().bcq_device_timeout_flag(C.byref(flag), 1 if reset else 0), "bcq_device_timeout_flag")
    return flag.value
