"""Thin binding over libwcc.so (the C ABI of include/wcc.h): argument marshalling only.

Every step runs in the library's CUDA kernels; torch is used for device memory and the current stream.
There is no fallback: if the library is missing, or a call returns an error code, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libwcc.so")

F32, BF16 = 0, 1
_STATUS = {0: "ok", 1: "null pointer", 2: "bad shape", 3: "k out of range", 4: "bad bits", 5: "bad dtype",
           6: "misaligned pointer", 7: "workspace too small", 8: "CUDA error", 9: "device wait timed out",
           10: "non-finite input"}

EXPORTS = ("wcc_staged_workspace_bytes", "wcc_forward_staged", "wcc_workspace_bytes", "wcc_select_workspace_bytes", "wcc_haar_fwd", "wcc_haar_inv", "wcc_select_topk",
           "wcc_forward", "wcc_forward_debug", "wcc_kpad", "wcc_last_status", "wcc_status_str",
           "wcc_profile_enable", "wcc_profile_read", "wcc_kernel_launches", "wcc_select_topk_static",
           "wcc_debug_set_wait_limit", "wcc_debug_wait_selftest", "wcc_forward_ex", "wcc_chain_workspace_bytes",
           "wcc_chain_forward", "wcc_select_bitmap_workspace_bytes", "wcc_select_topk_bitmap",
           "wcc_padded_workspace_bytes", "wcc_forward_padded", "wcc_dwconv_haar_fwd", "wcc_block_workspace_bytes",
           "wcc_block_forward", "wcc_dwt_fwd", "wcc_dwt_inv", "wcc_wavelet_workspace_bytes", "wcc_forward_wavelet")
STATIC_SCRATCH_BYTES = 512 * 1024
STAGES = ("haar_fwd_norms", "select_topk", "weight_quant", "gather_quant", "contract", "scatter_inv")   # wcc_forward_staged
FUSED_STAGES = ("clear", "haar_norms", "select_topk", "fused_pass2")                                      # wcc_forward


class WccError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__("%s: %s (status %d)" % (where, _STATUS.get(code, "?"), code))
        self.code = code


class Taps(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("coef", "nrm2", "idx", "Xq", "Xb", "scale_a", "Wq", "scale_w", "acc")]


class Options(C.Structure):
    _fields_ = [("alpha", C.c_float), ("weight_bits", C.c_int), ("relu", C.c_int), ("residual", C.c_void_p),
                ("Wq", C.c_void_p), ("scale_w", C.c_void_p)]


class ChainLayer(C.Structure):
    _fields_ = [("Wt", C.c_void_p), ("Cin", C.c_int), ("Cout", C.c_int), ("alpha", C.c_float), ("relu", C.c_int)]


_lib = None


def lib() -> C.CDLL:
    """The loaded library; raises if it has not been built (``python -m paper_2205_12268_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError("libwcc.so is not built: run `python -m paper_2205_12268_b200.build` "
                                    "(needs nvcc; there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        i, vp, sz = C.c_int, C.c_void_p, C.c_size_t
        L.wcc_workspace_bytes.restype = sz
        L.wcc_workspace_bytes.argtypes = [i] * 9
        L.wcc_staged_workspace_bytes.restype = sz
        L.wcc_staged_workspace_bytes.argtypes = [i] * 9
        L.wcc_select_workspace_bytes.restype = sz
        L.wcc_select_workspace_bytes.argtypes = [i, i]
        L.wcc_kpad.restype = i
        L.wcc_kpad.argtypes = [i, i]
        L.wcc_haar_fwd.restype = i
        L.wcc_haar_fwd.argtypes = [vp, i, i, i, i, i, i, vp, vp, vp]
        L.wcc_haar_inv.restype = i
        L.wcc_haar_inv.argtypes = [vp, i, i, i, i, i, i, vp, vp]
        L.wcc_select_topk.restype = i
        L.wcc_select_topk.argtypes = [vp, i, i, i, vp, vp, vp, sz, vp]
        L.wcc_select_topk_static.restype = i
        L.wcc_select_topk_static.argtypes = [vp, i, i, i, vp, vp, vp]
        fwd = [vp, vp, i, i, i, i, i, i, i, i, vp, i, vp, sz, vp]
        L.wcc_forward.restype = i
        L.wcc_forward.argtypes = fwd
        L.wcc_forward_debug.restype = i
        L.wcc_forward_debug.argtypes = fwd + [C.POINTER(Taps)]
        L.wcc_forward_staged.restype = i
        L.wcc_forward_staged.argtypes = fwd + [C.POINTER(Taps)]
        L.wcc_forward_ex.restype = i
        L.wcc_forward_ex.argtypes = fwd + [C.POINTER(Options), C.POINTER(Taps)]
        L.wcc_select_bitmap_workspace_bytes.restype = sz
        L.wcc_select_bitmap_workspace_bytes.argtypes = [i, i, i]
        L.wcc_select_topk_bitmap.restype = i
        L.wcc_select_topk_bitmap.argtypes = [vp, i, i, i, vp, vp, vp, sz, vp]
        L.wcc_padded_workspace_bytes.restype = sz
        L.wcc_padded_workspace_bytes.argtypes = [i] * 9
        L.wcc_forward_padded.restype = i
        L.wcc_forward_padded.argtypes = fwd
        L.wcc_dwconv_haar_fwd.restype = i
        L.wcc_dwconv_haar_fwd.argtypes = [vp, vp, i, i, i, i, i, i, vp, vp, vp]
        L.wcc_block_workspace_bytes.restype = sz
        L.wcc_block_workspace_bytes.argtypes = [i] * 9
        L.wcc_block_forward.restype = i
        L.wcc_block_forward.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, i, i, vp, i, vp, sz, vp]
        fp = C.POINTER(C.c_float)
        L.wcc_dwt_fwd.restype = i
        L.wcc_dwt_fwd.argtypes = [vp, i, i, i, i, i, i, fp, fp, i, vp, vp, vp, sz, vp]
        L.wcc_dwt_inv.restype = i
        L.wcc_dwt_inv.argtypes = [vp, i, i, i, i, i, i, fp, fp, i, vp, vp, sz, vp]
        L.wcc_wavelet_workspace_bytes.restype = sz
        L.wcc_wavelet_workspace_bytes.argtypes = [i] * 9
        L.wcc_forward_wavelet.restype = i
        L.wcc_forward_wavelet.argtypes = [vp, vp, i, i, i, i, i, i, i, i, fp, fp, fp, fp, i, vp, i, vp, sz, vp, C.POINTER(Taps)]
        L.wcc_chain_workspace_bytes.restype = sz
        L.wcc_chain_workspace_bytes.argtypes = [C.POINTER(ChainLayer), i, i, i, i, i, i, i, i]
        L.wcc_chain_forward.restype = i
        L.wcc_chain_forward.argtypes = [vp, C.POINTER(ChainLayer), i, i, i, i, i, i, i, vp, i, vp, sz, vp]
        L.wcc_last_status.restype = i
        L.wcc_last_status.argtypes = [vp]
        L.wcc_profile_enable.restype = i
        L.wcc_profile_enable.argtypes = [i]
        L.wcc_profile_read.restype = i
        L.wcc_profile_read.argtypes = [C.POINTER(C.c_float)]
        L.wcc_kernel_launches.restype = C.c_ulonglong
        L.wcc_kernel_launches.argtypes = []
        L.wcc_debug_set_wait_limit.restype = i
        L.wcc_debug_set_wait_limit.argtypes = [C.c_uint]
        L.wcc_debug_wait_selftest.restype = i
        L.wcc_debug_wait_selftest.argtypes = [vp]
        L.wcc_status_str.restype = C.c_char_p
        L.wcc_status_str.argtypes = [i]
        _lib = L
    return _lib


def _check(code: int, where: str):
    if code != 0:
        raise WccError(code, where)


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError("activations must be float32 or bfloat16, got %s" % t.dtype)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t):
    return None if t is None else t.data_ptr()


def _dev(t: torch.Tensor, name: str):
    if not (t.is_cuda and t.is_contiguous()):
        raise ValueError("%s must be a contiguous CUDA tensor" % name)


def workspace_bytes(N, Cin, Cout, H, W, levels, k, bits, dt) -> int:
    return int(lib().wcc_workspace_bytes(N, Cin, Cout, H, W, levels, k, bits, dt))


def kpad(Cin: int, bits: int) -> int:
    return int(lib().wcc_kpad(Cin, bits))


def haar_fwd(x: torch.Tensor, levels: int, want_norms: bool = True):
    """x [N][C][H][W] -> (coef fp32 [N][C][H][W] quadrant layout, nrm2 fp32 [N][H*W] or None)."""
    _dev(x, "x")
    N, Cc, H, W = x.shape
    coef = torch.empty((N, Cc, H, W), dtype=torch.float32, device=x.device)
    nrm2 = torch.empty((N, H * W), dtype=torch.float32, device=x.device) if want_norms else None
    _check(lib().wcc_haar_fwd(x.data_ptr(), N, Cc, H, W, levels, _dt(x), coef.data_ptr(), _ptr(nrm2), _stream()),
           "wcc_haar_fwd")
    return coef, nrm2


def dwconv_haar_fwd(u: torch.Tensor, Wdw: torch.Tensor, levels: int):
    """Depthwise 3x3 convolution (Wdw fp32 [C][3][3]) fused with the forward transform -> (coef, nrm2) as ``haar_fwd``."""
    _dev(u, "u")
    _dev(Wdw, "Wdw")
    N, Cc, H, W = u.shape
    if Wdw.dtype != torch.float32 or tuple(Wdw.shape) != (Cc, 3, 3):
        raise ValueError("Wdw must be float32 [C][3][3]")
    coef = torch.empty((N, Cc, H, W), dtype=torch.float32, device=u.device)
    nrm2 = torch.empty((N, H * W), dtype=torch.float32, device=u.device)
    _check(lib().wcc_dwconv_haar_fwd(u.data_ptr(), Wdw.data_ptr(), N, Cc, H, W, levels, _dt(u), coef.data_ptr(),
                                     nrm2.data_ptr(), _stream()), "wcc_dwconv_haar_fwd")
    return coef, nrm2


def _taps(f):
    import numpy as np
    a = np.ascontiguousarray(f, dtype=np.float32)
    return a, a.ctypes.data_as(C.POINTER(C.c_float))


def dwt_fwd(x: torch.Tensor, levels: int, dec_lo, dec_hi):
    """Generic wavelet transform (host filter arrays, see wcc.h) -> (coef fp32, nrm2 fp32 [N][P])."""
    _dev(x, "x")
    N, Cc, H, W = x.shape
    lo, plo = _taps(dec_lo)
    hi, phi = _taps(dec_hi)
    coef = torch.empty((N, Cc, H, W), dtype=torch.float32, device=x.device)
    nrm2 = torch.empty((N, H * W), dtype=torch.float32, device=x.device)
    ws = torch.empty((N * Cc * H * W * 4,), dtype=torch.uint8, device=x.device)
    _check(lib().wcc_dwt_fwd(x.data_ptr(), N, Cc, H, W, levels, _dt(x), plo, phi, lo.size, coef.data_ptr(), nrm2.data_ptr(),
                             ws.data_ptr(), ws.numel(), _stream()), "wcc_dwt_fwd")
    return coef, nrm2


def dwt_inv(coef: torch.Tensor, levels: int, rec_lo, rec_hi, dtype: torch.dtype = torch.float32) -> torch.Tensor:
    _dev(coef, "coef")
    N, Cc, H, W = coef.shape
    lo, plo = _taps(rec_lo)
    hi, phi = _taps(rec_hi)
    out = torch.empty((N, Cc, H, W), dtype=dtype, device=coef.device)
    ws = torch.empty((2 * (N * Cc * H * W * 4 + 256),), dtype=torch.uint8, device=coef.device)
    _check(lib().wcc_dwt_inv(coef.data_ptr(), N, Cc, H, W, levels, _dt(out), plo, phi, lo.size, out.data_ptr(),
                             ws.data_ptr(), ws.numel(), _stream()), "wcc_dwt_inv")
    return out


def forward_wavelet(x: torch.Tensor, Wt: torch.Tensor, levels: int, k: int, bits: int, bank, taps: bool = False):
    """The layer with another wavelet: ``bank`` = (dec_lo, dec_hi, rec_lo, rec_hi) host arrays of equal even length."""
    _dev(x, "x")
    _dev(Wt, "Wt")
    N, Cin, H, W = x.shape
    Cout = Wt.shape[0]
    f = [_taps(b) for b in bank]
    nbytes = int(lib().wcc_wavelet_workspace_bytes(N, Cin, Cout, H, W, levels, k, bits, _dt(x)))
    if nbytes == 0:
        raise WccError(2, "wcc_wavelet_workspace_bytes")
    ws = torch.empty((nbytes,), dtype=torch.uint8, device=x.device)
    y = torch.empty((N, Cout, H, W), dtype=x.dtype, device=x.device)
    t, s = {}, None
    if taps:
        P, M, kp = H * W, N * k, kpad(Cin, bits)
        t = dict(coef=torch.empty((N, Cin, P), dtype=torch.float32, device=x.device),
                 nrm2=torch.empty((N, P), dtype=torch.float32, device=x.device),
                 idx=torch.empty((N, k), dtype=torch.int32, device=x.device),
                 acc=torch.empty((M, Cout), dtype=torch.int32, device=x.device))
        if bits >= 2:
            t["Xq"] = torch.empty((M, kp), dtype=torch.int8, device=x.device)
        s = Taps(**{name: _ptr(t.get(name)) for name, _ in Taps._fields_})
    _check(lib().wcc_forward_wavelet(x.data_ptr(), Wt.data_ptr(), N, Cin, Cout, H, W, levels, k, bits, f[0][1], f[1][1], f[2][1],
                                     f[3][1], f[0][0].size, y.data_ptr(), _dt(x), ws.data_ptr(), nbytes, _stream(),
                                     C.byref(s) if s is not None else None), "wcc_forward_wavelet")
    return (y, t) if taps else y


class Block:
    """The inverted residual block y = x + WCC(W3, dw3x3(Wdw, WCC(W1, x))) (wcc_block_forward); the workspace, which
    also holds the expanded map, is allocated once, here."""

    def __init__(self, x: torch.Tensor, W1: torch.Tensor, Wdw: torch.Tensor, W3: torch.Tensor, levels: int, k: int, bits: int = 8):
        _dev(x, "x")
        for t, name in ((W1, "W1"), (Wdw, "Wdw"), (W3, "W3")):
            _dev(t, name)
            if t.dtype != torch.float32:
                raise TypeError("%s must be float32" % name)
        self.N, self.C, self.H, self.W = x.shape
        self.E = W1.shape[0]
        if tuple(W1.shape) != (self.E, self.C) or tuple(Wdw.shape) != (self.E, 3, 3) or tuple(W3.shape) != (self.C, self.E):
            raise ValueError("W1 [E][C], Wdw [E][3][3], W3 [C][E] expected")
        self.W1, self.Wdw, self.W3, self.levels, self.k, self.bits, self.dt = W1, Wdw, W3, levels, k, bits, _dt(x)
        n = int(lib().wcc_block_workspace_bytes(self.N, self.C, self.E, self.H, self.W, levels, k, bits, self.dt))
        if n == 0:
            raise WccError(2, "wcc_block_workspace_bytes")
        self.ws = Workspace(n, x.device)

    def __call__(self, x: torch.Tensor, y: torch.Tensor | None = None) -> torch.Tensor:
        _dev(x, "x")
        if y is None:
            y = torch.empty_like(x)
        _check(lib().wcc_block_forward(x.data_ptr(), self.W1.data_ptr(), self.Wdw.data_ptr(), self.W3.data_ptr(), self.N,
                                       self.C, self.E, self.H, self.W, self.levels, self.k, self.bits, y.data_ptr(), self.dt,
                                       self.ws.buf.data_ptr(), self.ws.nbytes, _stream()), "wcc_block_forward")
        return y


def haar_inv(coef: torch.Tensor, levels: int, dtype: torch.dtype = torch.float32) -> torch.Tensor:
    _dev(coef, "coef")
    if coef.dtype != torch.float32:
        raise TypeError("coef must be float32")
    N, Cc, H, W = coef.shape
    out = torch.empty((N, Cc, H, W), dtype=dtype, device=coef.device)
    _check(lib().wcc_haar_inv(coef.data_ptr(), N, Cc, H, W, levels, _dt(out), out.data_ptr(), _stream()), "wcc_haar_inv")
    return out


def select_topk(nrm2: torch.Tensor, k: int):
    """nrm2 fp32 [N][P] -> (idx int32 [N][k] ascending, tau fp32 [N])."""
    _dev(nrm2, "nrm2")
    if nrm2.dtype != torch.float32:
        raise TypeError("nrm2 must be float32")
    N, P = nrm2.shape
    idx = torch.empty((N, max(k, 1)), dtype=torch.int32, device=nrm2.device)
    tau = torch.empty((N,), dtype=torch.float32, device=nrm2.device)
    nbytes = int(lib().wcc_select_workspace_bytes(N, P))
    ws = torch.empty((max(nbytes, 256),), dtype=torch.uint8, device=nrm2.device)
    _check(lib().wcc_select_topk(nrm2.data_ptr(), N, P, k, idx.data_ptr(), tau.data_ptr(), ws.data_ptr(), nbytes, _stream()),
           "wcc_select_topk")
    return idx, tau


def select_topk_bitmap(nrm2: torch.Tensor, k: int):
    """nrm2 fp32 [N][P] -> (bitmap int32 [N][ceil(P/32)] with bit p % 32 of word p // 32 set for kept p, tau fp32 [N])."""
    _dev(nrm2, "nrm2")
    N, P = nrm2.shape
    bitmap = torch.empty((N, (P + 31) // 32), dtype=torch.int32, device=nrm2.device)
    tau = torch.empty((N,), dtype=torch.float32, device=nrm2.device)
    nbytes = int(lib().wcc_select_bitmap_workspace_bytes(N, P, k))
    ws = torch.empty((max(nbytes, 256),), dtype=torch.uint8, device=nrm2.device)
    _check(lib().wcc_select_topk_bitmap(nrm2.data_ptr(), N, P, k, bitmap.data_ptr(), tau.data_ptr(), ws.data_ptr(), nbytes,
                                        _stream()), "wcc_select_topk_bitmap")
    return bitmap, tau


def forward_padded(x: torch.Tensor, Wt: torch.Tensor, levels: int, k: int, bits: int = 8) -> torch.Tensor:
    """The layer on a map whose sides need not be multiples of 2^levels (zero padding, see wcc_forward_padded);
    k counts positions of the padded map."""
    _dev(x, "x")
    _dev(Wt, "Wt")
    N, Cin, H, W = x.shape
    Cout = Wt.shape[0]
    nbytes = int(lib().wcc_padded_workspace_bytes(N, Cin, Cout, H, W, levels, k, bits, _dt(x)))
    if nbytes == 0:
        raise WccError(2, "wcc_padded_workspace_bytes")
    ws = torch.empty((nbytes,), dtype=torch.uint8, device=x.device)
    y = torch.empty((N, Cout, H, W), dtype=x.dtype, device=x.device)
    _check(lib().wcc_forward_padded(x.data_ptr(), Wt.data_ptr(), N, Cin, Cout, H, W, levels, k, bits, y.data_ptr(), _dt(x),
                                    ws.data_ptr(), nbytes, _stream()), "wcc_forward_padded")
    return y


def select_topk_static(nrm2: torch.Tensor, k: int, idx: torch.Tensor, tau: torch.Tensor):
    """``select_topk`` for callers that cannot provide scratch memory: the library's built-in scratch array is used
    and nothing is allocated, here or in the library (the caller passes the output tensors).  Raises ``WccError``
    with code 7 when N and P need more than ``STATIC_SCRATCH_BYTES``.  Calls on one device share the scratch, so
    they must not overlap on the GPU."""
    _dev(nrm2, "nrm2")
    N, P = nrm2.shape
    _check(lib().wcc_select_topk_static(nrm2.data_ptr(), N, P, k, idx.data_ptr(), tau.data_ptr(), _stream()),
           "wcc_select_topk_static")
    return idx, tau


class Workspace:
    """Caller-owned scratch for ``forward``; reuse it across calls of the same (or smaller) problem."""

    def __init__(self, nbytes: int, device):
        self.nbytes = int(nbytes)
        self.buf = torch.empty((max(self.nbytes, 256),), dtype=torch.uint8, device=device)

    @classmethod
    def for_problem(cls, x: torch.Tensor, Cout: int, levels: int, k: int, bits: int, staged: bool = False):
        N, Cin, H, W = x.shape
        fn = lib().wcc_staged_workspace_bytes if staged else lib().wcc_workspace_bytes
        n = int(fn(N, Cin, Cout, H, W, levels, k, bits, _dt(x)))
        if n == 0:
            raise WccError(2, "wcc_workspace_bytes")
        return cls(n, x.device)


def forward(x: torch.Tensor, Wt: torch.Tensor | None, levels: int, k: int, bits: int = 8, y: torch.Tensor | None = None,
            ws: Workspace | None = None, taps: bool = False, staged: bool = False, alpha: float = 0.0, wbits: int = 0,
            relu: bool = False, residual: torch.Tensor | None = None, Wq: torch.Tensor | None = None,
            scale_w: torch.Tensor | None = None):
    """The WCC layer.  Returns y, or (y, dict of intermediate tensors) when ``taps`` is set (True: all of them; or an
    iterable of names out of coef, nrm2, idx, acc, Xq / Xb, scale_a, Wq, scale_w).
    ``staged`` selects wcc_forward_staged (every intermediate in memory) instead of the fused wcc_forward.
    ``alpha``, ``wbits``, ``relu``, ``residual``, ``Wq`` + ``scale_w``: the options of wcc_forward_ex (see wcc.h);
    with pre-quantized weights ``Wt`` may be None."""
    _dev(x, "x")
    N, Cin, H, W = x.shape
    use_ex = bool(alpha > 0.0 or wbits or relu or residual is not None or Wq is not None)
    if Wq is not None:
        _dev(Wq, "Wq")
        if scale_w is not None:
            _dev(scale_w, "scale_w")
        Cout = Wq.shape[0]
    else:
        _dev(Wt, "Wt")
        if Wt.dtype != torch.float32:
            raise TypeError("Wt must be float32")
        Cout = Wt.shape[0]
        if Wt.shape[1] != Cin:
            raise ValueError("Wt must be [Cout][Cin]")
    if use_ex and staged:
        raise ValueError("options are only available on the fused path")
    if residual is not None:
        _dev(residual, "residual")
        if residual.shape != (N, Cout, H, W) or residual.dtype != x.dtype:
            raise ValueError("residual must have the output's shape and type")
    if y is None:
        y = torch.empty((N, Cout, H, W), dtype=x.dtype, device=x.device)
    if ws is None:
        ws = Workspace.for_problem(x, Cout, levels, k, bits, staged=staged)
    args = (x.data_ptr(), _ptr(Wt), N, Cin, Cout, H, W, levels, k, bits, y.data_ptr(), _dt(x),
            ws.buf.data_ptr(), ws.nbytes, _stream())
    opt = Options(float(alpha), int(wbits), int(bool(relu)), _ptr(residual), _ptr(Wq), _ptr(scale_w)) if use_ex else None
    if not taps:
        if staged:
            _check(lib().wcc_forward_staged(*args, None), "wcc_forward_staged")
        elif use_ex:
            _check(lib().wcc_forward_ex(*args, C.byref(opt), None), "wcc_forward_ex")
        else:
            _check(lib().wcc_forward(*args), "wcc_forward")
        return y
    P, M, kp = H * W, N * k, kpad(Cin, bits)
    dev = x.device
    t = dict(coef=torch.empty((N, Cin, P), dtype=torch.float32, device=dev),
             nrm2=torch.empty((N, P), dtype=torch.float32, device=dev),
             idx=torch.empty((N, k), dtype=torch.int32, device=dev),
             acc=torch.empty((M, Cout), dtype=torch.int32, device=dev))
    if bits >= 2:
        t.update(Xq=torch.empty((M, kp), dtype=torch.int8, device=dev), scale_a=torch.empty((1,), dtype=torch.float32, device=dev),
                 Wq=torch.empty((Cout, kp), dtype=torch.int8, device=dev), scale_w=torch.empty((Cout,), dtype=torch.float32, device=dev))
    else:
        t.update(Xb=torch.empty((M, kp), dtype=torch.bfloat16, device=dev))
    if taps is not True:
        t = {name: v for name, v in t.items() if name in set(taps)}
    for name in ("Xq", "Xb", "acc"):          # every row is a kept position and gets written; start from zeros anyway
        if name in t:
            t[name].zero_()
    s = Taps(**{name: _ptr(t.get(name)) for name, _ in Taps._fields_})
    if staged:
        _check(lib().wcc_forward_staged(*args, C.byref(s)), "wcc_forward_staged")
    elif use_ex:
        _check(lib().wcc_forward_ex(*args, C.byref(opt), C.byref(s)), "wcc_forward_ex")
    else:
        _check(lib().wcc_forward_debug(*args, C.byref(s)), "wcc_forward_debug")
    return y, t


class Chain:
    """A chain of pointwise WCC layers (wcc_chain_forward): ``weights[i]`` is layer i's fp32 [Cout][Cin] device tensor;
    a ReLU follows every layer but (unless ``relu_last``) the last; ``alphas[i]`` > 0 fixes layer i's clipping parameter.
    The workspace (intermediate maps included) is allocated once, here."""

    def __init__(self, x: torch.Tensor, weights, levels: int, k: int, bits: int = 8, relu_last: bool = False, alphas=None):
        _dev(x, "x")
        self.N, cin, self.H, self.W = x.shape
        self.levels, self.k, self.bits, self.dt = levels, k, bits, _dt(x)
        self.weights = list(weights)
        n = len(self.weights)
        self.layers = (ChainLayer * n)()
        for i, Wt in enumerate(self.weights):
            _dev(Wt, "weights[%d]" % i)
            if Wt.dtype != torch.float32 or Wt.shape[1] != cin:
                raise ValueError("weights[%d] must be float32 [Cout][%d]" % (i, cin))
            self.layers[i] = ChainLayer(Wt.data_ptr(), cin, Wt.shape[0], 0.0 if alphas is None else float(alphas[i]),
                                        int(relu_last or i + 1 < n))
            cin = Wt.shape[0]
        self.Cout = cin
        nbytes = int(lib().wcc_chain_workspace_bytes(self.layers, n, self.N, self.H, self.W, levels, k, bits, self.dt))
        if nbytes == 0:
            raise WccError(2, "wcc_chain_workspace_bytes")
        self.ws = Workspace(nbytes, x.device)

    def __call__(self, x: torch.Tensor, y: torch.Tensor | None = None) -> torch.Tensor:
        _dev(x, "x")
        if y is None:
            y = torch.empty((self.N, self.Cout, self.H, self.W), dtype=x.dtype, device=x.device)
        _check(lib().wcc_chain_forward(x.data_ptr(), self.layers, len(self.weights), self.N, self.H, self.W, self.levels,
                                       self.k, self.bits, y.data_ptr(), self.dt, self.ws.buf.data_ptr(), self.ws.nbytes,
                                       _stream()), "wcc_chain_forward")
        return y


def last_status() -> int:
    """Synchronises the current stream and returns (and clears) the device status word."""
    return int(lib().wcc_last_status(_stream()))


def debug_set_wait_limit(polls: int):
    """Polls every device-side wait makes before it gives up (0 restores the default)."""
    _check(lib().wcc_debug_set_wait_limit(int(polls)), "wcc_debug_set_wait_limit")


def debug_wait_selftest():
    """Enqueues one warp that waits on a barrier nobody arrives on (it gives up after the wait limit)."""
    _check(lib().wcc_debug_wait_selftest(_stream()), "wcc_debug_wait_selftest")


def profile_enable(on: bool):
    _check(lib().wcc_profile_enable(int(on)), "wcc_profile_enable")


def profile_read():
    """Milliseconds of each stage (see ``STAGES``) of the last ``forward`` issued with profiling on."""
    ms = (C.c_float * len(STAGES))()
    _check(lib().wcc_profile_read(ms), "wcc_profile_read")
    return [float(v) for v in ms]


def kernel_launches() -> int:
    return int(lib().wcc_kernel_launches())
