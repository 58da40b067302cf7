"""ctypes front end of the CPU oracle (``wcc_oracle.c``) -- TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the bench's CPU-baseline leg import this
package.  It knows nothing about the CUDA library and the CUDA library knows
nothing about it.  ``build()`` compiles the C file with gcc; importing the
package compiles it on first use.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = [os.path.join(_HERE, "wcc_oracle.c"), os.path.join(_HERE, "wcc_oracle_impl.h")]
_LIB = os.environ.get("WCC_ORACLE_LIB") or os.path.join(_HERE, "liboracle.so")   # the override serves the mutation test only
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle (contraction off: every written operation rounds once)."""
    if os.environ.get("WCC_ORACLE_LIB"):
        return _LIB                                  # a library built by someone else (the mutation test): use as it is
    stale = force or not os.path.exists(_LIB) or any(os.path.getmtime(s) > os.path.getmtime(_LIB) for s in _SRC)
    if stale:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        cmd = ["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-shared", "-fPIC",
               "-Wall", "-o", tmp, _SRC[0], "-lm"]
        subprocess.check_call(cmd)
        os.replace(tmp, _LIB)
    return _LIB


def _L():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_quantize.restype = C.c_float
        _lib.orc_quantize_alpha.restype = C.c_float
    return _lib


def _p(a, ty):
    return None if a is None else a.ctypes.data_as(C.POINTER(ty))


def _real(dtype):
    dtype = np.dtype(dtype)
    if dtype == np.float32:
        return "f32", C.c_float
    if dtype == np.float64:
        return "f64", C.c_double
    raise TypeError(dtype)


def num_threads() -> int:
    return int(_L().orc_num_threads())


def haar_fwd(x: np.ndarray, levels: int) -> np.ndarray:
    """x [N][C][H][W] (float32 or float64) -> coefficients in the quadrant layout."""
    x = np.ascontiguousarray(x)
    suf, ty = _real(x.dtype)
    N, Cc, H, W = x.shape
    out = np.empty_like(x)
    rc = getattr(_L(), "orc_haar_fwd_" + suf)(_p(x, ty), N, Cc, H, W, levels, _p(out, ty))
    if rc:
        raise ValueError("orc_haar_fwd rc=%d" % rc)
    return out


def haar_inv(coef: np.ndarray, levels: int) -> np.ndarray:
    coef = np.ascontiguousarray(coef)
    suf, ty = _real(coef.dtype)
    N, Cc, H, W = coef.shape
    out = np.empty_like(coef)
    rc = getattr(_L(), "orc_haar_inv_" + suf)(_p(coef, ty), N, Cc, H, W, levels, _p(out, ty))
    if rc:
        raise ValueError("orc_haar_inv rc=%d" % rc)
    return out


def concat_order(plane: np.ndarray, levels: int) -> np.ndarray:
    """One transformed plane [H][W] re-read as the concatenated sub-band vector of Eq. 6."""
    plane = np.ascontiguousarray(plane)
    suf, ty = _real(plane.dtype)
    H, W = plane.shape
    out = np.empty(H * W, dtype=plane.dtype)
    getattr(_L(), "orc_concat_order_" + suf)(_p(plane, ty), H, W, levels, _p(out, ty))
    return out


def norms(coef: np.ndarray) -> np.ndarray:
    """coef [N][C][H][W] -> squared channel norm per position, [N][H*W]."""
    coef = np.ascontiguousarray(coef)
    suf, ty = _real(coef.dtype)
    N, Cc, H, W = coef.shape
    out = np.empty((N, H * W), dtype=coef.dtype)
    getattr(_L(), "orc_norms_" + suf)(_p(coef, ty), N, Cc, C.c_long(H * W), _p(out, ty))
    return out


def select_topk(nrm2: np.ndarray, k: int):
    """nrm2 [N][P] -> (idx int32 [N][k] ascending, tau [N])."""
    nrm2 = np.ascontiguousarray(nrm2)
    suf, ty = _real(nrm2.dtype)
    N, P = nrm2.shape
    idx = np.empty((N, k), dtype=np.int32)
    tau = np.empty(N, dtype=nrm2.dtype)
    rc = getattr(_L(), "orc_select_topk_" + suf)(_p(nrm2, ty), N, C.c_long(P), k, _p(idx, C.c_int32), _p(tau, ty))
    if rc:
        raise ValueError("orc_select_topk rc=%d" % rc)
    return idx, tau


def quantize(x: np.ndarray, bits: int = 8):
    """Per-tensor signed symmetric quantizer -> (int8 codes, scale)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    q = np.empty(x.shape, dtype=np.int8)
    s = _L().orc_quantize(_p(x, C.c_float), C.c_long(x.size), bits, _p(q, C.c_int8))
    return q, np.float32(s)


def quantize_weights(Wt: np.ndarray, bits: int = 8):
    """Per-output-channel quantizer on Wt [Cout][Cin] -> (int8 [Cout][Cin], scale_w [Cout])."""
    Wt = np.ascontiguousarray(Wt, dtype=np.float32)
    Cout, Cin = Wt.shape
    q = np.empty((Cout, Cin), dtype=np.int8)
    s = np.empty(Cout, dtype=np.float32)
    _L().orc_quantize_weights(_p(Wt, C.c_float), Cout, Cin, bits, _p(q, C.c_int8), _p(s, C.c_float))
    return q, s


def round_bf16(a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    out = np.empty_like(a)
    _L().orc_round_bf16(_p(a, C.c_float), C.c_long(a.size), _p(out, C.c_float))
    return out


def quantize_alpha(x: np.ndarray, alpha: float, bits: int = 8):
    """The same quantizer with a given clipping parameter (values beyond +-alpha clip) -> (int8 codes, scale)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    q = np.empty(x.shape, dtype=np.int8)
    s = _L().orc_quantize_alpha(_p(x, C.c_float), C.c_long(x.size), bits, C.c_float(alpha), _p(q, C.c_int8))
    return q, np.float32(s)


def forward(x: np.ndarray, Wt: np.ndarray, levels: int, k: int, bits: int, out_bf16: bool = False,
            idx_in: np.ndarray | None = None, taps: bool = False, wbits: int | None = None, alpha: float = 0.0,
            residual: np.ndarray | None = None, relu: bool = False):
    """The WCC layer in fp32.  Returns y, or (y, dict of taps) when ``taps`` is set.
    Options: ``wbits`` bits of the weight codes (default: ``bits``), ``alpha`` > 0 a given clipping parameter of the
    activation quantizer (default: the largest kept magnitude), ``residual`` a map added to the output, ``relu``."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    Wt = np.ascontiguousarray(Wt, dtype=np.float32)
    N, Cin, H, W = x.shape
    Cout = Wt.shape[0]
    assert Wt.shape[1] == Cin
    P = H * W
    y = np.empty((N, Cout, H, W), dtype=np.float32)
    t = {}
    if taps:
        t = dict(coef=np.empty((N, Cin, H, W), np.float32), nrm2=np.empty((N, P), np.float32),
                 idx=np.empty((N, k), np.int32))
        if bits > 0:
            t.update(Xq=np.empty((N, k, Cin), np.int8), scale_a=np.empty(1, np.float32),
                     Wq=np.empty((Cout, Cin), np.int8), scale_w=np.empty(Cout, np.float32),
                     acc=np.empty((N, k, Cout), np.int32))
    if idx_in is not None:
        idx_in = np.ascontiguousarray(idx_in, dtype=np.int32)
        assert idx_in.shape == (N, k)
    if residual is not None:
        residual = np.ascontiguousarray(residual, dtype=np.float32)
        assert residual.shape == y.shape
    rc = _L().orc_forward_ex_f32(
        _p(x, C.c_float), _p(Wt, C.c_float), N, Cin, Cout, H, W, levels, k, bits, bits if wbits is None else wbits,
        C.c_float(alpha), _p(residual, C.c_float), int(relu), int(out_bf16),
        _p(idx_in, C.c_int32), _p(y, C.c_float),
        _p(t.get("coef"), C.c_float), _p(t.get("nrm2"), C.c_float), _p(t.get("idx"), C.c_int32),
        _p(t.get("Xq"), C.c_int8), _p(t.get("scale_a"), C.c_float), _p(t.get("Wq"), C.c_int8),
        _p(t.get("scale_w"), C.c_float), _p(t.get("acc"), C.c_int32))
    if rc:
        raise ValueError("orc_forward_ex_f32 rc=%d" % rc)
    return (y, t) if taps else y


def chain(x: np.ndarray, weights, levels: int, k: int, bits: int = 8, out_bf16: bool = False, relu_last: bool = False,
          alphas=None):
    """A chain of pointwise WCC layers with a ReLU after every layer but (unless ``relu_last``) the last: layer i maps
    the previous layer's output with ``weights[i]`` ([Cout_i][Cin_i]).  ``alphas[i]`` > 0 gives layer i a fixed
    clipping parameter.  Nothing but a loop over ``forward``.  Returns the list of the layers' outputs."""
    outs = []
    cur = np.ascontiguousarray(x, dtype=np.float32)
    for i, Wt in enumerate(weights):
        last = i == len(weights) - 1
        cur = forward(cur, Wt, levels, k, bits, out_bf16=out_bf16, relu=(relu_last or not last),
                      alpha=0.0 if alphas is None else float(alphas[i]))
        outs.append(cur)
    return outs


def bitmap_of(idx: np.ndarray, P: int) -> np.ndarray:
    """Index lists [N][k] -> bitmaps uint32 [N][ceil(P/32)]: bit p % 32 of word p // 32 set for every kept p
    (the kept set in the other of the two forms Sec. 4 names)."""
    N = idx.shape[0]
    words = (P + 31) // 32
    out = np.zeros((N, words), dtype=np.uint32)
    for n in range(N):
        for p in idx[n]:
            out[n, p >> 5] |= np.uint32(1) << np.uint32(p & 31)
    return out


def forward_padded(x: np.ndarray, Wt: np.ndarray, levels: int, k: int, bits: int, out_bf16: bool = False):
    """The layer on a map whose sides are no multiples of 2^levels: zero padding at the bottom and on the right up to
    the next multiples, the layer on the padded map (k counts padded positions), cropping."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    N, Cin, H, W = x.shape
    unit = 1 << levels
    Hp, Wp = -(-H // unit) * unit, -(-W // unit) * unit
    xp = np.zeros((N, Cin, Hp, Wp), dtype=np.float32)
    xp[:, :, :H, :W] = x
    return np.ascontiguousarray(forward(xp, Wt, levels, k, bits, out_bf16=out_bf16)[:, :, :H, :W])


def dwconv3x3(x: np.ndarray, w: np.ndarray) -> np.ndarray:
    """Depthwise 3x3 convolution, stride 1, zero padding 1, no bias: x [N][C][H][W], w [C][3][3] -> [N][C][H][W] (fp32)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    w = np.ascontiguousarray(w, dtype=np.float32)
    N, Cc, H, W = x.shape
    assert w.shape == (Cc, 3, 3)
    y = np.empty_like(x)
    _L().orc_dwconv3x3_f32(_p(x, C.c_float), _p(w, C.c_float), N, Cc, H, W, _p(y, C.c_float))
    return y


def block(x: np.ndarray, W1: np.ndarray, Wdw: np.ndarray, W3: np.ndarray, levels: int, k: int, bits: int = 8,
          out_bf16: bool = False, taps: bool = False):
    """The inverted residual block of Eq. 13 with both pointwise convolutions as WCC layers and no non-linearities:
    y = x + WCC(W3, dw3x3(Wdw, WCC(W1, x))).  The expanded map u = WCC(W1, x) is rounded to the activation type like any
    layer output; the depthwise convolution feeds the second layer's transform directly in fp32 (the two are one fused
    step), and the skip connection is added after the second layer's inverse transform."""
    u = forward(x, W1, levels, k, bits, out_bf16=out_bf16)
    v = dwconv3x3(u, Wdw)
    y = forward(v, W3, levels, k, bits, out_bf16=out_bf16, residual=np.ascontiguousarray(x, dtype=np.float32))
    return (y, dict(u=u, v=v)) if taps else y


def dwt(x: np.ndarray, levels: int, lo, hi, inverse: bool = False) -> np.ndarray:
    """Multi-level 2-D wavelet transform of every plane with a two-channel filter bank (periodic extension, quadrant
    layout): forward with the decomposition filters ``lo, hi``, or (``inverse``) the synthesis with the reconstruction
    filters.  x float32 or float64 [N][C][H][W]; the taps are taken in x's precision."""
    x = np.ascontiguousarray(x)
    suf, ty = _real(x.dtype)
    lo = np.ascontiguousarray(lo, dtype=x.dtype)
    hi = np.ascontiguousarray(hi, dtype=x.dtype)
    assert lo.shape == hi.shape and lo.ndim == 1
    N, Cc, H, W = x.shape
    out = np.empty_like(x)
    rc = getattr(_L(), "orc_dwt_" + suf)(_p(x, ty), N, Cc, H, W, levels, _p(lo, ty), _p(hi, ty), lo.size, int(inverse), _p(out, ty))
    if rc:
        raise ValueError("orc_dwt rc=%d" % rc)
    return out


def forward_wavelet(x: np.ndarray, Wt: np.ndarray, levels: int, k: int, bits: int, dec_lo, dec_hi, rec_lo, rec_hi,
                    out_bf16: bool = False, taps: bool = False):
    """The WCC layer (Alg. 1) with another wavelet in place of Haar: the same steps, the transform and its inverse
    swapped for the given filter bank.  The steps are composed here from the oracle's own parts."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    Wt = np.ascontiguousarray(Wt, dtype=np.float32)
    N, Cin, H, W = x.shape
    Cout, P = Wt.shape[0], H * W
    coef = dwt(x, levels, dec_lo, dec_hi)
    nrm2 = norms(coef)
    idx, _ = select_topk(nrm2, k)
    cols = np.stack([coef[n].reshape(Cin, P)[:, idx[n]].T for n in range(N)])            # [N][k][Cin]
    t = dict(coef=coef.reshape(N, Cin, P), nrm2=nrm2, idx=idx)
    if bits > 0:
        Xq, scale_a = quantize(cols, bits)
        Wq, scale_w = quantize_weights(Wt, bits)
        acc = np.einsum("oc,nkc->nko", Wq.astype(np.int64), Xq.astype(np.int64)).astype(np.int32)
        Yc = acc.astype(np.float32) * (np.float32(scale_a) * scale_w)[None, None, :]
        t.update(Xq=Xq, scale_a=np.array([scale_a], np.float32), Wq=Wq, scale_w=scale_w, acc=acc)
    else:
        Yc = np.einsum("oc,nkc->nko", Wt.astype(np.float64), cols.astype(np.float64)).astype(np.float32)
    Ywt = np.zeros((N, Cout, P), dtype=np.float32)
    for n in range(N):
        Ywt[n][:, idx[n]] = Yc[n].T
    y = dwt(Ywt.reshape(N, Cout, H, W), levels, rec_lo, rec_hi, inverse=True)
    if out_bf16:
        y = round_bf16(y)
    return (y, t) if taps else y


def forward_f64(x: np.ndarray, Wt: np.ndarray, levels: int, k: int, idx_in: np.ndarray | None = None,
                taps: bool = False):
    """The unquantized layer entirely in double (invariant tests)."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    Wt = np.ascontiguousarray(Wt, dtype=np.float64)
    N, Cin, H, W = x.shape
    Cout = Wt.shape[0]
    y = np.empty((N, Cout, H, W), dtype=np.float64)
    nrm2 = np.empty((N, H * W), np.float64) if taps else None
    idx = np.empty((N, k), np.int32) if taps else None
    if idx_in is not None:
        idx_in = np.ascontiguousarray(idx_in, dtype=np.int32)
    rc = _L().orc_forward_f64(_p(x, C.c_double), _p(Wt, C.c_double), N, Cin, Cout, H, W, levels, k,
                              _p(idx_in, C.c_int32), _p(y, C.c_double), _p(nrm2, C.c_double), _p(idx, C.c_int32))
    if rc:
        raise ValueError("orc_forward_f64 rc=%d" % rc)
    return (y, dict(nrm2=nrm2, idx=idx)) if taps else y
