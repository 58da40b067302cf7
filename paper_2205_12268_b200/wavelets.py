"""Filter banks for the generic wavelet entry points (wcc_dwt_fwd, wcc_dwt_inv, wcc_forward_wavelet): decomposition and
reconstruction filters as plain float32 arrays of even length, in the library's indexing (origin T/2 - 1, periodic
extension, see wcc.h).  No layer arithmetic here: these are inputs, used by the CUDA path's callers and by the tests of
the oracle alike.

Haar and db2 have closed forms; the Daubechies family in general is built from the roots of its defining polynomial
(Daubechies 1988: the minimum-phase spectral factor of the half-band product filter); bior2.2 is the 5/3 spline pair
with rational taps.
"""
from __future__ import annotations

import math

import numpy as np


def _qmf(lo: np.ndarray) -> np.ndarray:
    """The high-pass partner of an orthogonal low-pass filter: hi[t] = (-1)^t lo[T - 1 - t]."""
    T = lo.size
    return np.array([(-1) ** t * lo[T - 1 - t] for t in range(T)], dtype=np.float64)


def daubechies(p: int) -> np.ndarray:
    """Low-pass decomposition filter of the Daubechies wavelet with p vanishing moments (2p taps), float64.
    |H(w)|^2 = cos^{2p}(w/2) * Q(sin^2(w/2)), Q(y) = sum_{k<p} C(p-1+k, k) y^k; the filter is the factor of that
    product whose roots lie inside the unit circle, times (1 + z^-1)^p, normalised to sum sqrt 2."""
    if p == 1:
        return np.array([1.0, 1.0]) / math.sqrt(2.0)
    q = [math.comb(p - 1 + k, k) for k in range(p)]                  # Q(y), ascending powers of y
    # y = (2 - z - 1/z) / 4: z^(p-1) * Q(y(z)) as a polynomial in z
    poly = np.zeros(2 * p - 1)
    base = np.array([-0.25, 0.5, -0.25])                             # z * y(z) = -z^2/4 + z/2 - 1/4
    term = np.array([1.0])
    for kk in range(p):
        shifted = np.zeros(2 * p - 1)
        off = (p - 1) - kk                                           # z^(p-1-k) * (z y)^k
        shifted[off:off + term.size] = term
        poly += q[kk] * shifted
        term = np.convolve(term, base)
    roots = np.roots(poly[::-1])
    inside = roots[np.abs(roots) < 1.0]
    h = np.array([1.0])
    for r in inside:
        h = np.convolve(h, [1.0, -r])
    for _ in range(p):
        h = np.convolve(h, [1.0, 1.0])
    h = np.real(h)
    return h * (math.sqrt(2.0) / h.sum())


def filter_bank(name: str):
    """(dec_lo, dec_hi, rec_lo, rec_hi) as float32 arrays for 'haar', 'db2', 'db3', 'db4', 'bior2.2'."""
    name = name.lower()
    if name in ("haar", "db1"):
        lo = daubechies(1)
    elif name == "db2":
        r3 = math.sqrt(3.0)
        lo = np.array([1 + r3, 3 + r3, 3 - r3, 1 - r3]) / (4.0 * math.sqrt(2.0))
    elif name.startswith("db") and name[2:].isdigit() and 3 <= int(name[2:]) <= 8:
        lo = daubechies(int(name[2:]))
    elif name == "bior2.2":
        s = math.sqrt(2.0) / 8.0
        bank = (np.array([-1, 2, 6, 2, -1, 0]) * s, np.array([0, 0, 2, -4, 2, 0]) * s,
                np.array([0, 2, 4, 2, 0, 0]) * s, np.array([0, 1, 2, -6, 2, 1]) * s)
        return tuple(np.asarray(f, dtype=np.float32) for f in bank)
    else:
        raise ValueError("unknown wavelet %r" % name)
    hi = _qmf(lo)
    lo32, hi32 = lo.astype(np.float32), hi.astype(np.float32)
    return lo32, hi32, lo32, hi32
