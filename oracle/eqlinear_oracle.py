"""Float64 CPU oracle for the cyclic-group equivariant linear layer (EQ-Linear).

THIS FILE IS TEST INFRASTRUCTURE.  It is the slow, plain definition that the CUDA
library is checked against; only the tests, the smoke check and the benchmark's
CPU-baseline leg may import it.  It shares no code with the CUDA path and imports
nothing from the product package.

What it computes (Eq. 1, the dense block-circulant form of EQ-Linear): the learnable
weight ``w[o, i, r]`` (``[Co, Ci, T]``) is unrolled into the dense matrix

    W[(o, t), (i, s)] = w[o, i, (t - s) mod T]          row = o*T + t,  col = i*T + s

and the layer is the ordinary affine map ``y = x W^T + tile_T(b)`` on row-major
``[N, C*T]`` features whose group index is the fastest one.  The fast algorithm of the
paper (Algorithm 1: group DFT, one complex channel GEMM per retained frequency, inverse
DFT) reaches exactly this result, so the oracle is the definition written out, in
float64, with a library matmul as its only primitive.

Index convention.  The paper's Eq. 1-2 print the circulant with index ``(s - t)``
(a circular correlation), while its Eq. 3-5 and the appendix kernel equations
(Eq. 19-21) compute the true circular convolution ``(t - s)``.  The convolution is the
default here; ``correlation=True`` gives the other reading (the same operator with the
weight reversed along the group axis).

Pins (tests/test_oracle_pins.py): brute-force four-loop evaluation of the definition,
the p4 closed form of Eq. 19-21 restated independently, numpy.fft's rfft/irfft along
the group axis (convolution theorem, Eq. 3), the equivariance invariant, the delta-weight
special cases, the adjoint identities for both gradients, and a hand-worked T=4 example
stored under tests/golden/.  No function in this file is "parity unpinned".
"""

from __future__ import annotations

import numpy as np


def _as_f64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def unroll_dense(w, correlation: bool = False) -> np.ndarray:
    """Dense block-circulant weight of Eq. 1.

    w: [Co, Ci, T].  Returns W: [Co*T, Ci*T] with
    W[o*T + t, i*T + s] = w[o, i, (t - s) mod T]   (or (s - t) mod T if ``correlation``).
    """
    w = _as_f64(w)
    Co, Ci, T = w.shape
    t = np.arange(T).reshape(T, 1)
    s = np.arange(T).reshape(1, T)
    r = (s - t) % T if correlation else (t - s) % T          # [T(t), T(s)]
    blocks = w[:, :, r]                                      # [Co, Ci, T(t), T(s)]
    return np.ascontiguousarray(blocks.transpose(0, 2, 1, 3).reshape(Co * T, Ci * T))


def fwd(x, w, bias=None, correlation: bool = False) -> np.ndarray:
    """Forward of Eq. 1: y[N, Co*T] = x[N, Ci*T] . W^T + tile_T(bias).

    ``bias`` is [Co], shared by all T group components of an output channel and by all tokens.
    """
    x = _as_f64(x)
    W = unroll_dense(w, correlation)
    y = x @ W.T
    if bias is not None:
        T = np.asarray(w).shape[2]
        y = y + np.repeat(_as_f64(bias), T)[None, :]
    return y


def bwd_data(dy, w, correlation: bool = False) -> np.ndarray:
    """Gradient of the forward with respect to x: dx[N, Ci*T] = dy[N, Co*T] . W."""
    dy = _as_f64(dy)
    W = unroll_dense(w, correlation)
    return dy @ W


def bwd_weight(x, dy, T: int, correlation: bool = False):
    """Gradients with respect to the original parameters.

    G = dy^T . x is the gradient of the dense W ([Co*T, Ci*T]); every w[o, i, r] appears in
    W at the T positions (t, s) with (t - s) mod T = r, so its gradient is the sum of G there:
        dw[o, i, r] = sum_t G[o*T + t, i*T + (t - r) mod T].
    The bias gradient is db[o] = sum_n sum_t dy[n, o, t].
    Returns (dw [Co, Ci, T], db [Co]).
    """
    x = _as_f64(x)
    dy = _as_f64(dy)
    N, Din = x.shape
    Dout = dy.shape[1]
    Ci, Co = Din // T, Dout // T
    G = (dy.T @ x).reshape(Co, T, Ci, T)                     # [o, t, i, s]
    dw = np.zeros((Co, Ci, T), dtype=np.float64)
    for r in range(T):
        for t in range(T):
            s = (t + r) % T if correlation else (t - r) % T
            dw[:, :, r] += G[:, t, :, s]
    db = dy.reshape(N, Co, T).sum(axis=(0, 2))
    return dw, db
