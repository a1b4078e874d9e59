"""Float64 CPU oracle of the EQ-Linear layer for the DIHEDRAL group D_T (rotations and reflections, order 2T).

Test infrastructure only: nothing in the product path imports this file.

The paper's construction (Eq. 1: a dense weight obtained by replicating and permuting one small weight along the group)
is stated for the cyclic group and names reflections as the next group to cover (Conclusion).  This file writes the same
definition out for D_T, with no Fourier transform, blocking or reordering:

    y[n, o, g] = b[o] + sum_i sum_h  w[o, i, h^-1 g] * x[n, i, h]            g, h in D_T

i.e. the group convolution whose restriction to the rotation subgroup is the cyclic layer's (t - s) mod T reading.
Group elements are indexed g = f*T + t  <->  r^t s^f  (t in Z_T rotations, f in {0, 1} the reflection flag), with
s r = r^-1 s.  Features are [N, C * 2T] with the group index fastest, the weight is [C_out, C_in, 2T].
"""

from __future__ import annotations

import numpy as np


def group_tables(T: int):
    """Multiplication and inverse tables of D_T for the indexing g = f*T + t <-> r^t s^f.
    (r^a s^f)(r^b s^e) = r^(a + (-1)^f b) s^(f + e);  rotations invert to r^-a, reflections are involutions."""
    L = 2 * T
    mul = np.empty((L, L), dtype=np.int64)
    inv = np.empty(L, dtype=np.int64)
    for g in range(L):
        f, a = divmod(g, T)
        inv[g] = ((-a) % T) if f == 0 else g
        for h in range(L):
            e, b = divmod(h, T)
            t = (a + (b if f == 0 else -b)) % T
            mul[g, h] = ((f + e) % 2) * T + t
    return mul, inv


def unroll_dense(w: np.ndarray, T: int) -> np.ndarray:
    """W[(o, g), (i, h)] = w[o, i, h^-1 g]: the dense [C_out*2T, C_in*2T] weight of the D_T-equivariant layer."""
    w = np.asarray(w, dtype=np.float64)
    Co, Ci, L = w.shape
    assert L == 2 * T
    mul, inv = group_tables(T)
    k = mul[inv[None, :], np.arange(L)[:, None]]          # k[g, h] = h^-1 g
    return w[:, :, k].transpose(0, 2, 1, 3).reshape(Co * L, Ci * L)


def fwd(x, w, bias, T):
    W = unroll_dense(w, T)
    y = np.asarray(x, dtype=np.float64) @ W.T
    if bias is not None:
        y = y + np.repeat(np.asarray(bias, dtype=np.float64), 2 * T)[None, :]
    return y


def bwd_data(dy, w, T):
    return np.asarray(dy, dtype=np.float64) @ unroll_dense(w, T)


def bwd_weight(x, dy, T):
    """dw[o, i, k] = sum over the entries (o, g), (i, h) of dy^T x with h^-1 g = k;  db[o] = sum_n sum_g dy[n, o, g]."""
    x = np.asarray(x, dtype=np.float64)
    dy = np.asarray(dy, dtype=np.float64)
    L = 2 * T
    Ci, Co = x.shape[1] // L, dy.shape[1] // L
    G = (dy.T @ x).reshape(Co, L, Ci, L)                  # [o, g, i, h]
    mul, inv = group_tables(T)
    dw = np.zeros((Co, Ci, L))
    for g in range(L):
        for h in range(L):
            dw[:, :, mul[inv[h], g]] += G[:, g, :, h]
    db = dy.reshape(-1, Co, L).sum(axis=(0, 2))
    return dw, db
