"""Pins for the float64 oracle: each check is an independent route to the same numbers.

None of these re-types the oracle's own formula (dense unroll + matmul): they use
 (1) a four-loop evaluation of the circular-convolution definition,
 (2) the paper's p4 closed form (Eq. 19-21) restated here,
 (3) numpy.fft's rfft / irfft along the group axis (convolution theorem, Eq. 3-7),
 (4) invariants of the operator (equivariance, delta weights, adjoint identities, linearity),
 (5) a hand-worked example stored under tests/golden/.
"""

import itertools
import os

import numpy as np
import pytest

from oracle import eqlinear_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rnd(seed, *shape):
    return np.random.Generator(np.random.PCG64(seed)).standard_normal(shape)


# ---------------------------------------------------------------- (1) brute force
def brute_fwd(x, w, b, T, correlation=False):
    """y[n,o,t] = b[o] + sum_i sum_s w[o,i,(t-s) mod T] x[n,i,s], one scalar at a time."""
    N = x.shape[0]
    Co, Ci, _ = w.shape
    y = np.zeros((N, Co, T))
    for n in range(N):
        for o in range(Co):
            for t in range(T):
                acc = 0.0 if b is None else float(b[o])
                for i in range(Ci):
                    for s in range(T):
                        r = (s - t) % T if correlation else (t - s) % T
                        acc += w[o, i, r] * x[n, i * T + s]
                y[n, o, t] = acc
    return y.reshape(N, Co * T)


@pytest.mark.parametrize("T", [1, 2, 3, 4, 5, 6, 7, 8, 12, 16, 32])
@pytest.mark.parametrize("Ci,Co,N", [(1, 1, 1), (3, 2, 2), (2, 5, 3), (8, 3, 5)])
@pytest.mark.parametrize("correlation", [False, True])
def test_forward_matches_brute_force(T, Ci, Co, N, correlation):
    x, w, b = rnd(1, N, Ci * T), rnd(2, Co, Ci, T), rnd(3, Co)
    ref = brute_fwd(x, w, b, T, correlation)
    got = orc.fwd(x, w, b, correlation)
    assert np.abs(got - ref).max() <= 1e-13 * max(1.0, np.abs(ref).max())
    got_nb = orc.fwd(x, w, None, correlation)
    assert np.abs(got_nb - brute_fwd(x, w, None, T, correlation)).max() <= 1e-13 * max(1.0, np.abs(ref).max())


@pytest.mark.parametrize("T", [1, 2, 3, 4, 5, 6, 7, 8, 12])
@pytest.mark.parametrize("correlation", [False, True])
def test_gradients_match_finite_structure(T, correlation):
    """The layer is linear, so its exact gradients are read off scalar by scalar:
    dx[n,i,s] = sum_{o,t} dy[n,o,t] w[o,i,(t-s)], dw[o,i,r] = sum_{n,t} dy[n,o,t] x[n,i,(t-r)]."""
    N, Ci, Co = 3, 2, 3
    x, w, dy = rnd(4, N, Ci * T), rnd(5, Co, Ci, T), rnd(6, N, Co * T)
    dx = np.zeros((N, Ci * T))
    dw = np.zeros((Co, Ci, T))
    for n, o, t, i, s in itertools.product(range(N), range(Co), range(T), range(Ci), range(T)):
        r = (s - t) % T if correlation else (t - s) % T
        dx[n, i * T + s] += dy[n, o * T + t] * w[o, i, r]
        dw[o, i, r] += dy[n, o * T + t] * x[n, i * T + s]
    db = dy.reshape(N, Co, T).sum(axis=(0, 2))
    got_dx = orc.bwd_data(dy, w, correlation)
    got_dw, got_db = orc.bwd_weight(x, dy, T, correlation)
    assert np.abs(got_dx - dx).max() <= 1e-13
    assert np.abs(got_dw - dw).max() <= 1e-13
    assert np.abs(got_db - db).max() <= 1e-13


# ---------------------------------------------------------------- (2) p4 closed form, Eq. 19-21
def p4_planes(v):
    """Eq. 19 on the last axis (length 4): (k=0, Re k=1, k=2, Im k=1)."""
    v0, v1, v2, v3 = v[..., 0], v[..., 1], v[..., 2], v[..., 3]
    return v0 + v1 + v2 + v3, v0 - v2, v0 - v1 + v2 - v3, v3 - v1


def p4_closed_form(x, w, b):
    N = x.shape[0]
    Co, Ci, _ = w.shape
    f0, f1, f2, f3 = p4_planes(x.reshape(N, Ci, 4))          # [N, Ci]
    w0, w1, w2, w3 = p4_planes(w)                            # [Co, Ci]
    a0 = f0 @ w0.T                                           # Eq. 20
    a1 = f1 @ w1.T - f3 @ w3.T
    a2 = f2 @ w2.T
    a3 = f1 @ w3.T + f3 @ w1.T
    y = np.stack([a0 / 4 + a1 / 2 + a2 / 4,                  # Eq. 21
                  a0 / 4 - a2 / 4 - a3 / 2,
                  a0 / 4 - a1 / 2 + a2 / 4,
                  a0 / 4 - a2 / 4 + a3 / 2], axis=-1)        # [N, Co, 4]
    return (y + b[None, :, None]).reshape(N, Co * 4)


def test_p4_closed_form_pins_the_convolution_reading():
    N, Ci, Co = 7, 5, 6
    x, w, b = rnd(7, N, Ci * 4), rnd(8, Co, Ci, 4), rnd(9, Co)
    ref = p4_closed_form(x, w, b)
    assert np.abs(orc.fwd(x, w, b) - ref).max() <= 1e-13
    # the correlation reading is a different operator: it must NOT agree
    assert np.abs(orc.fwd(x, w, b, correlation=True) - ref).max() > 1e-2


# ---------------------------------------------------------------- (3) convolution theorem through numpy.fft
@pytest.mark.parametrize("T", [1, 2, 3, 4, 5, 8, 16, 32])
def test_spectral_path_agrees_with_dense(T):
    N, Ci, Co = 6, 4, 3
    x, w, b, dy = rnd(10, N, Ci * T), rnd(11, Co, Ci, T), rnd(12, Co), rnd(13, N, Co * T)
    xh = np.fft.rfft(x.reshape(N, Ci, T), axis=-1)           # Eq. 4, k = 0..floor(T/2)
    wh = np.fft.rfft(w, axis=-1)
    gh = np.fft.rfft(dy.reshape(N, Co, T), axis=-1)
    yh = np.einsum("nik,oik->nok", xh, wh)                   # Eq. 5, one complex GEMM per k
    y = np.fft.irfft(yh, n=T, axis=-1) + b[None, :, None]    # Eq. 7
    assert np.abs(orc.fwd(x, w, b) - y.reshape(N, Co * T)).max() <= 1e-12
    dxh = np.einsum("nok,oik->nik", gh, np.conj(wh))
    dx = np.fft.irfft(dxh, n=T, axis=-1).reshape(N, Ci * T)
    assert np.abs(orc.bwd_data(dy, w) - dx).max() <= 1e-12
    dwh = np.einsum("nok,nik->oik", gh, np.conj(xh))
    dw = np.fft.irfft(dwh, n=T, axis=-1)
    got_dw, got_db = orc.bwd_weight(x, dy, T)
    assert np.abs(got_dw - dw).max() <= 1e-12
    assert np.abs(got_db - gh[:, :, 0].real.sum(axis=0)).max() <= 1e-12
    # correlation reading = conjugated weight spectrum
    yc = np.fft.irfft(np.einsum("nik,oik->nok", xh, np.conj(wh)), n=T, axis=-1) + b[None, :, None]
    assert np.abs(orc.fwd(x, w, b, correlation=True) - yc.reshape(N, Co * T)).max() <= 1e-12


# ---------------------------------------------------------------- (4) invariants
@pytest.mark.parametrize("T", [2, 3, 4, 8, 32])
@pytest.mark.parametrize("correlation", [False, True])
def test_equivariance_under_group_shift(T, correlation):
    N, Ci, Co = 4, 3, 5
    x, w, b = rnd(14, N, Ci * T), rnd(15, Co, Ci, T), rnd(16, Co)
    y = orc.fwd(x, w, b, correlation).reshape(N, Co, T)
    for r in range(T):
        xr = np.roll(x.reshape(N, Ci, T), r, axis=-1).reshape(N, Ci * T)
        yr = orc.fwd(xr, w, b, correlation).reshape(N, Co, T)
        assert np.abs(yr - np.roll(y, r, axis=-1)).max() <= 1e-12


@pytest.mark.parametrize("T", [2, 4, 5, 8])
def test_delta_weights(T):
    N, Ci, Co = 3, 4, 2
    x, M = rnd(17, N, Ci * T), rnd(18, Co, Ci)
    xs = x.reshape(N, Ci, T)
    w0 = np.zeros((Co, Ci, T)); w0[:, :, 0] = M              # identity on the group axis
    y0 = orc.fwd(x, w0).reshape(N, Co, T)
    assert np.abs(y0 - np.einsum("oi,nit->not", M, xs)).max() <= 1e-13
    w1 = np.zeros((Co, Ci, T)); w1[:, :, 1] = M              # delta at r = 1 shifts by +1 (convolution)
    y1 = orc.fwd(x, w1).reshape(N, Co, T)
    assert np.abs(y1 - np.einsum("oi,nit->not", M, np.roll(xs, 1, axis=-1))).max() <= 1e-13
    y1c = orc.fwd(x, w1, correlation=True).reshape(N, Co, T)  # ... and by -1 for the correlation
    assert np.abs(y1c - np.einsum("oi,nit->not", M, np.roll(xs, -1, axis=-1))).max() <= 1e-13


@pytest.mark.parametrize("T", [1, 3, 4, 8, 16])
@pytest.mark.parametrize("correlation", [False, True])
def test_adjoint_identities(T, correlation):
    N, Ci, Co = 5, 3, 4
    x, w, dy = rnd(19, N, Ci * T), rnd(20, Co, Ci, T), rnd(21, N, Co * T)
    lhs = np.vdot(dy, orc.fwd(x, w, None, correlation))
    dx = orc.bwd_data(dy, w, correlation)
    dw, db = orc.bwd_weight(x, dy, T, correlation)
    assert abs(lhs - np.vdot(dx, x)) <= 1e-11 * abs(lhs)
    assert abs(lhs - np.vdot(dw, w)) <= 1e-11 * abs(lhs)
    assert np.abs(db - dy.reshape(N, Co, T).sum(axis=(0, 2))).max() <= 1e-12


def test_linearity_and_dense_shape():
    T, N, Ci, Co = 4, 3, 2, 3
    x1, x2, w1, w2 = rnd(22, N, Ci * T), rnd(23, N, Ci * T), rnd(24, Co, Ci, T), rnd(25, Co, Ci, T)
    assert orc.unroll_dense(w1).shape == (Co * T, Ci * T)
    assert np.abs(orc.fwd(2 * x1 - x2, w1) - (2 * orc.fwd(x1, w1) - orc.fwd(x2, w1))).max() <= 1e-12
    assert np.abs(orc.fwd(x1, w1 + 3 * w2) - (orc.fwd(x1, w1) + 3 * orc.fwd(x1, w2))).max() <= 1e-12
    # every dense row holds each w[o, i, :] exactly once: row sums equal the per-channel weight sums
    W = orc.unroll_dense(w1)
    assert np.abs(W.sum(axis=1) - np.repeat(w1.sum(axis=(1, 2)), T)).max() <= 1e-12


# ---------------------------------------------------------------- (5) golden worked example
def load_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, vals = line.split(":")
            out[key.strip()] = np.array([float(v) for v in vals.split()])
    return out


def test_worked_p4_example():
    g = load_golden("p4_worked_example.txt")
    T = int(g["T"][0])
    x, w, b, dy = g["x"][None, :], g["w"].reshape(1, 1, T), g["bias"], g["dy"][None, :]
    assert np.array_equal(orc.fwd(x, w, b)[0], g["y"])
    assert np.array_equal(orc.bwd_data(dy, w)[0], g["dx"])
    dw, db = orc.bwd_weight(x, dy, T)
    assert np.array_equal(dw[0, 0], g["dw"])
    assert np.array_equal(db, g["db"])
    # the intermediate values in the fixture are the paper's p4 coordinates (Eq. 19-20)
    assert np.array_equal(np.array(p4_planes(g["x"])), g["f"])
    assert np.array_equal(np.array(p4_planes(g["w"])), g["w_planes"])
