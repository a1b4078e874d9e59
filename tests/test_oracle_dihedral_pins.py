"""Pins of the dihedral-group oracle (oracle/eqlinear_oracle_dihedral.py) to things other than itself: the group law
re-derived from D_T's action on the T-gon, a brute-force loop of the definition, the equivariance invariant, delta
weights, the cyclic oracle on the rotation subgroup, the irreducible-representation (Fourier) route, and the adjoint
identities of the gradients."""

import itertools

import numpy as np
import pytest

from oracle import eqlinear_oracle as cyc
from oracle import eqlinear_oracle_dihedral as dih


def act(g, T):
    """r^t s^f as a permutation of the T corners of a polygon: p -> t + p (rotation), p -> t - p (after a reflection)."""
    f, t = divmod(g, T)
    return tuple((t + (-p if f else p)) % T for p in range(T))


def compose(a, b):
    return tuple(a[b[p]] for p in range(len(a)))      # first b, then a


@pytest.mark.parametrize("T", [3, 4, 5, 8])
def test_group_tables_match_the_action_on_the_polygon(T):
    mul, inv = dih.group_tables(T)
    L = 2 * T
    perms = [act(g, T) for g in range(L)]
    index = {p: g for g, p in enumerate(perms)}
    assert len(index) == L                              # the action is faithful for T >= 3
    for g, h in itertools.product(range(L), repeat=2):
        assert mul[g, h] == index[compose(perms[g], perms[h])]
    ident = index[tuple(range(T))]
    assert ident == 0
    for g in range(L):
        assert mul[g, inv[g]] == ident and mul[inv[g], g] == ident
    r, s = 1, T
    assert mul[s, r] == mul[inv[r], s]                  # s r = r^-1 s
    assert mul[r, s] != mul[s, r]                       # not abelian


def brute_force(x, w, b, T):
    L = 2 * T
    perms = [act(g, T) for g in range(L)]
    index = {p: g for g, p in enumerate(perms)}
    inv_perm = lambda p: tuple(np.argsort(p))
    N, Ci, Co = x.shape[0], w.shape[1], w.shape[0]
    xr = x.reshape(N, Ci, L)
    y = np.zeros((N, Co, L))
    for n in range(N):
        for o in range(Co):
            for g in range(L):
                acc = 0.0 if b is None else b[o]
                for i in range(Ci):
                    for h in range(L):
                        k = index[compose(inv_perm(perms[h]), perms[g])]        # h^-1 g
                        acc += w[o, i, k] * xr[n, i, h]
                y[n, o, g] = acc
    return y.reshape(N, Co * L)


@pytest.mark.parametrize("T", [3, 4, 5])
def test_forward_matches_brute_force(T):
    g = np.random.default_rng(T)
    L = 2 * T
    x, w, b = g.standard_normal((3, 2 * L)), g.standard_normal((3, 2, L)), g.standard_normal(3)
    assert np.allclose(dih.fwd(x, w, b, T), brute_force(x, w, b, T), rtol=0, atol=1e-12)
    assert np.allclose(dih.fwd(x, w, None, T), brute_force(x, w, None, T), rtol=0, atol=1e-12)


@pytest.mark.parametrize("T", [3, 4, 6])
def test_equivariance_under_every_group_element(T):
    g = np.random.default_rng(10 + T)
    L = 2 * T
    mul, inv = dih.group_tables(T)
    x, w, b = g.standard_normal((4, 3 * L)), g.standard_normal((2, 3, L)), g.standard_normal(2)
    y = dih.fwd(x, w, b, T).reshape(4, 2, L)
    for u in range(L):
        perm = mul[inv[u], np.arange(L)]                # (L_u x)(g) = x(u^-1 g)
        xu = x.reshape(4, 3, L)[:, :, perm].reshape(4, 3 * L)
        yu = dih.fwd(xu, w, b, T).reshape(4, 2, L)
        assert np.allclose(yu, y[:, :, perm], rtol=0, atol=1e-12)


@pytest.mark.parametrize("T", [3, 4])
def test_delta_weights(T):
    g = np.random.default_rng(20 + T)
    L = 2 * T
    mul, inv = dih.group_tables(T)
    M = g.standard_normal((3, 2))
    x = g.standard_normal((5, 2 * L))
    xr = x.reshape(5, 2, L)
    for u in (0, 1, T, T + 1):
        w = np.zeros((3, 2, L)); w[:, :, u] = M
        y = dih.fwd(x, w, None, T).reshape(5, 3, L)
        # y(g) = sum_h w(h^-1 g) x(h) = M x(g u^-1)
        src = mul[np.arange(L), inv[u]]
        assert np.allclose(y, np.einsum("oi,nig->nog", M, xr[:, :, src]), rtol=0, atol=1e-12)


@pytest.mark.parametrize("T", [3, 4, 8])
def test_rotation_subgroup_reduces_to_the_cyclic_layer(T):
    """A weight and an input supported on the rotations: on the rotations the output is the cyclic layer's (t - s)
    convolution, and nothing reaches the reflection coset."""
    g = np.random.default_rng(30 + T)
    L = 2 * T
    wc, xc, b = g.standard_normal((3, 2, T)), g.standard_normal((4, 2 * T)), g.standard_normal(3)
    w = np.zeros((3, 2, L)); w[:, :, :T] = wc
    x = np.zeros((4, 2, L)); x[:, :, :T] = xc.reshape(4, 2, T)
    y = dih.fwd(x.reshape(4, 2 * L), w, None, T).reshape(4, 3, L)
    assert np.allclose(y[:, :, :T].reshape(4, 3 * T), cyc.fwd(xc, wc, None), rtol=0, atol=1e-12)
    assert np.allclose(y[:, :, T:], 0.0)


def irreps(T):
    """Real irreducible representations of D_T: list of (dimension, function g -> matrix)."""
    L = 2 * T
    out = []
    def one(sr, ss):
        return lambda g: np.array([[(sr ** (g % T)) * (ss ** (g // T))]], dtype=np.float64)
    out.append((1, one(1, 1))); out.append((1, one(1, -1)))
    if T % 2 == 0:
        out.append((1, one(-1, 1))); out.append((1, one(-1, -1)))
    for k in range(1, (T + 1) // 2):
        def rho(g, k=k):
            f, t = divmod(g, T)
            th = 2 * np.pi * k * t / T
            R = np.array([[np.cos(th), -np.sin(th)], [np.sin(th), np.cos(th)]])
            return R @ np.diag([1.0, -1.0]) if f else R
        out.append((2, rho))
    assert sum(d * d for d, _ in out) == L
    return out


def fourier_fwd(x, w, b, T):
    """The convolution theorem on D_T: y^(rho) = x^(rho) w^(rho) with f^(rho) = sum_g f(g) rho(g), then
    y(g) = 1/|G| sum_rho d_rho tr(rho(g)^T y^(rho))."""
    L = 2 * T
    N, Ci, Co = x.shape[0], w.shape[1], w.shape[0]
    xr = x.reshape(N, Ci, L)
    y = np.zeros((N, Co, L))
    for d, rho in irreps(T):
        mats = np.stack([rho(g) for g in range(L)])                       # [L, d, d]
        xh = np.einsum("nig,gab->niab", xr, mats)
        wh = np.einsum("oig,gab->oiab", w, mats)
        yh = np.einsum("niab,oibc->noac", xh, wh)
        y += (d / L) * np.einsum("noac,gac->nog", yh, mats)
    if b is not None:
        y += b[None, :, None]
    return y.reshape(N, Co * L)


@pytest.mark.parametrize("T", [2, 3, 4, 5, 8])
def test_fourier_route_agrees_with_dense(T):
    g = np.random.default_rng(40 + T)
    L = 2 * T
    x, w, b = g.standard_normal((5, 3 * L)), g.standard_normal((4, 3, L)), g.standard_normal(4)
    assert np.allclose(fourier_fwd(x, w, b, T), dih.fwd(x, w, b, T), rtol=0, atol=1e-11)


@pytest.mark.parametrize("T", [3, 4, 5])
def test_gradients(T):
    """Adjoint identities of a linear map, db = sum dy, and dw scalar by scalar on a small case."""
    g = np.random.default_rng(50 + T)
    L = 2 * T
    x, w, dy = g.standard_normal((6, 2 * L)), g.standard_normal((3, 2, L)), g.standard_normal((6, 3 * L))
    dx = dih.bwd_data(dy, w, T)
    dw, db = dih.bwd_weight(x, dy, T)
    lhs = np.vdot(dy, dih.fwd(x, w, None, T))
    assert abs(lhs - np.vdot(dx, x)) <= 1e-10 * abs(lhs)
    assert abs(lhs - np.vdot(dw, w)) <= 1e-10 * abs(lhs)
    assert np.allclose(db, dy.reshape(6, 3, L).sum(axis=(0, 2)))
    for (o, i, k) in [(0, 0, 0), (1, 1, 1), (2, 0, T), (0, 1, L - 1)]:
        e = np.zeros_like(w); e[o, i, k] = 1.0
        assert abs(np.vdot(dy, dih.fwd(x, e, None, T)) - dw[o, i, k]) <= 1e-10
    for (n, c) in [(0, 0), (3, L + 1), (5, 2 * L - 1)]:
        e = np.zeros_like(x); e[n, c] = 1.0
        assert abs(np.vdot(dy, dih.fwd(e, w, None, T)) - dx[n, c]) <= 1e-10
