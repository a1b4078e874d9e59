"""GPU parity of the dihedral-group layer (EQL_FLAG_DIHEDRAL) against its float64 dense-unroll oracle, through the C ABI."""

import numpy as np
import pytest
import torch

import paper_2607_21271_b200 as eq
from oracle import eqlinear_oracle_dihedral as dih
from tests.harness import TOL, GpuLayer, rel_max_err
from paper_2607_21271_b200.workloads import round_to_bf16

pytestmark = pytest.mark.gpu

D = eq.EQL_FLAG_DIHEDRAL


def draw(T, Ci, Co, N, dtype, seed, bias=True):
    """Seeded Gaussians in the layer's I/O type: x, dy ~ N(0, 1), w ~ N(0, 1 / (C_in * 2T)), bias ~ N(0, 0.02)."""
    g = np.random.Generator(np.random.PCG64(seed))
    L = 2 * T
    x = g.standard_normal((N, Ci * L), dtype=np.float32)
    w = g.standard_normal((Co, Ci, L), dtype=np.float32) / np.float32(np.sqrt(Ci * L))
    b = g.standard_normal(Co, dtype=np.float32) * np.float32(np.sqrt(0.02))
    dy = g.standard_normal((N, Co * L), dtype=np.float32)
    narrow = {"fp32": lambda a: a, "fp16": lambda a: a.astype(np.float16), "bf16": round_to_bf16}[dtype]
    return narrow(x), narrow(w), (narrow(b) if bias else None), narrow(dy)


@pytest.mark.parametrize("dtype", ["fp32", "fp16", "bf16"])
@pytest.mark.parametrize("T,Ci,Co,N", [(2, 8, 12, 333), (3, 8, 16, 200), (4, 24, 40, 1000), (5, 8, 8, 129), (6, 4, 12, 65),
                                        (8, 16, 24, 500), (4, 2, 70, 1)])
def test_dihedral_matches_oracle(dtype, T, Ci, Co, N):
    x, w, b, dy = draw(T, Ci, Co, N, dtype, 100 + T)
    layer = GpuLayer(T, Ci, Co, dtype, w, b, D)
    try:
        info = eq.eqlinear_plan_info(layer.plan)
        assert (info.T, info.fwd_kernel, info.bwd_data_kernel, info.bwd_weight_kernel) == (T, 0, 0, 0)
        n1, k2 = (4, T // 2 - 1) if T % 2 == 0 else (2, (T - 1) // 2)
        assert info.macs_per_token == (n1 + 8 * k2) * Ci * Co and info.dense_macs_per_token == (2 * T) ** 2 * Ci * Co
        y, dx = layer.fwd(x), layer.bwd_data(dy)
        dw, db = layer.bwd_weight(x, dy)
        dw2, _ = layer.bwd_weight(x, dy)
        assert np.array_equal(dw, dw2)                                  # fixed reduction order
    finally:
        layer.close()
    rdw, rdb = dih.bwd_weight(x, dy, T)
    errs = {"y": rel_max_err(y, dih.fwd(x, w, b, T)), "dx": rel_max_err(dx, dih.bwd_data(dy, w, T)),
            "dw": rel_max_err(dw, rdw), "db": rel_max_err(db, rdb)}
    for k, v in errs.items():
        assert v <= TOL[dtype], f"D_{T} {dtype} {Ci}->{Co} N={N}: {k} error {v:.3e}"


def test_dihedral_equivariance_on_the_gpu_and_gelu():
    """The GPU output alone: translating the input by any group element translates the output (also with the fused GELU,
    a pointwise map); and GELU(layer) against the oracle."""
    from scipy.special import erf
    T, Ci, Co, N = 4, 8, 12, 64
    x, w, b, _ = draw(T, Ci, Co, N, "fp32", 7)
    mul, inv = dih.group_tables(T)
    L = 2 * T
    for flags in (D, D | eq.EQL_FLAG_GELU):
        layer = GpuLayer(T, Ci, Co, "fp32", w, b, flags)
        try:
            y = layer.fwd(x).astype(np.float64).reshape(N, Co, L)
            for u in (1, T, T + 3):
                perm = mul[inv[u], np.arange(L)]
                xu = np.ascontiguousarray(x.reshape(N, Ci, L)[:, :, perm].reshape(N, Ci * L))
                yu = layer.fwd(xu).astype(np.float64).reshape(N, Co, L)
                assert ((yu - y[:, :, perm]) ** 2).sum() <= 1e-12 * (y ** 2).sum()
        finally:
            layer.close()
    ref = dih.fwd(x, w, b, T)
    assert rel_max_err(y.reshape(N, Co * L), 0.5 * ref * (1.0 + erf(ref / np.sqrt(2.0)))) <= TOL["fp32"]


def test_dihedral_argument_errors():
    lib, B = eq.load_library(), eq.binding
    with pytest.raises(eq.EqlError) as e:
        eq.eqlinear_workspace_bytes_flags(7, 8, 8, eq.EQL_FP32, D)       # D_7 is not among the built orders
    assert e.value.status == B.EQL_ERR_UNSUPPORTED
    assert eq.eqlinear_workspace_bytes_flags(5, 8, 8, eq.EQL_FP32, D) >= 2 * 10 * 64 * 4
    x, w, b, _ = draw(4, 8, 8, 16, "fp32", 1)
    for bad in (eq.EQL_FLAG_CORRELATION, eq.EQL_FLAG_FORCE_STREAMING, eq.EQL_FLAG_CTA_PAIR):
        with pytest.raises(eq.EqlError) as e:
            GpuLayer(4, 8, 8, "fp32", w, b, D | bad)
        assert e.value.status == B.EQL_ERR_INVALID_ARG
