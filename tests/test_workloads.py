"""CPU checks of the seeded input recipes (they serve the oracle and the CUDA path alike and hold none of the
method's arithmetic): determinism, dtypes and shapes, the statistics the recipe states, the row sampler used for
full-size parity on sampled outputs, and the shapes of the paper's operator-level benchmark (Tables 1-2)."""

import numpy as np
import pytest

from paper_2607_21271_b200.workloads import (ALL_WORKLOADS, BLOCK_SHAPES, CONFIGS, HEADLINE, OPERATOR_SHAPES, Workload, generate,
                                              sample_rows)


def test_bf16_rounding_is_round_to_nearest_even():
    """bf16 workloads are float32 arrays of bfloat16-representable values: the rounding must be the IEEE one (checked
    against torch's conversion, and on the tie cases by hand)."""
    import torch
    from paper_2607_21271_b200.workloads import round_to_bf16
    g = np.random.Generator(np.random.PCG64(3))
    a = (g.standard_normal(100000) * np.exp(g.uniform(-20, 20, 100000))).astype(np.float32)
    ref = torch.from_numpy(a).to(torch.bfloat16).float().numpy()
    assert np.array_equal(round_to_bf16(a), ref)
    ties = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -(1.0 + 2.0 ** -8)], dtype=np.float32)   # halfway cases
    assert np.array_equal(round_to_bf16(ties), np.array([1.0, 1.0 + 2.0 ** -6, -1.0], dtype=np.float32))
    wl = Workload("b", "bf16", 4, 8, 8, 16, "normal", ("fwd",), 1)
    d = generate(wl)
    for k in ("x", "w", "bias", "dy"):
        assert d[k].dtype == np.float32 and np.array_equal(round_to_bf16(d[k]), d[k])


def test_tables_are_consistent():
    assert HEADLINE in CONFIGS
    assert set(CONFIGS) | set(OPERATOR_SHAPES) | set(BLOCK_SHAPES) == set(ALL_WORKLOADS)
    assert not set(CONFIGS) & set(OPERATOR_SHAPES)
    for name, wl in ALL_WORKLOADS.items():
        assert wl.name == name
        assert wl.dtype in ("fp32", "fp16", "bf16") and wl.bias in ("none", "zero", "normal")
        assert wl.Din == wl.Ci * wl.T and wl.Dout == wl.Co * wl.T
        esz = 4 if wl.dtype == "fp32" else 2
        assert (wl.Din * esz) % 16 == 0 and (wl.Dout * esz) % 16 == 0          # rows are whole 16-byte units


def test_operator_shapes_follow_the_paper_setup():
    # batch 32 x 1024 tokens, the p4 group, equal widths on both sides, bias, forward and full backward
    for wl in OPERATOR_SHAPES.values():
        assert (wl.T, wl.N, wl.bias) == (4, 32 * 1024, "normal")
        assert wl.Ci == wl.Co and set(wl.passes) == {"fwd", "bwd_data", "bwd_weight"}
    assert {wl.Ci for wl in OPERATOR_SHAPES.values() if wl.dtype == "fp16"} >= {64, 256, 1024, 2048}


@pytest.mark.parametrize("dtype", ["fp32", "fp16"])
def test_generate_is_deterministic_and_typed(dtype):
    wl = Workload("w", dtype, 8, 12, 20, 257, "normal", ("fwd",), 42)
    a, b = generate(wl), generate(wl)
    want = np.float32 if dtype == "fp32" else np.float16
    for k in ("x", "w", "bias", "dy"):
        assert a[k].dtype == want and np.array_equal(a[k], b[k])
    assert a["x"].shape == (257, 96) and a["dy"].shape == (257, 160)
    assert a["w"].shape == (20, 12, 8) and a["bias"].shape == (20,)
    other = generate(Workload("w", dtype, 8, 12, 20, 257, "normal", ("fwd",), 43))
    assert not np.array_equal(a["x"], other["x"])


def test_generate_bias_kinds_and_statistics():
    base = dict(dtype="fp32", T=4, Ci=64, Co=48, N=4096, passes=("fwd",), seed=7)
    assert generate(Workload(name="n", bias="none", **base))["bias"] is None
    z = generate(Workload(name="z", bias="zero", **base))["bias"]
    assert z.shape == (48,) and not z.any()
    d = generate(Workload(name="g", bias="normal", **base))
    # x, dy ~ N(0, 1); w ~ N(0, variance 1 / (Ci T)): unit-variance outputs for unit-variance inputs
    assert abs(float(d["x"].std()) - 1.0) < 0.02 and abs(float(d["dy"].mean())) < 0.02
    assert abs(float(d["w"].std()) * np.sqrt(64 * 4) - 1.0) < 0.05
    # the draws do not depend on the bias kind (same order, same stream)
    assert np.array_equal(d["x"], generate(Workload(name="z", bias="zero", **base))["x"])


def test_fp16_inputs_are_the_rounded_fp32_draws():
    kw = dict(T=4, Ci=8, Co=8, N=100, bias="normal", passes=("fwd",), seed=3)
    f32, f16 = generate(Workload(name="a", dtype="fp32", **kw)), generate(Workload(name="b", dtype="fp16", **kw))
    for k in ("x", "w", "bias", "dy"):
        assert np.array_equal(f32[k].astype(np.float16), f16[k])


def test_sample_rows():
    assert np.array_equal(sample_rows(5, 96), np.arange(5))
    r = sample_rows(32768, 96, seed=1)
    assert r[0] == 0 and r[-1] == 32767 and len(r) <= 96 and len(r) >= 90
    assert np.all(np.diff(r) > 0)                                             # sorted, no duplicates
    assert np.array_equal(r, sample_rows(32768, 96, seed=1)) and not np.array_equal(r, sample_rows(32768, 96, seed=2))


def test_with_tokens_keeps_everything_else():
    wl = CONFIGS[HEADLINE].with_tokens(100)
    assert wl.N == 100 and (wl.T, wl.Ci, wl.Co, wl.dtype) == (8, 96, 384, "fp16")
