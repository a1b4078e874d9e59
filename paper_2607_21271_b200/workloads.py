"""Seeded synthetic workloads: shapes and random tensors only, none of the method's arithmetic.

Both the CUDA path's tests/benchmarks and the CPU oracle's tests draw their inputs here so
that they see identical bytes.  The shapes follow the ViT / Swin token shapes of the paper's
model table (Table 6: ViT at 224x224, patch 16 -> 197 tokens; Swin stage 1 at patch 4 ->
56x56 tokens); activations, weights and upstream gradients are Gaussians standing in for the
ImageNet-100 activations the paper's network-level experiments use.
"""

from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    dtype: str            # "fp32" | "fp16" | "bf16"  (fp16 / bf16 = 16-bit I/O, float accumulate)
    T: int                # order of the cyclic group
    Ci: int               # input channels per group element
    Co: int               # output channels per group element
    N: int                # tokens
    bias: str             # "none" | "zero" | "normal"
    passes: tuple         # subset of ("fwd", "bwd_data", "bwd_weight")
    seed: int

    @property
    def Din(self) -> int:
        return self.Ci * self.T

    @property
    def Dout(self) -> int:
        return self.Co * self.T

    @property
    def np_dtype(self):
        """Host array type of the inputs.  numpy has no bfloat16: bf16 workloads are float32 arrays whose values are
        exactly representable in bfloat16 (the device copy is an exact narrowing)."""
        return np.float16 if self.dtype == "fp16" else np.float32

    def with_tokens(self, N: int) -> "Workload":
        return replace(self, N=N, name=f"{self.name}@N={N}")


_FB = ("fwd", "bwd_data", "bwd_weight")

CONFIGS = {
    "tiny_fp32": Workload("tiny_fp32", "fp32", 4, 8, 8, 64, "none", ("fwd",), 0),
    "vit_s_fp32": Workload("vit_s_fp32", "fp32", 8, 48, 48, 64 * 197, "normal", _FB, 1),
    "vit_b_fc1_fp16": Workload("vit_b_fc1_fp16", "fp16", 8, 96, 384, 128 * 197, "zero", _FB, 2),
    "swin_t_s1_fp16": Workload("swin_t_s1_fp16", "fp16", 4, 24, 96, 128 * 56 * 56, "normal", ("fwd",), 3),
    "sweep_T4_fp16": Workload("sweep_T4_fp16", "fp16", 4, 256, 256, 65536, "normal", _FB, 4),
    "sweep_T8_fp16": Workload("sweep_T8_fp16", "fp16", 8, 128, 128, 65536, "normal", _FB, 4),
    "sweep_T16_fp16": Workload("sweep_T16_fp16", "fp16", 16, 64, 64, 65536, "normal", _FB, 4),
    "sweep_T32_fp16": Workload("sweep_T32_fp16", "fp16", 32, 32, 32, 65536, "normal", _FB, 4),
}

# The configuration the headline metric is quoted on.
HEADLINE = "vit_b_fc1_fp16"

# The shapes of the paper's operator-level benchmark (Tables 1 and 2): batch 32 x 1024 tokens, the p4 group (T = 4),
# c channels per group element on both sides (total width C = D = 4c), bias, forward and full backward.  The wide
# ones are the compute-bound end of the path.  Too large for a full oracle pass: tests compare sampled outputs.
OPERATOR_SHAPES = {
    **{f"op_c{c}_fp16": Workload(f"op_c{c}_fp16", "fp16", 4, c, c, 32 * 1024, "normal", _FB, 5)
       for c in (16, 64, 256, 512, 1024, 2048)},
    **{f"op_c{c}_fp32": Workload(f"op_c{c}_fp32", "fp32", 4, c, c, 32 * 1024, "normal", _FB, 5)
       for c in (16, 64, 256, 512, 1024, 2048)},
}

# The other linear layers of the EQ-ViT-B block the headline layer (fc1) comes from, at the same token count: the fused
# q/k/v projection is ONE layer with three blocks of output channels (x is read and transformed once for all three),
# fc2 is the MLP's second layer (384 -> 96 channels per group element).
BLOCK_SHAPES = {
    "vit_b_qkv_fp16": Workload("vit_b_qkv_fp16", "fp16", 8, 96, 3 * 96, 128 * 197, "normal", _FB, 6),
    "vit_b_fc2_fp16": Workload("vit_b_fc2_fp16", "fp16", 8, 384, 96, 128 * 197, "normal", _FB, 7),
    # the headline layer with bfloat16 I/O
    "vit_b_fc1_bf16": Workload("vit_b_fc1_bf16", "bf16", 8, 96, 384, 128 * 197, "zero", _FB, 2),
}

ALL_WORKLOADS = {**CONFIGS, **OPERATOR_SHAPES, **BLOCK_SHAPES}


def generate(wl: Workload) -> dict:
    """Draw x, w, bias, dy for a workload, in this fixed order, from PCG64(seed).

    x  ~ N(0, 1)                    [N, Ci*T]   (group index fastest)
    w  ~ N(0, variance 1/(Ci*T))    [Co, Ci, T]
    b  ~ N(0, variance 0.02) | 0 | None   [Co]
    dy ~ N(0, 1)                    [N, Co*T]
    Values are drawn as float32 and, for fp16 workloads, rounded once to half precision
    (round-to-nearest-even); the returned arrays are exactly the bytes both sides consume.
    """
    g = np.random.Generator(np.random.PCG64(wl.seed))
    dt = wl.np_dtype
    if wl.dtype == "bf16":
        narrow = round_to_bf16
    else:
        def narrow(a):
            return a.astype(dt)
    x = g.standard_normal((wl.N, wl.Ci * wl.T), dtype=np.float32)
    w = g.standard_normal((wl.Co, wl.Ci, wl.T), dtype=np.float32) / np.float32(np.sqrt(wl.Ci * wl.T))
    b = g.standard_normal(wl.Co, dtype=np.float32) * np.float32(np.sqrt(0.02))
    dy = g.standard_normal((wl.N, wl.Co * wl.T), dtype=np.float32)
    if wl.bias == "none":
        bias = None
    elif wl.bias == "zero":
        bias = np.zeros(wl.Co, dtype=dt)
    else:
        bias = narrow(b)
    return {"x": narrow(x), "w": narrow(w), "bias": bias, "dy": narrow(dy)}


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """float32 values rounded to the nearest bfloat16 (ties to even), returned as float32."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(a.shape)


def sample_rows(N: int, count: int, seed: int = 0) -> np.ndarray:
    """A sorted, duplicate-free sample of token indices that always includes both ends."""
    if N <= count:
        return np.arange(N)
    g = np.random.Generator(np.random.PCG64(seed + 1234567))
    idx = g.choice(N, size=count - 2, replace=False)
    return np.unique(np.concatenate([[0, N - 1], idx]))
