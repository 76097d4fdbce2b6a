"""Seeded synthetic inputs for the fused linear + epilogue + row-norm operator.

Data preparation only: this module holds none of the operator's arithmetic and imports neither
the CUDA binding nor the CPU oracle, so both can be fed the same bit patterns from here.

The paper scores kernels on benchmark-suite tasks whose shapes it does not print (Section 4,
"Benchmarks"); the five configurations below stand in for them: dense i.i.d. Gaussian matrices
with the shapes, dtypes, scales and seeds of this build's target configurations.

Recipe: ``numpy.random.Generator(PCG64(seed)).standard_normal`` in float64, drawn in the order
X, W, bias, residual, gamma, beta (absent tensors are skipped), scaled (and shifted for gamma),
cast to float32, then for bf16 configurations rounded to nearest-even bf16 and kept as uint16
bit patterns.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest, ties to even); returns the uint16 bit patterns."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    bits = a.view(np.uint32)
    lsb = (bits >> np.uint32(16)) & np.uint32(1)
    rounded = bits + np.uint32(0x7FFF) + lsb
    out = (rounded >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(a)
    if nan.any():
        out[nan] = np.uint16(0x7FC0)
    return out


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to float32."""
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def to_f64(a: np.ndarray) -> np.ndarray:
    """Exact widening of a stored tensor (float32, float64 or bf16 bits) to float64."""
    if a.dtype == np.uint16:
        return bf16_bits_to_f32(a).astype(np.float64)
    return a.astype(np.float64)


@dataclass
class Problem:
    """One operator instance.  Arrays are float32, or uint16 bf16 bit patterns when dtype=='bf16'."""
    name: str
    dtype: str                      # "f32" | "bf16"
    M: int
    N: int
    K: int                          # 0 for stand-alone row ops (X is then [M,N])
    X: np.ndarray = None
    W: Optional[np.ndarray] = None
    bias: Optional[np.ndarray] = None
    residual: Optional[np.ndarray] = None
    gamma: Optional[np.ndarray] = None
    beta: Optional[np.ndarray] = None
    act: str = "none"
    scale: float = 1.0
    norm: str = "none"
    eps: float = 1e-5
    call: str = "linear_epilogue_rownorm"   # which entry point serves it
    seed: int = 0
    meta: dict = field(default_factory=dict)

    @property
    def flops(self) -> int:
        return 2 * self.M * self.N * self.K

    @property
    def algorithmic_bytes(self) -> int:
        """One read of every input plus one write of Y."""
        es = 4 if self.dtype == "f32" else 2
        total = self.M * self.N * es                      # Y
        for t in (self.X, self.W, self.bias, self.residual, self.gamma, self.beta):
            if t is not None:
                total += t.size * es
        return total


def _store(a64: np.ndarray, dtype: str) -> np.ndarray:
    a32 = a64.astype(np.float32)
    return f32_to_bf16_bits(a32) if dtype == "bf16" else a32


def make_problem(name, dtype, M, N, K, *, seed, std_x, std_w=None, bias_std=None, residual_std=None,
                 gamma_std=None, beta_std=None, act="none", scale=1.0, norm="none", eps=1e-5,
                 call="linear_epilogue_rownorm") -> Problem:
    """Draw one problem.  K == 0 makes a stand-alone row problem with X of shape [M,N]."""
    rng = np.random.Generator(np.random.PCG64(seed))
    p = Problem(name=name, dtype=dtype, M=M, N=N, K=K, act=act, scale=scale, norm=norm, eps=eps,
                call=call, seed=seed)
    if K > 0:
        p.X = _store(rng.standard_normal((M, K)) * std_x, dtype)
        p.W = _store(rng.standard_normal((N, K)) * (std_w if std_w is not None else std_x), dtype)
    else:
        p.X = _store(rng.standard_normal((M, N)) * std_x, dtype)
    if bias_std is not None:
        p.bias = _store(rng.standard_normal(N) * bias_std, dtype)
    if residual_std is not None:
        p.residual = _store(rng.standard_normal((M, N)) * residual_std, dtype)
    if gamma_std is not None:
        p.gamma = _store(1.0 + rng.standard_normal(N) * gamma_std, dtype)
    if beta_std is not None:
        p.beta = _store(rng.standard_normal(N) * beta_std, dtype)
    return p


def config(idx: int, *, rows: Optional[int] = None) -> Problem:
    """The five target configurations (1-based).  ``rows`` keeps only the first rows of X (and of
    the residual): rows are independent, so this is the same problem on fewer rows, drawn from
    the same stream."""
    if idx == 1:     # fp32 linear + bias + GELU(erf) + row softmax
        p = make_problem("C1_f32_linear_bias_gelu_softmax", "f32", 128, 256, 256, seed=0,
                         std_x=1.0 / 16.0, bias_std=1.0 / 16.0, act="gelu_erf", norm="softmax")
    elif idx == 2:   # bf16 row LayerNorm, memory bound
        p = make_problem("C2_bf16_row_layernorm", "bf16", 16384, 4096, 0, seed=1, std_x=1.0,
                         gamma_std=0.1, beta_std=0.1, norm="layernorm", eps=1e-5, call="row_layernorm")
    elif idx == 3:   # bf16 linear + bias + SiLU + scale 0.5 + residual
        p = make_problem("C3_bf16_linear_bias_silu_scale_residual", "bf16", 8192, 4096, 4096, seed=2,
                         std_x=0.02, bias_std=0.02, residual_std=0.02, act="silu", scale=0.5,
                         call="linear_epilogue")
    elif idx == 4:   # bf16 linear + bias + GELU(erf) + row LayerNorm over N=8192
        p = make_problem("C4_bf16_linear_bias_gelu_layernorm", "bf16", 4096, 8192, 2048, seed=3,
                         std_x=0.02, bias_std=0.02, gamma_std=0.1, beta_std=0.1, act="gelu_erf",
                         norm="layernorm", eps=1e-5)
    elif idx == 5:   # bf16 linear + row softmax over N=32768, large-magnitude logits
        p = make_problem("C5_bf16_linear_softmax", "bf16", 2048, 32768, 1024, seed=4,
                         std_x=8.0 / 32.0, norm="softmax")
    else:
        raise ValueError("config index must be 1..5")
    if rows is not None and rows < p.M:
        p.M = rows
        p.X = np.ascontiguousarray(p.X[:rows])
        if p.residual is not None:
            p.residual = np.ascontiguousarray(p.residual[:rows])
    return p


def take_rows(p: Problem, rows) -> Problem:
    """The same problem restricted to the given row indices (rows are independent)."""
    rows = np.asarray(rows, dtype=np.int64)
    q = Problem(**{**p.__dict__})
    q.M = int(rows.size)
    q.X = np.ascontiguousarray(p.X[rows])
    if p.residual is not None:
        q.residual = np.ascontiguousarray(p.residual[rows])
    return q


def to_torch(a, dtype: str, device="cuda"):
    """numpy float32 array, or uint16 bf16 bit patterns, -> torch tensor of that dtype on `device`."""
    import torch
    if a is None:
        return None
    if dtype == "bf16":
        return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16).to(device)
    return torch.from_numpy(np.ascontiguousarray(a)).to(device)


def problem_to_torch(p: Problem, device="cuda") -> dict:
    """The tensors of a problem on `device`, keyed X, W, bias, residual, gamma, beta (absent ones None)."""
    return {k: to_torch(getattr(p, k), p.dtype, device) for k in ("X", "W", "bias", "residual", "gamma", "beta")}
