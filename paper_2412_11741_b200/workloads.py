"""Seeded synthetic inputs shaped like the KV tensors the CSR paper encodes.

This module only draws random numbers and lays them out; it holds none of the codec's
arithmetic.  Both the CPU oracle's tests and the CUDA path's tests read their inputs from
here so that the two see identical bit patterns.

The paper runs on real prompts through Llama-2-7B-chat, Llama-3-8B-Instruct and
Baichuan2-7B (head size d_h = 128; 32 attention heads or 8 grouped KV heads; dictionary
sizes 2048-8192; MP levels 4-16).  Neither the prompts nor the weights are available
here, so Gaussian stand-ins of the same shapes are used.  Keys get a few large "outlier"
channels per head, the structure the paper's observation section describes for key
caches; values are plain Gaussians.

All dictionaries are [N][d] fp32, one atom per row, rows normalised to unit l2 norm in
fp32.  "bf16" inputs are fp32 arrays whose values are exactly representable in bf16,
together with their 16-bit patterns.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np


# ---------------------------------------------------------------------------------------
# bf16 helpers (bit manipulation only)
# ---------------------------------------------------------------------------------------

def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (uint16), round to nearest even."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> fp32, exact."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    return from_bf16_bits(to_bf16_bits(x))


def normalise_rows(a: np.ndarray) -> np.ndarray:
    """Scale every row to unit l2 norm, in fp32 (the paper's ReNorm applied once)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    n = np.sqrt((a * a).sum(axis=1, keepdims=True, dtype=np.float32)).astype(np.float32)
    return (a / n).astype(np.float32)


# ---------------------------------------------------------------------------------------
# workload container
# ---------------------------------------------------------------------------------------

@dataclass
class Workload:
    name: str
    D: np.ndarray            # [N][d] fp32, unit-norm rows
    X: np.ndarray            # [M][d] fp32 values (bf16-exact when x_dtype == "bf16")
    s: int
    x_dtype: str             # "f32" or "bf16"
    meta: dict = field(default_factory=dict)

    @property
    def M(self) -> int:
        return int(self.X.shape[0])

    @property
    def N(self) -> int:
        return int(self.D.shape[0])

    @property
    def d(self) -> int:
        return int(self.D.shape[1])

    def X_bits(self) -> np.ndarray:
        """bf16 bit patterns of X (only for bf16 workloads)."""
        assert self.x_dtype == "bf16"
        return to_bf16_bits(self.X)


def _outlier_channels(rng: np.random.Generator, heads: int, d: int, per_head: int) -> np.ndarray:
    return np.stack([rng.choice(d, size=per_head, replace=False) for _ in range(heads)])


def _gauss(rng: np.random.Generator, rows: int, d: int) -> np.ndarray:
    out = np.empty((rows, d), np.float32)
    step = 1 << 16
    for r0 in range(0, rows, step):
        r1 = min(rows, r0 + step)
        out[r0:r1] = rng.standard_normal((r1 - r0, d), dtype=np.float32)
    return out


def _key_like_atoms(rng: np.random.Generator, n: int, d: int, chans: np.ndarray, scale: float) -> np.ndarray:
    a = _gauss(rng, n, d)
    heads = chans.shape[0]
    for j in range(n):
        a[j, chans[j % heads]] *= np.float32(scale)
    return a


def stratified_rows(M: int, n: int, seed: int = 0) -> np.ndarray:
    """n distinct row numbers spread evenly over [0, M): one random pick per stratum, so
    that every head and both the key and the value half of a workload are sampled."""
    n = min(n, M)
    if n == 0:
        return np.zeros(0, np.int64)
    rng = np.random.default_rng([seed, M, n])
    edges = np.linspace(0, M, n + 1).astype(np.int64)
    width = np.maximum(edges[1:] - edges[:-1], 1)
    return edges[:-1] + (rng.integers(0, 1 << 62, size=n) % width)


# ---------------------------------------------------------------------------------------
# the five configurations
# ---------------------------------------------------------------------------------------

def tiny(M: int = 4096, N: int = 1024, d: int = 128, s: int = 8, seed: int = 0) -> Workload:
    """Config 1: Gaussian fp32 atoms and inputs, followed by 64 vectors that are exact
    8-sparse combinations of distinct atoms with coefficients in +-[1, 2]."""
    rng = np.random.default_rng(seed)
    D = normalise_rows(_gauss(rng, N, d))
    X = _gauss(rng, M, d)
    n_sparse, k = 64, min(8, N)
    support = np.stack([rng.choice(N, size=k, replace=False) for _ in range(n_sparse)])
    amp = rng.uniform(1.0, 2.0, size=(n_sparse, k)) * rng.choice([-1.0, 1.0], size=(n_sparse, k))
    Xs = np.einsum("ik,ikd->id", amp, D[support].astype(np.float64)).astype(np.float32)
    return Workload("tiny", D, np.concatenate([X, Xs]), s, "f32",
                    {"sparse_rows": (M, M + n_sparse), "support": support, "amp": amp})


def _kv_workload(name: str, seed: int, groups: int, tokens: int, N: int, s: int, d: int = 128,
                 heads: int = 32, with_values: bool = True) -> Workload:
    """Keys: N(0,1) with 4 channels per head multiplied by 10; values: N(0,1).
    Row order: [kv][group (head or sequence x kv_head)][token]; the head of a group is
    group % heads.  Atoms come from an independent stream of the same distributions."""
    ss = np.random.SeedSequence(seed)
    s_chan, s_x, s_d = ss.spawn(3)
    chans = _outlier_channels(np.random.default_rng(s_chan), heads, d, 4)
    rng = np.random.default_rng(s_x)
    K = _gauss(rng, groups * tokens, d).reshape(groups, tokens, d)
    for g in range(groups):
        K[g][:, chans[g % heads]] *= np.float32(10.0)
    K = K.reshape(groups * tokens, d)
    parts = [K]
    if with_values:
        parts.append(_gauss(rng, groups * tokens, d))
    X = round_to_bf16(np.concatenate(parts) if len(parts) > 1 else K)
    rng_d = np.random.default_rng(s_d)
    n_key = N // 2 if with_values else N
    atoms = [_key_like_atoms(rng_d, n_key, d, chans, 10.0)]
    if with_values:
        atoms.append(_gauss(rng_d, N - n_key, d))
    D = normalise_rows(np.concatenate(atoms))
    return Workload(name, D, X, s, "bf16",
                    {"groups": groups, "tokens": tokens, "n_key_rows": groups * tokens,
                     "outlier_channels": chans})


def llama2_layer(tokens: int = 4096, N: int = 4096, s: int = 8) -> Workload:
    """Config 2: one Llama-2-7B-shaped layer at prefill, 32 heads x tokens x {K, V}."""
    return _kv_workload("llama2_7b_layer_prefill", 2, 32, tokens, N, s, heads=32)


def gqa_long(tokens: int = 16384, N: int = 8192, s: int = 16, seqs: int = 8, kv_heads: int = 8) -> Workload:
    """Config 3: 8 sequences x 16384 tokens x 8 KV heads x {K, V}."""
    return _kv_workload("gqa_long_context", 3, seqs * kv_heads, tokens, N, s, heads=kv_heads)


def sparsity_sweep(s: int, tokens: int = 32768, N: int = 8192) -> Workload:
    """Config 4: 2^20 key-like rows (32 heads), key-like atoms, s in {4, 8, 16, 32}."""
    w = _kv_workload("sparsity_sweep", 4, 32, tokens, N, s, heads=32, with_values=False)
    w.name = f"sparsity_sweep_s{s}"
    return w


def dict_sweep(N: int, d: int = 128, M: int = 1 << 20, s: int = 8) -> Workload:
    """Config 5: N(0,1) inputs with 2 % of the channels multiplied by 8; Gaussian atoms."""
    ss = np.random.SeedSequence([5, d])
    s_chan, s_x, s_d = ss.spawn(3)
    n_out = max(1, round(0.02 * d))
    chans = np.random.default_rng(s_chan).choice(d, size=n_out, replace=False)
    X = _gauss(np.random.default_rng(s_x), M, d)
    X[:, chans] *= np.float32(8.0)
    X = round_to_bf16(X)
    # draw the largest dictionary once and take a prefix, so that sizes nest
    D = normalise_rows(_gauss(np.random.default_rng(s_d), N, d))
    return Workload(f"dict_sweep_N{N}_d{d}", D, X, s, "bf16", {"outlier_channels": chans})
