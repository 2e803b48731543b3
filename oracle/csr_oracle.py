"""ctypes front end of the CPU oracle (``csr_oracle.c``) plus the storage-format step.

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the benchmark's CPU legs call this.
Nothing here is shared with, or imported by, the CUDA path.

Paper passages: Eq. 2-4 (matching pursuit), Eq. 12 (de-sparse), and the "Analysis for
CSR" paragraph (each kept entry is stored as an INT16 index and an fp16 coefficient, so a
vector of d_h channels costs 32*s*s_n bits).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "csr_oracle.c")
_LIB = os.path.join(_HERE, "libcsr_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP, no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, i32, p = ctypes.c_int64, ctypes.c_int, ctypes.c_void_p
        lib.csr_oracle_encode.argtypes = [p, p, i64, i32, i32, i32, p, p, p, p, p]
        lib.csr_oracle_encode.restype = None
        lib.csr_oracle_reconstruct.argtypes = [p, p, p, i64, i32, i32, i32, p]
        lib.csr_oracle_reconstruct.restype = None
        lib.csr_oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().csr_oracle_num_threads())


@dataclass
class MPResult:
    idx: np.ndarray       # [M][s] int32, selection order
    coef: np.ndarray      # [M][s] float64, signed
    gap: np.ndarray       # [M][s] relative gap between the two largest |correlations|
    resnorm: np.ndarray   # [M][s] ||R_{g+1}|| after iteration g
    residual: np.ndarray  # [M][d] R_s


def _f32c(a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype != np.float32:
        raise TypeError("the oracle takes fp32 bit patterns (widen bf16 to fp32 first)")
    return a


def mp_encode(D: np.ndarray, X: np.ndarray, s: int) -> MPResult:
    """Matching pursuit, Eq. 2-4.  D [N][d] fp32 (one atom per row), X [M][d] fp32."""
    D = _f32c(D)
    X = _f32c(X)
    N, d = D.shape
    M = X.shape[0]
    if X.ndim != 2 or X.shape[1] != d or s < 1:
        raise ValueError("shape mismatch")
    idx = np.empty((M, s), np.int32)
    coef = np.empty((M, s), np.float64)
    gap = np.empty((M, s), np.float64)
    resnorm = np.empty((M, s), np.float64)
    residual = np.empty((M, d), np.float64)
    if M:
        _load().csr_oracle_encode(D.ctypes.data, X.ctypes.data, M, d, N, s, idx.ctypes.data,
                                  coef.ctypes.data, gap.ctypes.data, resnorm.ctypes.data,
                                  residual.ctypes.data)
    return MPResult(idx, coef, gap, resnorm, residual)


def reconstruct(D: np.ndarray, idx: np.ndarray, coef: np.ndarray) -> np.ndarray:
    """De-sparse, Eq. 12: X_hat = sum over the stored entries of coef * atom (fp64)."""
    D = _f32c(D)
    N, d = D.shape
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    coef = np.ascontiguousarray(coef, dtype=np.float64)
    M, s = idx.shape
    if coef.shape != (M, s):
        raise ValueError("shape mismatch")
    if M and (idx.min() < 0 or idx.max() >= N):
        raise ValueError("index out of range")
    out = np.empty((M, d), np.float64)
    if M:
        _load().csr_oracle_reconstruct(D.ctypes.data, idx.ctypes.data, coef.ctypes.data, M, d, N, s,
                                       out.ctypes.data)
    return out


# --- chunks and the online part of a dictionary -------------------------------------------

def mp_encode_chunked(Ds, X: np.ndarray, s: int):
    """"KV Decomposition and Sparse Storage" with s_n = len(Ds) chunks: a head vector of d_h
    channels is cut into s_n consecutive pieces of d_h / s_n channels and piece c is encoded
    by matching pursuit over its own dictionary Ds[c] ([N_c][d_h / s_n]).  Returns one
    MPResult per chunk."""
    s_n = len(Ds)
    d_h = X.shape[1]
    if s_n < 1 or d_h % s_n:
        raise ValueError("d_h must be a multiple of the number of chunks")
    dc = d_h // s_n
    return [mp_encode(Ds[c], np.ascontiguousarray(X[:, c * dc:(c + 1) * dc]), s) for c in range(s_n)]


def reconstruct_chunked(Ds, idx_list, coef_list) -> np.ndarray:
    """Eq. 12 per chunk; the pieces are put back side by side."""
    return np.concatenate([reconstruct(Ds[c], idx_list[c], coef_list[c]) for c in range(len(Ds))], axis=1)


def dict_append(D: np.ndarray, N_cur: int, X: np.ndarray, rows) -> np.ndarray:
    """Online part of a dictionary ("Build dictionary": atoms sampled from the KV cache just
    computed; "NeuralDict": ReNorm keeps every atom at unit l2-norm).  Returns a copy of D
    ([N_cap][d] fp32) in which rows N_cur .. N_cur+len(rows)-1 are X[rows] divided by their
    l2-norm, computed in fp64 and rounded once to fp32; a zero row stays zero."""
    D = np.array(D, dtype=np.float32, copy=True)
    rows = np.asarray(rows, dtype=np.int64)
    if N_cur < 0 or N_cur + rows.size > D.shape[0]:
        raise ValueError("atoms do not fit")
    for i, r in enumerate(rows):
        x = np.asarray(X[r], np.float64)
        n = np.sqrt(np.sum(x * x))
        D[N_cur + i] = (x / n if n > 0 else x * 0).astype(np.float32)
    return D


# --- attention from the restored tensors ("De-Sparse to restore") ---------------------------

def key_scores(D: np.ndarray, Q: np.ndarray, idx: np.ndarray, coef: np.ndarray, scale: float = 1.0) -> np.ndarray:
    """scores[b][h][t] = scale * Q[b][h] . X~[b][t], with X~ = Eq. 12 restored from the codes
    [B][T][s]; Q is [B][H][d].  The restored tensor is formed explicitly, fp64 throughout."""
    B, T, s = idx.shape
    out = np.empty((B, Q.shape[1], T), np.float64)
    for b in range(B):
        xt = reconstruct(D, idx[b], coef[b])                  # [T][d]
        out[b] = scale * (np.asarray(Q[b], np.float64) @ xt.T)
    return out


def value_mix(D: np.ndarray, W: np.ndarray, idx: np.ndarray, coef: np.ndarray) -> np.ndarray:
    """out[b][h] = sum_t W[b][h][t] * X~[b][t] with X~ restored by Eq. 12; W is [B][H][T]."""
    B, T, s = idx.shape
    out = np.empty((B, W.shape[1], D.shape[1]), np.float64)
    for b in range(B):
        xt = reconstruct(D, idx[b], coef[b])
        out[b] = np.asarray(W[b], np.float64) @ xt
    return out


def decode_attention(Dk, Dv, Q, k_idx, k_coef, v_idx, v_coef, scale: float):
    """softmax_t(scale * Q . X~_K[t]) applied to X~_V, both tensors restored by Eq. 12; returns
    (out [B][H][d], weights [B][H][T]) in fp64."""
    sc = key_scores(Dk, Q, k_idx, k_coef, scale)
    sc = sc - sc.max(axis=2, keepdims=True)
    w = np.exp(sc)
    w /= w.sum(axis=2, keepdims=True)
    return value_mix(Dv, w, v_idx, v_coef), w


# --- one training step of the offline dictionary ("NeuralDict") -----------------------------

def mse_loss_and_grad(D: np.ndarray, X: np.ndarray, idx: np.ndarray, coef: np.ndarray):
    """L_MSE = sum_x ||x - W_D r(x)||^2 for given (fixed) codes, and its gradient with respect
    to the atoms, [N][d]: every stored entry (x, g) contributes -2 c_g (x - x^) to atom i_g."""
    Dd = np.asarray(D, np.float64)
    E = np.asarray(X, np.float64) - reconstruct(D, idx, coef)
    grad = np.zeros_like(Dd)
    for g in range(idx.shape[1]):
        np.add.at(grad, idx[:, g], -2.0 * coef[:, g][:, None] * E)
    return float(np.sum(E * E)), grad


def div_loss_and_grad(D: np.ndarray):
    """L_div = ||I - W^T W||_F^2 / N^2 (W = D^T, one atom per column) and its gradient
    (4 / N^2) (D D^T - I) D, [N][d]."""
    Dd = np.asarray(D, np.float64)
    N = Dd.shape[0]
    G = Dd @ Dd.T - np.eye(N)
    return float(np.sum(G * G) / N ** 2), (4.0 / N ** 2) * (G @ Dd)


def adaptive_beta(l_mse: float, l_div: float) -> float:
    """beta = min(0.1 * L_MSE / L_div, 1.0), from the last batch's loss values."""
    return 1.0 if l_div <= 0 else min(0.1 * l_mse / l_div, 1.0)


def dict_train_step(D: np.ndarray, X: np.ndarray, s: int, lr: float, beta: float):
    """One batch of TrainNeurDict (Algorithm 1): codes by matching pursuit over the current
    dictionary, L = L_MSE + beta * L_div differentiated with the codes held fixed, a plain
    gradient step and ReNorm.  Returns (new D as fp32, L_MSE, L_div, MPResult); the losses
    are those of the dictionary before the update."""
    res = mp_encode(D, X, s)
    l_mse, g_mse = mse_loss_and_grad(D, X, res.idx, res.coef)
    l_div, g_div = div_loss_and_grad(D)
    W = np.asarray(D, np.float64) - lr * (g_mse + beta * g_div)
    n = np.linalg.norm(W, axis=1, keepdims=True)
    W = np.where(n > 0, W / np.where(n > 0, n, 1.0), 0.0)
    return W.astype(np.float32), l_mse, l_div, res


# --- storage format ("Analysis for CSR") -------------------------------------------------

def pack_codes(idx: np.ndarray, coef: np.ndarray):
    """Stored form of r: 16-bit index and fp16 coefficient per kept entry.

    The coefficient goes fp64 -> fp32 -> fp16, round-to-nearest-even each time (the
    kernel's coefficient leaves its arithmetic as fp32).  Indices are kept unsigned so
    that dictionaries of up to 65536 atoms fit.
    """
    if idx.size and (idx.min() < 0 or idx.max() > 0xFFFF):
        raise ValueError("index does not fit 16 bits")
    return idx.astype(np.uint16), coef.astype(np.float32).astype(np.float16)


def unpack_codes(idx16: np.ndarray, coef16: np.ndarray):
    return idx16.astype(np.int32), coef16.astype(np.float64)


def code_bits_per_channel(d_h: int, s: int, s_n: int = 1) -> float:
    """Equivalent quantisation bits per channel: (16 + 16) * s * s_n / d_h."""
    return 32.0 * s * s_n / d_h


def code_bytes_per_vector(s: int, s_n: int = 1) -> int:
    return 4 * s * s_n


def relative_error(X: np.ndarray, X_hat: np.ndarray) -> np.ndarray:
    """Per-vector ||x - x_hat|| / ||x|| in fp64 (0 for a zero vector)."""
    X = np.asarray(X, np.float64)
    num = np.linalg.norm(X - np.asarray(X_hat, np.float64), axis=1)
    den = np.linalg.norm(X, axis=1)
    return np.where(den > 0, num / np.where(den > 0, den, 1.0), 0.0)
