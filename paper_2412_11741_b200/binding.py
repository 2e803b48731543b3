"""ctypes binding of libcsr.so: argument marshalling only.

Every function here has the name of the C entry point it forwards to (see include/csr.h).
torch is used for device memory and the current stream; no arithmetic of the codec is
done in Python.  If the shared library is missing or cannot be loaded the import of a
function fails loudly: there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
# CSR_LIBRARY_PATH selects another build of the same library (e.g. libcsr_debug.so, built with
# device-side index checks by `python -m paper_2412_11741_b200.build --debug`)
LIB_PATH = os.environ.get("CSR_LIBRARY_PATH") or os.path.join(_PKG, "libcsr.so")

CSR_OK = 0
CSR_ERR_INVALID_ARG = -1
CSR_ERR_UNSUPPORTED = -2
CSR_ERR_ALIGNMENT = -3
CSR_ERR_CUDA = -4
CSR_ERR_TIMEOUT = -5
CSR_ERR_WORKSPACE = -6
CSR_ERR_BOUNDS = -7

CSR_DTYPE_F32 = 0
CSR_DTYPE_BF16 = 1
CSR_DTYPE_F16 = 2

CSR_MODE_FP32_EXACT = 0
CSR_MODE_BF16_FAST = 1

EXPORTS = (
    "csr_encode", "csr_encode_ex", "csr_encode_workspace_bytes", "csr_reconstruct", "csr_reconstruct_ex",
    "csr_encode_host", "csr_reconstruct_host", "csr_encode_grouped", "csr_reconstruct_grouped", "csr_decode_attention", "csr_dict_append", "csr_dict_create", "csr_dict_destroy", "csr_dict_train_step", "csr_key_scores", "csr_pack_coefficients", "csr_value_mix",
    "csr_encode_static", "csr_dict_check_norms", "csr_set_option", "csr_device_status", "csr_release_workspace", "csr_last_error_string", "csr_version", "csr_debug_checks", "csr_debug_read",
)


class csr_encode_params_t(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32), ("mode", ctypes.c_int32),
        ("D", ctypes.c_void_p), ("X", ctypes.c_void_p),
        ("x_dtype", ctypes.c_int32), ("coef_dtype", ctypes.c_int32),
        ("M", ctypes.c_int64),
        ("d", ctypes.c_int32), ("N", ctypes.c_int32), ("s", ctypes.c_int32), ("reserved0", ctypes.c_int32),
        ("out_idx", ctypes.c_void_p), ("out_coef", ctypes.c_void_p),
        ("stream", ctypes.c_void_p), ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
        ("ldx", ctypes.c_int64), ("ld_code", ctypes.c_int64),
        ("dict", ctypes.c_void_p),
        ("dev_status", ctypes.c_void_p),
    ]


class csr_reconstruct_params_t(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32), ("reserved0", ctypes.c_int32),
        ("D", ctypes.c_void_p), ("idx", ctypes.c_void_p), ("coef", ctypes.c_void_p),
        ("coef_dtype", ctypes.c_int32), ("out_dtype", ctypes.c_int32),
        ("M", ctypes.c_int64),
        ("d", ctypes.c_int32), ("N", ctypes.c_int32), ("s", ctypes.c_int32), ("reserved1", ctypes.c_int32),
        ("X_hat", ctypes.c_void_p), ("stream", ctypes.c_void_p),
        ("ld_code", ctypes.c_int64), ("ld_xhat", ctypes.c_int64),
        ("dict", ctypes.c_void_p),
    ]


class csr_train_params_t(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32), ("mode", ctypes.c_int32),
        ("D", ctypes.c_void_p), ("X", ctypes.c_void_p),
        ("x_dtype", ctypes.c_int32), ("d", ctypes.c_int32), ("N", ctypes.c_int32), ("s", ctypes.c_int32),
        ("M", ctypes.c_int64),
        ("lr", ctypes.c_float), ("beta", ctypes.c_float),
        ("losses", ctypes.c_void_p), ("stream", ctypes.c_void_p),
    ]


class CsrError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"libcsr error {code}: {msg}")
        self.code = code


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libcsr.so (built in-tree by paper_2412_11741_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2412_11741_b200.build` "
                              "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i64, f32 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_float
        L.csr_encode.argtypes = [vp, vp, i64, i32, i32, i32, vp, vp]
        L.csr_encode.restype = i32
        L.csr_encode_ex.argtypes = [ctypes.POINTER(csr_encode_params_t)]
        L.csr_encode_ex.restype = i32
        L.csr_encode_host.argtypes = [ctypes.POINTER(csr_encode_params_t)]
        L.csr_encode_host.restype = i32
        L.csr_encode_static.argtypes = [vp, vp, i64, i32, i32, i32, vp, vp, vp, vp]
        L.csr_encode_static.restype = i32
        L.csr_encode_workspace_bytes.argtypes = [i32, i32, i32]
        L.csr_encode_workspace_bytes.restype = i64
        L.csr_reconstruct.argtypes = [vp, vp, vp, i64, i32, i32, i32, vp]
        L.csr_reconstruct.restype = i32
        L.csr_reconstruct_ex.argtypes = [ctypes.POINTER(csr_reconstruct_params_t)]
        L.csr_reconstruct_ex.restype = i32
        L.csr_reconstruct_host.argtypes = [ctypes.POINTER(csr_reconstruct_params_t)]
        L.csr_reconstruct_host.restype = i32
        L.csr_encode_grouped.argtypes = [ctypes.POINTER(csr_encode_params_t), i32]
        L.csr_encode_grouped.restype = i32
        L.csr_reconstruct_grouped.argtypes = [ctypes.POINTER(csr_reconstruct_params_t), i32]
        L.csr_reconstruct_grouped.restype = i32
        L.csr_dict_append.argtypes = [vp, i32, i32, i32, vp, i32, i64, i64, vp, i32, vp]
        L.csr_dict_append.restype = i32
        L.csr_key_scores.argtypes = [vp, i32, i32, vp, i32, i32, i32, vp, vp, i32, i64, i32, f32, vp, vp]
        L.csr_key_scores.restype = i32
        L.csr_value_mix.argtypes = [vp, i32, i32, vp, i32, i32, vp, vp, i32, i64, i32, vp, vp]
        L.csr_value_mix.restype = i32
        L.csr_decode_attention.argtypes = [vp, i32, vp, i32, i32, vp, i32, i32, i32, vp, vp, i32, vp, vp, i32, i32, i64, f32,
                                           vp, vp, vp]
        L.csr_decode_attention.restype = i32
        L.csr_pack_coefficients.argtypes = [vp, i64, vp, vp]
        L.csr_pack_coefficients.restype = i32
        L.csr_dict_create.argtypes = [vp, i32, i32, vp, ctypes.POINTER(vp)]
        L.csr_dict_create.restype = i32
        L.csr_dict_destroy.argtypes = [vp]
        L.csr_dict_destroy.restype = i32
        L.csr_dict_train_step.argtypes = [ctypes.POINTER(csr_train_params_t)]
        L.csr_dict_train_step.restype = i32
        L.csr_dict_check_norms.argtypes = [vp, i32, i32, f32, vp, ctypes.POINTER(f32)]
        L.csr_dict_check_norms.restype = i32
        L.csr_set_option.argtypes = [ctypes.c_char_p, i64]
        L.csr_set_option.restype = i32
        L.csr_device_status.argtypes = [vp]
        L.csr_device_status.restype = i32
        L.csr_release_workspace.argtypes = []
        L.csr_release_workspace.restype = i32
        L.csr_last_error_string.argtypes = []
        L.csr_last_error_string.restype = ctypes.c_char_p
        L.csr_version.argtypes = []
        L.csr_version.restype = i32
        L.csr_debug_checks.argtypes = []
        L.csr_debug_checks.restype = i32
        L.csr_debug_read.argtypes = [ctypes.c_char_p, ctypes.POINTER(ctypes.c_double)]
        L.csr_debug_read.restype = i32
        _lib = L
    return _lib


def csr_last_error_string() -> str:
    return lib().csr_last_error_string().decode()


def csr_version() -> int:
    return int(lib().csr_version())


def csr_debug_checks() -> bool:
    return bool(lib().csr_debug_checks())


def csr_debug_read(name: str) -> float:
    """A quantity only the checked build records (CSRError otherwise); reading resets it."""
    v = ctypes.c_double(0.0)
    _check(lib().csr_debug_read(name.encode(), ctypes.byref(v)))
    return v.value


def _check(rc: int) -> None:
    if rc != CSR_OK:
        raise CsrError(rc, csr_last_error_string())


_TORCH_DTYPE = {torch.float32: CSR_DTYPE_F32, torch.bfloat16: CSR_DTYPE_BF16, torch.float16: CSR_DTYPE_F16}


def _stream_ptr(t: torch.Tensor) -> int:
    return int(torch.cuda.current_stream(t.device).cuda_stream)


def csr_encode_workspace_bytes(mode: int, d: int, N: int) -> int:
    n = int(lib().csr_encode_workspace_bytes(mode, d, N))
    if n < 0:
        raise CsrError(n, csr_last_error_string())
    return n


def csr_pack_coefficients(coef32: torch.Tensor, coef16: Optional[torch.Tensor] = None) -> torch.Tensor:
    """csr_pack_coefficients: fp32 coefficients -> the stored fp16 form (round to nearest even)."""
    assert coef32.is_cuda and coef32.is_contiguous() and coef32.dtype == torch.float32
    if coef16 is None:
        coef16 = torch.empty(coef32.shape, dtype=torch.float16, device=coef32.device)
    assert coef16.is_contiguous() and coef16.dtype == torch.float16 and coef16.numel() == coef32.numel()
    with torch.cuda.device(coef32.device):
        _check(lib().csr_pack_coefficients(coef32.data_ptr(), coef32.numel(), coef16.data_ptr(), _stream_ptr(coef32)))
    return coef16


def csr_dict_create(D: torch.Tensor) -> int:
    """csr_dict_create: builds the fast mode's bf16 copy of D once (on torch's current stream);
    returns the handle to pass as `dict=` to csr_encode_ex.  Free it with csr_dict_destroy."""
    assert D.is_cuda and D.is_contiguous() and D.dtype == torch.float32 and D.dim() == 2
    h = ctypes.c_void_p()
    with torch.cuda.device(D.device):
        _check(lib().csr_dict_create(D.data_ptr(), D.shape[0], D.shape[1], _stream_ptr(D), ctypes.byref(h)))
    return h.value


def csr_dict_destroy(handle: int) -> None:
    _check(lib().csr_dict_destroy(handle))


def _encode_params(D, X, s, out_idx, out_coef, mode, stream, workspace) -> csr_encode_params_t:
    p = csr_encode_params_t()
    p.struct_size = ctypes.sizeof(csr_encode_params_t)
    p.mode = mode
    p.D = D.data_ptr()
    p.X = X.data_ptr()
    p.x_dtype = _TORCH_DTYPE[X.dtype]
    p.coef_dtype = _TORCH_DTYPE[out_coef.dtype]
    p.M = X.shape[0]
    p.d = D.shape[1]
    p.N = D.shape[0]
    p.s = s
    p.out_idx = out_idx.data_ptr()
    p.out_coef = out_coef.data_ptr()
    p.stream = stream
    if X.dim() == 2 and X.shape[0] > 1 and X.stride(0) != X.shape[1]:
        p.ldx = X.stride(0)
    if out_idx.shape[0] > 1 and out_idx.stride(0) != s:
        assert out_coef.stride(0) == out_idx.stride(0), "out_idx and out_coef must share their row stride"
        p.ld_code = out_idx.stride(0)
    elif out_idx.data_ptr() % 16 or out_coef.data_ptr() % 16:
        p.ld_code = s                                     # a view into wider arrays: element alignment is enough
    if workspace is not None:
        p.workspace = workspace.data_ptr()
        p.workspace_bytes = workspace.numel() * workspace.element_size()
    return p


def csr_encode_ex(D: torch.Tensor, X: torch.Tensor, s: int, *, mode: int = CSR_MODE_BF16_FAST,
                  coef_dtype: torch.dtype = torch.float16, out_idx: Optional[torch.Tensor] = None,
                  out_coef: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                  dict: Optional[int] = None, dev_status: Optional[torch.Tensor] = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """csr_encode_ex on CUDA tensors: D [N][d] fp32, X [M][d] fp32 or bf16.
    Returns (idx [M][s] uint16, coef [M][s] coef_dtype); runs on torch's current stream.
    dev_status: optional int32/uint32 CUDA tensor of one element that receives the wait status."""
    assert D.is_cuda and X.is_cuda and D.is_contiguous() and X.dim() == 2 and X.stride(1) == 1
    assert D.dtype == torch.float32 and D.dim() == 2 and X.shape[1] == D.shape[1]
    M = X.shape[0]
    if out_idx is None:
        out_idx = torch.empty((M, s), dtype=torch.uint16, device=X.device)
    if out_coef is None:
        out_coef = torch.empty((M, s), dtype=coef_dtype, device=X.device)
    p = _encode_params(D, X, s, out_idx, out_coef, mode, _stream_ptr(X), workspace)
    if dict is not None:
        p.dict = dict
    if dev_status is not None:
        assert dev_status.is_cuda and dev_status.element_size() == 4 and dev_status.numel() >= 1
        p.dev_status = dev_status.data_ptr()
    with torch.cuda.device(X.device):
        _check(lib().csr_encode_ex(ctypes.byref(p)))
    return out_idx, out_coef


def csr_encode(D: torch.Tensor, X: torch.Tensor, s: int, out_idx: Optional[torch.Tensor] = None,
               out_coef: Optional[torch.Tensor] = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """The 8-argument csr_encode: bf16 X, fp16 coefficients, fast mode, legacy default stream."""
    assert D.is_cuda and X.is_cuda and D.is_contiguous() and X.is_contiguous()
    assert D.dtype == torch.float32 and X.dtype == torch.bfloat16
    M, d = X.shape
    N = D.shape[0]
    if out_idx is None:
        out_idx = torch.empty((M, s), dtype=torch.uint16, device=X.device)
    if out_coef is None:
        out_coef = torch.empty((M, s), dtype=torch.float16, device=X.device)
    with torch.cuda.device(X.device):
        _check(lib().csr_encode(D.data_ptr(), X.data_ptr(), M, d, N, s, out_idx.data_ptr(), out_coef.data_ptr()))
    return out_idx, out_coef


def csr_encode_static(D: torch.Tensor, X: torch.Tensor, s: int, out_idx: torch.Tensor, out_coef: torch.Tensor,
                      dev_status: Optional[torch.Tensor] = None) -> None:
    """csr_encode_static: the fast encode for callers that must not allocate.  Outputs are
    passed in (this wrapper allocates nothing either); runs on torch's current stream."""
    assert D.is_cuda and X.is_cuda and D.is_contiguous() and X.is_contiguous()
    assert D.dtype == torch.float32 and X.dtype == torch.bfloat16
    assert out_idx.dtype == torch.uint16 and out_coef.dtype == torch.float16
    M, d = X.shape
    assert tuple(out_idx.shape) == (M, s) and tuple(out_coef.shape) == (M, s)
    st = None if dev_status is None else dev_status.data_ptr()
    with torch.cuda.device(X.device):
        _check(lib().csr_encode_static(D.data_ptr(), X.data_ptr(), M, d, D.shape[0], s, out_idx.data_ptr(),
                                       out_coef.data_ptr(), _stream_ptr(X), st))


def csr_encode_host(D: torch.Tensor, X_host: torch.Tensor, s: int, out_idx_host: torch.Tensor,
                    out_coef_host: torch.Tensor, *, mode: int = CSR_MODE_BF16_FAST, dict: Optional[int] = None) -> None:
    """csr_encode_host: D on the device; X and the outputs are host tensors (pinned for speed).
    Returns after the codes have arrived in the host tensors."""
    assert D.is_cuda and not X_host.is_cuda and not out_idx_host.is_cuda and not out_coef_host.is_cuda
    assert X_host.is_contiguous() and out_idx_host.is_contiguous() and out_coef_host.is_contiguous()
    assert out_idx_host.dtype == torch.uint16 and tuple(out_idx_host.shape) == (X_host.shape[0], s)
    p = _encode_params(D, X_host, s, out_idx_host, out_coef_host, mode, None, None)
    if dict is not None:
        p.dict = dict
    with torch.cuda.device(D.device):
        _check(lib().csr_encode_host(ctypes.byref(p)))


def _reconstruct_params(D, idx, coef, out_dtype, X_hat):
    assert D.is_cuda and idx.is_cuda and coef.is_cuda
    assert D.is_contiguous() and idx.stride(1) == 1 and coef.stride(1) == 1
    assert D.dtype == torch.float32 and idx.dtype == torch.uint16 and idx.shape == coef.shape
    M, s = idx.shape
    N, d = D.shape
    if X_hat is None:
        X_hat = torch.empty((M, d), dtype=out_dtype, device=D.device)
    assert tuple(X_hat.shape) == (M, d) and X_hat.stride(1) == 1
    p = csr_reconstruct_params_t()
    p.struct_size = ctypes.sizeof(csr_reconstruct_params_t)
    p.D = D.data_ptr()
    p.idx = idx.data_ptr()
    p.coef = coef.data_ptr()
    p.coef_dtype = _TORCH_DTYPE[coef.dtype]
    p.out_dtype = _TORCH_DTYPE[X_hat.dtype]
    p.M, p.d, p.N, p.s = M, d, N, s
    p.X_hat = X_hat.data_ptr()
    p.stream = _stream_ptr(D)
    if M > 1 and idx.stride(0) != s:
        assert coef.stride(0) == idx.stride(0), "idx and coef must share their row stride"
        p.ld_code = idx.stride(0)
    elif idx.data_ptr() % 16 or coef.data_ptr() % 16:
        p.ld_code = s                                     # a view into wider arrays: element alignment is enough
    if M > 1 and X_hat.stride(0) != d:
        p.ld_xhat = X_hat.stride(0)
    return p, X_hat


def csr_encode_grouped(problems, *, mode: int = CSR_MODE_BF16_FAST) -> None:
    """csr_encode_grouped: `problems` is a sequence of (D, X, s, out_idx, out_coef) or
    (D, X, s, out_idx, out_coef, dict) with CUDA tensors (dict: a csr_dict_create handle of D);
    X, out_idx and out_coef may be column slices of wider arrays (row strides are passed on).
    All problems are validated before any is enqueued; neighbouring fast-mode problems that
    each bring a handle are enqueued side by side."""
    arr = (csr_encode_params_t * len(problems))()
    for i, prob in enumerate(problems):
        D, X, s, out_idx, out_coef = prob[:5]
        assert D.is_cuda and X.is_cuda and D.is_contiguous() and X.stride(1) == 1 and D.dtype == torch.float32
        assert out_idx.dtype == torch.uint16 and out_idx.stride(1) == 1 and out_coef.stride(1) == 1
        arr[i] = _encode_params(D, X, s, out_idx, out_coef, mode, _stream_ptr(X), None)
        if len(prob) > 5 and prob[5] is not None:
            arr[i].dict = prob[5]
    if len(problems):
        with torch.cuda.device(problems[0][0].device):
            _check(lib().csr_encode_grouped(arr, len(problems)))


def csr_reconstruct_grouped(problems) -> None:
    """csr_reconstruct_grouped: `problems` is a sequence of (D, idx, coef, X_hat)."""
    arr = (csr_reconstruct_params_t * len(problems))()
    for i, (D, idx, coef, X_hat) in enumerate(problems):
        arr[i], _ = _reconstruct_params(D, idx, coef, X_hat.dtype, X_hat)
    if len(problems):
        with torch.cuda.device(problems[0][0].device):
            _check(lib().csr_reconstruct_grouped(arr, len(problems)))


def csr_dict_append(D: torch.Tensor, N_cur: int, X: torch.Tensor, rows: torch.Tensor) -> int:
    """csr_dict_append: writes normalised copies of X[rows] as atoms N_cur .. N_cur+len(rows)-1 of
    D ([N_cap][d] fp32, CUDA); rows is an int64 CUDA tensor.  Returns the new atom count."""
    assert D.is_cuda and X.is_cuda and rows.is_cuda and D.is_contiguous() and D.dtype == torch.float32
    assert X.dim() == 2 and X.stride(1) == 1 and rows.dtype == torch.int64 and rows.is_contiguous()
    n = int(rows.numel())
    with torch.cuda.device(D.device):
        _check(lib().csr_dict_append(D.data_ptr(), N_cur, D.shape[0], D.shape[1], X.data_ptr(), _TORCH_DTYPE[X.dtype],
                                     X.shape[0], X.stride(0) if X.shape[0] > 1 else 0, rows.data_ptr(), n,
                                     _stream_ptr(D)))
    return N_cur + n


def _check_codes(D, idx, coef):
    assert D.is_cuda and D.is_contiguous() and D.dtype == torch.float32
    assert idx.is_cuda and coef.is_cuda and idx.is_contiguous() and coef.is_contiguous()
    assert idx.dtype == torch.uint16 and idx.dim() == 3 and idx.shape == coef.shape


def csr_key_scores(D: torch.Tensor, Q: torch.Tensor, idx: torch.Tensor, coef: torch.Tensor, scale: float = 1.0,
                   scores: Optional[torch.Tensor] = None) -> torch.Tensor:
    """csr_key_scores: Q [B][H][d] (fp32 or bf16), codes [B][T][s]; returns scores [B][H][T] fp32."""
    _check_codes(D, idx, coef)
    B, T, s = idx.shape
    N, d = D.shape
    assert Q.is_cuda and Q.is_contiguous() and Q.dim() == 3 and Q.shape[0] == B and Q.shape[2] == d
    H = Q.shape[1]
    if scores is None:
        scores = torch.empty((B, H, T), dtype=torch.float32, device=D.device)
    assert scores.is_contiguous() and scores.dtype == torch.float32 and tuple(scores.shape) == (B, H, T)
    with torch.cuda.device(D.device):
        _check(lib().csr_key_scores(D.data_ptr(), N, d, Q.data_ptr(), _TORCH_DTYPE[Q.dtype], B, H, idx.data_ptr(),
                                    coef.data_ptr(), _TORCH_DTYPE[coef.dtype], T, s, float(scale), scores.data_ptr(),
                                    _stream_ptr(D)))
    return scores


def csr_value_mix(D: torch.Tensor, W: torch.Tensor, idx: torch.Tensor, coef: torch.Tensor,
                  out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """csr_value_mix: W [B][H][T] fp32 attention weights, codes [B][T][s]; returns [B][H][d] fp32."""
    _check_codes(D, idx, coef)
    B, T, s = idx.shape
    N, d = D.shape
    assert W.is_cuda and W.is_contiguous() and W.dtype == torch.float32 and W.dim() == 3
    assert W.shape[0] == B and W.shape[2] == T
    H = W.shape[1]
    if out is None:
        out = torch.empty((B, H, d), dtype=torch.float32, device=D.device)
    assert out.is_contiguous() and out.dtype == torch.float32 and tuple(out.shape) == (B, H, d)
    with torch.cuda.device(D.device):
        _check(lib().csr_value_mix(D.data_ptr(), N, d, W.data_ptr(), B, H, idx.data_ptr(), coef.data_ptr(),
                                   _TORCH_DTYPE[coef.dtype], T, s, out.data_ptr(), _stream_ptr(D)))
    return out


def csr_dict_train_step(D: torch.Tensor, X: torch.Tensor, s: int, lr: float, beta: float, *,
                        mode: int = CSR_MODE_FP32_EXACT, losses: Optional[torch.Tensor] = None) -> torch.Tensor:
    """csr_dict_train_step: updates D ([N][d] fp32, CUDA) in place on the batch X ([M][d]);
    returns the device tensor [L_MSE, L_div] (float64) of the dictionary before the update."""
    assert D.is_cuda and X.is_cuda and D.is_contiguous() and X.is_contiguous() and D.dtype == torch.float32
    assert X.dim() == 2 and X.shape[1] == D.shape[1]
    if losses is None:
        losses = torch.empty(2, dtype=torch.float64, device=D.device)
    assert losses.dtype == torch.float64 and losses.numel() >= 2 and losses.is_cuda
    p = csr_train_params_t()
    p.struct_size = ctypes.sizeof(csr_train_params_t)
    p.mode = mode
    p.D = D.data_ptr()
    p.X = X.data_ptr()
    p.x_dtype = _TORCH_DTYPE[X.dtype]
    p.d, p.N, p.s, p.M = D.shape[1], D.shape[0], s, X.shape[0]
    p.lr, p.beta = float(lr), float(beta)
    p.losses = losses.data_ptr()
    p.stream = _stream_ptr(D)
    with torch.cuda.device(D.device):
        _check(lib().csr_dict_train_step(ctypes.byref(p)))
    return losses


def csr_decode_attention(Dk: torch.Tensor, Dv: torch.Tensor, Q: torch.Tensor, k_idx: torch.Tensor, k_coef: torch.Tensor,
                         v_idx: torch.Tensor, v_coef: torch.Tensor, scale: float,
                         weights: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None):
    """csr_decode_attention: softmax(scale * Q K~^T) V~ straight from the codes.  Q [B][H][d]; key
    codes [B][T][sk], value codes [B][T][sv]; returns (out [B][H][d], weights [B][H][T]), fp32."""
    _check_codes(Dk, k_idx, k_coef)
    _check_codes(Dv, v_idx, v_coef)
    B, T, sk = k_idx.shape
    sv = v_idx.shape[2]
    d = Dk.shape[1]
    assert v_idx.shape[:2] == (B, T) and Dv.shape[1] == d and k_coef.dtype == v_coef.dtype
    assert Q.is_cuda and Q.is_contiguous() and Q.dim() == 3 and Q.shape[0] == B and Q.shape[2] == d
    H = Q.shape[1]
    if weights is None:
        weights = torch.empty((B, H, T), dtype=torch.float32, device=Dk.device)
    if out is None:
        out = torch.empty((B, H, d), dtype=torch.float32, device=Dk.device)
    assert weights.is_contiguous() and weights.dtype == torch.float32 and tuple(weights.shape) == (B, H, T)
    assert out.is_contiguous() and out.dtype == torch.float32 and tuple(out.shape) == (B, H, d)
    with torch.cuda.device(Dk.device):
        _check(lib().csr_decode_attention(Dk.data_ptr(), Dk.shape[0], Dv.data_ptr(), Dv.shape[0], d, Q.data_ptr(),
                                          _TORCH_DTYPE[Q.dtype], B, H, k_idx.data_ptr(), k_coef.data_ptr(), sk,
                                          v_idx.data_ptr(), v_coef.data_ptr(), sv, _TORCH_DTYPE[k_coef.dtype], T,
                                          float(scale), weights.data_ptr(), out.data_ptr(), _stream_ptr(Dk)))
    return out, weights


def csr_reconstruct_ex(D: torch.Tensor, idx: torch.Tensor, coef: torch.Tensor, *,
                       out_dtype: torch.dtype = torch.bfloat16,
                       X_hat: Optional[torch.Tensor] = None, dict: Optional[int] = None) -> torch.Tensor:
    """csr_reconstruct_ex on CUDA tensors; returns X_hat [M][d].  dict: a csr_dict_create handle of
    D, to gather bf16 atoms."""
    p, X_hat = _reconstruct_params(D, idx, coef, out_dtype, X_hat)
    if dict is not None:
        p.dict = dict
    with torch.cuda.device(D.device):
        _check(lib().csr_reconstruct_ex(ctypes.byref(p)))
    return X_hat


def csr_reconstruct_host(D: torch.Tensor, idx_host: torch.Tensor, coef_host: torch.Tensor,
                         X_hat_host: torch.Tensor, *, dict: Optional[int] = None) -> None:
    """csr_reconstruct_host: D on the device; the codes and X_hat are host tensors (pinned for
    speed).  Returns after X_hat has arrived in the host tensor."""
    assert D.is_cuda and not idx_host.is_cuda and not coef_host.is_cuda and not X_hat_host.is_cuda
    assert idx_host.is_contiguous() and coef_host.is_contiguous() and X_hat_host.is_contiguous()
    assert D.dtype == torch.float32 and idx_host.dtype == torch.uint16 and idx_host.shape == coef_host.shape
    M, s = idx_host.shape
    N, d = D.shape
    assert tuple(X_hat_host.shape) == (M, d)
    p = csr_reconstruct_params_t()
    p.struct_size = ctypes.sizeof(csr_reconstruct_params_t)
    p.D = D.data_ptr()
    p.idx = idx_host.data_ptr()
    p.coef = coef_host.data_ptr()
    p.coef_dtype = _TORCH_DTYPE[coef_host.dtype]
    p.out_dtype = _TORCH_DTYPE[X_hat_host.dtype]
    p.M, p.d, p.N, p.s = M, d, N, s
    p.X_hat = X_hat_host.data_ptr()
    if dict is not None:
        p.dict = dict
    with torch.cuda.device(D.device):
        _check(lib().csr_reconstruct_host(ctypes.byref(p)))


def csr_reconstruct(D: torch.Tensor, idx: torch.Tensor, coef: torch.Tensor,
                    X_hat: Optional[torch.Tensor] = None) -> torch.Tensor:
    """The 8-argument csr_reconstruct: fp16 coefficients in, bf16 X_hat out, legacy default stream."""
    assert D.is_cuda and D.dtype == torch.float32 and idx.dtype == torch.uint16 and coef.dtype == torch.float16
    M, s = idx.shape
    N, d = D.shape
    if X_hat is None:
        X_hat = torch.empty((M, d), dtype=torch.bfloat16, device=D.device)
    with torch.cuda.device(D.device):
        _check(lib().csr_reconstruct(D.data_ptr(), idx.data_ptr(), coef.data_ptr(), M, d, N, s, X_hat.data_ptr()))
    return X_hat


def csr_dict_check_norms(D: torch.Tensor, tol: float = -1.0) -> float:
    """csr_dict_check_norms: returns max_n | ||D[n]|| - 1 | (synchronises torch's current stream);
    raises CsrError if it exceeds tol (tol < 0: report only)."""
    assert D.is_cuda and D.is_contiguous() and D.dtype == torch.float32 and D.dim() == 2
    out = ctypes.c_float(0.0)
    with torch.cuda.device(D.device):
        _check(lib().csr_dict_check_norms(D.data_ptr(), D.shape[0], D.shape[1], float(tol), _stream_ptr(D), ctypes.byref(out)))
    return float(out.value)


def csr_set_option(name: str, value: int) -> None:
    """csr_set_option: process-wide tuning / diagnostic switches (see include/csr.h)."""
    _check(lib().csr_set_option(name.encode(), int(value)))


def csr_device_status(device=None) -> int:
    """Synchronises torch's current stream and returns CSR_OK or CSR_ERR_TIMEOUT."""
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    with torch.cuda.device(dev):
        return int(lib().csr_device_status(int(torch.cuda.current_stream(dev).cuda_stream)))


def csr_release_workspace() -> None:
    _check(lib().csr_release_workspace())
