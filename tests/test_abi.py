"""The C-ABI library builds, loads and exports every symbol include/csr.h declares; the
host-side argument checks answer without touching a GPU."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2412_11741_b200 import build
    build.build()
    from paper_2412_11741_b200 import binding
    return binding.lib()


def _declared_functions():
    src = open(os.path.join(ROOT, "include", "csr.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(csr_[a-z_]+)\s*\(", src)))


def test_exports_match_header(lib):
    from paper_2412_11741_b200 import binding
    names = _declared_functions()
    assert names, "no declarations found"
    for n in names:
        assert hasattr(lib, n), f"{n} declared in csr.h but not exported"
    assert sorted(binding.EXPORTS) == names


def test_version_and_struct_sizes(lib):
    from paper_2412_11741_b200 import binding
    assert binding.csr_version() == 120
    assert ctypes.sizeof(binding.csr_encode_params_t) == 128
    assert ctypes.sizeof(binding.csr_reconstruct_params_t) == 104


def _params(binding, **kw):
    p = binding.csr_encode_params_t()
    p.struct_size = ctypes.sizeof(p)
    p.mode = binding.CSR_MODE_BF16_FAST
    p.D, p.X, p.out_idx, p.out_coef = 0x1000, 0x2000, 0x3000, 0x4000
    p.x_dtype, p.coef_dtype = binding.CSR_DTYPE_BF16, binding.CSR_DTYPE_F16
    p.M, p.d, p.N, p.s = 1024, 128, 1024, 8
    for k, v in kw.items():
        setattr(p, k, v)
    return p


@pytest.mark.parametrize("kw,code", [
    (dict(d=96), -2), (dict(N=0), -1), (dict(N=70000), -1), (dict(s=0), -1), (dict(s=65), -1), (dict(M=-1), -1),
    (dict(D=0), -1), (dict(X=0), -1), (dict(out_idx=0), -1), (dict(D=0x1008), -3),
    (dict(X=0x2004), -3), (dict(mode=7), -1), (dict(x_dtype=3), -1), (dict(coef_dtype=1), -1),
    (dict(struct_size=8), -1), (dict(workspace=0x5008), -3), (dict(dev_status=0x6002), -3),
])
def test_encode_argument_errors(lib, kw, code):
    from paper_2412_11741_b200 import binding
    p = _params(binding, **kw)
    assert lib.csr_encode_ex(ctypes.byref(p)) == code
    assert binding.csr_last_error_string() != ""


def test_null_params_and_empty_input(lib):
    from paper_2412_11741_b200 import binding
    assert lib.csr_encode_ex(None) == binding.CSR_ERR_INVALID_ARG
    assert lib.csr_reconstruct_ex(None) == binding.CSR_ERR_INVALID_ARG
    # M == 0 is a successful no-op (no device work, no allocation)
    p = _params(binding, M=0, X=0, out_idx=0, out_coef=0)
    assert lib.csr_encode_ex(ctypes.byref(p)) == binding.CSR_OK
    assert lib.csr_encode(0x1000, 0, 0, 128, 1024, 8, 0, 0) == binding.CSR_OK
    assert lib.csr_reconstruct(0x1000, 0, 0, 0, 128, 1024, 8, 0) == binding.CSR_OK


def test_reconstruct_argument_errors(lib):
    from paper_2412_11741_b200 import binding
    assert lib.csr_reconstruct(0x1000, 0x2000, 0x3000, 10, 100, 1024, 8, 0x4000) == binding.CSR_ERR_UNSUPPORTED
    assert lib.csr_reconstruct(0x1000, 0x2000, 0x3000, 10, 128, 1024, 0, 0x4000) == binding.CSR_ERR_INVALID_ARG
    assert lib.csr_reconstruct(0x1000, 0x2002, 0x3000, 10, 128, 1024, 8, 0x4000) == binding.CSR_ERR_ALIGNMENT
    assert lib.csr_reconstruct(0, 0x2000, 0x3000, 10, 128, 1024, 8, 0x4000) == binding.CSR_ERR_INVALID_ARG


def test_stride_and_group_argument_errors(lib):
    from paper_2412_11741_b200 import binding
    assert lib.csr_encode_ex(ctypes.byref(_params(binding, ldx=64))) == binding.CSR_ERR_INVALID_ARG      # < d
    assert lib.csr_encode_ex(ctypes.byref(_params(binding, ld_code=4))) == binding.CSR_ERR_INVALID_ARG   # < s
    assert lib.csr_encode_ex(ctypes.byref(_params(binding, ldx=132))) == binding.CSR_ERR_ALIGNMENT       # rows off 16 B
    assert lib.csr_encode_host(ctypes.byref(_params(binding, ldx=256))) == binding.CSR_ERR_UNSUPPORTED
    assert lib.csr_encode_grouped(None, 1) == binding.CSR_ERR_INVALID_ARG
    assert lib.csr_encode_grouped(None, 0) == binding.CSR_OK
    arr = (binding.csr_encode_params_t * 2)(_params(binding, M=0, X=0, out_idx=0, out_coef=0), _params(binding, d=96))
    assert lib.csr_encode_grouped(arr, 2) == binding.CSR_ERR_UNSUPPORTED      # second problem invalid: nothing runs
    assert lib.csr_reconstruct_grouped(None, 0) == binding.CSR_OK
    # dict_append: capacity, dtype and alignment are checked before any device work
    f = lib.csr_dict_append
    assert f(0x1000, 10, 16, 128, 0x2000, 0, 100, 0, 0x3000, 7, None) == binding.CSR_ERR_INVALID_ARG    # 10 + 7 > 16
    assert f(0x1000, 0, 16, 96, 0x2000, 0, 100, 0, 0x3000, 4, None) == binding.CSR_ERR_UNSUPPORTED
    assert f(0x1000, 0, 16, 128, 0x2000, 7, 100, 0, 0x3000, 4, None) == binding.CSR_ERR_INVALID_ARG     # unknown dtype
    assert f(0x1000, 0, 16, 128, 0x2004, 0, 100, 0, 0x3000, 4, None) == binding.CSR_ERR_ALIGNMENT
    assert f(0x1000, 0, 16, 128, 0x2000, 0, 100, 0, 0x3000, 0, None) == binding.CSR_OK                  # nothing to add


def test_dict_handle_argument_errors(lib):
    from paper_2412_11741_b200 import binding
    h = ctypes.c_void_p()
    assert lib.csr_dict_create(0x1000, 1024, 96, None, ctypes.byref(h)) == binding.CSR_ERR_UNSUPPORTED
    assert lib.csr_dict_create(0, 1024, 128, None, ctypes.byref(h)) == binding.CSR_ERR_INVALID_ARG
    assert lib.csr_dict_create(0x1000, 1024, 128, None, None) == binding.CSR_ERR_INVALID_ARG
    assert lib.csr_dict_destroy(None) == binding.CSR_OK


def test_workspace_query(lib):
    from paper_2412_11741_b200 import binding
    assert binding.csr_encode_workspace_bytes(binding.CSR_MODE_FP32_EXACT, 128, 8192) == 0
    n = binding.csr_encode_workspace_bytes(binding.CSR_MODE_BF16_FAST, 128, 8192)
    assert 8192 * 128 * 2 <= n <= 8192 * 128 * 2 + 4096
    with pytest.raises(binding.CsrError):
        binding.csr_encode_workspace_bytes(binding.CSR_MODE_BF16_FAST, 100, 8192)


def test_options_and_norm_check_argument_errors(lib):
    from paper_2412_11741_b200 import binding
    assert lib.csr_set_option(b"fast_group", 4) == binding.CSR_OK
    assert lib.csr_set_option(b"fast_group", 0) == binding.CSR_OK
    assert lib.csr_set_option(b"fast_group", 3) == binding.CSR_ERR_INVALID_ARG
    assert lib.csr_set_option(b"fast_split", 3) == binding.CSR_ERR_INVALID_ARG
    assert lib.csr_set_option(b"exact_split", -1) == binding.CSR_ERR_INVALID_ARG
    assert lib.csr_set_option(b"wait_limit_ns", -5) == binding.CSR_ERR_INVALID_ARG
    assert lib.csr_set_option(b"wait_limit_ns", 2_000_000_000) == binding.CSR_OK
    assert lib.csr_set_option(b"no_such_option", 1) == binding.CSR_ERR_INVALID_ARG
    assert lib.csr_set_option(None, 1) == binding.CSR_ERR_INVALID_ARG
    out = ctypes.c_float()
    assert lib.csr_dict_check_norms(0, 1024, 128, 1e-3, None, ctypes.byref(out)) == binding.CSR_ERR_INVALID_ARG
    assert lib.csr_dict_check_norms(0x1000, 1024, 96, 1e-3, None, ctypes.byref(out)) == binding.CSR_ERR_UNSUPPORTED
    assert lib.csr_dict_check_norms(0x1004, 1024, 128, 1e-3, None, ctypes.byref(out)) == binding.CSR_ERR_ALIGNMENT
