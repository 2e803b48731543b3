"""B200-native sparse codec of CSR (arXiv 2412.11741): matching-pursuit encode and de-sparse.

The product is libcsr.so (hand-written sm_100a CUDA behind a C ABI, see include/csr.h);
this package only loads it and marshals torch tensors to it.
"""
from .binding import (  # noqa: F401
    CSR_DTYPE_BF16, CSR_DTYPE_F16, CSR_DTYPE_F32, CSR_ERR_ALIGNMENT, CSR_ERR_BOUNDS, CSR_ERR_CUDA, CSR_ERR_INVALID_ARG,
    CSR_ERR_TIMEOUT, CSR_ERR_UNSUPPORTED, CSR_ERR_WORKSPACE, CSR_MODE_BF16_FAST, CSR_MODE_FP32_EXACT, CSR_OK,
    CsrError, csr_device_status, csr_encode, csr_encode_ex, csr_decode_attention, csr_dict_append, csr_dict_check_norms, csr_dict_create, csr_dict_destroy, csr_dict_train_step, csr_encode_grouped, csr_encode_host, csr_encode_static, csr_encode_workspace_bytes, csr_key_scores, csr_pack_coefficients, csr_value_mix,
    csr_last_error_string, csr_reconstruct, csr_reconstruct_ex, csr_reconstruct_grouped, csr_reconstruct_host, csr_release_workspace, csr_set_option, csr_version, csr_debug_checks, csr_debug_read,
)
