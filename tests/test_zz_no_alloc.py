"""csr_encode_static, the encode entry point for callers that must not allocate device
memory (a server with a fixed memory plan, a process whose free memory belongs to a
caching allocator, a loop that cannot take the implicit synchronisation of cudaMalloc or
cudaFree).  Its scratch is an array inside the library image; this test checks, through
the C ABI, that it returns exactly what the allocating entry point returns, twice in a
row with different dictionaries (the array keeps the previous call's contents), that it
leaves the amount of free device memory unchanged once a start-up call per shape class has
been made (many rows; the few rows of a decoding step, which run as thread-block clusters),
and that it refuses dictionaries larger than the array.  Collected last on purpose."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2412_11741_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _np_idx(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def test_static_scratch_encode_matches_allocating_entry_point():
    from paper_2412_11741_b200 import build
    build.build()
    import paper_2412_11741_b200 as csr

    # N = 8192 (the limit) with 1024 rows (clusters of CTAs share the rows), then N = 1024 with 40960
    # rows (one CTA per pair of row tiles), then the 16 new rows of a decoding step (one row tile)
    cases = [wl.gqa_long(tokens=8), wl.llama2_layer(tokens=640, N=1024), wl.gqa_long(tokens=1, seqs=1)]
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    # start-up: the first call on a device loads the array, and each kernel's first launch its code
    for w in cases:
        oi = torch.zeros((w.M, w.s), dtype=torch.int16, device=DEV).view(torch.uint16)
        oc = torch.zeros((w.M, w.s), dtype=torch.float16, device=DEV)
        csr.csr_encode_static(torch.from_numpy(w.D).to(DEV), torch.from_numpy(w.X).to(DEV).to(torch.bfloat16), w.s, oi, oc)
    torch.cuda.synchronize()
    for call, w in enumerate(cases):
        D = torch.from_numpy(w.D).to(DEV)
        X = torch.from_numpy(w.X).to(DEV).to(torch.bfloat16)
        ref_idx, ref_coef = csr.csr_encode(D, X, w.s)                    # existing entry point
        torch.cuda.synchronize()
        out_idx = torch.full((w.M, w.s), -1, dtype=torch.int16, device=DEV).view(torch.uint16)
        out_coef = torch.full((w.M, w.s), float("nan"), dtype=torch.float16, device=DEV)
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        csr.csr_encode_static(D, X, w.s, out_idx, out_coef, dev_status=status)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert int(status.item()) == 0
        assert free_after == free_before
        assert np.array_equal(_np_idx(out_idx), _np_idx(ref_idx))
        assert torch.equal(out_coef.cpu(), ref_coef.cpu())

    # beyond the array: 16384 atoms of 128 channels
    big = torch.zeros((16384, 128), dtype=torch.float32, device=DEV)
    X = torch.zeros((256, 128), dtype=torch.bfloat16, device=DEV)
    oi = torch.zeros((256, 8), dtype=torch.int16, device=DEV).view(torch.uint16)
    oc = torch.zeros((256, 8), dtype=torch.float16, device=DEV)
    with pytest.raises(csr.CsrError) as ei:
        csr.csr_encode_static(big, X, 8, oi, oc)
    assert ei.value.code == csr.CSR_ERR_UNSUPPORTED and "CSR_STATIC_MAX_DICT_ELEMS" in str(ei.value)
    # without a caller status word
    w = cases[1]
    D = torch.from_numpy(w.D).to(DEV)
    X = torch.from_numpy(w.X).to(DEV).to(torch.bfloat16)
    ref_idx, ref_coef = csr.csr_encode(D, X, w.s)
    oi = torch.zeros((w.M, w.s), dtype=torch.int16, device=DEV).view(torch.uint16)
    oc = torch.zeros((w.M, w.s), dtype=torch.float16, device=DEV)
    csr.csr_encode_static(D, X, w.s, oi, oc)
    torch.cuda.synchronize()
    assert np.array_equal(_np_idx(oi), _np_idx(ref_idx)) and torch.equal(oc.cpu(), ref_coef.cpu())
