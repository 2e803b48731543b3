"""The checked build of the library (python -m paper_2412_11741_b200.build --debug: device-side
checks of every index a kernel gathers with, in place of a memory checker) returns the release
build's codes, stays silent on sound inputs in every encoder path, and reports an out-of-range
index that the release build would clamp without a word.  It runs in a child process because a
process loads one build of the library."""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r'''
import sys
import numpy as np, torch
sys.path.insert(0, %(root)r)
import paper_2412_11741_b200 as csr
from paper_2412_11741_b200 import workloads as wl

assert csr.csr_debug_checks() == %(debug)d
dev = "cuda:0"
sums = []
# many rows (one CTA per pair of row tiles), few rows (clusters), the exact mode; N not a multiple of 8
for tokens, mode in ((160, csr.CSR_MODE_BF16_FAST), (4, csr.CSR_MODE_BF16_FAST), (8, csr.CSR_MODE_FP32_EXACT)):
    w = wl.llama2_layer(tokens=tokens, N=1001)
    D = torch.from_numpy(w.D).to(dev)
    X = torch.from_numpy(w.X).to(dev).to(torch.bfloat16)
    idx, coef = csr.csr_encode_ex(D, X, w.s, mode=mode)
    assert csr.csr_device_status() == csr.CSR_OK, csr.csr_last_error_string()
    xh = csr.csr_reconstruct(D, idx, coef)
    h = csr.csr_dict_create(D)
    xh2 = csr.csr_reconstruct_ex(D, idx, coef, dict=h)
    csr.csr_dict_destroy(h)
    assert csr.csr_device_status() == csr.CSR_OK, csr.csr_last_error_string()
    sums.append((int(idx.view(torch.int16).to(torch.int64).sum()), float(coef.double().sum()), float(xh.double().sum()), float(xh2.double().sum())))
print("SUMS", repr(sums))
# an index past the dictionary: clamped by both builds, reported by the checked one
bad = idx.clone().view(torch.int16)
bad[5, 2] = 5000
bad[77, 0] = -1                                            # 65535
out = csr.csr_reconstruct(D, bad.view(torch.uint16), coef)
assert bool(torch.isfinite(out.float()).all())
print("STATUS", csr.csr_device_status(), csr.csr_device_status())
'''


def _run(debug: bool):
    from paper_2412_11741_b200 import build
    lib = build.build(debug=debug)
    env = dict(os.environ, CSR_LIBRARY_PATH=lib)
    res = subprocess.run([sys.executable, "-c", CHILD % {"root": ROOT, "debug": int(debug)}], env=env, capture_output=True,
                         text=True, timeout=900)
    assert res.returncode == 0, res.stdout + res.stderr
    lines = dict(l.split(" ", 1) for l in res.stdout.splitlines() if l.startswith(("SUMS", "STATUS")))
    return lines["SUMS"], lines["STATUS"].split()


def test_checked_build_matches_release_and_reports_clamped_indices():
    sums_release, status_release = _run(False)
    sums_debug, status_debug = _run(True)
    assert sums_debug == sums_release                       # same codes, same restored tensors
    assert status_release == ["0", "0"]                     # CSR_OK: the release build clamps silently
    assert status_debug == ["-7", "0"]                      # CSR_ERR_BOUNDS once, cleared by reading it


CHILD_TENSOR = r'''
import sys
import numpy as np, torch
sys.path.insert(0, %(root)r)
import paper_2412_11741_b200 as csr
from paper_2412_11741_b200 import workloads as wl

dev = "cuda:0"
worst = 0.0
for w in (wl.dict_sweep(4096, M=8192), wl.dict_sweep(4096, d=64, M=8192), wl.sparsity_sweep(32, tokens=128, N=8192),
          wl.gqa_long(tokens=64)):
    D = torch.from_numpy(w.D).to(dev)
    X = torch.from_numpy(w.X).to(dev).to(torch.bfloat16)
    csr.csr_set_option("exact_engine", 2)
    idx, coef = csr.csr_encode_ex(D, X, w.s, mode=csr.CSR_MODE_FP32_EXACT, coef_dtype=torch.float32)
    csr.csr_set_option("exact_engine", 0)
    assert csr.csr_device_status() == csr.CSR_OK, csr.csr_last_error_string()
    worst = max(worst, csr.csr_debug_read("exact_tensor_error"))
print("TCERR", repr(worst))
'''


def test_tensor_core_correlations_stay_far_inside_the_band():
    """The exact mode's tensor-core encoder decides a row by its largest key only when the runner-up is
    more than 2^-12 ||R|| below it, which is sound while a tensor-core correlation is within half
    of that of the fp64 value.  The checked build records the largest deviation over all picks it
    took that way: it must stay below a quarter of the band on the paper-shaped workloads (the
    split of the operands alone accounts for up to 1.2e-5 ||R||)."""
    from paper_2412_11741_b200 import build
    lib = build.build(debug=True)
    env = dict(os.environ, CSR_LIBRARY_PATH=lib)
    res = subprocess.run([sys.executable, "-c", CHILD_TENSOR % {"root": ROOT}], env=env, capture_output=True, text=True, timeout=900)
    assert res.returncode == 0, res.stdout + res.stderr
    worst = float([l for l in res.stdout.splitlines() if l.startswith("TCERR")][0].split(" ", 1)[1])
    assert 0.0 < worst < 2.0 ** -14, worst
