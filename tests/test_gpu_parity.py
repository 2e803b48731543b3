"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs (paper Eq. 2-4 for the encoder, Eq. 12 for the de-sparse)."""
import numpy as np
import pytest
import torch

from oracle import csr_oracle as orc
from paper_2412_11741_b200 import workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def _np_idx(t):
    """uint16 tensor -> numpy (through an int16 view: few torch ops take uint16)."""
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def _take_rows(t, rows):
    return t.view(torch.int16)[rows].view(torch.uint16) if t.dtype == torch.uint16 else t[rows]


@pytest.fixture(scope="module")
def csr():
    from paper_2412_11741_b200 import build
    build.build()
    import paper_2412_11741_b200 as pkg
    return pkg


@pytest.fixture
def opts(csr):
    """Sets library options (csr_set_option) for one test and restores the defaults afterwards."""
    yield csr.csr_set_option
    for name, value in (("fast_group", 0), ("fast_split", 0), ("exact_split", 0), ("exact_engine", 0), ("wait_limit_ns", 2_000_000_000)):
        csr.csr_set_option(name, value)


@pytest.fixture(params=["library", "alu", "tensor"])
def engine(request, csr):
    """Runs an exact-mode test with the library's choice of encoder, with the plain-ALU encoders
    only, and with the tensor-core encoder whatever the number of rows."""
    csr.csr_set_option("exact_engine", {"library": 0, "alu": 1, "tensor": 2}[request.param])
    yield request.param
    csr.csr_set_option("exact_engine", 0)


def _dev_x(w, X=None):
    X = w.X if X is None else X
    t = torch.from_numpy(np.ascontiguousarray(X)).to(DEV)
    return t.to(torch.bfloat16) if w.x_dtype == "bf16" else t


def _encode(csr, w, X, mode, coef_dtype=torch.float32):
    D = torch.from_numpy(w.D).to(DEV)
    idx, coef = csr.csr_encode_ex(D, _dev_x(w, X), w.s, mode=mode, coef_dtype=coef_dtype)
    assert csr.csr_device_status() == csr.CSR_OK
    return _np_idx(idx), coef.float().cpu().numpy()


# ---------------------------------------------------------------------------------------
# exact mode
# ---------------------------------------------------------------------------------------

def test_exact_tiny_config_all_rows(csr, engine):
    w = wl.tiny()
    idx, coef = _encode(csr, w, w.X, csr.CSR_MODE_FP32_EXACT)
    rep = parity.compare_exact(w.D, w.X, w.s, idx, coef)
    assert rep.ok, rep.detail
    assert rep.unexplained_rows == 0 and rep.coef_max_rel < 1e-4
    # the stored fp16 coefficient is the round-to-nearest-even of the fp32 one
    idx16, coef16 = _encode(csr, w, w.X, csr.CSR_MODE_FP32_EXACT, torch.float16)
    assert np.array_equal(idx16, idx)
    assert np.array_equal(coef16, coef.astype(np.float16).astype(np.float32))
    # exactly sparse rows: same picks as the oracle, first pick inside the true support
    lo, hi = w.meta["sparse_rows"]
    assert all(idx[m, 0] in w.meta["support"][m - lo] for m in range(lo, hi))


@pytest.mark.parametrize("make,rows", [
    (lambda: wl.llama2_layer(tokens=64), 2048),
    (lambda: wl.gqa_long(tokens=32), 1536),
    (lambda: wl.sparsity_sweep(32, tokens=64, N=8192), 768),
    (lambda: wl.dict_sweep(2048, M=4096), 2048),
    (lambda: wl.dict_sweep(4096, d=64, M=4096), 2048),
])
def test_exact_configs_subsample(csr, make, rows, engine):
    w = make()
    sel = wl.stratified_rows(w.M, rows, seed=7)
    X = w.X[sel]
    idx, coef = _encode(csr, w, X, csr.CSR_MODE_FP32_EXACT)
    rep = parity.compare_exact(w.D, X, w.s, idx, coef)
    assert rep.ok, rep.detail


@pytest.mark.parametrize("M", [0, 1, 2, 63, 64, 65, 127, 129, 200])
def test_exact_ragged_rows(csr, M, engine):
    rng = np.random.default_rng(M)
    D = wl.normalise_rows(rng.standard_normal((272, 128)).astype(np.float32))   # N not a tile multiple
    X = rng.standard_normal((M, 128)).astype(np.float32)
    w = wl.Workload("ragged", D, X, 5, "f32")
    if M == 0:
        Dd = torch.from_numpy(D).to(DEV)
        i, c = csr.csr_encode_ex(Dd, torch.empty((0, 128), device=DEV), 5, mode=csr.CSR_MODE_FP32_EXACT,
                                 coef_dtype=torch.float32)
        assert i.shape == (0, 5)
        return
    idx, coef = _encode(csr, w, X, csr.CSR_MODE_FP32_EXACT)
    rep = parity.compare_exact(D, X, 5, idx, coef)
    assert rep.ok, rep.detail


@pytest.mark.parametrize("N,s", [(1, 3), (16, 1), (130, 7), (1024, 64)])
def test_exact_small_dictionaries(csr, N, s, engine):
    rng = np.random.default_rng(N * 100 + s)
    D = wl.normalise_rows(rng.standard_normal((N, 64)).astype(np.float32))
    X = rng.standard_normal((150, 64)).astype(np.float32)
    idx, coef = _encode(csr, wl.Workload("small", D, X, s, "f32"), X, csr.CSR_MODE_FP32_EXACT)
    rep = parity.compare_exact(D, X, s, idx, coef)
    assert rep.ok, rep.detail


def test_exact_degenerate_inputs(csr, engine):
    """Zero vectors, exact ties, an input that is itself an atom, a duplicated atom."""
    rng = np.random.default_rng(5)
    D = wl.normalise_rows(rng.standard_normal((256, 128)).astype(np.float32))
    D[200] = D[3]                       # duplicate atom: the lower index must win
    D[17] = -D[9]                       # sign-flipped duplicate
    X = rng.standard_normal((64, 128)).astype(np.float32)
    X[0] = 0.0
    X[1] = D[42] * np.float32(2.0)      # exactly one atom: residual becomes (nearly) zero
    X[2] = D[3] * np.float32(-1.5)
    X[3] = D[9]
    idx, coef = _encode(csr, wl.Workload("deg", D, X, 6, "f32"), X, csr.CSR_MODE_FP32_EXACT)
    res = orc.mp_encode(D, X, 6)
    assert idx[0].tolist() == [0] * 6 and np.all(coef[0] == 0)
    assert idx[1, 0] == 42 and idx[2, 0] == 3 and idx[3, 0] == 9
    assert np.array_equal(idx[:, 0], res.idx[:, 0])
    rep = parity.compare_exact(D, X, 6, idx, coef, res)
    assert rep.ok, rep.detail


def test_exact_identity_dictionary_recovers_exactly(csr, engine):
    rng = np.random.default_rng(8)
    D = np.eye(64, dtype=np.float32)
    X = rng.standard_normal((130, 64)).astype(np.float32)
    idx, coef = _encode(csr, wl.Workload("eye", D, X, 64, "f32"), X, csr.CSR_MODE_FP32_EXACT)
    order = np.argsort(-np.abs(X), axis=1, kind="stable")
    assert np.array_equal(idx, order)
    assert np.array_equal(coef, np.take_along_axis(X, order, 1))


@pytest.mark.parametrize("M,N,d,s", [(1, 8192, 128, 16), (128, 8192, 128, 16), (200, 272, 128, 5), (1000, 4096, 64, 8),
                                     (4000, 2048, 128, 4)])
def test_exact_few_rows_split_dictionary_path(csr, M, N, d, s, opts):
    """Few rows (what one decoding step adds): the dictionary is split across CTAs.  The codes
    must be those of the one-CTA-per-row-tile encoder bit for bit, and the oracle's."""
    rng = np.random.default_rng(M + N)
    D = wl.normalise_rows(rng.standard_normal((N, d)).astype(np.float32))
    D[N // 2] = D[3]                                     # a duplicated atom: the lower index must win
    X = rng.standard_normal((M, d)).astype(np.float32)
    X[0] = D[3] * np.float32(1.25)
    w = wl.Workload("decode", D, X, s, "f32")
    idx, coef = _encode(csr, w, X, csr.CSR_MODE_FP32_EXACT)
    opts("exact_split", 1)
    idx2, coef2 = _encode(csr, w, X, csr.CSR_MODE_FP32_EXACT)
    opts("exact_split", 0)
    assert np.array_equal(idx, idx2) and np.array_equal(coef, coef2)
    assert idx[0, 0] == 3
    rep = parity.compare_exact(D, X, s, idx, coef)
    assert rep.ok, rep.detail


# ---------------------------------------------------------------------------------------
# fast mode
# ---------------------------------------------------------------------------------------

def test_fast_tiny_config(csr):
    w = wl.tiny()
    idx, coef = _encode(csr, w, w.X, csr.CSR_MODE_BF16_FAST)
    rep = parity.compare_fast(w.D, w.X, w.s, idx, coef)
    assert rep.ok, rep.detail
    assert rep.same_rows > 0.8 * rep.rows


@pytest.mark.parametrize("make,rows", [
    (lambda: wl.llama2_layer(tokens=64), 2048),
    (lambda: wl.gqa_long(tokens=32), 1536),
    (lambda: wl.sparsity_sweep(4, tokens=64, N=8192), 1024),
    (lambda: wl.sparsity_sweep(32, tokens=64, N=8192), 768),
    (lambda: wl.dict_sweep(2048, M=4096), 2048),
    (lambda: wl.dict_sweep(16384, M=4096), 768),
    (lambda: wl.dict_sweep(4096, d=64, M=4096), 2048),
])
def test_fast_configs_subsample(csr, make, rows):
    w = make()
    sel = wl.stratified_rows(w.M, rows, seed=11)
    X = w.X[sel]
    idx, coef = _encode(csr, w, X, csr.CSR_MODE_BF16_FAST)
    rep = parity.compare_fast(w.D, X, w.s, idx, coef)
    assert rep.ok, rep.detail


@pytest.mark.parametrize("M", [1, 127, 128, 129, 255, 256, 257, 300 * 256 + 5])
def test_fast_ragged_rows_match_full_tiles(csr, M):
    """Rows of a ragged tail get the same codes as the same rows inside full tiles, and
    rows past M are not written."""
    rng = np.random.default_rng(3)
    D = wl.normalise_rows(rng.standard_normal((512, 128)).astype(np.float32))
    Mfull = ((M + 255) // 256 + 1) * 256
    X = wl.round_to_bf16(rng.standard_normal((Mfull, 128)).astype(np.float32))
    Dd = torch.from_numpy(D).to(DEV)
    Xd = torch.from_numpy(X).to(DEV).to(torch.bfloat16)
    s = 8
    i_full, c_full = csr.csr_encode_ex(Dd, Xd, s, coef_dtype=torch.float32)
    out_i = torch.full((Mfull, s), -1, dtype=torch.int16, device=DEV).view(torch.uint16)
    out_c = torch.full((Mfull, s), -7.0, dtype=torch.float32, device=DEV)
    csr.csr_encode_ex(Dd, Xd[:M].contiguous(), s, coef_dtype=torch.float32, out_idx=out_i[:M], out_coef=out_c[:M])
    assert csr.csr_device_status() == csr.CSR_OK
    assert np.array_equal(_np_idx(out_i)[:M], _np_idx(i_full)[:M])
    assert torch.equal(out_c[:M].cpu(), c_full[:M].cpu())
    assert np.all(_np_idx(out_i)[M:] == 0xFFFF) and bool((out_c[M:] == -7.0).all())
    if M <= 300:
        rep = parity.compare_fast(D, X[:M], s, _np_idx(out_i)[:M], out_c[:M].cpu().numpy())
        assert rep.mean_ratio < 1.05 and rep.ratio_max < 1.5, rep


@pytest.mark.parametrize("N", [1, 5, 100, 1000, 4100])
@pytest.mark.parametrize("G", [0, 8])
def test_fast_any_dictionary_size(csr, N, G, opts):
    """N need not be a multiple of anything: the bf16 copy is padded with zero atoms, which
    are never selected (indices stay below N) unless the residual is zero (then atom 0)."""
    opts("fast_group", G)
    rng = np.random.default_rng(N)
    D = wl.normalise_rows(rng.standard_normal((N, 128)).astype(np.float32))
    X = wl.round_to_bf16(rng.standard_normal((600, 128)).astype(np.float32))
    X[11] = 0.0
    s = 4
    idx, coef = _encode(csr, wl.Workload("anyN", D, X, s, "bf16"), X, csr.CSR_MODE_BF16_FAST)
    assert int(idx.max()) < N and idx[11].tolist() == [0] * s and np.all(coef[11] == 0)
    if N >= 5:
        rep = parity.compare_fast(D, X, s, idx, coef)
        assert rep.ok, rep.detail
    else:                                                 # one atom: every step projects onto it
        res = orc.mp_encode(D, X, s)
        xn = np.linalg.norm(X.astype(np.float64), axis=1)
        assert np.array_equal(idx, res.idx) and np.all(np.abs(coef[:, 0] - res.coef[:, 0]) <= 2.0 ** -8 * xn)   # bf16 atom


@pytest.mark.parametrize("M,N,d,s,kind", [(1, 8192, 128, 16, "bf16"), (128, 8192, 128, 16, "bf16"), (300, 1000, 128, 5, "f32"),
                                          (2000, 4096, 64, 8, "f16"), (9000, 2048, 128, 4, "bf16"), (16, 65536, 64, 3, "bf16"),
                                          (24500, 65536, 128, 2, "bf16"),      # more row pairs than clusters fit at once
                                          (16, 4096, 128, 8, "bf16"), (100, 6144, 128, 5, "f32"), (64, 2048, 64, 4, "f16"),
                                          (128, 16384, 128, 6, "bf16"), (129, 8192, 128, 4, "bf16"),    # one row tile: 1, 1-2, 1, 4 tiles per CTA; just over
                                          (5, 300, 128, 3, "bf16"), (130, 600, 64, 2, "f32"), (7, 257, 64, 9, "f16")])   # two or three dictionary tiles
def test_fast_few_rows_split_dictionary_path(csr, M, N, d, s, kind, opts):
    """Few rows: the dictionary is split across the CTAs of a cluster (one launch) or, without
    clusters, across CTAs with one sweep and one pick launch per iteration.  Both must return
    the codes of the one-CTA-per-row-pair kernel bit for bit."""
    rng = np.random.default_rng(M * 7 + N)
    D = wl.normalise_rows(rng.standard_normal((N, d)).astype(np.float32))
    X = rng.standard_normal((M, d)).astype(np.float32)
    if N >= 1024:
        D[512 + 3] = D[3]                # the same atom at the same place of two 256-atom tiles: equal keys,
        X[0] = 3.0 * D[3] + 0.05 * X[0]  # and a row whose first pick it is: the lower index must win
    X = wl.round_to_bf16(X) if kind == "bf16" else X.astype(np.float16).astype(np.float32) if kind == "f16" else X
    if M > 2:
        X[1] = 0.0
    Dd = torch.from_numpy(D).to(DEV)
    Xd = torch.from_numpy(X).to(DEV).to({"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}[kind])
    i1, c1 = csr.csr_encode_ex(Dd, Xd, s, coef_dtype=torch.float32)
    assert csr.csr_device_status() == csr.CSR_OK
    if N >= 1024:
        assert int(_np_idx(i1)[0, 0]) == 3
    h = csr.csr_dict_create(Dd)
    i3, c3 = csr.csr_encode_ex(Dd, Xd, s, coef_dtype=torch.float16, dict=h)       # handle + packed coefficients
    csr.csr_dict_destroy(h)
    opts("fast_split", 2)                                         # the launch-per-iteration split
    i4, c4 = csr.csr_encode_ex(Dd, Xd, s, coef_dtype=torch.float32)
    assert csr.csr_device_status() == csr.CSR_OK
    opts("fast_split", 1)                                         # one CTA per pair of row tiles
    i2, c2 = csr.csr_encode_ex(Dd, Xd, s, coef_dtype=torch.float32)
    opts("fast_split", 0)
    assert np.array_equal(_np_idx(i1), _np_idx(i2)) and torch.equal(c1, c2)
    assert np.array_equal(_np_idx(i4), _np_idx(i2)) and torch.equal(c4, c2)
    assert np.array_equal(_np_idx(i3), _np_idx(i2)) and torch.equal(c3, c2.to(torch.float16))
    if N >= 1000 and M >= 100 and M * N <= 2e7:
        rep = parity.compare_fast(D, wl.round_to_bf16(X), s, _np_idx(i1), c1.cpu().numpy())
        assert rep.ok, rep.detail


@pytest.mark.parametrize("G", [1, 2, 4, 8])
@pytest.mark.parametrize("M,d", [(100, 128), (1000, 128), (40, 64)])
def test_fast_few_rows_every_group_size(csr, G, M, d, opts):
    """The clustered kernels exist for every arg-max group size: with the group size fixed, few
    rows must get the codes of the one-CTA-per-row-pair kernel bit for bit."""
    rng = np.random.default_rng(G * 1000 + M)
    N, s = 8192, 6
    Dd = torch.from_numpy(wl.normalise_rows(rng.standard_normal((N, d)).astype(np.float32))).to(DEV)
    Xd = torch.from_numpy(rng.standard_normal((M, d)).astype(np.float32)).to(DEV).to(torch.bfloat16)
    opts("fast_group", G)
    i1, c1 = csr.csr_encode_ex(Dd, Xd, s)
    opts("fast_split", 1)
    i2, c2 = csr.csr_encode_ex(Dd, Xd, s)
    assert csr.csr_device_status() == csr.CSR_OK
    assert np.array_equal(_np_idx(i1), _np_idx(i2)) and torch.equal(c1, c2)


@pytest.mark.parametrize("M", [16, 1024, 70000])
def test_encode_captured_in_a_cuda_graph(csr, M):
    """A decoding loop replays its step as a CUDA graph: after one ordinary call (which sizes
    the library's buffers) the encode, clustered or not, can be captured and replayed."""
    rng = np.random.default_rng(M)
    N, d, s = 4096, 128, 8
    Dd = torch.from_numpy(wl.normalise_rows(rng.standard_normal((N, d)).astype(np.float32))).to(DEV)
    X1 = torch.from_numpy(rng.standard_normal((M, d)).astype(np.float32)).to(DEV).to(torch.bfloat16)
    X2 = torch.from_numpy(rng.standard_normal((M, d)).astype(np.float32)).to(DEV).to(torch.bfloat16)
    want1 = csr.csr_encode_ex(Dd, X1, s)
    want2 = csr.csr_encode_ex(Dd, X2, s)
    h = csr.csr_dict_create(Dd)
    X = X1.clone()
    idx = torch.zeros((M, s), dtype=torch.int16, device=DEV).view(torch.uint16)
    coef = torch.zeros((M, s), dtype=torch.float16, device=DEV)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        csr.csr_encode_ex(Dd, X, s, out_idx=idx, out_coef=coef, dict=h)
    for want, src in ((want1, X1), (want2, X2)):
        X.copy_(src)
        g.replay()
        torch.cuda.synchronize()
        assert np.array_equal(_np_idx(idx), _np_idx(want[0])) and torch.equal(coef, want[1])
    assert csr.csr_device_status() == csr.CSR_OK
    del g
    csr.csr_dict_destroy(h)


def test_fast_fp32_input_and_odd_s(csr):
    rng = np.random.default_rng(13)
    D = wl.normalise_rows(rng.standard_normal((1024, 128)).astype(np.float32))
    X = rng.standard_normal((1000, 128)).astype(np.float32)
    for s in (1, 3, 11):
        w = wl.Workload("f32in", D, X, s, "f32")
        idx, coef = _encode(csr, w, X, csr.CSR_MODE_BF16_FAST)
        rep = parity.compare_fast(D, X, s, idx, coef)
        assert rep.ok, rep.detail
        idx16, coef16 = _encode(csr, w, X, csr.CSR_MODE_BF16_FAST, torch.float16)
        assert np.array_equal(idx16, idx)
        assert np.array_equal(coef16, coef.astype(np.float16).astype(np.float32))


@pytest.mark.parametrize("n", [0, 1, 7, 8, 1000003])
def test_pack_coefficients_is_round_to_nearest_even(csr, n):
    rng = np.random.default_rng(n)
    c = (rng.standard_normal(n) * np.exp(rng.uniform(-12, 8, n))).astype(np.float32)
    if n > 5:
        c[:5] = [0.0, -0.0, 65504.0, 1e-8, -70000.0]      # signed zero, largest, subnormal underflow, overflow
    with np.errstate(over="ignore"):                    # -70000 becomes -inf, as it must
        _, want = orc.pack_codes(np.zeros(n, np.int32), c.astype(np.float64))
    got = csr.csr_pack_coefficients(torch.from_numpy(c).to(DEV)).cpu().numpy()
    assert np.array_equal(got.view(np.uint16), want.view(np.uint16))


def test_fp16_inputs_and_outputs(csr, engine):
    """fp16 is the paper's model precision: X may be fp16 (read exactly by the exact mode,
    rounded to bf16 by the fast mode) and X_hat may be written as fp16."""
    rng = np.random.default_rng(16)
    D = wl.normalise_rows(rng.standard_normal((1024, 128)).astype(np.float32))
    X = (rng.standard_normal((900, 128)) * 3).astype(np.float16).astype(np.float32)
    Dd = torch.from_numpy(D).to(DEV)
    Xh = torch.from_numpy(X).to(DEV).to(torch.float16)
    s = 6
    idx, coef = csr.csr_encode_ex(Dd, Xh, s, mode=csr.CSR_MODE_FP32_EXACT, coef_dtype=torch.float32)
    rep = parity.compare_exact(D, X, s, _np_idx(idx), coef.cpu().numpy())
    assert rep.ok, rep.detail
    idx, coef = csr.csr_encode_ex(Dd, Xh, s, coef_dtype=torch.float32)
    i2, c2 = csr.csr_encode_ex(Dd, Xh.to(torch.bfloat16), s, coef_dtype=torch.float32)   # = rounding to bf16 first
    assert np.array_equal(_np_idx(idx), _np_idx(i2)) and torch.equal(coef, c2)
    rep = parity.compare_fast(D, X, s, _np_idx(idx), coef.cpu().numpy())
    assert rep.ok, rep.detail
    x32 = csr.csr_reconstruct_ex(Dd, idx, coef, out_dtype=torch.float32)
    x16 = csr.csr_reconstruct_ex(Dd, idx, coef, out_dtype=torch.float16)
    assert torch.equal(x16, x32.to(torch.float16))


def test_fast_zero_rows_and_eight_arg_form(csr):
    w = wl.llama2_layer(tokens=8, N=1024)
    X = w.X.copy()
    X[5] = 0.0
    D = torch.from_numpy(w.D).to(DEV)
    Xd = torch.from_numpy(X).to(DEV).to(torch.bfloat16)
    idx, coef = csr.csr_encode(D, Xd, w.s)
    torch.cuda.synchronize()
    assert csr.csr_device_status() == csr.CSR_OK
    assert idx.dtype == torch.uint16 and coef.dtype == torch.float16
    assert _np_idx(idx)[5].tolist() == [0] * w.s and bool((coef[5] == 0).all())
    rep = parity.compare_fast(w.D, X, w.s, _np_idx(idx), coef.float().cpu().numpy())
    assert rep.ok, rep.detail
    # caller-provided workspace gives the same codes
    nbytes = csr.csr_encode_workspace_bytes(csr.CSR_MODE_BF16_FAST, 128, 1024)
    ws = torch.empty(nbytes, dtype=torch.uint8, device=DEV)
    idx2, coef2 = csr.csr_encode_ex(D, Xd, w.s, workspace=ws)
    assert np.array_equal(_np_idx(idx2), _np_idx(idx)) and torch.equal(coef2.cpu(), coef.cpu())
    with pytest.raises(csr.CsrError):
        csr.csr_encode_ex(D, Xd, w.s, workspace=ws[:1024])


def test_prepared_dictionary_handle(csr):
    """A handle encodes exactly as the plain call does, keeps its snapshot when D changes
    afterwards, and refuses a call made for another dictionary."""
    w = wl.llama2_layer(tokens=8, N=1000)                # N not a multiple of 8 * 128 either
    D = torch.from_numpy(w.D).to(DEV)
    X = torch.from_numpy(w.X).to(DEV).to(torch.bfloat16)
    i0, c0 = csr.csr_encode_ex(D, X, w.s)
    h = csr.csr_dict_create(D)
    try:
        i1, c1 = csr.csr_encode_ex(D, X, w.s, dict=h)
        assert csr.csr_device_status() == csr.CSR_OK
        assert np.array_equal(_np_idx(i1), _np_idx(i0)) and torch.equal(c1.cpu(), c0.cpu())
        D.mul_(-1.0)                                     # the copy is a snapshot: same codes as before
        i2, c2 = csr.csr_encode_ex(D, X, w.s, dict=h)
        assert np.array_equal(_np_idx(i2), _np_idx(i0)) and torch.equal(c2.cpu(), c0.cpu())
        i3, c3 = csr.csr_encode_ex(D, X, w.s)            # the plain call sees the negated atoms
        assert np.array_equal(_np_idx(i3), _np_idx(i0)) and torch.equal(c3.cpu(), -c0.cpu())
        with pytest.raises(csr.CsrError):
            csr.csr_encode_ex(D[:512].contiguous(), X, w.s, dict=h)
    finally:
        csr.csr_dict_destroy(h)


def test_fast_full_size_llama2_layer_sampled(csr):
    """Config 2 at full size in the launch configuration the benchmark times; the oracle
    checks a stratified sample of the outputs."""
    w = wl.llama2_layer()
    assert w.M == 262144 and w.N == 4096 and w.s == 8
    D = torch.from_numpy(w.D).to(DEV)
    Xd = torch.from_numpy(w.X).to(DEV).to(torch.bfloat16)
    idx, coef = csr.csr_encode(D, Xd, w.s)
    assert csr.csr_device_status() == csr.CSR_OK
    sel = wl.stratified_rows(w.M, 2048, seed=21)
    st = torch.from_numpy(sel).to(DEV)
    rep = parity.compare_fast(w.D, w.X[sel], w.s, _np_idx(_take_rows(idx, st)), coef[st].float().cpu().numpy())
    assert rep.ok, rep.detail
    # every row got a valid code and the whole tensor reconstructs with the sample's error level
    assert int(_np_idx(idx).max()) < w.N
    xh = csr.csr_reconstruct(D, idx, coef)
    err = ((xh.float() - Xd.float()).norm(dim=1) / Xd.float().norm(dim=1)).mean().item()
    assert abs(err / rep.mean_err - 1) < 0.02


def _full_size_sampled(csr, w, rows, seed):
    """Encodes the whole workload in the launch configuration the benchmark times and lets the
    oracle check a stratified sample of the outputs; every index must be in range and the
    whole tensor must reconstruct at the sample's error level."""
    D = torch.from_numpy(w.D).to(DEV)
    Xd = torch.from_numpy(w.X).to(DEV).to(torch.bfloat16)
    idx, coef = csr.csr_encode(D, Xd, w.s)
    assert csr.csr_device_status() == csr.CSR_OK
    sel = wl.stratified_rows(w.M, rows, seed=seed)
    st = torch.from_numpy(sel).to(DEV)
    rep = parity.compare_fast(w.D, w.X[sel], w.s, _np_idx(_take_rows(idx, st)), coef[st].float().cpu().numpy())
    assert rep.ok, rep.detail
    assert int(idx.view(torch.int16).to(torch.int32).bitwise_and(0xFFFF).max()) < w.N
    err = 0.0
    step = 1 << 18
    for r0 in range(0, w.M, step):                      # in slices: X_hat of the whole job is large
        xh = csr.csr_reconstruct(D, _take_rows(idx, slice(r0, r0 + step)).contiguous(), coef[r0:r0 + step].contiguous())
        xs = Xd[r0:r0 + step].float()
        err += float(((xh.float() - xs).norm(dim=1) / xs.norm(dim=1)).sum())
    assert abs(err / w.M / rep.mean_err - 1) < 0.03
    return rep


def test_fast_full_size_gqa_long_sampled(csr):
    """Config 3 (the benchmark's workload) at full size."""
    w = wl.gqa_long()
    assert w.M == 2097152 and w.N == 8192 and w.s == 16
    _full_size_sampled(csr, w, 1024, seed=31)


@pytest.mark.parametrize("s", [4, 32])
def test_fast_full_size_sparsity_sweep_sampled(csr, s):
    """Config 4 at full size, the two ends of the sparsity sweep."""
    w = wl.sparsity_sweep(s)
    assert w.M == 1 << 20 and w.N == 8192
    _full_size_sampled(csr, w, 768, seed=41 + s)


@pytest.mark.parametrize("N,d", [(2048, 128), (16384, 128), (4096, 64)])
def test_fast_full_size_dict_sweep_sampled(csr, N, d):
    """Config 5 at full size: smallest and largest dictionary at d = 128, and d = 64."""
    w = wl.dict_sweep(N, d=d)
    assert w.M == 1 << 20
    _full_size_sampled(csr, w, 768, seed=51 + N // 1024 + d)


@pytest.mark.parametrize("G", [1, 2, 4, 8])
@pytest.mark.parametrize("d", [64, 128])
def test_fast_every_group_size(csr, G, d, opts):
    """The arg-max group size is a tuning knob: every setting must meet the same gates, also
    with a dictionary that ends in half an atom tile (N = 384) or is smaller than one (N = 128)."""
    opts("fast_group", G)
    rng = np.random.default_rng(100 * G + d)
    for N, M, s in ((384, 700, 6), (128, 300, 3), (2048, 1500, 9)):
        D = wl.normalise_rows(rng.standard_normal((N, d)).astype(np.float32))
        X = wl.round_to_bf16(rng.standard_normal((M, d)).astype(np.float32))
        X[7] = 0.0
        w = wl.Workload("grp", D, X, s, "bf16")
        idx, coef = _encode(csr, w, X, csr.CSR_MODE_BF16_FAST)
        assert idx[7].tolist() == [0] * s and np.all(coef[7] == 0)
        rep = parity.compare_fast(D, X, s, idx, coef)
        assert rep.ok, (G, d, N, rep.detail)


def test_largest_dictionary_and_most_iterations(csr, engine):
    """The limits of the interface: N = 65536 (indices fill the uint16 range) and s = 64, in
    both modes, against the oracle."""
    rng = np.random.default_rng(65536)
    N, d, M, s = 65536, 64, 192, 64
    D = wl.normalise_rows(rng.standard_normal((N, d)).astype(np.float32))
    X = wl.round_to_bf16(rng.standard_normal((M, d)).astype(np.float32))
    X[3] = D[65535] * np.float32(2.0)                     # the last atom must be reachable
    X = wl.round_to_bf16(X)
    w = wl.Workload("limits", D, X, s, "bf16")
    res = orc.mp_encode(D, X, s)
    idx, coef = _encode(csr, w, X, csr.CSR_MODE_FP32_EXACT)
    rep = parity.compare_exact(D, X, s, idx, coef, res)
    assert rep.ok, rep.detail
    assert idx[3, 0] == 65535 and int(idx.max()) > 60000
    # Fast mode at s = d with 65536 atoms: the oracle drives the error down to 5e-5 of ||x||.
    # The fast mode carries its residual in bf16, and the rounding of every intermediate
    # residual (2^-9 of its size) stays in the true error for good, so its error cannot
    # fall below about 2^-8 ||x|| (mean 3e-3, worst row 4e-3 here); down to that floor it
    # must follow the oracle.
    idx, coef = _encode(csr, w, X, csr.CSR_MODE_BF16_FAST)
    assert int(idx.max()) < N and idx[3, 0] == 65535
    e_gpu = orc.relative_error(X, orc.reconstruct(D, idx.astype(np.int32), coef.astype(np.float64)))
    e_or = res.resnorm[:, -1] / np.linalg.norm(X.astype(np.float64), axis=1)
    assert e_or.mean() < 1e-4
    assert np.all(e_gpu <= 1.05 * e_or + 2.0 ** -7.5) and e_gpu.mean() < 2.0 ** -8, float(e_gpu.max())
    # and at s = 16, where the error (0.1) is far above the floor, the usual gates hold
    # (row 3 is left out: it is one atom up to bf16 rounding, so after its first step both
    # sides chase rounding noise)
    keep = np.arange(M) != 3
    rep = parity.compare_fast(D, X[keep], 16, idx[keep, :16], coef[keep, :16])
    assert rep.ok, rep.detail


# ---------------------------------------------------------------------------------------
# de-sparse
# ---------------------------------------------------------------------------------------

@pytest.mark.parametrize("d,N,s,M", [(128, 1024, 8, 4096), (64, 300, 5, 1001), (128, 65536, 33, 517), (128, 16, 64, 64)])
def test_reconstruct_matches_oracle(csr, d, N, s, M):
    rng = np.random.default_rng(d + N + s)
    D = wl.normalise_rows(rng.standard_normal((N, d)).astype(np.float32))
    idx = rng.integers(0, N, size=(M, s)).astype(np.int32)
    idx[:, -1] = idx[:, 0]                     # repeated atoms accumulate
    coef = (rng.standard_normal((M, s)) * 3).astype(np.float32)
    idx16, coef16 = orc.pack_codes(idx, coef.astype(np.float64))
    Dd = torch.from_numpy(D).to(DEV)
    it = torch.from_numpy(idx16).to(DEV)
    ref32 = orc.reconstruct(D, idx, coef.astype(np.float64))
    scale = np.abs(coef).sum(1, keepdims=True) + 1e-30
    out32 = csr.csr_reconstruct_ex(Dd, it, torch.from_numpy(coef).to(DEV), out_dtype=torch.float32).cpu().numpy()
    assert np.abs(out32 - ref32).max() <= 1e-6 * scale.max()
    assert np.all(np.abs(out32 - ref32) <= 2e-6 * scale)
    # stored form: fp16 coefficients in, bf16 out
    ref16 = orc.reconstruct(D, idx, coef16.astype(np.float64))
    out16 = csr.csr_reconstruct(Dd, it, torch.from_numpy(coef16).to(DEV)).float().cpu().numpy()
    assert np.all(np.abs(out16 - ref16) <= 2.0 ** -8 * np.abs(ref16) + 2e-6 * scale)


def test_encode_then_reconstruct_round_trip(csr):
    w = wl.gqa_long(tokens=16)
    D = torch.from_numpy(w.D).to(DEV)
    Xd = torch.from_numpy(w.X).to(DEV).to(torch.bfloat16)
    idx, coef = csr.csr_encode(D, Xd, w.s)
    xh = csr.csr_reconstruct(D, idx, coef).float().cpu().numpy()
    ref = orc.reconstruct(w.D, _np_idx(idx).astype(np.int32), coef.float().cpu().numpy().astype(np.float64))
    assert np.all(np.abs(xh - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-3)


def test_host_entry_point(csr):
    w = wl.llama2_layer(tokens=600, N=1024)         # 38400 rows: more than one chunk
    D = torch.from_numpy(w.D).to(DEV)
    Xh = torch.from_numpy(w.X).to(torch.bfloat16).pin_memory()
    oi = torch.empty((w.M, w.s), dtype=torch.uint16).pin_memory()
    oc = torch.empty((w.M, w.s), dtype=torch.float16).pin_memory()
    csr.csr_encode_host(D, Xh, w.s, oi, oc)
    idx, coef = csr.csr_encode(D, Xh.to(DEV), w.s)
    torch.cuda.synchronize()
    assert np.array_equal(_np_idx(oi), _np_idx(idx)) and torch.equal(oc, coef.cpu())
    # and back: host codes in, host X_hat out, equal to the device entry point bit for bit
    xh_host = torch.empty((w.M, w.d), dtype=torch.bfloat16).pin_memory()
    csr.csr_reconstruct_host(D, oi, oc, xh_host)
    xh_dev = csr.csr_reconstruct(D, idx, coef)
    torch.cuda.synchronize()
    assert torch.equal(xh_host.view(torch.int16), xh_dev.cpu().view(torch.int16))
    xh32 = torch.empty((w.M, w.d), dtype=torch.float32)          # pageable memory and fp32 output work too
    csr.csr_reconstruct_host(D, oi, oc, xh32)
    assert torch.equal(xh32, csr.csr_reconstruct_ex(D, idx, coef, out_dtype=torch.float32).cpu())
    # with a prepared dictionary: the same codes, and the fp16-atom restore of the device entry point
    h = csr.csr_dict_create(D)
    oi2, oc2 = torch.zeros_like(oi), torch.zeros_like(oc)
    csr.csr_encode_host(D, Xh, w.s, oi2, oc2, dict=h)
    assert np.array_equal(_np_idx(oi2), _np_idx(idx)) and torch.equal(oc2, coef.cpu())
    csr.csr_reconstruct_host(D, oi, oc, xh_host, dict=h)
    assert torch.equal(xh_host.view(torch.int16), csr.csr_reconstruct_ex(D, idx, coef, dict=h).cpu().view(torch.int16))
    csr.csr_dict_destroy(h)


def test_host_entry_point_exact_mode_in_several_chunks(csr):
    """The exact mode through the host entry point: the chunks' encodes share the library's
    scratch, so they are chained one after the other while the copies overlap them; the codes
    are those of the device entry point on the whole tensor, and the oracle's."""
    w = wl.llama2_layer(tokens=1100, N=1024)        # 70400 rows: three chunks of 32768, the last ragged
    D = torch.from_numpy(w.D).to(DEV)
    Xh = torch.from_numpy(w.X).to(torch.bfloat16).pin_memory()
    oi = torch.empty((w.M, w.s), dtype=torch.uint16).pin_memory()
    oc = torch.empty((w.M, w.s), dtype=torch.float32).pin_memory()
    csr.csr_encode_host(D, Xh, w.s, oi, oc, mode=csr.CSR_MODE_FP32_EXACT)
    assert csr.csr_device_status() == csr.CSR_OK
    idx, coef = csr.csr_encode_ex(D, Xh.to(DEV), w.s, mode=csr.CSR_MODE_FP32_EXACT, coef_dtype=torch.float32)
    torch.cuda.synchronize()
    assert np.array_equal(_np_idx(oi), _np_idx(idx)) and torch.equal(oc, coef.cpu())
    sel = wl.stratified_rows(w.M, 1024, seed=3)
    rep = parity.compare_exact(w.D, w.X[sel], w.s, _np_idx(oi)[sel], oc.numpy()[sel])
    assert rep.ok, rep.detail


# (114, 141, 534: two atoms and many iterations, the picks end up below the oracle's own rounding noise;
# 214, 421: an overcomplete d = 64 dictionary taken to a small error, where the error ratios spread)
@pytest.mark.parametrize("seed", list(range(24)) + [114, 141, 214, 421, 534])
def test_random_shapes_both_modes(csr, seed):
    """Seeded random (M, N, d, s, input type) combinations, ragged in every dimension, through
    both encoders and the de-sparse kernel against the oracle."""
    rng = np.random.default_rng(1000 + seed)
    d = int(rng.choice([64, 128]))
    N = int(rng.choice([1, 2, 17, 100, 255, 256, 257, 600, 1023, 3000, 5000]))
    M = int(rng.choice([1, 3, 100, 255, 257, 700, 1500, 5000]))
    s = int(rng.integers(1, 20))
    kind = str(rng.choice(["f32", "bf16", "f16"]))
    D = wl.normalise_rows(rng.standard_normal((N, d)).astype(np.float32))
    if N > 2 and seed % 3 == 0:
        D[N // 2] = D[0]                                  # a duplicated atom
    X = (rng.standard_normal((M, d)) * rng.choice([0.01, 1.0, 30.0])).astype(np.float32)
    if kind == "bf16":
        X = wl.round_to_bf16(X)
    elif kind == "f16":
        X = X.astype(np.float16).astype(np.float32)
    if M > 2:
        X[M // 2] = 0.0
    Dd = torch.from_numpy(D).to(DEV)
    Xd = torch.from_numpy(X).to(DEV).to({"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}[kind])
    res = orc.mp_encode(D, X, s)
    idx, coef = csr.csr_encode_ex(Dd, Xd, s, mode=csr.CSR_MODE_FP32_EXACT, coef_dtype=torch.float32)
    rep = parity.compare_exact(D, X, s, _np_idx(idx), coef.cpu().numpy(), res)
    assert rep.ok, (d, N, M, s, kind, rep.detail)
    csr.csr_set_option("exact_engine", 2)                 # the tensor-core encoder, whatever the number of rows
    try:
        idx_t, coef_t = csr.csr_encode_ex(Dd, Xd, s, mode=csr.CSR_MODE_FP32_EXACT, coef_dtype=torch.float32)
    finally:
        csr.csr_set_option("exact_engine", 0)
    assert csr.csr_device_status() == csr.CSR_OK
    rep = parity.compare_exact(D, X, s, _np_idx(idx_t), coef_t.cpu().numpy(), res)
    assert rep.ok, ("tensor", d, N, M, s, kind, rep.detail)
    xh = csr.csr_reconstruct_ex(Dd, idx, coef, out_dtype=torch.float32).cpu().numpy()
    ref = orc.reconstruct(D, _np_idx(idx).astype(np.int32), coef.cpu().numpy().astype(np.float64))
    scale = np.abs(coef.cpu().numpy()).sum(1, keepdims=True) + 1e-30
    assert np.all(np.abs(xh - ref) <= 2e-6 * scale)
    idx, coef = csr.csr_encode_ex(Dd, Xd, s, coef_dtype=torch.float32)
    assert csr.csr_device_status() == csr.CSR_OK
    gi, gc = _np_idx(idx), coef.cpu().numpy()
    assert int(gi.max()) < N
    if M > 2:
        assert gi[M // 2].tolist() == [0] * s and np.all(gc[M // 2] == 0)
    if N >= 100 and M >= 100:
        Xb = wl.round_to_bf16(X)                          # what the fast mode encodes
        rep = parity.compare_fast(D, Xb, s, gi, gc)
        assert rep.ok, (d, N, M, s, kind, rep.detail)
    else:                                                 # tiny problems: the codes must at least describe x
        e_gpu = orc.relative_error(X, orc.reconstruct(D, gi.astype(np.int32), gc.astype(np.float64)))
        e_or = res.resnorm[:, -1] / np.maximum(np.linalg.norm(X.astype(np.float64), axis=1), 1e-300)
        assert np.all(e_gpu <= 1.3 * e_or + 2.0 ** -6), (d, N, M, s, kind)


@pytest.mark.parametrize("M,N", [(700, 1000), (64, 8192)])
def test_nan_and_inf_rows_do_no_harm(csr, M, N):
    """NaN or Inf in X: those rows' codes are unspecified, but the calls return, no device-side
    wait expires, every index stays below 65536 and inside what the de-sparse kernel accepts,
    and the other rows get exactly the codes they get without the bad rows."""
    rng = np.random.default_rng(M)
    D = wl.normalise_rows(rng.standard_normal((N, 128)).astype(np.float32))
    X = wl.round_to_bf16(rng.standard_normal((M, 128)).astype(np.float32))
    bad = X.copy()
    bad[5, 3] = np.nan
    bad[9] = np.inf
    bad[17, 100] = -np.inf
    good = np.ones(M, bool)
    good[[5, 9, 17]] = False
    Dd = torch.from_numpy(D).to(DEV)
    for mode, dt, eng in ((csr.CSR_MODE_BF16_FAST, torch.bfloat16, 0), (csr.CSR_MODE_FP32_EXACT, torch.float32, 1),
                          (csr.CSR_MODE_FP32_EXACT, torch.float32, 2)):
        csr.csr_set_option("exact_engine", eng)
        try:
            i0, c0 = csr.csr_encode_ex(Dd, torch.from_numpy(X).to(DEV).to(dt), 6, mode=mode, coef_dtype=torch.float32)
            i1, c1 = csr.csr_encode_ex(Dd, torch.from_numpy(bad).to(DEV).to(dt), 6, mode=mode, coef_dtype=torch.float32)
        finally:
            csr.csr_set_option("exact_engine", 0)
        assert csr.csr_device_status() == csr.CSR_OK
        g = torch.from_numpy(good).to(DEV)
        assert torch.equal(i0.view(torch.int16)[g], i1.view(torch.int16)[g]) and torch.equal(c0[g], c1[g])
        xh = csr.csr_reconstruct_ex(Dd, i1, c1, out_dtype=torch.float32)       # clamps whatever the bad rows hold
        assert bool(torch.isfinite(xh[g]).all())
