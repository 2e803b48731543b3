"""GPU parity at the sizes the kernels' loops need: the exact-mode encoder with several row
tiles per CTA (its persistent loop), the de-sparse kernel with several rows per warp (its
grid-stride loop), one NeuralDict step at a dictionary of many atom blocks; and the library's
robustness promises (a bounded wait that runs out, calls on two streams with their own
scratch, the unit-norm check, the per-call status word).  Paper passages: "Sparse
representation" Eq. 2-4, "De-Sparse to restore" Eq. 12, Algorithm 1 (TrainNeurDict)."""
import numpy as np
import pytest
import torch

from oracle import csr_oracle as orc
from paper_2412_11741_b200 import workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def _np_idx(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def _rows(t, sel):
    return t.view(torch.int16)[sel].view(torch.uint16) if t.dtype == torch.uint16 else t[sel]


@pytest.fixture(scope="module")
def csr():
    from paper_2412_11741_b200 import build
    build.build()
    import paper_2412_11741_b200 as pkg
    return pkg


@pytest.fixture
def opts(csr):
    yield csr.csr_set_option
    for name, value in (("fast_group", 0), ("fast_split", 0), ("exact_split", 0), ("exact_engine", 0), ("wait_limit_ns", 2_000_000_000)):
        csr.csr_set_option(name, value)


@pytest.fixture(params=["alu", "tensor"])
def engine(request, csr):
    """The exact mode's plain-ALU encoders, then its tensor-core encoder."""
    csr.csr_set_option("exact_engine", {"alu": 1, "tensor": 2}[request.param])
    yield request.param
    csr.csr_set_option("exact_engine", 0)


# ---------------------------------------------------------------------------------------
# exact mode: every CTA takes several row tiles
# ---------------------------------------------------------------------------------------

def _exact_many_tiles(csr, w, n_rows, sample, seed):
    """Encodes n_rows rows spread over the whole workload (every head, keys and values) in the
    exact mode and lets the oracle check a stratified sample of the outputs row by row."""
    take = wl.stratified_rows(w.M, n_rows, seed=seed)
    X = np.ascontiguousarray(w.X[take])
    D = torch.from_numpy(w.D).to(DEV)
    Xd = torch.from_numpy(X).to(DEV).to(torch.bfloat16)
    n_tiles = (X.shape[0] + 63) // 64
    resident = 2 * torch.cuda.get_device_properties(0).multi_processor_count
    assert n_tiles >= 2 * resident + 1, "the persistent tile loop must take more than two trips"
    # (the tensor-core encoder holds 256 rows per CTA, one CTA per SM: more than one trip there too)
    assert (X.shape[0] + 255) // 256 > resident // 2
    idx, coef = csr.csr_encode_ex(D, Xd, w.s, mode=csr.CSR_MODE_FP32_EXACT, coef_dtype=torch.float32)
    assert csr.csr_device_status() == csr.CSR_OK
    sel = wl.stratified_rows(X.shape[0], sample, seed=seed + 1)
    sel[-1] = X.shape[0] - 1                                   # the last row of the last trip
    st = torch.from_numpy(sel).to(DEV)
    res = orc.mp_encode(w.D, X[sel], w.s)
    gi = _np_idx(_rows(idx, st))
    rep = parity.compare_exact(w.D, X[sel], w.s, gi, coef[st].cpu().numpy(), res)
    assert rep.ok, rep.detail
    assert rep.unexplained_rows == 0 and rep.coef_max_rel < 1e-4
    # every row of every trip was written: indices in range, and the codes restore x at the
    # sample's error level (a tile skipped or encoded twice from stale shared memory would not)
    assert int(idx.view(torch.int16).to(torch.int32).bitwise_and(0xFFFF).max()) < w.N
    xh = csr.csr_reconstruct_ex(D, idx, coef, out_dtype=torch.float32)
    err = ((xh - Xd.float()).norm(dim=1) / Xd.float().norm(dim=1))
    e_or = res.resnorm[:, -1] / np.linalg.norm(X[sel].astype(np.float64), axis=1)
    same = (gi == res.idx).all(1)                              # (a tie-excused row may end elsewhere)
    assert same.mean() > 0.99 and np.allclose(err[st].cpu().numpy()[same], e_or[same], rtol=2e-3, atol=1e-6)
    assert abs(float(err.mean()) / float(e_or.mean()) - 1) < 0.03
    return rep


def test_exact_full_size_llama2_layer(csr, engine):
    """Config 2 whole (262,144 rows: 4096 row tiles over 296 resident CTAs, 14 trips)."""
    w = wl.llama2_layer()
    _exact_many_tiles(csr, w, w.M, 2048, seed=61)


def test_exact_many_tiles_gqa_long(csr, engine):
    """Config 3: 65,536 rows spread over all sequences, heads, keys and values (N = 8192, s = 16)."""
    _exact_many_tiles(csr, wl.gqa_long(), 65536, 1024, seed=62)


def test_exact_many_tiles_sparsity_sweep_s32(csr, engine):
    """Config 4 at s = 32: 49,152 rows."""
    _exact_many_tiles(csr, wl.sparsity_sweep(32), 49152, 512, seed=63)


@pytest.mark.parametrize("N,d", [(16384, 128), (4096, 64)])
def test_exact_many_tiles_dict_sweep(csr, N, d, engine):
    """Config 5: the largest dictionary, and the d = 64 chunk shape; 49,152 rows."""
    _exact_many_tiles(csr, wl.dict_sweep(N, d=d), 49152, 768, seed=64 + d)


# ---------------------------------------------------------------------------------------
# de-sparse: every warp takes several rows
# ---------------------------------------------------------------------------------------

@pytest.mark.parametrize("d,N,s", [(128, 8192, 4), (128, 8192, 33), (64, 4096, 8), (128, 8192, 16)])
def test_reconstruct_one_million_rows_sampled(csr, d, N, s):
    """Eq. 12 at M = 2^20 (more rows than the grid has warps): a stratified sample of 4096 rows
    of X_hat against the oracle element by element, fp32 and bf16 output, fp32 and fp16
    coefficients; plus the first and the last row."""
    M = 1 << 20
    rng = np.random.default_rng(d + N + s)
    D = wl.normalise_rows(rng.standard_normal((N, d)).astype(np.float32))
    g = torch.Generator(device=DEV).manual_seed(d + s)
    idx = torch.randint(0, N, (M, s), device=DEV, generator=g, dtype=torch.int32)
    idx[:, -1] = idx[:, 0]                                     # repeated atoms accumulate
    coef = torch.randn((M, s), device=DEV, generator=g) * 3
    idx16 = idx.to(torch.int16).view(torch.uint16)             # wraps to the same 16 bits
    Dd = torch.from_numpy(D).to(DEV)
    sel = wl.stratified_rows(M, 4096, seed=s)
    sel[0], sel[-1] = 0, M - 1
    st = torch.from_numpy(sel).to(DEV)
    idx_s = idx[st].cpu().numpy()
    coef_s = coef[st].cpu().numpy()
    scale = np.abs(coef_s).sum(1, keepdims=True) + 1e-30
    ref32 = orc.reconstruct(D, idx_s, coef_s.astype(np.float64))
    out32 = csr.csr_reconstruct_ex(Dd, idx16, coef, out_dtype=torch.float32)
    assert np.all(np.abs(out32[st].cpu().numpy() - ref32) <= 2e-6 * scale)
    del out32
    coef16 = coef.to(torch.float16)
    ref16 = orc.reconstruct(D, idx_s, coef16[st].float().cpu().numpy().astype(np.float64))
    out16 = csr.csr_reconstruct(Dd, idx16, coef16)
    assert np.all(np.abs(out16[st].float().cpu().numpy() - ref16) <= 2.0 ** -8 * np.abs(ref16) + 2e-6 * scale)
    # no row left unwritten anywhere: a second call into a poisoned buffer overwrites all of it
    buf = torch.full((M, d), float("nan"), dtype=torch.bfloat16, device=DEV)
    csr.csr_reconstruct(Dd, idx16, coef16, X_hat=buf)
    assert bool(torch.isfinite(buf).all()) and torch.equal(buf, out16)
    del buf, out16
    # atoms gathered from a prepared dictionary's fp16 copy: Eq. 12 over the rounded atoms, i.e.
    # the oracle fed the fp16-rounded dictionary, to fp32 accuracy; and within the stated bound
    # sum_g |coef_g| (2^-11 |atom_g[k]| + 2^-25) of the fp32-atom result
    h = csr.csr_dict_create(Dd)
    Dh = D.astype(np.float16).astype(np.float32)
    refh = orc.reconstruct(Dh, idx_s, coef_s.astype(np.float64))
    outb = csr.csr_reconstruct_ex(Dd, idx16, coef, out_dtype=torch.float32, dict=h)       # fp32 coefficients
    gotb = outb[st].cpu().numpy()
    assert np.all(np.abs(gotb - refh) <= 2e-6 * scale)
    bound = (np.abs(coef_s.astype(np.float64))[:, :, None] * (2.0 ** -11 * np.abs(D[idx_s].astype(np.float64)) + 2.0 ** -25)).sum(1)
    assert np.all(np.abs(gotb - ref32) <= bound + 2e-6 * scale)
    refh16 = orc.reconstruct(Dh, idx_s, coef16[st].float().cpu().numpy().astype(np.float64))
    outh = csr.csr_reconstruct_ex(Dd, idx16, coef16, out_dtype=torch.float32, dict=h)      # fp16 coefficients: mixed-precision FMA
    assert np.all(np.abs(outh[st].cpu().numpy() - refh16) <= 2e-6 * scale)
    del outb, outh
    outb16 = csr.csr_reconstruct_ex(Dd, idx16, coef16, dict=h)
    assert torch.equal(outb16[st], csr.csr_reconstruct_ex(Dd, idx16, coef16, out_dtype=torch.float32, dict=h)[st].to(torch.bfloat16))
    with pytest.raises(csr.CsrError):
        csr.csr_reconstruct_ex(Dd[:N // 2].contiguous(), idx16, coef, dict=h)       # another dictionary
    csr.csr_dict_destroy(h)


# ---------------------------------------------------------------------------------------
# NeuralDict step with many atom blocks
# ---------------------------------------------------------------------------------------

@pytest.mark.parametrize("mode_name", ["exact", "fast"])
def test_training_step_at_2048_atoms(csr, mode_name):
    """One step at N = 2048, d = 128, M = 8192, s = 8 (32 blocks of 64 atoms; every atom is
    selected by several rows, so the gradient scatter adds many rows per atom).  The oracle's
    step is computed from the codes the GPU encoder produced (the fast mode's picks differ
    from an fp64 pursuit by design; the exact mode's must equal them)."""
    N, d, M, s = 2048, 128, 8192, 8
    w = wl.sparsity_sweep(s, tokens=M // 32, N=N)
    D0, X = w.D, w.X
    lr, beta = 2e-5, 0.6
    mode = csr.CSR_MODE_FP32_EXACT if mode_name == "exact" else csr.CSR_MODE_BF16_FAST
    Dd = torch.from_numpy(D0.copy()).to(DEV)
    Xd = torch.from_numpy(X).to(DEV).to(torch.bfloat16)
    idx, coef = csr.csr_encode_ex(Dd, Xd, s, mode=mode, coef_dtype=torch.float32)
    gi, gc = _np_idx(idx).astype(np.int32), coef.cpu().numpy().astype(np.float64)
    losses = csr.csr_dict_train_step(Dd, Xd, s, lr, beta, mode=mode).cpu().numpy()
    assert csr.csr_device_status() == csr.CSR_OK
    if mode_name == "exact":
        rep = parity.compare_exact(D0, X, s, gi, gc.astype(np.float32))
        assert rep.ok and rep.exempt_rows == 0, rep.detail
    # the step of Algorithm 1 on those codes, from the oracle's own pieces
    l_mse, g_mse = orc.mse_loss_and_grad(D0, X, gi, gc)
    l_div, g_div = orc.div_loss_and_grad(D0)
    W = D0.astype(np.float64) - lr * (g_mse + beta * g_div)
    want = (W / np.linalg.norm(W, axis=1, keepdims=True)).astype(np.float32)
    got = Dd.cpu().numpy()
    assert losses[0] == pytest.approx(l_mse, rel=2e-5) and losses[1] == pytest.approx(l_div, rel=2e-5)
    # fp32 sums of up to a few hundred gradient rows per atom: |g| ~ 1e2-1e3, times lr, in fp32
    scale = lr * np.abs(g_mse).max(axis=1, keepdims=True) + 1.0
    assert np.all(np.abs(got - want) <= 4e-6 * scale), float(np.abs(got - want).max())
    assert np.allclose(np.linalg.norm(got.astype(np.float64), axis=1), 1.0, atol=3e-7)
    assert np.abs(got - D0).max() > 1e-2                       # a real step, far above the tolerance
    if mode_name == "exact":
        want2 = orc.dict_train_step(D0, X, s, lr, beta)[0]
        assert np.all(np.abs(got - want2) <= 4e-6 * scale)
    # The diversity term is a few 1e-9 of that step (4 / N^2 in front of it), so it is checked
    # alone: an empty batch leaves ReNorm(D - lr * beta * grad L_div), taken with a large lr.
    Dd = torch.from_numpy(D0.copy()).to(DEV)
    lr2, beta2 = 400.0, 1.5
    losses = csr.csr_dict_train_step(Dd, Xd[:0], s, lr2, beta2, mode=mode).cpu().numpy()
    W = D0.astype(np.float64) - lr2 * beta2 * g_div
    want = (W / np.linalg.norm(W, axis=1, keepdims=True)).astype(np.float32)
    got = Dd.cpu().numpy()
    assert losses[0] == 0.0 and losses[1] == pytest.approx(l_div, rel=2e-5)
    assert np.abs(want - D0).max() > 2e-3 and np.abs(got - want).max() <= 1e-6


@pytest.mark.parametrize("N,d", [(4200, 128), (2500, 64)])
def test_diversity_step_alone_ragged_and_in_several_passes(csr, N, d):
    """The diversity term by itself (an empty batch) on dictionaries whose size is no multiple of
    the kernels' 128-atom blocks; at N = 4200, d = 128 the scratch copy of D D^T - I is filled and
    consumed in two passes of rows.  Against the oracle's loss and gradient, to the tolerance of
    the full step."""
    rng = np.random.default_rng(N)
    D0 = wl.normalise_rows(rng.standard_normal((N, d)).astype(np.float32) + np.float32(0.3))    # coherent atoms: a large gradient
    l_div, g_div = orc.div_loss_and_grad(D0)
    lr, beta = 2000.0, 0.5
    Dd = torch.from_numpy(D0.copy()).to(DEV)
    X0 = torch.empty((0, d), dtype=torch.float32, device=DEV)
    losses = csr.csr_dict_train_step(Dd, X0, 4, lr, beta).cpu().numpy()
    assert csr.csr_device_status() == csr.CSR_OK
    W = D0.astype(np.float64) - lr * beta * g_div
    want = (W / np.linalg.norm(W, axis=1, keepdims=True)).astype(np.float32)
    got = Dd.cpu().numpy()
    assert losses[0] == 0.0 and losses[1] == pytest.approx(l_div, rel=2e-5)
    assert np.abs(want - D0).max() > 2e-3 and np.abs(got - want).max() <= 1e-6, (float(np.abs(want - D0).max()), float(np.abs(got - want).max()))


# ---------------------------------------------------------------------------------------
# robustness
# ---------------------------------------------------------------------------------------

def test_bounded_wait_runs_out_and_the_library_recovers(csr, opts):
    """With the wait limit at zero the first hand-off that is not complete when it is first
    looked at expires: the kernel stops, lets its copies land, frees its tensor memory and
    returns; the status word says so; the next call, with the default limit, is unaffected."""
    rng = np.random.default_rng(9)
    M, N, s = 256, 512, 2
    D = wl.normalise_rows(rng.standard_normal((N, 128)).astype(np.float32))
    X = wl.round_to_bf16(rng.standard_normal((M, 128)).astype(np.float32))
    Dd = torch.from_numpy(D).to(DEV)
    Xd = torch.from_numpy(X).to(DEV).to(torch.bfloat16)
    opts("fast_split", 1)                                      # the one-CTA-per-row-pair kernel
    want_i, want_c = csr.csr_encode_ex(Dd, Xd, s, coef_dtype=torch.float32)
    assert csr.csr_device_status() == csr.CSR_OK
    word = torch.zeros(1, dtype=torch.int32, device=DEV)
    opts("wait_limit_ns", 0)
    csr.csr_encode_ex(Dd, Xd, s, coef_dtype=torch.float32)                       # library status word
    assert csr.csr_device_status() == csr.CSR_ERR_TIMEOUT
    assert "wait expired" in csr.csr_last_error_string()
    assert csr.csr_device_status() == csr.CSR_OK                                # reading it clears it
    csr.csr_encode_ex(Dd, Xd, s, coef_dtype=torch.float32, dev_status=word)      # the caller's word
    torch.cuda.synchronize()
    assert int(word.item()) != 0 and csr.csr_device_status() == csr.CSR_OK
    opts("wait_limit_ns", 2_000_000_000)
    got_i, got_c = csr.csr_encode_ex(Dd, Xd, s, coef_dtype=torch.float32, dev_status=word)
    torch.cuda.synchronize()
    assert int(word.item()) == 0
    assert np.array_equal(_np_idx(got_i), _np_idx(want_i)) and torch.equal(got_c, want_c)
    rep = parity.compare_fast(D, X, s, _np_idx(got_i), got_c.cpu().numpy())
    assert rep.ok, rep.detail


def test_bounded_wait_runs_out_in_the_exact_tensor_encoder(csr, opts):
    """The same for the exact mode's tensor-core encoder (its eight arg-max warps also meet at
    named barriers: they all learn of the expiry at the first one after it and leave together)."""
    rng = np.random.default_rng(10)
    M, N, s = 700, 600, 3
    D = wl.normalise_rows(rng.standard_normal((N, 128)).astype(np.float32))
    X = wl.round_to_bf16(rng.standard_normal((M, 128)).astype(np.float32))
    Dd = torch.from_numpy(D).to(DEV)
    Xd = torch.from_numpy(X).to(DEV).to(torch.bfloat16)
    opts("exact_engine", 2)
    want_i, want_c = csr.csr_encode_ex(Dd, Xd, s, mode=csr.CSR_MODE_FP32_EXACT, coef_dtype=torch.float32)
    assert csr.csr_device_status() == csr.CSR_OK
    word = torch.zeros(1, dtype=torch.int32, device=DEV)
    opts("wait_limit_ns", 0)
    csr.csr_encode_ex(Dd, Xd, s, mode=csr.CSR_MODE_FP32_EXACT, coef_dtype=torch.float32)
    assert csr.csr_device_status() == csr.CSR_ERR_TIMEOUT
    assert csr.csr_device_status() == csr.CSR_OK
    csr.csr_encode_ex(Dd, Xd, s, mode=csr.CSR_MODE_FP32_EXACT, coef_dtype=torch.float32, dev_status=word)
    torch.cuda.synchronize()
    assert int(word.item()) != 0 and csr.csr_device_status() == csr.CSR_OK
    opts("wait_limit_ns", 2_000_000_000)
    got_i, got_c = csr.csr_encode_ex(Dd, Xd, s, mode=csr.CSR_MODE_FP32_EXACT, coef_dtype=torch.float32, dev_status=word)
    torch.cuda.synchronize()
    assert int(word.item()) == 0
    assert np.array_equal(_np_idx(got_i), _np_idx(want_i)) and torch.equal(got_c, want_c)
    rep = parity.compare_exact(D, X, s, _np_idx(got_i), got_c.cpu().numpy())
    assert rep.ok, rep.detail


def test_two_streams_with_their_own_scratch_do_not_disturb_each_other(csr):
    """Keys and values have their own dictionaries and may be encoded side by side: with a
    workspace (or a handle) and a status word each, two calls on two streams return what each
    returns alone."""
    wk, wv = wl.sparsity_sweep(8, tokens=1024, N=4096), wl.dict_sweep(2048, M=32768)
    jobs = []
    for w in (wk, wv):
        D = torch.from_numpy(w.D).to(DEV)
        X = torch.from_numpy(w.X).to(DEV).to(torch.bfloat16)
        alone = csr.csr_encode_ex(D, X, w.s)
        ws = torch.empty(csr.csr_encode_workspace_bytes(csr.CSR_MODE_BF16_FAST, w.d, w.N), dtype=torch.uint8, device=DEV)
        jobs.append((w, D, X, alone, ws, torch.zeros(1, dtype=torch.int32, device=DEV), torch.cuda.Stream()))
    handle = csr.csr_dict_create(jobs[1][1])
    torch.cuda.synchronize()
    for rep in range(3):
        outs = []
        for j, (w, D, X, alone, ws, word, stream) in enumerate(jobs):
            with torch.cuda.stream(stream):
                if j == 0:
                    outs.append(csr.csr_encode_ex(D, X, w.s, workspace=ws, dev_status=word))
                else:
                    outs.append(csr.csr_encode_ex(D, X, w.s, dict=handle, dev_status=word))
        torch.cuda.synchronize()
        for (w, D, X, alone, ws, word, stream), (i, c) in zip(jobs, outs):
            assert int(word.item()) == 0
            assert np.array_equal(_np_idx(i), _np_idx(alone[0])) and torch.equal(c, alone[1])
    csr.csr_dict_destroy(handle)


def test_dictionary_norm_check(csr):
    rng = np.random.default_rng(4)
    D = wl.normalise_rows(rng.standard_normal((1000, 128)).astype(np.float32))
    Dd = torch.from_numpy(D).to(DEV)
    dev = csr.csr_dict_check_norms(Dd, tol=1e-5)
    want = np.abs(np.linalg.norm(D.astype(np.float64), axis=1) - 1.0).max()
    assert dev <= 3e-7 and abs(dev - want) <= 2e-7
    Dd[777] *= 1.25
    assert csr.csr_dict_check_norms(Dd) == pytest.approx(0.25, abs=1e-6)          # report only
    with pytest.raises(csr.CsrError) as ei:
        csr.csr_dict_check_norms(Dd, tol=1e-3)
    assert ei.value.code == csr.CSR_ERR_INVALID_ARG and "l2-norm" in str(ei.value)
    Dd[3] = float("nan")
    assert csr.csr_dict_check_norms(Dd) == float("inf")
    D64 = torch.from_numpy(wl.normalise_rows(rng.standard_normal((77, 64)).astype(np.float32))).to(DEV)
    assert csr.csr_dict_check_norms(D64, tol=1e-6) <= 3e-7


def test_scratch_growth_keeps_earlier_graphs_valid(csr):
    """A graph captured with the library's scratch keeps working after a later call has made
    that scratch grow (the outgrown block is kept), and a call that would have to grow it
    during capture is refused instead of allocating."""
    csr.csr_release_workspace()
    rng = np.random.default_rng(12)
    d, s = 128, 4
    D1 = torch.from_numpy(wl.normalise_rows(rng.standard_normal((1024, d)).astype(np.float32))).to(DEV)
    X = torch.from_numpy(rng.standard_normal((40000, d)).astype(np.float32)).to(DEV).to(torch.bfloat16)
    want = csr.csr_encode_ex(D1, X, s)                        # sizes the scratch for N = 1024
    idx = torch.zeros((X.shape[0], s), dtype=torch.int16, device=DEV).view(torch.uint16)
    coef = torch.zeros((X.shape[0], s), dtype=torch.float16, device=DEV)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        csr.csr_encode_ex(D1, X, s, out_idx=idx, out_coef=coef)
    D2 = torch.from_numpy(wl.normalise_rows(rng.standard_normal((16384, d)).astype(np.float32))).to(DEV)
    csr.csr_encode_ex(D2, X, s)                               # the scratch grows: a new block
    torch.cuda.synchronize()
    g.replay()
    torch.cuda.synchronize()
    assert np.array_equal(_np_idx(idx), _np_idx(want[0])) and torch.equal(coef, want[1])
    assert csr.csr_device_status() == csr.CSR_OK
    del g
    # growth during capture is refused (and the capture survives: nothing was enqueued)
    D3 = torch.from_numpy(wl.normalise_rows(rng.standard_normal((40000, d)).astype(np.float32))).to(DEV)
    g2 = torch.cuda.CUDAGraph()
    refused = False
    with torch.cuda.graph(g2):
        try:
            csr.csr_encode_ex(D3, X, s, out_idx=idx, out_coef=coef)
        except csr.CsrError as e:
            refused = e.code == csr.CSR_ERR_WORKSPACE
    assert refused
    del g2
    csr.csr_release_workspace()
