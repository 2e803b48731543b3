"""GPU parity of the chunked / multi-dictionary calls and of the online dictionary atoms
("KV Decomposition and Sparse Storage", "Build dictionary") against the CPU oracle."""
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


@pytest.fixture(scope="module")
def csr():
    from paper_2412_11741_b200 import build
    build.build()
    import paper_2412_11741_b200 as pkg
    return pkg


def _value_cache(M, seed):
    rng = np.random.default_rng(seed)
    X = wl.round_to_bf16(rng.standard_normal((M, 128)).astype(np.float32))
    Ds = [wl.normalise_rows(rng.standard_normal((1024, 64)).astype(np.float32)) for _ in range(2)]
    return X, Ds


@pytest.mark.parametrize("mode_name,s", [("exact", 4), ("fast", 4), ("fast", 8)])
def test_two_chunks_with_their_own_dictionaries_in_place(csr, mode_name, s):
    """Value cache with s_n = 2: both halves of every 128-channel head vector are encoded in
    place (row stride 128) into one [M][2*s] code array by one grouped call, then restored
    into one [M][128] array; each half must agree with the oracle's chunked pursuit."""
    M = 3000
    X, Ds = _value_cache(M, seed=s)
    mode = csr.CSR_MODE_FP32_EXACT if mode_name == "exact" else csr.CSR_MODE_BF16_FAST
    Xd = torch.from_numpy(X).to(DEV).to(torch.bfloat16)
    Dd = [torch.from_numpy(D).to(DEV) for D in Ds]
    idx = torch.zeros((M, 2 * s), dtype=torch.int16, device=DEV).view(torch.uint16)
    coef = torch.zeros((M, 2 * s), dtype=torch.float32, device=DEV)
    csr.csr_encode_grouped([(Dd[c], Xd[:, 64 * c:64 * (c + 1)], s, idx[:, s * c:s * (c + 1)], coef[:, s * c:s * (c + 1)])
                            for c in range(2)], mode=mode)
    assert csr.csr_device_status() == csr.CSR_OK
    ref = orc.mp_encode_chunked(Ds, X, s)
    gi, gc = _np_idx(idx), coef.cpu().numpy()
    for c in range(2):
        Xc = np.ascontiguousarray(X[:, 64 * c:64 * (c + 1)])
        ic, cc = gi[:, s * c:s * (c + 1)], gc[:, s * c:s * (c + 1)]
        rep = (parity.compare_exact if mode_name == "exact" else parity.compare_fast)(Ds[c], Xc, s, ic, cc, ref[c])
        assert rep.ok, (c, rep.detail)
        # in place == on a contiguous copy of the chunk, bit for bit
        i2, c2 = csr.csr_encode_ex(Dd[c], Xd[:, 64 * c:64 * (c + 1)].contiguous(), s, mode=mode, coef_dtype=torch.float32)
        assert np.array_equal(_np_idx(i2), ic) and np.array_equal(c2.cpu().numpy(), cc)
    # restore both halves side by side
    xh = torch.full((M, 128), 7.0, dtype=torch.float32, device=DEV)
    csr.csr_reconstruct_grouped([(Dd[c], idx[:, s * c:s * (c + 1)], coef[:, s * c:s * (c + 1)], xh[:, 64 * c:64 * (c + 1)])
                                 for c in range(2)])
    want = orc.reconstruct_chunked(Ds, [gi[:, s * c:s * (c + 1)].astype(np.int32) for c in range(2)],
                                   [gc[:, s * c:s * (c + 1)].astype(np.float64) for c in range(2)])
    scale = np.abs(gc).sum(1, keepdims=True) + 1e-30
    assert np.all(np.abs(xh.cpu().numpy() - want) <= 2e-6 * scale)


def test_packed_codes_of_two_chunks_use_vector_stores_when_they_can(csr):
    """s = 8 with fp16 coefficients: chunk c's codes start 16 bytes into the row, so the
    16-byte store path is taken with a row stride; the result equals the dense call's."""
    M, s = 1000, 8
    X, Ds = _value_cache(M, seed=11)
    Xd = torch.from_numpy(X).to(DEV).to(torch.bfloat16)
    Dd = [torch.from_numpy(D).to(DEV) for D in Ds]
    idx = torch.zeros((M, 2 * s), dtype=torch.int16, device=DEV).view(torch.uint16)
    coef = torch.zeros((M, 2 * s), dtype=torch.float16, device=DEV)
    csr.csr_encode_grouped([(Dd[c], Xd[:, 64 * c:64 * (c + 1)], s, idx[:, s * c:s * (c + 1)], coef[:, s * c:s * (c + 1)])
                            for c in range(2)])
    for c in range(2):
        i2, c2 = csr.csr_encode(Dd[c], Xd[:, 64 * c:64 * (c + 1)].contiguous(), s)
        assert np.array_equal(_np_idx(i2), _np_idx(idx)[:, s * c:s * (c + 1)])
        assert torch.equal(c2.cpu(), coef[:, s * c:s * (c + 1)].cpu())


@pytest.mark.parametrize("M", [64, 3000])
def test_grouped_problems_with_handles_run_side_by_side(csr, M):
    """The K rows and the V rows of a decoding step: two dictionaries, two handles, one grouped
    call.  Such problems are enqueued side by side; the codes are those of separate calls, and
    work enqueued afterwards on the caller's stream sees all of them (the join)."""
    rng = np.random.default_rng(M)
    N, d, s = 2048, 128, 8
    Ds = [torch.from_numpy(wl.normalise_rows(rng.standard_normal((N, d)).astype(np.float32))).to(DEV) for _ in range(3)]
    Xs = [torch.from_numpy(rng.standard_normal((M, d)).astype(np.float32)).to(DEV).to(torch.bfloat16) for _ in range(3)]
    want = [csr.csr_encode_ex(D, X, s) for D, X in zip(Ds, Xs)]
    hs = [csr.csr_dict_create(D) for D in Ds]
    idx = [torch.zeros((M, s), dtype=torch.int16, device=DEV).view(torch.uint16) for _ in range(3)]
    coef = [torch.zeros((M, s), dtype=torch.float16, device=DEV) for _ in range(3)]
    # the third problem brings no handle: it runs after the first two, in order
    csr.csr_encode_grouped([(Ds[0], Xs[0], s, idx[0], coef[0], hs[0]), (Ds[1], Xs[1], s, idx[1], coef[1], hs[1]),
                            (Ds[2], Xs[2], s, idx[2], coef[2])])
    total = sum(c.float().sum() for c in coef)                        # on the caller's stream, after the join
    torch.cuda.synchronize()
    assert csr.csr_device_status() == csr.CSR_OK
    for k in range(3):
        assert np.array_equal(_np_idx(idx[k]), _np_idx(want[k][0])) and torch.equal(coef[k], want[k][1])
    assert float(total) == float(sum(w[1].float().sum() for w in want))
    # the same call captured into a CUDA graph (the fork and the join become graph edges)
    for k in range(3):
        idx[k].zero_()
        coef[k].zero_()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        csr.csr_encode_grouped([(Ds[0], Xs[0], s, idx[0], coef[0], hs[0]), (Ds[1], Xs[1], s, idx[1], coef[1], hs[1])])
    g.replay()
    torch.cuda.synchronize()
    for k in range(2):
        assert np.array_equal(_np_idx(idx[k]), _np_idx(want[k][0])) and torch.equal(coef[k], want[k][1])
    del g
    for h in hs:
        csr.csr_dict_destroy(h)


@pytest.mark.parametrize("d,dtype", [(128, "bf16"), (64, "f32")])
def test_online_atoms_match_oracle_and_are_used_by_the_encoder(csr, d, dtype):
    """Sampled rows of the cache become unit-norm atoms behind the offline part; the encoder
    then finds each sampled row's own atom first."""
    rng = np.random.default_rng(d)
    N_off, n_on, M = 896, 128, 5000
    D0 = np.zeros((N_off + n_on, d), np.float32)
    D0[:N_off] = wl.normalise_rows(rng.standard_normal((N_off, d)).astype(np.float32))
    Xw = rng.standard_normal((M, 2 * d)).astype(np.float32)          # rows are slices of a wider array
    Xw[17] = 0.0
    if dtype == "bf16":
        Xw = wl.round_to_bf16(Xw)
    X = Xw[:, d:]
    rows = rng.choice(M, n_on, replace=False).astype(np.int64)
    rows[5] = 17                                                      # a zero row gives a zero atom
    Dd = torch.from_numpy(D0).to(DEV)
    Xd = torch.from_numpy(Xw).to(DEV)
    if dtype == "bf16":
        Xd = Xd.to(torch.bfloat16)
    n_new = csr.csr_dict_append(Dd, N_off, Xd[:, d:], torch.from_numpy(rows).to(DEV))
    assert n_new == N_off + n_on
    got = Dd.cpu().numpy()
    want = orc.dict_append(D0, N_off, X, rows)
    assert np.array_equal(got[:N_off], D0[:N_off])
    assert np.all(got[N_off + 5] == 0)
    assert np.all(np.abs(got - want) <= 4e-7 * np.abs(want) + 1e-9)   # fp32 norm against fp64
    # downstream: the oracle and the exact encoder, both on the GPU-built dictionary
    sel = np.delete(rows, 5)[:64]
    Xs = np.ascontiguousarray(X[sel])
    i, c = csr.csr_encode_ex(Dd, torch.from_numpy(Xs).to(DEV), 3, mode=csr.CSR_MODE_FP32_EXACT, coef_dtype=torch.float32)
    rep = parity.compare_exact(got, Xs, 3, _np_idx(i), c.cpu().numpy())
    assert rep.ok, rep.detail
    own = N_off + np.array([int(np.flatnonzero(rows == r)[0]) for r in sel])
    assert np.array_equal(_np_idx(i)[:, 0].astype(np.int64), own)


@pytest.mark.parametrize("B,H,T,N,d,s,coef_dtype", [
    (3, 4, 5000, 2048, 128, 8, torch.float16), (2, 1, 1500, 8192, 128, 16, torch.float32),
    (2, 8, 700, 1024, 64, 4, torch.float16), (1, 9, 300, 16384, 128, 3, torch.float32), (2, 2, 0, 256, 64, 2, torch.float16),
    (1, 4, 20000, 1024, 128, 8, torch.float16),       # one stream cut into many token ranges
    (200, 2, 1100, 512, 64, 4, torch.float16),        # more streams than SMs
])
def test_attention_from_codes_matches_oracle(csr, B, H, T, N, d, s, coef_dtype):
    """Scores and weighted value sums computed straight from the codes against the oracle,
    which restores the tensor (Eq. 12) and multiplies in fp64."""
    rng = np.random.default_rng(B * 1000 + T + N)
    D = wl.normalise_rows(rng.standard_normal((N, d)).astype(np.float32))
    idx = rng.integers(0, N, (B, T, s)).astype(np.int32)
    if T:
        idx[:, :, -1] = idx[:, :, 0]                                   # repeated atoms accumulate
    coef = (rng.standard_normal((B, T, s)) * 2).astype(np.float32)
    if coef_dtype == torch.float16:
        coef = coef.astype(np.float16).astype(np.float32)
    Q = rng.standard_normal((B, H, d)).astype(np.float32)
    W = rng.random((B, H, T)).astype(np.float32)
    W /= np.maximum(W.sum(-1, keepdims=True), 1e-30)                   # rows of a softmax
    Dd = torch.from_numpy(D).to(DEV)
    it = torch.from_numpy(idx.astype(np.uint16).view(np.int16)).to(DEV).view(torch.uint16)
    ct = torch.from_numpy(coef).to(DEV).to(coef_dtype)
    scale = 1.0 / np.sqrt(d)
    sc = csr.csr_key_scores(Dd, torch.from_numpy(Q).to(DEV), it, ct, scale).cpu().numpy()
    want = orc.key_scores(D, Q, idx, coef.astype(np.float64), scale)
    bound = scale * np.linalg.norm(Q, axis=2)[:, :, None] * np.abs(coef).sum(2)[:, None, :]   # sum |coef| ||q|| ||atom||
    assert sc.shape == want.shape and np.all(np.abs(sc - want) <= 2e-6 * bound + 1e-30)
    Qb = wl.round_to_bf16(Q)                                            # bf16 queries are read exactly
    sc = csr.csr_key_scores(Dd, torch.from_numpy(Qb).to(DEV).to(torch.bfloat16), it, ct, scale).cpu().numpy()
    assert np.all(np.abs(sc - orc.key_scores(D, Qb, idx, coef.astype(np.float64), scale)) <= 2e-6 * bound + 1e-30)
    mix = csr.csr_value_mix(Dd, torch.from_numpy(W).to(DEV), it, ct).cpu().numpy()
    want = orc.value_mix(D, W, idx, coef.astype(np.float64))
    mbound = (W[:, :, :, None] * np.abs(coef)[:, None, :, :]).sum((2, 3))[:, :, None]       # sum w |coef| ||atom||
    assert mix.shape == want.shape and np.all(np.abs(mix - want) <= 4e-6 * mbound + 1e-30)
    if T:
        # fixed-point tables and ordered sums: the same bits on every run
        again = csr.csr_value_mix(Dd, torch.from_numpy(W).to(DEV), it, ct).cpu().numpy()
        assert np.array_equal(mix, again)
        # weights that are not a softmax row: one large, the rest tiny, some negative
        Wp = (W * 1e-4).astype(np.float32)
        Wp[:, :, T // 2] = 3.0
        Wp[:, :, ::7] *= -1.0
        mix = csr.csr_value_mix(Dd, torch.from_numpy(Wp).to(DEV), it, ct).cpu().numpy()
        want = orc.value_mix(D, Wp, idx, coef.astype(np.float64))
        mbound = (np.abs(Wp)[:, :, :, None] * np.abs(coef)[:, None, :, :]).sum((2, 3))[:, :, None]
        assert np.all(np.abs(mix - want) <= 4e-6 * mbound + 1e-30)
        # a NaN weight still reaches the output of its own head, and only that one
        Wn = W.copy()
        Wn[0, 0, T // 3] = np.nan
        mix = csr.csr_value_mix(Dd, torch.from_numpy(Wn).to(DEV), it, ct).cpu().numpy()
        assert np.all(np.isnan(mix[0, 0])) and np.all(np.isfinite(mix[0, 1:])) and np.all(np.isfinite(mix[1:]))


def test_value_mix_table_cannot_overflow(csr):
    """The value mix accumulates in 32-bit fixed point scaled from a bound on the table entries.
    The bound must hold in the worst case: every entry of every token names the same atom, with
    equal coefficients and equal weights, so one table entry receives everything."""
    B, H, T, N, d, s = 2, 3, 40000, 512, 64, 64
    rng = np.random.default_rng(5)
    D = wl.normalise_rows(rng.standard_normal((N, d)).astype(np.float32))
    idx = np.full((B, T, s), 7, dtype=np.int32)
    idx[1] = 300
    coef = np.full((B, T, s), 2.5, dtype=np.float32)
    coef[1] *= -1.0
    W = np.ones((B, H, T), dtype=np.float32)
    it = torch.from_numpy(idx.astype(np.uint16).view(np.int16)).to(DEV).view(torch.uint16)
    mix = csr.csr_value_mix(torch.from_numpy(D).to(DEV), torch.from_numpy(W).to(DEV), it,
                            torch.from_numpy(coef).to(DEV).to(torch.float16)).cpu().numpy()
    want = np.stack([np.tile(2.5 * s * T * D[7].astype(np.float64), (H, 1)), np.tile(-2.5 * s * T * D[300].astype(np.float64), (H, 1))])
    assert np.all(np.abs(mix - want) <= 1e-6 * 2.5 * s * T)


def test_scores_from_codes_equal_scores_from_the_restored_tensor(csr):
    """End to end on key-like data: encode, then q . x~ from the codes equals q . x~ from the
    de-sparse kernel's output (fp32), to fp32 rounding."""
    w = wl.llama2_layer(tokens=256, N=1024)
    T = 256
    D = torch.from_numpy(w.D).to(DEV)
    X = torch.from_numpy(w.X[:32 * T]).to(DEV).to(torch.bfloat16)          # 32 key heads x 256 tokens
    idx, coef = csr.csr_encode(D, X, w.s)
    xh = csr.csr_reconstruct_ex(D, idx, coef, out_dtype=torch.float32).view(32, T, 128)
    Q = torch.randn((32, 2, 128), device=DEV, generator=torch.Generator(device=DEV).manual_seed(1))
    sc = csr.csr_key_scores(D, Q, idx.view(32, T, w.s), coef.view(32, T, w.s))
    ref = torch.einsum("bhd,btd->bht", Q.double(), xh.double())
    tol = 2e-6 * (Q.norm(dim=2)[:, :, None] * coef.float().abs().sum(1).view(32, 1, T))
    assert bool(((sc.double() - ref).abs() <= tol.double() + 1e-30).all())


@pytest.mark.parametrize("N,d,M,s", [(256, 128, 3000, 8), (200, 64, 1000, 4)])
def test_dictionary_training_step_matches_oracle(csr, N, d, M, s):
    """One batch of NeuralDict training (matching pursuit forward, both gradients, gradient
    step, ReNorm) against the oracle; then the adaptive weight and a few more steps."""
    rng = np.random.default_rng(N + M)
    D0 = wl.normalise_rows(rng.standard_normal((N, d)).astype(np.float32))
    X = rng.standard_normal((M, d)).astype(np.float32)
    lr, beta = 1e-3, 0.7
    Dd = torch.from_numpy(D0.copy()).to(DEV)
    Xd = torch.from_numpy(X).to(DEV)
    losses = csr.csr_dict_train_step(Dd, Xd, s, lr, beta).cpu().numpy()
    want_D, l_mse, l_div, res = orc.dict_train_step(D0, X, s, lr, beta)
    assert res.gap.min() > 2e-6                              # no tie in this batch: same codes on both sides
    assert losses[0] == pytest.approx(l_mse, rel=2e-6) and losses[1] == pytest.approx(l_div, rel=2e-5)
    got = Dd.cpu().numpy()
    assert np.abs(got - want_D).max() <= 2e-6
    assert np.allclose(np.linalg.norm(got.astype(np.float64), axis=1), 1.0, atol=3e-7)
    moved = np.abs(got - D0).max(axis=1) > 0
    assert moved.all()                                       # the diversity term reaches every atom
    # a short run with the adaptive weight lowers the MSE loss on this batch; the tensor-core
    # encoder may drive the forward pass just as well
    first = losses[0]
    for mode in (csr.CSR_MODE_FP32_EXACT,) * 8 + (csr.CSR_MODE_BF16_FAST,) * 4:
        beta = orc.adaptive_beta(float(losses[0]), float(losses[1]))
        losses = csr.csr_dict_train_step(Dd, Xd, s, 2e-3, beta, mode=mode).cpu().numpy()
    assert csr.csr_device_status() == csr.CSR_OK
    assert losses[0] < first and np.isfinite(losses).all()


def test_decode_attention_over_encoded_cache(csr):
    """A decoding step end to end: keys and values of 12 streams are encoded (separate
    dictionaries, s = 8 for keys and 4 for values), then softmax(q K~^T / sqrt(d)) V~ is taken
    straight from the codes and compared with the oracle, which restores both tensors."""
    rng = np.random.default_rng(77)
    B, H, T, d, Nk, Nv = 12, 4, 700, 128, 1024, 512
    Dk = wl.normalise_rows(rng.standard_normal((Nk, d)).astype(np.float32))
    Dv = wl.normalise_rows(rng.standard_normal((Nv, d)).astype(np.float32))
    K = wl.round_to_bf16(rng.standard_normal((B * T, d)).astype(np.float32))
    V = wl.round_to_bf16(rng.standard_normal((B * T, d)).astype(np.float32))
    Q = (rng.standard_normal((B, H, d)) * 2).astype(np.float32)
    Dkd, Dvd = torch.from_numpy(Dk).to(DEV), torch.from_numpy(Dv).to(DEV)
    ki, kc = csr.csr_encode(Dkd, torch.from_numpy(K).to(DEV).to(torch.bfloat16), 8)
    vi, vc = csr.csr_encode(Dvd, torch.from_numpy(V).to(DEV).to(torch.bfloat16), 4)
    scale = 1.0 / np.sqrt(d)
    out, w = csr.csr_decode_attention(Dkd, Dvd, torch.from_numpy(Q).to(DEV), ki.view(B, T, 8), kc.view(B, T, 8),
                                      vi.view(B, T, 4), vc.view(B, T, 4), scale)
    want_out, want_w = orc.decode_attention(Dk, Dv, Q, _np_idx(ki).astype(np.int32).reshape(B, T, 8),
                                            kc.float().cpu().numpy().astype(np.float64).reshape(B, T, 8),
                                            _np_idx(vi).astype(np.int32).reshape(B, T, 4),
                                            vc.float().cpu().numpy().astype(np.float64).reshape(B, T, 4), scale)
    w, out = w.cpu().numpy(), out.cpu().numpy()
    assert np.allclose(w.sum(-1), 1.0, atol=1e-5)
    assert np.all(np.abs(w - want_w) <= 1e-4 * want_w + 1e-9)             # exp of scores good to ~1e-5
    assert np.all(np.abs(out - want_out) <= 2e-4 * np.abs(vc.float().cpu().numpy()).max())
