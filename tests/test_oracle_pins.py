"""Pins for the CPU oracle: each test checks it against something the paper or the
mathematics fixes, not against its own formula.

Matching pursuit: paper Eq. 2-4; de-sparse: Eq. 12; storage format: "Analysis for CSR".
"""
import itertools
import os

import numpy as np
import pytest

from oracle import csr_oracle as orc
from paper_2412_11741_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand_dict(rng, N, d):
    return wl.normalise_rows(rng.standard_normal((N, d)).astype(np.float32))


# --- brute force on tiny inputs (pins Eq. 2-3 and the order of Eq. 4) --------------------

def _brute_force_mp(D, x, s):
    """Independent restatement: stable descending sort of |D R| picks the atom."""
    D = D.astype(np.float64)
    R = x.astype(np.float64).copy()
    idx, coef = [], []
    for _ in range(s):
        c = np.array([float(np.dot(R, D[n])) for n in range(D.shape[0])])
        order = sorted(range(len(c)), key=lambda n: (-abs(c[n]), n))
        i = order[0]
        idx.append(i)
        coef.append(c[i])
        R = R - c[i] * D[i]
    return np.array(idx), np.array(coef), R


@pytest.mark.parametrize("d,N,s", [(2, 3, 2), (4, 7, 3), (8, 16, 4), (5, 16, 4), (8, 1, 2)])
def test_brute_force_tiny(d, N, s):
    rng = np.random.default_rng(100 + d * N)
    D = _rand_dict(rng, N, d)
    X = rng.standard_normal((37, d)).astype(np.float32)
    res = orc.mp_encode(D, X, s)
    for m in range(X.shape[0]):
        bi, bc, bR = _brute_force_mp(D, X[m], s)
        assert np.array_equal(res.idx[m], bi)
        np.testing.assert_allclose(res.coef[m], bc, rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(res.residual[m], bR, rtol=0, atol=1e-13)


def test_exhaustive_best_single_atom():
    """For s = 1 the pick must minimise ||x - c d_n|| over every atom and every scalar c
    (Eq. 1 restricted to one atom): the optimum is c = x.d_n / ||d_n||^2."""
    rng = np.random.default_rng(7)
    D = _rand_dict(rng, 12, 6)
    X = rng.standard_normal((50, 6)).astype(np.float32)
    res = orc.mp_encode(D, X, 1)
    Dd = D.astype(np.float64)
    for m in range(50):
        errs = []
        for n in range(12):
            c = np.dot(X[m], Dd[n]) / np.dot(Dd[n], Dd[n])
            errs.append(np.linalg.norm(X[m] - c * Dd[n]))
        # unit-norm atoms (to ~1e-7): the arg-max of |x.d_n| is the arg-min of the error
        assert res.idx[m, 0] == int(np.argmin(errs))


# --- s = 1 reduces to a library matmul ---------------------------------------------------

def test_s1_matches_matmul_argmax():
    rng = np.random.default_rng(3)
    D = _rand_dict(rng, 300, 64)
    X = rng.standard_normal((500, 64)).astype(np.float32)
    C = X.astype(np.float64) @ D.astype(np.float64).T
    res = orc.mp_encode(D, X, 1)
    assert np.array_equal(res.idx[:, 0], np.argmax(np.abs(C), axis=1))
    np.testing.assert_allclose(res.coef[:, 0], C[np.arange(500), res.idx[:, 0]], rtol=1e-12)
    srt = np.sort(np.abs(C), axis=1)
    np.testing.assert_allclose(res.gap[:, 0], (srt[:, -1] - srt[:, -2]) / srt[:, -1], rtol=1e-9, atol=1e-13)


# --- energy identity and monotone residual (pins the update and the signed coefficient) --

@pytest.mark.parametrize("seed", [0, 1])
def test_energy_identity_and_monotone(seed):
    rng = np.random.default_rng(seed)
    D = _rand_dict(rng, 256, 32)
    X = (rng.standard_normal((200, 32)) * 3).astype(np.float32)
    s = 12
    res = orc.mp_encode(D, X, s)
    x2 = (X.astype(np.float64) ** 2).sum(1)
    dn2 = (D.astype(np.float64) ** 2).sum(1)
    # exact identity for arbitrary atom norms: each step removes c^2 (2 - ||d||^2)
    removed = (res.coef ** 2 * (2.0 - dn2[res.idx])).sum(1)
    np.testing.assert_allclose(x2, (res.residual ** 2).sum(1) + removed, rtol=1e-12)
    # unit-norm atoms: ||x||^2 = ||R_s||^2 + sum c^2 up to the 1e-7 normalisation error
    np.testing.assert_allclose(x2, (res.residual ** 2).sum(1) + (res.coef ** 2).sum(1), rtol=5e-6)
    norms = np.concatenate([np.sqrt(x2)[:, None], res.resnorm], axis=1)
    assert np.all(np.diff(norms, axis=1) <= 1e-12)
    np.testing.assert_allclose(res.resnorm[:, -1], np.linalg.norm(res.residual, axis=1), rtol=1e-12)
    # |c_g| is non-increasing is NOT a property of MP; but |c_g| <= ||R_g|| always is
    assert np.all(np.abs(res.coef) <= norms[:, :-1] * (1 + 1e-6))


def test_sign_of_coefficient_is_kept():
    D = np.eye(4, dtype=np.float32)
    X = np.array([[0.5, -3.0, 1.0, 0.0]], np.float32)
    res = orc.mp_encode(D, X, 2)
    assert res.idx.tolist() == [[1, 2]]
    assert res.coef.tolist() == [[-3.0, 1.0]]


# --- orthonormal dictionary: textbook closed form ---------------------------------------

def test_identity_dictionary_exact_recovery():
    rng = np.random.default_rng(11)
    d = 16
    D = np.eye(d, dtype=np.float32)
    X = rng.standard_normal((64, d)).astype(np.float32)
    res = orc.mp_encode(D, X, d)
    order = np.argsort(-np.abs(X), axis=1, kind="stable")
    assert np.array_equal(res.idx, order)
    assert np.array_equal(res.coef, np.take_along_axis(X.astype(np.float64), order, 1))
    assert np.all(res.residual == 0.0)


def test_orthogonal_dictionary_closed_form():
    rng = np.random.default_rng(12)
    d = 24
    Q, _ = np.linalg.qr(rng.standard_normal((d, d)))
    D = Q.T.astype(np.float32)  # rows orthonormal to fp32 rounding
    X = rng.standard_normal((40, d)).astype(np.float32)
    res = orc.mp_encode(D, X, d)
    proj = X.astype(np.float64) @ D.astype(np.float64).T
    order = np.argsort(-np.abs(proj), axis=1, kind="stable")
    assert np.array_equal(res.idx, order)
    np.testing.assert_allclose(res.coef, np.take_along_axis(proj, order, 1), atol=1e-5)
    assert np.abs(res.residual).max() < 1e-5


# --- metamorphic relations ----------------------------------------------------------------

def test_metamorphic():
    rng = np.random.default_rng(21)
    N, d, s = 128, 32, 6
    D = _rand_dict(rng, N, d)
    X = rng.standard_normal((100, d)).astype(np.float32)
    base = orc.mp_encode(D, X, s)
    # scaling the input by a power of two scales the coefficients, same atoms
    sc = orc.mp_encode(D, (X * np.float32(4.0)), s)
    assert np.array_equal(sc.idx, base.idx)
    np.testing.assert_allclose(sc.coef, 4.0 * base.coef, rtol=1e-13)
    # negating one atom negates its coefficients only
    D2 = D.copy()
    D2[5] = -D2[5]
    ng = orc.mp_encode(D2, X, s)
    assert np.array_equal(ng.idx, base.idx)
    sign = np.where(base.idx == 5, -1.0, 1.0)
    np.testing.assert_allclose(ng.coef, sign * base.coef, rtol=1e-13)
    # permuting the atoms permutes the indices
    perm = rng.permutation(N)
    pm = orc.mp_encode(D[perm], X, s)
    assert np.array_equal(perm[pm.idx], base.idx)
    np.testing.assert_allclose(pm.coef, base.coef, rtol=1e-13)
    # appended zero atoms are never picked
    zp = orc.mp_encode(np.concatenate([D, np.zeros((16, d), np.float32)]), X, s)
    assert np.array_equal(zp.idx, base.idx)


def test_tie_break_lowest_index_and_zero_residual():
    D = np.array([[1, 0], [0, 1], [1, 0], [-1, 0]], np.float32)
    X = np.array([[2.0, 0.0], [0.0, 0.0]], np.float32)
    res = orc.mp_encode(D, X, 3)
    # atoms 0, 2, 3 tie in |correlation| at step 0: the lowest index wins; after that the
    # residual is exactly zero and (0, 0) is emitted
    assert res.idx[0].tolist() == [0, 0, 0]
    assert res.coef[0].tolist() == [2.0, 0.0, 0.0]
    assert res.idx[1].tolist() == [0, 0, 0] and res.coef[1].tolist() == [0.0, 0.0, 0.0]
    assert res.gap[0, 0] == 0.0


def test_repeated_atoms_accumulate_in_reconstruction():
    # two coherent atoms: MP returns to the first one; Eq. 12 must add both entries
    D = wl.normalise_rows(np.array([[1.0, 0.0], [1.0, 1.0]], np.float32))
    X = np.array([[1.0, 0.45]], np.float32)
    res = orc.mp_encode(D, X, 4)
    assert len(set(res.idx[0].tolist())) < 4
    xh = orc.reconstruct(D, res.idx, res.coef)
    np.testing.assert_allclose(xh + res.residual, X.astype(np.float64), atol=1e-14)


# --- de-sparse equals dense r times D (Eq. 12) -------------------------------------------

def test_reconstruct_is_dense_product():
    rng = np.random.default_rng(5)
    N, d, s, M = 64, 16, 5, 80
    D = _rand_dict(rng, N, d)
    idx = rng.integers(0, N, size=(M, s)).astype(np.int32)
    idx[:, 1] = idx[:, 0]  # force duplicates
    coef = rng.standard_normal((M, s))
    r = np.zeros((M, N))
    for m in range(M):
        for g in range(s):
            r[m, idx[m, g]] += coef[m, g]
    np.testing.assert_allclose(orc.reconstruct(D, idx, coef), r @ D.astype(np.float64), atol=1e-13)


def test_codes_plus_residual_give_back_x():
    w = wl.tiny(M=256)
    res = orc.mp_encode(w.D, w.X, w.s)
    xh = orc.reconstruct(w.D, res.idx, res.coef)
    np.testing.assert_allclose(xh + res.residual, w.X.astype(np.float64), atol=1e-13)
    np.testing.assert_allclose(orc.relative_error(w.X, xh),
                               res.resnorm[:, -1] / np.linalg.norm(w.X.astype(np.float64), axis=1), rtol=1e-9)


# --- exactly sparse inputs (config 1's extra rows) ---------------------------------------

def test_sparse_rows_first_pick_in_support_and_decay():
    w = wl.tiny(M=0)
    lo, hi = w.meta["sparse_rows"]
    X = w.X[lo:hi]
    support = w.meta["support"]
    errs = []
    for s in (8, 16, 32):
        res = orc.mp_encode(w.D, X, s)
        if s == 8:
            assert all(res.idx[m, 0] in support[m] for m in range(X.shape[0]))
        errs.append((res.resnorm[:, -1] / np.linalg.norm(X, axis=1)).mean())
    # MP (unlike OMP) does not recover a sparse combination of coherent atoms in s steps,
    # but the residual must fall quickly
    assert errs[0] < 0.3 and errs[1] < 0.25 * errs[0] and errs[2] < 0.1 * errs[1]


def test_error_falls_with_s_and_N():
    """Qualitative trend of the paper's MSE tables: more entries or more atoms, less error."""
    rng = np.random.default_rng(9)
    X = rng.standard_normal((300, 32)).astype(np.float32)
    Dbig = _rand_dict(rng, 512, 32)

    def err(D, s):
        r = orc.mp_encode(D, X, s)
        return orc.relative_error(X, orc.reconstruct(D, r.idx, r.coef)).mean()

    assert err(Dbig, 2) > err(Dbig, 4) > err(Dbig, 8)
    assert err(Dbig[:64], 4) > err(Dbig[:256], 4) > err(Dbig, 4)


# --- storage format -------------------------------------------------------------------------

def test_format_golden():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "code_format.txt")) if l.strip() and not l.startswith("#")]
    for d_h, s, s_n, bits, ratio in rows:
        d_h, s, s_n = int(d_h), int(s), int(s_n)
        assert orc.code_bits_per_channel(d_h, s, s_n) == float(bits)
        assert 2 * d_h / orc.code_bytes_per_vector(s, s_n) == float(ratio)
    idx = np.array([[0, 65535, 7]], np.int32)
    coef = np.array([[1.0, -0.333333333, 48.123]])
    i16, c16 = orc.pack_codes(idx, coef)
    assert i16.dtype == np.uint16 and c16.dtype == np.float16
    assert i16.nbytes + c16.nbytes == orc.code_bytes_per_vector(3)
    bi, bc = orc.unpack_codes(i16, c16)
    assert np.array_equal(bi, idx)
    np.testing.assert_allclose(bc, coef, rtol=2.0 ** -11)
    with pytest.raises(ValueError):
        orc.pack_codes(np.array([[70000]], np.int32), np.array([[1.0]]))


# --- planted mistakes must be caught (the pins are not vacuous) -----------------------------

def test_unsigned_reading_of_eq2_is_not_what_the_oracle_computes():
    """Eq. 2 prints the coefficient as a supremum of absolute values.  Taken literally (subtract
    |c| d) the residual GAINS energy whenever the best correlation is negative; the oracle keeps
    the sign.  On an input whose first pick has a negative correlation the oracle's output
    satisfies the energy identity and the literal reading, written out here, does not; the two
    residuals differ from the first step on."""
    rng = np.random.default_rng(0)
    D = _rand_dict(rng, 64, 16)
    x = rng.standard_normal(16).astype(np.float32)
    res = orc.mp_encode(D, x[None, :], 4)
    assert res.coef[0, 0] < 0                              # the case that tells the readings apart
    R = x.astype(np.float64).copy()
    e = 0.0
    for _ in range(4):
        c = D.astype(np.float64) @ R
        i = int(np.argmax(np.abs(c)))
        R = R - abs(c[i]) * D[i]                           # the literal reading of Eq. 2
        e += c[i] ** 2
    x64 = x.astype(np.float64)
    assert abs((x64 ** 2).sum() - (R ** 2).sum() - e) > 1e-3                       # literal reading: identity broken
    e_or = float((res.coef[0] ** 2 * (2.0 - (D[res.idx[0]].astype(np.float64) ** 2).sum(1))).sum())
    assert abs((x64 ** 2).sum() - (res.residual[0] ** 2).sum() - e_or) < 1e-12     # the oracle: identity holds
    assert np.linalg.norm(res.residual[0]) < np.linalg.norm(R) - 1e-3


# ---------------------------------------------------------------------------------------
# chunks and the online part of a dictionary
# ---------------------------------------------------------------------------------------

def test_dict_append_closed_forms():
    """3-4-0 triangle, unit norm, direction, scale invariance, zero row, untouched atoms."""
    rng = np.random.default_rng(3)
    D = np.zeros((6, 4), np.float32)
    D[0] = [1, 0, 0, 0]
    X = np.array([[3, 4, 0, 0], [0, 0, 0, 0], [-2, 0, 0, 0], [1, 1, 1, 1]], np.float32)
    out = orc.dict_append(D, 1, X, [0, 1, 2, 3])
    assert np.array_equal(out[0], D[0]) and np.array_equal(out[5], D[5])
    assert np.allclose(out[1], [0.6, 0.8, 0, 0], rtol=0, atol=1e-7)
    assert np.array_equal(out[2], np.zeros(4, np.float32))
    assert np.array_equal(out[3], np.array([-1, 0, 0, 0], np.float32))
    assert np.allclose(out[4], 0.5)
    Y = rng.standard_normal((50, 64)).astype(np.float32)
    E = orc.dict_append(np.zeros((50, 64), np.float32), 0, Y, np.arange(50))
    assert np.allclose(np.linalg.norm(E.astype(np.float64), axis=1), 1.0, atol=1e-7)
    cos = np.sum(E.astype(np.float64) * Y, axis=1) / np.linalg.norm(Y.astype(np.float64), axis=1)
    assert np.allclose(cos, 1.0, atol=1e-7)
    E2 = orc.dict_append(np.zeros((50, 64), np.float32), 0, Y * np.float32(8.0), np.arange(50))
    assert np.array_equal(E, E2)                          # scaling by a power of two changes nothing
    with pytest.raises(ValueError):
        orc.dict_append(D, 4, X, [0, 1, 2])


def test_an_appended_atom_encodes_its_own_row_in_one_step():
    """A sampled row becomes an atom that represents it exactly: first pick = that atom,
    coefficient = the row's norm, residual zero."""
    rng = np.random.default_rng(4)
    X = rng.standard_normal((8, 32)).astype(np.float32)
    D0 = np.zeros((40, 32), np.float32)
    D0[:32] = np.eye(32, dtype=np.float32)
    D = orc.dict_append(D0, 32, X, np.arange(8))
    res = orc.mp_encode(D, X, 1)
    assert np.array_equal(res.idx[:, 0], 32 + np.arange(8))
    assert np.allclose(res.coef[:, 0], np.linalg.norm(X.astype(np.float64), axis=1), rtol=1e-6)
    assert np.all(res.resnorm[:, 0] < 1e-6 * np.linalg.norm(X, axis=1))


def test_chunked_encode_is_independent_per_chunk():
    """s_n = 2 with an orthonormal dictionary per chunk and s = d_h / s_n recovers x exactly;
    changing chunk 1 of x or its dictionary leaves the codes of chunk 0 alone; the stored size
    is 4 * s * s_n bytes per head vector."""
    rng = np.random.default_rng(5)
    d_h, s_n = 16, 2
    Q0 = np.linalg.qr(rng.standard_normal((8, 8)))[0].astype(np.float32)
    Q1 = np.linalg.qr(rng.standard_normal((8, 8)))[0].astype(np.float32)
    X = rng.standard_normal((20, d_h)).astype(np.float32)
    res = orc.mp_encode_chunked([Q0, Q1], X, 8)
    xh = orc.reconstruct_chunked([Q0, Q1], [r.idx for r in res], [r.coef for r in res])
    assert np.allclose(xh, X, atol=1e-5)
    X2 = X.copy()
    X2[:, 8:] = rng.standard_normal((20, 8)).astype(np.float32)
    res2 = orc.mp_encode_chunked([Q0, Q0], X2, 8)
    assert np.array_equal(res2[0].idx, res[0].idx) and np.array_equal(res2[0].coef, res[0].coef)
    assert orc.code_bytes_per_vector(8, s_n) == 4 * 8 * 2 and orc.code_bits_per_channel(d_h, 8, s_n) == 32.0
    with pytest.raises(ValueError):
        orc.mp_encode_chunked([Q0, Q1, Q0], X, 4)


# ---------------------------------------------------------------------------------------
# attention from the restored tensors
# ---------------------------------------------------------------------------------------

def test_attention_from_codes_closed_forms():
    """Identity dictionary: the restored row is the scatter of its coefficients, so the score
    is sum_g coef * q[idx] and the mix is a weighted scatter (written here with np.add.at,
    not with the oracle's reconstruct); repeated indices accumulate; scale is linear; with
    the oracle's own codes plus the final residual the exact q . x comes back."""
    rng = np.random.default_rng(9)
    B, H, T, s, d = 2, 3, 40, 4, 16
    D = np.eye(d, dtype=np.float32)
    idx = rng.integers(0, d, (B, T, s)).astype(np.int32)
    idx[:, :, 3] = idx[:, :, 0]
    coef = rng.standard_normal((B, T, s))
    Q = rng.standard_normal((B, H, d))
    W = rng.random((B, H, T))
    sc = orc.key_scores(D, Q, idx, coef, scale=0.5)
    want = 0.5 * np.einsum("btg,bhtg->bht", coef, Q[np.arange(B)[:, None, None, None], np.arange(H)[None, :, None, None], idx[:, None]])
    assert np.allclose(sc, want, atol=1e-12)
    mix = orc.value_mix(D, W, idx, coef)
    want = np.zeros((B, H, d))
    for b in range(B):
        for h in range(H):
            np.add.at(want[b, h], idx[b].ravel(), (W[b, h][:, None] * coef[b]).ravel())
    assert np.allclose(mix, want, atol=1e-12)
    # real dictionary: q . x = scores from the codes + q . final residual
    Dn = wl.normalise_rows(rng.standard_normal((64, d)).astype(np.float32))
    X = rng.standard_normal((T, d)).astype(np.float32)
    res = orc.mp_encode(Dn, X, 5)
    q = rng.standard_normal((1, 1, d))
    sc = orc.key_scores(Dn, q, res.idx[None], res.coef[None])
    assert np.allclose(sc[0, 0] + res.residual @ q[0, 0], X.astype(np.float64) @ q[0, 0], atol=1e-12)


def test_decode_attention_is_dense_softmax_attention_of_the_restored_cache():
    """decode_attention against the textbook: restore K and V as dense matrices with a plain
    matrix product of a scattered code matrix (not the oracle's reconstruct), then
    softmax(scale * q K^T) V with scipy's softmax.  The weights are rows of a distribution;
    with one key far ahead of the rest the output is that token's restored value row."""
    from scipy.special import softmax
    rng = np.random.default_rng(21)
    B, H, T, s, d, N = 2, 3, 50, 4, 16, 40
    Dk = wl.normalise_rows(rng.standard_normal((N, d)).astype(np.float32))
    Dv = wl.normalise_rows(rng.standard_normal((N, d)).astype(np.float32))
    ki, vi = rng.integers(0, N, (B, T, s)).astype(np.int32), rng.integers(0, N, (B, T, s)).astype(np.int32)
    kc, vc = rng.standard_normal((B, T, s)), rng.standard_normal((B, T, s))
    Q = rng.standard_normal((B, H, d))
    out, w = orc.decode_attention(Dk, Dv, Q, ki, kc, vi, vc, scale=0.25)

    def dense(D, idx, coef):                              # [B][T][d] from a [T][N] code matrix times D
        X = np.zeros((B, T, d))
        for b in range(B):
            R = np.zeros((T, N))
            np.add.at(R, (np.repeat(np.arange(T), s), idx[b].ravel()), coef[b].ravel())
            X[b] = R @ D.astype(np.float64)
        return X

    K, V = dense(Dk, ki, kc), dense(Dv, vi, vc)
    want_w = softmax(0.25 * np.einsum("bhd,btd->bht", Q, K), axis=2)
    assert np.allclose(w, want_w, atol=1e-12) and np.allclose(w.sum(2), 1.0, atol=1e-12)
    assert np.allclose(out, np.einsum("bht,btd->bhd", want_w, V), atol=1e-12)
    # one key per stream with a huge score: the output is that token's restored value row
    kc2 = kc.copy()
    ki2 = ki.copy()
    ki2[:, 7, :] = 3
    kc2[:, 7, :] = 0.0
    kc2[:, 7, 0] = 1.0                                     # K[7] = atom 3
    Q2 = np.broadcast_to(1e4 * Dk[3].astype(np.float64), (B, H, d)).copy()
    out2, w2 = orc.decode_attention(Dk, Dv, Q2, ki2, kc2 * np.where(np.arange(T)[None, :, None] == 7, 1.0, 1e-3), vi, vc, scale=1.0)
    assert np.allclose(w2[:, :, 7], 1.0, atol=1e-9) and np.allclose(out2, V[:, None, 7, :], atol=1e-6)


# ---------------------------------------------------------------------------------------
# one training step of the offline dictionary
# ---------------------------------------------------------------------------------------

def test_training_gradients_match_finite_differences():
    """Both gradients against central differences of the losses themselves (codes fixed)."""
    rng = np.random.default_rng(21)
    N, d, M, s = 12, 6, 30, 3
    D = wl.normalise_rows(rng.standard_normal((N, d)).astype(np.float32))
    X = rng.standard_normal((M, d)).astype(np.float32)
    res = orc.mp_encode(D, X, s)
    l0, g_mse = orc.mse_loss_and_grad(D, X, res.idx, res.coef)
    _, g_div = orc.div_loss_and_grad(D)
    h = 1e-3                                              # fp32 storage of D limits the step size
    for (n, k) in [(0, 0), (3, 2), (7, 5), (11, 1), (int(res.idx[0, 0]), 4)]:
        Dp, Dm = D.copy(), D.copy()
        Dp[n, k] += np.float32(h)
        Dm[n, k] -= np.float32(h)
        step = float(Dp[n, k]) - float(Dm[n, k])
        fd = (orc.mse_loss_and_grad(Dp, X, res.idx, res.coef)[0] - orc.mse_loss_and_grad(Dm, X, res.idx, res.coef)[0]) / step
        assert abs(fd - g_mse[n, k]) <= 1e-3 * max(1.0, abs(fd)), (n, k, fd, g_mse[n, k])
        fd = (orc.div_loss_and_grad(Dp)[0] - orc.div_loss_and_grad(Dm)[0]) / step
        assert abs(fd - g_div[n, k]) <= 1e-3 * max(1e-3, abs(fd)), (n, k, fd, g_div[n, k])
    assert l0 == pytest.approx(float(np.sum(res.resnorm[:, -1] ** 2)), rel=1e-12)   # L_MSE is the squared MP residual


def test_diversity_loss_closed_forms_and_beta():
    """Orthonormal atoms: L_div = 0 and zero gradient; two copies of one atom among
    orthonormal ones: ||I - G||_F^2 = 2, so L_div = 2 / N^2; beta's cap and ratio."""
    Q = np.linalg.qr(np.random.default_rng(2).standard_normal((8, 8)))[0].astype(np.float64)
    l, g = orc.div_loss_and_grad(Q)
    assert l < 1e-28 and np.abs(g).max() < 1e-14
    D = Q[:5].copy()
    D[4] = D[0]
    l, _ = orc.div_loss_and_grad(D)
    assert l == pytest.approx(2.0 / 25.0, rel=1e-12)
    assert orc.adaptive_beta(5.0, 1.0) == 0.5 and orc.adaptive_beta(50.0, 1.0) == 1.0 and orc.adaptive_beta(1.0, 0.0) == 1.0


def test_training_steps_renormalise_and_lower_the_loss():
    rng = np.random.default_rng(22)
    N, d, M, s = 64, 16, 400, 4
    basis = wl.normalise_rows(rng.standard_normal((N, d)).astype(np.float32))
    codes = rng.integers(0, N, (M, 2))
    X = (basis[codes[:, 0]] * 2 + basis[codes[:, 1]] + 0.05 * rng.standard_normal((M, d))).astype(np.float32)
    D = wl.normalise_rows(rng.standard_normal((N, d)).astype(np.float32))
    beta, first = 0.0, None
    for it in range(30):
        D, l_mse, l_div, _ = orc.dict_train_step(D, X, s, lr=2e-3, beta=beta)
        beta = orc.adaptive_beta(l_mse, l_div)
        first = l_mse if first is None else first
        assert np.allclose(np.linalg.norm(D.astype(np.float64), axis=1), 1.0, atol=1e-6)
    assert l_mse < 0.8 * first


def test_train_step_with_zero_mse_gradient_is_the_diversity_step_in_closed_form():
    """Rows of X that ARE atoms (orthogonal to every other atom) are encoded exactly with s = 1, so
    grad L_MSE = 0 and the step is ReNorm(D - lr * beta * grad L_div).  With all atoms
    orthonormal except d_0 and d_1 at a known angle (d_0 . d_1 = c), D D^T - I has the single
    pair of entries c, so grad L_div is (4 / N^2) * c * d_1 on atom 0, (4 / N^2) * c * d_0 on atom 1
    and zero elsewhere: written out by hand below.  A doubled lr, beta applied to the wrong
    gradient or a wrong 4 / N^2 changes atoms 0 and 1."""
    N, d = 6, 8
    D = np.zeros((N, d), np.float32)
    D[0, 0] = 1.0
    D[1, 0], D[1, 1] = 0.6, 0.8
    for n in range(2, N):
        D[n, n] = 1.0
    X = np.stack([D[2], 2.5 * D[4], -1.5 * D[3]]).astype(np.float32)
    lr, beta = 0.05, 0.3
    Dn, l_mse, l_div, res = orc.dict_train_step(D, X, 1, lr, beta)
    assert res.idx[:, 0].tolist() == [2, 4, 3] and l_mse == 0.0
    D64 = D.astype(np.float64)
    c = float(D64[0] @ D64[1])
    n1 = float(D64[1] @ D64[1])                           # 0.6^2 + 0.8^2 in fp32 values: 1 up to 1e-8
    want = D64.copy()
    # (D D^T - I) D, rows 0 and 1: row 0 = c d_1, row 1 = c d_0 + (|d_1|^2 - 1) d_1
    want[0] = D64[0] - lr * beta * (4.0 / N ** 2) * (c * D64[1])
    want[1] = D64[1] - lr * beta * (4.0 / N ** 2) * (c * D64[0] + (n1 - 1.0) * D64[1])
    want /= np.linalg.norm(want, axis=1, keepdims=True)
    assert np.abs(Dn.astype(np.float64) - want).max() < 1e-7
    assert l_div == pytest.approx((2 * c * c + (n1 - 1.0) ** 2) / N ** 2, rel=1e-9)
    assert np.abs(Dn[0] - D[0]).max() > 1e-4              # the step is not a no-op


def test_train_step_with_orthonormal_atoms_is_the_mse_step_in_closed_form():
    """Orthonormal atoms: grad L_div = 0 whatever beta is, and the step is ReNorm(D - lr * grad
    L_MSE).  One row x = (3, 1, 0, 0) over the identity dictionary with s = 1: the pursuit takes
    atom 0 with c = 3, the error is e = (0, 1, 0, 0), the only gradient row is
    -2 c e = (0, -6, 0, 0) on atom 0, so atom 0 becomes (1, 6 lr, 0, 0) / norm and the others stay."""
    D = np.eye(4, dtype=np.float32)
    X = np.array([[3.0, 1.0, 0.0, 0.0]], np.float32)
    lr, beta = 0.01, 7.0                                  # a large beta: it must not touch this step
    Dn, l_mse, l_div, res = orc.dict_train_step(D, X, 1, lr, beta)
    assert res.idx[0, 0] == 0 and res.coef[0, 0] == 3.0
    assert l_mse == pytest.approx(1.0, abs=1e-15) and l_div == 0.0
    want = np.eye(4)
    want[0] = np.array([1.0, 6.0 * lr, 0.0, 0.0]) / np.sqrt(1.0 + 36.0 * lr * lr)
    assert np.abs(Dn.astype(np.float64) - want).max() < 1e-7
    # two rows sharing an atom add up: x_2 = (-2, 0, 1, 0) also takes atom 0 (c = -2, e = (0, 0, 1, 0))
    X2 = np.array([[3.0, 1.0, 0.0, 0.0], [-2.0, 0.0, 1.0, 0.0]], np.float32)
    Dn2, l_mse2, _, _ = orc.dict_train_step(D, X2, 1, lr, beta)
    w0 = np.array([1.0, 6.0 * lr, -4.0 * lr, 0.0])        # -lr * (-2*3*e_1 + -2*(-2)*e_2)
    want[0] = w0 / np.linalg.norm(w0)
    assert np.abs(Dn2.astype(np.float64) - want).max() < 1e-7 and l_mse2 == pytest.approx(2.0, abs=1e-15)


def test_train_step_displacement_is_linear_in_lr_to_first_order():
    """Doubling lr doubles the displacement of every atom up to O(lr^2): the codes do not depend
    on lr, and ReNorm of a unit atom moved by a small step removes the step's radial part and
    changes the rest only to second order."""
    rng = np.random.default_rng(31)
    N, d, M, s = 24, 8, 200, 3
    D = wl.normalise_rows(rng.standard_normal((N, d)).astype(np.float32))
    X = rng.standard_normal((M, d)).astype(np.float32)
    lr, beta = 1e-4, 0.5
    D1 = orc.dict_train_step(D, X, s, lr, beta)[0].astype(np.float64)
    D2 = orc.dict_train_step(D, X, s, 2 * lr, beta)[0].astype(np.float64)
    d1, d2 = D1 - D, D2 - D
    assert np.abs(d1).max() > 1e-4                        # far above the fp32 rounding of the outputs (6e-8)
    assert np.abs(d2 - 2 * d1).max() < 0.02 * np.abs(d1).max() + 3e-7
    # and beta scales the diversity part alone: the difference of two betas is lr * dbeta * grad L_div (tangential part)
    Da = orc.dict_train_step(D, X, s, lr, 0.0)[0].astype(np.float64)
    g = (4.0 / N ** 2) * ((D.astype(np.float64) @ D.astype(np.float64).T - np.eye(N)) @ D.astype(np.float64))
    tang = g - (g * D).sum(1, keepdims=True) * D          # ReNorm removes the radial part to first order
    assert np.abs((Da - D1) - lr * beta * tang).max() < 0.02 * np.abs(lr * beta * tang).max() + 3e-7
