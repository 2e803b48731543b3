"""The comparison rules used by the GPU parity tests, exercised on CPU: the oracle's own
output passes, planted mistakes fail, and a bf16-operand emulation of matching pursuit
(the arithmetic the fast mode uses) passes the fast-mode gates."""
import numpy as np

from oracle import csr_oracle as orc
from paper_2412_11741_b200 import workloads as wl
from tests import parity


def test_exact_rules_accept_oracle_and_reject_mistakes():
    w = wl.tiny(M=300)
    res = orc.mp_encode(w.D, w.X, w.s)
    rep = parity.compare_exact(w.D, w.X, w.s, res.idx, res.coef.astype(np.float32), res)
    assert rep.ok and rep.unexplained_rows == 0 and rep.exempt_rows == 0
    bad = res.idx.copy()
    bad[17, 3] = (bad[17, 3] + 1) % w.N
    assert not parity.compare_exact(w.D, w.X, w.s, bad, res.coef, res).ok
    c = res.coef.copy()
    c[5, 0] *= 1.001
    assert not parity.compare_exact(w.D, w.X, w.s, res.idx, c, res).ok
    c = res.coef.copy()
    c[5, 2] = -c[5, 2]
    assert not parity.compare_exact(w.D, w.X, w.s, res.idx, c, res).ok


def test_exact_rules_excuse_only_true_ties():
    D = np.array([[1, 0], [0, 1], [1, 0]], np.float32)
    X = np.array([[2.0, 1.0]] * 8, np.float32)
    res = orc.mp_encode(D, X, 2)
    alt = res.idx.copy()
    alt[:, 0] = 2                      # atom 2 equals atom 0: an exact tie at step 0
    # eight excused rows out of eight is flagged as "too many ties": a real bug looks like that
    assert not parity.compare_exact(D, X, 2, alt, res.coef, res).ok
    rep = parity.compare_exact(D, X[:1], 2, alt[:1], res.coef[:1])
    assert rep.exempt_rows == 1 and rep.unexplained_rows == 0 and rep.ok


def _bf16_mp(D, X, s):
    Db = wl.round_to_bf16(D)
    R = wl.round_to_bf16(X.astype(np.float32))
    idx = np.zeros((X.shape[0], s), np.int32)
    coef = np.zeros((X.shape[0], s), np.float32)
    for g in range(s):
        C = R @ Db.T
        i = np.argmax(np.abs(C), axis=1)
        a = Db[i]
        c = np.einsum("ij,ij->i", R, a).astype(np.float32)
        R = wl.round_to_bf16(R - c[:, None] * a)
        idx[:, g], coef[:, g] = i, c
    return idx, coef


def test_fast_rules_accept_bf16_emulation_and_reject_mistakes():
    w = wl.llama2_layer(tokens=8, N=1024)
    X = w.X[wl.stratified_rows(w.M, 512, 3)]
    res = orc.mp_encode(w.D, X, w.s)
    idx, coef = _bf16_mp(w.D, X, w.s)
    i16, c16 = orc.pack_codes(idx, coef.astype(np.float64))
    rep = parity.compare_fast(w.D, X, w.s, i16, c16.astype(np.float32), res)
    assert rep.ok, rep.detail
    assert 0.5 * rep.rows < rep.same_rows
    # a wrong sign, a stale residual (no update), an off-by-one index: all must fail
    c = coef.copy()
    c[:, 1] = -c[:, 1]
    assert not parity.compare_fast(w.D, X, w.s, idx, c, res).ok
    shifted = (idx + 1) % w.N
    assert not parity.compare_fast(w.D, X, w.s, shifted, coef, res).ok
    stale = np.repeat(idx[:, :1], w.s, axis=1)
    assert not parity.compare_fast(w.D, X, w.s, stale, np.repeat(coef[:, :1], w.s, axis=1), res).ok
