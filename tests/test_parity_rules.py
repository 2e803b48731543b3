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


def _emulated_report(w, rows, seed):
    X = w.X[wl.stratified_rows(w.M, rows, seed)]
    if w.x_dtype != "bf16":
        X = wl.round_to_bf16(X)                          # what the fast mode encodes
    res = orc.mp_encode(w.D, X, w.s)
    idx, coef = _bf16_mp(w.D, X, w.s)
    return parity.compare_fast(w.D, X, w.s, idx, coef, res)


def test_fast_gate_constants_come_from_the_bf16_emulation(capsys):
    """Where the fast-mode gates' numbers come from: bf16-operand matching pursuit (operands
    rounded to bf16, fp32 sums, residual rounded to bf16 after every update) on samples of every
    configuration, and on an overcomplete d = 64 dictionary taken far (s = 16), first leaves the
    oracle's trajectory at steps whose best two atoms are at most about 1.2 accumulated
    roundings apart (the gate allows FAST_GAP_C = 2.5), and its error ratios, scaled by the
    error level, stay at 0.8 of the caps or below.  Prints the distribution per case."""
    rng = np.random.default_rng(5)
    over = wl.Workload("overcomplete_d64", wl.normalise_rows(rng.standard_normal((5000, 64)).astype(np.float32)),
                       wl.round_to_bf16(rng.standard_normal((1500, 64)).astype(np.float32)), 16, "bf16")
    cases = [(wl.llama2_layer(tokens=64), 2048), (wl.gqa_long(tokens=64), 2048), (wl.sparsity_sweep(4, tokens=64), 2048),
             (wl.sparsity_sweep(32, tokens=64), 1024), (wl.dict_sweep(2048, M=4096), 2048),
             (wl.dict_sweep(16384, M=2048), 1024), (wl.dict_sweep(4096, d=64, M=4096), 2048), (wl.tiny(), 2048), (over, 1500)]
    lines = []
    for seed, (w, rows) in enumerate(cases):
        rep = _emulated_report(w, rows, seed)
        e = rep.oracle_mean_err
        lines.append(f"{w.name:26s} s={w.s:2d} N={w.N:5d} d={w.d:3d} rows={rep.rows}: err {e:.3f} same {rep.same_rows / rep.rows:.3f} "
                     f"margin max {rep.max_first_margin:.3f} rel gap max {rep.max_first_gap:.4f} "
                     f"ratio p50 {rep.ratio_p50:.4f} p99 {rep.ratio_p99:.4f} max {rep.ratio_max:.4f} mean {rep.mean_ratio:.5f} "
                     f"(p99-1)e {(rep.ratio_p99 - 1) * e:.4f} (max-1)e {(rep.ratio_max - 1) * e:.4f}")
        assert rep.ok, (w.name, rep.detail)
        assert rep.max_first_margin <= 0.6 * parity.FAST_GAP_C, (w.name, rep.max_first_margin)
        assert (rep.ratio_p99 - 1) * e <= 0.8 * parity.FAST_RATIO_P99_C, (w.name, rep.ratio_p99, e)
        assert (rep.ratio_max - 1) * e <= 0.8 * parity.FAST_RATIO_MAX_C, (w.name, rep.ratio_max, e)
    with capsys.disabled():
        print("\n" + "\n".join(lines))


def test_exact_rules_excuse_picks_below_the_oracles_own_noise_floor():
    """Two atoms, many iterations: the residual soon is orthogonal to both atoms, the correlations
    fall to 1e-16 ||x|| and the oracle's pick is decided by the rounding of its own sums: run on
    the same numbers with the channels in reverse order it picks differently, at exactly the
    steps the rule excuses (|c| <= 8 d 2^-53 ||R||), and nowhere else."""
    rng = np.random.default_rng(1141)
    for d, s in ((128, 12), (64, 18)):
        D = wl.normalise_rows(rng.standard_normal((2, d)).astype(np.float32))
        X = wl.round_to_bf16(rng.standard_normal((200, d)).astype(np.float32))
        res = orc.mp_encode(D, X, s)
        rev = orc.mp_encode(np.ascontiguousarray(D[:, ::-1]), np.ascontiguousarray(X[:, ::-1]), s)
        assert (rev.idx != res.idx).any()                  # the oracle disagrees with itself ...
        rep = parity.compare_exact(D, X, s, rev.idx, rev.coef, res)
        assert rep.ok and rep.unexplained_rows == 0, rep.detail      # ... only where the rule excuses it
        xn = np.linalg.norm(X.astype(np.float64), axis=1)
        prev = np.concatenate([xn[:, None], res.resnorm[:, :-1]], axis=1)
        first = np.where((rev.idx != res.idx).any(1), (rev.idx != res.idx).argmax(1), 0)
        rows = np.flatnonzero((rev.idx != res.idx).any(1))
        assert np.all(np.abs(res.coef[rows, first[rows]]) <= 8 * d * 2.0 ** -53 * prev[rows, first[rows]])
        # a wrong pick where the correlations are large is still rejected
        bad = res.idx.copy()
        bad[:, 1] = 1 - bad[:, 1]
        assert not parity.compare_exact(D, X, s, bad, res.coef, res).ok


def test_fast_gate_scales_with_the_residual_not_with_a_flat_gap():
    """Dictionaries of a handful of atoms: after a few steps the residual is nearly orthogonal to
    every atom, all correlations are tiny and RELATIVE gaps of 10 % and more separate atoms that
    bf16 cannot tell apart, while the absolute rule of the gate still holds; and a pick that is
    wrong by a clear margin at the first step is rejected whatever its relative gap."""
    rng = np.random.default_rng(77)
    for N in (5, 100):
        D = wl.normalise_rows(rng.standard_normal((N, 128)).astype(np.float32))
        X = wl.round_to_bf16(rng.standard_normal((600, 128)).astype(np.float32))
        res = orc.mp_encode(D, X, 4)
        idx, coef = _bf16_mp(D, X, 4)
        rep = parity.compare_fast(D, X, 4, idx, coef, res)
        assert rep.ok, (N, rep.detail)
    # second-best atom at step 0 for every row: relative gaps of a few per cent, far outside the gate
    w = wl.llama2_layer(tokens=8, N=1024)
    X = w.X[:256]
    res = orc.mp_encode(w.D, X, 1)
    C = np.abs(X.astype(np.float64) @ w.D.astype(np.float64).T)
    second = np.argsort(-C, axis=1)[:, 1].astype(np.int32)[:, None]
    c2 = np.take_along_axis(X.astype(np.float64) @ w.D.astype(np.float64).T, second.astype(np.int64), 1)
    rep = parity.compare_fast(w.D, X, 1, second, c2, res)
    assert not rep.ok and "roundings apart" in rep.detail
