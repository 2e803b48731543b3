"""Host-side checks of the seeded input generators (shapes, dtypes, determinism)."""
import numpy as np

from paper_2412_11741_b200 import workloads as wl


def test_bf16_round_trip_and_rne():
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, 0.0, 3.0e38, 1e-40], np.float32)
    b = wl.to_bf16_bits(x)
    y = wl.from_bf16_bits(b)
    assert y[0] == 1.0 and y[3] == -2.5 and y[4] == 0.0
    # 1 + 2^-8 is a tie between 1.0 and 1 + 2^-7: goes to the even mantissa (1.0)
    assert y[1] == 1.0
    # 1 + 3*2^-8 is a tie between 1+2^-7 (odd) and 1+2^-6 (even)
    assert y[2] == 1.015625
    assert np.array_equal(wl.to_bf16_bits(y), b)
    r = np.random.default_rng(0).standard_normal(10000).astype(np.float32)
    assert np.all(np.abs(wl.round_to_bf16(r) - r) <= np.abs(r) * 2.0 ** -8)


def test_tiny_config():
    w = wl.tiny()
    assert w.X.shape == (4096 + 64, 128) and w.D.shape == (1024, 128) and w.s == 8
    assert w.X.dtype == np.float32 and w.D.dtype == np.float32
    np.testing.assert_allclose(np.linalg.norm(w.D.astype(np.float64), axis=1), 1.0, atol=3e-7)
    w2 = wl.tiny()
    assert np.array_equal(w.X, w2.X) and np.array_equal(w.D, w2.D)
    lo, hi = w.meta["sparse_rows"]
    sup, amp = w.meta["support"], w.meta["amp"]
    assert np.all((np.abs(amp) >= 1) & (np.abs(amp) <= 2))
    x0 = (amp[0][:, None] * w.D[sup[0]].astype(np.float64)).sum(0)
    np.testing.assert_allclose(w.X[lo], x0, rtol=1e-6, atol=1e-6)


def test_kv_configs_small():
    w = wl.llama2_layer(tokens=16, N=256)
    assert w.X.shape == (2 * 32 * 16, 128) and w.D.shape == (256, 128) and w.x_dtype == "bf16"
    assert np.array_equal(wl.round_to_bf16(w.X), w.X)
    nk = w.meta["n_key_rows"]
    ch = w.meta["outlier_channels"]
    k0 = w.X[:16]
    assert np.abs(k0[:, ch[0]]).mean() > 4 * np.abs(np.delete(k0, ch[0], axis=1)).mean()
    assert abs(w.X[nk:].std() - 1.0) < 0.05
    np.testing.assert_allclose(np.linalg.norm(w.D.astype(np.float64), axis=1), 1.0, atol=3e-7)
    w3 = wl.gqa_long(tokens=8, N=128)
    assert w3.X.shape == (2 * 64 * 8, 128) and w3.s == 16
    w4 = wl.sparsity_sweep(4, tokens=8, N=128)
    assert w4.X.shape == (32 * 8, 128) and w4.s == 4
    w5 = wl.dict_sweep(256, d=64, M=512)
    assert w5.X.shape == (512, 64) and w5.D.shape == (256, 64)
    assert len(w5.meta["outlier_channels"]) == 1
    assert len(wl.dict_sweep(64, d=128, M=8).meta["outlier_channels"]) == 3


def test_stratified_rows():
    r = wl.stratified_rows(1000, 100, seed=1)
    assert len(np.unique(r)) == 100 and r.min() >= 0 and r.max() < 1000
    assert np.all(np.diff(r) > 0)
    assert np.array_equal(r, wl.stratified_rows(1000, 100, seed=1))
    assert len(wl.stratified_rows(5, 100)) == 5
