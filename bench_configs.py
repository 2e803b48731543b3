"""Throughput and reconstruction error of the codec on every synthetic configuration.

  python bench_configs.py [--configs c1,c2,c3,c4,c5,decode,attention,train,pack] [--reps 30] [--rows M] [--exact-rows E]

(`c5d64`, `c5n2048` ... `c5n16384`, `c4s4` ... `c4s32` name single cases; --rows shortens a case to
its first M rows, for profiler captures of one kernel.)

One JSON line per case: vectors/s and TFLOP/s of the fast encoder (median of the last two
thirds of `reps` back-to-back launches, i.e. after the clocks have settled under the power
cap), mean relative reconstruction error ||x - x_hat|| / ||x|| over all rows, the de-sparse
kernel's time with its HBM and L2-gather rates, and the fp32-exact encoder's rate on a
prefix of the rows.  Timed with CUDA events on torch's current stream; inputs are larger
than L2 except for the tiny configuration.
"""
from __future__ import annotations

import argparse
import json

import torch

import os
import sys

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))

from paper_2412_11741_b200 import binding as csr  # noqa: E402
from paper_2412_11741_b200 import build, workloads as wl  # noqa: E402


def _median_tail(xs):
    tail = sorted(xs[len(xs) // 3:])
    return tail[len(tail) // 2]


def _time(fn, reps):
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
    for a, b in ev:
        a.record()
        fn()
        b.record()
    torch.cuda.synchronize()
    return _median_tail([a.elapsed_time(b) for a, b in ev])


def run_case(w, reps, exact_rows=16384, rows=0):
    dev = torch.device("cuda", torch.cuda.current_device())
    if rows and rows < w.M:
        w.X = w.X[:rows]
    M, N, d, s = w.M, w.N, w.d, w.s
    D = torch.from_numpy(w.D).to(dev)
    X = torch.from_numpy(w.X).to(dev)
    if w.x_dtype == "bf16":
        X = X.to(torch.bfloat16)
    idx = torch.empty((M, s), dtype=torch.uint16, device=dev)
    coef = torch.empty((M, s), dtype=torch.float16, device=dev)
    enc_ms = _time(lambda: csr.csr_encode_ex(D, X, s, out_idx=idx, out_coef=coef), reps)
    if csr.csr_device_status() != csr.CSR_OK:
        raise RuntimeError(csr.csr_last_error_string())
    handle = csr.csr_dict_create(D)
    enc_prepared_ms = _time(lambda: csr.csr_encode_ex(D, X, s, out_idx=idx, out_coef=coef, dict=handle), reps)
    xh = torch.empty((M, d), dtype=torch.bfloat16, device=dev)
    rec_prepared_ms = _time(lambda: csr.csr_reconstruct_ex(D, idx, coef, X_hat=xh, dict=handle), max(5, reps // 3))
    csr.csr_dict_destroy(handle)
    rec_ms = _time(lambda: csr.csr_reconstruct_ex(D, idx, coef, X_hat=xh), max(5, reps // 3))
    err_sum, step = 0.0, 1 << 18
    for r0 in range(0, M, step):
        xs = X[r0:r0 + step].float()
        err_sum += float(((xh[r0:r0 + step].float() - xs).norm(dim=1) / xs.norm(dim=1).clamp_min(1e-30)).sum())
    me = min(M, exact_rows)
    ex_ms = float("nan")
    if me > 0:
        Xe = X[:me].contiguous()
        ie = torch.empty((me, s), dtype=torch.uint16, device=dev)
        ce = torch.empty((me, s), dtype=torch.float32, device=dev)
        ex_ms = _time(lambda: csr.csr_encode_ex(D, Xe, s, mode=csr.CSR_MODE_FP32_EXACT, out_idx=ie, out_coef=ce), 5)
    flops = 2.0 * M * N * d * s
    return {
        "case": w.name, "M": M, "N": N, "d": d, "s": s, "x_dtype": w.x_dtype,
        "encode_ms": round(enc_ms, 4), "encode_ms_prepared_dict": round(enc_prepared_ms, 4), "vectors_per_s": M / (enc_ms * 1e-3), "tflops": flops / (enc_ms * 1e-3) / 1e12,
        "mean_rel_error": err_sum / M,
        "reconstruct_ms": round(rec_ms, 4),
        "reconstruct_hbm_gbs": M * (4 * s + 2 * d) / (rec_ms * 1e-3) / 1e9,
        "reconstruct_l2_gather_gbs": M * s * d * 4 / (rec_ms * 1e-3) / 1e9,
        "reconstruct_ms_prepared_dict": round(rec_prepared_ms, 4),
        "reconstruct_prepared_hbm_gbs": M * (4 * s + 2 * d) / (rec_prepared_ms * 1e-3) / 1e9,
        "reconstruct_prepared_l2_gather_gbs": M * s * d * 2 / (rec_prepared_ms * 1e-3) / 1e9,
        "exact_mode_vectors_per_s": me / (ex_ms * 1e-3) if me else None, "exact_mode_rows": me,
    }


def run_decode_case(seqs, kv_heads, N, s, reps):
    """Latency of encoding the vectors ONE decoding step adds (seqs x kv_heads x {K, V} rows of
    d = 128) in each mode."""
    dev = torch.device("cuda", torch.cuda.current_device())
    w = wl.gqa_long(tokens=1, N=N, s=s, seqs=seqs, kv_heads=kv_heads)
    D = torch.from_numpy(w.D).to(dev)
    X = torch.from_numpy(w.X).to(dev)
    Xb = X.to(torch.bfloat16)
    M = w.M
    idx = torch.empty((M, s), dtype=torch.uint16, device=dev)
    coef = torch.empty((M, s), dtype=torch.float16, device=dev)
    out = {"case": f"decode_step_{seqs}x{kv_heads}x2", "M": M, "N": N, "d": w.d, "s": s}
    out["exact_split_us"] = 1e3 * _time(lambda: csr.csr_encode_ex(D, X, s, mode=csr.CSR_MODE_FP32_EXACT, out_idx=idx, out_coef=coef), reps)
    csr.csr_set_option("exact_split", 1)
    out["exact_row_tile_us"] = 1e3 * _time(lambda: csr.csr_encode_ex(D, X, s, mode=csr.CSR_MODE_FP32_EXACT, out_idx=idx, out_coef=coef), 3)
    csr.csr_set_option("exact_split", 0)
    out["fast_cluster_us"] = 1e3 * _time(lambda: csr.csr_encode_ex(D, Xb, s, out_idx=idx, out_coef=coef), reps)
    csr.csr_set_option("fast_split", 2)
    out["fast_split_us"] = 1e3 * _time(lambda: csr.csr_encode_ex(D, Xb, s, out_idx=idx, out_coef=coef), reps)
    csr.csr_set_option("fast_split", 1)
    out["fast_one_launch_us"] = 1e3 * _time(lambda: csr.csr_encode_ex(D, Xb, s, out_idx=idx, out_coef=coef), reps)
    csr.csr_set_option("fast_split", 0)
    # the step as a cache sees it: the K rows and the V rows (half of M each) against their own
    # dictionaries, one grouped call with dictionary handles
    D2 = torch.nn.functional.normalize(D.flip(0) + 0.5 * D, dim=1).contiguous()     # a second dictionary
    h1, h2 = csr.csr_dict_create(D), csr.csr_dict_create(D2)
    half = M // 2
    parts = [(D, Xb[:half], s, idx[:half], coef[:half], h1), (D2, Xb[half:], s, idx[half:], coef[half:], h2)]
    out["fast_k_and_v_grouped_us"] = 1e3 * _time(lambda: csr.csr_encode_grouped(parts), reps)
    out["fast_k_then_v_us"] = 1e3 * _time(lambda: [csr.csr_encode_ex(p[0], p[1], s, out_idx=p[3], out_coef=p[4], dict=p[5]) for p in parts], reps)
    csr.csr_dict_destroy(h1)
    csr.csr_dict_destroy(h2)
    return out


def run_attention_case(reps):
    """Attention straight from the codes on the GQA long-context shape: 64 code streams (8
    sequences x 8 KV heads) of 16384 tokens, s = 16, 4 query heads per KV head.  Rates are
    algorithmic HBM bytes (codes read once, scores written / weights read once) over time, with
    inputs rotated so that they come from HBM;
    the restored-tensor route (de-sparse kernel to bf16, then reading it back once) is timed
    beside it as the traffic it avoids."""
    dev = torch.device("cuda", torch.cuda.current_device())
    B, H, T, s, N, d = 64, 4, 16384, 16, 8192, 128
    g = torch.Generator(device=dev).manual_seed(0)
    D = torch.nn.functional.normalize(torch.randn((N, d), device=dev, generator=g), dim=1).contiguous()
    idx = torch.randint(0, N, (B, T, s), device=dev, generator=g, dtype=torch.int32).to(torch.int16).view(torch.uint16)
    coef = torch.randn((B, T, s), device=dev, generator=g).to(torch.float16)
    Q = torch.randn((B, H, d), device=dev, generator=g)
    W = torch.softmax(torch.randn((B, H, T), device=dev, generator=g), dim=-1)
    out = torch.empty((B, H, d), dtype=torch.float32, device=dev)
    xh = torch.empty((B * T, d), dtype=torch.bfloat16, device=dev)
    # three copies of the codes, weights and score arrays taken in turn: 250 MB, twice the L2, so
    # every call streams its codes from HBM as a decoding step over a long cache does
    copies = [(idx.clone(), coef.clone(), W.clone(), torch.empty((B, H, T), dtype=torch.float32, device=dev)) for _ in range(3)]
    turn = [0]

    def nxt():
        turn[0] = (turn[0] + 1) % len(copies)
        return copies[turn[0]]

    def f_scores():
        i, c, _, sc = nxt()
        csr.csr_key_scores(D, Q, i, c, 1.0, scores=sc)

    def f_mix():
        i, c, w, _ = nxt()
        csr.csr_value_mix(D, w, i, c, out=out)

    def f_restore():
        i, c, _, _ = nxt()
        csr.csr_reconstruct_ex(D, i.view(B * T, s), c.view(B * T, s), X_hat=xh)

    def f_attention():
        i, c, _, sc = nxt()
        csr.csr_decode_attention(D, D, Q, i, c, i, c, 1.0 / d ** 0.5, weights=sc, out=out)

    # one layer's whole decoding step: the B new K rows and B new V rows are encoded (two
    # dictionaries, handles, one grouped call), then the attention over the coded cache
    D2 = torch.nn.functional.normalize(D.flip(0) + 0.5 * D, dim=1).contiguous()
    hk, hv = csr.csr_dict_create(D), csr.csr_dict_create(D2)
    k_new = torch.randn((B, d), device=dev, generator=g).to(torch.bfloat16)
    v_new = torch.randn((B, d), device=dev, generator=g).to(torch.bfloat16)
    ni = [torch.empty((B, s), dtype=torch.uint16, device=dev) for _ in range(2)]
    nc = [torch.empty((B, s), dtype=torch.float16, device=dev) for _ in range(2)]

    def f_step():
        i, c, _, sc = nxt()
        csr.csr_encode_grouped([(D, k_new, s, ni[0], nc[0], hk), (D2, v_new, s, ni[1], nc[1], hv)])
        csr.csr_decode_attention(D, D2, Q, i, c, i, c, 1.0 / d ** 0.5, weights=sc, out=out)

    t_sc = _time(f_scores, reps)
    t_mx = _time(f_mix, reps)
    t_rc = _time(f_restore, reps)
    t_da = _time(f_attention, reps)
    t_st = _time(f_step, reps)
    csr.csr_dict_destroy(hk)
    csr.csr_dict_destroy(hv)
    code_b, sw_b = B * T * s * 4.0, B * H * T * 4.0
    return {"case": "attention_from_codes", "B": B, "H": H, "T": T, "N": N, "d": d, "s": s,
            "key_scores_ms": round(t_sc, 4), "key_scores_hbm_gbs": (code_b + sw_b) / (t_sc * 1e-3) / 1e9,
            "value_mix_ms": round(t_mx, 4), "value_mix_hbm_gbs": (code_b + sw_b) / (t_mx * 1e-3) / 1e9,
            "decode_attention_ms": round(t_da, 4), "encode_new_rows_plus_attention_ms": round(t_st, 4), "restore_to_bf16_ms": round(t_rc, 4), "restored_bytes": B * T * d * 2.0, "code_bytes": code_b}


def run_train_case(reps):
    """One NeuralDict training step (N = 8192 atoms, d = 128, s = 8 as in the paper's training,
    batch of 65536 key-like rows) with the tensor-core encoder as forward pass."""
    dev = torch.device("cuda", torch.cuda.current_device())
    w = wl.sparsity_sweep(8, tokens=2048)                    # 65536 key-like rows, 8192 atoms
    D = torch.from_numpy(w.D).to(dev)
    X = torch.from_numpy(w.X).to(dev).to(torch.bfloat16)
    losses = torch.empty(2, dtype=torch.float64, device=dev)
    t = _time(lambda: csr.csr_dict_train_step(D, X, 8, 1e-4, 0.1, mode=csr.CSR_MODE_BF16_FAST, losses=losses), max(5, reps // 3))
    idx = torch.empty((w.M, 8), dtype=torch.uint16, device=dev)
    coef = torch.empty((w.M, 8), dtype=torch.float32, device=dev)
    t_enc = _time(lambda: csr.csr_encode_ex(D, X, 8, out_idx=idx, out_coef=coef), max(5, reps // 3))
    l = losses.cpu().tolist()
    return {"case": "neuraldict_train_step", "M": w.M, "N": w.N, "d": w.d, "s": 8, "step_ms": round(t, 4),
            "encode_part_ms": round(t_enc, 4), "gradient_update_part_ms": round(t - t_enc, 4),
            "rows_per_s": w.M / (t * 1e-3), "L_MSE": l[0], "L_div": l[1]}


def run_pack_case(reps):
    """The stored-form writer alone: 2^28 fp32 coefficients -> fp16 (1 GiB in, 0.5 GiB out)."""
    dev = torch.device("cuda", torch.cuda.current_device())
    n = 1 << 28
    c32 = torch.randn(n, device=dev)
    c16 = torch.empty(n, dtype=torch.float16, device=dev)
    t = _time(lambda: csr.csr_pack_coefficients(c32, c16), reps)
    return {"case": "pack_coefficients", "n": n, "ms": round(t, 4), "hbm_gbs": 6.0 * n / (t * 1e-3) / 1e9}


def cases(names):
    for n in names:
        if n == "c1":
            yield wl.tiny()
        elif n == "c2":
            yield wl.llama2_layer()
        elif n == "c3":
            yield wl.gqa_long()
        elif n == "c4":
            for s in (4, 8, 16, 32):
                yield wl.sparsity_sweep(s)
        elif n == "c5":
            for N in (2048, 4096, 8192, 16384):
                yield wl.dict_sweep(N)
            yield wl.dict_sweep(4096, d=64)
        elif n == "c5d64":
            yield wl.dict_sweep(4096, d=64)
        elif n.startswith("c5n"):
            yield wl.dict_sweep(int(n[3:]))
        elif n.startswith("c4s"):
            yield wl.sparsity_sweep(int(n[3:]))
        else:
            raise SystemExit(f"unknown configuration {n}")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--configs", default="c1,c2,c3,c4,c5,decode,attention,train,pack")
    ap.add_argument("--reps", type=int, default=30)
    ap.add_argument("--rows", type=int, default=0, help="use only the first ROWS rows of each encode case")
    ap.add_argument("--exact-rows", type=int, default=16384, help="rows given to the fp32-exact encoder (0 = skip it)")
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device (there is no CPU fallback)")
    build.build()
    names = args.configs.split(",")
    for w in cases([n for n in names if n not in ("decode", "attention", "train", "pack")]):
        print(json.dumps(run_case(w, args.reps, args.exact_rows, args.rows)), flush=True)
    if "decode" in names:
        for seqs, kv_heads in ((1, 8), (8, 8), (64, 8)):
            print(json.dumps(run_decode_case(seqs, kv_heads, 8192, 16, args.reps)), flush=True)
    if "attention" in names:
        print(json.dumps(run_attention_case(args.reps)), flush=True)
    if "train" in names:
        print(json.dumps(run_train_case(args.reps)), flush=True)
    if "pack" in names:
        print(json.dumps(run_pack_case(args.reps)), flush=True)


if __name__ == "__main__":
    main()
