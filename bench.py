#!/usr/bin/env python
"""Benchmark of the CSR sparse codec hot path on B200.

One step = one pass of the whole path over one synthetic batch: csr_encode (load,
correlation, arg-max, residual update, packed code write) followed by csr_reconstruct.
The workload is the GQA long-context configuration: 8 sequences x 16384 tokens x 8 KV
heads x {K, V}, d = 128 (2,097,152 bf16 vectors), 8192 atoms, s = 16.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Prints ONE JSON line (rank 0).  `value` is vectors per second with inputs resident in
HBM; `e2e` is the same metric through csr_encode_host with pinned host buffers (copies
inside the timed region); `roofline` is the encoder kernel against the measured bf16
tensor peak; `cpu_baseline` is the fp64 oracle on the host cores on a bounded sample.
With --impl reference the oracle itself is the timed program.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "kv_vectors_encoded_per_sec"
UNIT = "vectors/s"
WORKLOAD = "gqa_long_context: 8 seq x 16384 tok x 8 kv_heads x {K,V}, d=128, M=2097152, N=8192, s=16, bf16"


# dram__bytes_read.sum + dram__bytes_write.sum of encode_fast_kernel<128, 1, 0> at M = 524288, N = 8192,
# s = 16 (profiles/encode_fast_small_case_ncu_full.md), per row; traffic grows in proportion to M.
DRAM_BYTES_PER_ROW_NCU = (137.220352e6 + 19.116288e6) / 524288


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"bf16_tflops": float(p["bf16_tflops"]), "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", 0)),
                "hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


def _make_workload(tokens: int, rank: int):
    from paper_2412_11741_b200 import workloads as wl
    w = wl.gqa_long(tokens=tokens)
    if rank:
        # other ranks encode their own batch: same recipe, rows rotated by a rank-dependent offset
        w.X = np.roll(w.X, 4099 * rank, axis=0)
    return w


# ---------------------------------------------------------------------------------------
# clocks
# ---------------------------------------------------------------------------------------

class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1]))
                    mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            # the sampler runs only around the timed region: the median over all samples is the clock under load
            out["sm_mhz"] = statistics.median(sm)
            out["sm_max_mhz"] = max(mx)
            out["samples"] = len(sm)
        out["reasons"] = sorted(reasons)
        return out


# ---------------------------------------------------------------------------------------
# CPU legs (the oracle as it stands)
# ---------------------------------------------------------------------------------------

def _oracle_rate(w, target_seconds: float):
    """Times the oracle (encode + reconstruct) on a prefix sample sized for about target_seconds."""
    from oracle import csr_oracle as orc
    probe = 256
    t0 = time.perf_counter()
    r = orc.mp_encode(w.D, w.X[:probe], w.s)
    orc.reconstruct(w.D, r.idx, r.coef)
    dt = max(time.perf_counter() - t0, 1e-3)
    rows = int(min(w.M, max(probe, (target_seconds / dt) * probe)))
    rows = max(256, (rows // 256) * 256)
    sel = np.linspace(0, w.M - 1, rows).astype(np.int64)
    X = np.ascontiguousarray(w.X[sel])
    t0 = time.perf_counter()
    r = orc.mp_encode(w.D, X, w.s)
    orc.reconstruct(w.D, r.idx, r.coef)
    dt = time.perf_counter() - t0
    return rows / dt, rows, dt, orc.num_threads()


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from oracle import csr_oracle as orc
    orc.build()
    w = _make_workload(args.tokens, 0)
    per_step_target = max(2.0, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
    rates, rows_used = [], 0
    for i in range(args.warmup + args.steps):
        rate, rows, dt, cores = _oracle_rate(w, per_step_target)
        if i >= args.warmup:
            rates.append((rows, dt))
        rows_used = rows
    tot_rows = sum(r for r, _ in rates)
    tot_t = sum(t for _, t in rates)
    value = tot_rows / tot_t
    sample = f"{rows_used} evenly spaced rows of the workload per step (oracle encode + reconstruct, fp64)"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * tot_t / max(1, len(rates)), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "tokens_per_sequence": args.tokens, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


# ---------------------------------------------------------------------------------------
# the CUDA arm
# ---------------------------------------------------------------------------------------

def run_cuda(args):
    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    from paper_2412_11741_b200 import build
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    import paper_2412_11741_b200 as csr

    w = _make_workload(args.tokens, rank)
    M, N, d, s = w.M, w.N, w.d, w.s
    D = torch.from_numpy(w.D).to(dev)
    X_host = torch.from_numpy(w.X).to(torch.bfloat16).pin_memory()
    X = X_host.to(dev)
    out_idx = torch.empty((M, s), dtype=torch.uint16, device=dev)
    out_coef = torch.empty((M, s), dtype=torch.float16, device=dev)
    X_hat = torch.empty((M, d), dtype=torch.bfloat16, device=dev)
    idx_host = torch.empty((M, s), dtype=torch.uint16).pin_memory()
    coef_host = torch.empty((M, s), dtype=torch.float16).pin_memory()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # the dictionary is fixed for a layer's lifetime: its 16-bit copies are made once, as a cache does
    handle = csr.csr_dict_create(D)

    def step(ev=None):
        if ev:
            ev[0].record()
        csr.csr_encode_ex(D, X, s, out_idx=out_idx, out_coef=out_coef, dict=handle)
        if ev:
            ev[1].record()
        csr.csr_reconstruct_ex(D, out_idx, out_coef, X_hat=X_hat, dict=handle)
        if ev:
            ev[2].record()

    for _ in range(max(3, args.warmup)):
        step()
    torch.cuda.synchronize()
    if csr.csr_device_status() != csr.CSR_OK:
        raise SystemExit("device-side wait expired during warm-up: " + csr.csr_last_error_string())

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    barrier()
    for i in range(args.steps):
        step(evs[i])
    barrier()
    enc_ms = [e[0].elapsed_time(e[1]) for e in evs]
    rec_ms = [e[1].elapsed_time(e[2]) for e in evs]
    total_ms = evs[0][0].elapsed_time(evs[-1][2])
    clocks = sampler.stop() if rank == 0 else {}
    if csr.csr_device_status() != csr.CSR_OK:
        raise SystemExit("device-side wait expired: " + csr.csr_last_error_string())

    # end to end through the host entry points (pinned host buffers, every copy inside the
    # timing): X in, codes out, then codes in, X_hat out
    xhat_host = torch.empty((M, d), dtype=torch.bfloat16).pin_memory()

    def e2e_step():
        csr.csr_encode_host(D, X_host, s, idx_host, coef_host, dict=handle)
        csr.csr_reconstruct_host(D, idx_host, coef_host, xhat_host, dict=handle)

    e2e_steps = max(1, min(args.steps, 5))
    e2e_step()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    barrier()
    e2e_s = (time.perf_counter() - t0) / e2e_steps

    # beside the timed steps: the same workload through the exact mode (the oracle's picks index for
    # index; its sweep runs on the tensor cores with three bf16 products per correlation)
    ex_idx = torch.empty((M, s), dtype=torch.uint16, device=dev)
    ex_coef = torch.empty((M, s), dtype=torch.float32, device=dev)
    ex_ms = []
    for i in range(3):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        csr.csr_encode_ex(D, X, s, mode=csr.CSR_MODE_FP32_EXACT, out_idx=ex_idx, out_coef=ex_coef, coef_dtype=torch.float32)
        b.record()
        torch.cuda.synchronize()
        if i:
            ex_ms.append(a.elapsed_time(b))
    if csr.csr_device_status() != csr.CSR_OK:
        raise RuntimeError(csr.csr_last_error_string())
    exact_ms = max(ex_ms)
    del ex_idx, ex_coef

    t = torch.tensor([total_ms, e2e_s, exact_ms], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    total_ms, e2e_s, exact_ms = float(t[0]), float(t[1]), float(t[2])

    if rank == 0:
        peaks = _peaks()
        ms_per_step = total_ms / args.steps
        value = world * M / (ms_per_step * 1e-3)
        enc = statistics.mean(enc_ms)
        flops = 2.0 * M * N * d * s
        achieved = flops / (enc * 1e-3) / 1e12
        hbm_bytes = M * d * 2 + N * d * 4 + M * s * 4
        roof = {
            "bound": "tensor", "kernel": "encode_fast_kernel<128, 1, 0>", "achieved": achieved, "peak": peaks["bf16_tflops"],
            "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"], "peak_source": peaks["source"] + " (burst)",
            "frac_of_sustained": achieved / peaks["bf16_tflops_sustained"] if peaks["bf16_tflops_sustained"] else None,
            "flops_per_launch": flops, "kernel_ms": enc, "traffic": DRAM_BYTES_PER_ROW_NCU * M,
            "traffic_source": "ncu dram read+write of one launch at M=524288 (profiles/), scaled by rows",
            "algorithmic_hbm_bytes": hbm_bytes,
        }
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup),
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "tokens_per_sequence": args.tokens, "M_per_gpu": M, "N": N, "d": d, "s": s,
                       "mode": "bf16_fast", "l2": "inputs (537 MB per step) larger than L2; no flush",
                       "step": "csr_encode_ex + csr_reconstruct_ex with a prepared dictionary handle (csr_dict_create once, "
                               "outside the timed region)",
                       "parallelism": f"rows sharded x{world}, no collective"},
            "encode_ms": enc, "reconstruct_ms": statistics.mean(rec_ms),
            "encode_vectors_per_sec": M / (enc * 1e-3),
            "clocks": clocks,
            "e2e": {"value": world * M / e2e_s, "unit": UNIT, "h2d_bytes_per_step": M * d * 2 + M * s * 4,
                    "d2h_bytes_per_step": M * s * 4 + M * d * 2, "ms_per_step": e2e_s * 1e3,
                    "call": "csr_encode_host (pinned host X in, host codes out) + csr_reconstruct_host "
                            "(host codes in, pinned host X_hat out)"},
            "gpu_launches": 2 * args.steps,
            "roofline": roof,
            "exact_mode": {"value": world * M / (exact_ms * 1e-3), "unit": UNIT, "ms": exact_ms,
                           "tflops_algorithmic": flops / (exact_ms * 1e-3) / 1e12,
                           "frac_of_bf16_burst": flops / (exact_ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                           "note": "csr_encode_ex in CSR_MODE_FP32_EXACT on the same rows, outside the timed steps: "
                                   "three bf16 MMAs per correlation, fp64 re-scoring inside the error band"},
        }
        if not args.no_cpu_baseline and world == 1:
            from oracle import csr_oracle as orc
            orc.build()
            rate, rows, dt, cores = _oracle_rate(w, 15.0)
            line["cpu_baseline"] = {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle",
                                    "sample": f"{rows} evenly spaced rows of the workload, {dt:.1f} s (fp64 encode + reconstruct)"}
        print(json.dumps(line), flush=True)
    csr.csr_dict_destroy(handle)
    if world > 1:
        dist.destroy_process_group()
    return 0


def launch_ranks(n: int, argv, script: str = None, backend_env: dict = None) -> int:
    """Starts n ranks of `script` (this file) on one node, one process per GPU, the way the
    multi-GPU form of this benchmark is meant to be launched, and returns the exit code.  Rank 0's
    single JSON line reaches this process's stdout unchanged.  NCCL's own log (which states the
    communicator's rank count) goes to files that are then copied to stderr."""
    import socket
    sock = socket.socket()
    sock.bind(("127.0.0.1", 0))
    port = sock.getsockname()[1]
    sock.close()
    env = dict(os.environ)
    logdir = tempfile.mkdtemp(prefix="bench_nccl_")
    env.setdefault("NCCL_DEBUG", "INFO")
    env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    env.setdefault("NCCL_DEBUG_FILE", os.path.join(logdir, "nccl_%h_%p.log"))
    env.update(backend_env or {})
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), script or os.path.abspath(__file__)] + list(argv)
    rc = subprocess.call(cmd, env=env)
    try:
        for name in sorted(os.listdir(logdir)):
            for line in open(os.path.join(logdir, name), errors="replace"):
                if "nranks" in line or "Init COMPLETE" in line:
                    sys.stderr.write(line)
            os.unlink(os.path.join(logdir, name))
        os.rmdir(logdir)
    except OSError:
        pass
    return rc


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--tokens", type=int, default=16384, help="tokens per sequence (16384 = the full configuration)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # called as `python bench.py --gpus N`: start the N ranks here
        return launch_ranks(args.gpus, sys.argv[1:])
    return run_cuda(args)


if __name__ == "__main__":
    sys.exit(main())
