"""The multi-GPU path shards rows and has no data-path collective; its host logic is
covered here with two gloo ranks on CPU."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2412_11741_b200 import sharding


@pytest.mark.parametrize("M,world", [(0, 2), (1, 2), (255, 2), (256, 2), (257, 2), (2097152, 8), (1000003, 4), (700, 3)])
def test_shard_rows_partition(M, world):
    spans = [sharding.shard_rows(M, r, world) for r in range(world)]
    assert spans[0][0] == 0 and spans[-1][1] == M
    for (a0, a1), (b0, b1) in zip(spans, spans[1:]):
        assert a1 == b0 and a0 <= a1
    for b, e in spans:
        assert b % sharding.ROW_ALIGN == 0 or b == M
    sizes = [e - b for b, e in spans]
    assert max(sizes) - min(sizes) < 2 * sharding.ROW_ALIGN   # one extra block plus the ragged tail


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, M, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import csr_oracle as orc
    from paper_2412_11741_b200 import workloads as wl
    w = wl.llama2_layer(tokens=4, N=128)
    b, e = sharding.shard_rows(M, rank, world)
    res = orc.mp_encode(w.D, w.X[b:e], 4)          # each rank encodes only its rows
    Dl = torch.from_numpy(w.D.copy()) if rank == 0 else torch.zeros(w.D.shape)
    sharding.install_dictionary(Dl, src=0)         # rank 1 starts without the dictionary
    assert np.array_equal(Dl.numpy(), w.D)
    rate = sharding.job_rate(e - b, 1.0 + rank)    # rank 1 is "slower"
    np.save(os.path.join(out, f"idx{rank}.npy"), res.idx)
    np.save(os.path.join(out, f"meta{rank}.npy"), np.array([b, e, rate]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_cover_all_rows_and_agree_on_rate(tmp_path):
    from oracle import csr_oracle as orc
    from paper_2412_11741_b200 import workloads as wl
    orc.build()
    M, world = 256, 2
    mp.spawn(_worker, args=(world, _free_port(), M, str(tmp_path)), nprocs=world, join=True)
    w = wl.llama2_layer(tokens=4, N=128)
    full = orc.mp_encode(w.D, w.X[:M], 4).idx
    metas = [np.load(tmp_path / f"meta{r}.npy") for r in range(world)]
    parts = [np.load(tmp_path / f"idx{r}.npy") for r in range(world)]
    assert int(metas[0][0]) == 0 and int(metas[0][1]) == int(metas[1][0]) and int(metas[1][1]) == M
    assert np.array_equal(np.concatenate(parts), full)           # sharding changes no result
    assert metas[0][2] == metas[1][2] == M / 2.0                 # all units / slowest rank's time


def test_bench_launcher_starts_one_rank_per_gpu(capfd):
    """`python bench.py --gpus N` without torchrun's environment starts the N ranks itself:
    the launcher, run here on a stub worker over gloo, brings up a process group of N ranks
    and passes rank 0's single JSON line through."""
    import importlib.util
    import json
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    spec = importlib.util.spec_from_file_location("bench_under_test", os.path.join(root, "bench.py"))
    bench = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(bench)
    stub = os.path.join(root, "tests", "_stub_rank_worker.py")
    rc = bench.launch_ranks(2, ["--gpus", "2", "--steps", "3"], script=stub)
    out = capfd.readouterr().out
    assert rc == 0
    lines = [json.loads(l) for l in out.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    assert lines[0]["n_gpus"] == 2 and lines[0]["units"] == 2.0 and lines[0]["slowest"] == 2.0
    assert lines[0]["argv"] == ["--gpus", "2", "--steps", "3"] and "x2" in lines[0]["parallelism"]
