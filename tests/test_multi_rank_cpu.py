"""The N > 1 path on CPU: two gloo ranks.

The hot path is elementwise, so N workers are N independent shards with no
collective on the data path; what has to hold is the host-side contract:
shards cut by `shard_range` tile the tensor, every shard's packed words are
whole, the concatenation of the shards' outputs is the single-worker bit
stream, and the timing reduction (max over ranks) that bench.py uses works.
The per-shard computation here is done by the oracle (the CUDA library has no
CPU path), which is exactly what makes the concatenation property checkable
without a GPU.
"""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2202_00441_b200 import workloads as wl


def test_shard_ranges_tile_and_align():
    for n in (0, 1, 127, 128, 129, 1000, 2 ** 20, 2 ** 24 + 7):
        for world in (1, 2, 3, 8):
            cuts = [wl.shard_range(n, r, world) for r in range(world)]
            assert cuts[0][0] == 0 and cuts[-1][1] == n
            for (a, b), (c, d) in zip(cuts, cuts[1:]):
                assert b == c and a <= b
            for lo, hi in cuts[:-1]:
                assert hi % 128 == 0 or hi == n
    with pytest.raises(ValueError):
        wl.shard_range(10, 2, 2)
    # cuts on 32 elements (the unit the library's alignment rule allows): whole packed words for every width
    for n in (31, 32, 33, 2 ** 24 + 7):
        for world in (2, 5, 8):
            cuts = [wl.shard_range(n, r, world, align=32) for r in range(world)]
            assert cuts[0][0] == 0 and cuts[-1][1] == n and all(b == c for (_, b), (c, _) in zip(cuts, cuts[1:]))
            assert all(lo % 32 == 0 for lo, _ in cuts)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, n, bits, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        case = wl.Case("shard_test", ("silu",), (bits,), "bf16", (n,), 1.5, 1.0, 123)
        x, g = wl.draw(case, "cpu")                       # every rank draws the same tensor, then cuts its shard
        lo, hi = wl.shard_range(n, rank, world)
        r = oracle.dp_solve("silu", bits)
        s, lev = r["s"].astype(np.float32), r["lev"].astype(np.float32)
        xs, gs = wl.to_numpy_bits(x[lo:hi]), wl.to_numpy_bits(g[lo:hi])
        y, packed = oracle.fwd("silu", bits, s, xs)
        gi = oracle.bwd(bits, lev, packed, gs)
        # gather the shards on rank 0 (object gather: sizes differ per rank)
        gathered = [None] * world
        dist.gather_object((lo, hi, y, packed, gi), gathered if rank == 0 else None, dst=0)
        # the timing reduction bench.py uses: max over ranks
        t = torch.tensor([float(rank + 1)], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        assert t.item() == float(world)
        if rank == 0:
            y_all = np.concatenate([p[2] for p in gathered])
            gi_all = np.concatenate([p[4] for p in gathered])
            words = []
            for lo_r, hi_r, _, packed_r, _ in gathered:
                assert lo_r * bits % 32 == 0               # every shard starts on a word boundary
                words.append(packed_r if hi_r == n else packed_r[:(hi_r - lo_r) * bits // 32])
            p_all = np.concatenate(words)
            y_ref, p_ref = oracle.fwd("silu", bits, s, wl.to_numpy_bits(x))
            gi_ref = oracle.bwd(bits, lev, p_ref, wl.to_numpy_bits(g))
            ok = np.array_equal(y_all, y_ref) and np.array_equal(p_all, p_ref) and np.array_equal(gi_all, gi_ref)
            open(os.path.join(out_dir, "ok" if ok else "bad"), "w").close()
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("bits", [1, 3])
def test_two_gloo_ranks_reproduce_the_single_stream(tmp_path, bits):
    world, n = 2, 100000 + 37
    mp.spawn(_worker, args=(world, _free_port(), n, bits, str(tmp_path)), nprocs=world, join=True)
    assert os.path.exists(tmp_path / "ok")


def test_bench_starts_its_own_ranks_when_asked_for_more_than_one_gpu():
    """`python bench.py --gpus 2` started plainly (no torchrun) re-launches itself as two ranks on
    127.0.0.1.  Checked with the reference arm, which needs no GPU: rank 0 alone prints the line, and
    the line reports the two ranks."""
    import json
    import subprocess
    import sys

    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    res = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--impl", "reference", "--steps", "1",
                          "--warmup", "0", "--ref-sample", "65536"], capture_output=True, text=True, env=env, timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [json.loads(ln) for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    assert lines[0]["impl"] == "reference" and lines[0]["n_gpus"] == 2 and lines[0]["ranks_started"] == 2
