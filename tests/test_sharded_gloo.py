"""Worker-sharded round over two CPU ranks (gloo): the sharding, worker_base and all-gather logic of
paper_2005_10761_b200/sharded.py must reproduce the single-process result.  The CPU oracle stands in
for the CUDA calls here (this is a test of the host logic, not of the kernels)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2005_10761_b200 import sharded


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


W_TOTAL, D, R, K, SEED, STEP = 5, 3001, 300, 30, 17, 4


def _inputs():
    rng = np.random.default_rng(123)
    g = (rng.standard_normal((W_TOTAL, D)) * np.exp(rng.standard_normal((W_TOTAL, D)))).astype(np.float32)
    m = (rng.standard_normal((W_TOTAL, D)) * 0.1).astype(np.float32)
    return g, m


def _rank_main(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    g, m = _inputs()
    begin, rows = sharded.shard_rows(W_TOTAL, world, rank)
    g_l = torch.from_numpy(g[begin:begin + rows].copy())
    m_l = torch.from_numpy(m[begin:begin + rows].copy())

    def sparsify(gl, ml, worker_base):
        idx, val = oracle.sparsify(gl.numpy(), ml.numpy(), D, R, K, SEED, STEP, worker_base)
        return torch.from_numpy(idx.view(np.int32)), torch.from_numpy(val)

    def aggregate(idx_all, val_all):
        return torch.from_numpy(oracle.aggregate(idx_all.numpy().view(np.uint32), val_all.numpy(), D)[1])

    idx_all, val_all, out = sharded.sharded_round(sparsify, aggregate, g_l, m_l, W_TOTAL, world, rank)
    np.savez(os.path.join(out_dir, f"rank{rank}.npz"), idx=idx_all.numpy(), val=val_all.numpy(), out=out.numpy(),
             m=m_l.numpy(), begin=begin, rows=rows)
    dist.destroy_process_group()


def test_two_rank_round_equals_single_process(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    g, m = _inputs()
    m_ref = m.copy()
    idx_ref, val_ref = oracle.sparsify(g, m_ref, D, R, K, SEED, STEP, 0)
    out_ref = oracle.aggregate(idx_ref, val_ref, D)[1]
    covered = 0
    for rank in range(world):
        z = np.load(os.path.join(str(tmp_path), f"rank{rank}.npz"))
        assert np.array_equal(z["idx"].view(np.uint32), idx_ref)          # every rank holds all W messages
        assert np.array_equal(z["val"].view(np.uint32), val_ref.view(np.uint32))
        assert np.array_equal(z["out"].view(np.uint32), out_ref.view(np.uint32))
        b, n = int(z["begin"]), int(z["rows"])
        assert np.array_equal(z["m"].view(np.uint32), m_ref[b:b + n].view(np.uint32))
        covered += n
    assert covered == W_TOTAL


def test_shard_rows_partition():
    for W in (1, 5, 8, 33):
        for world in (1, 2, 3, 8):
            spans = [sharded.shard_rows(W, world, r) for r in range(world)]
            assert spans[0][0] == 0 and sum(n for _, n in spans) == W
            for (b0, n0), (b1, _) in zip(spans, spans[1:]):
                assert b0 + n0 == b1
            assert max(n for _, n in spans) - min(n for _, n in spans) <= 1
