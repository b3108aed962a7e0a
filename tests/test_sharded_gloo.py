"""Worker-sharded round over CPU ranks (gloo): the sharding, worker_base and the single all-gather of
paper_2005_10761_b200/sharded.py must reproduce the single-process result -- with two ranks, and with
three ranks whose shards are uneven (one of them shorter than the others).  The CPU oracle stands in for
the CUDA calls here (this is a test of the host logic, not of the kernels)."""
import os
import socket

import numpy as np
import pytest
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
    ex = sharded.Exchange(W_TOTAL, K, world, rank, "cpu")
    g_l = torch.from_numpy(g[ex.begin:ex.begin + ex.rows].copy())
    m_l = torch.from_numpy(m[ex.begin:ex.begin + ex.rows].copy())
    calls = {"gather": 0}
    real = dist.all_gather_into_tensor

    def counting(*a, **kw):
        calls["gather"] += 1
        return real(*a, **kw)
    dist.all_gather_into_tensor = counting

    def sparsify_pairs(gl, ml, worker_base, pairs):
        idx, val = oracle.sparsify(gl.numpy(), ml.numpy(), D, R, K, SEED, STEP, worker_base)
        pairs.copy_(sharded.pack_pairs(torch.from_numpy(idx.view(np.int32)), torch.from_numpy(val)))

    def aggregate_pairs(pairs_all):
        idx, val = sharded.unpack_pairs(pairs_all)
        return torch.from_numpy(oracle.aggregate(idx.numpy().view(np.uint32), val.numpy(), D)[1])

    pairs_all, out = sharded.sharded_round(sparsify_pairs, aggregate_pairs, g_l, m_l, ex)
    idx_all, val_all = sharded.unpack_pairs(pairs_all)
    np.savez(os.path.join(out_dir, f"rank{rank}.npz"), idx=idx_all.numpy(), val=val_all.numpy(), out=out.numpy(),
             m=m_l.numpy(), begin=ex.begin, rows=ex.rows, gathers=calls["gather"])
    dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_sharded_round_equals_single_process(tmp_path, world):
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    g, m = _inputs()
    m_ref = m.copy()
    idx_ref, val_ref = oracle.sparsify(g, m_ref, D, R, K, SEED, STEP, 0)
    out_ref = oracle.aggregate(idx_ref, val_ref, D)[1]
    covered, sizes = 0, []
    for rank in range(world):
        z = np.load(os.path.join(str(tmp_path), f"rank{rank}.npz"))
        assert int(z["gathers"]) == 1                                     # one exchange per round
        assert np.array_equal(z["idx"].view(np.uint32), idx_ref)          # every rank holds all W messages
        assert np.array_equal(z["val"].view(np.uint32), val_ref.view(np.uint32))
        assert np.array_equal(z["out"].view(np.uint32), out_ref.view(np.uint32))
        b, n = int(z["begin"]), int(z["rows"])
        assert np.array_equal(z["m"].view(np.uint32), m_ref[b:b + n].view(np.uint32))
        covered += n
        sizes.append(n)
    assert covered == W_TOTAL
    if world == 3:
        assert sizes == [2, 2, 1]                                         # an uneven split


def test_shard_rows_partition():
    for W in (1, 5, 8, 9, 33):
        for world in (1, 2, 3, 8):
            spans = [sharded.shard_rows(W, world, r) for r in range(world)]
            c = sharded.shard_block(W, world)
            assert spans[0][0] == 0 and sum(n for _, n in spans) == W
            for (b0, n0), (b1, _) in zip(spans, spans[1:]):
                assert b0 + n0 == b1
            assert max(n for _, n in spans) == c                          # the largest shard sets the step time
            assert all(b == min(W, r * c) for r, (b, _) in enumerate(spans))   # rank r's rows start at row r * c of the gathered buffer


def test_pairs_round_trip():
    idx = torch.tensor([[0, 5, 2_000_000_000]], dtype=torch.int32)
    val = torch.tensor([[-0.0, float("nan"), -3.5e38]], dtype=torch.float32)
    i2, v2 = sharded.unpack_pairs(sharded.pack_pairs(idx, val))
    assert torch.equal(i2, idx) and torch.equal(v2.view(torch.int32), val.view(torch.int32))
