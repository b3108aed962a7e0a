"""Parity of the threshold-then-subsample encoder (proof of Theorem 1) with the CPU oracle.

Bar: message indices, values, counts, the number of marked coordinates and the residual are
bit-exact; the estimate equals the binary32 rounding of the oracle's double-precision result (same
operations in the same order) and is within 1e-6 * max|g| of it.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2005_10761_b200 import workloads as wl

pytestmark = pytest.mark.gpu

PAD = 0xFFFFFFFF


@pytest.fixture(scope="module")
def lib():
    import paper_2005_10761_b200 as pkg
    from paper_2005_10761_b200 import build
    build.build()
    return pkg


def _bits(x):
    return np.ascontiguousarray(x).view(np.uint32)


def _pad(a, mult=8):
    W, d = a.shape
    out = np.zeros((W, wl.round_up(d, mult)), dtype=a.dtype)
    out[:, :d] = a
    return out


def _spiky(rng, W, d, p=0.02):
    x = rng.standard_normal((W, d)) * 1e-3
    m = rng.random((W, d)) < p
    return np.where(m, rng.standard_normal((W, d)), x).astype(np.float32)


def run_both(lib, g, m0, d, theta, k, r_max, seed=3, step=0, worker_base=0, bf16=False, ctx=None, use_step=False,
             signs=False):
    W = g.shape[0]
    ctx = ctx or lib.RTopK(d_max=d, W_max=W, r_max=r_max, k_max=k)
    ctx.set_option(3, 1 if signs else 0)
    tg = torch.from_numpy(g).cuda()
    g_or = g
    if bf16:
        tg = tg.to(torch.bfloat16)
        g_or = tg.view(torch.int16).cpu().numpy().view(np.uint16)
    tm = torch.from_numpy(m0.copy()).cuda()
    idx = torch.full((W, k), 7, dtype=torch.int32, device="cuda")
    val = torch.full((W, k), float("nan"), dtype=torch.float32, device="cuda")
    cnt = torch.full((W,), -1, dtype=torch.int32, device="cuda")
    ones = torch.full((W,), -1, dtype=torch.int32, device="cuda")
    out = torch.full((wl.round_up(d, 4),), float("nan"), dtype=torch.float32, device="cuda")
    if use_step:
        ctx.step_threshold(tg, tm, d, theta, k, seed, step, idx, val, cnt, ones, out, worker_base=worker_base)
    else:
        ctx.sparsify_threshold(tg, tm, d, theta, k, seed, step, idx, val, cnt, ones, worker_base=worker_base)
        ctx.aggregate_threshold(idx, val, cnt, ones, d, out)
    ctx.poll_status()
    m_or = m0.copy()
    o_idx, o_val, o_cnt, o_ones = oracle.sparsify_threshold(g_or, m_or, d, theta, k, seed, step, worker_base, signs)
    o64, o32 = oracle.aggregate_threshold(o_idx, o_val, o_cnt, o_ones, d)
    assert np.array_equal(ones.cpu().numpy().view(np.uint32), o_ones)
    assert np.array_equal(cnt.cpu().numpy().view(np.uint32), o_cnt)
    assert np.array_equal(idx.cpu().numpy().view(np.uint32), o_idx)
    assert np.array_equal(_bits(val.cpu().numpy()), _bits(o_val))
    assert np.array_equal(_bits(tm.cpu().numpy()[:, :d]), _bits(m_or[:, :d]))
    got = out.cpu().numpy()[:d]
    assert np.array_equal(_bits(got), _bits(o32))
    finite = g[:, :d][np.isfinite(g[:, :d])]
    scale = (float(np.abs(finite).max()) if finite.size else 0.0) or 1.0
    assert np.abs(got.astype(np.float64) - o64).max() <= 1e-6 * scale * max(1.0, float((o_ones / np.maximum(o_cnt, 1)).max()))
    return o_cnt, o_ones, tm, ctx


@pytest.mark.parametrize("d,k,theta", [(1, 1, 0.5), (5, 2, 0.0), (33, 7, 0.01), (1023, 10, 0.5), (4097, 41, 0.1),
                                       (4098, 400, 0.5), (100003, 300, 0.3), (100003, 3000, 0.3)])
def test_small_and_ragged_sizes(lib, d, k, theta):
    rng = np.random.default_rng(d * 7 + k)
    W = 3
    g = _pad(_spiky(rng, W, d, p=0.05))
    m0 = _pad(_spiky(rng, W, d, p=0.05) * 0.5)
    run_both(lib, g, m0, d, theta, k, r_max=d, worker_base=4)


@pytest.mark.parametrize("d,k,theta", [(5, 2, 0.0), (4097, 41, 0.1), (100003, 300, 0.3), (100003, 3000, 0.3)])
def test_sign_mode(lib, d, k, theta):
    rng = np.random.default_rng(d + 3 * k)
    W = 3
    g = _pad(_spiky(rng, W, d, p=0.05))
    g[0, d // 2] = np.nan
    g[1, 0] = np.inf
    m0 = _pad(_spiky(rng, W, d, p=0.05) * 0.5)
    run_both(lib, g, m0, d, theta, k, r_max=d, worker_base=2, signs=True)
    run_both(lib, g, m0, d, theta, k, r_max=d, worker_base=2, signs=True, bf16=True, use_step=True)


def test_subsampled_kept_all_and_empty_rows_in_one_call(lib):
    # row 0 marks far more than k (subsampled), row 1 fewer than k (all sent), row 2 none, row 3 exactly k
    d, k = 50000, 64
    rng = np.random.default_rng(1)
    g = (rng.standard_normal((4, d)) * 1e-3).astype(np.float32)
    g[0, rng.choice(d, 5000, replace=False)] = 2.0
    g[1, rng.choice(d, 17, replace=False)] = -3.0
    g[3, rng.choice(d, k, replace=False)] = 1.5
    cnt, ones, _, _ = run_both(lib, _pad(g), np.zeros_like(_pad(g)), d, 0.5, k, r_max=8192)
    assert ones.tolist() == [5000, 17, 0, k] and cnt.tolist() == [k, 17, 0, k]
    run_both(lib, _pad(g), np.zeros_like(_pad(g)), d, 0.5, k, r_max=8192, use_step=True)


def test_multi_tile_rows_bf16_and_carried_residual(lib):
    cfg = wl.scaled(wl.configs()["c2"], d=300001, W=5)
    theta, k = 0.8, 700
    ctx = lib.RTopK(d_max=cfg.d, W_max=cfg.W, r_max=20000, k_max=k)
    m = np.zeros((cfg.W, cfg.ld), dtype=np.float32)
    for t in range(3):
        g = wl.gradient(cfg, t, "cpu").numpy()
        cnt, ones, tm, _ = run_both(lib, g, m, cfg.d, theta, k, r_max=20000, seed=cfg.seed, step=t, ctx=ctx,
                                    use_step=(t == 1))
        assert (ones > k).all()
        m = tm.cpu().numpy()
    g = wl.gradient(cfg, 5, "cpu").numpy()
    run_both(lib, g, m, cfg.d, theta, k, r_max=20000, seed=cfg.seed, step=5, ctx=ctx, bf16=True)


def test_context_serves_rtopk_and_threshold_calls_in_turn(lib):
    # the threshold call rewrites the context's slice table on the device; the next rTop-k call must not see it
    d, W, r, k = 70001, 3, 700, 70
    rng = np.random.default_rng(9)
    g = _pad(_spiky(rng, W, d))
    ctx = lib.RTopK(d_max=d, W_max=W, r_max=4 * r, k_max=k)
    for rnd in range(2):
        run_both(lib, g, np.zeros_like(g), d, 0.4, k, r_max=4 * r, ctx=ctx, step=rnd)
        tg, tm = torch.from_numpy(g).cuda(), torch.zeros(g.shape, device="cuda")
        idx = torch.zeros((W, k), dtype=torch.int32, device="cuda")
        val = torch.zeros((W, k), dtype=torch.float32, device="cuda")
        ctx.sparsify(tg, tm, d, r, k, 11, rnd, idx, val)
        ctx.poll_status()
        m_or = np.zeros_like(g)
        o_idx, o_val = oracle.sparsify(g, m_or, d, r, k, 11, rnd)
        assert np.array_equal(idx.cpu().numpy().view(np.uint32), o_idx)
        assert np.array_equal(_bits(val.cpu().numpy()), _bits(o_val))
        assert np.array_equal(_bits(tm.cpu().numpy()), _bits(m_or))


def test_too_many_marked_coordinates_are_reported_not_written(lib):
    d, k, W = 20000, 16, 2
    g = np.zeros((W, wl.round_up(d, 8)), dtype=np.float32)
    g[0, :3000] = 1.0                      # 3000 marked > the context's r_max of 1024
    g[1, 5:25] = -1.0                      # 20 marked: fine
    ctx = lib.RTopK(d_max=d, W_max=W, r_max=1024, k_max=k)
    tg, tm = torch.from_numpy(g).cuda(), torch.zeros(g.shape, device="cuda")
    idx = torch.zeros((W, k), dtype=torch.int32, device="cuda")
    val = torch.zeros((W, k), dtype=torch.float32, device="cuda")
    cnt = torch.zeros(W, dtype=torch.int32, device="cuda")
    ones = torch.zeros(W, dtype=torch.int32, device="cuda")
    ctx.sparsify_threshold(tg, tm, d, 0.5, k, 1, 0, idx, val, cnt, ones)
    with pytest.raises(lib.RTopKError) as e:
        ctx.poll_status()
    assert e.value.status == 5
    assert ones.tolist() == [3000, 20] and cnt.tolist() == [0, k]
    assert (idx[0].cpu().numpy().view(np.uint32) == PAD).all()
    assert np.array_equal(tm[0].cpu().numpy(), g[0])              # the overflowing worker keeps all of a
    ctx.poll_status()                                              # the flag was cleared


def test_bad_arguments(lib):
    d, W, k = 1000, 2, 10
    ctx = lib.RTopK(d_max=d, W_max=W, r_max=100, k_max=k)
    g = torch.zeros((W, 1000), device="cuda")
    m = torch.zeros((W, 1000), device="cuda")
    idx = torch.full((W, k), 5, dtype=torch.int32, device="cuda")
    val = torch.zeros((W, k), device="cuda")
    cnt = torch.zeros(W, dtype=torch.int32, device="cuda")
    ones = torch.zeros(W, dtype=torch.int32, device="cuda")
    for theta, kk in [(-1.0, k), (float("nan"), k), (float("inf"), k), (0.5, 0), (0.5, k + 1)]:
        with pytest.raises(lib.RTopKError) as e:
            ctx.sparsify_threshold(g, m, d, theta, kk, 1, 0, idx, val, cnt, ones)
        assert e.value.status == 1
    torch.cuda.synchronize()
    assert (idx == 5).all()


@pytest.mark.parametrize("name,theta,k", [("c2", 0.5, 11173), ("c3_bf16", 150.0, 25557)])
def test_full_size_all_rows(lib, name, theta, k):
    # The encoder's oracle needs no sort, so every row of the full-size workloads is compared bit for bit,
    # through rtopk_step_threshold, over two rounds with the residual carried.
    cfg = wl.configs()[name]
    oracle.set_threads(8)
    ctx = lib.RTopK(d_max=cfg.d, W_max=cfg.W, r_max=cfg.r * 4, k_max=k)
    tm = wl.zero_residual(cfg, "cuda")
    m_or = np.zeros((cfg.W, cfg.ld), dtype=np.float32)
    idx = torch.zeros((cfg.W, k), dtype=torch.int32, device="cuda")
    val = torch.zeros((cfg.W, k), dtype=torch.float32, device="cuda")
    cnt = torch.zeros(cfg.W, dtype=torch.int32, device="cuda")
    ones = torch.zeros(cfg.W, dtype=torch.int32, device="cuda")
    out = torch.zeros(wl.round_up(cfg.d, 4), dtype=torch.float32, device="cuda")
    for t in range(2):
        g = wl.gradient(cfg, t, "cuda")
        ctx.step_threshold(g, tm, cfg.d, theta, k, cfg.seed, t, idx, val, cnt, ones, out)
        ctx.poll_status()
        g_or = g.cpu().view(torch.int16).numpy().view(np.uint16) if cfg.grad_dtype == "bf16" else g.cpu().numpy()
        o_idx, o_val, o_cnt, o_ones = oracle.sparsify_threshold(np.ascontiguousarray(g_or), m_or, cfg.d, theta, k,
                                                                cfg.seed, t)
        _, o32 = oracle.aggregate_threshold(o_idx, o_val, o_cnt, o_ones, cfg.d)
        assert np.array_equal(ones.cpu().numpy().view(np.uint32), o_ones)
        assert np.array_equal(cnt.cpu().numpy().view(np.uint32), o_cnt)
        assert np.array_equal(idx.cpu().numpy().view(np.uint32), o_idx)
        assert np.array_equal(_bits(val.cpu().numpy()), _bits(o_val))
        assert np.array_equal(_bits(tm.cpu().numpy()), _bits(m_or))
        assert np.array_equal(_bits(out.cpu().numpy()[:cfg.d]), _bits(o32))
        assert (o_ones > k).any()                      # some rows subsample
    oracle.set_threads(1)
