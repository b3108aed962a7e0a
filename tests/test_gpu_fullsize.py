"""Parity at the full sizes of the named configurations, in the launch configuration bench.py times
(rtopk_step / rtopk_step_segmented on all W rows).

The oracle's full sort is too slow for every row at these sizes, so per configuration
  * a sample of worker rows is followed through the steps by the oracle and compared bit for bit
    (indices, values, residual row);
  * every row is checked on the GPU against properties that hold at any size: exactly k strictly
    ascending in-range indices, values are a bit copy of a = g + m at those indices, sent + residual
    reassembles a exactly, sent slots hold +0, every sent key is at least the reported threshold and
    the number of keys above the threshold matches the reported count;
  * the dense update is compared with the oracle's aggregate of the very messages the GPU produced
    (all W rows), bit for bit, which also meets the 1e-6 * max|g| bar.
"""
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

import oracle
from paper_2005_10761_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lib():
    import paper_2005_10761_b200 as pkg
    from paper_2005_10761_b200 import build
    build.build()
    oracle.set_threads(8)
    return pkg


def _free_bytes() -> int:
    """Free device memory once this process has given back what its allocator only caches."""
    import gc
    gc.collect()
    torch.cuda.empty_cache()
    return torch.cuda.mem_get_info()[0]


def _bits(t: torch.Tensor) -> torch.Tensor:
    return t.view(torch.int32)


def _host_grad(cfg, g_rows: torch.Tensor) -> np.ndarray:
    if cfg.grad_dtype == "bf16":
        return g_rows.cpu().view(torch.int16).numpy().view(np.uint16).copy()
    return g_rows.cpu().numpy().copy()


def _check_rows_on_gpu(cfg, ctx, g, m_prev, m_new, idx, val, seg):
    """Size-independent properties, all W rows, computed with torch on the device."""
    d = cfg.d
    S = len(cfg.seg_r) if seg else 1
    for w in range(cfg.W):
        # (m_prev None: the residual before the step was zero; the add still happens: -0 + +0 = +0)
        a = g[w, :d].to(torch.float32) + (m_prev[w, :d] if m_prev is not None else 0.0)
        i = idx[w].to(torch.int64)
        assert bool((i[1:] > i[:-1]).all()) and int(i[0]) >= 0 and int(i[-1]) < d
        assert torch.equal(_bits(val[w]), _bits(a[i]))
        assert bool((_bits(m_new[w, :d][i]) == 0).all())
        back = m_new[w, :d].clone()
        back[i] = val[w]
        assert torch.equal(_bits(back), _bits(a))
        key = _bits(a) & 0x7FFFFFFF
        at = 0
        for s in range(S):
            st = ctx.stats(w * S + s)
            lo, hi = (cfg.seg_off[s], cfg.seg_off[s + 1]) if seg else (0, d)
            r_s, k_s = (cfg.seg_r[s], cfg.seg_k[s]) if seg else (cfg.r, cfg.k)
            if r_s < hi - lo:
                ks = key[lo:hi]
                n_gt = int((ks > st["tau_key"]).sum())
                n_eq = int((ks == st["tau_key"]).sum())
                assert n_gt == st["n_greater"] and n_gt < r_s <= n_gt + n_eq      # tau is the r-th largest
                assert st["tie_quota"] == r_s - n_gt
                sent = key[i[at:at + k_s]]
                assert bool((sent >= st["tau_key"]).all())                        # U is inside the top-r set
            at += k_s


def _run_config(lib, cfg, steps, sample_rows, path=0, finish=0):
    seg = cfg.seg_off is not None
    K = cfg.k_total
    ctx = lib.RTopK(d_max=cfg.d, W_max=cfg.W, r_max=cfg.r, k_max=K, segments_max=len(cfg.seg_r) if seg else 1)
    ctx.set_option(0, path)                          # RTOPK_OPT_SELECT_PATH
    ctx.set_option(5, finish)                        # RTOPK_OPT_FINISH_PATH
    m = wl.zero_residual(cfg, "cuda")
    idx = torch.zeros((cfg.W, K), dtype=torch.int32, device="cuda")
    val = torch.zeros((cfg.W, K), dtype=torch.float32, device="cuda")
    out = torch.empty(wl.round_up(cfg.d, 4), dtype=torch.float32, device="cuda")
    m_or = np.zeros((len(sample_rows), cfg.ld), dtype=np.float32)
    for t in range(steps):
        g = wl.gradient(cfg, t, "cuda")
        m_prev = m.clone() if t > 0 else None          # m^0 = 0: no copy needed for the first step
        if seg:
            ctx.step_segmented(g, m, cfg.d, cfg.seg_off, cfg.seg_r, cfg.seg_k, cfg.seed, t, idx, val, out)
        else:
            ctx.step(g, m, cfg.d, cfg.r, cfg.k, cfg.seed, t, idx, val, out)
        ctx.poll_status()
        _check_rows_on_gpu(cfg, ctx, g, m_prev, m, idx, val, seg)
        del m_prev
        # sampled rows against the oracle (each row is an independent worker: worker_base = its id);
        # the rows' full sorts run side by side on host threads (the oracle call releases the GIL)
        idx_h, val_h = idx.cpu().numpy().view(np.uint32), val.cpu().numpy()

        def follow(n_w):
            n, w = n_w
            g_h = _host_grad(cfg, g[w:w + 1])
            if seg:
                return oracle.sparsify_segmented(g_h, m_or[n:n + 1], cfg.d, cfg.seg_off, cfg.seg_r, cfg.seg_k,
                                                 cfg.seed, t, worker_base=w)
            return oracle.sparsify(g_h, m_or[n:n + 1], cfg.d, cfg.r, cfg.k, cfg.seed, t, worker_base=w)
        with ThreadPoolExecutor(max_workers=max(1, min(4, len(sample_rows)))) as pool:
            followed = list(pool.map(follow, enumerate(sample_rows)))
        for n, w in enumerate(sample_rows):
            o_idx, o_val = followed[n]
            assert np.array_equal(idx_h[w], o_idx[0]), f"{cfg.name} step {t} worker {w}: indices"
            assert np.array_equal(val_h[w].view(np.uint32), o_val[0].view(np.uint32)), f"{cfg.name} step {t} worker {w}: values"
            assert np.array_equal(m[w].cpu().numpy().view(np.uint32), m_or[n].view(np.uint32)), f"{cfg.name} step {t} worker {w}: residual"
        # the update against the oracle's aggregate of the GPU's own messages
        o64, o32 = oracle.aggregate(idx_h, val_h, cfg.d)
        got = out.cpu().numpy()[: cfg.d]
        gmax = float(g.to(torch.float32).abs().max())
        assert np.abs(got.astype(np.float64) - o64).max() <= 1e-6 * gmax
        assert np.array_equal(got.view(np.uint32), o32.view(np.uint32))
        del g
    fallbacks = sum(ctx.stats(s)["used_fallback"] for s in range(cfg.W * (len(cfg.seg_r) if seg else 1)))
    ctx.close()
    return fallbacks


def test_c1_every_row(lib):
    cfg = wl.configs()["c1"]
    _run_config(lib, cfg, 1, list(range(cfg.W)))


def test_c2_three_steps_with_carried_residual(lib):
    assert _run_config(lib, wl.configs()["c2"], 3, [0, 5]) == 0       # the sampled bracket holds on this data


def test_c2_paper_setting_five_nodes(lib):
    _run_config(lib, wl.configs()["c2_n5"], 1, [4])


def test_c2_exact_path_full_size(lib):
    _run_config(lib, wl.configs()["c2"], 1, [7], path=1)


@pytest.mark.parametrize("name", ["c3_f32", "c3_bf16"])
def test_c3_two_steps(lib, name):
    _run_config(lib, wl.configs()[name], 2, [3])


def test_c3_and_c4_finished_from_the_runs(lib):
    # the three grid-wide kernels the d = 2^28 configurations take by themselves, forced at these sizes
    _run_config(lib, wl.configs()["c3_f32"], 2, [9], finish=2)
    _run_config(lib, wl.configs()["c4"], 1, [2], finish=2)


def test_c4_per_tensor_lstm_shapes(lib):
    _run_config(lib, wl.configs()["c4"], 1, [6])


def test_c5_quarter_billion_coordinates(lib):
    cfg = wl.configs()["c5_W4_r100_k10"]
    free = _free_bytes()
    if free < 24e9:
        pytest.skip("not enough free device memory on this (shared) GPU")
    _run_config(lib, cfg, 1, [2])


@pytest.mark.parametrize("name,rows", [("c5_W16_r1000_k4", [0, 5, 10, 15]), ("c5_W32_r100_k10", [1, 12, 23, 31]),
                                       ("c5_W4_r1000_k10", [0, 3]), ("c5_W4_r100_k4", [1])])
def test_c5_sweep_points_many_workers(lib, name, rows):
    # the remaining corners of the d = 2^28 sweep: W in {16, 32}, r / d = 0.1 %, k / r = 1 / 4.  Properties on
    # every row, the oracle on four sampled rows, the update against the oracle's aggregate of all messages.
    cfg = wl.configs()[name]
    free = _free_bytes()
    need = cfg.W * cfg.ld * 4 * 2.3 + 8e9            # g, m, scratch, temporaries of the checks
    if free < need:
        pytest.skip(f"not enough free device memory on this (shared) GPU: {free / 1e9:.0f} GB of {need / 1e9:.0f} GB")
    _run_config(lib, cfg, 1, rows)


def test_slice_longer_than_2_to_28_uses_wider_chunk_groups(lib):
    # above 2^28 coordinates a slice has more than 2048 x 32 chunks and k_finish takes its
    # group-walking layout path; properties only (the oracle's sort of such a row takes minutes)
    free = _free_bytes()
    if free < 16e9:
        pytest.skip("not enough free device memory on this (shared) GPU")
    import dataclasses
    d = (1 << 28) + (1 << 26) + 6
    cfg = dataclasses.replace(wl.configs()["c5_W1_r100_k10"], d=d, r=d // 1000, k=d // 10000, name="long_slice")
    _run_config(lib, cfg, 1, [])


def test_c5_limits_topk_and_randomk(lib):
    free = _free_bytes()
    if free < 16e9:
        pytest.skip("not enough free device memory on this (shared) GPU")
    # k = r (Definition 1): every member of the top-r set is sent -- properties on the device
    _run_config(lib, wl.configs()["c5_W1_topk"], 1, [])
    # r = d (Definition 2): the subset does not depend on the values; positions are indices
    cfg = wl.configs()["c5_W1_randk"]
    ctx = lib.RTopK(d_max=cfg.d, W_max=1, r_max=cfg.r, k_max=cfg.k)
    g = wl.gradient(cfg, 0, "cuda")
    m = wl.zero_residual(cfg, "cuda")
    idx = torch.zeros((1, cfg.k), dtype=torch.int32, device="cuda")
    val = torch.zeros((1, cfg.k), dtype=torch.float32, device="cuda")
    out = torch.empty(cfg.d, dtype=torch.float32, device="cuda")
    ctx.step(g, m, cfg.d, cfg.r, cfg.k, cfg.seed, 0, idx, val, out)
    ctx.poll_status()
    want = oracle.sample_positions(cfg.d, cfg.k, cfg.seed, 0, 0)
    assert np.array_equal(idx.cpu().numpy().view(np.uint32)[0], want)
    i = idx[0].to(torch.int64)
    assert torch.equal(_bits(val[0]), _bits(g[0, : cfg.d][i]))
    back = m[0, : cfg.d].clone()
    back[i] = val[0]
    assert torch.equal(_bits(back), _bits(g[0, : cfg.d]))
    assert torch.equal(_bits(out[i]), _bits(val[0]))                  # W = 1: the update is the message
    assert int((out != 0).sum()) <= cfg.k
    ctx.close()


def test_c3_message_formats_and_master_updates_at_full_size(lib):
    # The messages of one c3_f32 round through everything that follows the sparsifier: the bit-packed and the
    # span-table format (encoder outputs against the oracle's, the aggregation with the decoder fused in against
    # the oracle's average of the decoded messages), the master update and the momentum update of all 25.6 M
    # coordinates, bit for bit.
    cfg = wl.configs()["c3_f32"]
    d, W, k = cfg.d, cfg.W, cfg.k
    ctx = lib.RTopK(d_max=d, W_max=W, r_max=cfg.r, k_max=k)
    g = wl.gradient(cfg, 0, "cuda")
    m = wl.zero_residual(cfg, "cuda")
    idx = torch.zeros((W, k), dtype=torch.int32, device="cuda")
    val = torch.zeros((W, k), dtype=torch.float32, device="cuda")
    out = torch.empty(wl.round_up(d, 4), dtype=torch.float32, device="cuda")
    ctx.step(g, m, d, cfg.r, k, cfg.seed, 0, idx, val, out)
    del g, m
    idx_h, val_h = idx.cpu().numpy().view(np.uint32), val.cpu().numpy()
    # span table
    spans, ll, lh = lib.tiled_layout(d, k)
    tab = torch.zeros((W, spans + 1), dtype=torch.int32, device="cuda")
    low = torch.zeros((W, ll), dtype=torch.int16, device="cuda")
    qv = torch.zeros((W, lh), dtype=torch.int16, device="cuda")
    ctx.encode_tiled(idx, val, d, tab, low, qv)
    o_tab, o_low, o_qv = oracle.encode_tiled(idx_h, val_h, d)
    assert np.array_equal(tab.cpu().numpy().view(np.uint32), o_tab)
    assert np.array_equal(low.cpu().numpy().view(np.uint16)[:, :k], o_low)
    assert np.array_equal(qv.cpu().numpy().view(np.uint16)[:, :k], o_qv)
    d_idx, d_val = oracle.decode_tiled(o_tab, o_low, o_qv, d, k)
    assert np.array_equal(d_idx, idx_h)
    want = oracle.aggregate(d_idx, d_val, d)[1]
    ctx.aggregate_tiled(tab, low, qv, d, k, out)
    assert np.array_equal(out.cpu().numpy()[:d].view(np.uint32), want.view(np.uint32))
    # bit-packed
    bits, lw, lh = lib.packed_layout(d, k)
    pi = torch.zeros((W, lw), dtype=torch.int32, device="cuda")
    pv = torch.zeros((W, lh), dtype=torch.int16, device="cuda")
    ctx.encode(idx, val, d, pi, pv)
    o_pi, o_pv = oracle.encode(idx_h, val_h, d)
    assert np.array_equal(pi.cpu().numpy().view(np.uint32)[:, :o_pi.shape[1]], o_pi)
    ctx.aggregate_packed(pi, pv, d, k, out)
    assert np.array_equal(out.cpu().numpy()[:d].view(np.uint32), want.view(np.uint32))
    # master updates
    rng = np.random.default_rng(3)
    w0 = rng.standard_normal(d).astype(np.float32)
    v0 = (rng.standard_normal(d) * 0.1).astype(np.float32)
    w, v = torch.zeros_like(out), torch.zeros_like(out)
    w[:d] = torch.from_numpy(w0).cuda()
    v[:d] = torch.from_numpy(v0).cuda()
    ctx.apply_momentum(idx, val, d, 0.05, 0.9, v, w)
    o_v, o_w = oracle.apply_momentum(idx_h, val_h, d, 0.05, 0.9, v0, w0)
    assert np.array_equal(v.cpu().numpy()[:d].view(np.uint32), o_v.view(np.uint32))
    assert np.array_equal(w.cpu().numpy()[:d].view(np.uint32), o_w.view(np.uint32))
    w[:d] = torch.from_numpy(w0).cuda()
    ctx.apply_update(idx, val, d, 0.05, w)
    assert np.array_equal(w.cpu().numpy()[:d].view(np.uint32), oracle.apply_update(idx_h, val_h, d, 0.05, w0).view(np.uint32))
    ctx.poll_status()
    ctx.close()


def test_eight_rank_job_of_c3_run_rank_by_rank_on_one_gpu(lib):
    # The sharded job bench.py runs with --gpus 8 (16 rows of c3_f32 per GPU, 128 workers), as one process
    # over all ranks' data: every rank's rows are sparsified in turn with that rank's worker_base into its
    # block of the gathered pair buffer (what the all-gather leaves on every GPU), then the buffer is
    # aggregated in place.  Two sampled workers per rank position against the oracle with their global
    # worker ids, the average of all 128 messages against the oracle's, bit for bit.
    import dataclasses
    from paper_2005_10761_b200 import sharded
    base = wl.configs()["c3_f32"]
    world, c = 8, base.W
    W_total = world * c
    if _free_bytes() < 12e9:
        pytest.skip("not enough free device memory")
    cfg = dataclasses.replace(base, W=W_total)
    d, r, k = cfg.d, cfg.r, cfg.k
    ctx = lib.RTopK(d_max=d, W_max=W_total, r_max=r, k_max=k)
    pairs_all = torch.zeros((W_total, k), dtype=torch.int64, device="cuda")
    sampled = {0: [3], 3: [0, 15], 7: [9]}             # rank -> local rows followed by the oracle
    for p in range(world):
        begin, rows = sharded.shard_rows(W_total, world, p)
        assert (begin, rows) == (p * c, c)
        g = wl.gradient(cfg, 0, "cuda", workers=range(begin, begin + rows))
        m = wl.zero_residual(base, "cuda")
        ctx.sparsify_pairs(g, m, d, r, k, cfg.seed, 0, pairs_all[begin:begin + rows], worker_base=begin)
        ctx.poll_status()
        idx_p, val_p = sharded.unpack_pairs(pairs_all[begin:begin + rows])
        for w in sampled.get(p, []):
            m_or = np.zeros((1, cfg.ld), dtype=np.float32)
            o_idx, o_val = oracle.sparsify(_host_grad(cfg, g[w:w + 1]), m_or, d, r, k, cfg.seed, 0, worker_base=begin + w)
            assert np.array_equal(idx_p[w].cpu().numpy().view(np.uint32), o_idx[0]), f"rank {p} row {w}: indices"
            assert np.array_equal(val_p[w].cpu().numpy().view(np.uint32), o_val[0].view(np.uint32)), f"rank {p} row {w}: values"
            assert np.array_equal(m[w].cpu().numpy().view(np.uint32), m_or[0].view(np.uint32)), f"rank {p} row {w}: residual"
        del g, m
    out = torch.empty(wl.round_up(d, 4), dtype=torch.float32, device="cuda")
    ctx.aggregate_pairs(pairs_all, d, out)
    ctx.poll_status()
    idx_all, val_all = sharded.unpack_pairs(pairs_all)
    idx_h, val_h = idx_all.cpu().numpy().view(np.uint32), val_all.cpu().numpy()
    assert bool((idx_h[:, 1:] > idx_h[:, :-1]).all()) and int(idx_h.max()) < d
    o64, o32 = oracle.aggregate(idx_h, val_h, d)
    assert np.array_equal(out.cpu().numpy()[:d].view(np.uint32), o32.view(np.uint32))
    ctx.close()
