"""Parity of the CUDA library (through its C ABI) with the CPU oracle, element by element.

Bar: message indices, message values and the residual are bit-exact; the aggregated update is
within 1e-6 * max|g| of the oracle's double-precision result (and, because the library sums in a
fixed order in double precision, in fact equal to its binary32 rounding).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2005_10761_b200 import workloads as wl

pytestmark = pytest.mark.gpu

# how a context selects: the sampled bracket finished by the cluster kernel (what AUTO takes at these
# sizes), the full-vector radix select, or the sampled bracket finished from the runs by the three
# grid-wide kernels (what AUTO takes for slices of 2^26 coordinates or more)
AUTO, EXACT, RUNS = 0, 1, 2


@pytest.fixture(scope="module")
def lib():
    import paper_2005_10761_b200 as pkg
    from paper_2005_10761_b200 import build
    build.build()
    return pkg


def _ctx(lib, d, W, r, k, S=1, path=AUTO):
    ctx = lib.RTopK(d_max=d, W_max=W, r_max=r, k_max=k, segments_max=S)
    ctx.set_option(0, EXACT if path == EXACT else AUTO)          # RTOPK_OPT_SELECT_PATH
    ctx.set_option(5, 2 if path == RUNS else 0)                  # RTOPK_OPT_FINISH_PATH
    return ctx


def _bits(x):
    return np.ascontiguousarray(x).view(np.uint32)


def _pad(a: np.ndarray, mult=8, fill=0.0):
    W, d = a.shape
    ld = wl.round_up(d, mult)
    out = np.full((W, ld), fill, dtype=a.dtype)
    out[:, :d] = a
    return out


def run_gpu(lib, g, m0, d, r, k, seed, step, worker_base=0, path=AUTO, ctx=None, bf16=False):
    """g, m0: float32 numpy [W, ld] (g is converted to bfloat16 on request).  Returns numpy
    (idx, val, m') from rtopk_sparsify."""
    W = g.shape[0]
    own = ctx is None
    if own:
        ctx = _ctx(lib, d, W, r, k, path=path)
    tg = torch.from_numpy(g).cuda()
    if bf16:
        tg = tg.to(torch.bfloat16)
    tm = torch.from_numpy(m0.copy()).cuda()
    idx = torch.full((W, k), -1, dtype=torch.int32, device="cuda")
    val = torch.full((W, k), float("nan"), dtype=torch.float32, device="cuda")
    ctx.sparsify(tg, tm, d, r, k, seed, step, idx, val, worker_base=worker_base)
    ctx.poll_status()
    stats = [ctx.stats(w) for w in range(W)]
    # the same round as one fused call (its aggregation works from the run table the sparsifier keeps): the
    # messages must come out the same, and the update is returned for the comparison with the oracle's average
    tm2 = torch.from_numpy(m0.copy()).cuda()
    idx2, val2 = torch.full_like(idx, -1), torch.full_like(val, float("nan"))
    out = torch.full((g.shape[1],), float("nan"), dtype=torch.float32, device="cuda")
    ctx.step(tg, tm2, d, r, k, seed, step, idx2, val2, out, worker_base=worker_base)
    ctx.poll_status()
    assert torch.equal(idx2, idx) and torch.equal(val2.view(torch.int32), val.view(torch.int32))
    assert torch.equal(tm2.view(torch.int32), tm.view(torch.int32))
    run_gpu.last_update = out.cpu().numpy()[:d]
    if own:
        ctx.close()
    return idx.cpu().numpy().view(np.uint32), val.cpu().numpy(), tm.cpu().numpy(), stats


def check_against_oracle(lib, g, m0, d, r, k, seed=1, step=0, worker_base=0, path=AUTO, bf16=False):
    if bf16:
        gb = torch.from_numpy(g).to(torch.bfloat16)
        g_or = gb.view(torch.int16).numpy().view(np.uint16).copy()
    else:
        g_or = g
    m_or = m0.copy()
    o_idx, o_val = oracle.sparsify(g_or, m_or, d, r, k, seed, step, worker_base)
    g_idx, g_val, g_m, stats = run_gpu(lib, g, m0, d, r, k, seed, step, worker_base, path, bf16=bf16)
    for w in range(g.shape[0]):
        assert np.array_equal(g_idx[w], o_idx[w]), (
            f"indices differ: worker {w} d={d} r={r} k={k} path={path} stats={stats[w]} "
            f"first mismatch at {np.flatnonzero(g_idx[w] != o_idx[w])[:5]} gpu={g_idx[w][:8]} oracle={o_idx[w][:8]}")
        assert np.array_equal(_bits(g_val[w]), _bits(o_val[w])), f"values differ: worker {w}"
        assert np.array_equal(_bits(g_m[w, :d]), _bits(m_or[w, :d])), (
            f"residual differs: worker {w}, at {np.flatnonzero(_bits(g_m[w, :d]) != _bits(m_or[w, :d]))[:5]}")
        # padding columns are neither read nor written
        assert np.array_equal(_bits(g_m[w, d:]), _bits(m0[w, d:]))
    _, want = oracle.aggregate(o_idx, o_val, d)
    got = run_gpu.last_update
    both_nan = np.isnan(got) & np.isnan(want)          # (IEEE 754 leaves the payload of a NaN sum open)
    assert np.array_equal(_bits(got)[~both_nan], _bits(want)[~both_nan]), "update of the fused call differs"
    return stats


def _spiky(rng, W, d, p=0.02):
    x = rng.standard_normal((W, d)) * 1e-3
    m = rng.random((W, d)) < p
    return np.where(m, rng.standard_normal((W, d)), x).astype(np.float32)


SMALL = [(1, 1, 1), (2, 2, 1), (3, 2, 2), (5, 3, 2), (31, 7, 3), (33, 33, 4), (1023, 100, 10), (4097, 41, 41),
         (4098, 4098, 17), (5003, 1, 1), (12289, 900, 90), (40001, 400, 40)]


@pytest.mark.parametrize("path", [AUTO, EXACT, RUNS])
@pytest.mark.parametrize("d,r,k", SMALL)
def test_small_and_ragged_sizes(lib, d, r, k, path):
    rng = np.random.default_rng(d * 7 + r)
    W = 3
    g = _pad(_spiky(rng, W, d), fill=7.0)          # poisoned padding: must never be selected
    m0 = _pad(_spiky(rng, W, d) * 0.5, fill=-9.0)
    check_against_oracle(lib, g, m0, d, r, k, seed=d, step=3, worker_base=5, path=path)


@pytest.mark.parametrize("path", [AUTO, EXACT, RUNS])
def test_heavy_ties(lib, path):
    rng = np.random.default_rng(2)
    W, d = 2, 70001
    cases = {
        "all_equal": np.full((W, d), -3.25, dtype=np.float32),
        "mostly_zero": np.where(rng.random((W, d)) < 0.01, rng.standard_normal((W, d)), 0.0).astype(np.float32),
        "signed_zero": np.where(rng.random((W, d)) < 0.5, 0.0, -0.0).astype(np.float32),
        "three_levels": rng.choice(np.array([0.5, -0.5, 1.0, -2.0, 0.0], dtype=np.float32), (W, d)),
        "quantised": (np.round(rng.standard_normal((W, d)) * 4) / 4).astype(np.float32),
    }
    for name, g in cases.items():
        g = _pad(g)
        m0 = np.zeros_like(g)
        for r, k in [(700, 70), (35000, 35), (1, 1), (d, 700), (d - 1, d - 1)]:
            stats = check_against_oracle(lib, g, m0, d, r, k, seed=9, step=1, path=path)
            assert stats is not None, name


@pytest.mark.parametrize("path", [AUTO, EXACT, RUNS])
def test_non_finite_and_denormal_values(lib, path):
    rng = np.random.default_rng(3)
    W, d = 2, 9001
    g = _spiky(rng, W, d)
    g[:, 5] = np.nan; g[:, 77] = np.inf; g[:, 4000] = -np.inf; g[:, 8999] = 1e-45; g[:, 100] = -1e-42
    g = _pad(g)
    m0 = np.zeros_like(g)
    for r, k in [(3, 3), (90, 9), (9001, 90)]:
        check_against_oracle(lib, g, m0, d, r, k, seed=4, step=0, path=path)


def test_multi_tile_many_workers_and_worker_base(lib):
    rng = np.random.default_rng(4)
    W, d, r, k = 7, 300007, 3000, 300
    g = _pad(_spiky(rng, W, d, p=0.01))
    m0 = _pad(_spiky(rng, W, d, p=0.01) * 0.3)
    for path in (AUTO, EXACT, RUNS):
        check_against_oracle(lib, g, m0, d, r, k, seed=0xDEADBEEF12345, step=77, worker_base=1000, path=path)


def test_limits_topk_and_randomk(lib):
    rng = np.random.default_rng(5)
    W, d = 2, 50000
    g = _pad(_spiky(rng, W, d))
    m0 = np.zeros_like(g)
    for path in (AUTO, EXACT, RUNS):
        check_against_oracle(lib, g, m0, d, 500, 500, seed=1, step=2, path=path)      # k = r: Definition 1
        check_against_oracle(lib, g, m0, d, d, 50, seed=1, step=2, path=path)         # r = d: Definition 2
        check_against_oracle(lib, g, m0, d, d, d, seed=1, step=2, path=path)          # everything is sent


def test_bf16_gradient(lib):
    rng = np.random.default_rng(6)
    W, d, r, k = 3, 100003, 1000, 100
    g = _pad(_spiky(rng, W, d))
    m0 = _pad(_spiky(rng, W, d) * 0.25)
    for path in (AUTO, EXACT, RUNS):
        check_against_oracle(lib, g, m0, d, r, k, seed=6, step=6, path=path, bf16=True)


@pytest.mark.parametrize("name", ["c2", "c3_f32"])
def test_ten_steps_with_carried_residual(lib, name):
    cfg = wl.scaled(wl.configs()[name], d=250007, W=3)
    ctx = _ctx(lib, cfg.d, cfg.W, cfg.r, cfg.k)
    m_gpu = wl.zero_residual(cfg, "cuda")
    m_or = np.zeros((cfg.W, cfg.ld), dtype=np.float32)
    idx = torch.zeros((cfg.W, cfg.k), dtype=torch.int32, device="cuda")
    val = torch.zeros((cfg.W, cfg.k), dtype=torch.float32, device="cuda")
    for t in range(cfg.steps):
        g = wl.gradient(cfg, t, "cuda")
        ctx.sparsify(g, m_gpu, cfg.d, cfg.r, cfg.k, cfg.seed, t, idx, val)
        o_idx, o_val = oracle.sparsify(g.cpu().numpy(), m_or, cfg.d, cfg.r, cfg.k, cfg.seed, t)
        assert np.array_equal(idx.cpu().numpy().view(np.uint32), o_idx), f"step {t}"
        assert np.array_equal(_bits(val.cpu().numpy()), _bits(o_val)), f"step {t}"
        assert np.array_equal(_bits(m_gpu.cpu().numpy()), _bits(m_or)), f"step {t}"
    ctx.poll_status()
    ctx.close()


def test_segmented_per_tensor_selection(lib):
    rng = np.random.default_rng(7)
    W = 3
    sizes = [70001, 3, 4099, 12288, 50001, 1]       # unaligned cuts, tiny tensors, multi-tile tensors
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    d = int(off[-1])
    seg_r = [700, 3, 4099, 100, 5000, 1]
    seg_k = [70, 1, 40, 100, 50, 1]
    K = sum(seg_k)
    g = _pad(_spiky(rng, W, d))
    m0 = _pad(_spiky(rng, W, d) * 0.5)
    m_or = m0.copy()
    o_idx, o_val = oracle.sparsify_segmented(g, m_or, d, off, seg_r, seg_k, seed=8, step=5, worker_base=2)
    for path in (AUTO, EXACT, RUNS):
        ctx = _ctx(lib, d, W, sum(seg_r), K, S=len(sizes), path=path)
        tg, tm = torch.from_numpy(g).cuda(), torch.from_numpy(m0.copy()).cuda()
        idx = torch.zeros((W, K), dtype=torch.int32, device="cuda")
        val = torch.zeros((W, K), dtype=torch.float32, device="cuda")
        out = torch.empty(wl.round_up(d, 4), dtype=torch.float32, device="cuda")
        ctx.step_segmented(tg, tm, d, off, seg_r, seg_k, 8, 5, idx, val, out, worker_base=2)
        ctx.poll_status()
        assert np.array_equal(idx.cpu().numpy().view(np.uint32), o_idx)
        assert np.array_equal(_bits(val.cpu().numpy()), _bits(o_val))
        assert np.array_equal(_bits(tm.cpu().numpy()[:, :d]), _bits(m_or[:, :d]))
        o64, o32 = oracle.aggregate(o_idx, o_val, d)
        assert np.array_equal(_bits(out.cpu().numpy()[:d]), _bits(o32))
        ctx.close()


@pytest.mark.parametrize("case", range(16))
def test_random_segmented_steps(lib, case):
    # Seeded random tensor layouts (1 to 8 tensors of 1 to 60,000 coordinates, unaligned cuts), per-tensor r and
    # k, every finishing path: messages, residual and the update of the fused call against the oracle.
    rng = np.random.default_rng(50000 + case)
    S, W = int(rng.integers(1, 9)), int(rng.integers(1, 5))
    sizes = [int(rng.choice([rng.integers(1, 40), rng.integers(40, 9000), rng.integers(9000, 60000)])) for _ in range(S)]
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    d = int(off[-1])
    seg_r = [int(rng.integers(1, n + 1)) if rng.random() < 0.3 else max(1, n // int(rng.choice([3, 20, 100]))) for n in sizes]
    seg_k = [int(rng.integers(1, r + 1)) if rng.random() < 0.4 else max(1, r // int(rng.choice([2, 4, 10]))) for r in seg_r]
    K = sum(seg_k)
    g = _pad(_spiky(rng, W, d, p=float(rng.choice([0.0, 0.02, 0.2]))))
    m0 = _pad(_spiky(rng, W, d) * 0.5)
    if rng.random() < 0.3:                             # many equal magnitudes, signed zeros
        g = (np.round(g * 5) / 5).astype(np.float32)
    m_or = m0.copy()
    seed, step, wb = int(rng.integers(0, 2**40)), int(rng.integers(0, 99)), int(rng.integers(0, 9))
    o_idx, o_val = oracle.sparsify_segmented(g, m_or, d, off, seg_r, seg_k, seed=seed, step=step, worker_base=wb)
    ctx = _ctx(lib, d, W, sum(seg_r), K, S=S, path=int(rng.choice([AUTO, EXACT, RUNS])))
    tg, tm = torch.from_numpy(g).cuda(), torch.from_numpy(m0.copy()).cuda()
    idx = torch.zeros((W, K), dtype=torch.int32, device="cuda")
    val = torch.zeros((W, K), dtype=torch.float32, device="cuda")
    out = torch.full((wl.round_up(d, 4),), float("nan"), dtype=torch.float32, device="cuda")
    ctx.step_segmented(tg, tm, d, off, seg_r, seg_k, seed, step, idx, val, out, worker_base=wb)
    ctx.poll_status()
    assert np.array_equal(idx.cpu().numpy().view(np.uint32), o_idx)
    assert np.array_equal(_bits(val.cpu().numpy()), _bits(o_val))
    assert np.array_equal(_bits(tm.cpu().numpy()[:, :d]), _bits(m_or[:, :d]))
    assert np.array_equal(_bits(out.cpu().numpy()[:d]), _bits(oracle.aggregate(o_idx, o_val, d)[1]))
    ctx.close()


@pytest.mark.parametrize("W,d,k", [(1, 1000, 10), (4, 4096, 400), (5, 100001, 2000), (16, 300000, 3000),
                                   (32, 50000, 50000 // 3), (300, 20000, 50)])
def test_aggregate_against_oracle(lib, W, d, k):
    rng = np.random.default_rng(W * 31 + k)
    idx = np.stack([np.sort(rng.choice(d, k, replace=False)) for _ in range(W)]).astype(np.uint32)
    val = (rng.standard_normal((W, k)) * np.exp(2 * rng.standard_normal((W, k)))).astype(np.float32)
    ctx = _ctx(lib, d, W, k, k)
    t_idx = torch.from_numpy(idx.view(np.int32)).cuda()
    t_val = torch.from_numpy(val).cuda()
    out = torch.full((wl.round_up(d, 4),), float("nan"), dtype=torch.float32, device="cuda")
    for mode in (lib.SCALE_MEAN, lib.SCALE_SUM):
        ctx.aggregate(t_idx, t_val, d, out, scale_mode=mode)
        o64, o32 = oracle.aggregate(idx, val, d, mode)
        got = out.cpu().numpy()[:d]
        tol = 1e-6 * float(np.abs(val).max())
        assert np.abs(got.astype(np.float64) - o64).max() <= tol      # the stated bar
        assert np.array_equal(_bits(got), _bits(o32))                  # and the stronger fact
    ctx.close()


def test_aggregate_sparse_path_many_workers_and_crowded_tiles(lib):
    rng = np.random.default_rng(99)
    cases = []
    d, W, k = 3_000_017, 300, 500                      # more workers than one block batch
    cases.append((d, np.stack([np.sort(rng.choice(d, k, replace=False)) for _ in range(W)])))
    d, W, k = 1_000_000, 8, 2000                       # every entry inside the first output tiles
    cases.append((d, np.stack([np.sort(rng.choice(6000, k, replace=False)) for _ in range(W)])))
    d, W, k = 3_000_000, 16, 3000                      # identical supports: every coordinate shared by all
    same = np.sort(rng.choice(d, k, replace=False))
    cases.append((d, np.stack([same] * W)))
    d, W, k = 2_000_003, 13, 777                       # a worker count that is no multiple of the warps per block
    cases.append((d, np.stack([np.sort(rng.choice(d, k, replace=False)) for _ in range(W)])))
    d, W, k = 70_001, 3, 1                             # one entry per worker: the shortest sorted rows
    cases.append((d, np.array([[70_000], [0], [16_384]])))
    d, W, k = 1_000_000, 5, 40                         # runs that end exactly at tile borders
    edge = np.sort(np.concatenate([np.arange(16_380, 16_400), np.arange(32_758, 32_778)]))
    cases.append((d, np.stack([edge] * W)))
    # Messages that concentrate on a part of the vector: tiles with several times the entries the stage holds,
    # taken in parts.  (a) 80 % of every row inside 20000 coordinates, the rest anywhere; (b) a tile border in the
    # middle of the hot range, and rows that differ in how much they send there; (c) 200 workers that all send
    # the same 96 neighbouring coordinates: no part of 32 coordinates fits the stage, the searched path runs.
    d, W, k = 2_000_000, 12, 6000
    hot = [np.sort(np.concatenate([rng.choice(20_000, 4800, replace=False),
                                   20_000 + rng.choice(d - 20_000, 1200, replace=False)])) for _ in range(W)]
    cases.append((d, np.stack(hot)))
    d, W, k = 1_500_000, 9, 5000
    rows = []
    for w in range(W):
        n_hot = 500 * w + 500
        rows.append(np.sort(np.concatenate([10_000 + rng.choice(12_000, n_hot, replace=False),
                                            30_000 + rng.choice(d - 30_000, k - n_hot, replace=False)])))
    cases.append((d, np.stack(rows)))
    d, W, k = 400_000, 200, 100
    same = np.concatenate([np.arange(50_000, 50_096), np.array([123_456, 200_000, 300_001, 399_999])])
    cases.append((d, np.stack([same] * W)))
    for d, idx in cases:
        idx = idx.astype(np.uint32)
        W, k = idx.shape
        val = (rng.standard_normal((W, k)) * np.exp(2 * rng.standard_normal((W, k)))).astype(np.float32)
        ctx = _ctx(lib, d, W, k, k)
        out = torch.full((wl.round_up(d, 4),), float("nan"), dtype=torch.float32, device="cuda")
        ctx.aggregate(torch.from_numpy(idx.view(np.int32)).cuda(), torch.from_numpy(val).cuda(), d, out)
        o64, o32 = oracle.aggregate(idx, val, d)
        got = out.cpu().numpy()[:d]
        assert np.abs(got.astype(np.float64) - o64).max() <= 1e-6 * float(np.abs(val).max())
        assert np.array_equal(_bits(got), _bits(o32))
        ctx.close()


def test_packed_messages_against_oracle(lib):
    """Encoder (bit-packed indices, bfloat16 values, rounding error into the residual) and the
    aggregation that decodes on the fly: bit-equal to the oracle's encoder and to the oracle's
    aggregate of the decoded messages."""
    rng = np.random.default_rng(2024)
    cases = [(2_000_003, 8, 900), (100_003, 6, 20_000), (1 << 20, 3, 4097), (37, 2, 37), (5, 70, 3)]
    for d, W, k in cases:
        idx = np.stack([np.sort(rng.choice(d, k, replace=False)) for _ in range(W)]).astype(np.uint32)
        val = (rng.standard_normal((W, k)) * np.exp(3 * rng.standard_normal((W, k)))).astype(np.float32)
        val[0, 0] = 3.4e38                      # rounds to +inf in bfloat16
        val[W - 1, k - 1] = np.float32(np.nan)
        bits, lw, lh = lib.packed_layout(d, k)
        assert bits == oracle.index_bits(d) and lw >= oracle.packed_words(d, k) and lw % 4 == 0 and lh >= k and lh % 8 == 0
        ld = wl.round_up(d, 4)
        m0 = rng.standard_normal((W, ld)).astype(np.float32)
        for w in range(W):
            m0[w, idx[w].astype(np.int64)] = 0.0
        m_ref = m0.copy()
        o_pi, o_pv = oracle.encode(idx, val, d, residual=m_ref)
        ctx = _ctx(lib, d, W, k, k)
        t_idx, t_val = torch.from_numpy(idx.view(np.int32)).cuda(), torch.from_numpy(val).cuda()
        m = torch.from_numpy(m0.copy()).cuda()
        pi = torch.full((W, lw), -1, dtype=torch.int32, device="cuda")
        pv = torch.full((W, lh), -1, dtype=torch.int16, device="cuda")
        ctx.encode(t_idx, t_val, d, pi, pv, residual=m)
        got_pi = pi.cpu().numpy().view(np.uint32)
        got_pv = pv.cpu().numpy().view(np.uint16)
        nw = o_pi.shape[1]
        assert np.array_equal(got_pi[:, :nw], o_pi) and not got_pi[:, nw:].any()
        assert np.array_equal(got_pv[:, :k], o_pv) and not got_pv[:, k:].any()
        assert np.array_equal(_bits(m.cpu().numpy()), _bits(m_ref))
        d_idx, d_val = oracle.decode(o_pi, o_pv, d, k)
        assert np.array_equal(d_idx, idx)
        out = torch.full((ld,), float("nan"), dtype=torch.float32, device="cuda")
        for mode, omode in ((lib.SCALE_MEAN, oracle.SCALE_MEAN), (lib.SCALE_COUNT, oracle.SCALE_COUNT)):
            ctx.aggregate_packed(pi, pv, d, k, out, scale_mode=mode)
            _, want = oracle.aggregate(d_idx, d_val, d, omode)
            assert np.array_equal(_bits(out.cpu().numpy()[:d]), _bits(want))
        ctx.close()


def test_aggregate_scalings_against_oracle(lib):
    """UNBIASED (r / (W k), the estimator in the proof of Theorem 1) and COUNT (sum over senders /
    number of senders) on the sparse path, the dense path and with shared coordinates."""
    rng = np.random.default_rng(77)
    cases = []
    d, W, k = 2_000_003, 8, 900
    cases.append((d, np.stack([np.sort(rng.choice(d, k, replace=False)) for _ in range(W)])))
    d, W, k = 100_003, 6, 20_000
    cases.append((d, np.stack([np.sort(rng.choice(d, k, replace=False)) for _ in range(W)])))
    d, W, k = 50_000, 300, 2_000                       # dense path, more workers than one block batch
    cases.append((d, np.stack([np.sort(rng.choice(d, k, replace=False)) for _ in range(W)])))
    d, W, k = 1_000_000, 5, 3000
    same = np.sort(rng.choice(d, k, replace=False))
    cases.append((d, np.stack([same] * W)))
    for d, idx in cases:
        idx = idx.astype(np.uint32)
        W, k = idx.shape
        val = (rng.standard_normal((W, k)) * np.exp(2 * rng.standard_normal((W, k)))).astype(np.float32)
        ctx = _ctx(lib, d, W, k, k)
        t_idx, t_val = torch.from_numpy(idx.view(np.int32)).cuda(), torch.from_numpy(val).cuda()
        out = torch.full((wl.round_up(d, 4),), float("nan"), dtype=torch.float32, device="cuda")
        r = min(d, 7 * k + 3)
        ctx.aggregate_unbiased(t_idx, t_val, d, r, out)
        _, want = oracle.aggregate(idx, val, d, oracle.SCALE_UNBIASED, r=r)
        assert np.array_equal(_bits(out.cpu().numpy()[:d]), _bits(want))
        out.fill_(float("nan"))
        ctx.aggregate(t_idx, t_val, d, out, scale_mode=lib.SCALE_COUNT)
        _, want = oracle.aggregate(idx, val, d, oracle.SCALE_COUNT)
        assert np.array_equal(_bits(out.cpu().numpy()[:d]), _bits(want))
        # the update with by-count scaling
        w0 = rng.standard_normal(wl.round_up(d, 4)).astype(np.float32)
        w = torch.from_numpy(w0.copy()).cuda()
        ctx.apply_update(t_idx, t_val, d, 0.25, w, scale_mode=lib.SCALE_COUNT)
        want = oracle.apply_update(idx, val, d, 0.25, w0[:d], oracle.SCALE_COUNT)
        assert np.array_equal(_bits(w.cpu().numpy()[:d]), _bits(want))
        with pytest.raises(RuntimeError):                # UNBIASED needs r
            ctx.aggregate(t_idx, t_val, d, out, scale_mode=lib.SCALE_UNBIASED)
        ctx.close()


def test_step_with_unbiased_scaling(lib):
    cfg = wl.scaled(wl.configs()["c1"], d=300_007, W=4)
    ctx = _ctx(lib, cfg.d, cfg.W, cfg.r, cfg.k)
    g = wl.gradient(cfg, 0, "cuda")
    m = wl.zero_residual(cfg, "cuda")
    m_ref = np.zeros((cfg.W, cfg.ld), dtype=np.float32)
    idx = torch.zeros((cfg.W, cfg.k), dtype=torch.int32, device="cuda")
    val = torch.zeros((cfg.W, cfg.k), dtype=torch.float32, device="cuda")
    out = torch.full((cfg.ld,), float("nan"), dtype=torch.float32, device="cuda")
    ctx.step(g, m, cfg.d, cfg.r, cfg.k, cfg.seed, 0, idx, val, out, scale_mode=lib.SCALE_UNBIASED)
    o_idx, o_val = oracle.sparsify(g.cpu().numpy(), m_ref, cfg.d, cfg.r, cfg.k, cfg.seed, 0)
    _, want = oracle.aggregate(o_idx, o_val, cfg.d, oracle.SCALE_UNBIASED, r=cfg.r)
    assert np.array_equal(idx.cpu().numpy().view(np.uint32), o_idx)
    assert np.array_equal(_bits(out.cpu().numpy()[:cfg.d]), _bits(want))
    w0 = np.linspace(-1, 1, cfg.ld).astype(np.float32)
    w = torch.from_numpy(w0.copy()).cuda()
    ctx.step_apply(g, m, cfg.d, cfg.r, cfg.k, cfg.seed, 1, 0.5, idx, val, w, scale_mode=lib.SCALE_UNBIASED)
    o_idx, o_val = oracle.sparsify(g.cpu().numpy(), m_ref, cfg.d, cfg.r, cfg.k, cfg.seed, 1)
    want = oracle.apply_update(o_idx, o_val, cfg.d, 0.5, w0[:cfg.d], oracle.SCALE_UNBIASED, r=cfg.r)
    assert np.array_equal(_bits(w.cpu().numpy()[:cfg.d]), _bits(want))
    ctx.poll_status()
    ctx.close()


def test_master_update_against_oracle(lib):
    """Algorithm 1's w <- w - eta * ghat straight from the messages: bit-equal to the oracle on the
    sparse path (few entries per tile), the dense path, shared coordinates and -0.0 weights."""
    rng = np.random.default_rng(123)
    cases = []
    d, W, k = 2_000_003, 8, 900                        # sparse path, own run search
    cases.append((d, np.stack([np.sort(rng.choice(d, k, replace=False)) for _ in range(W)])))
    d, W, k = 3_000_017, 70, 400                       # sparse path behind the table of run starts
    cases.append((d, np.stack([np.sort(rng.choice(d, k, replace=False)) for _ in range(W)])))
    d, W, k = 100_003, 6, 20_000                       # dense path, ragged last tile
    cases.append((d, np.stack([np.sort(rng.choice(d, k, replace=False)) for _ in range(W)])))
    d, W, k = 1_000_000, 5, 3000                       # identical supports: every coordinate shared by all
    same = np.sort(rng.choice(d, k, replace=False))
    cases.append((d, np.stack([same] * W)))
    for d, idx in cases:
        idx = idx.astype(np.uint32)
        W, k = idx.shape
        val = (rng.standard_normal((W, k)) * np.exp(2 * rng.standard_normal((W, k)))).astype(np.float32)
        w0 = rng.standard_normal(wl.round_up(d, 4)).astype(np.float32)
        w0[idx[0, :5].astype(np.int64)] = -0.0
        w0[::1001] = -0.0
        ctx = _ctx(lib, d, W, k, k)
        for mode, eta in ((lib.SCALE_MEAN, 0.05), (lib.SCALE_SUM, 1.0), (lib.SCALE_MEAN, 0.0)):
            w = torch.from_numpy(w0.copy()).cuda()
            ctx.apply_update(torch.from_numpy(idx.view(np.int32)).cuda(), torch.from_numpy(val).cuda(), d, eta, w,
                             scale_mode=mode)
            want = oracle.apply_update(idx, val, d, eta, w0[:d], mode)
            got = w.cpu().numpy()
            assert np.array_equal(_bits(got[:d]), _bits(want))
            assert np.array_equal(_bits(got[d:]), _bits(w0[d:]))          # padding is never touched
        with pytest.raises(RuntimeError):
            ctx.apply_update(torch.from_numpy(idx.view(np.int32)).cuda(), torch.from_numpy(val).cuda(), d, -0.1,
                             torch.from_numpy(w0.copy()).cuda())
        ctx.close()


def test_step_apply_is_sparsify_then_update(lib):
    cfg = wl.scaled(wl.configs()["c1"], d=300_007, W=4)
    ctx = _ctx(lib, cfg.d, cfg.W, cfg.r, cfg.k)
    rng = np.random.default_rng(5)
    w0 = rng.standard_normal(cfg.ld).astype(np.float32)
    w = torch.from_numpy(w0.copy()).cuda()
    m = wl.zero_residual(cfg, "cuda")
    m_ref = np.zeros((cfg.W, cfg.ld), dtype=np.float32)
    idx = torch.zeros((cfg.W, cfg.k), dtype=torch.int32, device="cuda")
    val = torch.zeros((cfg.W, cfg.k), dtype=torch.float32, device="cuda")
    want = w0[:cfg.d].copy()
    for t in range(3):
        g = wl.gradient(cfg, t, "cuda")
        ctx.step_apply(g, m, cfg.d, cfg.r, cfg.k, cfg.seed, t, 0.1, idx, val, w)
        o_idx, o_val = oracle.sparsify(g.cpu().numpy(), m_ref, cfg.d, cfg.r, cfg.k, cfg.seed, t)
        want = oracle.apply_update(o_idx, o_val, cfg.d, 0.1, want)
        assert np.array_equal(idx.cpu().numpy().view(np.uint32), o_idx)
        assert np.array_equal(_bits(val.cpu().numpy()), _bits(o_val))
        assert np.array_equal(_bits(m.cpu().numpy()), _bits(m_ref))
        assert np.array_equal(_bits(w.cpu().numpy()[:cfg.d]), _bits(want))
    ctx.poll_status()
    ctx.close()


def test_span_table_messages_against_oracle(lib):
    """Encoder of the span-table format (entry counts per span of 16384 coordinates, 14 low index bits,
    bfloat16 values, rounding error into the residual) and the aggregation that decodes on the fly:
    bit-equal to the oracle's encoder and to the oracle's aggregate of the decoded messages.  Cases: few
    entries per tile (sparse kernel, the table serves as its run starts), many (dense kernel), one span,
    a ragged last span, rows that leave spans empty, more workers than one block's pass."""
    rng = np.random.default_rng(2025)
    cases = [(2_000_003, 8, 900), (100_003, 6, 20_000), (1 << 20, 3, 4097), (37, 2, 37), (16384, 5, 16384),
             (16385, 4, 3), (5_000_000, 2, 40), (300_000, 300, 50)]
    for d, W, k in cases:
        idx = np.stack([np.sort(rng.choice(d, k, replace=False)) for _ in range(W)]).astype(np.uint32)
        val = (rng.standard_normal((W, k)) * np.exp(3 * rng.standard_normal((W, k)))).astype(np.float32)
        val[0, 0] = 3.4e38                      # rounds to +inf in bfloat16
        val[W - 1, k - 1] = np.float32(np.nan)
        spans, ll, lh = lib.tiled_layout(d, k)
        assert spans == oracle.tiled_spans(d) and ll >= k and ll % 8 == 0 and lh >= k and lh % 8 == 0
        ld = wl.round_up(d, 4)
        m0 = rng.standard_normal((W, ld)).astype(np.float32)
        for w in range(W):
            m0[w, idx[w].astype(np.int64)] = 0.0
        m_ref = m0.copy()
        o_tab, o_low, o_qv = oracle.encode_tiled(idx, val, d, residual=m_ref)
        ctx = _ctx(lib, d, W, k, k)
        t_idx, t_val = torch.from_numpy(idx.view(np.int32)).cuda(), torch.from_numpy(val).cuda()
        m = torch.from_numpy(m0.copy()).cuda()
        tab = torch.full((W, spans + 1), -1, dtype=torch.int32, device="cuda")
        low = torch.full((W, ll), -1, dtype=torch.int16, device="cuda")
        qv = torch.full((W, lh), -1, dtype=torch.int16, device="cuda")
        ctx.encode_tiled(t_idx, t_val, d, tab, low, qv, residual=m)
        assert np.array_equal(tab.cpu().numpy().view(np.uint32), o_tab)
        got_low, got_qv = low.cpu().numpy().view(np.uint16), qv.cpu().numpy().view(np.uint16)
        assert np.array_equal(got_low[:, :k], o_low) and not got_low[:, k:].any()
        assert np.array_equal(got_qv[:, :k], o_qv) and not got_qv[:, k:].any()
        assert np.array_equal(_bits(m.cpu().numpy()), _bits(m_ref))
        d_idx, d_val = oracle.decode_tiled(o_tab, o_low, o_qv, d, k)
        assert np.array_equal(d_idx, idx)
        out = torch.full((ld,), float("nan"), dtype=torch.float32, device="cuda")
        for mode, omode in ((lib.SCALE_MEAN, oracle.SCALE_MEAN), (lib.SCALE_SUM, oracle.SCALE_SUM),
                            (lib.SCALE_COUNT, oracle.SCALE_COUNT)):
            ctx.aggregate_tiled(tab, low, qv, d, k, out, scale_mode=mode)
            _, want = oracle.aggregate(d_idx, d_val, d, omode)
            assert np.array_equal(_bits(out.cpu().numpy()[:d]), _bits(want)), (d, W, k, mode)
        # a table that claims more entries than the row holds is read as ending at k (nothing out of bounds)
        bad = tab.clone()
        bad[:, -1] = 2**31 - 1
        ctx.aggregate_tiled(bad, low, qv, d, k, out)
        torch.cuda.synchronize()
        with pytest.raises(lib.RTopKError):
            ctx.aggregate_tiled(tab, low, qv, d, k, out, scale_mode=lib.SCALE_UNBIASED)    # needs r
        ctx.poll_status()
        ctx.close()


def test_momentum_update_against_oracle(lib):
    """Heavy-ball master update: every coordinate's velocity and weight, bit for bit, over several rounds,
    from given messages (all scalings) and fused behind the sparsifier."""
    rng = np.random.default_rng(77)
    for d, W, k in [(300_007, 4, 300), (5000, 3, 2500), (4096, 2, 1), (70_001, 70, 20)]:
        ctx = _ctx(lib, d, W, k, k)
        ld = wl.round_up(d, 4)
        w0 = rng.standard_normal(ld).astype(np.float32)
        v0 = (rng.standard_normal(ld) * 0.1).astype(np.float32)
        for mode, omode, r in ((lib.SCALE_MEAN, oracle.SCALE_MEAN, 0), (lib.SCALE_COUNT, oracle.SCALE_COUNT, 0),
                               (lib.SCALE_UNBIASED, oracle.SCALE_UNBIASED, min(d, 3 * k))):
            w, v = torch.from_numpy(w0.copy()).cuda(), torch.from_numpy(v0.copy()).cuda()
            want_v, want_w = v0[:d].copy(), w0[:d].copy()
            for t in range(3):
                idx = np.stack([np.sort(rng.choice(d, k, replace=False)) for _ in range(W)]).astype(np.uint32)
                val = (rng.standard_normal((W, k)) * np.exp(rng.standard_normal((W, k)))).astype(np.float32)
                ctx.apply_momentum(torch.from_numpy(idx.view(np.int32)).cuda(), torch.from_numpy(val).cuda(), d, 0.05,
                                   0.9, v, w, scale_mode=mode, r=r)
                want_v, want_w = oracle.apply_momentum(idx, val, d, 0.05, 0.9, want_v, want_w, omode, r)
                assert np.array_equal(_bits(v.cpu().numpy()[:d]), _bits(want_v)), (d, W, k, mode, t)
                assert np.array_equal(_bits(w.cpu().numpy()[:d]), _bits(want_w)), (d, W, k, mode, t)
            assert np.array_equal(_bits(w.cpu().numpy()[d:]), _bits(w0[d:]))       # the padding is not touched
        idx_t = torch.zeros((W, k), dtype=torch.int32, device="cuda")
        val_t = torch.zeros((W, k), dtype=torch.float32, device="cuda")
        w, v = torch.from_numpy(w0.copy()).cuda(), torch.from_numpy(v0.copy()).cuda()
        for bad in (dict(eta=-0.1, mu=0.5), dict(eta=0.1, mu=1.0), dict(eta=0.1, mu=float("nan"))):
            with pytest.raises(lib.RTopKError):
                ctx.apply_momentum(idx_t, val_t, d, bad["eta"], bad["mu"], v, w)
        with pytest.raises(lib.RTopKError):
            ctx.apply_momentum(idx_t, val_t, d, 0.1, 0.5, w, w)
        ctx.close()
    # fused behind the sparsifier: three rounds of Algorithm 1 with the momentum master
    cfg = wl.scaled(wl.configs()["c1"], d=300_007, W=4)
    ctx = _ctx(lib, cfg.d, cfg.W, cfg.r, cfg.k)
    w0 = rng.standard_normal(cfg.ld).astype(np.float32)
    w = torch.from_numpy(w0.copy()).cuda()
    v = torch.zeros(cfg.ld, dtype=torch.float32, device="cuda")
    m = wl.zero_residual(cfg, "cuda")
    m_ref = np.zeros((cfg.W, cfg.ld), dtype=np.float32)
    idx = torch.zeros((cfg.W, cfg.k), dtype=torch.int32, device="cuda")
    val = torch.zeros((cfg.W, cfg.k), dtype=torch.float32, device="cuda")
    want_w, want_v = w0[:cfg.d].copy(), np.zeros(cfg.d, dtype=np.float32)
    for t in range(3):
        g = wl.gradient(cfg, t, "cuda")
        ctx.step_momentum(g, m, cfg.d, cfg.r, cfg.k, cfg.seed, t, 0.1, 0.9, idx, val, v, w)
        o_idx, o_val = oracle.sparsify(g.cpu().numpy(), m_ref, cfg.d, cfg.r, cfg.k, cfg.seed, t)
        want_v, want_w = oracle.apply_momentum(o_idx, o_val, cfg.d, 0.1, 0.9, want_v, want_w)
        assert np.array_equal(idx.cpu().numpy().view(np.uint32), o_idx)
        assert np.array_equal(_bits(m.cpu().numpy()), _bits(m_ref))
        assert np.array_equal(_bits(v.cpu().numpy()[:cfg.d]), _bits(want_v))
        assert np.array_equal(_bits(w.cpu().numpy()[:cfg.d]), _bits(want_w))
    ctx.poll_status()
    ctx.close()


def test_aggregate_of_signed_zeros_and_cancelling_values(lib):
    # The sum of a coordinate starts from +0 (as the oracle's accumulator does): a lone -0 gives +0, values that
    # cancel give +0, and both hold for coordinates with one sender and with several.
    d, W, k = 70_000, 3, 4
    idx = np.array([[5, 100, 20_000, 60_000], [5, 101, 20_000, 60_001], [6, 102, 20_000, 60_002]], dtype=np.uint32)
    val = np.array([[-0.0, -0.0, 1.5, -0.0], [-0.0, 2.0, -1.5, 0.0], [-0.0, -2.0, -0.0, -3.0]], dtype=np.float32)
    ctx = _ctx(lib, d, W, k, k)
    out = torch.full((wl.round_up(d, 4),), float("nan"), dtype=torch.float32, device="cuda")
    t_idx, t_val = torch.from_numpy(idx.view(np.int32)).cuda(), torch.from_numpy(val).cuda()
    for mode, omode in ((lib.SCALE_MEAN, oracle.SCALE_MEAN), (lib.SCALE_SUM, oracle.SCALE_SUM),
                        (lib.SCALE_COUNT, oracle.SCALE_COUNT)):
        ctx.aggregate(t_idx, t_val, d, out, scale_mode=mode)
        _, want = oracle.aggregate(idx, val, d, omode)
        assert np.array_equal(_bits(out.cpu().numpy()[:d]), _bits(want)), mode
    w = torch.zeros_like(out)
    ctx.apply_update(t_idx, t_val, d, 0.5, w)
    assert np.array_equal(_bits(w.cpu().numpy()[:d]), _bits(oracle.apply_update(idx, val, d, 0.5, np.zeros(d, dtype=np.float32))))
    ctx.close()


def test_threshold_reuse_changes_nothing_but_the_path(lib):
    """RTOPK_OPT_REUSE_THRESHOLD: consecutive rounds predict the first threshold from the last exact
    ones.  Messages, residual and update stay bit-equal to the oracle; the brackets are predicted
    once two successive thresholds are close to each other; an abrupt collapse of the magnitudes is
    repaired by the exact path and the next two rounds sample again."""
    from paper_2005_10761_b200.binding import OPT_REUSE_THRESHOLD
    cfg = wl.scaled(wl.configs()["c2"], d=400_003, W=3)
    ctx = _ctx(lib, cfg.d, cfg.W, cfg.r, cfg.k)
    ctx.set_option(OPT_REUSE_THRESHOLD, 1)
    m = wl.zero_residual(cfg, "cuda")
    m_ref = np.zeros((cfg.W, cfg.ld), dtype=np.float32)
    idx = torch.zeros((cfg.W, cfg.k), dtype=torch.int32, device="cuda")
    val = torch.zeros((cfg.W, cfg.k), dtype=torch.float32, device="cuda")
    out = torch.empty(cfg.ld, dtype=torch.float32, device="cuda")
    scale = [1.0] * 12 + [None, 1.0, 1.0]
    predicted, fell = [], []
    for t, sc in enumerate(scale):
        g = wl.gradient(cfg, t, "cuda")
        if sc is None:
            g = g * 1e-4 - m                    # a = g + m collapses to a thousandth of its size: every prediction misses
        ctx.step(g, m, cfg.d, cfg.r, cfg.k, cfg.seed, t, idx, val, out)
        o_idx, o_val = oracle.sparsify(g.cpu().numpy(), m_ref, cfg.d, cfg.r, cfg.k, cfg.seed, t)
        _, o_out = oracle.aggregate(o_idx, o_val, cfg.d)
        assert np.array_equal(idx.cpu().numpy().view(np.uint32), o_idx), t
        assert np.array_equal(_bits(val.cpu().numpy()), _bits(o_val)), t
        assert np.array_equal(_bits(m.cpu().numpy()), _bits(m_ref)), t
        assert np.array_equal(_bits(out.cpu().numpy()[:cfg.d]), _bits(o_out)), t
        st = [ctx.stats(w) for w in range(cfg.W)]
        predicted.append(all(s["bracket_predicted"] for s in st))
        fell.append(any(s["used_fallback"] for s in st))
    ctx.poll_status()
    assert not predicted[0] and not predicted[1]              # two exact thresholds are needed before the first prediction
    assert sum(predicted[2:12]) >= 6                          # while the residual builds up the history is not smooth yet
    assert predicted[10] and predicted[11] and not fell[10] and not fell[11]   # steady state: predictions hold
    assert predicted[12] and fell[12] and not predicted[13] and not predicted[14]   # the collapse is missed, repaired, and sampled after
    ctx.close()


def test_step_is_sparsify_then_aggregate(lib):
    cfg = wl.configs()["c1"]
    ctx = _ctx(lib, cfg.d, cfg.W, cfg.r, cfg.k)
    g = wl.gradient(cfg, 0, "cuda")
    m = wl.zero_residual(cfg, "cuda")
    idx = torch.zeros((cfg.W, cfg.k), dtype=torch.int32, device="cuda")
    val = torch.zeros((cfg.W, cfg.k), dtype=torch.float32, device="cuda")
    out = torch.empty(cfg.d, dtype=torch.float32, device="cuda")
    ctx.step(g, m, cfg.d, cfg.r, cfg.k, cfg.seed, 0, idx, val, out)
    ctx.poll_status()
    m_or = np.zeros((cfg.W, cfg.ld), dtype=np.float32)
    g_host = g.cpu().numpy()
    o_idx, o_val = oracle.sparsify(g_host, m_or, cfg.d, cfg.r, cfg.k, cfg.seed, 0)
    o64, o32 = oracle.aggregate(o_idx, o_val, cfg.d)
    assert np.array_equal(idx.cpu().numpy().view(np.uint32), o_idx)
    assert np.array_equal(_bits(val.cpu().numpy()), _bits(o_val))
    assert np.array_equal(_bits(m.cpu().numpy()), _bits(m_or))
    got = out.cpu().numpy()
    assert np.abs(got.astype(np.float64) - o64).max() <= 1e-6 * float(np.abs(g_host).max())
    assert np.array_equal(_bits(got), _bits(o32))
    # the sampled threshold did its job on this configuration (no fallback)
    assert all(ctx.stats(w)["used_fallback"] == 0 for w in range(cfg.W))
    ctx.close()


def test_pairs_format_equals_the_two_array_format(lib):
    # one buffer of 8-byte (index, value) pairs per worker -- what a sharded run all-gathers -- through
    # both finishing paths and the random-k limit, and its aggregation, against the two-array calls
    from paper_2005_10761_b200 import sharded
    cfg = wl.scaled(wl.configs()["c2"], d=300011, W=5)
    g = wl.gradient(cfg, 0, "cuda")
    for path, (r, k) in [(AUTO, (cfg.r, cfg.k)), (RUNS, (cfg.r, cfg.k)), (AUTO, (cfg.d, cfg.k)), (EXACT, (cfg.r, cfg.r))]:
        ctx = _ctx(lib, cfg.d, cfg.W, r, k, path=path)
        m1, m2 = wl.zero_residual(cfg, "cuda"), wl.zero_residual(cfg, "cuda")
        idx = torch.zeros((cfg.W, k), dtype=torch.int32, device="cuda")
        val = torch.zeros((cfg.W, k), dtype=torch.float32, device="cuda")
        pairs = torch.zeros((cfg.W, k), dtype=torch.int64, device="cuda")
        out1 = torch.empty(cfg.ld, dtype=torch.float32, device="cuda")
        out2 = torch.empty(cfg.ld, dtype=torch.float32, device="cuda")
        ctx.sparsify(g, m1, cfg.d, r, k, 21, 3, idx, val, worker_base=7)
        ctx.sparsify_pairs(g, m2, cfg.d, r, k, 21, 3, pairs, worker_base=7)
        ctx.aggregate(idx, val, cfg.d, out1)
        ctx.aggregate_pairs(pairs, cfg.d, out2)
        ctx.poll_status()
        i2, v2 = sharded.unpack_pairs(pairs)
        assert torch.equal(i2, idx) and torch.equal(v2.view(torch.int32), val.view(torch.int32)), (path, r, k)
        assert torch.equal(m1.view(torch.int32), m2.view(torch.int32))
        assert torch.equal(out1[: cfg.d].view(torch.int32), out2[: cfg.d].view(torch.int32))
        ctx.close()


def test_step_host_matches_device_call(lib):
    cfg = wl.scaled(wl.configs()["c1"], d=200003, W=3)
    ctx = _ctx(lib, cfg.d, cfg.W, cfg.r, cfg.k)
    g = wl.gradient(cfg, 0, "cpu").pin_memory()
    m1, m2 = wl.zero_residual(cfg, "cuda"), wl.zero_residual(cfg, "cuda")
    idx_d = torch.zeros((cfg.W, cfg.k), dtype=torch.int32, device="cuda")
    val_d = torch.zeros((cfg.W, cfg.k), dtype=torch.float32, device="cuda")
    out_d = torch.empty(cfg.ld, dtype=torch.float32, device="cuda")
    ctx.step(g.cuda(), m1, cfg.d, cfg.r, cfg.k, 3, 1, idx_d, val_d, out_d)
    idx_h = torch.zeros((cfg.W, cfg.k), dtype=torch.int32).pin_memory()
    val_h = torch.zeros((cfg.W, cfg.k), dtype=torch.float32).pin_memory()
    out_h = torch.zeros(cfg.d, dtype=torch.float32).pin_memory()
    ctx.step_host(g, m2, cfg.d, cfg.r, cfg.k, 3, 1, idx_h, val_h, out_h)
    torch.cuda.synchronize()
    assert torch.equal(idx_h, idx_d.cpu()) and torch.equal(val_h.view(torch.int32), val_d.cpu().view(torch.int32))
    assert torch.equal(out_h.view(torch.int32), out_d.cpu()[: cfg.d].view(torch.int32))
    assert torch.equal(m1.view(torch.int32), m2.view(torch.int32))
    ctx.close()


def test_step_host_sequence_without_waiting_in_between(lib):
    # Five calls in a row on one stream, each with its own gradient and result buffers and no wait between
    # them: uploads, steps and downloads of neighbouring calls overlap inside the library, and every
    # call must still give what the device call gives on the same data (residual carried).
    cfg = wl.scaled(wl.configs()["c2"], d=600011, W=4)
    ctx = _ctx(lib, cfg.d, cfg.W, cfg.r, cfg.k)
    n = 5
    gs = [wl.gradient(cfg, t, "cpu").pin_memory() for t in range(n)]
    idx_h = [torch.zeros((cfg.W, cfg.k), dtype=torch.int32).pin_memory() for _ in range(n)]
    val_h = [torch.zeros((cfg.W, cfg.k), dtype=torch.float32).pin_memory() for _ in range(n)]
    out_h = [torch.zeros(cfg.d, dtype=torch.float32).pin_memory() for _ in range(n)]
    m_h = wl.zero_residual(cfg, "cuda")
    for t in range(n):
        ctx.step_host(gs[t], m_h, cfg.d, cfg.r, cfg.k, cfg.seed, t, idx_h[t], val_h[t], out_h[t])
    torch.cuda.synchronize()
    ctx.poll_status()
    ctx2 = _ctx(lib, cfg.d, cfg.W, cfg.r, cfg.k)
    m_d = wl.zero_residual(cfg, "cuda")
    idx_d = torch.zeros((cfg.W, cfg.k), dtype=torch.int32, device="cuda")
    val_d = torch.zeros((cfg.W, cfg.k), dtype=torch.float32, device="cuda")
    out_d = torch.empty(cfg.ld, dtype=torch.float32, device="cuda")
    for t in range(n):
        ctx2.step(gs[t].cuda(), m_d, cfg.d, cfg.r, cfg.k, cfg.seed, t, idx_d, val_d, out_d)
        torch.cuda.synchronize()
        assert torch.equal(idx_h[t], idx_d.cpu()), t
        assert torch.equal(val_h[t].view(torch.int32), val_d.cpu().view(torch.int32)), t
        assert torch.equal(out_h[t].view(torch.int32), out_d.cpu()[: cfg.d].view(torch.int32)), t
    assert torch.equal(m_h.view(torch.int32), m_d.view(torch.int32))


def test_step_host_calls_of_changing_shape(lib):
    # W = 8, then W = 4, then W = 8 again through one context with no wait in between: the smaller call
    # divides the staging buffers differently, which must not disturb the call before it (whose step may
    # still be reading its gradient) nor the call after it.
    base = wl.scaled(wl.configs()["c2"], d=400009, W=8)
    shapes = [base, wl.scaled(wl.configs()["c2"], d=400009, W=4), base]
    ctx = _ctx(lib, base.d, 8, base.r, base.k)
    gs, res, m_h = [], [], []
    for t, cfg in enumerate(shapes):
        gs.append(wl.gradient(cfg, t, "cpu").pin_memory())
        res.append((torch.zeros((cfg.W, cfg.k), dtype=torch.int32).pin_memory(),
                    torch.zeros((cfg.W, cfg.k), dtype=torch.float32).pin_memory(),
                    torch.zeros(cfg.d, dtype=torch.float32).pin_memory()))
        m_h.append(wl.zero_residual(cfg, "cuda"))
    for t, cfg in enumerate(shapes):
        ctx.step_host(gs[t], m_h[t], cfg.d, cfg.r, cfg.k, cfg.seed, t, *res[t])
    torch.cuda.synchronize()
    ctx.poll_status()
    ctx2 = _ctx(lib, base.d, 8, base.r, base.k)
    for t, cfg in enumerate(shapes):
        m_d = wl.zero_residual(cfg, "cuda")
        idx_d = torch.zeros((cfg.W, cfg.k), dtype=torch.int32, device="cuda")
        val_d = torch.zeros((cfg.W, cfg.k), dtype=torch.float32, device="cuda")
        out_d = torch.empty(cfg.ld, dtype=torch.float32, device="cuda")
        ctx2.step(gs[t].cuda(), m_d, cfg.d, cfg.r, cfg.k, cfg.seed, t, idx_d, val_d, out_d)
        torch.cuda.synchronize()
        assert torch.equal(res[t][0], idx_d.cpu()), t
        assert torch.equal(res[t][1].view(torch.int32), val_d.cpu().view(torch.int32)), t
        assert torch.equal(res[t][2].view(torch.int32), out_d.cpu()[: cfg.d].view(torch.int32)), t
        assert torch.equal(m_h[t].view(torch.int32), m_d.view(torch.int32)), t
    ctx.close(); ctx2.close()


@pytest.mark.parametrize("r,k", [(1, 1), (2, 1), (7, 3), (64, 64), (1000, 1), (1000, 999), (16384, 1024),
                                 (111739, 11173), (2684354, 671088)])
def test_sampler_positions_against_oracle(lib, r, k):
    ctx = _ctx(lib, r, 1, r, k)
    pos = torch.zeros(k, dtype=torch.int32, device="cuda")
    for seed, step, worker, seg in [(0, 0, 0, 0), (0xABCDEF0123456789, 9, 31, 5)]:
        ctx.sample_positions(r, k, seed, step, worker, seg, pos)
        want = oracle.sample_positions(r, k, seed, step, worker, seg)
        assert np.array_equal(pos.cpu().numpy().view(np.uint32), want)
    ctx.close()


def test_repeated_runs_are_bit_identical(lib):
    cfg = wl.scaled(wl.configs()["c1"], d=500000, W=4)
    g = wl.gradient(cfg, 0, "cuda")
    ref = None
    ctx = _ctx(lib, cfg.d, cfg.W, cfg.r, cfg.k)
    for _ in range(20):
        m = wl.zero_residual(cfg, "cuda")
        idx = torch.zeros((cfg.W, cfg.k), dtype=torch.int32, device="cuda")
        val = torch.zeros((cfg.W, cfg.k), dtype=torch.float32, device="cuda")
        out = torch.empty(cfg.ld, dtype=torch.float32, device="cuda")
        ctx.step(g, m, cfg.d, cfg.r, cfg.k, 5, 5, idx, val, out)
        got = (idx.cpu(), val.cpu().view(torch.int32), m.cpu().view(torch.int32), out.cpu().view(torch.int32))
        if ref is None:
            ref = got
        else:
            assert all(torch.equal(a, b) for a, b in zip(ref, got))
    ctx.close()


def test_fallback_is_taken_and_exact_when_the_sample_misleads(lib):
    # large values only in a region the strided sample sees little of: the estimate is too high or
    # too low, the count check fails and the exact path must repair it
    W, d, r, k = 2, 400000, 4000, 400
    rng = np.random.default_rng(11)
    g = (rng.standard_normal((W, d)) * 1e-3).astype(np.float32)
    g[:, 1000:1000 + 6000] = rng.standard_normal((W, 6000)).astype(np.float32) * 5     # a dense hot band
    g = _pad(g)
    m0 = np.zeros_like(g)
    stats = check_against_oracle(lib, g, m0, d, r, k, seed=12, step=0, path=AUTO)
    g2 = np.zeros((W, d), dtype=np.float32)                                              # ties overflow the list
    g2[:, ::2] = 1.0
    g2 = _pad(g2)
    stats2 = check_against_oracle(lib, g2, np.zeros_like(g2), d, r, k, seed=12, step=0, path=AUTO)
    assert any(s["used_fallback"] for s in stats + stats2)


def test_a_wait_that_gives_up_is_reported_and_leaves_the_context_usable(lib):
    # The waits inside the kernels are bounded (the streaming pass's waits for its bulk copies and for free
    # stages are the only ones).  A test-only option makes every block of that pass take the exit of a wait
    # that ran out (no GPU fault, no hang is involved; the copies all arrive and are waited for): the call
    # returns, nothing outside the caller's buffers is written (canaries around the messages and the
    # residual), the status poll reports the internal error, and the same context then serves a normal
    # call correctly.
    from paper_2005_10761_b200.binding import OPT_TEST_STREAM_GIVEUP
    rng = np.random.default_rng(77)
    W, d, r, k = 2, 20000, 5000, 500                 # five chunks per row
    g = _pad(_spiky(rng, W, d))
    ld = g.shape[1]
    ctx = _ctx(lib, d, W, r, k)
    tg = torch.from_numpy(g).cuda()
    pad = 4096
    res_buf = torch.full((W * ld + 2 * pad,), 123.0, dtype=torch.float32, device="cuda")
    idx_buf = torch.full((W * k + 2 * pad,), -7, dtype=torch.int32, device="cuda")
    val_buf = torch.full((W * k + 2 * pad,), -7.0, dtype=torch.float32, device="cuda")
    tm = res_buf[pad:pad + W * ld].view(W, ld)
    tm.zero_()
    idx = idx_buf[pad:pad + W * k].view(W, k)
    val = val_buf[pad:pad + W * k].view(W, k)
    ctx.set_option(OPT_TEST_STREAM_GIVEUP, 1)
    ctx.sparsify(tg, tm, d, r, k, 5, 0, idx, val)
    torch.cuda.synchronize()
    with pytest.raises(lib.RTopKError) as e:
        ctx.poll_status()
    assert e.value.status == 5                                       # RTOPK_ERR_INTERNAL
    for buf, fill in ((res_buf, 123.0), (idx_buf, -7), (val_buf, -7.0)):
        assert bool((buf[:pad] == fill).all()) and bool((buf[-pad:] == fill).all())
    assert bool((tm[:, d:] == 0).all())                              # padding columns untouched
    ctx.poll_status()                                                # the flag was cleared by the failed poll
    # back to normal: the same context gives the oracle's result
    ctx.set_option(OPT_TEST_STREAM_GIVEUP, 0)
    tm.zero_()
    m_or = np.zeros_like(g)
    ctx.sparsify(tg, tm, d, r, k, 5, 1, idx, val)
    ctx.poll_status()
    o_idx, o_val = oracle.sparsify(g, m_or, d, r, k, 5, 1)
    assert np.array_equal(idx.cpu().numpy().view(np.uint32), o_idx)
    assert np.array_equal(_bits(val.cpu().numpy()), _bits(o_val))
    assert np.array_equal(_bits(tm.cpu().numpy()), _bits(m_or))
    ctx.close()


def test_bad_arguments_return_invalid_arg_and_write_nothing(lib):
    d, W, r, k = 4096, 2, 64, 8
    ctx = _ctx(lib, d, W, r, k)
    g = torch.zeros((W, d), dtype=torch.float32, device="cuda")
    m = torch.ones((W, d), dtype=torch.float32, device="cuda")
    idx = torch.zeros((W, k), dtype=torch.int32, device="cuda")
    val = torch.zeros((W, k), dtype=torch.float32, device="cuda")
    out = torch.zeros(d, dtype=torch.float32, device="cuda")
    bad = [dict(r=8, k=9), dict(r=d + 1, k=8), dict(r=64, k=0), dict(d=d + 4), dict(r=128, k=8)]
    for kw in bad:
        a = dict(d=d, r=r, k=k)
        a.update(kw)
        with pytest.raises(lib.RTopKError) as e:
            ctx.sparsify(g, m, a["d"], a["r"], a["k"], 0, 0, idx, val)
        assert e.value.status == 1
    with pytest.raises(lib.RTopKError):
        ctx.sparsify(g[:, 1:], m, d - 1, r, k, 0, 0, idx, val)          # misaligned base / stride
    with pytest.raises(lib.RTopKError):
        ctx.aggregate(idx, val, d, out, scale_mode=7)
    with pytest.raises(lib.RTopKError):
        lib.RTopK(d_max=1 << 31, W_max=1, r_max=1, k_max=1)
    torch.cuda.synchronize()
    assert bool((m == 1).all())
    ctx.poll_status()
    ctx.close()


def test_step_can_be_captured_in_a_cuda_graph_and_replayed(lib):
    # The call only enqueues work (its side stream forks from and rejoins the caller's stream), so a
    # caller may capture it; the replay must give what the oracle gives for the captured (seed, step).
    cfg = wl.scaled(wl.configs()["c2"], d=400003, W=3)
    ctx = _ctx(lib, cfg.d, cfg.W, cfg.r, cfg.k)
    g = wl.gradient(cfg, 0, "cuda")
    m = wl.zero_residual(cfg, "cuda")
    idx = torch.zeros((cfg.W, cfg.k), dtype=torch.int32, device="cuda")
    val = torch.zeros((cfg.W, cfg.k), dtype=torch.float32, device="cuda")
    out = torch.zeros(wl.round_up(cfg.d, 4), dtype=torch.float32, device="cuda")
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        ctx.step(g, m, cfg.d, cfg.r, cfg.k, cfg.seed, 0, idx, val, out)      # first call outside the capture
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=s):
            ctx.step(g, m, cfg.d, cfg.r, cfg.k, cfg.seed, 1, idx, val, out)
        m.zero_()
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        ctx.poll_status()
    m_or = np.zeros((cfg.W, cfg.ld), dtype=np.float32)
    o_idx, o_val = oracle.sparsify(g.cpu().numpy(), m_or, cfg.d, cfg.r, cfg.k, cfg.seed, 1)
    _, o32 = oracle.aggregate(o_idx, o_val, cfg.d)
    assert np.array_equal(idx.cpu().numpy().view(np.uint32), o_idx)
    assert np.array_equal(_bits(val.cpu().numpy()), _bits(o_val))
    assert np.array_equal(_bits(m.cpu().numpy()), _bits(m_or))
    assert np.array_equal(_bits(out.cpu().numpy()[:cfg.d]), _bits(o32))


def test_a_captured_first_call_sends_its_slice_table_from_the_context(lib):
    # The first call of a shape sends the table of its slices to the device.  When that call is captured, the
    # copy in the graph reads a buffer of the context (not one of the call), so replays long after the call
    # has returned still send the right table.
    cfg = wl.scaled(wl.configs()["c2"], d=300017, W=2)
    ctx = _ctx(lib, cfg.d, cfg.W, cfg.r, cfg.k)
    g = wl.gradient(cfg, 0, "cuda")
    m = wl.zero_residual(cfg, "cuda")
    idx = torch.zeros((cfg.W, cfg.k), dtype=torch.int32, device="cuda")
    val = torch.zeros((cfg.W, cfg.k), dtype=torch.float32, device="cuda")
    out = torch.zeros(wl.round_up(cfg.d, 4), dtype=torch.float32, device="cuda")
    s = torch.cuda.Stream()
    m_or = np.zeros((cfg.W, cfg.ld), dtype=np.float32)
    with torch.cuda.stream(s):
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=s):
            ctx.step(g, m, cfg.d, cfg.r, cfg.k, cfg.seed, 3, idx, val, out)   # the context's very first call
        junk = [torch.empty(1 << 20, dtype=torch.uint8).random_() for _ in range(8)]   # host allocations come and go
        del junk
        for _ in range(2):                                                   # same step both times: residual carried
            graph.replay()
            torch.cuda.synchronize()
            ctx.poll_status()
            o_idx, o_val = oracle.sparsify(g.cpu().numpy(), m_or, cfg.d, cfg.r, cfg.k, cfg.seed, 3)
            _, o32 = oracle.aggregate(o_idx, o_val, cfg.d)
            assert np.array_equal(idx.cpu().numpy().view(np.uint32), o_idx)
            assert np.array_equal(_bits(val.cpu().numpy()), _bits(o_val))
            assert np.array_equal(_bits(m.cpu().numpy()), _bits(m_or))
            assert np.array_equal(_bits(out.cpu().numpy()[:cfg.d]), _bits(o32))
    ctx.close()


@pytest.mark.parametrize("case", range(24))
def test_random_shapes_values_and_paths(lib, case):
    # Seeded random draws of everything a caller chooses: length, workers, r, k, first worker id, step,
    # gradient type, selection path, and how heavy the ties are (values quantised to a few levels).
    rng = np.random.default_rng(1000 + case)
    d = int(rng.choice([rng.integers(1, 64), rng.integers(64, 5000), rng.integers(5000, 200000)]))
    W = int(rng.integers(1, 6))
    r = int(rng.integers(1, d + 1)) if rng.random() < 0.3 else int(max(1, d * rng.choice([0.001, 0.01, 0.05, 0.3])))
    k = int(rng.integers(1, r + 1)) if rng.random() < 0.5 else max(1, r // int(rng.choice([2, 4, 10])))
    g = _spiky(rng, W, d, p=float(rng.choice([0.0, 0.01, 0.2])))
    m0 = _spiky(rng, W, d) * 0.5
    levels = int(rng.choice([0, 0, 3, 17]))
    if levels:                                   # many equal magnitudes, some across the threshold
        g = (np.round(g * levels) / levels).astype(np.float32)
        m0 = (np.round(m0 * levels) / levels).astype(np.float32)
    check_against_oracle(lib, _pad(g), _pad(m0), d, r, k, seed=int(rng.integers(0, 2**40)), step=int(rng.integers(0, 1000)),
                         worker_base=int(rng.integers(0, 50)), path=int(rng.choice([AUTO, EXACT, RUNS])),
                         bf16=bool(rng.random() < 0.3))


def test_device_round_counter_and_graph_replay_draw_fresh_subsets(lib):
    # With the round counter on the device the `step` argument is ignored and every call advances the
    # counter, so a captured round can be replayed and still follows Algorithm 1's t = 0, 1, 2, ...:
    # eager calls with explicit steps, eager calls on the counter and graph replays must agree bit for bit.
    cfg = wl.scaled(wl.configs()["c2"], d=300007, W=3)
    g = wl.gradient(cfg, 0, "cuda")
    n, first = 4, 7

    def buffers():
        return (wl.zero_residual(cfg, "cuda"), torch.zeros((cfg.W, cfg.k), dtype=torch.int32, device="cuda"),
                torch.zeros((cfg.W, cfg.k), dtype=torch.float32, device="cuda"),
                torch.zeros(wl.round_up(cfg.d, 4), dtype=torch.float32, device="cuda"))

    want = []
    ctx = _ctx(lib, cfg.d, cfg.W, cfg.r, cfg.k)
    m, idx, val, out = buffers()
    for t in range(first, first + n):
        ctx.step(g, m, cfg.d, cfg.r, cfg.k, cfg.seed, t, idx, val, out)
        want.append((idx.clone(), val.clone(), out.clone(), m.clone()))
    ctx.close()

    ctx = _ctx(lib, cfg.d, cfg.W, cfg.r, cfg.k)
    ctx.set_option(4, 1)
    ctx.set_device_step(first)
    m, idx, val, out = buffers()
    for i in range(n):
        ctx.step(g, m, cfg.d, cfg.r, cfg.k, cfg.seed, 12345, idx, val, out)       # the argument is ignored
        for got, ref in zip((idx, val, out, m), want[i]):
            assert torch.equal(got.view(torch.int32), ref.view(torch.int32)), i
    ctx.poll_status()

    # the same rounds as replays of one captured call
    m, idx, val, out = buffers()
    ctx.set_device_step(first)
    s = torch.cuda.Stream()
    torch.cuda.synchronize()
    with torch.cuda.stream(s):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=s):
            ctx.step(g, m, cfg.d, cfg.r, cfg.k, cfg.seed, 0, idx, val, out)
        for i in range(n):
            graph.replay()
            torch.cuda.synchronize()
            for got, ref in zip((idx, val, out, m), want[i]):
                assert torch.equal(got.view(torch.int32), ref.view(torch.int32)), i
    ctx.poll_status()
    ctx.close()


def test_device_round_counter_in_segmented_threshold_and_limit_calls(lib):
    # every sparsify-type call reads and advances the counter: per-tensor, threshold encoder, r = d (no
    # selection kernel) and k = r (no subset kernels); each must match the oracle at the counter's value
    rng = np.random.default_rng(31)
    W, d = 2, 50021
    g = _pad(_spiky(rng, W, d))
    tg = torch.from_numpy(g).cuda()
    ctx = lib.RTopK(d_max=d, W_max=W, r_max=d, k_max=600, segments_max=2)
    ctx.set_option(4, 1)
    ctx.set_device_step(40)
    tm = torch.zeros(g.shape, device="cuda")
    m_or = np.zeros_like(g)
    out = torch.empty(wl.round_up(d, 4), dtype=torch.float32, device="cuda")

    def msgs(k):
        return (torch.zeros((W, k), dtype=torch.int32, device="cuda"), torch.zeros((W, k), dtype=torch.float32, device="cuda"))

    # t = 40: per-tensor
    off, seg_r, seg_k = [0, 20003, d], [300, 500], [30, 50]
    idx, val = msgs(80)
    ctx.step_segmented(tg, tm, d, off, seg_r, seg_k, 9, 999, idx, val, out)
    o_idx, o_val = oracle.sparsify_segmented(g, m_or, d, off, seg_r, seg_k, seed=9, step=40)
    assert np.array_equal(idx.cpu().numpy().view(np.uint32), o_idx) and np.array_equal(_bits(val.cpu().numpy()), _bits(o_val))
    # t = 41: threshold encoder
    idx, val = msgs(60)
    cnt = torch.zeros(W, dtype=torch.int32, device="cuda")
    ones = torch.zeros(W, dtype=torch.int32, device="cuda")
    ctx.step_threshold(tg, tm, d, 0.3, 60, 9, 999, idx, val, cnt, ones, out)
    o_idx, o_val, o_cnt, o_ones = oracle.sparsify_threshold(g, m_or, d, 0.3, 60, 9, 41)
    assert (o_ones > 60).all()
    assert np.array_equal(idx.cpu().numpy().view(np.uint32), o_idx) and np.array_equal(_bits(val.cpu().numpy()), _bits(o_val))
    # t = 42: r = d (random-k), t = 43: k = r (top-k, draws nothing), t = 44: plain again
    for r, k, t in ((d, 100, 42), (400, 400, 43), (600, 60, 44)):
        idx, val = msgs(k)
        ctx.step(tg, tm, d, r, k, 9, 999, idx, val, out)
        o_idx, o_val = oracle.sparsify(g, m_or, d, r, k, 9, t)
        assert np.array_equal(idx.cpu().numpy().view(np.uint32), o_idx), (r, k)
        assert np.array_equal(_bits(val.cpu().numpy()), _bits(o_val)), (r, k)
    assert np.array_equal(_bits(tm.cpu().numpy()), _bits(m_or))
    ctx.poll_status()
    ctx.close()


def test_checkpoint_and_resume_with_a_new_context(lib):
    # The only state of Algorithm 1's node loop is the residual and the round number: ten rounds in one go
    # equal five rounds, a checkpoint of the residual on the host, a new context, and five more rounds.
    cfg = wl.scaled(wl.configs()["c2"], d=250003, W=3)
    gs = [wl.gradient(cfg, t, "cuda") for t in range(10)]

    def run(ctx, m, t0, t1, keep):
        idx = torch.zeros((cfg.W, cfg.k), dtype=torch.int32, device="cuda")
        val = torch.zeros((cfg.W, cfg.k), dtype=torch.float32, device="cuda")
        out = torch.zeros(wl.round_up(cfg.d, 4), dtype=torch.float32, device="cuda")
        for t in range(t0, t1):
            ctx.step(gs[t], m, cfg.d, cfg.r, cfg.k, cfg.seed, t, idx, val, out)
            keep.append((idx.cpu().clone(), val.cpu().clone(), out.cpu().clone()))
        ctx.poll_status()

    straight, resumed = [], []
    ctx = _ctx(lib, cfg.d, cfg.W, cfg.r, cfg.k)
    ctx.set_option(2, 1)                                  # threshold reuse: its history is not part of the state
    m = wl.zero_residual(cfg, "cuda")
    run(ctx, m, 0, 10, straight)
    m_straight = m.cpu().clone()
    ctx.close()

    ctx = _ctx(lib, cfg.d, cfg.W, cfg.r, cfg.k)
    ctx.set_option(2, 1)
    m = wl.zero_residual(cfg, "cuda")
    run(ctx, m, 0, 5, resumed)
    checkpoint = m.cpu().clone()
    ctx.close()
    del m
    ctx = _ctx(lib, cfg.d, cfg.W, cfg.r, cfg.k)           # a fresh context and a fresh residual buffer
    m = checkpoint.cuda()
    run(ctx, m, 5, 10, resumed)
    for a, b in zip(straight, resumed):
        for x, y in zip(a, b):
            assert torch.equal(x.view(torch.int32), y.view(torch.int32))
    assert torch.equal(m.cpu().view(torch.int32), m_straight.view(torch.int32))


@pytest.mark.parametrize("bf16", [False, True])
def test_exact_selection_inside_the_finishing_cluster(lib, bf16):
    # Every slice is made to miss its first bracket (threshold reuse, then a collapse of the magnitudes), with
    # many workers (small clusters), long rows (several CTAs and chunks per slice) and values quantised to a
    # few levels, so that ties straddle the r-th largest magnitude and the tie quota decides.
    from paper_2005_10761_b200.binding import OPT_REUSE_THRESHOLD
    rng = np.random.default_rng(77)
    W, d, r, k = 12, 150001, 3000, 300
    ctx = _ctx(lib, d, W, r, k)
    ctx.set_option(OPT_REUSE_THRESHOLD, 1)
    tm = torch.zeros((W, wl.round_up(d, 8)), dtype=torch.float32, device="cuda")
    m_or = np.zeros((W, wl.round_up(d, 8)), dtype=np.float32)
    idx = torch.zeros((W, k), dtype=torch.int32, device="cuda")
    val = torch.zeros((W, k), dtype=torch.float32, device="cuda")
    fell = []
    for t in range(8):
        g = _pad(_spiky(rng, W, d, p=0.05))
        if t >= 5:
            g = (np.round(g * 4) / 4).astype(np.float32) * (1e-3 if t == 5 else 1.0)   # few levels; t = 5 collapses
            g = g - (m_or if t == 5 else 0)
        tg = torch.from_numpy(g).cuda()
        g_or = g
        if bf16:
            tg = tg.to(torch.bfloat16)
            g_or = tg.view(torch.int16).cpu().numpy().view(np.uint16).copy()
        ctx.sparsify(tg, tm, d, r, k, 5, t, idx, val)
        ctx.poll_status()
        o_idx, o_val = oracle.sparsify(g_or, m_or, d, r, k, 5, t)
        assert np.array_equal(idx.cpu().numpy().view(np.uint32), o_idx), t
        assert np.array_equal(_bits(val.cpu().numpy()), _bits(o_val)), t
        assert np.array_equal(_bits(tm.cpu().numpy()), _bits(m_or)), t
        fell.append(sum(ctx.stats(w)["used_fallback"] for w in range(W)))
    assert max(fell) == W                      # in some round every slice took the exact path
    ctx.close()


def test_reused_thresholds_settle_on_a_gaussian_gradient(lib):
    # A plain Gaussian bulk has a steep tail: a predicted bracket at its widest lets about three times r
    # candidates through and overflows the list.  Such a miss has to narrow the next brackets (widening them
    # made every third round miss for ever).  Thirty rounds with a fresh gradient each, residual carried: the
    # brackets of nearly all rounds are predicted and at most three of the sixty slices-rounds are repaired.
    from paper_2005_10761_b200 import binding as B
    d, W = 4_000_000, 2
    r, k = d // 100, d // 1000
    ctx = _ctx(lib, d, W, r, k)
    ctx.set_option(B.OPT_REUSE_THRESHOLD, 1)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(11)
    m = torch.zeros((W, d), device="cuda")
    idx = torch.zeros((W, k), dtype=torch.int32, device="cuda")
    val = torch.zeros((W, k), device="cuda")
    out = torch.zeros(d, device="cuda")
    repaired = predicted = 0
    for t in range(30):
        g = torch.randn((W, d), generator=gen, device="cuda") * 1e-3
        a = g + m
        ctx.step(g, m, d, r, k, 7, t, idx, val, out)
        ctx.poll_status()
        for w in range(W):
            st = ctx.stats(w)
            repaired += st["used_fallback"]
            predicted += st["bracket_predicted"]
            i = idx[w].to(torch.int64)                     # whatever the path, the round is a valid one
            back = m[w].clone()
            back[i] = val[w]
            assert torch.equal(back.view(torch.int32), a[w].view(torch.int32))
            key = a[w].view(torch.int32) & 0x7FFFFFFF
            assert int((key > st["tau_key"]).sum()) == st["n_greater"] < r
    assert predicted >= 40 and repaired <= 3, (predicted, repaired)
    ctx.close()
