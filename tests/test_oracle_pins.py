"""Pins for the CPU oracle: what the paper and the mathematics fix, checked without a GPU.

Each test ties one piece of ``oracle/`` to something other than itself: published
known answers (Philox), big-integer arithmetic (draw scaling), exhaustive enumeration
(Floyd yields every k-subset equally often, Definition 3's "uniformly at random"),
brute force and library sorts (Definition 1), the closed form in the proof of
Proposition 1, the limits k = r (Definition 1) and r = d (Definition 2), and the
identities of Algorithm 1 (m' = a - ghat; the master's 1/n average).
"""
import itertools
import math
import os
from collections import Counter

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------- Philox
def _golden_lines(kind):
    with open(os.path.join(GOLDEN, "philox4x32_10_known_answers.txt")) as f:
        for line in f:
            tok = line.split()
            if tok and tok[0] == kind:
                yield tok[1:]


def test_philox_known_answers():
    n = 0
    for tok in _golden_lines("kat"):
        w = [int(t, 16) for t in tok]
        got = oracle.philox4x32_10(w[0:4], w[4:6])
        assert [int(x) for x in got] == w[6:10]
        n += 1
    assert n >= 2


def test_philox_cxx_standard_10000th_value():
    for tok in _golden_lines("nth"):
        n, seed, want = (int(t) for t in tok)
        block, word = divmod(n - 1, 4)
        got = oracle.philox4x32_10([block, 0, 0, 0], [seed, 0])
        assert int(got[word]) == want


def test_scale_draw_matches_big_integer_floor():
    rng = np.random.default_rng(1)
    cases = [(0, 1), (0, 7), (2**64 - 1, 1), (2**64 - 1, 7), (2**63, 2), (2**63 - 1, 2),
             (2**64 - 1, 2**31), (2**64 - 1, 2**32 - 1)]
    for _ in range(2000):
        cases.append((int(rng.integers(0, 2**64, dtype=np.uint64)), int(rng.integers(1, 2**32))))
    for u, n in cases:
        assert oracle.scale_draw(u, n) == (u * n) >> 64


def test_draw_uses_words_0_and_1_and_counter_layout():
    # t_j = floor(((x1 << 32) | x0) * (j + 1) / 2^64), counter = (j, worker, segment, step),
    # key = (seed lo, seed hi): the library's reading of "uniformly at random".
    seed = 0x0123456789ABCDEF
    for step, worker, seg, j in [(0, 0, 0, 0), (3, 2, 1, 77), (9, 31, 5, 2**28 - 1)]:
        x = oracle.philox4x32_10([j, worker, seg, step], [seed & 0xFFFFFFFF, seed >> 32])
        u = (int(x[1]) << 32) | int(x[0])
        assert oracle.draw(seed, step, worker, seg, j) == (u * (j + 1)) >> 64


def test_draw_streams_differ_across_seed_step_worker_segment():
    base = [oracle.draw(7, 1, 2, 3, j) for j in range(1000, 1200)]
    for args in [(8, 1, 2, 3), (7, 2, 2, 3), (7, 1, 3, 3), (7, 1, 2, 4), (7 + 2**32, 1, 2, 3)]:
        other = [oracle.draw(*args, j) for j in range(1000, 1200)]
        assert sum(a == b for a, b in zip(base, other)) < 10
    assert all(0 <= t <= j for t, j in zip(base, range(1000, 1200)))


# ----------------------------------------------------------------------------- Floyd
@pytest.mark.parametrize("r", [1, 2, 3, 4, 5, 6, 7])
def test_floyd_is_uniform_over_k_subsets_exhaustively(r):
    # Over all admissible draw tuples every k-subset of {0..r-1} must appear equally often.
    for k in range(1, r + 1):
        ranges = [range(j + 1) for j in range(r - k, r)]
        counts = Counter()
        for t in itertools.product(*ranges):
            pos = oracle.floyd_from_draws(r, k, np.array(t, dtype=np.uint32))
            assert len(set(pos.tolist())) == k and list(pos) == sorted(pos)
            counts[tuple(pos.tolist())] += 1
        total = math.prod(j + 1 for j in range(r - k, r))
        assert len(counts) == math.comb(r, k)
        assert set(counts.values()) == {total // math.comb(r, k)}


def test_floyd_limits():
    # k = r: every position; k = 1: the single draw of iteration r-1
    for r in (1, 5, 64):
        t = np.array([oracle.draw(3, 0, 0, 0, j) for j in range(r)], dtype=np.uint32)
        assert oracle.floyd_from_draws(r, r, t).tolist() == list(range(r))
        assert oracle.sample_positions(r, r, 3, 0, 0).tolist() == list(range(r))
    for r in (1, 9, 1000):
        assert oracle.sample_positions(r, 1, 11, 4, 2, 1).tolist() == [oracle.draw(11, 4, 2, 1, r - 1)]
    with pytest.raises(ValueError):
        oracle.floyd_from_draws(4, 2, np.array([3, 0], dtype=np.uint32))  # t_2 = 3 > 2


def _chi2_ok(observed, expected, dof, z=5.0):
    stat = float(((observed - expected) ** 2 / expected).sum())
    return abs(stat - dof) < z * math.sqrt(2 * dof), stat


def test_sampler_inclusion_frequencies_are_k_over_r():
    # each position is kept with probability k/r: its hit count over n seeds is Binomial(n, k/r)
    r, k, n = 50, 10, 20000
    hits = np.zeros(r)
    for seed in range(n):
        hits[oracle.sample_positions(r, k, seed, 0, 0)] += 1
    assert hits.sum() == n * k
    p = k / r
    stat = float(((hits - n * p) ** 2 / (n * p * (1 - p))).sum())
    assert abs(stat - r) < 6 * math.sqrt(2 * r), stat


def test_sampler_subset_frequencies_small_case():
    r, k, n = 5, 2, 20000
    counts = Counter()
    for step in range(n):
        counts[tuple(oracle.sample_positions(r, k, 99, step, 1).tolist())] += 1
    obs = np.array([counts[c] for c in itertools.combinations(range(r), k)], dtype=float)
    ok, stat = _chi2_ok(obs, n / math.comb(r, k), math.comb(r, k) - 1)
    assert ok, stat


# ----------------------------------------------------------------------------- top-r
def _key(x: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(x, dtype=np.float32).view(np.uint32) & 0x7FFFFFFF


def brute_top_r(a, r):
    """Definition 1 with ties to the lower index, by a plain Python sort."""
    key = _key(a).tolist()
    order = sorted(range(len(key)), key=lambda i: (-key[i], i))
    return sorted(order[:r])


def test_top_r_brute_force_tiny_with_ties():
    values = np.array([0.0, -0.0, 0.5, -0.5, 1.0, -2.0], dtype=np.float32)
    for d in range(1, 6):
        for combo in itertools.product(range(len(values)), repeat=d):
            a = values[list(combo)]
            for r in range(1, d + 1):
                assert oracle.top_r(a, r).tolist() == brute_top_r(a, r)


def test_top_r_matches_library_sorts_on_tie_free_data():
    rng = np.random.default_rng(5)
    d = 20011
    mags = rng.permutation(d).astype(np.float32) * np.float32(0.125) + np.float32(1.0)
    a = (mags * rng.choice([-1.0, 1.0], d)).astype(np.float32)
    assert len(np.unique(np.abs(a))) == d
    order = np.argsort(-np.abs(a).astype(np.float64), kind="stable")
    for r in (1, 2, 100, d // 100, d - 1, d):
        got = oracle.top_r(a, r)
        assert got.tolist() == sorted(order[:r].tolist())
        tk = torch.topk(torch.from_numpy(np.abs(a)), r).indices.numpy()
        assert set(got.tolist()) == set(tk.tolist())


def test_top_r_adversarial_ties_and_specials():
    a = np.full(1000, -3.25, dtype=np.float32)
    assert oracle.top_r(a, 17).tolist() == list(range(17))
    # duplicated magnitudes across the threshold: the lower indices win
    a = np.array([1, -2, 2, 1, -2, 0, 2, 1], dtype=np.float32)
    assert oracle.top_r(a, 3).tolist() == [1, 2, 4]
    assert oracle.top_r(a, 5).tolist() == [0, 1, 2, 4, 6]
    # order by bit pattern with the sign cleared: NaN > Inf > finite > denormal > zero
    a = np.array([0.0, 1e-45, -np.inf, np.nan, 3e38, -1e-45, -0.0], dtype=np.float32)
    assert oracle.top_r(a, 1).tolist() == [3]
    assert oracle.top_r(a, 2).tolist() == [2, 3]
    assert oracle.top_r(a, 3).tolist() == [2, 3, 4]
    assert oracle.top_r(a, 4).tolist() == [1, 2, 3, 4]
    assert oracle.top_r(a, 6).tolist() == [0, 1, 2, 3, 4, 5]


# ----------------------------------------------------------------------------- node body
def _spiky(rng, W, d):
    x = rng.standard_normal((W, d)) * 1e-3
    m = rng.random((W, d)) < 0.05
    return np.where(m, rng.standard_normal((W, d)), x).astype(np.float32)


def _scatter(idx, val, d):
    out = np.zeros(d, dtype=np.float32)
    out[idx] = val
    return out


@pytest.mark.parametrize("d,r,k", [(1, 1, 1), (2, 2, 1), (5, 3, 2), (33, 7, 7), (1023, 100, 10),
                                   (4097, 4097, 41), (4098, 400, 1)])
def test_sparsify_identities_of_algorithm_1(d, r, k):
    rng = np.random.default_rng(d)
    W = 3
    g = _spiky(rng, W, d)
    m0 = _spiky(rng, W, d) * 0.5
    a = g + m0                                     # numpy float32 add: IEEE round-to-nearest
    m = m0.copy()
    idx, val = oracle.sparsify(g, m, d, r, k, seed=42, step=6, worker_base=10)
    for w in range(W):
        T = brute_top_r(a[w], r)
        pos = oracle.sample_positions(r, k, 42, 6, 10 + w, 0)
        want = [T[p] for p in pos]
        assert idx[w].tolist() == want                           # U = k-subset of the top-r set
        assert len(set(want)) == k and set(want) <= set(T)
        assert val[w].view(np.uint32).tolist() == a[w][want].view(np.uint32).tolist()
        assert (m[w][want].view(np.uint32) == 0).all()           # sent slots hold +0.0
        back = m[w].copy()
        back[want] = val[w]
        assert (back.view(np.uint32) == a[w].view(np.uint32)).all()   # sent + residual = a
        assert np.count_nonzero(_scatter(idx[w], val[w], d)) <= k


def test_limit_k_equals_r_is_top_r():
    rng = np.random.default_rng(8)
    d, r = 5000, 123
    g = np.stack([rng.permutation(d) + 1.0 for _ in range(2)]) * rng.choice([-1.0, 1.0], (2, d))
    g = (g * 0.25).astype(np.float32)               # distinct magnitudes: top-r is unique
    m = np.zeros_like(g)
    idx, val = oracle.sparsify(g, m, d, r, r, seed=1, step=0)
    for w in range(2):
        want = np.sort(np.argsort(-np.abs(g[w]), kind="stable")[:r])
        assert idx[w].tolist() == want.tolist()
        # top_r(a) itself: a - m' is a on the top-r set and 0 elsewhere
        assert np.array_equal(g[w] - m[w], _scatter(want, g[w][want], d))


def test_limit_r_equals_d_is_random_k():
    rng = np.random.default_rng(9)
    d, k = 3001, 30
    g1 = rng.standard_normal((2, d)).astype(np.float32)
    g2 = rng.standard_normal((2, d)).astype(np.float32)
    i1, v1 = oracle.sparsify(g1, np.zeros_like(g1), d, d, k, seed=5, step=2)
    i2, v2 = oracle.sparsify(g2, np.zeros_like(g2), d, d, k, seed=5, step=2)
    assert np.array_equal(i1, i2)                     # the subset does not look at the values
    for w in range(2):
        assert i1[w].tolist() == oracle.sample_positions(d, k, 5, 2, w).tolist()
        assert np.array_equal(v1[w], g1[w][i1[w]])


def test_proposition_1_closed_form_monte_carlo():
    # E||a - rTop_k(a)||^2 = (1 - k/r) sum_{j<=r} a_(j)^2 + sum_{j>r} a_(j)^2   (proof of Prop. 1),
    # E[rTop_k(a)] = (k/r) top_r(a), and every draw satisfies ||a - C(a)||^2 <= ||a||^2.
    rng = np.random.default_rng(10)
    d, r, k, n = 300, 40, 10, 6000
    a = (rng.standard_normal(d) * np.exp(rng.standard_normal(d))).astype(np.float32)
    sq = np.sort(a.astype(np.float64) ** 2)[::-1]
    closed = (1 - k / r) * sq[:r].sum() + sq[r:].sum()
    errs = np.zeros(n)
    mean_vec = np.zeros(d)
    g = np.repeat(a[None, :], 1, axis=0)
    for s in range(n):
        m = np.zeros((1, d), dtype=np.float32)
        idx, val = oracle.sparsify(g, m, d, r, k, seed=1000 + s, step=s % 7)
        errs[s] = (m[0].astype(np.float64) ** 2).sum()
        mean_vec[idx[0]] += val[0]
    assert (errs <= (a.astype(np.float64) ** 2).sum() + 1e-9).all()
    assert abs(errs.mean() - closed) < 4 * errs.std() / math.sqrt(n)
    assert abs(closed - (1 - k / d) * sq.sum()) >= 0 and closed <= (1 - k / d) * sq.sum() + 1e-9
    top = np.zeros(d)
    T = brute_top_r(a, r)
    top[T] = a[T]
    dev = mean_vec / n - (k / r) * top
    sigma = np.sqrt((k / r) * (1 - k / r) / n) * np.abs(top)
    assert (np.abs(dev) <= 5 * sigma + 1e-12).all()


def test_nan_sums_are_stored_as_the_default_quiet_nan():
    # IEEE 754 does not fix the payload of a NaN result; the contract does (0x7FC00000)
    g = np.zeros((1, 8), dtype=np.float32)
    g.view(np.uint32)[0, 2] = 0x7FFFFFFF
    g.view(np.uint32)[0, 5] = 0xFFC12345
    g[0, 6] = np.inf
    m = np.zeros((1, 8), dtype=np.float32)
    m[0, 6] = -np.inf                                  # inf - inf
    idx, val = oracle.sparsify(g, m, 8, 3, 3, seed=0, step=0)
    assert idx[0].tolist() == [2, 5, 6]                # equal keys: lower index first
    assert val.view(np.uint32)[0].tolist() == [0x7FC00000] * 3


def test_step_counter_and_resume():
    rng = np.random.default_rng(11)
    W, d, r, k = 2, 2000, 100, 20
    grads = [_spiky(rng, W, d) for _ in range(6)]
    m_all = np.zeros((W, d), dtype=np.float32)
    out_all = [oracle.sparsify(grads[t], m_all, d, r, k, seed=3, step=t) for t in range(6)]
    m_a = np.zeros((W, d), dtype=np.float32)
    for t in range(3):
        oracle.sparsify(grads[t], m_a, d, r, k, seed=3, step=t)
    m_b = m_a.copy()                                  # "checkpoint": the residual is the only state
    out_b = [oracle.sparsify(grads[t], m_b, d, r, k, seed=3, step=t) for t in range(3, 6)]
    assert np.array_equal(m_b.view(np.uint32), m_all.view(np.uint32))
    for (i1, v1), (i2, v2) in zip(out_all[3:], out_b):
        assert np.array_equal(i1, i2) and np.array_equal(v1.view(np.uint32), v2.view(np.uint32))


def test_bf16_gradient_is_widened_exactly():
    rng = np.random.default_rng(12)
    W, d, r, k = 2, 999, 50, 5
    gf = torch.from_numpy(_spiky(rng, W, d)).to(torch.bfloat16)
    bits = gf.view(torch.int16).numpy().view(np.uint16).copy()
    m0 = _spiky(rng, W, d)
    m1, m2 = m0.copy(), m0.copy()
    i1, v1 = oracle.sparsify(bits, m1, d, r, k, seed=1, step=1)
    i2, v2 = oracle.sparsify(gf.to(torch.float32).numpy().copy(), m2, d, r, k, seed=1, step=1)
    assert np.array_equal(i1, i2) and np.array_equal(v1.view(np.uint32), v2.view(np.uint32))
    assert np.array_equal(m1.view(np.uint32), m2.view(np.uint32))


def test_segmented_is_rtopk_per_slice():
    rng = np.random.default_rng(13)
    W, sizes = 2, [700, 301, 1024, 5]
    off = np.concatenate([[0], np.cumsum(sizes)])
    d = int(off[-1])
    seg_r = [70, 301, 10, 2]
    seg_k = [7, 30, 10, 1]
    g = _spiky(rng, W, d)
    m0 = _spiky(rng, W, d)
    m = m0.copy()
    idx, val = oracle.sparsify_segmented(g, m, d, off, seg_r, seg_k, seed=21, step=4, worker_base=3)
    a = g + m0
    for w in range(W):
        at = 0
        for s, (lo, n) in enumerate(zip(off[:-1], sizes)):
            T = brute_top_r(a[w, lo:lo + n], seg_r[s])
            pos = oracle.sample_positions(seg_r[s], seg_k[s], 21, 4, 3 + w, s)
            want = [int(lo) + T[p] for p in pos]
            assert idx[w, at:at + seg_k[s]].tolist() == want
            assert np.array_equal(val[w, at:at + seg_k[s]], a[w][want])
            at += seg_k[s]
        back = m[w].copy()
        back[idx[w]] = val[w]
        assert np.array_equal(back.view(np.uint32), a[w].view(np.uint32))
    # one segment covering the vector is the plain operator
    m1, m2 = m0.copy(), m0.copy()
    i1, v1 = oracle.sparsify_segmented(g, m1, d, [0, d], [90], [9], seed=2, step=0)
    i2, v2 = oracle.sparsify(g, m2, d, 90, 9, seed=2, step=0)
    assert np.array_equal(i1, i2) and np.array_equal(v1, v2) and np.array_equal(m1, m2)


# ----------------------------------------------------------------------------- master
def test_aggregate_worked_example():
    # two workers, d = 4: worker 0 sends (0: 1, 2: 2), worker 1 sends (2: 4, 3: 8)
    idx = np.array([[0, 2], [2, 3]], dtype=np.uint32)
    val = np.array([[1, 2], [4, 8]], dtype=np.float32)
    o64, o32 = oracle.aggregate(idx, val, 4)
    assert o64.tolist() == [0.5, 0.0, 3.0, 4.0] and o32.tolist() == [0.5, 0.0, 3.0, 4.0]
    s64, _ = oracle.aggregate(idx, val, 4, oracle.SCALE_SUM)
    assert s64.tolist() == [1.0, 0.0, 6.0, 8.0]


def test_aggregate_against_numpy_and_special_cases():
    rng = np.random.default_rng(14)
    d, W, k = 5000, 5, 400
    idx = np.stack([np.sort(rng.choice(d, k, replace=False)) for _ in range(W)]).astype(np.uint32)
    val = (rng.standard_normal((W, k)) * np.exp(3 * rng.standard_normal((W, k)))).astype(np.float32)
    o64, o32 = oracle.aggregate(idx, val, d)
    ref = np.zeros(d)
    np.add.at(ref, idx.ravel().astype(np.int64), val.ravel().astype(np.float64))
    # the sum of five doubles depends on order only in the last bits
    assert np.allclose(o64, ref / W, rtol=1e-14, atol=0)
    assert np.array_equal(o32, o64.astype(np.float32))
    # W = 1: the update is the message itself
    o64, o32 = oracle.aggregate(idx[:1], val[:1], d)
    assert np.array_equal(o32, _scatter(idx[0], val[0], d))
    # disjoint supports: exact
    idx_d = np.arange(W * k, dtype=np.uint32).reshape(W, k)
    o64, _ = oracle.aggregate(idx_d, val, d)
    assert np.array_equal(o64[: W * k], val.ravel().astype(np.float64) / W)


def test_master_update_worked_example_and_textbook_sgd():
    # Algorithm 1, master update w <- w - eta * ghat.  d = 4, two workers as in the average's worked
    # example: ghat = [0.5, 0, 3, 4]; with eta = 0.5 and w = [1, 1, 1, 1] the update is exact.
    idx = np.array([[0, 2], [2, 3]], dtype=np.uint32)
    val = np.array([[1, 2], [4, 8]], dtype=np.float32)
    w = oracle.apply_update(idx, val, 4, 0.5, np.ones(4, dtype=np.float32))
    assert w.tolist() == [0.75, 1.0, -0.5, -1.0]
    # one worker, sum scaling: plain SGD on the sent coordinates, every other weight bit-unchanged
    rng = np.random.default_rng(21)
    d, k, eta = 3000, 200, np.float32(0.0371)
    idx = np.sort(rng.choice(d, k, replace=False)).astype(np.uint32)[None, :]
    val = (rng.standard_normal((1, k)) * np.exp(2 * rng.standard_normal((1, k)))).astype(np.float32)
    w0 = rng.standard_normal(d).astype(np.float32)
    w0[idx[0, 0]] = -0.0
    w0[(idx[0, 0] + 1) % d if (idx[0, 0] + 1) % d not in idx[0] else idx[0, 0]] = -0.0
    w1 = oracle.apply_update(idx, val, d, float(eta), w0, oracle.SCALE_SUM)
    ref = w0.astype(np.float64)
    ref[idx[0].astype(np.int64)] -= np.float64(eta) * val[0].astype(np.float64)
    assert np.array_equal(w1.view(np.uint32), ref.astype(np.float32).view(np.uint32))
    untouched = np.ones(d, dtype=bool)
    untouched[idx[0].astype(np.int64)] = False
    assert np.array_equal(w1.view(np.uint32)[untouched], w0.view(np.uint32)[untouched])
    # eta = 0 changes no value (a sent -0.0 weight may become +0.0: -0 - (0 * negative) = -0 + 0), and
    # no bit at unsent coordinates; the update agrees with the (separately pinned) average applied densely
    z = oracle.apply_update(idx, val, d, 0.0, w0)
    assert np.array_equal(z, w0) and np.array_equal(z.view(np.uint32)[untouched], w0.view(np.uint32)[untouched])
    W = 4
    idx4 = np.stack([np.sort(rng.choice(d, k, replace=False)) for _ in range(W)]).astype(np.uint32)
    val4 = rng.standard_normal((W, k)).astype(np.float32)
    _, g32 = oracle.aggregate(idx4, val4, d)
    dense = (w0.astype(np.float64) - np.float64(eta) * g32.astype(np.float64)).astype(np.float32)
    assert np.array_equal(oracle.apply_update(idx4, val4, d, float(eta), w0).view(np.uint32), dense.view(np.uint32))
    with pytest.raises(ValueError):
        oracle.apply_update(idx4, val4, d, -1.0, w0)


def test_momentum_update_worked_example_limits_and_library_optimizer():
    # Section IV trains with momentum SGD; reading: heavy ball on the master, v <- mu v + ghat, w <- w - eta v.
    # Worked example with exact binary fractions: ghat = [0.5, 0, 3, 4] (the average's worked example),
    # v0 = [1, 2, 0, -8], mu = 0.5, eta = 0.25, w0 = 1:  v1 = [1, 1, 3, 0],  w1 = [0.75, 0.75, 0.25, 1].
    idx = np.array([[0, 2], [2, 3]], dtype=np.uint32)
    val = np.array([[1, 2], [4, 8]], dtype=np.float32)
    v1, w1 = oracle.apply_momentum(idx, val, 4, 0.25, 0.5, np.array([1, 2, 0, -8], dtype=np.float32), np.ones(4, dtype=np.float32))
    assert v1.tolist() == [1.0, 1.0, 3.0, 0.0] and w1.tolist() == [0.75, 0.75, 0.25, 1.0]
    # a second step with the same messages: v2 = 0.5 v1 + ghat = [1, 0.5, 4.5, 4], w2 = w1 - 0.25 v2
    v2, w2 = oracle.apply_momentum(idx, val, 4, 0.25, 0.5, v1, w1)
    assert v2.tolist() == [1.0, 0.5, 4.5, 4.0] and w2.tolist() == [0.5, 0.625, -0.875, 0.0]
    rng = np.random.default_rng(41)
    d, k, W, eta, mu = 4000, 300, 3, 0.05, 0.9
    w0 = rng.standard_normal(d).astype(np.float32)
    msgs = []
    for _ in range(6):
        i = np.stack([np.sort(rng.choice(d, k, replace=False)) for _ in range(W)]).astype(np.uint32)
        msgs.append((i, rng.standard_normal((W, k)).astype(np.float32)))
    # mu = 0 is the (separately pinned) master update, bit for bit, and v is then the average itself
    v, w = oracle.apply_momentum(msgs[0][0], msgs[0][1], d, eta, 0.0, rng.standard_normal(d).astype(np.float32), w0)
    assert np.array_equal(w.view(np.uint32), oracle.apply_update(msgs[0][0], msgs[0][1], d, eta, w0).view(np.uint32))
    assert np.array_equal(v, oracle.aggregate(msgs[0][0], msgs[0][1], d)[1])
    # against the library optimizer (torch.optim.SGD with momentum, dampening 0, no Nesterov) run in float64 on
    # the same averages: the oracle rounds to binary32 twice per step and coordinate, so the two stay within a
    # few binary32 roundings of each other over six steps
    p = torch.nn.Parameter(torch.from_numpy(w0.astype(np.float64)))
    opt = torch.optim.SGD([p], lr=eta, momentum=mu)
    v, w = np.zeros(d, dtype=np.float32), w0.copy()
    for i, x in msgs:
        v, w = oracle.apply_momentum(i, x, d, eta, mu, v, w)
        p.grad = torch.from_numpy(oracle.aggregate(i, x, d)[1].astype(np.float64))
        opt.step()
    ref = p.detach().numpy()
    assert np.max(np.abs(w.astype(np.float64) - ref)) <= 6 * 2.0**-23 * max(1.0, float(np.max(np.abs(ref))))
    # a constant average g: v_n = g (1 - mu^n) / (1 - mu), the geometric series
    gi = np.arange(0, d, 7, dtype=np.uint32)[None, :]
    gv = rng.standard_normal((1, gi.shape[1])).astype(np.float32)
    v, w = np.zeros(d, dtype=np.float32), w0.copy()
    n = 12
    for _ in range(n):
        v, w = oracle.apply_momentum(gi, gv, d, eta, mu, v, w)
    g = np.zeros(d); g[gi[0].astype(np.int64)] = gv[0].astype(np.float64)
    assert np.allclose(v, g * (1 - mu**n) / (1 - mu), rtol=1e-5, atol=1e-7)
    # unsent coordinates: v decays by mu per step there and the weight keeps moving along it
    quiet = np.ones(d, dtype=bool); quiet[gi[0].astype(np.int64)] = False
    v0 = rng.standard_normal(d).astype(np.float32)
    v1, w1 = oracle.apply_momentum(gi, gv, d, eta, mu, v0, w0)
    assert np.array_equal(v1[quiet], (np.float64(np.float32(mu)) * v0[quiet].astype(np.float64)).astype(np.float32))
    assert np.array_equal(w1[quiet], (w0[quiet].astype(np.float64) - np.float64(np.float32(eta)) * v1[quiet].astype(np.float64)).astype(np.float32))
    for bad in [dict(eta=-1.0, mu=0.5), dict(eta=0.1, mu=1.0), dict(eta=0.1, mu=-0.1), dict(eta=0.1, mu=float("nan"))]:
        with pytest.raises(ValueError):
            oracle.apply_momentum(gi, gv, d, bad["eta"], bad["mu"], v0, w0)


def test_aggregate_scalings_unbiased_and_by_count():
    # the worked example again: S = [1, 0, 6, 8], senders c = [1, 0, 2, 1], W = 2, k = 2
    idx = np.array([[0, 2], [2, 3]], dtype=np.uint32)
    val = np.array([[1, 2], [4, 8]], dtype=np.float32)
    u64, _ = oracle.aggregate(idx, val, 4, oracle.SCALE_UNBIASED, r=3)       # S * 3 / 4
    assert u64.tolist() == [0.75, 0.0, 4.5, 6.0]
    c64, _ = oracle.aggregate(idx, val, 4, oracle.SCALE_COUNT)               # S / c
    assert c64.tolist() == [1.0, 0.0, 3.0, 8.0]
    # k = r: the unbiased scaling is the mean; disjoint supports: by-count is the sum; identical
    # supports: by-count is the mean
    rng = np.random.default_rng(8)
    d, W, k = 4000, 6, 300
    idx = np.stack([np.sort(rng.choice(d, k, replace=False)) for _ in range(W)]).astype(np.uint32)
    val = rng.standard_normal((W, k)).astype(np.float32)
    m64, _ = oracle.aggregate(idx, val, d)
    u64, _ = oracle.aggregate(idx, val, d, oracle.SCALE_UNBIASED, r=k)
    assert np.allclose(u64, m64, rtol=1e-15, atol=0)
    u64, _ = oracle.aggregate(idx, val, d, oracle.SCALE_UNBIASED, r=4 * k)   # r / k = 4: exact scaling
    assert np.array_equal(u64, 4.0 * m64) or np.allclose(u64, 4.0 * m64, rtol=1e-15, atol=0)
    idx_d = np.arange(W * k, dtype=np.uint32).reshape(W, k)
    c64, _ = oracle.aggregate(idx_d, val, d, oracle.SCALE_COUNT)
    s64, _ = oracle.aggregate(idx_d, val, d, oracle.SCALE_SUM)
    assert np.array_equal(c64, s64)
    same = np.stack([idx[0]] * W)
    c64, _ = oracle.aggregate(same, val, d, oracle.SCALE_COUNT)
    m64, _ = oracle.aggregate(same, val, d)
    assert np.array_equal(c64, m64)
    # by-count against numpy: sums and sender counts by np.add.at
    ref, cnt = np.zeros(d), np.zeros(d)
    np.add.at(ref, idx.ravel().astype(np.int64), val.ravel().astype(np.float64))
    np.add.at(cnt, idx.ravel().astype(np.int64), 1.0)
    c64, c32 = oracle.aggregate(idx, val, d, oracle.SCALE_COUNT)
    want = np.divide(ref, cnt, out=np.zeros(d), where=cnt > 0)
    assert np.allclose(c64, want, rtol=1e-14, atol=0) and np.array_equal(c32, c64.astype(np.float32))
    # unbiasedness (Definition 3 + the estimator's 1/S): averaged over many subsets of a fixed top-r
    # list, (r/k) * message converges to the list itself
    r, k2, trials = 12, 3, 6000
    vals = np.arange(1, r + 1, dtype=np.float64)
    acc = np.zeros(r)
    for t in range(trials):
        pos = oracle.sample_positions(r, k2, seed=99, worker=0, segment=0, step=t)
        acc[pos] += vals[pos] * r / k2
    assert np.allclose(acc / trials, vals, rtol=0.08)
    with pytest.raises(ValueError):
        oracle.aggregate(idx, val, d, oracle.SCALE_UNBIASED, r=k - 1)


def test_bad_arguments_are_rejected():
    g = np.zeros((1, 8), dtype=np.float32)
    m = np.zeros((1, 8), dtype=np.float32)
    for d, r, k in [(8, 4, 5), (8, 9, 1), (8, 4, 0), (9, 4, 1)]:
        with pytest.raises(ValueError):
            oracle.sparsify(g, m, d, r, k, seed=0, step=0)


# ----------------------------------------------------------------------------- message codec
def test_codec_index_bits_and_hand_packed_words():
    # Section III: an index costs log d bits.  b = ceil(log2 d), at least 1.
    for d, b in [(1, 1), (2, 1), (3, 2), (4, 2), (5, 3), (1000, 10), (1024, 10), (1025, 11), (2**31, 31), (2**32 - 1, 32)]:
        assert oracle.index_bits(d) == b
    # d = 1000 (b = 10), indices 1, 2, 1023 -> not allowed (>= d); use 999: the bit stream is the
    # little-endian integer sum idx_j << (10 j): written out by hand for three entries
    idx = np.array([[1, 2, 999, 512]], dtype=np.uint32)
    val = np.array([[1.0, -2.0, 0.5, 3.0]], dtype=np.float32)
    pi, pv = oracle.encode(idx, val, 1000)
    stream = 1 | (2 << 10) | (999 << 20) | (512 << 30)             # 40 bits
    assert pi.shape == (1, 2) and int(pi[0, 0]) == stream & 0xFFFFFFFF and int(pi[0, 1]) == stream >> 32
    assert pv[0].tolist() == [0x3F80, 0xC000, 0x3F00, 0x4040]


def test_codec_bit_stream_against_big_integers_and_round_trip():
    rng = np.random.default_rng(31)
    for d, k in [(2, 5), (37, 64), (1000, 333), (1 << 20, 1000), ((1 << 24) + 1, 257), (2**32 - 1, 50)]:
        b = oracle.index_bits(d)
        idx = np.sort(rng.choice(min(d, 1 << 40), size=min(k, d), replace=False) if d <= (1 << 26)
                      else np.unique(rng.integers(0, d, size=4 * k))[:k]).astype(np.uint32)[None, :]
        kk = idx.shape[1]
        val = rng.standard_normal((1, kk)).astype(np.float32)
        pi, pv = oracle.encode(idx, val, d)
        big = 0
        for j, v in enumerate(idx[0].tolist()):
            big |= v << (j * b)
        words = [(big >> (32 * w)) & 0xFFFFFFFF for w in range(pi.shape[1])]
        assert pi[0].tolist() == words and pi.shape[1] == (kk * b + 31) // 32
        i2, v2 = oracle.decode(pi, pv, d, kk)
        assert np.array_equal(i2, idx)
        assert np.array_equal(v2.view(np.uint32), pv.astype(np.uint32) << 16)


def test_codec_bfloat16_rounding_against_torch_and_rules():
    import torch
    rng = np.random.default_rng(32)
    x = np.concatenate([
        (rng.standard_normal(20000) * np.exp(8 * rng.standard_normal(20000))).astype(np.float32),
        rng.integers(0, 2**32, size=20000, dtype=np.uint64).astype(np.uint32).view(np.float32),
        np.array([0.0, -0.0, 1.0, np.inf, -np.inf, 3.3895314e38, 3.4028235e38, 1e-45, 1.17549435e-38], dtype=np.float32),
        np.array([0x3F808000, 0x3F818000, 0x3F807FFF, 0x3F808001, 0x7F7F8000], dtype=np.uint32).view(np.float32),
    ])
    x = x[~np.isnan(x)]
    ours = np.array([oracle.bf16_rne(float(v)) for v in x], dtype=np.uint16)
    theirs = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(ours, theirs)
    # the rules spelled out: exact halves go to the even neighbour, NaN is the default quiet NaN
    assert oracle.bf16_rne(float(np.array([0x3F808000], dtype=np.uint32).view(np.float32)[0])) == 0x3F80   # tie -> even (down)
    assert oracle.bf16_rne(float(np.array([0x3F818000], dtype=np.uint32).view(np.float32)[0])) == 0x3F82   # tie -> even (up)
    assert oracle.bf16_rne(float("nan")) == 0x7FC0
    assert oracle.bf16_rne(3.4028235e38) == 0x7F80                                                    # rounds to +inf


def test_codec_rounding_error_goes_to_the_residual():
    # Algorithm 1: m = a - ghat, with ghat the value that is sent.  The decoded value plus the
    # residual slot gives back a exactly (the rounding error of bfloat16 is a binary32 number).
    rng = np.random.default_rng(33)
    d, k = 5000, 400
    idx = np.sort(rng.choice(d, k, replace=False)).astype(np.uint32)[None, :]
    val = (rng.standard_normal((1, k)) * np.exp(3 * rng.standard_normal((1, k)))).astype(np.float32)
    val[0, 0] = 3.4e38          # rounds to +inf: no finite error to keep
    val[0, 1] = 1.0             # exact in bfloat16: the slot stays +0.0
    m = rng.standard_normal((1, d)).astype(np.float32)
    m[0, idx[0].astype(np.int64)] = 0.0
    m0 = m.copy()
    pi, pv = oracle.encode(idx, val, d, residual=m)
    _, back = oracle.decode(pi, pv, d, k)
    sent = idx[0].astype(np.int64)
    ok = np.isfinite(back[0])
    assert np.array_equal((back[0][ok].astype(np.float64) + m[0, sent][ok].astype(np.float64)), val[0][ok].astype(np.float64))
    assert m[0, sent[0]] == 0.0 and m[0, sent[1]] == 0.0 and not np.signbit(m[0, sent[1]])
    untouched = np.ones(d, dtype=bool); untouched[sent] = False
    assert np.array_equal(m[0, untouched].view(np.uint32), m0[0, untouched].view(np.uint32))
    assert np.all(np.abs(m[0, sent][ok]) <= np.abs(val[0][ok]) * 2.0**-8)


def test_tiled_codec_hand_example():
    # Spans of 16384 coordinates; d = 40000 has T = 3 of them: [0, 16384), [16384, 32768), [32768, 40000).
    # Row 3, 16383 | 16384, 16390 | 39999: two entries below 16384, four below 32768, five in all.
    idx = np.array([[3, 16383, 16384, 16390, 39999]], dtype=np.uint32)
    val = np.array([[1.0, -2.0, 0.5, 3.0, -0.15625]], dtype=np.float32)
    assert oracle.tiled_spans(40000) == 3 and oracle.tiled_spans(16384) == 1 and oracle.tiled_spans(16385) == 2
    tab, low, qv = oracle.encode_tiled(idx, val, 40000)
    assert tab.tolist() == [[0, 2, 4, 5]]
    assert low.tolist() == [[3, 16383, 0, 6, 39999 - 32768]]
    assert qv.tolist() == [[0x3F80, 0xC000, 0x3F00, 0x4040, 0xBE20]]
    i2, v2 = oracle.decode_tiled(tab, low, qv, 40000, 5)
    assert np.array_equal(i2, idx) and np.array_equal(v2, val)
    # a row that skips spans: the table repeats itself over the empty ones
    tab, low, _ = oracle.encode_tiled(np.array([[5, 70000]], dtype=np.uint32), np.ones((1, 2), dtype=np.float32), 100000)
    assert tab.tolist() == [[0, 1, 1, 1, 1, 2, 2, 2]] and low.tolist() == [[5, 70000 - 4 * 16384]]
    for bad in [np.array([[5, 5]]), np.array([[9, 3]]), np.array([[1, 100000]])]:       # not ascending / out of range
        with pytest.raises(ValueError):
            oracle.encode_tiled(bad.astype(np.uint32), np.ones((1, 2), dtype=np.float32), 100000)


def test_tiled_codec_against_library_search_round_trip_and_size():
    rng = np.random.default_rng(51)
    for d, k in [(1, 1), (16384, 16384), (16385, 9), (100003, 1000), (1 << 20, 5000), ((1 << 22) + 17, 300)]:
        idx = np.sort(rng.choice(d, size=k, replace=False)).astype(np.uint32)[None, :]
        val = (rng.standard_normal((1, k)) * np.exp(3 * rng.standard_normal((1, k)))).astype(np.float32)
        tab, low, qv = oracle.encode_tiled(idx, val, d)
        T = (d + 16383) // 16384
        # the table is a lower-bound search of the span boundaries in the sorted row (library routine)
        assert tab.shape == (1, T + 1)
        assert np.array_equal(tab[0], np.searchsorted(idx[0], np.arange(T + 1, dtype=np.int64) * 16384, side="left"))
        assert np.array_equal(low[0], idx[0] & 16383) and int(low.max()) < 16384
        # values: the bfloat16 rounding pinned above, here against torch once more
        assert np.array_equal(qv[0], torch.from_numpy(val[0]).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16))
        i2, v2 = oracle.decode_tiled(tab, low, qv, d, k)
        assert np.array_equal(i2, idx)
        assert np.array_equal(v2.view(np.uint32), qv.astype(np.uint32) << 16)
        # both codecs carry the same message
        pi, pv = oracle.encode(idx, val, d)
        i3, v3 = oracle.decode(pi, pv, d, k)
        assert np.array_equal(i3, i2) and np.array_equal(v3.view(np.uint32), v2.view(np.uint32))
    # size at the paper's scale (ResNet-18, 0.1 % of 11.17 M coordinates): 32 (T + 1) + 32 k bits against
    # (24 + 16) k for the bit-packed indices and 64 k for plain pairs
    d, k = 11173962, 11173
    T = oracle.tiled_spans(d)
    assert T == 683 and 32 * (T + 1) + 32 * k < (oracle.index_bits(d) + 16) * k < 64 * k


def test_tiled_codec_rounding_error_goes_to_the_residual():
    # the same error feedback as the bit-packed format: decoded value + residual slot = a exactly
    rng = np.random.default_rng(52)
    d, k = 50000, 700
    idx = np.sort(rng.choice(d, k, replace=False)).astype(np.uint32)[None, :]
    val = (rng.standard_normal((1, k)) * np.exp(3 * rng.standard_normal((1, k)))).astype(np.float32)
    val[0, 0] = 3.4e38
    val[0, 1] = 1.0
    m = rng.standard_normal((1, d)).astype(np.float32)
    m[0, idx[0].astype(np.int64)] = 0.0
    m0, m_packed = m.copy(), m.copy()
    tab, low, qv = oracle.encode_tiled(idx, val, d, residual=m)
    oracle.encode(idx, val, d, residual=m_packed)
    assert np.array_equal(m.view(np.uint32), m_packed.view(np.uint32))
    _, back = oracle.decode_tiled(tab, low, qv, d, k)
    sent = idx[0].astype(np.int64)
    ok = np.isfinite(back[0])
    assert np.array_equal(back[0][ok].astype(np.float64) + m[0, sent][ok].astype(np.float64), val[0][ok].astype(np.float64))
    assert m[0, sent[0]] == 0.0 and m[0, sent[1]] == 0.0 and not np.signbit(m[0, sent[1]])
    untouched = np.ones(d, dtype=bool); untouched[sent] = False
    assert np.array_equal(m[0, untouched].view(np.uint32), m0[0, untouched].view(np.uint32))


# ----------------------------------------------------------------------------- warm-up schedule
def test_warmup_schedule_geometric_sequence_and_limits():
    # Section IV: sparsity grows exponentially over the warm-up, k / r = 1 / n.  With density going
    # from 1/4 to 1/1024 in 4 steps every step divides the density by 4 (exact powers of two).
    d, n = 1 << 20, 8
    ks = [oracle.warmup_sizes(d, n, 0.25, 1.0 / 1024, 4, t)[1] for t in range(7)]
    assert ks == [d // 4, d // 16, d // 64, d // 256, d // 1024, d // 1024, d // 1024]
    for t in range(7):
        r, k = oracle.warmup_sizes(d, n, 0.25, 1.0 / 1024, 4, t)
        assert r == min(d, n * k) and 1 <= k <= r <= d
    # monotone, ends at floor(final d), never below one coordinate, r capped at d
    seq = [oracle.warmup_sizes(11_173_962, 5, 0.3, 0.001, 50, t) for t in range(60)]
    assert all(a[1] >= b[1] for a, b in zip(seq, seq[1:])) and seq[50][1] == 11_173
    assert seq[0] == (11_173_962, int(0.3 * 11_173_962))
    assert oracle.warmup_sizes(100, 4, 0.001, 0.001, 0, 3) == (4, 1)
    # against numpy's power on a grid (floor may differ by one where density * d is an integer)
    for t in range(0, 50, 7):
        want = int(np.floor(0.3 * np.power(0.001 / 0.3, t / 50) * 11_173_962))
        assert abs(seq[t][1] - want) <= 1
    with pytest.raises(ValueError):
        oracle.warmup_sizes(100, 4, 0.001, 0.01, 5, 0)
