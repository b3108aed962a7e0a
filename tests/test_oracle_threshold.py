"""Pins for the oracle's threshold-then-subsample encoder (the scheme in the proof of Theorem 1).

What the paper fixes and the tests check without a GPU: the marked set is what a library comparison
of magnitudes gives; at most k' marked coordinates are kept, all of them when there are no more than
k'; the kept set is a uniformly random k'-subset (every subset equally often over all draw tuples);
the estimator (1/n) sum X~_i / S_i is unbiased (its mean over all equally likely subsets is the
thresholded vector, in exact rational arithmetic); for 0/1 data each worker's scaled message sums to
||X_i||_1 (the identity used for the error bound); and Algorithm 1's m' = a - ghat.
"""
import itertools
import math
from collections import Counter
from fractions import Fraction

import numpy as np
import pytest

import oracle

PAD = 0xFFFFFFFF


def _spiky(rng, W, d, frac=0.1):
    x = rng.standard_normal((W, d)) * 1e-3
    m = rng.random((W, d)) < frac
    return np.where(m, rng.standard_normal((W, d)), x).astype(np.float32)


@pytest.mark.parametrize("d,k,theta", [(1, 1, 0.5), (7, 3, 0.0), (64, 5, 0.3), (1000, 40, 0.2), (1000, 400, 0.2),
                                       (4099, 64, 1e-3)])
def test_marked_set_counts_messages_and_residual(d, k, theta):
    rng = np.random.default_rng(d + k)
    W = 4
    g = _spiky(rng, W, d)
    m0 = (_spiky(rng, W, d) * 0.5).astype(np.float32)
    a = g + m0
    m = m0.copy()
    idx, val, count, ones = oracle.sparsify_threshold(g, m, d, theta, k, seed=5, step=3, worker_base=7)
    for w in range(W):
        marked = np.flatnonzero(np.abs(a[w]) > np.float32(theta))          # library comparison of magnitudes
        assert ones[w] == marked.size
        assert count[w] == min(marked.size, k)
        n = int(count[w])
        sent = idx[w, :n].astype(np.int64)
        assert (idx[w, n:] == PAD).all() and (val[w, n:].view(np.uint32) == 0).all()
        assert list(sent) == sorted(set(sent.tolist())) and set(sent.tolist()) <= set(marked.tolist())
        if marked.size <= k:
            assert sent.tolist() == marked.tolist()                            # nothing is dropped
        else:
            pos = oracle.sample_positions(marked.size, k, 5, 3, 7 + w, 0)      # the pinned k-of-n subset
            assert sent.tolist() == marked[pos].tolist()
        assert val[w, :n].view(np.uint32).tolist() == a[w][sent].view(np.uint32).tolist()
        back = m[w].copy()
        assert (back[sent].view(np.uint32) == 0).all()
        back[sent] = val[w, :n]
        assert (back.view(np.uint32) == a[w].view(np.uint32)).all()           # sent + residual = a


def test_threshold_comparison_is_strict_and_by_magnitude():
    a = np.array([[0.5, -0.5, 0.50000006, -0.75, 0.0, -0.0, np.inf, -np.inf, 0.25]], dtype=np.float32)
    m = np.zeros_like(a)
    idx, val, count, ones = oracle.sparsify_threshold(a, m, a.shape[1], 0.5, 9, seed=1, step=0)
    assert idx[0, :4].tolist() == [2, 3, 6, 7] and ones[0] == 4 and count[0] == 4
    # theta = 0: every non-zero magnitude is marked, zeros of either sign are not
    m[:] = 0
    idx, val, count, ones = oracle.sparsify_threshold(a, m, a.shape[1], 0.0, 9, seed=1, step=0)
    assert idx[0, :7].tolist() == [0, 1, 2, 3, 6, 7, 8] and ones[0] == 7
    # nothing marked: an empty message, the residual keeps everything
    m[:] = 0
    b = np.full((1, 5), 0.1, dtype=np.float32)
    mb = np.zeros_like(b)
    idx, val, count, ones = oracle.sparsify_threshold(b, mb, 5, 0.2, 2, seed=1, step=0)
    assert ones[0] == 0 and count[0] == 0 and (idx == PAD).all() and (mb == b).all()
    for bad in (-1.0, float("nan"), float("inf")):
        with pytest.raises(ValueError):
            oracle.sparsify_threshold(b, mb, 5, bad, 2, seed=1, step=0)


def test_kept_subset_is_uniform_and_estimator_unbiased_exhaustively():
    # One worker, n marked coordinates, k' kept.  Over all admissible draw tuples (equally likely) every
    # k'-subset appears equally often, and the mean of X~ / S is exactly X (here: the marked values).
    for n, k in [(4, 2), (5, 3), (6, 1), (6, 5)]:
        values = [Fraction(3 * j + 1, 7) * (-1) ** j for j in range(n)]
        ranges = [range(j + 1) for j in range(n - k, n)]
        counts, mean = Counter(), [Fraction(0)] * n
        total = 0
        for t in itertools.product(*ranges):
            pos = oracle.floyd_from_draws(n, k, np.array(t, dtype=np.uint32)).tolist()
            counts[tuple(pos)] += 1
            inv_S = Fraction(n, k)                        # S = k' / ||X||_1
            for p in pos:
                mean[p] += values[p] * inv_S
            total += 1
        assert len(counts) == math.comb(n, k) and len(set(counts.values())) == 1
        assert [x / total for x in mean] == values


def test_estimator_scaling_and_average():
    # Worker 0 marks 6 coordinates and keeps 2 (S = 1/3), worker 1 marks 2 and keeps both (S = 1).
    d, k = 8, 2
    g = np.array([[1, -2, 3, 0, 4, -5, 6, 0], [0, 0, 0, 7, 0, 0, 0, -8]], dtype=np.float32)
    m = np.zeros_like(g)
    idx, val, count, ones = oracle.sparsify_threshold(g, m, d, 0.5, k, seed=2, step=1)
    assert ones.tolist() == [6, 2] and count.tolist() == [2, 2]
    o64, o32 = oracle.aggregate_threshold(idx, val, count, ones, d)
    want = np.zeros(d)
    for j in range(2):
        want[idx[0, j]] += float(val[0, j]) * 3.0
        want[idx[1, j]] += float(val[1, j]) * 1.0
    want /= 2
    assert np.array_equal(o64, want) and np.array_equal(o32, want.astype(np.float32))
    # a worker that marked nothing contributes nothing but still counts in 1/n
    idx2 = np.vstack([idx, np.full((1, k), PAD, dtype=np.uint32)])
    val2 = np.vstack([val, np.zeros((1, k), dtype=np.float32)])
    o64b, _ = oracle.aggregate_threshold(idx2, val2, np.append(count, 0), np.append(ones, 0), d)
    assert np.allclose(o64b * 3, o64 * 2, rtol=0, atol=1e-15)
    with pytest.raises(ValueError):                                       # more sent than marked
        oracle.aggregate_threshold(idx, val, count, np.array([1, 2], dtype=np.uint32), d)


def test_bernoulli_observations_scaled_message_sums_to_the_number_of_ones():
    # The sparse Bernoulli model itself: X in {0,1}^d.  Each worker's X~ / S sums to ||X||_1 (k' * ||X||_1 / k'
    # when subsampled), and with all n workers holding the same X the estimate sums to ||X||_1 too.
    rng = np.random.default_rng(11)
    d, W, k = 500, 5, 12
    X = (rng.random((W, d)) < 0.08).astype(np.float32)
    m = np.zeros_like(X)
    idx, val, count, ones = oracle.sparsify_threshold(X, m, d, 0.5, k, seed=9, step=0)
    assert ones.tolist() == X.sum(axis=1).astype(int).tolist()
    o64, _ = oracle.aggregate_threshold(idx, val, count, ones, d)
    assert abs(o64.sum() * W - float(ones.sum())) < 1e-9
    assert (m + 0 == X - np.stack([np.bincount(idx[w, :count[w]], minlength=d) for w in range(W)])).all()


def test_estimator_mean_over_seeds_approaches_the_thresholded_vector():
    rng = np.random.default_rng(3)
    d, W, k, theta, n = 60, 3, 4, 0.5, 4000
    g = _spiky(rng, W, d, frac=0.3)
    target = np.where(np.abs(g) > theta, g, 0).astype(np.float64).mean(axis=0)
    acc = np.zeros(d)
    sq = np.zeros(d)
    for seed in range(n):
        m = np.zeros_like(g)
        idx, val, count, ones = oracle.sparsify_threshold(g, m, d, theta, k, seed=seed, step=0)
        o64, _ = oracle.aggregate_threshold(idx, val, count, ones, d)
        acc += o64
        sq += o64 * o64
    mean = acc / n
    sd = np.sqrt(np.maximum(sq / n - mean * mean, 0) / n)
    assert (np.abs(mean - target) <= 5 * sd + 1e-12).all()
    assert (ones > k).all()                                               # the case really subsamples


def test_sign_mode_sends_plus_minus_two_theta_and_keeps_the_difference():
    rng = np.random.default_rng(21)
    d, W, k, theta = 3000, 3, 50, 0.25
    g = _spiky(rng, W, d, frac=0.05)
    m0 = (_spiky(rng, W, d, frac=0.05) * 0.5).astype(np.float32)
    a = g + m0
    m_v, m_s = m0.copy(), m0.copy()
    idx_v, val_v, cnt_v, ones_v = oracle.sparsify_threshold(g, m_v, d, theta, k, seed=4, step=2)
    idx_s, val_s, cnt_s, ones_s = oracle.sparsify_threshold(g, m_s, d, theta, k, seed=4, step=2, signs=True)
    assert np.array_equal(idx_v, idx_s) and np.array_equal(cnt_v, cnt_s) and np.array_equal(ones_v, ones_s)
    M = np.float32(2 * theta)
    for w in range(W):
        n = int(cnt_s[w])
        sent = idx_s[w, :n].astype(np.int64)
        assert np.array_equal(val_s[w, :n], np.copysign(M, a[w][sent]))          # library copysign
        want = a[w].copy()
        want[sent] = a[w][sent] - np.copysign(M, a[w][sent])                      # numpy binary32 subtraction
        assert np.array_equal(m_s[w].view(np.uint32), want.view(np.uint32))
    with pytest.raises(ValueError):
        oracle.sparsify_threshold(g, m0.copy(), d, 3e38, k, seed=4, step=2, signs=True)   # 2 theta overflows


def test_sign_mode_on_the_scaled_signed_bernoulli_model_is_lossless_at_kept_coordinates():
    # X in {0, +-M}^d, threshold M / 2: a kept coordinate is reproduced exactly and leaves nothing behind,
    # and the estimate of n identical workers that keep everything is X itself.
    rng = np.random.default_rng(8)
    d, W, M = 400, 4, np.float32(0.75)
    X = (np.where(rng.random(d) < 0.05, 1.0, 0.0) * np.where(rng.random(d) < 0.5, -1.0, 1.0)).astype(np.float32) * M
    g = np.tile(X, (W, 1))
    m = np.zeros_like(g)
    n_ones = int(np.count_nonzero(X))
    idx, val, cnt, ones = oracle.sparsify_threshold(g, m, d, float(M) / 2, n_ones, seed=1, step=0, signs=True)
    assert (ones == n_ones).all() and (cnt == n_ones).all() and not m.any()
    o64, o32 = oracle.aggregate_threshold(idx, val, cnt, ones, d)
    assert np.array_equal(o32, X)
