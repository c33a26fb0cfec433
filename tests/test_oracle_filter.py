"""Pins of the oracle's token filter (Sec. 3.3): kept count, head average, ranking with
ties to the lower index, ascending output, byte-exact gather."""
import os

import numpy as np
import pytest

import oracle
import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_keep_counts_golden():
    n = 0
    for line in open(os.path.join(GOLD, "keep_counts.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        npatch, keep, k = line.split()
        assert oracle.keep_count(int(npatch), float(keep)) == int(k)
        n += 1
    assert n >= 8
    for bad in (0.0, -0.1, 1.5, float("nan")):
        with pytest.raises(ValueError):
            oracle.keep_count(10, bad)
    ks = [oracle.keep_count(1000, r / 100.0) for r in range(1, 101)]
    assert ks == sorted(ks) and ks[-1] == 1000


def _brute_force_keep(scores, k):
    """numpy restatement: fp32 sequential head sum, one division, lexsort on (-mean, index)."""
    acc = np.zeros(scores.shape[1], dtype=np.float32)
    for h in range(scores.shape[0]):
        acc = (acc + scores[h]).astype(np.float32)
    mean = (acc / np.float32(scores.shape[0])).astype(np.float32)
    order = np.lexsort((np.arange(mean.size), -mean.astype(np.float64)))
    return np.sort(order[:k]).astype(np.int32), mean


@pytest.mark.parametrize("grid,keep,quantum", [(64, 0.5, None), (64, 0.6, 2.0 ** -12),
                                               (16, 0.3, 2.0 ** -8), (37, 0.5, None)])
def test_filter_matches_lexsort(grid, keep, quantum):
    sc = synth.filter_scores(1, 2, 16, grid, grid, tie_quantum=quantum)
    tok = synth.token_rows(9, 2, 1 + grid * grid, 32)
    out, kept, mean = oracle.token_filter(sc, tok, n_global=1, keep_ratio=keep)
    k = oracle.keep_count(grid * grid, keep)
    for b in range(2):
        want, wmean = _brute_force_keep(sc[b], k)
        assert np.array_equal(kept[b], want)
        assert np.array_equal(mean[b], wmean)
        assert np.array_equal(out[b, 0], tok[b, 0])
        assert np.array_equal(out[b, 1:], tok[b, 1 + want])
    if quantum is not None:   # the tie stress really has ties at the threshold
        kth = np.sort(mean[0])[::-1][k - 1]
        assert (mean[0] == kth).sum() > 1


def test_filter_all_equal_and_identity_and_nesting():
    sc = np.full((1, 4, 50), 0.02, dtype=np.float32)
    _, kept, _ = oracle.token_filter(sc, None, keep_ratio=0.3)
    assert kept.tolist() == [list(range(15))]                 # ties -> lowest indices
    sc = synth.filter_scores(4, 1, 8, 12, 12)
    tok = synth.token_rows(5, 1, 2 + 144, 16)
    out, kept, _ = oracle.token_filter(sc, tok, n_global=2, keep_ratio=1.0)
    assert kept.tolist() == [list(range(144))] and np.array_equal(out, tok)   # keep 1.0 = identity
    prev = set()
    for k in range(1, 145, 13):
        _, kk, _ = oracle.token_filter(sc, None, keep_ratio=k / 144.0)
        assert kk.shape[1] == k and set(kk[0]) >= prev
        prev = set(kk[0])


def test_filter_signed_zero_and_order():
    # means: [0, -0, 1, 0] -> with k=2 keep index 2 and the first zero (index 0): -0 == +0
    sc = np.array([[[0.0, -0.0, 1.0, 0.0]]], dtype=np.float32)
    _, kept, _ = oracle.token_filter(sc, None, keep_ratio=0.5)
    assert kept.tolist() == [[0, 2]]
    # head average really averages over heads (not max / first head)
    sc = np.array([[[0.9, 0.0, 0.5], [0.0, 0.8, 0.5]]], dtype=np.float32)
    _, kept, mean = oracle.token_filter(sc, None, keep_ratio=1 / 3)
    assert kept.tolist() == [[2]] and np.allclose(mean, [[0.45, 0.4, 0.5]])
