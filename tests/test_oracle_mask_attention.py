"""Pins of the oracle's sparsification rule and masked attention (Sec. 3.2).

The oracle is checked against things other than itself: hand-enumerated neighbour sets,
closed-form pair counts, an independently written dense attention, a library masked
attention in fp64, and algebraic identities of softmax attention."""
import os

import numpy as np
import pytest
import torch

import oracle
import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _read_neighbours(name):
    rows = {}
    for line in open(os.path.join(GOLD, name)):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        k, v = line.split(":")
        rows[int(k)] = sorted(int(t) for t in v.split())
    return rows


@pytest.mark.parametrize("name,h,w,b,r", [
    ("neighbours_4x4_b1_r1.txt", 4, 4, 1, 1),
    ("neighbours_4x4_b2_r0.txt", 4, 4, 2, 0),
    ("neighbours_5x5_b2_r1.txt", 5, 5, 2, 1),
])
def test_mask_matches_hand_enumeration(name, h, w, b, r):
    m = oracle.mask(h, w, b, r, n_global=1)
    gold = _read_neighbours(name)
    assert gold
    for p, allowed in gold.items():
        got = sorted(int(j) for j in np.nonzero(m[1 + p, 1:])[0])
        assert got == allowed, (p, got, allowed)
    # global token: full row and full column
    assert m[0].all() and m[:, 0].all()


def test_mask_pair_counts_closed_form():
    for line in open(os.path.join(GOLD, "pair_counts.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        h, w, b, r, g, total = (int(t) for t in line.split())
        if h * w > 5000:   # the 146x146 row is checked through the separable row sums below
            continue
        m = oracle.mask(h, w, b, r, n_global=g) if h * w <= 800 else None
        if m is not None:
            assert int(m.sum()) == total
            assert (m == m.T).all()


def _axis_pairs(n, b, r):
    sizes = [min(b, n - i * b) for i in range((n + b - 1) // b)]
    return sum(sizes[i] * sizes[j] for i in range(len(sizes)) for j in range(len(sizes))
               if abs(i - j) <= r)


@pytest.mark.parametrize("h,w,b,r,total", [(64, 64, 8, 1, 1990657), (146, 146, 8, 2, 29679769)])
def test_mask_row_sums_large_grids(h, w, b, r, total):
    """Row sums of the oracle's predicate, sampled rows, against per-axis counting; the closed-form
    totals of the golden file are re-derived from the per-axis block sizes."""
    assert _axis_pairs(h, b, r) * _axis_pairs(w, b, r) + h * w + 1 + h * w == total
    import ctypes as C
    d = oracle._desc(1, h, w, b, r, 1, 1, 1, h * w, None, 0.0)
    f = oracle.lib().spvo_allowed
    rng = np.random.default_rng(0)
    for p in rng.integers(0, h * w, size=6):
        y, x = divmod(int(p), w)
        by, bx = y // b, x // b
        ny = sum(min(b, h - c * b) for c in range(max(0, by - r), min((h + b - 1) // b, by + r + 1)))
        nx = sum(min(b, w - c * b) for c in range(max(0, bx - r), min((w + b - 1) // b, bx + r + 1)))
        cnt = sum(f(C.byref(d), 0, 1 + int(p), j) for j in range(1 + h * w))
        assert cnt == ny * nx + 1


def test_mask_after_filter_uses_original_positions():
    # survivors 0, 5, 10, 15 of a 4x4 grid (the diagonal), block 2, radius 0:
    # (0,0),(1,1) share block (0,0); (2,2),(3,3) share block (1,1)
    m = oracle.mask(4, 4, 2, 0, n_global=1, patch_pos=np.array([[0, 5, 10, 15]], dtype=np.int32))
    want = np.array([[1, 1, 1, 1, 1],
                     [1, 1, 1, 0, 0],
                     [1, 1, 1, 0, 0],
                     [1, 0, 0, 1, 1],
                     [1, 0, 0, 1, 1]], dtype=bool)
    assert (m == want).all()


def _torch_masked_attention(q, k, v, mask, scale):
    qt, kt, vt = (torch.from_numpy(a.astype(np.float64)).permute(0, 2, 1, 3) for a in (q, k, v))
    o = torch.nn.functional.scaled_dot_product_attention(
        qt, kt, vt, attn_mask=torch.from_numpy(mask)[None, None], scale=scale)
    return o.permute(0, 2, 1, 3).numpy()


def test_sparse_equals_dense_when_radius_covers_grid():
    # 28x28 grid, block 7: radius 3 covers all 4x4 blocks
    q, k, v = synth.attention_qkv(0, 1, 785, 2, 64)
    o_sparse, _ = oracle.attention(q, k, v, 28, 28, 7, 3)
    o_dense = oracle.dense_attention(q, k, v)
    assert np.abs(o_sparse - o_dense).max() < 2e-6


@pytest.mark.parametrize("h,w,b,r,G", [(6, 5, 2, 1, 1), (9, 7, 3, 0, 2), (8, 8, 4, 1, 1)])
def test_sparse_attention_matches_library_masked_attention(h, w, b, r, G):
    n = G + h * w
    q, k, v = synth.attention_qkv(11, 2, n, 3, 16)
    # the boolean mask is rebuilt here from block coordinates, not taken from the oracle
    ys, xs = np.divmod(np.arange(h * w), w)
    by, bx = ys // b, xs // b
    pm = (np.abs(by[:, None] - by[None]) <= r) & (np.abs(bx[:, None] - bx[None]) <= r)
    mask = np.ones((n, n), dtype=bool)
    mask[G:, G:] = pm
    o, sc = oracle.attention(q, k, v, h, w, b, r, n_global=G, want_scores=True)
    ref = _torch_masked_attention(q, k, v, mask, 1.0 / 4.0)
    assert np.abs(o - ref).max() < 2e-6
    # CLS scores: softmax row of token 0 at the patch columns (Sec. 3.3)
    s = np.einsum("bhe,bjhe->bhj", q[:, 0].astype(np.float64), k.astype(np.float64)) / 4.0
    p = np.exp(s - s.max(-1, keepdims=True))
    p /= p.sum(-1, keepdims=True)
    assert np.abs(sc - p[:, :, G:]).max() < 1e-6
    assert np.all(sc.sum(-1) < 1.0)      # the global columns hold the rest of the row


def test_constant_and_one_hot_values():
    h, w, b, r = 6, 6, 2, 1
    n = 1 + h * w
    q, k, _ = synth.attention_qkv(3, 1, n, 2, 8)
    v = np.broadcast_to(np.arange(8, dtype=np.float32), (1, n, 2, 8)).copy()
    o, _ = oracle.attention(q, k, v, h, w, b, r)
    assert np.abs(o - v).max() < 1e-6            # rows of p sum to one
    m = oracle.mask(h, w, b, r)
    # V = one-hot(j) in dimension 0 => o[i, 0] = p_ij: zero exactly where masked, positive else
    for j in (0, 1, 17, 36):
        v1 = np.zeros((1, n, 2, 8), dtype=np.float32)
        v1[0, j, :, 0] = 1.0
        o1, _ = oracle.attention(q, k, v1, h, w, b, r)
        col = o1[0, :, 0, 0]
        assert np.all(col[~m[:, j]] == 0.0)
        assert np.all(col[m[:, j]] > 0.0)


def test_rows_argument_and_scale():
    q, k, v = synth.attention_qkv(5, 1, 1 + 16, 2, 8)
    full, _ = oracle.attention(q, k, v, 4, 4, 2, 0, scale=0.25)
    part, _ = oracle.attention(q, k, v, 4, 4, 2, 0, scale=0.25, rows=[3, 0, 9])
    for i in (3, 0, 9):
        assert np.array_equal(part[:, i], full[:, i])
    assert np.all(part[:, 5] == 0)
    other, _ = oracle.attention(q, k, v, 4, 4, 2, 0)   # default scale 1/sqrt(8)
    assert np.abs(other - full).max() > 1e-4


def test_filtered_positions_match_masked_subset():
    """Attention over survivors with original positions == library attention on the subset."""
    h, w, b, r = 8, 8, 2, 1
    rng = np.random.default_rng(2)
    keep = np.sort(rng.choice(h * w, size=29, replace=False)).astype(np.int32)
    n = 1 + keep.size
    q, k, v = synth.attention_qkv(7, 1, n, 2, 16)
    o, _ = oracle.attention(q, k, v, h, w, b, r, patch_pos=keep[None])
    ys, xs = np.divmod(keep, w)
    pm = (np.abs(ys[:, None] // b - ys[None] // b) <= r) & (np.abs(xs[:, None] // b - xs[None] // b) <= r)
    mask = np.ones((n, n), dtype=bool)
    mask[1:, 1:] = pm
    ref = _torch_masked_attention(q, k, v, mask, 0.25)
    assert np.abs(o - ref).max() < 2e-6


def test_permutation_inside_blocks_leaves_attention_unchanged():
    """The key set of Sec. 3.2 depends on a token's block only: presenting the tokens of every block in
    another order (positions, Q, K and V permuted alike) permutes the output rows and nothing else; the
    same holds for the order of whole blocks."""
    h, w, b, r = 8, 12, 4, 1
    rng = np.random.default_rng(8)
    pos = np.arange(h * w, dtype=np.int32)
    n = 1 + pos.size
    q, k, v = synth.attention_qkv(12, 1, n, 2, 16)
    base, bsc = oracle.attention(q, k, v, h, w, b, r, patch_pos=pos[None], want_scores=True)
    blk = (pos // w) // b * (w // b) + (pos % w) // b
    # shuffle inside blocks, then shuffle the blocks themselves
    key = rng.permutation(blk.max() + 1)[blk] * 1000.0 + rng.random(pos.size)
    perm = np.argsort(key)
    assert not np.array_equal(perm, pos)

    def reorder(a):
        out = a.copy()
        out[:, 1:] = a[:, 1 + perm]
        return out
    got, gsc = oracle.attention(reorder(q), reorder(k), reorder(v), h, w, b, r, patch_pos=pos[perm][None],
                                want_scores=True)
    assert np.abs(got - reorder(base)).max() < 1e-6
    assert np.abs(gsc - bsc[:, :, perm]).max() < 1e-7
