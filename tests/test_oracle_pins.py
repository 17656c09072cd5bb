"""Pins of the CPU oracle against things other than itself: closed forms, brute force on tiny
inputs, a hand-worked example, an independent linear-algebra routine and the invariants that
Def. 1-2 and Eq. 7, 9, 10 of the paper imply.  CPU only."""
import itertools
import json
import math
import os

import numpy as np
import pytest

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf16_bits(x):
    """float array (values exactly representable in bf16, or rounded to nearest even) -> uint16 bits."""
    a = np.asarray(x, np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def bf16_vals(bits):
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def rand_tokens(rng, n, d, scale=1.0):
    bits = bf16_bits(rng.standard_normal((n, d)) * scale)
    return bits, bf16_vals(bits)


# ----------------------------------------------------------------------------- scores (K-norm, Eq. 7 norms)

def test_scores_closed_forms(oracle):
    d = 96
    rows = np.zeros((5, d), np.float32)
    rows[0, :] = -0.75            # constant row c: l1 = d|c|, l2 = |c| sqrt(d)
    rows[1, 17] = 3.0             # one-hot: l1 = l2 = |value|
    rows[2, :] = 0.0              # zero row
    rows[3, ::2], rows[3, 1::2] = 2.0, -2.0
    rows[4, :3] = [3.0, -4.0, 12.0]   # 3-4-12-13 quadruple
    l1, l2 = oracle.scores(bf16_bits(rows), 0, 5)
    assert l1.tolist() == [0.75 * d, 3.0, 0.0, 2.0 * d, 19.0]
    assert l2[0] == pytest.approx(0.75 * math.sqrt(d), rel=1e-15)
    assert l2[1] == 3.0 and l2[2] == 0.0 and l2[4] == 13.0
    assert l2[3] == pytest.approx(2.0 * math.sqrt(d), rel=1e-15)


def test_scores_exact_sum_and_scaling(oracle):
    rng = np.random.default_rng(1)
    bits, vals = rand_tokens(rng, 7, 333)
    l1, l2 = oracle.scores(bits, 0, 7)
    for j in range(7):
        # math.fsum is the correctly rounded sum: an independent exact reference
        assert l1[j] == pytest.approx(math.fsum(abs(v) for v in vals[j]), rel=1e-13)
        assert l2[j] == pytest.approx(math.sqrt(math.fsum(v * v for v in vals[j])), rel=1e-13)
    # scaling by a power of two is exact in bf16 and scales both norms by |alpha|
    l1s, l2s = oracle.scores(bf16_bits(vals * -4.0), 0, 7)
    assert np.array_equal(l1s, 4.0 * l1) and np.array_equal(l2s, 4.0 * l2)


def test_scores_respect_vision_window(oracle):
    rng = np.random.default_rng(2)
    bits, vals = rand_tokens(rng, 12, 40)
    l1, _ = oracle.scores(bits, 3, 5)
    assert l1 == pytest.approx(np.abs(vals[3:8]).sum(1), rel=1e-13)


# ----------------------------------------------------------------------------- pivots (Def. 1)

def test_pivots_match_rank_counting(oracle):
    rng = np.random.default_rng(3)
    for n, P in [(1, 1), (9, 3), (64, 8), (64, 64), (33, 5)]:
        s = rng.standard_normal(n) ** 2
        s[rng.integers(0, n, size=n // 4)] = s[0]          # plant ties
        piv, _ = oracle.pivots(s, P)
        # brute force: rank of j = number of tokens that beat it (larger score, or equal and lower index)
        rank = [sum(1 for t in range(n) if s[t] > s[j] or (s[t] == s[j] and t < j)) for j in range(n)]
        expect = [j for r in range(P) for j in range(n) if rank[j] == r]
        assert piv.tolist() == expect
        assert len(set(piv.tolist())) == P
        others = np.setdiff1d(np.arange(n), piv)
        if len(others):
            assert s[piv].min() >= s[others].max()


def test_pivots_min_variant_and_gap(oracle):
    s = np.array([5.0, 1.0, 4.0, 2.0, 8.0])
    piv, gap = oracle.pivots(s, 2, largest=True)
    assert piv.tolist() == [4, 0]
    assert gap == pytest.approx(min((8 - 5) / 8, (5 - 4) / 5))
    piv, gap = oracle.pivots(s, 2, largest=False)
    assert piv.tolist() == [1, 3]
    assert gap == pytest.approx(min((2 - 1) / 1, (4 - 2) / 2))


# ----------------------------------------------------------------------------- similarity (Def. 2, Eq. 7)

def test_similarity_against_numpy_matmul(oracle):
    rng = np.random.default_rng(4)
    bits, vals = rand_tokens(rng, 50, 128)
    vis_offset, n_vis = 4, 40
    l1, l2 = oracle.scores(bits, vis_offset, n_vis)
    piv = np.array([7, 0, 39, 21], np.int32)
    dup = oracle.similarity(bits, vis_offset, n_vis, piv, l2)
    X = vals[vis_offset:vis_offset + n_vis]
    Xn = X / np.linalg.norm(X, axis=1, keepdims=True)
    ref = Xn[piv] @ Xn.T                                     # independent fp64 library routine
    assert np.abs(dup - ref).max() < 1e-14
    assert np.all(np.abs(dup) <= 1.0 + 1e-15)
    assert np.allclose(dup[np.arange(4), piv], 1.0, atol=1e-15)
    assert np.allclose(dup[:, piv], dup[:, piv].T, atol=1e-15)  # pivot x pivot block is symmetric
    # Lemma 1's algebra on unit vectors: |p^ - x^|^2 = 2 (1 - dup)
    dist2 = ((Xn[piv][:, None, :] - Xn[None, :, :]) ** 2).sum(-1)
    assert np.abs(dist2 - 2.0 * (1.0 - dup)).max() < 1e-13


def test_similarity_closed_forms(oracle):
    d = 8
    X = np.zeros((6, d), np.float32)
    X[0, 0] = 2.0                    # e0
    X[1, 1] = 5.0                    # e1: orthogonal to e0
    X[2, 0] = -0.5                   # -e0/4: dup = -1
    X[3, 0] = 16.0                   # 8 e0: dup = +1
    X[4, :2] = [1.0, 1.0]            # 45 degrees from e0 and e1
    # row 5 stays zero: dup := 0
    bits = bf16_bits(X)
    _, l2 = oracle.scores(bits, 0, 6)
    dup = oracle.similarity(bits, 0, 6, np.array([0, 4], np.int32), l2)
    assert dup[0].tolist() == pytest.approx([1.0, 0.0, -1.0, 1.0, 1 / math.sqrt(2), 0.0], abs=1e-15)
    assert dup[1].tolist() == pytest.approx([1 / math.sqrt(2), 1 / math.sqrt(2), -1 / math.sqrt(2),
                                             1 / math.sqrt(2), 1.0, 0.0], abs=1e-15)


def test_similarity_detects_transposed_or_unnormalised(oracle):
    """dup must be normalised by BOTH norms: scaling a token by 2 must not change its column."""
    rng = np.random.default_rng(5)
    bits, vals = rand_tokens(rng, 10, 64)
    _, l2 = oracle.scores(bits, 0, 10)
    piv = np.array([2, 6], np.int32)
    dup = oracle.similarity(bits, 0, 10, piv, l2)
    vals2 = vals.copy()
    vals2[3] *= 2.0
    vals2[6] *= 0.5
    bits2 = bf16_bits(vals2)
    _, l22 = oracle.scores(bits2, 0, 10)
    dup2 = oracle.similarity(bits2, 0, 10, piv, l22)
    assert np.abs(dup - dup2).max() < 1e-15


# ----------------------------------------------------------------------------- retention (Eq. 9-10)

def quotas(P, n_keep):
    q, r = divmod(n_keep - P, P)
    return [q + (1 if i < r else 0) for i in range(P)]


def test_retention_is_stepwise_minimal_by_exhaustion(oracle):
    """On tiny inputs every pivot's retained set has the minimal sum of dup over ALL subsets of its
    candidates of that size (unique without ties): the definition of 'the q_i lowest'."""
    rng = np.random.default_rng(6)
    for trial in range(40):
        n = int(rng.integers(4, 12))
        P = int(rng.integers(1, min(4, n) + 1))
        n_keep = int(rng.integers(P, n + 1))
        dup = rng.uniform(-1, 1, (P, n))
        piv = rng.permutation(n)[:P].astype(np.int32)
        keep, owner, eps, gap = oracle.retention(dup, piv, n_keep)
        assert int(keep.sum()) == n_keep and np.all(keep[piv] == 1)
        kept = set(piv.tolist())
        for i, qi in enumerate(quotas(P, n_keep)):
            cands = [j for j in range(n) if j not in kept]
            mine = [j for j in range(n) if owner[j] == i]
            assert len(mine) == qi
            if qi:
                best = min(itertools.combinations(cands, qi), key=lambda c: sum(dup[i, j] for j in c))
                assert sorted(best) == sorted(mine)
                assert eps[i] == max(dup[i, j] for j in mine)
            else:
                assert math.isnan(eps[i])
            kept |= set(mine)
        assert kept == set(np.nonzero(keep)[0].tolist())


def test_retention_invariants_eq9_eq10(oracle):
    rng = np.random.default_rng(7)
    n, P, n_keep = 300, 6, 57      # (57 - 6) % 6 = 3: the three highest-ranked pivots take one extra
    dup = rng.uniform(-1, 1, (P, n))
    piv = rng.permutation(n)[:P].astype(np.int32)
    keep, owner, eps, gap = oracle.retention(dup, piv, n_keep)
    assert int(keep.sum()) == n_keep                       # |R| = n_keep
    assert np.all(keep[piv] == 1)                          # P subset of R (Eq. 10)
    assert [int((owner == i).sum()) for i in range(P)] == [9, 9, 9, 8, 8, 8]
    assert [int(owner[p]) for p in piv] == [P + i for i in range(P)]
    dropped = np.nonzero(keep == 0)[0]
    for i in range(P):
        mine = np.nonzero(owner == i)[0]
        assert np.all(dup[i, mine] <= eps[i])              # R_i = {x_j : dup <= eps_i} (Eq. 9)
        assert np.all(dup[i, dropped] >= eps[i])           # a dropped token was a candidate of every pivot
    best_left = min(dup[i, dropped].min() - eps[i] for i in range(P))
    assert gap <= best_left + 1e-18 and gap >= 0.0


def test_retention_ties_take_lower_index_and_mask_earlier_picks(oracle):
    # two pivots that rank every candidate identically: the second must not re-pick the first's tokens
    dup = np.array([[9, 9, .1, .2, .2, .3, .4, .5],
                    [9, 9, .1, .2, .2, .3, .4, .5]], float)
    piv = np.array([0, 1], np.int32)
    keep, owner, eps, gap = oracle.retention(dup, piv, 6)
    assert owner.tolist() == [2, 3, 0, 0, 1, 1, -1, -1]
    assert eps.tolist() == [.2, .3]
    assert gap == 0.0                                      # pivot 0 left an equal candidate (index 4) behind


def test_retention_single_pivot_is_partial_sort(oracle):
    rng = np.random.default_rng(8)
    n, n_keep = 200, 31
    dup = rng.uniform(-1, 1, (1, n))
    keep, owner, eps, gap = oracle.retention(dup, np.array([17], np.int32), n_keep)
    row = dup[0].copy()
    row[17] = np.inf
    expect = set(np.argsort(row, kind="stable")[: n_keep - 1].tolist()) | {17}
    assert set(np.nonzero(keep)[0].tolist()) == expect
    srt = np.sort(row)
    assert eps[0] == srt[n_keep - 2] and gap == pytest.approx(srt[n_keep - 1] - srt[n_keep - 2])


def test_retention_all_pivots_and_identity(oracle):
    rng = np.random.default_rng(9)
    dup = rng.uniform(-1, 1, (5, 20))
    piv = np.array([3, 9, 1, 0, 19], np.int32)
    keep, owner, eps, gap = oracle.retention(dup, piv, 5)        # n_keep = P: R = P
    assert sorted(np.nonzero(keep)[0].tolist()) == sorted(piv.tolist())
    assert np.all(np.isnan(eps)) and gap == math.inf
    keep, owner, eps, gap = oracle.retention(dup, piv, 20)       # n_keep = n_vis: everything stays
    assert np.all(keep == 1) and np.all(owner >= 0)


def test_retention_rejects_bad_shapes(oracle):
    dup = np.zeros((2, 5))
    with pytest.raises(RuntimeError):
        oracle.retention(dup, np.array([0, 1], np.int32), 1)      # fewer kept than pivots
    with pytest.raises(RuntimeError):
        oracle.retention(dup, np.array([0, 1], np.int32), 6)      # more kept than tokens
    with pytest.raises(RuntimeError):
        oracle.retention(dup, np.array([1, 1], np.int32), 3)      # repeated pivot


# ----------------------------------------------------------------------------- compaction

def test_compact_properties(oracle):
    rng = np.random.default_rng(10)
    S, d, vo, nv = 23, 16, 5, 11
    bits, _ = rand_tokens(rng, S, d)
    keep = np.array([1, 0, 0, 1, 1, 0, 1, 0, 0, 0, 1], np.uint8)
    pos = rng.integers(0, 10_000_000_000, S).astype(np.int64)
    oh, oi, op = oracle.compact(keep, bits, vo, nv, pos)
    assert oi.tolist() == [0, 1, 2, 3, 4, 5, 8, 9, 11, 15, 16, 17, 18, 19, 20, 21, 22]
    assert np.all(np.diff(oi) > 0)
    assert np.array_equal(oh, bits[oi]) and np.array_equal(op, pos[oi])
    _, oi2, op2 = oracle.compact(keep, bits, vo, nv, None)
    assert np.array_equal(op2, oi2.astype(np.int64))
    oh3, oi3, _ = oracle.compact(np.ones(nv, np.uint8), bits, vo, nv, None)
    assert np.array_equal(oi3, np.arange(S)) and np.array_equal(oh3, bits)


# ----------------------------------------------------------------------------- the whole step

def test_hand_worked_example(oracle):
    with open(os.path.join(GOLDEN, "worked_2d.json")) as f:
        g = json.load(f)
    tok = np.array(g["tokens"], np.float32)
    vo, na = g["vis_offset"], g["n_after"]
    text = np.array([[7.0, 7.0]] * vo + [[9.0, -9.0]] * na, np.float32)   # large-norm text rows must be ignored
    seq = np.concatenate([text[:vo], tok, text[vo:]])[None]
    bits = bf16_bits(seq)
    r = oracle.reduce(bits, bits, vo, len(tok), g["n_pivot"], g["n_keep"])
    assert r.l1[0].tolist() == g["l1"]
    assert (r.l2[0] ** 2).tolist() == pytest.approx(g["l2_squared"], rel=1e-15)
    assert r.pivot_idx[0].tolist() == g["pivot_idx"]
    s2, s17, s34 = math.sqrt(2), math.sqrt(17), math.sqrt(34)
    assert (r.dup[0, 0, :5] * s2).tolist() == pytest.approx([1, s2, 1, 0, s2], abs=1e-15)
    assert r.dup[0, 1, [0, 2, 4]].tolist() == pytest.approx([-4 / s17, -1 / s17, -5 / s34], abs=1e-15)
    assert r.keep[0].tolist() == g["keep"]
    assert r.owner[0].tolist() == g["owner"]
    assert r.eps[0].tolist() == pytest.approx([0.0, -4 / s17], abs=1e-15)
    assert r.retain_gap[0] == pytest.approx(4 / s17 - 5 / s34, abs=1e-15)
    assert r.pivot_gap[0] == pytest.approx(min(1 / 6, 1 / 5), abs=1e-15)   # ranking 6, 5, then 4
    assert r.out_idx[0].tolist() == g["out_idx"]
    assert np.array_equal(r.out_hidden[0], bits[0][g["out_idx"]])
    assert r.out_pos[0].tolist() == g["out_idx"]


def test_scaled_copies_of_a_pivot_are_dropped(oracle):
    """'Duplicates collapse to one': copies alpha * p (0 < alpha < 1) have dup = 1, the highest possible,
    so they are never retained while other candidates remain; and they cannot be pivots themselves."""
    rng = np.random.default_rng(11)
    n, d = 60, 64
    _, vals = rand_tokens(rng, n, d)
    vals[5] *= 4.0                                   # the single pivot
    for j, a in [(9, 0.5), (23, 0.25), (41, 0.125)]:
        vals[j] = vals[5] * a
    bits = bf16_bits(vals)[None]
    r = oracle.reduce(bits, bits, 0, n, 1, n - 3)
    assert r.pivot_idx[0].tolist() == [5]
    assert set(np.nonzero(r.keep[0] == 0)[0].tolist()) == {9, 23, 41}
    assert r.dup[0, 0, [9, 23, 41]].tolist() == pytest.approx([1.0, 1.0, 1.0], abs=1e-15)


def test_permutation_equivariance(oracle):
    rng = np.random.default_rng(12)
    n, d, P, Kp = 90, 48, 4, 30
    bits, _ = rand_tokens(rng, n, d)
    perm = rng.permutation(n)
    a = oracle.reduce(bits[None], None, 0, n, P, Kp)
    b = oracle.reduce(bits[perm][None], None, 0, n, P, Kp)
    kept_a = set(np.nonzero(a.keep[0])[0].tolist())
    kept_b = set(perm[np.nonzero(b.keep[0])[0]].tolist())
    assert kept_a == kept_b
    assert a.pivot_idx[0].tolist() == perm[b.pivot_idx[0]].tolist()


def test_reduce_equals_its_steps_and_keeps_order(oracle):
    rng = np.random.default_rng(13)
    B, S, d, vo, nv, P, Kp = 3, 70, 32, 6, 50, 3, 17
    hb, _ = rand_tokens(rng, B * S, d)
    kb, _ = rand_tokens(rng, B * S, d)
    hb, kb = hb.reshape(B, S, d), kb.reshape(B, S, d)
    pos = rng.integers(0, 1 << 40, (B, S)).astype(np.int64)
    r = oracle.reduce(hb, kb, vo, nv, P, Kp, pos_in=pos)
    assert r.out_idx.shape == (B, S - nv + Kp)
    for b in range(B):
        l1, l2 = oracle.scores(kb[b], vo, nv)
        piv, _ = oracle.pivots(l1, P)
        dup = oracle.similarity(kb[b], vo, nv, piv, l2)
        keep, owner, eps, _ = oracle.retention(dup, piv, Kp)
        oh, oi, op = oracle.compact(keep, hb[b], vo, nv, pos[b])
        assert np.array_equal(r.pivot_idx[b], piv) and np.array_equal(r.keep[b], keep)
        assert np.array_equal(r.out_idx[b], oi) and np.array_equal(r.out_pos[b], op)
        assert np.array_equal(r.out_hidden[b], oh)          # hidden rows, not key rows, are gathered
        assert np.all(np.diff(r.out_idx[b]) > 0)            # original order preserved
        assert set(range(vo)) <= set(oi.tolist()) and set(range(vo + nv, S)) <= set(oi.tolist())
    # keys = None means the hidden states are scored
    r2 = oracle.reduce(hb, None, vo, nv, P, Kp)
    r3 = oracle.reduce(hb, hb, vo, nv, P, Kp)
    assert np.array_equal(r2.out_idx, r3.out_idx)


def test_l2_score_variant_changes_only_the_ranking(oracle):
    # a spiky row wins under L2, a flat row wins under L1
    d = 16
    X = np.zeros((3, d), np.float32)
    X[0, :] = 1.0          # L1 16, L2 4
    X[1, 0] = 8.0          # L1 8,  L2 8
    X[2, :4] = 1.5         # L1 6,  L2 3
    bits = bf16_bits(X)[None]
    assert oracle.reduce(bits, None, 0, 3, 1, 1, norm_kind=1).pivot_idx[0].tolist() == [0]
    assert oracle.reduce(bits, None, 0, 3, 1, 1, norm_kind=2).pivot_idx[0].tolist() == [1]
    assert oracle.reduce(bits, None, 0, 3, 1, 1, largest=False).pivot_idx[0].tolist() == [2]
