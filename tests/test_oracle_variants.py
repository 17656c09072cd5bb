"""Pins of the oracle's variants (caller-chosen pivots, one threshold for all pivots, row gather by the packed
index list) against things other than themselves: brute force on tiny inputs, numpy routines, invariants and
the special cases in which a variant must coincide with the main method.  CPU only."""
import itertools
import math

import numpy as np
import pytest

from test_oracle_pins import bf16_bits, rand_tokens


# ----------------------------------------------------------------------------- one threshold for all pivots

def test_global_threshold_is_minimal_by_exhaustion(oracle):
    """Among ALL subsets of the non-pivot tokens of the right size the retained one has the smallest sum of
    u_j = max_i dup[i][j] (unique without ties): 'the tokens least duplicated by any pivot'."""
    rng = np.random.default_rng(21)
    for trial in range(40):
        n = int(rng.integers(4, 12))
        P = int(rng.integers(1, min(4, n) + 1))
        n_keep = int(rng.integers(P, n + 1))
        dup = rng.uniform(-1, 1, (P, n))
        piv = rng.permutation(n)[:P].astype(np.int32)
        keep, owner, eps, gap = oracle.retention_global(dup, piv, n_keep)
        u = dup.max(axis=0)
        cands = [j for j in range(n) if j not in set(piv.tolist())]
        mine = [j for j in cands if keep[j]]
        assert int(keep.sum()) == n_keep and np.all(keep[piv] == 1) and len(mine) == n_keep - P
        if mine:
            best = min(itertools.combinations(cands, len(mine)), key=lambda c: sum(u[j] for j in c))
            assert sorted(best) == sorted(mine)
            assert np.all(eps == max(u[j] for j in mine))
            assert all(owner[j] == int(np.argmax(dup[:, j])) for j in mine)
        else:
            assert np.all(np.isnan(eps)) and gap == math.inf


def test_global_threshold_against_numpy_and_invariants(oracle):
    rng = np.random.default_rng(22)
    n, P, n_keep = 400, 7, 90
    dup = rng.uniform(-1, 1, (P, n))
    piv = rng.permutation(n)[:P].astype(np.int32)
    keep, owner, eps, gap = oracle.retention_global(dup, piv, n_keep)
    u = dup.max(axis=0)
    u[piv] = np.inf                                          # pivots are no candidates
    order = np.argsort(u, kind="stable")                     # an independent routine: stable sort = ties to lower index
    expect = set(order[: n_keep - P].tolist()) | set(piv.tolist())
    assert set(np.nonzero(keep)[0].tolist()) == expect
    dropped = np.nonzero(keep == 0)[0]
    kept_np = np.array(sorted(expect - set(piv.tolist())))
    assert np.all(u[kept_np] <= eps[0]) and np.all(u[dropped] >= eps[0])   # R = P u {x_j : max_i dup <= eps}
    assert gap == pytest.approx(u[dropped].min() - eps[0]) and gap >= 0
    assert [int(owner[p]) for p in piv] == [P + i for i in range(P)]
    assert np.all(owner[dropped] == -1)


def test_global_threshold_special_cases(oracle):
    rng = np.random.default_rng(23)
    dup = rng.uniform(-1, 1, (1, 60))
    piv = np.array([11], np.int32)
    a = oracle.retention_global(dup, piv, 20)                # one pivot: both rules are the same partial sort
    b = oracle.retention(dup, piv, 20)
    assert np.array_equal(a[0], b[0]) and a[2][0] == b[2][0] and a[3] == b[3]
    # ties: equal u_j go to the lower index; the nearest pivot is the first of equal dups
    dup = np.array([[9, 9, .3, .3, .1, .3],
                    [9, 9, .3, .2, .1, .3]], float)
    keep, owner, eps, gap = oracle.retention_global(dup, np.array([0, 1], np.int32), 4)
    assert keep.tolist() == [1, 1, 1, 0, 1, 0] and owner.tolist() == [2, 3, 0, -1, 0, -1]
    assert eps.tolist() == [.3, .3] and gap == 0.0
    with pytest.raises(RuntimeError):
        oracle.retention_global(dup, np.array([1, 1], np.int32), 4)   # repeated pivot
    with pytest.raises(RuntimeError):
        oracle.retention_global(dup, np.array([0, 1], np.int32), 7)   # more kept than tokens


def test_global_rule_differs_from_quotas_where_it_should(oracle):
    """Two pivots; token 2 is far from pivot 0 but a near copy of pivot 1.  Under per-pivot quotas pivot 0 keeps
    it (its own lowest dup); under one threshold its duplication is 0.99 and it is dropped."""
    dup = np.array([[9, 9, -.9, .1, .2, .3],
                    [9, 9, .99, .5, .4, .3]], float)
    piv = np.array([0, 1], np.int32)
    assert oracle.retention(dup, piv, 4)[0].tolist() == [1, 1, 1, 0, 0, 1]
    assert oracle.retention_global(dup, piv, 4)[0].tolist() == [1, 1, 0, 0, 1, 1]


# ----------------------------------------------------------------------------- pivots chosen by the caller

def test_given_pivots_replace_only_the_pivot_step(oracle):
    rng = np.random.default_rng(24)
    B, S, d, vo, nv, P, Kp = 3, 64, 32, 4, 50, 4, 19
    hb, _ = rand_tokens(rng, B * S, d)
    kb, _ = rand_tokens(rng, B * S, d)
    hb, kb = hb.reshape(B, S, d), kb.reshape(B, S, d)
    base = oracle.reduce(hb, kb, vo, nv, P, Kp)
    same = oracle.reduce(hb, kb, vo, nv, P, Kp, pivots_in=base.pivot_idx)      # its own pivots: nothing changes
    assert np.array_equal(same.out_idx, base.out_idx) and np.array_equal(same.owner, base.owner)
    assert np.all(np.isinf(same.pivot_gap))                                    # nothing was ranked
    given = np.stack([rng.permutation(nv)[:P] for _ in range(B)]).astype(np.int32)
    r = oracle.reduce(hb, kb, vo, nv, P, Kp, pivots_in=given)
    for b in range(B):                                                         # = the steps, composed by hand
        l1, l2 = oracle.scores(kb[b], vo, nv)
        dup = oracle.similarity(kb[b], vo, nv, given[b], l2)
        keep, owner, eps, _ = oracle.retention(dup, given[b], Kp)
        oh, oi, op = oracle.compact(keep, hb[b], vo, nv)
        assert np.array_equal(r.pivot_idx[b], given[b]) and np.array_equal(r.owner[b], owner)
        assert np.array_equal(r.out_idx[b], oi) and np.array_equal(r.out_hidden[b], oh)
        assert np.all(r.keep[b][given[b]] == 1)                                # P subset of R whatever the pivots
    swapped = given[:, ::-1].copy()                                            # the order given is the order of the turns
    r2 = oracle.reduce(hb, kb, vo, nv, P, Kp, pivots_in=swapped)
    assert np.array_equal(r2.pivot_idx, swapped)
    assert not np.array_equal(r2.owner, r.owner)
    bad = given.copy()
    bad[1, 2] = bad[1, 0]
    with pytest.raises(RuntimeError):
        oracle.reduce(hb, kb, vo, nv, P, Kp, pivots_in=bad)                    # repeated pivot
    g = oracle.reduce(hb, kb, vo, nv, P, Kp, pivots_in=given, rule=1)          # both variants together
    for b in range(B):
        l1, l2 = oracle.scores(kb[b], vo, nv)
        dup = oracle.similarity(kb[b], vo, nv, given[b], l2)
        assert np.array_equal(g.keep[b], oracle.retention_global(dup, given[b], Kp)[0])


# ----------------------------------------------------------------------------- rows gathered by the packed list

def test_gather_rows_against_numpy(oracle):
    rng = np.random.default_rng(25)
    B, S, w, S_out = 3, 40, 24, 17
    src = rng.integers(0, 1 << 16, (B, S, w)).astype(np.uint16)
    idx = np.stack([np.sort(rng.permutation(S)[:S_out]) for _ in range(B)]).astype(np.int32)
    out = oracle.gather_rows(src, idx)
    assert np.array_equal(out, np.take_along_axis(src, idx[:, :, None].astype(np.int64), axis=1))
    ident = np.tile(np.arange(S, dtype=np.int32), (B, 1))
    assert np.array_equal(oracle.gather_rows(src, ident), src)                 # the identity list copies
    idx[2, 5] = S
    with pytest.raises(RuntimeError):
        oracle.gather_rows(src, idx)                                           # index past the end


def test_gather_rows_follows_the_reduction(oracle):
    """The packed list of a reduction applied to the hidden states themselves gives the packed hidden states."""
    rng = np.random.default_rng(26)
    B, S, d, vo, nv, P, Kp = 2, 50, 16, 3, 40, 2, 9
    hb, _ = rand_tokens(rng, B * S, d)
    hb = hb.reshape(B, S, d)
    r = oracle.reduce(hb, None, vo, nv, P, Kp)
    assert np.array_equal(oracle.gather_rows(hb, r.out_idx), r.out_hidden)


# ----------------------------------------------------------------------------- Eq. 7 on the hidden rows

def test_cosine_on_hidden_rows_is_the_composition_of_the_steps(oracle):
    """Pivots ranked by the key rows, dup evaluated on the hidden rows: equal to the step functions composed by
    hand, to numpy's cosine of the hidden rows, and to the main method when both tensors are the same."""
    rng = np.random.default_rng(27)
    B, S, d, vo, nv, P, Kp = 3, 60, 32, 5, 48, 3, 14
    hb, hv = rand_tokens(rng, B * S, d)
    kb, _ = rand_tokens(rng, B * S, d)
    hb, kb, hv = hb.reshape(B, S, d), kb.reshape(B, S, d), hv.reshape(B, S, d)
    r = oracle.reduce(hb, kb, vo, nv, P, Kp, cosine_on_hidden=True)
    base = oracle.reduce(hb, kb, vo, nv, P, Kp)
    assert np.array_equal(r.pivot_idx, base.pivot_idx) and np.array_equal(r.l1, base.l1)   # the ranking is the keys'
    assert not np.array_equal(r.keep, base.keep)
    for b in range(B):
        kl1, _ = oracle.scores(kb[b], vo, nv)
        piv, _ = oracle.pivots(kl1, P)
        _, hl2 = oracle.scores(hb[b], vo, nv)
        dup = oracle.similarity(hb[b], vo, nv, piv, hl2)
        keep, owner, eps, _ = oracle.retention(dup, piv, Kp)
        assert np.array_equal(r.pivot_idx[b], piv) and np.array_equal(r.l2[b], hl2)
        assert np.array_equal(r.dup[b], dup) and np.array_equal(r.keep[b], keep)
        X = hv[b, vo:vo + nv]
        Xn = X / np.linalg.norm(X, axis=1, keepdims=True)
        assert np.allclose(r.dup[b], Xn[piv] @ Xn.T, rtol=0, atol=1e-12)                    # an independent routine
    same = oracle.reduce(hb, hb, vo, nv, P, Kp, cosine_on_hidden=True)                      # one tensor: nothing changes
    plain = oracle.reduce(hb, hb, vo, nv, P, Kp)
    assert np.array_equal(same.out_idx, plain.out_idx) and np.array_equal(same.dup, plain.dup)
    none = oracle.reduce(hb, None, vo, nv, P, Kp, cosine_on_hidden=True)                    # keys = None: likewise
    assert np.array_equal(none.out_idx, plain.out_idx)


# ----------------------------------------------------------------------------- pivots taken from the text tokens

def test_text_pivots_similarity_and_budget(oracle):
    """Pivots outside the vision block: their cosines against numpy, the budget split over all pivots but counted
    in vision tokens only, and the coincidence with the plain functions when every pivot is a vision token."""
    rng = np.random.default_rng(28)
    S, d, vo, nv = 70, 32, 8, 50
    kb, kv = rand_tokens(rng, S, d)
    piv = np.array([3, -5, 17, nv + 6, -8], np.int32)            # vision, text before, vision, text after, first token
    dup = oracle.similarity_any(kb, vo, nv, piv)
    X = kv[vo:vo + nv]
    Xn = X / np.linalg.norm(X, axis=1, keepdims=True)
    Pr = kv[vo + piv]
    Pn = Pr / np.linalg.norm(Pr, axis=1, keepdims=True)
    assert np.allclose(dup, Pn @ Xn.T, rtol=0, atol=1e-12)       # an independent routine
    n_keep = 20                                                  # 2 vision pivots + 18 over 5 pivots: quotas 4,4,4,3,3
    keep, owner, eps, gap = oracle.retention_any(dup, piv, n_keep)
    assert int(keep.sum()) == n_keep and keep[3] == 1 and keep[17] == 1
    assert [int((owner == i).sum()) for i in range(5)] == [4, 4, 4, 3, 3]
    assert owner[3] == 5 + 0 and owner[17] == 5 + 2
    kept = {3, 17}
    for i, qi in enumerate([4, 4, 4, 3, 3]):                     # every turn takes the lowest dup among what is left
        cands = [j for j in range(nv) if j not in kept]
        best = sorted(cands, key=lambda j: (dup[i, j], j))[:qi]
        assert sorted(best) == sorted(np.nonzero(owner == i)[0].tolist())
        assert eps[i] == max(dup[i, j] for j in best)
        kept |= set(best)
    vis_only = np.array([3, 17, 30], np.int32)                   # no text pivot: the plain functions
    _, l2 = oracle.scores(kb, vo, nv)
    assert np.allclose(oracle.similarity_any(kb, vo, nv, vis_only), oracle.similarity(kb, vo, nv, vis_only, l2), rtol=0, atol=1e-15)
    d2 = oracle.similarity(kb, vo, nv, vis_only, l2)
    a, b = oracle.retention_any(d2, vis_only, 12), oracle.retention(d2, vis_only, 12)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    with pytest.raises(RuntimeError):
        oracle.similarity_any(kb, vo, nv, np.array([-9], np.int32))          # before the sequence
    with pytest.raises(RuntimeError):
        oracle.retention_any(dup, np.array([3, -5, 17, -5, -8], np.int32), n_keep)   # repeated text pivot
    with pytest.raises(RuntimeError):
        oracle.retention(dup, piv, n_keep)                                   # the plain rule takes vision pivots only


def test_text_pivots_through_the_whole_step(oracle):
    rng = np.random.default_rng(29)
    B, S, d, vo, nv, P, Kp = 2, 64, 32, 6, 50, 4, 15
    hb, _ = rand_tokens(rng, B * S, d)
    kb, _ = rand_tokens(rng, B * S, d)
    hb, kb = hb.reshape(B, S, d), kb.reshape(B, S, d)
    piv = np.array([[4, -2, nv + 3, 20], [-6, -1, nv, nv + 7]], np.int32)   # sample 1: text pivots only
    r = oracle.reduce(hb, kb, vo, nv, P, Kp, pivots_in=piv, text_pivots=True)
    for b in range(B):
        dup = oracle.similarity_any(kb[b], vo, nv, piv[b])
        keep, owner, eps, _ = oracle.retention_any(dup, piv[b], Kp)
        oh, oi, op = oracle.compact(keep, hb[b], vo, nv)
        assert np.array_equal(r.keep[b], keep) and np.array_equal(r.out_idx[b], oi) and np.array_equal(r.out_hidden[b], oh)
        assert int(keep.sum()) == Kp                                        # the budget counts vision tokens
        assert r.out_idx.shape[1] == S - nv + Kp
    with pytest.raises(RuntimeError):
        oracle.reduce(hb, kb, vo, nv, P, Kp, pivots_in=piv)                 # text pivots must be asked for


# ----------------------------------------------------------------------------- independent pivots (the literal union of Eq. 10)

def test_union_retention_against_brute_force_and_its_invariants(oracle):
    rng = np.random.default_rng(31)
    for trial in range(20):
        nv = int(rng.integers(6, 40))
        P = int(rng.integers(1, 5))
        Kp = int(rng.integers(P, nv + 1))
        dup = rng.uniform(-1, 1, (P, nv))
        piv = rng.permutation(nv)[:P].astype(np.int32)
        keep, owner, eps, gap, cnt = oracle.retention_union(dup, piv, Kp)
        q, r = divmod(Kp - P, P)
        expect = set(piv.tolist())
        others = [j for j in range(nv) if j not in set(piv.tolist())]
        first = {}
        for i in range(P):
            qi = q + (1 if i < r else 0)
            mine = sorted(others, key=lambda j: (dup[i, j], j))[:qi]      # whatever the other pivots took
            for j in mine:
                first.setdefault(j, i)
            expect |= set(mine)
            if qi:
                assert eps[i] == max(dup[i, j] for j in mine)
                assert all(dup[i, j] >= eps[i] for j in others if j not in mine)
            else:
                assert np.isnan(eps[i])
        assert set(np.nonzero(keep)[0].tolist()) == expect and cnt == len(expect)
        assert P <= cnt <= Kp                                              # Eq. 10's union can fall short of the budget
        assert all(owner[p] == P + i for i, p in enumerate(piv))
        assert all(owner[j] == i for j, i in first.items())
        assert (owner[~keep.astype(bool)] == -1).all()


def test_union_coincides_with_the_quota_rule_when_the_picks_are_disjoint(oracle):
    """One pivot: nothing to mask.  Pivots with disjoint neighbourhoods: masking never bites."""
    rng = np.random.default_rng(32)
    dup = rng.uniform(-1, 1, (1, 30))
    a, b = oracle.retention_union(dup, [4], 11), oracle.retention(dup, [4], 11)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1]) and a[4] == 11
    dup = np.ones((2, 20))
    dup[0, 2:6] = [-.9, -.8, -.7, -.6]        # pivot 0 (token 0) is far from tokens 2..5
    dup[1, 10:14] = [-.9, -.8, -.7, -.6]      # pivot 1 (token 1) from tokens 10..13
    a, b = oracle.retention_union(dup, [0, 1], 10), oracle.retention(dup, [0, 1], 10)
    assert np.array_equal(a[0], b[0]) and a[4] == 10
    dup[1] = dup[0]                            # the same neighbourhood: the union keeps it once
    keep, owner, eps, gap, cnt = oracle.retention_union(dup, [0, 1], 10)
    assert cnt == 2 + 4 and (owner[2:6] == 0).all()


def test_union_through_the_whole_step_is_packed_without_padding(oracle):
    rng = np.random.default_rng(33)
    B, S, d, vo, nv, P, Kp = 3, 50, 16, 4, 40, 3, 12
    hb, _ = rand_tokens(rng, B * S, d)
    kb, _ = rand_tokens(rng, B * S, d)
    hb, kb = hb.reshape(B, S, d), kb.reshape(B, S, d)
    r = oracle.reduce(hb, kb, vo, nv, P, Kp, rule=2)
    cu = r.cu_seqlens
    assert cu[0] == 0 and np.all(np.diff(cu) >= S - nv + P) and np.all(np.diff(cu) <= S - nv + Kp)
    for b in range(B):
        _, l2 = oracle.scores(kb[b], vo, nv)
        dup = oracle.similarity(kb[b], vo, nv, r.pivot_idx[b], l2)
        keep, owner, eps, _, cnt = oracle.retention_union(dup, r.pivot_idx[b], Kp)
        oh, oi, op = oracle.compact(keep, hb[b], vo, nv)
        assert cu[b + 1] - cu[b] == S - nv + cnt
        assert np.array_equal(r.out_idx[cu[b]:cu[b + 1]], oi) and np.array_equal(r.out_hidden[cu[b]:cu[b + 1]], oh)
        assert np.array_equal(r.out_pos[cu[b]:cu[b + 1]], op) and np.array_equal(r.keep[b], keep)
    assert (r.out_idx[cu[B]:] == -1).all()


# ----------------------------------------------------------------------------- text pivots under the other two retention rules

def test_text_pivots_under_one_threshold_and_independent_pivots(oracle):
    """Text pivots count among the pivots a token is compared with but not among the vision tokens kept: replayed by
    brute force with hand-written budgets; with vision pivots only the functions coincide with the plain ones."""
    rng = np.random.default_rng(41)
    nv, P = 40, 5
    dup = rng.uniform(-1, 1, (P, nv))
    piv = np.array([7, -3, 22, nv + 4, -1], np.int32)            # two vision pivots, three text pivots
    n_keep = 16                                                  # 2 vision pivots + 14 more vision tokens
    # one threshold: the 14 non-pivot tokens of lowest max_i dup
    keep, owner, eps, gap = oracle.retention_global(dup, piv, n_keep, text_pivots=True)
    u = dup.max(axis=0)
    cands = [j for j in range(nv) if j not in (7, 22)]
    best = sorted(cands, key=lambda j: (u[j], j))[:14]
    assert int(keep.sum()) == n_keep and keep[7] == 1 and keep[22] == 1
    assert sorted(best) == sorted(j for j in cands if keep[j])
    assert np.all(eps == max(u[j] for j in best)) and owner[7] == P + 0 and owner[22] == P + 2
    assert all(owner[j] == int(np.argmax(dup[:, j])) for j in best)
    rest = sorted(cands, key=lambda j: (u[j], j))[14:]
    assert math.isclose(gap, u[rest[0]] - max(u[j] for j in best))
    # independent pivots: 14 over 5 pivots: quotas 3, 3, 3, 3, 2, every pivot from all non-pivot tokens
    keep, owner, eps, gap, cnt = oracle.retention_union(dup, piv, n_keep, text_pivots=True)
    kept = {7, 22}
    for i, qi in enumerate([3, 3, 3, 3, 2]):
        mine = sorted(cands, key=lambda j: (dup[i, j], j))[:qi]
        assert eps[i] == max(dup[i, j] for j in mine)
        for j in mine:
            if j not in kept:
                assert owner[j] == i                               # the first pivot in rank order that took it
            kept.add(j)
    assert set(np.nonzero(keep)[0].tolist()) == kept and cnt == len(kept) and 2 + 3 <= cnt <= n_keep
    # vision pivots only: the plain functions
    vis = np.array([7, 22, 30], np.int32)
    d3 = dup[:3]
    for a, b in [(oracle.retention_global(d3, vis, 12, text_pivots=True), oracle.retention_global(d3, vis, 12)),
                 (oracle.retention_union(d3, vis, 12, text_pivots=True), oracle.retention_union(d3, vis, 12))]:
        assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1]) and np.array_equal(a[2], b[2], equal_nan=True)
    with pytest.raises(RuntimeError):
        oracle.retention_global(dup, piv, n_keep)                # text pivots must be asked for
    with pytest.raises(RuntimeError):
        oracle.retention_union(dup, np.array([7, -3, 22, -3, -1], np.int32), n_keep, text_pivots=True)   # repeated


# ----------------------------------------------------------------------------- pivots from both modalities, random pivots

def test_pivots_from_both_modalities_against_numpy(oracle):
    """Pv vision and Pt text tokens of best score, each group in rank order: numpy's stable argsort on the same
    scores is the independent routine; planted equal scores go to the earlier token."""
    rng = np.random.default_rng(42)
    S, vo, nv = 60, 9, 40
    s = rng.uniform(1, 2, S)
    s[vo + 5] = s[vo + 31] = 3.0            # a tie among the vision tokens
    s[2] = s[S - 1] = 2.5                   # a tie among the text tokens (before and after the block)
    for largest in (True, False):
        key = -s if largest else s
        vis = np.argsort(key[vo:vo + nv], kind="stable")
        text_pos = np.array([t for t in range(S) if not vo <= t < vo + nv])
        txt = text_pos[np.argsort(key[text_pos], kind="stable")] - vo
        for Pv, Pt in [(4, 4), (0, 3), (5, 0), (nv, S - nv)]:
            got = oracle.pivots_mixed(s, vo, nv, Pv, Pt, largest)
            assert got[:Pv].tolist() == vis[:Pv].tolist() and got[Pv:].tolist() == txt[:Pt].tolist()
    got = oracle.pivots_mixed(s, vo, nv, 2, 2, True)
    assert got.tolist() == [5, 31, 2 - vo, S - 1 - vo]           # the ties, lower position first; text tokens outside [0, nv)
    with pytest.raises(RuntimeError):
        oracle.pivots_mixed(s, vo, nv, 2, S - nv + 1)            # more text pivots than text tokens


def test_splitmix64_reference_outputs(oracle):
    """The generator behind the random pivots against the outputs that the reference implementation of SplitMix64
    (Steele, Lea and Flood, OOPSLA 2014) is commonly tabulated with for the seed 1234567."""
    expect = [6457827717110365317, 3203168211198807973, 9817491932198370423, 4593380528125082431, 16408922859458223821]
    assert [oracle.splitmix64(1234567, k) for k in range(5)] == expect
    assert oracle.splitmix64(0, 0) == 0xE220A8397B1DCDAF         # the first output for seed 0 (the xoshiro seeding example)


def test_random_pivots_are_a_uniform_draw_without_replacement(oracle):
    nv, P = 50, 6
    a = oracle.pivots_random(99, 3, nv, P)
    assert len(set(a.tolist())) == P and a.min() >= 0 and a.max() < nv
    assert np.array_equal(a, oracle.pivots_random(99, 3, nv, P))                     # a function of (seed, sample) only
    assert not np.array_equal(a, oracle.pivots_random(99, 4, nv, P)) and not np.array_equal(a, oracle.pivots_random(100, 3, nv, P))
    # re-derived from the pinned generator: tickets = upper halves of outputs b * 2^32 + j, smallest first, ties by index
    tickets = np.array([oracle.splitmix64(99, (3 << 32) | j) >> 32 for j in range(nv)], np.uint64)
    assert a.tolist() == np.argsort(tickets, kind="stable")[:P].tolist()
    assert sorted(oracle.pivots_random(5, 0, nv, nv).tolist()) == list(range(nv))     # P = n_vis: a permutation
    # every token is drawn about equally often: 4000 draws of 6 of 50 -> 480 expected per token, sigma ~ 21
    hits = np.zeros(nv, np.int64)
    for seed in range(4000):
        hits[oracle.pivots_random(seed, 0, nv, P)] += 1
    assert hits.sum() == 4000 * P and abs(hits - 480).max() < 6 * 21


def test_pivot_sources_through_the_whole_step(oracle):
    """The batch entry point with pivots from both modalities / random pivots = the step functions composed by hand."""
    rng = np.random.default_rng(43)
    B, S, d, vo, nv, P, Kp = 3, 70, 32, 8, 50, 6, 18
    hb, _ = rand_tokens(rng, B * S, d)
    kb, _ = rand_tokens(rng, B * S, d)
    hb, kb = hb.reshape(B, S, d), kb.reshape(B, S, d)
    for rule in (0, 1, 2):
        r = oracle.reduce(hb, kb, vo, nv, P, Kp, pivot_source=1, n_text_pivots=2, rule=rule)
        cu = r.cu_seqlens
        for b in range(B):
            l1_all, _ = oracle.scores(kb[b], 0, S)
            piv = oracle.pivots_mixed(l1_all, vo, nv, P - 2, 2)
            assert np.array_equal(r.pivot_idx[b], piv) and (piv[:4] >= 0).all() and ((piv[4:] < 0) | (piv[4:] >= nv)).all()
            dup = oracle.similarity_any(kb[b], vo, nv, piv)
            keep = (oracle.retention_any(dup, piv, Kp) if rule == 0 else oracle.retention_global(dup, piv, Kp, True) if rule == 1
                    else oracle.retention_union(dup, piv, Kp, True))[0]
            assert np.array_equal(r.keep[b], keep)
            oh, oi, op = oracle.compact(keep, hb[b], vo, nv)
            got = r.out_idx[b] if rule != 2 else r.out_idx[cu[b]:cu[b + 1]]
            assert np.array_equal(got, oi)
    r = oracle.reduce(hb, kb, vo, nv, P, Kp, pivot_source=2, seed=2024)
    for b in range(B):
        piv = oracle.pivots_random(2024, b, nv, P)
        assert np.array_equal(r.pivot_idx[b], piv)
        _, l2 = oracle.scores(kb[b], vo, nv)
        keep = oracle.retention(oracle.similarity(kb[b], vo, nv, piv, l2), piv, Kp)[0]
        assert np.array_equal(r.keep[b], keep)
    with pytest.raises(RuntimeError):
        oracle.reduce(hb, kb, vo, nv, P, Kp, pivot_source=1, n_text_pivots=S - nv + 1)
