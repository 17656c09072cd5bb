"""Parity rules between a candidate implementation's outputs and the oracle (TEST INFRASTRUCTURE).

Takes plain numpy arrays from both sides; imports nothing from the CUDA path.

Rules (bf16 inputs, fp32 accumulation on the candidate side, fp64 in the oracle):
  * norms and similarities: relative error <= 1e-2 (similarities: |d| <= 1e-2 |dup| + 1e-4, since a
    relative bound is void near 0);
  * wherever the oracle's selection margin exceeds 1e-3 (relative score gap along the pivot ranking,
    absolute dup gap at every retention boundary) pivots, kept indices, gathered rows and position ids
    are bit-exact;
  * below that margin several results are equally right: the candidate's choice must be *valid under
    tolerance* - replaying its own per-pivot assignment against the oracle's fp64 similarities, no
    token it left behind beats its threshold by more than the tolerance - and everything that does
    not depend on the near-tie (counts, order, text rows, gathered bits, position ids) is exact.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from . import dart_oracle as _o

REL_TOL = 1e-2
SIM_ABS_FLOOR = 1e-4
MARGIN = 1e-3


@dataclass
class ParityReport:
    samples: int = 0
    exact: int = 0                 # samples whose out_idx equals the oracle's
    above_margin: int = 0          # samples with margin > MARGIN (exactness enforced)
    max_rel_l1: float = 0.0
    max_rel_l2: float = 0.0
    max_abs_sim: float = 0.0
    min_margin: float = float("inf")
    notes: list = field(default_factory=list)

    def merge(self, o: "ParityReport"):
        self.samples += o.samples
        self.exact += o.exact
        self.above_margin += o.above_margin
        self.max_rel_l1 = max(self.max_rel_l1, o.max_rel_l1)
        self.max_rel_l2 = max(self.max_rel_l2, o.max_rel_l2)
        self.max_abs_sim = max(self.max_abs_sim, o.max_abs_sim)
        self.min_margin = min(self.min_margin, o.min_margin)
        self.notes += o.notes
        return self


def quotas_any(pivot_idx, n_vis: int, n_keep: int):
    """Quotas when pivots outside [0, n_vis) are text tokens: only the vision pivots count against the budget."""
    P = len(pivot_idx)
    Pv = int(sum(0 <= int(p) < n_vis for p in pivot_idx))
    q, r = divmod(n_keep - Pv, P)
    return [q + (1 if i < r else 0) for i in range(P)]


def quotas(P: int, n_keep: int):
    q, r = divmod(n_keep - P, P)
    return [q + (1 if i < r else 0) for i in range(P)]


def check_packed_outputs(out_hidden, out_idx, out_pos, hidden_bits, pos_in, vis_offset, n_vis, n_keep):
    """Rules that hold whatever the near-ties decide (one sample)."""
    S = hidden_bits.shape[0]
    S_out = S - n_vis + n_keep
    assert out_idx.shape == (S_out,), "packed length"
    assert np.all(np.diff(out_idx.astype(np.int64)) > 0), "out_idx must be strictly ascending (original order)"
    assert np.array_equal(out_idx[:vis_offset], np.arange(vis_offset)), "text rows before the vision block"
    n_after = S - vis_offset - n_vis
    assert np.array_equal(out_idx[S_out - n_after:], np.arange(vis_offset + n_vis, S)), "text rows after"
    mid = out_idx[vis_offset:vis_offset + n_keep]
    assert mid.min() >= vis_offset and mid.max() < vis_offset + n_vis, "kept rows lie in the vision block"
    expect_pos = out_idx.astype(np.int64) if pos_in is None else pos_in[out_idx]
    assert np.array_equal(out_pos, expect_pos), "position ids follow the kept rows"
    if out_hidden is not None:
        assert np.array_equal(out_hidden, hidden_bits[out_idx]), "gathered rows are bit copies of hidden rows"


def check_scores(l1, ssq, ora_l1, ora_l2, rep: ParityReport, tol=REL_TOL):
    rl1 = np.abs(l1.astype(np.float64) - ora_l1) / np.maximum(ora_l1, 1e-300)
    l2 = np.sqrt(ssq.astype(np.float64))
    rl2 = np.abs(l2 - ora_l2) / np.maximum(ora_l2, 1e-300)
    rep.max_rel_l1 = max(rep.max_rel_l1, float(rl1.max()))
    rep.max_rel_l2 = max(rep.max_rel_l2, float(rl2.max()))
    assert rl1.max() <= tol, "L1 scores off by %g relative" % rl1.max()
    assert rl2.max() <= tol, "Euclidean norms off by %g relative" % rl2.max()


def check_sim(sim, ora_dup, rep: ParityReport, tol=REL_TOL, floor=SIM_ABS_FLOOR):
    err = np.abs(sim.astype(np.float64) - ora_dup)
    rep.max_abs_sim = max(rep.max_abs_sim, float(err.max()))
    bad = err > tol * np.abs(ora_dup) + floor
    assert not bad.any(), "similarities off by up to %g" % err.max()


def check_valid_under_tolerance(keys_bits, vis_offset, n_vis, n_keep, pivot_idx, owner, ora_score, ora_l2,
                                largest=True, tol=MARGIN, pivots_given=False, rule=0, text_pivots=False):
    """Replay the candidate's own pivots and assignment against fp64 quantities (one sample).
    ora_score is the oracle's ranking score (L1 norms, or the Euclidean norms for that variant); with
    pivots_given the caller chose the pivots and nothing about their ranking is checked; rule 1 is the
    variant with one threshold for all pivots; text_pivots (with pivots_given, rule 0): pivots outside [0, n_vis) are
    text tokens."""
    if text_pivots and rule == 0:
        assert pivots_given
        return _replay_text_pivots(keys_bits, vis_offset, n_vis, n_keep, pivot_idx, owner, tol)
    if text_pivots:
        assert pivots_given and rule == 1
        return _replay_text_pivots_one_threshold(keys_bits, vis_offset, n_vis, n_keep, pivot_idx, owner, tol)
    P = len(pivot_idx)
    assert len(set(pivot_idx.tolist())) == P, "pivots must be distinct"
    s = ora_score
    sgn = 1.0 if largest else -1.0
    others = np.setdiff1d(np.arange(n_vis), pivot_idx)
    if len(others) and not pivots_given:
        worst_piv = (sgn * s[pivot_idx]).min()
        best_other = (sgn * s[others]).max()
        assert worst_piv >= best_other - tol * abs(best_other), "a non-pivot beats a pivot beyond tolerance"
    ranked = sgn * s[pivot_idx]
    if not pivots_given:
        assert np.all(ranked[:-1] >= ranked[1:] - tol * np.abs(ranked[:-1])), "pivot rank order beyond tolerance"
    dup = _o.similarity(keys_bits, vis_offset, n_vis, pivot_idx, ora_l2)
    kept = np.zeros(n_vis, bool)
    kept[pivot_idx] = True
    assert [int(owner[p]) for p in pivot_idx] == [P + i for i in range(P)], "pivots carry their rank in owner"
    if rule == 1:
        u = dup.max(axis=0)
        mine = np.nonzero((owner >= 0) & (owner < P))[0]
        assert len(mine) == n_keep - P, "retained %d tokens beside the pivots, budget %d" % (len(mine), n_keep - P)
        if len(mine):
            assert np.all(dup[owner[mine], mine] >= u[mine] - tol), "owner is not (nearly) the most similar pivot"
            left = np.ones(n_vis, bool)
            left[pivot_idx] = False
            left[mine] = False
            if left.any():
                assert u[left].min() >= u[mine].max() - tol, \
                    "a token %g below the threshold was left behind" % (u[mine].max() - u[left].min())
        kept[mine] = True
        assert int(kept.sum()) == n_keep
        return kept
    for i, qi in enumerate(quotas(P, n_keep)):
        mine = np.nonzero(owner == i)[0]
        assert len(mine) == qi, "pivot %d retained %d tokens, quota %d" % (i, len(mine), qi)
        if qi == 0:
            continue
        assert not kept[mine].any(), "pivot %d retained a token that was already kept" % i
        eps_i = dup[i, mine].max()
        left = ~kept
        left[mine] = False
        if left.any():
            assert dup[i, left].min() >= eps_i - tol, \
                "pivot %d left behind a token %g below its threshold" % (i, eps_i - dup[i, left].min())
        kept[mine] = True
    assert int(kept.sum()) == n_keep
    assert np.array_equal(np.nonzero(owner >= 0)[0], np.nonzero(kept)[0]), "owner and kept set disagree"
    return kept


def _replay_text_pivots_one_threshold(keys_bits, vis_offset, n_vis, n_keep, pivot_idx, owner, tol):
    """One threshold for all pivots, some of which are text tokens: n_keep - Pv tokens beside the vision pivots."""
    P = len(pivot_idx)
    assert len(set(pivot_idx.tolist())) == P, "pivots must be distinct"
    dup = _o.similarity_any(keys_bits, vis_offset, n_vis, pivot_idx)
    kept = np.zeros(n_vis, bool)
    for i, p in enumerate(pivot_idx.tolist()):
        if 0 <= p < n_vis:
            kept[p] = True
            assert int(owner[p]) == P + i, "vision pivots carry their rank in owner"
    Pv = int(kept.sum())
    assert int((owner >= P).sum()) == Pv, "only vision pivots are marked as pivots"
    u = dup.max(axis=0)
    mine = np.nonzero((owner >= 0) & (owner < P))[0]
    assert len(mine) == n_keep - Pv, "retained %d tokens beside the pivots, budget %d" % (len(mine), n_keep - Pv)
    if len(mine):
        assert np.all(dup[owner[mine], mine] >= u[mine] - tol), "owner is not (nearly) the most similar pivot"
        left = ~kept
        left[mine] = False
        if left.any():
            assert u[left].min() >= u[mine].max() - tol, "a token %g below the threshold was left behind" % (u[mine].max() - u[left].min())
    kept[mine] = True
    assert int(kept.sum()) == n_keep
    return kept


def _replay_text_pivots(keys_bits, vis_offset, n_vis, n_keep, pivot_idx, owner, tol):
    P = len(pivot_idx)
    assert len(set(pivot_idx.tolist())) == P, "pivots must be distinct"
    dup = _o.similarity_any(keys_bits, vis_offset, n_vis, pivot_idx)
    kept = np.zeros(n_vis, bool)
    for i, p in enumerate(pivot_idx.tolist()):
        if 0 <= p < n_vis:
            kept[p] = True
            assert int(owner[p]) == P + i, "vision pivots carry their rank in owner"
    assert int((owner >= P).sum()) == int(kept.sum()), "only vision pivots are marked as pivots"
    for i, qi in enumerate(quotas_any(pivot_idx, n_vis, n_keep)):
        mine = np.nonzero(owner == i)[0]
        assert len(mine) == qi, "pivot %d retained %d tokens, quota %d" % (i, len(mine), qi)
        if qi == 0:
            continue
        assert not kept[mine].any(), "pivot %d retained a token that was already kept" % i
        eps_i = dup[i, mine].max()
        left = ~kept
        left[mine] = False
        if left.any():
            assert dup[i, left].min() >= eps_i - tol, \
                "pivot %d left behind a token %g below its threshold" % (i, eps_i - dup[i, left].min())
        kept[mine] = True
    assert int(kept.sum()) == n_keep
    assert np.array_equal(np.nonzero(owner >= 0)[0], np.nonzero(kept)[0]), "owner and kept set disagree"
    return kept


def check_batch(ora: _o.OracleResult, keys_bits, hidden_bits, vis_offset, n_vis, n_pivot, n_keep,
                out_hidden, out_idx, out_pos, dbg=None, pos_in=None, largest=True, norm_kind=1,
                require_exact_above=MARGIN, pivots_given=False, rule=0, sim_bits=None, text_pivots=False) -> ParityReport:
    """All rules over a batch.  ``dbg`` (optional) holds the candidate's per-step outputs as numpy arrays:
    l1, ssq, pivot_idx, sim, eps, keep, owner.  Without it only the packed outputs are checked.
    ``sim_bits``: the tensor Eq. 7 is evaluated on when it is not the scored one (cosine on the hidden rows)."""
    B = out_idx.shape[0]
    rep = ParityReport()
    margin = ora.margin
    for b in range(B):
        rep.samples += 1
        rep.min_margin = min(rep.min_margin, float(margin[b]))
        pin = None if pos_in is None else pos_in[b]
        check_packed_outputs(None if out_hidden is None else out_hidden[b], out_idx[b], out_pos[b], hidden_bits[b],
                             pin, vis_offset, n_vis, n_keep)
        same = np.array_equal(out_idx[b], ora.out_idx[b])
        rep.exact += int(same)
        if margin[b] > require_exact_above:
            rep.above_margin += 1
            assert same, "sample %d: kept indices differ although the margin is %g" % (b, margin[b])
            if out_hidden is not None and ora.out_hidden is not None:
                assert np.array_equal(out_hidden[b], ora.out_hidden[b])
            assert np.array_equal(out_pos[b], ora.out_pos[b])
        if dbg is None:
            continue
        check_scores(dbg["l1"][b], dbg["ssq"][b], ora.l1[b], ora.l2[b], rep)
        kept_gpu = np.zeros(n_vis, bool)
        kept_gpu[out_idx[b][vis_offset:vis_offset + n_keep] - vis_offset] = True
        assert np.array_equal(dbg["keep"][b].astype(bool), kept_gpu), "keep flags and out_idx disagree"
        assert np.array_equal(dbg["owner"][b] >= 0, kept_gpu), "owner and out_idx disagree"
        same_piv = np.array_equal(dbg["pivot_idx"][b], ora.pivot_idx[b])
        if ora.pivot_gap[b] > require_exact_above:
            assert same_piv, "sample %d: pivots differ although the score gap is %g" % (b, ora.pivot_gap[b])
        if same_piv and ora.dup is not None:
            check_sim(dbg["sim"][b], ora.dup[b], rep)
        if margin[b] > require_exact_above:
            assert np.array_equal(dbg["owner"][b], ora.owner[b])
            Pv_b = int(sum(0 <= int(x) < n_vis for x in dbg["pivot_idx"][b]))
            qs = ([n_keep - Pv_b] * n_pivot if rule == 1 else
                  quotas_any(dbg["pivot_idx"][b], n_vis, n_keep) if text_pivots else quotas(n_pivot, n_keep))
            has = np.array([q > 0 for q in qs])
            e = dbg["eps"][b].astype(np.float64)
            assert np.all(np.isnan(e[~has])) and np.all(np.abs(e[has] - ora.eps[b][has]) <= REL_TOL * np.abs(ora.eps[b][has]) + SIM_ABS_FLOOR)
        else:
            check_valid_under_tolerance(keys_bits[b] if sim_bits is None else sim_bits[b], vis_offset, n_vis, n_keep,
                                        dbg["pivot_idx"][b], dbg["owner"][b],
                                        ora.l1[b] if norm_kind == 1 else ora.l2[b], ora.l2[b], largest=largest,
                                        pivots_given=pivots_given, rule=rule, text_pivots=text_pivots)
            if not same:
                rep.notes.append("sample %d differs below margin %.2e (valid under tolerance)" % (b, margin[b]))
    return rep


def check_union_batch(ora: _o.OracleResult, keys_bits, hidden_bits, vis_offset, n_vis, n_pivot, n_keep,
                      out_hidden, out_idx, out_pos, cu_seqlens, dbg, pos_in=None, largest=True, norm_kind=1,
                      require_exact_above=MARGIN, text_pivots=False) -> ParityReport:
    """Retention with independent pivots: flat outputs, sample b's rows are cu_seqlens[b] .. cu_seqlens[b + 1] - 1.
    Above the margin everything equals the oracle; below it every pivot's picks are replayed against the oracle's
    fp64 similarities with the candidate's own thresholds (dbg["eps"])."""
    B, S = hidden_bits.shape[0], hidden_bits.shape[1]
    rep = ParityReport()
    margin = ora.margin
    cu = np.asarray(cu_seqlens, np.int64)
    assert cu[0] == 0 and len(cu) == B + 1
    for b in range(B):
        rep.samples += 1
        rep.min_margin = min(rep.min_margin, float(margin[b]))
        lo, hi = int(cu[b]), int(cu[b + 1])
        kept = hi - lo - (S - n_vis)
        Pv_b = int(sum(0 <= int(x) < n_vis for x in dbg["pivot_idx"][b]))
        assert Pv_b <= kept <= n_keep, "sample %d keeps %d vision tokens" % (b, kept)
        pin = None if pos_in is None else pos_in[b]
        check_packed_outputs(None if out_hidden is None else out_hidden[lo:hi], out_idx[lo:hi], out_pos[lo:hi],
                             hidden_bits[b], pin, vis_offset, n_vis, kept)
        olo, ohi = int(ora.cu_seqlens[b]), int(ora.cu_seqlens[b + 1])
        same = hi - lo == ohi - olo and np.array_equal(out_idx[lo:hi], ora.out_idx[olo:ohi])
        rep.exact += int(same)
        check_scores(dbg["l1"][b], dbg["ssq"][b], ora.l1[b], ora.l2[b], rep)
        kept_gpu = np.zeros(n_vis, bool)
        kept_gpu[out_idx[lo:hi][vis_offset:vis_offset + kept] - vis_offset] = True
        assert np.array_equal(dbg["keep"][b].astype(bool), kept_gpu), "keep flags and out_idx disagree"
        assert np.array_equal(dbg["owner"][b] >= 0, kept_gpu), "owner and out_idx disagree"
        piv = dbg["pivot_idx"][b]
        same_piv = np.array_equal(piv, ora.pivot_idx[b])
        if ora.pivot_gap[b] > require_exact_above:
            assert same_piv, "sample %d: pivots differ although the score gap is %g" % (b, ora.pivot_gap[b])
        if same_piv and ora.dup is not None:
            check_sim(dbg["sim"][b], ora.dup[b], rep)
        if margin[b] > require_exact_above:
            rep.above_margin += 1
            assert same, "sample %d: kept indices differ although the margin is %g" % (b, margin[b])
            assert np.array_equal(dbg["owner"][b], ora.owner[b])
            continue
        # valid under tolerance: every pivot's own threshold separates what it took from what it left
        assert len(set(piv.tolist())) == n_pivot
        score = ora.l1[b] if norm_kind == 1 else ora.l2[b]
        sgn = 1.0 if largest else -1.0
        others = np.setdiff1d(np.arange(n_vis), piv)
        if len(others) and not text_pivots:   # (text pivots are the caller's: nothing about their ranking to check)
            assert (sgn * score[piv]).min() >= (sgn * score[others]).max() * (1 - MARGIN * np.sign((sgn * score[others]).max()))
        dup = (_o.similarity_any(keys_bits[b], vis_offset, n_vis, piv) if text_pivots else
               _o.similarity(keys_bits[b], vis_offset, n_vis, piv, ora.l2[b]))
        e = dbg["eps"][b].astype(np.float64)
        allowed = np.zeros(n_vis, bool)
        allowed[piv[(piv >= 0) & (piv < n_vis)]] = True
        for i, qi in enumerate(quotas_any(piv, n_vis, n_keep) if text_pivots else quotas(n_pivot, n_keep)):
            if qi == 0:
                assert np.isnan(e[i])
                continue
            below = dup[i, others] < e[i] - MARGIN
            upto = dup[i, others] <= e[i] + MARGIN
            assert below.sum() <= qi <= upto.sum(), "pivot %d: its threshold does not cut off %d tokens" % (i, qi)
            assert kept_gpu[others[below]].all(), "pivot %d left behind a token well below its threshold" % i
            allowed[others[upto]] = True
        assert not (kept_gpu & ~allowed).any(), "a kept token lies above every pivot's threshold"
        if not same:
            rep.notes.append("sample %d differs below margin %.2e (valid under tolerance)" % (b, margin[b]))
    return rep
