"""The parity rules themselves, exercised on the CPU: the oracle's own output (rounded to fp32) must
pass, and mistakes planted into a copy of it must be caught.  CPU only."""
import numpy as np
import pytest

from oracle import parity
from test_oracle_pins import rand_tokens


def _case(oracle, seed=0, B=3, S=80, d=64, vo=7, nv=60, P=4, Kp=21):
    rng = np.random.default_rng(seed)
    hb, _ = rand_tokens(rng, B * S, d)
    kb, _ = rand_tokens(rng, B * S, d)
    hb, kb = hb.reshape(B, S, d), kb.reshape(B, S, d)
    ora = oracle.reduce(hb, kb, vo, nv, P, Kp)
    dbg = {"l1": ora.l1.astype(np.float32), "ssq": (ora.l2 ** 2).astype(np.float32),
           "pivot_idx": ora.pivot_idx.copy(), "sim": ora.dup.astype(np.float32),
           "eps": ora.eps.astype(np.float32), "keep": ora.keep.copy(), "owner": ora.owner.copy()}
    outs = [ora.out_hidden.copy(), ora.out_idx.copy(), ora.out_pos.copy()]
    return ora, kb, hb, (vo, nv, P, Kp), outs, dbg


def _run(ora, kb, hb, shp, outs, dbg, **kw):
    return parity.check_batch(ora, kb, hb, *shp, outs[0], outs[1], outs[2], dbg=dbg, **kw)


def test_oracle_output_passes_its_own_rules(oracle):
    ora, kb, hb, shp, outs, dbg = _case(oracle)
    rep = _run(ora, kb, hb, shp, outs, dbg)
    assert rep.samples == 3 and rep.exact == 3 and rep.max_rel_l1 < 1e-6 and rep.max_abs_sim < 1e-6


def _swap_kept_for_dropped(ora, outs, dbg, b, vo, worst=True):
    """Replace one token retained by pivot 0 with a dropped token (the most similar one if `worst`)."""
    mine = np.nonzero(ora.owner[b] == 0)[0]
    dropped = np.nonzero(ora.keep[b] == 0)[0]
    order = np.argsort(ora.dup[b, 0, dropped])
    new = dropped[order[-1]] if worst else dropped[order[0]]
    old = mine[0]
    dbg["owner"][b, old], dbg["owner"][b, new] = -1, 0
    dbg["keep"][b, old], dbg["keep"][b, new] = 0, 1
    kept = np.nonzero(dbg["keep"][b])[0] + vo
    n_keep = len(kept)
    outs[1][b, vo:vo + n_keep] = kept
    outs[2][b] = outs[1][b]
    return old, new


def test_wrong_retained_token_is_caught(oracle):
    ora, kb, hb, shp, outs, dbg = _case(oracle)
    _swap_kept_for_dropped(ora, outs, dbg, 1, shp[0])
    outs[0][1] = hb[1][outs[1][1]]
    with pytest.raises(AssertionError):
        _run(ora, kb, hb, shp, outs, dbg)
    # even when exactness is not demanded, the replay must reject it
    with pytest.raises(AssertionError, match="left behind"):
        _run(ora, kb, hb, shp, outs, dbg, require_exact_above=np.inf)


def test_near_tie_swap_is_valid_under_tolerance(oracle):
    """Plant an exact-in-direction near-duplicate of the boundary token: either may be retained."""
    rng = np.random.default_rng(5)
    S, d, nv, P, Kp = 40, 256, 40, 1, 9
    kb, vals = rand_tokens(rng, S, d)
    ora0 = oracle.reduce(kb[None], None, 0, nv, P, Kp)
    piv = ora0.pivot_idx[0, 0]
    row = ora0.dup[0, 0].copy()
    row[piv] = np.inf
    order = np.argsort(row)
    last_in, first_out = order[Kp - 2], order[Kp - 1]
    from test_oracle_pins import bf16_bits
    vals[first_out] = vals[last_in] * 0.5            # same direction: dup identical up to rounding
    kb = bf16_bits(vals)
    ora = oracle.reduce(kb[None], None, 0, nv, P, Kp)
    assert ora.retain_gap[0] < 1e-12
    dbg = {"l1": ora.l1.astype(np.float32), "ssq": (ora.l2 ** 2).astype(np.float32), "pivot_idx": ora.pivot_idx.copy(),
           "sim": ora.dup.astype(np.float32), "eps": ora.eps.astype(np.float32), "keep": ora.keep.copy(),
           "owner": ora.owner.copy()}
    outs = [ora.out_hidden.copy(), ora.out_idx.copy(), ora.out_pos.copy()]
    a, b_ = (last_in, first_out) if ora.keep[0, last_in] else (first_out, last_in)
    dbg["owner"][0, a], dbg["owner"][0, b_] = -1, 0
    dbg["keep"][0, a], dbg["keep"][0, b_] = 0, 1
    outs[1][0] = np.nonzero(dbg["keep"][0])[0]
    outs[2][0] = outs[1][0]
    outs[0][0] = kb[outs[1][0]]
    rep = parity.check_batch(ora, kb[None], kb[None], 0, nv, P, Kp, outs[0], outs[1], outs[2], dbg=dbg)
    assert rep.exact == 0 and rep.above_margin == 0 and len(rep.notes) == 1


@pytest.mark.parametrize("what", ["order", "pos", "row", "text", "score", "sim", "pivot"])
def test_planted_output_mistakes_are_caught(oracle, what):
    ora, kb, hb, shp, outs, dbg = _case(oracle, seed=3)
    vo, nv, P, Kp = shp
    if what == "order":
        outs[1][0, vo], outs[1][0, vo + 1] = outs[1][0, vo + 1], outs[1][0, vo]
    elif what == "pos":
        outs[2][2, 5] += 1
    elif what == "row":
        outs[0][1, vo + 2, 7] ^= 1
    elif what == "text":
        outs[1][0, 0] = 1
    elif what == "score":
        dbg["l1"][0, 3] *= 1.02
    elif what == "sim":
        dbg["sim"][1, 2, 11] += 0.02
    elif what == "pivot":
        dbg["pivot_idx"][0, 0], dbg["pivot_idx"][0, 1] = dbg["pivot_idx"][0, 1], dbg["pivot_idx"][0, 0]
    with pytest.raises(AssertionError):
        _run(ora, kb, hb, shp, outs, dbg)
