"""The variants next to the main method, CUDA path vs oracle through the C ABI (needs a B200): pivots chosen
by the caller, retention with one threshold for all pivots, row gather by the packed index list."""
import ctypes

import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import parity  # noqa: E402
from paper_2502_11494_b200 import dart, workloads as W  # noqa: E402
from test_gpu_parity import PATH_IDS, PATHS, _np, gaussian  # noqa: E402

pytestmark = pytest.mark.gpu


def run(keys, hidden, vo, nv, P, Kp, path, pivots=None, rule=dart.DART_RULE_QUOTAS, expect_status=dart.DART_OK,
        on_hidden=False, text=False):
    B, S, d = hidden.shape
    if path in (dart.DART_PATH_FUSED, dart.DART_PATH_TWO_PASS) and (d % 64 or P > 256):
        pytest.skip("the tensor-core paths need d % 64 == 0 and at most 256 pivots")
    ctx = dart.Dart(B, S, d, P, Kp)
    try:
        opts = dart.dart_opts(path=path, rule=rule, cosine_on_hidden=int(on_hidden), text_pivots=int(text),
                              pivots_in=None if pivots is None else pivots.data_ptr())
        res = ctx.reduce(hidden, keys, vo, nv, P, Kp, opts=opts, debug=True)
        torch.cuda.synchronize()
        st = ctx.status()
        detail = dart.dart_status_detail(ctx.handle)
        assert st == expect_status, (st, detail)
    finally:
        ctx.close()
    return _np(res[0]), _np(res[1]), _np(res[2]), {k: _np(v) for k, v in res[3].items()}, detail


def random_pivots(B, nv, P, seed):
    rng = np.random.default_rng(seed)
    return np.stack([rng.permutation(nv)[:P] for _ in range(B)]).astype(np.int32)


SHAPES = [
    (2, 120, 64, 5, 100, 4, 30),
    (3, 333, 264, 17, 301, 7, 60),       # d not a multiple of 64: staged kernels only
    (2, 700, 4096, 40, 576, 8, 64),      # the LLaVA-1.5 shape
    (1, 3000, 512, 12, 2880, 16, 320),   # the LLaVA-NeXT token count
    (2, 700, 512, 10, 640, 128, 320),    # many pivots: large pivot tiles, fewer atoms per stage of the one-pass kernel
    (1, 400, 3584, 0, 333, 40, 100),     # 56 atoms per row, a short last row tile, pivot count not a multiple of 4 x 8
]


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS.get)
@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_pivots_given_by_the_caller(oracle, shape, path):
    B, S, d, vo, nv, P, Kp = shape
    k, h = gaussian(B, S, d, seed=100 + sum(shape))
    piv = random_pivots(B, nv, P, seed=sum(shape))
    oh, oi, op, dbg, _ = run(k, h, vo, nv, P, Kp, path, pivots=torch.from_numpy(piv).cuda())
    kb, hb = W.bits(k), W.bits(h)
    ora = oracle.reduce(hb, kb, vo, nv, P, Kp, pivots_in=piv)
    assert np.array_equal(dbg["pivot_idx"], piv)
    rep = parity.check_batch(ora, kb, hb, vo, nv, P, Kp, oh, oi, op, dbg=dbg, pivots_given=True)
    assert rep.exact >= rep.above_margin and rep.max_abs_sim < 2e-5


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS.get)
def test_own_pivots_given_back_change_nothing(path):
    w = W.LLAVA15_B64.with_(B=5)
    k, h = W.make_batch(w, device="cuda")
    a = run(k, h, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, path)
    piv = torch.from_numpy(a[3]["pivot_idx"]).cuda()
    b = run(k, h, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, path, pivots=piv)
    assert all(np.array_equal(x, y) for x, y in zip(a[:3], b[:3]))
    for n in ("pivot_idx", "keep", "owner"):
        assert np.array_equal(a[3][n], b[3][n])
    # with the pivots given the fused path sums a row's norms in another order (one pass over swizzled tiles)
    for n in ("l1", "ssq", "sim", "eps"):
        assert np.allclose(a[3][n], b[3][n], rtol=1e-5, atol=1e-6, equal_nan=True)


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS.get)
@pytest.mark.parametrize("fault", ["repeated", "negative", "too large"])
def test_bad_pivots_are_reported_not_used(path, fault):
    k, h = gaussian(3, 200, 64, seed=31)
    piv = random_pivots(3, 180, 4, seed=32)
    piv[1, 3] = {"repeated": piv[1, 0], "negative": -1, "too large": 180}[fault]
    *_, detail = run(k, h, 10, 180, 4, 40, path, pivots=torch.from_numpy(piv).cuda(), expect_status=dart.DART_ERR_CHECK)
    assert detail[1][0] == 100 and detail[1][1] == 1 and detail[1][2] == 3   # which check, sample, rank


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS.get)
@pytest.mark.parametrize("shape", SHAPES + [(2, 64, 64, 0, 64, 5, 5), (2, 64, 64, 0, 64, 3, 64)],
                         ids=lambda s: "x".join(map(str, s)))
def test_one_threshold_for_all_pivots(oracle, shape, path):
    B, S, d, vo, nv, P, Kp = shape
    k, h = gaussian(B, S, d, seed=200 + sum(shape))
    oh, oi, op, dbg, _ = run(k, h, vo, nv, P, Kp, path, rule=dart.DART_RULE_GLOBAL)
    kb, hb = W.bits(k), W.bits(h)
    ora = oracle.reduce(hb, kb, vo, nv, P, Kp, rule=1)
    rep = parity.check_batch(ora, kb, hb, vo, nv, P, Kp, oh, oi, op, dbg=dbg, rule=1)
    assert rep.exact >= rep.above_margin and rep.max_abs_sim < 2e-5


def test_one_threshold_on_clustered_tokens(oracle):
    """The LLaVA-1.5-shaped workload (duplicates exist, boundary gaps are small): exact above the margin, valid
    under tolerance below it, and not the same selection as per-pivot quotas."""
    w = W.LLAVA15_B64.with_(B=6)
    k, h = W.make_batch(w, device="cuda")
    oh, oi, op, dbg, _ = run(k, h, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, dart.DART_PATH_AUTO, rule=dart.DART_RULE_GLOBAL)
    kb, hb = W.bits(k), W.bits(h)
    ora = oracle.reduce(hb, kb, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, rule=1)
    rep = parity.check_batch(ora, kb, hb, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, oh, oi, op, dbg=dbg, rule=1)
    assert rep.exact >= rep.above_margin and rep.exact >= 5, rep.notes
    quota = run(k, h, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, dart.DART_PATH_AUTO)
    assert not np.array_equal(quota[1], oi)


def test_both_variants_together(oracle):
    B, S, d, vo, nv, P, Kp = 2, 300, 128, 20, 260, 6, 50
    k, h = gaussian(B, S, d, seed=41)
    piv = random_pivots(B, nv, P, seed=42)
    oh, oi, op, dbg, _ = run(k, h, vo, nv, P, Kp, dart.DART_PATH_AUTO, pivots=torch.from_numpy(piv).cuda(),
                             rule=dart.DART_RULE_GLOBAL)
    kb, hb = W.bits(k), W.bits(h)
    ora = oracle.reduce(hb, kb, vo, nv, P, Kp, pivots_in=piv, rule=1)
    rep = parity.check_batch(ora, kb, hb, vo, nv, P, Kp, oh, oi, op, dbg=dbg, pivots_given=True, rule=1)
    assert rep.exact >= rep.above_margin


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS.get)
@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_cosine_on_the_hidden_rows(oracle, shape, path):
    """Pivots ranked by the key rows, Eq. 7 evaluated on the hidden rows."""
    B, S, d, vo, nv, P, Kp = shape
    k, h = gaussian(B, S, d, seed=300 + sum(shape))
    oh, oi, op, dbg, _ = run(k, h, vo, nv, P, Kp, path, on_hidden=True)
    kb, hb = W.bits(k), W.bits(h)
    ora = oracle.reduce(hb, kb, vo, nv, P, Kp, cosine_on_hidden=True)
    rep = parity.check_batch(ora, kb, hb, vo, nv, P, Kp, oh, oi, op, dbg=dbg, sim_bits=hb)
    assert rep.exact >= rep.above_margin and rep.max_abs_sim < 2e-5 and rep.max_rel_l1 < 5e-5 and rep.max_rel_l2 < 5e-5


def test_cosine_on_hidden_with_given_pivots_and_one_threshold(oracle):
    B, S, d, vo, nv, P, Kp = 2, 400, 256, 10, 380, 8, 70
    k, h = gaussian(B, S, d, seed=51)
    piv = random_pivots(B, nv, P, seed=52)
    oh, oi, op, dbg, _ = run(k, h, vo, nv, P, Kp, dart.DART_PATH_AUTO, pivots=torch.from_numpy(piv).cuda(),
                             rule=dart.DART_RULE_GLOBAL, on_hidden=True)
    kb, hb = W.bits(k), W.bits(h)
    ora = oracle.reduce(hb, kb, vo, nv, P, Kp, pivots_in=piv, rule=1, cosine_on_hidden=True)
    rep = parity.check_batch(ora, kb, hb, vo, nv, P, Kp, oh, oi, op, dbg=dbg, pivots_given=True, rule=1, sim_bits=hb)
    assert rep.exact >= rep.above_margin


def test_cosine_on_hidden_needs_the_l1_score():
    k, h = gaussian(1, 64, 64, seed=53)
    ctx = dart.Dart(1, 64, 64, 2, 8)
    with pytest.raises(dart.DartError) as e:
        ctx.reduce(h, k, 0, 64, 2, 8, opts=dart.dart_opts(norm_kind=2, cosine_on_hidden=1))
    assert e.value.code == dart.DART_ERR_UNSUPPORTED
    ctx.close()


def test_unknown_rule_is_rejected():
    k, h = gaussian(1, 64, 64, seed=43)
    ctx = dart.Dart(1, 64, 64, 2, 8)
    with pytest.raises(dart.DartError) as e:
        ctx.reduce(h, k, 0, 64, 2, 8, opts=dart.dart_opts(rule=7))
    assert e.value.code == dart.DART_ERR_UNSUPPORTED
    ctx.close()


# ----------------------------------------------------------------------------- rows gathered by the packed list

def _gather(src, idx, out=None, S_out=None):
    B, S, w = src.shape
    S_out = idx.shape[1] if S_out is None else S_out
    out = torch.empty((B, S_out, w), dtype=src.dtype, device="cuda") if out is None else out
    P = lambda t: ctypes.c_void_p(t.data_ptr())  # noqa: E731
    rc = dart.dart_gather_rows(P(src), P(idx), B, S, S_out, w * src.element_size(), P(out), 0,
                               ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
    return rc, out


@pytest.mark.parametrize("B,S,w,S_out", [(1, 16, 8, 16), (3, 700, 4096, 164), (2, 3000, 3584, 420), (5, 90, 24, 1)])
def test_gather_rows_against_the_oracle(oracle, B, S, w, S_out):
    g = torch.Generator(device="cuda").manual_seed(B + S + w)
    src = torch.randint(-32768, 32767, (B, S, w), generator=g, device="cuda", dtype=torch.int16)
    rng = np.random.default_rng(S_out)
    idx = np.stack([np.sort(rng.permutation(S)[:S_out]) for _ in range(B)]).astype(np.int32)
    rc, out = _gather(src, torch.from_numpy(idx).cuda())
    torch.cuda.synchronize()
    assert rc == dart.DART_OK
    assert np.array_equal(out.cpu().numpy().view(np.uint16), oracle.gather_rows(src.cpu().numpy().view(np.uint16), idx))


def test_gather_rows_packs_a_kv_cache_like_the_hidden_states(oracle):
    """The packed list of a reduction, applied to the key states, gives the key rows of the retained tokens."""
    w = W.LLAVA15_B64.with_(B=3)
    k, h = W.make_batch(w, device="cuda")
    ctx = dart.Dart(w.B, w.S, w.d, w.n_pivot, w.n_keep)
    oh, oi, op = ctx.reduce(h, k, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep)
    rc_h, again = _gather(h, oi)
    rc_k, packed_k = _gather(k, oi)
    torch.cuda.synchronize()
    assert ctx.status() == dart.DART_OK and rc_h == dart.DART_OK and rc_k == dart.DART_OK
    ctx.close()
    assert torch.equal(again.view(torch.int16), oh.view(torch.int16))
    assert np.array_equal(W.bits(packed_k), oracle.gather_rows(W.bits(k), oi.cpu().numpy()))


def test_gather_rows_argument_checks():
    src = torch.zeros((2, 10, 8), dtype=torch.int16, device="cuda")
    idx = torch.zeros((2, 4), dtype=torch.int32, device="cuda")
    P = lambda t: ctypes.c_void_p(t.data_ptr())  # noqa: E731
    out = torch.empty((2, 4, 8), dtype=torch.int16, device="cuda")
    assert dart.dart_gather_rows(None, P(idx), 2, 10, 4, 16, P(out), 0, None) == dart.DART_ERR_NULL
    assert dart.dart_gather_rows(P(src), P(idx), 2, 10, 4, 24, P(out), 0, None) == dart.DART_ERR_BAD_SHAPE   # not a multiple of 16
    assert dart.dart_gather_rows(P(src), P(idx), 0, 10, 4, 16, P(out), 0, None) == dart.DART_ERR_BAD_SHAPE
    assert dart.dart_gather_rows(ctypes.c_void_p(src.data_ptr() + 2), P(idx), 2, 10, 4, 16, P(out), 0, None) == dart.DART_ERR_ALIGN
    assert dart.dart_gather_rows(P(src), P(idx), 2, 10, 4, 16, P(src), 0, None) == dart.DART_ERR_ALIAS
    assert dart.dart_gather_rows(P(src), P(idx), 2, 10, 4, 16, P(out), 0, None) == dart.DART_OK
    torch.cuda.synchronize()


# ----------------------------------------------------------------------------- pivots taken from the text tokens (Sec. 5.4)

def text_pivots(B, vo, nv, S, P, seed, n_text=None):
    """Distinct pivots anywhere in the sample, relative to the vision block; at least one text token when there is one."""
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(B):
        p = rng.permutation(S)[:P] - vo
        text = np.concatenate([np.arange(-vo, 0), np.arange(nv, S - vo)])
        if len(text) and not ((p < 0) | (p >= nv)).any():
            p[rng.integers(P)] = rng.choice(text)
        if n_text == "all":
            p = rng.permutation(text)[:P]
        out.append(p)
    return np.stack(out).astype(np.int32)


TEXT_SHAPES = [
    (2, 120, 64, 9, 100, 4, 30),
    (2, 700, 4096, 40, 576, 8, 64),      # the LLaVA-1.5 shape
    (1, 3000, 512, 60, 2880, 16, 320),   # the LLaVA-NeXT token count
    (2, 700, 512, 30, 640, 128, 320),    # the compact pivot tile
    (1, 400, 3584, 0, 333, 40, 100),     # text after the vision block only
    (3, 96, 64, 20, 60, 6, 6),           # n_keep = P: text pivots free budget for their own picks
]


@pytest.mark.parametrize("path", [dart.DART_PATH_AUTO, dart.DART_PATH_FUSED, dart.DART_PATH_STAGED], ids=lambda p: PATH_IDS.get(p, "auto"))
@pytest.mark.parametrize("retention", [dart.DART_RETAIN_SERIAL, dart.DART_RETAIN_LISTS, dart.DART_RETAIN_BANDS], ids=["serial", "lists", "bands"])
@pytest.mark.parametrize("shape", TEXT_SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_pivots_from_the_text_tokens(oracle, shape, retention, path):
    B, S, d, vo, nv, P, Kp = shape
    k, h = gaussian(B, S, d, seed=400 + sum(shape))
    piv = text_pivots(B, vo, nv, S, P, seed=sum(shape))
    ctx = dart.Dart(B, S, d, P, Kp)
    try:
        piv_t = torch.from_numpy(piv).cuda()
        res = ctx.reduce(h, k, vo, nv, P, Kp, debug=True,
                         opts=dart.dart_opts(path=path, retention=retention, text_pivots=1, pivots_in=piv_t.data_ptr()))
        torch.cuda.synchronize()
        assert ctx.status() == dart.DART_OK, dart.dart_status_detail(ctx.handle)
    finally:
        ctx.close()
    oh, oi, op = _np(res[0]), _np(res[1]), _np(res[2])
    dbg = {n: _np(v) for n, v in res[3].items()}
    kb, hb = W.bits(k), W.bits(h)
    ora = oracle.reduce(hb, kb, vo, nv, P, Kp, pivots_in=piv, text_pivots=True)
    assert np.array_equal(dbg["pivot_idx"], piv)
    rep = parity.check_batch(ora, kb, hb, vo, nv, P, Kp, oh, oi, op, dbg=dbg, pivots_given=True, text_pivots=True)
    assert rep.exact >= rep.above_margin and rep.max_abs_sim < 2e-5


def test_text_pivots_only(oracle):
    """Every pivot a text token: nothing is kept but the pivots' picks, n_keep of them."""
    B, S, d, vo, nv, P, Kp = 2, 300, 128, 40, 200, 8, 50
    k, h = gaussian(B, S, d, seed=61)
    piv = text_pivots(B, vo, nv, S, P, seed=62, n_text="all")
    oh, oi, op, dbg, _ = run(k, h, vo, nv, P, Kp, dart.DART_PATH_AUTO, pivots=torch.from_numpy(piv).cuda(), text=True)
    kb, hb = W.bits(k), W.bits(h)
    ora = oracle.reduce(hb, kb, vo, nv, P, Kp, pivots_in=piv, text_pivots=True)
    rep = parity.check_batch(ora, kb, hb, vo, nv, P, Kp, oh, oi, op, dbg=dbg, pivots_given=True, text_pivots=True)
    assert rep.exact >= rep.above_margin and (dbg["owner"] < P).all()


def test_vision_pivots_with_the_text_option_change_nothing():
    k, h = gaussian(2, 200, 64, seed=63)
    piv = torch.from_numpy(random_pivots(2, 150, 5, seed=64)).cuda()
    a = run(k, h, 20, 150, 5, 40, dart.DART_PATH_AUTO, pivots=piv)
    b = run(k, h, 20, 150, 5, 40, dart.DART_PATH_AUTO, pivots=piv, text=True)
    assert all(np.array_equal(x, y) for x, y in zip(a[:3], b[:3]))
    assert all(np.array_equal(a[3][n], b[3][n], equal_nan=True) for n in a[3])


@pytest.mark.parametrize("fault", ["repeated text", "before the sample", "after the sample"])
def test_bad_text_pivots_are_reported_not_used(fault):
    k, h = gaussian(3, 200, 64, seed=65)
    piv = random_pivots(3, 150, 4, seed=66)
    piv[0, 1] = -7
    piv[1, 0] = 160
    piv[1, 3] = {"repeated text": 160, "before the sample": -21, "after the sample": 180}[fault]
    *_, detail = run(k, h, 20, 150, 4, 40, dart.DART_PATH_AUTO, pivots=torch.from_numpy(piv).cuda(), text=True,
                     expect_status=dart.DART_ERR_CHECK)
    assert detail[1][0] == 100 and detail[1][1] == 1 and detail[1][2] in (0, 3)


def test_text_pivots_need_given_pivots():
    k, h = gaussian(1, 64, 64, seed=67)
    ctx = dart.Dart(1, 64, 64, 2, 8)
    with pytest.raises(dart.DartError) as e:
        ctx.reduce(h, k, 4, 50, 2, 8, opts=dart.dart_opts(text_pivots=1))
    assert e.value.code == dart.DART_ERR_UNSUPPORTED
    ctx.close()


@pytest.mark.parametrize("path", [dart.DART_PATH_STAGED, dart.DART_PATH_FUSED], ids=PATH_IDS.get)
@pytest.mark.parametrize("shape", TEXT_SHAPES[:3] + [(3, 333, 264, 17, 301, 7, 60)], ids=lambda s: "x".join(map(str, s)))
def test_text_pivots_under_one_threshold(oracle, shape, path):
    B, S, d, vo, nv, P, Kp = shape
    k, h = gaussian(B, S, d, seed=440 + sum(shape))
    piv = text_pivots(B, vo, nv, S, P, seed=1 + sum(shape))
    oh, oi, op, dbg, _ = run(k, h, vo, nv, P, Kp, path, pivots=torch.from_numpy(piv).cuda(), rule=dart.DART_RULE_GLOBAL, text=True)
    kb, hb = W.bits(k), W.bits(h)
    ora = oracle.reduce(hb, kb, vo, nv, P, Kp, pivots_in=piv, text_pivots=True, rule=1)
    rep = parity.check_batch(ora, kb, hb, vo, nv, P, Kp, oh, oi, op, dbg=dbg, pivots_given=True, text_pivots=True, rule=1)
    assert rep.exact >= rep.above_margin and rep.max_abs_sim < 2e-5


@pytest.mark.parametrize("path", [dart.DART_PATH_STAGED, dart.DART_PATH_FUSED], ids=PATH_IDS.get)
@pytest.mark.parametrize("shape", TEXT_SHAPES[:3] + [(3, 333, 264, 17, 301, 7, 60)], ids=lambda s: "x".join(map(str, s)))
def test_text_pivots_with_independent_pivots(oracle, shape, path):
    B, S, d, vo, nv, P, Kp = shape
    k, h = gaussian(B, S, d, seed=470 + sum(shape))
    piv = text_pivots(B, vo, nv, S, P, seed=2 + sum(shape))
    oh, oi, op, dbg, cu = run_union(k, h, vo, nv, P, Kp, path, pivots=torch.from_numpy(piv).cuda(), text=True)
    kb, hb = W.bits(k), W.bits(h)
    ora = oracle.reduce(hb, kb, vo, nv, P, Kp, pivots_in=piv, text_pivots=True, rule=2)
    rep = parity.check_union_batch(ora, kb, hb, vo, nv, P, Kp, oh, oi, op, cu, dbg, text_pivots=True)
    assert rep.exact >= rep.above_margin and rep.max_abs_sim < 2e-5


# ----------------------------------------------------------------------------- pivots chosen inside the library from other sources

SOURCE_SHAPES = [
    (2, 120, 64, 9, 100, 4, 30),
    (3, 333, 264, 17, 301, 7, 60),       # d not a multiple of 64: plain kernels only
    (2, 700, 4096, 40, 576, 8, 64),      # the LLaVA-1.5 shape: 4 visual and 4 text pivots
    (1, 3000, 512, 60, 2880, 16, 320),
    (1, 400, 3584, 0, 333, 40, 100),     # text after the vision block only
]


def run_source(keys, hidden, vo, nv, P, Kp, path, source, n_text=0, seed=0, base=0, rule=dart.DART_RULE_QUOTAS, norm_kind=0, smallest=0):
    B, S, d = hidden.shape
    if path in (dart.DART_PATH_FUSED, dart.DART_PATH_TWO_PASS) and d % 64:
        pytest.skip("the tensor-core paths need d % 64 == 0")
    ctx = dart.Dart(B, S, d, P, Kp)
    try:
        res = ctx.reduce(hidden, keys, vo, nv, P, Kp, debug=True,
                         opts=dart.dart_opts(path=path, rule=rule, pivot_source=source, n_text_pivots=n_text, seed=seed, sample_base=base,
                                             norm_kind=norm_kind, pivot_smallest=smallest))
        torch.cuda.synchronize()
        assert ctx.status() == dart.DART_OK, dart.dart_status_detail(ctx.handle)
    finally:
        ctx.close()
    return _np(res[0]), _np(res[1]), _np(res[2]), {n: _np(v) for n, v in res[3].items()}


@pytest.mark.parametrize("path", [dart.DART_PATH_AUTO, dart.DART_PATH_STAGED, dart.DART_PATH_FUSED], ids=lambda p: PATH_IDS.get(p, "auto"))
@pytest.mark.parametrize("shape", SOURCE_SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_pivots_from_both_modalities(oracle, shape, path):
    """Half of the pivots are the text tokens of largest K-norm, half the vision tokens (the ablation's 4 + 4)."""
    B, S, d, vo, nv, P, Kp = shape
    k, h = gaussian(B, S, d, seed=520 + sum(shape))
    Pt = min(P // 2, S - nv)
    oh, oi, op, dbg = run_source(k, h, vo, nv, P, Kp, path, dart.DART_PIVOTS_MIXED, n_text=Pt)
    kb, hb = W.bits(k), W.bits(h)
    ora = oracle.reduce(hb, kb, vo, nv, P, Kp, pivot_source=1, n_text_pivots=Pt)
    assert np.array_equal(dbg["pivot_idx"], ora.pivot_idx)       # Gaussian scores: no near-ties at these seeds
    assert ((ora.pivot_idx[:, P - Pt:] < 0) | (ora.pivot_idx[:, P - Pt:] >= nv)).all()
    rep = parity.check_batch(ora, kb, hb, vo, nv, P, Kp, oh, oi, op, dbg=dbg, pivots_given=True, text_pivots=True)
    assert rep.samples == B and rep.max_abs_sim < 2e-5


@pytest.mark.parametrize("norm_kind,smallest,rule", [(2, 0, dart.DART_RULE_QUOTAS), (1, 1, dart.DART_RULE_GLOBAL)])
def test_pivots_from_both_modalities_variants(oracle, norm_kind, smallest, rule):
    B, S, d, vo, nv, P, Kp = 2, 300, 128, 30, 220, 6, 40
    k, h = gaussian(B, S, d, seed=530)
    oh, oi, op, dbg = run_source(k, h, vo, nv, P, Kp, dart.DART_PATH_AUTO, dart.DART_PIVOTS_MIXED, n_text=2, rule=rule,
                                 norm_kind=norm_kind, smallest=smallest)
    kb, hb = W.bits(k), W.bits(h)
    ora = oracle.reduce(hb, kb, vo, nv, P, Kp, pivot_source=1, n_text_pivots=2, rule=rule, norm_kind=norm_kind, largest=not smallest)
    assert np.array_equal(dbg["pivot_idx"], ora.pivot_idx)
    rep = parity.check_batch(ora, kb, hb, vo, nv, P, Kp, oh, oi, op, dbg=dbg, pivots_given=True, text_pivots=True, rule=rule,
                             norm_kind=norm_kind, largest=not smallest)
    assert rep.samples == B


@pytest.mark.parametrize("path", [dart.DART_PATH_AUTO, dart.DART_PATH_STAGED, dart.DART_PATH_FUSED], ids=lambda p: PATH_IDS.get(p, "auto"))
@pytest.mark.parametrize("shape", SOURCE_SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_random_pivots_from_a_seed(oracle, shape, path):
    """The tickets are integers: the pivots equal the oracle's bit for bit, on every path and every run."""
    B, S, d, vo, nv, P, Kp = shape
    k, h = gaussian(B, S, d, seed=560 + sum(shape))
    oh, oi, op, dbg = run_source(k, h, vo, nv, P, Kp, path, dart.DART_PIVOTS_RANDOM, seed=20240229 + sum(shape))
    kb, hb = W.bits(k), W.bits(h)
    ora = oracle.reduce(hb, kb, vo, nv, P, Kp, pivot_source=2, seed=20240229 + sum(shape))
    assert np.array_equal(dbg["pivot_idx"], ora.pivot_idx)
    rep = parity.check_batch(ora, kb, hb, vo, nv, P, Kp, oh, oi, op, dbg=dbg, pivots_given=True)
    assert rep.exact >= rep.above_margin and rep.max_abs_sim < 2e-5


def test_random_pivots_of_a_split_batch_are_those_of_the_whole_batch(oracle):
    B, S, d, vo, nv, P, Kp = 5, 200, 64, 10, 170, 5, 30
    k, h = gaussian(B, S, d, seed=590)
    whole = run_source(k, h, vo, nv, P, Kp, dart.DART_PATH_AUTO, dart.DART_PIVOTS_RANDOM, seed=7)[3]["pivot_idx"]
    tail = run_source(k[3:].contiguous(), h[3:].contiguous(), vo, nv, P, Kp, dart.DART_PATH_AUTO, dart.DART_PIVOTS_RANDOM, seed=7, base=3)[3]["pivot_idx"]
    assert np.array_equal(whole[3:], tail)
    assert np.array_equal(whole, np.stack([oracle.pivots_random(7, b, nv, P) for b in range(B)]))


def test_pivot_sources_say_what_they_do_not_take():
    k, h = gaussian(1, 64, 64, seed=591)
    piv = torch.zeros(1, 2, dtype=torch.int32, device="cuda")
    ctx = dart.Dart(1, 64, 64, 2, 8)
    for o, code in [(dart.dart_opts(pivot_source=3), dart.DART_ERR_UNSUPPORTED),
                    (dart.dart_opts(pivot_source=1, pivots_in=piv.data_ptr()), dart.DART_ERR_UNSUPPORTED),
                    (dart.dart_opts(pivot_source=2, path=dart.DART_PATH_RESIDENT), dart.DART_ERR_UNSUPPORTED),
                    (dart.dart_opts(pivot_source=1, n_text_pivots=3), dart.DART_ERR_BAD_SHAPE),          # more than n_pivot
                    (dart.dart_opts(pivot_source=2, sample_base=-1), dart.DART_ERR_BAD_SHAPE)]:
        with pytest.raises(dart.DartError) as e:
            ctx.reduce(h, k, 4, 50, 2, 8, opts=o)
        assert e.value.code == code
    ctx.close()


@pytest.mark.parametrize("seed", range(16))
def test_text_pivots_random_shapes(oracle, seed):
    rng = np.random.default_rng(2000 + seed)
    d = int(rng.choice([64, 128, 192, 320, 512, 1024]))
    nv = int(rng.integers(1, 500))
    vo, after = int(rng.integers(0, 40)), int(rng.integers(0, 40))
    S = vo + nv + after
    P = int(rng.integers(1, min(S, nv, 40) + 1))
    Kp = int(rng.integers(P, nv + 1))
    B = int(rng.integers(1, 4))
    k, h = gaussian(B, S, d, seed=500 + seed)
    piv = text_pivots(B, vo, nv, S, P, seed=seed)
    ctx = dart.Dart(B, S, d, P, Kp)
    try:
        piv_t = torch.from_numpy(piv).cuda()
        res = ctx.reduce(h, k, vo, nv, P, Kp, debug=True,
                         opts=dart.dart_opts(retention=int(rng.integers(0, 5)), text_pivots=1, pivots_in=piv_t.data_ptr()))
        torch.cuda.synchronize()
        assert ctx.status() == dart.DART_OK, dart.dart_status_detail(ctx.handle)
    finally:
        ctx.close()
    oh, oi, op = _np(res[0]), _np(res[1]), _np(res[2])
    dbg = {n: _np(v) for n, v in res[3].items()}
    kb, hb = W.bits(k), W.bits(h)
    ora = oracle.reduce(hb, kb, vo, nv, P, Kp, pivots_in=piv, text_pivots=True)
    rep = parity.check_batch(ora, kb, hb, vo, nv, P, Kp, oh, oi, op, dbg=dbg, pivots_given=True, text_pivots=True)
    assert rep.exact >= rep.above_margin and rep.max_abs_sim < 2e-5, (B, S, d, vo, nv, P, Kp)


# ----------------------------------------------------------------------------- independent pivots, variable-length outputs

def run_union(keys, hidden, vo, nv, P, Kp, path, pivots=None, text=False):
    B, S, d = hidden.shape
    if path in (dart.DART_PATH_FUSED, dart.DART_PATH_TWO_PASS) and (d % 64 or P > 256):
        pytest.skip("the tensor-core paths need d % 64 == 0 and at most 256 pivots")
    S_out = S - nv + Kp
    out = (torch.zeros((B * S_out, d), dtype=torch.bfloat16, device="cuda"),
           torch.full((B * S_out,), -1, dtype=torch.int32, device="cuda"),
           torch.full((B * S_out,), -1, dtype=torch.int64, device="cuda"))
    cu = torch.full((B + 1,), -7, dtype=torch.int32, device="cuda")
    ctx = dart.Dart(B, S, d, P, Kp)
    try:
        res = ctx.reduce(hidden, keys, vo, nv, P, Kp, out=out, debug=True,
                         opts=dart.dart_opts(path=path, rule=dart.DART_RULE_UNION, cu_seqlens=cu.data_ptr(), text_pivots=int(text),
                                             pivots_in=None if pivots is None else pivots.data_ptr()))
        torch.cuda.synchronize()
        assert ctx.status() == dart.DART_OK, dart.dart_status_detail(ctx.handle)
    finally:
        ctx.close()
    return _np(res[0]), _np(res[1]), _np(res[2]), {k: _np(v) for k, v in res[3].items()}, _np(cu)


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS.get)
@pytest.mark.parametrize("shape", SHAPES + [(2, 64, 64, 0, 64, 5, 5), (2, 64, 64, 0, 64, 3, 64), (300, 40, 64, 3, 30, 2, 9)],
                         ids=lambda s: "x".join(map(str, s)))
def test_independent_pivots_give_variable_lengths(oracle, shape, path):
    B, S, d, vo, nv, P, Kp = shape
    k, h = gaussian(B, S, d, seed=600 + sum(shape))
    oh, oi, op, dbg, cu = run_union(k, h, vo, nv, P, Kp, path)
    kb, hb = W.bits(k), W.bits(h)
    ora = oracle.reduce(hb, kb, vo, nv, P, Kp, rule=2)
    rep = parity.check_union_batch(ora, kb, hb, vo, nv, P, Kp, oh, oi, op, cu, dbg)
    assert rep.exact >= rep.above_margin and rep.max_abs_sim < 2e-5
    assert (oi[cu[-1]:] == -1).all() and (op[cu[-1]:] == -1).all() and not oh[cu[-1]:].any()   # nothing beyond the packed rows


def test_independent_pivots_on_clustered_tokens_keep_fewer_than_the_budget(oracle):
    """Duplicates make several pivots pick the same far-away tokens: the union falls short of n_keep."""
    w = W.LLAVA15_B64.with_(B=6)
    k, h = W.make_batch(w, device="cuda")
    oh, oi, op, dbg, cu = run_union(k, h, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, dart.DART_PATH_AUTO)
    kb, hb = W.bits(k), W.bits(h)
    ora = oracle.reduce(hb, kb, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, rule=2)
    rep = parity.check_union_batch(ora, kb, hb, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, oh, oi, op, cu, dbg)
    assert rep.exact >= rep.above_margin and rep.exact >= 5, rep.notes
    kept = np.diff(cu) - (w.S - w.n_vis)
    assert (kept <= w.n_keep).all() and (kept < w.n_keep).any()


@pytest.mark.parametrize("path", [dart.DART_PATH_STAGED, dart.DART_PATH_TWO_PASS], ids=PATH_IDS.get)
def test_independent_pivots_on_a_sample_beyond_48k_tokens(oracle, path):
    """The keep flags of a sample live in dynamic shared memory: past 48 KB the kernels need the opt-in limit."""
    B, S, d, vo, nv, P, Kp = 1, 50300, 64, 20, 50250, 3, 400
    k, h = gaussian(B, S, d, seed=77)
    oh, oi, op, dbg, cu = run_union(k, h, vo, nv, P, Kp, path)
    kb, hb = W.bits(k), W.bits(h)
    ora = oracle.reduce(hb, kb, vo, nv, P, Kp, rule=2)
    rep = parity.check_union_batch(ora, kb, hb, vo, nv, P, Kp, oh, oi, op, cu, dbg)
    assert rep.exact >= rep.above_margin and rep.max_abs_sim < 2e-5


def test_independent_pivots_need_cu_seqlens():
    k, h = gaussian(1, 64, 64, seed=68)
    ctx = dart.Dart(1, 64, 64, 2, 8)
    with pytest.raises(dart.DartError) as e:
        ctx.reduce(h, k, 0, 64, 2, 8, opts=dart.dart_opts(rule=dart.DART_RULE_UNION))
    assert e.value.code == dart.DART_ERR_NULL
    ctx.close()


@pytest.mark.parametrize("seed", range(12))
def test_independent_pivots_random_shapes(oracle, seed):
    rng = np.random.default_rng(3000 + seed)
    d = int(rng.choice([8, 24, 64, 128, 320, 1024]))
    nv = int(rng.integers(1, 600))
    vo, after = int(rng.integers(0, 40)), int(rng.integers(0, 40))
    P = int(rng.integers(1, min(nv, 24) + 1))
    Kp = int(rng.integers(P, nv + 1))
    B = int(rng.integers(1, 6))
    path = int(rng.choice(PATHS)) if d % 64 == 0 else dart.DART_PATH_STAGED
    k, h = gaussian(B, vo + nv + after, d, seed=800 + seed)
    oh, oi, op, dbg, cu = run_union(k, h, vo, nv, P, Kp, path)
    kb, hb = W.bits(k), W.bits(h)
    ora = oracle.reduce(hb, kb, vo, nv, P, Kp, rule=2)
    rep = parity.check_union_batch(ora, kb, hb, vo, nv, P, Kp, oh, oi, op, cu, dbg)
    assert rep.exact >= rep.above_margin and rep.max_abs_sim < 2e-5, (B, vo, nv, after, d, P, Kp, path)


# ----------------------------------------------------------------------------- the paper's other shapes (appendix)

@pytest.mark.parametrize("path", [dart.DART_PATH_AUTO] + PATHS, ids=lambda p: PATH_IDS.get(p, "auto"))
def test_vision_language_action_shape(oracle, path):
    """256 image tokens -> 56, 8 pivots, per control step of a batch of environments."""
    w = W.VLA_B16.with_(B=4)
    k, h = W.make_batch(w, device="cuda")
    oh, oi, op, dbg, _ = run(k, h, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, path)
    kb, hb = W.bits(k), W.bits(h)
    ora = oracle.reduce(hb, kb, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep)
    rep = parity.check_batch(ora, kb, hb, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, oh, oi, op, dbg=dbg)
    assert rep.exact >= rep.above_margin and rep.exact >= 3 and rep.max_abs_sim < 2e-5, rep.notes


@pytest.mark.parametrize("keep", W.AUDIO_KEEP)
def test_audio_token_shape(oracle, keep):
    """1500 audio tokens of width 3072 reduced by 20, 30 and 50 %."""
    w = W.AUDIO_B8.with_(B=2, n_keep=keep)
    k, h = W.make_batch(w, device="cuda")
    oh, oi, op, dbg, _ = run(k, h, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, dart.DART_PATH_AUTO)
    kb, hb = W.bits(k), W.bits(h)
    ora = oracle.reduce(hb, kb, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep)
    rep = parity.check_batch(ora, kb, hb, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, oh, oi, op, dbg=dbg)
    assert rep.exact >= rep.above_margin and rep.max_abs_sim < 2e-5, rep.notes
