"""CUDA path vs oracle, element by element, through the C ABI (needs a B200)."""
import ctypes

import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import parity  # noqa: E402
from paper_2502_11494_b200 import dart, workloads as W  # noqa: E402

pytestmark = pytest.mark.gpu

PATHS = [dart.DART_PATH_STAGED, dart.DART_PATH_FUSED, dart.DART_PATH_TWO_PASS]
PATH_IDS = {dart.DART_PATH_STAGED: "staged", dart.DART_PATH_FUSED: "fused", dart.DART_PATH_TWO_PASS: "two-pass"}


def _np(t):
    t = t.detach().cpu()
    return W.bits(t) if t.dtype == torch.bfloat16 else t.numpy()


def run_gpu(keys, hidden, vo, nv, P, Kp, pos_in=None, path=dart.DART_PATH_AUTO, norm_kind=0, smallest=0, debug=True,
            sweep_lag=0, retention=dart.DART_RETAIN_AUTO):
    B, S, d = hidden.shape
    if path in (dart.DART_PATH_FUSED, dart.DART_PATH_TWO_PASS) and (d % 64 or P > 256):
        pytest.skip("the tensor-core paths need d % 64 == 0 and at most 256 pivots")
    ctx = dart.Dart(B, S, d, P, Kp)
    try:
        opts = dart.dart_opts(norm_kind, smallest, path, 0, sweep_lag, 0, retention)
        res = ctx.reduce(hidden, keys, vo, nv, P, Kp, pos_in=pos_in, opts=opts, debug=debug)
        torch.cuda.synchronize()
        st = ctx.status()
        assert st == dart.DART_OK, (st, dart.dart_status_detail(ctx.handle))
    finally:
        ctx.close()
    oh, oi, op = _np(res[0]), _np(res[1]), _np(res[2])
    dbg = {k: _np(v) for k, v in res[3].items()} if debug else None
    return oh, oi, op, dbg


def compare(oracle, keys, hidden, vo, nv, P, Kp, pos_in=None, path=dart.DART_PATH_AUTO, norm_kind=1, smallest=0,
            debug=True, samples=None):
    """Run the CUDA path on the whole batch and the oracle on `samples` (default: all)."""
    oh, oi, op, dbg = run_gpu(keys, hidden, vo, nv, P, Kp, pos_in, path, norm_kind, smallest, debug)
    sel = list(range(hidden.shape[0])) if samples is None else list(samples)
    kb = W.bits(hidden[sel] if keys is None else keys[sel])
    hb = W.bits(hidden[sel])
    pin = None if pos_in is None else pos_in[sel].cpu().numpy()
    ora = oracle.reduce(hb, None if keys is None else kb, vo, nv, P, Kp, pos_in=pin, norm_kind=norm_kind,
                        largest=not smallest)
    d = None if dbg is None else {k: v[sel] for k, v in dbg.items()}
    return parity.check_batch(ora, kb, hb, vo, nv, P, Kp, oh[sel], oi[sel], op[sel], dbg=d, pos_in=pin,
                              largest=not smallest, norm_kind=norm_kind)


def gaussian(B, S, d, seed):
    g = torch.Generator(device="cuda").manual_seed(seed)
    k = torch.randn((B, S, d), generator=g, device="cuda").to(torch.bfloat16)
    h = torch.randn((B, S, d), generator=g, device="cuda").to(torch.bfloat16)
    return k, h


# (B, S, d, vis_offset, n_vis, P, Kp): small, odd, ragged and degenerate shapes
SHAPES = [
    (1, 16, 8, 0, 16, 1, 1),          # smallest row width, one pivot, only the pivot kept
    (2, 50, 64, 3, 40, 1, 40),        # identity: everything kept
    (3, 100, 128, 0, 100, 5, 5),      # n_keep = n_pivot: pure top-k by norm
    (2, 333, 264, 17, 301, 7, 60),    # nothing a multiple of anything; remainder quotas (53 % 7 = 4)
    (1, 700, 4096, 40, 576, 8, 64),   # the LLaVA-1.5 shape with Gaussian tokens
    (2, 1100, 3584, 0, 1100, 32, 512),  # vision block fills the sequence; Qwen2 width
    (1, 2200, 512, 100, 2050, 128, 320),  # many pivots: (320-128) % 128 = 64 -> half of the pivots keep 2, half 1
    (5, 64, 32, 60, 4, 2, 3),         # tiny vision block at the very end
    (1, 9000, 64, 5, 8990, 3, 1000),  # long sequence: many tiles and a ragged tail
]


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS.get)
@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_shapes_against_oracle(oracle, shape, path):
    B, S, d, vo, nv, P, Kp = shape
    k, h = gaussian(B, S, d, seed=sum(shape))
    rep = compare(oracle, k, h, vo, nv, P, Kp, path=path)
    assert rep.exact >= rep.above_margin
    assert rep.max_rel_l1 < 5e-5 and rep.max_rel_l2 < 5e-5 and rep.max_abs_sim < 2e-5   # fp32-accumulation level


RETENTION_SHAPES = SHAPES + [
    (3, 700, 64, 10, 640, 128, 640),    # every pivot keeps four: 128 short lists per sample
    (2, 5000, 64, 0, 5000, 2, 4098),    # 4096 kept beside the pivots: the longest candidate lists
    (2, 5000, 64, 0, 5000, 2, 4500),    # more than that: the two-phase form does not apply and the one-kernel form runs
    (150, 80, 64, 5, 70, 4, 30),        # more samples than SMs
]


@pytest.mark.parametrize("shape", RETENTION_SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_both_forms_of_the_retention_agree(oracle, shape):
    """One kernel per sample (the pivots' selections one after the other) and candidate lists + walks make the
    same selections: every output is bitwise equal, and one of them is checked against the oracle."""
    B, S, d, vo, nv, P, Kp = shape
    k, h = gaussian(B, S, d, seed=3 + sum(shape))
    a = run_gpu(k, h, vo, nv, P, Kp, path=dart.DART_PATH_STAGED, retention=dart.DART_RETAIN_SERIAL)
    b = run_gpu(k, h, vo, nv, P, Kp, path=dart.DART_PATH_STAGED, retention=dart.DART_RETAIN_LISTS)
    assert all(np.array_equal(x, y) for x, y in zip(a[:3], b[:3]))
    assert all(np.array_equal(a[3][n], b[3][n], equal_nan=(n == "eps")) for n in a[3])
    sel = list(range(min(B, 3)))
    kb, hb = W.bits(k[sel]), W.bits(h[sel])
    ora = oracle.reduce(hb, kb, vo, nv, P, Kp)
    rep = parity.check_batch(ora, kb, hb, vo, nv, P, Kp, b[0][sel], b[1][sel], b[2][sel],
                             dbg={n: v[sel] for n, v in b[3].items()})
    assert rep.exact >= rep.above_margin


def _band_inputs(kind, B, S, d, vo, nv, P, seed):
    """Key rows that drive the band retention through each of its routes."""
    k, h = gaussian(B, S, d, seed=seed)
    g = torch.Generator(device="cuda").manual_seed(seed + 1)
    v = torch.randn(d, generator=g, device="cuda")
    vis = slice(vo, vo + nv)
    if kind == "same pivots":
        # the P rows of largest norm are copies of one direction: every pivot ranks the tokens alike, so each band is
        # all but used up by the pivots before it
        idx = vo + torch.randperm(nv, generator=g, device="cuda")[:P]
        k[:, idx] = (3.0 * v + 0.01 * torch.randn(B, P, d, generator=g, device="cuda")).to(k.dtype)
    elif kind == "equal tokens":
        # all vision rows but the pivots are one and the same row: every dup of a row ties, no band fits its list and the
        # index decides
        k[:, vis] = k[:, vo:vo + 1].clone()
        idx = vo + torch.randperm(nv, generator=g, device="cuda")[:P]
        k[:, idx] = (2.0 * k[:, idx].float() + torch.randn(B, P, d, generator=g, device="cuda")).to(k.dtype)
    elif kind == "stretched range":
        # one token opposite to the pivots' direction and the rest packed within a sliver of the range: the first
        # level of bins holds nearly all tokens in one bin
        k[:, vis] = (v + 0.02 * torch.randn(B, nv, d, generator=g, device="cuda")).to(k.dtype)
        k[:, vo + nv // 3] = (-v).to(k.dtype)
        idx = vo + torch.randperm(nv, generator=g, device="cuda")[:P]
        k[:, idx] = (3.0 * v + 0.3 * torch.randn(B, P, d, generator=g, device="cuda")).to(k.dtype)
    elif kind == "lanes of large keys":
        # tokens whose index mod 32 is 12 or more lie along the pivots' direction, the others are unrelated to it
        j = torch.arange(nv, device="cuda")
        along = vo + j[(j % 32) >= 12]
        k[:, along] = (v + 0.05 * torch.randn(B, along.numel(), d, generator=g, device="cuda")).to(k.dtype)
        idx = vo + (torch.randperm(nv // 32, generator=g, device="cuda")[:P] * 32 + 20)
        k[:, idx] = (3.0 * v + 0.3 * torch.randn(B, P, d, generator=g, device="cuda")).to(k.dtype)
    else:
        assert kind == "gaussian"
    return k, h


BAND_CASES = [
    # (kind, (B, S, d, vis_offset, n_vis, P, Kp))
    ("gaussian", (3, 700, 64, 10, 640, 128, 640)),        # quotas of four
    ("gaussian", (2, 1000, 64, 0, 900, 20, 600)),         # quotas of 29
    ("gaussian", (2, 130, 64, 7, 101, 3, 40)),            # fewer tokens than bins; rows not a multiple of 16 bytes
    ("gaussian", (2, 7000, 64, 0, 7000, 2, 6146)),        # the longest bands: 6144 tokens beside the pivots
    ("gaussian", (2, 7000, 64, 0, 7000, 2, 6200)),        # more than that: the sorted lists or the one-kernel form run
    ("gaussian", (2, 2000, 64, 0, 2000, 60, 1900)),       # bands of several rounds of staging
    ("gaussian", (2, 3000, 128, 40, 2880, 32, 320)),      # a sweep cell's shape
    ("gaussian", (2, 700, 64, 10, 640, 128, 130)),        # most pivots keep nothing beside themselves
    ("same pivots", (2, 1100, 64, 20, 1000, 48, 300)),
    ("same pivots", (2, 700, 64, 10, 640, 128, 640)),
    ("equal tokens", (2, 700, 64, 10, 640, 16, 200)),
    ("equal tokens", (1, 2100, 64, 10, 2000, 4, 1500)),
    ("stretched range", (2, 1400, 64, 30, 1280, 16, 120)),
    ("stretched range", (2, 3000, 64, 0, 2880, 8, 320)),
    ("lanes of large keys", (2, 1400, 64, 30, 1280, 16, 120)),
    ("lanes of large keys", (1, 1400, 64, 30, 1280, 8, 264)),
]


@pytest.mark.parametrize("kind,shape", BAND_CASES, ids=lambda v: v if isinstance(v, str) else "x".join(map(str, v)))
def test_candidate_bands_make_the_same_selections(oracle, kind, shape):
    """Unsorted candidate bands (the lowest histogram band of each pivot's dups that holds the tokens it could need)
    against the one-kernel form, bitwise, and against the oracle: plain rows, pivots that rank the tokens alike, rows of
    equal values (the exact route), rows whose range an outlier stretches (the finer levels of bins)."""
    B, S, d, vo, nv, P, Kp = shape
    k, h = _band_inputs(kind, B, S, d, vo, nv, P, seed=11 + sum(shape))
    a = run_gpu(k, h, vo, nv, P, Kp, path=dart.DART_PATH_STAGED, retention=dart.DART_RETAIN_SERIAL)
    b = run_gpu(k, h, vo, nv, P, Kp, path=dart.DART_PATH_STAGED, retention=dart.DART_RETAIN_BANDS)
    c = run_gpu(k, h, vo, nv, P, Kp, path=dart.DART_PATH_STAGED, retention=dart.DART_RETAIN_FUSED)   # both phases in one launch
    for o in (b, c):
        assert all(np.array_equal(x, y) for x, y in zip(a[:3], o[:3]))
        assert all(np.array_equal(a[3][n], o[3][n], equal_nan=(n == "eps")) for n in a[3])
    kb, hb = W.bits(k), W.bits(h)
    ora = oracle.reduce(hb, kb, vo, nv, P, Kp)
    rep = parity.check_batch(ora, kb, hb, vo, nv, P, Kp, b[0], b[1], b[2], dbg=b[3])
    assert rep.exact >= rep.above_margin


# (B, S, d, vis_offset, n_vis, P, Kp): one, two and three row tiles, ragged and whole last tiles, few and many pivots
TWO_TILE_SHAPES = [
    (2, 140, 64, 5, 100, 3, 30),        # less than one tile
    (3, 300, 128, 10, 256, 8, 64),      # exactly two tiles: one task
    (2, 330, 64, 0, 300, 9, 50),        # two whole tiles and a ragged third: the last task has one tile
    (2, 700, 256, 40, 640, 16, 100),    # five whole tiles: the last task has one tile
    (1, 1500, 64, 7, 1410, 128, 600),   # pivot tiles as large as the row tiles, a ragged last tile that is a task's second
    (2, 3000, 4096, 40, 2880, 8, 320),  # the benchmark's shape
]


@pytest.mark.parametrize("tiles", [1, 2], ids=["one tile per task", "two tiles per task"])
@pytest.mark.parametrize("shape", TWO_TILE_SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_one_pass_kernel_with_one_and_two_row_tiles_per_task(oracle, shape, tiles):
    """The one-pass kernel takes one 128-row tile per task or two that share every pivot tile (two accumulators):
    both against the oracle, with pivots by score (score pass first) and with the caller's pivots."""
    B, S, d, vo, nv, P, Kp = shape
    k, h = gaussian(B, S, d, seed=21 + sum(shape))
    kb, hb = W.bits(k), W.bits(h)
    tune = 0x1000 if tiles == 1 else 0x2000
    g = torch.Generator(device="cuda").manual_seed(5)
    piv = torch.stack([torch.randperm(nv, generator=g, device="cuda")[:P] for _ in range(B)]).to(torch.int32).contiguous()
    for given in (False, True):
        ctx = dart.Dart(B, S, d, P, Kp)
        try:
            opts = dart.dart_opts(path=dart.DART_PATH_TWO_PASS, tune=tune, pivots_in=piv.data_ptr() if given else 0)
            res = ctx.reduce(h, k, vo, nv, P, Kp, opts=opts, debug=True)
            torch.cuda.synchronize()
            assert ctx.status() == dart.DART_OK, dart.dart_status_detail(ctx.handle)
        finally:
            ctx.close()
        dbg = {n: _np(v) for n, v in res[3].items()}
        ora = oracle.reduce(hb, kb, vo, nv, P, Kp, pivots_in=piv.cpu().numpy() if given else None)
        rep = parity.check_batch(ora, kb, hb, vo, nv, P, Kp, _np(res[0]), _np(res[1]), _np(res[2]), dbg=dbg, pivots_given=given)
        assert rep.exact >= rep.above_margin
        assert rep.max_rel_l2 < 5e-5 and rep.max_abs_sim < 2e-5


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS.get)
def test_keys_null_scores_the_hidden_states(oracle, path):
    _, h = gaussian(2, 120, 256, seed=7)
    rep = compare(oracle, None, h, 10, 100, 4, 30, path=path)
    assert rep.samples == 2


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS.get)
def test_position_ids_are_gathered(oracle, path):
    k, h = gaussian(2, 90, 64, seed=8)
    pos = torch.randint(0, 1 << 40, (2, 90), device="cuda", dtype=torch.int64)
    compare(oracle, k, h, 5, 70, 3, 20, pos_in=pos, path=path)


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS.get)
@pytest.mark.parametrize("norm_kind,smallest", [(2, 0), (1, 1), (2, 1)])
def test_score_variants(oracle, path, norm_kind, smallest):
    k, h = gaussian(2, 300, 128, seed=9)
    compare(oracle, k, h, 20, 260, 6, 50, path=path, norm_kind=norm_kind, smallest=smallest)


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS.get)
def test_ties_and_exact_duplicates(oracle, path):
    """Exact copies of rows tie on score and on similarity; the lower index must win on both sides.
    All values are small integers so that fp32 and fp64 sums agree exactly and every tie is a true tie."""
    g = torch.Generator().manual_seed(11)
    S, d = 200, 64
    base = torch.randint(-3, 4, (20, d), generator=g).float()
    labels = torch.randint(0, 20, (S,), generator=g)
    x = base[labels].to(torch.bfloat16)[None].cuda().contiguous()      # 200 rows, only 20 distinct
    oh, oi, op, dbg = run_gpu(x, x, 0, S, 4, 40, path=path)
    ora = oracle.reduce(W.bits(x), None, 0, S, 4, 40)
    assert np.array_equal(dbg["pivot_idx"], ora.pivot_idx)
    assert np.array_equal(dbg["l1"].astype(np.float64), ora.l1)         # integer sums: exact
    assert np.array_equal(dbg["owner"], ora.owner) and np.array_equal(oi, ora.out_idx)
    assert np.array_equal(oh, ora.out_hidden) and np.array_equal(op, ora.out_pos)


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS.get)
def test_zero_rows_and_all_equal_scores(oracle, path):
    S, d = 64, 32
    x = torch.zeros((1, S, d), dtype=torch.bfloat16, device="cuda")
    x[0, 10:] = 1.0                                 # rows 0..9 are zero (dup := 0), the rest identical
    oh, oi, op, dbg = run_gpu(x, x, 0, S, 2, 12, path=path)
    ora = oracle.reduce(W.bits(x), None, 0, S, 2, 12)
    assert np.array_equal(dbg["pivot_idx"], ora.pivot_idx) and ora.pivot_idx[0].tolist() == [10, 11]
    assert np.array_equal(oi, ora.out_idx) and np.array_equal(dbg["owner"], ora.owner)
    assert oi[0].tolist() == list(range(12))         # zero rows have the lowest dup (0 < 1) and are kept


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS.get)
def test_scaled_copies_of_the_pivot_are_dropped(oracle, path):
    k, h = gaussian(1, 80, 128, seed=12)
    k[0, 5] *= 4.0
    for j, a in [(9, 0.5), (23, 0.25), (41, 0.125)]:
        k[0, j] = k[0, 5] * a
    oh, oi, op, dbg = run_gpu(k, h, 0, 80, 1, 77, path=path)
    assert dbg["pivot_idx"][0].tolist() == [5]
    assert sorted(set(range(80)) - set(oi[0].tolist())) == [9, 23, 41]


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS.get)
@pytest.mark.parametrize("w", [W.LLAVA15_B1, W.LLAVA15_B64, W.LLAVA_NEXT_B8, W.VIDEO_B4], ids=lambda w: w.name)
def test_benchmark_configs(oracle, w, path):
    k, h = W.make_batch(w, device="cuda")
    rep = compare(oracle, k, h, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, path=path)
    assert rep.samples == w.B and rep.exact >= rep.above_margin
    # fp32 accumulation puts the CUDA path ~1e-6 from the oracle, far inside typical gaps: near-ties that
    # flip are rare, and every one of them has been checked for validity above
    assert rep.exact >= int(0.9 * w.B), rep.notes
    assert rep.max_rel_l1 < 5e-5 and rep.max_abs_sim < 2e-5


@pytest.fixture(scope="module")
def sweep_batch():
    """The benchmark's batch: 256 x 2980 x 4096 bf16 keys and hidden states (12.5 GB), generated once."""
    w = W.SWEEP_B256
    k, h = W.make_batch(w, device="cuda")
    yield w, k, h
    del k, h
    torch.cuda.empty_cache()


def _oracle_check_samples(oracle, w, P, Kp, k, h, oh, oi, op, dbg, sel, threads):
    """Oracle and every parity rule (validity replay below the margin included) for the samples in `sel`, one sample
    per task on a pool of host threads (the oracle is single-threaded C called through ctypes, which drops the GIL)."""
    from concurrent.futures import ThreadPoolExecutor

    rep = parity.ParityReport()
    chunk = 32                                  # samples whose bits are on the host at a time (0.8 GB per tensor)
    for c0 in range(0, len(sel), chunk):
        ids = sel[c0:c0 + chunk]
        kb, hb = W.bits(k[ids]), W.bits(h[ids])
        ohb, oib, opb = W.bits(oh[ids]), oi[ids].cpu().numpy(), op[ids].cpu().numpy()
        d = {n: (v[ids].cpu().numpy()) for n, v in dbg.items()}

        def one(i):
            ora = oracle.reduce(hb[i:i + 1], kb[i:i + 1], w.vis_offset, w.n_vis, P, Kp, want_dup=P <= 32)
            return parity.check_batch(ora, kb[i:i + 1], hb[i:i + 1], w.vis_offset, w.n_vis, P, Kp, ohb[i:i + 1],
                                      oib[i:i + 1], opb[i:i + 1], dbg={n: v[i:i + 1] for n, v in d.items()})

        with ThreadPoolExecutor(max_workers=threads) as pool:
            for r in pool.map(one, range(len(ids))):
                rep.merge(r)
    return rep


# every valid cell of the sweep (128 pivots cannot be kept within 64 tokens)
SWEEP_CELLS = [(8, 64), (8, 320), (8, 640), (32, 64), (32, 320), (32, 640), (128, 320), (128, 640)]


@pytest.mark.parametrize("cell", SWEEP_CELLS, ids=lambda c: "P%d_K%d" % c)
def test_full_size_sweep_cells(oracle, sweep_batch, cell):
    """Config 5 at its full size on the default path, the launch configuration bench.py times (the per-step outputs
    are copies out of the workspace after the same kernels).  8 pivots: ALL 256 samples go through the oracle;
    32 pivots: every fourth; 128 pivots: every sixteenth.  A sample whose kept set differs from the oracle's must lie
    below the margin AND pass the replay of its own assignment against the oracle's fp64 similarities (Eq. 9: nothing
    left behind beats a pivot's threshold by more than the tolerance): being rare is not enough."""
    import os

    w, k, h = sweep_batch
    P, Kp = cell
    ctx = dart.Dart(w.B, w.S, w.d, P, Kp)
    try:
        oh, oi, op, dbg = ctx.reduce(h, k, w.vis_offset, w.n_vis, P, Kp, debug=True)
        torch.cuda.synchronize()
        st = ctx.status()
        assert st == dart.DART_OK, (st, dart.dart_status_detail(ctx.handle))
    finally:
        ctx.close()
    S_out = w.S - w.n_vis + Kp
    # all samples: strictly ascending indices, text rows intact, position ids = indices, gathered rows = hidden rows
    d_oi = oi[:, 1:] - oi[:, :-1]
    assert bool((d_oi > 0).all()) and oi.shape == (w.B, S_out)
    assert bool((oi[:, :w.vis_offset] == torch.arange(w.vis_offset, device="cuda", dtype=torch.int32)).all())
    n_after = w.S - w.vis_offset - w.n_vis
    assert bool((oi[:, S_out - n_after:] == torch.arange(w.vis_offset + w.n_vis, w.S, device="cuda", dtype=torch.int32)).all())
    assert bool((op == oi.to(torch.int64)).all())
    rows = torch.gather(h.view(torch.int16), 1, oi.to(torch.int64).unsqueeze(-1).expand(-1, -1, w.d))
    assert bool((rows == oh.view(torch.int16)).all())
    del rows
    step = 1 if P <= 8 else 4 if P <= 32 else 16
    sel = sorted(set(range(0, w.B, step)) | {w.B - 1})
    rep = _oracle_check_samples(oracle, w, P, Kp, k, h, oh, oi, op, dbg, sel, threads=min(32, os.cpu_count() or 1))
    assert rep.samples == len(sel) and rep.exact >= rep.above_margin
    # every sample that differs from the oracle has been replayed by check_batch (it raises otherwise) and is listed
    assert rep.samples - rep.exact == len(rep.notes), rep.notes
    assert rep.max_rel_l1 < 5e-5 and rep.max_rel_l2 < 5e-5
    if P <= 32:
        assert rep.max_abs_sim < 2e-5


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS.get)
def test_runs_are_bitwise_reproducible(path):
    w = W.LLAVA15_B64.with_(B=4)
    k, h = W.make_batch(w, device="cuda")
    a = run_gpu(k, h, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, path=path)
    for _ in range(3):
        b = run_gpu(k, h, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, path=path)
        assert all(np.array_equal(x, y) for x, y in zip(a[:3], b[:3]))
        assert all(np.array_equal(a[3][n], b[3][n], equal_nan=(n == "eps")) for n in a[3])


def test_fused_path_rejects_what_it_cannot_do():
    k, h = gaussian(1, 64, 72, seed=15)                      # d = 72 is not a multiple of 64
    ctx = dart.Dart(1, 64, 72, 2, 8)
    with pytest.raises(dart.DartError) as e:
        ctx.reduce(h, k, 0, 64, 2, 8, opts=dart.dart_opts(0, 0, dart.DART_PATH_FUSED, 0, 0))
    assert e.value.code == dart.DART_ERR_UNSUPPORTED
    ctx.reduce(h, k, 0, 64, 2, 8)                            # AUTO falls back to the staged kernels
    torch.cuda.synchronize()
    assert ctx.status() == dart.DART_OK
    ctx.close()


@pytest.mark.parametrize("lag", [1, 40, 100000])
def test_fused_path_with_short_and_long_lags(oracle, lag):
    """The distance between a row's two sweeps only changes the schedule (how long sweep 2 waits for the
    pivots), never the result."""
    w = W.LLAVA15_B64.with_(B=6)
    k, h = W.make_batch(w, device="cuda")
    a = run_gpu(k, h, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, path=dart.DART_PATH_FUSED, sweep_lag=lag)
    b = run_gpu(k, h, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, path=dart.DART_PATH_FUSED)
    assert all(np.array_equal(x, y) for x, y in zip(a[:3], b[:3]))
    assert all(np.array_equal(a[3][n], b[3][n], equal_nan=(n == "eps")) for n in a[3])


@pytest.mark.parametrize("ahead", [2, 200, 2000])
def test_fused_path_with_the_second_pass_cut_into_column_chunks(oracle, ahead):
    """Option of the persistent sweep: every row tile's second pass as eight tasks of 512 columns whose shares of the
    similarities are added up afterwards, the first pass held within `ahead` steps of the second."""
    w = W.LLAVA_NEXT_B8.with_(B=3)
    k, h = W.make_batch(w, device="cuda")
    ctx = dart.Dart(w.B, w.S, w.d, w.n_pivot, w.n_keep)
    try:
        res = ctx.reduce(h, k, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, debug=True,
                         opts=dart.dart_opts(path=dart.DART_PATH_FUSED, tune=ahead))
        torch.cuda.synchronize()
        assert ctx.status() == dart.DART_OK, dart.dart_status_detail(ctx.handle)
    finally:
        ctx.close()
    kb, hb = W.bits(k), W.bits(h)
    ora = oracle.reduce(hb, kb, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep)
    rep = parity.check_batch(ora, kb, hb, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, _np(res[0]), _np(res[1]), _np(res[2]),
                             dbg={n: _np(v) for n, v in res[3].items()})
    assert rep.exact >= rep.above_margin and rep.max_abs_sim < 2e-5


def test_expired_wait_is_reported_not_hung():
    """Bounded waits: with the pivots withheld (a flag that nothing sets) the fused kernel must give up within
    its time limit, say where, exit normally, and leave the context usable for the next call."""
    w = W.LLAVA15_B64.with_(B=8)
    k, h = W.make_batch(w, device="cuda")
    ctx = dart.Dart(w.B, w.S, w.d, w.n_pivot, w.n_keep)
    opts = dart.dart_opts(0, 0, dart.DART_PATH_FUSED, 20000, 0, 1)        # 20 ms limit, pivots withheld
    ctx.reduce(h, k, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, opts=opts)
    torch.cuda.synchronize()
    assert ctx.status() == dart.DART_ERR_TIMEOUT
    rc, detail = dart.dart_status_detail(ctx.handle)
    assert rc == dart.DART_OK and detail[0] == 1                          # the wait for the pivots gave up first
    assert ctx.status() == dart.DART_OK                                   # reading cleared it
    good = ctx.reduce(h, k, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep)   # same context, normal call
    torch.cuda.synchronize()
    assert ctx.status() == dart.DART_OK
    ref = run_gpu(k, h, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, path=dart.DART_PATH_STAGED, debug=False)
    assert np.array_equal(_np(good[1]), ref[1]) and np.array_equal(_np(good[0]), ref[0])
    ctx.close()


def test_argument_validation_launches_nothing():
    k, h = gaussian(2, 64, 32, seed=13)
    ctx = dart.Dart(2, 64, 32, 4, 16)
    oh = torch.empty((2, 64, 32), dtype=torch.bfloat16, device="cuda")
    oi = torch.empty((2, 64), dtype=torch.int32, device="cuda")
    op = torch.empty((2, 64), dtype=torch.int64, device="cuda")
    P = lambda t: ctypes.c_void_p(t.data_ptr())  # noqa: E731
    n0 = dart.dart_launch_count(ctx.handle)

    def call(hid=h, key=k, vo=4, nv=50, p=4, kp=16, out=oh):
        return dart.dart_reduce(ctx.handle, P(hid), P(key), vo, nv, p, kp, P(out), P(oi), P(op), None)

    assert dart.dart_set_shape(ctx.handle, 3, 64) == dart.DART_ERR_BAD_SHAPE      # above B_max
    assert dart.dart_set_shape(ctx.handle, 2, 65) == dart.DART_ERR_BAD_SHAPE      # above S_max
    assert dart.dart_set_shape(ctx.handle, 2, 64) == dart.DART_OK
    assert call(p=0) == dart.DART_ERR_BAD_SHAPE
    assert call(p=5, kp=5) == dart.DART_ERR_BAD_SHAPE                             # above P_max
    assert call(kp=17) == dart.DART_ERR_BAD_SHAPE                                 # above Kp_max
    assert call(p=4, kp=3) == dart.DART_ERR_BAD_SHAPE                             # fewer kept than pivots
    assert call(nv=10, kp=11) == dart.DART_ERR_BAD_SHAPE                          # more kept than vision tokens
    assert call(vo=20, nv=50) == dart.DART_ERR_BAD_SHAPE                          # vision block past the end
    assert call(vo=-1) == dart.DART_ERR_BAD_SHAPE
    assert dart.dart_reduce(ctx.handle, None, P(k), 4, 50, 4, 16, P(oh), P(oi), P(op), None) == dart.DART_ERR_NULL
    assert dart.dart_reduce(ctx.handle, P(h), P(k), 4, 50, 4, 16, P(oh), None, P(op), None) == dart.DART_ERR_NULL
    assert dart.dart_reduce(ctx.handle, ctypes.c_void_p(h.data_ptr() + 2), P(k), 4, 50, 4, 16, P(oh), P(oi), P(op),
                            None) == dart.DART_ERR_ALIGN
    assert call(out=h) == dart.DART_ERR_ALIAS and call(out=k) == dart.DART_ERR_ALIAS
    assert dart.dart_launch_count(ctx.handle) == n0                               # nothing was launched
    assert call() == dart.DART_OK and dart.dart_launch_count(ctx.handle) > n0
    torch.cuda.synchronize()
    assert ctx.status() == dart.DART_OK
    assert dart.dart_workspace_bytes(ctx.handle) > 0
    ctx.close()


def test_profile_slots_cover_every_launch():
    k, h = gaussian(2, 200, 64, seed=14)
    ctx = dart.Dart(2, 200, 64, 4, 32)
    dart.dart_profile_enable(ctx.handle, True)
    ctx.reduce(h, k, 0, 200, 4, 32)
    rc, prof = dart.dart_profile_read(ctx.handle)
    assert rc == dart.DART_OK and sum(n for _, n in prof.values()) >= 1
    assert all(ms >= 0 for ms, _ in prof.values())
    ctx.close()


@pytest.mark.parametrize("B", [1, 6])
def test_the_call_can_be_captured_in_a_cuda_graph(B):
    """All work goes to the caller's stream and nothing synchronises the host: a captured call replays with the
    same outputs (one sample takes the resident sweep, six the persistent one; both launch cooperatively)."""
    w = W.LLAVA15_B64.with_(B=B)
    k, h = W.make_batch(w, device="cuda")
    ctx = dart.Dart(w.B, w.S, w.d, w.n_pivot, w.n_keep)
    try:
        ref = ctx.reduce(h, k, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep)
        torch.cuda.synchronize()
        out = tuple(torch.zeros_like(t) for t in ref)
        s, g = torch.cuda.Stream(), torch.cuda.CUDAGraph()
        with torch.cuda.stream(s):
            ctx.reduce(h, k, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, out=out, stream=s)
            s.synchronize()
            g.capture_begin()
            ctx.reduce(h, k, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, out=out, stream=s)
            g.capture_end()
        for t in out:
            t.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert ctx.status() == dart.DART_OK
        assert all(torch.equal(a, b) for a, b in zip(out, ref))
    finally:
        ctx.close()
