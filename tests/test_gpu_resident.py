"""The resident sweep (one read of the keys; rows wait on the chip for their sample's pivots) against the oracle,
through the C ABI (needs a B200)."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from paper_2502_11494_b200 import dart, workloads as W  # noqa: E402
from test_gpu_parity import compare, gaussian, run_gpu  # noqa: E402

pytestmark = pytest.mark.gpu

# (B, S, d, vis_offset, n_vis, P, Kp)
SHAPES = [
    (1, 16, 64, 0, 16, 1, 1),            # two octets in all: most CTAs hold nothing
    (2, 50, 64, 3, 40, 1, 40),           # identity: everything kept
    (3, 100, 128, 0, 100, 5, 5),         # n_keep = n_pivot: pure top-k by norm; a ragged last octet
    (2, 333, 320, 17, 301, 7, 60),       # row width not a multiple of 256: the 8-register tail batches
    (1, 700, 4096, 40, 576, 8, 64),      # the LLaVA-1.5 shape: one tensor-memory slot per quarter
    (7, 700, 4096, 40, 576, 8, 64),      # several samples in flight, fewer octets than CTAs
    (3, 3000, 4096, 40, 2880, 8, 320),   # the LLaVA-NeXT shape: 2-3 octets per CTA and sample, rotating
    (2, 1300, 3584, 0, 1300, 4, 100),    # Qwen2 width
    (5, 4800, 512, 30, 4736, 8, 500),    # the most octets per CTA and sample the kernel takes
    (9, 1300, 1024, 100, 1187, 3, 1187), # many samples, four slots per quarter
]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_resident_sweep_matches_the_oracle(oracle, shape):
    B, S, d, vo, nv, P, Kp = shape
    k, h = gaussian(B, S, d, seed=700 + sum(shape))
    rep = compare(oracle, k, h, vo, nv, P, Kp, path=dart.DART_PATH_RESIDENT)
    assert rep.exact >= rep.above_margin
    assert rep.max_rel_l1 < 5e-5 and rep.max_rel_l2 < 5e-5 and rep.max_abs_sim < 2e-5


def run_split(k, h, vo, nv, P, Kp, split):
    B, S, d = h.shape
    ctx = dart.Dart(B, S, d, P, Kp)
    try:
        res = ctx.reduce(h, k, vo, nv, P, Kp, debug=True, opts=dart.dart_opts(path=dart.DART_PATH_SPLIT, resident_split=split))
        torch.cuda.synchronize()
        assert ctx.status() == dart.DART_OK, dart.dart_status_detail(ctx.handle)
    finally:
        ctx.close()
    return res


@pytest.mark.parametrize("split", [0, 2, 3, -3, -4, 40], ids=lambda s: "split%d" % s)
@pytest.mark.parametrize("shape", [SHAPES[3], SHAPES[5], SHAPES[6], SHAPES[8]], ids=lambda s: "x".join(map(str, s)))
def test_split_between_chip_and_second_read_matches_the_oracle(oracle, shape, split):
    """Some 128-row tiles wait on the chip for the pivots, the others are read a second time by the one-pass
    kernel: whatever the share, every row gets its similarities from exactly one of the two."""
    from oracle import parity
    from test_gpu_parity import _np

    B, S, d, vo, nv, P, Kp = shape
    k, h = gaussian(B, S, d, seed=900 + sum(shape))
    res = run_split(k, h, vo, nv, P, Kp, split)
    kb, hb = W.bits(k), W.bits(h)
    ora = oracle.reduce(hb, kb, vo, nv, P, Kp)
    rep = parity.check_batch(ora, kb, hb, vo, nv, P, Kp, _np(res[0]), _np(res[1]), _np(res[2]),
                             dbg={n: _np(v) for n, v in res[3].items()})
    assert rep.exact >= rep.above_margin
    assert rep.max_rel_l1 < 5e-5 and rep.max_rel_l2 < 5e-5 and rep.max_abs_sim < 2e-5


@pytest.mark.parametrize("norm_kind,smallest", [(1, 1), (2, 0), (2, 1)])
def test_resident_sweep_ranking_variants(oracle, norm_kind, smallest):
    k, h = gaussian(3, 500, 256, seed=77)
    rep = compare(oracle, k, h, 20, 444, 6, 90, path=dart.DART_PATH_RESIDENT, norm_kind=norm_kind, smallest=smallest)
    assert rep.exact >= rep.above_margin and rep.max_abs_sim < 2e-5


def test_resident_sweep_equal_scores_rank_the_lower_index_first(oracle):
    """Rows that are copies of each other tie in score: the pivots must be the lower indices, in order."""
    k, h = gaussian(2, 300, 128, seed=78)
    k[:, 10:300] = k[:, 10:11] * 0.5          # all vision rows but the first equal; the first one larger
    k[:, 10] = k[:, 11] * 2
    oh, oi, op, dbg = run_gpu(k, h, 10, 290, 5, 40, path=dart.DART_PATH_RESIDENT)
    assert np.array_equal(dbg["pivot_idx"], np.tile(np.arange(5, dtype=np.int32), (2, 1)))
    rep = compare(oracle, k, h, 10, 290, 5, 40, path=dart.DART_PATH_RESIDENT)
    assert rep.exact >= rep.above_margin


def test_resident_sweep_on_the_clustered_workload(oracle):
    w = W.LLAVA15_B64.with_(B=12)
    k, h = W.make_batch(w, device="cuda")
    rep = compare(oracle, k, h, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, path=dart.DART_PATH_RESIDENT)
    assert rep.exact >= rep.above_margin and rep.exact >= 11, rep.notes
    a = run_gpu(k, h, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, path=dart.DART_PATH_RESIDENT)
    b = run_gpu(k, h, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, path=dart.DART_PATH_FUSED)
    assert np.array_equal(a[3]["pivot_idx"], b[3]["pivot_idx"])
    assert np.allclose(a[3]["sim"], b[3]["sim"], rtol=0, atol=4e-5)   # each within 2e-5 of the oracle


@pytest.mark.parametrize("shape", [(1, 64, 64, 0, 64, 9, 20), (1, 64, 8200, 0, 64, 2, 8), (1, 5000, 64, 0, 4744, 2, 8),
                                   (1, 64, 96, 0, 64, 2, 8)],
                         ids=["nine pivots", "rows wider than 8 KB", "too many rows per SM", "d not a multiple of 64"])
def test_resident_sweep_says_what_it_does_not_take(shape):
    B, S, d, vo, nv, P, Kp = shape
    k, h = gaussian(B, S, d, seed=79)
    ctx = dart.Dart(B, S, d, P, Kp)
    with pytest.raises(dart.DartError) as e:
        ctx.reduce(h, k, vo, nv, P, Kp, opts=dart.dart_opts(path=dart.DART_PATH_RESIDENT))
    assert e.value.code == dart.DART_ERR_UNSUPPORTED
    ctx.close()


@pytest.mark.parametrize("path,where,opts", [
    (dart.DART_PATH_RESIDENT, 83, {}),                       # no CTA counts itself in: the exchange warps wait for the others
    (dart.DART_PATH_TWO_PASS, 70, {}),                       # one-pass kernel: a norm warp never hands its norms to the epilogue
], ids=["resident sweep", "one-pass kernel"])
def test_expired_waits_of_the_other_kernels_are_reported_not_hung(path, where, opts):
    """Bounded waits of the resident sweep (what AUTO runs for up to four samples) and of the one-pass kernel: with one
    hand-over withheld - a counter that nothing advances, a barrier that one warp never arrives at - the kernel must
    give up within its time limit, say where, free its tensor memory, exit normally and leave the context usable."""
    w = W.LLAVA15_B64.with_(B=3)
    k, h = W.make_batch(w, device="cuda")
    ctx = dart.Dart(w.B, w.S, w.d, w.n_pivot, w.n_keep)
    ctx.reduce(h, k, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep,
               opts=dart.dart_opts(path=path, wait_limit=20000, test_withhold_pivots=1))      # 20 ms limit
    torch.cuda.synchronize()
    assert ctx.status() == dart.DART_ERR_TIMEOUT
    rc, detail = dart.dart_status_detail(ctx.handle)
    assert rc == dart.DART_OK and detail[0] == where, detail
    assert ctx.status() == dart.DART_OK                                   # reading cleared it
    good = ctx.reduce(h, k, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, opts=dart.dart_opts(path=path))   # same context
    torch.cuda.synchronize()
    assert ctx.status() == dart.DART_OK
    ref = run_gpu(k, h, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, path=dart.DART_PATH_STAGED, debug=False)
    assert np.array_equal(good[1].cpu().numpy(), ref[1]) and np.array_equal(W.bits(good[0]), ref[0])
    ctx.close()
