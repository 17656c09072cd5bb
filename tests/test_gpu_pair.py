"""The paired sweeps (the same SM reads a block of rows twice, a short time apart; every SM merges the SMs' candidate
lists into the sample's pivots) against the oracle, through the C ABI (needs a B200)."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from paper_2502_11494_b200 import dart, workloads as W  # noqa: E402
from test_gpu_parity import compare, gaussian, run_gpu  # noqa: E402

pytestmark = pytest.mark.gpu
PAIRED = dart.DART_PATH_PAIRED

# (B, S, d, vis_offset, n_vis, P, Kp)
SHAPES = [
    (1, 16, 64, 0, 16, 1, 1),            # one block in all: one CTA
    (2, 50, 64, 3, 40, 1, 40),           # identity: everything kept; ragged last block
    (3, 100, 128, 0, 100, 5, 5),         # n_keep = n_pivot: pure top-k by norm
    (2, 333, 320, 17, 301, 7, 60),       # five atoms: a single short stage per block
    (1, 700, 4096, 40, 576, 8, 64),      # the LLaVA-1.5 shape: fewer blocks than CTAs
    (7, 700, 4096, 40, 576, 8, 64),      # several samples, CTAs without a block in some of them
    (3, 3000, 4096, 40, 2880, 8, 320),   # the LLaVA-NeXT shape: one or two blocks per CTA and sample
    (8, 3000, 4096, 40, 2880, 16, 320),  # 16 pivots: pivot atoms of 16 rows
    (2, 1300, 3584, 0, 1300, 4, 100),    # Qwen2 width: 56 atoms, seven stages
    (4, 4708, 3584, 50, 4608, 16, 512),  # the video shape with 16 pivots
    (5, 4800, 512, 30, 4736, 9, 500),    # many blocks per CTA and sample, nine pivots
    (9, 1300, 1024, 100, 1187, 3, 1187), # many samples
    (1, 9000, 64, 5, 8990, 3, 1000),     # long sequence of one-atom rows
    (2, 300, 8192, 10, 280, 2, 30),      # the widest rows
]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_paired_sweeps_match_the_oracle(oracle, shape):
    B, S, d, vo, nv, P, Kp = shape
    k, h = gaussian(B, S, d, seed=1700 + sum(shape))
    rep = compare(oracle, k, h, vo, nv, P, Kp, path=PAIRED)
    assert rep.exact >= rep.above_margin
    # the tensor cores add each 16-column step to an fp32 accumulator that is cut, not rounded: a pivot's product with
    # itself (d positive terms) ends about (d / 16) / 2 units in the last place low, i.e. ~1e-5 at d = 4096, ~3e-5 at 8192
    assert rep.max_rel_l1 < 5e-5 and rep.max_rel_l2 < 5e-5 and rep.max_abs_sim < (2e-5 if d <= 4096 else 6e-5)


@pytest.mark.parametrize("norm_kind,smallest", [(1, 1), (2, 0), (2, 1)])
def test_paired_sweeps_ranking_variants(oracle, norm_kind, smallest):
    k, h = gaussian(3, 500, 256, seed=177)
    rep = compare(oracle, k, h, 20, 444, 6, 90, path=PAIRED, norm_kind=norm_kind, smallest=smallest)
    assert rep.exact >= rep.above_margin and rep.max_abs_sim < 2e-5


def test_paired_sweeps_equal_scores_rank_the_lower_index_first(oracle):
    """Rows that are copies of each other tie in score: the pivots must be the lower indices, in order, although they
    reach the merge through the lists of different CTAs."""
    k, h = gaussian(2, 300, 128, seed=178)
    k[:, 10:300] = k[:, 10:11] * 0.5          # all vision rows but the first equal; the first one larger
    k[:, 10] = k[:, 11] * 2
    oh, oi, op, dbg = run_gpu(k, h, 10, 290, 5, 40, path=PAIRED)
    assert np.array_equal(dbg["pivot_idx"], np.tile(np.arange(5, dtype=np.int32), (2, 1)))
    rep = compare(oracle, k, h, 10, 290, 5, 40, path=PAIRED)
    assert rep.exact >= rep.above_margin


@pytest.mark.parametrize("w", [W.LLAVA15_B1, W.LLAVA15_B64, W.LLAVA_NEXT_B8], ids=lambda w: w.name)
def test_paired_sweeps_on_the_benchmark_configs(oracle, w):
    k, h = W.make_batch(w, device="cuda")
    rep = compare(oracle, k, h, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, path=PAIRED)
    assert rep.samples == w.B and rep.exact >= rep.above_margin and rep.exact >= int(0.9 * w.B), rep.notes
    assert rep.max_rel_l1 < 5e-5 and rep.max_abs_sim < 2e-5
    a = run_gpu(k, h, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, path=PAIRED)
    b = run_gpu(k, h, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, path=dart.DART_PATH_TWO_PASS)
    assert np.array_equal(a[3]["pivot_idx"], b[3]["pivot_idx"])
    assert np.allclose(a[3]["sim"], b[3]["sim"], rtol=0, atol=4e-5)   # each within 2e-5 of the oracle


def test_paired_sweeps_are_bitwise_reproducible():
    w = W.LLAVA15_B64.with_(B=5)
    k, h = W.make_batch(w, device="cuda")
    a = run_gpu(k, h, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, path=PAIRED)
    for lead in (0, 1, 3):
        b = run_gpu(k, h, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, path=PAIRED, sweep_lag=lead)
        assert all(np.array_equal(x, y) for x, y in zip(a[:3], b[:3]))
        assert all(np.array_equal(a[3][n], b[3][n], equal_nan=(n == "eps")) for n in a[3])


@pytest.mark.parametrize("shape", [(1, 64, 64, 0, 64, 17, 20), (1, 64, 96, 0, 64, 2, 8)], ids=["17 pivots", "d not a multiple of 64"])
def test_paired_sweeps_say_what_they_do_not_take(shape):
    B, S, d, vo, nv, P, Kp = shape
    k, h = gaussian(B, S, d, seed=179)
    ctx = dart.Dart(B, S, d, P, Kp)
    with pytest.raises(dart.DartError) as e:
        ctx.reduce(h, k, vo, nv, P, Kp, opts=dart.dart_opts(path=PAIRED))
    assert e.value.code == dart.DART_ERR_UNSUPPORTED
    ctx.close()


# second status word: 44 = the sample's merging CTA still waits for the lists, 50 = another CTA waits for that CTA's result,
# 51 = the epilogue waits for the pivots' norms
@pytest.mark.parametrize("withhold,where", [(1, (44, 50)), (2, (51,))], ids=["lists never published", "norms never handed over"])
def test_paired_sweeps_expired_waits_are_reported_not_hung(withhold, where):
    """Bounded waits: with a sample's publication (or the pivots' norms) withheld - a counter that nothing advances -
    the kernel must give up within its time limit, say where, exit normally and leave the context usable."""
    w = W.LLAVA15_B64.with_(B=8)
    k, h = W.make_batch(w, device="cuda")
    ctx = dart.Dart(w.B, w.S, w.d, w.n_pivot, w.n_keep)
    opts = dart.dart_opts(path=PAIRED, wait_limit=20000, test_withhold_pivots=withhold)      # 20 ms limit
    ctx.reduce(h, k, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, opts=opts)
    torch.cuda.synchronize()
    assert ctx.status() == dart.DART_ERR_TIMEOUT
    rc, detail = dart.dart_status_detail(ctx.handle)
    assert rc == dart.DART_OK and detail[0] in where, detail
    assert ctx.status() == dart.DART_OK                                   # reading cleared it
    good = ctx.reduce(h, k, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, opts=dart.dart_opts(path=PAIRED))
    torch.cuda.synchronize()
    assert ctx.status() == dart.DART_OK
    ref = run_gpu(k, h, w.vis_offset, w.n_vis, w.n_pivot, w.n_keep, path=dart.DART_PATH_STAGED, debug=False)
    assert np.array_equal(good[1].cpu().numpy(), ref[1]) and np.array_equal(W.bits(good[0]), ref[0])
    ctx.close()
