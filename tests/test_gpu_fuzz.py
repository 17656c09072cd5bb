"""Seeded random shapes and options, every path against the oracle (needs a B200).  Shapes are small (the oracle
takes milliseconds) but ragged: odd token counts, vision blocks at either end, quotas with remainders, row
widths around the tile sizes of the tensor-core kernels."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import parity  # noqa: E402
from paper_2502_11494_b200 import dart, workloads as W  # noqa: E402
from test_gpu_parity import _np, gaussian  # noqa: E402

pytestmark = pytest.mark.gpu


def random_case(seed):
    rng = np.random.default_rng(1000 + seed)
    d = int(rng.choice([8, 24, 64, 128, 192, 320, 512, 1024, 3584]))
    n_vis = int(rng.integers(1, 700))
    before, after = int(rng.integers(0, 50)), int(rng.integers(0, 50))
    P = int(rng.integers(1, min(n_vis, 40) + 1))
    Kp = int(rng.integers(P, n_vis + 1))
    B = int(rng.integers(1, 5))
    return dict(B=B, S=before + n_vis + after, d=d, vo=before, nv=n_vis, P=P, Kp=Kp,
                path=int(rng.choice([dart.DART_PATH_STAGED, dart.DART_PATH_FUSED, dart.DART_PATH_TWO_PASS])),
                norm_kind=int(rng.choice([1, 2])), smallest=int(rng.integers(0, 2)),
                retention=int(rng.integers(0, 5)), rule=int(rng.integers(0, 2)),
                given=bool(rng.integers(0, 2)), on_hidden=bool(rng.integers(0, 2)), keys_null=bool(rng.integers(0, 4) == 0))


@pytest.mark.parametrize("seed", range(40))
def test_random_shapes_and_options(oracle, seed):
    c = random_case(seed)
    if c["path"] != dart.DART_PATH_STAGED and c["d"] % 64:
        c["path"] = dart.DART_PATH_STAGED
    if c["on_hidden"]:
        c["norm_kind"] = 1
    k, h = gaussian(c["B"], c["S"], c["d"], seed=seed)
    if c["keys_null"]:
        k = None
    piv = None
    if c["given"]:
        rng = np.random.default_rng(seed)
        piv = np.stack([rng.permutation(c["nv"])[:c["P"]] for _ in range(c["B"])]).astype(np.int32)
    piv_t = None if piv is None else torch.from_numpy(piv).cuda()
    ctx = dart.Dart(c["B"], c["S"], c["d"], c["P"], c["Kp"])
    try:
        opts = dart.dart_opts(norm_kind=c["norm_kind"], pivot_smallest=c["smallest"], path=c["path"], retention=c["retention"],
                              rule=c["rule"], cosine_on_hidden=int(c["on_hidden"]),
                              pivots_in=None if piv_t is None else piv_t.data_ptr())
        res = ctx.reduce(h, k, c["vo"], c["nv"], c["P"], c["Kp"], opts=opts, debug=True)
        torch.cuda.synchronize()
        assert ctx.status() == dart.DART_OK, (c, dart.dart_status_detail(ctx.handle))
    finally:
        ctx.close()
    oh, oi, op = _np(res[0]), _np(res[1]), _np(res[2])
    dbg = {n: _np(v) for n, v in res[3].items()}
    hb = W.bits(h)
    kb = hb if k is None else W.bits(k)
    on_hidden = c["on_hidden"] and k is not None
    ora = oracle.reduce(hb, None if k is None else kb, c["vo"], c["nv"], c["P"], c["Kp"], norm_kind=c["norm_kind"],
                        largest=not c["smallest"], pivots_in=piv, rule=c["rule"], cosine_on_hidden=on_hidden)
    rep = parity.check_batch(ora, kb, hb, c["vo"], c["nv"], c["P"], c["Kp"], oh, oi, op, dbg=dbg, largest=not c["smallest"],
                             norm_kind=c["norm_kind"], pivots_given=c["given"], rule=c["rule"],
                             sim_bits=hb if on_hidden else None)
    assert rep.exact >= rep.above_margin, c
    assert rep.max_rel_l1 < 5e-5 and rep.max_rel_l2 < 5e-5 and rep.max_abs_sim < 2e-5, c
