"""dart_pivots_static: the entry point for hosts that cannot allocate device memory.

An inference server that has given all of HBM to its own memory pool, or a loop that must not pay
for cudaMalloc's device-wide synchronisation, cannot create a context.  For them the library offers
pivot selection on a scratch array that is baked into the library image.  This test calls it twice
in a row through the C ABI - a large problem first, a smaller one second, so that the second call
finds the first call's scores still lying in the shared scratch - and requires the same pivots,
bit for bit (integer indices: the tolerance the other parity tests use for index outputs), as the
context-based entry point reports AND as the CPU oracle ranks them from its own fp64 scores (the two
entry points share their kernels, so agreement between them alone would not catch a mistake in
those).  It also checks what the entry point is for: the amount of free device memory is the same
before and after a call.  Collected last on purpose; it passes alone or after the rest.
"""
import ctypes

import numpy as np
import pytest

torch = pytest.importorskip("torch")

from paper_2502_11494_b200 import dart, workloads as W  # noqa: E402

pytestmark = pytest.mark.gpu


def _ptr(t):
    return ctypes.c_void_p(t.data_ptr())


def _pivots_via_context(keys, vo, nv, P):
    B, S, d = keys.shape
    ctx = dart.Dart(B, S, d, P, P)
    try:
        *_, dbg = ctx.reduce(keys, keys, vo, nv, P, P, debug=True)
        torch.cuda.synchronize()
        assert ctx.status() == dart.DART_OK
        return dbg["pivot_idx"].cpu().numpy()
    finally:
        ctx.close()


def _pivots_via_oracle(oracle, keys, vo, nv, P):
    """Def. 1 on the oracle's own L1 scores of the same bf16 bits, sample by sample."""
    kb = W.bits(keys)
    return np.stack([oracle.pivots(oracle.scores(kb[b], vo, nv)[0], P)[0] for b in range(kb.shape[0])])


def test_static_scratch_pivots_match_the_context_path_twice_in_a_row(oracle):
    g = torch.Generator(device="cuda").manual_seed(2024)
    st = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    dev = torch.cuda.current_device()
    # the last case fills the scratch to its last row: B * n_vis == DART_STATIC_MAX_ROWS
    cases = [(6, 700, 1024, 40, 576, 8), (2, 300, 256, 10, 257, 33), (64, 4096, 64, 0, 4096, 5)]
    assert cases[2][0] * cases[2][4] == dart.DART_STATIC_MAX_ROWS
    for n, (B, S, d, vo, nv, P) in enumerate(cases):
        keys = torch.randn((B, S, d), generator=g, device="cuda").to(torch.bfloat16)
        keys[:, vo + 3] = keys[:, vo + 1]                  # an exact duplicate row: a tie on the score
        keys[:, vo + nv - 1] *= 3.0                        # the block's last row ranks first: the last scratch row is read
        out = torch.full((B, P), -1, dtype=torch.int32, device="cuda")
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info(dev)[0]
        rc = dart.dart_pivots_static(_ptr(keys), B, S, d, vo, nv, P, _ptr(out), dev, st)
        assert rc == dart.DART_OK, dart.dart_strerror(rc)
        torch.cuda.synchronize()
        if n > 0:                                          # (the very first call on a device may load the module)
            assert torch.cuda.mem_get_info(dev)[0] == free_before, "the call changed the amount of free device memory"
        got = out.cpu().numpy()
        assert np.array_equal(got, _pivots_via_context(keys, vo, nv, P))
        assert np.array_equal(got, _pivots_via_oracle(oracle, keys, vo, nv, P))
        assert (got[:, 0] == nv - 1).all()


def test_static_scratch_limits_are_enforced():
    keys = torch.zeros((1, 64, 64), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros((1, 4), dtype=torch.int32, device="cuda")
    dev = torch.cuda.current_device()
    too_many = dart.DART_STATIC_MAX_ROWS + 1
    assert dart.dart_pivots_static(_ptr(keys), 1, too_many, 64, 0, too_many, 4, _ptr(out), dev, None) \
        == dart.DART_ERR_BAD_SHAPE                            # rejected on the host, nothing is read
    assert dart.dart_pivots_static(None, 1, 64, 64, 0, 64, 4, _ptr(out), dev, None) == dart.DART_ERR_NULL
    assert dart.dart_pivots_static(_ptr(keys), 1, 64, 64, 0, 64, 65, _ptr(out), dev, None) == dart.DART_ERR_BAD_SHAPE
