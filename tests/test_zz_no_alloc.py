"""The allocation-free Frame Cache match against the regular entry point.

Some callers of this library are not allowed to obtain device memory: a serving process that gave
its whole budget to one pool when it started, or code running under somebody else's allocator.
oc_match() is closed to them because a context owns cudaMalloc'd scratch; oc_match_frame_noalloc()
keeps its scratch in a fixed array inside the library instead.  This file checks, through the
C-ABI, that both entry points give the same answer and that this answer is the CPU oracle's - twice
in a row, because the second call finds the array dirty from the first - and that an oversized
layout is refused.  It is named so that pytest collects it last.
"""
import numpy as np
import pytest
import torch

from paper_2607_23844_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def oc():
    from paper_2607_23844_b200 import build
    build.build()
    from paper_2607_23844_b200 import omnicache
    assert torch.cuda.is_available()
    return omnicache


def _regular(oc, L, x):
    n = L.n_units
    sim = torch.full((n,), float("nan"), device="cuda")
    idx = torch.full((n,), -2, device="cuda", dtype=torch.int32)
    pair = torch.full((L.B, L.T - 1), float("nan"), device="cuda")
    with oc.Context(0, oc.match_workspace_bytes(L)) as ctx:
        ctx.match(L, x, sim, idx, None, pair)
        torch.cuda.synchronize()
    return sim, idx, pair


def test_noalloc_frame_match_equals_regular_entry_point_twice(oc, oracle):
    # two different inputs of two different shapes, one after the other: the second call starts
    # from whatever the first left in the shared array
    cases = [inputs.svd_frames(seed=51, T=9, H=24, W=40, C=64), inputs.svd_frames(seed=52, T=6, H=18, W=32, C=320)]
    for w in cases:
        L = oc.Layout(oc.KIND_FRAME, w.dtype, *w.shape)
        assert oc.match_workspace_bytes(L) <= oc.NOALLOC_SCRATCH_BYTES
        x = torch.from_numpy(w.x.view(np.int16)).cuda()
        want_sim, want_idx, want_pair = _regular(oc, L, x)
        ref = oracle.match_frame(oracle.Layout(oracle.KIND_FRAME, w.dtype, *w.shape), w.x)
        cand = np.isfinite(ref["best_sim"])
        for _ in range(2):
            n = L.n_units
            sim = torch.full((n,), float("nan"), device="cuda")
            idx = torch.full((n,), -2, device="cuda", dtype=torch.int32)
            pair = torch.full((L.B, L.T - 1), float("nan"), device="cuda")
            oc.match_frame_noalloc(0, L, x, sim, idx, pair)
            torch.cuda.synchronize()
            # same kernels, same fixed-order sums: the two entry points agree to the last bit, which
            # is well inside the 1e-3 the parity tests allow for bf16 inputs
            assert torch.equal(idx, want_idx)
            assert torch.equal(sim, want_sim)
            assert float((pair - want_pair).abs().max()) <= 1e-3
            assert torch.equal(pair, want_pair)
            # and against the oracle, under the parity tests' rules for bf16 inputs: similarities within
            # 1e-3, the chosen neighbour frame exact
            gs, gi = sim.cpu().numpy(), idx.cpu().numpy()
            assert np.array_equal(np.isneginf(gs), ~cand)
            assert np.abs(gs[cand] - ref["best_sim"][cand]).max() <= 1e-3
            assert np.array_equal(gi, ref["best_idx"])
            assert np.abs(pair.cpu().numpy() - ref["pair_sim"]).max() <= 1e-3


def test_noalloc_rejects_what_does_not_fit_or_is_not_a_frame_layout(oc):
    big = oc.Layout(oc.KIND_FRAME, oc.DTYPE_BF16, 4, 200, 72, 128, 320)
    assert oc.match_workspace_bytes(big) > oc.NOALLOC_SCRATCH_BYTES
    dummy = torch.zeros(64, device="cuda")
    sentinel = torch.full((800,), 5, device="cuda", dtype=torch.int32)
    out = sentinel.clone()
    assert oc.match_frame_noalloc(0, big, dummy, dummy, out, check=False) == oc.ERR_WORKSPACE
    tok = oc.Layout(oc.KIND_TOKEN, oc.DTYPE_BF16, 1, 1, 8, 8, 8)
    assert oc.match_frame_noalloc(0, tok, dummy, dummy, out, check=False) == oc.ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert torch.equal(out, sentinel)
