"""CPU-side checks of the C-ABI: the library loads, exports what the header declares, and its
host-only logic (layout validation, group counts, row geometry, reuse rule, argument rejection)
agrees with the oracle's independent statement of the same rules.  No kernel is launched here."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def oc():
    from paper_2607_23844_b200 import build
    build.build()
    from paper_2607_23844_b200 import omnicache
    return omnicache


def header_functions():
    text = open(os.path.join(ROOT, "include", "omnicache.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(oc_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(oc):
    names = header_functions()
    assert len(names) >= 20
    lib = C.CDLL(oc.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/omnicache.h but not exported"
    assert set(names) == set(oc.EXPORTS)


def test_status_and_kernel_names(oc):
    assert oc.status_str(0) == "OC_OK"
    assert oc.status_str(8) == "OC_CACHE_MISS"
    assert oc.status_str(99) == "OC_UNKNOWN_STATUS"
    assert len({oc.kernel_name(k) for k in range(oc.K_COUNT)}) == oc.K_COUNT
    assert oc.kernel_name(oc.K_MATCH_TC) == "match_tc"


def test_layout_check_rules(oc):
    L = oc.Layout
    ok = L(oc.KIND_TOKEN, oc.DTYPE_BF16, 2, 1, 64, 64, 1536)
    assert ok.check() == oc.OK
    assert L(oc.KIND_TOKEN, oc.DTYPE_BF16, 2, 1, 64, 64, 1532).check() == oc.ERR_ALIGNMENT   # C*2 % 16
    assert L(oc.KIND_TOKEN, oc.DTYPE_F32, 1, 1, 16, 16, 62).check() == oc.ERR_ALIGNMENT
    assert L(oc.KIND_TOKEN, oc.DTYPE_F32, 1, 1, 16, 16, 64).check() == oc.OK
    assert L(3, oc.DTYPE_BF16, 1, 1, 8, 8, 8).check() == oc.ERR_INVALID_ARG
    assert L(oc.KIND_TOKEN, 2, 1, 1, 8, 8, 8).check() == oc.ERR_INVALID_ARG
    assert L(oc.KIND_TOKEN, oc.DTYPE_BF16, 0, 1, 8, 8, 8).check() == oc.ERR_INVALID_ARG
    assert L(oc.KIND_TOKEN, oc.DTYPE_BF16, 1, 1, 9, 8, 8).check() == oc.ERR_INVALID_ARG      # H % sy
    assert L(oc.KIND_TOKEN, oc.DTYPE_BF16, 1, 1, 8, 8, 8, gy=3).check() == oc.ERR_INVALID_ARG
    assert L(oc.KIND_TOKEN, oc.DTYPE_BF16, 1, 1, 8, 8, 8, gy=4, gx=4).check() == oc.OK
    assert L(oc.KIND_TOKEN, oc.DTYPE_BF16, 1, 1, 8, 8, 8, gy=8).check() == oc.ERR_INVALID_ARG  # patch 1 row, sy 2
    assert L(oc.KIND_TOKEN, oc.DTYPE_BF16, 1, 1, 8, 8, 8, oy=2).check() == oc.ERR_INVALID_ARG
    assert L(oc.KIND_TOKEN, oc.DTYPE_BF16, 1, 1, 8, 8, 8, sy=1, sx=1).check() == oc.ERR_INVALID_ARG
    assert L(oc.KIND_TOKEN, oc.DTYPE_BF16, 1, 1, 8, 8, 8, sy=1, sx=1, self_match=1).check() == oc.OK
    assert L(oc.KIND_TOKEN, oc.DTYPE_BF16, 1, 1, 8, 8, 8, gy=2, self_match=1).check() == oc.ERR_UNSUPPORTED
    assert L(oc.KIND_TOKEN, oc.DTYPE_BF16, 1, 1, 8, 8, 8, eps=-1.0).check() == oc.ERR_INVALID_ARG
    assert L(oc.KIND_FRAME, oc.DTYPE_BF16, 1, 25, 72, 128, 320).check() == oc.OK
    assert L(oc.KIND_FRAME, oc.DTYPE_BF16, 1, 25, 72, 128, 320, frame_stat=2).check() == oc.ERR_INVALID_ARG
    assert L(oc.KIND_FRAME, oc.DTYPE_BF16, 1, 25, 72, 128, 320, gy=4, gx=4).check() == oc.OK     # patch-local
    assert L(oc.KIND_FRAME, oc.DTYPE_BF16, 1, 25, 72, 128, 320, gy=5).check() == oc.ERR_INVALID_ARG
    assert L(oc.KIND_FRAME, oc.DTYPE_BF16, 1, 25, 72, 128, 320, gx=-1).check() == oc.ERR_INVALID_ARG
    assert L(oc.KIND_FRAME, oc.DTYPE_BF16, 1, 25, 72, 128, 320, gy=0, gx=0).counts()[0] == 1
    assert L(oc.KIND_BLOCK, oc.DTYPE_BF16, 1, 16, 16, 16, 1152).check() == oc.OK
    assert L(oc.KIND_BLOCK, oc.DTYPE_BF16, 1, 16, 16, 16, 1152, gy=2).check() == oc.OK          # patch-local selection
    assert L(oc.KIND_BLOCK, oc.DTYPE_BF16, 1, 16, 16, 16, 1152, gy=16).check() == oc.ERR_INVALID_ARG  # cuts a 2x2 group
    assert L(oc.KIND_TOKEN, oc.DTYPE_BF16, 64, 64, 1024, 1024, 8).check() == oc.ERR_UNSUPPORTED   # > 2^31-1 units
    assert oc._lib.oc_layout_check(None) == oc.ERR_INVALID_ARG


@pytest.mark.parametrize("kind,shape,kw", [
    (0, (2, 1, 64, 64, 1536), {}), (0, (2, 1, 64, 64, 1536), dict(gy=4, gx=2)),
    (0, (1, 25, 18, 32, 1280), {}), (0, (1, 1, 16, 16, 64), dict(self_match=1)),
    (0, (1, 2, 12, 18, 8), dict(sy=3, sx=3, oy=1, ox=2, gy=2, gx=2)),
    (1, (3, 25, 72, 128, 320), {}), (2, (2, 16, 16, 16, 1152), {}),
    (1, (2, 25, 72, 128, 320), dict(gy=4, gx=4)), (1, (2, 5, 12, 16, 8), dict(gy=3, gx=1)),
    (1, (1, 4, 12, 16, 8), dict(gy=1, gx=8)), (2, (2, 16, 16, 24, 1152), dict(gy=2, gx=3)),
])
def test_counts_and_rows_agree_with_oracle(oc, oracle, kind, shape, kw):
    L = oc.Layout(kind, oc.DTYPE_BF16, *shape, **kw)
    Lo = oracle.Layout(kind, oracle.DT_BF16, *shape, **kw)
    g, u, r = L.counts()
    assert (g, u) == (Lo.n_groups, Lo.units_per_group)
    assert r == Lo.n_rep
    for ch, eb in ((shape[-1], 2), (24, 4)):
        a, b = oc.rows_from_layout(L, ch, eb), oracle.rows_for(Lo, ch, eb)
        # both describe the same byte offsets for every unit and segment
        assert (a.seg_bytes, a.n_seg) == (b.seg_bytes, b.n_seg)
        n_units = g * u
        for i in (0, 1, n_units // 2, n_units // 3 + 1, n_units - 1):
            for s in (0, a.n_seg - 1):
                off_a = (i // a.units_per_outer) * a.outer_pitch + (i % a.units_per_outer) * a.unit_pitch + s * a.seg_stride
                off_b = (i // b.units_per_outer) * b.outer_pitch + (i % b.units_per_outer) * b.unit_pitch + s * b.seg_stride
                assert off_a == off_b
    assert oc.match_workspace_bytes(L) > 0


def test_rows_from_layout_rejects(oc):
    L = oc.Layout(oc.KIND_TOKEN, oc.DTYPE_BF16, 1, 1, 8, 8, 8)
    rows = oc.CRows()
    cl = L.c()
    assert oc._lib.oc_rows_from_layout(C.byref(cl), 7, 2, C.byref(rows)) == oc.ERR_ALIGNMENT
    assert oc._lib.oc_rows_from_layout(C.byref(cl), 8, 3, C.byref(rows)) == oc.ERR_INVALID_ARG
    assert oc._lib.oc_rows_from_layout(C.byref(cl), 8, 2, None) == oc.ERR_INVALID_ARG


def test_layer_cache_rule_matches_oracle(oc, oracle):
    for s0 in (-3, 0, 7):
        for step in range(-5, 20):
            for n in (0, 1, 5):
                assert oc.layer_cache_would_hit(s0, step, n) == oracle.layer_cache_hit(s0, step, n)


def test_null_context_and_bad_arguments_are_rejected_before_any_launch(oc):
    lib = oc._lib
    L = oc.Layout(oc.KIND_TOKEN, oc.DTYPE_BF16, 1, 1, 8, 8, 8).c()
    rows = oc.CRows(16, 1, 0, 16, 1 << 40, 0)
    one = C.c_void_p(16)   # a non-null, 16-byte aligned dummy; never dereferenced on these paths
    assert lib.oc_match(None, C.byref(L), one, one, one, None, None, None) == oc.ERR_INVALID_ARG
    assert lib.oc_match_frame_levels(None, C.byref(L), one, 1, one, one, one, None, None, None) == oc.ERR_INVALID_ARG
    assert lib.oc_select(None, C.byref(L), one, one, 0, 0.5, 0, 64, one, one, one, one, None) == oc.ERR_INVALID_ARG
    assert lib.oc_joint_groups(None, C.byref(L), one, one, one, one, None) == oc.ERR_INVALID_ARG
    assert lib.oc_match_joint(None, C.byref(L), one, one, one, one, None) == oc.ERR_INVALID_ARG
    assert lib.oc_select_joint(None, C.byref(L), one, one, one, 0, 0.5, 0, 0, 64, one, one, one, one, None) == oc.ERR_INVALID_ARG
    assert lib.oc_joint_workspace_bytes(C.byref(L), None) == oc.ERR_INVALID_ARG
    assert lib.oc_gather(None, C.byref(rows), one, one, 4, one, None) == oc.ERR_INVALID_ARG
    assert lib.oc_restore(None, C.byref(rows), one, one, 4, one, one, one, 0, None) == oc.ERR_INVALID_ARG
    assert lib.oc_layer_cache_put(None, 0, 0, one, 16, None) == oc.ERR_INVALID_ARG
    assert lib.oc_layer_cache_get(None, 0, 0, 1, None, None, None, None) == oc.ERR_INVALID_ARG
    assert lib.oc_layer_cache_clear(None) == oc.ERR_INVALID_ARG
    assert lib.oc_destroy(None) == oc.ERR_INVALID_ARG
    assert lib.oc_device_status(None, None) == oc.ERR_INVALID_ARG
    assert lib.oc_profile_read(None, 0, None, None) == oc.ERR_INVALID_ARG
    assert lib.oc_profile_span_read(None, 1, None, None) == oc.ERR_INVALID_ARG
    assert lib.oc_profile_captured_read(None, 1, None, None) == oc.ERR_INVALID_ARG
    assert lib.oc_selftest_bounded_wait(None, 100, None) == oc.ERR_INVALID_ARG
    assert lib.oc_match_frame_noalloc(-1, C.byref(L), one, one, one, None, None) == oc.ERR_INVALID_ARG
    assert lib.oc_cache_step_host(None, C.byref(L), 0, 0.5, 0, one, one, one, None, None) == oc.ERR_INVALID_ARG
    h = C.c_void_p()
    assert lib.oc_create(None, 0, 0) == oc.ERR_INVALID_ARG
    assert lib.oc_create(C.byref(h), -1, 0) == oc.ERR_INVALID_ARG


def test_kernel_setup_runs_once_per_device_not_once_per_process(oc):
    """Kernel attributes (the opt-in to large dynamic shared memory) belong to a device; a process may use
    several.  The launchers' bookkeeping must run the set-up once for EVERY device it is asked about, remember
    a failure without retrying it, and refuse nothing else (host-only: a counting set-up routine stands in)."""
    lib = oc._lib
    n = 5
    runs, ok = (C.c_int * n)(), (C.c_int * n)()
    assert lib.oc_selftest_per_device_once(n, 4, -1, runs, ok) == oc.OK
    assert list(runs) == [1] * n and list(ok) == [4] * n
    assert lib.oc_selftest_per_device_once(n, 3, 2, runs, ok) == oc.OK
    assert list(runs) == [1] * n                       # the failing device's set-up is not run again either
    assert list(ok) == [3, 3, 0, 3, 3]
    assert lib.oc_selftest_per_device_once(0, 1, -1, runs, ok) == oc.ERR_INVALID_ARG
    assert lib.oc_selftest_per_device_once(65, 1, -1, runs, ok) == oc.ERR_INVALID_ARG
    assert lib.oc_selftest_per_device_once(n, 1, -1, None, ok) == oc.ERR_INVALID_ARG


def test_schedule_proposal_matches_oracle(oc, oracle):
    """Algorithm 1 is host logic: the library's answer must equal the oracle's to the index."""
    import numpy as np
    rng = np.random.default_rng(17)
    for trial in range(300):
        n = int(rng.integers(0, 40))
        L = rng.uniform(0.05, 5.0, n)
        Q = rng.uniform(0.0, 2.0, n)
        if n > 3 and trial % 3 == 0:                       # ties in the score and zero losses
            Q[1] = Q[0] / L[0] * L[1]; Q[2] = 0.0; Q[3] = 0.0
        s_r = float(rng.choice([1.0, 1.05, 1.5, 2.0, 3.7, 50.0]))
        got, saved = oc.schedule_propose(L, Q, s_r)
        ref = oracle.schedule_proposal(L, Q, s_r)
        assert got == ref
        assert abs(saved - L[ref].sum()) < 1e-9
    # the 28-layer x 25-step table of a DiT-sized model, as one call
    L = rng.uniform(0.5, 2.0, 28 * 25); Q = rng.gamma(2.0, 0.1, 28 * 25)
    got, saved = oc.schedule_propose(L, Q, 2.0)
    assert got == oracle.schedule_proposal(L, Q, 2.0) and saved >= 0.5 * L.sum() > saved - L[got[-1]]
    lib = oc._lib
    one = C.c_void_p(16)
    n_out = C.c_int64()
    assert lib.oc_schedule_propose(None, one, 1, 2.0, one, C.byref(n_out), None) == oc.ERR_INVALID_ARG
    bad = np.array([1.0, 0.0]); q = np.array([0.1, 0.1]); ch = np.empty(2, np.int32)
    assert lib.oc_schedule_propose(bad.ctypes.data_as(C.c_void_p), q.ctypes.data_as(C.c_void_p), 2, 2.0,
                                   ch.ctypes.data_as(C.c_void_p), C.byref(n_out), None) == oc.ERR_INVALID_ARG
    ok = np.array([1.0, 1.0])
    assert lib.oc_schedule_propose(ok.ctypes.data_as(C.c_void_p), q.ctypes.data_as(C.c_void_p), 2, 0.5,
                                   ch.ctypes.data_as(C.c_void_p), C.byref(n_out), None) == oc.ERR_INVALID_ARG


def test_create_fails_loudly_without_a_device(oc):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    h = C.c_void_p()
    assert oc._lib.oc_create(C.byref(h), 0, 0) == oc.ERR_CUDA
    assert not h.value
    with pytest.raises(oc.OmniCacheError):
        oc.Context(0, 0)
