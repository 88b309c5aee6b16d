"""GPU parity: every op of the path, called through the C-ABI binding, against the CPU oracle on the
same seeded inputs.  Tolerances: similarities 1e-3 absolute for bf16 inputs (fp32 accumulation),
1e-5 for fp32 inputs; indices exact except near-ties (oracle top-two gap, or distance to the
selection cut, below 1e-4); gather / restore / layered cache bit-exact."""
import numpy as np
import pytest
import torch

from paper_2607_23844_b200 import inputs

import gpu_harness as H

pytestmark = pytest.mark.gpu

TOL = {inputs.F32: 1e-5, inputs.BF16: 1e-3}


@pytest.fixture(scope="module")
def oc():
    from paper_2607_23844_b200 import build
    build.build()
    from paper_2607_23844_b200 import omnicache
    assert torch.cuda.is_available()
    return omnicache


def group_quanta(shape, groups=(1, 1), lattice=(2, 2, 0, 0)):
    """Boxes of 32 lattice points (2^k wide, at most 32) that cover one group's representative lattice."""
    sy, sx, oy, ox = lattice
    hp, wp = shape[2] // groups[0], shape[3] // groups[1]
    hs, ws = (hp - oy + sy - 1) // sy, (wp - ox + sx - 1) // sx
    bw = 1
    while bw < min(ws, 32):
        bw *= 2
    bh = 32 // bw
    return -(-ws // bw) * -(-hs // bh)


def expect_tensor_core(dtype, shape, lattice=(2, 2, 0, 0), self_match=False, groups=(1, 1)):
    """Whether oc_match must take the tcgen05 kernel for this Token Cache layout: bf16, no self-match, at most
    nine lattice members, rows of whole 16-byte chunks, a group whose column-scale tables fit beside the
    operand ring (150 boxes of 32 representatives).  Anything else belongs to the fp32-FMA kernel; a bf16
    layout that falls back silently would pass every numeric check and run an order of magnitude slower."""
    return (dtype == inputs.BF16 and not self_match and lattice[0] * lattice[1] <= 9 and shape[-1] % 8 == 0
            and group_quanta(shape, groups, lattice) <= 150)


def assert_matcher(rep, dtype, shape, lattice=(2, 2, 0, 0), groups=(1, 1)):
    want_tc = expect_tensor_core(dtype, shape, lattice, groups=groups)
    assert rep["launches"]["match_tc"] == (1 if want_tc else 0), rep["launches"]
    assert rep["launches"]["match_simt"] == (0 if want_tc else 1), rep["launches"]


def run_chain(oc, oracle, w, Cout=None, full_oracle=True, sample_rows=0, want_aux=False, **layout_kw):
    """match -> select -> gather -> restore for one workload, each stage compared with the oracle.
    Returns a small report dict."""
    L, Lo = H.layouts(oc, oracle, w, **layout_kw)
    rep = {}
    x_dev = H.to_dev(w.x)
    with H.make_ctx(oc, L) as ctx:
        # ---- match -----------------------------------------------------------------------------
        m = H.gpu_match(oc, ctx, L, x_dev, want_aux=want_aux and L.kind != oc.KIND_BLOCK,
                        want_pair=L.kind == oc.KIND_FRAME)
        gs, gi = m["best_sim"].cpu().numpy(), m["best_idx"].cpu().numpy()
        if L.kind == oc.KIND_TOKEN:
            if full_oracle:
                ref = oracle.match_token(Lo, w.x, want_full=want_aux)
                rows = None
            else:
                # the same number of rows from every group (frame or patch), so that every frame and, over
                # the groups, every position inside the matcher's tiles is looked at
                rng = np.random.default_rng(99)
                G, U = Lo.n_groups, Lo.units_per_group
                per = max(1, sample_rows // G)
                rows = np.sort(np.array([Lo.unit_index(g, int(u)) for g in range(G)
                                         for u in rng.choice(U, min(per, U), replace=False)], dtype=np.int64))
                ref = oracle.match_token(Lo, w.x, rows=rows)
            rep["near_tie_rows"], rep["near_tie_differ"] = H.check_match_against_oracle(
                oracle, Lo, w.x, gs, gi, ref, TOL[w.dtype], rows)
            if want_aux and full_oracle:
                a = m["aux"].cpu().numpy().astype(np.float64)
                f = ref["full_sim"]
                written = ~np.isnan(f)
                assert np.array_equal(~np.isnan(a), written), "aux rows written differ from the oracle's"
                assert np.abs(a[written] - f[written]).max() <= TOL[w.dtype]
        elif L.kind == oc.KIND_FRAME:
            ref = oracle.match_frame(Lo, w.x, want_pos=want_aux)
            H.check_match_against_oracle(oracle, Lo, w.x, gs, gi, ref, TOL[w.dtype])
            if L.T > 1:
                assert np.abs(m["pair_sim"].cpu().numpy() - ref["pair_sim"]).max() <= TOL[w.dtype]
            if want_aux and L.T > 1:
                assert np.abs(m["aux"].cpu().numpy() - ref["pos_sim"]).max() <= TOL[w.dtype]
        else:
            ref = oracle.match_block(Lo, w.x)
            H.check_match_against_oracle(oracle, Lo, w.x, gs, gi, ref, TOL[w.dtype])

        # ---- select: (a) on the GPU's own similarities, oracle given the same arrays (exact) -----
        mode = oc.SELECT_COUNT if w.mode == "count" else oc.SELECT_THRESHOLD
        U = L.units_per_group
        n_cand = U if w.self_match else U - L.reps_per_group
        stride = U - min(w.n_reuse, n_cand) if mode == oc.SELECT_COUNT else U
        s = H.gpu_select(oc, ctx, L, m["best_sim"], m["best_idx"], mode, w.thr, w.n_reuse, stride)
        ref_s = H.check_select_against_oracle(oracle, Lo, gs, gi, mode, w.thr, w.n_reuse, stride, s)
        # ---- select: (b) on the oracle's similarities uploaded to the GPU (exact, no exceptions) ---
        if full_oracle:
            os_, oi = ref["best_sim"], ref["best_idx"]
            s2 = H.gpu_select(oc, ctx, L, H.to_dev(os_), H.to_dev(oi), mode, w.thr, w.n_reuse, stride)
            ref_s2 = H.check_select_against_oracle(oracle, Lo, os_, oi, mode, w.thr, w.n_reuse, stride, s2)
            # (c) the two selections may differ only at units whose oracle similarity is within 1e-4
            # of the cut (count mode: the last reused value; threshold mode: thr)
            kept_a, kept_b = ref_s["slot_of"] >= 0, ref_s2["slot_of"] >= 0
            differ = np.nonzero(kept_a != kept_b)[0]
            if differ.size:
                G = Lo.n_groups
                grp_of = np.empty(Lo.n_units, np.int64)
                for g in range(G):
                    grp_of[[Lo.unit_index(g, u) for u in range(U)]] = g
                for i in differ:
                    if mode == oc.SELECT_COUNT:
                        ids = np.nonzero((grp_of == grp_of[i]) & ~kept_b & np.isfinite(os_))[0]
                        cut = os_[ids].min()
                    else:
                        cut = w.thr
                    assert abs(float(os_[i]) - float(cut)) < H.NEAR_TIE, (i, os_[i], cut)
            rep["cut_differ"] = int(differ.size)
            assert np.array_equal(ref_s["kept_count"], ref_s2["kept_count"]) or mode == oc.SELECT_THRESHOLD

        # ---- gather ------------------------------------------------------------------------------
        Ro = oracle.rows_for(Lo, w.shape[-1], w.elem_bytes)
        n_slots = s["kept_idx"].numel()
        y = torch.full((n_slots, Ro.row_bytes), 0xAB, device="cuda", dtype=torch.uint8)
        ctx.gather(H.crows(oc, Ro), x_dev, s["kept_idx"], n_slots, y)
        y_ref = oracle.gather(Ro, w.x, ref_s["kept_idx"], fill=0xAB)
        assert H.dev_bytes(y) == y_ref.tobytes()

        # ---- wrapped layer stand-in (outside the path) and restore ---------------------------------
        Cout = Cout or w.shape[-1]
        eb = w.elem_bytes
        Rz = oracle.rows_for(Lo, Cout, eb)
        rng = np.random.default_rng(123)
        if "layer_weight" in w.extra and Cout == w.shape[-1] and L.kind == oc.KIND_TOKEN:
            wt = w.extra["layer_weight"].astype(np.float64)
            yv = y_ref.view(np.float32).reshape(n_slots, -1).astype(np.float64)
            z_np = (yv @ wt).astype(np.float32)
            cache_np = (w.extra["x_prev"].reshape(-1, Cout).astype(np.float64) @ wt).astype(np.float32)
        else:
            n_el = n_slots * Rz.row_bytes // eb
            z_np = inputs.random_rows(5, (n_el,), w.dtype)
            cache_np = inputs.random_rows(6, w.shape[:-1] + (Cout,), w.dtype)
        z_dev, cache_dev = H.to_dev(z_np), H.to_dev(cache_np)
        n_units = Lo.n_units
        for src_mode in (oc.RESTORE_FROM_CACHE, oc.RESTORE_FROM_REPRESENTATIVE):
            out = torch.full((cache_np.nbytes,), 0xCD, device="cuda", dtype=torch.uint8)
            ctx.restore(H.crows(oc, Rz), z_dev, cache_dev, n_units, s["slot_of"], s["match_map"], out, src_mode)
            want = oracle.restore(Rz, z_np, cache_np, n_units, ref_s["slot_of"], ref_s["match_map"], src_mode)
            assert H.dev_bytes(out) == want.tobytes(), f"restore mode {src_mode}"
        inplace = cache_dev.clone()
        ctx.restore(H.crows(oc, Rz), z_dev, inplace, n_units, s["slot_of"], s["match_map"], inplace)
        want = oracle.restore(Rz, z_np, cache_np.copy(), n_units, ref_s["slot_of"], ref_s["match_map"], in_place=True)
        assert H.dev_bytes(inplace) == want.tobytes()
        torch.cuda.synchronize()
        assert ctx.device_status() == oc.OK
        rep["reused"] = int((ref_s["slot_of"] < 0).sum())
        rep["launches"] = ctx.launches()
    return rep


# ---------------------------------------------------------------------------------------------------
# config 1 exactly, and small versions of configs 2-4 that span several tiles with ragged tails
# ---------------------------------------------------------------------------------------------------
def test_config1_tiny_token_cache_fp32(oc, oracle):
    rep = run_chain(oc, oracle, inputs.tiny_token_cache(), want_aux=True)
    assert 40 <= rep["reused"] <= 110
    assert rep["launches"]["match_simt"] == 1


@pytest.mark.parametrize("shape,groups,lattice,dtype", [
    ((2, 1, 24, 40, 200), (1, 1), (2, 2, 0, 0), inputs.BF16),     # K tail (200 % 64), 240 reps
    ((1, 2, 32, 32, 128), (2, 2), (2, 2, 1, 1), inputs.BF16),     # patches, other lattice offset
    ((1, 1, 36, 72, 64), (1, 1), (2, 2, 0, 1), inputs.BF16),      # 18 x 36 lattice: ragged both ways
    ((2, 1, 16, 48, 96), (2, 4), (2, 2, 0, 0), inputs.BF16),      # 8 token groups per frame
    ((1, 1, 12, 18, 40), (1, 1), (3, 3, 1, 2), inputs.BF16),      # 3 x 3 neighbourhoods
    ((1, 2, 16, 16, 36), (1, 1), (2, 2, 0, 0), inputs.F32),       # fp32, C % 32 != 0
    ((1, 1, 64, 64, 320), (1, 1), (2, 2, 0, 0), inputs.BF16),     # 1024 reps: several N tiles
])
def test_token_chain_small(oc, oracle, shape, groups, lattice, dtype):
    B, T, Hh, W, C = shape
    w = inputs.sd3_token_cache(seed=21, B=B * T, H=Hh, W=W, C=C, groups=groups, dtype=dtype)
    w.x = w.x.reshape(shape); w.shape = shape
    sy, sx, oy, ox = lattice
    U = (Hh // groups[0]) * (W // groups[1])
    w.n_reuse = (U - U // (sy * sx)) // 2
    rep = run_chain(oc, oracle, w, want_aux=True, sy=sy, sx=sx, oy=oy, ox=ox)
    assert_matcher(rep, dtype, shape, lattice, groups)


def _random_token_layouts(n, seed):
    """Seeded random valid Token Cache shapes: lattice strides 2 or 3 with any offset, 1-8 patches per
    frame, ragged lattice sizes, channel counts with and without a 64-channel tail, 1-3 frames."""
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < n:
        sy, sx = int(rng.integers(2, 4)), int(rng.integers(2, 4))
        gy, gx = int(rng.choice([1, 1, 2, 3])), int(rng.choice([1, 1, 2, 4]))
        hp, wp = sy * int(rng.integers(2, 14)), sx * int(rng.integers(2, 22))
        C = int(rng.choice([8, 24, 64, 72, 128, 200, 320]))
        B, T = int(rng.integers(1, 3)), int(rng.integers(1, 3))
        if B * T * gy * hp * gx * wp * C > 6_000_000:
            continue
        out.append(((B, T, gy * hp, gx * wp, C), (gy, gx), (sy, sx, int(rng.integers(0, sy)), int(rng.integers(0, sx)))))
    return out


@pytest.mark.parametrize("shape,groups,lattice", _random_token_layouts(24, seed=20260701))
def test_token_chain_random_layouts(oc, oracle, shape, groups, lattice):
    """The whole chain against the oracle on shapes nobody picked by hand (the matcher's tiling,
    piece cutting and masking depend on every one of these numbers)."""
    B, T, Hh, W, C = shape
    w = inputs.sd3_token_cache(seed=int(np.prod(shape)) % 9973, B=B * T, H=Hh, W=W, C=C, groups=groups)
    w.x = w.x.reshape(shape); w.shape = shape
    sy, sx, oy, ox = lattice
    U = (Hh // groups[0]) * (W // groups[1])
    reps = ((Hh // groups[0]) // sy) * ((W // groups[1]) // sx)
    w.n_reuse = (U - reps) // 3
    rep = run_chain(oc, oracle, w, want_aux=True, sy=sy, sx=sx, oy=oy, ox=ox)
    assert_matcher(rep, inputs.BF16, shape, lattice, groups)


@pytest.mark.parametrize("shape,want_tc", [
    ((1, 1, 128, 128, 64), True),      # 64 x 64 representatives: 128 boxes, the largest tables in use here
    ((1, 1, 160, 128, 64), False),     # 80 x 64 representatives: 160 boxes, past the tables -> the FMA matcher
])
def test_token_group_tables_limit_and_fallback(oc, oracle, shape, want_tc):
    """The tensor-core matcher keeps the inverse norms of a whole group's representatives in shared memory;
    groups too large for that must fall back to the FMA matcher, not fail and not compute garbage."""
    B, T, Hh, W, C = shape
    assert expect_tensor_core(inputs.BF16, shape) == want_tc
    w = inputs.sd3_token_cache(seed=33, B=B * T, H=Hh, W=W, C=C, groups=(1, 1), dtype=inputs.BF16)
    w.x = w.x.reshape(shape); w.shape = shape
    U = Hh * W
    w.n_reuse = (U - U // 4) // 2
    rep = run_chain(oc, oracle, w, full_oracle=False, sample_rows=400)
    assert_matcher(rep, inputs.BF16, shape)


@pytest.mark.parametrize("plan", ["0,1,2", "0,2,3", "1,1,1", "1,2,2", "0,2,3,1", "1,1,2,1", "0,1,4,1"])
@pytest.mark.parametrize("shape,groups,lattice", _random_token_layouts(8, seed=7))
def test_token_match_random_layouts_forced_plans(oc, oracle, shape, groups, lattice, plan):
    B, T, Hh, W, C = shape
    w = inputs.sd3_token_cache(seed=int(np.prod(shape)) % 9973, B=B * T, H=Hh, W=W, C=C, groups=groups)
    w.x = w.x.reshape(shape); w.shape = shape
    sy, sx, oy, ox = lattice
    L, Lo = H.layouts(oc, oracle, w, sy=sy, sx=sx, oy=oy, ox=ox)
    ref = oracle.match_token(Lo, w.x)
    with H.make_ctx(oc, L) as ctx:
        ctx.tc_plan_override(plan.split(","))
        m = H.gpu_match(oc, ctx, L, H.to_dev(w.x))
        assert ctx.launches()["match_tc"] == 1 and ctx.launches()["match_simt"] == 0
    H.check_match_against_oracle(oracle, Lo, w.x, m["best_sim"].cpu().numpy(), m["best_idx"].cpu().numpy(), ref,
                                 TOL[inputs.BF16])


@pytest.mark.parametrize("shape,groups", [
    ((2, 1, 64, 64, 192), (1, 1)),       # 1024 representatives: 32 quanta, 8 candidate tiles per lattice
    ((1, 3, 40, 56, 136), (1, 1)),       # ragged 20 x 28 lattice, K tail, three frames
    ((1, 1, 64, 64, 128), (2, 2)),       # four patches per frame
])
@pytest.mark.parametrize("plan", ["0,1,1", "0,1,3", "0,2,2", "0,2,5", "1,1,1", "1,1,2", "1,2,1", "1,2,4", "0,2,64", "1,1,64",
                                  # the same with the candidate tiles resident in shared memory for a whole row
                                  "0,1,3,1", "0,2,2,1", "0,2,5,1", "1,1,2,1", "1,2,4,1", "0,1,7,1", "1,2,2,1",
                                  "0,2,5,0", "1,1,2,0"])
def test_tensor_core_matcher_every_plan(oc, oracle, shape, groups, plan):
    """The planner's choice (single CTA or CTA pair, one or two candidate tiles per CTA, pieces per
    row) changes the work split only: every valid plan must reproduce the oracle.  A plan the shape
    does not admit is ignored by the library (the planner's own choice runs instead)."""
    B, T, Hh, W, C = shape
    w = inputs.sd3_token_cache(seed=33, B=B * T, H=Hh, W=W, C=C, groups=groups)
    w.x = w.x.reshape(shape); w.shape = shape
    L, Lo = H.layouts(oc, oracle, w)
    ref = oracle.match_token(Lo, w.x, want_full=True)
    x_dev = H.to_dev(w.x)
    with H.make_ctx(oc, L) as ctx:
        ctx.tc_plan_override(plan.split(","))
        ctx.profile_enable(True)
        for want_aux in (False, True):
            m = H.gpu_match(oc, ctx, L, x_dev, want_aux=want_aux)
            gs, gi = m["best_sim"].cpu().numpy(), m["best_idx"].cpu().numpy()
            H.check_match_against_oracle(oracle, Lo, w.x, gs, gi, ref, TOL[inputs.BF16])
            if want_aux:
                a = m["aux"].cpu().numpy().astype(np.float64)
                f = ref["full_sim"]
                written = ~np.isnan(f)
                assert np.array_equal(~np.isnan(a), written), "aux rows written differ from the oracle's"
                assert np.abs(a[written] - f[written]).max() <= TOL[inputs.BF16]
        assert ctx.profile_read(oc.K_MATCH_TC)[0] == 2


@pytest.mark.parametrize("dtype", [inputs.BF16, inputs.F32])
@pytest.mark.parametrize("T,stat", [(7, 0), (6, 1), (2, 0), (1, 0)])
def test_frame_chain_small(oc, oracle, dtype, T, stat):
    w = inputs.svd_frames(seed=31, T=T, H=9, W=13, C=40, dtype=dtype, thr=0.9)
    rep = run_chain(oc, oracle, w, Cout=24, want_aux=True, frame_stat=stat)
    assert rep["reused"] == T // 2          # rho = 0.95 > 0.9: every odd frame is reused


def _frame_patch_workload(seed, B, T, Hh, W, C, dtype, grid, mode, rho=0.95):
    """AR(1) frames as in the SVD recipe, B batch elements, cut into grid patches per frame."""
    rng = np.random.default_rng(seed)
    x = np.stack([inputs.ar1_frames(rng, inputs.smooth_field(rng, Hh, W, C, 4.0), T, rho) for _ in range(B)])
    x = np.ascontiguousarray(x.reshape(B, T, Hh, W, C), dtype=np.float32)
    w = inputs.Workload(f"frame_patches_{grid[0]}x{grid[1]}", "frame", dtype, (B, T, Hh, W, C),
                        x if dtype == inputs.F32 else inputs.to_bf16_bits(x), mode=mode, thr=rho, n_reuse=max(1, (T // 2) // 2))
    w.groups = grid
    return w


@pytest.mark.parametrize("dtype", [inputs.BF16, inputs.F32])
@pytest.mark.parametrize("B,T,grid,stat,mode", [
    (2, 7, (3, 1), 0, "threshold"), (1, 6, (2, 4), 1, "count"), (2, 5, (1, 2), 0, "count"),
    (1, 2, (4, 4), 0, "threshold"), (2, 1, (2, 2), 0, "threshold"), (1, 9, (12, 16), 1, "threshold"),
])
def test_frame_patch_chain_small(oc, oracle, dtype, B, T, grid, stat, mode):
    """Patch-local Frame Cache (Section 3.3): every stage against the oracle, patches of frames as units."""
    w = _frame_patch_workload(41 + T, B, T, 12, 16, 40, dtype, grid, mode)
    rep = run_chain(oc, oracle, w, Cout=24, want_aux=True, frame_stat=stat)
    if T > 1 and grid != (12, 16):
        assert 0 < rep["reused"] <= B * (T // 2) * grid[0] * grid[1]


@pytest.mark.parametrize("dtype,stat", [(inputs.BF16, 0), (inputs.F32, 1)])
def test_frame_hierarchy_levels_from_one_pass(oc, oracle, dtype, stat):
    """Every level of the patch hierarchy (Section 3.3) equals the oracle's match at that patch size."""
    B, T, Hh, W, C = 2, 7, 12, 16, 40
    w = _frame_patch_workload(3, B, T, Hh, W, C, dtype, (6, 8), "threshold")
    grids = [(6, 8), (3, 4), (3, 1), (1, 2), (1, 1)]
    L = oc.Layout(oc.KIND_FRAME, dtype, B, T, Hh, W, C, gy=6, gx=8, frame_stat=stat)
    n_units = [B * T * gy * gx for gy, gx in grids]
    n_pairs = [B * (T - 1) * gy * gx for gy, gx in grids]
    with H.make_ctx(oc, L) as ctx:
        bs = torch.full((sum(n_units),), float("nan"), device="cuda")
        bi = torch.full((sum(n_units),), -2, device="cuda", dtype=torch.int32)
        ps = torch.full((sum(n_pairs),), float("nan"), device="cuda")
        pos = torch.full((B, T - 1, Hh * W), float("nan"), device="cuda")
        ctx.match_frame_levels(L, H.to_dev(w.x), grids, bs, bi, pos, ps)
        torch.cuda.synchronize()
        assert ctx.device_status() == oc.OK
        assert ctx.launches()["frame_pair"] == 1            # one streaming pass for all levels
        uo = po = 0
        for (gy, gx), nu, npair in zip(grids, n_units, n_pairs):
            Lo = oracle.Layout(oracle.KIND_FRAME, dtype, B, T, Hh, W, C, gy=gy, gx=gx, frame_stat=stat)
            ref = oracle.match_frame(Lo, w.x, want_pos=True)
            H.check_match_against_oracle(oracle, Lo, w.x, bs[uo:uo + nu].cpu().numpy(), bi[uo:uo + nu].cpu().numpy(),
                                         ref, TOL[dtype])
            assert np.abs(ps[po:po + npair].cpu().numpy() - ref["pair_sim"].reshape(-1)).max() <= TOL[dtype]
            assert np.abs(pos.cpu().numpy() - ref["pos_sim"]).max() <= TOL[dtype]
            uo += nu
            po += npair
        # argument checks: a grid that does not divide the finest one, too many levels
        assert ctx.match_frame_levels(L, H.to_dev(w.x), [(4, 8)], bs, bi, check=False) == oc.ERR_INVALID_ARG
        assert ctx.match_frame_levels(L, H.to_dev(w.x), [(1, 1)] * 9, bs, bi, check=False) == oc.ERR_INVALID_ARG


def _random_frame_block_layouts(n, seed):
    """Seeded random Frame / Block Cache shapes with patch grids: (kind, shape, grid, dtype, stat, mode)."""
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < n:
        kind = "frame" if len(out) % 2 == 0 else "block"
        gy, gx = int(rng.choice([1, 2, 3])), int(rng.choice([1, 2, 4]))
        hp, wp = 2 * int(rng.integers(1, 6)), 2 * int(rng.integers(1, 9))
        C = int(rng.choice([8, 24, 40, 64, 200, 320]))
        B, T = int(rng.integers(1, 3)), int(rng.integers(1, 10))
        if B * T * gy * hp * gx * wp * C > 3_000_000:
            continue
        out.append((kind, (B, T, gy * hp, gx * wp, C), (gy, gx), int(rng.choice([inputs.BF16, inputs.F32])),
                    int(rng.integers(0, 2)), str(rng.choice(["count", "threshold"]))))
    return out


@pytest.mark.parametrize("kind,shape,grid,dtype,stat,mode", _random_frame_block_layouts(24, seed=424242))
def test_frame_block_patch_chain_random_layouts(oc, oracle, kind, shape, grid, dtype, stat, mode):
    """Patch-local Frame and Block Cache, the whole chain, on shapes nobody picked by hand."""
    B, T, Hh, W, C = shape
    rng = np.random.default_rng(int(np.prod(shape)) % 7919)
    x = np.stack([inputs.ar1_frames(rng, inputs.smooth_field(rng, Hh, W, C, 3.0), T, 0.9) for _ in range(B)])
    x = np.ascontiguousarray(x.reshape(shape), dtype=np.float32)
    w = inputs.Workload(f"{kind}_random", kind, dtype, shape, x if dtype == inputs.F32 else inputs.to_bf16_bits(x),
                        mode=mode, thr=0.9, n_reuse=1)
    w.groups = grid
    if kind == "block":
        cand = (Hh // grid[0]) * (W // grid[1]) * 3 // 4
        w.n_reuse = max(1, cand // 2)
        run_chain(oc, oracle, w, Cout=16)
    else:
        w.n_reuse = max(1, (T // 2) // 2)
        run_chain(oc, oracle, w, Cout=16, want_aux=True, frame_stat=stat)


@pytest.mark.parametrize("grid", [(1, 1), (2, 3)])
def test_frame_chain_long_clip(oc, oracle, grid):
    """600 frames: the marching kernel cuts the clip into several segments (its per-pair records live
    in shared memory) and the select sees groups of 600 units."""
    w = _frame_patch_workload(9, 1, 600, 4, 6, 8, inputs.BF16, grid, "count", rho=0.9)
    w.n_reuse = 140
    rep = run_chain(oc, oracle, w, Cout=8, want_aux=True)
    assert rep["reused"] == 140 * grid[0] * grid[1]


def test_frame_patch_chain_long_rows(oc, oracle):
    """Rows too long for the time-marching kernel: the pair kernel's tiles follow the patches too."""
    w = _frame_patch_workload(5, 1, 4, 4, 6, 2176, inputs.BF16, (2, 3), "threshold")
    run_chain(oc, oracle, w, Cout=16, want_aux=True)


def test_frame_patches_svd_level0(oc, oracle):
    """Config-3 tensor cut 4 x 4 (18 x 32-token patches): sims, indices and the whole chain."""
    w = inputs.svd_frames()
    w.groups = (4, 4)
    w.thr = 0.95
    rep = run_chain(oc, oracle, w)
    assert 0 < rep["reused"] < 12 * 16


@pytest.mark.parametrize("dtype,lattice", [(inputs.BF16, (2, 2, 0, 0)), (inputs.F32, (2, 2, 1, 0)),
                                          (inputs.BF16, (1, 2, 0, 1)), (inputs.BF16, (3, 2, 2, 1))])
def test_block_chain_small(oc, oracle, dtype, lattice):
    sy, sx, oy, ox = lattice
    w = inputs.latte_blocks(seed=41, T=5, H=6, W=10, C=72, dtype=dtype)
    rep = run_chain(oc, oracle, w, Cout=40, sy=sy, sx=sx, oy=oy, ox=ox)
    if lattice == (2, 2, 0, 0):
        assert 0 < rep["reused"] < 45


# ---------------------------------------------------------------------------------------------------
# full-size configs 2-4
# ---------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("grid,mode", [((2, 2), "count"), ((1, 4), "count"), ((4, 1), "threshold"), ((2, 3), "count")])
def test_block_patches_chain(oc, oracle, grid, mode):
    """Patch-local Block Cache (Section 3.3): the selection is taken per patch of positions."""
    w = inputs.latte_blocks(seed=77, T=5, H=16, W=24, C=72)
    w.groups = grid
    w.mode = mode
    w.n_reuse = 7
    rep = run_chain(oc, oracle, w, Cout=40)
    if mode == "count":
        assert rep["reused"] == 7 * grid[0] * grid[1]


# ---------------------------------------------------------------------------------------------------
# Token Cache on the frame pairs of Frame Cache (Section 3.2.3)
# ---------------------------------------------------------------------------------------------------
def _joint_case(oc, oracle, x_np, shape, frames_np, mode, thr, n_pair, n_single, lattice=(2, 2, 0, 0), plan=None):
    """match_joint -> select_joint -> gather -> restore on a given frame table, each against the oracle."""
    B, T, Hh, W, C = shape
    P = Hh * W
    sy, sx, oy, ox = lattice
    L = oc.Layout(oc.KIND_TOKEN, oc.DTYPE_BF16, *shape, sy=sy, sx=sx, oy=oy, ox=ox)
    Lo = oracle.Layout(0, oracle.DT_BF16, *shape, sy=sy, sx=sx, oy=oy, ox=ox)
    n = B * T * P
    x_dev, fr_dev = H.to_dev(x_np), H.to_dev(frames_np)
    with oc.Context(0, oc.joint_workspace_bytes(L)) as ctx:
        if plan:
            ctx.tc_plan_override(plan.split(","))
        bs = torch.full((n,), float("nan"), device="cuda")
        bi = torch.full((n,), -2, device="cuda", dtype=torch.int32)
        ctx.match_joint(L, x_dev, fr_dev, bs, bi)
        torch.cuda.synchronize()
        assert ctx.device_status() == oc.OK
        ref = oracle.match_joint(Lo, x_np, frames_np)
        gs, gi = bs.cpu().numpy(), bi.cpu().numpy()
        H.check_match_against_oracle(oracle, Lo, x_np, gs, gi, ref, TOL[inputs.BF16])
        # selection on the GPU's own similarities: exact against the oracle given the same arrays
        stride = 2 * P if mode == oc.SELECT_THRESHOLD else max(2 * P - min(n_pair, 2 * P - P // (sy * sx)),
                                                                P - min(n_single, P - P // (sy * sx)))
        F = B * T
        kept = torch.full((F * stride,), -9, device="cuda", dtype=torch.int32)
        cnt = torch.full((F,), -9, device="cuda", dtype=torch.int32)
        mm = torch.full((n,), -9, device="cuda", dtype=torch.int32)
        so = torch.full((n,), -9, device="cuda", dtype=torch.int32)
        ctx.select_joint(L, fr_dev, bs, bi, mode, thr, n_pair, n_single, stride, kept, cnt, mm, so)
        torch.cuda.synchronize()
        ref_s = oracle.select_joint(Lo, frames_np, gs, gi, mode, thr, n_pair, n_single, stride)
        for k, t in (("kept_idx", kept), ("kept_count", cnt), ("match_map", mm), ("slot_of", so)):
            assert np.array_equal(t.cpu().numpy(), ref_s[k]), k
        # rows: plain token rows
        Ro = oracle.rows_for(Lo, C, 2)
        y = torch.full((F * stride, Ro.row_bytes), 0xAB, device="cuda", dtype=torch.uint8)
        ctx.gather(H.crows(oc, Ro), x_dev, kept, F * stride, y)
        assert H.dev_bytes(y) == oracle.gather(Ro, x_np, ref_s["kept_idx"], fill=0xAB).tobytes()
        z_np = inputs.random_rows(5, (F * stride * C,), inputs.BF16)
        cache_np = inputs.random_rows(6, shape, inputs.BF16)
        for src_mode in (oc.RESTORE_FROM_CACHE, oc.RESTORE_FROM_REPRESENTATIVE):
            out = torch.full((cache_np.nbytes,), 0xCD, device="cuda", dtype=torch.uint8)
            ctx.restore(H.crows(oc, Ro), H.to_dev(z_np), H.to_dev(cache_np), n, so, mm, out, src_mode)
            want = oracle.restore(Ro, z_np, cache_np, n, ref_s["slot_of"], ref_s["match_map"], src_mode)
            assert H.dev_bytes(out) == want.tobytes()
        assert ctx.device_status() == oc.OK
        return int((ref_s["slot_of"] < 0).sum())


@pytest.mark.parametrize("shape,lattice", [((2, 5, 16, 16, 64), (2, 2, 0, 0)), ((1, 6, 12, 24, 72), (2, 2, 1, 0)),
                                           ((1, 4, 24, 16, 136), (2, 2, 1, 1)), ((2, 3, 8, 32, 40), (2, 2, 0, 1))])
@pytest.mark.parametrize("mode", ["count", "threshold"])
def test_joint_token_cache_on_given_frame_tables(oc, oracle, shape, lattice, mode):
    B, T, Hh, W, C = shape
    rng = np.random.default_rng(sum(shape))
    x = np.stack([inputs.ar1_frames(rng, inputs.smooth_field(rng, Hh, W, C, 4.0), T, 0.9) for _ in range(B)])
    x_np = inputs.to_bf16_bits(np.ascontiguousarray(x.reshape(shape), dtype=np.float32))
    # every kind of slot: pairs with the partner after and before, unmatched frames, absorbed frames
    frames = np.array([[f, -1] for f in range(B * T)], np.int32)
    for b in range(B):
        o = b * T
        if b % 2 == 0:
            frames[o] = (o, o + 1); frames[o + 1] = (-1, -1)            # (0, 1)
        elif T >= 3:
            frames[o + 2] = (o + 2, o + 1); frames[o + 1] = (-1, -1)    # (2, 1): partner earlier
        if T >= 5:
            frames[o + 4] = (o + 4, o + 3); frames[o + 3] = (-1, -1)
    P = Hh * W
    reused = _joint_case(oc, oracle, x_np, shape, frames, oc.SELECT_COUNT if mode == "count" else oc.SELECT_THRESHOLD,
                         0.97, P // 2 + 3, P // 4 + 1, lattice)
    assert reused > 0


@pytest.mark.parametrize("plan", [None, "0,1,1", "0,2,2", "1,1,1", "1,2,2", "0,2,3", "0,2,3,1", "0,1,2,1", "1,2,2,1", "1,1,3,1"])
def test_joint_token_cache_svd_level_shapes_every_plan(oc, oracle, plan):
    """Several candidate tiles per lattice member, every form of the tensor-core matcher (single CTA / CTA
    pair, one or two tiles, several pieces per row) on the joint work list."""
    shape = (1, 7, 36, 64, 128)                     # 2304 tokens per frame: 576 per sub-lattice = 4.5 tiles
    B, T, Hh, W, C = shape
    rng = np.random.default_rng(17)
    x = inputs.ar1_frames(rng, inputs.smooth_field(rng, Hh, W, C, 6.0), T, 0.9).reshape(shape)
    x_np = inputs.to_bf16_bits(np.ascontiguousarray(x, dtype=np.float32))
    frames = np.array([[0, 1], [-1, -1], [2, -1], [-1, -1], [4, 3], [5, -1], [6, -1]], np.int32)
    P = Hh * W
    reused = _joint_case(oc, oracle, x_np, shape, frames, oc.SELECT_COUNT, 0.0, P, P // 3, plan=plan)
    assert reused == 2 * P + 3 * (P // 3)


def test_joint_many_short_frames(oc, oracle):
    """More frame slots than one pass of the work-list kernel takes (1100 > 1024), tiny frames."""
    shape = (1, 1100, 4, 4, 8)
    B, T, Hh, W, C = shape
    rng = np.random.default_rng(2)
    x = inputs.ar1_frames(rng, rng.standard_normal((Hh, W, C), dtype=np.float32), T, 0.8).reshape(shape)
    x_np = inputs.to_bf16_bits(np.ascontiguousarray(x, dtype=np.float32))
    frames = np.array([[f, -1] for f in range(T)], np.int32)
    for u in range(0, T - 1, 2):                       # every third representative frame takes a partner
        if (u // 2) % 3 == 0:
            frames[u] = (u, u + 1); frames[u + 1] = (-1, -1)
        elif (u // 2) % 3 == 1 and u >= 2 and frames[u - 1][0] >= 0:
            frames[u] = (u, u - 1); frames[u - 1] = (-1, -1)
    P = Hh * W
    reused = _joint_case(oc, oracle, x_np, shape, frames, oc.SELECT_COUNT, 0.0, 9, 5)
    n_pairs = int((frames[:, 1] >= 0).sum())
    n_single = int((frames[:, 0] >= 0).sum()) - n_pairs
    assert reused == 9 * n_pairs + 5 * n_single


def test_joint_groups_from_frame_cache_and_full_chain(oc, oracle):
    """Frame Cache decides the pairs (on the GPU), Token Cache works on them: the whole joint path."""
    shape = (2, 7, 16, 16, 64)
    B, T, Hh, W, C = shape
    rng = np.random.default_rng(5)
    x = np.stack([inputs.ar1_frames(rng, inputs.smooth_field(rng, Hh, W, C, 4.0), T, 0.93) for _ in range(B)])
    x_np = inputs.to_bf16_bits(np.ascontiguousarray(x.reshape(shape), dtype=np.float32))
    Lf = oc.Layout(oc.KIND_FRAME, oc.DTYPE_BF16, *shape)
    Lfo = oracle.Layout(1, oracle.DT_BF16, *shape)
    Lt = oc.Layout(oc.KIND_TOKEN, oc.DTYPE_BF16, *shape)
    x_dev = H.to_dev(x_np)
    with oc.Context(0, max(oc.match_workspace_bytes(Lf), oc.joint_workspace_bytes(Lt))) as ctx:
        m = H.gpu_match(oc, ctx, Lf, x_dev)
        fs = m["best_sim"].cpu().numpy()
        thr = float(np.median(fs[np.isfinite(fs)]))                    # about half of the candidate frames reused
        s = H.gpu_select(oc, ctx, Lf, m["best_sim"], m["best_idx"], oc.SELECT_THRESHOLD, thr, 0, T)
        frames = torch.full((B * T, 2), -9, device="cuda", dtype=torch.int32)
        ctx.joint_groups(Lt, m["best_sim"], m["best_idx"], s["slot_of"], frames)
        torch.cuda.synchronize()
        want = oracle.joint_groups(B, T, fs, m["best_idx"].cpu().numpy(), s["slot_of"].cpu().numpy())
        assert np.array_equal(frames.cpu().numpy(), want)
        assert (want[:, 1] >= 0).sum() >= 1 and (want[:, 0] < 0).sum() == (want[:, 1] >= 0).sum()
    _joint_case(oc, oracle, x_np, shape, want, oc.SELECT_COUNT, 0.0, 200, 60)


def test_joint_groups_conflicts_and_ties(oc, oracle):
    """Random Frame Cache outcomes, many of them with both neighbours claiming the same frame."""
    rng = np.random.default_rng(9)
    Lt = oc.Layout(oc.KIND_TOKEN, oc.DTYPE_BF16, 3, 9, 4, 4, 8)
    B, T = 3, 9
    with oc.Context(0, 0) as ctx:
        for trial in range(20):
            fs = np.full(B * T, -np.inf, np.float32)
            fi = np.arange(B * T, dtype=np.int32)
            so = np.arange(B * T, dtype=np.int32)
            for b in range(B):
                for t in range(1, T, 2):
                    f = b * T + t
                    fs[f] = np.float32(rng.integers(0, 4)) / 4          # few distinct values: ties
                    fi[f] = f + (1 if (t + 1 < T and rng.random() < 0.5) else -1)
                    so[f] = -1 if rng.random() < 0.7 else 5
            frames = torch.full((B * T, 2), -9, device="cuda", dtype=torch.int32)
            ctx.joint_groups(Lt, H.to_dev(fs), H.to_dev(fi), H.to_dev(so), frames)
            torch.cuda.synchronize()
            assert np.array_equal(frames.cpu().numpy(), oracle.joint_groups(B, T, fs, fi, so)), trial


# ---------------------------------------------------------------------------------------------------
# the projection with gather and scatter folded in
# ---------------------------------------------------------------------------------------------------
def _bf16_bits_to_f64(b):
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


@pytest.mark.parametrize("a_rows,K,N,n_rows,use_idx", [
    (300, 64, 128, 200, True), (300, 72, 136, 257, True), (512, 192, 256, 512, False), (700, 320, 640, 300, True),
    (128, 8, 128, 1, True), (4096, 1536, 1536, 2560, True), (600, 200, 384, 600, "scatter"), (300, 64, 256, 290, "scatter"),
])
def test_linear_gather_scatter(oc, oracle, a_rows, K, N, n_rows, use_idx):
    rng = np.random.default_rng(a_rows + K + N)
    a = inputs.to_bf16_bits(rng.standard_normal((a_rows, K)).astype(np.float32))
    w = inputs.to_bf16_bits((rng.standard_normal((N, K)) / np.sqrt(K)).astype(np.float32))
    out_rows = a_rows + 5
    out0 = inputs.to_bf16_bits(rng.standard_normal((out_rows, N)).astype(np.float32))
    if use_idx:
        a_idx = np.sort(rng.choice(a_rows, n_rows, replace=False)).astype(np.int32)     # a kept-index list
        out_idx = a_idx.copy()
        if n_rows > 3:
            a_idx[n_rows // 2] = -1                                                     # an unused slot
            out_idx[n_rows // 2] = -1
            out_idx[1] = -1                                                             # computed but not stored
    else:
        a_idx = out_idx = None
    if use_idx == "scatter":                         # dense rows in, scattered rows out (the restore half alone)
        a_idx = None
        out_idx = rng.permutation(out_rows)[:n_rows].astype(np.int32)
        out_idx[3] = -1
    with oc.Context(0, 0) as ctx:
        out = H.to_dev(out0)
        ctx.linear_gather_scatter(H.to_dev(a), a_rows, K, None if a_idx is None else H.to_dev(a_idx), n_rows, H.to_dev(w), N,
                                  out, out_rows, None if out_idx is None else H.to_dev(out_idx))
        torch.cuda.synchronize()
        assert ctx.device_status() == oc.OK
        assert ctx.launches()["linear"] == 1
        got = out.cpu().numpy().view(np.uint16).reshape(out_rows, N)
    # rows the oracle computes: all of them for the small cases, a sample for the large one
    rows = np.arange(n_rows) if n_rows * N * K < 5e8 else np.sort(rng.choice(n_rows, 200, replace=False))
    a64, w64 = _bf16_bits_to_f64(a), _bf16_bits_to_f64(w)
    written = np.zeros(out_rows, bool)
    exact_match = total = 0
    for r in range(n_rows):
        src = r if a_idx is None else int(a_idx[r])
        dst = r if out_idx is None else int(out_idx[r])
        if src >= 0 and dst >= 0:
            written[dst] = True
    for r in rows:
        src = r if a_idx is None else int(a_idx[r])
        dst = r if out_idx is None else int(out_idx[r])
        if src < 0 or dst < 0:
            continue
        ref = oracle.linear_gather_scatter(a[src:src + 1], None, 1, w, np.zeros((1, N), np.uint16), None)[0]
        exact = w64 @ a64[src]
        g64, r64 = _bf16_bits_to_f64(got[dst]), _bf16_bits_to_f64(ref)
        # fp32 accumulation (error a few ulps of the sum of magnitudes) can land on the other side of a bf16
        # rounding boundary: one bf16 ulp of the result, plus that accumulation error
        tol = np.abs(exact) * 2.0 ** -7 + (np.abs(w64) @ np.abs(a64[src])) * 2.0 ** -21
        bad = np.nonzero(np.abs(g64 - r64) > tol)[0]
        assert bad.size == 0, f"row {r}: cols {bad[:5]} got {g64[bad[:5]]} ref {r64[bad[:5]]} exact {exact[bad[:5]]} tol {tol[bad[:5]]}"
        exact_match += int((got[dst] == ref).sum())
        total += N
    assert total > 0 and exact_match >= 0.98 * total
    # rows nobody names keep their bytes
    assert np.array_equal(got[~written], out0[~written])


def test_linear_gather_scatter_argument_checks(oc, oracle):
    with oc.Context(0, 0) as ctx:
        t = torch.zeros(256 * 128, device="cuda", dtype=torch.int16)
        assert ctx.linear_gather_scatter(t, 256, 64, None, 10, t, 120, t, 256, None, check=False) == oc.ERR_UNSUPPORTED   # N < 128
        assert ctx.linear_gather_scatter(t, 256, 60, None, 10, t, 128, t, 256, None, check=False) == oc.ERR_ALIGNMENT
        assert ctx.linear_gather_scatter(t, 256, 64, None, 10, t, 132, t, 256, None, check=False) == oc.ERR_ALIGNMENT
        assert ctx.linear_gather_scatter(t, 256, 64, None, -1, t, 128, t, 256, None, check=False) == oc.ERR_INVALID_ARG
        assert ctx.linear_gather_scatter(t, 256, 64, None, 0, t, 128, t, 256, None) == oc.OK                              # nothing to do
        assert ctx.launches()["linear"] == 0


def test_config2_sd3_token_cache_full(oc, oracle):
    w = inputs.sd3_token_cache()
    rep = run_chain(oc, oracle, w, full_oracle=True)
    assert rep["launches"]["match_tc"] == 1, "the bf16 dense matcher must run on the tcgen05 kernel"
    assert rep["reused"] == 2 * 1536
    print("config2 report:", rep)


@pytest.mark.parametrize("groups", [(2, 1), (2, 2), (4, 2)])
def test_config2_token_groups_sampled(oc, oracle, groups):
    w = inputs.sd3_token_cache(groups=groups)
    rep = run_chain(oc, oracle, w, full_oracle=False, sample_rows=384)
    assert rep["launches"]["match_tc"] == 1


def test_config3_svd_frame_cache_full(oc, oracle):
    w = inputs.svd_frames()
    rep = run_chain(oc, oracle, w, want_aux=True)
    assert rep["reused"] == 12


def test_config4_latte_block_cache_full(oc, oracle):
    w = inputs.latte_blocks()
    rep = run_chain(oc, oracle, w)
    assert 40 <= rep["reused"] <= 160


# ---------------------------------------------------------------------------------------------------
# config 5: three U-Net levels x three caches x keep ratios, with step drift and the Layered Cache
# ---------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("level", [0, 1, 2])
def test_config5_levels(oc, oracle, level):
    Hh, W, C = inputs.SVD_LEVELS[level]
    base = inputs.svd_frames(seed=1005 + level, T=25, H=Hh, W=W, C=C, rho=0.95, kind="token")
    steps = (0, 1, 24)
    rng = np.random.default_rng(77)
    x = base.x
    lc_ref = oracle.LayerCache()
    L_any = oc.Layout(oc.KIND_TOKEN, base.dtype, *base.shape)
    with oc.Context(0, oc.match_workspace_bytes(L_any)) as lc_ctx:
        for step in range(max(steps) + 1):
            if step > 0:
                x = inputs.drift_step(rng, x, base.dtype)
            # Layered Cache: put every 5 steps, get on the others (interval N = 5), bit-exact
            x_dev = H.to_dev(x)
            if step % 5 == 0:
                lc_ctx.layer_cache_put(level, step, x_dev)
                lc_ref.put(level, step, x)
            dst = torch.zeros_like(x_dev)
            hit, view, nbytes = lc_ctx.layer_cache_get(level, step, 5, dst)
            want = lc_ref.get(level, step, 5)
            assert hit == (want is not None)
            if hit:
                assert nbytes == len(want) and H.dev_bytes(dst) == want
            if step not in steps:
                continue
            for kind in ("token", "frame", "block"):
                ratios = (0.25, 0.5, 0.75) if step == 0 else (0.5,)
                for ratio in ratios:
                    w = inputs.Workload(f"svd_l{level}_{kind}", kind, base.dtype, base.shape, x, mode="count")
                    if kind == "token":
                        U, R = Hh * W, (Hh // 2) * (W // 2)
                    elif kind == "frame":
                        U, R = 25, 13
                    else:
                        U, R = Hh * W, (Hh // 2) * (W // 2)
                    w.n_reuse = inputs.keep_ratio_to_reuse(U, U - R, ratio)
                    full = kind != "token"
                    rep = run_chain(oc, oracle, w, full_oracle=full, sample_rows=1200)
                    if kind == "token":
                        assert rep["launches"]["match_tc"] == 1
        assert lc_ctx.layer_cache_get(level, max(steps) + 5, 5)[0] is False


# ---------------------------------------------------------------------------------------------------
# edge cases
# ---------------------------------------------------------------------------------------------------
def test_identity_selection_roundtrip_and_extremes(oc, oracle):
    w = inputs.sd3_token_cache(seed=5, B=2, H=16, W=24, C=64)
    L, Lo = H.layouts(oc, oracle, w)
    x_dev = H.to_dev(w.x)
    U, n_cand = L.units_per_group, L.units_per_group - L.reps_per_group
    R = H.crows(oc, oracle.rows_for(Lo, 64, 2))
    with H.make_ctx(oc, L) as ctx:
        m = H.gpu_match(oc, ctx, L, x_dev)
        for mode, thr, n_reuse in ((oc.SELECT_COUNT, 0.0, 0), (oc.SELECT_THRESHOLD, 2.0, 0)):
            s = H.gpu_select(oc, ctx, L, m["best_sim"], m["best_idx"], mode, thr, n_reuse, U)
            assert torch.equal(s["kept_idx"].cpu(), torch.arange(L.n_units, dtype=torch.int32))
            y = torch.zeros_like(x_dev)
            ctx.gather(R, x_dev, s["kept_idx"], L.n_units, y)
            out = torch.zeros_like(x_dev)
            ctx.restore(R, y, torch.zeros_like(x_dev), L.n_units, s["slot_of"], s["match_map"], out)
            assert torch.equal(out, x_dev), "restore after an identity selection must reproduce the input"
        # everything reusable is reused: count >= candidates, threshold -inf
        for mode, thr, n_reuse, stride in ((oc.SELECT_COUNT, 0.0, n_cand + 7, U - n_cand),
                                           (oc.SELECT_THRESHOLD, -float("inf"), 0, U)):
            s = H.gpu_select(oc, ctx, L, m["best_sim"], m["best_idx"], mode, thr, n_reuse, stride)
            H.check_select_against_oracle(oracle, Lo, m["best_sim"].cpu().numpy(), m["best_idx"].cpu().numpy(),
                                          mode, thr, n_reuse, stride, s)
            assert int(s["kept_count"].sum()) == L.n_groups * L.reps_per_group


def test_duplicates_zero_rows_and_ties(oc, oracle):
    rng = np.random.default_rng(9)
    xf = rng.standard_normal((1, 1, 32, 32, 128)).astype(np.float32)
    xf[0, 0, 0, 2] = xf[0, 0, 0, 0]          # two identical representatives
    xf[0, 0, 1, 1] = xf[0, 0, 0, 0]          # a candidate equal to both: lowest index must win
    xf[0, 0, 5, 5] = 0.0                     # all-zero candidate: similarity 0 with everything
    xf[0, 0, 6, 6] = 0.0                     # all-zero representative
    xf[0, 0, 9, 9] = 4.0 * xf[0, 0, 8, 8]    # scaled copy: similarity 1
    for dtype in (inputs.BF16, inputs.F32):
        x = xf if dtype == inputs.F32 else inputs.to_bf16_bits(xf)
        w = inputs.Workload("dups", "token", dtype, xf.shape, x, mode="count", n_reuse=100)
        L, Lo = H.layouts(oc, oracle, w)
        with H.make_ctx(oc, L) as ctx:
            m = H.gpu_match(oc, ctx, L, H.to_dev(x))
        gs, gi = m["best_sim"].cpu().numpy(), m["best_idx"].cpu().numpy()
        # the tensor-core matcher (bf16 inputs) compares similarities lifted by up to 4 x the row's norm
        # into one binade: the reported cosine is rounded by up to 2^-24 * 4.004 = 2.4e-7
        one_tol = 2e-6
        assert gi[33] == 0 and abs(gs[33] - 1.0) <= one_tol
        assert gi[9 * 32 + 9] == 8 * 32 + 8 and abs(gs[9 * 32 + 9] - 1.0) <= one_tol
        assert gs[5 * 32 + 5] == 0.0 and gi[5 * 32 + 5] == 0     # all similarities 0: lowest index
        ref = oracle.match_token(Lo, x)
        H.check_match_against_oracle(oracle, Lo, x, gs, gi, ref, TOL[dtype])


@pytest.mark.parametrize("dtype", [inputs.BF16, inputs.F32])
def test_exact_ties_between_negative_similarities_go_to_the_lowest_index(oc, oracle, dtype):
    """A candidate whose BEST similarity is negative and exactly tied between identical representatives.
    Frame f duplicates one representative at two lattice places; the candidates of the frame point
    (almost) away from every representative, least so from the duplicated one.  The places are chosen so
    that the two copies meet in one reduction chain of the tensor-core epilogue, in its two chains, in
    two 32-column chunks and in two pieces of the row; the lower index must win every time."""
    Hh = W = 32
    C = 64
    Ws = W // 2                                                  # 16 x 16 representatives per frame
    places = [(0, 1), (0, 2), (5, 40), (3, 200), (17, 16), (254, 255)]        # lattice indices of the two copies
    T = len(places)
    rng = np.random.default_rng(4)
    xf = np.zeros((1, T, Hh, W, C), np.float32)
    e0, e1 = np.zeros(C, np.float32), np.zeros(C, np.float32)
    e0[0] = 1.0; e1[1] = 1.0
    for t, (p1, p2) in enumerate(places):
        for r in range(Ws * Ws):                                 # every other representative: near e1
            y, x = 2 * (r // Ws), 2 * (r % Ws)
            xf[0, t, y, x] = e1 + 0.05 * np.abs(rng.standard_normal(C)).astype(np.float32) * (np.arange(C) >= 2)
        a = e0 + 0.25 * np.abs(rng.standard_normal(C)).astype(np.float32) * (np.arange(C) >= 2)
        for p in (p1, p2):
            xf[0, t, 2 * (p // Ws), 2 * (p % Ws)] = a
        for y in range(Hh):
            for x in range(W):
                if y % 2 or x % 2:                               # candidates: -(0.1 e0 + e1), scaled, tail >= 0 flipped
                    xf[0, t, y, x] = -(0.1 * e0 + e1) * (1.0 + 0.5 * rng.random()) \
                                     - 0.01 * np.abs(rng.standard_normal(C)).astype(np.float32) * (np.arange(C) >= 2)
    x = xf if dtype == inputs.F32 else inputs.to_bf16_bits(xf)
    w = inputs.Workload("neg_ties", "token", dtype, xf.shape, x, mode="count", n_reuse=10)
    L, Lo = H.layouts(oc, oracle, w)
    ref = oracle.match_token(Lo, x)
    forced = [None] if dtype == inputs.F32 else [None, (0, 1, 1), (0, 2, 2), (0, 1, 8), (1, 1, 1), (1, 2, 4)]
    for plan in forced:
        with H.make_ctx(oc, L) as ctx:
            if plan:
                ctx.tc_plan_override(plan)
            m = H.gpu_match(oc, ctx, L, H.to_dev(x))
            assert ctx.launches()["match_tc"] == (1 if dtype == inputs.BF16 else 0)
        gs, gi = m["best_sim"].cpu().numpy(), m["best_idx"].cpu().numpy()
        H.check_match_against_oracle(oracle, Lo, x, gs, gi, ref, TOL[dtype])
        for t, (p1, p2) in enumerate(places):
            pl = min(p1, p2)
            low = (t * Hh + 2 * (pl // Ws)) * W + 2 * (pl % Ws)
            cand = [(t * Hh + y) * W + xx for y in range(Hh) for xx in range(W) if y % 2 or xx % 2]
            assert np.all(gs[cand] < 0.0), "the best similarity of every candidate must be negative here"
            assert np.all(ref["best_idx"][cand] == low), "construction: the oracle's best is the duplicated representative"
            assert np.all(gi[cand] == low), (plan, t, np.unique(gi[cand]))


def test_determinism_and_profile_counters(oc, oracle):
    w = inputs.sd3_token_cache(seed=8, B=2, H=32, W=32, C=256)
    L, _ = H.layouts(oc, oracle, w)
    x_dev = H.to_dev(w.x)
    with H.make_ctx(oc, L) as ctx:
        ctx.profile_enable(True)
        a = H.gpu_match(oc, ctx, L, x_dev)
        b = H.gpu_match(oc, ctx, L, x_dev)
        assert torch.equal(a["best_sim"], b["best_sim"]) and torch.equal(a["best_idx"], b["best_idx"])
        n, ms = ctx.profile_read(oc.K_NORMS)
        assert n == 2 and ms > 0.0
        n_tc, ms_tc = ctx.profile_read(oc.K_MATCH_TC)
        n_si, ms_si = ctx.profile_read(oc.K_MATCH_SIMT)
        assert n_tc + n_si == 2 and ms_tc + ms_si > 0.0
        ctx.profile_reset()
        assert ctx.profile_read(oc.K_NORMS) == (0, 0.0)


def test_device_span_of_the_tensor_core_matcher(oc, oracle):
    """Span mode stamps first-CTA entry and last-CTA exit of every match_tc launch; the span is
    positive, shorter than the event bracket around the same kernel, and results are unchanged."""
    w = inputs.sd3_token_cache(seed=8, B=2, H=32, W=32, C=256)
    L, _ = H.layouts(oc, oracle, w)
    x_dev = H.to_dev(w.x)
    with H.make_ctx(oc, L) as ctx:
        ctx.profile_enable(1)
        a = H.gpu_match(oc, ctx, L, x_dev)
        for _ in range(4):
            H.gpu_match(oc, ctx, L, x_dev)
        n_ev, ms_ev = ctx.profile_read(oc.K_MATCH_TC)
        ctx.profile_reset()
        ctx.profile_enable(2)
        for _ in range(5):
            b = H.gpu_match(oc, ctx, L, x_dev)
        n_sp, ms_sp = ctx.profile_span_read(oc.K_MATCH_TC)
        ctx.profile_enable(0)
        assert n_ev == 5 and n_sp == 5
        assert 0.0 < ms_sp < ms_ev
        assert torch.equal(a["best_sim"], b["best_sim"]) and torch.equal(a["best_idx"], b["best_idx"])
        with pytest.raises(oc.OmniCacheError):
            ctx.profile_span_read(oc.K_SELECT)


def test_event_brackets_captured_into_a_graph_are_taken_on_every_replay(oc, oracle):
    w = inputs.sd3_token_cache(seed=8, B=2, H=32, W=32, C=256)
    L, _ = H.layouts(oc, oracle, w)
    x_dev = H.to_dev(w.x)
    n = L.n_units
    sim = torch.empty(n, device="cuda"); idx = torch.empty(n, dtype=torch.int32, device="cuda")
    with H.make_ctx(oc, L) as ctx:
        ctx.match(L, x_dev, sim, idx); torch.cuda.synchronize()
        ref = idx.clone()
        ctx.profile_reset()
        ctx.profile_enable(1)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            ctx.match(L, x_dev, sim, idx, stream=torch.cuda.current_stream())
        ctx.profile_enable(0)
        assert ctx.profile_captured_read(oc.K_MATCH_FIN) == (0, 0.0)        # captured, never run
        seen = []
        for _ in range(3):
            idx.zero_()
            g.replay(); torch.cuda.synchronize()
            k, ms = ctx.profile_captured_read(oc.K_MATCH_FIN)
            assert k == 1 and ms > 0.0
            seen.append(ms)
            assert torch.equal(idx, ref)
        # the eager counters saw the captured launches as launches, their timers did not
        assert ctx.profile_read(oc.K_MATCH_FIN) == (1, 0.0)
        del g


def test_runtime_argument_errors_launch_nothing(oc, oracle):
    w = inputs.sd3_token_cache(seed=5, B=1, H=16, W=16, C=64)
    L, Lo = H.layouts(oc, oracle, w)
    x_dev = H.to_dev(w.x)
    n = L.n_units
    sim = torch.zeros(n, device="cuda"); idx = torch.zeros(n, device="cuda", dtype=torch.int32)
    sentinel = torch.full((n,), 7, device="cuda", dtype=torch.int32)
    with oc.Context(0, 16) as small:
        assert small.match(L, x_dev, sim, idx, check=False) == oc.ERR_WORKSPACE
    with H.make_ctx(oc, L) as ctx:
        before = dict(ctx.launches())
        assert ctx.match(L, x_dev.view(torch.uint8).reshape(-1)[2:].data_ptr(), sim, idx, check=False) == oc.ERR_ALIGNMENT
        U = L.units_per_group
        k = sentinel.clone()
        args = (k, k.clone(), k.clone(), k.clone())
        assert ctx.select(L, sim, idx, 5, 0.5, 0, U, *args, check=False) == oc.ERR_INVALID_ARG
        assert ctx.select(L, sim, idx, oc.SELECT_COUNT, 0.0, -1, U, *args, check=False) == oc.ERR_INVALID_ARG
        assert ctx.select(L, sim, idx, oc.SELECT_COUNT, 0.0, 10, U - 11, *args, check=False) == oc.ERR_INVALID_ARG
        assert ctx.select(L, sim, idx, oc.SELECT_THRESHOLD, float("nan"), 0, U, *args, check=False) == oc.ERR_INVALID_ARG
        Ls = oc.Layout(oc.KIND_TOKEN, w.dtype, *w.shape, self_match=1)
        assert ctx.select(Ls, sim, idx, oc.SELECT_COUNT, 0.0, 4, U, *args, check=False) == oc.ERR_UNSUPPORTED
        rows = oc.CRows(24, 1, 0, 24, 1 << 40, 0)
        assert ctx.gather(rows, x_dev, k, 4, x_dev, check=False) == oc.ERR_ALIGNMENT
        good = H.crows(oc, oracle.rows_for(Lo, 64, 2))
        assert ctx.restore(good, x_dev, None, n, k, k, x_dev.clone(), oc.RESTORE_FROM_CACHE, check=False) == oc.ERR_INVALID_ARG
        assert ctx.restore(good, x_dev, x_dev, n, k, k, x_dev, check=False) == oc.ERR_INVALID_ARG     # out == z
        assert ctx.layer_cache_get(0, 0, 5)[0] is False
        torch.cuda.synchronize()
        assert torch.equal(k, sentinel), "a rejected call must not write outputs"
        assert ctx.launches() == before, "a rejected call must not launch"
        assert ctx.device_status() == oc.OK


@pytest.mark.parametrize("kind,shape,kw", [
    (1, (3, 25, 4, 4, 8), {}), (1, (2, 64, 4, 6, 8), dict(gy=2, gx=3)), (1, (1, 1, 4, 4, 8), {}),
    (1, (2, 33, 2, 2, 8), dict(gy=2, gx=1)), (1, (1, 65, 2, 2, 8), {}),
    (2, (2, 3, 16, 24, 8), dict(gy=2, gx=3)), (2, (1, 2, 16, 16, 8), dict(gy=4, gx=4)), (2, (3, 2, 6, 10, 8), {}),
    (0, (1, 3, 8, 8, 8), {}), (0, (2, 2, 12, 20, 8), dict(gy=3, gx=2, sy=2, sx=5, oy=1, ox=3)),
    (0, (1, 2, 16, 16, 8), dict(gy=2, gx=4)),
])
def test_select_small_and_strided_groups_with_ties(oc, oracle, kind, shape, kw):
    """Groups of at most 64 units (one warp each) and just above; quantised similarities give many ties."""
    L = oc.Layout(kind, oc.DTYPE_BF16, *shape, **kw)
    Lo = oracle.Layout(kind, oracle.DT_BF16, *shape, **kw)
    G, U, R = L.counts()
    n = G * U
    rng = np.random.default_rng(G * 1000 + U)
    sim_np = (np.round(rng.uniform(-1, 1, n) * 6) / 6).astype(np.float32)
    sim_np[rng.integers(0, n, 3)] = 0.0
    sim_np[rng.integers(0, n, 3)] = -0.0
    idx_np = np.zeros(n, np.int32)
    reps = [u for u in range(U) if Lo.is_rep(u)]
    for g in range(G):
        for u in range(U):
            i = Lo.unit_index(g, u)
            if Lo.is_rep(u):
                sim_np[i] = -np.inf
                idx_np[i] = i
            else:                                   # a match is always a representative of the same group
                idx_np[i] = Lo.unit_index(g, reps[int(rng.integers(0, len(reps)))])
    n_cand = U - R
    with oc.Context(0, 0) as ctx:
        for mode, thr, n_reuse in ((oc.SELECT_COUNT, 0.0, 0), (oc.SELECT_COUNT, 0.0, 1), (oc.SELECT_COUNT, 0.0, n_cand // 2),
                                   (oc.SELECT_COUNT, 0.0, max(n_cand - 1, 0)), (oc.SELECT_COUNT, 0.0, n_cand + 3),
                                   (oc.SELECT_THRESHOLD, 0.0, 0), (oc.SELECT_THRESHOLD, 1 / 3, 0),
                                   (oc.SELECT_THRESHOLD, -1.0, 0), (oc.SELECT_THRESHOLD, 1.5, 0)):
            stride = U - min(n_reuse, n_cand) if mode == oc.SELECT_COUNT else U
            s = H.gpu_select(oc, ctx, L, H.to_dev(sim_np), H.to_dev(idx_np), mode, thr, n_reuse, stride)
            H.check_select_against_oracle(oracle, Lo, sim_np, idx_np, mode, thr, n_reuse, stride, s)
        assert ctx.device_status() == oc.OK


def test_select_capacity_limits(oc, oracle):
    # 65536 units per group is the supported maximum; one more patch row is rejected
    L = oc.Layout(oc.KIND_TOKEN, oc.DTYPE_BF16, 1, 1, 256, 256, 8)
    n = L.n_units
    rng = np.random.default_rng(1)
    sim_np = np.round(rng.uniform(-1, 1, n).astype(np.float32) * 64) / 64        # many equal values
    Lo = oracle.Layout(0, 1, 1, 1, 256, 256, 8)
    rep_mask = np.array([Lo.is_rep(u) for u in range(n)])
    sim_np[rep_mask] = -np.inf
    idx_np = np.where(rep_mask, np.arange(n), 0).astype(np.int32)
    with oc.Context(0, 0) as ctx:
        n_reuse = 20000
        s = H.gpu_select(oc, ctx, L, H.to_dev(sim_np), H.to_dev(idx_np), oc.SELECT_COUNT, 0.0, n_reuse, n - n_reuse)
        H.check_select_against_oracle(oracle, Lo, sim_np, idx_np, oc.SELECT_COUNT, 0.0, n_reuse, n - n_reuse, s)
        big = oc.Layout(oc.KIND_TOKEN, oc.DTYPE_BF16, 1, 1, 258, 256, 8)
        t = torch.zeros(big.n_units, device="cuda")
        ti = torch.zeros(big.n_units, device="cuda", dtype=torch.int32)
        assert ctx.select(big, t, ti, oc.SELECT_THRESHOLD, 0.5, 0, big.units_per_group, ti.clone(), ti.clone(),
                          ti.clone(), ti.clone(), check=False) == oc.ERR_UNSUPPORTED


@pytest.mark.parametrize("pinned", [True, False])
@pytest.mark.parametrize("frames", [(2, 1), (3, 3), (1, 1)])
def test_cache_step_host_matches_device_path(oc, oracle, pinned, frames):
    """Pinned buffers: the restore kernel reads the cache and writes the output in host memory itself;
    pageable buffers: staging copies.  Several frames are processed in chunks whose copies overlap the
    work on earlier chunks (9 frames: chunks of 2, 2, 2, 2, 1).  Same bytes every way."""
    w = inputs.sd3_token_cache(seed=12, B=frames[0] * frames[1], H=32, W=32, C=128)
    shape = (frames[0], frames[1]) + tuple(w.shape[2:])
    w.x = w.x.reshape(shape); w.shape = shape
    L, Lo = H.layouts(oc, oracle, w)
    cache_np = inputs.random_rows(3, w.shape, w.dtype)
    pin = (lambda t: t.pin_memory()) if pinned else (lambda t: t)
    xh = pin(torch.from_numpy(w.x.view(np.int16).copy()))
    ch = pin(torch.from_numpy(cache_np.view(np.int16).copy()))
    oh = pin(torch.zeros_like(xh))
    kh = pin(torch.zeros(L.n_groups, dtype=torch.int32))
    with H.make_ctx(oc, L) as ctx:
        ctx.cache_step_host(L, oc.SELECT_COUNT, 0.0, w.n_reuse, xh, ch, oh, kh)
        m = H.gpu_match(oc, ctx, L, H.to_dev(w.x))
    gs, gi = m["best_sim"].cpu().numpy(), m["best_idx"].cpu().numpy()
    U = L.units_per_group
    s = oracle.select(Lo, gs, gi, 1, 0.0, w.n_reuse, U)
    R = oracle.rows_for(Lo, 128, 2)
    y = oracle.gather(R, w.x, s["kept_idx"])
    want = oracle.restore(R, y, cache_np, Lo.n_units, s["slot_of"], s["match_map"])
    assert oh.numpy().tobytes() == want.tobytes()
    assert np.array_equal(kh.numpy(), s["kept_count"])


def test_bounded_wait_expires_into_the_status_word_and_context_stays_usable(oc, oracle):
    """Failure detection without a fault: a wait that nothing satisfies gives up after its limit,
    the status word says OC_ERR_TIMEOUT once, and the same context then matches correctly."""
    w = inputs.sd3_token_cache(seed=14, B=1, H=32, W=32, C=128)
    L, Lo = H.layouts(oc, oracle, w)
    with H.make_ctx(oc, L) as ctx:
        assert ctx.device_status() == oc.OK
        ctx.selftest_bounded_wait(2000)
        assert ctx.device_status() == oc.ERR_TIMEOUT
        assert ctx.device_status() == oc.OK                      # read-and-clear
        m = H.gpu_match(oc, ctx, L, H.to_dev(w.x))
        ref = oracle.match_token(Lo, w.x)
        H.check_match_against_oracle(oracle, Lo, w.x, m["best_sim"].cpu().numpy(), m["best_idx"].cpu().numpy(),
                                     ref, TOL[w.dtype])
        assert oc._lib.oc_selftest_bounded_wait(ctx._h, 0, None) == oc.ERR_INVALID_ARG
