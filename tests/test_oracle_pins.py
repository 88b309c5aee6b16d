"""Pins for the CPU oracle: brute force in NumPy, library special cases, closed forms, invariants.

None of these re-call the oracle's own routine: the NumPy side uses strided slicing, a normalised
matrix product and full sorts, i.e. different index arithmetic from the C loops.
"""
import os

import numpy as np
import pytest

from paper_2607_23844_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def as_f64(x, dtype):
    return x.astype(np.float64) if dtype == inputs.F32 else inputs.bf16_bits_to_f32(x).astype(np.float64)


def np_token_match(x64, sy, sx, oy, ox, gy, gx, self_match=False, eps=1e-8):
    """All-pairs brute force per patch with NumPy slicing. Returns best_sim(f64), best_idx, full list."""
    B, T, H, W, C = x64.shape
    Hp, Wp = H // gy, W // gx
    idx = np.arange(B * T * H * W).reshape(B, T, H, W)
    n = B * T * H * W
    best_sim = np.full(n, -np.inf)
    best_idx = np.arange(n)
    second = np.full(n, -np.inf)
    fulls = []
    for b in range(B):
        for t in range(T):
            for py in range(gy):
                for px in range(gx):
                    xs = x64[b, t, py * Hp:(py + 1) * Hp, px * Wp:(px + 1) * Wp]
                    ids = idx[b, t, py * Hp:(py + 1) * Hp, px * Wp:(px + 1) * Wp]
                    if self_match:
                        reps, rid = xs.reshape(-1, C), ids.reshape(-1)
                        cands, cid = reps, rid
                    else:
                        mask = np.zeros((Hp, Wp), bool)
                        mask[oy::sy, ox::sx] = True
                        reps, rid = xs[mask], ids[mask]
                        cands, cid = xs[~mask], ids[~mask]
                    rn = reps / np.maximum(np.linalg.norm(reps, axis=1, keepdims=True), eps)
                    cn = cands / np.maximum(np.linalg.norm(cands, axis=1, keepdims=True), eps)
                    S = np.clip(cn @ rn.T, -1, 1)
                    if self_match:
                        np.fill_diagonal(S, -np.inf)
                    a = S.argmax(axis=1)                      # first maximum = lowest index
                    best_sim[cid] = S[np.arange(len(cid)), a]
                    best_idx[cid] = rid[a]
                    S2 = S.copy()
                    S2[np.arange(len(cid)), a] = -np.inf
                    second[cid] = S2.max(axis=1)
                    fulls.append((cid, rid, S))
    return best_sim, best_idx, second, fulls


# ---------------------------------------------------------------------------------------------
# hand-worked values (tests/golden/cosine_hand_cases.txt: integer vectors with rational cosines)
# ---------------------------------------------------------------------------------------------
def test_cosine_hand_cases(oracle):
    rows = []
    with open(os.path.join(GOLDEN, "cosine_hand_cases.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            a, b, num, den = line.split(";")
            rows.append((np.array(a.split(), np.float32), np.array(b.split(), np.float32),
                         float(num) / float(den)))
    assert len(rows) >= 6
    for a, b, want in rows:
        x = np.concatenate([a, b])
        got = oracle.cosine(x, oracle.DT_F32, 0, a.size, a.size)
        assert abs(got - want) < 1e-15, (a, b, got, want)
        # same values stored as bf16 (small integers are exact in bf16)
        xb = inputs.to_bf16_bits(x)
        assert abs(oracle.cosine(xb, oracle.DT_BF16, 0, a.size, a.size) - want) < 1e-15


def test_cosine_closed_forms(oracle):
    rng = np.random.default_rng(3)
    a = rng.standard_normal(257).astype(np.float32)
    for s, want in ((2.0, 1.0), (0.5, 1.0), (-4.0, -1.0)):      # powers of two: scaling is exact
        x = np.concatenate([a, (a * np.float32(s))])
        assert abs(oracle.cosine(x, 0, 0, 257, 257) - want) < 1e-14
    z = np.zeros(16, np.float32)
    assert oracle.cosine(np.concatenate([z, a[:16]]), 0, 0, 16, 16) == 0.0   # zero row -> 0 (eps floor)
    # operand order does not matter, and a transposed/offset read would break this antisymmetry pin
    b = rng.standard_normal(257).astype(np.float32)
    x = np.concatenate([a, b])
    assert oracle.cosine(x, 0, 0, 257, 257) == oracle.cosine(x, 0, 257, 0, 257)
    assert abs(oracle.cosine(np.concatenate([a, -b]), 0, 0, 257, 257) + oracle.cosine(x, 0, 0, 257, 257)) < 1e-15


def test_bf16_widening_is_exact(oracle):
    # every finite bf16 pattern widens to the fp32 with the same top bits: check through cos(a, e_k)
    vals = np.array([1.0, -2.5, 3.0e-3, 1.5e10, -7.0], np.float32)
    bits = inputs.to_bf16_bits(vals)
    back = inputs.bf16_bits_to_f32(bits).astype(np.float64)
    for k in range(vals.size):
        e = np.zeros(vals.size, np.float32); e[k] = 1.0
        x = np.concatenate([bits, inputs.to_bf16_bits(e)])
        got = oracle.cosine(x, 1, 0, vals.size, vals.size)
        assert abs(got - back[k] / np.linalg.norm(back)) < 1e-15


# ---------------------------------------------------------------------------------------------
# dense match vs NumPy brute force
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("shape,groups,lattice,dtype", [
    ((1, 1, 16, 16, 64), (1, 1), (2, 2, 0, 0), inputs.F32),
    ((2, 1, 8, 12, 24), (1, 1), (2, 2, 0, 0), inputs.BF16),
    ((1, 3, 8, 8, 16), (2, 2), (2, 2, 1, 0), inputs.BF16),
    ((2, 2, 8, 16, 8), (2, 4), (2, 2, 0, 1), inputs.F32),
    ((1, 1, 6, 9, 8), (1, 1), (3, 3, 1, 2), inputs.F32),
    ((1, 2, 4, 8, 8), (1, 2), (1, 2, 0, 1), inputs.BF16),
])
def test_match_token_bruteforce(oracle, shape, groups, lattice, dtype):
    rng = np.random.default_rng(11)
    xf = rng.standard_normal(shape).astype(np.float32)
    # plant duplicates so that arg-max ties and high similarities occur
    flat = xf.reshape(-1, shape[-1])
    flat[5] = flat[0]; flat[9] = flat[0]; flat[-1] = 2 * flat[3]
    x = xf if dtype == inputs.F32 else inputs.to_bf16_bits(xf)
    sy, sx, oy, ox = lattice
    L = oracle.Layout(oracle.KIND_TOKEN, dtype, *shape, sy=sy, sx=sx, oy=oy, ox=ox,
                      gy=groups[0], gx=groups[1])
    got = oracle.match_token(L, x, want_full=True)
    bs, bi, sec, fulls = np_token_match(as_f64(x, dtype), sy, sx, oy, ox, *groups)
    assert np.array_equal(got["best_idx"], bi)
    cand = np.isfinite(bs)
    assert np.allclose(got["best_sim"][cand], bs[cand], atol=1e-7, rtol=0)   # fp32 rounding of output
    assert np.all(np.isneginf(got["best_sim"][~cand]))
    assert np.allclose(got["second_sim"][cand], sec[cand].astype(np.float32), atol=1e-7, rtol=0)
    # full matrix, element by element, to 1e-12
    U = L.units_per_group
    for g, (cid, rid, S) in enumerate(fulls):
        loc = {L.unit_index(g, u): u for u in range(U)}
        rows = [loc[i] for i in cid]
        assert np.max(np.abs(got["full_sim"][g][rows] - S)) < 1e-12
    # representative/candidate counts
    assert cand.sum() == L.n_groups * (U - L.n_rep)


def test_match_token_self_match_tiny_config(oracle):
    w = inputs.tiny_token_cache()
    L = oracle.Layout(oracle.KIND_TOKEN, w.dtype, *w.shape, self_match=1)
    got = oracle.match_token(L, w.x, want_full=True)
    bs, bi, sec, fulls = np_token_match(w.x.astype(np.float64), 2, 2, 0, 0, 1, 1, self_match=True)
    assert np.array_equal(got["best_idx"], bi)
    assert np.allclose(got["best_sim"], bs, atol=1e-7, rtol=0)
    S = fulls[0][2]
    off = ~np.eye(256, dtype=bool)
    assert np.max(np.abs(got["full_sim"][0][off] - S[off])) < 1e-12
    # sanity bands of the recipe: planted copies are near 1, everything else far below the threshold
    assert (bs > 0.999).sum() >= 100 and ((bs > 0.6) & (bs < 0.999)).sum() == 0


def test_match_token_rows_subset(oracle):
    rng = np.random.default_rng(5)
    x = inputs.to_bf16_bits(rng.standard_normal((2, 2, 8, 8, 16)).astype(np.float32))
    L = oracle.Layout(oracle.KIND_TOKEN, oracle.DT_BF16, 2, 2, 8, 8, 16, gy=2, gx=2)
    full = oracle.match_token(L, x)
    rows = rng.choice(L.n_units, 40, replace=False)
    sub = oracle.match_token(L, x, rows=rows)
    assert np.array_equal(sub["best_idx"][rows], full["best_idx"][rows])
    assert np.array_equal(sub["best_sim"][rows], full["best_sim"][rows])
    untouched = np.setdiff1d(np.arange(L.n_units), rows)
    assert np.all(sub["best_idx"][untouched] == -2)


def test_match_token_library_special_case_midsize(oracle):
    """Normalise rows, one float64 matrix product, row max: the textbook form, at several tiles' size."""
    w = inputs.sd3_token_cache(seed=7, B=1, H=32, W=32, C=192)
    L = oracle.Layout(oracle.KIND_TOKEN, w.dtype, *w.shape)
    got = oracle.match_token(L, w.x)
    x64 = as_f64(w.x, w.dtype)[0, 0]
    reps = x64[0::2, 0::2].reshape(-1, 192)
    rid = np.arange(32 * 32).reshape(32, 32)[0::2, 0::2].reshape(-1)
    rn = reps / np.linalg.norm(reps, axis=1, keepdims=True)
    xn = x64.reshape(-1, 192) / np.linalg.norm(x64.reshape(-1, 192), axis=1, keepdims=True)
    S = xn @ rn.T
    cand = np.setdiff1d(np.arange(1024), rid)
    assert np.array_equal(got["best_idx"][cand], rid[S[cand].argmax(1)])
    assert np.allclose(got["best_sim"][cand], S[cand].max(1), atol=1e-7, rtol=0)


def test_match_token_duplicates_and_onehot(oracle):
    # exact duplicate of a representative -> similarity exactly 1 and that representative wins,
    # the lowest-indexed one when several representatives are identical
    rng = np.random.default_rng(2)
    x = rng.standard_normal((1, 1, 4, 4, 32)).astype(np.float32)
    x[0, 0, 0, 2] = x[0, 0, 0, 0]        # rep (0,2) == rep (0,0)
    x[0, 0, 1, 1] = x[0, 0, 0, 0]        # candidate copies them
    x[0, 0, 3, 3] = 4 * x[0, 0, 2, 2]    # scaled copy of rep (2,2)
    L = oracle.Layout(oracle.KIND_TOKEN, 0, 1, 1, 4, 4, 32)
    got = oracle.match_token(L, x)
    assert got["best_idx"][5] == 0 and abs(got["best_sim"][5] - 1) < 1e-7
    assert abs(got["second_sim"][5] - 1) < 1e-7
    assert got["best_idx"][15] == 10 and abs(got["best_sim"][15] - 1) < 1e-7
    # one-hot rows: similarities are 0 or 1
    eye = np.zeros((1, 1, 4, 4, 16), np.float32)
    for k in range(16):
        eye[0, 0, k // 4, k % 4, k % 4] = 1.0
    got = oracle.match_token(oracle.Layout(0, 0, 1, 1, 4, 4, 16), eye, want_full=True)
    f = got["full_sim"][0]
    f = f[~np.isnan(f)]
    assert set(np.unique(f)) <= {0.0, 1.0}
    # permuting channels changes no index
    perm = rng.permutation(32)
    got_p = oracle.match_token(L, np.ascontiguousarray(x[..., perm]))
    assert np.array_equal(got_p["best_idx"], oracle.match_token(L, x)["best_idx"])


# ---------------------------------------------------------------------------------------------
# frame and block match vs NumPy
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("T", [2, 5, 6])
@pytest.mark.parametrize("stat", [0, 1])
def test_match_frame_bruteforce(oracle, T, stat):
    rng = np.random.default_rng(T)
    B, H, W, Cc = 2, 3, 5, 16
    xf = rng.standard_normal((B, T, H, W, Cc)).astype(np.float32)
    xf[:, 1:] = 0.7 * xf[:, :-1] + 0.3 * xf[:, 1:]
    x = inputs.to_bf16_bits(xf)
    x64 = as_f64(x, inputs.BF16)
    L = oracle.Layout(oracle.KIND_FRAME, oracle.DT_BF16, B, T, H, W, Cc, frame_stat=stat)
    got = oracle.match_frame(L, x, want_pos=True)
    a, b = x64[:, 1:], x64[:, :-1]
    pos = (a * b).sum(-1) / (np.linalg.norm(a, axis=-1) * np.linalg.norm(b, axis=-1))
    if stat == 0:
        pair = pos.mean(axis=(2, 3))
    else:
        af, bf = a.reshape(B, T - 1, -1), b.reshape(B, T - 1, -1)
        pair = (af * bf).sum(-1) / (np.linalg.norm(af, axis=-1) * np.linalg.norm(bf, axis=-1))
    assert np.allclose(got["pos_sim"], pos.reshape(B, T - 1, -1), atol=1e-7, rtol=0)
    assert np.allclose(got["pair_sim"], pair, atol=1e-7, rtol=0)
    for bb in range(B):
        for t in range(T):
            i = bb * T + t
            if t % 2 == 0:
                assert got["best_idx"][i] == i and np.isneginf(got["best_sim"][i])
                continue
            opts = [(pair[bb, t - 1], i - 1)]
            if t + 1 < T:
                opts.append((pair[bb, t], i + 1))
            want = max(opts, key=lambda o: (o[0], -o[1]))
            assert got["best_idx"][i] == want[1]
            assert abs(got["best_sim"][i] - want[0]) < 1e-7


def patch_major(x, gy, gx):
    """Section 3.3's rearrangement, written with NumPy: (B,T,k,H/k,k,W/k,C) -> (B*k*k, T, (H/k)*(W/k), C)."""
    B, T, H, W, Cc = x.shape
    hp, wp = H // gy, W // gx
    return x.reshape(B, T, gy, hp, gx, wp, Cc).transpose(0, 2, 4, 1, 3, 5, 6).reshape(B * gy * gx, T, hp * wp, Cc)


@pytest.mark.parametrize("grid", [(2, 2), (1, 3), (3, 1), (2, 4), (6, 12)])
@pytest.mark.parametrize("stat", [0, 1])
def test_match_frame_patch_local_is_the_reshaped_problem(oracle, grid, stat):
    """Patch-local Frame Cache = the whole-frame rule applied to every row of the rearranged array."""
    gy, gx = grid
    rng = np.random.default_rng(100 + gy * 16 + gx)
    B, T, H, W, Cc = 2, 6, 6, 12, 8
    xf = rng.standard_normal((B, T, H, W, Cc)).astype(np.float32)
    xf[:, 1:] = 0.6 * xf[:, :-1] + 0.4 * xf[:, 1:]
    x = inputs.to_bf16_bits(xf)
    x64 = as_f64(x, inputs.BF16)
    L = oracle.Layout(oracle.KIND_FRAME, oracle.DT_BF16, B, T, H, W, Cc, gy=gy, gx=gx, frame_stat=stat)
    got = oracle.match_frame(L, x, want_pos=True)
    npatch = gy * gx
    assert L.n_groups == B * npatch and L.units_per_group == T and L.n_units == B * T * npatch
    xp = patch_major(x64, gy, gx)                                  # [B*np, T, Pp, C]
    a, b = xp[:, 1:], xp[:, :-1]
    pos = (a * b).sum(-1) / (np.linalg.norm(a, axis=-1) * np.linalg.norm(b, axis=-1))
    if stat == 0:
        pair = pos.mean(axis=-1)                                   # [B*np, T-1]
    else:
        af, bf = a.reshape(B * npatch, T - 1, -1), b.reshape(B * npatch, T - 1, -1)
        pair = (af * bf).sum(-1) / (np.linalg.norm(af, axis=-1) * np.linalg.norm(bf, axis=-1))
    want_pair = pair.reshape(B, npatch, T - 1).transpose(0, 2, 1)  # [B, T-1, np]
    assert np.allclose(got["pair_sim"].reshape(B, T - 1, npatch), want_pair, atol=1e-7, rtol=0)
    # per-position cosines stay in frame order
    a5, b5 = x64[:, 1:], x64[:, :-1]
    pos5 = (a5 * b5).sum(-1) / (np.linalg.norm(a5, axis=-1) * np.linalg.norm(b5, axis=-1))
    assert np.allclose(got["pos_sim"], pos5.reshape(B, T - 1, -1), atol=1e-7, rtol=0)
    for bb in range(B):
        for t in range(T):
            for pt in range(npatch):
                i = ((bb * T + t) * gy + pt // gx) * gx + pt % gx
                assert L.unit_index(bb * npatch + pt, t) == i
                if t % 2 == 0:
                    assert got["best_idx"][i] == i and np.isneginf(got["best_sim"][i])
                    continue
                opts = [(want_pair[bb, t - 1, pt], i - npatch)]
                if t + 1 < T:
                    opts.append((want_pair[bb, t, pt], i + npatch))
                want = max(opts, key=lambda o: (o[0], -o[1]))
                assert got["best_idx"][i] == want[1]
                assert abs(got["best_sim"][i] - want[0]) < 1e-7


def test_match_frame_patch_local_equals_whole_frame_match_of_each_patch(oracle):
    """Cutting a patch out and matching it as a frame of its own gives that patch's results."""
    rng = np.random.default_rng(77)
    B, T, H, W, Cc, gy, gx = 2, 5, 4, 6, 8, 2, 3
    x = rng.standard_normal((B, T, H, W, Cc)).astype(np.float32)
    x[:, 1:] = 0.5 * x[:, :-1] + 0.5 * x[:, 1:]
    hp, wp, npatch = H // gy, W // gx, gy * gx
    for stat in (0, 1):
        L = oracle.Layout(oracle.KIND_FRAME, 0, B, T, H, W, Cc, gy=gy, gx=gx, frame_stat=stat)
        got = oracle.match_frame(L, x)
        for py in range(gy):
            for px in range(gx):
                sub = np.ascontiguousarray(x[:, :, py * hp:(py + 1) * hp, px * wp:(px + 1) * wp, :])
                Ls = oracle.Layout(oracle.KIND_FRAME, 0, B, T, hp, wp, Cc, frame_stat=stat)
                ws = oracle.match_frame(Ls, sub)
                pt = py * gx + px
                assert np.array_equal(got["pair_sim"][:, :, pt], ws["pair_sim"])
                assert np.array_equal(got["best_sim"][pt::npatch], ws["best_sim"])
                assert np.array_equal(got["best_idx"][pt::npatch], ws["best_idx"] * npatch + pt)
    # the patch means, weighted equally (equal areas), average to the whole-frame mean
    L1 = oracle.Layout(oracle.KIND_FRAME, 0, B, T, H, W, Cc)
    Lp = oracle.Layout(oracle.KIND_FRAME, 0, B, T, H, W, Cc, gy=gy, gx=gx)
    assert np.allclose(oracle.match_frame(Lp, x)["pair_sim"].astype(np.float64).mean(-1),
                       oracle.match_frame(L1, x)["pair_sim"], atol=2e-7, rtol=0)


def test_match_frame_ar1_expectation(oracle):
    """AR(1) frames: E[cos(x_t, x_{t-1})] = rho for unit-variance stationary rows (closed form)."""
    rho = 0.95
    rng = np.random.default_rng(8)
    f0 = rng.standard_normal((8, 8, 320), dtype=np.float32)
    x = inputs.ar1_frames(rng, f0, 9, rho).reshape(1, 9, 8, 8, 320)
    L = oracle.Layout(oracle.KIND_FRAME, 0, 1, 9, 8, 8, 320)
    got = oracle.match_frame(L, x)
    assert np.all(np.abs(got["pair_sim"] - rho) < 3 * (1 - rho ** 2) / np.sqrt(320 * 64) + 2e-3)


@pytest.mark.parametrize("lattice", [(2, 2, 0, 0), (2, 2, 1, 1), (1, 2, 0, 0)])
def test_match_block_bruteforce(oracle, lattice):
    sy, sx, oy, ox = lattice
    rng = np.random.default_rng(4)
    B, T, H, W, Cc = 2, 3, 4, 6, 8
    x = inputs.to_bf16_bits(rng.standard_normal((B, T, H, W, Cc)).astype(np.float32))
    x64 = as_f64(x, inputs.BF16)
    desc = x64.transpose(0, 2, 3, 1, 4).reshape(B, H, W, T * Cc)       # (B, H*W, T*C) reshape
    L = oracle.Layout(oracle.KIND_BLOCK, 1, B, T, H, W, Cc, sy=sy, sx=sx, oy=oy, ox=ox)
    got = oracle.match_block(L, x)
    for b in range(B):
        for y in range(H):
            for xx in range(W):
                i = b * H * W + y * W + xx
                ry, rx = (y // sy) * sy + oy, (xx // sx) * sx + ox
                if (ry, rx) == (y, xx):
                    assert got["best_idx"][i] == i and np.isneginf(got["best_sim"][i])
                    continue
                a, r = desc[b, y, xx], desc[b, ry, rx]
                want = a @ r / (np.linalg.norm(a) * np.linalg.norm(r))
                assert got["best_idx"][i] == b * H * W + ry * W + rx
                assert abs(got["best_sim"][i] - want) < 1e-7


# ---------------------------------------------------------------------------------------------
# selection vs full sort in NumPy, and its invariants
# ---------------------------------------------------------------------------------------------
def np_select(L, best_sim, best_idx, mode, thr, n_reuse, stride):
    G, U = L.n_groups, L.units_per_group
    gi = np.array([[L.unit_index(g, u) for u in range(U)] for g in range(G)])
    is_rep = np.array([L.is_rep(u) for u in range(U)])
    n = G * U
    reuse = np.zeros(n, bool)
    for g in range(G):
        cand = gi[g][~is_rep] if not L.self_match else gi[g]
        if mode == 0:
            r = best_sim[cand] >= np.float32(thr)
            if L.self_match:
                r &= best_idx[cand] < cand
            reuse[cand[r]] = True
        else:
            order = np.lexsort((cand, -best_sim[cand].astype(np.float64)))   # sim desc, index asc
            reuse[cand[order[:n_reuse]]] = True
    kept_idx = np.full(G * stride, -1, np.int64)
    slot_of = np.full(n, -1, np.int64)
    cnt = np.zeros(G, np.int64)
    for g in range(G):
        kept = np.sort(gi[g][~reuse[gi[g]]])
        kept_idx[g * stride: g * stride + kept.size] = kept
        slot_of[kept] = g * stride + np.arange(kept.size)
        cnt[g] = kept.size
    mm = np.arange(n)
    for i in np.nonzero(reuse)[0]:
        m = i
        while reuse[m]:
            m = best_idx[m]
        mm[i] = m
    return kept_idx, cnt, mm, slot_of


@pytest.mark.parametrize("kind,shape,groups", [
    (0, (2, 1, 8, 8, 8), (1, 1)), (0, (1, 2, 8, 16, 8), (2, 2)),
    (1, (3, 7, 2, 2, 8), (1, 1)), (2, (2, 3, 6, 8, 8), (1, 1)),
    (1, (2, 7, 4, 6, 8), (2, 3)), (2, (2, 3, 8, 12, 8), (2, 3)),
])
@pytest.mark.parametrize("mode", [0, 1])
def test_select_bruteforce(oracle, kind, shape, groups, mode):
    rng = np.random.default_rng(kind * 10 + mode)
    x = rng.standard_normal(shape).astype(np.float32)
    L = oracle.Layout(kind, 0, *shape, gy=groups[0], gx=groups[1])
    m = oracle.match(L, x)
    bs = m["best_sim"].copy()
    cand = np.isfinite(bs)
    # quantise so that equal similarities occur and the index tie-break is exercised
    bs[cand] = np.round(bs[cand] * 8) / 8
    U = L.units_per_group
    n_cand = U - L.n_rep
    for thr, n_reuse in ((0.0, n_cand // 2), (0.125, 1), (2.0, 0), (-1.0, n_cand), (0.25, n_cand + 5)):
        stride = U if mode == 0 else U - min(n_reuse, n_cand)
        got = oracle.select(L, bs, m["best_idx"], mode, thr, n_reuse, stride)
        ki, cnt, mm, so = np_select(L, bs, m["best_idx"], mode, thr, n_reuse, stride)
        assert np.array_equal(got["kept_idx"], ki)
        assert np.array_equal(got["kept_count"], cnt)
        assert np.array_equal(got["match_map"], mm)
        assert np.array_equal(got["slot_of"], so)
        if mode == 1:
            assert np.all(cnt == U - min(n_reuse, n_cand))


def test_block_patches_confine_the_selection_only(oracle):
    """Patch-local Block Cache: matching is unchanged (own 2x2 neighbourhood), the count-mode
    selection is taken per patch; unit indices stay the frame positions."""
    rng = np.random.default_rng(55)
    shape, gy, gx = (2, 3, 8, 12, 8), 2, 3
    x = rng.standard_normal(shape).astype(np.float32)
    L1 = oracle.Layout(2, 0, *shape)
    Lp = oracle.Layout(2, 0, *shape, gy=gy, gx=gx)
    m1, mp = oracle.match_block(L1, x), oracle.match_block(Lp, x)
    assert np.array_equal(m1["best_sim"], mp["best_sim"]) and np.array_equal(m1["best_idx"], mp["best_idx"])
    B, T, Hh, W, Cc = shape
    hp, wp = Hh // gy, W // gx
    assert Lp.n_groups == B * gy * gx and Lp.units_per_group == hp * wp and Lp.n_rep == hp * wp // 4
    pos = np.arange(B * Hh * W).reshape(B, gy, hp, gx, wp).transpose(0, 1, 3, 2, 4).reshape(B * gy * gx, hp * wp)
    for g in range(Lp.n_groups):
        for u in (0, 1, wp, hp * wp - 1):
            assert Lp.unit_index(g, u) == pos[g, u]
    n_reuse = 5
    s = oracle.select(Lp, mp["best_sim"], mp["best_idx"], 1, 0.0, n_reuse, hp * wp - n_reuse)
    reused = s["slot_of"] < 0
    for g in range(Lp.n_groups):
        ids = pos[g]
        assert reused[ids].sum() == n_reuse
        cand = ids[np.isfinite(mp["best_sim"][ids])]
        order = cand[np.lexsort((cand, -mp["best_sim"][cand].astype(np.float64)))]
        assert set(order[:n_reuse]) == set(ids[reused[ids]])
        assert np.array_equal(s["kept_idx"][g * (hp * wp - n_reuse):(g + 1) * (hp * wp - n_reuse)], ids[~reused[ids]][np.argsort(ids[~reused[ids]])])
    # rows are still whole blocks addressed by frame position
    R1, Rp = oracle.rows_for(L1, Cc, 4), oracle.rows_for(Lp, Cc, 4)
    assert R1 == Rp


def test_select_self_match_chain(oracle):
    w = inputs.tiny_token_cache()
    L = oracle.Layout(0, 0, *w.shape, self_match=1)
    m = oracle.match_token(L, w.x)
    got = oracle.select(L, m["best_sim"], m["best_idx"], 0, 0.9)
    ki, cnt, mm, so = np_select(L, m["best_sim"], m["best_idx"], 0, 0.9, 0, 256)
    assert np.array_equal(got["kept_idx"], ki) and np.array_equal(got["match_map"], mm)
    reused = got["slot_of"] < 0
    assert 40 <= reused.sum() <= 110
    # every reused token maps to a kept token with a lower index and similar features
    assert np.all(got["slot_of"][got["match_map"][reused]] >= 0)
    assert np.all(got["match_map"][reused] < np.nonzero(reused)[0])


def test_select_invariants(oracle):
    w = inputs.sd3_token_cache(seed=3, B=2, H=16, W=16, C=32, groups=(2, 2))
    L = oracle.Layout(0, w.dtype, *w.shape, gy=2, gx=2)
    m = oracle.match_token(L, w.x)
    U, G = L.units_per_group, L.n_groups
    got = oracle.select(L, m["best_sim"], m["best_idx"], 1, 0.0, w.n_reuse, U - w.n_reuse)
    stride = U - w.n_reuse
    ki = got["kept_idx"].reshape(G, stride)
    assert np.all(np.diff(ki, axis=1) > 0)                                    # strictly ascending
    assert np.all(got["kept_count"] == stride)
    reused = np.nonzero(got["slot_of"] < 0)[0]
    assert reused.size == G * w.n_reuse
    assert np.array_equal(np.sort(np.concatenate([ki.reshape(-1), reused])), np.arange(L.n_units))
    rep_ids = [L.unit_index(g, u) for g in range(G) for u in range(U) if L.is_rep(u)]
    assert np.all(got["slot_of"][rep_ids] >= 0)                               # representatives kept
    assert np.array_equal(got["slot_of"][ki.reshape(-1)], np.arange(G * stride))
    # match_map of a reused token is a kept representative of its own group
    grp = {L.unit_index(g, u): g for g in range(G) for u in range(U)}
    for i in reused:
        r = got["match_map"][i]
        assert grp[r] == grp[i] and got["slot_of"][r] >= 0 and r in set(rep_ids)
    # the cut: every reused candidate is at least as similar as every kept candidate of its group
    for g in range(G):
        ids = np.array([L.unit_index(g, u) for u in range(U) if not L.is_rep(u)])
        r = got["slot_of"][ids] < 0
        assert m["best_sim"][ids][r].min() >= m["best_sim"][ids][~r].max()


# ---------------------------------------------------------------------------------------------
# Token Cache on the frame pairs of Frame Cache (Section 3.2.3)
# ---------------------------------------------------------------------------------------------
def test_joint_groups_hand_cases(oracle):
    """Which frames pair up, written out by hand for one clip of five frames (candidates 1 and 3)."""
    ninf = -np.inf
    def groups(sim1, idx1, so1, sim3, idx3, so3):
        fs = np.array([ninf, sim1, ninf, sim3, ninf], np.float32)
        fi = np.array([0, idx1, 2, idx3, 4], np.int32)
        so = np.array([0, so1, 1, so3, 2], np.int32)
        return oracle.joint_groups(1, 5, fs, fi, so).tolist()
    # both candidates reused, different representatives
    assert groups(0.9, 0, -1, 0.8, 4, -1) == [[0, 1], [-1, -1], [2, -1], [-1, -1], [4, 3]]
    # both claim frame 2: the more similar one wins, the other stays a group of its own
    assert groups(0.9, 2, -1, 0.8, 2, -1) == [[0, -1], [-1, -1], [2, 1], [3, -1], [4, -1]]
    assert groups(0.7, 2, -1, 0.8, 2, -1) == [[0, -1], [1, -1], [2, 3], [-1, -1], [4, -1]]
    assert groups(0.8, 2, -1, 0.8, 2, -1) == [[0, -1], [-1, -1], [2, 1], [3, -1], [4, -1]]   # equal: the earlier frame
    # a candidate that Frame Cache keeps (slot >= 0) claims nothing
    assert groups(0.9, 2, 3, 0.8, 2, -1) == [[0, -1], [1, -1], [2, 3], [-1, -1], [4, -1]]
    assert groups(0.9, 0, 1, 0.8, 4, 3) == [[f, -1] for f in range(5)]
    # two batch elements are independent
    fs = np.array([ninf, 0.9, ninf, ninf, 0.5, ninf], np.float32)
    fi = np.array([0, 2, 2, 3, 3, 5], np.int32)
    so = np.array([0, -1, 1, 2, -1, 3], np.int32)
    assert oracle.joint_groups(2, 3, fs, fi, so).tolist() == [[0, -1], [-1, -1], [2, 1], [3, 4], [-1, -1], [5, -1]]


def np_joint(x64, frames, sy, sx, oy, ox):
    """NumPy brute force of the joint match: per group normalised matrix product, row arg-max."""
    B, T, Hh, W, Cc = x64.shape
    P = Hh * W
    tok = x64.reshape(B * T * P, Cc)
    nrm = tok / np.maximum(np.linalg.norm(tok, axis=1, keepdims=True), 1e-8)
    yy, xx = np.divmod(np.arange(P), W)
    lat = (yy % sy == oy) & (xx % sx == ox)
    best = np.full(B * T * P, -np.inf)
    arg = np.arange(B * T * P)
    is_rep = np.zeros(B * T * P, bool)
    for slot, (u, t) in enumerate(frames):
        if u < 0:
            continue
        reps = u * P + np.nonzero(lat)[0]
        is_rep[reps] = True
        cands = u * P + np.nonzero(~lat)[0]
        if t >= 0:
            cands = np.concatenate([cands, t * P + np.arange(P)])
        sim = np.clip(nrm[cands] @ nrm[reps].T, -1, 1)
        k = sim.argmax(axis=1)                      # first maximum = lowest representative index
        best[cands] = sim[np.arange(cands.size), k]
        arg[cands] = reps[k]
    return best, arg, is_rep


@pytest.mark.parametrize("lattice", [(2, 2, 0, 0), (2, 2, 1, 0), (1, 2, 0, 1)])
def test_match_joint_bruteforce(oracle, lattice):
    sy, sx, oy, ox = lattice
    rng = np.random.default_rng(sum(lattice) + 11)
    B, T, Hh, W, Cc = 2, 5, 4, 6, 16
    xf = rng.standard_normal((B, T, Hh, W, Cc)).astype(np.float32)
    xf[:, 1:] = 0.6 * xf[:, :-1] + 0.4 * xf[:, 1:]
    x = inputs.to_bf16_bits(xf)
    x64 = as_f64(x, inputs.BF16)
    frames = np.array([[0, 1], [-1, -1], [2, -1], [3, -1], [4, -1],        # b = 0: (0,1) pair, 3 unmatched
                       [5, -1], [-1, -1], [7, 6], [-1, -1], [9, 8]], np.int32)   # b = 1: pairs with t < u
    L = oracle.Layout(0, oracle.DT_BF16, B, T, Hh, W, Cc, sy=sy, sx=sx, oy=oy, ox=ox)
    got = oracle.match_joint(L, x, frames)
    best, arg, is_rep = np_joint(x64, frames, sy, sx, oy, ox)
    assert np.array_equal(np.isneginf(got["best_sim"]), is_rep)
    assert np.array_equal(got["best_idx"][is_rep], np.nonzero(is_rep)[0])
    c = ~is_rep
    assert np.abs(got["best_sim"][c] - best[c]).max() < 1e-7
    differ = np.nonzero(c & (got["best_idx"] != arg))[0]
    for i in differ:       # float32 rounding of the NumPy product can reorder exact ties only
        assert abs(best[i] - got["second_sim"][i]) < 1e-7


def test_match_joint_reduces_to_token_cache_and_to_copies(oracle):
    rng = np.random.default_rng(3)
    B, T, Hh, W, Cc = 1, 4, 4, 4, 8
    x = rng.standard_normal((B, T, Hh, W, Cc)).astype(np.float32)
    L = oracle.Layout(0, 0, B, T, Hh, W, Cc)
    # no pairs: every frame on its own = per-frame Token Cache
    singles = np.array([[f, -1] for f in range(T)], np.int32)
    a, b = oracle.match_joint(L, x, singles), oracle.match_token(L, x)
    assert np.array_equal(a["best_sim"], b["best_sim"]) and np.array_equal(a["best_idx"], b["best_idx"])
    s_a = oracle.select_joint(L, singles, a["best_sim"], a["best_idx"], 1, 0.0, 0, 5, 11)
    s_b = oracle.select(L, b["best_sim"], b["best_idx"], 1, 0.0, 5, 11)
    for k in ("kept_idx", "kept_count", "match_map", "slot_of"):
        assert np.array_equal(s_a[k], s_b[k])
    # frame 1 an exact copy of frame 0, paired: a copy of a lattice token matches that token with
    # similarity 1; a copy of any other token has the same match as its original
    x[0, 1] = x[0, 0]
    frames = np.array([[0, 1], [-1, -1], [2, -1], [3, -1]], np.int32)
    m = oracle.match_joint(L, x, frames)
    P = Hh * W
    yy, xx = np.divmod(np.arange(P), W)
    lat = (yy % 2 == 0) & (xx % 2 == 0)
    assert np.allclose(m["best_sim"][P + np.nonzero(lat)[0]], 1.0, atol=1e-7)
    assert np.array_equal(m["best_idx"][P + np.nonzero(lat)[0]], np.nonzero(lat)[0])
    assert np.array_equal(m["best_sim"][P + np.nonzero(~lat)[0]], m["best_sim"][np.nonzero(~lat)[0]])
    assert np.array_equal(m["best_idx"][P + np.nonzero(~lat)[0]], m["best_idx"][np.nonzero(~lat)[0]])


@pytest.mark.parametrize("mode", [0, 1])
def test_select_joint_bruteforce_and_invariants(oracle, mode):
    rng = np.random.default_rng(40 + mode)
    B, T, Hh, W, Cc = 2, 5, 4, 6, 8
    P = Hh * W
    x = rng.standard_normal((B, T, Hh, W, Cc)).astype(np.float32)
    frames = np.array([[0, 1], [-1, -1], [2, -1], [3, -1], [4, -1],
                       [5, -1], [-1, -1], [7, 6], [-1, -1], [9, 8]], np.int32)
    L = oracle.Layout(0, 0, B, T, Hh, W, Cc)
    m = oracle.match_joint(L, x, frames)
    bs = m["best_sim"].copy()
    c = np.isfinite(bs)
    bs[c] = np.round(bs[c] * 8) / 8                  # equal similarities: the index tie-break matters
    for thr, n_pair, n_single in ((0.0, 20, 7), (0.125, 1, 0), (2.0, 0, 0), (-1.0, 42, 18), (0.25, 100, 100)):
        stride = 2 * P
        got = oracle.select_joint(L, frames, bs, m["best_idx"], mode, thr, n_pair, n_single, stride)
        reused = got["slot_of"] < 0
        for slot, (u, t) in enumerate(frames):
            lo = slot * stride
            if u < 0:
                assert got["kept_count"][slot] == 0 and np.all(got["kept_idx"][lo:lo + stride] == -1)
                continue
            fr = sorted(f for f in (u, t) if f >= 0)
            ids = np.concatenate([f * P + np.arange(P) for f in fr])         # time order = ascending index
            cand = ids[np.isfinite(bs[ids])]
            if mode == 0:
                want = cand[bs[cand] >= np.float32(thr)]
            else:
                order = cand[np.lexsort((cand, -bs[cand].astype(np.float64)))]
                want = order[:min(n_pair if t >= 0 else n_single, cand.size)]
            assert set(ids[reused[ids]]) == set(want)
            kept = ids[~reused[ids]]
            n = kept.size
            assert got["kept_count"][slot] == n
            assert np.array_equal(got["kept_idx"][lo:lo + n], kept) and np.all(got["kept_idx"][lo + n:lo + stride] == -1)
            assert np.array_equal(got["slot_of"][kept], lo + np.arange(n))
            assert np.array_equal(got["match_map"][kept], kept)
            assert np.array_equal(got["match_map"][ids[reused[ids]]], m["best_idx"][ids[reused[ids]]])
            # a reused token's stand-in is a kept representative of its own group
            assert np.all(~reused[got["match_map"][ids]]) and np.all(got["match_map"][ids[reused[ids]]] // P == u)


# gather / restore
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("kind", [0, 1, 2])
def test_identity_selection_roundtrip(oracle, kind):
    """Identity selection => kept_idx = 0..n-1, gather is a copy, restore(gather(x)) == x bitwise."""
    rng = np.random.default_rng(kind)
    shape = (2, 4, 4, 6, 8)
    x = inputs.to_bf16_bits(rng.standard_normal(shape).astype(np.float32))
    L = oracle.Layout(kind, 1, *shape)
    m = oracle.match(L, x)
    for mode, thr, n_reuse in ((0, 2.0, 0), (1, 0.0, 0)):
        s = oracle.select(L, m["best_sim"], m["best_idx"], mode, thr, n_reuse)
        assert np.array_equal(s["kept_idx"], np.arange(L.n_units))
        assert np.array_equal(s["match_map"], np.arange(L.n_units))
        R = oracle.rows_for(L, 8, 2)
        y = oracle.gather(R, x, s["kept_idx"])
        back = oracle.restore(R, y, np.zeros_like(x), L.n_units, s["slot_of"], s["match_map"])
        assert back.tobytes() == x.tobytes()
        if kind != 2:
            assert y.tobytes() == x.tobytes()
        else:   # block rows: the (T, HW, C) -> (HW, T, C) permutation
            want = x.reshape(2, 4, 24, 8).transpose(0, 2, 1, 3)
            assert y.tobytes() == np.ascontiguousarray(want).tobytes()


@pytest.mark.parametrize("kind", [0, 1, 2])
def test_restore_sources_no_averaging(oracle, kind):
    rng = np.random.default_rng(20 + kind)
    shape = (2, 6, 4, 4, 8)
    Cout = 12
    x = rng.standard_normal(shape).astype(np.float32)
    L = oracle.Layout(kind, 0, *shape)
    m = oracle.match(L, x)
    n_cand = L.units_per_group - L.n_rep
    s = oracle.select(L, m["best_sim"], m["best_idx"], 1, 0.0, n_cand // 2, L.units_per_group - n_cand // 2)
    R = oracle.rows_for(L, Cout, 4)
    out_shape = shape[:-1] + (Cout,)
    cache = rng.standard_normal(out_shape).astype(np.float32)
    n_slots = s["kept_idx"].size
    z = rng.standard_normal((n_slots, R.row_bytes // 4)).astype(np.float32)
    out = oracle.restore(R, z, cache, L.n_units, s["slot_of"], s["match_map"]).view(np.float32)

    def unit_rows(t):      # [n_units, row elements] view of a [B,T,H,W,Cout] tensor, NumPy transposes
        if kind == 0:
            return t.reshape(-1, Cout)
        if kind == 1:
            return t.reshape(L.B * L.T, -1)
        return np.ascontiguousarray(t.reshape(L.B, L.T, L.H * L.W, Cout).transpose(0, 2, 1, 3)).reshape(L.B * L.H * L.W, -1)

    o, c = unit_rows(out.reshape(out_shape)), unit_rows(cache)
    for i in range(L.n_units):
        want = z[s["slot_of"][i]] if s["slot_of"][i] >= 0 else c[i]
        assert o[i].tobytes() == want.tobytes()
    # cold start: skipped units take the fresh row of their representative
    out2 = oracle.restore(R, z, None, L.n_units, s["slot_of"], s["match_map"],
                          src_mode=oracle.SRC_REPRESENTATIVE).view(np.float32)
    o2 = unit_rows(out2.reshape(out_shape))
    for i in range(L.n_units):
        assert o2[i].tobytes() == z[s["slot_of"][s["match_map"][i]]].tobytes()
    # in place: skipped rows untouched, computed rows overwritten
    c2 = cache.copy()
    oracle.restore(R, z, c2, L.n_units, s["slot_of"], s["match_map"], in_place=True)
    assert c2.tobytes() == out.tobytes()
    # gather lists exactly the kept rows of x in ascending order
    Rx = oracle.rows_for(L, shape[-1], 4)
    y = oracle.gather(Rx, x, s["kept_idx"]).view(np.float32)
    xr = unit_rows_generic(x, L)
    for slot, i in enumerate(s["kept_idx"]):
        if i >= 0:
            assert y[slot].tobytes() == xr[i].tobytes()


def patch_rows(t, gy, gx):
    """[B*T*gy*gx, (H/gy)*(W/gx)*C] rows of the frame patches, unit order ((b*T+t)*gy+py)*gx+px."""
    B, T, H, W, Cc = t.shape
    hp, wp = H // gy, W // gx
    return np.ascontiguousarray(t.reshape(B, T, gy, hp, gx, wp, Cc).transpose(0, 1, 2, 4, 3, 5, 6)).reshape(
        B * T * gy * gx, hp * wp * Cc)


@pytest.mark.parametrize("grid", [(2, 3), (1, 2), (4, 1)])
def test_frame_patch_rows_gather_restore(oracle, grid):
    """Patch-local Frame Cache moves patches of frames: the rows are the NumPy patch slices."""
    gy, gx = grid
    rng = np.random.default_rng(300 + gy * 8 + gx)
    shape = (2, 5, 4, 6, 8)
    Cout = 12
    x = rng.standard_normal(shape).astype(np.float32)
    x[:, 1:] = 0.5 * x[:, :-1] + 0.5 * x[:, 1:]
    L = oracle.Layout(oracle.KIND_FRAME, 0, *shape, gy=gy, gx=gx)
    m = oracle.match(L, x)
    # identity selection: gather is the patch-major copy, restore brings the frames back
    s0 = oracle.select(L, m["best_sim"], m["best_idx"], 0, 2.0, 0)
    Rx = oracle.rows_for(L, shape[-1], 4)
    y0 = oracle.gather(Rx, x, s0["kept_idx"]).view(np.float32)
    xr = patch_rows(x, gy, gx)
    assert np.array_equal(np.sort(s0["kept_idx"]), np.arange(L.n_units))
    assert y0.reshape(L.n_units, -1).tobytes() == xr[s0["kept_idx"]].tobytes()
    back = oracle.restore(Rx, y0, np.zeros_like(x), L.n_units, s0["slot_of"], s0["match_map"])
    assert back.tobytes() == x.tobytes()
    # a real selection: every output patch is bit-identical to exactly one source
    thr = float(np.median(m["best_sim"][np.isfinite(m["best_sim"])]))
    s = oracle.select(L, m["best_sim"], m["best_idx"], 0, thr, 0)
    assert 0 < (s["slot_of"] < 0).sum() < L.n_units
    y = oracle.gather(Rx, x, s["kept_idx"]).view(np.float32).reshape(s["kept_idx"].size, -1)
    for slot, i in enumerate(s["kept_idx"]):
        if i >= 0:
            assert y[slot].tobytes() == xr[i].tobytes()
    R = oracle.rows_for(L, Cout, 4)
    out_shape = shape[:-1] + (Cout,)
    cache = rng.standard_normal(out_shape).astype(np.float32)
    z = rng.standard_normal((s["kept_idx"].size, R.row_bytes // 4)).astype(np.float32)
    out = oracle.restore(R, z, cache, L.n_units, s["slot_of"], s["match_map"]).view(np.float32)
    o, c = patch_rows(out.reshape(out_shape), gy, gx), patch_rows(cache, gy, gx)
    for i in range(L.n_units):
        want = z[s["slot_of"][i]] if s["slot_of"][i] >= 0 else c[i]
        assert o[i].tobytes() == want.tobytes()
        # the stand-in of a skipped patch is the same patch position of an adjacent frame
        if s["slot_of"][i] < 0:
            assert abs(s["match_map"][i] - i) == gy * gx


def unit_rows_generic(t, L):
    Cc = t.shape[-1]
    if L.kind == 0:
        return t.reshape(-1, Cc)
    if L.kind == 1:
        return t.reshape(L.B * L.T, -1)
    return np.ascontiguousarray(t.reshape(L.B, L.T, L.H * L.W, Cc).transpose(0, 2, 1, 3)).reshape(L.B * L.H * L.W, -1)


def test_linear_gather_scatter_pins(oracle):
    """bf16 rounding by hand, identity weights, a library matmul, untouched rows."""
    # rounding to 8 significant bits, ties to even: 1 + 2^-8 is a tie -> 1.0 (even), 1 + 3*2^-8 -> 1 + 2^-6
    v = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20, -0.3, 3.0e5, 0.0])
    bits = oracle._f64_to_bf16_rne(v)
    back = oracle._bf16_to_f64(bits)
    assert back[0] == 1.0 and back[1] == 1.0 and back[2] == 1.0 + 2.0 ** -6 and back[3] == 1.0 + 2.0 ** -7
    assert back[6] == 0.0 and abs(back[4] + 0.3) <= 0.3 * 2.0 ** -8 and abs(back[5] - 3.0e5) <= 3.0e5 * 2.0 ** -8
    assert np.array_equal(oracle._f64_to_bf16_rne(back), bits)                 # bf16 values are fixed points
    rng = np.random.default_rng(12)
    Ra, K, N, Ro = 20, 24, 16, 30
    a = inputs.to_bf16_bits(rng.standard_normal((Ra, K)).astype(np.float32))
    w = inputs.to_bf16_bits(rng.standard_normal((N, K)).astype(np.float32))
    out0 = inputs.to_bf16_bits(rng.standard_normal((Ro, N)).astype(np.float32))
    a_idx = np.array([3, 7, -1, 19, 0, 7], np.int32)
    out_idx = np.array([5, 29, 2, -1, 11, 0], np.int32)
    got = oracle.linear_gather_scatter(a, a_idx, 6, w, out0, out_idx)
    a64, w64 = oracle._bf16_to_f64(a), oracle._bf16_to_f64(w)
    written = {5: 3, 29: 7, 11: 0, 0: 7}                                        # dst -> src (rows 2 and 3 skipped)
    for dst in range(Ro):
        if dst in written:
            exact = a64[written[dst]] @ w64.T                                   # library matmul in float64
            y = oracle._bf16_to_f64(got[dst])
            assert np.all(np.abs(y - exact) <= np.abs(exact) * 2.0 ** -8 + 1e-30)
        else:
            assert np.array_equal(got[dst], out0[dst])
    # identity weights: the output rows ARE the gathered rows; no index arrays: plain rows
    eye = inputs.to_bf16_bits(np.eye(K, dtype=np.float32))
    y = oracle.linear_gather_scatter(a, None, Ra, eye, np.zeros((Ra, K), np.uint16), None)
    assert np.array_equal(y, a)
    # one hand case: [1, 2] . [[3, 4], [0.5, -1]] = [11, -1.5]
    ah = inputs.to_bf16_bits(np.array([[1.0, 2.0]], np.float32))
    wh = inputs.to_bf16_bits(np.array([[3.0, 4.0], [0.5, -1.0]], np.float32))
    yh = oracle._bf16_to_f64(oracle.linear_gather_scatter(ah, None, 1, wh, np.zeros((1, 2), np.uint16), None))
    assert yh.tolist() == [[11.0, -1.5]]


def test_layer_cache_rule(oracle):
    lc = oracle.LayerCache()
    a = np.arange(100, dtype=np.float32)
    assert lc.get(3, 0, 5) is None
    lc.put(3, 10, a)
    for step, hit in ((9, False), (10, True), (14, True), (15, False), (100, False)):
        got = lc.get(3, step, 5)
        assert (got is not None) == hit
        if hit:
            assert got == a.tobytes()
    assert lc.get(4, 10, 5) is None
    lc.put(3, 15, a + 1)
    assert lc.get(3, 14, 5) is None and lc.get(3, 16, 5) == (a + 1).tobytes()
    lc.clear()
    assert lc.get(3, 16, 5) is None


# ---------------------------------------------------------------------------------------------
# Layered Cache schedule proposal (Algorithm 1)
# ---------------------------------------------------------------------------------------------
def test_schedule_proposal_hand_cases(oracle):
    path = os.path.join(os.path.dirname(__file__), "golden", "schedule_hand_cases.txt")
    n = 0
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        Ls, Qs, s_r, exp = [f.strip() for f in line.split(";")]
        got = oracle.schedule_proposal([float(v) for v in Ls.split()], [float(v) for v in Qs.split()], float(s_r))
        assert got == [int(v) for v in exp.split()], line
        n += 1
    assert n == 7


def test_schedule_proposal_is_the_shortest_sorted_prefix_that_meets_the_budget(oracle):
    """Exact-rational restatement: sort by (Q/L, index) with Fractions, take the shortest prefix whose
    latency sum reaches (1 - 1/s_r) * sum(L).  Inputs are small dyadic rationals, so the oracle's
    doubles are exact too and the two must agree to the index."""
    from fractions import Fraction as Fr
    rng = np.random.default_rng(5)
    for trial in range(200):
        n = int(rng.integers(1, 9))
        L = [Fr(int(rng.integers(1, 64)), 8) for _ in range(n)]
        Q = [Fr(int(rng.integers(0, 64)), 16) for _ in range(n)]
        s_r = Fr(int(rng.integers(8, 64)), 8)                       # 1 .. 8 in eighths
        order = sorted(range(n), key=lambda i: (Q[i] / L[i], i))
        target = (1 - 1 / s_r) * sum(L)
        exp, saved = [], Fr(0)
        for i in order:
            if not saved < target:
                break
            exp.append(i); saved += L[i]
        got = oracle.schedule_proposal([float(v) for v in L], [float(v) for v in Q], float(s_r))
        # 1/s_r may round in binary; the budget then moves by one ulp, which only matters when a prefix
        # sum lands exactly on it: accept either side in that single case
        if got != exp:
            pref = [sum(L[i] for i in order[:k]) for k in range(n + 1)]
            assert any(p == target for p in pref) and abs(len(got) - len(exp)) == 1 and got[:len(exp)] == exp[:len(got)]
        else:
            assert got == exp
        # invariants that hold whatever the rounding
        assert got == order[:len(got)]
        if got:
            assert sum(L[i] for i in got[:-1]) < target or abs(float(sum(L[i] for i in got[:-1]) - target)) < 1e-12
    assert oracle.schedule_proposal([1.0, 2.0], [0.5, 0.1], 1.0) == []
    assert oracle.schedule_proposal([1.0, 2.0], [0.5, 0.1], 1e9) == [1, 0]
    # a larger target speedup never takes fewer candidates
    L = list(rng.uniform(0.5, 4.0, 30)); Q = list(rng.uniform(0.0, 1.0, 30))
    sizes = [len(oracle.schedule_proposal(L, Q, s)) for s in (1.0, 1.1, 1.5, 2.0, 3.0, 10.0)]
    assert sizes == sorted(sizes) and sizes[0] == 0 and sizes[-1] <= 30


# ---------------------------------------------------------------------------------------------
# input recipes: sanity bands (properties of the generators, not parity targets)
# ---------------------------------------------------------------------------------------------
def test_input_recipes_shapes_and_bands(oracle):
    w = inputs.sd3_token_cache(seed=1002, B=1, H=32, W=32, C=96)
    assert w.x.dtype == np.uint16 and w.x.shape == (1, 1, 32, 32, 96)
    assert w.n_reuse == (1024 - 256) // 2
    f = inputs.bf16_bits_to_f32(w.x).astype(np.float64)
    assert 0.7 < f.var() < 1.4
    # neighbouring tokens of the smooth field are strongly correlated, distant ones are not
    a, b, c = f[0, 0, :, :-1], f[0, 0, :, 1:], np.roll(f[0, 0], 16, axis=1)
    near = (a * b).sum(-1) / (np.linalg.norm(a, axis=-1) * np.linalg.norm(b, axis=-1))
    far = (f[0, 0] * c).sum(-1) / (np.linalg.norm(f[0, 0], axis=-1) * np.linalg.norm(c, axis=-1))
    assert near.mean() > 0.95 and abs(far.mean()) < 0.3
    blk = inputs.latte_blocks(T=4, H=8, W=8, C=64)
    L = oracle.Layout(2, blk.dtype, *blk.shape)
    sims = oracle.match_block(L, blk.x)["best_sim"]
    sims = sims[np.isfinite(sims)]
    assert sims.min() < 0.85 < sims.max()
    assert inputs.keep_ratio_to_reuse(9216, 6912, 0.25) == 6912
    assert inputs.keep_ratio_to_reuse(9216, 6912, 0.5) == 4608
    assert inputs.keep_ratio_to_reuse(9216, 6912, 0.75) == 2304
    # bf16 rounding is round-to-nearest-even
    v = np.array([1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, 1.0 + 2 ** -9], np.float32)
    assert list(inputs.to_bf16_bits(v)) == [0x3F80, 0x3F82, 0x3F80]
