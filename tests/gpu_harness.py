"""Helpers of the GPU parity tests: run each op through the C-ABI binding on torch device buffers and
compare with the CPU oracle under the acceptance rules (similarities within tolerance; indices exact
except rows whose oracle top-two gap, or distance to the selection cut, is below 1e-4; data movement
bit-exact)."""
from __future__ import annotations

import numpy as np
import torch

from paper_2607_23844_b200 import inputs

NEAR_TIE = 1e-4


def to_dev(a: np.ndarray) -> torch.Tensor:
    """NumPy array -> CUDA tensor with the same bytes (uint16 bf16 patterns travel as int16)."""
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda()
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def dev_bytes(t: torch.Tensor) -> bytes:
    return t.contiguous().view(torch.uint8).cpu().numpy().tobytes()


def layouts(oc, oracle, w: inputs.Workload, **kw):
    kind = {"token": 0, "frame": 1, "block": 2}[w.kind]
    gy, gx = w.groups
    args = dict(gy=gy, gx=gx, self_match=int(w.self_match))
    args.update(kw)
    return oc.Layout(kind, w.dtype, *w.shape, **args), oracle.Layout(kind, w.dtype, *w.shape, **args)


def make_ctx(oc, L):
    return oc.Context(0, oc.match_workspace_bytes(L))


def gpu_match(oc, ctx, L, x_dev, want_aux=False, want_pair=False):
    n = L.n_units
    best_sim = torch.full((n,), float("nan"), device="cuda", dtype=torch.float32)
    best_idx = torch.full((n,), -2, device="cuda", dtype=torch.int32)
    aux = pair = None
    if want_aux:
        if L.kind == oc.KIND_TOKEN:
            g, u, r = L.counts()
            aux = torch.full((g, u, r), float("nan"), device="cuda", dtype=torch.float32)
        else:
            aux = torch.full((L.B, L.T - 1, L.H * L.W), float("nan"), device="cuda", dtype=torch.float32)
    if want_pair:
        shape = (L.B, max(L.T - 1, 0)) + ((L.gy * L.gx,) if L.kind == oc.KIND_FRAME and L.gy * L.gx > 1 else ())
        pair = torch.full(shape, float("nan"), device="cuda", dtype=torch.float32)
    ctx.match(L, x_dev, best_sim, best_idx, aux, pair)
    torch.cuda.synchronize()
    assert ctx.device_status() == oc.OK
    out = dict(best_sim=best_sim, best_idx=best_idx)
    if aux is not None:
        out["aux"] = aux
    if pair is not None:
        out["pair_sim"] = pair
    return out


def gpu_select(oc, ctx, L, best_sim, best_idx, mode, thr, n_reuse, stride):
    g, u, _ = L.counts()
    kept_idx = torch.full((g * stride,), -9, device="cuda", dtype=torch.int32)
    kept_count = torch.full((g,), -9, device="cuda", dtype=torch.int32)
    match_map = torch.full((g * u,), -9, device="cuda", dtype=torch.int32)
    slot_of = torch.full((g * u,), -9, device="cuda", dtype=torch.int32)
    ctx.select(L, best_sim, best_idx, mode, thr, n_reuse, stride, kept_idx, kept_count, match_map, slot_of)
    torch.cuda.synchronize()
    return dict(kept_idx=kept_idx, kept_count=kept_count, match_map=match_map, slot_of=slot_of)


def check_match_against_oracle(oracle, Lo, x_np, got_sim, got_idx, ref, tol, rows=None):
    """got_*: NumPy arrays from the GPU; ref: oracle dict with best_sim/best_idx/second_sim (token) or
    best_sim/best_idx.  Returns the number of near-tie rows and how many of them differ."""
    sel = np.arange(got_sim.size) if rows is None else np.asarray(rows)
    rs, ri = ref["best_sim"][sel], ref["best_idx"][sel]
    gs, gi = got_sim[sel], got_idx[sel]
    cand = np.isfinite(rs)
    assert np.array_equal(np.isneginf(gs), ~cand), "representative rows must carry -inf"
    assert np.array_equal(gi[~cand], ri[~cand])
    err = np.abs(gs[cand].astype(np.float64) - rs[cand].astype(np.float64))
    assert err.max(initial=0.0) <= tol, f"similarity error {err.max()} > {tol}"
    diff = np.nonzero(cand & (gi != ri))[0]
    near = 0
    if "second_sim" in ref:
        with np.errstate(invalid="ignore"):      # representative rows: -inf - -inf
            gap = rs.astype(np.float64) - ref["second_sim"][sel].astype(np.float64)
        near = int((cand & (gap < NEAR_TIE)).sum())
        C = Lo.C
        for k in diff:
            assert gap[k] < NEAR_TIE, f"row {sel[k]}: index differs although the top-two gap is {gap[k]}"
            # the GPU's choice must be (one of) the runner-up(s): its oracle similarity is within the gap
            s = oracle.cosine(x_np, Lo.dtype, int(sel[k]) * C, int(gi[k]) * C, C, Lo.eps)
            assert s >= rs[k] - NEAR_TIE
    else:
        assert diff.size == 0
    return near, int(diff.size)


def check_select_against_oracle(oracle, Lo, best_sim, best_idx, mode, thr, n_reuse, stride, got):
    """Exact comparison: oracle select on the very same best_sim / best_idx arrays."""
    ref = oracle.select(Lo, best_sim, best_idx, mode, thr, n_reuse, stride)
    for k in ("kept_idx", "kept_count", "match_map", "slot_of"):
        g = got[k].cpu().numpy()
        assert np.array_equal(g, ref[k]), f"select output {k} differs"
    return ref


def crows(oc, r):
    return oc.CRows(r.seg_bytes, r.n_seg, r.seg_stride, r.unit_pitch, r.units_per_outer, r.outer_pitch)
