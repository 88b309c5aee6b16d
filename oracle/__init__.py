"""CPU oracle for the OmniCache match / select / gather / restore / layered-cache path.

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's CPU-baseline leg may
import this package; the product package never does.  The arithmetic lives in
``omnicache_oracle.c`` (plain C, double precision, compiled here with gcc); this file only builds
it, marshals NumPy arrays into it and keeps the dictionary behind the Layered Cache oracle and the
few lines of the Layered Cache schedule proposal (Algorithm 1).
Nothing in here imports the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "omnicache_oracle.c")
_LIB = os.path.join(_HERE, "libomnicache_oracle.so")

KIND_TOKEN, KIND_FRAME, KIND_BLOCK = 0, 1, 2
DT_F32, DT_BF16 = 0, 1
MODE_THRESHOLD, MODE_COUNT = 0, 1
SRC_CACHE, SRC_REPRESENTATIVE = 0, 1


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2, OpenMP) if the shared object is missing or stale."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".{os.getpid()}.tmp"
    subprocess.run(["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"],
                   check=True)
    os.replace(tmp, _LIB)
    return _LIB


class _Layout(C.Structure):
    _fields_ = [(n, C.c_int) for n in
                ("kind", "dtype", "B", "T", "H", "W", "C", "sy", "sx", "oy", "ox", "gy", "gx",
                 "self_match", "frame_stat")] + [("eps", C.c_double)]


class _Rows(C.Structure):
    _fields_ = [(n, C.c_int64) for n in
                ("seg_bytes", "n_seg", "seg_stride", "unit_pitch", "units_per_outer", "outer_pitch")]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.ocr_cosine.restype = C.c_double
        _lib.ocr_cosine.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_int64, C.c_double]
        for name in ("ocr_num_groups", "ocr_units_per_group", "ocr_num_units"):
            getattr(_lib, name).restype = C.c_int64
            getattr(_lib, name).argtypes = [C.c_void_p]
        _lib.ocr_unit_index.restype = C.c_int64
        _lib.ocr_unit_index.argtypes = [C.c_void_p, C.c_int64, C.c_int64]
        _lib.ocr_is_rep.argtypes = [C.c_void_p, C.c_int64]
        _lib.ocr_match_token.argtypes = [C.c_void_p] * 3 + [C.c_int64] + [C.c_void_p] * 4
        _lib.ocr_match_frame.argtypes = [C.c_void_p] * 6
        _lib.ocr_match_block.argtypes = [C.c_void_p] * 4
        _lib.ocr_joint_groups.argtypes = [C.c_int, C.c_int] + [C.c_void_p] * 4
        _lib.ocr_match_joint.argtypes = [C.c_void_p] * 6
        _lib.ocr_select_joint.argtypes = ([C.c_void_p] * 4 + [C.c_int, C.c_float, C.c_int64, C.c_int64, C.c_int64]
                                          + [C.c_void_p] * 4)
        _lib.ocr_select.argtypes = ([C.c_void_p] * 3 + [C.c_int, C.c_float, C.c_int64, C.c_int64]
                                    + [C.c_void_p] * 4)
        _lib.ocr_gather.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]
        _lib.ocr_restore.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p,
                                     C.c_void_p, C.c_void_p, C.c_int]
        _lib.ocr_layer_cache_hit.argtypes = [C.c_int] * 3
    return _lib


@dataclass
class Layout:
    kind: int
    dtype: int
    B: int
    T: int
    H: int
    W: int
    C: int
    sy: int = 2
    sx: int = 2
    oy: int = 0
    ox: int = 0
    gy: int = 1
    gx: int = 1
    self_match: int = 0
    frame_stat: int = 0
    eps: float = 1e-8

    def c(self) -> _Layout:
        return _Layout(self.kind, self.dtype, self.B, self.T, self.H, self.W, self.C, self.sy,
                       self.sx, self.oy, self.ox, self.gy, self.gx, self.self_match,
                       self.frame_stat, self.eps)

    @property
    def n_groups(self) -> int:
        return lib().ocr_num_groups(C.byref(self.c()))

    @property
    def units_per_group(self) -> int:
        return lib().ocr_units_per_group(C.byref(self.c()))

    @property
    def n_units(self) -> int:
        return self.n_groups * self.units_per_group

    def unit_index(self, g: int, u: int) -> int:
        return lib().ocr_unit_index(C.byref(self.c()), g, u)

    def is_rep(self, u: int) -> bool:
        return bool(lib().ocr_is_rep(C.byref(self.c()), u))

    @property
    def n_rep(self) -> int:
        return sum(self.is_rep(u) for u in range(self.units_per_group))

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == DT_F32 else 2


@dataclass
class Rows:
    """Strided description of the unit rows of a [B,T,H,W,C'] tensor (see the C file)."""
    seg_bytes: int
    n_seg: int
    seg_stride: int
    unit_pitch: int
    units_per_outer: int
    outer_pitch: int

    def c(self) -> _Rows:
        return _Rows(self.seg_bytes, self.n_seg, self.seg_stride, self.unit_pitch,
                     self.units_per_outer, self.outer_pitch)

    @property
    def row_bytes(self) -> int:
        return self.seg_bytes * self.n_seg


def rows_for(L: Layout, channels: int, elem_bytes: int) -> Rows:
    """Row geometry of the units of layout ``L`` in a tensor with ``channels`` channels."""
    cb = channels * elem_bytes
    if L.kind == KIND_TOKEN:
        return Rows(cb, 1, 0, cb, 1 << 40, 0)
    if L.kind == KIND_FRAME:
        if L.gy * L.gx == 1:
            fb = L.H * L.W * cb
            return Rows(fb, 1, 0, fb, 1 << 40, 0)
        # a patch of a frame: H/gy segments of (W/gx)*C' elements, one per image row; the gx
        # patches of a patch row sit side by side, and patch rows follow one another uniformly
        # through frames and batch elements (Section 3.3)
        hp, wp = L.H // L.gy, L.W // L.gx
        return Rows(wp * cb, hp, L.W * cb, wp * cb, L.gx, hp * L.W * cb)
    return Rows(cb, L.T, L.H * L.W * cb, cb, L.H * L.W, L.T * L.H * L.W * cb)


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _check(x: np.ndarray, L: Layout):
    want = np.float32 if L.dtype == DT_F32 else np.uint16
    assert x.dtype == want and x.flags.c_contiguous
    assert x.size == L.B * L.T * L.H * L.W * L.C


def cosine(x: np.ndarray, dtype: int, a_off: int, b_off: int, n: int, eps: float = 1e-8) -> float:
    return lib().ocr_cosine(_p(x), dtype, a_off, b_off, n, eps)


def match_token(L: Layout, x: np.ndarray, rows=None, want_full: bool = False):
    """Dense (Token Cache) match. Returns dict(best_sim, best_idx, second_sim[, full_sim])."""
    _check(x, L)
    n = L.n_units
    best_sim = np.full(n, np.nan, np.float32)
    best_idx = np.full(n, -2, np.int32)
    second = np.full(n, np.nan, np.float32)
    full = np.full((L.n_groups, L.units_per_group, L.n_rep), np.nan, np.float64) if want_full else None
    r = None if rows is None else np.ascontiguousarray(rows, dtype=np.int32)
    rc = lib().ocr_match_token(C.byref(L.c()), _p(x), _p(r), 0 if r is None else r.size,
                               _p(best_sim), _p(best_idx), _p(second), _p(full))
    assert rc == 0, rc
    out = dict(best_sim=best_sim, best_idx=best_idx, second_sim=second)
    if want_full:
        out["full_sim"] = full
    return out


def match_frame(L: Layout, x: np.ndarray, want_pos: bool = False):
    _check(x, L)
    n = L.B * L.T * L.gy * L.gx
    best_sim = np.empty(n, np.float32)
    best_idx = np.empty(n, np.int32)
    pair = np.empty((L.B, max(L.T - 1, 0)) + ((L.gy * L.gx,) if L.gy * L.gx > 1 else ()), np.float32)
    pos = np.empty((L.B, max(L.T - 1, 0), L.H * L.W), np.float32) if want_pos else None
    rc = lib().ocr_match_frame(C.byref(L.c()), _p(x), _p(best_sim), _p(best_idx), _p(pair), _p(pos))
    assert rc == 0, rc
    out = dict(best_sim=best_sim, best_idx=best_idx, pair_sim=pair)
    if want_pos:
        out["pos_sim"] = pos
    return out


def match_block(L: Layout, x: np.ndarray):
    _check(x, L)
    n = L.B * L.H * L.W
    best_sim = np.empty(n, np.float32)
    best_idx = np.empty(n, np.int32)
    rc = lib().ocr_match_block(C.byref(L.c()), _p(x), _p(best_sim), _p(best_idx))
    assert rc == 0, rc
    return dict(best_sim=best_sim, best_idx=best_idx)


def match(L: Layout, x: np.ndarray):
    if L.kind == KIND_TOKEN:
        return match_token(L, x)
    if L.kind == KIND_FRAME:
        return match_frame(L, x)
    return match_block(L, x)


def select(L: Layout, best_sim: np.ndarray, best_idx: np.ndarray, mode: int, thr: float = 0.0,
           n_reuse: int = 0, y_group_stride: int | None = None):
    G, U = L.n_groups, L.units_per_group
    if y_group_stride is None:
        y_group_stride = U
    best_sim = np.ascontiguousarray(best_sim, np.float32)
    best_idx = np.ascontiguousarray(best_idx, np.int32)
    kept_idx = np.full(G * y_group_stride, -7, np.int32)
    kept_count = np.zeros(G, np.int32)
    match_map = np.full(G * U, -7, np.int32)
    slot_of = np.full(G * U, -7, np.int32)
    rc = lib().ocr_select(C.byref(L.c()), _p(best_sim), _p(best_idx), mode, thr, n_reuse,
                          y_group_stride, _p(kept_idx), _p(kept_count), _p(match_map), _p(slot_of))
    assert rc == 0, rc
    return dict(kept_idx=kept_idx, kept_count=kept_count, match_map=match_map, slot_of=slot_of)


def gather(R: Rows, x: np.ndarray, kept_idx: np.ndarray, fill: int = 0) -> np.ndarray:
    """Returns the dense buffer as bytes [n_slots, row_bytes]; unused slots keep ``fill``."""
    kept_idx = np.ascontiguousarray(kept_idx, np.int32)
    y = np.full((kept_idx.size, R.row_bytes), fill, np.uint8)
    rc = lib().ocr_gather(C.byref(R.c()), _p(x), _p(kept_idx), kept_idx.size, _p(y))
    assert rc == 0
    return y


def restore(R: Rows, z: np.ndarray, cache: np.ndarray | None, n_units: int, slot_of: np.ndarray,
            match_map: np.ndarray, src_mode: int = SRC_CACHE, in_place: bool = False) -> np.ndarray:
    """Returns the restored tensor as a flat byte array shaped like ``cache``."""
    slot_of = np.ascontiguousarray(slot_of, np.int32)
    match_map = np.ascontiguousarray(match_map, np.int32)
    if in_place:
        out = cache
    else:
        nbytes = cache.nbytes if cache is not None else n_units * R.row_bytes
        out = np.zeros(nbytes, np.uint8)
    rc = lib().ocr_restore(C.byref(R.c()), _p(z), _p(cache), n_units, _p(slot_of), _p(match_map),
                           _p(out), src_mode)
    assert rc == 0
    return out


def joint_groups(B: int, T: int, frame_best_sim, frame_best_idx, frame_slot_of) -> np.ndarray:
    """Frame pairs of Frame Cache as token groups (Section 3.2.3): [B*T, 2] int32 (u, t) per slot."""
    fs = np.ascontiguousarray(frame_best_sim, np.float32)
    fi = np.ascontiguousarray(frame_best_idx, np.int32)
    so = np.ascontiguousarray(frame_slot_of, np.int32)
    frames = np.empty((B * T, 2), np.int32)
    rc = lib().ocr_joint_groups(B, T, _p(fs), _p(fi), _p(so), _p(frames))
    assert rc == 0, rc
    return frames


def match_joint(L: Layout, x: np.ndarray, frames: np.ndarray):
    _check(x, L)
    n = L.B * L.T * L.H * L.W
    frames = np.ascontiguousarray(frames, np.int32)
    best_sim = np.full(n, np.nan, np.float32)
    best_idx = np.full(n, -7, np.int32)
    second = np.full(n, np.nan, np.float32)
    rc = lib().ocr_match_joint(C.byref(L.c()), _p(x), _p(frames), _p(best_sim), _p(best_idx), _p(second))
    assert rc == 0, rc
    return dict(best_sim=best_sim, best_idx=best_idx, second_sim=second)


def select_joint(L: Layout, frames: np.ndarray, best_sim, best_idx, mode: int, thr: float = 0.0,
                 n_reuse_pair: int = 0, n_reuse_single: int = 0, y_group_stride: int | None = None):
    F, P = L.B * L.T, L.H * L.W
    if y_group_stride is None:
        y_group_stride = 2 * P
    frames = np.ascontiguousarray(frames, np.int32)
    best_sim = np.ascontiguousarray(best_sim, np.float32)
    best_idx = np.ascontiguousarray(best_idx, np.int32)
    kept_idx = np.full(F * y_group_stride, -7, np.int32)
    kept_count = np.full(F, -7, np.int32)
    match_map = np.full(F * P, -7, np.int32)
    slot_of = np.full(F * P, -7, np.int32)
    rc = lib().ocr_select_joint(C.byref(L.c()), _p(frames), _p(best_sim), _p(best_idx), mode, thr,
                                n_reuse_pair, n_reuse_single, y_group_stride, _p(kept_idx),
                                _p(kept_count), _p(match_map), _p(slot_of))
    assert rc == 0, rc
    return dict(kept_idx=kept_idx, kept_count=kept_count, match_map=match_map, slot_of=slot_of)


def _bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def _f64_to_bf16_rne(v: np.ndarray) -> np.ndarray:
    """Round float64 values ONCE to bf16 (8 significant bits, ties to even); returns the 16-bit patterns.
    Normal range only (no subnormal / overflow handling: the tests stay far from both)."""
    v = np.asarray(v, np.float64)
    out = np.zeros(v.shape, np.float64)
    nz = v != 0
    e = np.floor(np.log2(np.abs(v[nz])))
    ulp = np.exp2(e - 7)
    out[nz] = np.rint(v[nz] / ulp) * ulp                 # exact scalings by powers of two; rint = half to even
    return (out.astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)


def linear_gather_scatter(a: np.ndarray, a_idx, n_rows: int, w: np.ndarray, out: np.ndarray, out_idx) -> np.ndarray:
    """The wrapped layer's projection with the gather folded into its operand load and the restore into
    its store (Appendix A's compaction and scatter, fused into the layer):
        out[dst(r), :] = bf16( sum_k a[src(r), k] * w[n, k] ),   r = 0 .. n_rows-1,
    src(r) = a_idx[r] (r if a_idx is None), dst(r) = out_idx[r] (r if None); a row whose src or dst is
    negative is skipped; rows of ``out`` that no r writes keep their contents.  bf16 bit patterns in and
    out, products and sums in float64, one rounding at the end."""
    a64, w64 = _bf16_to_f64(np.asarray(a, np.uint16)), _bf16_to_f64(np.asarray(w, np.uint16))
    res = np.array(out, np.uint16, copy=True)
    for r in range(n_rows):
        src = r if a_idx is None else int(a_idx[r])
        dst = r if out_idx is None else int(out_idx[r])
        if src < 0 or dst < 0:
            continue
        res[dst] = _f64_to_bf16_rne(w64 @ a64[src])
    return res


def layer_cache_hit(stored_step: int, step: int, interval: int) -> bool:
    return bool(lib().ocr_layer_cache_hit(stored_step, step, interval))


class LayerCache:
    """Layered Cache oracle (Section 3.4): a dictionary layer -> (stored step, bytes)."""

    def __init__(self):
        self.store: dict[int, tuple[int, bytes]] = {}

    def put(self, layer: int, step: int, data: np.ndarray) -> None:
        self.store[layer] = (step, data.tobytes())

    def get(self, layer: int, step: int, interval: int):
        if layer not in self.store:
            return None
        s0, blob = self.store[layer]
        return blob if layer_cache_hit(s0, step, interval) else None

    def clear(self) -> None:
        self.store.clear()


def schedule_proposal(L, Q, s_r: float):
    """Cache schedule proposal (Algorithm 1, Section 3.4), step by step in the paper's notation.

    L[i], Q[i]: latency and quality loss of candidate i (a layer-timestep pair); s_r: target speedup.
    Scores w = Q / L; candidates sorted by increasing w (equal scores: lower candidate index first,
    a point the paper leaves open); TargetSave = (1 - 1/s_r) * sum(L); candidates are taken in that
    order while Saved < TargetSave, each adding its L to Saved.  Returns the taken candidate indices
    in the order taken (every one of them carries the same cache interval N, which is not used to
    choose).  Double precision throughout."""
    L = [float(v) for v in L]
    Q = [float(v) for v in Q]
    assert len(L) == len(Q) and all(v > 0.0 for v in L) and s_r >= 1.0
    w = [Q[i] / L[i] for i in range(len(L))]
    order = sorted(range(len(L)), key=lambda i: (w[i], i))
    total = 0.0
    for v in L:
        total += v
    target_save = (1.0 - 1.0 / s_r) * total
    saved = 0.0
    chosen = []
    k = 0
    while saved < target_save and k < len(order):
        i = order[k]
        k += 1
        chosen.append(i)
        saved += L[i]
    return chosen


def num_threads() -> int:
    return lib().ocr_num_threads()


def set_num_threads(n: int) -> None:
    lib().ocr_set_num_threads(n)
