"""ctypes binding of the OmniCache C-ABI (``include/omnicache.h``); same names, marshalling only.

Every function here turns torch tensors into raw device pointers and the current torch stream into a
``cudaStream_t`` and calls the shared library: all arithmetic and data movement happen in the CUDA
kernels.  There is no CPU fallback: a missing library raises at import, a failing call raises
``OmniCacheError``.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libomnicache_b200.so")

OK, ERR_INVALID_ARG, ERR_ALIGNMENT, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_OOM, CACHE_MISS = range(9)
KIND_TOKEN, KIND_FRAME, KIND_BLOCK = 0, 1, 2
DTYPE_F32, DTYPE_BF16 = 0, 1
SELECT_THRESHOLD, SELECT_COUNT = 0, 1
RESTORE_FROM_CACHE, RESTORE_FROM_REPRESENTATIVE = 0, 1
FRAME_MEAN_POS_COS, FRAME_FLAT_COS = 0, 1
(K_NORMS, K_MATCH_TC, K_MATCH_SIMT, K_MATCH_FIN, K_FRAME, K_FRAME_FIN, K_BLOCK, K_BLOCK_FIN, K_SELECT,
 K_GATHER, K_RESTORE, K_COPY, K_LINEAR) = range(13)
K_COUNT = 13

EXPORTS = (
    "oc_status_str", "oc_layout_check", "oc_layout_counts", "oc_match_workspace_bytes",
    "oc_rows_from_layout", "oc_layer_cache_would_hit", "oc_kernel_name", "oc_create", "oc_destroy",
    "oc_device_status", "oc_profile_enable", "oc_profile_reset", "oc_profile_read", "oc_profile_span_read",
    "oc_profile_captured_read", "oc_match", "oc_match_frame_levels",
    "oc_select", "oc_gather", "oc_restore", "oc_layer_cache_put", "oc_layer_cache_get",
    "oc_layer_cache_clear", "oc_cache_step_host", "oc_match_frame_noalloc", "oc_selftest_bounded_wait", "oc_selftest_per_device_once",
    "oc_schedule_propose", "oc_joint_workspace_bytes", "oc_joint_groups", "oc_match_joint", "oc_select_joint",
    "oc_linear_gather_scatter", "oc_tc_plan_override", "oc_tc_plan_describe",
)


class OmniCacheError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_str(status)}")


class CLayout(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("kind", "dtype", "B", "T", "H", "W", "C", "sy", "sx", "oy", "ox",
                                      "gy", "gx", "self_match", "frame_stat")] + [("eps", C.c_float)]


class CRows(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("seg_bytes", "n_seg", "seg_stride", "unit_pitch",
                                        "units_per_outer", "outer_pitch")]


if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2607_23844_b200.build`")
_lib = C.CDLL(LIB_PATH)

_vp, _i, _i64, _f = C.c_void_p, C.c_int, C.c_int64, C.c_float
_lib.oc_status_str.restype = C.c_char_p
_lib.oc_status_str.argtypes = [_i]
_lib.oc_kernel_name.restype = C.c_char_p
_lib.oc_kernel_name.argtypes = [_i]
_lib.oc_layout_check.argtypes = [_vp]
_lib.oc_layout_counts.argtypes = [_vp, _vp, _vp, _vp]
_lib.oc_match_workspace_bytes.argtypes = [_vp, _vp]
_lib.oc_rows_from_layout.argtypes = [_vp, _i, _i, _vp]
_lib.oc_layer_cache_would_hit.argtypes = [_i, _i, _i]
_lib.oc_create.argtypes = [_vp, _i, C.c_size_t]
_lib.oc_destroy.argtypes = [_vp]
_lib.oc_device_status.argtypes = [_vp, _vp]
_lib.oc_selftest_bounded_wait.argtypes = [_vp, C.c_uint, _vp]
_lib.oc_selftest_per_device_once.argtypes = [C.c_int, C.c_int, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int)]
_lib.oc_profile_enable.argtypes = [_vp, _i]
_lib.oc_tc_plan_override.argtypes = [_vp, _i, _i, _i, _i, _i, _i]
_lib.oc_tc_plan_describe.argtypes = [_vp, _vp, _vp]
_lib.oc_profile_reset.argtypes = [_vp]
_lib.oc_profile_read.argtypes = [_vp, _i, _vp, _vp]
_lib.oc_profile_span_read.argtypes = [_vp, _i, _vp, _vp]
_lib.oc_profile_captured_read.argtypes = [_vp, _i, _vp, _vp]
_lib.oc_match.argtypes = [_vp] * 8
_lib.oc_match_frame_levels.argtypes = [_vp, _vp, _vp, _i, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.oc_select.argtypes = [_vp, _vp, _vp, _vp, _i, _f, _i64, _i64, _vp, _vp, _vp, _vp, _vp]
_lib.oc_linear_gather_scatter.argtypes = [_vp, _vp, _i64, _i64, _vp, _i64, _vp, _i64, _vp, _i64, _vp, _vp]
_lib.oc_joint_workspace_bytes.argtypes = [_vp, _vp]
_lib.oc_joint_groups.argtypes = [_vp] * 7
_lib.oc_match_joint.argtypes = [_vp] * 7
_lib.oc_select_joint.argtypes = [_vp, _vp, _vp, _vp, _vp, _i, _f, _i64, _i64, _i64, _vp, _vp, _vp, _vp, _vp]
_lib.oc_gather.argtypes = [_vp, _vp, _vp, _vp, _i64, _vp, _vp]
_lib.oc_restore.argtypes = [_vp, _vp, _vp, _vp, _i64, _vp, _vp, _vp, _i, _vp]
_lib.oc_layer_cache_put.argtypes = [_vp, _i, _i, _vp, C.c_size_t, _vp]
_lib.oc_layer_cache_get.argtypes = [_vp, _i, _i, _i, _vp, _vp, _vp, _vp]
_lib.oc_layer_cache_clear.argtypes = [_vp]
_lib.oc_cache_step_host.argtypes = [_vp, _vp, _i, _f, _i64, _vp, _vp, _vp, _vp, _vp]
_lib.oc_schedule_propose.argtypes = [_vp, _vp, _i64, C.c_double, _vp, _vp, _vp]
_lib.oc_match_frame_noalloc.argtypes = [_i, _vp, _vp, _vp, _vp, _vp, _vp]
NOALLOC_SCRATCH_BYTES = 1 << 20


def status_str(s: int) -> str:
    return _lib.oc_status_str(s).decode()


def kernel_name(k: int) -> str:
    return _lib.oc_kernel_name(k).decode()


def _chk(st: int, where: str) -> None:
    if st != OK:
        raise OmniCacheError(st, where)


_LAYOUT_CACHE: dict = {}


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

    def c(self) -> CLayout:
        key = (self.kind, self.dtype, self.B, self.T, self.H, self.W, self.C, self.sy, self.sx,
               self.oy, self.ox, self.gy, self.gx, self.self_match, self.frame_stat, self.eps)
        hit = _LAYOUT_CACHE.get(key)
        if hit is None:
            hit = _LAYOUT_CACHE[key] = CLayout(*key)
        return hit

    def check(self) -> int:
        return layout_check(self)

    def counts(self) -> tuple[int, int, int]:
        return layout_counts(self)

    @property
    def n_groups(self) -> int:
        return self.counts()[0]

    @property
    def units_per_group(self) -> int:
        return self.counts()[1]

    @property
    def reps_per_group(self) -> int:
        return self.counts()[2]

    @property
    def n_units(self) -> int:
        g, u, _ = self.counts()
        return g * u

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == DTYPE_F32 else 2


def layout_check(layout: Layout) -> int:
    """oc_layout_check: returns the status code (no exception), host only."""
    cl = layout.c()
    return _lib.oc_layout_check(C.byref(cl))


def layout_counts(layout: Layout) -> tuple[int, int, int]:
    cl = layout.c()
    g, u, r = C.c_int64(), C.c_int64(), C.c_int64()
    _chk(_lib.oc_layout_counts(C.byref(cl), C.byref(g), C.byref(u), C.byref(r)), "oc_layout_counts")
    return g.value, u.value, r.value


def match_workspace_bytes(layout: Layout) -> int:
    cl = layout.c()
    n = C.c_size_t()
    _chk(_lib.oc_match_workspace_bytes(C.byref(cl), C.byref(n)), "oc_match_workspace_bytes")
    return n.value


def joint_workspace_bytes(layout: Layout) -> int:
    cl = layout.c()
    n = C.c_size_t()
    _chk(_lib.oc_joint_workspace_bytes(C.byref(cl), C.byref(n)), "oc_joint_workspace_bytes")
    return n.value


def rows_from_layout(layout: Layout, channels: int, elem_bytes: int) -> CRows:
    cl, rows = layout.c(), CRows()
    _chk(_lib.oc_rows_from_layout(C.byref(cl), channels, elem_bytes, C.byref(rows)), "oc_rows_from_layout")
    return rows


def layer_cache_would_hit(stored_step: int, step: int, interval: int) -> bool:
    return bool(_lib.oc_layer_cache_would_hit(stored_step, step, interval))


def _ptr(t) -> int | None:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    assert t.is_contiguous(), "tensors handed to the C-ABI must be contiguous"
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream if isinstance(stream, int) else stream.cuda_stream


def schedule_propose(latency, quality_loss, target_speedup: float):
    """Layered Cache schedule proposal (Algorithm 1).  Returns (chosen candidate indices in the order
    taken, saved latency).  Host-side: no device work."""
    import numpy as np
    L = np.ascontiguousarray(latency, dtype=np.float64)
    Q = np.ascontiguousarray(quality_loss, dtype=np.float64)
    if L.shape != Q.shape or L.ndim != 1:
        raise ValueError("latency and quality_loss must be 1-D arrays of one length")
    chosen = np.empty(max(L.size, 1), dtype=np.int32)
    n, saved = C.c_int64(), C.c_double()
    _chk(_lib.oc_schedule_propose(L.ctypes.data_as(_vp), Q.ctypes.data_as(_vp), L.size, float(target_speedup),
                                  chosen.ctypes.data_as(_vp), C.byref(n), C.byref(saved)), "oc_schedule_propose")
    return chosen[:n.value].tolist(), saved.value


def match_frame_noalloc(device: int, layout: Layout, x, best_sim, best_idx, pair_sim=None, stream=None,
                        check: bool = True) -> int:
    """oc_match_frame_noalloc: the Frame Cache match for callers that may not allocate device memory.

    No context is involved: the partial sums go to a fixed array inside the library (at most
    NOALLOC_SCRATCH_BYTES; larger layouts come back as ERR_WORKSPACE).  Calls on one device share that
    array, so do not let two of them overlap on the GPU, and make the first call on a device outside
    of any stream capture."""
    cl = layout.c()
    st = _lib.oc_match_frame_noalloc(device, C.byref(cl), _ptr(x), _ptr(best_sim), _ptr(best_idx), _ptr(pair_sim),
                                     _stream(stream))
    if check:
        _chk(st, "oc_match_frame_noalloc")
    return st


class Context:
    """oc_create / oc_destroy and the per-context calls."""

    def __init__(self, device: int = 0, workspace_bytes: int = 0):
        self._h = C.c_void_p()
        _chk(_lib.oc_create(C.byref(self._h), device, workspace_bytes), "oc_create")
        self.device = device
        self.workspace_bytes = workspace_bytes

    def close(self) -> None:
        if self._h:
            _lib.oc_destroy(self._h)
            self._h = C.c_void_p()

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- status / profile ------------------------------------------------------------------------
    def device_status(self) -> int:
        code = C.c_int()
        _chk(_lib.oc_device_status(self._h, C.byref(code)), "oc_device_status")
        return code.value

    def selftest_bounded_wait(self, limit_us: int = 2000, stream=None) -> None:
        """Makes a bounded device-side wait run out on purpose (see oc_selftest_bounded_wait)."""
        _chk(_lib.oc_selftest_bounded_wait(self._h, limit_us, _stream(stream)), "oc_selftest_bounded_wait")

    def tc_plan_override(self, plan=None, single_accumulator: bool = False, candidates_resident: int = -1) -> None:
        """Test hook (oc_tc_plan_override): ``plan`` = (pair, tiles per CTA, pieces per row[, candidates
        resident]) forces the tensor-core matcher's work split; None returns to the planner."""
        if plan is None:
            _chk(_lib.oc_tc_plan_override(self._h, 0, 0, 1, 1, 0, -1), "oc_tc_plan_override")
        else:
            vals = [int(v) for v in plan]
            if len(vals) == 4:
                candidates_resident = vals[3]
            pair, tiles, pieces = vals[:3]
            _chk(_lib.oc_tc_plan_override(self._h, 1, pair, tiles, pieces, int(single_accumulator), int(candidates_resident)),
                 "oc_tc_plan_override")

    def tc_plan_describe(self, layout: Layout) -> dict:
        """Test hook (oc_tc_plan_describe): the tensor-core matcher's work split for this layout."""
        cl = layout.c()
        out = (C.c_int32 * 12)()
        _chk(_lib.oc_tc_plan_describe(self._h, C.byref(cl), out), "oc_tc_plan_describe")
        keys = ("pair", "tiles", "pieces_per_row", "two_acc_sets", "stages", "stage_bytes", "a_resident", "pieces",
                "walkers", "widest_cols", "kblocks")
        return dict(zip(keys, list(out)))

    def profile_enable(self, on) -> None:
        """False/0: timers off; True/1: CUDA events around every launch; 2: device-side spans of the
        tensor-core matcher (read with profile_span_read)."""
        _chk(_lib.oc_profile_enable(self._h, int(on)), "oc_profile_enable")

    def profile_reset(self) -> None:
        _chk(_lib.oc_profile_reset(self._h), "oc_profile_reset")

    def profile_read(self, kernel_id: int) -> tuple[int, float]:
        n, ms = C.c_int64(), C.c_double()
        _chk(_lib.oc_profile_read(self._h, kernel_id, C.byref(n), C.byref(ms)), "oc_profile_read")
        return n.value, ms.value

    def profile_captured_read(self, kernel_id: int) -> tuple[int, float]:
        """(brackets captured into CUDA graphs, sum of their most recent recordings in ms)."""
        n, ms = C.c_int64(), C.c_double()
        _chk(_lib.oc_profile_captured_read(self._h, kernel_id, C.byref(n), C.byref(ms)), "oc_profile_captured_read")
        return n.value, ms.value

    def profile_span_read(self, kernel_id: int) -> tuple[int, float]:
        """(launches stamped, summed first-CTA-entry -> last-CTA-exit time in ms); see profile_enable(2)."""
        n, ms = C.c_int64(), C.c_double()
        _chk(_lib.oc_profile_span_read(self._h, kernel_id, C.byref(n), C.byref(ms)), "oc_profile_span_read")
        return n.value, ms.value

    def launches(self) -> dict[str, int]:
        return {kernel_name(k): self.profile_read(k)[0] for k in range(K_COUNT)}

    # -- hot path --------------------------------------------------------------------------------
    def match(self, layout: Layout, x, best_sim, best_idx, aux_sim=None, pair_sim=None, stream=None,
              check: bool = True) -> int:
        cl = layout.c()
        st = _lib.oc_match(self._h, C.byref(cl), _ptr(x), _ptr(best_sim), _ptr(best_idx), _ptr(aux_sim),
                           _ptr(pair_sim), _stream(stream))
        if check:
            _chk(st, "oc_match")
        return st

    def linear_gather_scatter(self, a, a_rows: int, K: int, a_idx, n_rows: int, w, N: int, out, out_rows: int,
                              out_idx, stream=None, check: bool = True) -> int:
        st = _lib.oc_linear_gather_scatter(self._h, _ptr(a), a_rows, K, _ptr(a_idx), n_rows, _ptr(w), N, _ptr(out),
                                           out_rows, _ptr(out_idx), _stream(stream))
        if check:
            _chk(st, "oc_linear_gather_scatter")
        return st

    def joint_groups(self, layout: Layout, frame_best_sim, frame_best_idx, frame_slot_of, frames, stream=None,
                     check: bool = True) -> int:
        cl = layout.c()
        st = _lib.oc_joint_groups(self._h, C.byref(cl), _ptr(frame_best_sim), _ptr(frame_best_idx),
                                  _ptr(frame_slot_of), _ptr(frames), _stream(stream))
        if check:
            _chk(st, "oc_joint_groups")
        return st

    def match_joint(self, layout: Layout, x, frames, best_sim, best_idx, stream=None, check: bool = True) -> int:
        cl = layout.c()
        st = _lib.oc_match_joint(self._h, C.byref(cl), _ptr(x), _ptr(frames), _ptr(best_sim), _ptr(best_idx),
                                 _stream(stream))
        if check:
            _chk(st, "oc_match_joint")
        return st

    def select_joint(self, layout: Layout, frames, best_sim, best_idx, mode: int, thr: float, n_reuse_pair: int,
                     n_reuse_single: int, y_stride: int, kept_idx, kept_count, match_map, slot_of, stream=None,
                     check: bool = True) -> int:
        cl = layout.c()
        st = _lib.oc_select_joint(self._h, C.byref(cl), _ptr(frames), _ptr(best_sim), _ptr(best_idx), mode, thr,
                                  n_reuse_pair, n_reuse_single, y_stride, _ptr(kept_idx), _ptr(kept_count),
                                  _ptr(match_map), _ptr(slot_of), _stream(stream))
        if check:
            _chk(st, "oc_select_joint")
        return st

    def match_frame_levels(self, layout: Layout, x, grids, best_sim, best_idx, pos_sim=None, pair_sim=None,
                           stream=None, check: bool = True) -> int:
        """oc_match_frame_levels: ``grids`` is a sequence of (gy, gx) pairs (host side)."""
        cl = layout.c()
        flat = [int(v) for g in grids for v in g]
        arr = (C.c_int32 * max(len(flat), 1))(*flat)
        st = _lib.oc_match_frame_levels(self._h, C.byref(cl), _ptr(x), len(grids), arr, _ptr(best_sim),
                                        _ptr(best_idx), _ptr(pos_sim), _ptr(pair_sim), _stream(stream))
        if check:
            _chk(st, "oc_match_frame_levels")
        return st

    def select(self, layout: Layout, best_sim, best_idx, mode: int, thr: float, n_reuse_per_group: int,
               y_group_stride: int, kept_idx, kept_count, match_map, slot_of, stream=None,
               check: bool = True) -> int:
        cl = layout.c()
        st = _lib.oc_select(self._h, C.byref(cl), _ptr(best_sim), _ptr(best_idx), mode, thr,
                            n_reuse_per_group, y_group_stride, _ptr(kept_idx), _ptr(kept_count),
                            _ptr(match_map), _ptr(slot_of), _stream(stream))
        if check:
            _chk(st, "oc_select")
        return st

    def gather(self, rows: CRows, x, kept_idx, n_slots: int, y, stream=None, check: bool = True) -> int:
        st = _lib.oc_gather(self._h, C.byref(rows), _ptr(x), _ptr(kept_idx), n_slots, _ptr(y), _stream(stream))
        if check:
            _chk(st, "oc_gather")
        return st

    def restore(self, rows: CRows, z, cache, n_units: int, slot_of, match_map, out,
                src_mode: int = RESTORE_FROM_CACHE, stream=None, check: bool = True) -> int:
        st = _lib.oc_restore(self._h, C.byref(rows), _ptr(z), _ptr(cache), n_units, _ptr(slot_of),
                             _ptr(match_map), _ptr(out), src_mode, _stream(stream))
        if check:
            _chk(st, "oc_restore")
        return st

    def layer_cache_put(self, layer: int, step: int, src, nbytes: int | None = None, stream=None,
                        check: bool = True) -> int:
        if nbytes is None:
            nbytes = src.numel() * src.element_size()
        st = _lib.oc_layer_cache_put(self._h, layer, step, _ptr(src), nbytes, _stream(stream))
        if check:
            _chk(st, "oc_layer_cache_put")
        return st

    def layer_cache_get(self, layer: int, step: int, interval: int, dst=None, stream=None):
        """Returns (hit, view pointer, bytes).  Raises on errors other than a miss."""
        view, nbytes = C.c_void_p(), C.c_size_t()
        st = _lib.oc_layer_cache_get(self._h, layer, step, interval, _ptr(dst), C.byref(view), C.byref(nbytes),
                                     _stream(stream))
        if st == CACHE_MISS:
            return False, None, 0
        _chk(st, "oc_layer_cache_get")
        return True, view.value, nbytes.value

    def layer_cache_clear(self) -> None:
        _chk(_lib.oc_layer_cache_clear(self._h), "oc_layer_cache_clear")

    def cache_step_host(self, layout: Layout, mode: int, thr: float, n_reuse_per_group: int, x_host, cache_host,
                        out_host, kept_count_host=None, stream=None, check: bool = True) -> int:
        """Host-buffer call: tensors are CPU (ideally pinned) torch tensors."""
        cl = layout.c()
        st = _lib.oc_cache_step_host(self._h, C.byref(cl), mode, thr, n_reuse_per_group, _ptr(x_host),
                                     _ptr(cache_host), _ptr(out_host), _ptr(kept_count_host), _stream(stream))
        if check:
            _chk(st, "oc_cache_step_host")
        return st
