"""Seeded synthetic feature tensors shaped like the paper's SD3 / SVD-XT / Latte layers.

This module only *draws inputs*: random fields, AR(1) frame sequences, the bf16 rounding of the
stored values and the keep-ratio → reuse-count bookkeeping of a harness. It holds none of the
method's arithmetic (no similarity, selection, gather or restore), so both the CUDA path and the
CPU oracle may be fed from it without sharing any of the code under test.

All tensors are channel-last ``[B, T, H, W, C]`` (Section 3.2.2 writes spatial-layer inputs as
``(B, T, H, W, C)``); images have ``T = 1``.  bf16 tensors are returned as ``uint16`` bit patterns
(round-to-nearest-even of the fp32 draw) so that every consumer sees exactly the same stored values.

The experiments of Section 4.1 use real SD3-medium / SVD-XT / Latte-1 activations; those need
pretrained weights and datasets, so the recipes below stand in for them.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

# dtype tags (plain ints; the C-ABI and the oracle each define their own constants)
F32 = 0
BF16 = 1


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (uint16), round-to-nearest-even. Storage conversion only."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns -> the fp32 values they store (exact)."""
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def smooth_field(rng: np.random.Generator, H: int, W: int, C: int, ell: float) -> np.ndarray:
    """Periodic 2-D Gaussian random field per channel, covariance exp(-d^2 / (2 ell^2)), unit variance.

    White noise is filtered in the Fourier domain with the transfer function
    exp(-pi^2 ell^2 |f|^2) (a Gaussian kernel of std ell/sqrt(2)), then scaled so that the
    expected variance is one.  Returns float32 ``[H, W, C]``.
    """
    noise = rng.standard_normal((H, W, C), dtype=np.float32)
    fy = np.fft.fftfreq(H)[:, None]
    fx = np.fft.rfftfreq(W)[None, :]
    transfer = np.exp(-(np.pi ** 2) * (ell ** 2) * (fy ** 2 + fx ** 2))
    fy_full = np.fft.fftfreq(H)[:, None]
    fx_full = np.fft.fftfreq(W)[None, :]
    gain = np.sqrt(np.mean(np.exp(-2.0 * (np.pi ** 2) * (ell ** 2) * (fy_full ** 2 + fx_full ** 2))))
    spec = np.fft.rfft2(noise, axes=(0, 1))
    spec *= (transfer / gain)[:, :, None]
    out = np.fft.irfft2(spec, s=(H, W), axes=(0, 1))
    return out.astype(np.float32)


def ar1_frames(rng: np.random.Generator, frame0: np.ndarray, T: int, rho: float) -> np.ndarray:
    """``x_t = rho x_{t-1} + sqrt(1 - rho^2) N(0, 1)``; frame 0 given. Returns ``[T, *frame0.shape]``."""
    out = np.empty((T,) + frame0.shape, dtype=np.float32)
    out[0] = frame0
    s = np.float32(np.sqrt(1.0 - rho * rho))
    for t in range(1, T):
        out[t] = np.float32(rho) * out[t - 1] + s * rng.standard_normal(frame0.shape, dtype=np.float32)
    return out


@dataclass
class Workload:
    """One synthetic problem: stored features plus the layout/selection parameters of a harness."""

    name: str
    kind: str                      # "token" | "frame" | "block"
    dtype: int                     # F32 | BF16
    shape: tuple                   # (B, T, H, W, C)
    x: np.ndarray                  # float32 [B,T,H,W,C] (F32) or uint16 bits (BF16)
    mode: str                      # "threshold" | "count"
    thr: float = 0.0
    n_reuse: int = 0               # per group, count mode
    self_match: bool = False
    groups: tuple = (1, 1)         # (gy, gx) patches per frame
    extra: dict = field(default_factory=dict)

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == F32 else 2


def _store(a: np.ndarray, dtype: int) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32) if dtype == F32 else to_bf16_bits(a)


def tiny_token_cache(seed: int = 1001, H: int = 16, W: int = 16, C: int = 64,
                     dup_frac: float = 0.4, dup_noise: float = 0.01) -> Workload:
    """Config 1: one frame of H*W fp32 tokens, N(0,1) rows, ``dup_frac`` of them overwritten by a
    noisy copy (std ``dup_noise``) of a random other token; a fixed random C x C map stands in for
    the wrapped layer."""
    rng = np.random.default_rng(seed)
    n = H * W
    x = rng.standard_normal((n, C), dtype=np.float32)
    order = rng.permutation(n)[: int(round(dup_frac * n))]
    for i in order:
        j = int(rng.integers(0, n - 1))
        if j >= i:
            j += 1
        x[i] = x[j] + np.float32(dup_noise) * rng.standard_normal(C, dtype=np.float32)
    w = (rng.standard_normal((C, C), dtype=np.float32) / np.float32(np.sqrt(C))).astype(np.float32)
    x_prev = x - np.float32(0.02) * rng.standard_normal((n, C), dtype=np.float32)
    return Workload("tiny_token_fp32", "token", F32, (1, 1, H, W, C), x.reshape(1, 1, H, W, C),
                    mode="threshold", thr=0.9, self_match=True,
                    extra={"layer_weight": w, "x_prev": x_prev.reshape(1, 1, H, W, C)})


def sd3_token_cache(seed: int = 1002, B: int = 2, H: int = 64, W: int = 64, C: int = 1536,
                    groups: tuple = (1, 1), reuse_frac: float = 0.5, dtype: int = BF16,
                    ell: float = 8.0, noise: float = 0.1) -> Workload:
    """Config 2: classifier-free-guidance pair of 64x64-token DiT inputs; smooth field (correlation
    length ``ell`` tokens) plus iid N(0, noise) per channel; 2x2-strided representative split;
    the ``reuse_frac`` most similar candidates of every token group are reused."""
    rng = np.random.default_rng(seed)
    x = np.empty((B, 1, H, W, C), dtype=np.float32)
    for b in range(B):
        x[b, 0] = smooth_field(rng, H, W, C, ell)
        x[b, 0] += np.float32(noise) * rng.standard_normal((H, W, C), dtype=np.float32)
    gy, gx = groups
    n_tok = (H // gy) * (W // gx)
    n_rep = n_tok // 4
    n_reuse = int(np.floor(reuse_frac * (n_tok - n_rep)))
    return Workload(f"sd3_token_bf16_g{gy * gx}", "token", dtype, (B, 1, H, W, C), _store(x, dtype),
                    mode="count", n_reuse=n_reuse, groups=groups)


def svd_frames(seed: int = 1003, T: int = 25, H: int = 72, W: int = 128, C: int = 320,
               rho: float = 0.95, ell: float = 8.0, dtype: int = BF16, kind: str = "frame",
               thr: float = 0.9) -> Workload:
    """Config 3 (and the per-level tensors of config 5): AR(1) frames over a smooth frame 0."""
    rng = np.random.default_rng(seed)
    f0 = smooth_field(rng, H, W, C, ell)
    x = ar1_frames(rng, f0, T, rho).reshape(1, T, H, W, C)
    return Workload(f"svd_{kind}_{H}x{W}x{C}", kind, dtype, (1, T, H, W, C), _store(x, dtype),
                    mode="threshold", thr=thr)


def latte_blocks(seed: int = 1004, T: int = 16, H: int = 16, W: int = 16, C: int = 1152,
                 rho: float = 0.9, ell: float = 8.0, dtype: int = BF16, thr: float = 0.85) -> Workload:
    """Config 4: AR(1) frames (rho) plus, per 2x2 spatial group, a shared AR(1) motion term of
    amplitude U(0, 4), so that within-group block similarities straddle the threshold."""
    rng = np.random.default_rng(seed)
    f0 = smooth_field(rng, H, W, C, ell)
    f = ar1_frames(rng, f0, T, rho)                                   # [T,H,W,C]
    gh, gw = H // 2, W // 2
    m0 = rng.standard_normal((gh, gw, C), dtype=np.float32)
    m = ar1_frames(rng, m0, T, rho)                                   # [T,gh,gw,C]
    amp = rng.uniform(0.0, 4.0, size=(gh, gw)).astype(np.float32)
    shared = (m * amp[None, :, :, None]).repeat(2, axis=1).repeat(2, axis=2)
    x = (f + shared).reshape(1, T, H, W, C)
    return Workload("latte_block_bf16", "block", dtype, (1, T, H, W, C), _store(x, dtype),
                    mode="threshold", thr=thr)


SVD_LEVELS = ((72, 128, 320), (36, 64, 640), (18, 32, 1280))


def keep_ratio_to_reuse(n_tok: int, n_cand: int, keep_ratio: float) -> int:
    """Harness bookkeeping for the keep-ratio sweep: keep round(ratio * n_tok) units of a group,
    reuse the rest, never more than the candidates available."""
    n_keep = int(np.floor(keep_ratio * n_tok + 0.5))
    return int(min(max(n_tok - n_keep, 0), n_cand))


def drift_step(rng: np.random.Generator, stored: np.ndarray, dtype: int, sigma: float = 0.02) -> np.ndarray:
    """Config 5 step model ``x_s = x_{s-1} + N(0, sigma)``, re-rounded to the storage type."""
    prev = stored if dtype == F32 else bf16_bits_to_f32(stored)
    nxt = prev + np.float32(sigma) * rng.standard_normal(prev.shape, dtype=np.float32)
    return _store(nxt, dtype)


def random_rows(seed: int, shape: tuple, dtype: int) -> np.ndarray:
    """iid N(0,1) tensor of the given shape in the storage type (stand-in for layer outputs/caches)."""
    rng = np.random.default_rng(seed)
    return _store(rng.standard_normal(shape, dtype=np.float32), dtype)
