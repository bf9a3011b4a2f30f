"""Seeded synthetic inputs for the GKA hot path.

This module only draws random tensors with the shapes and value distributions of
the benchmark configurations; it contains none of the method's arithmetic (no
state recurrence, no solver).  Both the CUDA path and the CPU oracle consume the
arrays produced here, which is the only thing the two sides share.

Every (batch, head) pair has its own random substream ``default_rng([seed, b, h])``
and a fixed draw order (q, k, v, gate-normal, lambda-normal; the stress recipe
draws its factor, coefficients and noise in place of k), so any subset of heads
can be generated alone and is identical to the same heads of the full tensor.

Layouts follow the C ABI: q, k : [B, T, heads, d_k]; v : [B, T, heads, d_v];
gate, lam : [B, T, heads].  Values are drawn in float64 and returned as float32;
``round_bf16`` gives the value a bf16 buffer would hold (as float32).
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Iterable, Optional, Sequence, Tuple

import numpy as np


@dataclass(frozen=True)
class GkaConfig:
    """One benchmark configuration (shapes, distribution parameters, seed)."""

    name: str
    B: int
    heads: int
    T: int
    d: int
    chunk: int
    n_iter: int
    io_dtype: str  # "f32" | "bf16"
    seed: int
    gate_mean: float = 2.0  # gate = sigmoid(N(gate_mean, 1))
    lam_mean: float = 0.0  # lam = lam_scale * softplus(N(lam_mean, 1)) + lam_eps
    lam_eps: float = 1e-2
    lam_scale: float = 1.0
    key_rank: int = 0  # > 0: keys = normalise(z F + key_noise * N(0,1)), F of this rank
    key_noise: float = 0.0
    kind: str = "fwd"  # "fwd" | "decode"
    prefix_T: int = 0  # decode: length of the prefix that builds the state


CONFIGS = {
    0: GkaConfig("cfg0_fwd_f32_small", B=1, heads=2, T=256, d=64, chunk=64, n_iter=8,
                 io_dtype="f32", seed=0),
    1: GkaConfig("cfg1_fwd_bf16_train", B=4, heads=16, T=4096, d=128, chunk=64, n_iter=10,
                 io_dtype="bf16", seed=1),
    2: GkaConfig("cfg2_decode_bf16", B=256, heads=32, T=1, d=128, chunk=64, n_iter=10,
                 io_dtype="bf16", seed=2, kind="decode", prefix_T=2048),
    3: GkaConfig("cfg3_fwd_bf16_long", B=1, heads=32, T=131072, d=128, chunk=64, n_iter=10,
                 io_dtype="bf16", seed=3, gate_mean=4.0, lam_mean=-1.0, lam_eps=1e-3),
    4: GkaConfig("cfg4_fwd_stress", B=2, heads=8, T=8192, d=128, chunk=64, n_iter=8,
                 io_dtype="bf16", seed=4, gate_mean=6.0, lam_mean=0.0, lam_eps=0.0,
                 lam_scale=1e-4, key_rank=8, key_noise=0.01),
}


def shrink(cfg: GkaConfig, **kw) -> GkaConfig:
    """Copy of a configuration with some fields replaced (smaller B/heads/T for tests)."""
    return replace(cfg, **kw)


def round_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); result stays float32.  Finite inputs."""
    a = np.array(x, dtype=np.float32, order="C", copy=True)
    u = a.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    u += np.uint32(0x7FFF)
    u += lsb
    u &= np.uint32(0xFFFF0000)
    return a


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) of float32 values, round to nearest even."""
    r = round_bf16(x)
    return (r.view(np.uint32) >> 16).astype(np.uint16)


def _softplus(x: np.ndarray) -> np.ndarray:
    return np.log1p(np.exp(-np.abs(x))) + np.maximum(x, 0.0)


def _sigmoid(x: np.ndarray) -> np.ndarray:
    return 1.0 / (1.0 + np.exp(-x))


def _unit_rows(x: np.ndarray) -> np.ndarray:
    return x / np.linalg.norm(x, axis=-1, keepdims=True)


def draw_head(cfg: GkaConfig, b: int, h: int, T: Optional[int] = None, stream: int = 0):
    """Draw (q, k, v, gate, lam) for one (batch, head) pair, float64, shapes [T, d] / [T].

    ``stream`` selects an independent substream of the same (b, h) pair (the decode
    configuration uses stream 0 for the prefix and stream 1 for the step inputs).
    """
    T = cfg.T if T is None else T
    d = cfg.d
    key = [cfg.seed, b, h] if stream == 0 else [cfg.seed, b, h, stream]
    rng = np.random.default_rng(key)
    q = _unit_rows(rng.standard_normal((T, d)))
    if cfg.key_rank > 0:
        F = rng.standard_normal((cfg.key_rank, d))
        z = rng.standard_normal((T, cfg.key_rank))
        noise = rng.standard_normal((T, d))
        k = _unit_rows(z @ F + cfg.key_noise * noise)
    else:
        k = _unit_rows(rng.standard_normal((T, d)))
    v = rng.standard_normal((T, d))
    gate = _sigmoid(rng.normal(cfg.gate_mean, 1.0, T))
    lam = cfg.lam_scale * _softplus(rng.normal(cfg.lam_mean, 1.0, T)) + cfg.lam_eps
    return q, k, v, gate, lam


def make_inputs(cfg: GkaConfig, T: Optional[int] = None, stream: int = 0,
                pairs: Optional[Iterable[Tuple[int, int]]] = None):
    """Inputs of a configuration in ABI layout, float32.

    Returns dict(q, k, v [B,T,heads,d], gate, lam [B,T,heads]).  q, k, v are already
    rounded to bf16-representable values when ``cfg.io_dtype == "bf16"`` so that the
    oracle and the device see identical numbers.  ``pairs`` restricts generation to
    some (b, h) pairs (others stay zero; gate and lam stay 1 there).
    """
    T = cfg.T if T is None else T
    B, Hh, d = cfg.B, cfg.heads, cfg.d
    q = np.zeros((B, T, Hh, d), np.float32)
    k = np.zeros_like(q)
    v = np.zeros_like(q)
    gate = np.ones((B, T, Hh), np.float32)
    lam = np.ones((B, T, Hh), np.float32)
    todo: Sequence[Tuple[int, int]] = (
        [(b, h) for b in range(B) for h in range(Hh)] if pairs is None else list(pairs))
    for (b, h) in todo:
        qq, kk, vv, gg, ll = draw_head(cfg, b, h, T, stream)
        q[b, :, h] = qq
        k[b, :, h] = kk
        v[b, :, h] = vv
        gate[b, :, h] = gg
        lam[b, :, h] = ll
    # a float32 gate can round to exactly 1.0 but never above; keep lam strictly positive
    lam = np.maximum(lam, np.float32(1e-30))
    if cfg.io_dtype == "bf16":
        q, k, v = round_bf16(q), round_bf16(k), round_bf16(v)
    return dict(q=q, k=k, v=v, gate=gate, lam=lam)
