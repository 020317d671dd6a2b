"""Seeded synthetic workloads for the compress-and-calibrate + calibrated-decode path.

This module holds no arithmetic of the method itself: it only draws inputs.  It is the
one module both the CUDA path's tests/bench and the CPU oracle's tests take inputs from,
so that both sides see identical bf16 bit patterns.

The inputs are stand-ins for the shapes and statistics of long-prompt LLM attention
(the paper's Section 3.1.1 finds that nearby queries are similar; its introduction notes
that a few tokens carry most of the attention mass and that the first tokens act as
attention sinks).  No item of any public benchmark is reproduced here.

Recipe, per (layer, batch element):
  * every query head has a base direction u ~ N(0,1)^D; observation-window query j is
    u + 0.3 N(0,1)^D (adjacent-row cosine similarity about 0.9);
  * keys and values are N(0,1); `n_heavy` random prompt positions per kv head have their
    key scaled by 4 ("heavy hitters"); the first `n_sink` keys of a kv head are
    0.5 * (sum of the base directions of its query group), a strong logit for every head
    of the group (attention sinks);
  * optionally keys are rotated by a rotary position embedding at their position;
  * the decode query of step t is mean_j(Q_obs[j]) + sigma_t N(0,1)^D, and the step's new
    key/value rows are N(0,1).
All values are rounded to bf16 (round-to-nearest-even) and returned as uint16 bit patterns.

Random numbers come from numpy's counter-based Philox generator keyed by
(config id, seed, layer, batch element, kv head or tensor tag), so any single
(batch, kv-head) unit can be regenerated on its own.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, replace
import os

import numpy as np

D_HEAD = 128


@dataclass(frozen=True)
class WorkloadConfig:
    cfg_id: int
    B: int
    Hq: int
    Hkv: int
    L: int
    window: int
    pool: int
    budget: int
    steps: int
    n_sink: int
    n_heavy: int
    layers: int = 1
    sigma0: float = 0.3
    sigma1: float = 0.3
    rope: bool = False
    seed: int = 0
    seed_per_b: int = 0      # seed increment per batch element
    seed_per_layer: int = 0  # seed increment per layer
    D: int = D_HEAD

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    def sigma(self, t: int) -> float:
        if self.steps <= 1:
            return self.sigma0
        return self.sigma0 + (self.sigma1 - self.sigma0) * t / (self.steps - 1)

    def scaled(self, **kw) -> "WorkloadConfig":
        return replace(self, **kw)


# The five benchmark configurations (shapes, budgets, seeds and structure counts).
CONFIGS = {
    1: WorkloadConfig(1, B=1, Hq=8, Hkv=8, L=2048, window=32, pool=7, budget=128, steps=16,
                      n_sink=4, n_heavy=32),
    2: WorkloadConfig(2, B=1, Hq=32, Hkv=8, L=8192, window=32, pool=7, budget=512, steps=64,
                      n_sink=8, n_heavy=82),
    3: WorkloadConfig(3, B=4, Hq=32, Hkv=8, L=32768, window=64, pool=7, budget=2048,
                      steps=128, n_sink=8, n_heavy=164, seed_per_b=1),
    4: WorkloadConfig(4, B=8, Hq=32, Hkv=8, L=16384, window=32, pool=7, budget=128,
                      steps=256, n_sink=8, n_heavy=164, layers=32, rope=True,
                      seed_per_b=1, seed_per_layer=1000),
    5: WorkloadConfig(5, B=1, Hq=28, Hkv=4, L=131072, window=64, pool=7, budget=4096,
                      steps=512, n_sink=8, n_heavy=655, sigma0=0.1, sigma1=0.6),
}

_TAG_U, _TAG_QOBS, _TAG_DECODE = 0xF001, 0xF002, 0xF003


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest even); returns the uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


def _rng(cfg: WorkloadConfig, layer: int, b: int, tag: int) -> np.random.Generator:
    seed = cfg.seed + cfg.seed_per_b * b + cfg.seed_per_layer * layer
    k0 = (cfg.cfg_id << 48) | (layer << 32) | (b << 16) | tag
    return np.random.Generator(np.random.Philox(key=[k0, seed]))


def _normal(rng: np.random.Generator, shape) -> np.ndarray:
    return rng.standard_normal(shape, dtype=np.float32)


def base_directions(cfg: WorkloadConfig, layer: int, b: int) -> np.ndarray:
    """u[Hq, D] float32: the base query direction of every head."""
    return _normal(_rng(cfg, layer, b, _TAG_U), (cfg.Hq, cfg.D))


def gen_q_obs(cfg: WorkloadConfig, layer: int = 0) -> np.ndarray:
    """Observation-window queries, bf16 bits, [B, Hq, W, D]."""
    out = np.empty((cfg.B, cfg.Hq, cfg.window, cfg.D), dtype=np.uint16)
    for b in range(cfg.B):
        u = base_directions(cfg, layer, b)
        noise = _normal(_rng(cfg, layer, b, _TAG_QOBS), (cfg.Hq, cfg.window, cfg.D))
        out[b] = f32_to_bf16_bits(u[:, None, :] + np.float32(0.3) * noise)
    return out


def _rope_rotate(k: np.ndarray, base: float = 5.0e5) -> np.ndarray:
    """Rotate rows of k[L, D] by their position (rotate-half pairing (i, i + D/2))."""
    L, D = k.shape
    half = D // 2
    inv = base ** (-np.arange(half, dtype=np.float64) / half)
    ang = np.arange(L, dtype=np.float64)[:, None] * inv[None, :]
    c, s = np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)
    a, bb = k[:, :half], k[:, half:]
    return np.concatenate([a * c - bb * s, bb * c + a * s], axis=1)


def gen_kv_unit(cfg: WorkloadConfig, layer: int, b: int, h: int, u: np.ndarray | None = None):
    """K and V of one (batch element, kv head): two [L, D] uint16 arrays of bf16 bits."""
    if u is None:
        u = base_directions(cfg, layer, b)
    rng = _rng(cfg, layer, b, h)
    k = _normal(rng, (cfg.L, cfg.D))
    v = _normal(rng, (cfg.L, cfg.D))
    n_cand = cfg.L - cfg.window
    n_heavy = min(cfg.n_heavy, max(0, n_cand - cfg.n_sink))
    if n_heavy > 0:
        pos = cfg.n_sink + rng.choice(n_cand - cfg.n_sink, size=n_heavy, replace=False)
        k[pos] *= np.float32(4.0)
    n_sink = min(cfg.n_sink, cfg.L)
    if n_sink > 0:
        G = cfg.G
        k[:n_sink] = np.float32(0.5) * u[h * G:(h + 1) * G].sum(axis=0)[None, :]
    if cfg.rope:
        k = _rope_rotate(k)
    return f32_to_bf16_bits(k), f32_to_bf16_bits(v)


def gen_kv(cfg: WorkloadConfig, layer: int = 0, threads: int | None = None):
    """K, V bf16 bits, each [B, Hkv, L, D]."""
    K = np.empty((cfg.B, cfg.Hkv, cfg.L, cfg.D), dtype=np.uint16)
    V = np.empty_like(K)
    us = [base_directions(cfg, layer, b) for b in range(cfg.B)]

    def work(bh):
        b, h = bh
        K[b, h], V[b, h] = gen_kv_unit(cfg, layer, b, h, us[b])

    units = [(b, h) for b in range(cfg.B) for h in range(cfg.Hkv)]
    threads = threads or min(len(units), os.cpu_count() or 1)
    if threads > 1:
        with ThreadPoolExecutor(threads) as ex:
            list(ex.map(work, units))
    else:
        for bh in units:
            work(bh)
    return K, V


def gen_decode_inputs(cfg: WorkloadConfig, q_obs_bits: np.ndarray, layer: int = 0,
                      steps: int | None = None):
    """Per-step decode inputs, bf16 bits: q [T, B, Hq, D], k_new and v_new [T, B, Hkv, D]."""
    T = cfg.steps if steps is None else steps
    q = np.empty((T, cfg.B, cfg.Hq, cfg.D), dtype=np.uint16)
    kn = np.empty((T, cfg.B, cfg.Hkv, cfg.D), dtype=np.uint16)
    vn = np.empty_like(kn)
    for b in range(cfg.B):
        rng = _rng(cfg, layer, b, _TAG_DECODE)
        qbar = bf16_bits_to_f32(q_obs_bits[b]).mean(axis=1)  # [Hq, D]
        for t in range(T):
            q[t, b] = f32_to_bf16_bits(qbar + np.float32(cfg.sigma(t)) * _normal(rng, (cfg.Hq, cfg.D)))
            kn[t, b] = f32_to_bf16_bits(_normal(rng, (cfg.Hkv, cfg.D)))
            vn[t, b] = f32_to_bf16_bits(_normal(rng, (cfg.Hkv, cfg.D)))
    return q, kn, vn


def small_config(**kw) -> WorkloadConfig:
    """A config-1-shaped workload with overridable sizes, for unit tests."""
    base = dict(cfg_id=99, B=1, Hq=4, Hkv=2, L=300, window=8, pool=5, budget=40, steps=4,
                n_sink=2, n_heavy=6)
    base.update(kw)
    return WorkloadConfig(**base)
