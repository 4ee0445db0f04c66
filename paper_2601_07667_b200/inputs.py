"""Seeded synthetic workloads for the ASL prefill hot path.

This module only *makes inputs*: bf16 bit patterns for the observation-window
queries, the keys and the values of one layer, plus the shape parameters of a
workload.  It holds none of the method's arithmetic (no softmax, pooling,
ranking, selection), so both the CPU oracle's tests and the CUDA path's tests
can draw the same tensors from it without sharing any code of the method.

Every tensor comes from a counter-based generator (Philox) keyed by
(seed, workload, layer, tensor), so any layer of any workload can be made on
its own, in any order, on any machine, with identical bits.

Tensors are returned as ``uint16`` arrays holding bf16 bit patterns:
  q_obs  [B][H_q][w][d]      last-w query rows of every request
  k, v   [sum n_b][H_k][d]   requests packed back to back (cu_seqlens offsets)
The five named workloads follow the shapes of the long-context models the
method was evaluated on (32 q heads / 8 kv heads, d = 128, contexts 4k-128k,
budgets of a few thousand tokens, window 32-128, pooling kernel 5-7); the
values are synthetic stand-ins for real activations: Gaussian background,
per-channel scale outliers, rotary position phase, and a few planted "heavy"
keys the window queries lean toward.
"""
from __future__ import annotations

import dataclasses
import math
from dataclasses import dataclass
from typing import Dict, Optional, Tuple

import numpy as np

POOL_AVG = 0
POOL_MAX = 1


@dataclass(frozen=True)
class Workload:
    name: str
    wid: int                      # numeric id used in the RNG key
    layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    window: int
    pool_kernel: int
    pool_mode: int                # POOL_AVG / POOL_MAX
    seqlens: Tuple[int, ...]      # n_b per request, window included
    budgets: Tuple[int, ...]      # KV budget per request, window included
    l_min: int
    l_obs: int
    tau: float
    # --- value recipe ---
    query_bias: float = 1.0 / math.sqrt(3.0)   # beta: q = g + beta*sqrt(d)*u  (cosine 0.5)
    heavy_per_head: int = 8                    # planted keys per (request, kv head)
    heavy_scale: float = 3.0                   # planted key = heavy_scale*sqrt(d)*u
    heavy_decay: float = 1.0                   # strength multiplied by decay**layer
    chan_scale: str = "none"                   # none | lognormal | student3
    chan_sigma: float = 0.5
    rope_base: float = 0.0                     # 0 = no rotary phase
    distractors: int = 0                       # near-duplicates of the first planted key
    distractor_cos: float = 0.9
    salience_start: float = 0.0                # weight of the layer-persistent per-token
    salience_step: float = 0.0                 #   salience: a_l = start + step*layer
    fresh_scale: float = 1.0                   # std of the layer-fresh Gaussian part of K

    @property
    def batch(self) -> int:
        return len(self.seqlens)

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def total_tokens(self) -> int:
        return int(sum(self.seqlens))

    def cu_seqlens(self) -> np.ndarray:
        return np.concatenate([[0], np.cumsum(self.seqlens)]).astype(np.int32)

    def kept(self, b: int) -> int:
        return min(self.budgets[b], self.seqlens[b])


def _rng(seed: int, wid: int, layer: int, tensor: int) -> np.random.Generator:
    """Philox stream for one (seed, workload, layer, tensor)."""
    key = np.array([(seed & 0xFFFFFFFF) << 8 | (wid & 0xFF),
                    ((layer + 1) & 0xFFFFFF) << 8 | (tensor & 0xFF)], dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


# tensor ids of the streams
_T_Q, _T_K, _T_V, _T_DIR, _T_POS, _T_CHAN, _T_SAL, _T_DIS, _T_LEN = range(9)
_STATIC = -1   # "layer" of the streams that stay fixed over the stack


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(bits).astype(np.float64)


def _c4_lengths(seed: int) -> Tuple[int, ...]:
    g = _rng(seed, 4, _STATIC, _T_LEN)
    return tuple(int(8192 + x) for x in g.integers(0, 57345, size=8))


def workload(name: str, seed: int = 0, **override) -> Workload:
    """One of the five named workloads (C1..C5).  Keyword overrides (for
    example ``seqlens=(1000,)``, ``layers=3``) give scaled-down variants with
    the same recipe for CPU-sized tests."""
    name = name.upper()
    if name == "C1":    # tiny stack
        wl = Workload("C1", 1, 4, 8, 2, 128, 32, 7, POOL_AVG, (4096,), (512,), 1, 2, 0.3,
                      heavy_per_head=8)
    elif name == "C2":  # 8B-shaped layer sweep
        wl = Workload("C2", 2, 32, 32, 8, 128, 64, 7, POOL_AVG, (32768,), (2048,), 10, 8, 0.3,
                      heavy_per_head=16, heavy_decay=0.97, chan_scale="lognormal", chan_sigma=0.5,
                      rope_base=500000.0, salience_start=0.04, salience_step=0.035)
    elif name == "C3":  # long-context single request
        wl = Workload("C3", 3, 12, 32, 8, 128, 64, 7, POOL_AVG, (131072,), (4096,), 2, 8, 0.3,
                      heavy_per_head=1, distractors=64, distractor_cos=0.9)
    elif name == "C4":  # ragged batched prefill
        lens = _c4_lengths(seed)
        wl = Workload("C4", 4, 4, 32, 8, 128, 32, 7, POOL_AVG, lens, tuple(n // 10 for n in lens),
                      1, 2, 0.3, heavy_per_head=-4096)   # negative: one planted key per 4096 tokens
    elif name == "C5":  # wide GQA, max pooling
        wl = Workload("C5", 5, 80, 64, 8, 128, 128, 5, POOL_MAX, (65536,), (4096,), 26, 8, 0.3,
                      heavy_per_head=32, chan_scale="student3")
    else:
        raise ValueError(f"unknown workload {name!r}")
    if override:
        wl = dataclasses.replace(wl, **override)
    if len(wl.budgets) != len(wl.seqlens):
        raise ValueError("budgets and seqlens differ in length")
    return wl


def _n_heavy(wl: Workload, n: int) -> int:
    if wl.heavy_per_head >= 0:
        return wl.heavy_per_head
    return -(-n // (-wl.heavy_per_head))


def directions(wl: Workload, seed: int) -> np.ndarray:
    """Unit direction u[b][h][d] the window queries lean toward (fixed over layers)."""
    g = _rng(seed, wl.wid, _STATIC, _T_DIR)
    u = g.standard_normal((wl.batch, wl.n_kv_heads, wl.head_dim), dtype=np.float32)
    u /= np.linalg.norm(u, axis=-1, keepdims=True)
    return u


def planted_positions(wl: Workload, seed: int):
    """Request-local positions of the planted heavy keys: list over requests of
    int arrays [H_k][count], all inside the past part [0, n_b - w)."""
    g = _rng(seed, wl.wid, _STATIC, _T_POS)
    out = []
    for n in wl.seqlens:
        T = n - wl.window
        cnt = min(_n_heavy(wl, n), T)
        pos = np.stack([np.sort(g.choice(T, size=cnt, replace=False)) for _ in range(wl.n_kv_heads)])
        out.append(pos.astype(np.int64))
    return out


def distractor_positions(wl: Workload, seed: int):
    """Positions of the near-duplicate keys (C3): list over requests of [H_k][distractors]."""
    if wl.distractors == 0:
        return [np.zeros((wl.n_kv_heads, 0), dtype=np.int64) for _ in wl.seqlens]
    g = _rng(seed, wl.wid, _STATIC, _T_DIS)
    planted = planted_positions(wl, seed)
    out = []
    for b, n in enumerate(wl.seqlens):
        T = n - wl.window
        rows = []
        for h in range(wl.n_kv_heads):
            free = np.setdiff1d(np.arange(T), planted[b][h], assume_unique=False)
            cnt = min(wl.distractors, free.size)
            rows.append(np.sort(g.choice(free, size=cnt, replace=False)))
        out.append(np.stack(rows).astype(np.int64))
    return out


def _channel_scale(wl: Workload, seed: int) -> Optional[np.ndarray]:
    if wl.chan_scale == "none":
        return None
    g = _rng(seed, wl.wid, _STATIC, _T_CHAN)
    shape = (wl.n_kv_heads, wl.head_dim)
    if wl.chan_scale == "lognormal":
        return np.exp(wl.chan_sigma * g.standard_normal(shape)).astype(np.float32)
    if wl.chan_scale == "student3":
        return np.abs(g.standard_t(3.0, size=shape)).astype(np.float32)
    raise ValueError(wl.chan_scale)


def _rope(x: np.ndarray, pos: np.ndarray, base: float) -> np.ndarray:
    """Rotary phase on [..., tokens, heads, d] (token axis = -3), pairs (c, c + d/2)."""
    d = x.shape[-1]
    half = d // 2
    inv = base ** (-np.arange(half, dtype=np.float64) * 2.0 / d)
    ang = pos.astype(np.float64)[:, None] * inv[None, :]           # [tokens][half]
    cos = np.cos(ang).astype(np.float32)[:, None, :]
    sin = np.sin(ang).astype(np.float32)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * cos - x2 * sin, x2 * cos + x1 * sin], axis=-1)


def layer_inputs(wl: Workload, layer: int, seed: int = 0, want_v: bool = True) -> Dict[str, np.ndarray]:
    """bf16 bit patterns of one layer's q_obs, k, v for workload ``wl``."""
    d, w, Hq, Hk, G = wl.head_dim, wl.window, wl.n_q_heads, wl.n_kv_heads, wl.group
    sd = math.sqrt(d)
    total = wl.total_tokens
    cu = wl.cu_seqlens()
    u = directions(wl, seed)                              # [B][Hk][d]
    planted = planted_positions(wl, seed)
    distract = distractor_positions(wl, seed)
    chan = _channel_scale(wl, seed)

    gq = _rng(seed, wl.wid, layer, _T_Q)
    gk = _rng(seed, wl.wid, layer, _T_K)
    q = gq.standard_normal((wl.batch, Hq, w, d), dtype=np.float32)
    k = gk.standard_normal((total, Hk, d), dtype=np.float32)
    if wl.fresh_scale != 1.0:
        k *= np.float32(wl.fresh_scale)
    if chan is not None:
        k *= chan[None, :, :]
    if wl.rope_base > 0.0:
        for b in range(wl.batch):
            n = wl.seqlens[b]
            sl = slice(int(cu[b]), int(cu[b + 1]))
            k[sl] = _rope(k[sl], np.arange(n), wl.rope_base)
            qb = np.swapaxes(q[b], 0, 1)                  # [w][Hq][d]
            q[b] = np.swapaxes(_rope(qb, np.arange(n - w, n), wl.rope_base), 0, 1)

    sal_w = wl.salience_start + wl.salience_step * layer
    gs = _rng(seed, wl.wid, _STATIC, _T_SAL) if sal_w != 0.0 else None
    gd = _rng(seed, wl.wid, _STATIC, _T_DIS + 16) if wl.distractors else None
    strength = wl.heavy_scale * (wl.heavy_decay ** layer)
    for b in range(wl.batch):
        n = wl.seqlens[b]
        o = int(cu[b])
        # window queries lean toward u of their kv head
        for a in range(Hq):
            q[b, a] += np.float32(wl.query_bias * sd) * u[b, a // G][None, :]
        if gs is not None:   # layer-persistent per-token salience along u (same z_j at every layer)
            z = gs.standard_normal(n, dtype=np.float32)
            k[o:o + n] += np.float32(sal_w / wl.query_bias) * z[:, None, None] * u[b][None, :, :]
        for h in range(Hk):
            k[o + planted[b][h], h, :] = np.float32(strength * sd) * u[b, h]
            if wl.distractors:
                needle = u[b, h]
                m = distract[b][h].size
                noise = gd.standard_normal((m, d), dtype=np.float32)
                noise -= (noise @ needle)[:, None] * needle[None, :]
                noise /= np.linalg.norm(noise, axis=-1, keepdims=True)
                c = wl.distractor_cos
                k[o + distract[b][h], h, :] = np.float32(strength * sd) * (
                    c * needle[None, :] + math.sqrt(1.0 - c * c) * noise)
    out = {"q_obs": f32_to_bf16_bits(q), "k": f32_to_bf16_bits(k), "cu_seqlens": cu}
    if want_v:
        gv = _rng(seed, wl.wid, layer, _T_V)
        out["v"] = f32_to_bf16_bits(gv.standard_normal((total, Hk, d), dtype=np.float32))
    return out


def keys_to_fp8(k_bits: np.ndarray, scale=None):
    """An FP8 (E4M3) copy of a layer's keys, as a quantised K cache would hold them: uint8 codes
    [n][H_k][d] and one fp32 scale per kv head, chosen (unless given) so that the head's largest
    magnitude maps to the format's largest finite value (448).  Rounding to nearest by the library
    cast; input preparation only -- the keys the path is then asked to score ARE code x scale."""
    import torch
    k = torch.from_numpy(bf16_bits_to_f32(k_bits))
    if scale is None:
        amax = k.abs().amax(dim=(0, 2)).clamp_min(1e-30)
        scale = (amax / 448.0).to(torch.float32)
    else:
        scale = torch.as_tensor(np.asarray(scale, dtype=np.float32))
    codes = (k / scale[None, :, None]).clamp(-448.0, 448.0).to(torch.float8_e4m3fn).view(torch.uint8)
    return codes.numpy().copy(), scale.numpy().copy()


def quantised_scores(n_heads: int, T: int, levels: int, seed: int = 0) -> np.ndarray:
    """fp32 score rows [n_heads][T] drawn from only ``levels`` distinct values, so
    that the k-th boundary of a top-k falls inside a run of exact ties."""
    g = _rng(seed, 31, _STATIC, 0)
    return (g.integers(0, levels, size=(n_heads, T)).astype(np.float32) / np.float32(levels)) ** 2
