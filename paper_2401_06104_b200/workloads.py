"""Seeded synthetic workloads for the TOVA decode path.

This module only *draws inputs*: Gaussian queries, keys and values with the
layer geometry of the 6-7B models the paper evaluates (Section 5.3), rotary
position embedding applied to q/k where a workload says so, and a few
structured keys (sink / heavy hitters).  It holds none of the method's
arithmetic (no softmax, no eviction), so both the CUDA path and the CPU
checker may consume its arrays.

Every token's (q, k, v) is a pure function of (seed, layer, position): a
counter-based Philox stream is keyed by those three integers, so any token
can be regenerated alone, in any order, on any machine.

All arrays are float32.  For bf16 workloads the values are rounded once to
bf16 (round-to-nearest-even) and stored back as float32, so a float32 consumer
and a bf16 consumer see bit-identical numbers.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Tuple

import numpy as np

DTYPE_FP32 = 0
DTYPE_BF16 = 1


@dataclass(frozen=True)
class Workload:
    """Geometry and input recipe of one synthetic workload."""

    name: str
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    capacity: int
    dtype: int                 # DTYPE_FP32 or DTYPE_BF16 (storage of q, k, v)
    prompt: int                # prompt tokens (prefill)
    decode: int                # decode steps after the prompt
    comp_std: float            # std of every q and k component
    v_std: float = 1.0
    rope: bool = False         # rotate-half RoPE, base 10000, original positions
    # structured keys
    key0_gain: float = 1.0     # norm multiplier of the key at position 0
    sink_bias: float = 0.0     # persistent sink: see _token()
    heavy_frac: float = 0.0    # fraction of keys with norm x heavy_gain
    heavy_period: int = 0      # every heavy_period-th key gets norm x heavy_gain
    heavy_gain: float = 1.0
    n_layers: int = 1
    seed: int = 0

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def sm_scale(self) -> float:
        return 1.0 / float(np.sqrt(self.head_dim))

    @property
    def elem_bytes(self) -> int:
        return 2 if self.dtype == DTYPE_BF16 else 4

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)

    def step_bytes(self, live: int | None = None) -> int:
        """Algorithmic HBM bytes of one layer-step: the K/V cache read plus
        one slot written, for all sequences."""
        n = self.capacity if live is None else live
        row = self.n_kv_heads * self.head_dim * self.elem_bytes
        return self.batch * (2 * n * row + 2 * row)


_SQRT2 = float(np.sqrt(2.0))

WORKLOADS: Dict[str, Workload] = {
    # 1 layer, batch 1, 4 MHA heads, D 64, fp32, capacity 64; components
    # N(0,1)/8, key at position 0 has 8x norm.
    "tiny": Workload("tiny", 1, 4, 4, 64, 64, DTYPE_FP32, 32, 512,
                     comp_std=1.0 / 8.0, v_std=1.0 / 8.0, key0_gain=8.0, seed=0),
    # Same geometry, unit-variance components (logit std 1): separates the
    # scores better than "tiny".
    "tiny_unit": Workload("tiny_unit", 1, 4, 4, 64, 64, DTYPE_FP32, 32, 512,
                          comp_std=1.0, key0_gain=8.0, seed=0),
    # LLaMA-2-7B-shaped layer.
    "llama2_7b_layer": Workload("llama2_7b_layer", 8, 32, 32, 128, 512, DTYPE_BF16,
                                2048, 2048, comp_std=_SQRT2,
                                rope=True, sink_bias=3.0, seed=1),
    # Mistral-7B-shaped GQA layer (capacity swept by the caller).
    "mistral_7b_gqa": Workload("mistral_7b_gqa", 32, 32, 8, 128, 1024, DTYPE_BF16,
                               4096, 1024, comp_std=1.0, heavy_frac=0.02,
                               heavy_gain=3.0, seed=2),
    # 32 layers of the LLaMA-2-7B shape, batch 64, capacity 1024.
    "llama2_7b_full": Workload("llama2_7b_full", 64, 32, 32, 128, 1024, DTYPE_BF16,
                               8192, 1, comp_std=_SQRT2,
                               n_layers=32, seed=3),
    # Yi-6B-shaped GQA layer, long stream.
    "yi_6b_long": Workload("yi_6b_long", 4, 32, 4, 128, 4096, DTYPE_BF16,
                           4096, 65904, comp_std=1.0, heavy_period=1024,
                           heavy_gain=3.0, sink_bias=3.0, seed=4),
}
# "logit std ~ 2" with sm_scale = 1/sqrt(D) needs std_q * std_k = 2: every q and
# k component of the LLaMA-shaped workloads has std sqrt(2).


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); float32 out."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """Upper 16 bits of bf16-representable float32 values, as uint16."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    return (u >> np.uint32(16)).astype(np.uint16)


def _rng(seed: int, layer: int, pos: int, stream: int = 0) -> np.random.Generator:
    """Counter-based stream for one (seed, layer, position)."""
    key = [(int(seed) << 32) | (int(layer) << 8) | int(stream), int(pos)]
    return np.random.Generator(np.random.Philox(key=np.array(key, dtype=np.uint64)))


def _rope(x: np.ndarray, pos: int) -> np.ndarray:
    """Rotate-half rotary embedding at one position; x is [..., D] float64."""
    d = x.shape[-1]
    half = d // 2
    inv = 10000.0 ** (-np.arange(half, dtype=np.float64) * 2.0 / d)
    ang = float(pos) * inv
    c, s = np.cos(ang), np.sin(ang)
    a, b = x[..., :half], x[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def sink_direction(w: Workload, layer: int) -> np.ndarray:
    """Unit vectors [Hkv, D] shared by the sink key and every query's bias."""
    g = _rng(w.seed, layer, 0, stream=1)
    u = g.standard_normal((w.n_kv_heads, w.head_dim))
    return u / np.linalg.norm(u, axis=-1, keepdims=True)


def token(w: Workload, pos: int, layer: int = 0) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """(q [B,H,D], k [B,Hkv,D], v [B,Hkv,D]) of the token at one position.

    q and k are post-RoPE where the workload asks for RoPE.  Structured keys:
      * key0_gain: the key at position 0 is multiplied by it;
      * sink_bias s > 0: the key at position 0 is replaced by sqrt(D)*comp_std*u
        (u a fixed unit direction per KV head) and every query gets
        s*comp_std*u added, so that key's logit has mean s logit-stds at
        every step: a sink that stays attended, as the paper observes for the
        first token (Section 7.3);
      * heavy_frac / heavy_period: those keys get heavy_gain times the norm.
    """
    B, H, Hkv, D = w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim
    g = _rng(w.seed, layer, pos)
    q = g.standard_normal((B, H, D)) * w.comp_std
    k = g.standard_normal((B, Hkv, D)) * w.comp_std
    v = g.standard_normal((B, Hkv, D)) * w.v_std
    uni = g.random((B, Hkv))
    if w.rope:
        q = _rope(q, pos)
        k = _rope(k, pos)
    if w.heavy_frac > 0.0:
        k = np.where((uni < w.heavy_frac)[..., None], k * w.heavy_gain, k)
    if w.heavy_period > 0 and pos > 0 and pos % w.heavy_period == 0:
        k = k * w.heavy_gain
    if w.sink_bias > 0.0:
        u = sink_direction(w, layer)                              # [Hkv, D]
        q = q + (w.sink_bias * w.comp_std) * np.repeat(u, w.group, axis=0)[None]
        if pos == 0:
            k = np.broadcast_to(u[None] * (np.sqrt(D) * w.comp_std), k.shape).copy()
    if pos == 0 and w.key0_gain != 1.0:
        k = k * w.key0_gain
    out = [np.ascontiguousarray(a, dtype=np.float32) for a in (q, k, v)]
    if w.dtype == DTYPE_BF16:
        out = [round_to_bf16(a) for a in out]
    return out[0], out[1], out[2]


def tokens(w: Workload, first_pos: int, count: int, layer: int = 0):
    """Stack `count` consecutive tokens: q [T,B,H,D], k and v [T,B,Hkv,D]."""
    qs, ks, vs = [], [], []
    for t in range(first_pos, first_pos + count):
        q, k, v = token(w, t, layer)
        qs.append(q), ks.append(k), vs.append(v)
    shape_q = (0, w.batch, w.n_q_heads, w.head_dim)
    shape_k = (0, w.batch, w.n_kv_heads, w.head_dim)
    if count == 0:
        return (np.zeros(shape_q, np.float32), np.zeros(shape_k, np.float32),
                np.zeros(shape_k, np.float32))
    return np.stack(qs), np.stack(ks), np.stack(vs)
