"""Seeded synthetic inputs for the affix-cache refresh path.

This module only draws random numbers and lays them out; it holds none of the
method's arithmetic (no normalisation, projection, attention, scoring or
selection).  Both the CPU oracle's tests and the CUDA path's tests/benchmark
take their inputs from here, so that the two sides see identical bytes.

All "bf16" arrays are numpy ``uint16`` arrays holding the bf16 bit pattern
(numpy has no bf16 dtype).  The only numeric helpers are the format conversion
bf16 <-> fp32 and the rotary cos/sin *input table* (an argument of the
library, built once in fp64 and stored as fp32).

Shapes follow the paper's workloads: a shared affix F = {l..r} of L tokens at
the prefix, middle or end of a T-token context, a request-specific part, and a
masked generation region decoded in 32-token blocks (Section 3.1, Section 5
set-up: generation length 256, block 32).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, Optional

import numpy as np

SEED_BASE = 0xAC000000

# tensor ids inside one layer (added to the layer's seed)
_TENSOR_IDS = dict(attn_norm_g=0, wq=1, wk=2, wv=3, bq=4, bk=5, bv=6, wo=7,
                   mlp_norm_g=8, w_gate=9, w_up=10, w_down=11)


# --------------------------------------------------------------------------
# bf16 <-> fp32 format conversion (data formatting only)
# --------------------------------------------------------------------------
def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round an fp32 array to bf16 (round-to-nearest-even); returns uint16 bits."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) to fp32 exactly."""
    u = np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32)


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(int(seed) & 0xFFFFFFFFFFFFFFFF))


def normal_bf16(seed: int, shape, std: float, mean: float = 0.0) -> np.ndarray:
    """i.i.d. N(mean, std) drawn in fp32 from a Philox stream, stored as bf16 bits."""
    g = _rng(seed)
    a = g.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        a *= np.float32(std)
    if mean != 0.0:
        a += np.float32(mean)
    return f32_to_bf16_bits(a)


# --------------------------------------------------------------------------
# shapes
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class LayerShape:
    """One bidirectional transformer layer (pre-norm, RMSNorm, RoPE, SwiGLU)."""
    hidden: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    rms_eps: float = 1e-5
    qkv_bias: bool = False
    rope_theta: float = 5e5
    name: str = ""

    @property
    def q_dim(self) -> int:
        return self.n_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim

    def weight_bytes(self) -> int:
        D, F = self.hidden, self.ffn
        n = D * self.q_dim + 2 * D * self.kv_dim + self.q_dim * D + 3 * D * F
        return 2 * n


TINY = LayerShape(256, 4, 4, 64, 1024, 1e-5, False, 5e5, "tiny")
TINY_GQA = LayerShape(256, 4, 2, 64, 768, 1e-6, True, 1e6, "tiny-gqa")
LLADA_8B = LayerShape(4096, 32, 32, 128, 12288, 1e-5, False, 5e5, "llada-8b")
DREAM_7B = LayerShape(3584, 28, 4, 128, 18944, 1e-6, True, 1e6, "dream-7b")


@dataclass
class Layout:
    """Where the affix, the request-specific rows and the masked rows sit.

    ``masked_pos`` [B, m] and ``extra_rows`` [B, e] are absolute positions
    outside the affix span; ``extra_rows`` are the request-specific rows that
    are recomputed together with the anchors (may be empty).
    """
    batch: int
    ctx_len: int
    affix_start: int
    affix_len: int
    masked_pos: np.ndarray
    extra_rows: np.ndarray
    name: str = ""

    @property
    def n_masked(self) -> int:
        return int(self.masked_pos.shape[1])

    @property
    def n_extra(self) -> int:
        return int(self.extra_rows.shape[1])


def make_layout(batch: int, pre: int, affix: int, post: int, gen: int,
                n_masked: int, extra: str = "none", tail: int = 0,
                name: str = "") -> Layout:
    """Context = [pre request rows][affix][post request rows][gen rows][tail rows].

    The first ``n_masked`` generation rows are the masked positions M.
    ``extra``: "none" (anchors only), "all" (every non-affix row, the paper's
    recompute set of Section 3.3) or "masked" (only the masked rows).
    """
    T = pre + affix + post + gen + tail
    l = pre
    gen0 = pre + affix + post
    assert 0 <= n_masked <= gen
    masked = np.arange(gen0, gen0 + n_masked, dtype=np.int32)
    non_affix = np.concatenate([np.arange(0, l), np.arange(l + affix, T)]).astype(np.int32)
    if extra == "none":
        ex = np.zeros((0,), np.int32)
    elif extra == "all":
        ex = non_affix
    elif extra == "masked":
        ex = masked.copy()
    else:
        raise ValueError(extra)
    return Layout(batch, T, l, affix,
                  np.ascontiguousarray(np.broadcast_to(masked, (batch, masked.size))),
                  np.ascontiguousarray(np.broadcast_to(ex, (batch, ex.size))), name)


# the benchmark configurations (shape and layout only)
def config_layout(cfg: int, extra: str = "none", n_masked: Optional[int] = None,
                  batch: Optional[int] = None) -> Layout:
    if cfg == 1:   # 128 affix + 64 request + 32 masked + 32 already-decoded rows = 256
        return make_layout(batch or 1, 0, 128, 64, 32, 32 if n_masked is None else n_masked,
                           extra, tail=32, name="cfg1-tiny")
    if cfg == 2:   # 512 affix + 256 request + 256 generation (32-token blocks)
        return make_layout(batch or 1, 0, 512, 256, 256, 32 if n_masked is None else n_masked,
                           extra, name="cfg2-llada-layer")
    if cfg == 3:
        return make_layout(batch or 16, 0, 2048, 256, 256, 256 if n_masked is None else n_masked,
                           extra, name="cfg3-llada-b16")
    if cfg == 4:   # affix in the middle
        return make_layout(batch or 32, 128, 1024, 256, 256, 256 if n_masked is None else n_masked,
                           extra, name="cfg4-dream-b32")
    raise ValueError(cfg)


def sweep_layout(affix_len: int, batch: int, place: str, extra: str = "none") -> Layout:
    """Sweep point: 64 request rows + 32 masked rows around an affix of the given length."""
    if place == "prefix":
        return make_layout(batch, 0, affix_len, 64, 32, 32, extra, name=f"sweep-L{affix_len}-prefix")
    if place == "middle":
        return make_layout(batch, 32, affix_len, 32, 32, 32, extra, name=f"sweep-L{affix_len}-middle")
    if place == "suffix":
        # generation rows sit before the affix: [64 request][32 gen] affix
        T = 96 + affix_len
        masked = np.arange(64, 96, dtype=np.int32)
        non_affix = np.arange(0, 96, dtype=np.int32)
        ex = {"none": np.zeros((0,), np.int32), "all": non_affix, "masked": masked}[extra]
        return Layout(batch, T, 96, affix_len,
                      np.ascontiguousarray(np.broadcast_to(masked, (batch, 32))),
                      np.ascontiguousarray(np.broadcast_to(ex, (batch, ex.size))),
                      f"sweep-L{affix_len}-suffix")
    raise ValueError(place)


# --------------------------------------------------------------------------
# tensors
# --------------------------------------------------------------------------
def rope_table(n_pos: int, head_dim: int, theta: float):
    """cos/sin input table, fp32 [n_pos, head_dim/2], angles evaluated in fp64."""
    half = head_dim // 2
    inv = np.float64(theta) ** (-np.arange(half, dtype=np.float64) / half)
    ang = np.arange(n_pos, dtype=np.float64)[:, None] * inv[None, :]
    return np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)


def layer_weights(shape: LayerShape, cfg_id: int = 0, layer: int = 0,
                  std: float = 0.02) -> Dict[str, Optional[np.ndarray]]:
    """bf16 weights ~ N(0, std), [out, in] row-major; norm gains ~ N(1, 0.05)."""
    base = SEED_BASE + 4096 * cfg_id + 64 * layer
    D, F = shape.hidden, shape.ffn
    dims = dict(wq=(shape.q_dim, D), wk=(shape.kv_dim, D), wv=(shape.kv_dim, D),
                wo=(D, shape.q_dim), w_gate=(F, D), w_up=(F, D), w_down=(D, F))
    w: Dict[str, Optional[np.ndarray]] = {}
    for k, shp in dims.items():
        w[k] = normal_bf16(base + _TENSOR_IDS[k], shp, std)
    w["attn_norm_g"] = normal_bf16(base + _TENSOR_IDS["attn_norm_g"], (D,), 0.05, 1.0)
    w["mlp_norm_g"] = normal_bf16(base + _TENSOR_IDS["mlp_norm_g"], (D,), 0.05, 1.0)
    if shape.qkv_bias:
        w["bq"] = normal_bf16(base + _TENSOR_IDS["bq"], (shape.q_dim,), std)
        w["bk"] = normal_bf16(base + _TENSOR_IDS["bk"], (shape.kv_dim,), std)
        w["bv"] = normal_bf16(base + _TENSOR_IDS["bv"], (shape.kv_dim,), std)
    else:
        w["bq"] = w["bk"] = w["bv"] = None
    return w


def hidden_states(shape: LayerShape, lay: Layout, seed: int, ctx_seed: int,
                  rho: float = 0.3) -> np.ndarray:
    """Layer input x, bf16 bits [B, T, D].

    Affix rows share one base draw across the batch (the affix text is shared);
    every row also carries a context-dependent perturbation of relative size
    ``rho`` drawn from ``ctx_seed`` (the request-specific context).  Calling
    this twice with the same ``seed`` and different ``ctx_seed`` gives the
    "same affix under a different suffix" pair used for stale caches.
    """
    B, T, D = lay.batch, lay.ctx_len, shape.hidden
    l, L = lay.affix_start, lay.affix_len
    x = np.empty((B, T, D), np.float32)
    affix_base = _rng(seed).standard_normal((L, D), dtype=np.float32)
    for b in range(B):
        x[b] = _rng(seed + 7919 * (b + 1)).standard_normal((T, D), dtype=np.float32)
        x[b, l:l + L] = affix_base
        x[b] += np.float32(rho) * _rng(ctx_seed + 104729 * (b + 1)).standard_normal((T, D), dtype=np.float32)
    return f32_to_bf16_bits(x)


def random_kv_cache(shape: LayerShape, lay: Layout, seed: int, ctx_capacity: Optional[int] = None,
                    std: Optional[float] = None, hot_frac: float = 0.0):
    """Token-major K and V caches, bf16 bits [B, ctx_capacity, Hkv, d].

    Entries ~ N(0, std) with std defaulting to 0.02*sqrt(hidden), the scale a
    N(0,0.02) projection of a unit-RMS row produces.  The affix rows are one
    draw shared by the whole batch (a shared cache copied into each request's
    working cache).  ``hot_frac`` scales that fraction of affix K rows by 4 to
    give a skewed score distribution.
    """
    cap = ctx_capacity or lay.ctx_len
    B, l, L = lay.batch, lay.affix_start, lay.affix_len
    s = std if std is not None else 0.02 * float(np.sqrt(shape.hidden))
    shp = (B, cap, shape.n_kv_heads, shape.head_dim)
    k = np.empty(shp, np.uint16)
    v = np.empty(shp, np.uint16)
    ak = bf16_bits_to_f32(normal_bf16(seed + 1, (L,) + shp[2:], s))
    av = normal_bf16(seed + 2, (L,) + shp[2:], s)
    if hot_frac > 0.0:
        hot = _rng(seed + 3).random(L) < hot_frac
        ak[hot] *= np.float32(4.0)
    ak = f32_to_bf16_bits(ak)
    for b in range(B):
        k[b] = normal_bf16(seed + 11 + 2 * b, shp[1:], s)
        v[b] = normal_bf16(seed + 12 + 2 * b, shp[1:], s)
        k[b, l:l + L] = ak
        v[b, l:l + L] = av
    return k, v


def random_q_mask(shape: LayerShape, lay: Layout, seed: int, std: Optional[float] = None) -> np.ndarray:
    """Masked-row queries, bf16 bits [B, m, H, d], ~ N(0, 0.02*sqrt(hidden))."""
    s = std if std is not None else 0.02 * float(np.sqrt(shape.hidden))
    return normal_bf16(seed, (lay.batch, lay.n_masked, shape.n_heads, shape.head_dim), s)


@dataclass
class Case:
    """Everything one layer-step needs, as host arrays."""
    shape: LayerShape
    layout: Layout
    weights: Dict[str, Optional[np.ndarray]]
    x: np.ndarray            # bf16 bits [B, T, D]
    cache_k: np.ndarray      # bf16 bits [B, cap, Hkv, d]
    cache_v: np.ndarray
    rope_cos: np.ndarray     # fp32 [cap, d/2]
    rope_sin: np.ndarray
    ratio: float
    x_stale: Optional[np.ndarray] = None   # same affix under another context
    meta: dict = field(default_factory=dict)


def make_case(shape: LayerShape, lay: Layout, ratio: float, cfg_id: int = 0, layer: int = 0,
              with_stale_hidden: bool = False, hot_frac: float = 0.0,
              weights: Optional[Dict[str, Optional[np.ndarray]]] = None) -> Case:
    """One single-layer case with a randomly drawn (stale) cache.  ``weights`` reuses an
    earlier ``layer_weights`` draw (they depend only on shape, cfg_id and layer)."""
    base = SEED_BASE + 4096 * cfg_id + 64 * layer
    w = weights if weights is not None else layer_weights(shape, cfg_id, layer)
    x = hidden_states(shape, lay, base + 20, base + 21)
    xs = hidden_states(shape, lay, base + 20, base + 22) if with_stale_hidden else None
    ck, cv = random_kv_cache(shape, lay, base + 30, hot_frac=hot_frac)
    cos, sin = rope_table(lay.ctx_len, shape.head_dim, shape.rope_theta)
    return Case(shape, lay, w, x, ck, cv, cos, sin, ratio, xs)
