"""CPU oracle for the affix-cache refresh path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, step-by-step numpy restatement of what the path computes:
anchor scoring (Eq. 4-5), top-K anchor selection (Eq. 6), selective
recomputation of the anchor rows and request-specific rows (Section 3.3,
Section 4.3) and the construction of the working cache (Section 3.3,
Section 4.1).  Nothing here is used by the product: only the tests, the
smoke check and the benchmark's CPU-baseline leg import this module, and it
shares no code with the CUDA path.

Arithmetic: every contraction, normalisation and softmax runs in fp64
(numpy matmul is used as a library step).  Values are rounded to bf16
(round-to-nearest-even, via fp32) exactly where the path *stores* a bf16
tensor: the normalised rows, q/k/v (after the rotary embedding for q and k),
the attention output, the post-attention hidden, the second normalised rows,
the gated activation and the layer output.  Softmax weights are never
rounded.  ``round_storage=False`` switches every one of those roundings off
(pure fp64) so that the share of the error budget spent on storage rounding
can be measured.

The paper fixes the method, not the layer: the layer architecture (pre-norm
RMSNorm, rotate-half RoPE, SwiGLU MLP, residuals) is the LLaDA/Dream-style
layer named by the benchmark configurations; the paper is silent on it.

Readings taken where the paper is silent (each is a parameter or stated in
the function that takes it):
  * Eq. 4 softmax domain: the affix keys only, as the equation is written
    (``norm_full=False``).  ``norm_full=True`` normalises over every key of
    the logical context and keeps the affix columns (the prose of
    Section 3.2 describes the probe attending with the affix as past KV).
  * K from the ratio: ceil(ratio * L), clipped to [0, L]  (Eq. 6 gives K only).
  * TopK ties: the lower position wins; anchors are returned ascending.
  * Anchor queries attend the *refreshed* anchor K/V (store-then-attend,
    Appendix C.1), over all T positions with no mask (bidirectional).

Also here: the two ablation variants of the paper that are arithmetic (the KV-deviation
selector of the appendix, ``kv_deviation_scores``; the DropNA key layout of Section 5.3,
``dropna_key_keep`` / ``recompute_rows(key_keep=)``), each pinned like the rest.

Pins (tests marked "not gpu"): brute-force nested-loop scoring and selection
on tiny inputs, closed forms (zero queries -> uniform scores; score mass
= N*H*m), library special cases (torch scaled_dot_product_attention,
rms_norm, silu, a library rotary embedding), ratio 1.0 == a separately
written dense layer, ratio 0 == direct reuse, byte-identity of untouched
rows, attention rows summing to one.  The paper prints no intermediate
numeric value (no score vector, anchor list or K/V entry), so agreement with
the authors' own code is unpinned; every function is pinned to its definition.
"""
from __future__ import annotations

import math
from typing import Dict, Optional, Sequence, Tuple

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------
# storage format
# --------------------------------------------------------------------------
def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> exact fp64 values."""
    u = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(F64)


def f64_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """fp64 -> bf16 bits, round-to-nearest-even (through fp32)."""
    u = np.ascontiguousarray(np.asarray(a, dtype=F64).astype(np.float32)).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_round(a: np.ndarray) -> np.ndarray:
    """Value of ``a`` after being stored as bf16 and read back (fp64 in, fp64 out)."""
    return bf16_bits_to_f64(f64_to_bf16_bits(a))


def _store(a: np.ndarray, round_storage: bool) -> np.ndarray:
    return bf16_round(a) if round_storage else np.asarray(a, dtype=F64)


def _w(weights: Dict[str, Optional[np.ndarray]], name: str) -> Optional[np.ndarray]:
    """A weight as fp64; accepts bf16 bits (uint16) or a float array."""
    t = weights.get(name)
    if t is None:
        return None
    if t.dtype == np.uint16:
        return bf16_bits_to_f64(t)
    return np.asarray(t, dtype=F64)


# --------------------------------------------------------------------------
# layer pieces (architecture of the benchmark configurations)
# --------------------------------------------------------------------------
def rmsnorm(x: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    """x_i * rsqrt(mean_i(x_i^2) + eps) * g_i, per row."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * g


def rope(v: np.ndarray, pos: np.ndarray, cos: np.ndarray, sin: np.ndarray) -> np.ndarray:
    """Rotary embedding, rotate-half pairing (i, i + d/2).

    v [n, heads, d]; pos [n] absolute positions; cos/sin [n_pos, d/2] input table.
    out_i       = v_i * cos_i - v_{i+d/2} * sin_i
    out_{i+d/2} = v_{i+d/2} * cos_i + v_i * sin_i
    """
    half = v.shape[-1] // 2
    c = np.asarray(cos, F64)[pos][:, None, :]
    s = np.asarray(sin, F64)[pos][:, None, :]
    a, b = v[..., :half], v[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def silu(z: np.ndarray) -> np.ndarray:
    return z / (1.0 + np.exp(-z))


def softmax_rows(z: np.ndarray) -> np.ndarray:
    z = z - np.max(z, axis=-1, keepdims=True)
    e = np.exp(z)
    return e / np.sum(e, axis=-1, keepdims=True)


def project_q(weights, shape, xn: np.ndarray, pos: np.ndarray, cos, sin, round_storage=True) -> np.ndarray:
    """q = RoPE(Wq xn + bq) stored bf16; [n, H, d]."""
    q = xn @ _w(weights, "wq").T
    if weights.get("bq") is not None:
        q = q + _w(weights, "bq")
    q = q.reshape(-1, shape.n_heads, shape.head_dim)
    return _store(rope(q, pos, cos, sin), round_storage)


def project_kv(weights, shape, xn: np.ndarray, pos: np.ndarray, cos, sin, round_storage=True):
    """k = RoPE(Wk xn + bk), v = Wv xn + bv, both stored bf16; [n, Hkv, d]."""
    k = xn @ _w(weights, "wk").T
    v = xn @ _w(weights, "wv").T
    if weights.get("bk") is not None:
        k = k + _w(weights, "bk")
    if weights.get("bv") is not None:
        v = v + _w(weights, "bv")
    k = k.reshape(-1, shape.n_kv_heads, shape.head_dim)
    v = v.reshape(-1, shape.n_kv_heads, shape.head_dim)
    return _store(rope(k, pos, cos, sin), round_storage), _store(v, round_storage)


def normed_rows(weights, shape, x_rows: np.ndarray, round_storage=True) -> np.ndarray:
    """xn = RMSNorm(x) * g1 stored bf16."""
    return _store(rmsnorm(x_rows, _w(weights, "attn_norm_g"), shape.rms_eps), round_storage)


def masked_queries(weights, shape, x_rows: np.ndarray, pos: np.ndarray, cos, sin,
                   round_storage=True) -> np.ndarray:
    """Q_mask of Eq. 4: post-RoPE queries of the masked positions at this layer; [m, H, d]."""
    xn = normed_rows(weights, shape, x_rows, round_storage)
    return project_q(weights, shape, xn, pos, cos, sin, round_storage)


# --------------------------------------------------------------------------
# Eq. 4-5: anchor scoring
# --------------------------------------------------------------------------
def score_anchors(q_mask: np.ndarray, k_affix: np.ndarray, k_context: Optional[np.ndarray] = None,
                  affix_start: int = 0, norm_full: bool = False) -> np.ndarray:
    """One layer's contribution to s_j (Eq. 5), fp64 [L].

    q_mask  [m, H, d]    queries of the masked positions (post-RoPE)
    k_affix [L, Hkv, d]  precomputed keys of the affix tokens
    a_{j,k}^{(h)} = Softmax(Q_mask^{(h)} K_affix^{(h)T} / sqrt(d_h))[k, j]   (Eq. 4)
    s_j          += sum_h sum_{k in M} a_{j,k}^{(h)}                          (Eq. 5)
    With grouped-query attention query head h reads KV head h // (H / Hkv).
    ``norm_full``: the softmax runs over all keys of ``k_context`` [T, Hkv, d]
    (whose rows affix_start.. are the affix) and only the affix columns are kept.
    """
    m, H, d = q_mask.shape
    L, Hkv, _ = k_affix.shape
    group = H // Hkv
    s = np.zeros(L, F64)
    for h in range(H):
        kh = h // group
        if norm_full:
            z = q_mask[:, h, :] @ k_context[:, kh, :].T / math.sqrt(d)     # [m, T]
            a = softmax_rows(z)[:, affix_start:affix_start + L]
        else:
            z = q_mask[:, h, :] @ k_affix[:, kh, :].T / math.sqrt(d)       # [m, L]
            a = softmax_rows(z)
        s += a.sum(axis=0)
    return s


# --------------------------------------------------------------------------
# Eq. 6: anchor selection
# --------------------------------------------------------------------------
def k_from_ratio(affix_len: int, ratio: float) -> int:
    """K = ceil(ratio * L) clipped to [0, L]; ratio 0 -> 0, ratio 1 -> L."""
    k = int(math.ceil(ratio * affix_len - 1e-9))
    return max(0, min(int(affix_len), k))


def select_topk(scores: np.ndarray, K: int, band_rel: float = 1e-3):
    """A = TopK({s_j}, K) (Eq. 6) on the fp32 scores.

    Order by (score descending, position ascending), keep the first K, return
    them ascending.  Also returns tau (the K-th largest score) and the two
    index sets of the comparison band: ``must`` = scores above tau*(1+band),
    ``may`` = scores at least tau*(1-band).
    """
    s = np.asarray(scores, dtype=np.float32)
    L = s.shape[0]
    order = sorted(range(L), key=lambda j: (-float(s[j]), j))
    A = np.array(sorted(order[:K]), dtype=np.int32)
    if K == 0:
        return A, float("inf"), np.zeros(0, np.int32), np.zeros(0, np.int32)
    tau = float(s[order[K - 1]])
    s64 = s.astype(F64)
    must = np.nonzero(s64 > tau * (1.0 + band_rel))[0].astype(np.int32)
    may = np.nonzero(s64 >= tau * (1.0 - band_rel))[0].astype(np.int32)
    return A, tau, must, may


# --------------------------------------------------------------------------
# Section 3.3: selective recomputation and the working cache
# --------------------------------------------------------------------------
def recompute_set(anchor_idx: Sequence[int], affix_start: int, extra_rows: Sequence[int]) -> np.ndarray:
    """Absolute positions R: anchors (relative to the affix start) first, then the request rows."""
    a = np.asarray(anchor_idx, dtype=np.int64) + affix_start
    e = np.asarray(extra_rows, dtype=np.int64)
    return np.concatenate([a, e])


def scatter_kv(cache_k: np.ndarray, cache_v: np.ndarray, rows: np.ndarray,
               k_new: np.ndarray, v_new: np.ndarray):
    """Working cache: a copy of the shared cache with rows R overwritten, nothing else (bf16 bits)."""
    ck, cv = cache_k.copy(), cache_v.copy()
    ck[rows] = k_new
    cv[rows] = v_new
    return ck, cv


def dropna_key_keep(ctx_len: int, affix_start: int, affix_len: int, anchor_idx: Sequence[int]) -> np.ndarray:
    """Keys that exist under the DropNA layout (Section 5.3, "Is the Non-Anchor Cache Useful?"): every
    position outside the affix, and of the affix only the anchors; bool [ctx_len]."""
    keep = np.ones(ctx_len, bool)
    keep[affix_start:affix_start + affix_len] = False
    keep[affix_start + np.asarray(anchor_idx, dtype=np.int64)] = True
    return keep


def kv_deviation_scores(k_ref: np.ndarray, v_ref: np.ndarray, k_full: np.ndarray, v_full: np.ndarray) -> np.ndarray:
    """One layer's term of the KV-deviation selector the paper compares against (appendix
    "CacheBlend-Style Anchor Selection"): affix token j is ranked by how far its K/V in the affix-only
    cache lie from its K/V in the full-prompt cache,
        s_j += sum_{h, c} (K_full[j, h, c] - K_ref[j, h, c])^2 + (V_full[j, h, c] - V_ref[j, h, c])^2.
    The paper names the quantity ("KV difference") but not the norm; the squared Euclidean distance
    over K and V together is the reading taken.  Inputs [L, Hkv, d] fp64 (bf16 values); returns fp64 [L].
    The scores of several layers add, and Eq. 6 then picks the K largest."""
    dk = np.asarray(k_full, F64) - np.asarray(k_ref, F64)
    dv = np.asarray(v_full, F64) - np.asarray(v_ref, F64)
    return (dk * dk).sum(axis=(1, 2)) + (dv * dv).sum(axis=(1, 2))


def recompute_rows(weights, shape, x_rows: np.ndarray, rows: np.ndarray,
                   cache_k: np.ndarray, cache_v: np.ndarray, ctx_len: int, cos, sin,
                   round_storage: bool = True, key_keep: Optional[np.ndarray] = None):
    """Recompute the rows R of one request under the current context.

    x_rows  [n, D] fp64  layer input at the rows R (bf16 values)
    rows    [n]          absolute positions of R
    cache_k/cache_v [cap, Hkv, d] bf16 bits: the shared/stale cache of this request
    Returns dict with k_new/v_new (bf16 bits [n, Hkv, d]), the working cache
    (bf16 bits), y [n, D] fp64 (bf16 values), attention row sums [n, H].
    Queries are formed only for R; keys and values are the whole logical
    context [0, ctx_len) with rows R taken from the fresh k/v (Section 4.3).
    ``key_keep`` (bool [ctx_len], optional): positions whose key/value exist; the
    others are removed from every softmax (the DropNA layout of Section 5.3, which
    discards the non-anchor affix entries).
    """
    H, Hkv, d = shape.n_heads, shape.n_kv_heads, shape.head_dim
    group = H // Hkv
    n = x_rows.shape[0]
    xn = normed_rows(weights, shape, x_rows, round_storage)
    q = project_q(weights, shape, xn, rows, cos, sin, round_storage)            # [n, H, d]
    k_new, v_new = project_kv(weights, shape, xn, rows, cos, sin, round_storage)
    kb, vb = f64_to_bf16_bits(k_new), f64_to_bf16_bits(v_new)
    wk_bits, wv_bits = scatter_kv(cache_k, cache_v, rows, kb, vb)
    if round_storage:
        Kc = bf16_bits_to_f64(wk_bits[:ctx_len])
        Vc = bf16_bits_to_f64(wv_bits[:ctx_len])
    else:   # keep the unrounded fresh rows in the logical view
        Kc = bf16_bits_to_f64(cache_k[:ctx_len]); Kc[rows] = k_new
        Vc = bf16_bits_to_f64(cache_v[:ctx_len]); Vc[rows] = v_new
    o = np.zeros((n, H, d), F64)
    rowsum = np.zeros((n, H), F64)
    for h in range(H):
        kh = h // group
        z = q[:, h, :] @ Kc[:, kh, :].T / math.sqrt(d)        # [n, T]
        if key_keep is not None:
            z = np.where(np.asarray(key_keep, bool)[None, :], z, -np.inf)
        p = softmax_rows(z)
        rowsum[:, h] = p.sum(axis=1)
        o[:, h, :] = p @ Vc[:, kh, :]
    o = _store(o.reshape(n, H * d), round_storage)
    h1 = _store(x_rows + o @ _w(weights, "wo").T, round_storage)
    xn2 = _store(rmsnorm(h1, _w(weights, "mlp_norm_g"), shape.rms_eps), round_storage)
    act = _store(silu(xn2 @ _w(weights, "w_gate").T) * (xn2 @ _w(weights, "w_up").T), round_storage)
    y = _store(h1 + act @ _w(weights, "w_down").T, round_storage)
    return dict(k_new=kb, v_new=vb, cache_k=wk_bits, cache_v=wv_bits, y=y, rowsum=rowsum,
                q=q, o=o, h1=h1)


def layer_step(weights, shape, x: np.ndarray, cache_k: np.ndarray, cache_v: np.ndarray,
               ctx_len: int, affix_start: int, affix_len: int, masked_pos: np.ndarray,
               extra_rows: np.ndarray, cos, sin, ratio: Optional[float] = None,
               K: Optional[int] = None, anchor_idx: Optional[np.ndarray] = None,
               scores_in: Optional[np.ndarray] = None, norm_full: bool = False,
               round_storage: bool = True, drop_non_anchor: bool = False):
    """One request, one layer: score -> select -> recompute -> working cache.

    x [T, D] bf16 bits (layer input at every position).  If ``anchor_idx`` is
    given the scoring/selection is skipped (the anchor set is fixed per
    request after selection, Section 3.2).  ``scores_in`` is added to this
    layer's scores (Eq. 5 sums over layers).  ``drop_non_anchor``: the DropNA
    ablation of Section 5.3 (same anchors, the non-anchor affix entries are
    discarded: no query attends them).
    """
    xf = bf16_bits_to_f64(x)
    out = {}
    if anchor_idx is None:
        qm = masked_queries(weights, shape, xf[masked_pos], masked_pos, cos, sin, round_storage)
        Kall = bf16_bits_to_f64(cache_k[:ctx_len])
        s = score_anchors(qm, Kall[affix_start:affix_start + affix_len], Kall, affix_start, norm_full)
        if scores_in is not None:
            s = s + np.asarray(scores_in, F64)
        s32 = s.astype(np.float32)
        if K is None:
            K = k_from_ratio(affix_len, ratio)
        anchor_idx, tau, must, may = select_topk(s32, K)
        out.update(scores=s32, scores64=s, tau=tau, must=must, may=may, q_mask=qm)
    rows = recompute_set(anchor_idx, affix_start, extra_rows)
    keep = dropna_key_keep(ctx_len, affix_start, affix_len, anchor_idx) if drop_non_anchor else None
    r = recompute_rows(weights, shape, xf[rows], rows, cache_k, cache_v, ctx_len, cos, sin, round_storage, keep)
    out.update(r)
    out.update(anchor_idx=np.asarray(anchor_idx, np.int32), rows=rows)
    return out


# --------------------------------------------------------------------------
# A dense bidirectional layer over the whole sequence, written on its own
# (the ratio-1.0 / full-recompute end point, Section 5.2)
# --------------------------------------------------------------------------
def dense_layer(weights, shape, x: np.ndarray, cos, sin, round_storage: bool = True):
    """Full-sequence forward of the layer: every position is a query and a fresh key/value.

    x [T, D] bf16 bits.  Returns (y [T, D] fp64, K bits [T, Hkv, d], V bits [T, Hkv, d]).
    """
    H, Hkv, d = shape.n_heads, shape.n_kv_heads, shape.head_dim
    T = x.shape[0]
    pos = np.arange(T)
    X = bf16_bits_to_f64(x)
    Xn = _store(X * (1.0 / np.sqrt((X ** 2).mean(-1, keepdims=True) + shape.rms_eps))
                * _w(weights, "attn_norm_g"), round_storage)
    Wq, Wk, Wv = _w(weights, "wq"), _w(weights, "wk"), _w(weights, "wv")
    Q = np.einsum("td,od->to", Xn, Wq)
    Kp = np.einsum("td,od->to", Xn, Wk)
    Vp = np.einsum("td,od->to", Xn, Wv)
    if weights.get("bq") is not None:
        Q, Kp, Vp = Q + _w(weights, "bq"), Kp + _w(weights, "bk"), Vp + _w(weights, "bv")
    Q = _store(rope(Q.reshape(T, H, d), pos, cos, sin), round_storage)
    Kp = _store(rope(Kp.reshape(T, Hkv, d), pos, cos, sin), round_storage)
    Vp = _store(Vp.reshape(T, Hkv, d), round_storage)
    Kr = np.repeat(Kp, H // Hkv, axis=1)       # [T, H, d]
    Vr = np.repeat(Vp, H // Hkv, axis=1)
    Z = np.einsum("qhd,khd->hqk", Q, Kr) / math.sqrt(d)
    P = np.exp(Z - Z.max(-1, keepdims=True))
    P /= P.sum(-1, keepdims=True)
    O = _store(np.einsum("hqk,khd->qhd", P, Vr).reshape(T, H * d), round_storage)
    H1 = _store(X + O @ _w(weights, "wo").T, round_storage)
    Xn2 = _store(rmsnorm(H1, _w(weights, "mlp_norm_g"), shape.rms_eps), round_storage)
    G = Xn2 @ _w(weights, "w_gate").T
    U = Xn2 @ _w(weights, "w_up").T
    A = _store(G / (1.0 + np.exp(-G)) * U, round_storage)
    Y = _store(H1 + A @ _w(weights, "w_down").T, round_storage)
    return Y, f64_to_bf16_bits(Kp), f64_to_bf16_bits(Vp)


# --------------------------------------------------------------------------
# N layers: the one-shot probe of Section 3.2 and the refresh pass of Section 3.3
# --------------------------------------------------------------------------
def probe_forward(layers, shape, x0: np.ndarray, caches, ctx_len: int, affix_start: int, affix_len: int,
                  masked_pos: np.ndarray, probe_rows: np.ndarray, cos, sin, norm_full: bool = False,
                  round_storage: bool = True):
    """One-shot probe (Section 3.2): forward only the non-affix rows P through all N layers with the
    precomputed affix cache as fixed past KV; at every layer score the affix keys by the attention
    they receive from the masked rows and sum over layers (Eq. 5).

    layers: list of weight dicts; x0 [T, D] bf16 bits (layer-0 input); caches: list of
    (cache_k, cache_v) bf16 bits per layer; probe_rows: absolute positions P (must contain masked_pos).
    The affix keys are the cached (stale) ones.  With ``norm_full`` the softmax of Eq. 4 runs over every key the
    probe's own attention sees: the affix keys as cached plus the probe rows' fresh keys (Section 3.2: the probe
    attends with the affix as past KV), i.e. the working cache of this layer.
    Returns (scores fp64 [L], list of working caches, list of per-layer outputs y [|P|, D]).
    """
    rows = np.asarray(probe_rows, dtype=np.int64)
    where = {int(p): i for i, p in enumerate(rows)}
    mask_idx = np.array([where[int(p)] for p in masked_pos], dtype=np.int64)
    x_rows = bf16_bits_to_f64(x0)[rows]
    s = np.zeros(affix_len, F64)
    out_caches, ys = [], []
    for W, (ck, cv) in zip(layers, caches):
        r = recompute_rows(W, shape, x_rows, rows, ck, cv, ctx_len, cos, sin, round_storage)
        Kall = bf16_bits_to_f64((r["cache_k"] if norm_full else ck)[:ctx_len])
        s += score_anchors(r["q"][mask_idx], Kall[affix_start:affix_start + affix_len], Kall, affix_start, norm_full)
        x_rows = r["y"]
        out_caches.append((r["cache_k"], r["cache_v"]))
        ys.append(r["y"])
    return s, out_caches, ys


def refresh_forward(layers, shape, x0: np.ndarray, caches, ctx_len: int, affix_start: int,
                    anchor_idx: np.ndarray, extra_rows: np.ndarray, cos, sin, round_storage: bool = True):
    """Refresh pass (Section 3.3): recompute the anchors and the request rows through all N layers;
    layer n+1's input rows are layer n's output rows.  Returns (rows, working caches, per-layer y)."""
    rows = recompute_set(anchor_idx, affix_start, extra_rows)
    x_rows = bf16_bits_to_f64(x0)[rows]
    out_caches, ys = [], []
    for W, (ck, cv) in zip(layers, caches):
        r = recompute_rows(W, shape, x_rows, rows, ck, cv, ctx_len, cos, sin, round_storage)
        x_rows = r["y"]
        out_caches.append((r["cache_k"], r["cache_v"]))
        ys.append(r["y"])
    return rows, out_caches, ys


def dense_forward(layers, shape, x0: np.ndarray, cos, sin, round_storage: bool = True):
    """All positions through all N layers (the full-recompute end point); returns per-layer (y, K, V)."""
    x = x0
    outs = []
    for W in layers:
        y, kb, vb = dense_layer(W, shape, x, cos, sin, round_storage)
        outs.append((y, kb, vb))
        x = f64_to_bf16_bits(y)
    return outs


# --------------------------------------------------------------------------
# Eq. 2-3: predict the masked positions of the current block, commit the confident ones
# --------------------------------------------------------------------------
def predict_commit(h_rows: np.ndarray, final_norm_g: np.ndarray, w_lm: np.ndarray, eps: float, threshold: float,
                   round_storage: bool = True):
    """One request's block: z = W_lm (RMSNorm(h) g); token = argmax_v z (lowest index on ties);
    confidence = softmax(z)[token]; commit = confidence > threshold, or, if no row qualifies, the
    single most confident row (lowest index on ties) -- the threshold rule of the decoding
    schedule the paper builds on (Section 3.1; threshold 0.9 in Section 5).

    h_rows [n, D] fp64 (bf16 values); final_norm_g [D] and w_lm [V, D] bf16 bits or floats.
    Returns (token int32 [n], confidence fp64 [n], commit bool [n], logits fp64 [n, V]).
    """
    g = bf16_bits_to_f64(final_norm_g) if final_norm_g.dtype == np.uint16 else np.asarray(final_norm_g, F64)
    W = bf16_bits_to_f64(w_lm) if w_lm.dtype == np.uint16 else np.asarray(w_lm, F64)
    hn = _store(rmsnorm(h_rows, g, eps), round_storage)
    z = hn @ W.T
    token = np.argmax(z, axis=1).astype(np.int32)
    zmax = z.max(axis=1, keepdims=True)
    conf = 1.0 / np.exp(z - zmax).sum(axis=1)
    commit = conf > threshold
    if z.shape[0] and not commit.any():
        commit[int(np.argmax(conf))] = True
    return token, conf, commit, z


def commit_update(token_ids: np.ndarray, block_pos: np.ndarray, token: np.ndarray, confidence: np.ndarray,
                  mask_id: int, threshold: float) -> int:
    """Eq. 3 on one request's sequence: the block positions that still hold ``mask_id`` and whose
    confidence exceeds the threshold receive their predicted token; if there are masked positions
    but none qualifies, the single most confident masked one does (lowest index on ties).
    Already decoded positions are left alone.  ``token_ids`` [T] is updated in place; returns the
    number of masked positions left in the block."""
    masked = [i for i, p in enumerate(block_pos) if token_ids[p] == mask_id]
    if not masked:
        return 0
    hits = [i for i in masked if confidence[i] > threshold]
    if not hits:
        best = masked[0]
        for i in masked[1:]:
            if confidence[i] > confidence[best]:
                best = i
        hits = [best]
    for i in hits:
        token_ids[block_pos[i]] = token[i]
    return len(masked) - len(hits)


def generate_block(layers, shape, embed: np.ndarray, final_norm_g: np.ndarray, w_lm: np.ndarray,
                   token_ids: np.ndarray, caches, ctx_len: int, affix_start: int, anchor_idx: np.ndarray,
                   request_rows: np.ndarray, block_pos: np.ndarray, cos, sin, mask_id: int, threshold: float,
                   max_steps: int, round_storage: bool = True):
    """One request, one block, refresh-then-decode (Section 4.3 with the threshold schedule of
    Section 5): step 0 recomputes R = A u E (anchors + all request-specific rows) through all layers
    from the token embeddings, later steps only the block's rows over the caches the earlier steps
    left; after every step the block rows are predicted (Eq. 2) and Eq. 3 commits into ``token_ids``.

    embed [V, D] bf16 bits; token_ids [T] int (updated in place); caches: list of (K, V) bf16 bits.
    Returns (steps, working caches, history) where history[s] = (token, confidence, token_ids copy)."""
    history = []
    steps = 0
    for step in range(max_steps):
        if step == 0:
            a_idx, extra = np.asarray(anchor_idx), np.asarray(request_rows)
        else:
            a_idx, extra = np.zeros((0,), np.int64), np.asarray(block_pos)
        x0 = embed[np.asarray(token_ids[:ctx_len], dtype=np.int64)]
        rows, caches, ys = refresh_forward(layers, shape, x0, caches, ctx_len, affix_start, a_idx, extra, cos, sin,
                                           round_storage)
        where = {int(p): i for i, p in enumerate(rows)}
        h = ys[-1][[where[int(p)] for p in block_pos]]
        token, conf, _, _ = predict_commit(h, final_norm_g, w_lm, shape.rms_eps, threshold, round_storage)
        left = commit_update(token_ids, block_pos, token, conf, mask_id, threshold)
        history.append((token.copy(), conf.copy(), np.array(token_ids).copy()))
        steps = step + 1
        if left == 0:
            break
    return steps, caches, history


# --------------------------------------------------------------------------
# comparison helpers used by the parity tests
# --------------------------------------------------------------------------
def rel_err_gate(a: np.ndarray, b: np.ndarray, tol: float = 2e-2) -> Tuple[bool, float]:
    """Agreement of a bf16 tensor ``a`` with the reference ``b`` to max relative error ``tol``.

    Four conditions, all required:
      max |a-b| <= tol * max |b|                      (max error relative to the tensor's scale)
      rms(a-b) <= tol/2 * rms(b)                      (no systematic error)
      |a_i-b_i| <= 2*tol * max(|b_i|, rms(b)) for every element   (no single wrong element)
      |a_i-b_i| <= tol * max(|b_i|, rms(b)) for all but 1e-5 of the elements
    The last two exist because bf16 storage rounding alone (the same tensor with and without the
    roundings of the contract) already moves about one element in a million by 2 % of rms(b);
    an element-wise bound at exactly ``tol`` would sit in the tail of that noise.
    Returns (ok, worst element-wise ratio).
    """
    a = np.asarray(a, F64); b = np.asarray(b, F64)
    if b.size == 0:
        return a.size == 0, 0.0
    d = np.abs(a - b)
    rms = math.sqrt(float(np.mean(b * b)))
    bmax = float(np.max(np.abs(b)))
    denom = np.maximum(np.abs(b), rms)
    denom = np.where(denom == 0.0, 1.0, denom)
    ratio = d / denom
    worst = float(np.max(ratio))
    ok = (float(np.max(d)) <= tol * (bmax if bmax > 0 else 1.0)
          and math.sqrt(float(np.mean(d * d))) <= 0.5 * tol * (rms if rms > 0 else 1.0)
          and worst <= 2.0 * tol
          and float(np.mean(ratio > tol)) <= 1e-5)
    return ok, worst


def anchor_set_ok(gpu_idx: np.ndarray, K: int, L: int, must: np.ndarray, may: np.ndarray) -> Tuple[bool, str]:
    """The band rule: |A| = K, unique, ascending, in range, must <= A <= may."""
    g = np.asarray(gpu_idx).astype(np.int64)
    if g.shape != (K,):
        return False, f"shape {g.shape} != ({K},)"
    if K == 0:
        return True, ""
    if g.min() < 0 or g.max() >= L:
        return False, "index out of range"
    if np.any(np.diff(g) <= 0):
        return False, "not strictly ascending"
    gs = set(g.tolist())
    if not set(must.tolist()) <= gs:
        return False, f"missing {sorted(set(must.tolist()) - gs)[:8]}"
    if not gs <= set(may.tolist()):
        return False, f"outside band {sorted(gs - set(may.tolist()))[:8]}"
    return True, ""
