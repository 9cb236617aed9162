"""GPU parity at the batch sizes the benchmark times: the sweep's 64-request points (where the cache and
x pass 2^31 elements and the kernel selection changes: batched scoring, grouped attention, one
selection CTA per request), benchmark configuration 3 at 16 requests and configuration 4 at 32, one
layer each.  The inputs are drawn on the device (the host generator would take minutes for 4 GB
tensors); the requests that are checked (the first and the last of the batch) are copied to the host
and go through the CPU oracle exactly as in the small cases."""
import numpy as np
import pytest
import torch

from oracle import acache_oracle as orc
from paper_2608_26140_b200 import binding as ab
from paper_2608_26140_b200 import workloads as wl

from helpers import DEV, assert_close_bf16, cached_weights

pytestmark = pytest.mark.gpu


def draw_on_device(shape, lay, seed):
    """x [B, T, D] ~ N(0, 1) and K/V caches ~ N(0, 0.02 sqrt(D)), bf16, one request at a time; the affix rows of
    all three are request 0's (the affix is shared by the batch)."""
    B, T, l, L = lay.batch, lay.ctx_len, lay.affix_start, lay.affix_len
    gen = torch.Generator(device=DEV)
    gen.manual_seed(seed)
    std = 0.02 * float(np.sqrt(shape.hidden))
    x = torch.empty((B, T, shape.hidden), dtype=torch.bfloat16, device=DEV)
    ck = torch.empty((B, T, shape.n_kv_heads, shape.head_dim), dtype=torch.bfloat16, device=DEV)
    cv = torch.empty_like(ck)
    for b in range(B):
        x[b] = torch.randn((T, shape.hidden), generator=gen, device=DEV, dtype=torch.float32).to(torch.bfloat16)
        ck[b] = (torch.randn(ck.shape[1:], generator=gen, device=DEV, dtype=torch.float32) * std).to(torch.bfloat16)
        cv[b] = (torch.randn(cv.shape[1:], generator=gen, device=DEV, dtype=torch.float32) * std).to(torch.bfloat16)
    for t in (x, ck, cv):
        t[1:, l:l + L] = t[0:1, l:l + L]
    return x, ck, cv


def check_large_batch(shape, weights, lay, ratio, seed, norm_full=False):
    B, T, l, L = lay.batch, lay.ctx_len, lay.affix_start, lay.affix_len
    checked = sorted({0, B - 1})
    x, ck, cv = draw_on_device(shape, lay, seed)
    # host copies of the checked requests as they are BEFORE the step
    hx = {b: ab.to_host_bits(x[b]) for b in checked}
    hk = {b: ab.to_host_bits(ck[b]) for b in checked}
    hv = {b: ab.to_host_bits(cv[b]) for b in checked}
    w_dev = {k: (ab.to_device_bf16(v, DEV) if v is not None else None) for k, v in weights.items()}
    cos_h, sin_h = wl.rope_table(T, shape.head_dim, shape.rope_theta)
    cos, sin = torch.from_numpy(cos_h).to(DEV), torch.from_numpy(sin_h).to(DEV)
    masked = torch.from_numpy(lay.masked_pos.copy()).to(DEV)
    extra = torch.from_numpy(lay.extra_rows.copy()).to(DEV) if lay.n_extra else None
    req = ab.Context.request(B, T, l, L, masked, extra, cos, sin)
    K = orc.k_from_ratio(L, ratio)
    n = K + lay.n_extra
    ctx = ab.Context.for_shape(shape, B, T, L, max(n, 1), lay.n_masked, DEV)
    scores = torch.zeros((B, L), dtype=torch.float32, device=DEV)
    anchors = torch.full((B, max(K, 1)), -1, dtype=torch.int32, device=DEV)
    y = torch.zeros((B, max(n, 1), shape.hidden), dtype=torch.bfloat16, device=DEV)
    flags = ab.F_SCORE | ab.F_SELECT | (ab.F_SCORE_NORM_FULL if norm_full else 0)
    ctx.layer_step(ab.Context.weights(w_dev), req, ab.Context.kv(ck, cv), x, 0, ratio, flags, scores, anchors, y)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    s_gpu, a_gpu = scores.cpu().numpy(), anchors.cpu().numpy()
    w64 = {k: (orc.bf16_bits_to_f64(v) if v is not None else None) for k, v in weights.items()}
    for b in checked:
        args = (w64, shape, hx[b], hk[b], hv[b], T, l, L, lay.masked_pos[b], lay.extra_rows[b], cos_h, sin_h)
        free = orc.layer_step(*args, ratio=ratio, norm_full=norm_full)
        err = np.abs(s_gpu[b] - free["scores64"]) / np.maximum(free["scores64"], free["scores64"].mean())
        assert err.max() < 1e-3, (b, err.max())
        ok, why = orc.anchor_set_ok(a_gpu[b, :K], K, L, free["must"], free["may"])
        assert ok, (b, why)
        ref = free if np.array_equal(free["anchor_idx"], a_gpu[b, :K]) else orc.layer_step(*args, anchor_idx=a_gpu[b, :K])
        rows = ref["rows"]
        keep = np.setdiff1d(np.arange(T), rows)
        ckb, cvb = ab.to_host_bits(ck[b]), ab.to_host_bits(cv[b])
        assert np.array_equal(ckb[keep], hk[b][keep]) and np.array_equal(cvb[keep], hv[b][keep]), "untouched rows changed"
        assert_close_bf16(ckb[rows], ref["k_new"], f"request {b} K rows")
        assert_close_bf16(cvb[rows], ref["v_new"], f"request {b} V rows")
        assert_close_bf16(ab.to_host_bits(y[b, :n]), ref["y"], f"request {b} y")
    # the requests in between: every one selected K distinct anchors in range, ascending
    assert (a_gpu[:, :K] >= 0).all() and (a_gpu[:, :K] < L).all() and (np.diff(a_gpu[:, :K], axis=1) > 0).all()


@pytest.mark.parametrize("L,place,ratio", [(8192, "prefix", 0.05), (512, "middle", 0.2)])
def test_sweep_points_at_64_requests(L, place, ratio):
    """Configuration-5 sweep points at batch 64: at L = 8192 x and each cache hold 2.17 G elements."""
    lay = wl.sweep_layout(L, 64, place, "none")
    check_large_batch(wl.LLADA_8B, cached_weights(wl.LLADA_8B, 5), lay, ratio, seed=0x5EED0 + L)


def test_config3_layer_at_16_requests():
    """Configuration 3, one layer at its full batch: 16 x (410 anchors + 512 request rows) = 14 752 rows."""
    lay = wl.config_layout(3, "all", n_masked=256, batch=16)
    check_large_batch(wl.LLADA_8B, cached_weights(wl.LLADA_8B, 5), lay, 0.2, seed=0x5EED3)


def test_config4_layer_at_32_requests():
    """Configuration 4, one Dream-7B-shaped layer at its full batch: 32 x (205 anchors + 640 request rows)."""
    lay = wl.config_layout(4, "all", n_masked=256, batch=32)
    check_large_batch(wl.DREAM_7B, wl.layer_weights(wl.DREAM_7B, 4, 0), lay, 0.2, seed=0x5EED4)
