"""GPU parity at the shapes of the benchmark configurations 3, 4 and 5 (one layer, a slice of
the batch where the full batch would take the CPU oracle too long): LLaDA-8B layer with a
2048-token affix and all request rows recomputed, Dream-7B layer shapes (grouped-query
attention, QKV bias) with the affix in the middle, and sweep points over affix length,
placement and ratio."""
import numpy as np
import pytest
import torch

from oracle import acache_oracle as orc
from paper_2608_26140_b200 import binding as ab
from paper_2608_26140_b200 import workloads as wl

from helpers import DeviceCase, assert_close_bf16, cached_weights, oracle_step
from test_gpu_parity import run_layer_step

pytestmark = pytest.mark.gpu


def check_step(case, ratio, requests, norm_full=False):
    dc = DeviceCase(case)
    lay = case.layout
    flags = ab.F_SCORE | ab.F_SELECT | (ab.F_SCORE_NORM_FULL if norm_full else 0)
    K, s_gpu, a_gpu, y = run_layer_step(dc, ratio, flags)
    n = K + lay.n_extra
    ckb, cvb = ab.to_host_bits(dc.ck), ab.to_host_bits(dc.cv)
    worst = 0.0
    for b in requests:
        free = oracle_step(case, b, ratio=ratio, norm_full=norm_full)
        err = np.abs(s_gpu[b] - free["scores64"]) / np.maximum(free["scores64"], free["scores64"].mean())
        assert err.max() < 1e-3, err.max()
        ok, why = orc.anchor_set_ok(a_gpu[b, :K], K, lay.affix_len, free["must"], free["may"])
        assert ok, why
        ref = free if np.array_equal(free["anchor_idx"], a_gpu[b, :K]) else oracle_step(case, b, anchor_idx=a_gpu[b, :K])
        rows = ref["rows"]
        keep = np.setdiff1d(np.arange(lay.ctx_len), rows)
        assert np.array_equal(ckb[b][keep], case.cache_k[b][keep]) and np.array_equal(cvb[b][keep], case.cache_v[b][keep])
        if n:
            worst = max(worst, assert_close_bf16(ckb[b][rows], ref["k_new"], "K rows"))
            worst = max(worst, assert_close_bf16(cvb[b][rows], ref["v_new"], "V rows"))
            worst = max(worst, assert_close_bf16(ab.to_host_bits(y[b, :n]), ref["y"], "y"))
    assert dc.ctx.poll_status() == 0
    return worst


def test_config3_layer_slice():
    """LLaDA-8B layer, 2048-token prefix affix + 256 request + 256 generation rows, all request rows
    recomputed with the 410 anchors (922 rows per request); 2 of the 16 requests."""
    lay = wl.config_layout(3, "all", n_masked=256, batch=2)
    case = wl.make_case(wl.LLADA_8B, lay, 0.2, cfg_id=5, weights=cached_weights(wl.LLADA_8B, 5))
    check_step(case, 0.2, requests=[0, 1])


def test_config4_dream_layer_slice():
    """Dream-7B layer shapes (28 query / 4 KV heads, bias), affix in the middle; 2 of the 32 requests,
    the second one checked in full, masked rows = the whole 256-token generation."""
    lay = wl.config_layout(4, "all", n_masked=256, batch=2)
    case = wl.make_case(wl.DREAM_7B, lay, 0.2, cfg_id=4)
    check_step(case, 0.2, requests=[1])


@pytest.mark.parametrize("L,place,ratio,batch", [
    (512, "middle", 0.05, 2),
    (512, "suffix", 0.5, 1),
    (2048, "prefix", 0.35, 1),
    (2048, "suffix", 0.1, 2),
    (8192, "middle", 0.05, 1),
])
def test_config5_sweep_points(L, place, ratio, batch):
    lay = wl.sweep_layout(L, batch, place, "none")
    case = wl.make_case(wl.LLADA_8B, lay, ratio, cfg_id=5, weights=cached_weights(wl.LLADA_8B, 5))
    check_step(case, ratio, requests=[batch - 1])


def test_config5_full_context_normaliser_and_hot_keys():
    lay = wl.sweep_layout(2048, 1, "middle", "masked")
    case = wl.make_case(wl.LLADA_8B, lay, 0.2, cfg_id=5, hot_frac=0.05, weights=cached_weights(wl.LLADA_8B, 5))
    check_step(case, 0.2, requests=[0], norm_full=True)
