"""The selector and layout variants the paper ablates, against the oracle: the KV-deviation
(CacheBlend-style) anchor selector of the appendix, which feeds the same Eq. 6 selection, and the
DropNA layout of Section 5.3 (same anchors, the non-anchor affix entries do not exist as keys)."""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

from oracle import acache_oracle as orc
from paper_2608_26140_b200 import binding as ab
from paper_2608_26140_b200 import workloads as wl

from helpers import DEV, DeviceCase, assert_close_bf16, make_projected_case, oracle_step
from test_gpu_parity import MID128, dev_i32

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("shape,B,pre,L,post,n_layers,shared_ref", [
    (wl.TINY_GQA, 2, 5, 300, 33, 2, False),
    (MID128, 3, 0, 520, 40, 3, True),          # the affix-only cache is one copy for the batch
    (wl.LLADA_8B, 2, 16, 700, 48, 1, False),
])
def test_kv_deviation_scores_and_selection(shape, B, pre, L, post, n_layers, shared_ref):
    lay = wl.make_layout(B, pre, L, post, 32, 32)
    T, l = lay.ctx_len, lay.affix_start
    ctx = ab.Context.for_shape(shape, B, T, L, 1, 32, DEV)
    req = ab.Context.request(B, T, l, L, dev_i32(lay.masked_pos), None, None, None)
    scores = torch.full((B, L), 9.0, dtype=torch.float32, device=DEV)
    ref = np.zeros((B, L))
    for n in range(n_layers):
        rk, rv = wl.random_kv_cache(shape, lay, 8100 + 10 * n)
        fk, fv = wl.random_kv_cache(shape, lay, 8105 + 10 * n)
        # the full-prompt cache is the affix-only one moved a little, a few tokens moved a lot
        g = np.random.default_rng(n)
        hot = g.choice(L, 7, replace=False)
        mix = lambda a, b_: wl.f32_to_bf16_bits(wl.bf16_bits_to_f32(a) + 0.1 * wl.bf16_bits_to_f32(b_))   # noqa: E731
        fk2, fv2 = mix(rk, fk), mix(rv, fv)
        fk2[:, l + hot] = fk[:, l + hot]
        drk, drv, dfk, dfv = (ab.to_device_bf16(a, DEV) for a in (rk, rv, fk2, fv2))
        kv_ref = ab.KV(drk.data_ptr(), drv.data_ptr(), 0, T) if shared_ref else ab.Context.kv(drk, drv)
        ctx.score_kv_deviation(req, kv_ref, ab.Context.kv(dfk, dfv), scores, accumulate=n > 0)
        for b in range(B):
            rb = 0 if shared_ref else b
            ref[b] += orc.kv_deviation_scores(*(orc.bf16_bits_to_f64(a)[l:l + L] for a in (rk[rb], rv[rb], fk2[b], fv2[b])))
    torch.cuda.synchronize()
    s_gpu = scores.cpu().numpy()
    assert np.abs(s_gpu - ref).max() <= 1e-5 * ref.max()
    K = orc.k_from_ratio(L, 0.2)
    anchors = torch.zeros((B, K), dtype=torch.int32, device=DEV)
    ctx.select_topk(scores, B, L, K, anchors)
    torch.cuda.synchronize()
    for b in range(B):
        _, _, must, may = orc.select_topk(ref[b].astype(np.float32), K)
        ok, why = orc.anchor_set_ok(anchors.cpu().numpy()[b], K, L, must, may)
        assert ok, why
    assert ctx.poll_status() == 0


def run_dropna(dc, ratio, shared_storage, anchors_in=None):
    s, lay = dc.case.shape, dc.case.layout
    B, L = lay.batch, lay.affix_len
    K = orc.k_from_ratio(L, ratio)
    n = K + lay.n_extra
    scores = torch.zeros((B, L), dtype=torch.float32, device=DEV)
    anchors = torch.full((B, max(K, 1)), -1, dtype=torch.int32, device=DEV)
    y = torch.zeros((B, max(n, 1), s.hidden), dtype=torch.bfloat16, device=DEV)
    flags = ab.F_DROP_NON_ANCHOR
    if anchors_in is None:
        flags |= ab.F_SCORE | ab.F_SELECT
    else:
        anchors[:, :K] = dev_i32(anchors_in)
    k_new = v_new = None
    if shared_storage:
        k_new = torch.zeros((B, max(n, 1), s.n_kv_heads, s.head_dim), dtype=torch.bfloat16, device=DEV)
        v_new = torch.zeros_like(k_new)
        dc.ctx.layer_step_shared(dc.lw, dc.req, dc.kv(), dc.x, 0, ratio, flags, scores, anchors, k_new, v_new, y)
    else:
        dc.ctx.layer_step(dc.lw, dc.req, dc.kv(), dc.x, 0, ratio, flags, scores, anchors, y)
    torch.cuda.synchronize()
    return K, anchors.cpu().numpy(), y, k_new, v_new


CASES = [
    (wl.TINY, 2, 0, 200, 24, 32, 32, "all", 0.2),          # prefix affix: whole key tiles are dropped; head dim 64
    (wl.TINY_GQA, 2, 9, 100, 20, 40, 32, "masked", 0.35),
    (MID128, 2, 0, 400, 8, 32, 32, "none", 0.2),           # head dim 128: the tcgen05 kernels, anchors only
    (MID128, 2, 8, 260, 30, 34, 32, "all", 0.1),
    (MID128, 1, 4, 900, 30, 34, 32, "all", 0.5),           # more than 256 rows: two query tiles where forced
]


@pytest.mark.parametrize("shared_storage", [False, True])
@pytest.mark.parametrize("shape,B,pre,L,post,gen,m,extra,ratio", CASES)
def test_dropna_layer_step(shape, B, pre, L, post, gen, m, extra, ratio, shared_storage):
    lay = wl.make_layout(B, pre, L, post, gen, m, extra)
    case = make_projected_case(shape, lay, ratio, cfg_id=15)
    dc = DeviceCase(case)
    K, a_gpu, y, k_new, v_new = run_dropna(dc, ratio, shared_storage)
    n = K + lay.n_extra
    ckb, cvb = ab.to_host_bits(dc.ck), ab.to_host_bits(dc.cv)
    for b in range(B):
        free = oracle_step(case, b, ratio=ratio)                                 # selection is the KeepNA one
        ok, why = orc.anchor_set_ok(a_gpu[b, :K], K, L, free["must"], free["may"])
        assert ok, why
        ref = oracle_step(case, b, anchor_idx=a_gpu[b, :K], drop_non_anchor=True)
        keepna = oracle_step(case, b, anchor_idx=a_gpu[b, :K])
        rows = ref["rows"]
        if shared_storage:                                                      # nothing written, fresh K/V in the slots
            assert np.array_equal(ckb[b], case.cache_k[b]) and np.array_equal(cvb[b], case.cache_v[b])
            assert_close_bf16(ab.to_host_bits(k_new[b, :n]), ref["k_new"], "k_new")
            assert_close_bf16(ab.to_host_bits(v_new[b, :n]), ref["v_new"], "v_new")
        else:
            keep = np.setdiff1d(np.arange(lay.ctx_len), rows)
            assert np.array_equal(ckb[b][keep], case.cache_k[b][keep]) and np.array_equal(cvb[b][keep], case.cache_v[b][keep])
            assert_close_bf16(ckb[b][rows], ref["k_new"], "K rows")
            assert_close_bf16(cvb[b][rows], ref["v_new"], "V rows")
        assert_close_bf16(ab.to_host_bits(y[b, :n]), ref["y"], "y under DropNA")
        # the layouts really differ at this ratio: the DropNA output is far from the KeepNA one
        good, _ = orc.rel_err_gate(orc.bf16_bits_to_f64(ab.to_host_bits(y[b, :n])), keepna["y"], 2e-2)
        assert not good
    assert dc.ctx.poll_status() == 0


def test_dropna_equals_keepna_at_ratio_one():
    """Section 5.3: at ratio 1.0 no non-anchor token remains and both layouts are the full affix recomputation."""
    lay = wl.make_layout(2, 6, 150, 20, 32, 32, "all")
    case = make_projected_case(MID128, lay, 1.0, cfg_id=16)
    dc = DeviceCase(case)
    K, a1, y_drop, _, _ = run_dropna(dc, 1.0, False)
    ck_drop = ab.to_host_bits(dc.ck)
    dc.reset_cache()
    scores = torch.zeros((2, 150), dtype=torch.float32, device=DEV)
    anchors = torch.zeros((2, K), dtype=torch.int32, device=DEV)
    y_keep = torch.zeros_like(y_drop)
    dc.ctx.layer_step(dc.lw, dc.req, dc.kv(), dc.x, 0, 1.0, ab.F_SCORE | ab.F_SELECT, scores, anchors, y_keep)
    torch.cuda.synchronize()
    assert np.array_equal(ab.to_host_bits(y_keep), ab.to_host_bits(y_drop)) and np.array_equal(ab.to_host_bits(dc.ck), ck_drop)


@pytest.mark.parametrize("switch", ["ACACHE_ATTN_TC2Q=2", "ACACHE_ATTN_TC=0"])
def test_dropna_with_one_attention_kernel_forced(switch):
    """The two-query-tile tcgen05 kernel and the mma.sync kernel at head dim 128 are chosen by size or switch; the
    DropNA cases above run once more in a child process with each forced."""
    name, value = switch.split("=")
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider", "tests/test_gpu_selectors.py",
           "-k", "test_dropna_layer_step or ratio_one"]
    r = subprocess.run(cmd, cwd=ROOT, env={**os.environ, name: value}, capture_output=True, text=True, timeout=1200)
    assert r.returncode == 0, (r.stdout[-3000:], r.stderr[-1000:])
    assert " passed" in r.stdout and "no tests ran" not in r.stdout
