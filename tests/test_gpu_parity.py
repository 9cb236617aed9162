"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs.  Integer work (anchor indices, untouched cache rows) is compared exactly,
up to the 1e-3 relative band around the K-th score; bf16 tensors within 2e-2."""
import numpy as np
import pytest
import torch

from oracle import acache_oracle as orc
from paper_2608_26140_b200 import binding as ab
from paper_2608_26140_b200 import workloads as wl

from helpers import DEV, TOL, DeviceCase, assert_close_bf16, make_projected_case, oracle_step

pytestmark = pytest.mark.gpu

MID128 = wl.LayerShape(512, 4, 2, 128, 1024, 1e-5, True, 5e5, "mid-d128")


def dev_i32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(DEV)


# ------------------------------------------------------------------ Eq. 4-5
@pytest.mark.parametrize("shape,B,pre,L,post,m,norm_full", [
    (wl.TINY, 1, 0, 128, 64, 32, False),
    (wl.TINY, 2, 5, 300, 33, 70, False),       # ragged L and m, affix in the middle
    (wl.TINY_GQA, 2, 0, 257, 10, 1, True),
    (MID128, 2, 16, 520, 40, 32, False),
    (MID128, 1, 0, 1, 64, 3, False),           # one affix token
    (MID128, 1, 7, 700, 64, 130, True),
    (wl.LLADA_8B, 1, 0, 512, 256, 32, False),
    # short affixes scored by the one-launch cluster kernel: one or two key tiles per CTA, one to four row groups
    (wl.TINY, 1, 4, 450, 20, 50, False),
    (MID128, 2, 3, 1000, 20, 64, False),
    (MID128, 1, 0, 1024, 8, 17, False),
    (MID128, 2, 0, 65, 8, 64, False),
    # from 2048 keys (batch x range) on tcgen05: up to 64 masked rows in one pass with the logits kept in tensor memory
    # (ragged key ranges, CTAs of the cluster without keys, 32 and 64 columns, both normalisers), more rows in two passes
    (MID128, 2, 5, 3000, 33, 32, False),
    (MID128, 1, 0, 2500, 40, 64, True),
    (MID128, 3, 16, 700, 20, 33, False),
    (MID128, 1, 7, 2100, 64, 130, True),
])
def test_score_anchors(shape, B, pre, L, post, m, norm_full):
    lay = wl.make_layout(B, pre, L, post, max(m, 1), m)
    T = lay.ctx_len
    ck, _ = wl.random_kv_cache(shape, lay, 77)
    q = wl.random_q_mask(shape, lay, 78)
    ctx = ab.Context.for_shape(shape, B, T, L, 1, max(m, 1), DEV)
    dk = ab.to_device_bf16(ck, DEV)
    dq = ab.to_device_bf16(q, DEV)
    masked = dev_i32(lay.masked_pos)
    req = ab.Context.request(B, T, lay.affix_start, L, masked, None, None, None)
    scores = torch.full((B, L), 3.0, dtype=torch.float32, device=DEV)
    ctx.score_anchors(req, dq, ab.Context.kv(dk, dk), scores, accumulate=False, norm_full=norm_full)
    ctx.score_anchors(req, dq, ab.Context.kv(dk, dk), scores, accumulate=True, norm_full=norm_full)
    torch.cuda.synchronize()
    s_gpu = scores.cpu().numpy().astype(np.float64)
    for b in range(B):
        kf = orc.bf16_bits_to_f64(ck[b, :T])
        ref = 2.0 * orc.score_anchors(orc.bf16_bits_to_f64(q[b]), kf[lay.affix_start:lay.affix_start + L], kf,
                                      lay.affix_start, norm_full)
        err = np.abs(s_gpu[b] - ref) / np.maximum(ref, ref.mean())
        assert err.max() < 1e-3, (b, err.max())
        if not norm_full:
            assert abs(s_gpu[b].sum() - 2.0 * shape.n_heads * m) < 1e-3 * shape.n_heads * m
    assert ctx.poll_status() == 0


@pytest.mark.parametrize("L,m,norm_full", [(2300, 32, False),     # the one-pass tcgen05 kernel (ragged last tile)
                                           (2300, 64, True),      # 64 columns per tile, all keys in the denominator
                                           (2300, 130, False)])   # more than 64 masked rows: the two tcgen05 passes
def test_score_anchors_over_a_cache_shared_by_the_batch(L, m, norm_full):
    """batch_stride = 0 (Section 4.1: one copy of the affix K/V for every request) on the long-affix scoring kernels: every
    request reads the same keys with its own masked rows."""
    shape, B = MID128, 3
    lay = wl.make_layout(B, 4, L, 30, max(m, 1), m)
    T = lay.ctx_len
    ck, _ = wl.random_kv_cache(shape, lay, 91)
    q = wl.random_q_mask(shape, lay, 92)
    ctx = ab.Context.for_shape(shape, B, T, L, 1, m, DEV)
    dk = ab.to_device_bf16(ck[:1], DEV)                                   # one [T, Hkv, d] copy
    dq = ab.to_device_bf16(q, DEV)
    req = ab.Context.request(B, T, lay.affix_start, L, dev_i32(lay.masked_pos), None, None, None)
    scores = torch.full((B, L), -1.0, dtype=torch.float32, device=DEV)
    ctx.score_anchors(req, dq, ab.KV(dk.data_ptr(), dk.data_ptr(), 0, T), scores, accumulate=False, norm_full=norm_full)
    torch.cuda.synchronize()
    s_gpu = scores.cpu().numpy().astype(np.float64)
    kf = orc.bf16_bits_to_f64(ck[0, :T])
    for b in range(B):
        ref = orc.score_anchors(orc.bf16_bits_to_f64(q[b]), kf[lay.affix_start:lay.affix_start + L], kf, lay.affix_start, norm_full)
        err = np.abs(s_gpu[b] - ref) / np.maximum(ref, ref.mean())
        assert err.max() < 1e-3, (b, err.max())
    assert ctx.poll_status() == 0


def test_score_is_bitwise_reproducible():
    shape, B, L, m = MID128, 2, 1000, 64
    lay = wl.make_layout(B, 0, L, 8, m, m)
    ck, _ = wl.random_kv_cache(shape, lay, 5)
    q = wl.random_q_mask(shape, lay, 6)
    ctx = ab.Context.for_shape(shape, B, lay.ctx_len, L, 1, m, DEV)
    dk, dq = ab.to_device_bf16(ck, DEV), ab.to_device_bf16(q, DEV)
    req = ab.Context.request(B, lay.ctx_len, 0, L, dev_i32(lay.masked_pos), None, None, None)
    outs = []
    for _ in range(3):
        s = torch.empty((B, L), dtype=torch.float32, device=DEV)
        ctx.score_anchors(req, dq, ab.Context.kv(dk, dk), s)
        outs.append(s.cpu().numpy())
    assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[0], outs[2])


# ------------------------------------------------------------------ Eq. 6
@pytest.mark.parametrize("B,L", [(1, 1), (3, 7), (2, 1000), (2, 1024), (1, 8192), (2, 16384), (1, 20000)])
def test_select_topk_exact(B, L):
    g = np.random.default_rng(L)
    ctx = ab.Context.for_shape(wl.TINY, B, 256, 128, 1, 1, DEV)
    for trial, K in enumerate(sorted({0, 1, L // 5, L // 2, L - 1, L})):
        if K < 0:
            continue
        s = g.random((B, L)).astype(np.float32)
        if trial % 2 == 0 and L > 4:           # heavy ties around the threshold
            s = np.round(s * 8) / 8
        s[:, L // 2] = -0.0
        ds = torch.from_numpy(s).to(DEV)
        out = torch.full((B, max(K, 1)), -7, dtype=torch.int32, device=DEV)
        ctx.select_topk(ds, B, L, K, out)
        torch.cuda.synchronize()
        got = out.cpu().numpy()
        for b in range(B):
            ref = orc.select_topk(s[b], K)[0]
            assert np.array_equal(got[b, :K], ref), (B, L, K, b)
    # all-equal scores: lowest positions win
    ds = torch.full((B, L), 0.25, device=DEV)
    K = max(1, L // 3)
    out = torch.empty((B, K), dtype=torch.int32, device=DEV)
    ctx.select_topk(ds, B, L, K, out)
    assert np.array_equal(out.cpu().numpy(), np.broadcast_to(np.arange(K, dtype=np.int32), (B, K)))


# ------------------------------------------------------------------ selective recompute + scatter
def run_split_calls(dc: DeviceCase, anchor_idx_dev, K):
    s, lay = dc.case.shape, dc.case.layout
    n = K + lay.n_extra
    B = lay.batch
    k_new = torch.zeros((B, max(n, 1), s.n_kv_heads, s.head_dim), dtype=torch.bfloat16, device=DEV)
    v_new = torch.zeros_like(k_new)
    y = torch.zeros((B, max(n, 1), s.hidden), dtype=torch.bfloat16, device=DEV)
    dc.ctx.recompute_anchors(dc.lw, dc.req, dc.kv(), dc.x, 0, anchor_idx_dev, K, k_new, v_new, y)
    return k_new, v_new, y


def check_against_oracle(dc, anchors, k_new, v_new, y, cache_k_bits, cache_v_bits, K):
    """Teacher-forced comparison: the oracle recomputes with the GPU's anchor set."""
    case, lay = dc.case, dc.case.layout
    n = K + lay.n_extra
    worst = 0.0
    for b in range(lay.batch):
        ref = oracle_step(case, b, anchor_idx=anchors[b, :K])
        worst = max(worst, assert_close_bf16(ab.to_host_bits(k_new[b, :n]), ref["k_new"], "k_new"))
        worst = max(worst, assert_close_bf16(ab.to_host_bits(v_new[b, :n]), ref["v_new"], "v_new"))
        worst = max(worst, assert_close_bf16(ab.to_host_bits(y[b, :n]), ref["y"], "y"))
        if cache_k_bits is not None:
            rows = ref["rows"]
            keep = np.setdiff1d(np.arange(case.cache_k.shape[1]), rows)
            assert np.array_equal(cache_k_bits[b][keep], case.cache_k[b][keep]), "untouched K rows changed"
            assert np.array_equal(cache_v_bits[b][keep], case.cache_v[b][keep]), "untouched V rows changed"
            assert_close_bf16(cache_k_bits[b][rows], ref["k_new"], "cache K rows")
            assert_close_bf16(cache_v_bits[b][rows], ref["v_new"], "cache V rows")
    return worst


@pytest.mark.parametrize("shape,B,pre,L,post,gen,m,extra,ratio", [
    (wl.TINY, 1, 0, 128, 64, 32, 32, "none", 0.2),
    (wl.TINY, 2, 9, 100, 20, 40, 32, "all", 0.2),       # affix in the middle, ragged tiles
    (wl.TINY_GQA, 2, 0, 130, 31, 33, 33, "masked", 0.35),
    (MID128, 2, 4, 200, 30, 32, 32, "all", 0.1),
    (MID128, 1, 0, 64, 16, 16, 16, "none", 1.0),
    # row counts at the edges of the attention kernels' 128-row query tiles (128, 129, 256, 257, 384 rows)
    (MID128, 2, 0, 400, 8, 32, 32, "none", 0.32),
    (MID128, 2, 0, 400, 8, 32, 32, "none", 0.3225),
    (MID128, 2, 0, 400, 8, 32, 32, "none", 0.64),
    (MID128, 2, 0, 400, 8, 32, 32, "none", 0.6425),
    (MID128, 2, 0, 400, 8, 32, 32, "none", 0.96),
])
def test_recompute_then_scatter(shape, B, pre, L, post, gen, m, extra, ratio):
    lay = wl.make_layout(B, pre, L, post, gen, m, extra)
    case = make_projected_case(shape, lay, ratio, cfg_id=11)
    dc = DeviceCase(case)
    K = orc.k_from_ratio(L, ratio)
    # any valid anchor set will do for the split calls: take a seeded random one
    g = np.random.default_rng(3)
    anchors = np.stack([np.sort(g.choice(L, K, replace=False)) for _ in range(B)]).astype(np.int32)
    da = dev_i32(anchors)
    k_new, v_new, y = run_split_calls(dc, da, K)
    torch.cuda.synchronize()
    # recompute must not have touched the cache
    assert np.array_equal(ab.to_host_bits(dc.ck), case.cache_k) and np.array_equal(ab.to_host_bits(dc.cv), case.cache_v)
    dc.ctx.scatter_kv(dc.req, dc.kv(), da, K, k_new, v_new)
    torch.cuda.synchronize()
    ckb, cvb = ab.to_host_bits(dc.ck), ab.to_host_bits(dc.cv)
    check_against_oracle(dc, anchors, k_new, v_new, y, ckb, cvb, K)
    # the scattered rows are bit-identical to k_new / v_new
    n = K + lay.n_extra
    for b in range(B):
        rows = orc.recompute_set(anchors[b], lay.affix_start, lay.extra_rows[b])
        assert np.array_equal(ckb[b][rows], ab.to_host_bits(k_new[b, :n]))
        assert np.array_equal(cvb[b][rows], ab.to_host_bits(v_new[b, :n]))
    assert dc.ctx.poll_status() == 0


# ------------------------------------------------------------------ the chained layer-step
def run_layer_step(dc: DeviceCase, ratio, flags, anchors_in=None):
    s, lay = dc.case.shape, dc.case.layout
    B, L = lay.batch, lay.affix_len
    K = orc.k_from_ratio(L, ratio)
    n = K + lay.n_extra
    scores = torch.zeros((B, L), dtype=torch.float32, device=DEV)
    anchors = torch.full((B, max(K, 1)), -1, dtype=torch.int32, device=DEV)
    if anchors_in is not None:
        anchors[:, :K] = dev_i32(anchors_in)
    y = torch.zeros((B, max(n, 1), s.hidden), dtype=torch.bfloat16, device=DEV)
    dc.ctx.layer_step(dc.lw, dc.req, dc.kv(), dc.x, 0, ratio, flags, scores, anchors, y)
    torch.cuda.synchronize()
    return K, scores.cpu().numpy(), anchors.cpu().numpy(), y


@pytest.mark.parametrize("shape,B,pre,L,post,gen,m,extra", [
    (wl.TINY, 1, 0, 128, 64, 32, 32, "none"),          # benchmark config 1 (tail rows folded into gen)
    (wl.TINY, 2, 16, 128, 48, 64, 32, "all"),
    (wl.TINY_GQA, 2, 0, 200, 24, 32, 32, "all"),
    (MID128, 2, 8, 260, 30, 34, 32, "masked"),
])
@pytest.mark.parametrize("ratio", [0.0, 0.2, 1.0])
def test_layer_step(shape, B, pre, L, post, gen, m, extra, ratio):
    lay = wl.make_layout(B, pre, L, post, gen, m, extra)
    case = make_projected_case(shape, lay, ratio, cfg_id=12)
    dc = DeviceCase(case)
    K, s_gpu, a_gpu, y = run_layer_step(dc, ratio, ab.F_SCORE | ab.F_SELECT)
    n = K + lay.n_extra
    ckb, cvb = ab.to_host_bits(dc.ck), ab.to_host_bits(dc.cv)
    for b in range(B):
        free = oracle_step(case, b, ratio=ratio)                     # the oracle's own selection
        err = np.abs(s_gpu[b] - free["scores64"]) / np.maximum(free["scores64"], free["scores64"].mean())
        assert err.max() < 1e-3
        ok, why = orc.anchor_set_ok(a_gpu[b, :K], K, L, free["must"], free["may"])
        assert ok, why
        ref = oracle_step(case, b, anchor_idx=a_gpu[b, :K])          # teacher-forced on the GPU's set
        rows = ref["rows"]
        keep = np.setdiff1d(np.arange(lay.ctx_len), rows)
        assert np.array_equal(ckb[b][keep], case.cache_k[b][keep]) and np.array_equal(cvb[b][keep], case.cache_v[b][keep])
        if n:
            assert_close_bf16(ckb[b][rows], ref["k_new"], "K rows")
            assert_close_bf16(cvb[b][rows], ref["v_new"], "V rows")
            assert_close_bf16(ab.to_host_bits(y[b, :n]), ref["y"], "y")
        if ratio == 1.0 and extra == "all":
            # full recompute == the dense layer written separately in the oracle
            yd, kd, vd = orc.dense_layer(case.weights, shape, case.x[b], case.rope_cos, case.rope_sin)
            assert_close_bf16(ckb[b][:lay.ctx_len], kd, "K vs dense")
            assert_close_bf16(cvb[b][:lay.ctx_len], vd, "V vs dense")
            assert_close_bf16(ab.to_host_bits(y[b, :n]), yd[rows], "y vs dense")
        if ratio == 0.0:
            l = lay.affix_start
            assert np.array_equal(ckb[b][l:l + L], case.cache_k[b][l:l + L])
    assert dc.ctx.poll_status() == 0


def test_fused_step_equals_split_calls():
    lay = wl.make_layout(2, 6, 150, 20, 32, 32, "all")
    case = make_projected_case(MID128, lay, 0.2, cfg_id=13)
    dc = DeviceCase(case)
    K, s_gpu, a_gpu, y_fused = run_layer_step(dc, 0.2, ab.F_SCORE | ab.F_SELECT)
    ck_fused, cv_fused = ab.to_host_bits(dc.ck), ab.to_host_bits(dc.cv)
    dc.reset_cache()
    da = dev_i32(a_gpu[:, :K])
    k_new, v_new, y_split = run_split_calls(dc, da, K)
    dc.ctx.scatter_kv(dc.req, dc.kv(), da, K, k_new, v_new)
    torch.cuda.synchronize()
    assert np.array_equal(ab.to_host_bits(dc.ck), ck_fused) and np.array_equal(ab.to_host_bits(dc.cv), cv_fused)
    n = K + lay.n_extra
    assert_close_bf16(ab.to_host_bits(y_split[:, :n]), ab.to_host_bits(y_fused[:, :n]), "split vs fused y")
    # a second fused step with the anchors given (no scoring) reproduces the first bit for bit
    dc.reset_cache()
    _, _, _, y2 = run_layer_step(dc, 0.2, 0, anchors_in=a_gpu[:, :K])
    assert np.array_equal(ab.to_host_bits(y2), ab.to_host_bits(y_fused))
    assert np.array_equal(ab.to_host_bits(dc.ck), ck_fused)


def test_idempotent_when_cache_is_current():
    """Cache computed from the very hidden rows being refreshed: refreshed K/V stay within
    tolerance of the cached ones (the oracle gives identical bytes)."""
    lay = wl.make_layout(1, 0, 128, 32, 32, 32, "all")
    case = wl.make_case(wl.TINY, lay, 0.5, cfg_id=14)
    from helpers import projected_cache
    case.cache_k, case.cache_v = projected_cache(case, case.x)
    dc = DeviceCase(case)
    run_layer_step(dc, 0.5, ab.F_SCORE | ab.F_SELECT)
    assert_close_bf16(ab.to_host_bits(dc.ck), case.cache_k, "K idempotent")
    assert_close_bf16(ab.to_host_bits(dc.cv), case.cache_v, "V idempotent")


def test_compact_input_matches_gathered_input():
    lay = wl.make_layout(2, 0, 128, 16, 32, 32, "masked")
    case = make_projected_case(wl.TINY, lay, 0.25, cfg_id=15)
    dc = DeviceCase(case)
    K, _, a_gpu, y_full = run_layer_step(dc, 0.25, ab.F_SCORE | ab.F_SELECT)
    n = K + lay.n_extra
    rows = np.stack([orc.recompute_set(a_gpu[b, :K], lay.affix_start, lay.extra_rows[b]) for b in range(2)])
    xc = torch.stack([dc.x[b, torch.from_numpy(rows[b]).to(DEV)] for b in range(2)]).contiguous()
    dc.reset_cache()
    y = torch.zeros((2, n, case.shape.hidden), dtype=torch.bfloat16, device=DEV)
    anchors = dev_i32(a_gpu[:, :K])
    dc.ctx.layer_step(dc.lw, dc.req, dc.kv(), xc, 1, 0.25, 0, None, anchors, y)
    torch.cuda.synchronize()
    assert np.array_equal(ab.to_host_bits(y), ab.to_host_bits(y_full[:, :n]))


def test_out_of_range_index_is_flagged_and_skipped():
    lay = wl.make_layout(1, 0, 128, 16, 32, 32, "none")
    case = wl.make_case(wl.TINY, lay, 0.1, cfg_id=16)
    dc = DeviceCase(case)
    K = orc.k_from_ratio(128, 0.1)
    bad = np.arange(K, dtype=np.int32)[None].copy()
    bad[0, 3] = 100000
    da = dev_i32(bad)
    k_new, v_new, y = run_split_calls(dc, da, K)
    dc.ctx.scatter_kv(dc.req, dc.kv(), da, K, k_new, v_new)
    torch.cuda.synchronize()
    assert dc.ctx.poll_status() & ab.FLAG_BAD_INDEX
    assert dc.ctx.poll_status() == 0                                   # cleared by the poll
    ckb = ab.to_host_bits(dc.ck)
    keep = np.setdiff1d(np.arange(lay.ctx_len), np.delete(bad[0], 3))
    assert np.array_equal(ckb[0][keep], case.cache_k[0][keep])


@pytest.mark.parametrize("shape,L,extra,ratio", [
    (wl.TINY, 128, "masked", 0.2),       # the step needs most of x: staged by one copy
    (wl.TINY, 128, "none", 0.05),        # 38 of 192 rows: page-locked x is read in place, each row once
    (MID128, 600, "all", 0.05),          # in place with request rows among the recomputed ones (their residual comes
])                                       # from the device copy the row preparation leaves), head dimension 128
def test_host_buffer_entry_point(shape, L, extra, ratio):
    lay = wl.make_layout(2, 0, L, 32, 32, 32, extra)
    case = make_projected_case(shape, lay, ratio, cfg_id=17)
    dc = DeviceCase(case)
    K, s_dev, a_dev, y_dev = run_layer_step(dc, ratio, ab.F_SCORE | ab.F_SELECT)
    n = K + lay.n_extra
    dc.reset_cache()
    xh = torch.from_numpy(case.x.view(np.int16)).view(torch.bfloat16).pin_memory()
    sh = torch.zeros((2, L), dtype=torch.float32).pin_memory()
    ah = torch.zeros((2, K), dtype=torch.int32).pin_memory()
    yh = torch.zeros((2, n, case.shape.hidden), dtype=torch.bfloat16).pin_memory()
    dc.ctx.layer_step_host(dc.lw, dc.req, dc.kv(), xh, ratio, 0, sh, ah, yh)
    torch.cuda.synchronize()
    assert np.array_equal(sh.numpy(), s_dev) and np.array_equal(ah.numpy(), a_dev[:, :K])
    assert np.array_equal(ab.to_host_bits(yh), ab.to_host_bits(y_dev[:, :n]))
    # page-locked x is read in place by the kernels, pageable x is staged by a copy: same results; so are pageable outputs
    assert dc.ctx.host_x_in_place(xh)
    xp = torch.from_numpy(case.x.view(np.int16).copy()).view(torch.bfloat16)
    assert not dc.ctx.host_x_in_place(xp)
    dc.reset_cache()
    sh2, ah2, yh2 = (torch.zeros(t.shape, dtype=t.dtype) for t in (sh, ah, yh))
    dc.ctx.layer_step_host(dc.lw, dc.req, dc.kv(), xp, ratio, 0, sh2, ah2, yh2)
    torch.cuda.synchronize()
    assert np.array_equal(sh2.numpy(), s_dev) and np.array_equal(ah2.numpy(), a_dev[:, :K])
    assert np.array_equal(ab.to_host_bits(yh2), ab.to_host_bits(y_dev[:, :n]))


def test_invalid_arguments_enqueue_nothing():
    lay = wl.make_layout(1, 0, 128, 16, 32, 32, "none")
    case = wl.make_case(wl.TINY, lay, 0.1, cfg_id=18)
    dc = DeviceCase(case, max_rows=8)
    before = dc.ctx.launch_count()
    y = torch.zeros((1, 64, 256), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(ab.AcacheError) as e:      # K = 13 rows > max_rows = 8
        dc.ctx.layer_step(dc.lw, dc.req, dc.kv(), dc.x, 0, 0.1, 0, None, dev_i32(np.arange(13)[None]), y)
    assert e.value.status == ab.ERR_INVALID_ARG
    with pytest.raises(ab.AcacheError):           # misaligned x
        dc.ctx.layer_step(dc.lw, dc.req, dc.kv(), dc.x.data_ptr() + 2, 0, 0.05, 0, None, dev_i32(np.arange(7)[None]), y)
    assert dc.ctx.launch_count() == before


# ------------------------------------------------------------------ benchmark configuration 2, full size
@pytest.mark.parametrize("extra", ["none", "all"])
def test_llada_layer_full_size(extra):
    """512-token affix + 256 request + 256 generation rows at LLaDA-8B layer shapes, ratio 20 %,
    in the configuration the benchmark times (random stale cache)."""
    lay = wl.config_layout(2, extra)
    case = wl.make_case(wl.LLADA_8B, lay, 0.2, cfg_id=2)
    dc = DeviceCase(case)
    K, s_gpu, a_gpu, y = run_layer_step(dc, 0.2, ab.F_SCORE | ab.F_SELECT)
    assert K == 103
    n = K + lay.n_extra
    free = oracle_step(case, 0, ratio=0.2)
    err = np.abs(s_gpu[0] - free["scores64"]) / np.maximum(free["scores64"], free["scores64"].mean())
    assert err.max() < 1e-3
    ok, why = orc.anchor_set_ok(a_gpu[0, :K], K, 512, free["must"], free["may"])
    assert ok, why
    ref = free if np.array_equal(free["anchor_idx"], a_gpu[0, :K]) else oracle_step(case, 0, anchor_idx=a_gpu[0, :K])
    rows = ref["rows"]
    ckb, cvb = ab.to_host_bits(dc.ck), ab.to_host_bits(dc.cv)
    keep = np.setdiff1d(np.arange(lay.ctx_len), rows)
    assert np.array_equal(ckb[0][keep], case.cache_k[0][keep]) and np.array_equal(cvb[0][keep], case.cache_v[0][keep])
    assert_close_bf16(ckb[0][rows], ref["k_new"], "K rows")
    assert_close_bf16(cvb[0][rows], ref["v_new"], "V rows")
    assert_close_bf16(ab.to_host_bits(y[0, :n]), ref["y"], "y")
    assert dc.ctx.poll_status() == 0


# ------------------------------------------------------------------ shared affix storage (Section 4.1)
@pytest.mark.parametrize("L,ratio", [(160, 0.2), (400, 0.7)])    # 88 rows: one query tile; 336 rows: three (two per CTA + one)
def test_shared_affix_cache_with_private_rows(L, ratio):
    """One copy of the affix K/V (batch_stride = 0) serves three requests: scoring reads it, the
    refresh writes each request's anchors and request rows to its private k_new / v_new and its
    attention reads all other positions from the shared copy, which stays untouched."""
    shape, B = MID128, 3
    lay = wl.make_layout(B, 0, L, 24, 32, 32, "all")
    case = wl.make_case(shape, lay, ratio, cfg_id=19)
    T, L = lay.ctx_len, lay.affix_len
    shared_k, shared_v = case.cache_k[0].copy(), case.cache_v[0].copy()      # [T, Hkv, d]; only affix rows matter
    dc = DeviceCase(case)
    dsk, dsv = ab.to_device_bf16(shared_k[None], DEV), ab.to_device_bf16(shared_v[None], DEV)
    kv = ab.KV(dsk.data_ptr(), dsv.data_ptr(), 0, T)
    K = orc.k_from_ratio(L, ratio)
    n = K + lay.n_extra
    # scores from masked-row queries computed by the oracle (any queries would do)
    q = wl.random_q_mask(shape, lay, 91)
    dq = ab.to_device_bf16(q, DEV)
    scores = torch.zeros((B, L), dtype=torch.float32, device=DEV)
    dc.ctx.score_anchors(dc.req, dq, kv, scores)
    anchors = torch.zeros((B, K), dtype=torch.int32, device=DEV)
    dc.ctx.select_topk(scores, B, L, K, anchors)
    k_new = torch.zeros((B, n, shape.n_kv_heads, shape.head_dim), dtype=torch.bfloat16, device=DEV)
    v_new = torch.zeros_like(k_new)
    y = torch.zeros((B, n, shape.hidden), dtype=torch.bfloat16, device=DEV)
    dc.ctx.recompute_anchors(dc.lw, dc.req, kv, dc.x, 0, anchors, K, k_new, v_new, y)
    torch.cuda.synchronize()
    assert dc.ctx.poll_status() == 0
    assert np.array_equal(ab.to_host_bits(dsk[0]), shared_k) and np.array_equal(ab.to_host_bits(dsv[0]), shared_v)
    s_gpu, a_gpu = scores.cpu().numpy(), anchors.cpu().numpy()
    for b in range(B):
        kf = orc.bf16_bits_to_f64(shared_k[:T])
        s_ref = orc.score_anchors(orc.bf16_bits_to_f64(q[b]), kf[lay.affix_start:lay.affix_start + L])
        assert (np.abs(s_gpu[b] - s_ref) / np.maximum(s_ref, s_ref.mean())).max() < 1e-3
        _, _, must, may = orc.select_topk(s_ref.astype(np.float32), K)
        ok, why = orc.anchor_set_ok(a_gpu[b], K, L, must, may)
        assert ok, why
        # the oracle with a private copy of the shared cache for this request
        ref = orc.layer_step(case.weights, shape, case.x[b], shared_k, shared_v, T, lay.affix_start, L,
                             lay.masked_pos[b], lay.extra_rows[b], case.rope_cos, case.rope_sin, anchor_idx=a_gpu[b])
        assert_close_bf16(ab.to_host_bits(k_new[b]), ref["k_new"], "private K")
        assert_close_bf16(ab.to_host_bits(v_new[b]), ref["v_new"], "private V")
        assert_close_bf16(ab.to_host_bits(y[b]), ref["y"], "y")
    # the fused call over the same storage: the masked rows' queries now come from its own projection of x
    k2, v2, y2 = torch.zeros_like(k_new), torch.zeros_like(v_new), torch.zeros_like(y)
    scores2, anchors2 = torch.zeros_like(scores), torch.zeros_like(anchors)
    dc.ctx.layer_step_shared(dc.lw, dc.req, kv, dc.x, 0, ratio, ab.F_SCORE | ab.F_SELECT, scores2, anchors2, k2, v2, y2)
    torch.cuda.synchronize()
    assert dc.ctx.poll_status() == 0
    assert np.array_equal(ab.to_host_bits(dsk[0]), shared_k) and np.array_equal(ab.to_host_bits(dsv[0]), shared_v)
    s2, a2 = scores2.cpu().numpy(), anchors2.cpu().numpy()
    for b in range(B):
        free = orc.layer_step(case.weights, shape, case.x[b], shared_k, shared_v, T, lay.affix_start, L,
                              lay.masked_pos[b], lay.extra_rows[b], case.rope_cos, case.rope_sin, ratio=ratio)
        assert (np.abs(s2[b] - free["scores64"]) / np.maximum(free["scores64"], free["scores64"].mean())).max() < 1e-3
        ok, why = orc.anchor_set_ok(a2[b], K, L, free["must"], free["may"])
        assert ok, why
        ref = free if np.array_equal(free["anchor_idx"], a2[b]) else orc.layer_step(
            case.weights, shape, case.x[b], shared_k, shared_v, T, lay.affix_start, L, lay.masked_pos[b], lay.extra_rows[b],
            case.rope_cos, case.rope_sin, anchor_idx=a2[b])
        assert_close_bf16(ab.to_host_bits(k2[b]), ref["k_new"], "private K (fused call)")
        assert_close_bf16(ab.to_host_bits(v2[b]), ref["v_new"], "private V (fused call)")
        assert_close_bf16(ab.to_host_bits(y2[b]), ref["y"], "y (fused call)")
    # calls that write the cache refuse a shared one
    with pytest.raises(ab.AcacheError):
        dc.ctx.scatter_kv(dc.req, kv, anchors, K, k_new, v_new)
    with pytest.raises(ab.AcacheError):
        dc.ctx.layer_step(dc.lw, dc.req, kv, dc.x, 0, ratio, 0, None, anchors, y)


def test_duplicate_row_is_served_once_in_the_split_calls():
    """Two fresh rows naming the same position: the position -> row map lets the later one serve it, and the
    attention that reads cache and fresh rows as two key sources must not count the position twice."""
    shape, B = MID128, 1
    lay = wl.make_layout(B, 0, 140, 20, 32, 32, "all")
    dup = np.concatenate([lay.extra_rows, lay.extra_rows[:, 3:4]], axis=1)          # one position twice
    lay2 = wl.Layout(lay.batch, lay.ctx_len, lay.affix_start, lay.affix_len, lay.masked_pos, np.ascontiguousarray(dup), "dup")
    case = wl.make_case(shape, lay2, 0.25, cfg_id=23)
    dc = DeviceCase(case)
    K = orc.k_from_ratio(lay.affix_len, 0.25)
    g = np.random.default_rng(4)
    anchors = np.sort(g.choice(lay.affix_len, K, replace=False))[None].astype(np.int32)
    k_new, v_new, y = run_split_calls(dc, dev_i32(anchors), K)
    torch.cuda.synchronize()
    assert dc.ctx.poll_status() == 0
    ref = oracle_step(case, 0, anchor_idx=anchors[0])
    assert_close_bf16(ab.to_host_bits(y[0]), ref["y"], "y with a duplicated row")
    assert_close_bf16(ab.to_host_bits(k_new[0]), ref["k_new"], "k_new with a duplicated row")


def test_degenerate_inputs():
    """Empty batch, no masked rows, a one-token affix: nothing faults, the defined results come out."""
    shape = MID128
    lay = wl.make_layout(2, 3, 40, 9, 32, 32, "all")
    case = wl.make_case(shape, lay, 0.25, cfg_id=27)
    dc = DeviceCase(case)
    B, L, T = lay.batch, lay.affix_len, lay.ctx_len
    K = orc.k_from_ratio(L, 0.25)
    n = K + lay.n_extra
    scores = torch.full((B, L), 5.0, dtype=torch.float32, device=DEV)
    anchors = torch.full((B, K), -1, dtype=torch.int32, device=DEV)
    y = torch.zeros((B, n, shape.hidden), dtype=torch.bfloat16, device=DEV)
    # an empty batch launches nothing
    req0 = ab.Context.request(0, T, lay.affix_start, L, dc.masked, dc.extra, dc.cos, dc.sin)
    l0 = dc.ctx.launch_count()
    dc.ctx.layer_step(dc.lw, req0, dc.kv(), dc.x, 0, 0.25, ab.F_SCORE | ab.F_SELECT, scores, anchors, y)
    assert dc.ctx.launch_count() == l0
    # no masked rows: this layer adds nothing to the scores (they are zeroed unless accumulating), Eq. 6 on
    # all-equal scores takes the K lowest positions, and the refresh of those rows is the oracle's
    req1 = ab.Context.request(B, T, lay.affix_start, L, None, dc.extra, dc.cos, dc.sin)
    dc.ctx.layer_step(dc.lw, req1, dc.kv(), dc.x, 0, 0.25, ab.F_SCORE | ab.F_SELECT, scores, anchors, y)
    torch.cuda.synchronize()
    assert torch.count_nonzero(scores).item() == 0
    assert np.array_equal(anchors.cpu().numpy(), np.broadcast_to(np.arange(K, dtype=np.int32), (B, K)))
    for b in range(B):
        ref = oracle_step(case, b, anchor_idx=np.arange(K))
        assert_close_bf16(ab.to_host_bits(y[b]), ref["y"], "y with the K lowest positions as anchors")
    scores.fill_(2.0)
    dc.ctx.layer_step(dc.lw, req1, dc.kv(), dc.x, 0, 0.0, ab.F_SCORE | ab.F_ACCUMULATE | ab.F_NO_RECOMPUTE, scores, None, None)
    torch.cuda.synchronize()
    assert torch.all(scores == 2.0).item()
    assert dc.ctx.poll_status() == 0
    # a one-token affix at ratio 1: K = 1, the single affix row is refreshed
    lay1 = wl.make_layout(1, 5, 1, 6, 32, 32, "none")
    case1 = wl.make_case(shape, lay1, 1.0, cfg_id=28)
    dc1 = DeviceCase(case1)
    K1, s1, a1, y1 = run_layer_step(dc1, 1.0, ab.F_SCORE | ab.F_SELECT)
    assert K1 == 1 and a1[0, 0] == 0
    assert abs(s1[0, 0] - shape.n_heads * lay1.n_masked) < 1e-3 * shape.n_heads * lay1.n_masked     # softmax over one key
    ref = oracle_step(case1, 0, anchor_idx=np.array([0]))
    assert_close_bf16(ab.to_host_bits(y1[0, :1]), ref["y"], "y of the single affix row")
    assert dc1.ctx.poll_status() == 0
