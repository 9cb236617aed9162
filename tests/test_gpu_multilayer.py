"""N > 1 layers through the C ABI: the one-shot probe (scores accumulated over layers from the
non-affix rows only, Section 3.2), one selection, then the refresh pass with the fixed anchor
set (Section 3.3), each layer's compact output feeding the next layer."""
import numpy as np
import pytest
import torch

from oracle import acache_oracle as orc
from paper_2608_26140_b200 import binding as ab
from paper_2608_26140_b200 import workloads as wl

from helpers import DEV, TOL, assert_close_bf16, e2e_tol

pytestmark = pytest.mark.gpu


def build(shape, n_layers, B, pre, L, post, gen, m):
    lay = wl.make_layout(B, pre, L, post, gen, m, "all")
    layers = [wl.layer_weights(shape, 31, n) for n in range(n_layers)]
    x = wl.hidden_states(shape, lay, 500, 501)
    xs = wl.hidden_states(shape, lay, 500, 502)
    cos, sin = wl.rope_table(lay.ctx_len, shape.head_dim, shape.rope_theta)
    # stale caches per request and layer: exact K/V of a dense forward under another context
    caches = []
    for b in range(B):
        caches.append([(kb, vb) for (_, kb, vb) in orc.dense_forward(layers, shape, xs[b], cos, sin)])
    return lay, layers, x, caches, cos, sin


MID128 = wl.LayerShape(512, 4, 2, 128, 1024, 1e-5, True, 5e5, "mid-d128")


@pytest.mark.parametrize("shape,n_layers,norm_full,geom", [
    (wl.TINY, 2, False, (6, 96, 20, 32, 32)), (wl.TINY_GQA, 3, True, (6, 96, 20, 32, 32)),
    # head dim 128: the probe's scores come out of its own attention (Eq. 4 over the affix keys); one query tile, then
    # three with the masked rows straddling two of them and an affix that starts and ends inside key tiles
    (MID128, 2, False, (6, 96, 20, 32, 32)), (MID128, 3, False, (20, 300, 100, 100, 100)),
    (MID128, 2, True, (20, 300, 100, 100, 100)),          # normaliser over all keys: the separate scoring kernels
])
def test_probe_select_refresh(shape, n_layers, norm_full, geom):
    B, ratio = 2, 0.25
    lay, layers, x, caches, cos, sin = build(shape, n_layers, B, *geom)
    T, l, L, P = lay.ctx_len, lay.affix_start, lay.affix_len, lay.n_extra
    K = orc.k_from_ratio(L, ratio)
    dev_layers = [{k: (ab.to_device_bf16(v, DEV) if v is not None else None) for k, v in w.items()} for w in layers]
    lws = [ab.Context.weights(w) for w in dev_layers]
    dx = ab.to_device_bf16(x, DEV)
    # device caches [layer][B, T, Hkv, d]
    dk = [ab.to_device_bf16(np.stack([caches[b][n][0] for b in range(B)]), DEV) for n in range(n_layers)]
    dv = [ab.to_device_bf16(np.stack([caches[b][n][1] for b in range(B)]), DEV) for n in range(n_layers)]
    dcos, dsin = torch.from_numpy(cos).to(DEV), torch.from_numpy(sin).to(DEV)
    masked = torch.from_numpy(lay.masked_pos.copy()).to(DEV)
    extra = torch.from_numpy(lay.extra_rows.copy()).to(DEV)
    req = ab.Context.request(B, T, l, L, masked, extra, dcos, dsin)
    ctx = ab.Context.for_shape(shape, B, T, L, L + P, lay.n_masked, DEV)
    scores = torch.zeros((B, L), dtype=torch.float32, device=DEV)
    nf = ab.F_SCORE_NORM_FULL if norm_full else 0

    # ---- probe: K = 0 anchors, rows = all non-affix rows, scores accumulate over layers
    y = [torch.zeros((B, P, shape.hidden), dtype=torch.bfloat16, device=DEV) for _ in range(n_layers)]
    for n in range(n_layers):
        flags = ab.F_SCORE | nf | (ab.F_ACCUMULATE if n else 0)
        xin, compact = (dx, 0) if n == 0 else (y[n - 1], 1)
        ctx.layer_step(lws[n], req, ab.Context.kv(dk[n], dv[n]), xin, compact, 0.0, flags, scores, None, y[n])
    anchors = torch.zeros((B, K), dtype=torch.int32, device=DEV)
    ctx.select_topk(scores, B, L, K, anchors)
    torch.cuda.synchronize()
    s_gpu, a_gpu = scores.cpu().numpy(), anchors.cpu().numpy()

    # ---- the same through the single entry point, on fresh copies of the caches: identical bits
    dk2 = [ab.to_device_bf16(np.stack([caches[b][n][0] for b in range(B)]), DEV) for n in range(n_layers)]
    dv2 = [ab.to_device_bf16(np.stack([caches[b][n][1] for b in range(B)]), DEV) for n in range(n_layers)]
    scores2 = torch.full((B, L), 7.0, dtype=torch.float32, device=DEV)
    anchors2 = torch.zeros((B, K), dtype=torch.int32, device=DEV)
    ya, yb = torch.zeros_like(y[0]), torch.zeros_like(y[0])
    ctx.probe_select(lws, [ab.Context.kv(dk2[n], dv2[n]) for n in range(n_layers)], req, dx, ratio, nf, ya, yb, scores2, anchors2)
    torch.cuda.synchronize()
    assert np.array_equal(scores2.cpu().numpy(), s_gpu) and np.array_equal(anchors2.cpu().numpy(), a_gpu)
    for n in range(n_layers):
        assert torch.equal(dk2[n], dk[n]) and torch.equal(dv2[n], dv[n])
    assert torch.equal(yb if n_layers % 2 == 0 else ya, y[-1])

    # ---- refresh with the fixed anchor set
    yr = [torch.zeros((B, K + P, shape.hidden), dtype=torch.bfloat16, device=DEV) for _ in range(n_layers)]
    for n in range(n_layers):
        xin, compact = (dx, 0) if n == 0 else (yr[n - 1], 1)
        ctx.layer_step(lws[n], req, ab.Context.kv(dk[n], dv[n]), xin, compact, ratio, 0, None, anchors, yr[n])
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0

    for b in range(B):
        s_ref, probe_caches, probe_ys = orc.probe_forward(layers, shape, x[b], caches[b], T, l, L, lay.masked_pos[b],
                                                         lay.extra_rows[b], cos, sin, norm_full)
        # scores with teacher forcing: layer n's term (Eq. 4) from the oracle fed the GPU's own layer-n input rows,
        # summed over the layers (Eq. 5): the single-layer tolerance holds
        rows_p = np.asarray(lay.extra_rows[b], dtype=np.int64)
        where = {int(p): i for i, p in enumerate(rows_p)}
        mask_idx = np.array([where[int(p)] for p in lay.masked_pos[b]])
        s_tf = np.zeros(L)
        for n in range(n_layers):
            x_rows = orc.bf16_bits_to_f64(x[b])[rows_p] if n == 0 else orc.bf16_bits_to_f64(ab.to_host_bits(y[n - 1][b]))
            r = orc.recompute_rows(layers[n], shape, x_rows, rows_p, caches[b][n][0], caches[b][n][1], T, cos, sin)
            Kall = orc.bf16_bits_to_f64((r["cache_k"] if norm_full else caches[b][n][0])[:T])   # as orc.probe_forward
            s_tf += orc.score_anchors(r["q"][mask_idx], Kall[l:l + L], Kall, l, norm_full)
        err_tf = np.abs(s_gpu[b] - s_tf) / np.maximum(s_tf, s_tf.mean())
        assert err_tf.max() < 1e-3, err_tf.max()
        # end to end the later layers' queries come from hidden rows that already differ by the earlier layers'
        # rounding, so the scores' gate grows with the layer count like the outputs' (helpers.e2e_tol)
        err = np.abs(s_gpu[b] - s_ref) / np.maximum(s_ref, s_ref.mean())
        assert err.max() < 1e-3 * n_layers, err.max()
        _, _, must, may = orc.select_topk(s_ref.astype(np.float32), K)
        ok, why = orc.anchor_set_ok(a_gpu[b], K, L, must, may)
        assert ok, why
        assert_close_bf16(ab.to_host_bits(y[-1][b]), probe_ys[-1], "probe output, end to end", e2e_tol(n_layers))
        # end to end with the GPU's anchor set
        rows, ref_caches, ref_ys = orc.refresh_forward(layers, shape, x[b], caches[b], T, l, a_gpu[b],
                                                       lay.extra_rows[b], cos, sin)
        assert_close_bf16(ab.to_host_bits(yr[-1][b]), ref_ys[-1], "refresh output, end to end", e2e_tol(n_layers))
        keep = np.setdiff1d(np.arange(T), rows)
        for n in range(n_layers):
            ckb = ab.to_host_bits(dk[n][b])
            assert np.array_equal(ckb[keep], caches[b][n][0][keep]), "non-anchor affix rows changed"
            assert_close_bf16(ckb[rows], ref_caches[n][0][rows], f"layer {n} K rows", e2e_tol(n_layers))
        # layer-wise teacher forcing: the oracle fed the GPU's layer-n input reproduces its layer-n output
        for n in range(n_layers):
            xin = orc.bf16_bits_to_f64(x[b])[rows] if n == 0 else orc.bf16_bits_to_f64(ab.to_host_bits(yr[n - 1][b]))
            r = orc.recompute_rows(layers[n], shape, xin, rows, caches[b][n][0], caches[b][n][1],
                                   T, cos, sin)
            assert_close_bf16(ab.to_host_bits(yr[n][b]), r["y"], f"layer {n} output, teacher forced")
            assert_close_bf16(ab.to_host_bits(dv[n][b])[rows], r["v_new"], f"layer {n} V rows, teacher forced")
