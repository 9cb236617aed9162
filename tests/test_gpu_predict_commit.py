"""Predict-then-commit on the current block (Eq. 2-3): final norm + LM head + softmax confidence +
threshold rule, against the oracle."""
import numpy as np
import pytest
import torch

from oracle import acache_oracle as orc
from paper_2608_26140_b200 import binding as ab
from paper_2608_26140_b200 import workloads as wl

from helpers import DEV

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("shape,V,B,h_rows,n_blk", [
    (wl.TINY, 1280, 2, 40, 32),            # 2 x 32 rows, vocabulary of 10 half-tiles: split and whole tiles
    (wl.TINY, 128, 1, 5, 3),               # one half-tile, ragged rows
    (wl.LLADA_8B, 126464, 2, 96, 32),      # the LLaDA vocabulary
])
def test_predict_commit(shape, V, B, h_rows, n_blk):
    D = shape.hidden
    g = np.random.default_rng(V + n_blk)
    w_lm = wl.normal_bf16(7001, (V, D), 0.02)
    gain = wl.normal_bf16(7002, (D,), 0.05, 1.0)
    h = wl.normal_bf16(7003, (B, h_rows, D), 1.0)
    block_rows = np.stack([np.sort(g.choice(h_rows, n_blk, replace=False)) for _ in range(B)]).astype(np.int32)
    # make a few rows confident: point them along one vocabulary row (RMSNorm keeps the direction)
    Wf = wl.bf16_bits_to_f32(w_lm)
    hf = wl.bf16_bits_to_f32(h)
    for b in range(B):
        for j in g.choice(n_blk, max(1, n_blk // 4), replace=False):
            v = int(g.integers(0, V))
            hf[b, block_rows[b, j]] = Wf[v] / np.abs(Wf[v]).max() * 40.0 + 0.05 * hf[b, block_rows[b, j]]
    if B > 1:
        hf[B - 1] *= 0.0
        hf[B - 1] += wl.bf16_bits_to_f32(wl.normal_bf16(7004, (h_rows, D), 1.0))    # last request: nobody confident
    h = wl.f32_to_bf16_bits(hf)

    ctx = ab.Context.for_shape(shape, B, 64, 32, 8, 8, DEV, max_vocab=V, max_block=n_blk)
    dh, dw, dg = ab.to_device_bf16(h, DEV), ab.to_device_bf16(w_lm, DEV), ab.to_device_bf16(gain, DEV)
    dbr = torch.from_numpy(block_rows).to(DEV)
    token = torch.full((B, n_blk), -1, dtype=torch.int32, device=DEV)
    conf = torch.zeros((B, n_blk), dtype=torch.float32, device=DEV)
    commit = torch.full((B, n_blk), -1, dtype=torch.int32, device=DEV)
    ctx.predict_commit(dh, h_rows, dbr, B, n_blk, dg, dw, V, 0.9, token, conf, commit)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    t_gpu, c_gpu, k_gpu = token.cpu().numpy(), conf.cpu().numpy().astype(np.float64), commit.cpu().numpy()
    for b in range(B):
        rows = orc.bf16_bits_to_f64(h[b])[block_rows[b]]
        tok, cf, cm, z = orc.predict_commit(rows, gain, w_lm, shape.rms_eps, 0.9)
        zs = np.sort(z, axis=1)
        clear = (zs[:, -1] - zs[:, -2]) > 1e-3 * np.abs(zs[:, -1]).clip(1e-3)     # arg max not a near tie
        assert np.array_equal(t_gpu[b][clear], tok[clear])
        assert clear.mean() > 0.9
        assert np.allclose(c_gpu[b], cf, rtol=2e-3, atol=1e-7), np.abs(c_gpu[b] - cf).max()
        sure = np.abs(cf - 0.9) > 2e-3
        if cm.sum() > 1 or (cf > 0.9).any():
            assert np.array_equal(k_gpu[b][sure] != 0, cm[sure])
        else:                                                   # fallback: exactly one row, the most confident
            assert k_gpu[b].sum() == 1
            j = int(np.argmax(k_gpu[b]))
            assert cf[j] >= cf.max() * (1 - 2e-3)
    if B > 1:
        assert commit[B - 1].sum().item() == 1                  # the fallback path was exercised
    assert (commit[0] != 0).sum().item() >= 1


def test_denoise_step_two_layers_with_embedding_lookup():
    """acache_denoise_step: token ids -> embedding rows -> two refresh layers with a fixed anchor set ->
    LM head + commit, against the oracle's refresh_forward + predict_commit."""
    shape, n_layers, B, V = wl.TINY_GQA, 2, 2, 640
    lay = wl.make_layout(B, 4, 64, 12, 32, 32, "all")
    T, l, L, P = lay.ctx_len, lay.affix_start, lay.affix_len, lay.n_extra
    K = 16
    g = np.random.default_rng(5)
    layers = [wl.layer_weights(shape, 41, n) for n in range(n_layers)]
    embed = wl.normal_bf16(7101, (V, shape.hidden), 1.0)
    w_lm = wl.normal_bf16(7102, (V, shape.hidden), 0.02)
    gain = wl.normal_bf16(7103, (shape.hidden,), 0.05, 1.0)
    ids = g.integers(0, V, size=(B, T)).astype(np.int32)
    ids[:, l:l + L] = ids[0, l:l + L]                               # the affix text is shared
    x0 = embed[ids]                                                 # [B, T, D] bf16 bits
    cos, sin = wl.rope_table(T, shape.head_dim, shape.rope_theta)
    caches = [[wl.random_kv_cache(shape, wl.make_layout(1, 4, 64, 12, 32, 32, "all"), 900 + 10 * n + b) for n in range(n_layers)]
              for b in range(B)]
    caches = [[(ck[0], cv[0]) for (ck, cv) in per_b] for per_b in caches]
    anchors = np.stack([np.sort(g.choice(L, K, replace=False)) for _ in range(B)]).astype(np.int32)
    # current block = the masked rows; their compact rows: anchors first, then extras in order
    where = {int(p): i for i, p in enumerate(lay.extra_rows[0])}
    block_rows = np.stack([[K + where[int(p)] for p in lay.masked_pos[b]] for b in range(B)]).astype(np.int32)
    n_blk = block_rows.shape[1]

    ctx = ab.Context.for_shape(shape, B, T, L, K + P, lay.n_masked, DEV, max_vocab=V, max_block=n_blk)
    dl = [{k: (ab.to_device_bf16(v, DEV) if v is not None else None) for k, v in w.items()} for w in layers]
    lws = [ab.Context.weights(w) for w in dl]
    dk = [ab.to_device_bf16(np.stack([caches[b][n][0] for b in range(B)]), DEV) for n in range(n_layers)]
    dv = [ab.to_device_bf16(np.stack([caches[b][n][1] for b in range(B)]), DEV) for n in range(n_layers)]
    kvs = [ab.Context.kv(dk[n], dv[n]) for n in range(n_layers)]
    dcos, dsin = torch.from_numpy(cos).to(DEV), torch.from_numpy(sin).to(DEV)
    masked = torch.from_numpy(lay.masked_pos.copy()).to(DEV)
    extra = torch.from_numpy(lay.extra_rows.copy()).to(DEV)
    dids = torch.from_numpy(ids).to(DEV)
    req = ab.Context.request(B, T, l, L, masked, extra, dcos, dsin, token_ids=dids, n_embed=V)
    de, dw, dg = ab.to_device_bf16(embed, DEV), ab.to_device_bf16(w_lm, DEV), ab.to_device_bf16(gain, DEV)
    ya = torch.zeros((B, K + P, shape.hidden), dtype=torch.bfloat16, device=DEV)
    yb = torch.zeros_like(ya)
    da, dbr = torch.from_numpy(anchors).to(DEV), torch.from_numpy(block_rows).to(DEV)
    token = torch.full((B, n_blk), -1, dtype=torch.int32, device=DEV)
    conf = torch.zeros((B, n_blk), dtype=torch.float32, device=DEV)
    commit = torch.full((B, n_blk), -1, dtype=torch.int32, device=DEV)
    last = ctx.denoise_step(lws, kvs, req, de, da, K, ya, yb, dbr, n_blk, dg, dw, V, 0.9, token, conf, commit)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    assert last == yb.data_ptr()                                    # two layers: a then b
    from helpers import TOL, assert_close_bf16, e2e_tol
    for b in range(B):
        rows, ref_caches, ys = orc.refresh_forward(layers, shape, x0[b], caches[b], T, l, anchors[b], lay.extra_rows[b],
                                                   cos, sin)
        assert_close_bf16(ab.to_host_bits(yb[b]), ys[-1], "last layer output", e2e_tol(n_layers))
        for n in range(n_layers):
            assert_close_bf16(ab.to_host_bits(dk[n][b])[rows], ref_caches[n][0][rows], f"layer {n} K", e2e_tol(n_layers))
        # teacher-forced head: the oracle's head on the GPU's own last-layer rows
        hrows = orc.bf16_bits_to_f64(ab.to_host_bits(yb[b]))[block_rows[b]]
        tok, cf, cm, z = orc.predict_commit(hrows, gain, w_lm, shape.rms_eps, 0.9)
        zs = np.sort(z, axis=1)
        clear = (zs[:, -1] - zs[:, -2]) > 1e-3 * np.abs(zs[:, -1]).clip(1e-3)
        assert np.array_equal(token.cpu().numpy()[b][clear], tok[clear]) and clear.mean() > 0.8
        assert np.allclose(conf.cpu().numpy()[b], cf, rtol=2e-3)
        assert commit[b].sum().item() == cm.sum() == 1              # random weights: nobody is confident
        assert cf[int(np.argmax(commit.cpu().numpy()[b]))] >= cf.max() * (1 - 2e-3)


@pytest.mark.parametrize("shape", [wl.TINY_GQA, wl.LayerShape(512, 4, 2, 128, 1024, 1e-5, True, 5e5, "mid-d128")])
def test_denoise_step_shared_storage_equals_private_caches(shape):
    """acache_denoise_step_shared (one cache per layer for the whole batch, fresh rows in private slots,
    nothing written to the cache) against acache_denoise_step on per-request copies of the same cache:
    same fresh K/V bit for bit, same predictions, outputs within tolerance; the shared caches untouched."""
    n_layers, B, V = 2, 3, 256
    lay = wl.make_layout(B, 0, 150, 20, 32, 32, "all")
    T, l, L, P = lay.ctx_len, lay.affix_start, lay.affix_len, lay.n_extra
    K = 40
    g = np.random.default_rng(15)
    layers = [wl.layer_weights(shape, 43, n) for n in range(n_layers)]
    embed = wl.normal_bf16(7201, (V, shape.hidden), 1.0)
    w_lm = wl.normal_bf16(7202, (V, shape.hidden), 0.3)
    gain = wl.normal_bf16(7203, (shape.hidden,), 0.05, 1.0)
    ids = g.integers(0, V, size=(B, T)).astype(np.int32)
    ids[:, l:l + L] = ids[0, l:l + L]
    cos, sin = wl.rope_table(T, shape.head_dim, shape.rope_theta)
    one = wl.make_layout(1, 0, 150, 20, 32, 32, "all")
    shared = [wl.random_kv_cache(shape, one, 950 + n) for n in range(n_layers)]          # [1, T, Hkv, d] each
    anchors = np.stack([np.sort(g.choice(L, K, replace=False)) for _ in range(B)]).astype(np.int32)
    where = {int(p): i for i, p in enumerate(lay.extra_rows[0])}
    block_rows = np.stack([[K + where[int(p)] for p in lay.masked_pos[b][:8]] for b in range(B)]).astype(np.int32)
    n_blk, n = 8, K + P

    ctx = ab.Context.for_shape(shape, B, T, L, n, lay.n_masked, DEV, max_vocab=V, max_block=n_blk)
    dl = [{k: (ab.to_device_bf16(v, DEV) if v is not None else None) for k, v in w.items()} for w in layers]
    lws = [ab.Context.weights(w) for w in dl]
    dcos, dsin = torch.from_numpy(cos).to(DEV), torch.from_numpy(sin).to(DEV)
    masked = torch.from_numpy(lay.masked_pos.copy()).to(DEV)
    extra = torch.from_numpy(lay.extra_rows.copy()).to(DEV)
    dids = torch.from_numpy(ids).to(DEV)
    req = ab.Context.request(B, T, l, L, masked, extra, dcos, dsin, token_ids=dids, n_embed=V)
    de, dw, dg = ab.to_device_bf16(embed, DEV), ab.to_device_bf16(w_lm, DEV), ab.to_device_bf16(gain, DEV)
    da, dbr = torch.from_numpy(anchors).to(DEV), torch.from_numpy(block_rows).to(DEV)

    def outputs():
        return (torch.zeros((B, n, shape.hidden), dtype=torch.bfloat16, device=DEV), torch.zeros((B, n, shape.hidden), dtype=torch.bfloat16, device=DEV),
                torch.zeros((B, n_blk), dtype=torch.int32, device=DEV), torch.zeros((B, n_blk), dtype=torch.float32, device=DEV),
                torch.zeros((B, n_blk), dtype=torch.int32, device=DEV))

    # shared storage
    sk = [ab.to_device_bf16(shared[i][0], DEV) for i in range(n_layers)]
    sv = [ab.to_device_bf16(shared[i][1], DEV) for i in range(n_layers)]
    kvs_s = [ab.KV(sk[i].data_ptr(), sv[i].data_ptr(), 0, T) for i in range(n_layers)]
    k_new = [torch.zeros((B, n, shape.n_kv_heads, shape.head_dim), dtype=torch.bfloat16, device=DEV) for _ in range(n_layers)]
    v_new = [torch.zeros_like(k_new[0]) for _ in range(n_layers)]
    ya, yb, tok_s, conf_s, com_s = outputs()
    ctx.denoise_step_shared(lws, kvs_s, req, de, da, K, k_new, v_new, ya, yb, dbr, n_blk, dg, dw, V, 0.9, tok_s, conf_s, com_s)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    for i in range(n_layers):
        assert np.array_equal(ab.to_host_bits(sk[i]), shared[i][0]) and np.array_equal(ab.to_host_bits(sv[i]), shared[i][1])
    y_shared = ab.to_host_bits(yb)

    # one working cache per request, seeded with the same contents
    pk = [ab.to_device_bf16(np.repeat(shared[i][0], B, axis=0), DEV) for i in range(n_layers)]
    pv = [ab.to_device_bf16(np.repeat(shared[i][1], B, axis=0), DEV) for i in range(n_layers)]
    kvs_p = [ab.Context.kv(pk[i], pv[i]) for i in range(n_layers)]
    ya2, yb2, tok_p, conf_p, com_p = outputs()
    ctx.denoise_step(lws, kvs_p, req, de, da, K, ya2, yb2, dbr, n_blk, dg, dw, V, 0.9, tok_p, conf_p, com_p)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    from helpers import TOL, assert_close_bf16, e2e_tol
    assert_close_bf16(y_shared, ab.to_host_bits(yb2), "last layer output, shared vs private", TOL)
    rows_of = [np.concatenate([l + anchors[b], lay.extra_rows[b]]) for b in range(B)]
    for b in range(B):
        # layer 0 sees identical inputs in both runs: its fresh K/V are the same bits
        assert np.array_equal(ab.to_host_bits(k_new[0][b]), ab.to_host_bits(pk[0][b])[rows_of[b]])
        assert np.array_equal(ab.to_host_bits(v_new[0][b]), ab.to_host_bits(pv[0][b])[rows_of[b]])
        assert_close_bf16(ab.to_host_bits(k_new[1][b]), ab.to_host_bits(pk[1][b])[rows_of[b]], "layer 1 fresh K", TOL)
    assert np.allclose(conf_s.cpu().numpy(), conf_p.cpu().numpy(), rtol=5e-2, atol=1e-3)
    # and against the oracle, request by request (its private copy of the shared cache)
    for b in range(B):
        caches_b = [(shared[i][0][0], shared[i][1][0]) for i in range(n_layers)]
        rows, ref_caches, ys = orc.refresh_forward(layers, shape, embed[ids[b]], caches_b, T, l, anchors[b], lay.extra_rows[b], cos, sin)
        assert_close_bf16(y_shared[b], ys[-1], "last layer output vs oracle", e2e_tol(n_layers))
        assert_close_bf16(ab.to_host_bits(k_new[1][b]), ref_caches[1][0][rows], "layer 1 fresh K vs oracle", e2e_tol(n_layers))
