"""Block decoding through the C ABI (Section 4.3 schedule with the threshold commit of Eq. 3):
acache_commit_update bit for bit against the oracle's rule, acache_generate_block against the
oracle's refresh-then-decode loop on a small two-layer model."""
import numpy as np
import pytest
import torch

from oracle import acache_oracle as orc
from paper_2608_26140_b200 import binding as ab
from paper_2608_26140_b200 import workloads as wl

from helpers import DEV

pytestmark = pytest.mark.gpu

V, MASK = 256, 255


def small_model(shape, n_layers, B, seed):
    """Seeded layers, embedding, LM head and stale caches (a dense forward under another context)."""
    lay = wl.make_layout(B, 4, 80, 12, 32, 32, "all")
    layers = [wl.layer_weights(shape, 33, n) for n in range(n_layers)]
    embed = wl.normal_bf16(seed + 1, (V, shape.hidden), 1.0)
    w_lm = wl.normal_bf16(seed + 2, (V, shape.hidden), 0.6)
    gain = wl.normal_bf16(seed + 3, (shape.hidden,), 0.05, 1.0)
    g = np.random.default_rng(seed)
    ids = g.integers(0, V - 1, size=(B, lay.ctx_len)).astype(np.int32)
    ids[:, lay.affix_start:lay.affix_start + lay.affix_len] = ids[0, lay.affix_start:lay.affix_start + lay.affix_len]
    other = g.integers(0, V - 1, size=(B, lay.ctx_len)).astype(np.int32)
    cos, sin = wl.rope_table(lay.ctx_len, shape.head_dim, shape.rope_theta)
    caches = [[(kb, vb) for (_, kb, vb) in orc.dense_forward(layers, shape, embed[other[b]], cos, sin)] for b in range(B)]
    for b in range(B):
        ids[b, lay.masked_pos[b]] = MASK
    return lay, layers, embed, w_lm, gain, ids, caches, cos, sin


def test_commit_update_bitwise():
    g = np.random.default_rng(5)
    ctx = ab.Context.for_shape(wl.TINY, 8, 512, 128, 1, 1, DEV)
    for trial in range(6):
        B, T, n_blk = 7, 300, [1, 5, 32, 33, 64, 70][trial]
        ids = g.integers(0, 50, size=(B, T)).astype(np.int32)
        pos = np.stack([g.choice(T, n_blk, replace=False) for _ in range(B)]).astype(np.int32)
        for b in range(B):
            m = g.random(n_blk) < [0.0, 0.3, 0.6, 1.0, 0.9, 0.5, 0.05][b]
            ids[b, pos[b][m]] = MASK
        tok = g.integers(0, 50, size=(B, n_blk)).astype(np.int32)
        conf = g.random((B, n_blk)).astype(np.float32)
        if trial % 2:
            conf = np.round(conf * 4) / 4                 # ties, also at the maximum
            conf = np.minimum(conf, 0.75).astype(np.float32)   # nobody above 0.9: the fallback decides
        d_ids, d_pos = torch.from_numpy(ids.copy()).to(DEV), torch.from_numpy(pos).to(DEV)
        d_tok, d_conf = torch.from_numpy(tok).to(DEV), torch.from_numpy(conf).to(DEV)
        left = torch.full((B,), -1, dtype=torch.int32, device=DEV)
        ctx.commit_update(d_ids, T, d_pos, B, n_blk, d_tok, d_conf, MASK, 0.9, left)
        torch.cuda.synchronize()
        ref = ids.copy()
        ref_left = [orc.commit_update(ref[b], pos[b], tok[b], conf[b].astype(np.float64), MASK, np.float32(0.9)) for b in range(B)]
        assert np.array_equal(d_ids.cpu().numpy(), ref), trial
        assert left.cpu().numpy().tolist() == ref_left, trial
    assert ctx.poll_status() == 0


MID128 = wl.LayerShape(512, 4, 2, 128, 1024, 1e-5, True, 5e5, "mid-d128")


@pytest.mark.parametrize("shape,n_layers,threshold,storage,B", [
    (wl.TINY, 2, 0.9, "private", 2), (wl.TINY_GQA, 2, 0.35, "private", 2),
    (wl.TINY_GQA, 2, 0.35, "shared", 2), (MID128, 2, 0.5, "shared", 2),
    (MID128, 2, 0.5, "shared", 5)])       # five requests: one full group of four in a decode-pass attention tile + one
def test_generate_block_vs_oracle(shape, n_layers, threshold, storage, B):
    """Step by step with teacher forcing: before every step the oracle takes the GPU's token state
    (the masked rows of this small random model have nearly equal confidences, so which one the
    fallback commits is not unique); per step the predictions must agree and the GPU's commits must
    be valid under the oracle's confidences.  The C loop must then reproduce the stepwise run exactly.
    storage = "shared": one stale cache per layer serves both requests (batch_stride 0), the refresh
    pass fills private slots and the decode passes refresh the block's rows inside them; the oracle
    runs the same schedule on a private copy of that cache per request."""
    n_blk, ratio, band = 8, 0.25, 0.03
    shared = storage == "shared"
    lay, layers, embed, w_lm, gain, ids, caches, cos, sin = small_model(shape, n_layers, B, 4242)
    if shared:
        caches = [caches[0] for _ in range(B)]
    T, l, L, P = lay.ctx_len, lay.affix_start, lay.affix_len, lay.n_extra
    K = orc.k_from_ratio(L, ratio)
    g = np.random.default_rng(9)
    anchors = np.stack([np.sort(g.choice(L, K, replace=False)) for _ in range(B)]).astype(np.int32)
    block = np.stack([lay.masked_pos[b][:n_blk] for b in range(B)]).astype(np.int32)

    dev_layers = [{k: (ab.to_device_bf16(v, DEV) if v is not None else None) for k, v in w.items()} for w in layers]
    lws = [ab.Context.weights(w) for w in dev_layers]
    dcos, dsin = torch.from_numpy(cos).to(DEV), torch.from_numpy(sin).to(DEV)
    masked = torch.from_numpy(lay.masked_pos.copy()).to(DEV)
    extra = torch.from_numpy(lay.extra_rows.copy()).to(DEV)
    d_block = torch.from_numpy(block).to(DEV)
    d_anchors = torch.from_numpy(anchors).to(DEV)
    where = {int(p): i for i, p in enumerate(lay.extra_rows[0])}
    rows_r = torch.from_numpy(np.stack([[K + where[int(p)] for p in block[b]] for b in range(B)]).astype(np.int32)).to(DEV)
    rows_d = torch.from_numpy(np.broadcast_to(np.arange(n_blk, dtype=np.int32), (B, n_blk)).copy()).to(DEV)
    ctx = ab.Context.for_shape(shape, B, T, L, K + P, lay.n_masked, DEV, max_vocab=V, max_block=n_blk)
    d_embed, d_wlm, d_gain = ab.to_device_bf16(embed, DEV), ab.to_device_bf16(w_lm, DEV), ab.to_device_bf16(gain, DEV)
    ya = torch.zeros((B, K + P, shape.hidden), dtype=torch.bfloat16, device=DEV)
    yb = torch.zeros_like(ya)
    token = torch.zeros((B, n_blk), dtype=torch.int32, device=DEV)
    conf = torch.zeros((B, n_blk), dtype=torch.float32, device=DEV)
    commit = torch.zeros((B, n_blk), dtype=torch.int32, device=DEV)
    left = torch.zeros((B,), dtype=torch.int32, device=DEV)

    def device_state():
        nb = 1 if shared else B
        dk = [ab.to_device_bf16(np.stack([caches[b][n][0] for b in range(nb)]), DEV) for n in range(n_layers)]
        dv = [ab.to_device_bf16(np.stack([caches[b][n][1] for b in range(nb)]), DEV) for n in range(n_layers)]
        d_ids = torch.from_numpy(ids.copy()).to(DEV)
        req_r = ab.Context.request(B, T, l, L, masked, extra, dcos, dsin, token_ids=d_ids, n_embed=V)
        req_d = ab.Context.request(B, T, l, L, masked, d_block, dcos, dsin, token_ids=d_ids, n_embed=V)
        if shared:
            kvs = [ab.KV(dk[n].data_ptr(), dv[n].data_ptr(), 0, T) for n in range(n_layers)]
        else:
            kvs = [ab.Context.kv(dk[n], dv[n]) for n in range(n_layers)]
        return dk, dv, kvs, d_ids, req_r, req_d

    def slots():
        z = lambda: [torch.zeros((B, K + P, shape.n_kv_heads, shape.head_dim), dtype=torch.bfloat16, device=DEV)
                     for _ in range(n_layers)]
        return z(), z()

    def one_step(refresh, kvs, req_r, req_d, ks, vs):
        if not shared:
            ctx.denoise_step(lws, kvs, req_r if refresh else req_d, d_embed, d_anchors if refresh else None,
                             K if refresh else 0, ya, yb, rows_r if refresh else rows_d, n_blk, d_gain, d_wlm, V, threshold,
                             token, conf, commit)
        elif refresh:
            ctx.denoise_step_shared(lws, kvs, req_r, d_embed, d_anchors, K, ks, vs, ya, yb, rows_r, n_blk, d_gain, d_wlm, V,
                                    threshold, token, conf, commit)
        else:
            ctx.decode_step_shared(lws, kvs, req_d, req_r, d_embed, d_anchors, K, rows_r, ks, vs, ya, yb, rows_d, n_blk,
                                   d_gain, d_wlm, V, threshold, token, conf, commit)

    # ---- stepwise on the GPU, the oracle teacher-forced with the GPU's token state
    dk, dv, kvs, d_ids, req_r, req_d = device_state()
    ks, vs = slots()
    ref_ids = ids.copy()
    ref_caches = [list(caches[b]) for b in range(B)]
    steps_gpu = 0
    for step in range(2 * n_blk):
        refresh = step == 0
        one_step(refresh, kvs, req_r, req_d, ks, vs)
        ctx.commit_update(d_ids, T, d_block, B, n_blk, token, conf, MASK, threshold, left)
        torch.cuda.synchronize()
        steps_gpu += 1
        ids_gpu, tok_gpu, conf_gpu = d_ids.cpu().numpy(), token.cpu().numpy(), conf.cpu().numpy()
        for b in range(B):
            a_idx, ex = (anchors[b], lay.extra_rows[b]) if refresh else (np.zeros(0, np.int64), block[b])
            rows, ref_caches[b], ys = orc.refresh_forward(layers, shape, embed[ref_ids[b]], ref_caches[b], T, l, a_idx, ex, cos, sin)
            pos_row = {int(p): i for i, p in enumerate(rows)}
            h = ys[-1][[pos_row[int(p)] for p in block[b]]]
            tok_ref, conf_ref, _, z = orc.predict_commit(h, gain, w_lm, shape.rms_eps, threshold)
            assert np.allclose(conf_gpu[b], conf_ref, rtol=5e-2, atol=2e-3), (step, b)
            zs = np.sort(z, axis=1)
            clear = (zs[:, -1] - zs[:, -2]) > 0.05 * np.abs(zs[:, -1])
            assert np.array_equal(tok_gpu[b][clear], tok_ref[clear]), (step, b)
            was_masked = np.array([ref_ids[b][p] == MASK for p in block[b]])
            now_masked = np.array([ids_gpu[b][p] == MASK for p in block[b]])
            newly = was_masked & ~now_masked
            assert not np.any(~was_masked & (ids_gpu[b][block[b]] != ref_ids[b][block[b]])), "a decoded position changed"
            if was_masked.any():
                assert newly.any(), "a step must commit at least one position"
                assert np.array_equal(ids_gpu[b][block[b]][newly], tok_gpu[b][newly])
                if np.any(conf_ref[was_masked] > threshold + band):      # the threshold rule applies
                    assert np.all(conf_ref[newly] > threshold - band)
                    assert not np.any(was_masked & ~newly & (conf_ref > threshold + band))
                elif not np.any(conf_ref[was_masked] > threshold - band):  # the fallback applies
                    assert newly.sum() == 1 and conf_ref[newly][0] >= conf_ref[was_masked].max() * (1 - band)
            keep = np.setdiff1d(np.arange(T), block[b])
            assert np.array_equal(ids_gpu[b][keep], ref_ids[b][keep]), "a position outside the block changed"
            ref_ids[b] = ids_gpu[b]                              # teacher forcing
        if int(left.sum().item()) == 0:
            break
    assert not np.any(ref_ids[:, block] == MASK) or steps_gpu == 2 * n_blk
    from helpers import TOL, assert_close_bf16, e2e_tol
    final_ids = d_ids.cpu().numpy().copy()
    if shared:
        # the shared caches are untouched; every private slot row holds what the oracle's cache holds at its position
        final_k = [ab.to_host_bits(t) for t in ks]
        for n in range(n_layers):
            assert np.array_equal(ab.to_host_bits(dk[n])[0], caches[0][n][0]) and np.array_equal(ab.to_host_bits(dv[n])[0], caches[0][n][1])
            for b in range(B):
                pos = np.concatenate([l + anchors[b], lay.extra_rows[b]])
                assert_close_bf16(final_k[n][b], ref_caches[b][n][0][pos], f"layer {n} private K slots after the block", e2e_tol(n_layers))
                assert_close_bf16(ab.to_host_bits(vs[n])[b], ref_caches[b][n][1][pos], f"layer {n} private V slots after the block", e2e_tol(n_layers))
    else:
        final_k = [ab.to_host_bits(t) for t in dk]
        for b in range(B):
            for n in range(n_layers):
                assert_close_bf16(final_k[n][b], ref_caches[b][n][0], f"layer {n} K cache after the block", e2e_tol(n_layers))
    assert ctx.poll_status() == 0

    # ---- the C loop reproduces the stepwise run bit for bit
    dk, dv, kvs, d_ids, req_r, req_d = device_state()
    ks, vs = slots()
    if shared:
        steps = ctx.generate_block_shared(lws, kvs, req_r, req_d, d_embed, d_anchors, K, ks, vs, ya, yb, rows_r, rows_d, n_blk,
                                          d_gain, d_wlm, V, threshold, MASK, 2 * n_blk, token, conf, commit, left)
    else:
        steps = ctx.generate_block(lws, kvs, req_r, req_d, d_embed, d_anchors, K, ya, yb, rows_r, rows_d, n_blk, d_gain, d_wlm, V,
                                   threshold, MASK, 2 * n_blk, token, conf, commit, left)
    torch.cuda.synchronize()
    assert steps == steps_gpu
    assert np.array_equal(d_ids.cpu().numpy(), final_ids)
    assert left.cpu().numpy().tolist() == [0] * B
    for n in range(n_layers):
        assert np.array_equal(ab.to_host_bits(ks[n] if shared else dk[n]), final_k[n])
    assert ctx.poll_status() == 0


def test_decode_over_shared_storage_flags_a_bad_slot_row_and_rejects_mismatched_requests():
    """A slot row outside the slot array raises the bad-index flag and that row's K/V is not stored (the
    other rows are); requests that describe different contexts are refused before anything is enqueued."""
    shape, n_layers, B, n_blk, ratio = MID128, 1, 2, 8, 0.25
    lay, layers, embed, w_lm, gain, ids, caches, cos, sin = small_model(shape, n_layers, B, 77)
    T, l, L, P = lay.ctx_len, lay.affix_start, lay.affix_len, lay.n_extra
    K = orc.k_from_ratio(L, ratio)
    g = np.random.default_rng(2)
    anchors = torch.from_numpy(np.stack([np.sort(g.choice(L, K, replace=False)) for _ in range(B)]).astype(np.int32)).to(DEV)
    block = np.stack([lay.masked_pos[b][:n_blk] for b in range(B)]).astype(np.int32)
    where = {int(p): i for i, p in enumerate(lay.extra_rows[0])}
    rows_r = np.stack([[K + where[int(p)] for p in block[b]] for b in range(B)]).astype(np.int32)
    bad_rows = rows_r.copy()
    bad_rows[1, 2] = K + P                     # one past the end of the slot array
    w = {k: (ab.to_device_bf16(v, DEV) if v is not None else None) for k, v in layers[0].items()}
    lw = ab.Context.weights(w)
    dcos, dsin = torch.from_numpy(cos).to(DEV), torch.from_numpy(sin).to(DEV)
    masked, extra = torch.from_numpy(lay.masked_pos.copy()).to(DEV), torch.from_numpy(lay.extra_rows.copy()).to(DEV)
    d_block = torch.from_numpy(block).to(DEV)
    dk, dv = ab.to_device_bf16(caches[0][0][0][None], DEV), ab.to_device_bf16(caches[0][0][1][None], DEV)
    kv = ab.KV(dk.data_ptr(), dv.data_ptr(), 0, T)
    req_s = ab.Context.request(B, T, l, L, masked, extra, dcos, dsin)
    req_r = ab.Context.request(B, T, l, L, masked, d_block, dcos, dsin)
    ctx = ab.Context.for_shape(shape, B, T, L, K + P, lay.n_masked, DEV)
    ks = torch.zeros((B, K + P, shape.n_kv_heads, shape.head_dim), dtype=torch.bfloat16, device=DEV)
    vs = torch.zeros_like(ks)
    x = ab.to_device_bf16(wl.normal_bf16(3, (B, n_blk, shape.hidden), 1.0), DEV)
    y = torch.zeros((B, n_blk, shape.hidden), dtype=torch.bfloat16, device=DEV)
    ctx.recompute_rows_shared(lw, req_r, req_s, kv, x, 1, anchors, K, torch.from_numpy(bad_rows).to(DEV), ks, vs, y)
    torch.cuda.synchronize()
    assert ctx.poll_status() & ab.FLAG_BAD_INDEX
    kb = ab.to_host_bits(ks)
    written = np.zeros((B, K + P), dtype=bool)
    for b in range(B):
        for i in range(n_blk):
            if not (b == 1 and i == 2):
                written[b, rows_r[b, i]] = True
    assert np.all(kb[~written] == 0), "a row outside the block's slots was written"
    assert all(np.any(kb[b, r] != 0) for b in range(B) for r in np.flatnonzero(written[b])), "a block row was not stored"
    # a request pair that disagrees on the context is refused
    req_other = ab.Context.request(B, T, l, L - 1, masked, d_block, dcos, dsin)
    with pytest.raises(ab.AcacheError):
        ctx.recompute_rows_shared(lw, req_other, req_s, kv, x, 1, anchors, K, torch.from_numpy(rows_r).to(DEV), ks, vs, y)
    # and so is a cache with one copy per request where the call wants nothing written: allowed (reads only) -- but a
    # NULL slot_rows is not
    with pytest.raises(ab.AcacheError):
        ctx.recompute_rows_shared(lw, req_r, req_s, kv, x, 1, anchors, K, None, ks, vs, y)
    assert ctx.poll_status() == 0
