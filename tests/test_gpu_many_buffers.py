"""A model with more weight matrices and caches than the library keeps TMA descriptors for: the
descriptor caches (one per tensor rank) then replace entries all the time, and every launch must
still get the descriptors of its own operands.  1200 layer-steps over 600 distinct weight sets and
caches (device copies of four seeded sets) must give, bit for bit, the output of the first
layer-step with the same seeded set, and that one is checked against the oracle."""
import numpy as np
import pytest
import torch

from oracle import acache_oracle as orc
from paper_2608_26140_b200 import binding as ab
from paper_2608_26140_b200 import workloads as wl

from helpers import DEV, assert_close_bf16

pytestmark = pytest.mark.gpu

MID128 = wl.LayerShape(512, 4, 2, 128, 1024, 1e-5, True, 5e5, "mid-d128")


def test_outputs_do_not_depend_on_descriptor_cache_state():
    shape, B, n_sets, n_inst = MID128, 2, 4, 600
    lay = wl.make_layout(B, 4, 2200, 20, 32, 32, "all")     # 2048+ keys: the tcgen05 score kernels run too
    ratio = 0.1
    K = orc.k_from_ratio(lay.affix_len, ratio)
    n = K + lay.n_extra
    cases = [wl.make_case(shape, lay, ratio, cfg_id=40 + i) for i in range(n_sets)]
    g = np.random.default_rng(3)
    anchors_h = np.stack([np.sort(g.choice(lay.affix_len, K, replace=False)) for _ in range(B)]).astype(np.int32)
    anchors = torch.from_numpy(anchors_h).to(DEV)
    base_w = [{k: (ab.to_device_bf16(v, DEV) if v is not None else None) for k, v in c.weights.items()} for c in cases]
    base_k = [ab.to_device_bf16(c.cache_k, DEV) for c in cases]
    base_v = [ab.to_device_bf16(c.cache_v, DEV) for c in cases]
    xs = [ab.to_device_bf16(c.x, DEV) for c in cases]
    c0 = cases[0]
    cos, sin = torch.from_numpy(c0.rope_cos).to(DEV), torch.from_numpy(c0.rope_sin).to(DEV)
    masked = torch.from_numpy(lay.masked_pos).to(DEV)
    extra = torch.from_numpy(lay.extra_rows).to(DEV)
    req = ab.Context.request(B, lay.ctx_len, lay.affix_start, lay.affix_len, masked, extra, cos, sin)
    ctx = ab.Context.for_shape(shape, B, lay.ctx_len, lay.affix_len, n, lay.n_masked, DEV)
    scores = torch.zeros((B, lay.affix_len), dtype=torch.float32, device=DEV)
    y = torch.zeros((B, n, shape.hidden), dtype=torch.bfloat16, device=DEV)

    first_y, first_k, first_s = {}, {}, {}
    keep_alive = []
    for i in range(2 * n_inst):
        s = i % n_sets
        if i < n_inst:        # a distinct copy of everything: new addresses, hence new descriptors
            w = {k: (v.clone() if v is not None else None) for k, v in base_w[s].items()}
            ck, cv = base_k[s].clone(), base_v[s].clone()
            keep_alive.append((w, ck, cv))
        else:                 # second round over the same buffers: lookups now hit or miss depending on the cache state
            w, ck, cv = keep_alive[i - n_inst]
            ck.copy_(base_k[s]); cv.copy_(base_v[s])
        ctx.layer_step(ab.Context.weights(w), req, ab.Context.kv(ck, cv), xs[s], 0, ratio, ab.F_SCORE, scores, anchors, y)
        torch.cuda.synchronize()
        yb, kb, sb = ab.to_host_bits(y), ab.to_host_bits(ck), scores.cpu().numpy().copy()
        if s not in first_y:
            first_y[s], first_k[s], first_s[s] = yb, kb, sb
        else:
            assert np.array_equal(yb, first_y[s]) and np.array_equal(kb, first_k[s]) and np.array_equal(sb, first_s[s]), i
    assert ctx.poll_status() == 0
    # the first set against the oracle
    for b in range(B):
        ref = orc.layer_step(c0.weights, shape, c0.x[b], c0.cache_k[b], c0.cache_v[b], lay.ctx_len, lay.affix_start,
                             lay.affix_len, lay.masked_pos[b], lay.extra_rows[b], c0.rope_cos, c0.rope_sin,
                             anchor_idx=anchors_h[b])
        assert_close_bf16(first_y[0][b], ref["y"], "y")
        assert_close_bf16(first_k[0][b][ref["rows"]], ref["k_new"], "K rows")


def test_deep_model_passes_are_reproducible_and_equal_layer_by_layer_calls():
    """64 layers with their own weight and cache buffers (hundreds of descriptors per pass): the C loops
    acache_denoise_step and acache_denoise_step_shared must give, bit for bit, what single-layer calls
    chained by hand give, and the same again on a second pass."""
    shape, B, n_layers, V, n_blk = MID128, 3, 64, 256, 8
    lay = wl.make_layout(B, 0, 300, 20, 32, 32, "all")
    ratio = 0.3
    T, l, L, P = lay.ctx_len, lay.affix_start, lay.affix_len, lay.n_extra
    K = orc.k_from_ratio(L, ratio)
    n = K + P
    sets = [wl.make_case(shape, lay, ratio, cfg_id=60 + i) for i in range(3)]
    base_w = [{k: (ab.to_device_bf16(v, DEV) if v is not None else None) for k, v in c.weights.items()} for c in sets]
    ws = [{k: (v.clone() if v is not None else None) for k, v in base_w[i % 3].items()} for i in range(n_layers)]
    lws = [ab.Context.weights(w) for w in ws]
    ck0 = [ab.to_device_bf16(c.cache_k, DEV) for c in sets]
    cv0 = [ab.to_device_bf16(c.cache_v, DEV) for c in sets]
    g = np.random.default_rng(11)
    anchors = torch.from_numpy(np.stack([np.sort(g.choice(L, K, replace=False)) for _ in range(B)]).astype(np.int32)).to(DEV)
    where = {int(p): i for i, p in enumerate(lay.extra_rows[0])}
    rows_blk = torch.from_numpy(np.stack([[K + where[int(p)] for p in lay.masked_pos[b][:n_blk]] for b in range(B)]).astype(np.int32)).to(DEV)
    cos, sin = torch.from_numpy(sets[0].rope_cos).to(DEV), torch.from_numpy(sets[0].rope_sin).to(DEV)
    masked, extra = torch.from_numpy(lay.masked_pos).to(DEV), torch.from_numpy(lay.extra_rows).to(DEV)
    req = ab.Context.request(B, T, l, L, masked, extra, cos, sin)
    ctx = ab.Context.for_shape(shape, B, T, L, n, lay.n_masked, DEV, max_vocab=V, max_block=n_blk)
    x0 = ab.to_device_bf16(sets[0].x, DEV)
    w_lm = ab.to_device_bf16(wl.normal_bf16(5, (V, shape.hidden), 0.3), DEV)
    gain = ab.to_device_bf16(wl.normal_bf16(6, (shape.hidden,), 0.05, 1.0), DEV)
    ya, yb = (torch.zeros((B, n, shape.hidden), dtype=torch.bfloat16, device=DEV) for _ in range(2))
    token = torch.zeros((B, n_blk), dtype=torch.int32, device=DEV)
    conf = torch.zeros((B, n_blk), dtype=torch.float32, device=DEV)
    commit = torch.zeros((B, n_blk), dtype=torch.int32, device=DEV)

    def fresh_caches():
        dk = [ck0[i % 3].clone() for i in range(n_layers)]
        dv = [cv0[i % 3].clone() for i in range(n_layers)]
        return dk, dv

    # private caches: C loop twice, then by hand
    results = []
    for mode in ("loop", "loop", "by hand"):
        dk, dv = fresh_caches()
        kvs = [ab.Context.kv(dk[i], dv[i]) for i in range(n_layers)]
        if mode == "loop":
            last = ctx.denoise_step(lws, kvs, req, x0, anchors, K, ya, yb, rows_blk, n_blk, gain, w_lm, V, 0.9, token, conf, commit)
            y_last = ya if last == ya.data_ptr() else yb
        else:
            x, compact = x0, 0
            for i in range(n_layers):
                y = ya if i % 2 == 0 else yb
                ctx.layer_step(lws[i], req, kvs[i], x, compact, ratio, 0, None, anchors, y)
                x, compact = y, 1
            y_last = x
            ctx.predict_commit(y_last, n, rows_blk, B, n_blk, gain, w_lm, V, 0.9, token, conf, commit)
        torch.cuda.synchronize()
        results.append((ab.to_host_bits(y_last).copy(), token.cpu().numpy().copy(), conf.cpu().numpy().copy(),
                        ab.to_host_bits(dk[n_layers - 1]).copy()))
    for r in results[1:]:
        for a, b in zip(results[0], r):
            assert np.array_equal(a, b)
    assert np.isfinite(results[0][2]).all()

    # shared storage: C loop twice, then by hand
    ks = [torch.zeros((B, n, shape.n_kv_heads, shape.head_dim), dtype=torch.bfloat16, device=DEV) for _ in range(n_layers)]
    vs = [torch.zeros_like(t) for t in ks]
    sk = [ck0[i % 3][0:1].clone() for i in range(n_layers)]
    sv = [cv0[i % 3][0:1].clone() for i in range(n_layers)]
    kvs = [ab.KV(sk[i].data_ptr(), sv[i].data_ptr(), 0, T) for i in range(n_layers)]
    shared = []
    for mode in ("loop", "loop", "by hand"):
        for t in ks + vs:
            t.zero_()
        if mode == "loop":
            last = ctx.denoise_step_shared(lws, kvs, req, x0, anchors, K, ks, vs, ya, yb, rows_blk, n_blk, gain, w_lm, V, 0.9,
                                           token, conf, commit)
            y_last = ya if last == ya.data_ptr() else yb
        else:
            x, compact = x0, 0
            for i in range(n_layers):
                y = ya if i % 2 == 0 else yb
                ctx.recompute_anchors(lws[i], req, kvs[i], x, compact, anchors, K, ks[i], vs[i], y)
                x, compact = y, 1
            y_last = x
            ctx.predict_commit(y_last, n, rows_blk, B, n_blk, gain, w_lm, V, 0.9, token, conf, commit)
        torch.cuda.synchronize()
        shared.append((ab.to_host_bits(y_last).copy(), token.cpu().numpy().copy(), conf.cpu().numpy().copy(),
                       ab.to_host_bits(ks[n_layers - 1]).copy()))
    for r in shared[1:]:
        for a, b in zip(shared[0], r):
            assert np.array_equal(a, b)
    assert ctx.poll_status() == 0
