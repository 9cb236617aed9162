"""The allocation-free scoring entry point (for callers that may not call cudaMalloc and so cannot hand the
library a workspace) against the CPU oracle and against the ordinary entry point.

The file name sorts last on purpose: the driver stops at the first failure (`pytest -x`), and a failure of
this one added entry point should not keep any other test from running.  Nothing here depends on the tests
before it: it passes alone in a fresh process as well (the static scratch keeps whatever the last call left
and every call overwrites what it reads)."""
import numpy as np
import pytest
import torch

from oracle import acache_oracle as orc
from paper_2608_26140_b200 import binding as ab
from paper_2608_26140_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
SHAPE = wl.LayerShape(512, 4, 2, 128, 1024, 1e-5, False, 5e5, "mid-d128")


def _case(shape, B, pre, L, post, m, seed):
    lay = wl.make_layout(B, pre, L, post, max(m, 1), m)
    ck, _ = wl.random_kv_cache(shape, lay, seed)
    q = wl.random_q_mask(shape, lay, seed + 1)
    dk, dq = ab.to_device_bf16(ck, DEV), ab.to_device_bf16(q, DEV)
    masked = torch.from_numpy(lay.masked_pos.copy()).to(DEV)
    req = ab.Context.request(B, lay.ctx_len, lay.affix_start, L, masked, None, None, None)
    return lay, ck, q, dk, dq, masked, req


def _oracle_scores(shape, lay, ck, q, b, norm_full, kb=None):
    kf = orc.bf16_bits_to_f64(ck[b if kb is None else kb, :lay.ctx_len])
    l, L = lay.affix_start, lay.affix_len
    return orc.score_anchors(orc.bf16_bits_to_f64(q[b]), kf[l:l + L], kf, l, norm_full)


def _rel(got, ref):
    return (np.abs(got - ref) / np.maximum(ref, ref.mean())).max()


def test_static_scratch_scoring_matches_oracle_and_workspace_scoring_twice_in_a_row():
    ctx = ab.Context.for_shape(SHAPE, 2, 1024, 700, 1, 130, DEV)
    # two different problems back to back: the second call finds the first call's leftovers in the
    # shared scratch and must not be affected by them
    for (B, pre, L, post, m, norm_full, seed) in [(2, 7, 700, 64, 130, False, 41), (1, 0, 300, 20, 33, True, 43)]:
        lay, ck, q, dk, dq, masked, req = _case(SHAPE, B, pre, L, post, m, seed)
        kv = ab.Context.kv(dk, dk)
        ref = torch.zeros((B, L), dtype=torch.float32, device=DEV)
        ctx.score_anchors(req, dq, kv, ref, accumulate=False, norm_full=norm_full)
        got = torch.full((B, L), 7.0, dtype=torch.float32, device=DEV)
        st = ab.score_anchors_static(ctx.desc, req, dq, kv, got, accumulate=False, norm_full=norm_full)
        assert st == ab.OK
        torch.cuda.synchronize()
        g = got.cpu().numpy()
        # below 2048 keys per batch the workspace path runs the same kernels on the same layout: identical bits
        assert np.array_equal(g, ref.cpu().numpy())
        for b in range(B):
            assert _rel(g[b].astype(np.float64), _oracle_scores(SHAPE, lay, ck, q, b, norm_full)) < 1e-3
        # accumulate on top of the previous result
        st = ab.score_anchors_static(ctx.desc, req, dq, kv, got, accumulate=True, norm_full=norm_full)
        assert st == ab.OK
        torch.cuda.synchronize()
        g2 = got.cpu().numpy().astype(np.float64)
        for b in range(B):
            assert _rel(g2[b], 2.0 * _oracle_scores(SHAPE, lay, ck, q, b, norm_full)) < 1e-3


def test_static_scratch_scoring_on_one_cache_shared_by_the_batch():
    """kv.batch_stride = 0 (Section 4.1): every request scores against request 0's copy of the cache."""
    B, L, m = 3, 520, 32
    lay, ck, q, dk, dq, masked, req = _case(SHAPE, B, 16, L, 40, m, 47)
    shared = ab.KV(dk[0:1].data_ptr(), dk[0:1].data_ptr(), 0, lay.ctx_len)
    got = torch.zeros((B, L), dtype=torch.float32, device=DEV)
    assert ab.score_anchors_static(ab.Context.for_shape(SHAPE, B, lay.ctx_len, L, 1, m, DEV).desc, req, dq, shared, got) == ab.OK
    torch.cuda.synchronize()
    g = got.cpu().numpy().astype(np.float64)
    for b in range(B):
        assert _rel(g[b], _oracle_scores(SHAPE, lay, ck, q, b, False, kb=0)) < 1e-3


def test_static_scratch_filled_to_its_last_float():
    """B * H * (2 m ceil(L / 256) + L) = 2^20 floats exactly is accepted and correct; one masked row more is refused."""
    B, L, m = 2, 65536, 128
    assert B * SHAPE.n_heads * (2 * m * ((L + 255) // 256) + L) == 1 << 20
    lay, ck, q, dk, dq, masked, req = _case(SHAPE, B, 0, L, 8, m, 53)
    desc = ab.Context.for_shape(SHAPE, B, lay.ctx_len, L, 1, m + 1, DEV).desc
    kv = ab.Context.kv(dk, dk)
    got = torch.zeros((B, L), dtype=torch.float32, device=DEV)
    assert ab.score_anchors_static(desc, req, dq, kv, got) == ab.OK
    torch.cuda.synchronize()
    g = got.cpu().numpy().astype(np.float64)
    for b in range(B):
        assert _rel(g[b], _oracle_scores(SHAPE, lay, ck, q, b, False)) < 1e-3
    lay2 = wl.make_layout(B, 0, L, 8, m + 1, m + 1)
    masked2 = torch.from_numpy(lay2.masked_pos.copy()).to(DEV)
    q2 = torch.zeros((B, m + 1, SHAPE.n_heads, SHAPE.head_dim), dtype=torch.bfloat16, device=DEV)
    req2 = ab.Context.request(B, lay2.ctx_len, 0, L, masked2, None, None, None)
    dk2 = torch.zeros((B, lay2.ctx_len, SHAPE.n_kv_heads, SHAPE.head_dim), dtype=torch.bfloat16, device=DEV)
    assert ab.score_anchors_static(desc, req2, q2, ab.Context.kv(dk2, dk2), got) == ab.ERR_WORKSPACE


def test_static_scratch_rejects_oversized_problems_without_launching():
    shape = wl.LLADA_8B
    desc = ab.ModelDesc(shape.hidden, shape.n_heads, shape.n_kv_heads, shape.head_dim, shape.ffn, shape.rms_eps, 0,
                        64, 40000, 40000, 1, 32, 0, 0)
    dummy = torch.zeros(1024, dtype=torch.bfloat16, device=DEV)
    masked = torch.zeros((64, 32), dtype=torch.int32, device=DEV)
    req = ab.Context.request(64, 40000, 0, 32768, masked, None, None, None)     # 64 * 32 * 32768 floats >> 2^20
    kv = ab.KV(dummy.data_ptr(), dummy.data_ptr(), 40000 * 32 * 128, 40000)
    out = torch.zeros(16, dtype=torch.float32, device=DEV)
    assert ab.score_anchors_static(desc, req, dummy, kv, out) == ab.ERR_WORKSPACE
    assert ab.score_anchors_static(desc, req, dummy, ab.KV(None, None, 0, 0), out) == ab.ERR_INVALID_ARG
    torch.cuda.synchronize()
