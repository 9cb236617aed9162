"""The allocation-free scoring entry point (for callers that may not call cudaMalloc and so
cannot hand the library a workspace) must give what the ordinary entry point gives.  Runs
last in the suite on purpose; it also passes on its own in a fresh process."""
import numpy as np
import pytest
import torch

from paper_2608_26140_b200 import binding as ab
from paper_2608_26140_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _case(shape, B, pre, L, post, m, seed):
    lay = wl.make_layout(B, pre, L, post, max(m, 1), m)
    ck, _ = wl.random_kv_cache(shape, lay, seed)
    q = wl.random_q_mask(shape, lay, seed + 1)
    dk, dq = ab.to_device_bf16(ck, DEV), ab.to_device_bf16(q, DEV)
    masked = torch.from_numpy(lay.masked_pos.copy()).to(DEV)
    req = ab.Context.request(B, lay.ctx_len, lay.affix_start, L, masked, None, None, None)
    return lay, dk, dq, masked, req


def test_static_scratch_scoring_matches_workspace_scoring_twice_in_a_row():
    shape = wl.LayerShape(512, 4, 2, 128, 1024, 1e-5, False, 5e5, "mid-d128")
    ctx = ab.Context.for_shape(shape, 2, 1024, 700, 1, 130, DEV)
    # two different problems back to back: the second call finds the first call's leftovers in the
    # shared scratch and must not be affected by them
    for (B, pre, L, post, m, norm_full, seed) in [(2, 7, 700, 64, 130, False, 41), (1, 0, 300, 20, 33, True, 43)]:
        lay, dk, dq, masked, req = _case(shape, B, pre, L, post, m, seed)
        kv = ab.Context.kv(dk, dk)
        ref = torch.zeros((B, L), dtype=torch.float32, device=DEV)
        ctx.score_anchors(req, dq, kv, ref, accumulate=False, norm_full=norm_full)
        got = torch.full((B, L), 7.0, dtype=torch.float32, device=DEV)
        st = ab.score_anchors_static(ctx.desc, req, dq, kv, got, accumulate=False, norm_full=norm_full)
        assert st == ab.OK
        torch.cuda.synchronize()
        r, g = ref.cpu().numpy().astype(np.float64), got.cpu().numpy().astype(np.float64)
        err = np.abs(g - r) / np.maximum(r, r.mean())
        assert err.max() < 1e-3, err.max()
        # accumulate on top of the previous result
        st = ab.score_anchors_static(ctx.desc, req, dq, kv, got, accumulate=True, norm_full=norm_full)
        assert st == ab.OK
        torch.cuda.synchronize()
        g2 = got.cpu().numpy().astype(np.float64)
        assert np.abs(g2 - 2 * r).max() <= 2e-3 * np.maximum(r, r.mean()).max()


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
