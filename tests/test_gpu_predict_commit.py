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
