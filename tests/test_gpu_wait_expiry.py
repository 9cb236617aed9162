"""Failure detection on the device without a fault: a bounded wait inside a kernel is made to run out
(acache_debug_expire_next_wait gives one grid-wide barrier a target it cannot reach and a short poll
limit), and the test checks what the library promises for that case: the kernel returns, the status word
carries ACACHE_FLAG_WAIT_EXPIRED, acache_poll_status answers ACACHE_ERR_TIMEOUT and re-arms the barrier,
and the very next call on the same context gives the bits of a clean run."""
import numpy as np
import pytest
import torch

from oracle import acache_oracle as orc
from paper_2608_26140_b200 import binding as ab
from paper_2608_26140_b200 import workloads as wl

from helpers import DEV, DeviceCase
from test_gpu_parity import MID128, dev_i32

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,L,extra", [
    (1, 300, "none"),      # 60 rows: one CTA per tile, ring stages filled with weights before the barrier
    (2, 400, "all"),       # several 128-row tiles: the two-SM projection kernel
])
def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable(B, L, extra):
    lay = wl.make_layout(B, 4, L, 40, 32, 32, extra)
    case = wl.make_case(MID128, lay, 0.2, cfg_id=17)
    dc = DeviceCase(case)
    K = orc.k_from_ratio(L, 0.2)
    n = K + lay.n_extra
    g = np.random.default_rng(1)
    anchors = dev_i32(np.stack([np.sort(g.choice(L, K, replace=False)) for _ in range(B)]))

    def step():
        y = torch.zeros((B, n, MID128.hidden), dtype=torch.bfloat16, device=DEV)
        dc.ctx.layer_step(dc.lw, dc.req, dc.kv(), dc.x, 0, 0.2, 0, None, anchors, y)
        torch.cuda.synchronize()                     # returns: no kernel of the step is stuck
        return ab.to_host_bits(y), ab.to_host_bits(dc.ck), ab.to_host_bits(dc.cv)

    clean = step()
    assert dc.ctx.poll_status_code() == (ab.OK, 0)
    dc.reset_cache()
    dc.ctx.debug_expire_next_wait()
    step()                                           # its outputs are meaningless; only that it ends matters
    code, flags = dc.ctx.poll_status_code()
    assert code == ab.ERR_TIMEOUT and (flags & ab.FLAG_WAIT_EXPIRED)
    assert dc.ctx.poll_status_code() == (ab.OK, 0)   # the poll cleared the word
    dc.reset_cache()
    again = step()
    assert dc.ctx.poll_status_code() == (ab.OK, 0)
    for a, b in zip(clean, again):
        assert np.array_equal(a, b)
