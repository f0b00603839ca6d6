"""The give-up path of the bounded waits.  Every wait inside the kernels has a time limit after which the
kernel latches RR_ERR_TIMEOUT, lets go of what it holds (barrier words, TMEM, copies in flight) and
returns; the CUDA context stays usable.  With the testing aid rr_test_set_wait_limit_ns the limit is set
to one nanosecond, so waits run out while the awaited work is still under way -- nothing is broken,
nothing hangs -- and the next ordinary call must be exact again."""
import numpy as np
import pytest
import torch

from paper_2402_12399_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture
def short_waits():
    import paper_2402_12399_b200 as rr
    rr.test_set_wait_limit_ns(1)
    yield rr
    rr.test_set_wait_limit_ns(0)


def test_router_grid_barrier_gives_up_and_recovers(short_waits):
    import helpers
    from oracle import rr_oracle as orc
    rr = short_waits
    w = synth.WORKLOADS["c2"]
    a_np = synth.make_logits(w.T, w.E, w.bias, 77)
    a = torch.from_numpy(a_np).cuda()
    C = w.capacity(1.0)
    t = rr.route(a, w.k, C, w.G, 3)
    with pytest.raises(rr.RRError) as ei:
        rr.check(t._workspace)
    assert ei.value.code == 6                      # a block waited longer than 1 ns at a grid barrier
    rr.test_set_wait_limit_ns(0)
    # the kernel has put its barrier words back: the same workspace and tables serve the next call
    rr.route(a, w.k, C, w.G, 3, tables=t, workspace=t._workspace)
    rr.check(t._workspace)
    helpers.assert_tables_equal(t, orc.route(a_np, w.k, C, w.G, 3), "after a timed-out call")


def test_gemm_epilogue_wait_gives_up_and_recovers(short_waits):
    import helpers
    from oracle import rr_oracle as orc
    rr = short_waits
    T, E, k, G, d, d_ff, C = 1024, 4, 1, 2, 512, 1024, 256
    L = synth.make_layer(T, E, d, d_ff, ("normal", 0.5), 5, "bf16", w_std=0.05)
    hid, W1, W3, W2 = (helpers.to_torch(x, "bf16") for x in (L.hidden, L.W1, L.W3, L.W2))
    logits = torch.from_numpy(L.logits).cuda()
    rr.test_set_wait_limit_ns(0)
    tab = rr.route(logits, k, C, G, 3)
    rr.check(tab._workspace)
    rr.test_set_wait_limit_ns(1)
    out = rr.moe_fwd(hid, W1, W3, W2, logits, tab)
    with pytest.raises(rr.RRError) as ei:
        rr.check(out._workspace)
    assert ei.value.code == 6                      # the epilogue gave up on its accumulators
    rr.test_set_wait_limit_ns(0)
    out = rr.moe_fwd(hid, W1, W3, W2, logits, tab, out=out, workspace=out._workspace)
    rr.check(out._workspace)
    tc = orc.route(L.logits, k, C, G, 3)
    want = orc.forward_tokens(L.hidden, L.W1, L.W3, L.W2, L.logits, tc)
    rms = float(np.sqrt((want ** 2).mean()))
    assert float(np.abs(out.cpu().numpy() - want).max()) <= 2e-2 * rms
