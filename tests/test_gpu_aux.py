"""GPU parity of the load-balance loss (rr_aux_loss_fwd / rr_aux_loss_bwd) against the fp64 oracle.

Tolerances, from the fp32 arithmetic of the kernels: the counts are integers, so f = count / T is one
rounding away from the oracle's (2^-23 relative); P and L are sums of n = passes + warps + blocks
(< 900 here) non-negative fp32 terms in a fixed order, relative error <= n 2^-24 < 6e-5; a gradient
element is coef g_ij (f_j - sum_e f_e g_ie) with g good to about 1e-6 relative, so its absolute error
is about 2e-6 coef g_ij max(f), checked against 2e-5 of the largest gradient magnitude (the difference
in the bracket cancels up to a factor of ten on balanced routers)."""
import numpy as np
import pytest
import torch

from paper_2402_12399_b200 import synth

pytestmark = pytest.mark.gpu
TOL_F, TOL_P, TOL_G = 2.0 ** -22, 6e-5, 2e-5


def _both(a, k, alpha=1e-2, scale=1.0):
    import helpers
    import paper_2402_12399_b200 as rr
    from oracle import rr_oracle as orc
    T, E = a.shape
    tg, tc = helpers.route_both(a, k, max(1, k * T // E), 1, 0, "aux tables")
    ad = torch.from_numpy(a).cuda()
    loss, f, P = rr.aux_loss_fwd(ad, tg.topk_expert, alpha)
    rr.check(loss._workspace)
    L0, f0, P0 = orc.aux_loss(a, tc.topk_expert, alpha)
    np.testing.assert_allclose(f.cpu().numpy(), f0, rtol=TOL_F, atol=0)
    np.testing.assert_allclose(P.cpu().numpy(), P0, rtol=TOL_P, atol=0)
    assert abs(float(loss) - L0) <= TOL_P * L0, (float(loss), L0)
    g = rr.aux_loss_bwd(ad, f, alpha, scale)
    g0 = orc.aux_loss_bwd(a, f0, alpha, scale)
    err = float(np.abs(g.cpu().numpy() - g0).max())
    assert err <= TOL_G * float(np.abs(g0).max()) + 1e-30, (err, float(np.abs(g0).max()))
    return ad, f, g, g0


@pytest.mark.parametrize("E,k", [(1, 1), (2, 1), (3, 2), (5, 1), (8, 2), (12, 2), (16, 1), (24, 3), (32, 2),
                                 (33, 2), (64, 2), (100, 4), (128, 2), (200, 8), (256, 2)])
def test_small_shapes(E, k):
    for T in (1, 37, 1000, 4099):                 # less than one pass, ragged slabs, several blocks
        a = synth.make_logits(T, E, ("normal", 1.0), 900 + E + T)
        _both(a, k, alpha=0.37, scale=-1.5)


@pytest.mark.parametrize("name", ["c2", "c3", "c4", "c5"])
def test_workload_shapes(name):
    w = synth.WORKLOADS[name]
    a = synth.make_logits(w.T, w.E, w.bias, w.seed(0, w.mode))
    _both(a, w.k)


def test_largest_router_size():
    _both(synth.make_logits(1 << 20, 64, ("normal", 0.5), 3), 2)


def test_uniform_scores_give_alpha():
    import paper_2402_12399_b200 as rr
    a = torch.full((5000, 8), 0.75, device="cuda")
    te = torch.zeros(5000, 3, dtype=torch.int32, device="cuda")
    loss, f, P = rr.aux_loss_fwd(a, te, 0.01)
    assert abs(float(loss) - 0.01) < 1e-7 and f.tolist() == [1.0] + [0.0] * 7
    g = rr.aux_loss_bwd(a, f, 0.01)
    want = 0.01 / 5000 * (f.cpu().numpy() - 0.125)                      # closed form at g = 1/E
    np.testing.assert_allclose(g.cpu().numpy(), np.broadcast_to(want, (5000, 8)), rtol=1e-5, atol=1e-12)


def test_accumulate_adds_onto_existing_gradient():
    import paper_2402_12399_b200 as rr
    a = synth.make_logits(3000, 64, ("normal", 0.7), 11)
    ad, f, g, _ = _both(a, 2, alpha=1.0)
    base = torch.randn_like(g) * float(g.abs().max())
    acc = base.clone()
    out = rr.aux_loss_bwd(ad, f, 1.0, 1.0, dlogits=acc, accumulate=True)
    assert out is acc and torch.equal(acc, base + g)


def test_repeats_bit_for_bit():
    import paper_2402_12399_b200 as rr
    w = synth.WORKLOADS["c2"]
    a = torch.from_numpy(synth.make_logits(w.T, w.E, w.bias, 5)).cuda()
    t = rr.route(a, w.k, w.capacity(1.0), w.G, 3)
    ref = None
    ws = None
    for _ in range(5):
        loss, f, P = rr.aux_loss_fwd(a, t.topk_expert, 1e-2, workspace=ws)
        ws = loss._workspace
        cur = torch.cat([loss, f, P, rr.aux_loss_bwd(a, f, 1e-2).flatten()])
        if ref is None:
            ref = cur.clone()
        assert torch.equal(cur, ref)
    rr.check(ws)


def test_no_tokens_and_bad_arguments():
    import paper_2402_12399_b200 as rr
    a = torch.zeros(0, 8, device="cuda")
    te = torch.zeros(0, 3, dtype=torch.int32, device="cuda")
    loss, f, P = rr.aux_loss_fwd(a, te, 1.0)
    assert float(loss) == 0.0 and float(f.abs().sum()) == 0.0 and float(P.abs().sum()) == 0.0
    assert rr.aux_loss_bwd(a, f, 1.0).shape == (0, 8)
    a = torch.zeros(64, 8, device="cuda")
    te = torch.zeros(64, 3, dtype=torch.int32, device="cuda")
    with pytest.raises(rr.RRError) as ei:
        rr.aux_loss_fwd(a, te, 1.0, workspace=torch.zeros(256, dtype=torch.uint8, device="cuda"))
    assert ei.value.code == 3
    with pytest.raises(rr.RRError) as ei:
        rr.aux_loss_fwd(torch.zeros(4, 257, device="cuda"), te[:4], 1.0)
    assert ei.value.code == 1
    # a first choice outside 0..E-1 is reported through the status word, and skipped
    te[5, 0] = 8
    te[6, 0] = -1
    loss, f, _ = rr.aux_loss_fwd(a, te, 1.0)
    with pytest.raises(rr.RRError) as ei:
        rr.check(loss._workspace)
    assert ei.value.code == 1
    assert abs(float(f.sum()) - 62 / 64) < 1e-6


@pytest.mark.parametrize("T,E,k,G", [(2048, 8, 1, 2), (4096, 64, 2, 8), (3000, 24, 3, 2), (5000, 40, 2, 5), (65536, 64, 2, 8),
                                     (999, 7, 2, 1)])
def test_route_loss_in_the_routing_kernel(T, E, k, G):
    """rr_route_loss: the routing kernel's pass over the logits also adds up the softmax values, the first
    choices come from its totals.  Tables as rr_route (bit-exact against the oracle), f / P / L within the
    tolerances of the separate loss kernels, and bit-repeatable."""
    import helpers
    import paper_2402_12399_b200 as rr
    from oracle import rr_oracle as orc
    T = T // G * G
    a = synth.make_logits(T, E, ("normal", 1.0), 90 + E)
    C = max(1, k * T // E)
    for mode in (0, 3):
        if (mode & 2) and k >= E:
            continue
        tab, (loss, f, P) = rr.route_loss(torch.from_numpy(a).cuda(), k, C, G, mode, 1e-2)
        rr.check(tab._workspace)
        tc = orc.route(a, k, C, G, mode)
        helpers.assert_tables_equal(tab, tc, f"route_loss T{T} E{E} mode{mode}")
        L0, f0, P0 = orc.aux_loss(a, tc.topk_expert, 1e-2)
        np.testing.assert_allclose(f.cpu().numpy().astype(np.float64), f0, rtol=2.0 ** -22, atol=0)
        np.testing.assert_allclose(P.cpu().numpy().astype(np.float64), P0, rtol=6e-5, atol=1e-9)
        assert abs(float(loss) - L0) <= 6e-5 * L0
        tab2, (loss2, f2, P2) = rr.route_loss(torch.from_numpy(a).cuda(), k, C, G, mode, 1e-2)
        assert torch.equal(loss, loss2) and torch.equal(P, P2) and torch.equal(f, f2)
