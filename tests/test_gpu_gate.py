"""GPU parity of the gate projection (Eq. 1) and its gradients against the CPU oracle."""
import numpy as np
import pytest
import torch

from paper_2402_12399_b200 import synth

pytestmark = pytest.mark.gpu

# bf16 products are exact and summed in fp32 on both the tensor cores (forward) and the CUDA cores
# (backward): 1e-4 x RMS leaves room for the order of d (or T) fp32 additions.  fp32 inputs go
# through tf32 in the forward pass: both operands are cut to 10 mantissa bits, each product is off
# by up to 2^-9 of itself, and the largest of T*E sums of d such errors stays below 2^-7 x RMS
TOL_BF16, TOL_TF32, TOL_BWD = 1e-4, 2.0 ** -7, 1e-4


def _inputs(T, E, d, seed, dtype):
    rng = np.random.default_rng(seed)
    h = rng.standard_normal((T, d)).astype(np.float32)
    w = (rng.standard_normal((E, d)) / np.sqrt(d)).astype(np.float32)
    if dtype == "bf16":
        return synth.to_bf16_bits(h), synth.to_bf16_bits(w)
    return h, w


def _dev(a, dtype):
    import helpers
    return helpers.to_torch(a, dtype)


def _ratio(got, want, tol, what):
    rms = float(np.sqrt((want ** 2).mean()))
    err = float(np.abs(np.asarray(got, np.float64) - want).max())
    assert err <= tol * rms, f"{what}: max err {err:.3e} vs rms {rms:.3e} (ratio {err / rms:.2e})"


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("T,E,d", [(1, 1, 64), (300, 8, 128), (1000, 64, 256), (777, 5, 192), (2048, 256, 64),
                                   (129, 130, 320)])
def test_forward_and_backward_small(T, E, d, dtype):
    import paper_2402_12399_b200 as rr
    from oracle import rr_oracle as orc
    h, w = _inputs(T, E, d, 10 + T + E, dtype)
    hd, wd = _dev(h, dtype), _dev(w, dtype)
    a = rr.gate_fwd(hd, wd)
    rr.check(a._workspace)
    want = orc.gate_fwd(h, w)
    _ratio(a.cpu().numpy(), want, TOL_BF16 if dtype == "bf16" else TOL_TF32, "logits")

    rng = np.random.default_rng(3)
    dl = rng.standard_normal((T, E)).astype(np.float32)
    base = rng.standard_normal((T, d)).astype(np.float32)      # dhidden is added to
    dh = torch.from_numpy(base.copy()).cuda()
    dW = rr.gate_bwd(torch.from_numpy(dl).cuda(), hd, wd, dh)
    torch.cuda.synchronize()
    want_dW, want_dh = orc.gate_bwd(dl.astype(np.float64), h, w)
    _ratio(dW.cpu().numpy(), want_dW, TOL_BWD, "dWg")
    _ratio(dh.cpu().numpy() - base.astype(np.float64), want_dh, TOL_BWD * 10, "dhidden increment")


def test_forward_feeds_the_router():
    # logits made by the projection go straight into rr_route: same device buffer, no copy
    import helpers
    import paper_2402_12399_b200 as rr
    from oracle import rr_oracle as orc
    T, E, d = 4096, 16, 256
    h, w = _inputs(T, E, d, 5, "bf16")
    a = rr.gate_fwd(_dev(h, "bf16"), _dev(w, "bf16"))
    tg = rr.route(a, 2, 512, 4, 3)
    rr.check(tg._workspace)
    tc = orc.route(a.cpu().numpy(), 2, 512, 4, 3)     # the oracle routes the same fp32 logits
    helpers.assert_tables_equal(tg, tc, "tables from projected logits")


@pytest.mark.parametrize("name", ["c3", "c5"])
def test_full_size_sampled(name):
    import paper_2402_12399_b200 as rr
    from oracle import rr_oracle as orc
    w_ = synth.WORKLOADS[name]
    T, E, d = w_.T, w_.E, w_.d
    h, w = _inputs(T, E, d, 77, "bf16")
    hd, wd = _dev(h, "bf16"), _dev(w, "bf16")
    a = rr.gate_fwd(hd, wd)
    rr.check(a._workspace)
    rows = np.sort(np.random.default_rng(1).choice(T, 256, replace=False))
    _ratio(a.cpu().numpy()[rows], orc.gate_fwd(np.ascontiguousarray(h[rows]), w), TOL_BF16, "logits (sampled tokens)")
    # repeatable bit for bit (plain stores in the forward, fixed summation order in dWg)
    a2 = rr.gate_fwd(hd, wd)
    assert torch.equal(a, a2)
    dl = torch.randn(T, E, device="cuda")
    dh1, dh2 = torch.zeros(T, d, device="cuda"), torch.zeros(T, d, device="cuda")
    g1, g2 = rr.gate_bwd(dl, hd, wd, dh1), rr.gate_bwd(dl, hd, wd, dh2)
    assert torch.equal(g1, g2) and torch.equal(dh1, dh2)
    want_dW, _ = orc.gate_bwd(dl.cpu().numpy().astype(np.float64), h, w)
    _ratio(g1.cpu().numpy(), want_dW, TOL_BWD, "dWg")
    _, want_dh = orc.gate_bwd(dl.cpu().numpy()[rows].astype(np.float64), np.ascontiguousarray(h[rows]), w)
    _ratio(dh1.cpu().numpy()[rows], want_dh, TOL_BWD * 10, "dhidden (sampled tokens)")


def test_bad_arguments_are_refused():
    import paper_2402_12399_b200 as rr
    h = torch.zeros(8, 96, dtype=torch.bfloat16, device="cuda")      # d not a multiple of 64
    w = torch.zeros(4, 96, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(rr.RRError):
        rr.gate_fwd(h, w)
