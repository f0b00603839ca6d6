"""One training step through every entry point, in the order a layer calls them:
gate projection (Eq. 1) -> routing with IR and FR (Sections 3-4) -> expert FFN and combine (Eq. 2, 3)
-> load-balance loss (Section 5.1) -> backward of all four.  The total loss is <dout, out> + s L_aux.
The oracle takes the fp32 logits the GPU projection produced (the routing decisions are made on them)
and composes its own functions in fp64; hidden-state and gate-weight gradients within 2e-2 x RMS."""
import numpy as np
import pytest
import torch

from paper_2402_12399_b200 import synth

pytestmark = pytest.mark.gpu
TOL = 2e-2


def _ratio(got, want, what, tol=TOL):
    rms = float(np.sqrt((want ** 2).mean()))
    err = float(np.abs(np.asarray(got, np.float64) - want).max())
    assert rms > 0 and err <= tol * rms, f"{what}: max err {err:.3e} vs rms {rms:.3e} (ratio {err / rms:.2e})"


@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("T,E,k,G,d,d_ff,mode", [(2048, 8, 2, 4, 128, 256, 3), (3072, 16, 1, 2, 192, 128, 1)])
def test_training_step_with_gate_and_load_balance_loss(T, E, k, G, d, d_ff, mode, fused):
    import helpers
    import paper_2402_12399_b200 as rr
    from oracle import rr_oracle as orc
    L = synth.make_layer(T, E, d, d_ff, ("none", 0), 40 + E, "bf16", True, w_std=0.05)
    rng = np.random.default_rng(E)
    Wg_h = synth.to_bf16_bits((rng.standard_normal((E, d)) * 2.0 / np.sqrt(d)).astype(np.float32))
    hid, W1, W3, W2, dout, Wg = (helpers.to_torch(x, "bf16") for x in (L.hidden, L.W1, L.W3, L.W2, L.dout, Wg_h))
    C, alpha = k * T // E, 1e-2

    # forward
    if fused:   # projection, routing and loss in two launches, the selection in the projection's epilogue
        logits, tab, (loss, f, P) = rr.gate_route(hid, Wg, k, C, G, mode, alpha)
    else:
        logits = rr.gate_fwd(hid, Wg)
        tab = rr.route(logits, k, C, G, mode)
    nb = rr.moe_workspace_bytes(T, E, k, C, G, d, d_ff, 0, mode)[2]
    saved = torch.empty(nb, dtype=torch.uint8, device="cuda")
    out = rr.moe_fwd(hid, W1, W3, W2, logits, tab, saved=saved)
    if not fused:
        loss, f, P = rr.aux_loss_fwd(logits, tab.topk_expert, alpha)
        rr.check(loss._workspace)
    for t in (logits, tab, out):
        rr.check(t._workspace)

    a = logits.cpu().numpy()
    tc = orc.route(a, k, C, G, mode)
    helpers.assert_tables_equal(tab, tc, "tables")
    tokens = np.arange(T, dtype=np.int32)
    _ratio(out.cpu().numpy(), orc.forward_tokens(L.hidden, L.W1, L.W3, L.W2, a, tc, tokens), "out")
    L0, f0, _ = orc.aux_loss(a, tc.topk_expert, alpha)
    assert abs(float(loss) - L0) <= 1e-4 * L0

    # backward; the weight of the auxiliary loss is chosen so that both parts of dL/da count
    want_dh, want_dl = orc.backward_tokens(L.hidden, L.W1, L.W3, L.W2, L.dout, a, tc, tokens)
    unit = orc.aux_loss_bwd(a, f0, alpha, 1.0)
    s = float(np.sqrt((want_dl ** 2).mean()) / np.sqrt((unit ** 2).mean()))
    want_dl = want_dl + s * unit
    want_dWg, want_dh_gate = orc.gate_bwd(want_dl, L.hidden, Wg_h)

    dh, dl, dW1, dW3, dW2 = rr.moe_bwd(dout, hid, W1, W3, W2, logits, tab, saved)
    rr.aux_loss_bwd(logits, f, alpha, s, dlogits=dl, accumulate=True)
    dWg = rr.gate_bwd(dl, hid, Wg, dh)
    rr.check(dh._workspace)
    _ratio(dl.cpu().numpy(), want_dl, "dlogits (experts + load-balance loss)")
    _ratio(dWg.cpu().numpy(), want_dWg, "dWg")
    _ratio(dh.cpu().numpy(), want_dh + want_dh_gate, "dhidden (experts + gate)")
