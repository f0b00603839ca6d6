"""GPU parity of rr_moe_bwd against the fp64 oracle: every gradient within 2e-2 x RMS.

Shapes give every expert on the order of a thousand rows: the bound is a maximum over all
elements relative to the tensor's RMS, and with only a hundred rows per expert the column norms
of the bf16-rounded operands scatter so much that single columns dominate the maximum."""
import numpy as np
import pytest
import torch

from paper_2402_12399_b200 import synth

pytestmark = pytest.mark.gpu
TOL = 2e-2


def _close(got, want, what, mask=None):
    got = np.asarray(got, np.float64)
    if mask is not None:
        assert (got[~mask] == 0).all() and (want[~mask] == 0).all(), f"{what}: unrouted entries must be zero"
        if not mask.any():
            return 0.0
        rms = float(np.sqrt((want[mask] ** 2).mean()))
    else:
        rms = float(np.sqrt((want ** 2).mean()))
    err = float(np.abs(got - want).max())
    if rms == 0:
        assert err == 0, what
        return 0.0
    if err > TOL * rms:
        FAILS.append(f"{what}: max err {err:.3e} vs rms {rms:.3e} (ratio {err / rms:.3e})")
    return err / rms


FAILS = []


def _run(L, k, C, G, mode, grad_exact=False, tokens=None, experts=None):
    import helpers
    import paper_2402_12399_b200 as rr
    from oracle import rr_oracle as orc
    tg, tc = helpers.route_both(L.logits, k, C, G, mode, "bwd tables")
    hid, W1, W3, W2, dout = (helpers.to_torch(x, "bf16") for x in (L.hidden, L.W1, L.W3, L.W2, L.dout))
    logits = torch.from_numpy(L.logits).cuda()
    T, d = hid.shape
    E, d_ff, _ = W1.shape
    _, _, nb = rr.moe_workspace_bytes(T, E, k, C, G, d, d_ff, 0, mode)
    saved = torch.empty(nb, dtype=torch.uint8, device="cuda")
    out = rr.moe_fwd(hid, W1, W3, W2, logits, tg, saved=saved)
    rr.check(out._workspace)
    dh, dl, dW1, dW3, dW2 = rr.moe_bwd(dout, hid, W1, W3, W2, logits, tg, saved, grad_exact=grad_exact)
    rr.check(dh._workspace)
    tok = np.arange(T, dtype=np.int32) if tokens is None else tokens
    want_dh, want_dl = orc.backward_tokens(L.hidden, L.W1, L.W3, L.W2, L.dout, L.logits, tc, tok, grad_exact)
    routed = (tc.token_rows >= 0).any(1)[tok]
    r = {"dhidden": _close(dh.cpu().numpy()[tok], want_dh, "dhidden", routed),
         "dlogits": _close(dl.cpu().numpy()[tok], want_dl, "dlogits", routed)}
    for e in (range(E) if experts is None else experts):
        w1, w3, w2 = orc.backward_expert(L.hidden, L.W1, L.W3, L.W2, L.dout, tc, e)
        r[f"dW1[{e}]"] = _close(dW1[e].cpu().numpy(), w1, f"dW1[{e}]")
        r[f"dW3[{e}]"] = _close(dW3[e].cpu().numpy(), w3, f"dW3[{e}]")
        r[f"dW2[{e}]"] = _close(dW2[e].cpu().numpy(), w2, f"dW2[{e}]")
    print({k_: f"{v:.2e}" for k_, v in r.items()})
    fails = list(FAILS)
    FAILS.clear()
    assert not fails, fails
    return r


@pytest.mark.parametrize("T,E,k,G,d,d_ff,cf,mode", [
    (2048, 2, 1, 1, 128, 128, 1.0, 3),
    (2048, 4, 2, 2, 128, 256, 1.0, 3),
    (3200, 8, 2, 4, 192, 320, 1.0, 3),
    (4096, 8, 1, 2, 256, 384, 1.5, 2),
    (2048, 4, 2, 2, 320, 192, 1.0, 1),
    (2048, 4, 2, 2, 128, 256, 1.0, 3 | 16),          # per-source capacity
    (3200, 8, 2, 4, 192, 320, 1.0, 3 | 4 | 8 | 16),  # all three alternative readings at once
])
def test_small_gradients(T, E, k, G, d, d_ff, cf, mode):
    L = synth.make_layer(T, E, d, d_ff, ("normal", 0.8), 500 + T + E, "bf16", True, w_std=0.05)
    _run(L, k, int(cf * k * T / E), G, mode)


def test_exact_gate_gradient():
    L = synth.make_layer(2048, 4, 128, 256, ("normal", 0.8), 77, "bf16", True, w_std=0.05)
    _run(L, 2, 1024, 2, 3, grad_exact=True)


def test_expert_without_rows_gets_zero_weight_gradient():
    # a strongly negative bias empties expert 3: its weight gradients must be exactly zero
    L = synth.make_layer(256, 4, 64, 128, ("none", 0), 5, "bf16", True, w_std=0.05)
    L.logits[:, 3] = -50.0
    r = _run(L, 1, 256, 1, 0)
    assert r["dW1[3]"] == 0.0


@pytest.mark.parametrize("name", ["c4", "c5"])
def test_scaled_training_workloads(name):
    w = synth.scaled(synth.WORKLOADS[name], 8, 4)
    L = synth.make_layer(w.T, w.E, w.d, w.d_ff, w.bias, w.seed(), "bf16", True)
    rng = np.random.default_rng(2)
    tokens = np.sort(rng.choice(w.T, 192, replace=False)).astype(np.int32)
    _run(L, w.k, w.capacity(w.capacity_factors[0]), w.G, w.mode, tokens=tokens, experts=[0, w.E - 1])


def test_many_experts_odd_tile_counts():
    # 64 experts with two to four 128-row tiles each: CTA pairs with an empty second half in every
    # GEMM of the backward pass, weight gradients contracted over short row ranges
    L = synth.make_layer(8192, 64, 64, 128, ("normal", 0.6), 23, "bf16", True, w_std=0.1)
    _run(L, 2, 256, 8, 3, experts=[0, 31, 63])


def test_skewed_experts_weight_gradients():
    """A few hot experts hold most rows (their own capacity plus the IR rows of their group), others a handful:
    the weight-gradient items differ in cost by two orders of magnitude and are dealt out by falling cost in
    alternating direction.  Checked on the two largest experts and on two of middle size (the bound on the
    largest entry needs a few hundred rows per expert, see the module docstring)."""
    import helpers
    L = synth.make_layer(8192, 16, 128, 256, ("zipf", 1.5), 91, "bf16", True, w_std=0.1)
    k, C, G, mode = 2, 1024, 2, 3
    _, tc = helpers.route_both(L.logits, k, C, G, mode, "skewed tables")
    rows = np.diff(np.asarray(tc.row_offset))
    assert rows.max() >= 8 * max(1, int(np.median(rows))) and rows.min() < 64, rows   # the input is skewed
    order = [int(e) for e in np.argsort(-rows)]
    mid = [e for e in order[2:] if rows[e] >= 256][:2]
    _run(L, k, C, G, mode, experts=order[:2] + mid)
