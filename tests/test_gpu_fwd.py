"""GPU parity of rr_moe_fwd against the fp64 oracle: max |err| <= 2e-2 x RMS of the oracle output."""
import numpy as np
import pytest
import torch

from paper_2402_12399_b200 import synth

pytestmark = pytest.mark.gpu
TOL = 2e-2   # x RMS of the oracle tensor


def _run(L, k, C, G, mode, tokens=None, train=False):
    import helpers
    import paper_2402_12399_b200 as rr
    from oracle import rr_oracle as orc
    tg, tc = helpers.route_both(L.logits, k, C, G, mode, "fwd tables")
    hid, W1, W3, W2 = (helpers.to_torch(x, L.dtype) for x in (L.hidden, L.W1, L.W3, L.W2))
    T, d = hid.shape
    E, d_ff, _ = W1.shape
    saved = None
    if train:
        nb = rr.moe_workspace_bytes(T, E, k, C, G, d, d_ff, rr.binding._dtype_code(hid), mode)[2]
        saved = torch.empty(nb, dtype=torch.uint8, device="cuda")
    out = rr.moe_fwd(hid, W1, W3, W2, None, tg, saved=saved)
    rr.check(out._workspace)
    want = orc.forward_tokens(L.hidden, L.W1, L.W3, L.W2, L.logits, tc, tokens)
    got = out.cpu().numpy().astype(np.float64)
    if tokens is not None:
        got = got[tokens]
    # tokens without a live route must be exactly zero; the tolerance is relative to the RMS of
    # the rows the layer actually computes (zeros of dropped tokens would dilute it)
    routed = (tc.token_rows >= 0).any(1)
    routed = routed if tokens is None else routed[tokens]
    assert (got[~routed] == 0).all() and (want[~routed] == 0).all()
    if not routed.any():
        return out, tg, tc, 0.0
    rms = float(np.sqrt((want[routed] ** 2).mean()))
    err = float(np.abs(got - want).max())
    assert rms > 0 and err <= TOL * rms, f"max err {err:.3e} vs rms {rms:.3e} (ratio {err / rms:.3e})"
    return out, tg, tc, err / rms


def test_single_expert_plain_mlp():
    L = synth.make_layer(200, 1, 64, 128, ("none", 0), 1, "bf16", w_std=0.1)
    _run(L, 1, 200, 1, 0)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("T,E,k,G,d,d_ff,cf", [
    (256, 4, 1, 2, 64, 64, 1.0),
    (1024, 8, 2, 4, 128, 320, 1.0),
    (1536, 8, 2, 2, 192, 448, 0.5),
    (640, 16, 1, 4, 256, 128, 1.5),
])
def test_medium_all_modes(T, E, k, G, d, d_ff, cf, dtype):
    L = synth.make_layer(T, E, d, d_ff, ("normal", 0.8), 300 + T + E, dtype, w_std=0.05)
    C = int(cf * k * T / E)
    for mode in (0, 1, 2, 3):
        _run(L, k, C, G, mode)


def test_alternative_readings_feed_the_same_expert_kernels():
    # score-priority dropping, softmax-valued fill-in key, per-source capacity: other tables, same row space
    L = synth.make_layer(1536, 8, 128, 320, ("normal", 0.8), 77, "bf16", w_std=0.05)
    for k, G, cf in [(2, 4, 1.0), (1, 2, 0.5)]:
        C = int(cf * k * 1536 / 8)
        for mode in (3 | 4, 3 | 8, 3 | 16, 3 | 4 | 8 | 16):
            _run(L, k, C, G, mode)


def test_unrouted_tokens_are_zero_and_no_rows():
    L = synth.make_layer(512, 8, 64, 128, ("normal", 1.0), 5, "bf16", w_std=0.05)
    out, tg, tc, _ = _run(L, 1, 16, 2, 0)
    dropped = torch.from_numpy(tc.drop_count > 0).cuda()
    assert bool(dropped.any()) and float(out[dropped].abs().max()) == 0.0
    # capacity 0 without IR: no live row at all, output identically zero
    import paper_2402_12399_b200 as rr
    import helpers
    tg0 = helpers.gpu_route(L.logits, 1, 0, 2, 0)
    hid, W1, W3, W2 = (helpers.to_torch(x, L.dtype) for x in (L.hidden, L.W1, L.W3, L.W2))
    o = rr.moe_fwd(hid, W1, W3, W2, None, tg0)
    rr.check(o._workspace)
    assert float(o.abs().max()) == 0.0


def test_training_mode_saves_and_matches():
    L = synth.make_layer(1024, 8, 128, 256, ("normal", 0.8), 17, "bf16", w_std=0.05)
    _run(L, 2, 256, 4, 3, train=True)


def test_fp32_layer_leaves_saved_alone():
    """An fp32 layer has no backward pass: rr_moe_workspace_bytes reports 0 bytes of `saved`, and a buffer
    that is passed all the same is not written to."""
    import helpers
    import paper_2402_12399_b200 as rr
    L = synth.make_layer(512, 4, 64, 128, ("normal", 0.5), 77, "f32", w_std=0.05)
    k, C, G, mode = 2, 256, 2, 3
    tg, _ = helpers.route_both(L.logits, k, C, G, mode, "fp32 saved")
    hid, W1, W3, W2 = (helpers.to_torch(x, L.dtype) for x in (L.hidden, L.W1, L.W3, L.W2))
    assert rr.moe_workspace_bytes(512, 4, k, C, G, 64, 128, rr.binding._dtype_code(hid), mode)[2] == 0
    plain = rr.moe_fwd(hid, W1, W3, W2, None, tg).cpu()
    saved = torch.full((1 << 20,), 0x5A, dtype=torch.uint8, device="cuda")
    out = rr.moe_fwd(hid, W1, W3, W2, None, tg, saved=saved)
    rr.check(out._workspace)
    assert bool((saved == 0x5A).all())
    assert torch.allclose(out.cpu(), plain, rtol=0, atol=1e-5)   # (the combine adds rows with atomics)


def test_c1_full():
    w = synth.WORKLOADS["c1"]
    L = synth.make_workload(w)
    _, _, _, ratio = _run(L, w.k, w.capacity(1.0), w.G, w.mode)
    print("c1 err/rms", ratio)


@pytest.mark.parametrize("name", ["c3", "c4", "c5"])
def test_scaled_workloads(name):
    w = synth.scaled(synth.WORKLOADS[name], 8, 4)
    L = synth.make_layer(w.T, w.E, w.d, w.d_ff, w.bias, w.seed(), "bf16")
    rng = np.random.default_rng(1)
    tokens = np.sort(rng.choice(w.T, 256, replace=False)).astype(np.int32)
    _run(L, w.k, w.capacity(w.capacity_factors[0]), w.G, w.mode, tokens=tokens)


def test_many_experts_few_rows_each():
    # the largest expert count the library takes: one or two 128-row tiles per expert, so most
    # CTA pairs run with an empty second half, and several experts have no rows at all
    L = synth.make_layer(4096, 256, 64, 64, ("normal", 1.0), 41, "bf16", w_std=0.1)
    for k, G, mode in [(8, 8, 3), (1, 256, 1), (2, 1, 2)]:
        _run(L, k, max(1, int(k * 4096 / 256)), G, mode)


def test_no_tokens_is_a_no_op():
    import paper_2402_12399_b200 as rr
    dev = torch.device("cuda", 0)
    E, d, d_ff = 4, 64, 128
    W1 = torch.zeros(E, d_ff, d, dtype=torch.bfloat16, device=dev)
    W2 = torch.zeros(E, d, d_ff, dtype=torch.bfloat16, device=dev)
    hidden = torch.zeros(0, d, dtype=torch.bfloat16, device=dev)
    logits = torch.zeros(0, E, device=dev)
    tab = rr.route(logits, 2, 4, 2, 3)
    out = rr.moe_fwd(hidden, W1, W1, W2, logits, tab)
    assert out.shape == (0, d)
    nb = rr.moe_workspace_bytes(0, E, 2, 4, 2, d, d_ff, 0, 3)[2]
    saved = torch.empty(max(nb, 256), dtype=torch.uint8, device=dev)
    grads = rr.moe_bwd(hidden, hidden, W1, W1, W2, logits, tab, saved)
    torch.cuda.synchronize()
    assert all(float(g.abs().sum()) == 0.0 for g in grads[2:])
