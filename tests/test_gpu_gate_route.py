"""rr_gate_route: gate projection (Eq. 1) + routing (Sections 3, 4.1, 4.2) + load-balance loss (Section
5.1) with the selection made in the projection's epilogue.  The oracle takes the fp32 logits the GPU
wrote (every routing decision is an exact comparison of those numbers) and composes its own functions:
tables bit-exact, f / P / L within the tolerances of the load-balance loss, logits bit-identical to
rr_gate_fwd."""
import numpy as np
import pytest
import torch

from paper_2402_12399_b200 import synth

pytestmark = pytest.mark.gpu


def _inputs(T, E, d, seed, scale=2.0):
    rng = np.random.default_rng(seed)
    hid = synth.to_bf16_bits(rng.standard_normal((T, d), dtype=np.float32))
    Wg = synth.to_bf16_bits((rng.standard_normal((E, d)) * scale / np.sqrt(d)).astype(np.float32))
    bias_col = rng.normal(0.0, 0.5, E).astype(np.float32)           # skew the load: scale the expert embeddings
    Wg = synth.to_bf16_bits(synth.bf16_bits_to_f32(Wg) * (1.0 + 0.3 * bias_col[:, None]))
    return hid, Wg


def _check(T, E, k, G, d, C, mode, alpha, seed):
    import helpers
    import paper_2402_12399_b200 as rr
    from oracle import rr_oracle as orc
    hid_h, Wg_h = _inputs(T, E, d, seed)
    hid, Wg = helpers.to_torch(hid_h, "bf16"), helpers.to_torch(Wg_h, "bf16")
    logits, tab, aux = rr.gate_route(hid, Wg, k, C, G, mode, alpha)
    rr.check(tab._workspace)
    ref = rr.gate_fwd(hid, Wg)
    assert torch.equal(logits, ref), "logits differ from rr_gate_fwd"
    a = logits.cpu().numpy()
    tc = orc.route(a, k, C, G, mode)
    helpers.assert_tables_equal(tab, tc, f"gate_route T{T} E{E} k{k} mode{mode}")
    if alpha is not None:
        L0, f0, P0 = orc.aux_loss(a, tc.topk_expert, alpha)
        loss, f, P = (x.cpu().numpy().astype(np.float64) for x in aux)
        np.testing.assert_allclose(f, f0, rtol=2.0 ** -22, atol=0)
        np.testing.assert_allclose(P, P0, rtol=6e-5, atol=1e-9)
        assert abs(float(loss[0]) - L0) <= 6e-5 * L0
    return logits, tab, aux


@pytest.mark.parametrize("T,E,k,G,d", [(128, 8, 1, 2, 64), (1000, 8, 2, 4, 128), (4096, 64, 2, 8, 256), (3000, 24, 3, 2, 192),
                                       (2048, 16, 4, 4, 128), (777, 40, 2, 5, 64), (2048, 256, 2, 8, 128), (5000, 32, 1, 8, 320)])
def test_small_shapes_all_modes(T, E, k, G, d):
    T = T // G * G
    for mode in (0, 1, 2, 3):
        for cf in (0.5, 1.0, 2.0):
            C = int(np.ceil(cf * k * T / E))
            _check(T, E, k, G, d, C, mode, 1e-2 if mode == 3 else None, 7 + E + mode)


@pytest.mark.parametrize("name", ["c3", "c5"])
def test_full_size_shapes(name):
    w = synth.WORKLOADS[name]
    _check(w.T, w.E, w.k, w.G, w.d, w.capacity(1.0), 3, 1e-2, 11)


def test_repeats_bit_for_bit_and_reuses_buffers():
    import helpers
    import paper_2402_12399_b200 as rr
    T, E, k, G, d, C = 8192, 64, 2, 8, 256, 256
    hid_h, Wg_h = _inputs(T, E, d, 3)
    hid, Wg = helpers.to_torch(hid_h, "bf16"), helpers.to_torch(Wg_h, "bf16")
    logits, tab, aux = rr.gate_route(hid, Wg, k, C, G, 3, 1e-2)
    rr.check(tab._workspace)
    ref = {n: getattr(tab, n).clone() for n in helpers.INT_TABLES}
    ref_aux = [x.clone() for x in aux]
    for _ in range(5):
        for n in helpers.INT_TABLES:
            getattr(tab, n).fill_(-7)
        rr.gate_route(hid, Wg, k, C, G, 3, 1e-2, logits=logits, tables=tab, workspace=tab._workspace, aux=aux)
        rr.check(tab._workspace)
        for n in helpers.INT_TABLES:
            assert torch.equal(getattr(tab, n), ref[n]), n
        for x, y in zip(aux, ref_aux):
            assert torch.equal(x, y)


def test_nonfinite_scores_are_reported_and_other_modes_refused():
    import helpers
    import paper_2402_12399_b200 as rr
    T, E, k, G, d = 1024, 64, 2, 8, 128
    hid_h, Wg_h = _inputs(T, E, d, 5)
    hid_h[17, :] = 0x7FC0                                            # a NaN hidden state (bf16 bits)
    hid, Wg = helpers.to_torch(hid_h, "bf16"), helpers.to_torch(Wg_h, "bf16")
    logits, tab, _ = rr.gate_route(hid, Wg, k, 64, G, 3)
    with pytest.raises(rr.RRError) as ei:
        rr.check(tab._workspace)
    assert ei.value.code == 5
    assert int(tab.topk_expert.min()) >= 0 and int(tab.topk_expert.max()) < E and int(tab.route_slot.max()) < 64
    for mode in (3 | 4, 3 | 8, 3 | 16):
        with pytest.raises(rr.RRError) as ei:
            rr.gate_route(hid, Wg, k, 64, G, mode)
        assert ei.value.code == 2
    # no tokens
    e_h = torch.empty(0, d, dtype=torch.bfloat16, device="cuda")
    logits, tab, aux = rr.gate_route(e_h, Wg, k, 4, G, 3, 1e-2)
    rr.check(tab._workspace)
    assert float(aux[0]) == 0.0 and int(tab.expert_count.sum()) == 0
