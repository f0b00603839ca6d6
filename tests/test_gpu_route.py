"""GPU parity of rr_route against the CPU oracle: all integer tables bit-exact."""
import json
import os

import numpy as np
import pytest
import torch

from paper_2402_12399_b200 import synth

pytestmark = pytest.mark.gpu


def _h():
    import helpers
    return helpers


def test_capacity3_example_on_gpu():
    g = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "capacity3_example.json")))
    a = np.array(g["logits"], np.float32)
    for mode in (0, 1, 2, 3):
        tg, _ = _h().route_both(a, g["k"], g["C"], g["G"], mode, f"capacity3 mode {mode}")
    assert tg.slot_token.cpu().tolist() == g["fr"]["slot_token"]


@pytest.mark.parametrize("E,k,G", [(1, 1, 1), (2, 1, 2), (3, 2, 1), (4, 2, 2), (6, 3, 3), (8, 1, 2), (8, 2, 8),
                                   (16, 2, 4), (24, 3, 2), (32, 1, 8), (64, 2, 8), (96, 4, 4), (128, 2, 2),
                                   (200, 8, 5), (256, 2, 8)])
def test_small_all_modes(E, k, G):
    for T in (G, 40 * G, 333 * G):          # one ragged tile, several tiles with a ragged tail
        a = synth.make_logits(T, E, ("normal", 1.0), 100 + E + T)
        for cf in (0.5, 1.0, 2.0):
            C = int(np.ceil(cf * k * T / E))
            for mode in (0, 1, 2, 3):
                if (mode & 2) and k >= E:
                    continue
                _h().route_both(a, k, C, G, mode, f"T{T} E{E} k{k} G{G} C{C} mode{mode}")


def test_heavy_ties():
    rng = np.random.default_rng(3)
    for E, k, G in [(8, 2, 2), (64, 2, 8), (32, 1, 4)]:
        T = 1000 * G
        a = (rng.integers(-2, 3, (T, E)) * 0.5).astype(np.float32)
        a[rng.random((T, E)) < 0.2] = -0.0
        for C in (0, 1, T * k // E, T):
            _h().route_both(a, k, C, G, 3, f"ties E{E} C{C}")


def test_degenerate_capacities_and_empty():
    a = synth.make_logits(512, 8, ("normal", 0.7), 9)
    for C in (0, 1, 512, 2048):
        for mode in (0, 3):
            _h().route_both(a, 2, C, 4, mode, f"C{C} mode{mode}")
    _h().route_both(np.zeros((0, 8), np.float32), 2, 4, 2, 3, "empty")
    _h().route_both(a, 8, 600, 2, 1, "k == E")


@pytest.mark.parametrize("name", ["c1", "c2", "c3", "c4", "c5"])
def test_workload_shapes(name):
    w = synth.WORKLOADS[name]
    for ci, cf in enumerate(w.capacity_factors):
        modes = (0, 1, 2, 3) if name == "c2" else (w.mode,)
        for mode in modes:
            a = synth.make_logits(w.T, w.E, w.bias, w.seed(ci, mode))
            _h().route_both(a, w.k, w.capacity(cf), w.G, mode, f"{name} cf{cf} mode{mode}")


def test_extra_seeds_c2():
    w = synth.WORKLOADS["c2"]
    for extra in (1, 2, 3):
        a = synth.make_logits(w.T, w.E, w.bias, w.seed(0, 3, extra))
        _h().route_both(a, w.k, w.capacity(1.0), w.G, 3, f"c2 seed {extra}")


def test_inference_sweeps_from_the_paper():
    # capacity factors of Tables 3-4 and experts-per-group of Table 6
    T, E = 16384, 8
    a = synth.make_logits(T, E, ("normal", 0.5), 77)
    for k, cf, mode in [(1, 0.5, 1), (1, 0.75, 1), (2, 1.0, 1), (2, 1.5, 1), (1, 1.25, 2), (1, 1.5, 2),
                        (2, 2.5, 2), (2, 3.0, 2)]:
        for G in (8, 4, 2):
            _h().route_both(a, k, int(cf * T / E), G, mode, f"k{k} cf{cf} G{G}")


def test_logits_written_by_the_kernel_just_before():
    """The routing kernel may be set up while the kernel before it in the stream still runs; it must not read
    its logits before that kernel has finished.  The logits buffer is rewritten by a copy kernel right in
    front of every call, twelve different inputs without a synchronisation in between; every result is
    compared with the tables of the same input routed on its own."""
    import paper_2402_12399_b200 as rr
    w = synth.WORKLOADS["c2"]
    C = w.capacity(1.0)
    inputs = [torch.from_numpy(synth.make_logits(w.T, w.E, w.bias, 900 + i)).cuda() for i in range(12)]
    refs = []
    for x in inputs:
        t = rr.route(x, w.k, C, w.G, 3)
        rr.check(t._workspace)
        refs.append({n: getattr(t, n).clone() for n in _h().INT_TABLES})
    live = torch.empty_like(inputs[0])
    outs = [rr.alloc_tables(w.T, w.E, w.k, C, w.G, 3) for _ in inputs]
    ws = rr.alloc_workspace(rr.route_workspace_bytes(w.T, w.E, w.k, C, w.G, 3))
    torch.cuda.synchronize()
    for x, t in zip(inputs, outs):
        live.copy_(x)                                        # a kernel on the same stream writes the logits
        rr.route(live, w.k, C, w.G, 3, tables=t, workspace=ws)
    rr.check(ws)
    for i, (t, ref) in enumerate(zip(outs, refs)):
        for n in _h().INT_TABLES:
            assert torch.equal(getattr(t, n), ref[n]), (i, n)


def test_deterministic_and_reuses_buffers():
    import paper_2402_12399_b200 as rr
    w = synth.WORKLOADS["c5"]
    a = torch.from_numpy(synth.make_logits(w.T, w.E, w.bias, 5)).cuda()
    t = rr.route(a, w.k, w.capacity(1.0), w.G, 3)
    ref = {n: getattr(t, n).clone() for n in _h().INT_TABLES}
    ws = t._workspace
    for _ in range(10):
        for n in _h().INT_TABLES:
            getattr(t, n).fill_(-7)             # stale contents must be completely overwritten
        rr.route(a, w.k, w.capacity(1.0), w.G, 3, tables=t, workspace=ws)
        rr.check(ws)
        for n in _h().INT_TABLES:
            assert torch.equal(getattr(t, n), ref[n]), n


def test_nonfinite_logit_is_reported_not_fatal():
    import paper_2402_12399_b200 as rr
    a = synth.make_logits(1024, 8, ("none", 0), 1)
    a[17, 3] = np.nan
    t = rr.route(torch.from_numpy(a).cuda(), 2, 256, 2, 3)
    with pytest.raises(rr.RRError) as ei:
        rr.check(t._workspace)
    assert ei.value.code == 5
    rr.check(t._workspace)                      # reported once, then clear
    assert int(t.route_slot.max()) < 256 and int(t.topk_expert.max()) < 8


@pytest.mark.parametrize("E,k,G", [(64, 2, 8), (32, 1, 4), (8, 2, 2), (24, 3, 2), (256, 4, 8)])
@pytest.mark.parametrize("mode", [3, 3 | 4, 3 | 8, 3 | 16])
def test_rows_without_a_finite_logit_keep_every_index_in_range(E, k, G, mode):
    """Whole rows of NaN or of -inf (a NaN hidden state, every expert masked) and rows where fewer
    than k+1 logits are finite: the call reports RR_ERR_NONFINITE, nothing faults, and every index
    in every table names an expert / slot / token / row that exists."""
    import paper_2402_12399_b200 as rr
    T, C = 512 * G, 8 * G
    a = synth.make_logits(T, E, ("normal", 1.0), 55 + E)
    a[3, :] = np.nan
    a[40, :] = -np.inf
    a[T - 1, :] = -np.inf
    a[T - 1, E - 1] = 0.5              # one finite logit, k+1 wanted
    a[77, : E // 2] = np.nan
    a[300, 1:] = np.inf
    t = rr.route(torch.from_numpy(a).cuda(), k, C, G, mode)
    with pytest.raises(rr.RRError) as ei:
        rr.check(t._workspace)
    assert ei.value.code == 5
    R = E * C + T
    for name, lo, hi in [("topk_expert", -1, E), ("route_slot", -1, C), ("slot_token", -1, T), ("slot_rank", -1, k + 1),
                         ("drop_count", 0, k + 1), ("ir_expert", -1, E), ("ir_pos", -1, T), ("ir_offset", 0, T + 1),
                         ("ir_token", -1, T), ("expert_count", 0, C + 1), ("row_offset", 0, R + 1),
                         ("row_token", -1, T), ("token_rows", -1, R)]:
        x = getattr(t, name)
        assert int(x.min()) >= lo and int(x.max()) < hi, (name, int(x.min()), int(x.max()))
    assert int(t.topk_expert[:, :k].min()) >= 0       # the k routed experts always exist (k <= E)
    # a clean call on the same buffers afterwards is exact again
    b = synth.make_logits(T, E, ("normal", 1.0), 56 + E)
    rr.route(torch.from_numpy(b).cuda(), k, C, G, mode, tables=t, workspace=t._workspace)
    rr.check(t._workspace)
    from oracle import rr_oracle as orc
    _h().assert_tables_equal(t, orc.route(b, k, C, G, mode), f"after non-finite rows E{E} mode{mode}")


def test_bad_arguments_are_refused():
    import paper_2402_12399_b200 as rr
    a = torch.zeros(64, 8, device="cuda")
    for kw in [dict(k=0), dict(k=9), dict(G=3), dict(capacity=-1), dict(mode=32), dict(mode=8), dict(mode=9), dict(mode=16, capacity=9), dict(k=8, mode=2)]:
        args = dict(k=1, capacity=8, G=2, mode=0)
        args.update(kw)
        with pytest.raises(rr.RRError) as ei:
            rr.route(a, **args)
        assert ei.value.code == 1
    with pytest.raises(rr.RRError) as ei:
        rr.route(a, 1, 8, 2, 0, workspace=torch.zeros(256, dtype=torch.uint8, device="cuda"))
    assert ei.value.code == 3


# ---- score-priority dropping (mode bit 4: a full expert drops its lowest scores, Section 3's wording) ----
@pytest.mark.parametrize("E,k,G", [(1, 1, 1), (2, 1, 2), (3, 2, 1), (4, 2, 2), (6, 3, 3), (8, 2, 8), (16, 2, 4),
                                   (24, 3, 2), (32, 1, 8), (64, 2, 8), (96, 4, 4), (200, 8, 5), (256, 2, 8)])
def test_score_priority_small_all_modes(E, k, G):
    for T in (G, 40 * G, 333 * G):
        a = synth.make_logits(T, E, ("normal", 1.0), 300 + E + T)
        for cf in (0.5, 1.0, 2.0):
            C = int(np.ceil(cf * k * T / E))
            for mode in (4, 5, 6, 7):
                if (mode & 2) and k >= E:
                    continue
                _h().route_both(a, k, C, G, mode, f"score T{T} E{E} k{k} G{G} C{C} mode{mode}")


def test_score_priority_heavy_ties_and_degenerate_capacities():
    rng = np.random.default_rng(4)
    for E, k, G in [(8, 2, 2), (64, 2, 8), (32, 1, 4)]:
        T = 1000 * G
        a = (rng.integers(-2, 3, (T, E)) * 0.5).astype(np.float32)
        a[rng.random((T, E)) < 0.2] = -0.0
        for C in (0, 1, T * k // E, T):
            _h().route_both(a, k, C, G, 7, f"score ties E{E} C{C}")
    _h().route_both(np.zeros((0, 8), np.float32), 2, 4, 2, 7, "score empty")
    _h().route_both(synth.make_logits(512, 8, ("normal", 0.7), 9), 8, 600, 2, 5, "score k == E")


@pytest.mark.parametrize("name", ["c2", "c3", "c4", "c5"])
def test_score_priority_workload_shapes(name):
    w = synth.WORKLOADS[name]
    for ci, cf in enumerate(w.capacity_factors):
        for mode in ((4, 5, 6, 7) if name == "c2" else (w.mode | 4,)):
            a = synth.make_logits(w.T, w.E, w.bias, w.seed(ci, mode))
            _h().route_both(a, w.k, w.capacity(cf), w.G, mode, f"score {name} cf{cf} mode{mode}")


def test_score_priority_reuses_buffers_and_is_refused_without_allocation():
    import paper_2402_12399_b200 as rr
    w = synth.WORKLOADS["c5"]
    a = torch.from_numpy(synth.make_logits(w.T, w.E, w.bias, 6)).cuda()
    t = rr.route(a, w.k, w.capacity(1.0), w.G, 7)
    ref = {n: getattr(t, n).clone() for n in _h().INT_TABLES}
    for _ in range(5):
        for n in _h().INT_TABLES:
            getattr(t, n).fill_(-7)
        rr.route(a, w.k, w.capacity(1.0), w.G, 7, tables=t, workspace=t._workspace)
        rr.check(t._workspace)
        for n in _h().INT_TABLES:
            assert torch.equal(getattr(t, n), ref[n]), n
    with pytest.raises(rr.RRError) as ei:
        rr.route_noalloc(a, w.k, w.capacity(1.0), w.G, 7, t)
    assert ei.value.code == 1


# ---- softmax-valued FR key (mode bit 8: nominees ranked by g_ie, Appendix A's "routing scores") ----
@pytest.mark.parametrize("E,k,G", [(2, 1, 2), (3, 2, 1), (4, 2, 2), (6, 3, 3), (8, 2, 8), (16, 2, 4), (24, 3, 2),
                                   (32, 1, 8), (64, 2, 8), (96, 4, 4), (200, 7, 5), (256, 2, 8)])
def test_softmax_key_small_all_modes(E, k, G):
    for T in (G, 40 * G, 333 * G):
        a = synth.make_logits(T, E, ("normal", 1.0), 500 + E + T)
        for cf in (0.5, 1.0, 2.0):
            C = int(np.ceil(cf * k * T / E))
            for mode in (2 | 8, 3 | 8, 6 | 8, 7 | 8):
                _h().route_both(a, k, C, G, mode, f"softkey T{T} E{E} k{k} G{G} C{C} mode{mode}")


def test_softmax_key_wide_logits_ties_and_degenerate_capacities():
    rng = np.random.default_rng(14)
    for E, k, G in [(8, 2, 2), (64, 2, 8), (32, 1, 4)]:
        T = 1000 * G
        a = (rng.integers(-2, 3, (T, E)) * 0.5).astype(np.float32)           # few distinct rows: many equal keys
        a[rng.random((T, E)) < 0.2] = -0.0
        for C in (0, 1, T * k // E, T):
            _h().route_both(a, k, C, G, 3 | 8, f"softkey ties E{E} C{C}")
        b = (rng.normal(size=(T, E)) * 40.0).astype(np.float32)              # reaches the clamp at -80
        _h().route_both(b, k, T * k // E, G, 3 | 8, f"softkey wide E{E}")
    _h().route_both(np.zeros((0, 8), np.float32), 2, 4, 2, 3 | 8, "softkey empty")


@pytest.mark.parametrize("name", ["c2", "c3", "c4", "c5"])
def test_softmax_key_workload_shapes(name):
    w = synth.WORKLOADS[name]
    for ci, cf in enumerate(w.capacity_factors):
        for mode in ((2 | 8, 3 | 8) if name == "c2" else (3 | 8,)):
            a = synth.make_logits(w.T, w.E, w.bias, w.seed(ci, mode))
            tg, tc = _h().route_both(a, w.k, w.capacity(cf), w.G, mode, f"softkey {name} cf{cf} mode{mode}")
    # the key matters on these inputs: the logit-keyed router fills in other tokens
    plain = _h().gpu_route(a, w.k, w.capacity(cf), w.G, 3)
    assert not torch.equal(plain.route_slot, tg.route_slot)
    assert torch.equal(plain.route_slot[:, :w.k], tg.route_slot[:, :w.k])


def test_softmax_key_reuses_buffers_and_is_refused_without_allocation():
    import paper_2402_12399_b200 as rr
    w = synth.WORKLOADS["c5"]
    a = torch.from_numpy(synth.make_logits(w.T, w.E, w.bias, 6)).cuda()
    t = rr.route(a, w.k, w.capacity(1.0), w.G, 3 | 8)
    ref = {n: getattr(t, n).clone() for n in _h().INT_TABLES}
    for _ in range(5):
        for n in _h().INT_TABLES:
            getattr(t, n).fill_(-7)
        rr.route(a, w.k, w.capacity(1.0), w.G, 3 | 8, tables=t, workspace=t._workspace)
        rr.check(t._workspace)
        for n in _h().INT_TABLES:
            assert torch.equal(getattr(t, n), ref[n]), n
    with pytest.raises(rr.RRError) as ei:
        rr.route_noalloc(a, w.k, w.capacity(1.0), w.G, 3 | 8, t)
    assert ei.value.code == 1


# ---- per-source capacity (mode bit 16: every expert grants each source group capacity/G slots, Section 3's
# capacity as a device sees it that routes only its own tokens) ----
@pytest.mark.parametrize("E,k,G", [(1, 1, 1), (2, 1, 2), (3, 2, 1), (3, 2, 3), (4, 2, 2), (6, 3, 3), (8, 2, 8), (16, 2, 4),
                                   (24, 3, 2), (32, 1, 8), (64, 2, 8), (96, 4, 4), (200, 7, 5), (256, 2, 256)])
def test_local_capacity_small_all_modes(E, k, G):
    for Ts in (1, 40, 333):                       # tokens per group: tiles end inside a group, odd row addresses
        T = Ts * G
        a = synth.make_logits(T, E, ("normal", 1.0), 700 + E + T)
        for cf in (0.5, 1.0, 2.0):
            C = int(np.ceil(cf * k * Ts / E)) * G
            for mode in (16, 17, 18, 19, 23, 27):
                if (mode & 2) and k >= E:
                    continue
                _h().route_both(a, k, C, G, mode, f"localcap T{T} E{E} k{k} G{G} C{C} mode{mode}")


def test_local_capacity_ties_and_degenerate_capacities():
    rng = np.random.default_rng(24)
    for E, k, G in [(8, 2, 2), (64, 2, 8), (32, 1, 4)]:
        T = 1000 * G
        a = (rng.integers(-2, 3, (T, E)) * 0.5).astype(np.float32)
        a[rng.random((T, E)) < 0.2] = -0.0
        for Cs in (0, 1, 1000 * k // E, 1000):
            for mode in (19, 23, 31):
                _h().route_both(a, k, Cs * G, G, mode, f"localcap ties E{E} Cs{Cs} mode{mode}")
    _h().route_both(np.zeros((0, 8), np.float32), 2, 4, 2, 19, "localcap empty")


@pytest.mark.parametrize("name", ["c2", "c3", "c4", "c5"])
def test_local_capacity_workload_shapes(name):
    w = synth.WORKLOADS[name]
    for ci, cf in enumerate(w.capacity_factors):
        for mode in ((16, 17, 18, 19, 23) if name == "c2" else (19,)):
            a = synth.make_logits(w.T, w.E, w.bias, w.seed(ci, mode))
            tg, tc = _h().route_both(a, w.k, w.capacity(cf), w.G, mode, f"localcap {name} cf{cf} mode{mode}")
    plain = _h().gpu_route(a, w.k, w.capacity(cf), w.G, 3)
    assert not torch.equal(plain.route_slot, tg.route_slot)            # the flag matters on these inputs


def test_local_capacity_reuses_buffers_and_is_refused_without_allocation():
    import paper_2402_12399_b200 as rr
    w = synth.WORKLOADS["c5"]
    a = torch.from_numpy(synth.make_logits(w.T, w.E, w.bias, 6)).cuda()
    t = rr.route(a, w.k, w.capacity(1.0), w.G, 19)
    ref = {n: getattr(t, n).clone() for n in _h().INT_TABLES}
    for _ in range(5):
        for n in _h().INT_TABLES:
            getattr(t, n).fill_(-7)
        rr.route(a, w.k, w.capacity(1.0), w.G, 19, tables=t, workspace=t._workspace)
        rr.check(t._workspace)
        for n in _h().INT_TABLES:
            assert torch.equal(getattr(t, n), ref[n]), n
    with pytest.raises(rr.RRError) as ei:
        rr.route_noalloc(a, w.k, w.capacity(1.0), w.G, 19, t)
    assert ei.value.code == 1


@pytest.mark.parametrize("T,E,k,G,cf,bias", [(1 << 18, 8, 1, 4, 1.0, ("normal", 0.3)), (1 << 20, 64, 2, 8, 1.0, ("zipf", 1.1)),
                                             (200000, 16, 2, 4, 1.5, ("normal", 1.0))])
def test_long_nominee_lists(T, E, k, G, cf, bias):
    """Many tokens per expert: every expert's nominee list is far longer than one block holds in
    registers (the long-list path of the fill-in selection, with padding left to fill), the per-token
    records of the persistent kernel go through the workspace, and on heavy ties the equal keys are
    split by token order."""
    a = synth.make_logits(T, E, bias, 4242 + E)
    C = int(cf * T / E)
    _h().route_both(a, k, C, G, 3, f"long lists T{T} E{E}")
    if E == 8:
        rng = np.random.default_rng(1)
        b = (rng.integers(-3, 4, (T, E)) * 0.25).astype(np.float32)
        _h().route_both(b, k, C, G, 3, f"long lists with ties T{T} E{E}")
