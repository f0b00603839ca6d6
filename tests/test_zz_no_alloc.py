"""rr_route_noalloc: routing for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is off limits at routing time (a latency-critical
or stream-ordered section, a plug-in without an allocator, a fully committed memory pool).  For
them the library keeps the routing scratch in a fixed array of its own.  This test calls that entry
point through the C ABI twice in a row, on different inputs, and requires the same tables as the
regular rr_route gives (and as the CPU oracle computes): the array keeps the previous call's
contents, so the second call would expose anything that wrongly relied on a clean start.  It lives
in its own file, collected last.
"""
import numpy as np
import pytest
import torch

from paper_2402_12399_b200 import synth

pytestmark = pytest.mark.gpu

INT_TABLES = ["topk_expert", "route_slot", "slot_token", "slot_rank", "drop_count", "ir_expert", "ir_pos",
              "ir_offset", "ir_token", "expert_count", "n_routed", "row_offset", "row_token", "token_rows"]


def _compare(rr, logits_np, k, C, G, mode, status):
    a = torch.from_numpy(logits_np).cuda()
    T, E = a.shape
    want = rr.route(a, k, C, G, mode)
    rr.check(want._workspace)
    got = rr.alloc_tables(T, E, k, C, G, mode)          # outputs stay the caller's
    for n in INT_TABLES:
        getattr(got, n).fill_(-9)
    rr.route_noalloc(a, k, C, G, mode, got, status)
    rr.check(status)
    for n in INT_TABLES:                                    # integer tables: bit-exact
        assert torch.equal(getattr(got, n), getattr(want, n)), n
    # and directly against the CPU statement of the method, not only against the sibling entry point
    import helpers
    from oracle import rr_oracle as orc
    helpers.assert_tables_equal(got, orc.route(logits_np, k, C, G, mode), "rr_route_noalloc vs oracle")
    # weights: the tolerance of the routing parity tests
    np.testing.assert_allclose(got.combine_w.cpu().numpy(), want.combine_w.cpu().numpy(), rtol=1e-5, atol=1e-7)
    np.testing.assert_allclose(got.row_weight.cpu().numpy(), want.row_weight.cpu().numpy(), rtol=1e-5, atol=1e-7)


def test_two_calls_in_a_row_match_rr_route():
    import paper_2402_12399_b200 as rr
    status = torch.zeros(64, dtype=torch.int32, device="cuda")
    w = synth.WORKLOADS["c2"]
    # first call: the largest listed shape; second call: a smaller, differently shaped problem
    # that reuses (and must not be confused by) what the first one left in the array
    _compare(rr, synth.make_logits(w.T, w.E, w.bias, 11), w.k, w.capacity(1.0), w.G, 3, status)
    _compare(rr, synth.make_logits(3000, 24, ("normal", 1.0), 12), 3, 300, 4, 3, status)
    _compare(rr, synth.make_logits(w.T, w.E, w.bias, 13), w.k, w.capacity(1.25), w.G, 1, status)


def test_status_may_be_omitted_and_nonfinite_is_latched():
    import paper_2402_12399_b200 as rr
    a = synth.make_logits(2048, 8, ("normal", 0.7), 3)
    t = rr.alloc_tables(2048, 8, 1, 256, 2, 3)
    rr.route_noalloc(torch.from_numpy(a).cuda(), 1, 256, 2, 3, t, None)
    torch.cuda.synchronize()
    ref = rr.route(torch.from_numpy(a).cuda(), 1, 256, 2, 3)
    assert torch.equal(t.slot_token, ref.slot_token)
    a[5, 5] = np.inf
    status = torch.zeros(64, dtype=torch.int32, device="cuda")
    rr.route_noalloc(torch.from_numpy(a).cuda(), 1, 256, 2, 3, t, status)
    with pytest.raises(rr.RRError) as ei:
        rr.check(status)
    assert ei.value.code == 5


def test_shapes_beyond_the_fixed_array_are_refused():
    import paper_2402_12399_b200 as rr
    T, E, k = 1 << 20, 64, 2                               # needs ~50 MB of scratch
    a = torch.zeros(T, E, device="cuda")
    t = rr.alloc_tables(T, E, k, 64, 8, 0)
    with pytest.raises(rr.RRError) as ei:
        rr.route_noalloc(a, k, 64, 8, 0, t, None)
    assert ei.value.code == 7 and "fixed" in str(ei.value)
