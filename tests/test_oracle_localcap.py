"""Pins for the oracle's per-source capacity (mode bit 16): Section 3 spreads the experts over G
devices and derives the capacity from the number of tokens a router sees; a device routing its own
batch sees T/G tokens, so every expert grants each source group C/G slots of its own.

Checked against things other than the oracle's segment arithmetic: a hand-worked example; the
decomposition into G separate routing problems solved by the already pinned single-segment router;
G = 1, where the flag cannot matter; the invariants of the slot table and of the compact row space."""
import numpy as np
import pytest

from oracle import rr_oracle as orc
from paper_2402_12399_b200 import synth

L = orc.LOCAL_CAP


def test_hand_example():
    # 4 tokens in 2 groups of 2, 2 experts, top-1, C = 2 (one slot per group and expert).
    # Tokens 0, 1 (group 0) choose expert 0; tokens 2, 3 (group 1) choose expert 1.
    a = np.array([[2, 0], [3, 1], [0, 2], [1, 3]], np.float32)
    # over all tokens: both experts take their two tokens, nothing is dropped
    assert orc.route(a, 1, 2, 2, 0).slot_token.tolist() == [[0, 1], [2, 3]]
    # per source: group 0 owns slot 0 of each expert, group 1 slot 1; tokens 1 and 3 are dropped
    t = orc.route(a, 1, 2, 2, L)
    assert t.slot_token.tolist() == [[0, -1], [-1, 2]]
    assert t.route_slot[:, 0].tolist() == [0, -1, 1, -1]
    assert t.drop_count.tolist() == [0, 1, 0, 1]
    assert t.expert_count.tolist() == [1, 1] and t.n_routed.tolist() == [2, 2]
    assert t.row_offset.tolist() == [0, 1, 2] and t.row_token[:2].tolist() == [0, 2]
    assert t.token_rows[:, 0].tolist() == [0, -1, 1, -1]
    # with FR every token nominates its other expert; group 0's slot at expert 1 goes to the better
    # of tokens 0, 1 there (logits 0 and 1: token 1), group 1's slot at expert 0 to token 3 (1 > 0)
    f = orc.route(a, 1, 2, 2, L | orc.FR)
    assert f.slot_token.tolist() == [[0, 3], [1, 2]]
    assert f.slot_rank.tolist() == [[0, 1], [1, 0]]
    assert f.route_slot.tolist() == [[0, -1], [-1, 0], [1, -1], [-1, 1]]
    assert f.expert_count.tolist() == [2, 2]
    # rows follow slot order inside an expert: expert 0 rows (token 0, token 3), expert 1 (1, 2)
    assert f.row_token[:4].tolist() == [0, 3, 1, 2]
    # IR: the dropped tokens 1 and 3 go to the single expert of their own group, after its slots
    r = orc.route(a, 1, 2, 2, L | orc.IR)
    assert r.ir_expert.tolist() == [-1, 0, -1, 1]
    assert r.row_offset.tolist() == [0, 2, 4] and r.row_token[:4].tolist() == [0, 1, 2, 3]


@pytest.mark.parametrize("mode", [0, orc.FR, orc.SCORE, orc.SCORE | orc.FR, orc.FR | orc.FR_SOFTMAX])
def test_equals_one_routing_problem_per_group(mode):
    rng = np.random.default_rng(3)
    for T, E, G, k in [(240, 6, 3, 2), (512, 8, 4, 1), (96, 4, 2, 3), (64, 8, 8, 2)]:
        a = (rng.normal(size=(T, E)) + rng.normal(size=E)).astype(np.float32)
        a[rng.random((T, E)) < 0.1] = 0.5                                   # ties
        Ts = T // G
        for Cs in (0, 1, Ts * k // E, Ts):
            t = orc.route(a, k, Cs * G, G, mode | L)
            count = np.zeros(E, np.int64)
            nr = np.zeros(E, np.int64)
            for g in range(G):
                sub = orc.route(a[g * Ts:(g + 1) * Ts], k, Cs, 1, mode)      # the group alone, single segment
                want = np.where(sub.route_slot >= 0, sub.route_slot + g * Cs, -1)
                assert np.array_equal(t.route_slot[g * Ts:(g + 1) * Ts], want), (T, E, G, k, Cs, g)
                assert np.array_equal(t.drop_count[g * Ts:(g + 1) * Ts], sub.drop_count)
                seg = t.slot_token[:, g * Cs:(g + 1) * Cs]
                assert np.array_equal(seg, np.where(sub.slot_token >= 0, sub.slot_token + g * Ts, -1))
                assert np.array_equal(t.slot_rank[:, g * Cs:(g + 1) * Cs], sub.slot_rank)
                count += sub.expert_count
                nr += sub.n_routed
            assert np.array_equal(t.expert_count, count) and np.array_equal(t.n_routed, nr)


@pytest.mark.parametrize("mode", [0, 1, 2, 3, 7, 3 | orc.FR_SOFTMAX])
def test_one_group_changes_nothing(mode):
    a = synth.make_logits(1024, 8, ("normal", 0.7), 4)
    p, q = orc.route(a, 2, 200, 1, mode), orc.route(a, 2, 200, 1, mode | L)
    for name in ("route_slot", "slot_token", "slot_rank", "drop_count", "ir_expert", "ir_pos", "ir_token",
                 "expert_count", "n_routed", "row_offset", "row_token", "token_rows", "combine_w", "row_weight"):
        assert np.array_equal(getattr(p, name), getattr(q, name)), name


@pytest.mark.parametrize("mode", [L | 3, L | 7, L | 1, L | 2])
def test_invariants(mode):
    for T, E, G, k, Cs in [(2048, 8, 2, 2, 200), (4096, 16, 4, 2, 100), (1024, 32, 8, 1, 3), (960, 6, 3, 3, 170)]:
        a = synth.make_logits(T, E, ("normal", 0.8), 21 + T)
        C, Ts = Cs * G, T // G
        t = orc.route(a, k, C, G, mode)
        K1 = k + 1
        # every occupied slot lies in the segment of its token's group, segments fill from their start
        for e in range(E):
            for g in range(G):
                seg = t.slot_token[e, g * Cs:(g + 1) * Cs]
                n = int((seg >= 0).sum())
                assert (seg[:n] >= 0).all() and (seg[n:] < 0).all()
                assert ((seg[:n] // Ts) == g).all()
        # slot table and route table are inverse to each other
        ii, rr = np.nonzero(t.route_slot >= 0)
        assert (t.slot_token[t.topk_expert[ii, rr], t.route_slot[ii, rr]] == ii).all()
        assert (t.slot_rank[t.topk_expert[ii, rr], t.route_slot[ii, rr]] == rr).all()
        assert int((t.slot_token >= 0).sum()) == len(ii) == int(t.expert_count.sum())
        # drops: a top-k routing without a slot; IR exactly for the tokens with a drop
        assert np.array_equal(t.drop_count, (t.route_slot[:, :k] < 0).sum(1))
        if mode & orc.IR:
            assert ((t.ir_expert >= 0) == (t.drop_count > 0)).all()
        # compact row space: expert e's rows are its occupied slots in slot order, then its IR list
        n_ir = np.diff(t.ir_offset)
        assert np.array_equal(np.diff(t.row_offset), t.expert_count + n_ir)
        for e in range(E):
            occupied = t.slot_token[e][t.slot_token[e] >= 0]
            want = np.concatenate([occupied, t.ir_token[t.ir_offset[e]:t.ir_offset[e + 1]]])
            assert np.array_equal(t.row_token[t.row_offset[e]:t.row_offset[e + 1]], want), e
        live = t.token_rows >= 0
        assert (t.row_token[t.token_rows[live]] == np.nonzero(live)[0]).all()
        assert (t.row_weight[t.token_rows[live]] == t.combine_w[live]).all()
        np.testing.assert_allclose(t.combine_w.sum(1)[live.any(1)], 1.0, rtol=1e-12)
        # tighter than the capacity over all tokens: a group cannot borrow another group's slots
        glob = orc.route(a, k, C, G, mode & ~L)
        assert int(t.drop_count.sum()) >= int(glob.drop_count.sum())


def test_arguments():
    a = synth.make_logits(64, 4, ("normal", 0.5), 1)
    with pytest.raises(orc.OracleError):
        orc.route(a, 1, 17, 2, L)           # capacity not divisible by the number of groups
    orc.route(a, 1, 16, 2, L)
    orc.route(np.zeros((0, 4), np.float32), 1, 16, 2, L | 3)
