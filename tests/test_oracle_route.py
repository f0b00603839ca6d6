"""Pins for the routing oracle (CPU only).

Each test checks oracle/rr_oracle.c against something other than itself:
a hand-derived example in the setting of Fig. 1, the invariants Section 3
states, the special cases Sections 4.1 / 4.2 state, and an independent
definition-by-counting formulation enumerated over every small logit matrix.
"""
import itertools
import json
import math
import os

import numpy as np
import pytest

from oracle import rr_oracle as orc
from paper_2402_12399_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden", "capacity3_example.json")


def _gold():
    with open(GOLD) as f:
        return json.load(f)


# --------------------------------------------------------------------------
# P1: capacity-3 example (Fig. 1 caption; Section 3; Sections 4.1, 4.2)
# --------------------------------------------------------------------------
def test_capacity3_vanilla():
    g = _gold()
    a = np.array(g["logits"], np.float32)
    t = orc.route(a, g["k"], g["C"], g["G"], 0)
    assert t.slot_token.tolist() == g["vanilla"]["slot_token"]
    dropped = [i for i in range(g["T"]) if t.drop_count[i] > 0]
    assert dropped == g["vanilla"]["dropped_tokens"]
    assert int((t.slot_token < 0).sum()) == g["vanilla"]["n_padding"]
    assert int(t.drop_count.sum()) == g["vanilla"]["n_dropped"]
    for e, q in g["queues"].items():
        assert int(t.n_routed[int(e)]) == len(q)
    # dropped tokens have no route at all and weight zero
    for i in dropped:
        assert (t.route_slot[i] < 0).all() and (t.combine_w[i] == 0).all()
    assert (t.ir_expert == -1).all()


def test_capacity3_ir():
    g = _gold()
    a = np.array(g["logits"], np.float32)
    t = orc.route(a, g["k"], g["C"], g["G"], orc.IR)
    want = {int(i): e for i, e in g["ir"]["ir_expert"].items()}
    for i in range(g["T"]):
        assert int(t.ir_expert[i]) == want.get(i, -1)
    assert t.ir_offset.tolist() == g["ir"]["ir_offset"]
    for e, lst in g["ir"]["ir_lists"].items():
        e = int(e)
        assert t.ir_token[t.ir_offset[e]:t.ir_offset[e + 1]].tolist() == lst
    assert t.slot_token.tolist() == g["vanilla"]["slot_token"]  # IR never touches the slots


def test_capacity3_fr_and_weights():
    g = _gold()
    a = np.array(g["logits"], np.float32)
    t = orc.route(a, g["k"], g["C"], g["G"], orc.FR)
    assert t.slot_token.tolist() == g["fr"]["slot_token"]
    assert t.slot_rank.tolist() == g["fr"]["slot_rank"]
    t3 = orc.route(a, g["k"], g["C"], g["G"], orc.IR | orc.FR)
    assert t3.slot_token.tolist() == g["fr"]["slot_token"]
    for i, w in g["weights_mode3"].items():
        if i == "comment":
            continue
        np.testing.assert_allclose(t3.combine_w[int(i)], w, rtol=0, atol=1e-12)


# --------------------------------------------------------------------------
# P5: independent definition-by-counting formulation, exhaustive on tiny inputs
# --------------------------------------------------------------------------
def counting_router(a, k, C, G, mode):
    """Positions by counting earlier assignments; fill-in by counting better nominees."""
    T, E = len(a), len(a[0])
    order = [sorted(range(E), key=lambda j, i=i: (-a[i][j], j)) for i in range(T)]
    assign = [(r, i, order[i][r]) for r in range(k) for i in range(T)]
    route_slot = [[-1] * (k + 1) for _ in range(T)]
    drops = [0] * T
    n = [0] * E
    for (r, i, e) in assign:
        n[e] += 1
        pos = sum(1 for (r2, i2, e2) in assign if e2 == e and (r2, i2) < (r, i))
        if pos < C:
            route_slot[i][r] = pos
        else:
            drops[i] += 1
    kept = [min(x, C) for x in n]
    ir_expert = [-1] * T
    ir_pos = [-1] * T
    if mode & 1:
        tg, eg = T // G, E // G
        for i in range(T):
            if drops[i]:
                grp = i // tg
                ir_expert[i] = min(range(grp * eg, (grp + 1) * eg), key=lambda j: (-a[i][j], j))
        for i in range(T):
            if ir_expert[i] >= 0:
                ir_pos[i] = sum(1 for i2 in range(i) if ir_expert[i2] == ir_expert[i])
    if mode & 2:
        filled = [False] * T
        for i in range(T):
            e = order[i][k]
            better = sum(1 for i2 in range(T) if i2 != i and order[i2][k] == e and
                         (a[i2][e] > a[i][e] or (a[i2][e] == a[i][e] and i2 < i)))
            filled[i] = better < C - kept[e]
        for i in range(T):
            if filled[i]:
                e = order[i][k]
                route_slot[i][k] = kept[e] + sum(1 for i2 in range(i) if filled[i2] and order[i2][k] == e)
    return order, route_slot, drops, ir_expert, ir_pos


def _compare_with_counting(a, k, C, G, mode):
    an = np.array(a, np.float32)
    t = orc.route(an, k, C, G, mode)
    order, route_slot, drops, ir_expert, ir_pos = counting_router(an.tolist(), k, C, G, mode)
    T, E = an.shape
    for i in range(T):
        assert t.topk_expert[i].tolist() == (order[i][:k + 1] if E > k else order[i][:k] + [-1])
        assert t.route_slot[i].tolist() == route_slot[i], (a, k, C, G, mode)
        assert int(t.drop_count[i]) == drops[i]
        assert int(t.ir_expert[i]) == ir_expert[i]
        assert int(t.ir_pos[i]) == ir_pos[i]
    # the slot table is the inverse of route_slot
    want = -np.ones((E, C), np.int64)
    rank = -np.ones((E, C), np.int64)
    for i in range(T):
        for r in range(k + 1):
            if route_slot[i][r] >= 0:
                want[order[i][r], route_slot[i][r]] = i
                rank[order[i][r], route_slot[i][r]] = r
    assert (t.slot_token == want).all() and (t.slot_rank == rank).all()


@pytest.mark.parametrize("T,E,ks,Gs,Cs,modes", [
    (3, 3, (1, 2), (1, 3), (1,), (0, 1, 2, 3)),
    (3, 3, (1, 2), (3,), (2,), (3,)),
    (4, 2, (1,), (1, 2), (1, 2, 3), (0, 1, 2, 3)),
    (2, 3, (1, 2), (1,), (0, 1, 2), (0, 1, 2, 3)),
])
def test_exhaustive_small(T, E, ks, Gs, Cs, modes):
    alphabet = (-1.0, 0.0, 1.0)
    for flat in itertools.product(alphabet, repeat=T * E):
        a = [list(flat[i * E:(i + 1) * E]) for i in range(T)]
        for k in ks:
            for G in Gs:
                if T % G or E % G:
                    continue
                for C in Cs:
                    for mode in modes:
                        if (mode & 2) and k >= E:
                            continue
                        _compare_with_counting(a, k, C, G, mode)


def test_counting_random_medium():
    rng = np.random.default_rng(5)
    for trial in range(60):
        T, E = 24, 6
        k = int(rng.integers(1, 4))
        G = int(rng.choice([1, 2, 3, 6]))
        C = int(rng.integers(0, 14))
        # few distinct values -> many ties across tokens and experts
        a = rng.integers(-2, 3, (T, E)).astype(np.float32) * 0.5
        _compare_with_counting(a.tolist(), k, C, G, int(rng.integers(0, 4)))


def test_negative_zero_ties_with_positive_zero():
    a = np.array([[-0.0, 0.0, -1.0], [0.0, -0.0, -1.0]], np.float32)
    t = orc.route(a, 1, 2, 1, 0)
    assert t.topk_expert[:, 0].tolist() == [0, 0]  # equal under float comparison -> lower index


# --------------------------------------------------------------------------
# P2: invariants Section 3 states
# --------------------------------------------------------------------------
def _skewed(T, E, seed, sigma=0.8):
    return synth.make_logits(T, E, ("normal", sigma), seed)


@pytest.mark.parametrize("k", [1, 2, 3])
def test_dropped_equals_padding_when_cf_is_k(k):
    # Section 3: with capacity factor k the slots number exactly k*T, so drops == paddings.
    T, E = 960, 8
    a = _skewed(T, E, 11 + k)
    C = k * T // E
    t = orc.route(a, k, C, 2, 0)
    assert int(t.drop_count.sum()) == int((t.slot_token < 0).sum()) > 0


def test_capacity_factor_monotone():
    # larger CF: fewer drops, more padding; smaller CF: the reverse (Section 3)
    T, E, k = 1024, 8, 2
    a = _skewed(T, E, 3)
    prev = None
    for cf in (0.5, 1.0, 1.5, 2.0, 2.5, 3.0):
        t = orc.route(a, k, int(cf * T / E), 4, 0)
        cur = (int(t.drop_count.sum()), int((t.slot_token < 0).sum()))
        if prev:
            assert cur[0] <= prev[0] and cur[1] >= prev[1]
        prev = cur


@pytest.mark.parametrize("mode", [0, 1, 2, 3])
def test_structural_invariants(mode):
    T, E, k, G = 2048, 16, 2, 4
    a = _skewed(T, E, 77, 1.0)
    C = T * k // E
    t = orc.route(a, k, C, G, mode)
    # |R_i| <= k and only successful routes are in R_i
    assert ((t.route_slot[:, :k] >= 0).sum(1) + t.drop_count == k).all()
    assert t.route_slot.max() < C
    # every occupied slot names a token that ranks that expert at the recorded rank
    for e in range(E):
        occ = int(t.expert_count[e])
        assert (t.slot_token[e, :occ] >= 0).all() and (t.slot_token[e, occ:] == -1).all()
        keys = []
        for s in range(occ):
            i, r = int(t.slot_token[e, s]), int(t.slot_rank[e, s])
            assert t.topk_expert[i, r] == e and t.route_slot[i, r] == s
            keys.append((r, i))
        assert keys == sorted(keys)            # (rank, token) order inside an expert
        kept = min(int(t.n_routed[e]), C)
        assert all(r < k for r, _ in keys[:kept]) and all(r == k for r, _ in keys[kept:])
        if not (mode & 2):
            assert occ == kept
    # the top-(k+1) experts are ordered by score and beat every other expert
    for i in range(0, T, 97):
        sel = t.topk_expert[i]
        vals = a[i, sel]
        assert (np.diff(vals) <= 0).all()
        rest = np.setdiff1d(np.arange(E), sel)
        assert a[i, rest].max() <= vals[-1]
    # weights sum to one for routed tokens, zero otherwise
    s = t.combine_w.sum(1)
    routed = (t.token_rows >= 0).any(1)
    np.testing.assert_allclose(s[routed], 1.0, atol=1e-12)
    assert (s[~routed] == 0).all()
    # row space: a bijection between live routes and rows
    R = int(t.row_offset[E])
    assert sorted(t.token_rows[t.token_rows >= 0].tolist()) == list(range(R))
    assert (t.row_token[:R] >= 0).all() and (t.row_token[R:] == -1).all()
    for i in range(0, T, 53):
        for c in range(k + 2):
            row = t.token_rows[i, c]
            if row >= 0:
                assert t.row_token[row] == i and t.row_weight[row] == t.combine_w[i, c]


# --------------------------------------------------------------------------
# P3 / P6: IR special cases (Section 4.1)
# --------------------------------------------------------------------------
def test_ir_single_group_is_top1():
    # Section 4.1: with every expert in one group, IR coincides with top-1 routing.
    T, E = 512, 8
    a = _skewed(T, E, 5)
    t = orc.route(a, 2, 64, 1, orc.IR)
    dropped = t.drop_count > 0
    assert dropped.any()
    assert (t.ir_expert[dropped] == a.argmax(1)[dropped]).all()
    assert (t.ir_expert[~dropped] == -1).all()


def test_ir_one_expert_per_group_and_conservation():
    T, E, G = 1024, 8, 8   # the paper's main setup: one expert per GPU
    a = _skewed(T, E, 6)
    t = orc.route(a, 2, T * 2 // E, G, orc.IR)
    dropped = np.nonzero(t.drop_count > 0)[0]
    assert (t.ir_expert[dropped] == dropped // (T // G)).all()
    # cost of a group = its number of dropped tokens, whatever the routing outcome
    G2 = 4
    t2 = orc.route(a, 2, T * 2 // E, G2, orc.IR)
    for g in range(G2):
        lo, hi = g * T // G2, (g + 1) * T // G2
        n_drop = int((t2.drop_count[lo:hi] > 0).sum())
        e_lo, e_hi = g * E // G2, (g + 1) * E // G2
        assert int(t2.ir_offset[e_hi] - t2.ir_offset[e_lo]) == n_drop
        assert ((t2.ir_expert[lo:hi] == -1) | ((t2.ir_expert[lo:hi] >= e_lo) & (t2.ir_expert[lo:hi] < e_hi))).all()
    # IR lists are in token order
    for e in range(E):
        lst = t2.ir_token[t2.ir_offset[e]:t2.ir_offset[e + 1]]
        assert (np.diff(lst) > 0).all()


def test_dropped_twice_one_ir_route_weight_times_two():
    # k = 2, C = 0: both routings of every token are dropped; IR sends the token to
    # ONE expert with multiplicity 2, which normalises to weight 1 (Eq. 3).
    a = _skewed(64, 4, 9)
    t = orc.route(a, 2, 0, 2, orc.IR)
    assert (t.drop_count == 2).all()
    assert (t.ir_expert >= 0).all()
    np.testing.assert_allclose(t.combine_w[:, 3], 1.0)
    assert (t.combine_w[:, :3] == 0).all()


def test_eq3_weight_with_one_kept_one_dropped():
    # token 2: first routing kept at expert 0, second routing (expert 1) dropped, IR -> expert 0
    a = np.array([[0.0, 5.0], [0.0, 5.0], [2.0, 1.0], [0.0, 5.0]], np.float32)
    t = orc.route(a, 2, 3, 1, orc.IR)
    # rank 0: tokens 0,1,3 -> e1 (slots 0..2), token 2 -> e0.  rank 1: token 2 -> e1 is full -> dropped
    assert t.route_slot[2].tolist() == [0, -1, -1] and t.drop_count[2] == 1
    assert t.ir_expert[2] == 0
    # Eq. 3: (e^2 E_0 + 1 * e^2 E_0) / (e^2 + e^2): kept and IR routes weigh the same
    np.testing.assert_allclose(t.combine_w[2], [0.5, 0.0, 0.0, 0.5], atol=1e-15)


def test_eq3_reduces_to_eq2_without_drops():
    a = _skewed(256, 8, 10)
    big = orc.route(a, 2, 256 * 2, 2, orc.IR)
    assert (big.drop_count == 0).all() and (big.ir_expert == -1).all()
    i = np.arange(256)
    top = np.take_along_axis(a.astype(np.float64), big.topk_expert[:, :2].astype(np.int64), 1)
    w = np.exp(top - top.max(1, keepdims=True))
    w /= w.sum(1, keepdims=True)              # Eq. 2 written out
    np.testing.assert_allclose(big.combine_w[:, :2], w, rtol=1e-13)
    assert (big.combine_w[:, 2:] == 0).all()


# --------------------------------------------------------------------------
# P4: FR == top-(k+1) router at unchanged capacity when nobody is refused (Section 4.2)
# --------------------------------------------------------------------------
@pytest.mark.parametrize("k", [1, 2])
def test_fr_equals_top_k_plus_1_without_contention(k):
    T, E = 512, 8
    a = synth.make_logits(T, E, ("none", 0), 21)
    C = T * (k + 1)                      # nothing can be refused
    fr = orc.route(a, k, C, 2, orc.FR)
    kp1 = orc.route(a, k + 1, C, 2, 0)
    assert (fr.drop_count == 0).all()
    assert (fr.slot_token == kp1.slot_token).all()
    assert (fr.slot_rank == kp1.slot_rank).all()
    assert (fr.route_slot == kp1.route_slot[:, :k + 1]).all()
    np.testing.assert_allclose(fr.combine_w[:, :k + 1], kp1.combine_w[:, :k + 1], rtol=1e-14)
    # moderate capacity: still identical as long as every expert has room for all its nominees
    C2 = T
    fr2 = orc.route(a, k, C2, 2, orc.FR)
    kp2 = orc.route(a, k + 1, C2, 2, 0)
    assert (kp2.drop_count == 0).all()
    assert (fr2.slot_token == kp2.slot_token).all()


def test_fr_picks_highest_scores_and_fills_all_padding_it_can():
    T, E, k = 2048, 8, 1
    a = _skewed(T, E, 31, 0.5)
    C = T // E
    van = orc.route(a, k, C, 2, 0)
    fr = orc.route(a, k, C, 2, orc.FR)
    assert (fr.route_slot[:, :k] == van.route_slot[:, :k]).all()   # kept routes untouched
    for e in range(E):
        nominees = np.nonzero(fr.topk_expert[:, k] == e)[0]
        v = C - min(int(van.n_routed[e]), C)
        chosen = nominees[fr.route_slot[nominees, k] >= 0]
        assert len(chosen) == min(v, len(nominees))
        if len(chosen) and len(chosen) < len(nominees):
            refused = np.setdiff1d(nominees, chosen)
            assert a[chosen, e].min() >= a[refused, e].max()
    # share of unsuccessful routings grows to roughly 1/(k+1) or more (Appendix A remark)
    attempts = (k + 1) * T
    failed = attempts - int((fr.route_slot >= 0).sum())
    assert failed >= T * k * 0 + (attempts - E * C)


def test_modes_are_independent_post_passes():
    # FR and IR both start from the plain top-k result: with both on, the slot
    # table equals FR's and the IR lists equal IR's.
    a = _skewed(1024, 16, 41)
    van = orc.route(a, 2, 128, 4, 0)
    ir = orc.route(a, 2, 128, 4, orc.IR)
    fr = orc.route(a, 2, 128, 4, orc.FR)
    both = orc.route(a, 2, 128, 4, orc.IR | orc.FR)
    assert (both.slot_token == fr.slot_token).all()
    assert (both.ir_expert == ir.ir_expert).all() and (both.ir_token == ir.ir_token).all()
    assert (both.drop_count == van.drop_count).all()


# --------------------------------------------------------------------------
# argument rules
# --------------------------------------------------------------------------
@pytest.mark.parametrize("kw", [
    dict(k=0), dict(k=9), dict(G=3), dict(G=0), dict(C=-1), dict(mode=8), dict(k=8, mode=2),
])
def test_rejects_bad_arguments(kw):
    a = _skewed(64, 8, 1)
    args = dict(k=1, C=8, G=2, mode=0)
    args.update(kw)
    with pytest.raises(orc.OracleError):
        orc.route(a, args["k"], args["C"], args["G"], args["mode"])


def test_rejects_nonfinite_and_accepts_empty():
    a = _skewed(16, 4, 1)
    a[3, 2] = np.inf
    with pytest.raises(orc.OracleError):
        orc.route(a, 1, 4, 1, 0)
    t = orc.route(np.zeros((0, 4), np.float32), 1, 4, 2, 3)
    assert (t.slot_token == -1).all() and t.row_offset.tolist() == [0] * 5
