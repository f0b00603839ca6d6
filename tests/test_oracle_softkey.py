"""Pins for the oracle's softmax-valued FR key (mode bit 8): Appendix A calls the softmax values g_ij
"routing scores"; read that way, the second stage of Fill-in Rectification (Section 4.2) ranks an
expert's nominees by g_ie rather than by the raw logit a_ie.  The key is a single-precision softmax
with every operation fixed, so that it can decide an integer reproducibly.

Checked against things other than the oracle's own code: the textbook softmax in double precision
(accuracy and closed forms of the fixed recipe), a hand-worked example in which the two keys pick
different tokens, an independent definition by counting better nominees on double-precision softmax
values, and the cases in which both keys must give the same tables."""
import math

import numpy as np
import pytest

from oracle import rr_oracle as orc
from paper_2402_12399_b200 import synth

K = orc.FR_SOFTMAX


def softmax64(row):
    x = np.exp(row.astype(np.float64) - float(row.max()))
    return x / x.sum()


def test_fixed_softmax_is_the_softmax():
    rng = np.random.default_rng(1)
    for E in (2, 3, 8, 64, 256):
        for scale in (0.1, 1.0, 4.0, 20.0):
            row = (rng.normal(size=E) * scale).astype(np.float32)
            g = orc.softmax32(row)
            want = softmax64(row)
            big = want > 1e-30
            # a - m rounds to fp32 (half an ulp of |a - m|, which exp turns into a relative error), exp
            # itself to ~1e-7, E-1 additions of positive terms, one division
            tol = 3e-7 + E * 6e-8 + np.abs(row.astype(np.float64) - float(row.max())) * 6e-8
            assert (np.abs(g / want - 1.0)[big] < tol[big]).all(), (E, scale)
            assert abs(float(g.astype(np.float64).sum()) - 1.0) < E * 1e-7


def test_fixed_softmax_closed_forms():
    # equal logits: exactly 1/E when E is a power of two (e^0 = 1 exactly, exact sum, exact quotient)
    for E in (2, 4, 64):
        assert orc.softmax32(np.full(E, 3.25, np.float32)).tolist() == [1.0 / E] * E
    # two logits ln 2 apart (as close as fp32 allows): 2/3 and 1/3
    g = orc.softmax32(np.array([math.log(2.0), 0.0], np.float32))
    assert abs(g[0] - 2 / 3) < 1e-7 and abs(g[1] - 1 / 3) < 1e-7
    # shift invariance is exact when the shifted logits and their differences are representable
    row = np.array([0.5, -1.25, 2.0, 0.0], np.float32)
    assert orc.softmax32(row).tolist() == orc.softmax32(row + np.float32(8.0)).tolist()
    # order inside a row follows the logits, the largest has g = 1/Z
    row = np.random.default_rng(2).normal(size=32).astype(np.float32)
    g = orc.softmax32(row)
    assert (np.argsort(-g, kind="stable") == np.argsort(-row, kind="stable")).all()
    # far below the maximum the clamp at -80 takes over: tiny but positive and normal
    g = orc.softmax32(np.array([0.0, -500.0], np.float32))
    assert g[0] == 1.0 and 0.0 < g[1] < 1e-30 and g[1] >= np.finfo(np.float32).tiny


def test_hand_example_keys_disagree():
    # top-1 with FR, 3 experts, capacity 2.  Tokens 0 and 1 take expert 0; expert 1 receives nobody
    # and has two padding slots; tokens 2, 3, 4 take expert 2 (the last is dropped) and all three
    # nominate expert 1 as their second choice.
    #   token 2: a = (-9, 3.0, 9): g_1 = e^-6 / (1 + e^-6 + e^-18) ~ 0.00247
    #   token 3: a = (-9, 2.0, 3): g_1 = e^-1 / (1 + e^-1 + e^-12) ~ 0.269
    #   token 4: a = (-9, 1.0, 5): g_1 = e^-4 / (1 + e^-4 + e^-14) ~ 0.0180
    # tokens 0, 1 nominate expert 2, which is full.  By raw logit expert 1 takes tokens 2 and 3
    # (3.0 and 2.0); by softmax value it takes tokens 3 and 4.
    a = np.array([[9, 0, 1], [9, 0, 1], [-9, 3, 9], [-9, 2, 3], [-9, 1, 5]], np.float32)
    by_logit = orc.route(a, 1, 2, 1, orc.FR)
    by_soft = orc.route(a, 1, 2, 1, orc.FR | K)
    assert by_logit.slot_token.tolist() == [[0, 1], [2, 3], [2, 3]]
    assert by_soft.slot_token.tolist() == [[0, 1], [3, 4], [2, 3]]
    assert by_soft.slot_rank.tolist() == [[0, 0], [1, 1], [0, 0]]
    assert by_soft.route_slot.tolist() == [[0, -1], [1, -1], [0, -1], [1, 0], [-1, 1]]
    assert by_soft.drop_count.tolist() == by_logit.drop_count.tolist() == [0, 0, 0, 0, 1]
    # token 4: dropped at its first choice, filled in at expert 1: all its weight goes there
    assert by_soft.combine_w[4].tolist() == [0.0, 1.0, 0.0]


def counting_fill(a, k, C, t):
    """Fill-in by counting on double-precision softmax values: nominee i of expert e is placed iff
    fewer than v_e nominees of e have a larger g (ties: lower token); slot = kept_e + number of placed
    nominees of lower index.  `t` supplies only the top-k stage (kept counts and the nominations)."""
    T, E = a.shape
    g = np.stack([softmax64(a[i]) for i in range(T)])
    fill = [-1] * T
    for e in range(E):
        nom = [i for i in range(T) if t.topk_expert[i, k] == e]
        kept = min(int(t.n_routed[e]), C)
        v = C - kept
        placed = [i for i in nom
                  if sum(1 for j in nom if j != i and (g[j, e] > g[i, e] or (g[j, e] == g[i, e] and j < i))) < v]
        for p, i in enumerate(placed):
            fill[i] = kept + p
    return fill, g


def test_selection_matches_counting_on_double_precision_softmax():
    rng = np.random.default_rng(5)
    done = 0
    for seed in range(40):
        T, E = 96, 8
        a = (rng.normal(size=(T, E)) * 1.5 + rng.normal(size=E)).astype(np.float32)
        k, C = int(rng.integers(1, 3)), int(rng.integers(8, 30))
        t = orc.route(a, k, C, 2, orc.FR | orc.IR | K)
        fill, g = counting_fill(a, k, C, t)
        # the fp32 key is good to ~1e-6; skip inputs where two nominees of one expert are closer
        gk = np.array([g[i, t.topk_expert[i, k]] for i in range(T)])
        close = False
        for e in range(E):
            v = np.sort(gk[t.topk_expert[:, k] == e])
            if len(v) > 1 and (np.diff(v) / v[1:]).min() < 1e-4:
                close = True
        if close:
            continue
        assert t.route_slot[:, k].tolist() == fill, seed
        done += 1
    assert done >= 25


def test_differs_from_logit_key_under_contention_only():
    a = synth.make_logits(4096, 16, ("normal", 0.8), 7)
    # contention: fewer padding slots than nominees somewhere -> the keys choose differently
    p, s = orc.route(a, 2, 600, 4, orc.FR | orc.IR), orc.route(a, 2, 600, 4, orc.FR | orc.IR | K)
    for name in ("topk_expert", "drop_count", "ir_expert", "ir_pos", "n_routed", "expert_count"):
        assert np.array_equal(getattr(p, name), getattr(s, name)), name
    assert np.array_equal(p.route_slot[:, :2], s.route_slot[:, :2])          # the top-k stage is untouched
    assert int((p.route_slot[:, 2] >= 0).sum()) == int((s.route_slot[:, 2] >= 0).sum())
    assert not np.array_equal(p.route_slot[:, 2], s.route_slot[:, 2])
    # threshold property on the softmax key, per expert
    g = np.stack([orc.softmax32(a[i]) for i in range(a.shape[0])])
    for e in range(16):
        nom = np.nonzero(s.topk_expert[:, 2] == e)[0]
        inn, out = nom[s.route_slot[nom, 2] >= 0], nom[s.route_slot[nom, 2] < 0]
        if len(inn) and len(out):
            assert g[inn, e].min() >= g[out, e].max()
        assert (np.diff(s.route_slot[inn, 2]) > 0).all()
    # no contention (every nominee fits): the key cannot matter, tables are identical
    big = 4096 * 3
    p, s = orc.route(a, 2, big, 4, orc.FR), orc.route(a, 2, big, 4, orc.FR | K)
    for name in ("route_slot", "slot_token", "slot_rank", "token_rows", "combine_w"):
        assert np.array_equal(getattr(p, name), getattr(s, name)), name


def test_needs_fr():
    a = synth.make_logits(64, 4, ("normal", 0.5), 1)
    with pytest.raises(orc.OracleError):
        orc.route(a, 1, 16, 1, K)
    with pytest.raises(orc.OracleError):
        orc.route(a, 1, 16, 1, K | orc.IR)
    orc.route(a, 1, 16, 1, K | orc.FR | orc.SCORE)      # combines with score-priority dropping
