"""Pins for the oracle's score-priority dropping (mode bit 4): the other reading of Section 3, where a
full expert drops the tokens with the lowest routing scores rather than the latest ones.

Checked against things other than the oracle's selection loop: a hand-worked example, an independent
definition by counting better candidates (exhaustive over small logit matrices), the cases where the
two readings must coincide, the threshold property, invariance under a permutation of the tokens,
and the fact that only WHO is kept may change, never how many."""
import itertools

import numpy as np
import pytest

from oracle import rr_oracle as orc
from paper_2402_12399_b200 import synth

S = orc.SCORE


def test_hand_example():
    # 5 tokens, 2 experts, top-1, capacity 2.  First choices: tokens 0,1,2,4 -> expert 0 with scores
    # 1, 3, 2, 3; token 3 -> expert 1.  Token order keeps tokens 0,1; score priority keeps the two
    # highest scores at expert 0: tokens 1 and 4 (3 and 3), placed in token order.
    a = np.array([[1, 0], [3, 0], [2, 0], [0, 5], [3, 0]], np.float32)
    plain = orc.route(a, 1, 2, 1, 0)
    assert plain.slot_token.tolist() == [[0, 1], [3, -1]]
    t = orc.route(a, 1, 2, 1, S)
    assert t.slot_token.tolist() == [[1, 4], [3, -1]]
    assert t.route_slot[:, 0].tolist() == [-1, 0, -1, 0, 1]
    assert t.drop_count.tolist() == [1, 0, 1, 0, 0]
    # top-2: second choices come after all first choices and compete for what is left; expert 1 has
    # one free slot after token 3 and four second choices with scores 0: the lowest token gets it
    t2 = orc.route(a, 2, 2, 1, S)
    assert t2.slot_token.tolist() == [[1, 4], [3, 0]]
    assert t2.slot_rank.tolist() == [[0, 0], [0, 1]]
    assert t2.drop_count.tolist() == [1, 1, 2, 1, 1]
    # a tie on the threshold score goes to the lower token: capacity 1 keeps token 1, not token 4
    assert orc.route(a, 1, 1, 1, S).slot_token.tolist() == [[1], [3]]


def counting_score_router(a, k, C):
    """route_slot[T][k] by counting: within a rank, a candidate stays iff fewer than the remaining
    capacity of its expert score better; its slot counts the staying candidates of lower index."""
    T, E = len(a), len(a[0])
    order = [sorted(range(E), key=lambda j, i=i: (-a[i][j], j)) for i in range(T)]
    slot = [[-1] * k for _ in range(T)]
    used = [0] * E
    for r in range(k):
        stays = [False] * T
        for i in range(T):
            e = order[i][r]
            better = sum(1 for i2 in range(T) if i2 != i and order[i2][r] == e and
                         (a[i2][e] > a[i][e] or (a[i2][e] == a[i][e] and i2 < i)))
            stays[i] = better < C - used[e]
        for i in range(T):
            if stays[i]:
                e = order[i][r]
                slot[i][r] = used[e] + sum(1 for i2 in range(i) if stays[i2] and order[i2][r] == e)
        for e in range(E):
            used[e] = min(C, used[e] + sum(1 for i in range(T) if order[i][r] == e))
    return slot


def _check_counting(a, k, C):
    an = np.array(a, np.float32)
    t = orc.route(an, k, C, 1, S)
    want = counting_score_router(an.tolist(), k, C)
    assert t.route_slot[:, :k].tolist() == want, (a, k, C)
    assert t.drop_count.tolist() == [sum(1 for x in row if x < 0) for row in want]
    E = an.shape[1]
    inv = -np.ones((E, C), np.int64)
    for i, row in enumerate(want):
        for r, p in enumerate(row):
            if p >= 0:
                inv[t.topk_expert[i, r], p] = i
    assert (t.slot_token == inv).all()


@pytest.mark.parametrize("T,E,ks,Cs", [(3, 3, (1, 2), (1, 2)), (4, 2, (1, 2), (1, 2, 3)), (2, 3, (1, 2, 3), (0, 1, 2))])
def test_exhaustive_small(T, E, ks, Cs):
    for flat in itertools.product((-1.0, 0.0, 1.0), repeat=T * E):
        a = [list(flat[i * E:(i + 1) * E]) for i in range(T)]
        for k in ks:
            for C in Cs:
                _check_counting(a, k, C)


def test_counting_random_medium():
    rng = np.random.default_rng(8)
    for _ in range(60):
        T, E = 24, 6
        a = rng.integers(-2, 3, (T, E)).astype(np.float32) * 0.5       # many ties
        _check_counting(a.tolist(), int(rng.integers(1, 4)), int(rng.integers(0, 14)))


@pytest.mark.parametrize("mode", [0, 1, 2, 3])
def test_same_as_token_order_when_nothing_overflows(mode):
    a = synth.make_logits(512, 8, ("normal", 0.5), 3)
    for k in (1, 2):
        p, s = orc.route(a, k, 512 * k, 2, mode), orc.route(a, k, 512 * k, 2, mode | S)
        for name in ("route_slot", "slot_token", "slot_rank", "drop_count", "ir_expert", "token_rows", "combine_w"):
            assert np.array_equal(getattr(p, name), getattr(s, name)), name


def test_counts_do_not_change_only_who_is_kept():
    a = synth.make_logits(4096, 16, ("normal", 0.8), 5)
    for k, C in [(1, 256), (2, 384), (2, 512)]:
        p, s = orc.route(a, k, C, 4, 0), orc.route(a, k, C, 4, S)
        assert np.array_equal(p.n_routed, s.n_routed) and np.array_equal(p.expert_count, s.expert_count)
        assert np.array_equal(p.slot_rank, s.slot_rank)            # rank r occupies the same slot ranges
        assert int(p.drop_count.sum()) == int(s.drop_count.sum())
        assert not np.array_equal(p.slot_token, s.slot_token)
        # threshold property per (rank, expert): every kept score >= every dropped score
        for r in range(k):
            for e in range(16):
                cand = np.nonzero(s.topk_expert[:, r] == e)[0]
                kept = cand[s.route_slot[cand, r] >= 0]
                lost = cand[s.route_slot[cand, r] < 0]
                if len(kept) and len(lost):
                    assert a[kept, e].min() >= a[lost, e].max()
                assert (np.diff(s.route_slot[kept, r]) > 0).all()   # slots ascend with the token index
        # the kept scores can only be better in total
        gain = sum(a[s.slot_token[e][s.slot_token[e] >= 0], e].sum() - a[p.slot_token[e][p.slot_token[e] >= 0], e].sum()
                   for e in range(16))
        assert gain > 0


def test_kept_set_is_invariant_under_token_permutation():
    # distinct scores, no groups: who is kept does not depend on where a token sits in the batch
    rng = np.random.default_rng(11)
    T, E, k, C = 600, 6, 2, 130
    a = rng.permutation(T * E).reshape(T, E).astype(np.float32) / 7.0
    perm = rng.permutation(T)
    t0, t1 = orc.route(a, k, C, 1, S), orc.route(a[perm], k, C, 1, S)
    assert np.array_equal(t1.route_slot[:, :k] >= 0, (t0.route_slot[:, :k] >= 0)[perm])
    plain0, plain1 = orc.route(a, k, C, 1, 0), orc.route(a[perm], k, C, 1, 0)
    assert not np.array_equal(plain1.route_slot[:, :k] >= 0, (plain0.route_slot[:, :k] >= 0)[perm])


def test_rectifications_run_on_top_of_it():
    a = synth.make_logits(2048, 8, ("normal", 0.7), 9)
    base = orc.route(a, 2, 384, 2, S)
    both = orc.route(a, 2, 384, 2, S | orc.IR | orc.FR)
    assert np.array_equal(base.route_slot[:, :2], both.route_slot[:, :2])       # post-passes leave top-k alone
    assert ((both.ir_expert >= 0) == (base.drop_count > 0)).all()
    assert int((both.route_slot[:, 2] >= 0).sum()) > 0
    np.testing.assert_allclose(both.combine_w.sum(1)[(both.token_rows >= 0).any(1)], 1.0, rtol=1e-12)
