"""Pins for greedy verification, the confidence statistics and the KV index work."""
import math

import numpy as np
import pytest
import scipy.special
import scipy.stats

from oracle import recg_oracle as orc
from paper_2609_34388_b200 import synth


def test_stats_uniform_logits():
    V = 1000
    s = orc.row_stats(np.full(V, 3.25))
    assert s["top1"] == 0 and s["top2"] == 1
    assert abs(s["p1"] - 1.0 / V) < 1e-15 and abs(s["margin"]) < 1e-15
    assert abs(s["entropy"] - math.log(V)) < 1e-12


def test_stats_dominant_logit():
    x = np.zeros(500)
    x[123] = 50.0
    s = orc.row_stats(x)
    assert s["top1"] == 123 and s["top2"] == 0
    assert abs(s["p1"] - 1.0) < 1e-15 and s["entropy"] < 1e-15 + 60 * 499 * math.exp(-50)
    assert s["logit_gap"] == 50.0


def test_stats_two_equal_maxima_lowest_index_first():
    x = np.array([0.0, 2.0, -1.0, 2.0, 1.0])
    s = orc.row_stats(x)
    assert (s["top1"], s["top2"]) == (1, 3)
    assert s["margin"] == 0.0 and s["logit_gap"] == 0.0


def test_stats_two_point_closed_form():
    # logits (a, 0, -inf-like): p1 = sigmoid(a)
    a = 1.7
    x = np.array([-1e9, a, 0.0, -1e9])
    s = orc.row_stats(x)
    p = 1.0 / (1.0 + math.exp(-a))
    assert abs(s["p1"] - p) < 1e-15 and abs(s["p2"] - (1 - p)) < 1e-15
    H = -(p * math.log(p) + (1 - p) * math.log(1 - p))
    assert abs(s["entropy"] - H) < 1e-14


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_stats_vs_library(seed):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal(4096) * 3.0
    s = orc.row_stats(x)
    p = scipy.special.softmax(x)
    order = np.argsort(-x, kind="stable")
    assert s["top1"] == order[0] and s["top2"] == order[1]
    assert abs(s["p1"] - p[order[0]]) < 1e-14 and abs(s["p2"] - p[order[1]]) < 1e-14
    assert abs(s["entropy"] - scipy.stats.entropy(p)) < 1e-12
    assert s["entropy"] <= math.log(4096)


def test_greedy_accept_examples():
    # y0 is known; y1.. are drafts; top1[i] is the verifier's token after y_i
    assert orc.greedy_accept([5, 6, 7, 8], [1, 5, 6, 7]) == 3       # all drafts accepted
    assert orc.greedy_accept([5, 6, 7, 8], [1, 5, 9, 7]) == 1       # first mismatch at draft 2
    assert orc.greedy_accept([5, 6, 7, 8], [1, 4, 6, 7]) == 0       # later matches do not count
    assert orc.greedy_accept([5], [1]) == 0                         # nothing drafted


def test_verify_round_emits_prefix_plus_verifier_token():
    V = 16
    y = [3, 7, 2, 9]
    top = [7, 2, 5, 1, 11, 12]          # rows 0..3 verify, rows 4..5 draft
    logits = np.zeros((6, V))
    for r, t in enumerate(top):
        logits[r, t] = 4.0 + r
    r = orc.verify_round(logits, y, 2)
    assert r["accept_len"] == 2 and r["emitted"] == [7, 2, 5] and r["n_emitted"] == 3
    assert r["next_draft"] == [11, 12] and r["cont_hit"] is False
    ent = [orc.row_stats(logits[i])["entropy"] for i in range(3)]
    assert abs(r["entropy_mean"] - sum(ent) / 3) < 1e-15


def test_continuation_rule():
    V = 16
    y = [3, 7]
    logits = np.zeros((4, V))
    for r, t in enumerate([7, 9, 9, 4]):      # full accept, bonus 9, first drafted token 9
        logits[r, t] = 5.0
    assert orc.verify_round(logits, y, 2)["cont_hit"] is True
    logits[2, 9] = 0.0
    logits[2, 8] = 5.0                         # first drafted token 8 != bonus 9
    assert orc.verify_round(logits, y, 2)["cont_hit"] is False
    logits[2, 8] = 0.0
    logits[2, 9] = 5.0
    assert orc.verify_round(logits, [3, 6], 2)["cont_hit"] is False   # not fully accepted


@pytest.mark.parametrize("k", [4, 8, 16])
def test_planted_accept_lengths(k):
    B, V = 24, 512
    lg = synth.logits_normal(B * (k + 1), V, seed=6 + k).double().numpy()
    acc = synth.planted_accept_lengths(B, k, 0.25, seed=4 + k)
    acc[0], acc[1] = 0, k                      # both ends
    y = synth.plant_drafts(lg.argmax(axis=1), B, k, acc, V, seed=4)
    res = orc.verify_batch(lg, [k + 1] * B, [0] * B, y.reshape(-1))
    assert [r["accept_len"] for r in res] == acc.tolist()
    for r, a, yy in zip(res, acc, y):
        assert r["emitted"][:-1] == yy[1: a + 1].tolist()


def test_bf16_ties_resolve_to_lowest_index():
    # bf16 N(0,1) rows of this width often tie at the maximum
    lg = synth.logits_normal(64, 128256 // 8, seed=9)
    x = lg.double().numpy()
    ties = 0
    for r in range(x.shape[0]):
        s = orc.row_stats(x[r])
        m = x[r].max()
        idx = np.nonzero(x[r] == m)[0]
        assert s["top1"] == idx[0]
        if len(idx) > 1:
            ties += 1
            assert s["top2"] == idx[1] and s["margin"] == 0.0
    assert ties > 0


def test_kv_commit_bruteforce():
    ps = 4
    pt = [9, 2, 7, 5, 0]
    L, v, b, a = 6, 5, 3, 2
    r = orc.kv_commit(L, v, b, a, pt, ps)
    assert r["new_ctx_len"] == 9
    slot = {p: pt[p // ps] * ps + p % ps for p in range(20)}
    assert r["commit_slots"] == [slot[6], slot[7], slot[8]]
    assert r["rollback_slots"] == [slot[p] for p in range(9, 14)]
    # pages hold positions [0,4) [4,8) [8,12) [12,16): page 3 (phys 5) is wholly beyond 9
    assert r["freed_pages"] == [5]
    # commit + rollback exactly tile the new positions, no overlap
    assert len(set(r["commit_slots"]) | set(r["rollback_slots"])) == v + b


def test_kv_commit_page_boundary():
    ps = 16
    pt = list(range(100, 110))
    r = orc.kv_commit(31, 8, 8, 0, pt, ps)       # new length 32: exactly fills page 1
    assert r["new_ctx_len"] == 32 and r["freed_pages"] == [102]
    r = orc.kv_commit(31, 8, 8, 7, pt, ps)       # new length 39
    assert r["freed_pages"] == []
