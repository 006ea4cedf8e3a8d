"""Pins for the oracle's synthetic-acceptance chain (Table 1) and the bookkeeping between rounds."""
import os

import numpy as np
import torch

from oracle import recg_oracle as orc
from paper_2609_34388_b200 import synth
from tests._util import oracle_cfg, oracle_weights

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "table1_transitions.txt")


def printed_table():
    rows = [ln.split() for ln in open(GOLDEN) if ln.strip() and not ln.startswith("#")]
    return np.asarray(rows, dtype=np.float64)


def test_matrix_is_the_printed_table_normalised():
    T = printed_table()
    assert T.shape == (3, 3)
    assert np.array_equal(T, np.asarray(orc.TABLE1_PERCENT))
    assert np.all(np.abs(T.sum(axis=1) - 100.0) < 0.02)          # printed to two decimals
    P = orc.chain_matrix()
    assert np.allclose(P.sum(axis=1), 1.0, atol=1e-15)
    assert np.max(np.abs(P * 100.0 - T)) < 0.01                  # normalising moves nothing beyond the printed precision
    # what the text says about it: short and long rounds persist, medium rounds mostly fall back to short
    assert P[0, 0] > 0.5 and P[2, 2] > 0.5 and P[1, 0] > P[1, 1] and abs(P[1, 1] - 0.2242) < 1e-4
    assert orc.TABLE1_INTERVALS == ((1, 8), (9, 16), (17, 32))


def test_stationary_distribution_two_ways():
    P = orc.chain_matrix()
    pi = orc.chain_stationary(P)
    assert abs(pi.sum() - 1.0) < 1e-12 and np.all(pi > 0)
    assert np.max(np.abs(pi @ P - pi)) < 1e-12
    # power iteration and the eigenvector of eigenvalue one agree with the linear solve
    q = np.array([1.0, 0.0, 0.0])
    for _ in range(200):
        q = q @ P
    assert np.max(np.abs(q - pi)) < 1e-12
    w, V = np.linalg.eig(P.T)
    e = np.real(V[:, np.argmin(np.abs(w - 1.0))])
    assert np.max(np.abs(e / e.sum() - pi)) < 1e-10
    assert pi[0] > pi[2] > pi[1]            # short rounds dominate (the text's remark on the 22.42 % entry)


def test_long_walk_reproduces_the_table_and_the_intervals():
    P = orc.chain_matrix()
    rng = np.random.default_rng(4)
    n = 200000
    states, lengths = orc.acceptance_chain(P, orc.TABLE1_INTERVALS, 0, rng.random(n), rng.random(n))
    states, lengths = np.asarray(states), np.asarray(lengths)
    counts = np.zeros((3, 3))
    np.add.at(counts, (states[:-1], states[1:]), 1)
    emp = counts / counts.sum(axis=1, keepdims=True)
    sigma = np.sqrt(P * (1 - P) / counts.sum(axis=1, keepdims=True))
    assert np.all(np.abs(emp - P) < 4 * sigma)
    freq = np.bincount(states, minlength=3) / n
    assert np.max(np.abs(freq - orc.chain_stationary(P))) < 5e-3
    for s, (lo, hi) in enumerate(orc.TABLE1_INTERVALS):
        L = lengths[states == s]
        assert L.min() == lo and L.max() == hi
        assert abs(L.mean() - (lo + hi) / 2) < 0.1          # uniform inside the interval
    # deterministic corner cases: u = 0 takes the first column and the interval's low end, u -> 1 the last ones
    st, ln = orc.acceptance_chain(P, orc.TABLE1_INTERVALS, 1, [0.0, 0.999999, 0.0], [0.0, 0.0, 0.999999])
    assert st == [1, 0, 2] and ln == [9, 1, 32]
    # the boundary between two columns belongs to the later one (cumulative probability <= u)
    st, _ = orc.acceptance_chain(P, orc.TABLE1_INTERVALS, 0, [P[0, 0], np.nextafter(P[0, 0], 0)], [0.5, 0.5, ])
    assert st == [0, 1]


def test_advance_round_is_the_bookkeeping_of_the_pinned_loop():
    """spec_decode (pinned by losslessness) records every round; advance_round applied to a round's record must give the
    next round's context length and verify tokens."""
    shape = synth.ModelShape(n_layers=2, hidden=32, n_q_heads=4, n_kv_heads=2, head_dim=8, ffn=48, vocab=64)
    W = synth.model_weights(shape, seed=0, dtype=torch.float32)
    for k in ("wqkv", "wo", "w_gate_up", "w_down"):
        W[k] = [w * 8.0 for w in W[k]]
    W["embed"] = W["embed"] * 20.0
    W["lm_head"] = W["lm_head"] * 20.0
    cfg, W64 = oracle_cfg(shape), oracle_weights(W)
    prompt = synth.token_ids(12, shape.vocab, seed=7).tolist()
    truth = orc.greedy_ar(cfg, W64, prompt, 40)

    def plant(t, out, y):     # teacher-forced drafts with a mismatch in every third round: reuse, rejection and bonus occur
        if t % 3 == 2 or len(y) == 1:
            k = len(out)
            y = [y[0]] + truth[k: k + 4]
            if t % 3 == 2:
                y[2] = (y[2] + 1) % (shape.vocab - 1)
        return y

    _, trace, _ = orc.spec_decode(cfg, W64, prompt, 4, 9, plant=plant)
    seen_reuse = seen_reject = False
    for t in range(len(trace) - 1):
        r = trace[t]
        new_L, y = orc.advance_round(r["L"], r["y"], r["b"], r["accept_len"], r["emitted"][-1], r["cont_hit"], r["next_draft"])
        assert new_L == r["new_L"] == trace[t + 1]["L"]
        nxt = trace[t + 1]["y"]
        if (t + 1) % 3 != 2 and len(y) > 1:
            assert nxt == y                       # a reused block is verified as it is
        assert nxt[0] == y[0] == r["emitted"][-1]
        seen_reuse |= bool(r["cont_hit"])
        seen_reject |= r["accept_len"] < len(r["y"]) - 1
    assert seen_reject


def test_planted_rounds_lengths():
    # v = 1 first (only the known token), block 8 reused only after full acceptance
    tr = orc.planted_rounds(100, 1, [8, 8, 8, 8, 8], [5, 32, 3, 8, 1])
    #        L    v  b  a  emitted reused
    assert tr[0] == (100, 1, 8, 0, 1, True)      # a lone known token is always "fully accepted": its block is reused
    assert tr[1] == (101, 8, 8, 7, 8, True)      # 32 is cut to the 8 tokens there are
    assert tr[2] == (109, 8, 8, 2, 3, False)
    assert tr[3] == (112, 1, 8, 0, 1, True)
    assert tr[4] == (113, 8, 8, 0, 1, False)
    # context lengths grow by what was emitted
    assert all(tr[i + 1][0] == tr[i][0] + tr[i][4] for i in range(4))
    # no block: nothing to reuse
    assert orc.planted_rounds(10, 4, [0, 0], [4, 4]) == [(10, 4, 0, 3, 4, False), (14, 1, 0, 0, 1, False)]


def test_workload_generator_draws_from_the_same_chain():
    """The benchmark's input generator (synth.acceptance_chain_lengths) has its own copy of the table: its transition
    counts over a long run must match the oracle's matrix, and its lengths must stay inside the intervals."""
    assert synth.ACCEPT_TRANSITIONS == orc.TABLE1_PERCENT and synth.ACCEPT_INTERVALS == orc.TABLE1_INTERVALS
    L = synth.acceptance_chain_lengths(60000, 2, seed=8)
    assert L.min() == 1 and L.max() == 32
    P = orc.chain_matrix()
    for r in range(2):
        states = np.digitize(L[:, r], [9, 17])
        counts = np.zeros((3, 3))
        np.add.at(counts, (states[:-1], states[1:]), 1)
        emp = counts / counts.sum(axis=1, keepdims=True)
        sigma = np.sqrt(P * (1 - P) / counts.sum(axis=1, keepdims=True))
        assert np.all(np.abs(emp - P) < 4.5 * sigma)
