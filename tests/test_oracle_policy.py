"""Pins for the oracle's block-size rule (Sec. 5.2, Eq. 2-3): closed forms, pairwise-comparison brute force,
limits of the cost weight, tie breaking, binning at the edges and the state update."""
import itertools

import numpy as np
import pytest

from oracle import recg_oracle as orc
from paper_2609_34388_b200 import synth


def test_certainty_is_minus_the_mean_of_two_entropies():
    assert orc.policy_certainty(0.5, 1.5) == -1.0
    assert orc.policy_certainty(0.0, 0.0) == 0.0
    s = orc.policy_certainty(np.float32(0.1), np.float32(0.2), np.float32)
    assert s.dtype == np.float32 and s == np.float32(-0.5) * (np.float32(0.1) + np.float32(0.2))


def test_binning_at_and_between_edges():
    blocks = [8, 16, 32]
    edges = [-2.0, -1.0]
    # value depends on the bin only: candidate j is best in bin j
    value = np.zeros((3, 3, 3, 2))
    for j in range(3):
        value[j, j] = 1.0
    cost = np.zeros(3)
    for s, want in [(-5.0, 8), (-2.0000001, 8), (-2.0, 16), (-1.5, 16), (-1.0, 32), (0.0, 32)]:
        assert orc.policy_select(s, 0, 0, blocks, edges, value, cost)[1] == want, s


def test_cost_weight_limits_and_ties():
    t = synth.policy_table()
    blocks, edges, value = t["blocks"], t["s_edges"], t["value"]
    for s, jp, f in itertools.product([-2.9, -1.4, -0.1], range(3), (0, 1)):
        k = int(np.sum(edges <= s))
        # no cost: the candidate with the largest estimate; overwhelming cost: the cheapest candidate
        assert orc.policy_select(s, jp, f, blocks, edges, value, np.zeros(3))[0] == int(np.argmax(value[:, k, jp, f]))
        assert orc.policy_select(s, jp, f, blocks, edges, value, np.array([1e3, 2e3, 3e3]))[0] == 0
        assert orc.policy_select(s, jp, f, blocks, edges, value, np.array([3e3, 2e3, 1e3]))[0] == 2
    flat = np.ones((3, len(edges) + 1, 3, 2))
    assert orc.policy_select(-1.0, 1, 1, blocks, edges, flat, np.zeros(3)) == (0, 8)          # tie: smaller block
    assert orc.policy_select(-1.0, 1, 1, blocks, edges, flat, np.array([0.5, 0.0, 0.0])) == (1, 16)


def test_selection_equals_pairwise_comparisons_on_the_geometric_model():
    """With per-token acceptance probability p and a bonus token, a block of B drafts+1 emits (1 - p^B)/(1 - p) tokens
    in expectation.  Under a cost c per drafted token, doubling B pays iff the extra expected tokens exceed the extra
    cost; that chain of pairwise inequalities must select what the argmax selects."""
    blocks = [8, 16, 32]
    edges = np.linspace(-3.0, 0.0, 31)[1:-1]
    centres = np.linspace(-3.0, 0.0, 31)[:-1] + 0.05
    ps = 1.0 / (1.0 + np.exp(-(3.0 * centres + 5.0)))
    V = lambda p, B: (1.0 - p ** B) / (1.0 - p)
    value = np.zeros((3, 30, 3, 2))
    for j, B in enumerate(blocks):
        for k, p in enumerate(ps):
            value[j, k] = V(p, B)
    seen = set()
    for c in (0.02, 0.05, 0.1):
        cost = np.array([c * B for B in blocks])
        for k, (s, p) in enumerate(zip(centres, ps)):
            got = orc.policy_select(s, 0, 0, blocks, edges, value, cost)[1]
            want = 8
            if V(p, 16) - V(p, 8) > c * 8 and V(p, 16) - c * 16 >= V(p, 32) - c * 32:
                want = 16
            if V(p, 32) - V(p, 8) > c * 24 and V(p, 32) - V(p, 16) > c * 16:
                want = 32
            assert got == want, (c, p)
            seen.add(got)
        # more certainty never shrinks the block in this model
        picks = [orc.policy_select(s, 0, 0, blocks, edges, value, cost)[1] for s in centres]
        assert picks == sorted(picks)
    assert seen == {8, 16, 32}


def test_state_update_and_history():
    t = synth.policy_table()
    st = {"e1": [0.4, 0.4, 0.4, 0.4], "e2": [1.0, 1.0, 1.0, 1.0], "block_index": [0, 1, 2, 1], "full": [0, 1, 0, 1]}
    ent = [0.2, 0.3, 9.9, 0.1]
    acc = [3, 2, 0, 0]
    ver = [4, 4, 0, 1]          # full acceptance; partial; a request that verified nothing; one known token only
    before = {k: list(v) for k, v in st.items()}
    out = orc.policy_step(st, ent, acc, ver, t["blocks"], t["s_edges"], t["value"], t["cost"])
    assert st["e1"] == [0.2, 0.3, 0.4, 0.1] and st["e2"] == [0.4, 0.4, 1.0, 0.4]
    assert st["full"] == [1, 0, 0, 0]
    for r in range(4):
        s = -(st["e1"][r] + st["e2"][r]) / 2
        j, B = orc.policy_select(s, before["block_index"][r], st["full"][r], t["blocks"], t["s_edges"], t["value"], t["cost"])
        assert out[r] == B and st["block_index"][r] == j
    # the previous block size and the acceptance flag are really used: some table entry flips a decision
    flips = 0
    for s in np.linspace(-2.9, -0.1, 40):
        base = orc.policy_select(s, 0, 0, t["blocks"], t["s_edges"], t["value"], t["cost"])[0]
        flips += int(any(orc.policy_select(s, jp, f, t["blocks"], t["s_edges"], t["value"], t["cost"])[0] != base
                         for jp in range(3) for f in (0, 1)))
    assert flips > 0


def test_float32_mode_matches_float64_away_from_edges():
    t = synth.policy_table()
    rng = np.random.default_rng(0)
    for _ in range(200):
        e1, e2 = rng.uniform(0, 3, 2)
        s64 = float(orc.policy_certainty(e1, e2))
        if np.min(np.abs(t["s_edges"] - s64)) < 1e-4:
            continue
        s32 = orc.policy_certainty(np.float32(e1), np.float32(e2), np.float32)
        a = orc.policy_select(s64, 1, 0, t["blocks"], t["s_edges"], t["value"], t["cost"])
        b = orc.policy_select(s32, 1, 0, t["blocks"], t["s_edges"], t["value"], t["cost"], np.float32)
        assert a == b
