"""Pins for the oracle's predictive draft-verify overlap (Sec. 5.1): every branch row against the
standalone round it hypothesises, visibility by brute force over the definition, the selection and
reuse rules on hand-made cases, and losslessness of the recursive loop."""
import numpy as np
import pytest
import torch

from oracle import recg_oracle as orc
from paper_2609_34388_b200 import synth
from tests._util import oracle_cfg, oracle_weights


@pytest.fixture(scope="module")
def small():
    shape = synth.ModelShape(n_layers=2, hidden=32, n_q_heads=4, n_kv_heads=2, head_dim=8, ffn=48, vocab=64)
    W = synth.model_weights(shape, seed=0, dtype=torch.float32)
    for k in ("wqkv", "wo", "w_gate_up", "w_down"):
        W[k] = [w * 8.0 for w in W[k]]
    W["embed"] = W["embed"] * 20.0
    W["lm_head"] = W["lm_head"] * 20.0
    synth.perturb_norm_gains(W)
    return shape, oracle_cfg(shape), oracle_weights(W)


def test_visibility_by_brute_force():
    """Row by row from the words of Sec. 5.1: a branch sees the canonical prefix up to the draft it
    replaces, never the verifier's later tokens, never another branch."""
    L, v, b, bc = 5, 6, 3, 4
    corr = [(2, 11), (5, 12)]
    pos, vis, kind = orc.overlap_round_rows(L, v, b, corr, bc)
    n = v + b + 2 * (1 + bc)
    assert vis.shape == (n, L + n) and len(kind) == n
    owner = ["v"] * v + ["c"] * b + ["k0"] * (1 + bc) + ["k1"] * (1 + bc)
    idx_of = {"k0": 2, "k1": 5}
    for r in range(n):
        for c in range(L + n):
            if c < L:
                want = True                                  # committed context: everybody
            else:
                j = c - L
                o_r, o_c = owner[r], owner[j]
                if o_r == "v":
                    want = o_c == "v" and j <= r
                elif o_r == "c":
                    want = o_c in ("v", "c")
                else:
                    i = idx_of[o_r]
                    if o_c == "v":
                        want = j < i
                    elif o_c == o_r:
                        first = owner.index(o_r)
                        want = (j == r) if r == first else True   # replacement token: causal; masks: whole branch
                    else:
                        want = False
            assert bool(vis[r, c]) == want, (r, c)
    assert pos[:v].tolist() == list(range(L, L + v))
    assert pos[v: v + b].tolist() == list(range(L + v, L + v + b))
    assert pos[v + b: v + b + 1 + bc].tolist() == list(range(L + 2, L + 2 + 1 + bc))
    assert pos[v + b + 1 + bc:].tolist() == list(range(L + 5, L + 5 + 1 + bc))
    assert kind == ["v"] * v + ["c"] * b + (["r"] + ["m"] * bc) * 2


def test_no_branches_is_the_plain_round(small):
    shape, cfg, W = small
    ids = synth.token_ids(20, shape.vocab, seed=11).tolist()
    kv, L, _ = orc.prefill(cfg, W, ids[:15])
    y = ids[14:18]
    a, _, _ = orc.fused_round_cached(cfg, W, kv, L, y, 5)
    c, _, _ = orc.overlap_round_cached(cfg, W, kv, L, y, 5, [], 7)
    assert np.array_equal(a, c)


@pytest.mark.parametrize("b,bc", [(4, 4), (0, 3), (5, 0)])
def test_branch_rows_equal_the_round_they_hypothesise(small, b, bc):
    """If the verifier accepts y_1..y_{i-1} and emits the replacement r at index i, the next round is
    [r | block] over a context of L + i tokens.  The correction branch must already hold exactly
    those logits, and the verifier / continuation rows must not notice the branches."""
    shape, cfg, W = small
    ids = synth.token_ids(30, shape.vocab, seed=12).tolist()
    kv, L, _ = orc.prefill(cfg, W, ids[:17])
    y = ids[16:22]
    v = len(y)
    corr = [(2, 40), (4, 7)]
    logits, kv_new, _ = orc.overlap_round_cached(cfg, W, kv, L, y, b, corr, bc)
    plain, kv_plain, _ = orc.fused_round_cached(cfg, W, kv, L, y, b)
    assert np.max(np.abs(logits[: v + b] - plain)) < 1e-11
    for (K, V), (Kp, Vp) in zip(kv_new, kv_plain):
        assert np.max(np.abs(K[: L + v + b] - Kp)) < 1e-11 and np.max(np.abs(V[: L + v + b] - Vp)) < 1e-11
    for k, (i, tok) in enumerate(corr):
        pre = [(K[: L + i], V[: L + i]) for (K, V) in kv_plain]      # context + y_0 .. y_{i-1}
        alone, kv_alone, _ = orc.fused_round_cached(cfg, W, pre, L + i, [tok], bc)
        r0 = v + b + k * (1 + bc)
        assert np.max(np.abs(logits[r0: r0 + 1 + bc] - alone)) < 1e-10
        for (K, V), (Ka, Va) in zip(kv_new, kv_alone):
            assert np.max(np.abs(K[L + r0: L + r0 + 1 + bc] - Ka[L + i:])) < 1e-10
            assert np.max(np.abs(V[L + r0: L + r0 + 1 + bc] - Va[L + i:])) < 1e-10
    # changing the replacement token of one branch changes that branch only
    other, _, _ = orc.overlap_round_cached(cfg, W, kv, L, y, b, [(2, 41), (4, 7)], bc)
    r0, r1 = v + b, v + b + 1 + bc
    assert np.max(np.abs(other[:r0] - logits[:r0])) < 1e-12
    assert np.max(np.abs(other[r1:] - logits[r1:])) < 1e-12
    assert np.max(np.abs(other[r0] - logits[r0])) > 1e-9


def test_select_branches_rule():
    # index 0 is never a draft; threshold is strict; earliest two kept; continuation iff <= 2 risky
    m = [0.0, 0.9, 0.3, 0.5, 0.49, 0.1]
    s = [9, 10, 11, 12, 13, 14]
    corr, cont = orc.select_branches(m, s)
    assert corr == [(2, 11), (4, 13)] and cont is False      # three risky positions: 2, 4, 5
    corr, cont = orc.select_branches(m[:5], s[:5])
    assert corr == [(2, 11), (4, 13)] and cont is True
    corr, cont = orc.select_branches([0.0, 0.9, 0.8], [1, 2, 3])
    assert corr == [] and cont is True
    corr, cont = orc.select_branches([0.0], [1])
    assert corr == [] and cont is True
    corr, cont = orc.select_branches(m, s, delta=0.2)
    assert corr == [(5, 14)] and cont is True


def planted_logits(rows, vocab, top1, top2=None, gap=4.0):
    x = np.zeros((rows, vocab))
    for r in range(rows):
        x[r, top1[r]] = 10.0
        if top2 is not None:
            x[r, top2[r]] = 10.0 - gap
    return x


def test_reuse_rules_planted():
    V = 32
    y = [3, 4, 5, 6]                       # y_0 known, drafts 4 5 6
    v, b, bc = 4, 3, 2
    corr = [(2, 20), (3, 21)]
    n = v + b + 2 * (1 + bc)
    # verifier agrees with y_1, then says 20 where the draft was 5: accept length 1, correction 0 hits
    top1 = [4, 20, 9, 9] + [9, 8, 7] + [15, 16, 17] + [18, 19, 22]
    r = orc.verify_overlap_round(planted_logits(n, V, top1), y, b, corr, bc)
    assert r["accept_len"] == 1 and r["emitted"] == [4, 20]
    assert r["corr_hit"] == [True, False] and r["cont_hit"] is False
    assert r["corr_draft"] == [[16, 17], [19, 22]]
    # same position rejected but another token: no hit
    top1[1] = 23
    r = orc.verify_overlap_round(planted_logits(n, V, top1), y, b, corr, bc)
    assert r["accept_len"] == 1 and r["corr_hit"] == [False, False]
    # rejected at index 3 with the second branch's token
    top1[1], top1[2] = 5, 21
    r = orc.verify_overlap_round(planted_logits(n, V, top1), y, b, corr, bc)
    assert r["accept_len"] == 2 and r["corr_hit"] == [False, True]
    # the replacement token appears, but at an index no branch predicted
    top1[0] = 20
    r = orc.verify_overlap_round(planted_logits(n, V, top1), y, b, corr, bc)
    assert r["accept_len"] == 0 and r["emitted"] == [20] and r["corr_hit"] == [False, False]
    # full acceptance: continuation rule only
    top1[:4] = [4, 5, 6, 9]
    r = orc.verify_overlap_round(planted_logits(n, V, top1), y, b, corr, bc)
    assert r["accept_len"] == 3 and r["cont_hit"] is True and r["corr_hit"] == [False, False]


def test_next_round_risky_positions_planted():
    """Margins are planted through the top-2 logit gap: gap 4 gives M = 0.96.., gap 0.5 gives M < 0.5."""
    V = 32
    y = [3, 4, 5]
    v, b, bc = 3, 4, 3
    corr = [(1, 20)]
    n = v + b + 1 + bc
    top1 = [4, 5, 9] + [9, 8, 7, 6] + [15, 16, 17, 18]
    top2 = [1] * 3 + [24, 25, 26, 27] + [28, 29, 30, 31]
    x = planted_logits(n, V, top1, top2, gap=4.0)
    for row in (v + 0, v + 2, v + 3, v + b + 1, v + b + 3):      # low-margin rows
        x[row, top2[row]] = 10.0 - 0.5
    # two-candidate rows: M = tanh(gap / 2) exactly when only two logits matter; here 30 zeros add mass
    r = orc.verify_overlap_round(x, y, b, corr, bc)
    # continuation block: mask row 0 is not a draft of the next round; rows 2 and 3 are risky
    assert r["risky"][0] == (2, [(2, 26), (3, 27)])
    # correction block: mask row m becomes y'_{m+1}; rows 0 and 2 are risky -> indices 1 and 3
    assert r["risky"][1] == (2, [(1, 29), (3, 31)])
    st = r["stats"]
    assert len(st) == n
    assert st[v + 1]["margin"] > 0.5 > st[v + 2]["margin"]


@pytest.mark.parametrize("delta", [0.5, 0.05, 0.0])
def test_overlap_loop_is_lossless(small, delta):
    """Whatever branches are prepared and reused, the emitted text is the greedy continuation."""
    shape, cfg, W = small
    prompt = synth.token_ids(12, shape.vocab, seed=7).tolist()
    out, trace = orc.spec_decode_overlap(cfg, W, prompt, 4, rounds=6, delta=delta)
    ar = orc.greedy_ar(cfg, W, prompt, len(out))
    assert out == ar
    assert all(len(t["emitted"]) == t["accept_len"] + 1 for t in trace)
    if delta == 0.0:
        assert all(t["corr"] == [] and t["cont"] for t in trace)
        plain, ptrace, _ = orc.spec_decode(cfg, W, prompt, 4, rounds=6)
        assert plain == out and [t["accept_len"] for t in ptrace] == [t["accept_len"] for t in trace]
    for t in trace:
        assert len(t["corr"]) <= 2 and all(1 <= i < len(t["y"]) for i, _ in t["corr"])


def test_reused_correction_branch_feeds_the_next_round(small):
    """Teacher-forced case: drafts are the greedy continuation except one position whose replacement
    candidate is the true token.  The branch must hit, and its drafts must equal what a fresh round
    over the corrected context would draft."""
    shape, cfg, W = small
    prompt = synth.token_ids(12, shape.vocab, seed=8).tolist()
    ar = orc.greedy_ar(cfg, W, prompt, 12)
    kv, L, y0 = orc.prefill(cfg, W, prompt)
    v, b, i = 5, 4, 3
    y = [y0[0]] + ar[: v - 1]
    truth = y[i]
    y[i] = (truth + 1) % (shape.vocab - 1)
    corr = [(i, truth)]
    logits, kv_new, _ = orc.overlap_round_cached(cfg, W, kv, L, y, b, corr, b)
    r = orc.verify_overlap_round(logits, y, b, corr, b)
    assert r["accept_len"] == i - 1 and r["emitted"][-1] == truth and r["corr_hit"] == [True]
    # the round a server without the branch would have to run next
    new_L = L + i
    pre = [(K[:new_L], V[:new_L]) for (K, V) in kv_new]
    nxt, _, _ = orc.fused_round_cached(cfg, W, pre, new_L, [truth], b)
    fresh = orc.verify_round(nxt, [truth], b)
    assert r["corr_draft"][0] == fresh["next_draft"]
