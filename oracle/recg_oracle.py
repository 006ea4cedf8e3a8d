"""CPU oracle for the fused draft+verify round of diffusion-AR self-speculation.

THIS IS TEST INFRASTRUCTURE.  It is a plain, slow, fp64 numpy statement of what
the round computes, written from the paper's definitions so that a reader can
check it by eye.  It shares no code with the CUDA path and must never be
imported by the product: only the tests, the smoke check and the benchmark's
CPU-baseline leg call it.

What follows the paper, and where:

* the two attention masks, M^Diff and M^AR                      -- Eq. 1 (Sec. 3.1)
* one shared backbone serving both modes; accept the drafted
  prefix up to the first mismatch with the verifier             -- Sec. 3.1
* draft confidence C_i = P_1st(i), margin M_i = P_1st - P_2nd   -- Sec. 4.1
* mean verifier entropy e_t over causally valid positions       -- Sec. 5.2
* continuation-branch reuse rule (full acceptance and the
  first drafted token equals the verifier's bonus token)        -- Sec. 5.1
* co-batching the next draft block with the current verify
  rows in one forward over a shared prefix                      -- Sec. 5.1, 5.3
* risky positions (M_i < delta, earliest two), correction
  branches with the second candidate, their reuse rule, and
  the recursive loop over verifier + up to three branches       -- Sec. 5.1
* the certainty state and the table-lookup block-size rule      -- Sec. 5.2, Eq. 2-3
* the transition probabilities of acceptance intervals between
  adjacent rounds, as a Markov chain that supplies synthetic
  acceptance lengths                                            -- Sec. 4.2, Table 1

The backbone itself (RMSNorm, rotary embedding with rotate-half pairing,
grouped-query attention, SwiGLU, untied LM head) is the generic Llama-style
decoder the workload configuration names; the paper only says "shared
backbone".  Every floating-point quantity is float64.

Parity pins (see tests/test_oracle_*.py): brute-force loops over Eq. 1 on tiny
shapes, a library attention routine with the same boolean mask, an independent
library implementation of the causal decoder, losslessness of greedy
speculation against token-by-token greedy decoding, cached == dense, closed
forms for the statistics, and planted accept lengths; for the branches, each
branch row against the standalone round it hypothesises, visibility by brute
force, planted selection / reuse cases and losslessness of the recursive loop
(tests/test_oracle_overlap.py); for the block-size rule, pairwise comparisons
on a closed-form acceptance model, the limits of the cost weight, ties and
bin edges (tests/test_oracle_policy.py); for the acceptance chain, the printed
table itself (tests/golden/table1_transitions.txt), its stationary distribution
solved two ways and the transition counts of a long run
(tests/test_oracle_chain.py); for the bookkeeping between rounds, the trace of
the pinned round loop.  No value printed in the
paper exists for this path, so numeric parity with the paper itself is
unpinned; parity is with these definitions.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Callable, Dict, List, Optional, Sequence, Tuple

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------
# configuration
# --------------------------------------------------------------------------
@dataclass
class ModelConfig:
    n_layers: int
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    vocab: int
    rope_base: float = 10000.0
    rms_eps: float = 1e-5
    mask_token_id: int = -1  # -1 -> vocab - 1

    def mask_id(self) -> int:
        return self.vocab - 1 if self.mask_token_id < 0 else self.mask_token_id


# Weights are a dict of float64 arrays, all stored [out_features, in_features]:
#   embed [V,H]  final_norm [H]  lm_head [V,H]
#   attn_norm[l] [H]   wqkv[l] [(n_q+2 n_kv) d, H]  (q heads, then k heads, then v heads)
#   wo[l] [H, n_q d]   ffn_norm[l] [H]   w_gate_up[l] [2F, H] (gate rows, then up rows)
#   w_down[l] [H, F]
Weights = Dict[str, object]


# --------------------------------------------------------------------------
# Eq. 1: the masks, as visibility predicates (True <=> M_ij = 0)
# --------------------------------------------------------------------------
def mask_diff(i, j, P: int, B: int):
    """M^Diff of Eq. 1 with 0-based indices.

    Prefix positions are 0..P-1 and draft positions are P..P+B-1.  A prefix
    row sees prefix columns j <= i; a draft row sees every prefix and draft
    column; everything else is -inf.  Works on ints or broadcastable arrays.
    """
    i_in_P = (i >= 0) & (i < P)
    j_in_P = (j >= 0) & (j < P)
    i_in_D = (i >= P) & (i < P + B)
    j_in_PD = (j >= 0) & (j < P + B)
    return (i_in_P & j_in_P & (j <= i)) | (i_in_D & j_in_PD)


def mask_ar(i, j):
    """M^AR of Eq. 1: strict left-to-right visibility."""
    return j <= i


def visibility_matrix(P: int, B: int) -> np.ndarray:
    """Boolean [(P+B), (P+B)] matrix of Eq. 1's M^Diff, every (i, j) pair."""
    n = P + B
    i = np.arange(n).reshape(n, 1)
    j = np.arange(n).reshape(1, n)
    return np.asarray(mask_diff(i, j, P, B), dtype=bool)


def fused_round_visibility(L: int, v: int, b: int) -> np.ndarray:
    """Visibility of the n = v + b new rows of one fused round, [n, L + n].

    The request is laid out as committed context [0, L), pending verify tokens
    [L, L+v), mask tokens [L+v, L+v+b).  Eq. 1's prefix set is context plus
    verify tokens (they keep causal dependency); its draft set is the mask
    block.  Restricted to prefix rows this is M^AR, so verify rows are
    verified exactly as in the autoregressive mode.
    """
    return visibility_matrix(L + v, b)[L:, :]


# --------------------------------------------------------------------------
# backbone pieces
# --------------------------------------------------------------------------
def rmsnorm(h: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    ms = np.mean(h * h, axis=-1, keepdims=True)
    return h / np.sqrt(ms + eps) * g


def rope(x: np.ndarray, pos: np.ndarray, base: float) -> np.ndarray:
    """Rotary embedding, rotate-half pairing (i, i + d/2); x is [rows, heads, d]."""
    d = x.shape[-1]
    half = d // 2
    i = np.arange(half, dtype=F64)
    theta = base ** (-2.0 * i / d)                      # [half]
    ang = pos.astype(F64).reshape(-1, 1) * theta.reshape(1, -1)   # [rows, half]
    c = np.cos(ang)[:, None, :]
    s = np.sin(ang)[:, None, :]
    x1 = x[..., :half]
    x2 = x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def silu(z: np.ndarray) -> np.ndarray:
    return z / (1.0 + np.exp(-z))


def attention(q: np.ndarray, K: np.ndarray, V: np.ndarray, vis: np.ndarray) -> np.ndarray:
    """softmax(q K^T / sqrt(d) + M) V with grouped-query heads.

    q [rows, n_q, d]; K, V [keys, n_kv, d]; vis bool [rows, keys] (True = M is 0).
    Keys that are not visible are never read arithmetically (they may hold NaN).
    """
    rows, n_q, d = q.shape
    n_kv = K.shape[1]
    group = n_q // n_kv
    o = np.zeros((rows, n_q, d), dtype=F64)
    for r in range(rows):
        cols = np.nonzero(vis[r])[0]
        if cols.size == 0:
            continue
        for hq in range(n_q):
            hk = hq // group
            s = K[cols, hk, :] @ q[r, hq, :] / np.sqrt(F64(d))
            s = s - np.max(s)
            p = np.exp(s)
            p = p / np.sum(p)
            o[r, hq, :] = p @ V[cols, hk, :]
    return o


def hybrid_attention(q: np.ndarray, K: np.ndarray, V: np.ndarray, L: int, v: int, b: int) -> np.ndarray:
    """The round's attention for one request (Eq. 1 over a shared prefix).

    q [v+b, n_q, d] are the new rows (verify rows first, then mask rows);
    K, V [L+v+b, n_kv, d] hold the committed context followed by the new rows.
    """
    assert q.shape[0] == v + b and K.shape[0] == L + v + b
    return attention(q, K, V, fused_round_visibility(L, v, b))


def decoder_rows(cfg: ModelConfig, W: Weights, ids: Sequence[int], pos: np.ndarray, vis: np.ndarray,
                 kv_prefix: Optional[List[Tuple[np.ndarray, np.ndarray]]] = None,
                 act_round: Optional[Callable[[np.ndarray], np.ndarray]] = None):
    """Run the backbone over a set of rows.

    ids/pos give each row's token id and absolute position.  kv_prefix, if
    given, holds per layer the K and V ([L, n_kv, d]) of positions 0..L-1 that
    precede the rows; the rows' own K/V are appended after them, so vis is
    [rows, L + rows].  act_round, if given, is applied where an implementation
    that stores activations in a narrower type rounds them (normalised input,
    q/k/v, attention output, SwiGLU output); the default is pure float64.

    Returns (logits [rows, V], kv [(K_all, V_all)] per layer, hidden [rows, H]).
    """
    rd = act_round if act_round is not None else (lambda a: a)
    n_q, n_kv, d = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    ids = np.asarray(ids, dtype=np.int64)
    rows = ids.shape[0]
    h = np.array(W["embed"][ids], dtype=F64)
    kv_out = []
    for l in range(cfg.n_layers):
        x = rd(rmsnorm(h, W["attn_norm"][l], cfg.rms_eps))
        qkv = x @ W["wqkv"][l].T
        q = qkv[:, : n_q * d].reshape(rows, n_q, d)
        k = qkv[:, n_q * d: (n_q + n_kv) * d].reshape(rows, n_kv, d)
        vv = qkv[:, (n_q + n_kv) * d:].reshape(rows, n_kv, d)
        q = rd(rope(q, pos, cfg.rope_base))
        k = rd(rope(k, pos, cfg.rope_base))
        vv = rd(vv)
        if kv_prefix is not None:
            K_all = np.concatenate([kv_prefix[l][0], k], axis=0)
            V_all = np.concatenate([kv_prefix[l][1], vv], axis=0)
        else:
            K_all, V_all = k, vv
        kv_out.append((K_all, V_all))
        o = rd(attention(q, K_all, V_all, vis)).reshape(rows, n_q * d)
        h = h + o @ W["wo"][l].T
        x = rd(rmsnorm(h, W["ffn_norm"][l], cfg.rms_eps))
        gu = x @ W["w_gate_up"][l].T
        a = rd(silu(gu[:, : cfg.ffn]) * gu[:, cfg.ffn:])
        h = h + a @ W["w_down"][l].T
    logits = rd(rmsnorm(h, W["final_norm"], cfg.rms_eps)) @ W["lm_head"].T
    return logits, kv_out, h


# --------------------------------------------------------------------------
# the fused round, dense (the definition) and cached (what a server runs)
# --------------------------------------------------------------------------
def fused_round_dense(cfg: ModelConfig, W: Weights, context_ids: Sequence[int], verify_ids: Sequence[int], b: int,
                      act_round=None):
    """Recompute every position 0..L+n-1 from token ids under Eq. 1; no cache.

    Returns (logits of the n new rows [n, V], per-layer (K, V) of all L+n
    positions, hidden of the n new rows).
    """
    L, v = len(context_ids), len(verify_ids)
    ids = list(context_ids) + list(verify_ids) + [cfg.mask_id()] * b
    pos = np.arange(L + v + b)
    vis = visibility_matrix(L + v, b)
    logits, kv, h = decoder_rows(cfg, W, ids, pos, vis, None, act_round)
    return logits[L:], kv, h[L:]


def fused_round_cached(cfg: ModelConfig, W: Weights, kv_prefix, L: int, verify_ids: Sequence[int], b: int,
                       act_round=None):
    """Compute only the n new rows over given K/V of the committed context.

    kv_prefix[l] = (K [>=L, n_kv, d], V) ; only the first L positions are read.
    """
    v = len(verify_ids)
    ids = list(verify_ids) + [cfg.mask_id()] * b
    pos = np.arange(L, L + v + b)
    vis = fused_round_visibility(L, v, b)
    pre = [(K[:L], V[:L]) for (K, V) in kv_prefix]
    return decoder_rows(cfg, W, ids, pos, vis, pre, act_round)


# --------------------------------------------------------------------------
# greedy verification and the statistics
# --------------------------------------------------------------------------
def argmax_lowest(x: np.ndarray) -> int:
    """Index of the maximum; the lowest index wins a tie."""
    return int(np.argmax(x))


def row_stats(logits_row: np.ndarray) -> Dict[str, float]:
    """top-1 / top-2 ids, P_1st, P_2nd, margin M = P_1st - P_2nd (Sec. 4.1),
    entropy in nats, and the top-2 logit gap, for one row of logits."""
    x = np.asarray(logits_row, dtype=F64)
    t1 = argmax_lowest(x)
    y = x.copy()
    y[t1] = -np.inf
    t2 = argmax_lowest(y)
    z = x - x[t1]
    e = np.exp(z)
    s = np.sum(e)
    p = e / s
    # -sum p ln p, written without 0*log(0)
    logp = z - np.log(s)
    H = -float(np.sum(np.where(p > 0.0, p * logp, 0.0)))
    return {"top1": t1, "top2": t2, "p1": float(p[t1]), "p2": float(p[t2]),
            "margin": float(p[t1] - p[t2]), "entropy": H, "logit_gap": float(x[t1] - x[t2])}


def greedy_accept(verify_top1: Sequence[int], y: Sequence[int]) -> int:
    """Accept length a: the largest m in [0, v-1] with y[i+1] == top1[i] for all i < m.

    Row i of the verify segment holds token y[i]; its argmax predicts the token
    after it.  y[0] is known to be correct, y[1:] are drafts (Sec. 3.1).
    """
    v = len(y)
    a = 0
    while a < v - 1 and int(y[a + 1]) == int(verify_top1[a]):
        a += 1
    return a


def verify_round(logits: np.ndarray, y: Sequence[int], b: int) -> Dict[str, object]:
    """Everything one request's round reports, from its n = v + b rows of logits.

    Emitted tokens are y[1..a] followed by the verifier's own token at row a
    (the correction when a < v-1, the bonus token when a = v-1).  e_mean
    averages verifier entropy over rows 0..a, the causally valid ones
    (Sec. 5.2).  cont_hit is the continuation-branch reuse rule of Sec. 5.1.
    """
    v = len(y)
    n = v + b
    assert logits.shape[0] == n
    st = [row_stats(logits[r]) for r in range(n)]
    top1 = [s["top1"] for s in st]
    out: Dict[str, object] = {"stats": st}
    if v > 0:
        a = greedy_accept(top1[:v], y)
        emitted = [int(t) for t in y[1: a + 1]] + [top1[a]]
        e_mean = float(np.mean([st[i]["entropy"] for i in range(a + 1)]))
        n_emit = a + 1
    else:
        a, emitted, e_mean, n_emit = 0, [], 0.0, 0
    next_draft = top1[v:]
    cont_hit = bool(v > 0 and b > 0 and a == v - 1 and next_draft[0] == top1[v - 1])
    out.update({"accept_len": a, "n_emitted": n_emit, "emitted": emitted, "entropy_mean": e_mean,
                "next_draft": next_draft, "cont_hit": cont_hit})
    return out


def kv_commit(L: int, v: int, b: int, a: int, page_table: Sequence[int], page_size: int) -> Dict[str, object]:
    """KV bookkeeping after verification; index work only.

    Positions L..L+a (tokens y_0..y_a) become committed context; positions
    L+a+1..L+n-1 (rejected drafts and every mask row) are rolled back.  A page
    is freed when its first position is at or beyond the new length.
    """
    n = v + b
    new_L = L + (a + 1 if v > 0 else 0)
    slot = lambda p: int(page_table[p // page_size]) * page_size + p % page_size
    commit = [slot(p) for p in range(L, new_L)]
    rollback = [slot(p) for p in range(new_L, L + n)]
    first_free = -(-new_L // page_size)
    last = -(-(L + n) // page_size)
    freed = [int(page_table[i]) for i in range(first_free, last)]
    return {"new_ctx_len": new_L, "commit_slots": commit, "rollback_slots": rollback, "freed_pages": freed}


def verify_batch(logits: np.ndarray, verify_len: Sequence[int], block_size: Sequence[int],
                 verify_tokens: Sequence[int]) -> List[Dict[str, object]]:
    """Standalone verification of a ragged batch: rows are concatenated request by
    request (verify rows then draft rows), verify_tokens likewise."""
    res = []
    r0 = 0
    t0 = 0
    for v, b in zip(verify_len, block_size):
        res.append(verify_round(np.asarray(logits[r0: r0 + v + b], dtype=F64), list(verify_tokens[t0: t0 + v]), b))
        r0 += v + b
        t0 += v
    return res


# --------------------------------------------------------------------------
# decoding loops (tiny models only)
# --------------------------------------------------------------------------
def greedy_ar(cfg: ModelConfig, W: Weights, prompt: Sequence[int], n_new: int) -> List[int]:
    """Plain token-by-token greedy decoding: the whole sequence is recomputed
    densely under M^AR for every new token.  The ground truth for losslessness."""
    seq = list(prompt)
    for _ in range(n_new):
        n = len(seq)
        i = np.arange(n).reshape(n, 1)
        j = np.arange(n).reshape(1, n)
        logits, _, _ = decoder_rows(cfg, W, seq, np.arange(n), np.asarray(mask_ar(i, j)), None)
        seq.append(argmax_lowest(logits[-1]))
    return seq[len(prompt):]


def prefill(cfg: ModelConfig, W: Weights, prompt: Sequence[int]):
    """Commit K/V of all but the last prompt token; the last one is y_0 of the
    first round.  Returns (per-layer (K, V) of length L = len(prompt)-1, L, y)."""
    ctx = list(prompt[:-1])
    n = len(ctx)
    i = np.arange(n).reshape(n, 1)
    j = np.arange(n).reshape(1, n)
    _, kv, _ = decoder_rows(cfg, W, ctx, np.arange(n), np.asarray(mask_ar(i, j)), None)
    return kv, n, [int(prompt[-1])]


def spec_decode(cfg: ModelConfig, W: Weights, prompt: Sequence[int], b: int, rounds: int,
                plant: Optional[Callable[[int, List[int], List[int]], List[int]]] = None,
                poison_rollback: bool = True):
    """Self-speculative decoding with the next draft co-batched into the verify forward.

    Every round runs ONE forward over the pending verify tokens y (causal) and
    b mask tokens (bidirectional), verifies greedily, commits K/V of y_0..y_a
    and rolls the rest back.  If the block was fully accepted and the first
    drafted token equals the bonus token, the drafted block becomes the next
    round's verify tokens (the continuation branch is reused); otherwise the
    branch is discarded and the next round verifies the single emitted token.

    plant(round_index, emitted_so_far, y) may replace y before the round (used
    to teacher-force drafts with a planted first mismatch).  Rolled-back cache
    positions are overwritten with NaN so that any later read would poison the
    output.  Returns (emitted tokens, per-round trace).
    """
    kv, L, y = prefill(cfg, W, prompt)
    out: List[int] = []
    trace = []
    for t in range(rounds):
        if plant is not None:
            y = plant(t, out, y)
        v = len(y)
        logits, kv_new, _ = fused_round_cached(cfg, W, kv, L, y, b)
        r = verify_round(logits, y, b)
        a = r["accept_len"]
        new_L = L + a + 1
        kv = []
        for (K, V) in kv_new:
            K = K.copy()
            V = V.copy()
            if poison_rollback:
                K[new_L:] = np.nan
                V[new_L:] = np.nan
            kv.append((K, V))
        out += r["emitted"]
        trace.append({"L": L, "y": list(y), "b": b, "accept_len": a, "emitted": list(r["emitted"]),
                      "cont_hit": r["cont_hit"], "next_draft": list(r["next_draft"]), "new_L": new_L})
        L = new_L
        bonus = r["emitted"][-1]
        if r["cont_hit"]:
            y = [bonus] + [int(t_) for t_ in r["next_draft"][1:]]
        else:
            y = [bonus]
    return out, trace, (kv, L)


# --------------------------------------------------------------------------
# predictive draft-verify overlap: correction and continuation branches (Sec. 5.1)
# --------------------------------------------------------------------------
# One request's round then holds up to four logical rows that share the
# canonical prefix (Sec. 5.1, 5.3):
#   verifier      y_0 .. y_{v-1}                       causal
#   continuation  b mask tokens after the whole y      sees prefix + y + its block
#   correction k  for a risky draft index i_k (1 <= i_k <= v-1): the replacement
#                 token r_k standing where y_{i_k} stands, then bc mask tokens;
#                 sees prefix + y_0 .. y_{i_k - 1} + its own tokens
# New rows are ordered [verifier | continuation | correction 0 | correction 1];
# their K/V occupy cache indices L, L+1, ... in that order, while the rotary
# position of a branch token is the position it would have in the sequence the
# branch hypothesises (r_k at L + i_k, its masks at L + i_k + 1 ...).
DELTA_RISKY = 0.5   # margin threshold of the risky-position rule (Sec. 5.1 / experimental setup)


def select_branches(margin: Sequence[float], second: Sequence[int], delta: float = DELTA_RISKY, keep: int = 2):
    """Risky-position rule of Sec. 5.1 for the pending drafts y_1 .. y_{v-1}.

    margin[i], second[i] are M_i and the second-ranked token id of the draft
    row that produced y_i (entry 0 is ignored: y_0 is known to be correct).
    A position is risky when M_i < delta; the earliest `keep` risky positions
    get a correction branch (the draft replaced by its second candidate), and
    the continuation branch is prepared only when no more than `keep`
    positions are risky.  Returns ([(i, replacement)], continuation?).
    """
    risky = [i for i in range(1, len(margin)) if float(margin[i]) < delta]
    corr = [(i, int(second[i])) for i in risky[:keep]]
    return corr, len(risky) <= keep


def overlap_round_rows(L: int, v: int, b: int, corr: Sequence[Tuple[int, int]], bc: int):
    """Positions and visibility of the rows of a round with branches.

    Returns (pos [n], vis [n, L + n], kind [n]) with n = v + b + len(corr) * (1 + bc);
    kind is 'v' (verifier), 'c' (continuation mask), 'r' (replacement token)
    or 'm' (mask of a correction branch).  Column j < L is committed context,
    column L + j is new row j.
    """
    n = v + b + len(corr) * (1 + bc)
    pos = np.zeros(n, dtype=np.int64)
    vis = np.zeros((n, L + n), dtype=bool)
    kind = []
    for j in range(v):                      # verifier: M^AR
        pos[j] = L + j
        vis[j, : L + j + 1] = True
        kind.append("v")
    for j in range(b):                      # continuation: Eq. 1 with prefix = context + y
        pos[v + j] = L + v + j
        vis[v + j, : L + v] = True
        vis[v + j, L + v: L + v + b] = True
        kind.append("c")
    for k, (i, _tok) in enumerate(corr):
        assert 1 <= i <= v - 1, "a correction replaces one of the drafts y_1 .. y_{v-1}"
        r0 = v + b + k * (1 + bc)           # row of the replacement token
        pos[r0] = L + i
        vis[r0, : L + i] = True             # context + y_0 .. y_{i-1}
        vis[r0, L + r0] = True              # itself (causal token)
        kind.append("r")
        for j in range(bc):                 # the branch's own block: Eq. 1 with prefix = ... + replacement
            pos[r0 + 1 + j] = L + i + 1 + j
            vis[r0 + 1 + j, : L + i] = True
            vis[r0 + 1 + j, L + r0: L + r0 + 1 + bc] = True
            kind.append("m")
    return pos, vis, kind


def overlap_round_cached(cfg: ModelConfig, W: Weights, kv_prefix, L: int, verify_ids: Sequence[int], b: int,
                         corr: Sequence[Tuple[int, int]], bc: int, act_round=None):
    """One forward over the verifier and all prospective branches of a request."""
    ids = list(verify_ids) + [cfg.mask_id()] * b
    for (_i, tok) in corr:
        ids += [int(tok)] + [cfg.mask_id()] * bc
    pos, vis, _ = overlap_round_rows(L, len(verify_ids), b, corr, bc)
    pre = [(K[:L], V[:L]) for (K, V) in kv_prefix]
    return decoder_rows(cfg, W, ids, pos, vis, pre, act_round)


def verify_overlap_round(logits: np.ndarray, y: Sequence[int], b: int, corr: Sequence[Tuple[int, int]], bc: int,
                         delta: float = DELTA_RISKY) -> Dict[str, object]:
    """verify_round() plus the branch reuse rules and the next round's risky positions.

    corr_hit[k]: the verifier rejected exactly the draft the branch replaced
    (accept length a = i_k - 1) and its own token there equals the replacement
    (Sec. 5.1).  corr_draft[k]: argmax of the branch's mask rows, the drafts
    that follow the replacement if the branch is reused.
    risky[j] describes draft block j (0 = continuation, 1 + k = correction k)
    in the indexing of the verify row it would become: the continuation gives
    y' = [bonus, d_1, ..], so mask row m is y'_m (m >= 1); a correction gives
    y' = [replacement, d_0, ..], so mask row m is y'_{m+1}.  Each entry is
    (number of risky positions, [(index into y', second candidate)] for the
    earliest two).
    """
    v = len(y)
    n_corr = len(corr)
    assert logits.shape[0] == v + b + n_corr * (1 + bc)
    out = verify_round(logits[: v + b], y, b)
    a = out["accept_len"]
    st_all = list(out["stats"])
    hits, drafts, risky = [], [], []

    def block_risky(stats, first_index):
        idx = [first_index + m for m, s in enumerate(stats) if s["margin"] < delta]
        sec = {first_index + m: s["top2"] for m, s in enumerate(stats)}
        return (len(idx), [(i, sec[i]) for i in idx[:2]])

    risky.append(block_risky(st_all[v + 1: v + b], 1))
    for k, (i, tok) in enumerate(corr):
        r0 = v + b + k * (1 + bc)
        st = [row_stats(logits[r]) for r in range(r0, r0 + 1 + bc)]
        st_all += st
        hits.append(bool(a == i - 1 and out["emitted"][-1] == int(tok)))
        drafts.append([s["top1"] for s in st[1:]])
        risky.append(block_risky(st[1:], 1))
    out.update({"stats": st_all, "corr_hit": hits, "corr_draft": drafts, "risky": risky})
    return out


def spec_decode_overlap(cfg: ModelConfig, W: Weights, prompt: Sequence[int], b: int, rounds: int,
                        delta: float = DELTA_RISKY, poison_rollback: bool = True):
    """Self-speculative decoding with predictive draft-verify overlap (Sec. 5.1).

    Every round runs one forward over the verifier row and the branches the
    risky-position rule selects, then keeps the branch the verification outcome
    confirms (a correction that predicted both the rejected position and the
    verifier's token, or the continuation after full acceptance); its drafts
    are the next round's verify tokens, and the rule is applied to them again.
    Returns (emitted tokens, per-round trace).
    """
    kv, L, y = prefill(cfg, W, prompt)
    margin: List[float] = [1.0]
    second: List[int] = [-1]
    out: List[int] = []
    trace = []
    for _t in range(rounds):
        corr, cont = select_branches(margin, second, delta)
        bb = b if cont else 0
        logits, kv_new, _ = overlap_round_cached(cfg, W, kv, L, y, bb, corr, b)
        r = verify_overlap_round(logits, y, bb, corr, b, delta)
        a = r["accept_len"]
        new_L = L + a + 1
        kv = []
        for (K, V) in kv_new:
            K = K[: L + len(y)].copy()
            V = V[: L + len(y)].copy()
            if poison_rollback:
                K[new_L:] = np.nan
                V[new_L:] = np.nan
            kv.append((K, V))
        out += r["emitted"]
        v = len(y)
        st = r["stats"]
        used = "none"
        bonus = r["emitted"][-1]
        if r["cont_hit"]:
            used = "continuation"
            rows = st[v + 1: v + bb]
            y_next = [bonus] + [s["top1"] for s in rows]
        elif any(r["corr_hit"]):
            k = r["corr_hit"].index(True)
            used = "correction%d" % k
            r0 = v + bb + k * (1 + b)
            rows = st[r0 + 1: r0 + 1 + b]
            y_next = [bonus] + [s["top1"] for s in rows]
        else:
            rows = []
            y_next = [bonus]
        trace.append({"L": L, "y": list(y), "corr": list(corr), "cont": cont, "accept_len": a,
                      "emitted": list(r["emitted"]), "used": used, "new_L": new_L})
        margin = [1.0] + [s["margin"] for s in rows]
        second = [-1] + [s["top2"] for s in rows]
        y = y_next
        L = new_L
    return out, trace


# --------------------------------------------------------------------------
# verification-guided adaptive drafting: the block-size rule (Sec. 5.2, Eq. 2-3)
# --------------------------------------------------------------------------
# The calibrated estimate V_B(s, z) is a table: the certainty s is binned by
# ascending edges (bin = number of edges <= s), z = (index of the previous
# block size among the candidates, full-acceptance flag).  cost[B] is
# rho_C * T_C(B), the profiled execution cost at the current load, already
# weighted.  value has shape [n_blocks (candidate B), n_bins, n_blocks (previous
# B), 2 (F)].
def policy_certainty(e1, e2, dtype=F64):
    """s_t = -(e_{t-1} + e_{t-2}) / 2 (Eq. 2), evaluated in `dtype`."""
    e1 = np.asarray(e1, dtype=dtype)
    e2 = np.asarray(e2, dtype=dtype)
    return (e1 + e2) * dtype(-0.5)


def policy_select(s, prev_index: int, full: int, blocks: Sequence[int], s_edges, value, cost, dtype=F64):
    """B* = argmax_B [V_B(s, z) - rho_C T_C(B)] (Eq. 3); the first maximum wins,
    i.e. the smaller block on a tie.  Returns (index into blocks, B*)."""
    edges = np.asarray(s_edges, dtype=dtype)
    k = int(np.sum(edges <= dtype(s)))
    value = np.asarray(value, dtype=dtype)
    cost = np.asarray(cost, dtype=dtype)
    score = [value[j, k, prev_index, int(full)] - cost[j] for j in range(len(blocks))]
    best = 0
    for j in range(1, len(blocks)):
        if score[j] > score[best]:
            best = j
    return best, int(blocks[best])


def policy_step(state: Dict[str, list], entropy_mean, accept_len, verify_len, blocks, s_edges, value, cost,
                dtype=F64):
    """One request-wise update after a finished round, then the choice for the next one.

    state holds per request e1 = e_{t-1}, e2 = e_{t-2}, block_index (the block
    size chosen last time, the B_{t-1} of Eq. 2) and full (F_{t-1}).  A round
    that verified at least one token shifts its mean verifier entropy into the
    history; F is set when the round verified drafts and accepted all of them.
    Returns the chosen block sizes; state is updated in place.
    """
    out = []
    for r in range(len(state["e1"])):
        v, a = int(verify_len[r]), int(accept_len[r])
        if v > 0:
            state["e2"][r] = state["e1"][r]
            state["e1"][r] = dtype(entropy_mean[r])
            state["full"][r] = 1 if (v > 1 and a == v - 1) else 0
        s = policy_certainty(state["e1"][r], state["e2"][r], dtype)
        j, B = policy_select(s, state["block_index"][r], state["full"][r], blocks, s_edges, value, cost, dtype)
        state["block_index"][r] = j
        out.append(B)
    return out


# --------------------------------------------------------------------------
# synthetic acceptance lengths: the interval chain of Table 1 (Sec. 4.2)
# --------------------------------------------------------------------------
# With block size 32 the paper sorts a round's acceptance length A (emitted
# tokens of the round, a + 1 here) into three intervals and prints the
# probability of the next round's interval given this round's.  Random-init
# weights accept almost nothing, so multi-round runs take their acceptance
# lengths from this chain instead.  The paper prints nothing about the
# distribution INSIDE an interval; it is taken uniform over the interval's
# integers.  All random numbers are inputs (uniforms in [0, 1)).
TABLE1_INTERVALS = ((1, 8), (9, 16), (17, 32))
TABLE1_PERCENT = ((70.30, 18.11, 11.60),
                  (58.39, 22.42, 19.19),
                  (20.83, 12.51, 66.66))


def chain_matrix(percent=TABLE1_PERCENT) -> np.ndarray:
    """Row-stochastic transition matrix from the printed percentages (the rows
    add up to 100 only to the printed precision; each row is divided by its sum)."""
    P = np.asarray(percent, dtype=F64)
    return P / P.sum(axis=1, keepdims=True)


def chain_stationary(P: np.ndarray) -> np.ndarray:
    """The distribution pi with pi P = pi and sum(pi) = 1, by solving the linear system."""
    n = P.shape[0]
    A = np.vstack([P.T - np.eye(n), np.ones((1, n))])
    rhs = np.concatenate([np.zeros(n), [1.0]])
    pi, *_ = np.linalg.lstsq(A, rhs, rcond=None)
    return pi


def acceptance_chain(P: np.ndarray, intervals, state0: int, u_state: Sequence[float], u_len: Sequence[float]):
    """Walk the chain: round t is in state s_t (s_0 = state0); its acceptance
    length is lo + floor(u_len[t] * (hi - lo + 1)) within the state's interval;
    the next state is the first j whose cumulative probability in row s_t
    exceeds u_state[t].  Returns (states, lengths)."""
    states, lengths = [], []
    s = int(state0)
    for t in range(len(u_len)):
        lo, hi = intervals[s]
        states.append(s)
        lengths.append(min(hi, lo + int(np.floor(F64(u_len[t]) * (hi - lo + 1)))))
        c = np.cumsum(P[s])
        j = int(np.sum(c <= F64(u_state[t])))
        s = min(j, len(intervals) - 1)
    return states, lengths


def advance_round(L: int, y: Sequence[int], b: int, accept_len: int, verifier_token: int, cont_hit: bool,
                  next_draft: Sequence[int]):
    """Bookkeeping between two rounds of the fused loop (Sec. 3.1, 5.1): K/V of
    y_0..y_a are committed, the verifier's token at row a is emitted last and
    becomes the next y_0; a reused continuation block supplies the next drafts
    (its first token only confirmed the bonus token), otherwise the next round
    verifies the single emitted token.  Returns (new L, next y)."""
    new_L = L + accept_len + 1
    if cont_hit:
        return new_L, [int(verifier_token)] + [int(t) for t in next_draft[1:]]
    return new_L, [int(verifier_token)]


def planted_rounds(L0: int, v0: int, blocks: Sequence[int], lengths: Sequence[int]):
    """Lengths-only trace of the loop under synthetic acceptance (token values
    play no role): round t has context L_t, v_t verify tokens and block
    blocks[t]; it accepts a_t = min(lengths[t], v_t) - 1 drafts, i.e. emits
    min(lengths[t], v_t) tokens; the continuation block is taken as reused
    exactly when the round accepted all its drafts and drafted a block.
    Returns per round (L, v, b, a, emitted, reused)."""
    L, v = int(L0), int(v0)
    out = []
    for t, b in enumerate(blocks):
        emitted = max(1, min(int(lengths[t]), v)) if v > 0 else 0
        a = emitted - 1 if v > 0 else 0
        reused = v > 0 and b > 0 and a == v - 1
        out.append((L, v, int(b), a, emitted, reused))
        L = L + (a + 1 if v > 0 else 0)
        v = int(b) if reused else 1
    return out
