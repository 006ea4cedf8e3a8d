"""Pins for the oracle's masks and attention (Eq. 1), independent of the oracle's own code paths."""
import math

import numpy as np
import pytest
import torch

from oracle import recg_oracle as orc


def brute_mask(P, B):
    """Eq. 1's M^Diff written with explicit sets and loops; returns additive mask (0 / -inf)."""
    n = P + B
    Pset = set(range(P))
    Dset = set(range(P, P + B))
    M = [[-math.inf] * n for _ in range(n)]
    for i in range(n):
        for j in range(n):
            if i in Pset and j in Pset and j <= i:
                M[i][j] = 0.0
            elif i in Dset and (j in Pset or j in Dset):
                M[i][j] = 0.0
    return M


def brute_attention(q, K, V, M, row0):
    """softmax(q K^T / sqrt(d) + M) V with scalar loops; rows of q are absolute rows row0.."""
    rows, n_q, d = q.shape
    keys, n_kv, _ = K.shape
    g = n_q // n_kv
    out = np.zeros_like(q)
    for r in range(rows):
        for h in range(n_q):
            s = []
            for j in range(keys):
                dot = 0.0
                for e in range(d):
                    dot += q[r, h, e] * K[j, h // g, e]
                s.append(dot / math.sqrt(d) + M[row0 + r][j])
            m = max(s)
            w = [math.exp(x - m) if x != -math.inf else 0.0 for x in s]
            z = sum(w)
            for e in range(d):
                acc = 0.0
                for j in range(keys):
                    if w[j] != 0.0:
                        acc += w[j] * V[j, h // g, e]
                out[r, h, e] = acc / z
    return out


CASES = [(L, v, b) for L in (0, 1, 15, 16, 17, 33) for v in (0, 1, 3, 8) for b in (0, 1, 2, 8) if v + b > 0]


def test_mask_matches_bruteforce_sets():
    for P in range(0, 7):
        for B in range(0, 5):
            M = brute_mask(P, B)
            vis = orc.visibility_matrix(P, B)
            for i in range(P + B):
                for j in range(P + B):
                    assert vis[i, j] == (M[i][j] == 0.0)
                    assert bool(orc.mask_diff(i, j, P, B)) == (M[i][j] == 0.0)


def test_mask_structure():
    L, v, b = 5, 4, 3
    vis = orc.fused_round_visibility(L, v, b)
    assert vis.shape == (v + b, L + v + b)
    # verify rows: exactly causal (row i sees L + i + 1 keys), never the mask block
    for i in range(v):
        assert vis[i].sum() == L + i + 1 and vis[i, : L + i + 1].all()
    # draft rows see everything
    assert vis[v:].all()
    # restricted to prefix rows/cols, M^Diff equals M^AR
    full = orc.visibility_matrix(L + v, b)
    i = np.arange(L + v)[:, None]
    j = np.arange(L + v)[None, :]
    assert (full[: L + v, : L + v] == orc.mask_ar(i, j)).all()


@pytest.mark.parametrize("L,v,b", CASES[::3])
def test_attention_bruteforce(L, v, b):
    rng = np.random.default_rng(L * 100 + v * 10 + b)
    n_q, n_kv, d = 2, 1, 8
    n = v + b
    q = rng.standard_normal((n, n_q, d))
    K = rng.standard_normal((L + n, n_kv, d))
    V = rng.standard_normal((L + n, n_kv, d))
    ref = brute_attention(q, K, V, brute_mask(L + v, b), L)
    got = orc.hybrid_attention(q, K, V, L, v, b)
    assert np.max(np.abs(ref - got)) < 1e-12


@pytest.mark.parametrize("L,v,b", CASES)
def test_attention_vs_library_sdpa(L, v, b):
    rng = np.random.default_rng(7 + L * 100 + v * 10 + b)
    n_q, n_kv, d = 4, 2, 16
    n = v + b
    q = rng.standard_normal((n, n_q, d))
    K = rng.standard_normal((L + n, n_kv, d))
    V = rng.standard_normal((L + n, n_kv, d))
    M = torch.tensor(brute_mask(L + v, b), dtype=torch.float64)[L:, :]
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]                      # [1, n_q, n, d]
    tk = torch.from_numpy(K).permute(1, 0, 2).repeat_interleave(n_q // n_kv, 0)[None]
    tv = torch.from_numpy(V).permute(1, 0, 2).repeat_interleave(n_q // n_kv, 0)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=(M == 0.0)[None, None])
    ref = ref[0].permute(1, 0, 2).numpy()
    got = orc.hybrid_attention(q, K, V, L, v, b)
    assert np.max(np.abs(ref - got)) < 1e-12


def test_invisible_keys_are_never_read():
    # verify rows must not touch the mask block's K/V: poison them
    L, v, b = 9, 3, 4
    rng = np.random.default_rng(3)
    q = rng.standard_normal((v + b, 2, 8))
    K = rng.standard_normal((L + v + b, 1, 8))
    V = rng.standard_normal((L + v + b, 1, 8))
    ref = orc.hybrid_attention(q, K, V, L, v, b)
    K2, V2 = K.copy(), V.copy()
    K2[L + v:] = np.nan
    V2[L + v:] = np.nan
    got = orc.hybrid_attention(q, K2, V2, L, v, b)
    assert np.array_equal(ref[:v], got[:v])
    assert np.isnan(got[v:]).all()


def test_attention_uniform_scores_average_values():
    # q = 0 -> uniform softmax over visible keys -> plain mean of visible V rows
    L, v, b = 4, 3, 2
    rng = np.random.default_rng(5)
    V = rng.standard_normal((L + v + b, 1, 8))
    K = rng.standard_normal((L + v + b, 1, 8))
    q = np.zeros((v + b, 2, 8))
    o = orc.hybrid_attention(q, K, V, L, v, b)
    for i in range(v):
        assert np.allclose(o[i, 0], V[: L + i + 1, 0].mean(0), atol=1e-14)
    for i in range(v, v + b):
        assert np.allclose(o[i, 1], V[:, 0].mean(0), atol=1e-14)
