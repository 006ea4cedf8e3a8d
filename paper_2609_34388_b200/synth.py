"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws numbers (weights, token ids, K/V values, batch
descriptors, logits with planted drafts).  It holds none of the method's
arithmetic and imports neither the CUDA binding nor the CPU oracle, so both
sides can be fed the very same arrays.

Seeds by convention: 0 weights, 1 token ids, 2 K/V values, 3.. descriptor
draws, 4 planting.  Weights are N(0, 0.02^2) with all norm gains 1.0; token
ids are uniform over [0, vocab-1) so that the mask id (vocab-1) never occurs
in a prompt; K/V and standalone logits are N(0, 1).
"""
from __future__ import annotations

from dataclasses import dataclass, asdict
from typing import Dict, List, Optional

import numpy as np
import torch


@dataclass
class ModelShape:
    n_layers: int
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    vocab: int
    rope_base: float = 10000.0
    rms_eps: float = 1e-5
    mask_token_id: int = -1

    def as_dict(self):
        return asdict(self)


def tiny_shape() -> ModelShape:
    """The small 2-layer model used for end-to-end parity."""
    return ModelShape(n_layers=2, hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=64, ffn=1024, vocab=2048,
                      rope_base=10000.0)


def llama8b_shape(n_layers: int = 32) -> ModelShape:
    """8B-class backbone shapes (hidden 4096, 32/8 heads, d 128, FFN 14336, vocab 128256)."""
    return ModelShape(n_layers=n_layers, hidden=4096, n_q_heads=32, n_kv_heads=8, head_dim=128, ffn=14336,
                      vocab=128256, rope_base=500000.0)


def dense14b_shape(n_layers: int = 40) -> ModelShape:
    """A 14B-class backbone.  The second model of the paper's evaluation is named but its dimensions are not given;
    these are an ASSUMPTION in the style of current dense 14B decoders: 40 layers, hidden 5120, 40 query / 8 kv heads
    (five query heads per kv head), head_dim 128, FFN 17408, vocab 152064 (about 14.8 B parameters)."""
    return ModelShape(n_layers=n_layers, hidden=5120, n_q_heads=40, n_kv_heads=8, head_dim=128, ffn=17408,
                      vocab=152064, rope_base=1000000.0)


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _normal(shape, std, gen, device, dtype):
    # drawn in fp32 then cast, in slabs so that the fp32 staging buffer stays small
    out = torch.empty(shape, dtype=dtype, device=device)
    flat = out.view(-1)
    n = flat.numel()
    step = 1 << 26
    for i in range(0, n, step):
        m = min(step, n - i)
        flat[i:i + m] = (torch.randn(m, generator=gen, device=device, dtype=torch.float32) * std).to(dtype)
    return out


def model_weights(shape: ModelShape, seed: int = 0, device="cpu", dtype=torch.bfloat16) -> Dict[str, object]:
    """Random-init weights, every matrix stored [out_features, in_features]."""
    g = _gen(seed, device)
    H, d, F, V = shape.hidden, shape.head_dim, shape.ffn, shape.vocab
    nq, nkv = shape.n_q_heads, shape.n_kv_heads
    W: Dict[str, object] = {}
    W["embed"] = _normal((V, H), 0.02, g, device, dtype)
    W["lm_head"] = _normal((V, H), 0.02, g, device, dtype)
    W["final_norm"] = torch.ones(H, dtype=dtype, device=device)
    for k in ("attn_norm", "wqkv", "wo", "ffn_norm", "w_gate_up", "w_down"):
        W[k] = []
    for _ in range(shape.n_layers):
        W["attn_norm"].append(torch.ones(H, dtype=dtype, device=device))
        W["wqkv"].append(_normal(((nq + 2 * nkv) * d, H), 0.02, g, device, dtype))
        W["wo"].append(_normal((H, nq * d), 0.02, g, device, dtype))
        W["ffn_norm"].append(torch.ones(H, dtype=dtype, device=device))
        W["w_gate_up"].append(_normal((2 * F, H), 0.02, g, device, dtype))
        W["w_down"].append(_normal((H, F), 0.02, g, device, dtype))
    return W


def perturb_norm_gains(W: Dict[str, object], seed: int = 7) -> None:
    """Replace the all-ones norm gains by 1 + N(0, 0.1^2) in place, so that a test
    can tell a gain that is applied from one that is dropped."""
    g = _gen(seed, "cpu")

    def draw(t):
        return (1.0 + 0.1 * torch.randn(t.shape, generator=g)).to(t.dtype).to(t.device)

    W["final_norm"] = draw(W["final_norm"])
    W["attn_norm"] = [draw(t) for t in W["attn_norm"]]
    W["ffn_norm"] = [draw(t) for t in W["ffn_norm"]]


def token_ids(n: int, vocab: int, seed: int = 1) -> np.ndarray:
    """Uniform ids in [0, vocab-1): the last id is reserved for the mask token."""
    rng = np.random.default_rng(seed)
    return rng.integers(0, vocab - 1, size=n, dtype=np.int64).astype(np.int32)


def kv_values(n_pos: int, n_kv_heads: int, head_dim: int, seed: int = 2, device="cpu",
              dtype=torch.bfloat16):
    """Logical K and V, each [n_pos, n_kv_heads, head_dim], N(0, 1)."""
    g = _gen(seed, device)
    k = _normal((n_pos, n_kv_heads, head_dim), 1.0, g, device, dtype)
    v = _normal((n_pos, n_kv_heads, head_dim), 1.0, g, device, dtype)
    return k, v


def queries(n_tok: int, n_q_heads: int, head_dim: int, seed: int = 5, device="cpu", dtype=torch.bfloat16):
    g = _gen(seed, device)
    return _normal((n_tok, n_q_heads, head_dim), 1.0, g, device, dtype)


@dataclass
class BatchDescriptor:
    """Per-request lengths of one round plus a scattered page table."""
    ctx_len: np.ndarray        # [C] committed context tokens L_r
    verify_len: np.ndarray     # [C] pending verify tokens v_r
    block_size: np.ndarray     # [C] mask tokens b_r
    page_table: np.ndarray     # [C, stride] physical page ids (int32), -1 where unused
    n_pages: int               # physical pages the pool must hold
    page_size: int
    # correction branches of the draft-verify overlap (None = none anywhere)
    n_corr: Optional[np.ndarray] = None      # [C] 0..2
    corr_index: Optional[np.ndarray] = None  # [C, 2] replaced draft index, increasing
    corr_token: Optional[np.ndarray] = None  # [C, 2] replacement token ids
    corr_block: Optional[np.ndarray] = None  # [C] mask tokens per branch

    @property
    def n_req(self) -> int:
        return int(self.ctx_len.shape[0])

    @property
    def rows(self) -> np.ndarray:
        """Rows of each request in the ragged batch."""
        n = self.verify_len + self.block_size
        if self.n_corr is not None:
            n = n + self.n_corr * (1 + self.corr_block)
        return n

    @property
    def n_tokens(self) -> int:
        return int(self.rows.sum())

    def branch_kwargs(self) -> dict:
        """The branch arguments of binding.Batch."""
        if self.n_corr is None:
            return {}
        return {"n_corr": self.n_corr, "corr_index": self.corr_index, "corr_token": self.corr_token,
                "corr_block": self.corr_block}


def page_tables(ctx_len, n_new, page_size: int, seed: int, spare_pages: int = 0, stride: Optional[int] = None):
    """Scattered page tables: the physical pages of all requests are one random
    permutation, so that neighbouring logical pages are never neighbours in memory."""
    rng = np.random.default_rng(seed)
    need = [-(-(int(l) + int(n)) // page_size) for l, n in zip(ctx_len, n_new)]
    total = int(sum(need)) + spare_pages
    perm = rng.permutation(total).astype(np.int32)
    stride = max(need) if stride is None else stride
    pt = np.full((len(need), stride), -1, dtype=np.int32)
    o = 0
    for r, k in enumerate(need):
        pt[r, :k] = perm[o:o + k]
        o += k
    return pt, total


def batch_descriptor(n_req: int, block_choices, block_probs, ctx_lo: int, ctx_hi: int, seed: int = 3,
                     page_size: int = 16, verify_equals_block: bool = True) -> BatchDescriptor:
    """A ragged batch: block sizes drawn from block_choices, context lengths
    uniform in [ctx_lo, ctx_hi], verify length equal to the block size (one known
    token plus b-1 drafts: the steady state after a reused continuation block)."""
    rng = np.random.default_rng(seed)
    probs = None if block_probs is None else np.asarray(block_probs, dtype=np.float64)
    b = rng.choice(np.asarray(block_choices), size=n_req, p=probs).astype(np.int32)
    L = rng.integers(ctx_lo, ctx_hi + 1, size=n_req).astype(np.int32)
    v = b.copy() if verify_equals_block else (b + 1).astype(np.int32)
    pt, total = page_tables(L, v + b, page_size, seed + 1000)
    return BatchDescriptor(L, v, b, pt, total, page_size)


def fixed_descriptor(ctx_len, verify_len, block_size, seed: int = 3, page_size: int = 16, corr=None,
                     corr_block=None) -> BatchDescriptor:
    """corr: per request a list of up to two (draft index, replacement token); corr_block: mask tokens per branch."""
    L = np.asarray(ctx_len, dtype=np.int32)
    v = np.asarray(verify_len, dtype=np.int32)
    b = np.asarray(block_size, dtype=np.int32)
    if corr is None:
        pt, total = page_tables(L, v + b, page_size, seed + 1000)
        return BatchDescriptor(L, v, b, pt, total, page_size)
    nc = np.asarray([len(c) for c in corr], dtype=np.int32)
    ci = np.zeros((len(corr), 2), dtype=np.int32)
    ct = np.zeros((len(corr), 2), dtype=np.int32)
    for r, c in enumerate(corr):
        for k, (i, tok) in enumerate(c):
            ci[r, k], ct[r, k] = i, tok
    cb = np.asarray(corr_block, dtype=np.int32)
    pt, total = page_tables(L, v + b + nc * (1 + cb), page_size, seed + 1000)
    return BatchDescriptor(L, v, b, pt, total, page_size, nc, ci, ct, cb)


def with_correction_branches(desc: BatchDescriptor, vocab: int, n_branches: int = 2, seed: int = 11) -> BatchDescriptor:
    """The same requests with n_branches correction branches each (where the verify row has that many drafts):
    replaced draft indices drawn without replacement from 1..v-1, replacement tokens uniform, one block of the
    request's own size per branch, and page tables that cover the extra rows."""
    rng = np.random.default_rng(seed)
    corr = []
    for v in desc.verify_len:
        k = min(n_branches, max(int(v) - 1, 0))
        idx = np.sort(rng.choice(np.arange(1, int(v)), size=k, replace=False)) if k else []
        corr.append([(int(i), int(rng.integers(0, vocab - 1))) for i in idx])
    return fixed_descriptor(desc.ctx_len, desc.verify_len, desc.block_size, seed=seed, page_size=desc.page_size,
                            corr=corr, corr_block=desc.block_size)


def logits_normal(rows: int, vocab: int, seed: int = 6, device="cpu", dtype=torch.bfloat16):
    g = _gen(seed, device)
    return _normal((rows, vocab), 1.0, g, device, dtype)


def planted_accept_lengths(n_req: int, k: int, p: float = 0.25, seed: int = 4) -> np.ndarray:
    """min(G, k) with P(G = j) = p (1-p)^j, j >= 0: every draft is rejected with probability p."""
    rng = np.random.default_rng(seed)
    g = rng.geometric(p, size=n_req) - 1
    return np.minimum(g, k).astype(np.int32)


def plant_drafts(row_argmax: np.ndarray, n_req: int, k: int, accept: np.ndarray, vocab: int,
                 seed: int = 4) -> np.ndarray:
    """Verify tokens [n_req, k+1] for logits laid out as k+1 rows per request.

    row_argmax[r*(k+1)+i] is the id that row i of request r selects (supplied by
    the caller).  Token 0 is arbitrary; tokens 1..a equal the ids selected by
    rows 0..a-1; token a+1 (if any) is forced to differ from row a's id; later
    tokens are uniform random.
    """
    rng = np.random.default_rng(seed + 17)
    y = rng.integers(0, vocab - 1, size=(n_req, k + 1), dtype=np.int64)
    am = np.asarray(row_argmax).reshape(n_req, k + 1)
    for r in range(n_req):
        a = int(accept[r])
        y[r, 1:a + 1] = am[r, :a]
        if a + 1 <= k:
            wrong = int(y[r, a + 1])
            if wrong == int(am[r, a]):
                wrong = (wrong + 1) % (vocab - 1)
            y[r, a + 1] = wrong
    return y.astype(np.int32)


def policy_table(blocks=(8, 16, 32), n_bins: int = 12, rho_cost=(0.9, 1.5, 2.6), seed: int = 13):
    """A synthetic stand-in for the calibrated estimate V_B(s, z) of the block-size rule and for the weighted
    execution cost rho_C * T_C(B): certainty bin edges evenly spaced over s in [-3, 0], and a value that grows with
    certainty and with the candidate block, a little more after a fully accepted block, plus seeded noise so that
    no two entries tie.  Shapes: value [n_blocks, n_bins, n_blocks, 2], cost [n_blocks].  Calibration data of the
    paper's models is not available; only the shape of the lookup matters here."""
    rng = np.random.default_rng(seed)
    nb = len(blocks)
    edges = np.linspace(-3.0, 0.0, n_bins + 1)[1:-1].astype(np.float32)
    centre = np.linspace(-3.0, 0.0, n_bins + 1)[:-1] + 1.5 / n_bins
    p = 1.0 / (1.0 + np.exp(-(2.0 * centre + 4.0)))                    # per-token acceptance grows with certainty
    value = np.zeros((nb, n_bins, nb, 2), dtype=np.float32)
    for j, B in enumerate(blocks):
        for k in range(n_bins):
            for jp in range(nb):
                for f in (0, 1):
                    pk = min(0.995, p[k] * (1.0 + 0.05 * f) * (1.0 + 0.01 * jp))
                    value[j, k, jp, f] = (1.0 - pk ** B) / (1.0 - pk) + 0.01 * rng.standard_normal()
    return {"blocks": np.asarray(blocks, dtype=np.int32), "s_edges": edges, "value": value,
            "cost": np.asarray(rho_cost, dtype=np.float32)}


# Transition percentages between acceptance intervals [1,8], (8,16], (16,32] of adjacent rounds at block size 32, as
# printed in the paper's transition table (Sec. 4.2).  Random-init weights accept almost nothing, so multi-round
# workloads draw their acceptance lengths from this chain: the interval follows the table, the length is uniform over
# the interval's integers (the paper prints nothing about the distribution inside an interval).
ACCEPT_INTERVALS = ((1, 8), (9, 16), (17, 32))
ACCEPT_TRANSITIONS = ((70.30, 18.11, 11.60), (58.39, 22.42, 19.19), (20.83, 12.51, 66.66))


def acceptance_chain_lengths(n_rounds: int, n_req: int, seed: int = 4) -> np.ndarray:
    """Emitted tokens per round and request, int32 [n_rounds, n_req]: one independent chain per request, started from
    a state drawn uniformly."""
    rng = np.random.default_rng(seed)
    P = np.asarray(ACCEPT_TRANSITIONS, dtype=np.float64)
    P = P / P.sum(axis=1, keepdims=True)
    out = np.zeros((n_rounds, n_req), dtype=np.int32)
    for r in range(n_req):
        s = int(rng.integers(0, 3))
        for t in range(n_rounds):
            lo, hi = ACCEPT_INTERVALS[s]
            out[t, r] = rng.integers(lo, hi + 1)
            s = int(rng.choice(3, p=P[s]))
    return out
