"""Test helpers: data conversion between the generators, the oracle and the binding."""
import numpy as np
import torch

from oracle import recg_oracle as orc


def oracle_cfg(shape) -> orc.ModelConfig:
    return orc.ModelConfig(**shape.as_dict())


def f64(t) -> np.ndarray:
    """Exact widening of a torch tensor (bf16/fp32) to float64 numpy."""
    return t.detach().to("cpu").to(torch.float64).numpy()


def oracle_weights(W) -> dict:
    out = {}
    for k, val in W.items():
        out[k] = [f64(t) for t in val] if isinstance(val, list) else f64(val)
    return out


def bf16_round(a: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even to bf16, returned as float64 (for the oracle's act_round hook)."""
    return torch.from_numpy(np.ascontiguousarray(a)).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()


def oracle_rounds_together(cfg, W, reqs, act_round=None):
    """Several requests' fused rounds in ONE call of the oracle's generic backbone (orc.decoder_rows), so that a deep
    model's weights are widened to float64 once per layer instead of once per request and layer.

    reqs: dicts with "kv" (per layer (K, V), at least L positions), "L", "y" (verify ids) and "b".  The call's prefix is
    the requests' contexts one after the other, its rows are the requests' new rows one after the other, and the
    visibility matrix is block diagonal: request i's rows see request i's context columns and request i's new rows
    exactly as orc.fused_round_visibility(L_i, v_i, b_i) says, and nothing of any other request.  Positions are each
    request's own (L_i ..).  Returns per request (logits [n_i, V], hidden [n_i, H]).
    tests/test_oracle_model.py checks that this equals one orc.fused_round_cached call per request.
    """
    Ls = [r["L"] for r in reqs]
    ns = [len(r["y"]) + r["b"] for r in reqs]
    Ltot, ntot = sum(Ls), sum(ns)
    ids, pos = [], []
    vis = np.zeros((ntot, Ltot + ntot), dtype=bool)
    c0 = r0 = 0
    for r, L, n in zip(reqs, Ls, ns):
        v = len(r["y"])
        ids += list(r["y"]) + [cfg.mask_id()] * r["b"]
        pos += list(range(L, L + n))
        block = orc.fused_round_visibility(L, v, r["b"])          # [n, L + n]
        vis[r0:r0 + n, c0:c0 + L] = block[:, :L]
        vis[r0:r0 + n, Ltot + r0:Ltot + r0 + n] = block[:, L:]
        c0 += L
        r0 += n
    n_layers = len(reqs[0]["kv"])
    prefix = [(np.concatenate([r["kv"][l][0][:r["L"]] for r in reqs], axis=0),
               np.concatenate([r["kv"][l][1][:r["L"]] for r in reqs], axis=0)) for l in range(n_layers)]
    logits, _, hidden = orc.decoder_rows(cfg, W, ids, np.asarray(pos), vis, prefix, act_round)
    out, r0 = [], 0
    for n in ns:
        out.append((logits[r0:r0 + n], hidden[r0:r0 + n]))
        r0 += n
    return out


GAP_BINS = (1e-3, 1e-2, 3e-2, 1e-1)


def flip_histogram(gaps) -> str:
    """Counts of rows whose top-1 differs from the oracle's, by the oracle's top-2 logit gap."""
    gaps = np.asarray(list(gaps), dtype=np.float64)
    edges = (0.0,) + GAP_BINS + (np.inf,)
    parts = []
    for lo, hi in zip(edges[:-1], edges[1:]):
        parts.append(f"[{lo:g}, {hi:g}): {int(((gaps >= lo) & (gaps < hi)).sum())}")
    return ", ".join(parts)
