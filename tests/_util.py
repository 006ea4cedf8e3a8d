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
