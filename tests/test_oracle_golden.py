"""The oracle against small fixtures written out by hand from the paper's equations and rules (tests/golden)."""
import os

import numpy as np

from oracle import recg_oracle as orc

HERE = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def read_sections(name):
    out, cur = {}, None
    for line in open(os.path.join(HERE, name)):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("["):
            cur = line.strip("[]")
            out[cur] = []
        else:
            out[cur].append([int(t) for t in line.split()])
    return {k: np.asarray(v) for k, v in out.items()}


def test_eq1_masks():
    g = read_sections("eq1_masks_P3_B2.txt")
    P, B = 3, 2
    assert np.array_equal(orc.visibility_matrix(P, B).astype(int), g["M_Diff"])
    n = P + B
    i, j = np.arange(n).reshape(n, 1), np.arange(n).reshape(1, n)
    assert np.array_equal(np.asarray(orc.mask_ar(i, j)).astype(int), g["M_AR"])
    # the fused round is the same mask with prefix = context + verify tokens, restricted to the new rows
    assert np.array_equal(orc.fused_round_visibility(1, 2, 2).astype(int), g["M_Diff"][1:])


def test_overlap_rows():
    g = read_sections("overlap_rows_L2_v3_b2.txt")
    pos, vis, kind = orc.overlap_round_rows(2, 3, 2, [(2, 99)], 1)
    assert np.array_equal(vis.astype(int), g["visibility"])
    assert pos.tolist() == g["positions"][0].tolist()
    assert kind == ["v", "v", "v", "c", "c", "r", "m"]
