"""The allocation-free row-statistics entry point against the context-based verify and the oracle, two calls in a row.

Collected last on purpose: if it fails, a run that stops at the first failure has already run everything
else.  It must pass alone in a fresh process and after the other tests.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import recg_oracle as orc
from paper_2609_34388_b200 import binding, synth

pytestmark = pytest.mark.gpu


def reference_stats(lg):
    """The existing entry point (recg_verify on a context) for the same logits."""
    rows, vocab = lg.shape
    shape = synth.ModelShape(n_layers=0, hidden=64, n_q_heads=4, n_kv_heads=2, head_dim=64, ffn=64, vocab=vocab)
    ctx = binding.Context(binding.make_config(shape, 1, rows, 1))
    got = ctx.recg_verify(binding.Batch([0], [0], [rows], None), lg)      # one request of `rows` mask rows
    ctx.recg_sync()
    ctx.recg_free()
    return got


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_static_scratch_matches_context_verify_twice(dtype):
    vocab = 128256
    first = synth.logits_normal(37, vocab, seed=71, device="cuda", dtype=dtype)
    second = synth.logits_normal(9, vocab, seed=72, device="cuda", dtype=dtype)      # fewer rows: stale partials remain
    for lg in (first, second):
        ref = reference_stats(lg)
        got = binding.recg_row_stats_static(lg)
        torch.cuda.synchronize()
        assert got["top1"].cpu().numpy().tolist() == ref["top1"].tolist()
        assert got["top2"].cpu().numpy().tolist() == ref["top2"].tolist()
        np.testing.assert_allclose(got["p1"].cpu().numpy(), ref["p1"], rtol=2e-4, atol=1e-7)
        np.testing.assert_allclose(got["p2"].cpu().numpy(), ref["p2"], rtol=2e-4, atol=1e-7)
        np.testing.assert_allclose(got["entropy"].cpu().numpy(), ref["entropy"], rtol=2e-4, atol=1e-5)
        # and against the oracle's definition of the per-row statistics on the same values (ids exact)
        host = lg.double().cpu().numpy()
        for r in range(host.shape[0]):
            want = orc.row_stats(host[r])
            assert int(got["top1"][r]) == want["top1"] and int(got["top2"][r]) == want["top2"]
            assert abs(float(got["p1"][r]) - want["p1"]) <= 2e-4 * want["p1"] + 1e-7
            assert abs(float(got["p2"][r]) - want["p2"]) <= 2e-4 * want["p2"] + 1e-7
            assert abs(float(got["entropy"][r]) - want["entropy"]) <= 2e-4 * want["entropy"] + 1e-5


def test_static_scratch_rejects_oversize_and_bad_arguments():
    lib = binding.lib()
    lg = torch.zeros((4, 2048), dtype=torch.float32, device="cuda")
    args = [None] * 5 + [None]
    assert lib.recg_row_stats_static(lg.data_ptr(), 1, 70000, 2048, *args) == 3          # beyond the static scratch
    assert lib.recg_row_stats_static(lg.data_ptr(), 1, 65537, 2048, *args) == 3
    assert b"65536" in lib.recg_row_stats_static_error()
    assert lib.recg_row_stats_static(None, 1, 4, 2048, *args) == 1
    assert lib.recg_row_stats_static(lg.data_ptr(), 7, 4, 2048, *args) == 1
    assert lib.recg_row_stats_static(lg.data_ptr(), 1, 0, 2048, *args) == 0               # nothing to do
    torch.cuda.synchronize()
