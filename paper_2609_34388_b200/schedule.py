"""Host-side batch scheduling helpers: bucketing requests by draft block size.

A server whose kernels pad every request of a batch to the longest one loses work when block sizes are mixed; the
usual remedy is to run one batch per block size.  The step of this library is ragged (it computes valid rows only),
so it can also run the mixed batch directly.  These helpers build both schedules from one batch descriptor so that
the two can be compared; they touch no GPU state.
"""
from __future__ import annotations

from typing import Dict, List

import numpy as np

from .synth import BatchDescriptor


def bucket_by_block(block_size) -> Dict[int, List[int]]:
    """Request indices grouped by block size, block sizes ascending, request order kept inside a bucket."""
    out: Dict[int, List[int]] = {}
    for r, b in enumerate(np.asarray(block_size).tolist()):
        out.setdefault(int(b), []).append(r)
    return dict(sorted(out.items()))


def sub_descriptor(desc: BatchDescriptor, idx: List[int]) -> BatchDescriptor:
    """The requests idx of desc as a batch of their own (same physical pages, same pool)."""
    idx = list(idx)
    pick = lambda a: None if a is None else np.ascontiguousarray(a[idx])
    return BatchDescriptor(pick(desc.ctx_len), pick(desc.verify_len), pick(desc.block_size), pick(desc.page_table),
                           desc.n_pages, desc.page_size, pick(desc.n_corr), pick(desc.corr_index), pick(desc.corr_token),
                           pick(desc.corr_block))


def bucketed(desc: BatchDescriptor) -> List[BatchDescriptor]:
    """One batch per block size."""
    return [sub_descriptor(desc, idx) for idx in bucket_by_block(desc.block_size).values()]


def verify_token_slices(desc: BatchDescriptor, idx: List[int]) -> List[slice]:
    """Where the verify tokens of requests idx sit in the concatenated verify_tokens array of desc."""
    off = np.concatenate([[0], np.cumsum(desc.verify_len)])
    return [slice(int(off[r]), int(off[r + 1])) for r in idx]


def padded_rows(desc: BatchDescriptor) -> int:
    """Rows a kernel that pads every request to the longest one would compute for this batch."""
    return int(desc.n_req * int(desc.rows.max())) if desc.n_req else 0
