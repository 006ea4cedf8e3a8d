"""Host-side scheduling helpers: bucketing by block size."""
import numpy as np

from paper_2609_34388_b200 import schedule, synth


def test_buckets_partition_the_batch_and_keep_order():
    desc = synth.batch_descriptor(64, [4, 8, 16, 32], None, 100, 900, seed=5)
    buckets = schedule.bucket_by_block(desc.block_size)
    assert list(buckets) == sorted(set(desc.block_size.tolist()))
    flat = [r for idx in buckets.values() for r in idx]
    assert sorted(flat) == list(range(64))
    for b, idx in buckets.items():
        assert idx == sorted(idx) and all(desc.block_size[r] == b for r in idx)
    subs = schedule.bucketed(desc)
    assert sum(s.n_req for s in subs) == 64 and sum(s.n_tokens for s in subs) == desc.n_tokens
    for s, idx in zip(subs, buckets.values()):
        assert np.array_equal(s.ctx_len, desc.ctx_len[idx]) and np.array_equal(s.page_table, desc.page_table[idx])
        assert s.n_pages == desc.n_pages and len(set(s.block_size.tolist())) == 1
        # a bucket has nothing to pad as long as verify lengths follow the block size
        assert schedule.padded_rows(s) == s.n_tokens
    assert schedule.padded_rows(desc) == 64 * int(desc.rows.max()) > desc.n_tokens


def test_sub_descriptor_keeps_branches_and_token_slices():
    base = synth.fixed_descriptor([10, 20, 30], [4, 1, 6], [4, 8, 4])
    desc = synth.with_correction_branches(base, 1000, 2, seed=3)
    sub = schedule.sub_descriptor(desc, [2, 0])
    assert sub.n_req == 2 and sub.rows.tolist() == [desc.rows[2], desc.rows[0]]
    assert np.array_equal(sub.corr_index, desc.corr_index[[2, 0]]) and np.array_equal(sub.corr_block, desc.corr_block[[2, 0]])
    sl = schedule.verify_token_slices(desc, [2, 0])
    assert (sl[0].start, sl[0].stop, sl[1].start, sl[1].stop) == (5, 11, 0, 4)
    plain = schedule.sub_descriptor(base, [1])
    assert plain.n_corr is None and plain.n_tokens == 9
