"""Device-resident rounds: N rounds enqueued back to back (step, verification, block-size rule, next-round bookkeeping)
with one synchronisation at the end, against the oracle."""
import numpy as np
import pytest
import torch

from oracle import recg_oracle as orc
from paper_2609_34388_b200 import binding, synth
from tests._util import oracle_cfg, oracle_weights

pytestmark = pytest.mark.gpu


def tiny():
    shape = synth.tiny_shape()
    W = synth.model_weights(shape, seed=0, dtype=torch.bfloat16)
    Wd = {k: ([t.cuda() for t in v] if isinstance(v, list) else v.cuda()) for k, v in W.items()}
    return shape, Wd, oracle_cfg(shape), oracle_weights(W)


def prefilled(ctx, ocfg, W64, prompts, pt, pool, n_pages):
    pre = [orc.prefill(ocfg, W64, p) for p in prompts]
    for i, (kv, L, _) in enumerate(pre):
        for l, (K, V) in enumerate(kv):
            ctx.recg_kv_write(pool, n_pages, l, pt[i], 0, torch.from_numpy(K).to(torch.bfloat16).cuda(),
                              torch.from_numpy(V).to(torch.bfloat16).cuda())
    return pre


def test_device_rounds_emit_the_greedy_text_and_the_rule_s_block_sizes():
    """Six rounds of three requests of the tiny model with no host round trip: the device assembles every next round from
    the verification results and the block-size rule's choice.  Afterwards (one sync) the logged tokens must be the
    oracle's greedy continuation of every prompt (speculation is lossless), the logged lengths must follow the oracle's
    bookkeeping between rounds, and the logged block sizes must be what the oracle's rule picks from the logged mean
    entropies (float32 decisions on the same inputs).  Request 0 starts with three teacher-forced drafts, so a round
    that accepts drafts occurs."""
    shape, Wd, ocfg, W64 = tiny()
    t = synth.policy_table((4, 8, 16), 16, rho_cost=(0.3, 0.6, 1.2), seed=3)
    t["s_edges"] = (t["s_edges"] / 3.0 * 0.2 - (np.log(shape.vocab) - 0.2)).astype(np.float32)   # bins around ln(vocab)
    C, rounds, max_verify = 3, 6, 16
    prompts = [synth.token_ids(30 + 7 * i, shape.vocab, seed=20 + i).tolist() for i in range(C)]
    ars = [orc.greedy_ar(ocfg, W64, p, rounds + 8) for p in prompts]
    Ls = [len(p) - 1 for p in prompts]
    pt, n_pages = synth.page_tables(Ls, [rounds * 17 + 40] * C, 16, seed=5)
    ctx = binding.Context(binding.make_config(shape, C, 128, pt.shape[1]), Wd)
    ctx.recg_policy_load(t["blocks"], t["s_edges"], t["value"], t["cost"])
    pool = binding.alloc_kv_pool(ctx, n_pages)
    pre = prefilled(ctx, ocfg, W64, prompts, pt, pool, n_pages)
    ys = [list(p[2]) for p in pre]
    ys[0] = ys[0] + ars[0][:3]                      # three correct drafts: round 0 of request 0 accepts all of them
    blocks0 = [8] * C
    db = binding.DeviceBatch(Ls, [len(y) for y in ys], blocks0, ys, max_verify, pt, pool, n_pages, rows_hint=32)
    st0 = {"e1": [np.float32(7.0)] * C, "e2": [np.float32(7.0)] * C, "block_index": [1] * C, "full": [0] * C}
    dst = {k: torch.tensor(v, dtype=torch.float32 if k[0] == "e" else torch.int32, device="cuda") for k, v in st0.items()}
    nxt = torch.zeros(C, dtype=torch.int32, device="cuda")
    log = binding.RoundLog(C, rounds, 64)
    for rnd in range(rounds):                       # nothing below waits for the device
        ctx.recg_step_device(db)
        ctx.recg_verify_device()
        ctx.recg_policy_step(dst, nxt)
        ctx.recg_next_round(db, rnd, next_block=nxt, log=log)
    ctx.recg_sync()
    assert int(log.n_rounds[0]) == rounds
    n_out = log.n_tokens.cpu().numpy()
    toks = log.tokens.cpu().numpy()
    acc, blk, ver = log.accept_len.cpu().numpy(), log.block_size.cpu().numpy(), log.verify_len.cpu().numpy()
    ent = log.entropy_mean.cpu().numpy()
    # text: lossless
    for i in range(C):
        assert toks[i, : n_out[i]].tolist() == ars[i][: n_out[i]], i
        assert n_out[i] == int(acc[:, i].sum()) + rounds
    assert acc[0, 0] == 3 and ver[0, 0] == 4 and acc[1:, 0].max() == 0       # random weights draft nothing acceptable later
    # bookkeeping between rounds: verify lengths and context lengths follow the oracle's rule (no block is reused here:
    # a random-weight draft never equals the bonus token)
    L = np.asarray(Ls)
    for rnd in range(rounds):
        if rnd:
            assert (ver[rnd] == 1).all()
        L = L + acc[rnd] + 1
    assert db.ctx_len.cpu().numpy().tolist() == L.tolist()
    # block sizes: the oracle's rule on the logged float32 entropies
    st = {k: list(v) for k, v in st0.items()}
    want_blocks = [blocks0]
    for rnd in range(rounds):
        want_blocks.append(orc.policy_step(st, ent[rnd], acc[rnd], ver[rnd], t["blocks"], t["s_edges"], t["value"], t["cost"],
                                           dtype=np.float32))
    for rnd in range(rounds):
        assert blk[rnd].tolist() == want_blocks[rnd], rnd
    assert db.block_size.cpu().numpy().tolist() == want_blocks[rounds]
    assert len({b for row in want_blocks for b in row}) > 1          # the rule did change sizes on the way
    ctx.recg_free()


def test_device_rounds_with_planted_acceptance_follow_the_chain():
    """Random weights accept nothing, so longer runs take their acceptance lengths from the interval chain of the paper's
    transition table.  The device's bookkeeping over 12 rounds (context, verify length, accepted drafts per round) must
    be the oracle's lengths-only trace for the same planted lengths, including rounds that reuse the drafted block."""
    shape, Wd, ocfg, W64 = tiny()
    C, rounds, b = 4, 12, 16
    rng = np.random.default_rng(9)
    P = orc.chain_matrix()
    planted = np.zeros((rounds, C), dtype=np.int32)
    for i in range(C):
        _, lens = orc.acceptance_chain(P, orc.TABLE1_INTERVALS, i % 3, rng.random(rounds), rng.random(rounds))
        planted[:, i] = lens
    Ls = [20 + 9 * i for i in range(C)]
    pt, n_pages = synth.page_tables(Ls, [rounds * 17 + 64] * C, 16, seed=6)
    ctx = binding.Context(binding.make_config(shape, C, 160, pt.shape[1]), Wd)
    pool = binding.alloc_kv_pool(ctx, n_pages, fill="normal")
    ys = [[5 + i] for i in range(C)]
    db = binding.DeviceBatch(Ls, [1] * C, [b] * C, ys, 32, pt, pool, n_pages)
    log = binding.RoundLog(C, rounds, 400)
    pl = torch.from_numpy(planted).cuda()
    for rnd in range(rounds):
        ctx.recg_step_device(db)
        ctx.recg_verify_device()
        ctx.recg_next_round(db, rnd, planted_emitted=pl[rnd], log=log)
    ctx.recg_sync()
    acc, blk, ver = log.accept_len.cpu().numpy(), log.block_size.cpu().numpy(), log.verify_len.cpu().numpy()
    reused = 0
    for i in range(C):
        trace = orc.planted_rounds(Ls[i], 1, [b] * rounds, planted[:, i].tolist())
        assert ver[:, i].tolist() == [t[1] for t in trace], i
        assert blk[:, i].tolist() == [t[2] for t in trace]
        assert acc[:, i].tolist() == [t[3] for t in trace]
        assert int(log.n_tokens[i]) == sum(t[4] for t in trace)
        assert int(db.ctx_len[i]) == trace[-1][0] + trace[-1][4]
        reused += sum(1 for t in trace if t[5] and t[1] > 1)
    assert reused > 0 and ver.max() == b
    ctx.recg_free()


def test_device_round_that_breaks_a_capacity_is_refused_on_the_device():
    shape, Wd, ocfg, W64 = tiny()
    pt, n_pages = synth.page_tables([10, 10], [40, 40], 16, seed=7)
    ctx = binding.Context(binding.make_config(shape, 2, 32, pt.shape[1]), Wd)
    pool = binding.alloc_kv_pool(ctx, n_pages, fill="normal")
    db = binding.DeviceBatch([10, 10], [1, 1], [30, 30], [[1], [2]], 8, pt, pool, n_pages)     # 62 rows > max_tokens = 32
    log = binding.RoundLog(2, 2, 16)
    ctx.recg_step_device(db)
    ctx.recg_verify_device()
    ctx.recg_next_round(db, 0, log=log)
    with pytest.raises(binding.RecgError) as e:
        ctx.recg_sync()
    assert e.value.status == 6
    assert db.ctx_len.cpu().tolist() == [10, 10] and log.n_tokens.cpu().tolist() == [0, 0]     # the empty round changed nothing
    with pytest.raises(binding.RecgError) as e:            # results of a device-resident round stay on the device
        ctx.recg_verify(None, None, host=True, n_req=2, n_tok=4, n_ver=2)
    assert e.value.status == 1
    db2 = binding.DeviceBatch([10, 10], [1, 1], [4, 4], [[1], [2]], 8, pt, pool, n_pages)
    ctx.recg_step_device(db2)                               # the context is still usable
    ctx.recg_verify_device()
    ctx.recg_sync()
    ctx.recg_free()


@pytest.mark.parametrize("n_req,capacity,blocks", [(12, 512, [4, 8, 16, 32]), (3, 128, [4, 8, 16]), (1, 64, [16]), (1, 32, [8])])
def test_device_round_on_8b_shaped_layers_equals_the_host_round(n_req, capacity, blocks):
    """The same ragged batch through two 8B-shaped layers (tcgen05 projections and attention) once with host descriptor
    arrays and once with device arrays (row count unknown to the host, launches sized for the capacity): logits agree
    within the batch-invariance tolerance, integers wherever the top-2 gap is not a near tie.  Capacities of at most 128
    rows take the projections whose cut tiles are handed over inside clusters, with the row count read on the device."""
    shape = synth.llama8b_shape(2)
    shape.vocab = 8192
    W = synth.model_weights(shape, seed=0, dtype=torch.bfloat16)
    Wd = {k: ([t.cuda() for t in v] if isinstance(v, list) else v.cuda()) for k, v in W.items()}
    desc = synth.batch_descriptor(n_req, blocks, None, 100, 2000, seed=31)
    T = desc.n_tokens
    assert T <= capacity
    ctx = binding.Context(binding.make_config(shape, n_req, capacity, desc.page_table.shape[1]), Wd)     # capacity above the row count
    pool = binding.alloc_kv_pool(ctx, desc.n_pages, fill="normal")
    ys = synth.token_ids(int(desc.verify_len.sum()), shape.vocab, seed=1)
    host = binding.Batch(desc.ctx_len, desc.verify_len, desc.block_size, ys, desc.page_table, pool, desc.n_pages)
    ref = ctx.logits_tensor(ctx.recg_step(host))
    g_ref = {k: v.copy() for k, v in ctx.recg_verify(host).items()}
    cuv = np.concatenate([[0], np.cumsum(desc.verify_len)])
    per_req = [ys[cuv[i]: cuv[i + 1]].tolist() for i in range(desc.n_req)]
    pt = np.where(desc.page_table >= 0, desc.page_table, 0)
    db = binding.DeviceBatch(desc.ctx_len, desc.verify_len, desc.block_size, per_req, 32, pt, pool, desc.n_pages, rows_hint=T)
    lg = ctx.recg_step_device(db)
    assert lg.n_rows == capacity
    got = binding.device_view(lg.data, (lg.n_rows, lg.vocab), torch.float32)[:T].clone()
    out = binding.VerifyOut(desc.n_req, T, int(desc.verify_len.sum()), host=False)
    ctx.recg_verify(None, None, host=False, out=out)
    ctx.recg_sync()
    assert float((got - ref).abs().max()) <= 1e-2 * float(ref.abs().max())
    top2 = torch.topk(ref, 2, dim=1).values
    clear = ((top2[:, 0] - top2[:, 1]) >= 1e-2).cpu().numpy()
    v = out.views()
    assert (v["top1"].cpu().numpy()[clear] == g_ref["top1"][clear]).all()
    cu = np.concatenate([[0], np.cumsum(desc.rows)])
    for i in range(desc.n_req):
        if clear[cu[i]: cu[i + 1]].all():
            assert int(v["accept_len"][i]) == int(g_ref["accept_len"][i])
            assert int(v["new_ctx_len"][i]) == int(g_ref["new_ctx_len"][i])
    ctx.recg_free()
