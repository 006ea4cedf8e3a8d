"""GPU parity of the block-size rule (Sec. 5.2, Eq. 2-3) against the oracle, both deciding in float32."""
import numpy as np
import pytest
import torch

from oracle import recg_oracle as orc
from paper_2609_34388_b200 import binding, synth
from tests._util import oracle_cfg, oracle_weights

pytestmark = pytest.mark.gpu


def verify_only_ctx(n_req, vocab=512):
    shape = synth.ModelShape(n_layers=0, hidden=64, n_q_heads=4, n_kv_heads=2, head_dim=64, ffn=64, vocab=vocab)
    return binding.Context(binding.make_config(shape, n_req, 40 * n_req, 1))


def dev_state(st):
    return {"e1": torch.tensor(st["e1"], dtype=torch.float32, device="cuda"),
            "e2": torch.tensor(st["e2"], dtype=torch.float32, device="cuda"),
            "block_index": torch.tensor(st["block_index"], dtype=torch.int32, device="cuda"),
            "full": torch.tensor(st["full"], dtype=torch.int32, device="cuda")}


@pytest.mark.parametrize("blocks,n_bins,seed", [((8, 16, 32), 12, 13), ((2, 4, 8, 16), 64, 14), ((16,), 1, 15),
                                                ((4, 8, 16, 32, 64, 128, 256, 512), 5, 16)])
def test_policy_step_matches_oracle(blocks, n_bins, seed):
    rng = np.random.default_rng(seed)
    nb = len(blocks)
    t = synth.policy_table(blocks, n_bins, rho_cost=tuple(0.05 * b + 0.5 for b in blocks), seed=seed)
    C = 300
    ctx = verify_only_ctx(C)
    ctx.recg_policy_load(t["blocks"], t["s_edges"], t["value"], t["cost"])
    st = {"e1": rng.uniform(0, 3, C).astype(np.float32).tolist(), "e2": rng.uniform(0, 3, C).astype(np.float32).tolist(),
          "block_index": rng.integers(0, nb, C).tolist(), "full": rng.integers(0, 2, C).tolist()}
    st = {k: [np.float32(x) for x in v] if k in ("e1", "e2") else v for k, v in st.items()}
    dst = dev_state(st)
    nxt = torch.full((C,), -1, dtype=torch.int32, device="cuda")
    for rnd in range(3):
        v = rng.integers(0, 10, C)
        v[:3] = [0, 1, 9]
        a = np.array([rng.integers(0, max(x, 1)) for x in v])
        full_rows = rng.random(C) < 0.4
        a[full_rows] = np.maximum(v[full_rows] - 1, 0)
        ent = rng.uniform(0, 3, C).astype(np.float32)
        # lay the batch out (verify-only call on dummy logits), then the rule on explicit device arrays
        batch = binding.Batch([0] * C, v, [1] * C, np.zeros(int(v.sum()), np.int32))
        ctx.recg_verify(batch, torch.zeros((batch.n_tok, 512), dtype=torch.float32, device="cuda"))
        ctx.recg_policy_step(dst, nxt, torch.from_numpy(ent).cuda(), torch.from_numpy(a.astype(np.int32)).cuda())
        ctx.recg_sync()
        want = orc.policy_step(st, ent, a, v, t["blocks"], t["s_edges"], t["value"], t["cost"], dtype=np.float32)
        assert nxt.cpu().tolist() == want, rnd
        assert dst["block_index"].cpu().tolist() == st["block_index"]
        assert dst["full"].cpu().tolist() == st["full"]
        assert dst["e1"].cpu().numpy().tolist() == [float(x) for x in st["e1"]]
        assert dst["e2"].cpu().numpy().tolist() == [float(x) for x in st["e2"]]
    if nb > 1:
        assert len(set(nxt.cpu().tolist())) > 1        # the table really discriminates
    ctx.recg_free()


def test_policy_rejections():
    ctx = verify_only_ctx(4)
    t = synth.policy_table()
    st = dev_state({"e1": [0.0] * 4, "e2": [0.0] * 4, "block_index": [0] * 4, "full": [0] * 4})
    nxt = torch.zeros(4, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.RecgError):       # no table yet
        ctx.recg_policy_step(st, nxt)
    with pytest.raises(binding.RecgError):       # blocks not ascending
        ctx.recg_policy_load([8, 8, 32], t["s_edges"], t["value"], t["cost"])
    with pytest.raises(binding.RecgError):       # edges not ascending
        ctx.recg_policy_load(t["blocks"], t["s_edges"][::-1].copy(), t["value"], t["cost"])
    with pytest.raises(binding.RecgError):       # too many candidates
        big = synth.policy_table(tuple(range(1, 10)), 4, rho_cost=tuple([1.0] * 9))
        ctx.recg_policy_load(big["blocks"], big["s_edges"], big["value"], big["cost"])
    ctx.recg_policy_load(t["blocks"], t["s_edges"], t["value"], t["cost"])
    with pytest.raises(binding.RecgError):       # table loaded, but no batch has been laid out
        ctx.recg_policy_step(st, nxt)
    ctx.recg_free()


def test_policy_drives_block_sizes_of_a_tiny_loop():
    """Several rounds of the tiny model in which the device picks every request's next block size from the library's
    own verification results (no host copy of the entropies in between); the oracle's rule applied to the same
    float32 entropies must pick the same sizes, the chosen sizes are used for the next round, and the emitted text
    stays the oracle's greedy continuation."""
    shape = synth.tiny_shape()
    W = synth.model_weights(shape, seed=0, dtype=torch.bfloat16)
    ocfg, W64 = oracle_cfg(shape), oracle_weights(W)
    Wd = {k: ([t.cuda() for t in v] if isinstance(v, list) else v.cuda()) for k, v in W.items()}
    t = synth.policy_table((4, 8, 16), 16, rho_cost=(0.3, 0.6, 1.2), seed=3)
    # random weights give near-uniform rows: entropies close to ln(vocab); centre the bins there
    t["s_edges"] = (t["s_edges"] / 3.0 * 0.2 - (np.log(shape.vocab) - 0.2)).astype(np.float32)
    C, rounds = 3, 5
    prompts = [synth.token_ids(30 + 7 * i, shape.vocab, seed=20 + i).tolist() for i in range(C)]
    pre = [orc.prefill(ocfg, W64, p) for p in prompts]
    Ls = [p[1] for p in pre]
    ys = [list(p[2]) for p in pre]
    pt, n_pages = synth.page_tables(Ls, [rounds * 17 + 40] * C, 16, seed=5)
    ctx = binding.Context(binding.make_config(shape, C, 128, pt.shape[1]), Wd)
    ctx.recg_policy_load(t["blocks"], t["s_edges"], t["value"], t["cost"])
    pool = binding.alloc_kv_pool(ctx, n_pages)
    for i, (kv, L, _) in enumerate(pre):
        for l, (K, V) in enumerate(kv):
            ctx.recg_kv_write(pool, n_pages, l, pt[i], 0, torch.from_numpy(K).to(torch.bfloat16).cuda(),
                              torch.from_numpy(V).to(torch.bfloat16).cuda())
    st = {"e1": [np.float32(7.0)] * C, "e2": [np.float32(7.0)] * C, "block_index": [1] * C, "full": [0] * C}
    dst = dev_state(st)
    nxt = torch.zeros(C, dtype=torch.int32, device="cuda")
    blocks = [8] * C
    ars = [orc.greedy_ar(ocfg, W64, p, rounds * 3 + 8) for p in prompts]
    outs = [[] for _ in range(C)]
    picked = []
    for rnd in range(rounds):
        if rnd == 2:   # teacher-forced drafts for request 0 so that a full acceptance occurs
            ys[0] = [ys[0][0]] + ars[0][len(outs[0]): len(outs[0]) + 3]
        batch = binding.Batch(Ls, [len(y) for y in ys], blocks, [x for y in ys for x in y], pt, pool, n_pages)
        lg = ctx.recg_step(batch)
        g = ctx.recg_verify(batch)                # host results; the library's device buffers keep them too
        ctx.recg_policy_step(dst, nxt)            # entropy_mean / accept_len: the library's own buffers
        ctx.recg_sync()
        want = orc.policy_step(st, g["entropy_mean"], g["accept_len"], [len(y) for y in ys], t["blocks"], t["s_edges"],
                               t["value"], t["cost"], dtype=np.float32)
        assert nxt.cpu().tolist() == want
        if rnd == 2:
            assert int(g["accept_len"][0]) == 3 and st["full"][0] == 1
        tb0 = 0
        ver_off = np.concatenate([[0], np.cumsum([len(y) for y in ys])])
        for i in range(C):
            a = int(g["accept_len"][i])
            outs[i] += g["emitted"][ver_off[i]:][: a + 1].tolist()
            nd = g["next_draft"][tb0: tb0 + blocks[i]].tolist()
            tb0 += blocks[i]
            bonus = outs[i][-1]
            Ls[i] = int(g["new_ctx_len"][i])
            ys[i] = [bonus] + nd[1:] if int(g["cont_hit"][i]) else [bonus]
        blocks = nxt.cpu().tolist()
        picked.append(list(blocks))
    for i in range(C):
        assert outs[i] == ars[i][: len(outs[i])]
    assert all(b in (4, 8, 16) for row in picked for b in row)
    ctx.recg_free()
