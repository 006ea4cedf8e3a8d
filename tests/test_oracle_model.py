"""Pins for the oracle's backbone and round loop: an independent library decoder, losslessness
against token-by-token greedy decoding, cached == dense, and the reductions to textbook cases."""
import math

import numpy as np
import pytest
import torch

from oracle import recg_oracle as orc
from paper_2609_34388_b200 import synth
from tests._util import bf16_round, oracle_cfg, oracle_rounds_together, oracle_weights


def small_shape(n_layers=2):
    return synth.ModelShape(n_layers=n_layers, hidden=32, n_q_heads=4, n_kv_heads=2, head_dim=8, ffn=48, vocab=64)


@pytest.fixture(scope="module")
def small():
    shape = small_shape()
    W = synth.model_weights(shape, seed=0, dtype=torch.float32)
    # scale up so that logits separate well and norm gains matter
    for k in ("wqkv", "wo", "w_gate_up", "w_down"):
        W[k] = [w * 8.0 for w in W[k]]
    W["embed"] = W["embed"] * 20.0
    W["lm_head"] = W["lm_head"] * 20.0
    synth.perturb_norm_gains(W)
    return shape, oracle_cfg(shape), oracle_weights(W), W


def hf_model(shape, W):
    from transformers import LlamaConfig, LlamaForCausalLM

    cfg = LlamaConfig(vocab_size=shape.vocab, hidden_size=shape.hidden, intermediate_size=shape.ffn,
                      num_hidden_layers=shape.n_layers, num_attention_heads=shape.n_q_heads,
                      num_key_value_heads=shape.n_kv_heads, head_dim=shape.head_dim, rms_norm_eps=shape.rms_eps,
                      rope_theta=shape.rope_base, attention_bias=False, mlp_bias=False, tie_word_embeddings=False,
                      max_position_embeddings=512, attn_implementation="eager")
    m = LlamaForCausalLM(cfg).to(torch.float64).eval()
    nq, nkv, d, F = shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.ffn
    sd = {"model.embed_tokens.weight": W["embed"], "model.norm.weight": W["final_norm"], "lm_head.weight": W["lm_head"]}
    for l in range(shape.n_layers):
        p = f"model.layers.{l}."
        qkv = W["wqkv"][l]
        sd[p + "self_attn.q_proj.weight"] = qkv[: nq * d]
        sd[p + "self_attn.k_proj.weight"] = qkv[nq * d: (nq + nkv) * d]
        sd[p + "self_attn.v_proj.weight"] = qkv[(nq + nkv) * d:]
        sd[p + "self_attn.o_proj.weight"] = W["wo"][l]
        sd[p + "mlp.gate_proj.weight"] = W["w_gate_up"][l][:F]
        sd[p + "mlp.up_proj.weight"] = W["w_gate_up"][l][F:]
        sd[p + "mlp.down_proj.weight"] = W["w_down"][l]
        sd[p + "input_layernorm.weight"] = W["attn_norm"][l]
        sd[p + "post_attention_layernorm.weight"] = W["ffn_norm"][l]
    missing = m.load_state_dict({k: v.to(torch.float64) for k, v in sd.items()}, strict=False)
    assert not [k for k in missing.missing_keys if "rotary" not in k]
    return m


def test_causal_forward_matches_library_decoder(small):
    """b = 0 is a plain causal LM forward: compare with an independent Llama implementation."""
    shape, cfg, W64, W = small
    m = hf_model(shape, W)
    ids = synth.token_ids(23, shape.vocab, seed=1)
    with torch.no_grad():
        ref = m(input_ids=torch.from_numpy(ids.astype(np.int64))[None]).logits[0].numpy()
    got, _, _ = orc.fused_round_dense(cfg, W64, [], ids.tolist(), 0)
    assert np.max(np.abs(ref - got)) < 1e-5 * np.max(np.abs(ref))     # the library computes rotary angles in fp32


def test_fused_round_matches_library_decoder_with_explicit_mask(small):
    """The hybrid round through the library decoder, given Eq. 1 as an explicit additive mask."""
    shape, cfg, W64, W = small
    m = hf_model(shape, W)
    L, v, b = 11, 4, 5
    ids = synth.token_ids(L + v, shape.vocab, seed=2).tolist()
    full = ids + [cfg.mask_id()] * b
    n = L + v + b
    M = torch.full((n, n), -math.inf, dtype=torch.float64)
    for i in range(n):
        for j in range(n):
            if (i < L + v and j <= i) or (i >= L + v):
                M[i, j] = 0.0
    with torch.no_grad():
        ref = m(input_ids=torch.tensor(full)[None], attention_mask=M[None, None],
                position_ids=torch.arange(n)[None]).logits[0].numpy()
    got, _, _ = orc.fused_round_dense(cfg, W64, ids[:L], ids[L:], b)
    assert np.max(np.abs(ref[L:] - got)) < 1e-5 * np.max(np.abs(ref))


def test_rope_properties():
    rng = np.random.default_rng(0)
    d = 16
    q = rng.standard_normal((1, 1, d))
    k = rng.standard_normal((1, 1, d))
    assert np.allclose(orc.rope(q, np.array([0]), 10000.0), q, atol=0)          # position 0 is the identity
    for p in (1, 17, 400):
        assert abs(np.linalg.norm(orc.rope(q, np.array([p]), 10000.0)) - np.linalg.norm(q)) < 1e-12
    def dot(pq, pk):
        return float(np.sum(orc.rope(q, np.array([pq]), 10000.0) * orc.rope(k, np.array([pk]), 10000.0)))
    assert abs(dot(5, 3) - dot(105, 103)) < 1e-11 and abs(dot(40, 3) - dot(77, 40)) < 1e-11
    assert abs(dot(5, 3) - dot(6, 3)) > 1e-4
    # explicit pair rotation: element i with i + d/2, angle p * base^(-2i/d)
    p, base = 9, 10000.0
    x = q[0, 0]
    r = orc.rope(q, np.array([p]), base)[0, 0]
    for i in range(d // 2):
        th = p * base ** (-2.0 * i / d)
        assert abs(r[i] - (x[i] * math.cos(th) - x[i + d // 2] * math.sin(th))) < 1e-14
        assert abs(r[i + d // 2] - (x[i + d // 2] * math.cos(th) + x[i] * math.sin(th))) < 1e-14


def test_cached_equals_dense(small):
    shape, cfg, W64, _ = small
    L, v, b = 19, 3, 4
    ids = synth.token_ids(L + v, shape.vocab, seed=3).tolist()
    dense_logits, dense_kv, _ = orc.fused_round_dense(cfg, W64, ids[:L], ids[L:], b)
    kv, L0, y0 = orc.prefill(cfg, W64, ids[: L + 1])
    assert L0 == L and y0 == [ids[L]]
    for (K, V), (Kd, Vd) in zip(kv, dense_kv):
        assert np.max(np.abs(K - Kd[:L])) < 1e-12 and np.max(np.abs(V - Vd[:L])) < 1e-12
    cached_logits, cached_kv, _ = orc.fused_round_cached(cfg, W64, kv, L, ids[L:], b)
    assert np.max(np.abs(cached_logits - dense_logits)) < 1e-10
    for (K, V), (Kd, Vd) in zip(cached_kv, dense_kv):
        assert np.max(np.abs(K - Kd)) < 1e-11 and np.max(np.abs(V - Vd)) < 1e-11


def test_rounds_run_together_equal_rounds_run_alone(small):
    """The test helper that sends several requests through orc.decoder_rows at once (block-diagonal visibility over the
    concatenated contexts) gives each request what its own fused_round_cached call gives, also with the rounding hook."""
    shape, cfg, W64, _ = small
    reqs = []
    for i, (L, v, b) in enumerate([(19, 3, 4), (0, 2, 2), (33, 1, 8), (7, 5, 0), (16, 0, 3)]):
        ids = synth.token_ids(L + max(v, 1), shape.vocab, seed=30 + i).tolist()
        kv = orc.prefill(cfg, W64, ids[: L + 1])[0] if L else [(np.zeros((0, 2, 8)), np.zeros((0, 2, 8)))] * cfg.n_layers
        reqs.append({"kv": kv, "L": L, "y": ids[L: L + v], "b": b})
    for hook, tol in ((None, 1e-10), (bf16_round, 0.0)):
        together = oracle_rounds_together(cfg, W64, reqs, hook)
        for r, (lg, hd) in zip(reqs, together):
            alone_lg, _, alone_hd = orc.fused_round_cached(cfg, W64, r["kv"], r["L"], r["y"], r["b"], hook)
            if hook is None:
                assert np.max(np.abs(lg - alone_lg)) < tol and np.max(np.abs(hd - alone_hd)) < tol
            else:
                # with rounding, a last-bit difference of the fp64 sums can flip a bf16 rounding: compare loosely
                assert np.max(np.abs(lg - alone_lg)) < 2e-2 * np.max(np.abs(alone_lg))


def test_rounding_hook_is_applied_at_the_six_storage_points(small):
    """decoder_rows' act_round hook: the identity leaves the result unchanged; a hook that counts its calls is applied
    to the normalised input (twice per layer), q, k, v, the attention output and the SwiGLU output of every layer and
    to the final normalised input; rounding to bf16 moves the logits by about a bf16 ulp, not more."""
    shape, cfg, W64, _ = small
    L, v, b = 12, 3, 4
    ids = synth.token_ids(L + v, shape.vocab, seed=8).tolist()
    kv, _, _ = orc.prefill(cfg, W64, ids[: L + 1])
    base, _, _ = orc.fused_round_cached(cfg, W64, kv, L, ids[L:], b)
    same, _, _ = orc.fused_round_cached(cfg, W64, kv, L, ids[L:], b, lambda a: a)
    assert np.array_equal(base, same)
    shapes = []
    def counting(a):
        shapes.append(a.shape)
        return a
    orc.fused_round_cached(cfg, W64, kv, L, ids[L:], b, counting)
    n = v + b
    per_layer = [(n, shape.hidden), (n, 4, 8), (n, 2, 8), (n, 2, 8), (n, 4, 8), (n, shape.hidden), (n, shape.ffn)]
    assert shapes == per_layer * cfg.n_layers + [(n, shape.hidden)]
    rounded, _, _ = orc.fused_round_cached(cfg, W64, kv, L, ids[L:], b, bf16_round)
    rel = np.max(np.abs(rounded - base)) / np.max(np.abs(base))
    assert 0 < rel < 3e-2


def test_verify_rows_ignore_draft_block(small):
    shape, cfg, W64, _ = small
    L, v = 10, 4
    ids = synth.token_ids(L + v, shape.vocab, seed=4).tolist()
    base, _, _ = orc.fused_round_dense(cfg, W64, ids[:L], ids[L:], 0)
    for b in (1, 8):
        got, _, _ = orc.fused_round_dense(cfg, W64, ids[:L], ids[L:], b)
        assert np.max(np.abs(got[:v] - base)) < 1e-12
    cfg2 = orc.ModelConfig(**{**cfg.__dict__, "mask_token_id": 5})
    got, _, _ = orc.fused_round_dense(cfg2, W64, ids[:L], ids[L:], 8)
    assert np.max(np.abs(got[:v] - base)) < 1e-12


def test_special_cases(small):
    shape, cfg, W64, _ = small
    L, v = 7, 3
    ids = synth.token_ids(L + v, shape.vocab, seed=5).tolist()
    # b = 1: the single mask row sees exactly what a causal row at that position sees
    a, _, _ = orc.fused_round_dense(cfg, W64, ids[:L], ids[L:], 1)
    c, _, _ = orc.fused_round_dense(cfg, W64, ids[:L], ids[L:] + [cfg.mask_id()], 0)
    assert np.max(np.abs(a - c)) < 1e-12
    # L = 0: no cache at all
    d0, _, _ = orc.fused_round_dense(cfg, W64, [], ids, 2)
    d1, _, _ = orc.fused_round_cached(cfg, W64, [(np.zeros((0, 2, 8)), np.zeros((0, 2, 8)))] * cfg.n_layers, 0, ids, 2)
    assert np.max(np.abs(d0 - d1)) < 1e-12
    # v tokens at once == v single-token steps over a growing cache
    kv, L0, _ = orc.prefill(cfg, W64, ids[: L + 1])
    allat, _, _ = orc.fused_round_cached(cfg, W64, kv, L, ids[L:], 0)
    for i in range(v):
        one, kv, _ = orc.fused_round_cached(cfg, W64, kv, L + i, [ids[L + i]], 0)
        assert np.max(np.abs(one[0] - allat[i])) < 1e-10


def test_draft_rows_are_bidirectional(small):
    """Changing a LATER verify token must change... nothing earlier, but every draft row; and draft rows see each other."""
    shape, cfg, W64, _ = small
    L, v, b = 6, 3, 3
    ids = synth.token_ids(L + v, shape.vocab, seed=6).tolist()
    base, _, _ = orc.fused_round_dense(cfg, W64, ids[:L], ids[L:], b)
    ids2 = list(ids)
    ids2[-1] = (ids2[-1] + 1) % (shape.vocab - 1)
    got, _, _ = orc.fused_round_dense(cfg, W64, ids2[:L], ids2[L:], b)
    assert np.max(np.abs(got[: v - 1] - base[: v - 1])) < 1e-12
    assert all(np.max(np.abs(got[r] - base[r])) > 1e-9 for r in range(v - 1, v + b))
    # a draft row with 2 masks differs from the same row with 3 masks (it sees the later mask)
    two, _, _ = orc.fused_round_dense(cfg, W64, ids[:L], ids[L:], 2)
    assert np.max(np.abs(two[v] - base[v])) > 1e-9


@pytest.mark.parametrize("b", [4, 8])
def test_losslessness_self_drafted(small, b):
    shape, cfg, W64, _ = small
    prompt = synth.token_ids(12, shape.vocab, seed=7).tolist()
    out, trace, _ = orc.spec_decode(cfg, W64, prompt, b, rounds=5)
    ar = orc.greedy_ar(cfg, W64, prompt, len(out))
    assert out == ar
    assert all(len(t["emitted"]) == t["accept_len"] + 1 for t in trace)


@pytest.mark.parametrize("m", [0, 1, 3, 6, 7])
def test_losslessness_planted(small, m):
    """Drafts teacher-forced from the greedy continuation with one corrupted token: the accept
    length must equal the corruption index and the output must still be the greedy continuation."""
    shape, cfg, W64, _ = small
    prompt = synth.token_ids(12, shape.vocab, seed=8).tolist()
    v = 8
    ar = orc.greedy_ar(cfg, W64, prompt, 40)

    def plant(t, out, y):
        truth = ar[len(out): len(out) + v - 1]          # tokens after y_0
        y = [y[0]] + truth
        if m + 1 <= v - 1:
            y[m + 1] = (y[m + 1] + 1) % (shape.vocab - 1)
        return y

    out, trace, (kv, L) = orc.spec_decode(cfg, W64, prompt, 8, rounds=3, plant=plant)
    assert out == ar[: len(out)]
    assert [t["accept_len"] for t in trace] == [m, m, m]
    # the committed cache equals a dense recomputation of the committed tokens (rolled-back slots were NaN)
    seq = prompt + out
    _, dense_kv, _ = orc.fused_round_dense(cfg, W64, seq[:L], [], 0) if L else (None, [], None)
    for (K, V), (Kd, Vd) in zip(kv, dense_kv):
        assert np.max(np.abs(K[:L] - Kd)) < 1e-10 and np.max(np.abs(V[:L] - Vd)) < 1e-10
        assert np.isnan(K[L:]).all()


def test_tiny_config_losslessness():
    """The 2-layer / hidden-256 / vocab-2048 model with a 64-token prompt, block 8, 4 rounds."""
    shape = synth.tiny_shape()
    W = synth.model_weights(shape, seed=0, dtype=torch.float32)
    cfg, W64 = oracle_cfg(shape), oracle_weights(W)
    prompt = synth.token_ids(64, shape.vocab, seed=1).tolist()
    out, trace, _ = orc.spec_decode(cfg, W64, prompt, 8, rounds=4)
    assert out == orc.greedy_ar(cfg, W64, prompt, len(out))
