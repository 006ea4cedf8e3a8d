"""GPU parity of the standalone operations (attention, verify, projection, KV import/export) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import recg_oracle as orc
from paper_2609_34388_b200 import binding, synth
from tests._util import f64

pytestmark = pytest.mark.gpu


def ops_ctx(shape, max_req, max_tok, max_pages, flags=0):
    shape = synth.ModelShape(**{**shape.as_dict(), "n_layers": 1})
    return binding.Context(binding.make_config(shape, max_req, max_tok, max_pages, flags))


def run_attention_case(shape, reqs, seed, layer=0, poison=True):
    """reqs: list of (L, v, b).  Returns (max abs err / max |ref|, per-request refs)."""
    L = [r[0] for r in reqs]
    v = [r[1] for r in reqs]
    b = [r[2] for r in reqs]
    desc = synth.fixed_descriptor(L, v, b, seed=seed)
    T = desc.n_tokens
    ctx = ops_ctx(shape, len(reqs), max(T, 1), desc.page_table.shape[1])
    pool = binding.alloc_kv_pool(ctx, desc.n_pages, fill=None)
    if poison:
        pool.fill_(float("nan"))       # unwritten and invisible slots must never reach the output
    q = synth.queries(T, shape.n_q_heads, shape.head_dim, seed=seed + 5)
    ks, vs = [], []
    for r in range(len(reqs)):
        n = L[r] + v[r] + b[r]
        k_, v_ = synth.kv_values(n, shape.n_kv_heads, shape.head_dim, seed=seed * 100 + r)
        ks.append(k_)
        vs.append(v_)
        ctx.recg_kv_write(pool, desc.n_pages, layer, desc.page_table[r], 0, k_.cuda(), v_.cuda())
    batch = binding.Batch(desc.ctx_len, desc.verify_len, desc.block_size, None, desc.page_table, pool, desc.n_pages)
    o = torch.full((T, shape.n_q_heads, shape.head_dim), float("nan"), dtype=torch.bfloat16, device="cuda")
    ctx.recg_attention(batch, layer, q.cuda(), o)
    ctx.recg_sync()
    got = f64(o)
    worst = 0.0
    t0 = 0
    for r in range(len(reqs)):
        n = v[r] + b[r]
        ref = orc.hybrid_attention(f64(q[t0:t0 + n]), f64(ks[r]), f64(vs[r]), L[r], v[r], b[r])
        assert not np.isnan(got[t0:t0 + n]).any(), f"NaN in request {r}"
        worst = max(worst, np.max(np.abs(got[t0:t0 + n] - ref)) / np.max(np.abs(ref)))
        t0 += n
    # KV round trip through the pool layout
    k_back, v_back = ctx.recg_kv_read(pool, desc.n_pages, layer, desc.page_table[0], 0, L[0] + v[0] + b[0])
    assert torch.equal(k_back.cpu(), ks[0]) and torch.equal(v_back.cpu(), vs[0])
    ctx.recg_free()
    return worst


ATTN_TOL = 1e-2   # relative to max |ref| (attention outputs within 1e-2 relative)


@pytest.mark.parametrize("reqs", [
    [(0, 1, 0)], [(0, 0, 1)], [(1, 1, 1)], [(15, 1, 0)], [(16, 2, 2)], [(17, 3, 8)], [(33, 8, 8)],
    [(63, 1, 1)], [(64, 1, 0)], [(65, 0, 8)], [(200, 16, 16)], [(130, 5, 0)],
    [(100, 4, 4), (7, 1, 8), (300, 16, 16), (64, 2, 2), (0, 8, 8)],
])
def test_attention_small(reqs):
    for shape in (synth.tiny_shape(), synth.llama8b_shape(1)):
        assert run_attention_case(shape, reqs, seed=11) < ATTN_TOL


def test_attention_long_context_split_and_multi_tile():
    shape = synth.llama8b_shape(1)
    # 8B-class op: context 4096, 16 causal + 16 bidirectional rows (split over many KV ranges)
    assert run_attention_case(shape, [(4096, 16, 16)], seed=21) < ATTN_TOL
    # more rows than one tile (64 tokens x 4 heads = 256 rows) and a ragged tail
    assert run_attention_case(shape, [(1000, 33, 31), (5, 40, 0)], seed=22) < ATTN_TOL
    # many short requests next to a long one
    assert run_attention_case(shape, [(3000, 2, 2)] + [(50 + 37 * i, 2, 2) for i in range(20)], seed=23) < ATTN_TOL
    assert run_attention_case(synth.tiny_shape(), [(2500, 40, 30), (100, 70, 0)], seed=24) < ATTN_TOL


def test_attention_many_row_tiles_per_request():
    """Prefill-like chunks: many row tiles per request head (sibling pairs plus a tile without a sibling), next to
    ordinary requests, so that both lines of the work list and several items per CTA occur."""
    shape = synth.llama8b_shape(1)
    assert run_attention_case(shape, [(300, 200, 0), (700, 8, 8), (0, 95, 1)], seed=41) < ATTN_TOL
    assert run_attention_case(shape, [(64, 33, 0)] * 3 + [(2000, 16, 16)], seed=42) < ATTN_TOL
    assert run_attention_case(synth.tiny_shape(), [(100, 130, 0), (10, 3, 4)], seed=43) < ATTN_TOL


def test_attention_high_concurrency_mix():
    """128 requests with the high-concurrency block mix {2,4,8,16} @ (.4,.3,.2,.1): about a thousand small tiles."""
    shape = synth.llama8b_shape(1)
    desc = synth.batch_descriptor(128, [2, 4, 8, 16], [0.4, 0.3, 0.2, 0.1], 40, 700, seed=31)
    reqs = list(zip(desc.ctx_len.tolist(), desc.verify_len.tolist(), desc.block_size.tolist()))
    assert run_attention_case(shape, reqs, seed=32) < ATTN_TOL


@pytest.mark.parametrize("flags", [0, binding.FLAG_SIMT_ATTENTION])
def test_attention_five_query_heads_per_kv_head(flags):
    """40 query / 8 kv heads: a row tile is 25 tokens x 5 heads = 125 of the 128 rows."""
    shape = synth.dense14b_shape(1)
    L = [300, 77, 1500, 0, 40]
    v = [25, 26, 50, 3, 1]
    b = [25, 24, 14, 2, 8]
    desc = synth.fixed_descriptor(L, v, b, seed=31)
    T = desc.n_tokens
    ctx = ops_ctx(shape, len(L), T, desc.page_table.shape[1], flags)
    pool = binding.alloc_kv_pool(ctx, desc.n_pages, fill=None)
    pool.fill_(float("nan"))
    q = synth.queries(T, shape.n_q_heads, shape.head_dim, seed=36)
    ks, vs = [], []
    for r in range(len(L)):
        k_, v_ = synth.kv_values(L[r] + v[r] + b[r], shape.n_kv_heads, shape.head_dim, seed=3100 + r)
        ks.append(k_)
        vs.append(v_)
        ctx.recg_kv_write(pool, desc.n_pages, 0, desc.page_table[r], 0, k_.cuda(), v_.cuda())
    batch = binding.Batch(desc.ctx_len, desc.verify_len, desc.block_size, None, desc.page_table, pool, desc.n_pages)
    o = torch.full((T, shape.n_q_heads, shape.head_dim), float("nan"), dtype=torch.bfloat16, device="cuda")
    ctx.recg_attention(batch, 0, q.cuda(), o)
    ctx.recg_sync()
    got = f64(o)
    t0 = 0
    for r in range(len(L)):
        n = v[r] + b[r]
        ref = orc.hybrid_attention(f64(q[t0:t0 + n]), f64(ks[r]), f64(vs[r]), L[r], v[r], b[r])
        assert not np.isnan(got[t0:t0 + n]).any(), f"NaN in request {r}"
        assert np.max(np.abs(got[t0:t0 + n] - ref)) / np.max(np.abs(ref)) < ATTN_TOL, r
        t0 += n
    ctx.recg_free()


def test_attention_is_deterministic():
    shape = synth.llama8b_shape(1)
    desc = synth.fixed_descriptor([1500, 40], [8, 4], [8, 4], seed=3)
    ctx = ops_ctx(shape, 2, 32, desc.page_table.shape[1])
    pool = binding.alloc_kv_pool(ctx, desc.n_pages, fill="normal")
    batch = binding.Batch(desc.ctx_len, desc.verify_len, desc.block_size, None, desc.page_table, pool, desc.n_pages)
    q = synth.queries(desc.n_tokens, 32, 128, seed=1).cuda()
    o1, o2 = torch.empty_like(q), torch.empty_like(q)
    ctx.recg_attention(batch, 0, q, o1)
    ctx.recg_attention(None, 0, q, o2)      # reuse of the laid-out batch
    ctx.recg_sync()
    assert torch.equal(o1, o2)
    ctx.recg_free()


# ---------------------------------------------------------------- verification
def run_verify_case(B, k, vocab, dtype, seed, sample=None):
    shape = synth.ModelShape(n_layers=0, hidden=64, n_q_heads=4, n_kv_heads=2, head_dim=64, ffn=64, vocab=vocab)
    R = B * (k + 1)
    ctx = binding.Context(binding.make_config(shape, B, R, 1))
    lg = synth.logits_normal(R, vocab, seed=seed, device="cuda", dtype=dtype)
    lg_host = lg.cpu()
    am = np.empty(R, dtype=np.int64)
    for r0 in range(0, R, 256):          # planted drafts need each row's selected id: lowest index of the max
        am[r0:r0 + 256] = lg_host[r0:r0 + 256].double().numpy().argmax(axis=1)
    acc = synth.planted_accept_lengths(B, k, 0.25, seed=seed + 1)
    if B >= 2:
        acc[0], acc[1] = 0, k
    y = synth.plant_drafts(am, B, k, acc, vocab, seed=seed + 2)
    batch = binding.Batch([0] * B, [k + 1] * B, [0] * B, y.reshape(-1))
    got = ctx.recg_verify(batch, lg)
    ctx.recg_sync()
    # by construction
    assert got["accept_len"].tolist() == acc.tolist()
    assert got["n_emitted"].tolist() == (acc + 1).tolist()
    assert got["top1"].tolist() == am.tolist()
    # against the oracle, on all or on sampled requests
    reqs = range(B) if sample is None else sorted(set(np.random.default_rng(seed).integers(0, B, sample).tolist()) | {0, B - 1})
    for r in reqs:
        rows = slice(r * (k + 1), (r + 1) * (k + 1))
        ref = orc.verify_round(lg_host[rows].double().numpy(), y[r].tolist(), 0)
        assert int(got["accept_len"][r]) == ref["accept_len"]
        em = got["emitted"][rows]
        assert em[: ref["n_emitted"]].tolist() == ref["emitted"] and (em[ref["n_emitted"]:] == -1).all()
        assert int(got["new_ctx_len"][r]) == ref["accept_len"] + 1 and int(got["cont_hit"][r]) == 0
        st = ref["stats"]
        assert got["top1"][rows].tolist() == [s["top1"] for s in st]
        assert got["top2"][rows].tolist() == [s["top2"] for s in st]
        np.testing.assert_allclose(got["p1"][rows], [s["p1"] for s in st], rtol=2e-4, atol=1e-7)
        np.testing.assert_allclose(got["p2"][rows], [s["p2"] for s in st], rtol=2e-4, atol=1e-7)
        np.testing.assert_allclose(got["entropy"][rows], [s["entropy"] for s in st], rtol=2e-4, atol=1e-5)
        assert abs(float(got["entropy_mean"][r]) - ref["entropy_mean"]) < 2e-4 * max(1.0, ref["entropy_mean"])
    ctx.recg_free()


@pytest.mark.parametrize("B,k", [(1, 4), (8, 8), (32, 4), (3, 32), (32, 16)])
def test_verify_sweep_bf16(B, k):
    run_verify_case(B, k, 128256, torch.bfloat16, seed=40 + B + k)


def test_verify_fp32_and_odd_vocab():
    run_verify_case(4, 4, 128256, torch.float32, seed=7)
    run_verify_case(5, 3, 2048, torch.bfloat16, seed=8)
    run_verify_case(2, 2, 1000 * 16, torch.float32, seed=9)


def test_verify_full_size_sampled():
    # largest sweep point: 256 requests x 33 rows x 128256 logits (2.17 GB); oracle on sampled requests
    run_verify_case(256, 32, 128256, torch.bfloat16, seed=99, sample=6)


def test_verify_closed_forms_and_ties():
    V = 4096
    shape = synth.ModelShape(n_layers=0, hidden=64, n_q_heads=4, n_kv_heads=2, head_dim=64, ffn=64, vocab=V)
    ctx = binding.Context(binding.make_config(shape, 4, 16, 1))
    lg = torch.zeros((4, V), dtype=torch.float32)
    lg[0] = 1.5                                   # uniform
    lg[1, 777] = 60.0                             # dominant
    lg[2, 100] = lg[2, 3000] = 2.0                # two equal maxima
    lg[3] = torch.linspace(-3, 3, V)
    lg[3, 5] = lg[3, -1]                          # tie between index 5 and the last index
    lg[3, 100:3000] = float("-inf")               # banned ids contribute nothing and poison nothing
    batch = binding.Batch([0], [1], [3], [0])
    got = ctx.recg_verify(batch, lg.cuda())
    assert got["top1"].tolist() == [0, 777, 100, 5] and got["top2"].tolist() == [1, 0, 3000, V - 1]
    assert abs(got["p1"][0] - 1.0 / V) < 1e-9 and abs(got["entropy"][0] - np.log(V)) < 1e-4
    assert abs(got["p1"][1] - 1.0) < 5e-6 and abs(got["entropy"][1]) < 1e-4    # fp32 rounding of x log2(e) at x = 60
    assert got["p1"][2] == got["p2"][2]
    ref3 = orc.row_stats(lg[3].double().numpy())
    assert abs(got["p1"][3] - ref3["p1"]) < 1e-6 and abs(got["entropy"][3] - ref3["entropy"]) < 1e-4
    assert got["next_draft"].tolist() == [777, 100, 5] and got["accept_len"].tolist() == [0]
    ctx.recg_free()


def test_verify_commit_indices_and_continuation():
    """Ragged batch with a page table: slot states, freed pages, continuation rule, v = 0 and b = 0 requests."""
    V = 2048
    shape = synth.ModelShape(n_layers=0, hidden=64, n_q_heads=4, n_kv_heads=2, head_dim=64, ffn=64, vocab=V)
    L, v, b = [31, 5, 40, 16], [8, 0, 3, 1], [8, 4, 0, 15]
    desc = synth.fixed_descriptor(L, v, b, seed=5)
    T = desc.n_tokens
    ctx = binding.Context(binding.make_config(shape, 4, T, desc.page_table.shape[1]))
    lg = synth.logits_normal(T, V, seed=3, dtype=torch.float32)
    am = lg.double().numpy().argmax(axis=1)
    # request 0: accept 3 of 7 drafts; request 2: all accepted; request 3: v = 1 and the first draft row repeats the bonus
    y0 = [9] + am[0:3].tolist() + [(int(am[3]) + 1) % V, 1, 2, 3]
    y2 = [4] + am[20:22].tolist()
    lg[24] = lg[23]                                  # request 3: row 23 verify, row 24 first draft row
    y = y0 + y2 + [11]
    batch = binding.Batch(L, v, b, y, desc.page_table, None, 0)
    got = ctx.recg_verify(batch, lg.cuda())
    ref = orc.verify_batch(lg.double().numpy(), v, b, y)
    t0 = 0
    for r in range(4):
        rr = ref[r]
        assert int(got["accept_len"][r]) == rr["accept_len"] and int(got["cont_hit"][r]) == int(rr["cont_hit"])
        kc = orc.kv_commit(L[r], v[r], b[r], rr["accept_len"], desc.page_table[r], 16)
        assert int(got["new_ctx_len"][r]) == kc["new_ctx_len"] and int(got["freed_pages"][r]) == len(kc["freed_pages"])
        ss = got["slot_state"][t0:t0 + v[r] + b[r]].tolist()
        assert [s for s in ss if s >= 0] == kc["commit_slots"]
        assert [-(s + 1) for s in ss if s < 0] == kc["rollback_slots"]
        t0 += v[r] + b[r]
    assert got["accept_len"].tolist() == [3, 0, 2, 0] and got["cont_hit"].tolist() == [0, 0, 0, 1]
    nd = [d for r in ref for d in r["next_draft"]]
    assert got["next_draft"].tolist() == nd
    ctx.recg_free()


# ---------------------------------------------------------------- projection
@pytest.mark.parametrize("flags", [0, binding.FLAG_SIMT_GEMM])
@pytest.mark.parametrize("M,N,K", [(1, 128, 64), (31, 256, 256), (128, 512, 1024), (129, 6144, 4096), (300, 4096, 14336),
                                   (77, 2048, 256), (515, 1024, 4096), (32, 4096, 4096), (32, 4096, 14336),
                                   (470, 4096, 14336), (16, 6144, 4096), (130, 128256, 4096)])
def test_linear(M, N, K, flags):
    shape = synth.tiny_shape()
    ctx = ops_ctx(shape, 1, 8, 1, flags)
    g = torch.Generator().manual_seed(M * 7 + N)
    x = torch.randn((M, K), generator=g).to(torch.bfloat16)
    w = (torch.randn((N, K), generator=g) * 0.05).to(torch.bfloat16)
    ref = x.double().numpy() @ w.double().numpy().T
    y = ctx.recg_linear(x.cuda(), w.cuda(), torch.float32)
    ctx.recg_sync()
    err = np.max(np.abs(f64(y) - ref)) / np.max(np.abs(ref))
    assert err < 1e-4, err      # fp32 accumulation of exact bf16 products: ~sqrt(K) 2^-24 relative, K <= 14336
    yb = ctx.recg_linear(x.cuda(), w.cuda(), torch.bfloat16)
    assert np.max(np.abs(f64(yb) - ref)) / np.max(np.abs(ref)) < 5e-3
    y2 = ctx.recg_linear(x.cuda(), w.cuda(), torch.float32)      # K-split partials are reduced in a fixed order
    assert torch.equal(y, y2)
    ctx.recg_free()


def test_linear_random_shapes():
    """Seeded sweep over row counts, widths that are not multiples of the tile widths (N % 16 == 0 only) and depths:
    every tile decomposition the scheduler can pick, the clipped right edge and the clipped last rows, both output
    types.  The output buffer is poisoned and padded so that a store beyond the matrix would show."""
    rng = np.random.default_rng(77)
    shape = synth.tiny_shape()
    ctx = ops_ctx(shape, 1, 8, 1)
    for case in range(48):
        M = int(rng.choice([1, 2, 15, 17, 31, 32, 33, 63, 64, 65, 100, 127, 128, 129, 200, 255, 257, 376, 400, 480, 513, 700]))
        N = 16 * int(rng.integers(1, 80)) if case % 3 else 16 * int(rng.integers(80, 700))
        K = 64 * int(rng.integers(1, 24))
        out_dtype = torch.bfloat16 if case % 2 else torch.float32
        g = torch.Generator().manual_seed(1000 + case)
        x = torch.randn((M, K), generator=g).to(torch.bfloat16)
        w = (torch.randn((N, K), generator=g) * 0.05).to(torch.bfloat16)
        ref = x.double().numpy() @ w.double().numpy().T
        buf = torch.full((M + 2, N), float("nan"), dtype=out_dtype, device="cuda")   # two guard rows behind the matrix
        xd, wd = x.cuda(), w.cuda()
        ctx._check(binding.lib().recg_linear(ctx.h, xd.data_ptr(), wd.data_ptr(), buf.data_ptr(), M, N, K,
                                             binding.DTYPE_BF16 if out_dtype == torch.bfloat16 else binding.DTYPE_F32))
        ctx.recg_sync()
        got = f64(buf[:M])
        assert not np.isnan(got).any(), (M, N, K)
        assert torch.isnan(buf[M:].float()).all(), f"stored beyond the last row: {(M, N, K)}"
        tol = 1e-4 if out_dtype == torch.float32 else 5e-3       # bf16 output: half an ulp is 2^-9
        assert np.max(np.abs(got - ref)) / np.max(np.abs(ref)) < tol, (M, N, K, str(out_dtype))
    ctx.recg_free()


@pytest.mark.parametrize("force", ["512,0", "512,1", "384,0", "384,1", "256,1", "128,1", "64,1", "256,0"])
def test_linear_forced_decompositions(force):
    """Every tile width and decomposition of the projection kernel on shapes that make it cut tiles: CTA pairs
    (512 = 256-row tiles over clusters of two), stream-K with the reduction through the idle operand ring (last
    pieces) and through global memory (pieces followed by whole tiles), ragged M, M beyond one pair tile."""
    shape = synth.tiny_shape()
    ctx = ops_ctx(shape, 1, 8, 1)
    tile, sk = (int(t) for t in force.split(","))
    ctx.recg_debug_gemm_config(tile, sk)
    for (M, N, K) in [(300, 512, 1024), (130, 4096, 4096), (470, 1024, 14336), (600, 6144, 1024), (257, 28672, 512)]:
        g = torch.Generator().manual_seed(M * 7 + N)
        x = torch.randn((M, K), generator=g).to(torch.bfloat16)
        w = (torch.randn((N, K), generator=g) * 0.05).to(torch.bfloat16)
        ref = x.double().numpy() @ w.double().numpy().T
        y = ctx.recg_linear(x.cuda(), w.cuda(), torch.float32)
        ctx.recg_sync()
        err = np.max(np.abs(f64(y) - ref)) / np.max(np.abs(ref))
        assert err < 1e-4, (force, M, N, K, err)
        y2 = ctx.recg_linear(x.cuda(), w.cuda(), torch.float32)
        ctx.recg_sync()
        assert torch.equal(y, y2), (force, M, N, K)        # parts are added in a fixed order
    ctx.recg_free()


LLAMA8B_PROJECTIONS = {"qkv": (6144, 4096), "o": (4096, 4096), "gate_up": (28672, 4096), "down": (4096, 14336),
                       "lm_head": (128256, 4096)}


@pytest.mark.parametrize("name", list(LLAMA8B_PROJECTIONS))
def test_linear_at_the_row_counts_the_bench_times(name):
    """The five 8B-class projection shapes at the row counts of the concurrency-128 step, the concurrency sweep and the
    forward-time sweep (1331, 2000, 3792, 8192 rows: 6 to 64 row tiles, every decomposition the cost model picks
    there) and with every forced tile configuration at 1331 and 3792 rows.  The product is too large for a full float64
    reference, so 256 sampled output columns (the first and last 32 and 192 drawn at random) are compared with a
    float64 matmul of the same bf16 values; the whole output starts as NaN, so an unwritten tile shows anywhere, two
    guard rows behind the matrix must stay NaN, and a second run must give the same bits."""
    N, K = LLAMA8B_PROJECTIONS[name]
    shape = synth.tiny_shape()
    ctx = ops_ctx(shape, 1, 8, 1)
    g = torch.Generator(device="cuda").manual_seed(N + K)
    w = (torch.randn((N, K), generator=g, device="cuda") * 0.05).to(torch.bfloat16)
    rng = np.random.default_rng(N)
    cols = np.unique(np.concatenate([np.arange(32), np.arange(N - 32, N), rng.integers(32, N - 32, 192)]))
    w_ref = f64(w[torch.from_numpy(cols).cuda()])
    for M in (1331, 2000, 3792, 8192):
        x = torch.randn((M, K), generator=g, device="cuda").to(torch.bfloat16)
        ref = f64(x) @ w_ref.T
        scale = np.max(np.abs(ref))
        configs = [(0, False)]
        if M in (1331, 3792):
            configs += [(t, sk) for t in (64, 128, 256, 384, 512) for sk in (False, True)]
        for tile, sk in configs:
            if name == "lm_head" and tile in (64, 128) and M > 1331:
                continue            # (narrow tiles on the widest matrix: tens of thousands of tiles, nothing new)
            ctx.recg_debug_gemm_config(tile, sk)
            outs = []
            for rep in range(2):
                buf = torch.full((M + 2, N), float("nan"), dtype=torch.float32, device="cuda")
                ctx._check(binding.lib().recg_linear(ctx.h, x.data_ptr(), w.data_ptr(), buf.data_ptr(), M, N, K,
                                                     binding.DTYPE_F32))
                ctx.recg_sync()
                outs.append(buf)
            buf = outs[0]
            assert not torch.isnan(buf[:M]).any(), f"unwritten output: {(name, M, tile, sk)}"
            assert torch.isnan(buf[M:]).all(), f"stored beyond the last row: {(name, M, tile, sk)}"
            err = np.max(np.abs(f64(buf[:M][:, torch.from_numpy(cols).cuda()]) - ref)) / scale
            assert err < 1e-4, (name, M, tile, sk, err)
            assert torch.equal(outs[0][:M], outs[1][:M]), f"not deterministic: {(name, M, tile, sk)}"
            del outs, buf
    ctx.recg_free()


@pytest.mark.parametrize("name", ["qkv", "o", "down"])
def test_linear_thin_rows_hand_over_inside_clusters(name):
    """Problems of one row tile (at most 128 rows) whose tiles are cut over K: the CTAs that share a tile form a cluster and
    hand their partial tiles to the cluster's leader through distributed shared memory.  The 8B-class shapes at 1, 7, 32,
    33, 66, 100 and 128 rows,
    with the cost model's choice and with forced tile widths (which give clusters of 2 to 4), against a float64 product
    of the same bf16 values; the same launches with the hand-over through the partial-tile workspace (stream_k = 2) must
    agree with it as closely; reruns give the same bits; rows behind the last one stay untouched."""
    N, K = LLAMA8B_PROJECTIONS[name]
    shape = synth.tiny_shape()
    ctx = ops_ctx(shape, 1, 8, 1)
    g = torch.Generator(device="cuda").manual_seed(N + K + 1)
    w = (torch.randn((N, K), generator=g, device="cuda") * 0.05).to(torch.bfloat16)
    w64 = f64(w)
    for M in (1, 7, 32, 33, 66, 100, 128):
        x = torch.randn((M, K), generator=g, device="cuda").to(torch.bfloat16)
        ref = f64(x) @ w64.T
        scale = np.max(np.abs(ref))
        got = {}
        for tile, sk in [(0, 1), (0, 2), (64, 1), (64, 2), (128, 1), (128, 2), (256, 1)]:
            ctx.recg_debug_gemm_config(tile, sk)
            outs = []
            for rep in range(2):
                buf = torch.full((M + 2, N), float("nan"), dtype=torch.float32, device="cuda")
                ctx._check(binding.lib().recg_linear(ctx.h, x.data_ptr(), w.data_ptr(), buf.data_ptr(), M, N, K,
                                                     binding.DTYPE_F32))
                ctx.recg_sync()
                outs.append(buf)
            assert not torch.isnan(outs[0][:M]).any(), f"unwritten output: {(name, M, tile, sk)}"
            assert torch.isnan(outs[0][M:]).all(), f"stored beyond the last row: {(name, M, tile, sk)}"
            err = np.max(np.abs(f64(outs[0][:M]) - ref)) / scale
            assert err < 1e-4, (name, M, tile, sk, err)
            assert torch.equal(outs[0][:M], outs[1][:M]), f"not deterministic: {(name, M, tile, sk)}"
            got[(tile, sk)] = outs[0][:M].clone()
        # same tiles, other hand-over: the K ranges of the parts differ, so the sums differ in rounding only
        for tile in (0, 64, 128):
            d = float((got[(tile, 1)] - got[(tile, 2)]).abs().max()) / scale
            assert d < 1e-5, (name, M, tile, d)
    ctx.recg_free()


def test_bounded_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    """A kernel whose wait can never be satisfied gives up after its poll limit, returns and leaves the timeout in the
    status word: recg_sync reports RECG_ERR_TIMEOUT once, and the same context then computes a correct product
    (stream-K decomposition, whose arrival counters are reset after an error)."""
    shape = synth.tiny_shape()
    ctx = ops_ctx(shape, 1, 8, 1)
    ctx.recg_debug_wait_timeout(2000)
    with pytest.raises(binding.RecgError) as e:
        ctx.recg_sync()
    assert e.value.status == 5 and "gave up" in str(e.value)
    ctx.recg_sync()                                   # the status word was cleared
    ctx.recg_debug_gemm_config(256, True)
    g = torch.Generator().manual_seed(3)
    x = torch.randn((300, 1024), generator=g).to(torch.bfloat16)
    w = (torch.randn((512, 1024), generator=g) * 0.05).to(torch.bfloat16)
    y = ctx.recg_linear(x.cuda(), w.cuda(), torch.float32)
    ctx.recg_sync()
    ref = x.double().numpy() @ w.double().numpy().T
    assert np.max(np.abs(f64(y) - ref)) / np.max(np.abs(ref)) < 1e-4
    ctx.recg_free()


def test_debug_checks_guard_bands_and_page_ownership():
    """RECG_FLAG_DEBUG_CHECKS: a normal call passes; a write just past the end of a workspace region (done here
    through the address recg_debug_buffer hands out, inside the library's own allocation) is reported by the next
    recg_sync as RECG_ERR_INTERNAL, once; a page that receives new rows of two requests is refused on the host."""
    shape = synth.tiny_shape()
    W = synth.model_weights(shape, seed=0, dtype=torch.bfloat16)
    Wd = {k: ([t.cuda() for t in v] if isinstance(v, list) else v.cuda()) for k, v in W.items()}
    max_tok = 32
    ctx = binding.Context(binding.make_config(shape, 4, max_tok, 8, binding.FLAG_DEBUG_CHECKS), Wd)
    pool = binding.alloc_kv_pool(ctx, 32)
    pt = np.arange(16, dtype=np.int32).reshape(2, 8)
    batch = binding.Batch([20, 5], [2, 1], [4, 4], [1, 2, 3], pt, pool, 32)
    ctx.recg_step(batch)
    ctx.recg_verify(batch)
    ctx.recg_sync()
    # the rotated queries are [max_tokens, n_q * d] bf16; the guard band follows the region (256-byte aligned)
    import ctypes as C
    p, dt, r, c = C.c_void_p(), C.c_int32(), C.c_int32(), C.c_int32()
    ctx._check(binding.lib().recg_debug_buffer(ctx.h, 2, C.byref(p), C.byref(dt), C.byref(r), C.byref(c)))
    region = max_tok * shape.n_q_heads * shape.head_dim * 2
    band = binding.device_view(p.value + (region + 255) // 256 * 256, (64,), torch.float32)
    saved = band.clone()
    band[3] = 1.0
    with pytest.raises(binding.RecgError) as e:
        ctx.recg_sync()
    assert e.value.status == 6 and "guard band" in str(e.value)
    ctx.recg_sync()                                   # reported once; the bands were refilled
    assert torch.equal(band, saved)
    shared = pt.copy()
    shared[1, 0] = pt[0, 1]                           # request 1's first new page is request 0's page of new rows
    with pytest.raises(binding.RecgError) as e:
        ctx.recg_step(binding.Batch([20, 5], [2, 1], [4, 4], [1, 2, 3], shared, pool, 32))
    assert e.value.status == 1 and "named twice" in str(e.value)
    ctx.recg_free()


def test_host_side_rejections():
    shape = synth.tiny_shape()
    ctx = ops_ctx(shape, 2, 16, 4)
    lg = torch.zeros((4, shape.vocab), dtype=torch.float32, device="cuda")
    with pytest.raises(binding.RecgError) as e:
        ctx.recg_verify(binding.Batch([0, 0, 0], [1, 1, 1], [0, 0, 0], [0, 0, 0]), lg)     # too many requests
    assert e.value.status == 3
    with pytest.raises(binding.RecgError) as e:
        ctx.recg_verify(binding.Batch([0], [20], [0], [0] * 20), lg)                        # too many tokens
    assert e.value.status == 3
    with pytest.raises(binding.RecgError) as e:
        ctx.recg_verify(binding.Batch([0], [0], [0], None), lg)                             # a request without rows
    assert e.value.status == 1
    with pytest.raises(binding.RecgError) as e:
        ctx.recg_verify(binding.Batch([-1], [1], [0], [0]), lg)
    assert e.value.status == 1
    pool = torch.zeros(ctx.kv_pool_bytes(4) // 2, dtype=torch.bfloat16, device="cuda")
    q = torch.zeros((4, 4, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.RecgError) as e:      # page table too short for L + v + b = 100 tokens
        ctx.recg_attention(binding.Batch([96], [2], [2], None, np.zeros((1, 4), np.int32), pool, 4), 0, q, q.clone())
    assert e.value.status == 3
    with pytest.raises(binding.RecgError) as e:      # page id outside the pool
        ctx.recg_attention(binding.Batch([10], [2], [2], None, np.full((1, 4), 9, np.int32), pool, 4), 0, q, q.clone())
    assert e.value.status == 1
    with pytest.raises(binding.RecgError) as e:      # step on a context without weights
        ctx.recg_step(binding.Batch([10], [2], [2], [1, 2], np.zeros((1, 4), np.int32), pool, 4))
    assert e.value.status == 1
    ctx.recg_sync()
    ctx.recg_free()
