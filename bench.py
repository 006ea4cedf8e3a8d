"""Benchmark of the fused draft+verify step (one round = recg_step + recg_verify) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Workload (config.workload): the full 32-layer 8B-class random-init backbone at concurrency 16, per-request
block sizes drawn from {4, 8, 16, 32}, verify length equal to the block size, context lengths uniform in
[512, 8192], synthetic token ids, KV pool filled with N(0, 1).  `value` is processed tokens/s (all verify
and mask rows of the batch per step) with everything resident in HBM; `e2e` runs the same calls with host
descriptor arrays copied in and the verification results copied out every step.  Extra keys report the
standalone attention operation at the 8B low-concurrency shape, the verify sweep, per-kernel-class
rooflines and the concurrency-1 point.  With N > 1 every rank runs its own batch of the same shape
(requests are independent: no collective on the data path) and rank 0 prints the aggregate.
"""
import argparse
import json
import os
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2609_34388_b200 import synth  # noqa: E402
from paper_2609_34388_b200.dist import DistEnv  # noqa: E402

METRIC = "draft+verify step processed tokens/s (fused round over a ragged batch, 8B-class backbone)"
UNIT = "tokens/s"


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"], "bf16_tflops_sustained": d["bf16_tflops_sustained"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index=0, period=0.01):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            pass

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {nv.nvmlClocksThrottleReasonHwSlowdown: "hw_slowdown",
                 nv.nvmlClocksThrottleReasonHwThermalSlowdown: "hw_thermal_slowdown",
                 nv.nvmlClocksThrottleReasonSwThermalSlowdown: "sw_thermal_slowdown",
                 nv.nvmlClocksThrottleReasonSwPowerCap: "sw_power_cap"}
        while not self._stop_evt.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        med = int(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ------------------------------------------------------------------------------------------------
# workload construction
# ------------------------------------------------------------------------------------------------
def c16_descriptor(seed):
    return synth.batch_descriptor(16, [4, 8, 16, 32], None, 512, 8192, seed=seed)


def c128_descriptor(seed, ctx_scale=1.0):
    """configs[3]: concurrency 128, blocks {2,4,8,16} @ (.4,.3,.2,.1), context lengths U[1024,16384] x ctx_scale.  At
    full length the KV pool alone is about 146 GB; bench_c128 takes ctx_scale = 1 when the device has room for it
    beside weights and workspace and 0.5 otherwise, and says which in its result."""
    return synth.batch_descriptor(128, [2, 4, 8, 16], [0.4, 0.3, 0.2, 0.1], int(1024 * ctx_scale), int(16384 * ctx_scale),
                                  seed=seed)


def c1_descriptor(seed):
    return synth.fixed_descriptor([4096], [16], [16], seed=seed)


def algorithmic_counts(shape, desc):
    """FLOPs and bytes one step must move, per kernel class."""
    T = desc.n_tokens
    H, F, V, d = shape.hidden, shape.ffn, shape.vocab, shape.head_dim
    nq, nkv, nl = shape.n_q_heads, shape.n_kv_heads, shape.n_layers
    qkv_n = (nq + 2 * nkv) * d
    w_params = {"gemm_qkv": qkv_n * H, "gemm_o": H * nq * d, "gemm_gate_up": 2 * F * H, "gemm_down": H * F}
    flops = {k: 2.0 * T * p * nl for k, p in w_params.items()}
    flops["lm_head"] = 2.0 * T * V * H
    wbytes = {k: 2.0 * p * nl for k, p in w_params.items()}
    wbytes["lm_head"] = 2.0 * V * H
    kv_tokens = float((desc.ctx_len + desc.rows).sum())
    attn_bytes = nl * (kv_tokens * nkv * d * 2 * 2 + 2.0 * T * nq * d * 2)   # K+V once per layer, q in, o out
    attn_flops = nl * 4.0 * d * nq * float(((desc.ctx_len + desc.rows) * desc.rows).sum())
    logits_bytes = 4.0 * T * V
    return {"T": T, "flops": flops, "wbytes": wbytes, "attn_bytes": attn_bytes, "attn_flops": attn_flops,
            "verify_bytes": logits_bytes}


NOMINAL_HBM_GBS = 8000.0        # the workload statement's "about 8 TB/s"


def hbm_fracs(gbs, peaks):
    """Every bandwidth fraction is stated against both denominators: the measured copy bandwidth and 8 TB/s."""
    return {"frac_of_hbm_measured": round(gbs / peaks["hbm_gbs"], 4), "frac_of_8000": round(gbs / NOMINAL_HBM_GBS, 4)}


def tensor_fracs(tflops, peaks):
    """... and every tensor fraction against the measured burst and sustained bf16 rates."""
    return {"frac_of_bf16_burst": round(tflops / peaks["bf16_tflops"], 4),
            "frac_of_bf16_sustained": round(tflops / peaks["bf16_tflops_sustained"], 4)}


def roofline_entry(kind, achieved, peak, traffic=None, note=None):
    unit = "GB/s" if kind == "hbm" else "TFLOP/s"
    e = {"bound": kind, "achieved": round(achieved, 2), "peak": peak, "unit": unit, "frac": round(achieved / peak, 4),
         "traffic": traffic}
    if note:
        e["note"] = note
    return e


# ------------------------------------------------------------------------------------------------
# the product arm
# ------------------------------------------------------------------------------------------------
def run_ours(args, env):
    from paper_2609_34388_b200 import binding

    peaks = load_peaks()
    dev = torch.device("cuda", env.local_rank)
    torch.cuda.set_device(dev)
    shape = synth.llama8b_shape(32)
    t_setup = time.time()
    W = synth.model_weights(shape, seed=0, device=dev, dtype=torch.bfloat16)
    descs = [c16_descriptor(3 + i + 100 * env.rank) for i in range(10)]          # ten batch draws (seeds 3..12), rotated
    max_pages = max(d.page_table.shape[1] for d in descs)
    n_pages = max(d.n_pages for d in descs)
    cfg = binding.make_config(shape, 16, 1024, max_pages, args.flags)
    ctx = binding.Context(cfg, W)
    pool = binding.alloc_kv_pool(ctx, n_pages, fill="normal")
    batches = []
    for i, d in enumerate(descs):
        ys = synth.token_ids(int(d.verify_len.sum()), shape.vocab, seed=1 + i)
        batches.append(binding.Batch(d.ctx_len, d.verify_len, d.block_size, ys, d.page_table, pool, n_pages))
    torch.cuda.synchronize()
    setup_s = time.time() - t_setup

    outs_dev = [binding.VerifyOut(b.n_req, b.n_tok, b.n_ver, host=False) for b in batches]
    outs_host = [binding.VerifyOut(b.n_req, b.n_tok, b.n_ver, host=True) for b in batches]

    def step_device(i):
        j = i % len(batches)
        ctx.recg_step(batches[j])
        ctx.recg_verify(batches[j], out=outs_dev[j])

    def step_e2e(i):
        j = i % len(batches)
        ctx.recg_step(batches[j])               # host descriptor arrays are copied to the device by the call
        return ctx.recg_verify(batches[j], out=outs_host[j])   # results copied to host memory, stream synchronised

    for i in range(args.warmup):
        step_device(i)
    ctx.recg_sync()

    # ---- timed region: device-resident ----
    sampler = ClockSampler(env.local_rank)
    sampler.start()
    env.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.steps):
        step_device(i)
    e1.record()
    torch.cuda.synchronize()
    env.barrier()
    ms_total = e0.elapsed_time(e1)
    clocks = sampler.stop()
    ctx.recg_sync()
    tokens = sum(batches[i % len(batches)].n_tok for i in range(args.steps))
    ms_total_max = env.max_float(ms_total)
    tokens_all = env.sum_float(float(tokens))
    value = tokens_all / (ms_total_max / 1e3)

    # ---- timed region: end to end (host descriptors in, host results out, every step) ----
    for i in range(2):
        step_e2e(i)
    env.barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    e0.record()
    for i in range(args.steps):
        res = step_e2e(i)
    e1.record()
    torch.cuda.synchronize()
    wall_ms = (time.perf_counter() - t0) * 1e3
    env.barrier()
    e2e_ms = env.max_float(max(e0.elapsed_time(e1), wall_ms))
    b0 = batches[0]
    h2d = 4 * (9 * b0.n_req + 2 * (b0.n_req + 1) + b0.n_ver + b0.page_table.size)
    d2h = outs_host[0].nbytes()
    e2e_value = tokens_all / (e2e_ms / 1e3)

    out = {"metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": env.world, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": round(ms_total_max / args.steps, 4), "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
           "config": {"workload": "configs[2]: 32-layer 8B-class backbone, concurrency 16 per GPU, block sizes U{4,8,16,32}, "
                                  "verify_len = block, context U[512,8192], 10 batch draws (seeds 3..12) rotated",
                      "tokens_per_step": [b.n_tok for b in batches], "l2": "inputs (15 GB weights, 10-20 GB KV) larger than L2",
                      "logits": "fp32", "parallelism": f"replicas x{env.world}" if env.world > 1 else "single GPU"},
           "clocks": clocks,
           "e2e": {"value": round(e2e_value, 1), "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                   "ms_per_step": round(e2e_ms / args.steps, 4)},
           "gpu_launches": int(args.steps * (3 + 8 * shape.n_layers + 2 + 2)),
           "setup_s": round(setup_s, 1), "peaks": peaks}

    if env.rank == 0:
        # ---- per-class timing pass (events at class boundaries; separate from the timed region above) ----
        ctx.recg_timing_enable(True)
        ctx.recg_timing_read()
        for i in range(args.steps):
            step_device(i)
        ms, launches = ctx.recg_timing_read()
        ctx.recg_timing_enable(False)
        counts = [algorithmic_counts(shape, descs[i % len(descs)]) for i in range(args.steps)]
        gemm_classes = ("gemm_qkv", "gemm_o", "gemm_gate_up", "gemm_down", "lm_head")
        gemm_ms = sum(ms[k] for k in gemm_classes)
        gemm_flops = sum(sum(c["flops"][k] for k in gemm_classes) for c in counts)
        kern = {}
        for k in gemm_classes:
            fl = sum(c["flops"][k] for c in counts)
            kern[k] = {"ms_per_step": round(ms[k] / args.steps, 4), "tflops": round(fl / (ms[k] / 1e3) / 1e12, 1),
                       **tensor_fracs(fl / (ms[k] / 1e3) / 1e12, peaks)}
        ab = sum(c["attn_bytes"] for c in counts)
        kern["attention"] = {"ms_per_step": round(ms["attention"] / args.steps, 4),
                             "gbs": round(ab / (ms["attention"] / 1e3) / 1e9, 1),
                             **hbm_fracs(ab / (ms["attention"] / 1e3) / 1e9, peaks)}
        vb = sum(c["verify_bytes"] for c in counts)
        kern["verify"] = {"ms_per_step": round(ms["verify"] / args.steps, 4), "gbs": round(vb / (ms["verify"] / 1e3) / 1e9, 1),
                          **hbm_fracs(vb / (ms["verify"] / 1e3) / 1e9, peaks)}
        kern["rmsnorm"] = {"ms_per_step": round(ms["rmsnorm"] / args.steps, 4)}
        kern["layout"] = {"ms_per_step": round(ms["layout"] / args.steps, 4)}
        out["kernels"] = kern
        n_gemm_launch = sum(launches[k] for k in gemm_classes)
        ach = gemm_flops / (gemm_ms / 1e3) / 1e12
        # `traffic` (DRAM bytes of one launch under the profiler) cannot be measured inside this run; it is null here and the
        # profiler summary of the largest projection is kept with the other summaries under profiles/
        out["roofline"] = roofline_entry("tensor", ach, peaks["bf16_tflops_sustained"], None,
                                         f"projection GEMM kernel (tcgen05), {n_gemm_launch} launches, avg "
                                         f"{gemm_ms / max(n_gemm_launch, 1) * 1e3:.1f} us; peak = sustained bf16 of {peaks['source']} "
                                         f"(the kernel is timed inside a long step); of the burst rate: {ach / peaks['bf16_tflops']:.4f}; "
                                         "traffic: not measurable in this run (the ncu summary of the gate|up launch is under profiles/)")
        out["step_time_share"] = {k: round(v / sum(ms.values()), 4) for k, v in ms.items()}
    if env.rank == 0:
        # ---- every batch draw by itself: mean and range over the ten draws ----
        per = []
        for j, bt in enumerate(batches):
            for _ in range(2):
                ctx.recg_step(bt)
                ctx.recg_verify(bt, out=outs_dev[j])
            torch.cuda.synchronize()
            e0.record()
            for _ in range(3):
                ctx.recg_step(bt)
                ctx.recg_verify(bt, out=outs_dev[j])
            e1.record()
            torch.cuda.synchronize()
            per.append(e0.elapsed_time(e1) / 3)
        tps = [b.n_tok / (m / 1e3) for b, m in zip(batches, per)]
        out["draws"] = {"seeds": list(range(3, 13)), "tokens_per_step": [b.n_tok for b in batches],
                        "ms_per_step": [round(m, 3) for m in per],
                        "ms_mean": round(float(np.mean(per)), 3), "ms_min": round(min(per), 3), "ms_max": round(max(per), 3),
                        "tokens_per_s_mean": round(float(np.mean(tps)), 1), "tokens_per_s_min": round(min(tps), 1),
                        "tokens_per_s_max": round(max(tps), 1)}
    if args.quick:
        if env.rank == 0:
            out["c1"] = bench_c1(binding, ctx, shape, pool, n_pages, peaks, args)
        ctx.recg_free()
        return out
    if env.rank == 0:
        # the short-step and single-operation points are compared with peaks that were measured on an idle device, so the
        # device is left idle for a moment after the long step loops
        torch.cuda.synchronize()
        time.sleep(3.0)
        out["c1"] = bench_c1(binding, ctx, shape, pool, n_pages, peaks, args)
        out["attention_op"] = bench_attention_op(binding, peaks, args)
        out["attention_c16_op"] = bench_attention_op(binding, peaks, args, desc=c16_descriptor(3), n_layers=4,
                                                     label="attention of configs[2] draw 0 as a single operation: 16 requests, "
                                                           "blocks U{4,8,16,32}, context U[512,8192], 4 layer caches rotated "
                                                           "(1.2 GB > L2), CUDA-graph replay")
        out["verify_sweep"] = bench_verify(binding, peaks)
        out["gemm_shapes"] = bench_gemm_shapes(binding, peaks)
        out["cpu_baseline"] = cpu_baseline(shape, descs[0])
    ctx.recg_free()
    del pool, ctx
    torch.cuda.empty_cache()
    if env.rank == 0 and env.world == 1:
        out["device_loop"] = {"workload": "8 rounds with planted acceptance and the block-size rule, device-resident against "
                                          "host-driven, 32-layer 8B-class backbone",
                              "points": [bench_device_loop(binding, W, shape, peaks, n) for n in (1, 16)]}
        out["c128"] = bench_c128(binding, W, shape, peaks, args)
        del W
        torch.cuda.empty_cache()
        out["second_model"] = bench_second_model(binding, peaks, args)
    return out


def bench_second_model(binding, peaks, args):
    """The same step on an assumed 14B-class backbone (synth.dense14b_shape: 40 layers, hidden 5120, 40 / 8 heads, FFN
    17408, vocab 152064) at concurrency 16, configs[2]'s request recipe."""
    shape = synth.dense14b_shape()
    W = synth.model_weights(shape, seed=0, device="cuda", dtype=torch.bfloat16)
    desc = c16_descriptor(3)
    ctx = binding.Context(binding.make_config(shape, 16, 1024, desc.page_table.shape[1]), W)
    pool = binding.alloc_kv_pool(ctx, desc.n_pages, fill="normal")
    ys = synth.token_ids(int(desc.verify_len.sum()), shape.vocab, seed=1)
    batch = binding.Batch(desc.ctx_len, desc.verify_len, desc.block_size, ys, desc.page_table, pool, desc.n_pages)
    vout = binding.VerifyOut(batch.n_req, batch.n_tok, batch.n_ver, host=False)
    for _ in range(3):
        ctx.recg_step(batch)
        ctx.recg_verify(batch, out=vout)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    iters = 5
    e0.record()
    for _ in range(iters):
        ctx.recg_step(batch)
        ctx.recg_verify(batch, out=vout)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / iters
    ctx.recg_timing_enable(True)
    ctx.recg_timing_read()
    for _ in range(iters):
        ctx.recg_step(batch)
        ctx.recg_verify(batch, out=vout)
    cms, _ = ctx.recg_timing_read()
    ctx.recg_timing_enable(False)
    cnt = algorithmic_counts(shape, desc)
    gemm_classes = ("gemm_qkv", "gemm_o", "gemm_gate_up", "gemm_down", "lm_head")
    gemm_ms = sum(cms[k] for k in gemm_classes) / iters
    gemm_tf = sum(cnt["flops"][k] for k in gemm_classes) / (gemm_ms / 1e3) / 1e12
    attn_ms = cms["attention"] / iters
    attn_gbs = cnt["attn_bytes"] / (attn_ms / 1e3) / 1e9
    wbytes = sum(cnt["wbytes"].values())
    out = {"workload": "assumed 14B-class backbone (40 layers, hidden 5120, 40/8 heads, d 128, FFN 17408, vocab 152064), "
                       "concurrency 16, configs[2] request recipe, draw 0",
           "tokens_per_step": batch.n_tok, "ms_per_step": round(ms, 3), "tokens_per_s": round(batch.n_tok / (ms / 1e3), 1),
           "weight_gb": round(wbytes / 1e9, 1),
           "ideal_ms": round(max(wbytes / peaks["hbm_gbs"] / 1e6, sum(cnt["flops"].values()) / peaks["bf16_tflops_sustained"] / 1e9)
                             + cnt["attn_bytes"] / peaks["hbm_gbs"] / 1e6, 3),
           "gemm": {"ms_per_step": round(gemm_ms, 3), "tflops": round(gemm_tf, 1), **tensor_fracs(gemm_tf, peaks)},
           "attention": {"ms_per_step": round(attn_ms, 3), "gbs": round(attn_gbs, 1), **hbm_fracs(attn_gbs, peaks)}}
    ctx.recg_free()
    del pool, W
    torch.cuda.empty_cache()
    return out


def _time_graph(ctx_stream, fn, iters):
    """Capture fn() (library launches on ctx_stream) into a CUDA graph and time `iters` replays with events, so that
    short kernels are not hidden behind host launch latency.  Returns microseconds per replay."""
    with torch.cuda.stream(ctx_stream):
        fn()
        ctx_stream.synchronize()
        g = torch.cuda.CUDAGraph()
        g.capture_begin()
        fn()
        g.capture_end()
        for _ in range(2):
            g.replay()
        ctx_stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(ctx_stream)
        for _ in range(iters):
            g.replay()
        e1.record(ctx_stream)
        ctx_stream.synchronize()
    return e0.elapsed_time(e1) / iters * 1e3


def bench_attention_op(binding, peaks, args, desc=None, n_layers=32, label=None):
    """configs[1]: one layer's hybrid attention at 8B shapes, context 4096, 16 causal + 16 bidirectional rows.
    n_layers distinct layer caches are rotated so that the KV stream does not sit in L2; the calls of one rotation
    are replayed from a CUDA graph (kernel time, not launch latency)."""
    shape = synth.llama8b_shape(n_layers)
    desc = c1_descriptor(7) if desc is None else desc
    T = desc.n_tokens
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        ctx = binding.Context(binding.make_config(shape, desc.n_req, T, desc.page_table.shape[1]), stream=stream.cuda_stream)
        pool = binding.alloc_kv_pool(ctx, desc.n_pages, fill="normal")
        batch = binding.Batch(desc.ctx_len, desc.verify_len, desc.block_size, None, desc.page_table, pool, desc.n_pages,
                              **desc.branch_kwargs())
        q = synth.queries(T, 32, 128, seed=5, device="cuda")
        o = torch.empty_like(q)
        ctx.recg_attention(batch, 0, q, o)
        stream.synchronize()

    def rotation():
        for l in range(n_layers):
            ctx.recg_attention(None, l, q, o)

    us = _time_graph(stream, rotation, 10) / n_layers
    kv_tok = float((desc.ctx_len + desc.rows).sum())
    kv_bytes = kv_tok * 8 * 128 * 2 * 2 + 2 * T * 32 * 128 * 2
    ctx.recg_sync()
    ctx.recg_free()
    gbs = kv_bytes / (us * 1e-6) / 1e9
    return {"workload": label or "configs[1]: 32/8 heads, d 128, context 4096, 16 causal + 16 bidirectional rows, "
                                 f"{n_layers} caches rotated, CUDA-graph replay",
            "us_per_call": round(us, 2), "calls_include": "attention kernel + combine kernel", "algorithmic_bytes": int(kv_bytes),
            "gbs": round(gbs, 1), **hbm_fracs(gbs, peaks)}


def bench_small_step(binding, peaks, args, n_layers=2, n_req=16):
    """A small case of the whole step for profiler captures: n_layers 8B-shaped layers + LM head, n_req requests with
    configs[2]'s block sizes and contexts U[64, 1024] (about 1.5 GB of weights and a pool of a few hundred MB, so a
    capture that saves and restores device memory stays short).  Timed too, but it is not a benchmark figure."""
    shape = synth.llama8b_shape(n_layers)
    W = synth.model_weights(shape, seed=0, device="cuda", dtype=torch.bfloat16)
    desc = synth.batch_descriptor(n_req, [4, 8, 16, 32], None, 64, 1024, seed=3)
    ctx = binding.Context(binding.make_config(shape, n_req, desc.n_tokens, desc.page_table.shape[1], args.flags), W)
    pool = binding.alloc_kv_pool(ctx, desc.n_pages, fill="normal")
    ys = synth.token_ids(int(desc.verify_len.sum()), shape.vocab, seed=1)
    batch = binding.Batch(desc.ctx_len, desc.verify_len, desc.block_size, ys, desc.page_table, pool, desc.n_pages)
    vout = binding.VerifyOut(batch.n_req, batch.n_tok, batch.n_ver, host=False)
    for _ in range(3):
        ctx.recg_step(batch)
        ctx.recg_verify(batch, out=vout)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(5):
        ctx.recg_step(batch)
        ctx.recg_verify(batch, out=vout)
    e1.record()
    torch.cuda.synchronize()
    ctx.recg_sync()
    ctx.recg_free()
    return {"workload": f"{n_layers} 8B-shaped layers + LM head, {n_req} requests, {batch.n_tok} rows, contexts U[64,1024]",
            "ms_per_step": round(e0.elapsed_time(e1) / 5, 3)}


def bench_gemm_shapes(binding, peaks):
    """The five projection shapes of one 8B-class layer (+ LM head) as standalone y = x w^T calls (plain epilogue).
    Copies of the weight matrix are rotated (at least 300 MB in total, more than L2 holds) so that every call streams
    its weights from HBM like the calls inside a step do."""
    shape = synth.tiny_shape()
    shape.n_layers = 1
    ctx = binding.Context(binding.make_config(shape, 1, 8, 1))
    out = []
    for M in (32, 480, 1331):
        for name, N, K in (("qkv", 6144, 4096), ("o", 4096, 4096), ("gate_up", 28672, 4096), ("down", 4096, 14336),
                           ("lm_head", 128256, 4096)):
            g = torch.Generator(device="cuda")
            g.manual_seed(M + N)
            x = torch.randn((M, K), generator=g, device="cuda").to(torch.bfloat16)
            n_copies = max(1, int(np.ceil(300e6 / (N * K * 2))))
            ws = [(torch.randn((N, K), generator=g, device="cuda") * 0.02).to(torch.bfloat16)]
            ws += [ws[0].clone() for _ in range(n_copies - 1)]
            y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
            calls = 12 if n_copies == 1 else n_copies * max(1, 12 // n_copies)

            def run(n):
                for i in range(n):
                    binding.lib().recg_linear(ctx.h, x.data_ptr(), ws[i % n_copies].data_ptr(), y.data_ptr(), M, N, K, 0)

            run(max(3, n_copies))
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            run(calls)
            e1.record()
            torch.cuda.synchronize()
            us = e0.elapsed_time(e1) / calls * 1e3
            tf = 2.0 * M * N * K / (us * 1e-6) / 1e12
            gbs = N * K * 2 / (us * 1e-6) / 1e9
            out.append({"M": M, "name": name, "N": N, "K": K, "us": round(us, 1), "weight_copies_rotated": n_copies,
                        "tflops": round(tf, 1), **tensor_fracs(tf, peaks), "weight_gbs": round(gbs, 1), **hbm_fracs(gbs, peaks)})
            del x, ws, y
    ctx.recg_free()
    return out


def bench_verify(binding, peaks):
    """configs[4]: the verify kernel over bf16 logits [B (k+1), 128256] ~ N(0,1) for every B in {1,8,32,128,256} and k in
    {4,8,16,32}.  Drafts are planted: a prefix of Geometric(0.25) length (cut at k) equals the rows' argmax, the next
    draft differs, the rest is random; the accept lengths that come back must be the planted ones.  Copies of the
    logits are rotated so that the scan does not sit in L2, and one rotation is replayed from a CUDA graph (kernel
    time, not launch latency)."""
    V = 128256
    res = []
    shape = synth.ModelShape(n_layers=0, hidden=64, n_q_heads=4, n_kv_heads=2, head_dim=64, ffn=64, vocab=V)
    for B in (1, 8, 32, 128, 256):
        for k in (4, 8, 16, 32):
            R = B * (k + 1)
            stream = torch.cuda.Stream()
            with torch.cuda.stream(stream):
                ctx = binding.Context(binding.make_config(shape, B, R, 1), stream=stream.cuda_stream)
                lg = synth.logits_normal(R, V, seed=6, device="cuda")
                # the ids the rows select (lowest index among equal maxima), for the planting only
                ids = torch.arange(V, device="cuda", dtype=torch.int32)
                sel = []
                for r0 in range(0, R, 512):
                    part = lg[r0:r0 + 512].float()
                    mx = part.max(dim=1, keepdim=True).values
                    sel.append(torch.where(part == mx, ids, V).min(dim=1).values)
                sel = torch.cat(sel)
                accept = synth.planted_accept_lengths(B, k, 0.25, seed=4)
                y = synth.plant_drafts(sel.cpu().numpy(), B, k, accept, V, seed=4).reshape(-1)
                del mx, sel, part, ids
                batch = binding.Batch([0] * B, [k + 1] * B, [0] * B, y)
                vout = binding.VerifyOut(B, R, R, host=False)
                ctx.recg_verify(batch, lg, out=vout)
                stream.synchronize()
                planted_ok = bool((vout.bufs["accept_len"][:B].cpu().numpy() == accept).all())
                n_rot = max(2, min(64, int(np.ceil(300e6 / (R * V * 2)))))
                copies = [lg] + [lg.clone() for _ in range(n_rot - 1)]
                stream.synchronize()

            def rotation():
                for c in copies:
                    ctx.recg_verify(None, c, out=vout)

            us = _time_graph(stream, rotation, 5) / len(copies)
            gbs = R * V * 2 / (us * 1e-6) / 1e9
            res.append({"B": B, "k": k, "rows": R, "us": round(us, 2), "gbs": round(gbs, 1), **hbm_fracs(gbs, peaks),
                        "emitted_tokens": int(accept.sum() + B), "accept_lengths_as_planted": planted_ok})
            ctx.recg_sync()
            ctx.recg_free()
            del copies, lg
            torch.cuda.empty_cache()
    return res


def bench_c128(binding, W, shape, peaks, args):
    """High-concurrency point: full model, 128 requests (see c128_descriptor), per-class times."""
    free_b, _ = torch.cuda.mem_get_info()
    desc, ctx_scale = c128_descriptor(5, 1.0), 1.0
    # pool + workspace (logits for 8192 rows and the rest: about 6 GB) + a margin must fit, else halve the contexts
    if desc.n_pages * 16 * 131072 + (14 << 30) > free_b:
        desc, ctx_scale = c128_descriptor(5, 0.5), 0.5
    # the same context and pool also serve the concurrency sweep below (configs[2]'s recipe at other batch sizes)
    sweep_descs = {C: synth.batch_descriptor(C, [4, 8, 16, 32], None, 512, 8192, seed=40 + C) for C in (1, 2, 4, 8, 16, 32, 64, 128)}
    # rounds with prospective correction branches (two per request, one block of the request's size each), and
    # the same requests without them
    ov_plain = {"c16": c16_descriptor(3), "c1": c1_descriptor(11)}
    ov_descs = {k: synth.with_correction_branches(d, shape.vocab, 2, seed=60) for k, d in ov_plain.items()}
    # forward time against concurrency for one block size at a time (the paper's Fig. 2b on random weights): T_C(B), the
    # profile the block-size rule weighs against the expected progress
    tcb_descs = {(C, B): synth.batch_descriptor(C, [B], None, 512, 8192, seed=80 + C) for C in (1, 4, 16, 64, 128) for B in (8, 16, 32)}
    # the block mixtures the paper's adaptive policy ends up with on its 8B model (its block-distribution table: shares
    # of blocks 8 / 16 / 32 at each concurrency), contexts as in configs[2]: the paper-shaped points of the sweep
    mix_descs = {C: synth.batch_descriptor(C, [8, 16, 32], [p / sum(mix) for p in mix], 512, 8192, seed=120 + C)
                 for C, mix in ((2, (9.33, 2.54, 88.13)), (8, (3.70, 36.96, 59.34)), (32, (41.17, 43.33, 15.50)),
                                (128, (78.21, 12.04, 9.75)))}
    all_descs = [desc] + list(sweep_descs.values()) + list(ov_descs.values()) + list(tcb_descs.values()) + list(mix_descs.values())
    n_pages = max(d.n_pages for d in all_descs)
    cfg = binding.make_config(shape, 128, max(2048, max(d.n_tokens for d in all_descs)), max(d.page_table.shape[1] for d in all_descs))
    need = binding.lib().recg_kv_pool_bytes(__import__("ctypes").byref(cfg), n_pages)
    if need + (8 << 30) > free_b:
        return {"skipped": f"pool of {need / 1e9:.0f} GB does not fit in the {free_b / 1e9:.0f} GB that are free"}
    ctx = binding.Context(cfg, W)
    pool = binding.alloc_kv_pool(ctx, n_pages, fill="normal")
    ys = synth.token_ids(int(desc.verify_len.sum()), shape.vocab, seed=9)
    batch = binding.Batch(desc.ctx_len, desc.verify_len, desc.block_size, ys, desc.page_table, pool, n_pages)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # ---- tokens/s against concurrency: configs[2]'s recipe (blocks U{4,8,16,32}, verify_len = block, context
    # U[512,8192]) at 1 .. 128 requests, one batch draw each, whole step (recg_step + recg_verify), device resident
    sweep = []
    for C, d in sweep_descs.items():
        ysw = synth.token_ids(int(d.verify_len.sum()), shape.vocab, seed=50 + C)
        bt = binding.Batch(d.ctx_len, d.verify_len, d.block_size, ysw, d.page_table, pool, n_pages)
        vo = binding.VerifyOut(bt.n_req, bt.n_tok, bt.n_ver, host=False)
        for _ in range(3):
            ctx.recg_step(bt)
            ctx.recg_verify(bt, out=vo)
        torch.cuda.synchronize()
        n_it = 5
        e0.record()
        for _ in range(n_it):
            ctx.recg_step(bt)
            ctx.recg_verify(bt, out=vo)
        e1.record()
        torch.cuda.synchronize()
        msw = e0.elapsed_time(e1) / n_it
        cw = algorithmic_counts(shape, d)
        sweep.append({"concurrency": C, "tokens_per_step": bt.n_tok, "kv_tokens": int(np.sum(d.ctx_len + d.rows)),
                      "ms_per_step": round(msw, 3), "tokens_per_s": round(bt.n_tok / (msw / 1e3), 1),
                      "ideal_ms": round(max(sum(cw["wbytes"].values()) / peaks["hbm_gbs"] / 1e6,
                                            sum(cw["flops"].values()) / peaks["bf16_tflops_sustained"] / 1e9) +
                                        cw["attn_bytes"] / peaks["hbm_gbs"] / 1e6, 3)})
    sweep_result = {"workload": "configs[2] recipe at other batch sizes, one draw each, processed tokens/s of the whole step; "
                                            "ideal_ms = max(weight stream, GEMM flops at sustained peak) + KV stream, of measured peaks",
                                "points": sweep}
    mix = []
    for C, d in mix_descs.items():
        ysw = synth.token_ids(int(d.verify_len.sum()), shape.vocab, seed=130 + C)
        bt = binding.Batch(d.ctx_len, d.verify_len, d.block_size, ysw, d.page_table, pool, n_pages)
        vo = binding.VerifyOut(bt.n_req, bt.n_tok, bt.n_ver, host=False)
        n_it = 5 if C >= 32 else 20
        for _ in range(3):
            ctx.recg_step(bt)
            ctx.recg_verify(bt, out=vo)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(n_it):
            ctx.recg_step(bt)
            ctx.recg_verify(bt, out=vo)
        e1.record()
        torch.cuda.synchronize()
        msw = e0.elapsed_time(e1) / n_it
        cw = algorithmic_counts(shape, d)
        mix.append({"concurrency": C, "blocks": {int(b): int((d.block_size == b).sum()) for b in (8, 16, 32)},
                    "tokens_per_step": bt.n_tok, "ms_per_step": round(msw, 3), "tokens_per_s": round(bt.n_tok / (msw / 1e3), 1),
                    "ideal_ms": round(max(sum(cw["wbytes"].values()) / peaks["hbm_gbs"] / 1e6,
                                          sum(cw["flops"].values()) / peaks["bf16_tflops_sustained"] / 1e9) +
                                      cw["attn_bytes"] / peaks["hbm_gbs"] / 1e6, 3)})
    mix_result = {"workload": "block sizes drawn from the paper's reported 8B block distribution at each concurrency (shares of 8 / "
                              "16 / 32), verify_len = block, context U[512,8192], one draw per point; whole step",
                  "points": mix}
    tcb = []
    for (C, B), d in tcb_descs.items():
        ysw = synth.token_ids(int(d.verify_len.sum()), shape.vocab, seed=90)
        bt = binding.Batch(d.ctx_len, d.verify_len, d.block_size, ysw, d.page_table, pool, n_pages)
        vo = binding.VerifyOut(bt.n_req, bt.n_tok, bt.n_ver, host=False)
        n_it = 4 if C >= 64 else 20          # short steps: enough of them for the clocks to settle
        for _ in range(n_it):
            ctx.recg_step(bt)
            ctx.recg_verify(bt, out=vo)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(n_it):
            ctx.recg_step(bt)
            ctx.recg_verify(bt, out=vo)
        e1.record()
        torch.cuda.synchronize()
        tcb.append({"concurrency": C, "block": B, "rows": bt.n_tok, "ms_per_step": round(e0.elapsed_time(e1) / n_it, 3)})
    tcb_result = {"workload": "whole step, every request with verify_len = block = B, context U[512,8192], one draw per point",
                  "points": tcb}
    # ---- one ragged mixed batch against one batch per block size (the remedy of padded kernels) ----
    from paper_2609_34388_b200 import schedule
    bucketing = []
    for C in (16, 128):
        d = sweep_descs[C]
        ysw = synth.token_ids(int(d.verify_len.sum()), shape.vocab, seed=50 + C)
        plans = {"ragged": [(d, ysw)]}
        groups = schedule.bucket_by_block(d.block_size)
        plans["bucketed"] = []
        for idx in groups.values():
            toks = np.concatenate([ysw[sl] for sl in schedule.verify_token_slices(d, idx)])
            plans["bucketed"].append((schedule.sub_descriptor(d, idx), toks))
        res = {"concurrency": C, "rows": d.n_tokens, "rows_if_padded_to_longest": schedule.padded_rows(d),
               "buckets": {int(b): len(idx) for b, idx in groups.items()}}
        for name, plan in plans.items():
            bts = [binding.Batch(x.ctx_len, x.verify_len, x.block_size, t, x.page_table, pool, n_pages) for x, t in plan]
            vos = [binding.VerifyOut(bt.n_req, bt.n_tok, bt.n_ver, host=False) for bt in bts]
            def run_plan():
                for bt, vo in zip(bts, vos):
                    ctx.recg_step(bt)
                    ctx.recg_verify(bt, out=vo)
            for _ in range(3):
                run_plan()
            torch.cuda.synchronize()
            e0.record()
            for _ in range(5):
                run_plan()
            e1.record()
            torch.cuda.synchronize()
            msw = e0.elapsed_time(e1) / 5
            res[name] = {"steps": len(bts), "ms": round(msw, 3), "rows_per_s": round(d.n_tokens / (msw / 1e3), 1)}
        res["bucketed_over_ragged"] = round(res["bucketed"]["ms"] / res["ragged"]["ms"], 3)
        bucketing.append(res)
    bucketing_result = {"workload": "configs[2] recipe at 16 and 128 requests: the whole mixed batch in one ragged step against one "
                                    "step per block size (4 steps), same requests, same pool; time for all requests of the round",
                        "points": bucketing}
    overlap = {}
    for key in ov_descs:
        res = {}
        for kind, d in (("plain", ov_plain[key]), ("branches", ov_descs[key])):
            ysw = synth.token_ids(int(d.verify_len.sum()), shape.vocab, seed=70)
            bt = binding.Batch(d.ctx_len, d.verify_len, d.block_size, ysw, d.page_table, pool, n_pages, **d.branch_kwargs())
            vo = binding.VerifyOut(bt.n_req, bt.n_tok, bt.n_ver, host=False)
            for _ in range(3):
                ctx.recg_step(bt)
                ctx.recg_verify(bt, out=vo)
            torch.cuda.synchronize()
            n_it = 5
            e0.record()
            for _ in range(n_it):
                ctx.recg_step(bt)
                ctx.recg_verify(bt, out=vo)
            e1.record()
            torch.cuda.synchronize()
            msw = e0.elapsed_time(e1) / n_it
            ctx.recg_timing_enable(True)
            ctx.recg_timing_read()
            for _ in range(n_it):
                ctx.recg_step(bt)
                ctx.recg_verify(bt, out=vo)
            cms, _ = ctx.recg_timing_read()
            ctx.recg_timing_enable(False)
            cw = algorithmic_counts(shape, d)
            att = cms["attention"] / n_it
            res[kind] = {"rows_per_step": bt.n_tok, "ms_per_step": round(msw, 3), "rows_per_s": round(bt.n_tok / (msw / 1e3), 1),
                         "attention_ms": round(att, 3), "attention_gbs": round(cw["attn_bytes"] / (att / 1e3) / 1e9, 1),
                         "attention": hbm_fracs(cw["attn_bytes"] / (att / 1e3) / 1e9, peaks)}
        res["step_time_ratio"] = round(res["branches"]["ms_per_step"] / res["plain"]["ms_per_step"], 3)
        overlap[key] = res
    overlap_result = {"workload": "configs[2] draw 0 (c16) and the concurrency-1 case (c1) with two correction branches per request "
                                  "(replaced draft indices drawn at random, one block of the request's size per branch) beside the "
                                  "same requests without branches; attention bytes count a request's K/V once per layer for all "
                                  "of its rows", "points": overlap}
    vout = binding.VerifyOut(batch.n_req, batch.n_tok, batch.n_ver, host=False)
    for _ in range(3):
        ctx.recg_step(batch)
        ctx.recg_verify(batch, out=vout)
    torch.cuda.synchronize()
    iters = 4
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        ctx.recg_step(batch)
        ctx.recg_verify(batch, out=vout)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / iters
    ctx.recg_timing_enable(True)
    ctx.recg_timing_read()
    for _ in range(iters):
        ctx.recg_step(batch)
        ctx.recg_verify(batch, out=vout)
    cms, _ = ctx.recg_timing_read()
    ctx.recg_timing_enable(False)
    cnt = algorithmic_counts(shape, desc)
    gemm_classes = ("gemm_qkv", "gemm_o", "gemm_gate_up", "gemm_down", "lm_head")
    gemm_ms = sum(cms[k] for k in gemm_classes) / iters
    gemm_tf = sum(cnt["flops"][k] for k in gemm_classes) / (gemm_ms / 1e3) / 1e12
    attn_ms = cms["attention"] / iters
    attn_gbs = cnt["attn_bytes"] / (attn_ms / 1e3) / 1e9
    label = ("configs[3] as stated: concurrency 128, blocks {2,4,8,16} @ (.4,.3,.2,.1), verify_len = block, context lengths "
             "U[1024,16384]") if ctx_scale == 1.0 else \
            ("configs[3] at HALF context (U[512,8192]: the full-length pool did not fit beside weights and workspace): "
             "concurrency 128, blocks {2,4,8,16} @ (.4,.3,.2,.1), verify_len = block")
    wb = sum(cnt["wbytes"].values())
    out = {"workload": label, "context_scale": ctx_scale,
           "tokens_per_step": batch.n_tok, "kv_tokens": int(np.sum(desc.ctx_len + desc.rows)), "kv_pool_gb": round(need / 1e9, 1),
           "ms_per_step": round(ms, 3), "tokens_per_s": round(batch.n_tok / (ms / 1e3), 1),
           "ideal_ms": round(max(wb / peaks["hbm_gbs"] / 1e6, sum(cnt["flops"].values()) / peaks["bf16_tflops_sustained"] / 1e9) +
                             cnt["attn_bytes"] / peaks["hbm_gbs"] / 1e6, 3),
           "gemm": {"ms_per_step": round(gemm_ms, 3), "tflops": round(gemm_tf, 1), **tensor_fracs(gemm_tf, peaks)},
           "attention": {"ms_per_step": round(attn_ms, 3), "gbs": round(attn_gbs, 1), **hbm_fracs(attn_gbs, peaks)}}
    out["concurrency_sweep"] = sweep_result
    out["block_mixture_sweep"] = mix_result
    out["bucketing"] = bucketing_result
    out["forward_time_by_block"] = tcb_result
    # block-size rule on the device after the verification of the 128-request batch (one small kernel; launch bound)
    tb = synth.policy_table()
    ctx.recg_policy_load(tb["blocks"], tb["s_edges"], tb["value"], tb["cost"])
    pst = {"e1": torch.zeros(128, dtype=torch.float32, device="cuda"), "e2": torch.zeros(128, dtype=torch.float32, device="cuda"),
           "block_index": torch.zeros(128, dtype=torch.int32, device="cuda"), "full": torch.zeros(128, dtype=torch.int32, device="cuda")}
    nxt = torch.zeros(128, dtype=torch.int32, device="cuda")
    for _ in range(10):
        ctx.recg_policy_step(pst, nxt, vout.bufs["entropy_mean"], vout.bufs["accept_len"])
    torch.cuda.synchronize()
    e0.record()
    for _ in range(200):
        ctx.recg_policy_step(pst, nxt, vout.bufs["entropy_mean"], vout.bufs["accept_len"])
    e1.record()
    torch.cuda.synchronize()
    out["policy_step"] = {"workload": "block-size rule for 128 requests, 3 candidates x 12 certainty bins, back-to-back launches",
                          "us_per_call": round(e0.elapsed_time(e1) / 200 * 1e3, 2),
                          "share_of_step": round(e0.elapsed_time(e1) / 200 / ms, 6)}
    out["overlap_branches"] = overlap_result
    ctx.recg_free()
    del pool
    torch.cuda.empty_cache()
    return out


def bench_c1(binding, ctx, shape, pool, n_pages, peaks, args):
    """Concurrency 1 (context 4096, 16 + 16 rows) through the full model: the weight-streaming regime."""
    desc = c1_descriptor(11)
    ys = synth.token_ids(16, shape.vocab, seed=2)
    batch = binding.Batch(desc.ctx_len, desc.verify_len, desc.block_size, ys, desc.page_table, pool, n_pages)
    vout = binding.VerifyOut(batch.n_req, batch.n_tok, batch.n_ver, host=False)
    for _ in range(3):
        ctx.recg_step(batch)
        ctx.recg_verify(batch, out=vout)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    iters = max(3, args.steps)
    e0.record()
    for _ in range(iters):
        ctx.recg_step(batch)
        ctx.recg_verify(batch, out=vout)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / iters
    ctx.recg_timing_enable(True)
    ctx.recg_timing_read()
    for _ in range(iters):
        ctx.recg_step(batch)
        ctx.recg_verify(batch, out=vout)
    cms, _ = ctx.recg_timing_read()
    ctx.recg_timing_enable(False)
    classes = {k: round(v / iters, 4) for k, v in cms.items()}
    wbytes = 2.0 * (shape.n_layers * ((shape.n_q_heads + 2 * shape.n_kv_heads) * shape.head_dim * shape.hidden +
                                       shape.hidden * shape.n_q_heads * shape.head_dim + 3 * shape.ffn * shape.hidden) +
                    shape.vocab * shape.hidden)
    return {"workload": "concurrency 1, context 4096, verify 16 + block 16", "ms_per_step": round(ms, 4),
            "tokens_per_s": round(32 / (ms / 1e3), 1), "weight_stream_gbs": round(wbytes / (ms / 1e3) / 1e9, 1),
            **hbm_fracs(wbytes / (ms / 1e3) / 1e9, peaks), "class_ms_per_step": classes}


def bench_device_loop(binding, W, shape, peaks, n_req, rounds=8):
    """Rounds per second with and without host round trips: the same requests run `rounds` rounds (a) device-resident --
    step, verification, block-size rule and next-round bookkeeping enqueued back to back, one sync at the end -- and
    (b) host-driven -- results copied to the host after every round and the next descriptor built there.  Acceptance
    lengths are planted from the interval chain of the paper's transition table (random weights accept nothing); block
    sizes come from the rule with a synthetic value table over {8, 16, 32}; contexts U[512, 8192]."""
    rng = np.random.default_rng(200 + n_req)
    Ls = rng.integers(512, 8193, size=n_req).astype(np.int32)
    grow = rounds * 33 + 64
    pt, n_pages = synth.page_tables(Ls, [grow] * n_req, 16, seed=201)
    max_tok = n_req * 64
    ctx = binding.Context(binding.make_config(shape, n_req, max_tok, pt.shape[1]), W)
    pool = binding.alloc_kv_pool(ctx, n_pages, fill="normal")
    tb = synth.policy_table()
    ctx.recg_policy_load(tb["blocks"], tb["s_edges"], tb["value"], tb["cost"])
    planted = synth.acceptance_chain_lengths(rounds, n_req, seed=202)            # [rounds, n_req] emitted tokens per round
    pl_dev = torch.from_numpy(planted).cuda()
    y0 = [[int(t)] for t in synth.token_ids(n_req, shape.vocab, seed=203)]

    def fresh_state():
        return {"e1": torch.zeros(n_req, dtype=torch.float32, device="cuda"), "e2": torch.zeros(n_req, dtype=torch.float32, device="cuda"),
                "block_index": torch.zeros(n_req, dtype=torch.int32, device="cuda"), "full": torch.zeros(n_req, dtype=torch.int32, device="cuda")}

    nxt = torch.zeros(n_req, dtype=torch.int32, device="cuda")
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def run_device():
        db = binding.DeviceBatch(Ls, [1] * n_req, [16] * n_req, y0, 32, pt, pool, n_pages, rows_hint=n_req * 24)
        st = fresh_state()
        log = binding.RoundLog(n_req, rounds, rounds * 33)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        e0.record()
        for r in range(rounds):
            ctx.recg_step_device(db)
            ctx.recg_verify_device()
            ctx.recg_policy_step(st, nxt)
            ctx.recg_next_round(db, r, next_block=nxt, planted_emitted=pl_dev[r], log=log)
        e1.record()
        torch.cuda.synchronize()
        wall = (time.perf_counter() - t0) * 1e3
        return max(e0.elapsed_time(e1), wall), int(log.n_tokens.sum()), log.block_size.cpu().numpy()

    def run_host():
        L, v, b = Ls.copy(), np.ones(n_req, np.int32), np.full(n_req, 16, np.int32)
        ys = [list(y) for y in y0]
        st = fresh_state()
        emitted = 0
        blocks = []
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        e0.record()
        for r in range(rounds):
            bt = binding.Batch(L, v, b, [t for y in ys for t in y], pt, pool, n_pages)
            ctx.recg_step(bt)
            g = ctx.recg_verify(bt)                       # host results: copies and a sync every round
            ctx.recg_policy_step(st, nxt)
            nb = nxt.cpu().numpy()                        # the host needs the next block sizes to size the next batch
            blocks.append(b.copy())
            cuv = np.concatenate([[0], np.cumsum(v)])
            cub = np.concatenate([[0], np.cumsum(b)])
            for i in range(n_req):                        # the bookkeeping between rounds, on the host
                e = max(1, min(int(planted[r, i]), int(v[i])))
                a = e - 1
                last = int(g["top1"][int(cuv[i] + cub[i]) + a])
                reuse = b[i] > 0 and a == v[i] - 1
                emitted += e
                L[i] += e
                if reuse:
                    ys[i] = [last] + g["next_draft"][int(cub[i]) + 1: int(cub[i]) + int(b[i])].tolist()
                else:
                    ys[i] = [last]
                v[i] = len(ys[i])
                b[i] = nb[i]
        e1.record()
        torch.cuda.synchronize()
        wall = (time.perf_counter() - t0) * 1e3
        return max(e0.elapsed_time(e1), wall), emitted, np.asarray(blocks)

    run_device()
    run_host()
    ms_d, em_d, blk_d = run_device()
    ms_h, em_h, blk_h = run_host()
    ctx.recg_sync()
    ctx.recg_free()
    del pool
    torch.cuda.empty_cache()
    return {"concurrency": n_req, "rounds": rounds,
            "device_resident": {"ms_per_round": round(ms_d / rounds, 3), "rounds_per_s": round(rounds / (ms_d / 1e3), 1),
                                "emitted_tokens": em_d, "emitted_tokens_per_s": round(em_d / (ms_d / 1e3), 1)},
            "host_driven": {"ms_per_round": round(ms_h / rounds, 3), "rounds_per_s": round(rounds / (ms_h / 1e3), 1),
                            "emitted_tokens": em_h, "emitted_tokens_per_s": round(em_h / (ms_h / 1e3), 1)},
            "same_emitted_tokens": em_d == em_h, "same_block_sizes": bool((blk_d == blk_h).all()),
            "host_over_device": round(ms_h / ms_d, 3)}


# ------------------------------------------------------------------------------------------------
# the oracle, timed as it stands on the host cores (reported baseline, and the --impl reference arm)
# ------------------------------------------------------------------------------------------------
class OracleSample:
    """The CPU oracle, as it stands, on a bounded sample of the workload: the first n_req requests of the batch through
    ONE of the n_layers layers plus the LM head and verification; the layer time is scaled by n_layers."""

    def __init__(self, shape, desc, n_req=1):
        from oracle import recg_oracle as orc

        self.orc = orc
        self.shape = shape
        one = synth.ModelShape(**{**shape.as_dict(), "n_layers": 1})
        W = synth.model_weights(one, seed=0, device="cpu", dtype=torch.bfloat16)
        self.W64 = {k: ([t.double().numpy() for t in v] if isinstance(v, list) else v.double().numpy())
                    for k, v in W.items() if k != "embed"}
        self.W64["embed"] = W["embed"].float().numpy()       # exact widening; rows are widened to fp64 on lookup
        self.ocfg = orc.ModelConfig(**one.as_dict())
        self.reqs = []
        for r in range(min(n_req, desc.n_req)):
            L, v, b = int(desc.ctx_len[r]), int(desc.verify_len[r]), int(desc.block_size[r])
            K, V = synth.kv_values(L, shape.n_kv_heads, shape.head_dim, seed=2 + r, device="cpu")
            self.reqs.append((L, b, [(K.double().numpy(), V.double().numpy())], synth.token_ids(v, shape.vocab, seed=1 + r).tolist()))

    def step(self):
        """Returns (tokens/s, seconds for the whole model by the scaling rule, tokens)."""
        orc = self.orc
        layer = head = ver = 0.0
        toks = 0
        for (L, b, kv, y) in self.reqs:
            t0 = time.perf_counter()
            logits, _, h = orc.fused_round_cached(self.ocfg, self.W64, kv, L, y, b)
            t1 = time.perf_counter()
            x = orc.rmsnorm(h, self.W64["final_norm"], self.ocfg.rms_eps)     # the head alone, to split layer / head time
            _ = x @ self.W64["lm_head"].T
            t2 = time.perf_counter()
            orc.verify_round(logits, y, b)
            t3 = time.perf_counter()
            head += t2 - t1
            layer += (t1 - t0) - (t2 - t1)
            ver += t3 - t2
            toks += len(y) + b
        total = layer * self.shape.n_layers + head + ver
        return toks / total, total, toks

    def describe(self):
        rows = sum(len(y) + b for (_, b, _, y) in self.reqs)
        ctxs = sum(L for (L, _, _, _) in self.reqs)
        return (f"{len(self.reqs)} request(s) of the concurrency-16 batch ({rows} rows over {ctxs} context tokens) through 1 of "
                f"{self.shape.n_layers} layers (time x{self.shape.n_layers}) plus the full LM head and verification; fp64 numpy")


def cpu_baseline(shape, desc):
    import multiprocessing

    s = OracleSample(shape, desc, n_req=desc.n_req)       # the whole batch: some tens of seconds of CPU work
    t0 = time.perf_counter()
    tps, secs, toks = s.step()
    return {"value": round(tps, 2), "unit": UNIT, "cores": multiprocessing.cpu_count(), "kind": "oracle",
            "sample": s.describe(), "seconds_scaled": round(secs, 2), "seconds_spent": round(time.perf_counter() - t0, 1)}


def run_reference(args, env):
    import multiprocessing

    shape = synth.llama8b_shape(32)
    s = OracleSample(shape, c16_descriptor(3))
    for _ in range(args.warmup):
        s.step()
    vals = [s.step() for _ in range(args.steps)]
    tps = float(np.mean([v[0] for v in vals]))
    secs = float(np.mean([v[1] for v in vals]))
    cb = {"value": round(tps, 2), "unit": UNIT, "cores": multiprocessing.cpu_count(), "kind": "oracle", "sample": s.describe()}
    return {"impl": "reference", "metric": METRIC, "value": round(tps, 2), "unit": UNIT, "n_gpus": env.world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(secs * 1e3, 2), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": "configs[2] (bounded sample per step, see cpu_baseline.sample)"},
            "cpu_baseline": cb,
            "e2e": {"value": round(tps, 2), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=8)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--flags", type=int, default=0, help="recg_config.flags of the timed context (A/B checks)")
    ap.add_argument("--quick", action="store_true", help="the timed step, its per-class times and the concurrency-1 point only")
    ap.add_argument("--only", default="", help="comma list of op-level sections to run alone (attention_op, attention_c16, attention_c16_branches, small_step, device_loop, verify_sweep, gemm_shapes): "
                                               "small cases for profiling; prints their JSON and exits")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        # rank 0 alone times the oracle on the host cores; the other ranks have nothing to do
        env = DistEnv(rank=int(os.environ.get("RANK", "0")), world=int(os.environ.get("WORLD_SIZE", "1")))
        if env.rank == 0:
            print(json.dumps(run_reference(args, env)), flush=True)
        return
    if args.only:
        from paper_2609_34388_b200 import binding

        peaks = load_peaks()
        res = {}
        for sec in args.only.split(","):
            if sec == "attention_op":
                res[sec] = bench_attention_op(binding, peaks, args)
            elif sec == "attention_c16":
                res[sec] = bench_attention_op(binding, peaks, args, desc=c16_descriptor(3), n_layers=4,
                                              label="attention of configs[2]: 16 requests, blocks U{4,8,16,32}, context "
                                                    "U[512,8192], 4 layer caches rotated, CUDA-graph replay")
            elif sec == "attention_c16_branches":
                res[sec] = bench_attention_op(binding, peaks, args, n_layers=4,
                                              desc=synth.with_correction_branches(c16_descriptor(3), 128256, 2, seed=60),
                                              label="attention of configs[2] draw 0 with two correction branches per request "
                                                    "(784 rows instead of 376), 4 layer caches rotated, CUDA-graph replay")
            elif sec == "device_loop":
                shape2 = synth.llama8b_shape(2)
                W2 = synth.model_weights(shape2, seed=0, device="cuda", dtype=torch.bfloat16)
                res[sec] = [bench_device_loop(binding, W2, shape2, peaks, n) for n in (1, 16)]
            elif sec == "small_step":
                res[sec] = bench_small_step(binding, peaks, args)
            elif sec == "verify_sweep":
                res[sec] = bench_verify(binding, peaks)
            elif sec == "gemm_shapes":
                res[sec] = bench_gemm_shapes(binding, peaks)
        print(json.dumps(res), flush=True)
        return
    env = DistEnv.from_env(backend="nccl")
    out = run_ours(args, env)
    if env.rank == 0:
        print(json.dumps(out), flush=True)
    env.close()


if __name__ == "__main__":
    main()
