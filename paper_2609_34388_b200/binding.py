"""Thin ctypes binding of librecg.so: same names as the C ABI, argument marshalling only.

Every step of the path runs inside the CUDA library; this module converts Python/torch
objects to the plain pointers and sizes the C ABI takes (see include/recg.h).  There is no
fallback: if the library is missing, or there is no CUDA device, calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librecg.so")

RECG_OK = 0
DTYPE_BF16, DTYPE_F32 = 0, 1
MEM_DEVICE, MEM_HOST = 0, 1
FLAG_LOGITS_BF16, FLAG_SIMT_GEMM, FLAG_SIMT_ATTENTION, FLAG_DEBUG_CHECKS, FLAG_FOLD_NORM, FLAG_CHAIN = 1, 2, 4, 8, 16, 32
STATUS_NAMES = {0: "RECG_OK", 1: "RECG_ERR_INVALID_ARG", 2: "RECG_ERR_SHAPE", 3: "RECG_ERR_CAPACITY",
                4: "RECG_ERR_CUDA", 5: "RECG_ERR_TIMEOUT", 6: "RECG_ERR_INTERNAL"}


class RecgError(RuntimeError):
    def __init__(self, status: int, text: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {text}")
        self.status = status


class recg_config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "hidden", "n_q_heads", "n_kv_heads", "head_dim", "ffn", "vocab")] + \
               [("rope_base", C.c_float), ("rms_eps", C.c_float)] + \
               [(n, C.c_int32) for n in ("mask_token_id", "page_size", "max_requests", "max_tokens",
                                         "max_pages_per_request", "flags")]


class recg_weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("final_norm", C.c_void_p), ("lm_head", C.c_void_p)] + \
               [(n, C.POINTER(C.c_void_p)) for n in ("attn_norm", "wqkv", "wo", "ffn_norm", "w_gate_up", "w_down")]


class recg_batch(C.Structure):
    _fields_ = [("n_req", C.c_int32), ("ctx_len", C.c_void_p), ("verify_len", C.c_void_p), ("block_size", C.c_void_p),
                ("verify_tokens", C.c_void_p), ("page_table", C.c_void_p), ("page_table_stride", C.c_int32),
                ("kv_pool", C.c_void_p), ("kv_pool_pages", C.c_int64), ("n_corr", C.c_void_p),
                ("corr_index", C.c_void_p), ("corr_token", C.c_void_p), ("corr_block", C.c_void_p),
                ("risk_delta", C.c_float)]


class recg_logits(C.Structure):
    _fields_ = [("data", C.c_void_p), ("dtype", C.c_int32), ("n_rows", C.c_int32), ("vocab", C.c_int32)]


_INT_OUT = ("accept_len", "n_emitted", "emitted", "new_ctx_len", "slot_state", "freed_pages", "next_draft", "cont_hit",
            "top1", "top2")
_FLT_OUT = ("p1", "p2", "entropy", "entropy_mean")
_INT_OUT_BRANCH = ("corr_hit", "risky_n", "risky_index", "risky_token", "freed_page_ids")


class recg_verify_out(C.Structure):
    _fields_ = [("mem", C.c_int32)] + [(n, C.c_void_p) for n in _INT_OUT + _FLT_OUT + _INT_OUT_BRANCH]


class recg_policy_table(C.Structure):
    _fields_ = [("n_blocks", C.c_int32), ("n_bins", C.c_int32), ("blocks", C.c_void_p), ("s_edges", C.c_void_p),
                ("value", C.c_void_p), ("cost", C.c_void_p)]


class recg_policy_state(C.Structure):
    _fields_ = [("e1", C.c_void_p), ("e2", C.c_void_p), ("block_index", C.c_void_p), ("full", C.c_void_p)]


class recg_device_batch(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_req", "max_verify", "page_table_stride", "rows_hint")] + \
               [(n, C.c_void_p) for n in ("ctx_len", "verify_len", "block_size", "verify_tokens", "page_table", "kv_pool")] + \
               [("kv_pool_pages", C.c_int64)]


class recg_round_log(C.Structure):
    _fields_ = [("tokens", C.c_void_p), ("n_tokens", C.c_void_p), ("max_tokens_per_request", C.c_int32), ("max_rounds", C.c_int32),
                ("accept_len", C.c_void_p), ("block_size", C.c_void_p), ("verify_len", C.c_void_p), ("n_rounds", C.c_void_p),
                ("entropy_mean", C.c_void_p)]


_lib = None


def lib() -> C.CDLL:
    """Load librecg.so (built in-tree by __graft_entry__.build()); raises if it is absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not found: build it with `python -c 'import __graft_entry__ as g; g.build()'`")
        L = C.CDLL(LIB_PATH)
        L.recg_kv_pool_bytes.restype = C.c_size_t
        L.recg_kv_pool_bytes.argtypes = [C.POINTER(recg_config), C.c_int64]
        L.recg_last_error.restype = C.c_char_p
        L.recg_last_error.argtypes = [C.c_void_p]
        L.recg_init.argtypes = [C.POINTER(C.c_void_p), C.POINTER(recg_config), C.POINTER(recg_weights), C.c_void_p]
        L.recg_step.argtypes = [C.c_void_p, C.POINTER(recg_batch), C.POINTER(recg_logits)]
        L.recg_verify.argtypes = [C.c_void_p, C.POINTER(recg_batch), C.c_void_p, C.c_int32, C.POINTER(recg_verify_out)]
        L.recg_attention.argtypes = [C.c_void_p, C.POINTER(recg_batch), C.c_int32, C.c_void_p, C.c_void_p]
        kvio = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p,
                C.c_void_p]
        L.recg_kv_write.argtypes = kvio
        L.recg_kv_read.argtypes = kvio
        L.recg_linear.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32]
        L.recg_debug_buffer.argtypes = [C.c_void_p, C.c_int32, C.POINTER(C.c_void_p), C.POINTER(C.c_int32),
                                        C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        L.recg_sync.argtypes = [C.c_void_p]
        L.recg_row_stats_static.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32] + [C.c_void_p] * 6
        L.recg_row_stats_static.restype = C.c_int32
        L.recg_row_stats_static_error.restype = C.c_char_p
        L.recg_timing_enable.argtypes = [C.c_void_p, C.c_int32]
        L.recg_timing_read.argtypes = [C.c_void_p, C.POINTER(C.c_float), C.POINTER(C.c_int32)]
        L.recg_policy_load.argtypes = [C.c_void_p, C.POINTER(recg_policy_table)]
        L.recg_policy_step.argtypes = [C.c_void_p, C.POINTER(recg_policy_state), C.c_void_p, C.c_void_p, C.c_void_p]
        L.recg_free.argtypes = [C.c_void_p]
        L.recg_step_device.argtypes = [C.c_void_p, C.POINTER(recg_device_batch), C.POINTER(recg_logits)]
        L.recg_next_round.argtypes = [C.c_void_p, C.POINTER(recg_device_batch), C.c_void_p, C.c_void_p, C.POINTER(recg_round_log),
                                      C.c_int32]
        L.recg_debug_gemm_config.argtypes = [C.c_void_p, C.c_int32, C.c_int32]
        L.recg_debug_wait_timeout.argtypes = [C.c_void_p, C.c_int32]
        L.recg_debug_map_cache_selftest.argtypes = [C.c_int32, C.POINTER(C.c_int32)]
        L.recg_debug_map_cache_selftest.restype = C.c_int32
        for f in ("recg_init", "recg_step", "recg_verify", "recg_attention", "recg_kv_write", "recg_kv_read",
                  "recg_linear", "recg_debug_buffer", "recg_sync", "recg_free", "recg_timing_enable", "recg_timing_read",
                  "recg_policy_load", "recg_policy_step", "recg_debug_gemm_config", "recg_debug_wait_timeout",
                  "recg_step_device", "recg_next_round"):
            getattr(L, f).restype = C.c_int32
        _lib = L
    return _lib


EXPORTS = ("recg_kv_pool_bytes", "recg_init", "recg_step", "recg_verify", "recg_attention", "recg_kv_write",
           "recg_kv_read", "recg_linear", "recg_debug_buffer", "recg_sync", "recg_free", "recg_last_error",
           "recg_timing_enable", "recg_timing_read", "recg_row_stats_static", "recg_row_stats_static_error",
           "recg_policy_load", "recg_policy_step", "recg_debug_gemm_config", "recg_debug_wait_timeout",
           "recg_debug_map_cache_selftest", "recg_step_device", "recg_next_round")
TIMING_CLASSES = ("layout", "rmsnorm", "gemm_qkv", "attention", "gemm_o", "gemm_gate_up", "gemm_down", "lm_head", "verify")


def make_config(shape, max_requests: int, max_tokens: int, max_pages_per_request: int, flags: int = 0,
                page_size: int = 16) -> recg_config:
    """shape: any object with the model fields (n_layers, hidden, n_q_heads, ...)."""
    return recg_config(shape.n_layers, shape.hidden, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.ffn,
                       shape.vocab, float(shape.rope_base), float(shape.rms_eps), int(shape.mask_token_id), page_size,
                       max_requests, max_tokens, max_pages_per_request, flags)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _ptr(a) -> Optional[int]:
    if a is None:
        return None
    if isinstance(a, torch.Tensor):
        return a.data_ptr()
    return a.ctypes.data


class Batch:
    """Holds the host arrays of one recg_batch alive and exposes the C struct."""

    def __init__(self, ctx_len, verify_len, block_size, verify_tokens=None, page_table=None, kv_pool=None,
                 kv_pool_pages: int = 0, n_corr=None, corr_index=None, corr_token=None, corr_block=None,
                 risk_delta: float = 0.0):
        """n_corr [C], corr_index / corr_token [C, 2], corr_block [C]: the correction branches (all None = none)."""
        self.ctx_len, self.verify_len, self.block_size = _i32(ctx_len), _i32(verify_len), _i32(block_size)
        self.verify_tokens = _i32(verify_tokens) if verify_tokens is not None else np.zeros(0, np.int32)
        self.page_table = None if page_table is None else _i32(page_table)
        self.kv_pool = kv_pool
        stride = 0 if self.page_table is None else int(self.page_table.shape[1])
        self.n_req = len(self.ctx_len)
        self.n_corr = None if n_corr is None else _i32(n_corr)
        self.corr_index = None if n_corr is None else _i32(corr_index).reshape(self.n_req, 2)
        self.corr_token = None if n_corr is None else _i32(corr_token).reshape(self.n_req, 2)
        self.corr_block = None if n_corr is None else _i32(corr_block)
        self.c = recg_batch(len(self.ctx_len), _ptr(self.ctx_len), _ptr(self.verify_len), _ptr(self.block_size),
                            _ptr(self.verify_tokens) if self.verify_tokens.size else None, _ptr(self.page_table),
                            stride, _ptr(kv_pool), int(kv_pool_pages), _ptr(self.n_corr), _ptr(self.corr_index),
                            _ptr(self.corr_token), _ptr(self.corr_block), float(risk_delta))
        self.rows = self.verify_len + self.block_size          # rows of each request in the ragged batch
        if self.n_corr is not None:
            self.rows = self.rows + self.n_corr * (1 + self.corr_block)
        self.n_tok = int(self.rows.sum())
        self.n_ver = int(self.verify_len.sum())


class DeviceBatch:
    """A recg_device_batch: the descriptor arrays as CUDA int32 tensors that recg_next_round rewrites in place."""

    def __init__(self, ctx_len, verify_len, block_size, verify_tokens, max_verify: int, page_table, kv_pool, kv_pool_pages: int,
                 rows_hint: int = 0):
        """verify_tokens: per request a list of its y (padded here to max_verify)."""
        self.n_req = len(ctx_len)
        dev = kv_pool.device
        i32 = lambda a: torch.as_tensor(np.asarray(a, dtype=np.int32), device=dev).contiguous()
        self.ctx_len, self.verify_len, self.block_size = i32(ctx_len), i32(verify_len), i32(block_size)
        vt = np.zeros((self.n_req, max_verify), dtype=np.int32)
        for r, y in enumerate(verify_tokens):
            vt[r, :len(y)] = y
        self.verify_tokens = i32(vt)
        self.page_table = i32(page_table)
        self.kv_pool = kv_pool
        self.c = recg_device_batch(self.n_req, max_verify, int(self.page_table.shape[1]), rows_hint, self.ctx_len.data_ptr(),
                                   self.verify_len.data_ptr(), self.block_size.data_ptr(), self.verify_tokens.data_ptr(),
                                   self.page_table.data_ptr(), kv_pool.data_ptr(), int(kv_pool_pages))


class RoundLog:
    """Device logs of a run of device-resident rounds."""

    def __init__(self, n_req: int, max_rounds: int, max_tokens_per_request: int, device="cuda"):
        z = lambda *shape: torch.zeros(shape, dtype=torch.int32, device=device)
        self.tokens, self.n_tokens = z(n_req, max_tokens_per_request), z(n_req)
        self.accept_len, self.block_size, self.verify_len = z(max_rounds, n_req), z(max_rounds, n_req), z(max_rounds, n_req)
        self.n_rounds = z(1)
        self.entropy_mean = torch.zeros((max_rounds, n_req), dtype=torch.float32, device=device)
        self.c = recg_round_log(self.tokens.data_ptr(), self.n_tokens.data_ptr(), max_tokens_per_request, max_rounds,
                                self.accept_len.data_ptr(), self.block_size.data_ptr(), self.verify_len.data_ptr(),
                                self.n_rounds.data_ptr(), self.entropy_mean.data_ptr())


class VerifyOut:
    """Caller-provided result buffers of recg_verify (host numpy arrays or CUDA tensors)."""

    def __init__(self, n_req: int, n_tok: int, n_ver: int, host: bool = True):
        self.sizes = {"accept_len": n_req, "n_emitted": n_req, "emitted": n_ver, "new_ctx_len": n_req,
                      "slot_state": n_tok, "freed_pages": n_req, "next_draft": n_tok - n_ver, "cont_hit": n_req,
                      "top1": n_tok, "top2": n_tok, "p1": n_tok, "p2": n_tok, "entropy": n_tok, "entropy_mean": n_req,
                      "corr_hit": 2 * n_req, "risky_n": 3 * n_req, "risky_index": 6 * n_req, "risky_token": 6 * n_req,
                      "freed_page_ids": n_tok}
        self.bufs = {}
        self.c = recg_verify_out()
        self.c.mem = MEM_HOST if host else MEM_DEVICE
        for name, n in self.sizes.items():
            isf = name in _FLT_OUT
            if host:
                self.bufs[name] = np.zeros(max(n, 1), dtype=np.float32 if isf else np.int32)
            else:
                self.bufs[name] = torch.zeros(max(n, 1), dtype=torch.float32 if isf else torch.int32, device="cuda")
            setattr(self.c, name, _ptr(self.bufs[name]))

    def views(self):
        return {k: v[:self.sizes[k]] for k, v in self.bufs.items()}

    def nbytes(self) -> int:
        return 4 * sum(self.sizes.values())


class Context:
    """recg_ctx wrapper.  weights: dict of CUDA bf16 tensors as produced by synth.model_weights."""

    def __init__(self, cfg: recg_config, weights: Optional[Dict[str, object]] = None, stream: Optional[int] = None):
        if not torch.cuda.is_available():
            raise RuntimeError("recg needs a CUDA device (there is no CPU fallback)")
        self.cfg = cfg
        self._keep = weights
        self.h = C.c_void_p()
        wptr = None
        if weights is not None:
            n = cfg.n_layers
            arrs = {}
            for k in ("attn_norm", "wqkv", "wo", "ffn_norm", "w_gate_up", "w_down"):
                arrs[k] = (C.c_void_p * max(n, 1))(*[t.data_ptr() for t in weights[k]])
            self._arrs = arrs
            self._w = recg_weights(weights["embed"].data_ptr(), weights["final_norm"].data_ptr(),
                                   weights["lm_head"].data_ptr(), *[C.cast(arrs[k], C.POINTER(C.c_void_p)) for k in
                                                                    ("attn_norm", "wqkv", "wo", "ffn_norm", "w_gate_up",
                                                                     "w_down")])
            wptr = C.byref(self._w)
        self.stream = torch.cuda.current_stream().cuda_stream if stream is None else stream
        st = lib().recg_init(C.byref(self.h), C.byref(cfg), wptr, C.c_void_p(self.stream))
        if st != RECG_OK:
            raise RecgError(st, lib().recg_last_error(None).decode())

    def _check(self, st: int):
        if st != RECG_OK:
            raise RecgError(st, lib().recg_last_error(self.h).decode())

    def kv_pool_bytes(self, n_pages: int) -> int:
        return lib().recg_kv_pool_bytes(C.byref(self.cfg), n_pages)

    def recg_step(self, batch: Batch):
        """Returns a torch view [T, vocab] of the library-owned logits (valid until the next step)."""
        lg = recg_logits()
        self._check(lib().recg_step(self.h, C.byref(batch.c), C.byref(lg)))
        return lg

    def logits_tensor(self, lg: recg_logits) -> torch.Tensor:
        """Copy of the logits view as a torch tensor (device to device)."""
        dt = torch.bfloat16 if lg.dtype == DTYPE_BF16 else torch.float32
        return device_view(lg.data, (lg.n_rows, lg.vocab), dt).clone()

    def recg_verify(self, batch: Optional[Batch], logits: Optional[torch.Tensor] = None, host: bool = True,
                    n_req: Optional[int] = None, n_tok: Optional[int] = None, n_ver: Optional[int] = None,
                    out: Optional["VerifyOut"] = None):
        """Runs verification; returns a dict of numpy arrays (host=True) or CUDA tensors.  Pass a
        preallocated VerifyOut to avoid allocating the result buffers on every call."""
        if out is None:
            C_ = batch.n_req if batch is not None else n_req
            T = batch.n_tok if batch is not None else n_tok
            Tv = batch.n_ver if batch is not None else n_ver
            out = VerifyOut(C_, T, Tv, host)
        dt = 0
        lp = None
        if logits is not None:
            dt = DTYPE_BF16 if logits.dtype == torch.bfloat16 else DTYPE_F32
            lp = logits.data_ptr()
        self._check(lib().recg_verify(self.h, C.byref(batch.c) if batch is not None else None, lp, dt, C.byref(out.c)))
        return out.views()

    def recg_attention(self, batch: Optional[Batch], layer: int, q: torch.Tensor, o: torch.Tensor):
        self._check(lib().recg_attention(self.h, C.byref(batch.c) if batch is not None else None, layer, q.data_ptr(),
                                         o.data_ptr()))

    def recg_kv_write(self, pool: torch.Tensor, n_pages: int, layer: int, page_row, pos0: int, k: torch.Tensor,
                      v: torch.Tensor):
        row = _i32(page_row)
        self._check(lib().recg_kv_write(self.h, pool.data_ptr(), n_pages, layer, _ptr(row), len(row), pos0, k.shape[0],
                                        k.data_ptr(), v.data_ptr()))

    def recg_kv_read(self, pool: torch.Tensor, n_pages: int, layer: int, page_row, pos0: int, n_pos: int):
        row = _i32(page_row)
        k = torch.empty((n_pos, self.cfg.n_kv_heads, self.cfg.head_dim), dtype=torch.bfloat16, device="cuda")
        v = torch.empty_like(k)
        self._check(lib().recg_kv_read(self.h, pool.data_ptr(), n_pages, layer, _ptr(row), len(row), pos0, n_pos,
                                       k.data_ptr(), v.data_ptr()))
        return k, v

    def recg_linear(self, x: torch.Tensor, w: torch.Tensor, out_dtype=torch.float32) -> torch.Tensor:
        M, K = x.shape
        N = w.shape[0]
        y = torch.empty((M, N), dtype=out_dtype, device="cuda")
        self._check(lib().recg_linear(self.h, x.data_ptr(), w.data_ptr(), y.data_ptr(), M, N, K,
                                      DTYPE_BF16 if out_dtype == torch.bfloat16 else DTYPE_F32))
        return y

    def recg_policy_load(self, blocks, s_edges, value, cost):
        """Host arrays of the block-size rule: blocks [nb], s_edges [n_bins-1], value [nb, n_bins, nb, 2], cost [nb]."""
        b = _i32(blocks)
        e = np.ascontiguousarray(np.asarray(s_edges, dtype=np.float32))
        v = np.ascontiguousarray(np.asarray(value, dtype=np.float32))
        c = np.ascontiguousarray(np.asarray(cost, dtype=np.float32))
        n_bins = e.size + 1
        if v.shape != (b.size, n_bins, b.size, 2) or c.size != b.size:
            raise ValueError("value must be [n_blocks, n_bins, n_blocks, 2] and cost [n_blocks]")
        t = recg_policy_table(b.size, n_bins, _ptr(b), _ptr(e) if e.size else None, _ptr(v), _ptr(c))
        self._check(lib().recg_policy_load(self.h, C.byref(t)))

    def recg_policy_step(self, state: Dict[str, torch.Tensor], next_block: torch.Tensor,
                         entropy_mean: Optional[torch.Tensor] = None, accept_len: Optional[torch.Tensor] = None):
        """state: CUDA tensors e1, e2 (float32), block_index, full (int32), updated in place; next_block: CUDA int32."""
        st = recg_policy_state(state["e1"].data_ptr(), state["e2"].data_ptr(), state["block_index"].data_ptr(),
                               state["full"].data_ptr())
        self._check(lib().recg_policy_step(self.h, C.byref(st), _ptr(entropy_mean), _ptr(accept_len),
                                           next_block.data_ptr()))

    def recg_debug_buffer(self, which: int) -> torch.Tensor:
        p, dt, r, c = C.c_void_p(), C.c_int32(), C.c_int32(), C.c_int32()
        self._check(lib().recg_debug_buffer(self.h, which, C.byref(p), C.byref(dt), C.byref(r), C.byref(c)))
        return device_view(p.value, (r.value, c.value),
                           torch.bfloat16 if dt.value == DTYPE_BF16 else torch.float32).clone()

    def recg_step_device(self, batch: "DeviceBatch"):
        lg = recg_logits()
        self._check(lib().recg_step_device(self.h, C.byref(batch.c), C.byref(lg)))
        return lg

    def recg_verify_device(self):
        """Verification of the last recg_step_device into the library's own device buffers (nothing is copied)."""
        out = recg_verify_out()
        out.mem = MEM_DEVICE
        self._check(lib().recg_verify(self.h, None, None, 0, C.byref(out)))

    def recg_next_round(self, batch: "DeviceBatch", round_index: int, next_block: Optional[torch.Tensor] = None,
                        planted_emitted: Optional[torch.Tensor] = None, log: Optional["RoundLog"] = None):
        self._check(lib().recg_next_round(self.h, C.byref(batch.c), _ptr(next_block), _ptr(planted_emitted),
                                          C.byref(log.c) if log is not None else None, int(round_index)))

    def recg_debug_gemm_config(self, tile: int, stream_k: int):
        self._check(lib().recg_debug_gemm_config(self.h, int(tile), int(stream_k)))

    def recg_debug_wait_timeout(self, max_polls: int):
        self._check(lib().recg_debug_wait_timeout(self.h, int(max_polls)))

    def recg_timing_enable(self, enable: bool):
        self._check(lib().recg_timing_enable(self.h, 1 if enable else 0))

    def recg_timing_read(self):
        """Returns ({class: ms}, {class: launches}) accumulated since the last read."""
        ms = (C.c_float * len(TIMING_CLASSES))()
        ln = (C.c_int32 * len(TIMING_CLASSES))()
        self._check(lib().recg_timing_read(self.h, ms, ln))
        return dict(zip(TIMING_CLASSES, list(ms))), dict(zip(TIMING_CLASSES, list(ln)))

    def recg_sync(self):
        self._check(lib().recg_sync(self.h))

    def recg_free(self):
        if self.h:
            lib().recg_free(self.h)
            self.h = C.c_void_p()

    def __del__(self):
        try:
            self.recg_free()
        except Exception:
            pass


class _DevView:
    """Zero-copy torch view of library-owned device memory through the CUDA array interface."""

    def __init__(self, ptr: int, shape, dtype):
        ts = "<f4" if dtype == torch.float32 else "<i2"
        self.__cuda_array_interface__ = {"shape": tuple(shape), "typestr": ts, "data": (int(ptr), False), "version": 3}


def device_view(ptr: int, shape, dtype) -> torch.Tensor:
    t = torch.as_tensor(_DevView(ptr, shape, dtype), device="cuda")
    return t.view(torch.bfloat16) if dtype == torch.bfloat16 else t


def alloc_kv_pool(ctx: Context, n_pages: int, fill: Optional[str] = "zero") -> torch.Tensor:
    """Caller-owned pool as a flat bf16 CUDA tensor of the size the library asks for."""
    n = ctx.kv_pool_bytes(n_pages) // 2
    if fill == "normal":
        pool = torch.empty(n, dtype=torch.bfloat16, device="cuda")
        step = 1 << 28
        g = torch.Generator(device="cuda")
        g.manual_seed(2)
        for i in range(0, n, step):
            m = min(step, n - i)
            pool[i:i + m] = torch.randn(m, generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
        return pool
    if fill == "zero":
        return torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    return torch.empty(n, dtype=torch.bfloat16, device="cuda")


def recg_row_stats_static(logits: torch.Tensor, stream: Optional[int] = None):
    """Per-row statistics through the entry point that allocates nothing inside the library (the result
    tensors below are the CALLER's buffers).  For callers that must not trigger a device allocation:
    see include/recg.h.  Returns a dict of CUDA tensors; does not synchronise."""
    rows, vocab = logits.shape
    out = {"top1": torch.empty(rows, dtype=torch.int32, device=logits.device),
           "top2": torch.empty(rows, dtype=torch.int32, device=logits.device),
           "p1": torch.empty(rows, dtype=torch.float32, device=logits.device),
           "p2": torch.empty(rows, dtype=torch.float32, device=logits.device),
           "entropy": torch.empty(rows, dtype=torch.float32, device=logits.device)}
    st = torch.cuda.current_stream().cuda_stream if stream is None else stream
    rc = lib().recg_row_stats_static(logits.data_ptr(), DTYPE_BF16 if logits.dtype == torch.bfloat16 else DTYPE_F32,
                                     rows, vocab, out["top1"].data_ptr(), out["top2"].data_ptr(), out["p1"].data_ptr(),
                                     out["p2"].data_ptr(), out["entropy"].data_ptr(), C.c_void_p(st))
    if rc != RECG_OK:
        raise RecgError(rc, lib().recg_row_stats_static_error().decode())
    return out
