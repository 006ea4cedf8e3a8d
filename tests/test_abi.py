"""The C-ABI library loads and exports every entry point the header declares (no GPU needed)."""
import ctypes as C
import os
import re

import torch

from paper_2609_34388_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "recg.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(recg_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported():
    import __graft_entry__ as g

    g.build()
    lib = binding.lib()
    names = declared_symbols()
    assert "recg_init" in names and "recg_step" in names and "recg_verify" in names and "recg_free" in names
    for n in names:
        assert hasattr(lib, n), f"{n} declared in recg.h but not exported"
    assert set(names) == set(binding.EXPORTS)


def test_struct_sizes_match_header_layout(tmp_path):
    # 7 ints, 2 floats, 6 ints
    assert C.sizeof(binding.recg_config) == 15 * 4
    # int + 5 ptr + int + ptr + int64, then 4 ptr + float, with padding
    assert C.sizeof(binding.recg_batch) == 8 * 8 + 8 + 4 * 8 + 8
    assert C.sizeof(binding.recg_verify_out) == 8 + 19 * 8
    # and against the header itself, as the C compiler lays the structs out
    import subprocess
    src = tmp_path / "sizes.c"
    src.write_text('#include <stdio.h>\n#include <stddef.h>\n#include "recg.h"\n'
                   'int main(void) { printf("%zu %zu %zu %zu %zu %zu %zu %zu %zu %zu %zu\\n", sizeof(recg_config), sizeof(recg_batch), '
                   'sizeof(recg_verify_out), offsetof(recg_batch, n_corr), offsetof(recg_batch, risk_delta), '
                   'offsetof(recg_verify_out, corr_hit), offsetof(recg_verify_out, freed_page_ids), sizeof(recg_device_batch), '
                   'offsetof(recg_device_batch, kv_pool_pages), sizeof(recg_round_log), offsetof(recg_round_log, entropy_mean)); '
                   'return 0; }\n')
    exe = tmp_path / "sizes"
    subprocess.run(["gcc", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)], check=True)
    got = [int(t) for t in subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split()]
    want = [C.sizeof(binding.recg_config), C.sizeof(binding.recg_batch), C.sizeof(binding.recg_verify_out),
            binding.recg_batch.n_corr.offset, binding.recg_batch.risk_delta.offset,
            binding.recg_verify_out.corr_hit.offset, binding.recg_verify_out.freed_page_ids.offset,
            C.sizeof(binding.recg_device_batch), binding.recg_device_batch.kv_pool_pages.offset,
            C.sizeof(binding.recg_round_log), binding.recg_round_log.entropy_mean.offset]
    assert got == want


def test_tensor_map_cache_hands_out_copies_across_evictions():
    """More distinct keys than the cache holds, three lookups per simulated launch: a map taken before a later lookup
    of the same launch emptied the cache must still be the right one (host logic only, fake encoder)."""
    lib = binding.lib()
    ev = C.c_int32(0)
    assert lib.recg_debug_map_cache_selftest(3 * 5000, C.byref(ev)) == 0
    assert ev.value >= 3          # 15000 keys through a 4096-entry cache
    assert lib.recg_debug_map_cache_selftest(30, C.byref(ev)) == 0 and ev.value == 0


def test_init_rejects_capacities_the_launches_cannot_serve():
    lib = binding.lib()
    h = C.c_void_p()
    big = binding.recg_config(2, 256, 4, 2, 64, 1024, 2048, 1e4, 1e-5, -1, 16, 5000, 64, 8, 0)     # requests
    assert lib.recg_init(C.byref(h), C.byref(big), None, None) == 3
    big = binding.recg_config(2, 256, 4, 2, 64, 1024, 2048, 1e4, 1e-5, -1, 16, 4, (1 << 20) + 1, 8, 0)   # rows
    assert lib.recg_init(C.byref(h), C.byref(big), None, None) == 3 and b"4096 requests" in lib.recg_last_error(None)


def test_pool_bytes_formula():
    lib = binding.lib()
    cfg = binding.recg_config(32, 4096, 32, 8, 128, 14336, 128256, 5e5, 1e-5, -1, 16, 16, 1024, 600, 0)
    # 2 (K,V) * 8 heads * 128 dims * 2 bytes * 32 layers = 131072 bytes per token
    assert lib.recg_kv_pool_bytes(C.byref(cfg), 10) == 10 * 16 * 131072
    assert lib.recg_kv_pool_bytes(C.byref(cfg), 0) == 0


def test_init_fails_loudly_without_a_device_or_with_bad_config():
    lib = binding.lib()
    h = C.c_void_p()
    bad = binding.recg_config(2, 256, 4, 2, 48, 1024, 2048, 1e4, 1e-5, -1, 16, 4, 64, 8, 0)   # head_dim 48
    st = lib.recg_init(C.byref(h), C.byref(bad), None, None)
    assert st == 2 and b"head_dim" in lib.recg_last_error(None)
    bad = binding.recg_config(2, 256, 4, 2, 64, 1024, 2048, 1e4, 1e-5, -1, 32, 4, 64, 8, 0)   # page size 32
    assert lib.recg_init(C.byref(h), C.byref(bad), None, None) == 2
    assert lib.recg_init(C.byref(h), None, None, None) == 1
    if not torch.cuda.is_available():
        ok = binding.recg_config(2, 256, 4, 2, 64, 1024, 2048, 1e4, 1e-5, -1, 16, 4, 64, 8, 0)
        st = lib.recg_init(C.byref(h), C.byref(ok), None, None)
        assert st == 4 and b"no CPU fallback" in lib.recg_last_error(None)
        try:
            binding.Context(ok)
            assert False, "Context() must raise without a CUDA device"
        except RuntimeError:
            pass


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2609_34388_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.replace("the CPU oracle", "").replace("CPU oracle", ""), f
