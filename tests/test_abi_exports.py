"""The C-ABI library loads and exports every symbol the public header declares (no GPU, no compute)."""
import ctypes
import os
import re


def test_library_exports_every_declared_symbol(repo_root):
    lib_path = os.path.join(repo_root, "paper_2511_18793_b200", "libnezha.so")
    if not os.path.exists(lib_path):
        from paper_2511_18793_b200 import build
        build.build()
    header = open(os.path.join(repo_root, "include", "nezha.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = sorted(set(re.findall(r"\b(nezha_[a-z_0-9]+)\s*\(", header)))
    assert len(declared) >= 14
    lib = ctypes.CDLL(lib_path)
    for name in declared:
        assert hasattr(lib, name), name
    from paper_2511_18793_b200 import binding
    assert sorted(binding.EXPORTS) == declared


def test_arena_bytes_rejects_bad_configs_without_a_gpu(repo_root):
    from paper_2511_18793_b200 import binding, synth
    import ctypes as C
    cfg = binding.make_config(synth.WORKLOADS["tiny"])
    assert binding.lib.nezha_arena_bytes(C.byref(cfg), 5000, 0.5) > 0
    assert binding.lib.nezha_arena_bytes(C.byref(cfg), 5000, 1.5) == 0
    cfg.L = 9
    assert binding.lib.nezha_arena_bytes(C.byref(cfg), 5000, 0.5) == 0
    cfg = binding.make_config(synth.WORKLOADS["tiny"])
    cfg.n_kv_heads = 3
    assert binding.lib.nezha_arena_bytes(C.byref(cfg), 5000, 0.5) == 0
    big = binding.make_config(synth.WORKLOADS["7b"])
    gb = binding.lib.nezha_arena_bytes(C.byref(big), 100_000_000, 0.5) / 2 ** 30
    assert 20 < gb < 120          # weights + KV + scratch of the largest workload fit one 180 GB GPU
