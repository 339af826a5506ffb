"""CPU-only checks of the boundary: the shared library builds, loads, and exports every declared symbol."""
import ctypes
import os
import re

from paper_2605_09649_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "trimkv.h")).read()
    return sorted(set(re.findall(r"TRIMKV_API\s+[\w\s\*]+?\b(trimkv_\w+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build()
    assert os.path.exists(path)
    lib = ctypes.CDLL(path)
    names = _declared()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), f"{n} declared in trimkv.h but not exported"
    assert sorted(binding.EXPORTS) == names


def test_binding_declares_signatures_without_a_gpu():
    L = binding.lib()
    assert L.trimkv_last_error() is not None
    assert binding.select_workspace_bytes(1 << 20) >= 16384 * 16
    assert binding.kernel_launches() >= 0
    cfg = binding.Config()
    L.trimkv_default_config(ctypes.byref(cfg), 1024, 4, 2, 128)
    assert (cfg.budget_entries, cfg.layers, cfg.kv_heads, cfg.q_heads, cfg.head_dim) == (1024, 4, 2, 2, 128)
    assert (cfg.page_size, cfg.gate_hidden, cfg.horizon, cfg.max_batch) == (64, 512, 2, 1)
