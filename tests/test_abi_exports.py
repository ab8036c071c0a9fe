"""The C-ABI library builds, loads without a GPU and exports every function include/pmkvq.h declares;
host-side argument checks that need no device answer as documented."""
import ctypes
import os
import re

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    with open(os.path.join(ROOT, "include", "pmkvq.h")) as f:
        text = re.sub(r"/\*.*?\*/", "", f.read(), flags=re.S)
    return sorted(set(re.findall(r"\b(pmkvq_[a-z0-9_]+)\s*\(", text)))


def test_header_functions_are_exported():
    from paper_2505_18610_b200 import binding
    lib = binding.lib()
    names = _declared_functions()
    assert {"pmkvq_cache_create", "pmkvq_append", "pmkvq_progressive_reduce", "pmkvq_decode_attention"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in pmkvq.h but not exported by libpmkvq.so"


def test_binding_mirrors_the_header():
    """The Python binding sets argument types for every declared function (same names)."""
    from paper_2505_18610_b200 import binding
    lib = binding.lib()
    for n in _declared_functions():
        assert getattr(lib, n).argtypes is not None, f"binding does not marshal {n}"


def test_binding_argument_counts_match_the_prototypes():
    """Every prototype of pmkvq.h has as many parameters as the binding marshals (a drifted signature would
    otherwise pass garbage in the trailing registers)."""
    from paper_2505_18610_b200 import binding
    lib = binding.lib()
    with open(os.path.join(ROOT, "include", "pmkvq.h")) as f:
        text = re.sub(r"/\*.*?\*/", "", f.read(), flags=re.S)
    protos = re.findall(r"\b(pmkvq_[a-z0-9_]+)\s*\(([^()]*)\)\s*;", text)
    assert len(protos) >= 18
    for name, params in protos:
        params = params.strip()
        n = 0 if params in ("", "void") else params.count(",") + 1
        assert len(getattr(lib, name).argtypes) == n, f"{name}: header has {n} parameters"
    # alpha grid search: host-side argument errors are answered before anything touches a device
    a = (ctypes.c_float * 2)(0.0, 0.5)
    out = (ctypes.c_double * 2)()
    one = ctypes.c_void_p(256)
    assert lib.pmkvq_alpha_grid_search(one, one, one, 4, 1, 1, 1, 3, a, 2, 1.0, 10000.0, 1e-5, one, out, None, None) == binding.INVALID_ARG
    assert lib.pmkvq_alpha_grid_search(one, one, one, 4, 1, 1, 1, 2, a, 65, 1.0, 10000.0, 1e-5, one, out, None, None) == binding.INVALID_ARG
    assert lib.pmkvq_alpha_grid_search(one, one, one, 4, 1, 1, 1, 2, a, 2, 1.0, 10000.0, 1e-5, ctypes.c_void_p(8), out, None, None) == binding.INVALID_ARG
    assert lib.pmkvq_alpha_grid_workspace_bytes(0, 1, 1, 1) == 0
    assert lib.pmkvq_alpha_grid_workspace_bytes(2048, 8, 4, 7) >= 2048 * 8 * 4 * 512 * (3 + 7)


def test_host_side_validation_without_a_device():
    from paper_2505_18610_b200 import binding
    lib = binding.lib()
    fbit = (ctypes.c_uint8 * 2)(4, 2)
    cfg = binding._Config()
    cfg.layers, cfg.q_heads, cfg.kv_heads, cfg.head_dim, cfg.batch, cfg.max_tokens = 2, 8, 2, 128, 1, 1024
    cfg.fbit = ctypes.cast(fbit, ctypes.POINTER(ctypes.c_uint8))
    cfg.n_sink, cfg.window, cfg.evict_chunk, cfg.count_metadata = 1, 128, 1, 1
    need = lib.pmkvq_arena_bytes_required(ctypes.byref(cfg))
    # at least the cache itself: 129 INT16 tokens + 895 tokens at Fbit per (K|V, kv head), for both blocks
    floor = sum(2 * 2 * (129 * 264 + 895 * (16 * b + 8)) for b in (4, 2))
    assert need >= floor and need < floor * 4 + (64 << 20)
    cfg.head_dim = 64
    assert lib.pmkvq_arena_bytes_required(ctypes.byref(cfg)) == 0          # head_dim must be 128
    cfg.head_dim, cfg.q_heads = 128, 18
    assert lib.pmkvq_arena_bytes_required(ctypes.byref(cfg)) == 0          # GQA group 9 > 8
    cfg.q_heads = 8
    bad = (ctypes.c_uint8 * 2)(4, 3)
    cfg.fbit = ctypes.cast(bad, ctypes.POINTER(ctypes.c_uint8))
    assert lib.pmkvq_arena_bytes_required(ctypes.byref(cfg)) == 0          # Fbit must be 2, 4, 8 or 16
    h = ctypes.c_void_p()
    cfg.fbit = ctypes.cast(fbit, ctypes.POINTER(ctypes.c_uint8))
    cfg.d_arena = None
    assert lib.pmkvq_cache_create(ctypes.byref(cfg), ctypes.byref(h)) == binding.INVALID_ARG and not h
    assert lib.pmkvq_append(None, 0, None, None, 1, None) == binding.INVALID_ARG
    assert lib.pmkvq_decode_attention(None, 0, None, None, None) == binding.INVALID_ARG
    assert lib.pmkvq_progressive_reduce(None, 0, None) == binding.INVALID_ARG
    assert lib.pmkvq_status_string(binding.BUDGET_FULL).decode().startswith("budget full")
    assert np.isfinite(need)
