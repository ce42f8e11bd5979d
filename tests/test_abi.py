"""The C-ABI library without a GPU: it loads, exports every symbol the public headers declare,
and its host-side argument checks reject bad calls before any device work."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def library():
    from paper_2602_03295_b200 import _build, binding
    _build.build()
    return binding.PopLibrary()


def declared_symbols():
    names = set()
    for h in ("pop.h", "pop_kernels.h"):
        text = open(os.path.join(ROOT, "include", h)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(pop_[a-z0-9_]+)\s*\(", text))
    return names


def test_every_declared_symbol_is_exported_and_bound(library):
    from paper_2602_03295_b200 import binding
    syms = declared_symbols()
    assert len(syms) >= 18
    for s in syms:
        assert hasattr(library.dll, s), f"{s} declared in include/ but not exported"
    assert syms == set(binding.SIGNATURES), syms ^ set(binding.SIGNATURES)


def test_missing_library_fails_loudly(tmp_path):
    from paper_2602_03295_b200 import binding
    with pytest.raises(ImportError):
        binding.PopLibrary(str(tmp_path / "nope.so"))


def test_strerror_and_config_validation(library):
    from paper_2602_03295_b200 import binding
    import pop_synth as ps
    assert library.dll.pop_strerror(0) == b"ok"
    assert b"invalid" in library.dll.pop_strerror(binding.POP_E_INVALID)
    cfg = binding.make_config(ps.C2_LLAMA8B)
    n = library.dll.pop_weight_arena_bytes(C.byref(cfg))
    params = 32 * 218_112_000 + 2 * 128256 * 4096
    assert 2 * params <= n < 2 * params * 1.01
    cfg.struct_size = 12
    assert library.dll.pop_weight_arena_bytes(C.byref(cfg)) == 0
    bad = binding.make_config(ps.C1_TINY.replace(head_dim=80))
    assert library.dll.pop_weight_arena_bytes(C.byref(bad)) == 0
    bad = binding.make_config(ps.C1_TINY.replace(n_q_heads=3))
    assert library.dll.pop_weight_arena_bytes(C.byref(bad)) == 0


def test_null_and_misaligned_arguments_are_rejected_on_the_host(library):
    from paper_2602_03295_b200 import binding
    import pop_synth as ps
    d = library.dll
    assert d.pop_k_gemm(None, 8, 0, None, 8, 0, None, 8, 0, 128, 128, 64, 1, 0, 0, 0, None) == binding.POP_E_INVALID
    assert d.pop_k_gemm(1024, 8, 0, 2048, 8, 0, 4096, 8, 0, 128, 128, 60, 1, 0, 0, 0, None) == binding.POP_E_INVALID
    assert d.pop_k_attention(None, 0, None, None, None, None, 0, 1, 1, 0, 1, 1, 1, 64, 16, 1, 1, 0, None) \
        == binding.POP_E_INVALID
    assert d.pop_k_gemv(None, 0, 0, None, 0, None, 0, 1, 1, 8, 0, 0, 0, None) == binding.POP_E_INVALID
    cfg = binding.make_config(ps.C1_TINY)
    out = C.c_void_p()
    assert d.pop_load_weights(C.byref(cfg), None, 0, None, 0, None, C.byref(out)) == binding.POP_E_INVALID
    assert d.pop_prefill(None, None, 1, 1, 1, None, None, None) == binding.POP_E_INVALID
    assert d.pop_full_prefill(None, None, 1, 1, None, None, None) == binding.POP_E_INVALID
    assert d.pop_workspace_bytes(None, 8, 1) == 0
    assert d.pop_set_workspace(None, None, 0) == binding.POP_E_INVALID
    assert d.pop_last_launch_count(None) == 0
    d.pop_free(None)
