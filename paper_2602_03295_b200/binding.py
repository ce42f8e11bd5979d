"""ctypes binding of libpop_b200.so (the C ABI declared in include/pop.h and include/pop_kernels.h).

Argument marshalling only: tensors are torch CUDA tensors used as device memory; every step runs
in the library's kernels. There is no fallback: if the shared library is missing or does not load,
`lib()` raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

from . import _build

POP_OK = 0
POP_E_INVALID = -1
POP_E_NOSPACE = -2
POP_E_CUDA = -3
POP_E_DEVICE_TIMEOUT = -4
POP_E_MISSING = -5


class PopError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: status {code}")
        self.code = code


class pop_config_t(C.Structure):
    _fields_ = [("struct_size", C.c_uint32),
                ("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_q_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("d_ffn", C.c_int32), ("vocab", C.c_int32),
                ("rms_eps", C.c_float), ("rope_theta", C.c_float),
                ("act", C.c_int32), ("qk_norm", C.c_int32), ("post_norms", C.c_int32),
                ("window", C.c_int32), ("global_every", C.c_int32)]


class pop_tensor_t(C.Structure):
    _fields_ = [("name", C.c_char_p), ("dev_ptr", C.c_void_p), ("dtype", C.c_int32), ("ndim", C.c_int32),
                ("shape", C.c_int64 * 2)]


class pop_kv_cache_t(C.Structure):
    _fields_ = [("k_pool", C.c_void_p), ("v_pool", C.c_void_p), ("block_table", C.c_void_p),
                ("page_size", C.c_int32), ("num_pages", C.c_int32), ("max_pages_per_seq", C.c_int32)]


class pop_input_t(C.Structure):
    _fields_ = [("tokens", C.c_void_p), ("embeds", C.c_void_p)]


# name -> (restype, argtypes); every symbol declared in include/*.h
_I32, _I64, _P, _F = C.c_int32, C.c_int64, C.c_void_p, C.c_float
SIGNATURES = {
    "pop_weight_arena_bytes": (C.c_size_t, [C.POINTER(pop_config_t)]),
    "pop_load_weights": (C.c_int, [C.POINTER(pop_config_t), C.POINTER(pop_tensor_t), _I32, _P, C.c_size_t, _P,
                                   C.POINTER(_P)]),
    "pop_workspace_bytes": (C.c_size_t, [_P, _I32, _I32]),
    "pop_set_workspace": (C.c_int, [_P, _P, C.c_size_t]),
    "pop_prefill": (C.c_int, [_P, C.POINTER(pop_input_t), _I32, _I32, _I32, C.POINTER(pop_kv_cache_t), _P, _P]),
    "pop_full_prefill": (C.c_int, [_P, C.POINTER(pop_input_t), _I32, _I32, C.POINTER(pop_kv_cache_t), _P, _P]),
    "pop_last_status": (C.c_int, [_P, _P]),
    "pop_last_launch_count": (_I64, [_P]),
    "pop_free": (None, [_P]),
    "pop_strerror": (C.c_char_p, [C.c_int]),
    "pop_k_gemm": (C.c_int, [_P, _I64, _I64, _P, _I64, _I64, _P, _I64, _I64, _I32, _I32, _I32, _I32, _I32, _I32,
                             _I32, _P]),
    "pop_k_status": (C.c_int, [_P]),
    "pop_k_launch_count": (_I64, []),
    "pop_k_reset_launch_count": (None, []),
}


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


class PopLibrary:
    """The loaded shared library with typed entry points."""

    def __init__(self, path: Optional[str] = None):
        path = path or _build.LIB_PATH
        if not os.path.exists(path):
            raise ImportError(f"{path} is missing: build it with __graft_entry__.build() "
                              "(nvcc, sm_100a); there is no fallback path")
        self.path = path
        self.dll = C.CDLL(path)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(self.dll, name)   # AttributeError if the symbol is not exported
            fn.restype, fn.argtypes = res, args

    # -------------------------------------------------------------- helpers
    def check(self, code: int, what: str):
        if code != POP_OK:
            msg = self.dll.pop_strerror(code)
            raise PopError(code, f"{what} ({msg.decode() if msg else '?'})")

    def status(self, stream=None) -> int:
        return self.dll.pop_k_status(_stream_ptr(stream))

    def launch_count(self) -> int:
        return self.dll.pop_k_launch_count()

    def reset_launch_count(self):
        self.dll.pop_k_reset_launch_count()

    # -------------------------------------------------------------- kernel-level calls
    def gemm(self, A: torch.Tensor, B: torch.Tensor, out: torch.Tensor, epilogue: int = 0, act: int = 0,
             n_valid: int = 0, stream=None):
        """out = epilogue(A @ B^T). A [M,K] or [G,M,K] bf16, B [N,K] or [G,N,K] bf16 (inner dim contiguous)."""
        if A.dim() == 2:
            A, B, out3 = A.unsqueeze(0), B.unsqueeze(0), out.unsqueeze(0)
        else:
            out3 = out
        G, M, K = A.shape
        N = B.shape[1]
        assert A.stride(2) == 1 and B.stride(2) == 1 and out3.stride(2) == 1
        code = self.dll.pop_k_gemm(A.data_ptr(), A.stride(1), A.stride(0) if G > 1 else 0,
                                   B.data_ptr(), B.stride(1), B.stride(0) if G > 1 else 0,
                                   out3.data_ptr(), out3.stride(1), out3.stride(0) if G > 1 else 0,
                                   M, N, K, G, epilogue, act, n_valid, _stream_ptr(stream))
        self.check(code, "pop_k_gemm")
        return out


class PopModel:
    """Placeholder until the model-level calls are bound (see PopLibrary for kernel-level calls)."""


_LIB: Optional[PopLibrary] = None


def lib() -> PopLibrary:
    """The process-wide library handle; raises if the CUDA extension is not built."""
    global _LIB
    if _LIB is None:
        _LIB = PopLibrary()
    return _LIB
