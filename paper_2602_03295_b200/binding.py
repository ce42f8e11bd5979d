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
POP_NO_BOUNDARY, POP_NO_INDEP_KV = 1, 2

SIGNATURES = {
    "pop_weight_arena_bytes": (C.c_size_t, [C.POINTER(pop_config_t)]),
    "pop_load_weights": (C.c_int, [C.POINTER(pop_config_t), C.POINTER(pop_tensor_t), _I32, _P, C.c_size_t, _P,
                                   C.POINTER(_P)]),
    "pop_workspace_bytes": (C.c_size_t, [_P, _I32, _I32]),
    "pop_set_workspace": (C.c_int, [_P, _P, C.c_size_t]),
    "pop_prefill": (C.c_int, [_P, C.POINTER(pop_input_t), _I32, _I32, _I32, C.POINTER(pop_kv_cache_t), _P, _P]),
    "pop_full_prefill": (C.c_int, [_P, C.POINTER(pop_input_t), _I32, _I32, C.POINTER(pop_kv_cache_t), _P, _P]),
    "pop_prefill_ragged": (C.c_int, [_P, C.POINTER(pop_input_t), C.POINTER(_I32), _I32, _I32, C.POINTER(pop_kv_cache_t),
                                     _P, _P]),
    "pop_prefill_skip": (C.c_int, [_P, C.POINTER(pop_input_t), _I32, _I32, C.c_char_p, C.POINTER(pop_kv_cache_t), _P,
                                   _P]),
    "pop_fp8_arena_bytes": (C.c_size_t, [_P]),
    "pop_enable_fp8": (C.c_int, [_P, _P, C.c_size_t, _P]),
    "pop_prefill_chunked": (C.c_int, [_P, C.POINTER(pop_input_t), _I32, _I32, _I32, _I32, C.POINTER(pop_kv_cache_t),
                                      _P, _P]),
    "pop_prefill_ablation": (C.c_int, [_P, C.POINTER(pop_input_t), _I32, _I32, C.c_char_p, _I32,
                                       C.POINTER(pop_kv_cache_t), _P, _P]),
    "pop_decode_step": (C.c_int, [_P, _P, _I32, _I32, C.POINTER(pop_kv_cache_t), _P, _P]),
    "pop_decode_step_from": (C.c_int, [_P, _P, _I32, _I32, C.POINTER(_I32), C.POINTER(pop_kv_cache_t), _P, _P]),
    "pop_generate_greedy": (C.c_int, [_P, _P, _I32, _I32, _I32, C.POINTER(pop_kv_cache_t), _P, _P, _P]),
    "pop_read_hidden": (C.c_int, [_P, _I32, _I32, _P, _P, _P]),
    "pop_last_status": (C.c_int, [_P, _P]),
    "pop_last_launch_count": (_I64, [_P]),
    "pop_free": (None, [_P]),
    "pop_strerror": (C.c_char_p, [C.c_int]),
    "pop_k_gemm": (C.c_int, [_P, _I64, _I64, _P, _I64, _I64, _P, _I64, _I64, _I32, _I32, _I32, _I32, _I32, _I32,
                             _I32, _P]),
    "pop_k_gemv_e4m3": (C.c_int, [_P, _I64, _P, _I64, _P, _P, _I64] + [_I32] * 6 + [_P]),
    "pop_k_gemm_e4m3": (C.c_int, [_P, _I64, _P, _P, _I64, _P, _P, _I64, _I32, _I32, _I32, _I32, _I32, _I32, _P]),
    "pop_k_rmsnorm_e4m3": (C.c_int, [_P, _I64, _P, _P, _I64, _P, _I32, _I32, _F, _P]),
    "pop_k_quantize_e4m3": (C.c_int, [_P, _I64, _P, _P, _P, _P]),
    "pop_k_quant_rows_e4m3": (C.c_int, [_P, _I64, _P, _I64, _P, _I32, _I32, _P]),
    "pop_k_gemm_norm": (C.c_int, [_P, _I64, _P, _I64, _P, _I64, _I32, _I32, _I32, _I32, _I32, _I32, _P, _I64, _P, _P, _I32,
                                  _P, _I32, _I32, _I32, _F, _P]),
    "pop_k_gemm_qkv_rope": (C.c_int, [_P, _I64, _I64, _P, _I64, _I64, _I32, _I32, _I32, _P, _I64, _P, _P, _I64, _I32,
                                      _P, _I32, _I32, _P, _P, _I64, _P] + [_I32] * 6 + [_F, _P]),
    "pop_k_attention": (C.c_int, [_P, _I64, _P, _P, _P, _P, _I64] + [_I32] * 11 + [_P]),
    "pop_k_rmsnorm": (C.c_int, [_P, _I64, _P, _I64, _P, _I64, _I64, _I32, _I32, _I32, _F, _I32, _P]),
    "pop_k_rope_table": (C.c_int, [_P, _I32, _I32, _F, _P]),
    "pop_k_rope_cache": (C.c_int, [_P, _I64, _I64, _P, _I64, _P, _P, _I64, _I32, _P, _I32, _I32, _P, _P, _I64, _P]
                         + [_I32] * 8 + [_F, _P]),
    "pop_k_gemv": (C.c_int, [_P, _I64, _I32, _P, _I64, _P, _I64] + [_I32] * 6 + [_P]),
    "pop_k_decode_attention": (C.c_int, [_P, _I64, _P, _P, _P, _I32, _I32, _P, _P, _P, _I64] + [_I32] * 6 + [_P]),
    "pop_k_decode_attention_qkv": (C.c_int, [_P, _I64, _P, _P, C.c_float, _P, _P, _P, _P, _I32, _I32, _I32, _P, _P, _P,
                                             _I64] + [_I32] * 6 + [_P]),
    "pop_k_decode_attention_static": (C.c_int, [_P, _I64, _P, _P, _P, _I32, _I32, _P, _I64] + [_I32] * 6 + [_P]),
    "pop_k_profile": (None, [_I32]),
    "pop_k_profile_summary": (C.c_int, [_I32, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(_I64)]),
    "pop_k_status": (C.c_int, [_P]),
    "pop_k_wait_selftest": (C.c_int, [_I64, _P]),
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

    def wait_selftest(self, limit_cycles: int = 200000, stream=None):
        """Launch the bounded-wait self-test kernel (raises the status word to POP_E_DEVICE_TIMEOUT)."""
        self.check(self.dll.pop_k_wait_selftest(limit_cycles, _stream_ptr(stream)), "pop_k_wait_selftest")

    def launch_count(self) -> int:
        return self.dll.pop_k_launch_count()

    def reset_launch_count(self):
        self.dll.pop_k_reset_launch_count()

    PROF_KINDS = ("gemm", "attention", "elementwise", "gemv", "decode_attention")

    def profile(self, enable: bool):
        self.dll.pop_k_profile(1 if enable else 0)

    def profile_summary(self) -> dict:
        """{kind: (total_ms, total_work, launches)} of the launches recorded since the last call."""
        out = {}
        for i, name in enumerate(self.PROF_KINDS):
            ms, work, n = C.c_double(), C.c_double(), _I64()
            self.check(self.dll.pop_k_profile_summary(i, C.byref(ms), C.byref(work), C.byref(n)),
                       "pop_k_profile_summary")
            out[name] = (ms.value, work.value, n.value)
        return out

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


    def gemv_e4m3(self, x, w8, w_scale, out, mode=0, act=0, n_valid=0, stream=None):
        """pop_k_gemv_e4m3: x bf16 [B, K]; w8 uint8 codes [N, K]; w_scale fp32 [1]."""
        B, K = x.shape
        code = self.dll.pop_k_gemv_e4m3(x.data_ptr(), x.stride(0), w8.data_ptr(), w8.stride(0), w_scale.data_ptr(),
                                        out.data_ptr(), out.stride(0), B, w8.shape[0], K, mode, act, n_valid,
                                        _stream_ptr(stream))
        self.check(code, "pop_k_gemv_e4m3")
        return out

    def rmsnorm_e4m3(self, x, gain, eps, stream=None, out=None, scale=None):
        """pop_k_rmsnorm_e4m3: returns (codes uint8 [rows, d], scale fp32 [rows]); out / scale may be given."""
        rows, d = x.shape
        if out is None:
            out = torch.empty(rows, d, dtype=torch.uint8, device=x.device)
        if scale is None:
            scale = torch.empty(rows, dtype=torch.float32, device=x.device)
        code = self.dll.pop_k_rmsnorm_e4m3(x.data_ptr(), x.stride(0), gain.data_ptr(), out.data_ptr(), out.stride(0),
                                           scale.data_ptr(), rows, d, eps, _stream_ptr(stream))
        self.check(code, "pop_k_rmsnorm_e4m3")
        return out, scale

    def quant_rows_e4m3(self, x, in_place=False, stream=None):
        """pop_k_quant_rows_e4m3 of bf16 rows [rows, d]: returns (codes uint8 [rows, d], scale fp32 [rows]);
        in_place writes each row's codes over the start of the row (the view returned has row stride 2 d)."""
        rows, d = x.shape
        scale = torch.empty(rows, dtype=torch.float32, device=x.device)
        out = x.view(torch.uint8)[:, :d] if in_place else torch.empty(rows, d, dtype=torch.uint8, device=x.device)
        code = self.dll.pop_k_quant_rows_e4m3(x.data_ptr(), x.stride(0), out.data_ptr(), out.stride(0),
                                              scale.data_ptr(), rows, d, _stream_ptr(stream))
        self.check(code, "pop_k_quant_rows_e4m3")
        return out, scale

    def quantize_e4m3(self, w, stream=None):
        """pop_k_quantize_e4m3 of a contiguous bf16 tensor: returns (codes uint8 of w's shape, scale fp32 [1])."""
        assert w.is_contiguous() and w.dtype == torch.bfloat16
        out = torch.empty(w.shape, dtype=torch.uint8, device=w.device)
        scale = torch.empty(1, dtype=torch.float32, device=w.device)
        scratch = torch.empty(1, dtype=torch.int32, device=w.device)
        code = self.dll.pop_k_quantize_e4m3(w.data_ptr(), w.numel(), out.data_ptr(), scale.data_ptr(),
                                            scratch.data_ptr(), _stream_ptr(stream))
        self.check(code, "pop_k_quantize_e4m3")
        return out, scale

    def gemm_e4m3(self, A, a_scale, B, b_scale, out, epilogue=1, act=0, n_valid=0, stream=None):
        """pop_k_gemm_e4m3: A [M,K], B [N,K] uint8 codes; a_scale fp32 [M]; b_scale fp32 [1]."""
        M, K = A.shape
        N = B.shape[0]
        code = self.dll.pop_k_gemm_e4m3(A.data_ptr(), A.stride(0), a_scale.data_ptr(), B.data_ptr(), B.stride(0),
                                        b_scale.data_ptr(), out.data_ptr(), out.stride(0), M, N, K, epilogue, act,
                                        n_valid, _stream_ptr(stream))
        self.check(code, "pop_k_gemm_e4m3")
        return out

    def gemm_norm(self, A, B, out, epilogue, act=0, n_valid=0, hn_out=None, gain_next=None, ss_out=None,
                  ss_in=None, norm_d=0, norm_eps=0.0, stream=None):
        """pop_k_gemm_norm: 2-D operands; hn_out/gain_next/ss_out = producer side, ss_in [M, cnt] fp32 =
        consumer side (None to leave a side out)."""
        M, K = A.shape
        N = B.shape[0]
        code = self.dll.pop_k_gemm_norm(A.data_ptr(), A.stride(0), B.data_ptr(), B.stride(0), out.data_ptr(),
                                        out.stride(0), M, N, K, epilogue, act, n_valid, _ptr(hn_out),
                                        0 if hn_out is None else hn_out.stride(0), _ptr(gain_next), _ptr(ss_out),
                                        0 if ss_out is None else ss_out.stride(0), _ptr(ss_in),
                                        0 if ss_in is None else ss_in.shape[1],
                                        0 if ss_in is None else ss_in.stride(0), norm_d, norm_eps,
                                        _stream_ptr(stream))
        self.check(code, "pop_k_gemm_norm")
        return out

    def gemm_qkv_rope(self, A, W, q_out, k_pool, v_pool, layer0, block_table, page_size, q_gain, k_gain, table,
                      n_q, n_kv, hd, rows_per_seq, rows_written, pos0, eps, stream=None):
        """Fused QKV projection + per-head norm + RoPE + cache write. A [M,K] or [G,M,K] bf16; W
        [(n_q+2 n_kv) hd, K] or [G, ..., K] bf16; pools [layers, pages, page_size, n_kv, hd]."""
        if A.dim() == 2:
            A, W = A.unsqueeze(0), W.unsqueeze(0)
        G, M, K = A.shape
        gain_gs = 0 if (k_gain is None or k_gain.dim() == 1) else k_gain.stride(0)
        code = self.dll.pop_k_gemm_qkv_rope(A.data_ptr(), A.stride(1), A.stride(0) if G > 1 else 0, W.data_ptr(),
                                            W.stride(1), W.stride(0) if G > 1 else 0, M, K, G, _ptr(q_out),
                                            0 if q_out is None else q_out.stride(0), k_pool.data_ptr(),
                                            v_pool.data_ptr(), k_pool.stride(0), layer0, block_table.data_ptr(),
                                            block_table.shape[1], page_size, _ptr(q_gain), _ptr(k_gain), gain_gs,
                                            table.data_ptr(), n_q, n_kv, hd, rows_per_seq, rows_written, pos0, eps,
                                            _stream_ptr(stream))
        self.check(code, "pop_k_gemm_qkv_rope")

    def attention(self, q, k_pool, v_pool, block_table, out, batch, seq_len, kv_len, n_q, n_kv, hd, page_size,
                  window=0, q_pos0=0, stream=None):
        """q [batch*seq_len, >= n_q*hd] bf16; k_pool/v_pool one cache layer [pages, page_size, n_kv, hd]."""
        code = self.dll.pop_k_attention(q.data_ptr(), q.stride(0), k_pool.data_ptr(), v_pool.data_ptr(),
                                        block_table.data_ptr(), out.data_ptr(), out.stride(0), batch, seq_len,
                                        q_pos0, kv_len, n_q, n_kv, hd, page_size, k_pool.shape[0],
                                        block_table.shape[1], window, _stream_ptr(stream))
        self.check(code, "pop_k_attention")
        return out

    def rmsnorm(self, x, gain, out, eps, stream=None):
        """x fp32 [rows, d]; gain fp32 [d] or [groups, d]; out bf16/fp32 [rows, d] or [groups, rows, d]."""
        groups = 1 if gain.dim() == 1 else gain.shape[0]
        rows, d = x.shape
        code = self.dll.pop_k_rmsnorm(x.data_ptr(), x.stride(0), gain.data_ptr(),
                                      0 if gain.dim() == 1 else gain.stride(0), out.data_ptr(), out.stride(-2),
                                      0 if out.dim() == 2 else out.stride(0), rows, d, groups, eps,
                                      1 if out.dtype == torch.float32 else 0, _stream_ptr(stream))
        self.check(code, "pop_k_rmsnorm")
        return out

    def rope_table(self, table, n_pos, hd, theta, stream=None):
        self.check(self.dll.pop_k_rope_table(table.data_ptr(), n_pos, hd, theta, _stream_ptr(stream)),
                   "pop_k_rope_table")
        return table

    def rope_cache(self, x, q_out, k_pool, v_pool, layer0, block_table, page_size, q_gain, k_gain, table, n_q, n_kv,
                   hd, rows_per_seq, rows_written, pos0, eps, stream=None):
        """x fp32 [rows, (n_q+2 n_kv) hd] or [groups, rows, ...]; pools [layers, pages, page_size, n_kv, hd]."""
        groups = 1 if x.dim() == 2 else x.shape[0]
        rows = x.shape[-2]
        gain_gs = 0 if (k_gain is None or k_gain.dim() == 1) else k_gain.stride(0)
        code = self.dll.pop_k_rope_cache(x.data_ptr(), x.stride(-2), 0 if x.dim() == 2 else x.stride(0),
                                         _ptr(q_out), 0 if q_out is None else q_out.stride(0), k_pool.data_ptr(),
                                         v_pool.data_ptr(), k_pool.stride(0), layer0, block_table.data_ptr(),
                                         block_table.shape[1], page_size, _ptr(q_gain), _ptr(k_gain), gain_gs,
                                         table.data_ptr(), n_q, n_kv, hd, rows, rows_per_seq, rows_written, pos0,
                                         groups, eps, _stream_ptr(stream))
        self.check(code, "pop_k_rope_cache")

    def gemv(self, x, w, out, mode=0, act=0, n_valid=0, stream=None):
        B, K = x.shape
        code = self.dll.pop_k_gemv(x.data_ptr(), x.stride(0), 1 if x.dtype == torch.float32 else 0, w.data_ptr(),
                                   w.stride(0), out.data_ptr(), out.stride(0), B, w.shape[0], K, mode, act, n_valid,
                                   _stream_ptr(stream))
        self.check(code, "pop_k_gemv")
        return out

    def decode_attention(self, q, k_pool, v_pool, block_table, out, n_q, n_kv, hd, kv_len, page_size, window=0,
                         stream=None, counters=None, partial=None):
        """pop_k_decode_attention. `counters`: a zeroed int32 tensor of batch * n_kv entries (left zero by
        the call) makes it a single launch; without, a second kernel merges the key splits."""
        batch = q.shape[0]
        if partial is None:
            partial = torch.empty(batch * n_q * 64 * (hd + 2), dtype=torch.float32, device=q.device)
        code = self.dll.pop_k_decode_attention(q.data_ptr(), q.stride(0), k_pool.data_ptr(), v_pool.data_ptr(),
                                               block_table.data_ptr(), block_table.shape[1], page_size,
                                               partial.data_ptr(), 0 if counters is None else counters.data_ptr(),
                                               out.data_ptr(), out.stride(0), batch, n_q, n_kv,
                                               hd, kv_len, window, _stream_ptr(stream))
        self.check(code, "pop_k_decode_attention")
        return out

    def decode_attention_qkv(self, qkv, q_gain, k_gain, eps, rope_row, k_pool, v_pool, block_table, out, n_q, n_kv, hd,
                             kv_len, page_size, counters, window=0, partial=None, stream=None):
        """pop_k_decode_attention_qkv: qkv fp32 [B, (n_q + 2 n_kv) hd]; rope_row float2 [hd/2] of position
        kv_len - 1; pools of one layer [pages, page_size, n_kv, hd] (the new position is appended)."""
        batch = qkv.shape[0]
        if partial is None:
            partial = torch.empty(batch * n_q * 64 * (hd + 2), dtype=torch.float32, device=qkv.device)
        code = self.dll.pop_k_decode_attention_qkv(
            qkv.data_ptr(), qkv.stride(0), 0 if q_gain is None else q_gain.data_ptr(),
            0 if k_gain is None else k_gain.data_ptr(), eps, rope_row.data_ptr(), k_pool.data_ptr(), v_pool.data_ptr(),
            block_table.data_ptr(), block_table.shape[1], page_size, k_pool.shape[0], partial.data_ptr(),
            counters.data_ptr(), out.data_ptr(), out.stride(0), batch, n_q, n_kv, hd, kv_len, window,
            _stream_ptr(stream))
        self.check(code, "pop_k_decode_attention_qkv")
        return out

    def decode_attention_static(self, q, k_pool, v_pool, block_table, out, n_q, n_kv, hd, kv_len, page_size,
                                window=0, stream=None):
        """pop_k_decode_attention_static: same arguments as decode_attention, but the split-KV partials
        live in the library's own fixed device array, so this call allocates nothing (not even a
        torch tensor). Raises PopError(POP_E_NOSPACE) beyond the array's stated size."""
        code = self.dll.pop_k_decode_attention_static(q.data_ptr(), q.stride(0), k_pool.data_ptr(),
                                                      v_pool.data_ptr(), block_table.data_ptr(),
                                                      block_table.shape[1], page_size, out.data_ptr(),
                                                      out.stride(0), q.shape[0], n_q, n_kv, hd, kv_len, window,
                                                      _stream_ptr(stream))
        self.check(code, "pop_k_decode_attention_static")
        return out


_LIB: Optional[PopLibrary] = None


def lib() -> PopLibrary:
    """The process-wide library handle; raises if the CUDA extension is not built."""
    global _LIB
    if _LIB is None:
        _LIB = PopLibrary()
    return _LIB


def make_config(cfg) -> pop_config_t:
    """pop_config_t from any object with the fields of pop_synth.ModelConfig."""
    c = pop_config_t()
    c.struct_size = C.sizeof(pop_config_t)
    for f in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab", "act", "qk_norm",
              "post_norms", "window", "global_every"):
        setattr(c, f, int(getattr(cfg, f)))
    c.rms_eps = float(cfg.rms_eps)
    c.rope_theta = float(cfg.rope_theta)
    return c


class KVCache:
    """Caller-owned paged KV cache: bf16 pools [n_layers, num_pages, page_size, n_kv, hd] and an
    int32 block table [batch, max_pages_per_seq] (identity paging unless `block_table` is given)."""

    def __init__(self, cfg, batch: int, seq_len: int, page_size: int = 128, device="cuda",
                 block_table: Optional[torch.Tensor] = None, num_pages: Optional[int] = None, fill: float = 0.0):
        pps = (seq_len + page_size - 1) // page_size
        self.page_size = page_size
        self.num_pages = num_pages or batch * pps
        shape = (cfg.n_layers, self.num_pages, page_size, cfg.n_kv_heads, cfg.head_dim)
        self.k = torch.full(shape, fill, dtype=torch.bfloat16, device=device)
        self.v = torch.full(shape, fill, dtype=torch.bfloat16, device=device)
        if block_table is None:
            block_table = torch.arange(batch * pps, dtype=torch.int32).reshape(batch, pps)
        self.block_table = block_table.to(device=device, dtype=torch.int32).contiguous()
        self.batch, self.seq_len = batch, seq_len

    def struct(self) -> pop_kv_cache_t:
        s = pop_kv_cache_t()
        s.k_pool, s.v_pool, s.block_table = self.k.data_ptr(), self.v.data_ptr(), self.block_table.data_ptr()
        s.page_size, s.num_pages, s.max_pages_per_seq = self.page_size, self.num_pages, self.block_table.shape[1]
        return s

    def gather(self, layer: int, seq_len: Optional[int] = None):
        """(K, V) of 0-based `layer` as dense [batch, seq_len, n_kv, hd] tensors (a host-side view for checks)."""
        n = seq_len or self.seq_len
        pos = torch.arange(n, device=self.k.device)
        pages = self.block_table[:, pos // self.page_size].long()          # [batch, n]
        slots = (pos % self.page_size)[None, :].expand_as(pages)
        return self.k[layer][pages, slots], self.v[layer][pages, slots]


class PopModel:
    """A loaded model: repacked weights in a device arena plus a workspace, both torch tensors."""

    def __init__(self, cfg, weights, library: Optional[PopLibrary] = None, device="cuda"):
        """`weights.get(name, layer)` must return bf16 matrices / fp32 gains on `device`
        (layer 1-based, 0 for embed, final_norm, lm_head)."""
        self.lib = library or lib()
        self.cfg = cfg
        self.device = device
        self.c_cfg = make_config(cfg)
        nbytes = self.lib.dll.pop_weight_arena_bytes(C.byref(self.c_cfg))
        if nbytes == 0:
            raise PopError(POP_E_INVALID, "pop_weight_arena_bytes")
        self.arena = torch.empty(nbytes + 1024, dtype=torch.uint8, device=device)
        base = (self.arena.data_ptr() + 1023) // 1024 * 1024
        names = [("embed", 0), ("final_norm", 0), ("lm_head", 0)]
        per_layer = ["ln_in", "wq", "wk", "wv", "wo", "ln_ffn", "w_gate", "w_up", "w_down"]
        if cfg.qk_norm:
            per_layer += ["q_norm", "k_norm"]
        if cfg.post_norms:
            per_layer += ["post_attn_norm", "post_ffn_norm"]
        self.handle = C.c_void_p()
        # load layer by layer so that only one layer's source tensors are alive at a time
        groups = [names] + [[(n, l) for n in per_layer] for l in range(1, cfg.n_layers + 1)]
        tensors, keep = [], []
        for grp in groups:
            for name, layer in grp:
                t = weights.get(name, layer).to(device).contiguous()
                keep.append(t)
                pt = pop_tensor_t()
                pt.name = (name if layer == 0 else f"layers.{layer}.{name}").encode()
                pt.dev_ptr = t.data_ptr()
                pt.dtype = 0 if t.dtype == torch.bfloat16 else 1
                pt.ndim = t.dim()
                pt.shape[0] = t.shape[0]
                pt.shape[1] = t.shape[1] if t.dim() > 1 else 0
                tensors.append(pt)
        arr = (pop_tensor_t * len(tensors))(*tensors)
        code = self.lib.dll.pop_load_weights(C.byref(self.c_cfg), arr, len(tensors), base, nbytes,
                                             _stream_ptr(None), C.byref(self.handle))
        self.lib.check(code, "pop_load_weights")
        torch.cuda.current_stream().synchronize()
        del keep
        self.ws = None
        self.ws_shape = None

    def ensure_workspace(self, seq_len: int, batch: int):
        need = self.lib.dll.pop_workspace_bytes(self.handle, seq_len, batch)
        if self.ws is None or self.ws.numel() < need + 1024:
            self.ws = torch.empty(need + 1024, dtype=torch.uint8, device=self.device)
        base = (self.ws.data_ptr() + 1023) // 1024 * 1024
        self.lib.check(self.lib.dll.pop_set_workspace(self.handle, base, self.ws.numel() - 1024),
                       "pop_set_workspace")

    def _input(self, tokens, embeds):
        inp = pop_input_t()
        inp.tokens = tokens.data_ptr()
        inp.embeds = None if embeds is None else embeds.data_ptr()
        return inp

    def prefill(self, tokens, embeds, l_keep: int, cache: KVCache, logits: Optional[torch.Tensor] = None,
                stream=None):
        """pop_prefill on device tensors: tokens int32 [B, N], embeds bf16 [B, N, d] or None."""
        B, N = tokens.shape
        self.ensure_workspace(N, B)
        if logits is None:
            logits = torch.empty(B, self.cfg.vocab, dtype=torch.float32, device=self.device)
        inp, kc = self._input(tokens, embeds), cache.struct()
        code = self.lib.dll.pop_prefill(self.handle, C.byref(inp), N, B, l_keep, C.byref(kc), logits.data_ptr(),
                                        _stream_ptr(stream))
        self.lib.check(code, "pop_prefill")
        return logits

    def full_prefill(self, tokens, embeds, cache: KVCache, logits: Optional[torch.Tensor] = None, stream=None):
        B, N = tokens.shape
        self.ensure_workspace(N, B)
        if logits is None:
            logits = torch.empty(B, self.cfg.vocab, dtype=torch.float32, device=self.device)
        inp, kc = self._input(tokens, embeds), cache.struct()
        code = self.lib.dll.pop_full_prefill(self.handle, C.byref(inp), N, B, C.byref(kc), logits.data_ptr(),
                                             _stream_ptr(stream))
        self.lib.check(code, "pop_full_prefill")
        return logits

    def prefill_ragged(self, tokens, embeds, seq_lens, l_keep: int, cache: KVCache,
                       logits: Optional[torch.Tensor] = None, stream=None):
        """pop_prefill_ragged: tokens int32 [sum(seq_lens)] packed on the device, seq_lens a host list."""
        B = len(seq_lens)
        self.ensure_workspace(max(seq_lens), B)
        if logits is None:
            logits = torch.empty(B, self.cfg.vocab, dtype=torch.float32, device=self.device)
        lens = (_I32 * B)(*[int(x) for x in seq_lens])
        inp, kc = self._input(tokens, embeds), cache.struct()
        code = self.lib.dll.pop_prefill_ragged(self.handle, C.byref(inp), lens, B, l_keep, C.byref(kc),
                                               logits.data_ptr(), _stream_ptr(stream))
        self.lib.check(code, "pop_prefill_ragged")
        return logits

    def prefill_skip(self, tokens, embeds, skip, cache: KVCache, logits: Optional[torch.Tensor] = None, stream=None):
        """pop_prefill_skip: `skip` is a collection of 1-based layer numbers pruned during the prefill."""
        B, N = tokens.shape
        self.ensure_workspace(N, B)
        if logits is None:
            logits = torch.empty(B, self.cfg.vocab, dtype=torch.float32, device=self.device)
        mask = bytes(1 if (l + 1) in set(skip) else 0 for l in range(self.cfg.n_layers))
        inp, kc = self._input(tokens, embeds), cache.struct()
        code = self.lib.dll.pop_prefill_skip(self.handle, C.byref(inp), N, B, mask, C.byref(kc), logits.data_ptr(),
                                             _stream_ptr(stream))
        self.lib.check(code, "pop_prefill_skip")
        return logits

    def enable_fp8(self, on: bool = True, stream=None):
        """pop_enable_fp8: E4M3 copies of the kept layers' QKV and gate/up weights (the arena is a torch
        tensor this object keeps); on=False goes back to bf16 operands."""
        if not on:
            self.lib.check(self.lib.dll.pop_enable_fp8(self.handle, None, 0, _stream_ptr(stream)), "pop_enable_fp8")
            self.fp8_arena = None
            return
        need = self.lib.dll.pop_fp8_arena_bytes(self.handle)
        self.fp8_arena = torch.empty(need + 1024, dtype=torch.uint8, device=self.device)
        base = (self.fp8_arena.data_ptr() + 1023) // 1024 * 1024
        self.lib.check(self.lib.dll.pop_enable_fp8(self.handle, base, need, _stream_ptr(stream)), "pop_enable_fp8")

    def prefill_chunked(self, tokens, embeds, l_keep: int, chunk_len: int, cache: KVCache,
                        logits: Optional[torch.Tensor] = None, stream=None):
        """pop_prefill_chunked: pop_prefill in chunks of chunk_len positions (workspace for one chunk)."""
        B, N = tokens.shape
        self.ensure_workspace(min(chunk_len, N), B)
        if logits is None:
            logits = torch.empty(B, self.cfg.vocab, dtype=torch.float32, device=self.device)
        inp, kc = self._input(tokens, embeds), cache.struct()
        code = self.lib.dll.pop_prefill_chunked(self.handle, C.byref(inp), N, B, l_keep, chunk_len, C.byref(kc),
                                                logits.data_ptr(), _stream_ptr(stream))
        self.lib.check(code, "pop_prefill_chunked")
        return logits

    def prefill_ablation(self, tokens, embeds, skip, cache: KVCache, boundary: bool = True, indep_kv: bool = True,
                         logits: Optional[torch.Tensor] = None, stream=None):
        """pop_prefill_ablation: pop_prefill_skip without boundary handling and / or without the pruned
        layers' independent KV projections. Returns (logits, layer_first_pos) where layer_first_pos is
        what later decode_step calls must be given (None when every layer holds the whole prompt)."""
        B, N = tokens.shape
        self.ensure_workspace(N, B)
        if logits is None:
            logits = torch.empty(B, self.cfg.vocab, dtype=torch.float32, device=self.device)
        skip = set(skip)
        mask = bytes(1 if (l + 1) in skip else 0 for l in range(self.cfg.n_layers))
        flags = (0 if boundary else POP_NO_BOUNDARY) | (0 if indep_kv else POP_NO_INDEP_KV)
        inp, kc = self._input(tokens, embeds), cache.struct()
        code = self.lib.dll.pop_prefill_ablation(self.handle, C.byref(inp), N, B, mask, flags, C.byref(kc),
                                                 logits.data_ptr(), _stream_ptr(stream))
        self.lib.check(code, "pop_prefill_ablation")
        horizon = N - 1 if boundary else N       # without the full-depth pass a pruned layer holds nothing at all
        first = None if indep_kv else [horizon if (l + 1) in skip else 0 for l in range(self.cfg.n_layers)]
        return logits, first

    def decode_step(self, tokens, pos: int, cache: KVCache, logits: Optional[torch.Tensor] = None, stream=None,
                    layer_first_pos=None):
        """pop_decode_step: tokens int32 [B] on the device, each at position `pos` of its sequence.
        layer_first_pos (n_layers ints) -> pop_decode_step_from: per-layer attention horizon."""
        B = tokens.shape[0]
        self.ensure_workspace(1, B) if self.ws is None else None
        if logits is None:
            logits = torch.empty(B, self.cfg.vocab, dtype=torch.float32, device=self.device)
        kc = cache.struct()
        if layer_first_pos is None:
            code = self.lib.dll.pop_decode_step(self.handle, tokens.data_ptr(), pos, B, C.byref(kc),
                                                logits.data_ptr(), _stream_ptr(stream))
            self.lib.check(code, "pop_decode_step")
        else:
            arr = (_I32 * self.cfg.n_layers)(*[int(v) for v in layer_first_pos])
            code = self.lib.dll.pop_decode_step_from(self.handle, tokens.data_ptr(), pos, B, arr, C.byref(kc),
                                                     logits.data_ptr(), _stream_ptr(stream))
            self.lib.check(code, "pop_decode_step_from")
        return logits

    def generate_greedy(self, first_tokens, pos0: int, n_steps: int, cache: KVCache,
                        logits: Optional[torch.Tensor] = None, stream=None):
        """pop_generate_greedy: returns (tokens int32 [B, n_steps] on the device, last logits)."""
        B = first_tokens.shape[0]
        if self.ws is None:
            self.ensure_workspace(1, B)
        if logits is None:
            logits = torch.empty(B, self.cfg.vocab, dtype=torch.float32, device=self.device)
        out = torch.full((B, n_steps), -1, dtype=torch.int32, device=self.device)
        kc = cache.struct()
        code = self.lib.dll.pop_generate_greedy(self.handle, first_tokens.data_ptr(), pos0, n_steps, B, C.byref(kc),
                                                out.data_ptr(), logits.data_ptr(), _stream_ptr(stream))
        self.lib.check(code, "pop_generate_greedy")
        return out, logits

    def read_hidden(self, seq_len: int, batch: int, stream=None):
        """(hidden fp32 [B, N, d], last fp32 [B, d]) left in the workspace by the last prefill of this shape."""
        hidden = torch.empty(batch, seq_len, self.cfg.d_model, dtype=torch.float32, device=self.device)
        last = torch.empty(batch, self.cfg.d_model, dtype=torch.float32, device=self.device)
        code = self.lib.dll.pop_read_hidden(self.handle, seq_len, batch, hidden.data_ptr(), last.data_ptr(),
                                            _stream_ptr(stream))
        self.lib.check(code, "pop_read_hidden")
        return hidden, last

    def last_status(self, stream=None) -> int:
        return self.lib.dll.pop_last_status(self.handle, _stream_ptr(stream))

    def last_launch_count(self) -> int:
        return self.lib.dll.pop_last_launch_count(self.handle)

    def close(self):
        if self.handle:
            self.lib.dll.pop_free(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
