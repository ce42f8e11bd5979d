"""Seeded synthetic inputs for the POP prefill path: model shapes, weights, prompts.

This module only *describes and draws inputs*. It holds none of the method's
arithmetic (no norm, no projection, no attention): the CPU oracle and the CUDA
library each implement that on their own and merely receive what is drawn here.

Every value is a pure function of ``(seed, tensor id, element index)`` through a
counter-based integer hash, so any tensor (or any row range of it) can be drawn
on demand, on the CPU or on a CUDA device, with bit-identical results: only
64-bit integer operations and one correctly rounded fp32 multiply are used, no
transcendental function whose last bit could differ between devices.

Normal deviates are the centred sum of twelve 16-bit uniforms (Irwin-Hall, unit
variance, support +-6 sigma), scaled by ``std`` in fp32 and rounded to bf16
(round to nearest even).
"""
from __future__ import annotations

import dataclasses
import zlib
from typing import Optional

import torch

MASK64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB

DEFAULT_SEED = 20260203


def _s64(v: int) -> int:
    """Python int -> the int64 two's-complement value with the same low 64 bits."""
    v &= MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


def _lsr(x: torch.Tensor, n: int) -> torch.Tensor:
    """Logical right shift of an int64 tensor."""
    return (x >> n) & ((1 << (64 - n)) - 1)


def _mix(z: torch.Tensor) -> torch.Tensor:
    """splitmix64 finaliser on int64 tensors (wrap-around arithmetic)."""
    z = (z ^ _lsr(z, 30)) * _s64(_M1)
    z = (z ^ _lsr(z, 27)) * _s64(_M2)
    return z ^ _lsr(z, 31)


def _mix_int(z: int) -> int:
    z &= MASK64
    z = ((z ^ (z >> 30)) * _M1) & MASK64
    z = ((z ^ (z >> 27)) * _M2) & MASK64
    return z ^ (z >> 31)


def stream_key(seed: int, tensor_id: int) -> int:
    """Key of one tensor's random stream."""
    return _mix_int(_mix_int(seed & MASK64) + (tensor_id & MASK64) * _GOLDEN)


def tensor_id(name: str, layer: int = 0) -> int:
    """Stable id of a named tensor (CRC32 of the name, layer in the high bits)."""
    return (layer << 32) | zlib.crc32(name.encode())


def _hash_at(key: int, counter: torch.Tensor) -> torch.Tensor:
    return _mix(counter * _s64(_GOLDEN) + _s64(key))


_CHUNK = 1 << 20


def _mix_(z: torch.Tensor, t: torch.Tensor) -> torch.Tensor:
    """In-place splitmix64 finaliser; `t` is scratch of the same shape."""
    for shift, mult in ((30, _M1), (27, _M2)):
        torch.bitwise_right_shift(z, shift, out=t)
        t.bitwise_and_((1 << (64 - shift)) - 1)
        z.bitwise_xor_(t)
        z.mul_(_s64(mult))
    torch.bitwise_right_shift(z, 31, out=t)
    t.bitwise_and_((1 << 33) - 1)
    z.bitwise_xor_(t)
    return z


def _irwin_hall_int(key: int, start: int, count: int, device) -> torch.Tensor:
    """Centred sum of twelve 16-bit uniforms for elements [start, start+count): int64,
    value = 2 * (sum - 12 * 32767.5), an exact integer in [-786420, 786420]."""
    out = torch.empty(count, dtype=torch.int64, device=device)
    for c0 in range(0, count, _CHUNK):
        c1 = min(count, c0 + _CHUNK)
        idx3 = torch.arange(start + c0, start + c1, dtype=torch.int64, device=device).mul_(3)
        acc = out[c0:c1].zero_()
        z = torch.empty_like(idx3)
        t = torch.empty_like(idx3)
        for j in range(3):
            torch.add(idx3, j, out=z)
            z.mul_(_s64(_GOLDEN)).add_(_s64(key))
            _mix_(z, t)
            for sh in (0, 16, 32):
                torch.bitwise_right_shift(z, sh, out=t)
                t.bitwise_and_(0xFFFF)
                acc.add_(t)
            torch.bitwise_right_shift(z, 48, out=t)
            t.bitwise_and_(0xFFFF)
            acc.add_(t)
        acc.mul_(2).sub_(786420)
    return out


def normal_bf16(seed: int, tid: int, shape, std: float, device="cpu",
                row_start: int = 0, row_count: Optional[int] = None) -> torch.Tensor:
    """bf16 tensor of approximately N(0, std^2) values; optionally only rows
    [row_start, row_start+row_count) of the leading dimension."""
    shape = tuple(int(s) for s in shape)
    inner = 1
    for s in shape[1:]:
        inner *= s
    rows = shape[0] if row_count is None else int(row_count)
    key = stream_key(seed, tid)
    s = _irwin_hall_int(key, row_start * inner, rows * inner, device)
    # s / 2 / 65536 has unit variance; s is exact in fp32 (|s| < 2^24).
    scale = torch.tensor(float(std) / 131072.0, dtype=torch.float32, device=device)
    x = s.to(torch.float32) * scale
    return x.to(torch.bfloat16).reshape((rows,) + shape[1:])


def gains(seed: int, tid: int, n: int, distinct: bool, device="cpu") -> torch.Tensor:
    """Norm gains, fp32: all ones, or k/128 + 0.5 with k uniform in [0,128)
    (every value exactly representable in bf16)."""
    if not distinct:
        return torch.ones(n, dtype=torch.float32, device=device)
    key = stream_key(seed, tid)
    h = _hash_at(key, torch.arange(n, dtype=torch.int64, device=device))
    k = _lsr(h, 57)  # 7 bits
    return 0.5 + k.to(torch.float32) / 128.0


def uniform_tokens(seed: int, batch: int, seq_len: int, vocab: int) -> torch.Tensor:
    """int32 [batch, seq_len] token ids uniform over [0, vocab) (CPU tensor);
    sequence b uses stream ``seed + 1 + b``."""
    out = torch.empty(batch, seq_len, dtype=torch.int32)
    for b in range(batch):
        key = stream_key(seed + 1 + b, tensor_id("tokens"))
        h = _hash_at(key, torch.arange(seq_len, dtype=torch.int64))
        out[b] = (_lsr(h, 11) % vocab).to(torch.int32)
    return out


def visual_embeds(seed: int, batch: int, n_rows: int, d_model: int) -> torch.Tensor:
    """bf16 [batch, n_rows, d_model] stand-ins for projected visual tokens: N(0,1)
    entries, every row rescaled to RMS 1, then rounded to bf16. Drawn on the CPU only."""
    out = torch.empty(batch, n_rows, d_model, dtype=torch.bfloat16)
    for b in range(batch):
        key = stream_key(seed + 1 + b, tensor_id("visual_embeds"))
        s = _irwin_hall_int(key, 0, n_rows * d_model, "cpu").to(torch.float64) / 131072.0
        s = s.reshape(n_rows, d_model)
        s = s / s.pow(2).mean(dim=1, keepdim=True).sqrt()
        out[b] = s.to(torch.float32).to(torch.bfloat16)
    return out


# --------------------------------------------------------------------------------------
# Model shapes
# --------------------------------------------------------------------------------------

@dataclasses.dataclass(frozen=True)
class ModelConfig:
    name: str
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0
    act: int = 0            # 0 SiLU-gated, 1 tanh-GELU-gated
    qk_norm: int = 0        # per-head RMSNorm on q and k before RoPE
    post_norms: int = 0     # RMSNorm on each sublayer output before the residual add
    window: int = 0         # 0: all layers global
    global_every: int = 0   # layer l (1-based) is global iff l % global_every == 0
    distinct_gains: bool = False
    weight_std: float = 0.02

    @property
    def q_dim(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim

    def layer_window(self, layer: int) -> int:
        """Attention window of 1-based layer `layer` (0 = global)."""
        if self.window <= 0:
            return 0
        if self.global_every > 0 and layer % self.global_every == 0:
            return 0
        return self.window

    def replace(self, **kw) -> "ModelConfig":
        return dataclasses.replace(self, **kw)


@dataclasses.dataclass(frozen=True)
class Workload:
    """One benchmark / parity configuration: a model shape plus a prompt recipe."""
    key: str
    model: ModelConfig
    batch: int
    seq_len: int
    l_keep: int
    n_visual: int = 0       # leading positions given as embeddings instead of token ids


C1_TINY = ModelConfig("tiny-llama", 4, 256, 4, 2, 64, 688, 1024, 1e-5, 10000.0)
C2_LLAMA8B = ModelConfig("llama-3.1-8b-shape", 32, 4096, 32, 8, 128, 14336, 128256, 1e-5, 500000.0)
C3_QWEN8B = ModelConfig("qwen3-8b-vlm-backbone-shape", 36, 4096, 32, 8, 128, 12288, 151936, 1e-6,
                        1000000.0, qk_norm=1)
C4_GEMMA12B = ModelConfig("gemma-3-12b-shape", 48, 3840, 16, 8, 256, 15360, 262144, 1e-6,
                          1000000.0, act=1, post_norms=1, window=1024, global_every=6)

WORKLOADS = {
    "c1": Workload("c1", C1_TINY, 1, 128, 3),
    "c2": Workload("c2", C2_LLAMA8B, 1, 8192, 24),
    "c3": Workload("c3", C3_QWEN8B, 1, 6656, 27, n_visual=6144),
    "c4": Workload("c4", C4_GEMMA12B, 1, 16384, 36),
}

# per-layer tensors: name -> shape as a function of the config ([out, in]; y = x W^T)
def layer_tensor_shapes(cfg: ModelConfig) -> dict:
    s = {
        "ln_in": (cfg.d_model,),
        "wq": (cfg.q_dim, cfg.d_model),
        "wk": (cfg.kv_dim, cfg.d_model),
        "wv": (cfg.kv_dim, cfg.d_model),
        "wo": (cfg.d_model, cfg.q_dim),
        "ln_ffn": (cfg.d_model,),
        "w_gate": (cfg.d_ffn, cfg.d_model),
        "w_up": (cfg.d_ffn, cfg.d_model),
        "w_down": (cfg.d_model, cfg.d_ffn),
    }
    if cfg.qk_norm:
        s["q_norm"] = (cfg.head_dim,)
        s["k_norm"] = (cfg.head_dim,)
    if cfg.post_norms:
        s["post_attn_norm"] = (cfg.d_model,)
        s["post_ffn_norm"] = (cfg.d_model,)
    return s


def global_tensor_shapes(cfg: ModelConfig) -> dict:
    return {"embed": (cfg.vocab, cfg.d_model), "final_norm": (cfg.d_model,),
            "lm_head": (cfg.vocab, cfg.d_model)}


class SynthWeights:
    """Draws the weights of a random-init model on demand.

    ``get(name, layer)`` returns matrices as bf16 and norm gains as fp32, on
    ``device``; ``layer`` is 1-based, 0 for the global tensors. ``rows(...)``
    draws a row range of a matrix (used to look up a few embedding rows without
    materialising a [vocab, d] table)."""

    def __init__(self, cfg: ModelConfig, seed: int = DEFAULT_SEED, device="cpu"):
        self.cfg, self.seed, self.device = cfg, seed, device

    def shape(self, name: str, layer: int = 0):
        tbl = layer_tensor_shapes(self.cfg) if layer > 0 else global_tensor_shapes(self.cfg)
        return tbl[name]

    def get(self, name: str, layer: int = 0) -> torch.Tensor:
        shp = self.shape(name, layer)
        tid = tensor_id(name, layer)
        if len(shp) == 1:
            return gains(self.seed, tid, shp[0], self.cfg.distinct_gains, self.device)
        return normal_bf16(self.seed, tid, shp, self.cfg.weight_std, self.device)

    def rows(self, name: str, layer: int, row_start: int, row_count: int) -> torch.Tensor:
        shp = self.shape(name, layer)
        return normal_bf16(self.seed, tensor_id(name, layer), shp, self.cfg.weight_std,
                           self.device, row_start, row_count)

    def embedding_rows(self, ids: torch.Tensor) -> torch.Tensor:
        """bf16 [len(ids), d_model] rows of the embedding table."""
        ids = ids.reshape(-1).tolist()
        out = torch.empty(len(ids), self.cfg.d_model, dtype=torch.bfloat16, device=self.device)
        cache = {}
        for i, t in enumerate(ids):
            if t not in cache:
                cache[t] = self.rows("embed", 0, int(t), 1)[0]
            out[i] = cache[t]
        return out


def make_prompt(wl: Workload, seed: int = DEFAULT_SEED):
    """(tokens int32 [B,N] with -1 at positions fed by embeddings, embeds bf16 [B,N,d] or None)."""
    cfg = wl.model
    tokens = uniform_tokens(seed, wl.batch, wl.seq_len, cfg.vocab)
    embeds = None
    if wl.n_visual > 0:
        embeds = torch.zeros(wl.batch, wl.seq_len, cfg.d_model, dtype=torch.bfloat16)
        embeds[:, :wl.n_visual] = visual_embeds(seed, wl.batch, wl.n_visual, cfg.d_model)
        tokens[:, :wl.n_visual] = -1
    return tokens, embeds
