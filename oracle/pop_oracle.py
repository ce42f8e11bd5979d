"""CPU oracle for the POP pruned-prefill path.  TEST INFRASTRUCTURE, not product code.

A plain, slow, step-by-step statement of what the path computes, in plain PyTorch
CPU ops (fp64 by default), written from the paper's definitions:

  * decoder layer         y_l = x_l + Attn(x_l, K, V);  x_{l+1} = y_l + FFN(y_l)      (Sec. 2.1, Eq. 1)
  * KV generation         k = RoPE(LN(x_l) W^K),  v = LN(x_l) W^V                     (Eq. 2)
  * KV append             K_cur = Concat(K_past, k), attention uses the updated cache (Eq. 3)
  * pruned layer          k_l, v_l from the layer's own LN / W^K / W^V on x_l (Eq. 14);
                          hidden state passed on unchanged (Eq. 15 = Eq. 4)
  * boundary handling     pruned prefill covers x_{1:N-1}; x_N is the first decode step
                          of the full model                                        (Sec. 3.3)

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
module. It shares no code with the CUDA library and never imports it. Weights and
inputs are handed in by the caller (a provider with ``get(name, layer)``).

Readings taken where the paper is silent (each also listed in the design notes):
RMSNorm with fp statistics over the feature axis; rotate-half RoPE pairing
(j, j + hd/2) with angle pos * theta^(-2j/hd), 0-based positions; per-head QK
RMSNorm (when the model has it) between projection and RoPE; softmax scale
1/sqrt(hd); sliding window of W keys including the query's own position; query
head h uses KV head floor(h * n_kv / n_q); tanh-approximated GELU for the
GELU-gated FFN; logits for the last prompt position only.

``precision="exact"`` evaluates everything in ``dtype``.  ``precision="bf16ops"``
additionally rounds intermediate tensors to bf16 at the points where a bf16
tensor-core pipeline stores or feeds them (GEMM operands, q/k/v, softmax
probabilities entering P.V, attention output, gated activation); it exists so
that integer decisions (the argmax token) can be compared in the kernel's
precision.  The residual stream, norm statistics, softmax and all accumulations
stay in ``dtype`` in both modes.

Pins (tests/test_oracle_*.py): closed forms and invariants of each primitive, an
independent brute-force single-sequence evaluator with explicit N x N score
matrices and no cache, prefix-recomputation (causality), the structural
identities of POP (L_keep = L and L_keep = L-1 reproduce the full prefill; kept
layers and the first pruned layer have the full model's KV; deeper pruned layers
equal a separate three-line evaluation of Eq. 14), and fault-injection checks
that a planted mistake fails them.  The accuracy effect of pruning on trained
models (the paper's Tables 1, 3, 4) is parity unpinned: it needs trained weights
and public datasets that are not available to this repository.
"""
from __future__ import annotations

import math
from typing import Optional

import torch


# ---------------------------------------------------------------------------------------
# primitives
# ---------------------------------------------------------------------------------------

def _rnd(x: torch.Tensor, precision: str) -> torch.Tensor:
    """Identity in "exact" mode; otherwise ("bf16ops": bf16 operands; "fp8": E4M3 operands for the four
    projections of a layer; "fp8w": E4M3 weights of those projections, bf16 activations; bf16 for
    attention and everything stored in all three) round to bf16 and back."""
    if precision == "exact":
        return x
    if precision not in ("bf16ops", "fp8", "fp8w"):
        raise ValueError(f"unknown precision {precision!r}")
    return x.to(torch.float32).to(torch.bfloat16).to(x.dtype)


# ---------------------------------------------------------------------------------------
# FP8 operands (stage-aware quantisation is the paper's stated future direction, Sec. 6; the paper
# fixes no format: this is the OCP E4M3 format with one scale per activation row and one per weight
# matrix, the reading stated in the design notes)
# ---------------------------------------------------------------------------------------
E4M3_MAX = 448.0


def e4m3_round(x: torch.Tensor) -> torch.Tensor:
    """Nearest value of the OCP FP8 E4M3 format (1 sign, 4 exponent bits with bias 7, 3 mantissa
    bits; no infinities; largest finite value 448; subnormals are multiples of 2^-9), ties to the
    even mantissa, magnitudes above 448 saturate. Returned in float64."""
    x = x.double()
    a = x.abs().clamp(max=E4M3_MAX)
    _, ex = torch.frexp(a)                       # a = m * 2^ex, m in [0.5, 1)
    e = (ex - 1).clamp(min=-6)                   # exponent of the binade; subnormals share the lowest
    quantum = torch.pow(torch.tensor(2.0, dtype=torch.float64), (e - 3).double())
    q = torch.round(a / quantum) * quantum       # torch.round: halves to even
    return torch.where(a == 0, torch.zeros_like(a), q) * torch.sign(x)


def quant_rows_e4m3(h: torch.Tensor):
    """One scale per row: codes e4m3(h * (448 / amax_row)) and the scale amax_row / 448 that maps
    them back (a row of zeros gets scale 1). The decision is taken in fp32 as the kernel takes it.
    h: [T, d] -> (codes [T, d] float64 holding E4M3 values, scale [T, 1] float64)."""
    h32 = h.to(torch.float32)
    amax = h32.abs().amax(dim=-1, keepdim=True)
    safe = torch.where(amax > 0, amax, torch.ones_like(amax))
    inv = torch.tensor(E4M3_MAX, dtype=torch.float32) / safe
    scale = torch.where(amax > 0, amax / torch.tensor(E4M3_MAX, dtype=torch.float32), torch.ones_like(amax))
    return e4m3_round(h32 * inv), scale.double()


def quant_tensors_e4m3(ws):
    """One scale for a group of weight matrices that the kernel stores as one fused matrix:
    codes e4m3(w * (448 / amax)) for every matrix and the common scale amax / 448."""
    amax = max(float(w.to(torch.float32).abs().max()) for w in ws)
    amax32 = torch.tensor(amax if amax > 0 else E4M3_MAX, dtype=torch.float32)
    inv = torch.tensor(E4M3_MAX, dtype=torch.float32) / amax32
    scale = float(amax32 / torch.tensor(E4M3_MAX, dtype=torch.float32))
    return [e4m3_round(w.to(torch.float32) * inv) for w in ws], scale


def rmsnorm(x: torch.Tensor, gain: torch.Tensor, eps: float) -> torch.Tensor:
    """LN(.) of Eq. 2 for the RMSNorm models evaluated in Sec. 4: x * g / sqrt(mean(x^2) + eps)."""
    ms = x.pow(2).mean(dim=-1, keepdim=True)
    return x / torch.sqrt(ms + eps) * gain


def rope(x: torch.Tensor, positions: torch.Tensor, theta: float) -> torch.Tensor:
    """RoPE(.) of Eq. 2. x: [..., T, heads, hd]; positions: [T] (0-based).
    Pair (j, j + hd/2) is rotated by the angle pos * theta^(-2j/hd)."""
    hd = x.shape[-1]
    half = hd // 2
    j = torch.arange(half, dtype=torch.float64)
    inv_freq = torch.pow(torch.tensor(float(theta), dtype=torch.float64), -2.0 * j / hd)
    ang = positions.to(torch.float64)[:, None] * inv_freq[None, :]          # [T, half]
    cos = torch.cos(ang).to(x.dtype)[:, None, :]
    sin = torch.sin(ang).to(x.dtype)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return torch.cat([x1 * cos - x2 * sin, x2 * cos + x1 * sin], dim=-1)


def gated_act(gate: torch.Tensor, up: torch.Tensor, act: int) -> torch.Tensor:
    """act(gate) * up: SiLU (act=0) or tanh-approximated GELU (act=1)."""
    if act == 0:
        a = gate * torch.sigmoid(gate)
    else:
        a = 0.5 * gate * (1.0 + torch.tanh(math.sqrt(2.0 / math.pi) * (gate + 0.044715 * gate.pow(3))))
    return a * up


def attention(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, q_pos: torch.Tensor,
              window: int, precision: str = "exact", k_pos0: int = 0) -> torch.Tensor:
    """Attn of Eq. 1 for one sequence. q: [T, n_q, hd] at absolute positions q_pos [T];
    k, v: [S, n_kv, hd] holding cache positions k_pos0..k_pos0+S-1. Query at position i sees keys
    j <= i, and j > i - window when window > 0. Returns [T, n_q, hd]."""
    T, n_q, hd = q.shape
    S, n_kv, _ = k.shape
    out = torch.empty_like(q)
    kpos = torch.arange(S) + k_pos0
    allowed = kpos[None, :] <= q_pos[:, None]
    if window > 0:
        allowed &= kpos[None, :] > (q_pos[:, None] - window)
    scale = 1.0 / math.sqrt(hd)
    for h in range(n_q):
        g = (h * n_kv) // n_q
        s = (q[:, h, :] @ k[:, g, :].T) * scale
        s = s.masked_fill(~allowed, float("-inf"))
        p = torch.exp(s - s.max(dim=-1, keepdim=True).values)
        denom = p.sum(dim=-1, keepdim=True)
        out[:, h, :] = (_rnd(p, precision) @ v[:, g, :]) / denom
    return out


# ---------------------------------------------------------------------------------------
# model pieces
# ---------------------------------------------------------------------------------------

def _w(weights, name, layer, dtype):
    return weights.get(name, layer).to(dtype)


def embed(cfg, weights, tokens: torch.Tensor, embeds: Optional[torch.Tensor], dtype) -> torch.Tensor:
    """x_1 for one sequence: tokens int [N] (a negative id means "take the row of
    `embeds`"), embeds [N, d] or None."""
    N = tokens.shape[0]
    x = torch.empty(N, cfg.d_model, dtype=dtype)
    is_tok = tokens >= 0
    if is_tok.any():
        if hasattr(weights, "embedding_rows"):
            rows = weights.embedding_rows(tokens[is_tok])
        else:
            rows = weights.get("embed", 0)[tokens[is_tok].long()]
        x[is_tok] = rows.to(dtype)
    if (~is_tok).any():
        x[~is_tok] = embeds[~is_tok].to(dtype)
    return x


def _qkv_fp8(cfg, weights, layer: int, x: torch.Tensor, dtype):
    """q, k, v projections of LN(x) with E4M3 operands: one scale per row of LN(x), one for the fused
    [W^Q; W^K; W^V] matrix; the products are exact, the scales multiply the sum."""
    hq, sa = quant_rows_e4m3(rmsnorm(x, _w(weights, "ln_in", layer, dtype), cfg.rms_eps))
    (wq, wk, wv), sw = quant_tensors_e4m3([weights.get(n, layer) for n in ("wq", "wk", "wv")])
    hq = hq.to(dtype)
    return tuple((hq @ w.to(dtype).T) * sa.to(dtype) * sw for w in (wq, wk, wv))


def _w_deq(weights, names, layer: int, dtype):
    """The matrices `names` of a layer as the E4M3 kernels see them when only the weights are
    quantised (precision "fp8w": single-position passes stream codes and keep bf16 activations):
    code * scale, one scale for the group (it is stored as one fused matrix)."""
    qs, sw = quant_tensors_e4m3([weights.get(n, layer) for n in names])
    return [(q * sw).to(dtype) for q in qs]


def _proj_fp8(a: torch.Tensor, w: torch.Tensor, dtype) -> torch.Tensor:
    """a @ w^T with E4M3 operands: one scale per row of a (already rounded to bf16, as it is stored),
    one for the matrix."""
    aq, sa = quant_rows_e4m3(a)
    (wq,), sw = quant_tensors_e4m3([w])
    return (aq.to(dtype) @ wq.to(dtype).T) * sa.to(dtype) * sw


def kv_generation(cfg, weights, layer: int, x: torch.Tensor, positions: torch.Tensor,
                  dtype, precision: str):
    """Eq. 2 (and, applied to a pruned layer's input, Eq. 14): the layer's own input norm,
    K/V projections, optional per-head K norm, RoPE on k. x: [T, d] -> k, v [T, n_kv, hd]."""
    if precision == "fp8":
        _, k, v = _qkv_fp8(cfg, weights, layer, x, dtype)
        k = k.reshape(-1, cfg.n_kv_heads, cfg.head_dim)
        v = v.reshape(-1, cfg.n_kv_heads, cfg.head_dim)
    else:
        h = _rnd(rmsnorm(x, _w(weights, "ln_in", layer, dtype), cfg.rms_eps), precision)
        if precision == "fp8w":
            _, wk, wv = _w_deq(weights, ("wq", "wk", "wv"), layer, dtype)
        else:
            wk, wv = _w(weights, "wk", layer, dtype), _w(weights, "wv", layer, dtype)
        k = (h @ wk.T).reshape(-1, cfg.n_kv_heads, cfg.head_dim)
        v = (h @ wv.T).reshape(-1, cfg.n_kv_heads, cfg.head_dim)
    if cfg.qk_norm:
        k = rmsnorm(k, _w(weights, "k_norm", layer, dtype), cfg.rms_eps)
    k = rope(k, positions, cfg.rope_theta)
    return _rnd(k, precision), _rnd(v, precision)


def layer_forward(cfg, weights, layer: int, x: torch.Tensor, positions: torch.Tensor,
                  k_past: Optional[torch.Tensor], v_past: Optional[torch.Tensor],
                  dtype, precision: str, k_pos0: int = 0):
    """One full decoder layer (Eq. 1-3) on the T new positions `positions` of one sequence,
    given the cache of earlier positions (its first entry is position k_pos0; with no past
    entries the new positions are the whole cache). Returns x_{l+1} [T, d], K_cur, V_cur."""
    k_new, v_new = kv_generation(cfg, weights, layer, x, positions, dtype, precision)
    if k_past is not None and k_past.shape[0] > 0:
        k_cur = torch.cat([k_past, k_new], dim=0)                       # Eq. 3
        v_cur = torch.cat([v_past, v_new], dim=0)
    else:
        k_cur, v_cur = k_new, v_new
        k_pos0 = int(positions[0])
    if precision == "fp8":
        q = _qkv_fp8(cfg, weights, layer, x, dtype)[0].reshape(-1, cfg.n_q_heads, cfg.head_dim)
    else:
        h = _rnd(rmsnorm(x, _w(weights, "ln_in", layer, dtype), cfg.rms_eps), precision)
        wq_ = _w_deq(weights, ("wq", "wk", "wv"), layer, dtype)[0] if precision == "fp8w" else _w(weights, "wq", layer, dtype)
        q = (h @ wq_.T).reshape(-1, cfg.n_q_heads, cfg.head_dim)
    if cfg.qk_norm:
        q = rmsnorm(q, _w(weights, "q_norm", layer, dtype), cfg.rms_eps)
    q = _rnd(rope(q, positions, cfg.rope_theta), precision)
    a = attention(q, k_cur, v_cur, positions, cfg.layer_window(layer), precision, k_pos0)
    a = _rnd(a.reshape(-1, cfg.q_dim), precision)
    if precision == "fp8":
        o = _proj_fp8(a, weights.get("wo", layer), dtype)
    elif precision == "fp8w":
        o = a @ _w_deq(weights, ("wo",), layer, dtype)[0].T
    else:
        o = a @ _w(weights, "wo", layer, dtype).T
    if cfg.post_norms:
        o = rmsnorm(o, _w(weights, "post_attn_norm", layer, dtype), cfg.rms_eps)
    y = x + o                                                           # Eq. 1, first line
    if precision == "fp8":
        h2q, sa = quant_rows_e4m3(rmsnorm(y, _w(weights, "ln_ffn", layer, dtype), cfg.rms_eps))
        (wg, wu), sw = quant_tensors_e4m3([weights.get(n, layer) for n in ("w_gate", "w_up")])
        gate = (h2q.to(dtype) @ wg.to(dtype).T) * sa.to(dtype) * sw
        up = (h2q.to(dtype) @ wu.to(dtype).T) * sa.to(dtype) * sw
    else:
        h2 = _rnd(rmsnorm(y, _w(weights, "ln_ffn", layer, dtype), cfg.rms_eps), precision)
        if precision == "fp8w":
            wg_, wu_ = _w_deq(weights, ("w_gate", "w_up"), layer, dtype)
        else:
            wg_, wu_ = _w(weights, "w_gate", layer, dtype), _w(weights, "w_up", layer, dtype)
        gate = h2 @ wg_.T
        up = h2 @ wu_.T
    if precision == "fp8":
        f = _proj_fp8(_rnd(gated_act(gate, up, cfg.act), precision), weights.get("w_down", layer), dtype)
    elif precision == "fp8w":
        f = _rnd(gated_act(gate, up, cfg.act), precision) @ _w_deq(weights, ("w_down",), layer, dtype)[0].T
    else:
        f = _rnd(gated_act(gate, up, cfg.act), precision) @ _w(weights, "w_down", layer, dtype).T
    if cfg.post_norms:
        f = rmsnorm(f, _w(weights, "post_ffn_norm", layer, dtype), cfg.rms_eps)
    return y + f, k_cur, v_cur                                          # Eq. 1, second line


def lm_logits(cfg, weights, x_last: torch.Tensor, dtype) -> torch.Tensor:
    """Final norm and output head on one position: [d] -> [vocab]."""
    h = rmsnorm(x_last, _w(weights, "final_norm", 0, dtype), cfg.rms_eps)
    V = cfg.vocab
    out = torch.empty(V, dtype=dtype)
    step = 16384
    for r0 in range(0, V, step):
        r1 = min(V, r0 + step)
        if hasattr(weights, "rows"):
            w = weights.rows("lm_head", 0, r0, r1 - r0).to(dtype)
        else:
            w = weights.get("lm_head", 0)[r0:r1].to(dtype)
        out[r0:r1] = w @ h
    return out


# ---------------------------------------------------------------------------------------
# the two prefill procedures
# ---------------------------------------------------------------------------------------

def full_prefill(cfg, weights, tokens: torch.Tensor, embeds: Optional[torch.Tensor] = None,
                 dtype=torch.float64, precision: str = "exact", n_layers: Optional[int] = None):
    """Standard prefill of the unpruned model over x_{1:N} (Sec. 3.3, the ordinary
    pipeline POP is compared with). tokens: int [B, N]; embeds: [B, N, d] or None.

    Returns dict: K, V lists over layers of [B, N, n_kv, hd]; logits [B, vocab];
    hidden [B, N, d] = the state leaving the last evaluated layer."""
    L = cfg.n_layers if n_layers is None else n_layers
    B, N = tokens.shape
    K = [torch.empty(B, N, cfg.n_kv_heads, cfg.head_dim, dtype=dtype) for _ in range(L)]
    V = [torch.empty(B, N, cfg.n_kv_heads, cfg.head_dim, dtype=dtype) for _ in range(L)]
    hidden = torch.empty(B, N, cfg.d_model, dtype=dtype)
    logits = torch.empty(B, cfg.vocab, dtype=dtype)
    pos = torch.arange(N)
    for b in range(B):
        x = embed(cfg, weights, tokens[b], None if embeds is None else embeds[b], dtype)
        for l in range(1, L + 1):
            x, K[l - 1][b], V[l - 1][b] = layer_forward(cfg, weights, l, x, pos, None, None,
                                                        dtype, precision)
        hidden[b] = x
        logits[b] = lm_logits(cfg, weights, x[N - 1], dtype)
    return {"K": K, "V": V, "logits": logits, "hidden": hidden}


def pop_prefill(cfg, weights, tokens: torch.Tensor, embeds: Optional[torch.Tensor], l_keep: int,
                dtype=torch.float64, precision: str = "exact", skip=None, boundary: bool = True,
                indep_kv: bool = True, fp8_kept: bool = False):
    """POP inference up to the first generated token, in the paper's two phases (Sec. 3.3).

    Phase 1, pruned prefill on x_{1:N-1}: layers 1..L_keep run in full; each layer
    l > L_keep only stores k_l, v_l computed from its own norm and projections on the state
    it receives (Eq. 14) and passes that state on unchanged (Eq. 15), so all pruned layers
    of the deep suffix see H = x_{L_keep+1}.

    Phase 2, first decode step on x_N: one position through all L layers, each appending
    its k, v to the cache (Eq. 2-3) and attending over positions 1..N.

    `skip` (a collection of 1-based layer numbers) states the pruned set S_skip of Eq. 4 / Eq. 14-15
    explicitly instead of the deep suffix {l_keep+1..L}; it may be shallow or interleaved (the
    layer-selection ablation of Sec. 4.4). A pruned layer projects whatever state reaches it.

    The two component ablations of Sec. 4.4.1 (Table "design choices"):
      boundary=False (the row without boundary handling): x_N is processed by the pruned prefill model like
        every other position: phase 1 covers all N positions, there is no phase 2, and the logits
        come from the state that leaves phase 1 at position N.
      indep_kv=False (the row without independent KV projections): pruned layers generate no cache entries in phase 1;
        in phase 2 (and in later decode steps) such a layer can only attend to positions >= N.
        Their K, V rows of positions 1..N-1 are returned as NaN ("absent").

    fp8_kept (deep-suffix set only): every position, x_N included, passes the kept layers with
    E4M3 operands in their four projections (precision "fp8"); x_N's pass through the deep layers
    streams E4M3 weights with bf16 activations ("fp8w"); the pruned layers' Eq. 14 projections use
    `precision`.

    Returns dict: K, V (N entries for every layer), logits [B, vocab],
    H [B, N-1, d] (the state leaving the last layer of phase 1 at positions 1..N-1; for the
    deep-suffix set this is the state leaving the kept stack), first_pos (per layer, 0-based: the
    first cache position later decode steps may attend to: 0, or for pruned layers when
    indep_kv is off N-1, the entry phase 2 wrote -- N if there was no phase 2 either),
    x_last [B, d] (the state of x_N that enters the final norm)."""
    L = cfg.n_layers
    if skip is None:
        assert 1 <= l_keep <= L
        skip = set(range(l_keep + 1, L + 1))
    skip = set(int(l) for l in skip)
    assert all(1 <= l <= L for l in skip)
    B, N = tokens.shape
    K = [torch.empty(B, N, cfg.n_kv_heads, cfg.head_dim, dtype=dtype) for _ in range(L)]
    V = [torch.empty(B, N, cfg.n_kv_heads, cfg.head_dim, dtype=dtype) for _ in range(L)]
    H = torch.empty(B, max(N - 1, 0), cfg.d_model, dtype=dtype)
    logits = torch.empty(B, cfg.vocab, dtype=dtype)
    x_out = torch.empty(B, cfg.d_model, dtype=dtype)
    for b in range(B):
        x_all = embed(cfg, weights, tokens[b], None if embeds is None else embeds[b], dtype)
        kc = [None] * L
        vc = [None] * L
        # ---- phase 1: pruned prefill on positions 0..N-2 (on all N positions without boundary handling)
        n1 = N - 1 if boundary else N
        if n1 > 0:
            pos = torch.arange(n1)
            x = x_all[:n1]
            for l in range(1, L + 1):
                if l not in skip:
                    x, kc[l - 1], vc[l - 1] = layer_forward(cfg, weights, l, x, pos, None, None,
                                                            dtype, "fp8" if fp8_kept else precision)
                elif indep_kv:
                    kc[l - 1], vc[l - 1] = kv_generation(cfg, weights, l, x, pos, dtype, precision)
                    # Eq. 15: x is handed to layer l+1 unchanged
            H[b] = x[: N - 1]
        if boundary:
            # ---- phase 2: x_N as the first decode step of the full model
            posN = torch.tensor([N - 1])
            x = x_all[N - 1: N]
            for l in range(1, L + 1):
                x, kc[l - 1], vc[l - 1] = layer_forward(cfg, weights, l, x, posN, kc[l - 1], vc[l - 1], dtype,
                                                        ("fp8" if l not in skip else "fp8w") if fp8_kept else precision)
            x_last = x[0]
        else:
            x_last = x[N - 1]
        for l in range(L):
            if kc[l] is None:                    # pruned layer without cache entries, no phase 2
                K[l][b] = float("nan")
                V[l][b] = float("nan")
            else:
                absent = N - kc[l].shape[0]      # positions a pruned layer holds nothing for
                K[l][b, :absent] = float("nan")
                V[l][b, :absent] = float("nan")
                K[l][b, absent:], V[l][b, absent:] = kc[l], vc[l]
        logits[b] = lm_logits(cfg, weights, x_last, dtype)
        x_out[b] = x_last
    horizon = N - 1 if boundary else N           # without phase 2 a pruned layer holds nothing at all
    first_pos = [horizon if (not indep_kv and (l + 1) in skip) else 0 for l in range(L)]
    return {"K": K, "V": V, "logits": logits, "H": H, "first_pos": first_pos, "x_last": x_out}


def decode_step(cfg, weights, tokens: torch.Tensor, K, V, dtype=torch.float64, precision: str = "exact",
                first_pos=None):
    """One decode step of the FULL model over an existing cache (the decode stage D of Sec. 3.2, Eq. 11, kept at full depth by Sec. 3.3; Eq. 1-3):
    POP prunes nothing in this stage. tokens: int [B], the token at
    position n = current cache length; K, V: lists (one per layer) of [B, n, n_kv, hd].
    first_pos (per layer, 0-based) is the first cache position a layer may attend to: positions
    before it hold nothing (the ablation without independent KV projections, Sec. 4.4.1).
    Returns (K', V', logits): caches with n + 1 entries and the next-token logits [B, vocab]."""
    L = cfg.n_layers
    B = tokens.shape[0]
    n = K[0].shape[1]
    K2 = [torch.empty(B, n + 1, cfg.n_kv_heads, cfg.head_dim, dtype=dtype) for _ in range(L)]
    V2 = [torch.empty(B, n + 1, cfg.n_kv_heads, cfg.head_dim, dtype=dtype) for _ in range(L)]
    logits = torch.empty(B, cfg.vocab, dtype=dtype)
    pos = torch.tensor([n])
    for b in range(B):
        x = embed(cfg, weights, tokens[b: b + 1], None, dtype)
        for l in range(1, L + 1):
            f = 0 if first_pos is None else int(first_pos[l - 1])
            x, k_cur, v_cur = layer_forward(cfg, weights, l, x, pos, K[l - 1][b, f:].to(dtype),
                                            V[l - 1][b, f:].to(dtype), dtype, precision, k_pos0=f)
            K2[l - 1][b, :f], V2[l - 1][b, :f] = K[l - 1][b, :f], V[l - 1][b, :f]
            K2[l - 1][b, f:], V2[l - 1][b, f:] = k_cur, v_cur
        logits[b] = lm_logits(cfg, weights, x[0], dtype)
    return K2, V2, logits


# ---------------------------------------------------------------------------------------
# cost model (counts of the work the method defines; no arithmetic of the method)
# ---------------------------------------------------------------------------------------

def layer_params(cfg) -> int:
    return cfg.d_model * (cfg.q_dim + 2 * cfg.kv_dim) + cfg.q_dim * cfg.d_model + 3 * cfg.d_model * cfg.d_ffn


def deep_third(n_layers: int):
    """The pruned set the paper uses throughout (Sec. 3.3: the deepest third of the layers): the last
    floor(L / 3) layers, as 1-based layer numbers."""
    p = n_layers // 3
    return set(range(n_layers - p + 1, n_layers + 1))


def kv_param_share(cfg) -> float:
    """Share of a layer's matrix parameters held by W^K and W^V (compare Sec. 3.3's "<5%")."""
    return 2 * cfg.kv_dim * cfg.d_model / layer_params(cfg)


def attention_pairs(n: int, window: int) -> int:
    if window <= 0 or window >= n:
        return n * (n + 1) // 2
    return window * (window + 1) // 2 + (n - window) * window


def prefill_flops(cfg, batch: int, n: int, l_keep: Optional[int]) -> float:
    """Algorithmic FLOPs: full layers on n positions (GEMMs + unmasked attention pairs) and,
    when l_keep < L, the K/V projections of pruned layers on n-1 positions. The boundary
    token's deep-layer pass and the head are bandwidth terms and are not counted."""
    L = cfg.n_layers
    lk = L if l_keep is None else l_keep
    total = 0.0
    for l in range(1, lk + 1):
        total += 2.0 * n * batch * layer_params(cfg)
        total += 4.0 * cfg.q_dim * batch * attention_pairs(n, cfg.layer_window(l))
    total += (L - lk) * 2.0 * (n - 1) * batch * cfg.d_model * 2 * cfg.kv_dim
    return total
