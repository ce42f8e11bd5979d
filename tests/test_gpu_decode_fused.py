"""The single-kernel form of a decode step / of the boundary token's pass (paper Sec. 3.3; Sec. 3.2
Eq. 11): the library takes it for one sequence of a model with head_dim 128 and K extents that are
multiples of 256, i.e. at the true layer widths, which the tiny test models never reach. Here: layer
shapes of config 2 (Llama-3.1-8B: d 4096, 32/8 heads, FFN 14336) and of config 3 (Qwen3-8B: per-head
q/k norm, FFN 12288) at reduced depth and vocabulary, cache lengths chosen so that the key ranges of
the CTAs are empty, a single partial tile, and several tiles with a ragged last group.

Against the oracle's decode_step (fp64) with the tolerances of the other true-width tests: cache
entries per tensor max|err|/max|ref| <= 2e-2 (depth <= 3), logits within the depth budget of a
bf16-operand pipeline; and against the chain of single kernels (POP_DECODE_FUSED=0), which computes the
same roundings in a different summation order.
"""
import pytest
import torch

import pop_synth as ps
from oracle import pop_oracle as po
from tests.full_parity import DeviceDrawnWeights
from tests.gpu_util import logits_budget, rel_err
from tests.test_gpu_prefill import CachedWeights, build, KV_TOL

pytestmark = pytest.mark.gpu
DEV = "cuda"

WIDTHS = {
    "llama": ps.C2_LLAMA8B.replace(n_layers=2, vocab=8192, name="llama8b-width-2-layers"),
    "qwen": ps.C3_QWEN8B.replace(n_layers=2, vocab=8192, name="qwen3-8b-width-2-layers"),
    "window": ps.C2_LLAMA8B.replace(n_layers=3, vocab=8192, window=96, global_every=3, name="llama8b-width-windowed"),
}


def _steps(model, cfg, tokens, N, T, l_keep, page, cache=None):
    from paper_2602_03295_b200.binding import KVCache
    cache = cache or KVCache(cfg, 1, N + T, page, fill=float("nan"))
    out = [model.prefill(tokens[:, :N].contiguous().to(DEV), None, l_keep, cache).clone()]
    assert model.last_status() == 0
    for i in range(T):
        out.append(model.decode_step(tokens[:, N + i].contiguous().to(DEV), N + i, cache).clone())
        assert model.last_status() == 0
    return out, cache


@pytest.mark.parametrize("variant,N,T,l_keep,page", [("llama", 1, 3, 1, 16), ("llama", 200, 3, 1, 128),
                                                     ("qwen", 333, 2, 1, 64), ("window", 300, 3, 2, 128),
                                                     ("llama", 1500, 2, 2, 128)])
def test_fused_decode_steps_against_the_oracle(variant, N, T, l_keep, page):
    cfg = WIDTHS[variant]
    tokens = ps.uniform_tokens(41, 1, N + T, cfg.vocab)
    w = CachedWeights(DeviceDrawnWeights(cfg))
    ref = po.pop_prefill(cfg, w, tokens[:, :N], None, l_keep, dtype=torch.float64)
    K, V = ref["K"], ref["V"]
    model = build(cfg)
    got, cache = _steps(model, cfg, tokens, N, T, l_keep, page)
    assert model.last_launch_count() < 20          # the step is a handful of launches, not a chain per layer
    want = [ref["logits"]]
    for i in range(T):
        K, V, lg = po.decode_step(cfg, w, tokens[:, N + i].contiguous(), K, V)
        want.append(lg)
    for i, (g, r) in enumerate(zip(got, want)):
        assert torch.isfinite(g).all()
        d = g.cpu().double() - r.double()
        rms_b, max_b = logits_budget(cfg.n_layers, r.double().std().item())
        assert d.pow(2).mean().sqrt().item() <= rms_b and d.abs().max().item() <= max_b, (i, d.abs().max().item(), max_b)
    for l in range(cfg.n_layers):
        k, v = cache.gather(l, N + T)
        assert rel_err(k, K[l]) <= KV_TOL and rel_err(v, V[l]) <= KV_TOL, f"layer {l + 1}"


@pytest.mark.parametrize("variant,N", [("llama", 700), ("qwen", 129)])
def test_fused_kernel_follows_the_chain_of_single_kernels(variant, N, monkeypatch):
    cfg = WIDTHS[variant]
    T, l_keep = 3, 1
    tokens = ps.uniform_tokens(43, 1, N + T, cfg.vocab)
    model = build(cfg)
    fused, cf = _steps(model, cfg, tokens, N, T, l_keep, 128)
    n_fused = model.last_launch_count()
    monkeypatch.setenv("POP_DECODE_FUSED", "0")
    chain, cc = _steps(model, cfg, tokens, N, T, l_keep, 128)
    assert model.last_launch_count() > n_fused
    for a, b in zip(fused, chain):
        assert (a - b).abs().max().item() <= 2e-2 * max(1.0, b.abs().max().item())
    for l in range(cfg.n_layers):
        ka, va = cf.gather(l, N + T)
        kb, vb = cc.gather(l, N + T)
        assert rel_err(ka, kb) <= 1e-2 and rel_err(va, vb) <= 1e-2


def test_graph_replayed_greedy_loop_with_the_fused_kernel():
    # the cooperative kernel inside the captured step: tokens must be (or tie with) the arg-max of the
    # step-by-step logits for the same history
    from paper_2602_03295_b200.binding import KVCache
    cfg = WIDTHS["llama"]
    N, T, l_keep = 150, 6, 1
    tokens = ps.uniform_tokens(77, 1, N, cfg.vocab)
    model = build(cfg)
    ca = KVCache(cfg, 1, N + T + 1, 128)
    cb = KVCache(cfg, 1, N + T + 1, 128)
    la = model.prefill(tokens.to(DEV), None, l_keep, ca)
    model.prefill(tokens.to(DEV), None, l_keep, cb)
    first = la.argmax(-1).to(torch.int32)
    gen, last_logits = model.generate_greedy(first, N, T, ca)
    assert model.last_status() == 0
    gen = gen.cpu()
    tok = first
    for i in range(T):
        lg = model.decode_step(tok.contiguous(), N + i, cb)
        choice = gen[:, i].to(DEV).long()
        picked = lg.gather(1, choice[:, None])[:, 0]
        assert (lg.max(-1).values - picked).max().item() <= 1e-2
        tok = gen[:, i].to(DEV)
    assert (last_logits - lg).abs().max().item() <= 1e-2
    for l in range(cfg.n_layers):
        ka, va = ca.gather(l, N + T)
        kb, vb = cb.gather(l, N + T)
        assert rel_err(ka, kb) <= 1e-2 and rel_err(va, vb) <= 1e-2
