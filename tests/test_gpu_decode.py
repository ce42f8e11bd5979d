"""pop_decode_step (the full model's decode stage over the cache a prefill built, paper Sec. 3.2 Eq. 11 /
Sec. 3.3, where decoding keeps every layer) against the oracle's decode_step.

Tolerances as for the prefill: every layer's K and V per tensor max|err|/max|ref| <= 2e-2, logits
max|err| <= 5e-2 against the fp64 oracle; the greedy token (a decision taken in floating point) is
compared with the oracle in the kernel's precision, and a disagreement is only accepted where the
oracle's two best logits are a near-tie."""
import pytest
import torch

import pop_synth as ps
from oracle import pop_oracle as po
from tests.gpu_util import rel_err
from tests.test_gpu_prefill import TINY_VARIANTS, build, KV_TOL, LOGIT_TOL

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("variant", list(TINY_VARIANTS))
@pytest.mark.parametrize("B,N,T,l_keep,page", [(1, 1, 3, 1, 16), (2, 30, 5, 2, 16), (3, 127, 4, 1, 64)])
def test_decode_steps_after_a_pruned_prefill(variant, B, N, T, l_keep, page):
    from paper_2602_03295_b200.binding import KVCache
    cfg = TINY_VARIANTS[variant]
    tokens = ps.uniform_tokens(31, B, N + T, cfg.vocab)          # the last T are fed one by one
    w = ps.SynthWeights(cfg)
    ref = po.pop_prefill(cfg, w, tokens[:, :N], None, l_keep)
    K, V = ref["K"], ref["V"]
    model = build(cfg)
    cache = KVCache(cfg, B, N + T, page, fill=float("nan"))
    logits = model.prefill(tokens[:, :N].contiguous().to(DEV), None, l_keep, cache)
    assert model.last_status() == 0
    for i in range(T):
        tok = tokens[:, N + i].contiguous()
        K, V, want = po.decode_step(cfg, w, tok, K, V)
        logits = model.decode_step(tok.to(DEV), N + i, cache)
        assert model.last_status() == 0
        assert not torch.isnan(logits).any()
        assert (logits.cpu().double() - want).abs().max().item() <= LOGIT_TOL, f"step {i}"
    for l in range(cfg.n_layers):
        k, v = cache.gather(l, N + T)
        assert rel_err(k, K[l]) <= KV_TOL and rel_err(v, V[l]) <= KV_TOL, f"layer {l + 1}"


def test_greedy_continuation_agrees_with_the_oracle_in_kernel_precision():
    from paper_2602_03295_b200.binding import KVCache
    cfg = ps.C1_TINY
    n_prompts, N, T, l_keep = 32, 64, 6, 2
    tokens = ps.uniform_tokens(2000, n_prompts, N, cfg.vocab)
    w = ps.SynthWeights(cfg)
    ref = po.pop_prefill(cfg, w, tokens, None, l_keep, precision="bf16ops")
    K, V, want = ref["K"], ref["V"], ref["logits"]
    model = build(cfg)
    cache = KVCache(cfg, n_prompts, N + T, 16)
    got = model.prefill(tokens.to(DEV), None, l_keep, cache)
    agree = total = 0
    for i in range(T + 1):
        g, r = got.argmax(-1).cpu(), want.argmax(-1)
        top2 = want.topk(2, dim=-1).values
        for j in (g != r).nonzero().flatten().tolist():
            assert (top2[j, 0] - top2[j, 1]).item() < 1e-2       # only near-ties may differ
        agree += (g == r).sum().item()
        total += n_prompts
        if i == T:
            break
        tok = g.to(torch.int32)                                   # both sides continue with the GPU's choice
        K, V, want = po.decode_step(cfg, w, tok, K, V, precision="bf16ops")
        got = model.decode_step(tok.to(DEV), N + i, cache)
        assert model.last_status() == 0
    assert agree / total >= 0.99, (agree, total)


def test_decode_step_rejects_a_full_cache():
    from paper_2602_03295_b200 import PopError, POP_E_NOSPACE, POP_E_INVALID
    from paper_2602_03295_b200.binding import KVCache
    cfg = ps.C1_TINY
    model = build(cfg)
    tokens = ps.uniform_tokens(3, 1, 16, cfg.vocab).to(DEV)
    cache = KVCache(cfg, 1, 16, 16)                               # exactly one page
    model.prefill(tokens, None, 2, cache)
    logits = torch.full((1, cfg.vocab), 9.0, device=DEV)
    with pytest.raises(PopError) as e:
        model.decode_step(tokens[:, 0].contiguous(), 16, cache, logits)
    assert e.value.code == POP_E_NOSPACE
    with pytest.raises(PopError) as e:
        model.decode_step(tokens[:, 0].contiguous(), -1, cache, logits)
    assert e.value.code == POP_E_INVALID
    torch.cuda.synchronize()
    assert (logits == 9.0).all()


@pytest.mark.parametrize("variant", ["c1", "gemma", "hd256"])
def test_graph_replayed_greedy_loop_follows_the_step_by_step_path(variant):
    # pop_generate_greedy (one captured step replayed with a device-side position) against the same
    # steps issued one by one with the arg-max taken on the host: every generated token must be the
    # arg-max of the step-by-step logits for the same history (or tie with it to rounding), and the
    # caches must agree
    from paper_2602_03295_b200.binding import KVCache
    cfg = TINY_VARIANTS[variant]
    B, N, T, l_keep = 3, 40, 7, 2
    tokens = ps.uniform_tokens(77, B, N, cfg.vocab)
    model = build(cfg)
    ca = KVCache(cfg, B, N + T + 1, 16)
    cb = KVCache(cfg, B, N + T + 1, 16)
    la = model.prefill(tokens.to(DEV), None, l_keep, ca)
    lb = model.prefill(tokens.to(DEV), None, l_keep, cb)
    first = la.argmax(-1).to(torch.int32)
    gen, last_logits = model.generate_greedy(first, N, T, ca)
    assert model.last_status() == 0
    gen = gen.cpu()
    assert (gen >= 0).all() and (gen < cfg.vocab).all()
    tok = first
    for i in range(T):
        lg = model.decode_step(tok.contiguous(), N + i, cb)
        choice = gen[:, i].to(DEV).long()
        picked = lg.gather(1, choice[:, None])[:, 0]
        assert (lg.max(-1).values - picked).max().item() <= 1e-2      # the graph's token is (or ties with) the arg-max
        tok = gen[:, i].to(DEV)
    # (the graph path cannot size its key splits by the length, the step path does: the attention
    # outputs differ by bf16 roundings)
    assert (last_logits - lg).abs().max().item() <= 1e-2
    for l in range(cfg.n_layers):
        ka, va = ca.gather(l, N + T)
        kb, vb = cb.gather(l, N + T)
        assert rel_err(ka, kb) <= 1e-2 and rel_err(va, vb) <= 1e-2
