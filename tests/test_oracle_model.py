"""Pins for the oracle's two prefill procedures.

* an independent brute-force evaluator (pure Python / numpy loops, explicit N x N score
  matrix, no cache, every position recomputed from its prefix) on tiny shapes;
* third-party decoder implementations (transformers' Llama and Qwen3 modules) loaded with
  the same synthetic weights, as a library routine the textbook model reduces to;
* the structural identities that the paper's definitions of POP imply (Sec. 2.2, 3.3);
* planted mistakes in the oracle that these pins must catch.
"""
import math

import numpy as np
import pytest
import torch

import pop_synth as ps
from oracle import pop_oracle as po

D = torch.float64

TINY = ps.ModelConfig("pin", 3, 16, 4, 2, 4, 24, 40, 1e-5, 100.0, distinct_gains=True, weight_std=0.3)
VARIANTS = {
    "llama": TINY,
    "qknorm": TINY.replace(qk_norm=1),
    "gemma": TINY.replace(n_layers=4, act=1, post_norms=1, window=3, global_every=2, head_dim=8),
}


class DictWeights:
    def __init__(self, cfg, seed=11):
        sw = ps.SynthWeights(cfg, seed)
        self.t = {}
        for l in range(1, cfg.n_layers + 1):
            for name in ps.layer_tensor_shapes(cfg):
                self.t[(name, l)] = sw.get(name, l)
        for name in ps.global_tensor_shapes(cfg):
            self.t[(name, 0)] = sw.get(name, 0)

    def get(self, name, layer=0):
        return self.t[(name, layer)]


# ------------------------------------------------------------------ brute force (numpy, loops)

def _np(w, name, l):
    return w.get(name, l).double().numpy()


def _bf_norm(x, g, eps):
    return [x[i] * g[i] / math.sqrt(sum(v * v for v in x) / len(x) + eps) for i in range(len(x))]


def _bf_rope(vec, pos, theta):
    hd = len(vec)
    out = list(vec)
    for j in range(hd // 2):
        a = pos * theta ** (-2.0 * j / hd)
        out[j] = vec[j] * math.cos(a) - vec[j + hd // 2] * math.sin(a)
        out[j + hd // 2] = vec[j + hd // 2] * math.cos(a) + vec[j] * math.sin(a)
    return out


def brute_force_layer(cfg, w, l, X):
    """One decoder layer over all rows of X (list of N vectors), returning the new X and the
    K, V of every position, through an explicit N x N masked score matrix."""
    N = len(X)
    hd, nq, nkv = cfg.head_dim, cfg.n_q_heads, cfg.n_kv_heads
    Wq, Wk, Wv, Wo = (_np(w, n, l) for n in ("wq", "wk", "wv", "wo"))
    Q, K, V = [], [], []
    for i in range(N):
        h = np.array(_bf_norm(list(X[i]), _np(w, "ln_in", l), cfg.rms_eps))
        q, k, v = Wq @ h, Wk @ h, Wv @ h
        qh, kh = [], []
        for a in range(nq):
            t = list(q[a * hd:(a + 1) * hd])
            if cfg.qk_norm:
                t = _bf_norm(t, _np(w, "q_norm", l), cfg.rms_eps)
            qh.append(_bf_rope(t, i, cfg.rope_theta))
        for a in range(nkv):
            t = list(k[a * hd:(a + 1) * hd])
            if cfg.qk_norm:
                t = _bf_norm(t, _np(w, "k_norm", l), cfg.rms_eps)
            kh.append(_bf_rope(t, i, cfg.rope_theta))
        Q.append(qh)
        K.append(kh)
        V.append([list(v[a * hd:(a + 1) * hd]) for a in range(nkv)])
    win = cfg.layer_window(l)
    newX = []
    for i in range(N):
        att = []
        for a in range(nq):
            g = a * nkv // nq
            scores = np.full(N, -np.inf)
            for j in range(N):
                if j <= i and (win <= 0 or j > i - win):
                    scores[j] = sum(Q[i][a][c] * K[j][g][c] for c in range(hd)) / math.sqrt(hd)
            p = np.exp(scores - scores.max())
            p /= p.sum()
            att += [sum(p[j] * V[j][g][c] for j in range(N)) for c in range(hd)]
        o = Wo @ np.array(att)
        if cfg.post_norms:
            o = np.array(_bf_norm(list(o), _np(w, "post_attn_norm", l), cfg.rms_eps))
        y = np.array(X[i]) + o
        h2 = np.array(_bf_norm(list(y), _np(w, "ln_ffn", l), cfg.rms_eps))
        gate, up = _np(w, "w_gate", l) @ h2, _np(w, "w_up", l) @ h2
        if cfg.act == 0:
            a_ = gate / (1 + np.exp(-gate))
        else:
            a_ = 0.5 * gate * (1 + np.tanh(math.sqrt(2 / math.pi) * (gate + 0.044715 * gate ** 3)))
        f = _np(w, "w_down", l) @ (a_ * up)
        if cfg.post_norms:
            f = np.array(_bf_norm(list(f), _np(w, "post_ffn_norm", l), cfg.rms_eps))
        newX.append(y + f)
    return newX, np.array(K), np.array(V)


def brute_force_full(cfg, w, tokens):
    emb = _np(w, "embed", 0)
    X = [emb[t] for t in tokens]
    Ks, Vs = [], []
    for l in range(1, cfg.n_layers + 1):
        X, K, V = brute_force_layer(cfg, w, l, X)
        Ks.append(K)
        Vs.append(V)
    h = np.array(_bf_norm(list(X[-1]), _np(w, "final_norm", 0), cfg.rms_eps))
    return Ks, Vs, _np(w, "lm_head", 0) @ h


@pytest.mark.parametrize("variant", list(VARIANTS))
def test_full_prefill_matches_brute_force(variant):
    cfg = VARIANTS[variant]
    w = DictWeights(cfg)
    tokens = ps.uniform_tokens(3, 1, 6, cfg.vocab)
    out = po.full_prefill(cfg, w, tokens)
    Ks, Vs, logits = brute_force_full(cfg, w, tokens[0].tolist())
    for l in range(cfg.n_layers):
        assert np.allclose(out["K"][l][0].numpy(), Ks[l], atol=1e-10)
        assert np.allclose(out["V"][l][0].numpy(), Vs[l], atol=1e-10)
    assert np.allclose(out["logits"][0].numpy(), logits, atol=1e-10)


def test_full_prefill_is_causal_prefix_recomputation():
    cfg = VARIANTS["gemma"]
    w = DictWeights(cfg)
    tokens = ps.uniform_tokens(4, 1, 7, cfg.vocab)
    out = po.full_prefill(cfg, w, tokens)
    for n in (1, 4):
        pre = po.full_prefill(cfg, w, tokens[:, :n])
        for l in range(cfg.n_layers):
            assert torch.allclose(pre["K"][l][0], out["K"][l][0, :n], atol=1e-12)
            assert torch.allclose(pre["V"][l][0], out["V"][l][0, :n], atol=1e-12)


def test_batch_rows_are_independent_sequences():
    cfg = VARIANTS["llama"]
    w = DictWeights(cfg)
    tokens = ps.uniform_tokens(5, 2, 5, cfg.vocab)
    both = po.pop_prefill(cfg, w, tokens, None, 2)
    one = po.pop_prefill(cfg, w, tokens[1:], None, 2)
    assert torch.allclose(both["logits"][1], one["logits"][0], atol=1e-12)
    assert torch.allclose(both["K"][2][1], one["K"][2][0], atol=1e-12)


# ------------------------------------------------------------------ third-party decoders

def _load_hf(model, cfg, w):
    sd = {}
    pre = "model."
    sd[pre + "embed_tokens.weight"] = w.get("embed").double()
    sd[pre + "norm.weight"] = w.get("final_norm").double()
    sd["lm_head.weight"] = w.get("lm_head").double()
    names = {"wq": "self_attn.q_proj", "wk": "self_attn.k_proj", "wv": "self_attn.v_proj",
             "wo": "self_attn.o_proj", "w_gate": "mlp.gate_proj", "w_up": "mlp.up_proj",
             "w_down": "mlp.down_proj", "ln_in": "input_layernorm", "ln_ffn": "post_attention_layernorm",
             "q_norm": "self_attn.q_norm", "k_norm": "self_attn.k_norm"}
    for l in range(1, cfg.n_layers + 1):
        for n in ps.layer_tensor_shapes(cfg):
            sd[f"{pre}layers.{l-1}.{names[n]}.weight"] = w.get(n, l).double()
    missing, unexpected = model.load_state_dict(sd, strict=False)
    assert not unexpected and all("rotary" in m or "inv_freq" in m for m in missing), (missing, unexpected)


@pytest.mark.parametrize("family", ["llama", "qwen3"])
def test_full_prefill_matches_third_party_decoder(family):
    tr = pytest.importorskip("transformers")
    cfg = ps.ModelConfig("hf", 3, 32, 4, 2, 8, 48, 64, 1e-5, 10000.0, distinct_gains=True,
                         weight_std=0.2, qk_norm=1 if family == "qwen3" else 0)
    w = DictWeights(cfg)
    kw = dict(vocab_size=cfg.vocab, hidden_size=cfg.d_model, intermediate_size=cfg.d_ffn,
              num_hidden_layers=cfg.n_layers, num_attention_heads=cfg.n_q_heads,
              num_key_value_heads=cfg.n_kv_heads, head_dim=cfg.head_dim, rms_norm_eps=cfg.rms_eps,
              rope_theta=cfg.rope_theta, max_position_embeddings=64, tie_word_embeddings=False,
              attention_bias=False, hidden_act="silu", attn_implementation="eager")
    try:
        if family == "llama":
            hf_cfg = tr.LlamaConfig(mlp_bias=False, **kw)
            model = tr.LlamaForCausalLM(hf_cfg)
        else:
            hf_cfg = tr.Qwen3Config(use_sliding_window=False, **kw)
            model = tr.Qwen3ForCausalLM(hf_cfg)
    except Exception as e:  # library API drift: the other pins still hold
        pytest.skip(f"cannot build the third-party model: {e}")
    model = model.double().eval()
    _load_hf(model, cfg, w)
    tokens = ps.uniform_tokens(6, 2, 9, cfg.vocab)
    with torch.no_grad():
        ref = model(input_ids=tokens.long(), use_cache=True)
    out = po.full_prefill(cfg, w, tokens)
    # the library keeps its rotary tables in fp32, hence 1e-5 and not round-off of fp64
    assert torch.allclose(out["logits"], ref.logits[:, -1].double(), atol=1e-5)
    pkv = ref.past_key_values
    for l in range(cfg.n_layers):
        try:
            k_ref, v_ref = pkv.layers[l].keys, pkv.layers[l].values
        except AttributeError:
            k_ref, v_ref = pkv[l][0], pkv[l][1]
        assert torch.allclose(out["K"][l], k_ref.transpose(1, 2).double(), atol=1e-5)
        assert torch.allclose(out["V"][l], v_ref.transpose(1, 2).double(), atol=1e-5)


# ------------------------------------------------------------------ POP structure

def _setup(variant="gemma", n=8, batch=1, seed=9):
    cfg = VARIANTS[variant]
    w = DictWeights(cfg)
    tokens = ps.uniform_tokens(seed, batch, n, cfg.vocab)
    return cfg, w, tokens


def _maxdiff(a, b):
    return (a - b).abs().max().item()


@pytest.mark.parametrize("variant", list(VARIANTS))
def test_keeping_all_layers_is_the_full_prefill(variant):
    cfg, w, tokens = _setup(variant)
    full = po.full_prefill(cfg, w, tokens)
    pop = po.pop_prefill(cfg, w, tokens, None, cfg.n_layers)
    assert _maxdiff(full["logits"], pop["logits"]) < 1e-11
    for l in range(cfg.n_layers):
        assert _maxdiff(full["K"][l], pop["K"][l]) < 1e-11
        assert _maxdiff(full["V"][l], pop["V"][l]) < 1e-11


@pytest.mark.parametrize("variant", list(VARIANTS))
def test_pruning_only_the_last_layer_changes_nothing(variant):
    # the single pruned layer receives the exact x_L, so Eq. 14 equals Eq. 2 there, and the
    # boundary token runs the whole stack: cache and logits equal the full model's
    cfg, w, tokens = _setup(variant)
    full = po.full_prefill(cfg, w, tokens)
    pop = po.pop_prefill(cfg, w, tokens, None, cfg.n_layers - 1)
    assert _maxdiff(full["logits"], pop["logits"]) < 1e-11
    for l in range(cfg.n_layers):
        assert _maxdiff(full["K"][l], pop["K"][l]) < 1e-11
        assert _maxdiff(full["V"][l], pop["V"][l]) < 1e-11


def test_kept_layers_and_first_pruned_layer_have_the_full_models_cache():
    cfg, w, tokens = _setup("gemma")
    L = cfg.n_layers
    full = po.full_prefill(cfg, w, tokens)
    for l_keep in (1, 2):
        pop = po.pop_prefill(cfg, w, tokens, None, l_keep)
        for l in range(l_keep + 1):            # layers 1..L_keep and layer L_keep+1
            assert _maxdiff(full["K"][l], pop["K"][l]) < 1e-11
            assert _maxdiff(full["V"][l], pop["V"][l]) < 1e-11
        # deeper layers hold an approximation: they must differ from the full model's ...
        assert _maxdiff(full["K"][L - 1][:, :-1], pop["K"][L - 1][:, :-1]) > 1e-3
        # ... and so does the first token's distribution
        assert _maxdiff(full["logits"], pop["logits"]) > 1e-4


def test_pruned_layers_hold_eq14_of_the_kept_stacks_output():
    cfg, w, tokens = _setup("qknorm", n=7)
    l_keep = 1
    pop = po.pop_prefill(cfg, w, tokens, None, l_keep)
    N = tokens.shape[1]
    # H = x_{L_keep+1} on positions 0..N-2, from an independent run of the kept stack alone
    H = po.full_prefill(cfg, w, tokens[:, : N - 1], n_layers=l_keep)["hidden"][0]
    assert _maxdiff(H, pop["H"][0]) < 1e-12
    for l in range(l_keep + 1, cfg.n_layers + 1):
        g = w.get("ln_in", l).double()
        h = H * g / torch.sqrt(H.pow(2).mean(-1, keepdim=True) + cfg.rms_eps)
        k = (h @ w.get("wk", l).double().T).reshape(N - 1, cfg.n_kv_heads, cfg.head_dim)
        v = (h @ w.get("wv", l).double().T).reshape(N - 1, cfg.n_kv_heads, cfg.head_dim)
        gk = w.get("k_norm", l).double()
        k = k * gk / torch.sqrt(k.pow(2).mean(-1, keepdim=True) + cfg.rms_eps)
        # rotate with complex arithmetic instead of the oracle's rotate-half code
        half = cfg.head_dim // 2
        ang = torch.arange(N - 1, dtype=D)[:, None] * cfg.rope_theta ** (-2.0 * torch.arange(half, dtype=D) / cfg.head_dim)
        z = torch.complex(k[..., :half], k[..., half:]) * torch.polar(torch.ones_like(ang), ang)[:, None, :]
        k = torch.cat([z.real, z.imag], dim=-1)
        assert _maxdiff(pop["K"][l - 1][0, : N - 1], k) < 1e-11
        assert _maxdiff(pop["V"][l - 1][0, : N - 1], v) < 1e-11


def test_boundary_entry_of_deep_layers_comes_from_the_full_stack_state():
    # the last prompt position is a decode step of the full model (Sec. 3.3): its deep-layer
    # k, v come from the state that position really has there, not from H
    cfg, w, tokens = _setup("llama", n=6)
    pop = po.pop_prefill(cfg, w, tokens, None, 1)
    N = tokens.shape[1]
    l = cfg.n_layers
    H_all = po.full_prefill(cfg, w, tokens, n_layers=1)["hidden"][0]
    k_from_H, _ = po.kv_generation(cfg, w, l, H_all[N - 1:], torch.tensor([N - 1]), D, "exact")
    assert _maxdiff(pop["K"][l - 1][0, N - 1:], k_from_H) > 1e-4


def test_two_phase_boundary_equals_running_the_kept_stack_on_all_positions():
    # causality: in layers <= L_keep position N-1 depends on exact states only, so "prefill
    # N-1 then decode one" and "prefill N through the kept stack" agree
    cfg, w, tokens = _setup("gemma", n=9)
    l_keep = 2
    pop = po.pop_prefill(cfg, w, tokens, None, l_keep)
    fused = po.full_prefill(cfg, w, tokens, n_layers=l_keep)
    for l in range(l_keep):
        assert _maxdiff(pop["K"][l], fused["K"][l]) < 1e-11
        assert _maxdiff(pop["V"][l], fused["V"][l]) < 1e-11
    assert _maxdiff(pop["H"][0], fused["hidden"][0, :-1]) < 1e-11


def test_first_token_depends_on_the_projected_cache():
    cfg, w, tokens = _setup("llama", n=8)
    pop = po.pop_prefill(cfg, w, tokens, None, 1)

    class Zeroed(DictWeights):
        pass
    wz = Zeroed(cfg)
    wz.t[("wv", 3)] = torch.zeros_like(wz.t[("wv", 3)])
    popz = po.pop_prefill(cfg, wz, tokens, None, 1)
    assert _maxdiff(pop["logits"], popz["logits"]) > 1e-4


@pytest.mark.parametrize("variant", list(VARIANTS))
def test_decode_steps_reproduce_the_full_prefill_of_the_longer_prompt(variant):
    # the decode stage is the full model on one more position over the cache (Sec. 3.2, Eq. 11): feeding the
    # tokens of a longer prompt one by one after a full prefill of its first part must give that
    # longer prompt's cache and last-position logits (causality; nothing of the future is used)
    cfg, w, tokens = _setup(variant, n=11, batch=2)
    n0 = 7
    ref = po.full_prefill(cfg, w, tokens)
    part = po.full_prefill(cfg, w, tokens[:, :n0])
    K, V = part["K"], part["V"]
    for i in range(n0, tokens.shape[1]):
        K, V, logits = po.decode_step(cfg, w, tokens[:, i], K, V)
        assert K[0].shape[1] == i + 1
    assert _maxdiff(logits, ref["logits"]) < 1e-10
    for l in range(cfg.n_layers):
        assert _maxdiff(K[l], ref["K"][l]) < 1e-10 and _maxdiff(V[l], ref["V"][l]) < 1e-10
    # after a pruned prefill the decode step consumes the projected entries: the result differs
    # from the full model's unless at most one layer was pruned
    pop = po.pop_prefill(cfg, w, tokens[:, :n0], None, 1)
    _, _, lg = po.decode_step(cfg, w, tokens[:, n0], pop["K"], pop["V"])
    part2 = po.decode_step(cfg, w, tokens[:, n0], part["K"], part["V"])[2]
    assert _maxdiff(lg, part2) > 1e-6


def test_explicit_skip_sets():
    cfg, w, tokens = _setup("gemma", n=9, batch=2)      # 4 layers
    L = cfg.n_layers
    # the deep suffix given as a set is the l_keep form; the empty set is the full model
    a = po.pop_prefill(cfg, w, tokens, None, 2)
    b = po.pop_prefill(cfg, w, tokens, None, 0, skip={3, 4})
    full = po.full_prefill(cfg, w, tokens)
    none = po.pop_prefill(cfg, w, tokens, None, 0, skip=set())
    assert _maxdiff(a["logits"], b["logits"]) == 0 and _maxdiff(none["logits"], full["logits"]) < 1e-11
    for l in range(L):
        assert _maxdiff(a["K"][l], b["K"][l]) == 0 and _maxdiff(none["V"][l], full["V"][l]) < 1e-11
    # interleaved set {2, 4}: layer 1 is exact; layer 2 projects x_2 (Eq. 14) and hands it on (Eq. 15),
    # so kept layer 3 generates its K/V from x_2 as well -- both restated here from the full model's x_2
    r = po.pop_prefill(cfg, w, tokens, None, 0, skip={2, 4})
    N = tokens.shape[1]
    pos = torch.arange(N - 1)
    for bi in range(tokens.shape[0]):
        x1 = po.embed(cfg, w, tokens[bi], None, torch.float64)
        x2, k1, v1 = po.layer_forward(cfg, w, 1, x1, torch.arange(N), None, None, torch.float64, "exact")
        assert _maxdiff(r["K"][0][bi], k1) < 1e-11
        k2, v2 = po.kv_generation(cfg, w, 2, x2[: N - 1], pos, torch.float64, "exact")
        k3, v3 = po.kv_generation(cfg, w, 3, x2[: N - 1], pos, torch.float64, "exact")
        assert _maxdiff(r["K"][1][bi, : N - 1], k2) < 1e-11 and _maxdiff(r["V"][1][bi, : N - 1], v2) < 1e-11
        assert _maxdiff(r["K"][2][bi, : N - 1], k3) < 1e-11 and _maxdiff(r["V"][2][bi, : N - 1], v3) < 1e-11
    # the boundary position runs the full stack: through layer 3 it only meets exact cache entries
    # (layer 2 projected the exact x_2), so its entries equal the full model's; layer 3's context
    # entries came from x_2 instead of x_3, which shows in the boundary entry of layer 4
    for l in range(3):
        assert _maxdiff(r["K"][l][:, N - 1], full["K"][l][:, N - 1]) < 1e-10
    assert _maxdiff(r["K"][3][:, N - 1], full["K"][3][:, N - 1]) > 1e-6
    # a shallow set changes the result differently from a deep set of the same size
    sh = po.pop_prefill(cfg, w, tokens, None, 0, skip={1, 2})
    assert _maxdiff(sh["logits"], po.pop_prefill(cfg, w, tokens, None, 2)["logits"]) > 1e-6


def test_without_boundary_handling_the_last_token_sees_the_pruned_model():
    # Sec. 4.4.1, the variant without boundary handling: x_N goes through the pruned prefill model. Pruned layers pass
    # the state on unchanged (Eq. 15), so the logits are those of the model truncated to its kept
    # layers, and every position of a pruned layer -- the last included -- holds Eq. 14 of the kept
    # stack's output.
    for variant in ("llama", "gemma"):
        cfg, w, tokens = _setup(variant, n=9, batch=2)
        L, lk, N = cfg.n_layers, 2, tokens.shape[1]
        r = po.pop_prefill(cfg, w, tokens, None, lk, boundary=False)
        trunc = po.full_prefill(cfg, w, tokens, n_layers=lk)
        assert _maxdiff(r["logits"], trunc["logits"]) < 1e-11
        assert _maxdiff(r["logits"], po.pop_prefill(cfg, w, tokens, None, lk)["logits"]) > 1e-6
        for l in range(lk):
            assert _maxdiff(r["K"][l], trunc["K"][l]) < 1e-11 and _maxdiff(r["V"][l], trunc["V"][l]) < 1e-11
        for bi in range(tokens.shape[0]):
            for l in range(lk + 1, L + 1):
                k, v = po.kv_generation(cfg, w, l, trunc["hidden"][bi], torch.arange(N), torch.float64, "exact")
                assert _maxdiff(r["K"][l - 1][bi], k) < 1e-11 and _maxdiff(r["V"][l - 1][bi], v) < 1e-11
        assert r["first_pos"] == [0] * L


def test_without_independent_kv_a_pruned_layer_attends_to_the_last_token_only():
    # Sec. 4.4.1, the variant without independent KV projections: pruned layers generate no cache in the prefill, so in the first
    # decode step such a layer sees one key, its own: softmax over one score is 1 and the attention
    # output is the token's own value vector (repeated over the query heads of a group), whatever q is.
    cfg, w, tokens = _setup("llama", n=7, batch=2)          # 3 layers, no window, no post norms
    L, lk, N = cfg.n_layers, 2, tokens.shape[1]
    r = po.pop_prefill(cfg, w, tokens, None, lk, indep_kv=False)
    ref = po.pop_prefill(cfg, w, tokens, None, lk)
    assert r["first_pos"] == [0, 0, N - 1]
    # kept layers are untouched; the pruned layer holds nothing before the last position
    for l in range(lk):
        assert _maxdiff(r["K"][l], ref["K"][l]) == 0 and _maxdiff(r["V"][l], ref["V"][l]) == 0
    assert torch.isnan(r["K"][lk][:, : N - 1]).all() and torch.isnan(r["V"][lk][:, : N - 1]).all()
    # its entry of the last position comes from the true state, as with boundary handling
    assert _maxdiff(r["K"][lk][:, N - 1], ref["K"][lk][:, N - 1]) < 1e-11
    # closed form of the pruned layer for the last token, written with plain matrix products
    f64 = torch.float64
    G = cfg.n_q_heads // cfg.n_kv_heads
    for bi in range(tokens.shape[0]):
        full = po.full_prefill(cfg, w, tokens[bi: bi + 1], n_layers=lk)
        x = full["hidden"][0, N - 1]                         # the last token's state entering layer lk + 1
        v_own = r["V"][lk][bi, N - 1]                        # [n_kv, hd]
        a = v_own.repeat_interleave(G, dim=0).reshape(-1)    # attention output = own value per query head
        y = x + w.get("wo", lk + 1).to(f64) @ a
        h2 = po.rmsnorm(y, w.get("ln_ffn", lk + 1).to(f64), cfg.rms_eps)
        f = w.get("w_down", lk + 1).to(f64) @ po.gated_act(w.get("w_gate", lk + 1).to(f64) @ h2,
                                                             w.get("w_up", lk + 1).to(f64) @ h2, cfg.act)
        assert _maxdiff(r["logits"][bi], po.lm_logits(cfg, w, y + f, f64)) < 1e-10
    assert _maxdiff(r["logits"], ref["logits"]) > 1e-6
    # later decode steps keep that horizon: the pruned layer attends from position N-1 on, which is the
    # same as handing it a cache that starts there
    nxt = torch.tensor([5, 11])
    K2, V2, lg = po.decode_step(cfg, w, nxt, r["K"], r["V"], first_pos=r["first_pos"])
    Kc = [k.clone() for k in r["K"]]
    Vc = [v.clone() for v in r["V"]]
    for bi in range(2):
        x = po.embed(cfg, w, nxt[bi: bi + 1], None, f64)
        for l in range(1, L + 1):
            f0 = r["first_pos"][l - 1]
            x, kk, vv = po.layer_forward(cfg, w, l, x, torch.tensor([N]), Kc[l - 1][bi, f0:], Vc[l - 1][bi, f0:],
                                         f64, "exact", k_pos0=f0)
            assert _maxdiff(K2[l - 1][bi, f0:], kk) < 1e-12
        assert _maxdiff(lg[bi], po.lm_logits(cfg, w, x[0], f64)) < 1e-12
    # and the horizon matters: with the (NaN) rows before it the result would not even be finite
    assert torch.isfinite(lg).all()
    # a windowed model: the horizon and the window combine (keys must satisfy both)
    cfg, w, tokens = _setup("gemma", n=9, batch=1)           # window 3 in local layers
    r = po.pop_prefill(cfg, w, tokens, None, 2, indep_kv=False)
    assert torch.isfinite(r["logits"]).all()
    K2, V2, lg = po.decode_step(cfg, w, torch.tensor([3]), r["K"], r["V"], first_pos=r["first_pos"])
    assert torch.isfinite(lg).all()


def test_single_token_prompt_has_an_empty_first_phase():
    cfg, w, tokens = _setup("llama", n=1)
    pop = po.pop_prefill(cfg, w, tokens, None, 1)
    full = po.full_prefill(cfg, w, tokens)
    assert pop["H"].shape[1] == 0
    assert _maxdiff(pop["logits"], full["logits"]) < 1e-12


def test_embedding_rows_can_replace_tokens():
    cfg, w, tokens = _setup("llama", n=6)
    emb = w.get("embed")[tokens[0].long()].reshape(1, 6, -1)
    mixed = tokens.clone()
    mixed[:, :4] = -1
    a = po.pop_prefill(cfg, w, tokens, None, 2)
    b = po.pop_prefill(cfg, w, mixed, emb, 2)
    assert _maxdiff(a["logits"], b["logits"]) < 1e-12


def test_kernel_precision_mode_stays_close_to_exact_mode():
    cfg, w, tokens = _setup("gemma", n=8)
    a = po.pop_prefill(cfg, w, tokens, None, 2)
    b = po.pop_prefill(cfg, w, tokens, None, 2, precision="bf16ops")
    err = _maxdiff(a["logits"], b["logits"])
    assert 0 < err < 0.1 * a["logits"].abs().max().item()


# ------------------------------------------------------------------ planted mistakes

def _pins_hold(cfg, w, tokens):
    """Re-runs the cheap structural and brute-force pins; True when all hold."""
    try:
        out = po.full_prefill(cfg, w, tokens)
        Ks, Vs, logits = brute_force_full(cfg, w, tokens[0].tolist())
        ok = np.allclose(out["logits"][0].numpy(), logits, atol=1e-9)
        ok &= all(np.allclose(out["K"][l][0].numpy(), Ks[l], atol=1e-9) for l in range(cfg.n_layers))
        ok &= all(np.allclose(out["V"][l][0].numpy(), Vs[l], atol=1e-9) for l in range(cfg.n_layers))
        pop = po.pop_prefill(cfg, w, tokens, None, cfg.n_layers - 1)
        ok &= _maxdiff(out["logits"], pop["logits"]) < 1e-9
        ok &= all(_maxdiff(out["K"][l], pop["K"][l]) < 1e-9 for l in range(cfg.n_layers))
        pop1 = po.pop_prefill(cfg, w, tokens, None, 1)
        ok &= _maxdiff(out["K"][1], pop1["K"][1]) < 1e-9 and _maxdiff(out["V"][1], pop1["V"][1]) < 1e-9
        return bool(ok)
    except Exception:
        return False


MISTAKES = {
    "rope_sign": ("rope", lambda orig: (lambda x, p, t: orig(x, -p, t))),
    "rope_interleaved_pairs": ("rope", lambda orig: (lambda x, p, t: orig(
        x.reshape(*x.shape[:-1], -1, 2).transpose(-1, -2).reshape(x.shape), p, t))),
    "norm_without_gain": ("rmsnorm", lambda orig: (lambda x, g, e: orig(x, torch.ones_like(g), e))),
    "norm_eps_outside_root": ("rmsnorm", lambda orig: (lambda x, g, e: x / (x.pow(2).mean(-1, keepdim=True).sqrt() + e) * g)),
    "window_off_by_one": ("attention", lambda orig: (lambda q, k, v, qp, w, pr="exact": orig(q, k, v, qp, w + 1 if w > 0 else 0, pr))),
    "act_swapped": ("gated_act", lambda orig: (lambda g, u, a: orig(g, u, 1 - a))),
    "gate_up_swapped": ("gated_act", lambda orig: (lambda g, u, a: orig(u, g, a))),
    "pruned_layer_uses_previous_layers_weights": ("kv_generation", lambda orig: (
        lambda cfg, w, l, x, pos, dt, pr: orig(cfg, w, l - 1 if x.shape[0] > 1 and l == cfg.n_layers else l, x, pos, dt, pr))),
}


def test_pins_hold_unmodified():
    cfg, w, tokens = _setup("gemma", n=6)
    assert _pins_hold(cfg, w, tokens)


@pytest.mark.parametrize("name", list(MISTAKES))
def test_planted_mistake_is_caught(name, monkeypatch):
    cfg, w, tokens = _setup("gemma", n=6)
    attr, make = MISTAKES[name]
    monkeypatch.setattr(po, attr, make(getattr(po, attr)))
    assert not _pins_hold(cfg, w, tokens)
