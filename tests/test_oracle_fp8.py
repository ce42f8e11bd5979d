"""Pins of the oracle's FP8 (E4M3) rounding and scaling: against the format's definition enumerated
value by value, against torch's own float8_e4m3fn cast (a library routine the oracle does not call),
and closed forms."""
import itertools

import torch

from oracle import pop_oracle as po


def _all_e4m3_values():
    # every finite non-negative value from the format's definition: exponent field E (0..15), mantissa M (0..7);
    # E = 0: M/8 * 2^-6; else (1 + M/8) * 2^(E-7); the pattern E = 15, M = 7 is NaN
    vals = []
    for E, M in itertools.product(range(16), range(8)):
        if E == 15 and M == 7:
            continue
        vals.append(M / 8 * 2.0 ** -6 if E == 0 else (1 + M / 8) * 2.0 ** (E - 7))
    return sorted(vals)


def test_representable_values_are_fixed_points_and_the_largest_is_448():
    v = torch.tensor(_all_e4m3_values(), dtype=torch.float64)
    assert v.max().item() == 448.0 and v[1].item() == 2.0 ** -9 and len(v) == 127
    assert torch.equal(po.e4m3_round(v), v)
    assert torch.equal(po.e4m3_round(-v), -v)


def test_rounding_goes_to_the_nearest_value_ties_to_even():
    v = _all_e4m3_values()
    for lo, hi in zip(v[:-1], v[1:]):
        mid = (lo + hi) / 2
        x = torch.tensor([lo + 0.49 * (hi - lo), lo + 0.51 * (hi - lo), mid], dtype=torch.float64)
        r = po.e4m3_round(x)
        assert r[0].item() == lo and r[1].item() == hi
        # the tie goes to the value whose mantissa is even: consecutive values alternate parity
        even = lo if v.index(lo) % 2 == 0 else hi
        assert r[2].item() == even, (lo, hi)
    assert po.e4m3_round(torch.tensor([1e9, -1e9, 460.0, 0.0, 2.0 ** -11])).tolist() == [448.0, -448.0, 448.0, 0.0, 0.0]


def test_agrees_with_the_library_cast():
    g = torch.Generator().manual_seed(3)
    x = torch.cat([torch.randn(20000, generator=g) * s for s in (1e-3, 0.05, 1.0, 30.0, 200.0)])
    x = x.clamp(-448, 448)                                    # the library cast does not saturate
    lib = x.to(torch.float8_e4m3fn).to(torch.float64)
    assert torch.equal(po.e4m3_round(x), lib)


def test_row_and_tensor_scales():
    g = torch.Generator().manual_seed(4)
    h = torch.randn(5, 64, generator=g) * torch.tensor([[1e-3], [1.0], [50.0], [0.0], [7.0]])
    q, s = po.quant_rows_e4m3(h)
    assert s[3].item() == 1.0 and (q[3] == 0).all()
    for r in (0, 1, 2, 4):
        assert q[r].abs().max().item() == 448.0               # the row's largest magnitude maps to the format's
        # dequantised values are within half a quantum (2^-4 relative for normal numbers) of the input
        assert ((q[r] * s[r] - h[r].double()).abs() <= h[r].abs().double() * 2.0 ** -4 + s[r] * 2.0 ** -10).all()
    ws = [torch.randn(8, 16, generator=g) * 0.02, torch.randn(4, 16, generator=g) * 0.05]
    qs, sc = po.quant_tensors_e4m3(ws)
    assert max(float(t.abs().max()) for t in qs) == 448.0
    assert abs(sc - max(float(w.abs().max()) for w in ws) / 448.0) < 1e-9


def test_fp8_projections_restated_with_the_library_cast():
    # the QKV and gate/up products of a layer in "fp8" precision, restated with torch's float8 cast:
    # codes of LN(x) per row and of the fused weight matrices per matrix, exact products, scales last
    import pop_synth as ps
    cfg = ps.ModelConfig("pin8", 2, 32, 4, 2, 8, 48, 50, 1e-5, 100.0, distinct_gains=True, weight_std=0.3)
    w = ps.SynthWeights(cfg)
    x = torch.randn(6, cfg.d_model, generator=torch.Generator().manual_seed(8), dtype=torch.float64) * 3
    f8 = torch.float8_e4m3fn

    def rows(h):
        h32 = h.float()
        amax = h32.abs().amax(-1, keepdim=True)
        return (h32 * (448.0 / amax)).to(f8).double(), (amax / 448.0).double()

    def mats(names, layer):
        ws = [w.get(n, layer).float() for n in names]
        amax = torch.stack([t.abs().max() for t in ws]).max()
        return [(t * (448.0 / amax)).to(f8).double() for t in ws], float(amax / 448.0)

    pos = torch.arange(6)
    k, v = po.kv_generation(cfg, w, 1, x, pos, torch.float64, "fp8")
    hq, sa = rows(po.rmsnorm(x, w.get("ln_in", 1).double(), cfg.rms_eps))
    (wq, wk, wv), sw = mats(("wq", "wk", "wv"), 1)
    v_ref = ((hq @ wv.T) * sa * sw).reshape(6, cfg.n_kv_heads, cfg.head_dim)
    v_ref = v_ref.float().to(torch.bfloat16).double()                      # cache entries are bf16
    assert (v - v_ref).abs().max().item() < 1e-12
    k_ref = po.rope(((hq @ wk.T) * sa * sw).reshape(6, cfg.n_kv_heads, cfg.head_dim), pos, cfg.rope_theta)
    assert (k - k_ref.float().to(torch.bfloat16).double()).abs().max().item() < 1e-12
    # output and down projections: rows of the bf16-stored operand, one scale each; the matrix one scale
    a = (torch.randn(6, cfg.q_dim, generator=torch.Generator().manual_seed(9)) * 2).to(torch.bfloat16)
    aq, sa2 = rows(a.double())
    (wo8,), swo = mats(("wo",), 2)
    assert (po._proj_fp8(a.double(), w.get("wo", 2), torch.float64) - (aq @ wo8.T) * sa2 * swo).abs().max().item() < 1e-12
    # the quantised model stays near the unquantised one, and is not it
    tokens = ps.uniform_tokens(3, 1, 12, cfg.vocab)
    a = po.full_prefill(cfg, w, tokens, precision="fp8")
    b = po.full_prefill(cfg, w, tokens, precision="bf16ops")
    for l in range(cfg.n_layers):
        err = (a["V"][l] - b["V"][l]).abs().max() / b["V"][l].abs().max()
        assert 0 < err.item() < 0.35          # 3 mantissa bits, rows of 32 terms
    # kept layers only: with every layer pruned but the first, the deep layers' entries of positions < N-1
    # are bf16 projections of an fp8-computed state
    r = po.pop_prefill(cfg, w, tokens, None, 1, precision="bf16ops", fp8_kept=True)
    r0 = po.pop_prefill(cfg, w, tokens, None, 1, precision="bf16ops")
    assert (r["K"][0] - a["K"][0]).abs().max().item() == 0                 # layer 1 is the fp8 layer of the full run
    assert (r["K"][1] - r0["K"][1]).abs().max().item() > 0                 # H differs
    kk, vv = po.kv_generation(cfg, w, 2, r["H"][0], torch.arange(11), torch.float64, "bf16ops")
    assert (r["K"][1][0, :11] - kk).abs().max().item() == 0


def test_weight_only_precision_is_the_kernel_precision_on_dequantised_weights():
    # "fp8w": a layer in kernel (bf16) precision whose four projection matrices are replaced by
    # code * scale -- restated by running kernel precision on a weight set patched that way
    import pop_synth as ps
    cfg = ps.ModelConfig("pin8w", 2, 32, 4, 2, 8, 48, 50, 1e-5, 100.0, distinct_gains=True, weight_std=0.3)
    w = ps.SynthWeights(cfg)
    f8 = torch.float8_e4m3fn

    class Patched:
        def get(self, name, layer):
            groups = [("wq", "wk", "wv"), ("w_gate", "w_up"), ("wo",), ("w_down",)]
            for g in groups:
                if name in g:
                    amax = max(float(w.get(n, layer).float().abs().max()) for n in g)
                    t = w.get(name, layer).float()
                    return (t * (448.0 / amax)).to(f8).double() * (amax / 448.0)
            return w.get(name, layer)
    x = torch.randn(5, cfg.d_model, generator=torch.Generator().manual_seed(12), dtype=torch.float64)
    pos = torch.arange(5)
    a = po.layer_forward(cfg, w, 2, x, pos, None, None, torch.float64, "fp8w")
    b = po.layer_forward(cfg, Patched(), 2, x, pos, None, None, torch.float64, "bf16ops")
    for u, v in zip(a, b):
        assert (u - v).abs().max().item() < 1e-5          # the scale is an fp32 number in the oracle
    c = po.layer_forward(cfg, w, 2, x, pos, None, None, torch.float64, "bf16ops")
    assert (a[0] - c[0]).abs().max().item() > 1e-4
