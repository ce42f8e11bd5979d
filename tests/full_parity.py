"""The whole CPU oracle against the library at the benchmark configurations' own sizes.

`compare(wl)` runs pop_prefill on the GPU in the launch configuration bench.py times (page size 128,
the workload's batch and L_keep), then the oracle's literal two-phase POP prefill (fp32, precision
"exact") on the same seeded weights and prompt, and returns one row per layer: the error of the
layer's K and V over all positions, of the boundary position alone, plus the state H leaving the
kept stack, the boundary token's final state and the logits. Nothing is asserted here; the tests
assert, and `python -m tests.full_parity <config> [--emu] [--layers L --keep K]` prints the table
(with --emu also the oracle in bf16-operand precision against the exact oracle, i.e. what rounding
the operands to bf16 costs by itself, no GPU involved).

The weights are drawn on the GPU by the shared generator (bit-identical to the CPU draw, which the
synth tests check) and handed to the oracle as CPU tensors: drawing 8-12 G parameters on the host
would take longer than the oracle itself.
"""
from __future__ import annotations

import argparse
import time

import torch

import pop_synth as ps
from oracle import pop_oracle as po

DEV = "cuda"


class DeviceDrawnWeights:
    """Weight provider for the oracle: tensors drawn on the GPU by pop_synth, returned on the CPU."""

    def __init__(self, cfg, seed=ps.DEFAULT_SEED):
        self.g = ps.SynthWeights(cfg, seed, device=DEV)

    def get(self, name, layer=0):
        return self.g.get(name, layer).cpu()

    def rows(self, name, layer, row_start, row_count):
        return self.g.rows(name, layer, row_start, row_count).cpu()

    def embedding_rows(self, ids):
        table = self.g.get("embed", 0)
        return table[ids.reshape(-1).long().to(DEV)].cpu()


def _err(got, ref):
    """(max|got-ref| / max|ref|, rms(got-ref) / rms(ref)) with the arithmetic done on the GPU in fp32/fp64."""
    ref = ref.to(DEV).float()
    d = got.to(DEV).float() - ref
    return ((d.abs().max() / ref.abs().max().clamp_min(1e-30)).item(),
            (d.double().pow(2).mean().sqrt() / ref.double().pow(2).mean().sqrt().clamp_min(1e-30)).item())


def compare(wl: ps.Workload, emu: bool = False, seed: int = ps.DEFAULT_SEED, log=print):
    from paper_2602_03295_b200.binding import KVCache, PopModel
    cfg, N, B, Lk, L = wl.model, wl.seq_len, wl.batch, wl.l_keep, wl.model.n_layers
    tokens, embeds = ps.make_prompt(wl, seed)
    model = PopModel(cfg, ps.SynthWeights(cfg, seed, device=DEV))
    cache = KVCache(cfg, B, N, 128, fill=float("nan"))
    t0 = time.time()
    logits = model.prefill(tokens.to(DEV), None if embeds is None else embeds.to(DEV), Lk, cache)
    assert model.last_status() == 0
    hidden, last = model.read_hidden(N, B)
    torch.cuda.synchronize()
    log(f"[{wl.key}] gpu prefill {time.time() - t0:.2f} s (first call, includes workspace set-up)")
    model.close()
    del model
    torch.cuda.empty_cache()

    w = DeviceDrawnWeights(cfg, seed)
    t0 = time.time()
    ref = po.pop_prefill(cfg, w, tokens, embeds, Lk, dtype=torch.float32, precision="exact")
    t_oracle = time.time() - t0
    log(f"[{wl.key}] oracle exact fp32 {t_oracle:.1f} s on {torch.get_num_threads()} threads")
    ref_emu = None
    if emu:
        t0 = time.time()
        ref_emu = po.pop_prefill(cfg, w, tokens, embeds, Lk, dtype=torch.float32, precision="bf16ops")
        log(f"[{wl.key}] oracle bf16ops fp32 {time.time() - t0:.1f} s")

    rows = []
    for l in range(L):
        k, v = cache.gather(l)
        r = {"layer": l + 1, "kind": "kept" if l < Lk else "pruned"}
        r["K"], r["K_rms"] = _err(k, ref["K"][l])
        r["V"], r["V_rms"] = _err(v, ref["V"][l])
        r["K_last"], _ = _err(k[:, N - 1], ref["K"][l][:, N - 1])
        r["V_last"], _ = _err(v[:, N - 1], ref["V"][l][:, N - 1])
        r["finite"] = bool(torch.isfinite(k.float()).all() and torch.isfinite(v.float()).all())
        if ref_emu is not None:
            r["K_emu"], _ = _err(ref_emu["K"][l], ref["K"][l])
            r["V_emu"], _ = _err(ref_emu["V"][l], ref["V"][l])
            r["K_vs_emu"], _ = _err(k, ref_emu["K"][l])
            r["V_vs_emu"], _ = _err(v, ref_emu["V"][l])
        rows.append(r)
    out = {"rows": rows, "oracle_s": t_oracle, "threads": torch.get_num_threads()}
    if N > 1:
        out["H"], out["H_rms"] = _err(hidden[:, : N - 1], ref["H"])
    out["x_last"], out["x_last_rms"] = _err(last, ref["x_last"])
    lg, rl = logits.cpu().double(), ref["logits"].double()
    out["logits"] = (lg - rl).abs().max().item()
    out["logits_rms"] = (lg - rl).pow(2).mean().sqrt().item()
    out["logits_std"] = rl.std().item()
    top2 = rl.topk(2, dim=-1).values
    out["argmax_agree"] = (lg.argmax(-1) == rl.argmax(-1)).tolist()
    out["top2_gap"] = (top2[:, 0] - top2[:, 1]).tolist()
    if ref_emu is not None:
        le = ref_emu["logits"].double()
        out["logits_emu"] = (le - rl).abs().max().item()
        out["logits_vs_emu"] = (lg - le).abs().max().item()
        out["H_emu"], _ = _err(ref_emu["H"], ref["H"])
        out["x_last_emu"], _ = _err(ref_emu["x_last"], ref["x_last"])
        out["argmax_agree_emu"] = (lg.argmax(-1) == le.argmax(-1)).tolist()
        out["argmax_emu_vs_exact"] = (le.argmax(-1) == rl.argmax(-1)).tolist()
    return out


def table(res) -> str:
    emu = "K_emu" in res["rows"][0]
    head = "layer kind    K_max    K_rms    V_max    V_rms   K_last   V_last"
    if emu:
        head += "  | K_emu    V_emu   K_vs_emu V_vs_emu"
    lines = [head]
    for r in res["rows"]:
        s = (f"{r['layer']:5d} {r['kind']:6s} {r['K']:8.2e} {r['K_rms']:8.2e} {r['V']:8.2e} {r['V_rms']:8.2e} "
             f"{r['K_last']:8.2e} {r['V_last']:8.2e}")
        if emu:
            s += f"  | {r['K_emu']:8.2e} {r['V_emu']:8.2e} {r['K_vs_emu']:8.2e} {r['V_vs_emu']:8.2e}"
        lines.append(s)
    for k in ("H", "H_rms", "x_last", "x_last_rms", "logits", "logits_rms", "logits_std", "argmax_agree", "top2_gap",
              "H_emu", "x_last_emu", "logits_emu", "logits_vs_emu", "argmax_agree_emu", "argmax_emu_vs_exact",
              "oracle_s", "threads"):
        if k in res:
            lines.append(f"{k}: {res[k]}")
    return "\n".join(lines)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("config", choices=sorted(ps.WORKLOADS))
    ap.add_argument("--emu", action="store_true", help="also run the oracle in bf16-operand precision")
    ap.add_argument("--layers", type=int, default=0, help="truncate the model to this many layers")
    ap.add_argument("--keep", type=int, default=0, help="L_keep of the truncated model")
    ap.add_argument("--seq", type=int, default=0, help="prompt length (default: the workload's)")
    ap.add_argument("--seed", type=int, default=ps.DEFAULT_SEED)
    a = ap.parse_args()
    wl = ps.WORKLOADS[a.config]
    if a.layers:
        wl = ps.Workload(wl.key, wl.model.replace(n_layers=a.layers), wl.batch, wl.seq_len, a.keep or a.layers,
                         wl.n_visual)
    if a.seq:
        wl = ps.Workload(wl.key, wl.model, wl.batch, a.seq, wl.l_keep, min(wl.n_visual, a.seq))
    print(f"{wl.key}: {wl.model.name} L={wl.model.n_layers} L_keep={wl.l_keep} N={wl.seq_len} seed={a.seed}", flush=True)
    print(table(compare(wl, emu=a.emu, seed=a.seed)), flush=True)


if __name__ == "__main__":
    main()
