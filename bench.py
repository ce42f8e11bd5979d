#!/usr/bin/env python
"""Benchmark of the POP pruned-prefill path on B200.

A step is one pop_prefill call (embedding, L_keep full layers over the prompt, the pruned layers'
independent K/V projections, the boundary token through the deep layers, final norm + output
head) on one batch of seeded synthetic input. Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2|c3|c4|c1]
                  [--seq-len S --batch B --l-keep L] [--impl reference]

N > 1 (under torchrun): independent replicas, one prompt batch per GPU, no data-path collective
("weak" scaling); time is the maximum over ranks.  --impl reference times the CPU oracle, as it
stands, on a bounded slice of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

import pop_synth as ps  # noqa: E402

METRIC = "pop_prefill_tokens_per_s"
UNIT = "tokens/s"
KERNELS = ["gemm_qkv", "gemm_o", "gemm_gateup", "gemm_down", "kvproj", "attention", "attention_local", "gemv_head",
           "gemv_gateup",
           "decode_attention", "decode_step", "rmsnorm", "rope_cache", "gemm_gateup_fp8", "gemm_qkvshape_fp8",
           "rmsnorm_fp8"]


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2", choices=sorted(ps.WORKLOADS))
    ap.add_argument("--seq-len", type=int, default=0)
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--l-keep", type=int, default=0)
    ap.add_argument("--page-size", type=int, default=128)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sweep", action="store_true",
                    help="config-5 sweep on the workload's model shape: prompt length x batch x L_keep/L, one "
                         "JSON line per point (POP vs full-depth prefill, tokens/s, TTFT, path TFLOP/s)")
    ap.add_argument("--precision", default="bf16", choices=["bf16", "fp8"],
                    help="fp8: E4M3 operands in the kept layers' four projection GEMMs (a second workload; "
                         "the default line is bf16 throughout)")
    ap.add_argument("--chunked", action="store_true",
                    help="long prompts through pop_prefill_chunked (one JSON line per point) instead of the default run")
    ap.add_argument("--kernel", default="", choices=[""] + KERNELS,
                    help="time ONE kernel of the path alone, at the workload's per-layer shape, through its "
                         "kernel-level C-ABI entry point (a small case for profiling)")
    return ap.parse_args()


def resolve_workload(a) -> ps.Workload:
    wl = ps.WORKLOADS[a.workload]
    n = a.seq_len or wl.seq_len
    nv = min(wl.n_visual, n - 1) if wl.n_visual else 0
    return ps.Workload(wl.key, wl.model, a.batch or wl.batch, n, a.l_keep or wl.l_keep, nv)


# DRAM read+write bytes of one down-projection GEMM launch at the c2 layer shape, from the ncu capture
# summarised in profiles/gemm_pair_kernel_c2.md; valid only for the kernel source it was taken on.
GEMM_TRAFFIC = {"bytes_per_launch": 1.516e9, "launch": "down projection, M 8192 N 4096 K 14336 (CTA-pair form)",
                "gemm_cu_sha256": "1ef20f01ac169023a3567ef5a93b5b790c5ffc32fe622ab0241bbd2919212d1e"}


def gemm_traffic():
    import hashlib
    try:
        with open(os.path.join(ROOT, "paper_2602_03295_b200", "csrc", "gemm.cu"), "rb") as f:
            sha = hashlib.sha256(f.read()).hexdigest()
    except OSError:
        return None
    return GEMM_TRAFFIC["bytes_per_launch"] if sha == GEMM_TRAFFIC["gemm_cu_sha256"] else None


def load_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    except Exception:
        return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons of one GPU with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows = []
        self.proc = None
        self.gpu = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            parts = [p.strip() for p in r.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v == "Active":
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def replica_seed(rank: int) -> int:
    """Prompt seed of replica `rank`: every replica works on its own batch of prompts."""
    return ps.DEFAULT_SEED + 101 * rank


def max_over_ranks(ms: float, device="cpu") -> float:
    """Elapsed time of the slowest replica (all-reduce MAX when a process group is up)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.item()


def aggregate_tokens_per_s(tokens_per_replica: int, world: int, ms_per_step: float) -> float:
    """Whole-job throughput of `world` independent replicas timed by the slowest one."""
    return tokens_per_replica * world / (ms_per_step * 1e-3)


# ------------------------------------------------------------------------------------ CPU oracle legs

class _CachedWeights:
    def __init__(self, w):
        self.w, self.c = w, {}

    def get(self, name, layer=0):
        if (name, layer) not in self.c:
            self.c[(name, layer)] = self.w.get(name, layer)
        return self.c[(name, layer)]

    def embedding_rows(self, ids):
        return self.w.embedding_rows(ids)


def oracle_sample(wl: ps.Workload, repeats: int, warmup: int):
    """Times the oracle, as it stands (fp32, torch CPU ops), on a bounded sample of the workload, the same
    one in the `cpu_baseline` leg and in `--impl reference`: at the workload's own prompt length (attention
    is quadratic in it, so a shorter slice would flatter the CPU) ONE full decoder layer (layer 1) over the
    first sequence, ONE pruned layer's K/V generation (Eq. 14) over it, ONE deep layer's single-position
    pass of the boundary token over a cache of that length, and the output head on one position.
    Returns (timed seconds per sample, extrapolated seconds per whole step, parts): a whole step is
    L_keep x layer + P x kv-projection + P x boundary layer + head, per sequence."""
    from oracle import pop_oracle as po
    cfg = wl.model
    tokens, embeds = ps.make_prompt(wl)
    w = _CachedWeights(ps.SynthWeights(cfg))
    n = wl.seq_len
    x = po.embed(cfg, w, tokens[0, :n], None if embeds is None else embeds[0, :n], torch.float32)
    for name in ps.layer_tensor_shapes(cfg):
        w.get(name, 1)
    w.get("lm_head", 0), w.get("final_norm", 0)
    pos = torch.arange(n)
    P = cfg.n_layers - wl.l_keep
    timed, whole = [], []
    parts = {}
    for i in range(warmup + repeats):
        t0 = time.perf_counter()
        po.layer_forward(cfg, w, 1, x, pos, None, None, torch.float32, "exact")
        t1 = time.perf_counter()
        k, v = po.kv_generation(cfg, w, 1, x[: n - 1], pos[: n - 1], torch.float32, "exact")
        t2 = time.perf_counter()
        po.layer_forward(cfg, w, 1, x[n - 1:], pos[n - 1:], k, v, torch.float32, "exact")
        t3 = time.perf_counter()
        po.lm_logits(cfg, w, x[-1], torch.float32)
        t4 = time.perf_counter()
        if i >= warmup:
            timed.append(t4 - t0)
            whole.append(wl.batch * (wl.l_keep * (t1 - t0) + P * (t2 - t1) + P * (t3 - t2) + (t4 - t3)))
            parts = {"layer_s": t1 - t0, "kv_projection_s": t2 - t1, "boundary_layer_s": t3 - t2, "head_s": t4 - t3}
    return timed, whole, parts


def oracle_sample_text(wl, parts):
    P = wl.model.n_layers - wl.l_keep
    return (f"oracle (fp32, torch CPU ops) at the workload's own length, {wl.seq_len} positions of one sequence: one "
            f"full decoder layer {parts['layer_s']:.2f} s, one pruned layer's K/V generation "
            f"{parts['kv_projection_s']:.2f} s, one deep layer's single-position boundary pass "
            f"{parts['boundary_layer_s']:.2f} s, output head {parts['head_s']:.3f} s; tokens/s = batch x {wl.seq_len} / "
            f"(batch x (L_keep={wl.l_keep} x layer + {P} x kv + {P} x boundary + head)), i.e. extrapolated over the "
            f"depth from that one-layer sample")


def run_reference(a, wl):
    rank, world, _ = dist_env()
    if rank != 0:
        return
    timed, whole, parts = oracle_sample(wl, a.steps, min(a.warmup, 1))
    t_sample = sum(timed) / len(timed)
    t_step = sum(whole) / len(whole)
    value = wl.seq_len * wl.batch / t_step
    cores = torch.get_num_threads()
    desc = oracle_sample_text(wl, parts)
    # ms_per_step is what one timed step of THIS run took (the one-layer sample); the whole-path time
    # the metric is quoted on is extrapolated from it and sits under its own key
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": a.gpus,
           "steps": a.steps, "warmup": min(a.warmup, 1), "ms_per_step": t_sample * 1e3,
           "extrapolated_whole_path_ms": t_step * 1e3, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
           "config": workload_config(wl, a), "gpu_launches": 0,
           "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out), flush=True)


def workload_config(wl, a):
    cfg = wl.model
    return {"workload": f"{wl.key}: {cfg.name}, L={cfg.n_layers}, batch {wl.batch} x {wl.seq_len} tokens"
                        f"{' (' + str(wl.n_visual) + ' as embeddings)' if wl.n_visual else ''}, L_keep={wl.l_keep}",
            "global_batch": wl.batch * max(1, a.gpus), "seq_len": wl.seq_len, "l_keep": wl.l_keep,
            "page_size": a.page_size, "parallelism": f"replicas x{max(1, a.gpus)}",
            "l2": "inputs larger than L2 (weights 2x params bytes stream every step)"}


# ------------------------------------------------------------------------------------ GPU leg

def run_ours(a, wl):
    from oracle import pop_oracle as po   # cost model + cpu_baseline leg only
    import paper_2602_03295_b200 as pk
    from paper_2602_03295_b200.binding import KVCache, PopModel

    rank, world, local = dist_env()
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    else:
        torch.cuda.set_device(0)
    dev = torch.device("cuda", local if world > 1 else 0)
    cfg = wl.model
    lib = pk.lib()
    model = PopModel(cfg, ps.SynthWeights(cfg, device=dev), device=dev)
    fp8 = a.precision == "fp8"
    if fp8:
        model.enable_fp8()
    tokens_h, embeds_h = ps.make_prompt(wl, replica_seed(rank))
    tokens_h = tokens_h.pin_memory()
    embeds_h = None if embeds_h is None else embeds_h.pin_memory()
    tokens = tokens_h.to(dev)
    embeds = None if embeds_h is None else embeds_h.to(dev)
    DECODE_STEPS = 32
    cache = KVCache(cfg, wl.batch, wl.seq_len + DECODE_STEPS, a.page_size, device=dev)   # room for the decode leg
    logits = torch.empty(wl.batch, cfg.vocab, dtype=torch.float32, device=dev)
    logits_h = torch.empty(wl.batch, cfg.vocab, dtype=torch.float32).pin_memory()

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    def step():
        model.prefill(tokens, embeds, wl.l_keep, cache, logits)

    def step_e2e():
        t = tokens_h.to(dev, non_blocking=True)
        e = None if embeds_h is None else embeds_h.to(dev, non_blocking=True)
        model.prefill(t, e, wl.l_keep, cache, logits)
        logits_h.copy_(logits, non_blocking=True)

    def timed(fn, steps):
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        barrier()
        return max_over_ranks(e0.elapsed_time(e1), dev)

    for _ in range(max(a.warmup, 3)):
        step()
    sampler = ClockSampler(local if world > 1 else 0)
    sampler.start()
    total_ms = timed(step, a.steps)
    clocks = sampler.stop()
    status = model.last_status()
    launches = model.last_launch_count()
    ms_step = total_ms / a.steps
    n_tok = wl.batch * wl.seq_len * world
    value = aggregate_tokens_per_s(wl.batch * wl.seq_len, world, ms_step)

    # end to end: host tokens (and embeddings) in, host logits out, copies inside the timed region
    step_e2e()
    e2e_ms = timed(step_e2e, a.steps) / a.steps
    h2d = tokens_h.numel() * 4 + (0 if embeds_h is None else embeds_h.numel() * 2)
    d2h = logits_h.numel() * 4

    # the library's own full-depth prefill, for the speedup POP is about
    def step_full():
        model.full_prefill(tokens, embeds, cache, logits)
    step_full()
    full_ms = timed(step_full, max(2, a.steps // 2)) / max(2, a.steps // 2)

    # decode stage over the cache the pruned prefill built: the full model, one position per call
    step()
    dec_tok = tokens[:, -1].contiguous()
    for i in range(3):
        model.decode_step(dec_tok, wl.seq_len + i, cache, logits)
    barrier()
    d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    d0.record()
    for i in range(DECODE_STEPS):
        model.decode_step(dec_tok, wl.seq_len + i, cache, logits)
    d1.record()
    barrier()
    dec_ms = max_over_ranks(d0.elapsed_time(d1), dev) / DECODE_STEPS
    dec_status = model.last_status()
    # the same steps as an on-device greedy loop: one captured step replayed per token
    model.generate_greedy(dec_tok.to(torch.int32), wl.seq_len, 4, cache, logits)
    barrier()
    d0.record()
    model.generate_greedy(dec_tok.to(torch.int32), wl.seq_len, DECODE_STEPS, cache, logits)
    d1.record()
    barrier()
    gen_ms = max_over_ranks(d0.elapsed_time(d1), dev) / DECODE_STEPS
    dec_status = dec_status or model.last_status()
    # bytes a decode step streams: bf16 weights, or E4M3 layer matrices (1 byte) and the bf16 output head
    weight_bytes = (1.0 if fp8 else 2.0) * cfg.n_layers * po.layer_params(cfg) + 2.0 * cfg.vocab * cfg.d_model

    # per-kernel-class durations of one more step, CUDA events on the launching stream
    # (as many steps as the timed region, back to back, so that clocks sit where they sat there)
    for _ in range(2):
        step()
    lib.profile(True)
    for _ in range(a.steps):
        step()
    torch.cuda.synchronize()
    lib.profile(False)
    prof = {k: (v[0] / a.steps, v[1] / a.steps, v[2] // a.steps) for k, v in lib.profile_summary().items()}
    peaks = load_peaks()
    gemm_ms, gemm_flops, gemm_n = prof["gemm"]
    att_ms, att_flops, att_n = prof["attention"]
    flops = po.prefill_flops(cfg, wl.batch, wl.seq_len, wl.l_keep)
    peak_tf = peaks["bf16_tflops_sustained"]          # the GEMM runs inside a long step
    achieved_tf = gemm_flops / (gemm_ms * 1e-3) / 1e12 if gemm_ms > 0 else 0.0
    breakdown = {k: {"ms": round(v[0], 3), "launches": v[2]} for k, v in prof.items()}
    breakdown["attention"]["tflops"] = round(att_flops / (att_ms * 1e-3) / 1e12, 1) if att_ms > 0 else None

    if fp8:
        # the GEMM class mixes dtypes: its peak is total flop / (fp8 flop / (2 x bf16 peak) + bf16 flop / bf16 peak),
        # 2 being the nominal fp8 : bf16 ratio
        f_pad = (cfg.d_ffn + 127) // 128 * 128
        rows = wl.batch * wl.seq_len
        qd_ = cfg.n_q_heads * cfg.head_dim
        f8 = 2.0 * rows * cfg.d_model * (qd_ + 2 * cfg.n_kv_heads * cfg.head_dim + 2 * f_pad + qd_ + cfg.d_ffn) * wl.l_keep
        tot = achieved_tf * 1e12 * gemm_ms * 1e-3
        peak_tf = tot / (f8 / (2 * peak_tf) + (tot - f8) / peak_tf) if peak_tf else peak_tf
    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": a.steps, "warmup": max(a.warmup, 3),
           "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
           "dtype": "e4m3 (the four projections of kept layers) + bf16" if fp8 else "bf16", "data": "synthetic",
           "config": workload_config(wl, a),
           "ttft_ms": ms_step, "full_prefill_ms": full_ms, "speedup_vs_full_prefill": full_ms / ms_step,
           "speedup_ceiling_flop_ratio": po.prefill_flops(cfg, wl.batch, wl.seq_len, None) / flops,
           "speedup_ceiling_layer_ratio": cfg.n_layers / wl.l_keep,
           "algorithmic_tflop": flops / 1e12,
           "path_tflops": flops / (ms_step * 1e-3) / 1e12,
           "path_frac_of_measured_burst_peak": flops / (ms_step * 1e-3) / 1e12 / peaks["bf16_tflops"],
           "path_frac_of_nominal_2250": flops / (ms_step * 1e-3) / 1e12 / 2250.0,
           "device_status": status,
           "clocks": clocks,
           "e2e": {"value": n_tok / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                   "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms},
           "decode": {"ms_per_step": dec_ms, "tokens_per_s": wl.batch * world / (dec_ms * 1e-3),
                      "context": wl.seq_len, "steps": DECODE_STEPS, "device_status": dec_status,
                      "graph_loop_ms_per_step": gen_ms, "graph_loop_tokens_per_s": wl.batch * world / (gen_ms * 1e-3),
                      "graph_loop_weight_stream_gbs": weight_bytes / (gen_ms * 1e-3) / 1e9,
                      "weight_stream_gbs": weight_bytes / (dec_ms * 1e-3) / 1e9,
                      "frac_of_measured_hbm": weight_bytes / (dec_ms * 1e-3) / 1e9 / load_peaks()["hbm_gbs"]},
           "gpu_launches": int(launches * a.steps),
           "roofline": {"kernel": "gemm_pair_kernel / gemm_kernel (tcgen05 projection GEMM, all epilogues)", "bound": "tensor",
                        "achieved": achieved_tf, "peak": peak_tf, "unit": "TFLOP/s",
                        "frac": achieved_tf / peak_tf if peak_tf else None,
                        "peak_source": f"{peaks['source']} sustained cuBLAS bf16 (burst {peaks['bf16_tflops']})"
                                       + (", fp8 launches at 2 x that (nominal ratio), flop-weighted" if fp8 else ""),
                        "launches_per_step": gemm_n, "ms_per_step": gemm_ms, "traffic": None if fp8 else gemm_traffic(),
                        "traffic_launch": GEMM_TRAFFIC["launch"]},
           "kernel_breakdown": breakdown}
    if rank == 0 and world == 1 and not a.no_cpu_baseline:
        _, whole, parts = oracle_sample(wl, 2, 1)
        t = sum(whole) / len(whole)
        out["cpu_baseline"] = {"value": wl.seq_len * wl.batch / t, "unit": UNIT, "cores": torch.get_num_threads(),
                               "kind": "oracle", "sample": oracle_sample_text(wl, parts)}
    if rank == 0:
        print(json.dumps(out), flush=True)
    if world > 1:
        torch.distributed.destroy_process_group()


def run_kernel(a, wl):
    """One kernel alone at the workload's per-layer shape: W warm-up launches, K timed launches between
    CUDA events on the launching stream. Every launch reads operands larger than L2 or, where they are
    smaller, rotates through enough operand sets to exceed it."""
    import paper_2602_03295_b200 as pk
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    lib = pk.lib()
    cfg = wl.model
    M, d, F, hd = wl.batch * wl.seq_len, cfg.d_model, cfg.d_ffn, cfg.head_dim
    qd, kvd = cfg.n_q_heads * hd, cfg.n_kv_heads * hd
    P = max(1, cfg.n_layers - wl.l_keep)
    g = torch.Generator(device=dev).manual_seed(ps.DEFAULT_SEED)

    def rnd(*shape, std=0.5, dtype=torch.bfloat16):
        return (torch.randn(*shape, generator=g, device=dev, dtype=torch.float32) * std).to(dtype)

    peaks = load_peaks()
    k = a.kernel
    bound, work, sets = "tensor", 0.0, 1
    if (k.startswith("gemm_") and not k.endswith("_fp8")) or k == "kvproj":
        f_pad = (F + 127) // 128 * 128
        shapes = {"gemm_qkv": (1, qd + 2 * kvd, d, 1), "gemm_o": (1, d, qd, 2), "gemm_gateup": (1, 2 * f_pad, d, 3),
                  "gemm_down": (1, d, F, 2), "kvproj": (P, 2 * kvd, d, 1)}
        G, N, K, epi = shapes[k]
        A, B = rnd(G, M, K), rnd(G, N, K, std=0.02)
        if epi == 3:
            out = torch.zeros(G, M, F, dtype=torch.bfloat16, device=dev)
        else:
            out = torch.zeros(G, M, N, dtype=torch.float32, device=dev)
        work = 2.0 * G * M * N * K

        if k in ("gemm_qkv", "kvproj"):
            # as the path runs them: per-head norm, RoPE and the paged-cache write in the epilogue
            from paper_2602_03295_b200.binding import KVCache
            del out
            n_q = cfg.n_q_heads if k == "gemm_qkv" else 0
            cache = KVCache(cfg.replace(n_layers=G), wl.batch, wl.seq_len, a.page_size, device=dev)
            table = torch.zeros(wl.seq_len, hd // 2, 2, dtype=torch.float32, device=dev)
            lib.rope_table(table, wl.seq_len, hd, cfg.rope_theta)
            q_out = torch.zeros(M, qd, dtype=torch.bfloat16, device=dev) if n_q else None
            gq = torch.ones(G, hd, dtype=torch.float32, device=dev) if cfg.qk_norm else None

            def launch(i):
                lib.gemm_qkv_rope(A if G > 1 else A[0], B if G > 1 else B[0], q_out, cache.k, cache.v, 0,
                                  cache.block_table, a.page_size, gq if (gq is None or G > 1) else gq[0],
                                  gq if (gq is None or G > 1) else gq[0], table, n_q, cfg.n_kv_heads, hd,
                                  wl.seq_len, wl.seq_len, 0, cfg.rms_eps)
        else:
            def launch(i):
                lib.gemm(A if G > 1 else A[0], B if G > 1 else B[0], out if G > 1 else out[0], epilogue=epi,
                         act=cfg.act, n_valid=F if epi == 3 else 0)
    elif k in ("gemm_gateup_fp8", "gemm_qkvshape_fp8"):
        # the E4M3 GEMM at the gate/up shape (gated epilogue) and at the QKV shape (plain fp32 store)
        f_pad = (F + 127) // 128 * 128
        N, epi = (2 * f_pad, 3) if k == "gemm_gateup_fp8" else (qd + 2 * kvd, 1)
        K = d
        A8, sa = lib.rmsnorm_e4m3(rnd(M, K, dtype=torch.float32), torch.ones(K, dtype=torch.float32, device=dev),
                                  cfg.rms_eps)
        B8, sb = lib.quantize_e4m3(rnd(N, K, std=0.02))
        out = torch.zeros(M, F if epi == 3 else N, dtype=torch.bfloat16 if epi == 3 else torch.float32, device=dev)
        work = 2.0 * M * N * K
        peaks = dict(peaks, bf16_tflops=2.0 * peaks["bf16_tflops"], source=peaks["source"] + " bf16 x 2 (nominal fp8 : bf16 ratio)")

        def launch(i):
            lib.gemm_e4m3(A8, sa, B8, sb, out, epilogue=epi, act=cfg.act, n_valid=F if epi == 3 else 0)
    elif k == "rmsnorm_fp8":
        bound = "hbm"
        x = rnd(M, d, dtype=torch.float32)
        gain = torch.ones(d, dtype=torch.float32, device=dev)
        work = 5.0 * M * d
        codes = torch.empty(M, d, dtype=torch.uint8, device=dev)
        scales = torch.empty(M, dtype=torch.float32, device=dev)

        def launch(i):
            lib.rmsnorm_e4m3(x, gain, cfg.rms_eps, out=codes, scale=scales)
    elif k in ("attention", "attention_local"):
        from paper_2602_03295_b200.binding import KVCache
        window = cfg.window if k == "attention_local" else 0
        q = rnd(M, qd, std=1.0)
        cache = KVCache(cfg.replace(n_layers=1), wl.batch, wl.seq_len, a.page_size, device=dev)
        cache.k.copy_(rnd(*cache.k.shape, std=1.0))
        cache.v.copy_(rnd(*cache.v.shape, std=1.0))
        out = torch.zeros(M, qd, dtype=torch.bfloat16, device=dev)
        N = wl.seq_len
        pairs = N * (N + 1) / 2 if not window or window >= N else window * (window + 1) / 2 + (N - window) * window
        work = 4.0 * hd * pairs * cfg.n_q_heads * wl.batch

        def launch(i):
            lib.attention(q, cache.k[0], cache.v[0], cache.block_table, out, wl.batch, N, N, cfg.n_q_heads,
                          cfg.n_kv_heads, hd, a.page_size, window)
    elif k == "gemv_head":
        bound = "hbm"
        W = rnd(cfg.vocab, d, std=0.02)
        x = rnd(wl.batch, d, dtype=torch.float32)
        out = torch.zeros(wl.batch, cfg.vocab, dtype=torch.float32, device=dev)
        work = 2.0 * cfg.vocab * d

        def launch(i):
            lib.gemv(x, W, out, mode=0)
    elif k == "gemv_gateup":
        # the boundary / decode path's widest matrix for wl.batch activation rows (--batch N): the scalar GEMV for
        # one or two rows, the tensor-core GEMV from three on; four weight sets so that L2 never helps
        bound = "hbm"
        F = (cfg.d_ffn + 127) // 128 * 128
        Ws = [rnd(2 * F, d, std=0.02) for _ in range(4)]
        x = rnd(wl.batch, d, std=1.0)
        out = torch.zeros(wl.batch, cfg.d_ffn, dtype=torch.bfloat16, device=dev)
        work = 2.0 * 2 * F * d

        def launch(i):
            lib.gemv(x, Ws[i % 4], out, mode=3, act=cfg.act, n_valid=cfg.d_ffn)
    elif k == "decode_attention":
        from paper_2602_03295_b200.binding import KVCache
        bound = "hbm"
        N = wl.seq_len
        per_set = 4.0 * wl.batch * N * kvd
        sets = int(2 * 126e6 // per_set) + 2
        cache = KVCache(cfg.replace(n_layers=sets), wl.batch, N, a.page_size, device=dev)
        cache.k.copy_(rnd(*cache.k.shape, std=1.0))
        cache.v.copy_(rnd(*cache.v.shape, std=1.0))
        q = rnd(wl.batch, qd, std=1.0)
        out = torch.zeros(wl.batch, qd, dtype=torch.bfloat16, device=dev)
        work = per_set
        # as the decode step calls it: zeroed arrival counters, so the kernel merges its own key splits
        ctr = torch.zeros(wl.batch * cfg.n_kv_heads, dtype=torch.int32, device=dev)
        part = torch.empty(wl.batch * cfg.n_q_heads * 64 * (hd + 2), dtype=torch.float32, device=dev)

        def launch(i):
            lib.decode_attention(q, cache.k[i % sets], cache.v[i % sets], cache.block_table, out, cfg.n_q_heads,
                                 cfg.n_kv_heads, hd, N, a.page_size, 0, counters=ctr, partial=part)
    elif k == "decode_step":
        # one position per sequence through all layers over the cache of a full-depth prefill (the
        # single-row kernels: GEMV, norm, RoPE + cache write, split-KV attention, output head)
        from paper_2602_03295_b200.binding import KVCache, PopModel
        bound = "hbm"
        N = wl.seq_len
        model = PopModel(cfg, ps.SynthWeights(cfg, device=dev), device=dev)
        if a.precision == "fp8":
            model.enable_fp8()
        cache = KVCache(cfg, wl.batch, N + 64, a.page_size, device=dev)
        tokens, embeds = ps.make_prompt(wl)
        model.prefill(tokens.to(dev), None if embeds is None else embeds.to(dev), cfg.n_layers, cache)
        tok = torch.zeros(wl.batch, dtype=torch.int32, device=dev)
        logits = torch.zeros(wl.batch, cfg.vocab, dtype=torch.float32, device=dev)
        per_layer = d * (qd + 2 * kvd) + qd * d + 3 * d * F
        wbytes = 1.0 if a.precision == "fp8" else 2.0
        work = wbytes * cfg.n_layers * per_layer + 2.0 * cfg.vocab * d + 4.0 * wl.batch * N * kvd * cfg.n_layers

        def launch(i):
            model.decode_step(tok, N + i % 64, cache, logits)
    elif k == "rmsnorm":
        bound = "hbm"
        x = rnd(M, d, dtype=torch.float32)
        gain = torch.ones(d, dtype=torch.float32, device=dev)
        out = torch.zeros(M, d, dtype=torch.bfloat16, device=dev)
        work = 6.0 * M * d

        def launch(i):
            lib.rmsnorm(x, gain, out, cfg.rms_eps)
    else:   # rope_cache
        from paper_2602_03295_b200.binding import KVCache
        bound = "hbm"
        N = wl.seq_len
        x = rnd(M, qd + 2 * kvd, dtype=torch.float32)
        cache = KVCache(cfg.replace(n_layers=1), wl.batch, N, a.page_size, device=dev)
        table = torch.zeros(N, hd // 2, 2, dtype=torch.float32, device=dev)
        lib.rope_table(table, N, hd, cfg.rope_theta)
        q_out = torch.zeros(M, qd, dtype=torch.bfloat16, device=dev)
        work = 6.0 * M * (qd + 2 * kvd)

        def launch(i):
            lib.rope_cache(x, q_out, cache.k, cache.v, 0, cache.block_table, a.page_size, None, None, table,
                           cfg.n_q_heads, cfg.n_kv_heads, hd, N, N, 0, cfg.rms_eps)

    for i in range(max(a.warmup, 3)):
        launch(i)
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(a.steps):
        launch(i)
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1) / a.steps
    assert lib.status() == 0
    if bound == "tensor":
        achieved, peak, unit = work / (ms * 1e-3) / 1e12, peaks["bf16_tflops"], "TFLOP/s"
    else:
        achieved, peak, unit = work / (ms * 1e-3) / 1e9, peaks["hbm_gbs"], "GB/s"
    print(json.dumps({"kernel": k, "config": workload_config(wl, a), "steps": a.steps, "warmup": max(a.warmup, 3),
                      "ms_per_launch": ms, "operand_sets": sets,
                      "roofline": {"bound": bound, "achieved": achieved, "peak": peak, "unit": unit,
                                   "frac": achieved / peak, "peak_source": peaks["source"] + " burst"},
                      "clocks": clocks}), flush=True)


def run_sweep(a, wl0):
    """Prompt length {512, 2048, 8192, 32768} x batch {1, 4, 8} (at most 64K tokens in total) x
    L_keep/L in {1, 0.875, 0.75, 0.625} on one loaded model. Every point: 3 warm-up calls, then
    `--steps` calls between CUDA events. Weights (2 bytes per parameter, far larger than L2) stream
    on every call."""
    from oracle import pop_oracle as po   # FLOP model only
    from paper_2602_03295_b200.binding import KVCache, PopModel
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    cfg = wl0.model
    model = PopModel(cfg, ps.SynthWeights(cfg, device=dev), device=dev)
    peaks = load_peaks()
    L = cfg.n_layers
    for n in (512, 2048, 8192, 32768):
        for bsz in (1, 4, 8):
            if n * bsz > 65536:
                continue
            tokens = ps.uniform_tokens(ps.DEFAULT_SEED + 1, bsz, n, cfg.vocab).to(dev)
            cache = KVCache(cfg, bsz, n, a.page_size, device=dev)
            logits = torch.empty(bsz, cfg.vocab, dtype=torch.float32, device=dev)
            full_ms = None
            for ratio in (1.0, 0.875, 0.75, 0.625):
                lk = int(round(L * ratio))

                def step():
                    model.prefill(tokens, None, lk, cache, logits)
                for _ in range(3):
                    step()
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                # short shapes are repeated until about a second of work has been timed: a handful of 10 ms
                # calls is over before the clocks have settled under the power cap
                e0.record()
                step()
                e1.record()
                torch.cuda.synchronize()
                steps = int(min(200, max(a.steps, 1000.0 / max(e0.elapsed_time(e1), 1e-3))))
                e0.record()
                for _ in range(steps):
                    step()
                e1.record()
                torch.cuda.synchronize()
                ms = e0.elapsed_time(e1) / steps
                assert model.last_status() == 0
                if ratio == 1.0:
                    full_ms = ms
                flops = po.prefill_flops(cfg, bsz, n, lk)
                print(json.dumps({
                    "sweep": wl0.key, "seq_len": n, "batch": bsz, "l_keep": lk, "keep_ratio": ratio,
                    "ttft_ms": ms, "tokens_per_s": bsz * n / (ms * 1e-3),
                    "speedup_vs_full_depth": full_ms / ms,
                    "speedup_ceiling_flop_ratio": po.prefill_flops(cfg, bsz, n, None) / flops,
                    "speedup_ceiling_layer_ratio": L / lk, "timed_calls": steps,
                    "path_tflops": flops / (ms * 1e-3) / 1e12,
                    "frac_of_measured_burst_peak": flops / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"]}), flush=True)
            if n == 8192 and bsz == 1:
                # the same number of pruned layers chosen deep, shallow or interleaved (pop_prefill_skip)
                P = L // 4
                sets = {"deep": set(range(L - P + 1, L + 1)), "shallow": set(range(1, P + 1)),
                        "interleaved": set(range(4, L + 1, 4))}
                for name, sk in sets.items():
                    def step_skip():
                        model.prefill_skip(tokens, None, sk, cache, logits)
                    for _ in range(3):
                        step_skip()
                    torch.cuda.synchronize()
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    for _ in range(a.steps):
                        step_skip()
                    e1.record()
                    torch.cuda.synchronize()
                    ms = e0.elapsed_time(e1) / a.steps
                    assert model.last_status() == 0
                    print(json.dumps({"sweep": wl0.key, "seq_len": n, "batch": bsz, "skip_set": name,
                                      "pruned_layers": sorted(sk), "ttft_ms": ms, "tokens_per_s": bsz * n / (ms * 1e-3),
                                      "speedup_vs_full_depth": full_ms / ms}), flush=True)
            if n == 8192 and bsz == 8:
                # a ragged batch of eight prompts packed without padding against the same prompts padded to 8192
                lens = [8192, 6144, 4096, 3072, 2048, 1024, 512, 128]
                packed = torch.cat([tokens[i, :m] for i, m in enumerate(lens)]).contiguous()

                def step_ragged():
                    model.prefill_ragged(packed, None, lens, L * 3 // 4, cache, logits)
                for _ in range(3):
                    step_ragged()
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(a.steps):
                    step_ragged()
                e1.record()
                torch.cuda.synchronize()
                ms = e0.elapsed_time(e1) / a.steps
                assert model.last_status() == 0
                print(json.dumps({"sweep": wl0.key, "ragged_lens": lens, "l_keep": L * 3 // 4, "ttft_ms": ms,
                                  "real_tokens_per_s": sum(lens) / (ms * 1e-3),
                                  "padded_to_8192_ttft_ms_same_l_keep": "see the N 8192, B 8 row"}), flush=True)
            del cache, tokens, logits


def run_chunked(a, wl0):
    """Long prompts on the workload's model, batch 1, L_keep = 3L/4: the one-shot call where its
    workspace is reasonable, and pop_prefill_chunked at several chunk lengths up to 131072 positions.
    Weights stream on every call and every chunk (far larger than L2)."""
    from oracle import pop_oracle as po   # FLOP model only
    from paper_2602_03295_b200.binding import KVCache, PopModel
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    cfg = wl0.model
    model = PopModel(cfg, ps.SynthWeights(cfg, device=dev), device=dev)
    peaks = load_peaks()
    lk = cfg.n_layers * 3 // 4
    for n, chunk in ((32768, 0), (32768, 16384), (32768, 8192), (32768, 2048), (131072, 8192)):
        tokens = ps.uniform_tokens(ps.DEFAULT_SEED + 1, 1, n, cfg.vocab).to(dev)
        cache = KVCache(cfg, 1, n, a.page_size, device=dev)
        logits = torch.empty(1, cfg.vocab, dtype=torch.float32, device=dev)
        model.ws = None                                   # size the workspace for this point alone

        def step():
            if chunk:
                model.prefill_chunked(tokens, None, lk, chunk, cache, logits)
            else:
                model.prefill(tokens, None, lk, cache, logits)
        for _ in range(3 if n <= 32768 else 1):
            step()
        torch.cuda.synchronize()
        steps = a.steps if n <= 32768 else max(1, min(a.steps, 2))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            step()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
        assert model.last_status() == 0
        flops = po.prefill_flops(cfg, 1, n, lk)
        print(json.dumps({"chunked": wl0.key, "seq_len": n, "chunk_len": chunk or None, "l_keep": lk, "ttft_ms": ms,
                          "tokens_per_s": n / (ms * 1e-3), "path_tflops": flops / (ms * 1e-3) / 1e12,
                          "frac_of_measured_burst_peak": flops / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                          "workspace_mb": model.ws.numel() / 2 ** 20,
                          "kv_cache_mb": 2 * cache.k.numel() * 2 / 2 ** 20, "steps": steps}), flush=True)
        del cache, tokens, logits


def main():
    a = parse_args()
    wl = resolve_workload(a)
    if a.chunked:
        run_chunked(a, wl)
    elif a.sweep:
        run_sweep(a, wl)
    elif a.kernel:
        run_kernel(a, wl)
    elif a.impl == "reference":
        run_reference(a, wl)
    else:
        run_ours(a, wl)


if __name__ == "__main__":
    main()
