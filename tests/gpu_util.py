"""Helpers shared by the GPU parity tests (no arithmetic of the method lives here)."""
import torch


def rel_err(got: torch.Tensor, ref: torch.Tensor) -> float:
    """max |got - ref| / max |ref| : the per-tensor relative error the tolerances are stated in."""
    ref = ref.double().cpu()
    return ((got.double().cpu() - ref).abs().max() / ref.abs().max().clamp_min(1e-30)).item()


def paged_pools(k, v, page_size, extra_pages=3, seed=0, garbage=float("nan")):
    """Scatter dense [B, N, n_kv, hd] bf16 K/V into shuffled pages; unused slots hold `garbage`."""
    B, N, n_kv, hd = k.shape
    pps = (N + page_size - 1) // page_size
    npages = B * pps + extra_pages
    g = torch.Generator().manual_seed(seed)
    bt = torch.randperm(npages, generator=g)[: B * pps].reshape(B, pps).int()
    kp = torch.full((npages, page_size, n_kv, hd), garbage, dtype=torch.bfloat16)
    vp = torch.full((npages, page_size, n_kv, hd), garbage, dtype=torch.bfloat16)
    pos = torch.arange(N)
    for b in range(B):
        pages = bt[b, pos // page_size].long()
        kp[pages, pos % page_size] = k[b]
        vp[pages, pos % page_size] = v[b]
    return kp, vp, bt


def interleave_gate_up(w_gate, w_up):
    """The fused gate/up operand layout of the gated GEMM / GEMV: blocks of 128 gate rows followed by the
    matching 128 up rows, the last block zero-padded to 128. [F, K] x 2 -> [2 * ceil(F/128)*128, K]."""
    F, K = w_gate.shape
    f_pad = (F + 127) // 128 * 128
    out = torch.zeros(2 * f_pad, K, dtype=w_gate.dtype, device=w_gate.device)
    for t in range(f_pad // 128):
        n = min(128, F - t * 128)
        out[256 * t: 256 * t + n] = w_gate[128 * t: 128 * t + n]
        out[256 * t + 128: 256 * t + 128 + n] = w_up[128 * t: 128 * t + n]
    return out
