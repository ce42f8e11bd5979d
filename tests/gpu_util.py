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
