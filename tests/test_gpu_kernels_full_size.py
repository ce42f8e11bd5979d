"""The two tensor-core kernels at the sizes they run at inside the benchmark configurations, checked on
sampled output rows the oracle computes one by one.

Attention (Attn of paper Eq. 1): the per-layer shapes of config 2 (8192 positions, 32/8 heads of 128),
config 4 (16384 positions, 16/8 heads of 256; a global layer and a local layer with window 1024) and
config 5's longest prompt (32768 positions): 64 sampled query rows incl. the first and last rows, both
sides of a 128-row tile edge and the rows where the window starts to cut, every head, against
po.attention in fp64. 64 to 256 query tiles per head: several waves of CTAs, every K/V ring wrap.

Projection GEMM (paper Eq. 1-2, Eq. 14): the four shapes of a config-2 layer at M = 8192 rows and the
batched pruned-layer K/V projection (8 layers at once) with its RoPE / cache-write epilogue: 1024 to
7168 output tiles, i.e. up to 48 per persistent CTA, so the TMEM double buffer, its phase flips and
the shared-memory ring carried across tiles are all exercised. 256 sampled rows x all columns against
fp64 products.

Tolerances as in the small-shape kernel tests: 1e-2 (per tensor, max|err| / max|ref|) for bf16
outputs, 1e-4 for fp32 outputs of fp32-accumulated bf16 products.
"""
import pytest
import torch

from oracle import pop_oracle as po
from tests.gpu_util import interleave_gate_up, rel_err

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(scope="module")
def L():
    import paper_2602_03295_b200 as pk
    return pk.lib()


@pytest.fixture(params=["single", "pair", "narrow"])
def gemm_form(request, monkeypatch):
    monkeypatch.setenv("POP_GEMM_PAIR", "1" if request.param == "pair" else "0")
    monkeypatch.setenv("POP_GEMM_NARROW", "1" if request.param == "narrow" else "0")
    return request.param


def _randn_bf16(shape, seed, std=1.0):
    g = torch.Generator(device=DEV).manual_seed(seed)
    return (torch.randn(*shape, generator=g, device=DEV) * std).bfloat16()


def _rows(n, count, seed, extra=()):
    g = torch.Generator().manual_seed(seed)
    fixed = [0, 1, 127, 128, 129, n // 2 - 1, n // 2, n - 129, n - 128, n - 2, n - 1] + list(extra)
    rnd = torch.randint(0, n, (max(0, count - len(fixed)),), generator=g).tolist()
    return torch.tensor(sorted({r for r in fixed + rnd if 0 <= r < n}))


@pytest.mark.parametrize("N,n_q,n_kv,hd,window", [(8192, 32, 8, 128, 0), (16384, 16, 8, 256, 0),
                                                  (16384, 16, 8, 256, 1024), (32768, 32, 8, 128, 0),
                                                  (8192, 32, 8, 128, 1024)])
def test_attention_at_the_benchmark_shapes(L, N, n_q, n_kv, hd, window):
    page = 128
    q = _randn_bf16((N, n_q * hd), 101, 1.5)
    k = _randn_bf16((N, n_kv, hd), 102)
    v = _randn_bf16((N, n_kv, hd), 103)
    # pages in shuffled order, unused slots and a few spare pages full of NaN
    pps = N // page
    perm = torch.randperm(pps + 3, generator=torch.Generator().manual_seed(5))[:pps]
    kp = torch.full((pps + 3, page, n_kv, hd), float("nan"), dtype=torch.bfloat16, device=DEV)
    vp = torch.full_like(kp, float("nan"))
    kp[perm.to(DEV)] = k.reshape(pps, page, n_kv, hd)
    vp[perm.to(DEV)] = v.reshape(pps, page, n_kv, hd)
    bt = perm.reshape(1, pps).int().to(DEV)
    out = torch.full((N, n_q * hd), float("nan"), dtype=torch.bfloat16, device=DEV)
    L.attention(q, kp, vp, bt, out, 1, N, N, n_q, n_kv, hd, page, window)
    assert L.status() == 0
    assert torch.isfinite(out.float()).all()
    edge = (window - 2, window - 1, window, window + 1, window + 127, window + 128) if window else ()
    rows = _rows(N, 64, 7, edge)
    ref = po.attention(q[rows.to(DEV)].cpu().double().reshape(len(rows), n_q, hd), k.cpu().double(), v.cpu().double(),
                       rows, window).reshape(len(rows), -1)
    got = out[rows.to(DEV)]
    assert rel_err(got, ref) < 1e-2
    # row by row as well: a single bad row must not hide behind the tensor's largest value
    per_row = (got.cpu().double() - ref).abs().amax(dim=1) / ref.abs().amax(dim=1)
    assert per_row.max().item() < 2e-2, (rows[per_row.argmax()].item(), per_row.max().item())


M_FULL = 8192


@pytest.mark.parametrize("name,N,K,epi", [("qkv-shape", 6144, 4096, 0), ("o-proj", 4096, 4096, 2),
                                          ("down", 4096, 14336, 2), ("store-f32", 4096, 4096, 1)])
def test_gemm_at_the_config2_shapes(L, gemm_form, name, N, K, epi):
    A = _randn_bf16((M_FULL, K), 201, 0.5)
    B = _randn_bf16((N, K), 202, 0.05)
    rows = _rows(M_FULL, 256, 11)
    ref = A[rows.to(DEV)].cpu().double() @ B.cpu().double().T
    if epi == 0:
        out = torch.full((M_FULL, N), float("nan"), dtype=torch.bfloat16, device=DEV)
    else:
        init = _randn_bf16((M_FULL, N), 203).float()
        out = init.clone()
        if epi == 2:
            ref = ref + init[rows.to(DEV)].cpu().double()
    L.gemm(A, B, out, epilogue=epi)
    assert L.status() == 0
    assert torch.isfinite(out.float()).all()
    assert rel_err(out[rows.to(DEV)], ref) < (1e-2 if epi == 0 else 1e-4)


def test_gated_gemm_at_the_config2_shape(L, gemm_form):
    F, K = 14336, 4096
    A = _randn_bf16((M_FULL, K), 211, 0.5)
    Wg, Wu = _randn_bf16((F, K), 212, 0.03), _randn_bf16((F, K), 213, 0.03)
    Wgu = interleave_gate_up(Wg, Wu)
    out = torch.full((M_FULL, F), float("nan"), dtype=torch.bfloat16, device=DEV)
    L.gemm(A, Wgu, out, epilogue=3, act=0, n_valid=F)
    assert L.status() == 0
    assert torch.isfinite(out.float()).all()
    rows = _rows(M_FULL, 256, 13)
    a = A[rows.to(DEV)].cpu().double()
    ref = po.gated_act(a @ Wg.cpu().double().T, a @ Wu.cpu().double().T, 0)
    assert rel_err(out[rows.to(DEV)], ref) < 1e-2


def test_batched_pruned_layer_projection_at_the_config2_shape(L, gemm_form):
    # Eq. 14 for 8 pruned layers in one launch: A holds 8 normalised copies of the state (one per
    # layer's gain), W the layers' [W^K; W^V]; the epilogue applies RoPE to k and writes both into the
    # layers' pages; the last position of the sequence is skipped (it belongs to the boundary token)
    G, N, K, n_kv, hd, page, theta = 8, M_FULL, 4096, 8, 128, 128, 500000.0
    A = _randn_bf16((G, N, K), 221, 1.0)
    W = _randn_bf16((G, 2 * n_kv * hd, K), 222, 0.02)
    table = torch.zeros(N, hd // 2, 2, dtype=torch.float32, device=DEV)
    L.rope_table(table, N, hd, theta)
    pps = N // page
    perm = torch.randperm(pps, generator=torch.Generator().manual_seed(3))
    bt = perm.reshape(1, pps).int().to(DEV)
    layers = G + 2
    kpool = torch.full((layers, pps, page, n_kv, hd), float("nan"), dtype=torch.bfloat16, device=DEV)
    vpool = torch.full_like(kpool, float("nan"))
    L.gemm_qkv_rope(A, W, None, kpool, vpool, 1, bt, page, None, None, table, 0, n_kv, hd, N, N - 1, 0, 1e-5)
    assert L.status() == 0
    rows = _rows(N - 1, 128, 17)
    pages, slots = perm[rows // page].to(DEV), (rows % page).to(DEV)
    for g in range(G):
        x = (A[g][rows.to(DEV)].cpu().double() @ W[g].cpu().double().T).reshape(len(rows), 2 * n_kv, hd)
        k_ref = po.rope(x[:, :n_kv], rows, theta)
        assert rel_err(kpool[1 + g][pages, slots], k_ref) < 1e-2, g
        assert rel_err(vpool[1 + g][pages, slots], x[:, n_kv:]) < 1e-2, g
        # every position but the last was written, the last one and the neighbouring layers were not
        flat_k = kpool[1 + g][perm.to(DEV)].reshape(N, n_kv, hd)
        assert torch.isfinite(flat_k[: N - 1].float()).all() and torch.isnan(flat_k[N - 1].float()).all()
    assert torch.isnan(kpool[0].float()).all() and torch.isnan(kpool[G + 1].float()).all()
