"""Kernel-by-kernel parity: each C-ABI kernel entry point against the oracle's statement of the
same step (fp64 on the CPU), on shapes spanning several tiles with ragged tails.

Tolerances: outputs stored as bf16 carry one rounding (2^-9 relative) on top of fp32 accumulation
of bf16 products, so a per-tensor max|err|/max|ref| of 1e-2 bounds them with margin; fp32 outputs
of fp32-accumulated bf16 products are held to 1e-4."""
import math

import pytest
import torch

import pop_synth as ps
from oracle import pop_oracle as po
from tests.gpu_util import paged_pools, rel_err

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(scope="module")
def L():
    import paper_2602_03295_b200 as pk
    return pk.lib()


@pytest.fixture(params=["single", "pair", "narrow"])
def gemm_form(request, monkeypatch):
    """Runs a GEMM test three times: with one CTA per 128 x 256 tile, with a CTA pair per 256 x 256 tile,
    and with one CTA per 128 x 128 tile (the plain-store and residual epilogues only; the other epilogues
    then run the 128 x 256 form). POP_GEMM_PAIR / POP_GEMM_NARROW force a form whatever the problem size."""
    monkeypatch.setenv("POP_GEMM_PAIR", "1" if request.param == "pair" else "0")
    monkeypatch.setenv("POP_GEMM_NARROW", "1" if request.param == "narrow" else "0")
    return request.param


def _bf(shape, seed, std=0.5):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(*shape, generator=g) * std).bfloat16()


@pytest.mark.parametrize("M,N,K,G", [(128, 256, 64, 1), (300, 264, 136, 1), (1000, 1024, 4096, 1),
                                     (200, 512, 128, 3), (1, 8, 8, 1), (129, 2056, 72, 2), (385, 520, 200, 1),
                                     (2100, 5000, 328, 1)])
@pytest.mark.parametrize("epi", [0, 1, 2])
def test_gemm_plain_epilogues(L, gemm_form, M, N, K, G, epi):
    A, B = _bf((G, M, K), 1), _bf((G, N, K), 2)
    ref = torch.matmul(A.double(), B.double().transpose(1, 2))
    if epi == 0:
        out = torch.zeros(G, M, N, dtype=torch.bfloat16, device=DEV)
    else:
        init = _bf((G, M, N), 3).float()
        out = init.clone().to(DEV)
        if epi == 2:
            ref = ref + init.double()
    L.gemm(A.to(DEV), B.to(DEV), out, epilogue=epi)
    assert L.status() == 0
    assert rel_err(out, ref) < (1e-2 if epi == 0 else 1e-4)


@pytest.mark.parametrize("M,F,K,act", [(384, 256, 320, 0), (130, 688, 256, 0), (257, 1000, 136, 1)])
def test_gemm_gated_epilogue(L, gemm_form, M, F, K, act):
    # gate/up rows interleaved in blocks of 128 with zero padding of the last block, as the
    # library's weight repacking lays them out
    Wg, Wu, A = _bf((F, K), 4), _bf((F, K), 5), _bf((M, K), 6)
    f_pad = (F + 127) // 128 * 128
    Wgu = torch.zeros(2 * f_pad, K, dtype=torch.bfloat16)
    for t in range(f_pad // 128):
        n = min(128, F - t * 128)
        Wgu[256 * t: 256 * t + n] = Wg[128 * t: 128 * t + n]
        Wgu[256 * t + 128: 256 * t + 128 + n] = Wu[128 * t: 128 * t + n]
    canary = 7.0
    out = torch.full((M, F + 8), canary, dtype=torch.bfloat16, device=DEV)
    L.gemm(A.to(DEV), Wgu.to(DEV), out[:, :F], epilogue=3, act=act, n_valid=F)
    assert L.status() == 0
    ref = po.gated_act(A.double() @ Wg.double().T, A.double() @ Wu.double().T, act)
    assert rel_err(out[:, :F], ref) < 1e-2
    assert (out[:, F:] == canary).all()          # nothing written past the valid columns


CASES = [  # B, N, n_q, n_kv, hd, page, window
    (1, 128, 2, 1, 128, 128, 0), (1, 300, 4, 2, 128, 64, 0), (2, 200, 4, 2, 64, 16, 0),
    (1, 300, 2, 2, 64, 128, 0), (1, 260, 2, 1, 256, 32, 0), (1, 500, 4, 1, 128, 128, 100),
    (1, 1, 4, 2, 64, 16, 0), (1, 2, 2, 1, 128, 16, 0), (1, 129, 8, 8, 128, 32, 0),
    (1, 700, 2, 2, 256, 128, 130), (1, 1000, 8, 2, 128, 256, 0), (3, 130, 4, 2, 128, 16, 128),
]


@pytest.mark.parametrize("B,N,n_q,n_kv,hd,page,window", CASES)
def test_attention_prefill(L, B, N, n_q, n_kv, hd, page, window):
    q, k, v = _bf((B * N, n_q * hd), 7, 1.0), _bf((B, N, n_kv, hd), 8, 1.0), _bf((B, N, n_kv, hd), 9, 1.0)
    kp, vp, bt = paged_pools(k, v, page)
    out = torch.zeros(B * N, n_q * hd, dtype=torch.bfloat16, device=DEV)
    L.attention(q.to(DEV), kp.to(DEV), vp.to(DEV), bt.to(DEV), out, B, N, N, n_q, n_kv, hd, page, window)
    assert L.status() == 0
    ref = torch.cat([po.attention(q[b * N:(b + 1) * N].double().reshape(N, n_q, hd), k[b].double(), v[b].double(),
                                  torch.arange(N), window).reshape(N, -1) for b in range(B)])
    assert not torch.isnan(out).any()            # non-finite garbage beyond the prompt never leaks
    assert rel_err(out, ref) < 1e-2


def test_attention_rejects_page_sizes_a_tile_would_straddle(L):
    from paper_2602_03295_b200 import PopError, POP_E_INVALID
    q = torch.zeros(16, 128, dtype=torch.bfloat16, device=DEV)
    pool = torch.zeros(1, 48, 1, 128, dtype=torch.bfloat16, device=DEV)
    bt = torch.zeros(1, 1, dtype=torch.int32, device=DEV)
    with pytest.raises(PopError) as e:
        L.attention(q, pool, pool, bt, q.clone(), 1, 16, 16, 1, 1, 128, 48, 0)
    assert e.value.code == POP_E_INVALID


def test_attention_query_offset_and_strided_q(L):
    # queries are the last 100 positions of a 356-entry cache, read out of a wider fused buffer
    B, T, S, n_q, n_kv, hd = 1, 100, 356, 4, 2, 128
    wide = _bf((T, n_q * hd + 512), 10, 1.0)
    k, v = _bf((B, S, n_kv, hd), 11, 1.0), _bf((B, S, n_kv, hd), 12, 1.0)
    kp, vp, bt = paged_pools(k, v, 32)
    wide_d = wide.to(DEV)
    out = torch.zeros(T, n_q * hd, dtype=torch.bfloat16, device=DEV)
    L.attention(wide_d[:, : n_q * hd], kp.to(DEV), vp.to(DEV), bt.to(DEV), out, B, T, S, n_q, n_kv, hd, 32, 0,
                q_pos0=S - T)
    assert L.status() == 0
    ref = po.attention(wide[:, : n_q * hd].double().reshape(T, n_q, hd), k[0].double(), v[0].double(),
                       torch.arange(S - T, S), 0).reshape(T, -1)
    assert rel_err(out, ref) < 1e-2


@pytest.mark.parametrize("rows,d,groups", [(5, 256, 1), (300, 4096, 1), (33, 3840, 3)])
def test_rmsnorm(L, rows, d, groups):
    x = _bf((rows, d), 13, 3.0).float() + 0.123
    gain = ps.gains(3, 9, groups * d, True).reshape(groups, d)
    out = torch.zeros(groups, rows, d, dtype=torch.bfloat16, device=DEV)
    L.rmsnorm(x.to(DEV), gain.to(DEV) if groups > 1 else gain[0].to(DEV), out if groups > 1 else out[0], 1e-5)
    ref = torch.stack([po.rmsnorm(x.double(), gain[g].double(), 1e-5) for g in range(groups)])
    assert rel_err(out, ref) < 1e-2
    out32 = torch.zeros(rows, d, dtype=torch.float32, device=DEV)
    L.rmsnorm(x.to(DEV), gain[0].to(DEV), out32, 1e-5)
    assert rel_err(out32, ref[0]) < 1e-5


@pytest.mark.parametrize("hd,n_q,n_kv,qk_norm", [(64, 4, 2, 0), (128, 4, 1, 1), (256, 2, 2, 1)])
def test_rope_and_cache_write(L, hd, n_q, n_kv, qk_norm):
    B, N, page, theta, eps, layers = 2, 45, 16, 500000.0, 1e-6, 3
    rows = B * N
    x = _bf((rows, (n_q + 2 * n_kv) * hd), 14, 1.0).float() * 1.7
    table = torch.zeros(N, hd // 2, 2, dtype=torch.float32, device=DEV)
    L.rope_table(table, N, hd, theta)
    ang = torch.arange(N, dtype=torch.float64)[:, None] * theta ** (-2.0 * torch.arange(hd // 2, dtype=torch.float64) / hd)
    assert (table[..., 0].cpu().double() - ang.cos()).abs().max() < 1e-7
    assert (table[..., 1].cpu().double() - ang.sin()).abs().max() < 1e-7
    qg = ps.gains(1, 1, hd, True) if qk_norm else None
    kg = ps.gains(1, 2, hd, True) if qk_norm else None
    pps = (N + page - 1) // page
    bt = torch.randperm(B * pps, generator=torch.Generator().manual_seed(1)).reshape(B, pps).int()
    canary = -77.0
    kpool = torch.full((layers, B * pps, page, n_kv, hd), canary, dtype=torch.bfloat16, device=DEV)
    vpool = torch.full_like(kpool, canary)
    q_out = torch.zeros(rows, n_q * hd, dtype=torch.bfloat16, device=DEV)
    written = N - 1                               # as for a pruned layer: the last position is skipped
    L.rope_cache(x.to(DEV), q_out, kpool, vpool, 1, bt.to(DEV), page, None if qg is None else qg.to(DEV),
                 None if kg is None else kg.to(DEV), table, n_q, n_kv, hd, N, written, 0, eps)
    xd = x.double().reshape(B, N, n_q + 2 * n_kv, hd)
    q, k, v = xd[:, :, :n_q], xd[:, :, n_q:n_q + n_kv], xd[:, :, n_q + n_kv:]
    if qk_norm:
        q, k = po.rmsnorm(q, qg.double(), eps), po.rmsnorm(k, kg.double(), eps)
    pos = torch.arange(N)
    for b in range(B):
        qr, kr = po.rope(q[b], pos, theta), po.rope(k[b], pos, theta)
        assert rel_err(q_out[b * N: b * N + written].reshape(written, n_q, hd), qr[:written]) < 1e-2
        pages = bt[b, pos // page].long()
        kg_, vg_ = kpool[1][pages.to(DEV), (pos % page).to(DEV)], vpool[1][pages.to(DEV), (pos % page).to(DEV)]
        assert rel_err(kg_[:written], kr[:written]) < 1e-2
        assert rel_err(vg_[:written], v[b, :written]) < 1e-2
        assert (kg_[written:] == canary).all() and (vg_[written:] == canary).all()
    assert (kpool[0] == canary).all() and (kpool[2] == canary).all()   # other layers untouched


@pytest.mark.parametrize("M,d,K,F", [(300, 520, 136, 688), (129, 256, 72, 264)])
def test_rmsnorm_folded_around_the_gemms(L, gemm_form, M, d, K, F):
    # residual GEMM that also emits the next operand and row sums of squares, then a gated and a
    # plain GEMM that consume them: together they must equal residual add -> RMSNorm -> GEMM
    eps = 1e-5
    A, Wo = _bf((M, K), 40), _bf((d, K), 41, 0.2)
    x0 = _bf((M, d), 42).float()
    gain = ps.gains(3, 11, d, True)
    n_t = (d + 255) // 256
    x = x0.clone().to(DEV)
    hn = torch.zeros(M, d, dtype=torch.bfloat16, device=DEV)
    ss = torch.full((M, n_t + 1), 1e9, dtype=torch.float32, device=DEV)
    L.gemm_norm(A.to(DEV), Wo.to(DEV), x, 2, hn_out=hn, gain_next=gain.to(DEV), ss_out=ss)
    assert L.status() == 0
    x_ref = x0.double() + A.double() @ Wo.double().T
    assert rel_err(x, x_ref) < 1e-4
    assert rel_err(ss[:, :n_t].sum(1), x_ref.pow(2).sum(1)) < 1e-4
    assert (ss[:, n_t] == 1e9).all()
    assert rel_err(hn, x_ref * gain.double()) < 1e-2
    h_ref = po.rmsnorm(x_ref, gain.double(), eps)
    # consumer 1: gated FFN projection
    Wg, Wu = _bf((F, d), 43, 0.1), _bf((F, d), 44, 0.1)
    f_pad = (F + 127) // 128 * 128
    Wgu = torch.zeros(2 * f_pad, d, dtype=torch.bfloat16)
    for t in range(f_pad // 128):
        n = min(128, F - t * 128)
        Wgu[256 * t: 256 * t + n] = Wg[128 * t: 128 * t + n]
        Wgu[256 * t + 128: 256 * t + 128 + n] = Wu[128 * t: 128 * t + n]
    act = torch.zeros(M, F, dtype=torch.bfloat16, device=DEV)
    L.gemm_norm(hn, Wgu.to(DEV), act, 3, act=0, n_valid=F, ss_in=ss[:, :n_t], norm_d=d, norm_eps=eps)
    assert rel_err(act, po.gated_act(h_ref @ Wg.double().T, h_ref @ Wu.double().T, 0)) < 1e-2
    # consumer 2: plain fp32 store
    out = torch.zeros(M, F, dtype=torch.float32, device=DEV)
    L.gemm_norm(hn, Wg.to(DEV), out, 1, ss_in=ss[:, :n_t], norm_d=d, norm_eps=eps)
    assert rel_err(out, h_ref @ Wg.double().T) < 1e-2
    assert L.status() == 0


@pytest.mark.parametrize("hd,n_q,n_kv,qk_norm,groups", [(64, 4, 2, 0, 1), (128, 4, 1, 1, 1), (256, 2, 2, 1, 1),
                                                        (128, 0, 2, 1, 3), (64, 3, 3, 0, 1)])
def test_fused_qkv_projection_rope_and_cache_write(L, gemm_form, hd, n_q, n_kv, qk_norm, groups):
    # the projection GEMM with norm, RoPE and the paged-cache write in its epilogue, against the
    # oracle's statement of Eq. 2-3 (fp64); several m tiles with a ragged tail, several n tiles
    B, N, K, page, theta, eps, layers = 2, 150, 136, 16, 500000.0, 1e-6, 5
    rows, heads = B * N, n_q + 2 * n_kv
    A = _bf((groups, rows, K), 30, 1.0)
    W = _bf((groups, heads * hd, K), 31, 0.1)
    table = torch.zeros(N, hd // 2, 2, dtype=torch.float32, device=DEV)
    L.rope_table(table, N, hd, theta)
    qg = ps.gains(1, 1, groups * hd, True).reshape(groups, hd) if qk_norm else None
    kg = ps.gains(1, 2, groups * hd, True).reshape(groups, hd) if qk_norm else None
    pps = (N + page - 1) // page
    bt = torch.randperm(B * pps, generator=torch.Generator().manual_seed(2)).reshape(B, pps).int()
    canary = -77.0
    kpool = torch.full((layers, B * pps, page, n_kv, hd), canary, dtype=torch.bfloat16, device=DEV)
    vpool = torch.full_like(kpool, canary)
    q_out = torch.zeros(rows, max(n_q, 1) * hd, dtype=torch.bfloat16, device=DEV)
    written = N - 1
    dev = lambda t: None if t is None else t.to(DEV)
    L.gemm_qkv_rope(A.to(DEV) if groups > 1 else A[0].to(DEV), W.to(DEV) if groups > 1 else W[0].to(DEV),
                    q_out if n_q else None, kpool, vpool, 1, bt.to(DEV), page,
                    dev(qg if groups > 1 or qg is None else qg[0]), dev(kg if groups > 1 or kg is None else kg[0]),
                    table, n_q, n_kv, hd, N, written, 0, eps)
    assert L.status() == 0
    pos = torch.arange(N)
    for g in range(groups):
        x = (A[g].double() @ W[g].double().T).reshape(B, N, heads, hd)
        q, k, v = x[:, :, :n_q], x[:, :, n_q:n_q + n_kv], x[:, :, n_q + n_kv:]
        if qk_norm:
            k = po.rmsnorm(k, kg[g].double(), eps)
            if n_q:
                q = po.rmsnorm(q, qg[g].double(), eps)
        for b in range(B):
            kr = po.rope(k[b], pos, theta)
            if n_q:
                qr = po.rope(q[b], pos, theta)
                assert rel_err(q_out[b * N: b * N + written].reshape(written, n_q, hd), qr[:written]) < 1e-2
            pages = bt[b, pos // page].long().to(DEV)
            slots = (pos % page).to(DEV)
            kg_, vg_ = kpool[1 + g][pages, slots], vpool[1 + g][pages, slots]
            assert rel_err(kg_[:written], kr[:written]) < 1e-2
            assert rel_err(vg_[:written], v[b, :written]) < 1e-2
            assert (kg_[written:] == canary).all() and (vg_[written:] == canary).all()
    assert (kpool[0] == canary).all() and (kpool[1 + groups:] == canary).all()


@pytest.fixture(params=["auto", "scalar"])
def gemv_form(request, monkeypatch):
    """GEMV tests run twice: with the library's choice (the tensor-core kernel from three activation rows
    on, bf16 activations, K a multiple of 32) and with the scalar kernel everywhere (POP_GEMV_MMA=0)."""
    monkeypatch.setenv("POP_GEMV_MMA", "0" if request.param == "scalar" else "1")
    return request.param


@pytest.mark.parametrize("B,N,K,xf32", [(1, 1024, 4096, False), (8, 520, 688, False), (3, 1000, 256, True),
                                        (11, 64, 64, False), (8, 4096, 4096, False), (5, 1000, 512, False),
                                        (3, 24, 96, False), (4, 4096, 14336, False), (8, 4096, 4096, True)])
def test_gemv_store_and_add(L, gemv_form, B, N, K, xf32):
    W = _bf((N, K), 15)
    x = _bf((B, K), 16)
    xin = x.float() if xf32 else x
    ref = x.double() @ W.double().T
    out = torch.zeros(B, N, dtype=torch.float32, device=DEV)
    L.gemv(xin.to(DEV), W.to(DEV), out, mode=0)
    assert rel_err(out, ref) < 1e-4
    L.gemv(xin.to(DEV), W.to(DEV), out, mode=2)
    assert rel_err(out, 2 * ref) < 1e-4


@pytest.mark.parametrize("B,F,K", [(4, 688, 256), (8, 14336, 4096), (3, 100, 64), (1, 688, 256)])
def test_gemv_gated(L, gemv_form, B, F, K):
    Wg, Wu, x = _bf((F, K), 17), _bf((F, K), 18), _bf((B, K), 19)
    f_pad = (F + 127) // 128 * 128
    Wgu = torch.zeros(2 * f_pad, K, dtype=torch.bfloat16)
    for t in range(f_pad // 128):
        n = min(128, F - t * 128)
        Wgu[256 * t: 256 * t + n] = Wg[128 * t: 128 * t + n]
        Wgu[256 * t + 128: 256 * t + 128 + n] = Wu[128 * t: 128 * t + n]
    for act in (0, 1):
        out = torch.zeros(B, F, dtype=torch.bfloat16, device=DEV)
        L.gemv(x.to(DEV), Wgu.to(DEV), out, mode=3, act=act, n_valid=F)
        ref = po.gated_act(x.double() @ Wg.double().T, x.double() @ Wu.double().T, act)
        assert rel_err(out, ref) < 1e-2


@pytest.mark.parametrize("B,S,n_q,n_kv,hd,page,window", [(1, 1, 4, 2, 64, 16, 0), (2, 300, 4, 2, 128, 16, 0),
                                                         (1, 5000, 8, 2, 128, 128, 0), (1, 700, 2, 1, 256, 64, 100),
                                                         (3, 77, 8, 1, 64, 32, 0)])
def test_decode_attention(L, B, S, n_q, n_kv, hd, page, window):
    q, k, v = _bf((B, n_q * hd), 20, 1.0), _bf((B, S, n_kv, hd), 21, 1.0), _bf((B, S, n_kv, hd), 22, 1.0)
    kp, vp, bt = paged_pools(k, v, page)
    out = torch.zeros(B, n_q * hd, dtype=torch.bfloat16, device=DEV)
    L.decode_attention(q.to(DEV), kp.to(DEV), vp.to(DEV), bt.to(DEV), out, n_q, n_kv, hd, S, page, window)
    ref = torch.stack([po.attention(q[b].double().reshape(1, n_q, hd), k[b].double(), v[b].double(),
                                    torch.tensor([S - 1]), window).reshape(-1) for b in range(B)])
    assert not torch.isnan(out).any()
    assert rel_err(out, ref) < 1e-2
    # with arrival counters the attention kernel merges its own splits: same bits, counters left at zero,
    # so the same array serves the next call
    ctr = torch.zeros(B * n_kv, dtype=torch.int32, device=DEV)
    for _ in range(2):
        out2 = torch.full_like(out, float("nan"))
        L.decode_attention(q.to(DEV), kp.to(DEV), vp.to(DEV), bt.to(DEV), out2, n_q, n_kv, hd, S, page, window,
                           counters=ctr)
        assert torch.equal(out2, out)
        assert (ctr == 0).all()


@pytest.mark.parametrize("B,S,n_q,n_kv,hd,page,window,norm", [(1, 1, 4, 2, 64, 16, 0, False), (2, 37, 8, 2, 128, 16, 0, True),
                                                              (1, 1000, 32, 8, 128, 128, 0, False),
                                                              (3, 300, 4, 1, 256, 64, 96, True),
                                                              (1, 2049, 8, 8, 64, 128, 0, True)])
def test_decode_attention_with_the_projection_finish(L, B, S, n_q, n_kv, hd, page, window, norm):
    # the form the boundary / decode path runs (Eq. 2-3 for the new position, then Attn of Eq. 1): fp32 QKV row in,
    # per-head norm + RoPE + cache append inside the attention kernel
    theta, eps = 10000.0, 1e-6
    g = torch.Generator().manual_seed(30)
    qkv = torch.randn(B, (n_q + 2 * n_kv) * hd, generator=g)
    k_old, v_old = _bf((B, S, n_kv, hd), 31, 1.0), _bf((B, S, n_kv, hd), 32, 1.0)
    kp, vp, bt = paged_pools(k_old, v_old, page)
    # the slot of position S - 1 holds garbage until the kernel appends
    for b in range(B):
        kp[bt[b, (S - 1) // page].long(), (S - 1) % page] = float("nan")
        vp[bt[b, (S - 1) // page].long(), (S - 1) % page] = float("nan")
    qg = (1.0 + 0.1 * torch.randn(hd, generator=g)) if norm else None
    kg = (1.0 + 0.1 * torch.randn(hd, generator=g)) if norm else None
    table = torch.zeros(S, hd // 2, 2, dtype=torch.float32, device=DEV)
    L.rope_table(table, S, hd, theta)
    kp, vp = kp.to(DEV), vp.to(DEV)
    out = torch.full((B, n_q * hd), float("nan"), dtype=torch.bfloat16, device=DEV)
    ctr = torch.zeros(B * n_kv, dtype=torch.int32, device=DEV)
    L.decode_attention_qkv(qkv.to(DEV), None if qg is None else qg.to(DEV), None if kg is None else kg.to(DEV), eps,
                           table[S - 1], kp, vp, bt.to(DEV), out, n_q, n_kv, hd, S, page, ctr, window)
    assert L.status() == 0 and (ctr == 0).all()
    x = qkv.double().reshape(B, 1, n_q + 2 * n_kv, hd)
    q, kn, vn = x[:, :, :n_q], x[:, :, n_q:n_q + n_kv], x[:, :, n_q + n_kv:]
    if norm:
        q, kn = po.rmsnorm(q, qg.double(), eps), po.rmsnorm(kn, kg.double(), eps)
    pos = torch.tensor([S - 1])
    q, kn = po.rope(q, pos, theta), po.rope(kn, pos, theta)
    for b in range(B):
        K = torch.cat([k_old[b, : S - 1].double(), kn[b]]), torch.cat([v_old[b, : S - 1].double(), vn[b]])
        ref = po.attention(q[b], K[0], K[1], pos, window).reshape(-1)
        assert rel_err(out[b], ref) < 1e-2, b
        page_id, slot = bt[b, (S - 1) // page].long(), (S - 1) % page
        assert rel_err(kp[page_id, slot], kn[b, 0]) < 1e-2 and rel_err(vp[page_id, slot], vn[b, 0]) < 1e-2
    assert not torch.isnan(out.float()).any()


@pytest.mark.parametrize("B,S", [(1, 100), (8, 700), (2, 250)])
def test_decode_attention_cluster_merge_matches_the_merge_through_memory(L, B, S, monkeypatch):
    # few splits per (sequence, kv head): the splits form a thread-block cluster and merge through
    # distributed shared memory; POP_DEC_CLUSTER=0 keeps partials + counters in global memory
    n_q, n_kv, hd, page = 32, 8, 128, 64
    q, k, v = _bf((B, n_q * hd), 40, 1.0), _bf((B, S, n_kv, hd), 41, 1.0), _bf((B, S, n_kv, hd), 42, 1.0)
    kp, vp, bt = paged_pools(k, v, page)
    outs = []
    for mode in ("1", "0"):
        monkeypatch.setenv("POP_DEC_CLUSTER", mode)
        out = torch.full((B, n_q * hd), float("nan"), dtype=torch.bfloat16, device=DEV)
        ctr = torch.zeros(B * n_kv, dtype=torch.int32, device=DEV)
        L.decode_attention(q.to(DEV), kp.to(DEV), vp.to(DEV), bt.to(DEV), out, n_q, n_kv, hd, S, page, 0, counters=ctr)
        assert (ctr == 0).all()
        outs.append(out)
    ref = torch.stack([po.attention(q[b].double().reshape(1, n_q, hd), k[b].double(), v[b].double(),
                                    torch.tensor([S - 1]), 0).reshape(-1) for b in range(B)])
    assert rel_err(outs[0], ref) < 1e-2 and rel_err(outs[1], ref) < 1e-2
    assert rel_err(outs[0], outs[1].cpu().double()) < 1e-2


def test_generators_agree_between_cpu_and_gpu():
    tid = ps.tensor_id("wq", 2)
    a = ps.normal_bf16(3, tid, (300, 1000), 0.02)
    b = ps.normal_bf16(3, tid, (300, 1000), 0.02, device=DEV)
    assert torch.equal(a, b.cpu())
    assert torch.equal(ps.gains(3, 7, 4096, True), ps.gains(3, 7, 4096, True, DEV).cpu())
