"""FP8 (E4M3) operand path against the oracle: quantisation kernels code by code, the tensor-core GEMM on
codes, and the model-level kept-stack use."""
import pytest
import torch

import pop_synth as ps
from oracle import pop_oracle as po
from tests.gpu_util import rel_err

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(scope="module")
def L():
    import paper_2602_03295_b200 as pk
    return pk.lib()


def _codes_to_values(codes):
    return codes.cpu().view(torch.float8_e4m3fn).to(torch.float64)


@pytest.mark.parametrize("rows,d", [(5, 64), (130, 4096), (3, 5120), (7, 688)])
def test_rmsnorm_e4m3_codes(L, rows, d):
    g = torch.Generator().manual_seed(5)
    x = torch.randn(rows, d, generator=g) * torch.logspace(-2, 2, rows)[:, None]
    x[0, 3] = 40.0 * x[0].abs().max()                       # an outlier channel sets its row's scale
    gain = 1.0 + 0.1 * torch.randn(d, generator=g)
    codes, scale = L.rmsnorm_e4m3(x.to(DEV), gain.to(DEV), 1e-5)
    assert L.status() == 0
    ref_q, ref_s = po.quant_rows_e4m3(po.rmsnorm(x.double(), gain.double(), 1e-5))
    got = _codes_to_values(codes)
    assert torch.allclose(scale.cpu().double(), ref_s[:, 0], rtol=1e-5)
    # both sides decide in fp32; the row sums differ in their last bits, so a value sitting on a rounding
    # boundary may fall to the neighbouring code: allow very few, and only neighbours
    diff = got != ref_q
    assert diff.double().mean().item() < 2e-3
    step = torch.maximum(ref_q.abs(), torch.tensor(2.0 ** -6, dtype=torch.float64)) * 2.0 ** -3
    assert ((got - ref_q).abs() <= step * 1.001).all()
    assert got.abs().max(dim=1).values.eq(448.0).all()


def test_weight_quantisation_codes(L):
    w = (torch.randn(300, 1000, generator=torch.Generator().manual_seed(6)) * 0.02).to(torch.bfloat16)
    codes, scale = L.quantize_e4m3(w.to(DEV))
    assert L.status() == 0
    (ref_q,), ref_s = po.quant_tensors_e4m3([w])
    assert abs(scale.item() - ref_s) <= 1e-6 * ref_s
    assert torch.equal(_codes_to_values(codes), ref_q)       # bf16 inputs, one fp32 product: identical decisions


@pytest.mark.parametrize("M,N,K", [(128, 256, 128), (300, 520, 1024), (1, 8, 16), (1000, 256, 4096)])
def test_gemm_on_codes(L, M, N, K):
    g = torch.Generator().manual_seed(7)
    a = torch.randn(M, K, generator=g)
    w = (torch.randn(N, K, generator=g) * 0.02).to(torch.bfloat16)
    aq, a_s = po.quant_rows_e4m3(a)
    (wq,), w_s = po.quant_tensors_e4m3([w])
    ref = (aq @ wq.T) * a_s * w_s                            # fp64 on the codes
    A8 = aq.to(torch.float32).to(torch.float8_e4m3fn).view(torch.uint8).to(DEV)   # exact: they are E4M3 values
    B8 = wq.to(torch.float32).to(torch.float8_e4m3fn).view(torch.uint8).to(DEV)
    sa = a_s[:, 0].float().to(DEV)
    sb = torch.tensor([w_s], dtype=torch.float32, device=DEV)
    out = torch.zeros(M, N, dtype=torch.float32, device=DEV)
    L.gemm_e4m3(A8, sa, B8, sb, out, epilogue=1)
    assert L.status() == 0
    assert rel_err(out, ref) < 1e-5                          # exact products, fp32 accumulation
    outb = torch.zeros(M, N, dtype=torch.bfloat16, device=DEV)
    L.gemm_e4m3(A8, sa, B8, sb, outb, epilogue=0)
    assert rel_err(outb, ref) < 1e-2
