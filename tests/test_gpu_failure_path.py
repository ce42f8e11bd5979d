"""The library's failure path on the GPU, exercised without a fault, a trap or an endless loop.

Two ways the device status word gets raised are driven here:
  * a bounded wait that runs out (pop_k_wait_selftest: the same wait the GEMM and attention kernels
    use, on a barrier nothing arrives at, limited to well under a millisecond);
  * a token id that cannot be looked up (negative with no embedding rows, or >= vocab), which only
    the device can see.
In both cases the word must read back once with the right code, kernels launched while it is raised
must return without writing, and the library must work normally after the word was read.
"""
import pytest
import torch

import pop_synth as ps
from oracle import pop_oracle as po
from tests.gpu_util import rel_err

pytestmark = pytest.mark.gpu
DEV = "cuda"


def test_a_wait_that_runs_out_raises_the_status_word_and_later_launches_return_at_once():
    import paper_2602_03295_b200 as pk
    L = pk.lib()
    assert L.status() == 0
    g = torch.Generator().manual_seed(1)
    A = torch.randn(300, 128, generator=g).bfloat16().to(DEV)
    B = torch.randn(264, 128, generator=g).bfloat16().to(DEV)
    ref = A.cpu().double() @ B.cpu().double().T
    out = torch.full((300, 264), 7.0, dtype=torch.float32, device=DEV)
    L.wait_selftest(200000)
    # queued behind the raised word: the GEMM and the attention kernel must not touch their outputs
    L.gemm(A, B, out, epilogue=1)
    q = torch.randn(128, 128, generator=g).bfloat16().to(DEV)
    pool = torch.randn(1, 128, 1, 128, generator=g).bfloat16().to(DEV)
    bt = torch.zeros(1, 1, dtype=torch.int32, device=DEV)
    ao = torch.full((128, 128), 5.0, dtype=torch.bfloat16, device=DEV)
    L.attention(q, pool, pool, bt, ao, 1, 128, 128, 1, 1, 128, 128, 0)
    torch.cuda.synchronize()
    assert (out == 7.0).all() and (ao == 5.0).all()
    assert L.status() == pk.POP_E_DEVICE_TIMEOUT
    assert L.status() == 0                       # read once, then clear
    L.gemm(A, B, out, epilogue=1)
    assert L.status() == 0
    assert rel_err(out, ref) < 1e-4
    with pytest.raises(pk.PopError) as e:        # the limit itself is bounded
        L.wait_selftest(10 ** 9)
    assert e.value.code == pk.POP_E_INVALID


@pytest.mark.parametrize("bad", [-1, 1024, 2 ** 30])
def test_an_unusable_token_id_is_reported_not_dereferenced(bad):
    from paper_2602_03295_b200 import POP_E_INVALID
    from paper_2602_03295_b200.binding import KVCache, PopModel
    cfg = ps.C1_TINY
    model = PopModel(cfg, ps.SynthWeights(cfg, device=DEV))
    tokens = ps.uniform_tokens(5, 1, 40, cfg.vocab)
    good = tokens.clone()
    tokens[0, 17] = bad
    cache = KVCache(cfg, 1, 40, 16, fill=float("nan"))
    model.prefill(tokens.to(DEV), None, 3, cache)           # no embedding rows supplied
    assert model.last_status() == POP_E_INVALID
    assert model.last_status() == 0
    # the same model and workspace then serve a valid prompt
    cache = KVCache(cfg, 1, 40, 16, fill=float("nan"))
    logits = model.prefill(good.to(DEV), None, 3, cache)
    assert model.last_status() == 0
    ref = po.pop_prefill(cfg, ps.SynthWeights(cfg), good, None, 3)
    assert (logits.cpu().double() - ref["logits"]).abs().max().item() <= 5e-2
    # a decode step never has embedding rows: a negative id there is caught the same way
    model.decode_step(torch.tensor([bad], dtype=torch.int32, device=DEV), 40, KVCache(cfg, 1, 41, 16))
    assert model.last_status() == POP_E_INVALID
    assert model.last_status() == 0


def test_a_block_table_entry_outside_the_pool_is_reported_not_dereferenced():
    # the block table lives on the device: the kernels that turn its entries into addresses check them
    from paper_2602_03295_b200 import POP_E_INVALID
    from paper_2602_03295_b200.binding import KVCache, PopModel
    cfg = ps.C1_TINY
    model = PopModel(cfg, ps.SynthWeights(cfg, device=DEV))
    tokens = ps.uniform_tokens(6, 1, 40, cfg.vocab).to(DEV)
    for bad in (-1, 3, 10 ** 6):
        bt = torch.tensor([[0, bad, 2]], dtype=torch.int32)
        cache = KVCache(cfg, 1, 40, 16, block_table=bt, num_pages=3, fill=5.0)
        model.prefill(tokens, None, 3, cache)
        assert model.last_status() == POP_E_INVALID, bad
        assert model.last_status() == 0
        assert (cache.k[:, [0, 2]] == 5.0).sum() < cache.k[:, [0, 2]].numel()     # valid pages were written
    cache = KVCache(cfg, 1, 40, 16, fill=float("nan"))
    logits = model.prefill(tokens, None, 3, cache)
    assert model.last_status() == 0 and torch.isfinite(logits).all()
