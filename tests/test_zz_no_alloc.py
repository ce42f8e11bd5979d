"""The allocation-free decode-attention entry point against the ordinary one.

pop_k_decode_attention_static serves callers that cannot allocate device memory when they call
(a serving loop or host callback where cudaMalloc is off limits, or a process that was only handed
input and output buffers): its split-KV partials live in a fixed array inside the library instead of
a caller-supplied scratch buffer. This file is collected last on purpose, so a failure here cannot
hide the result of any other test in a run that stops at the first failure; it must also pass when
run alone in a fresh process (the first call on a device performs the one-time address lookup).
"""
import pytest
import torch

from oracle import pop_oracle as po
from tests.gpu_util import paged_pools, rel_err

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _bf(shape, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(*shape, generator=g).bfloat16()


def _both(L, B, S, n_q, n_kv, hd, page, window, seed):
    """Runs the ordinary and the allocation-free entry point on the same inputs."""
    q, k, v = _bf((B, n_q * hd), seed), _bf((B, S, n_kv, hd), seed + 1), _bf((B, S, n_kv, hd), seed + 2)
    kp, vp, bt = paged_pools(k, v, page)
    q, kp, vp, bt = q.to(DEV), kp.to(DEV), vp.to(DEV), bt.to(DEV)
    want = torch.zeros(B, n_q * hd, dtype=torch.bfloat16, device=DEV)
    got = torch.full_like(want, float("nan"))
    L.decode_attention(q, kp, vp, bt, want, n_q, n_kv, hd, S, page, window)
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    L.decode_attention_static(q, kp, vp, bt, got, n_q, n_kv, hd, S, page, window)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before      # torch's allocator was not touched either
    assert L.status() == 0
    # and the arithmetic itself, not only the sibling: the oracle's attention of the same inputs (fp64)
    ref = torch.stack([po.attention(q[b].cpu().double().reshape(1, n_q, hd), k[b].double(), v[b].double(),
                                    torch.tensor([S - 1]), window).reshape(-1) for b in range(B)])
    assert rel_err(got, ref) < 1e-2
    return got, want


def test_static_scratch_variant_matches_the_ordinary_entry_point_on_two_calls_in_a_row():
    import paper_2602_03295_b200 as pk
    L = pk.lib()
    # first call: long cache, many splits fill a large part of the shared array
    got, want = _both(L, 2, 5000, 8, 2, 128, 128, 0, seed=31)
    assert not torch.isnan(got).any()
    assert rel_err(got, want) < 1e-2                     # the tolerance of the kernel parity tests
    assert torch.equal(got, want)                        # same kernels, same order: in fact identical
    # second call right behind it: other shape, fewer splits, a window; the array still holds the
    # first call's partials, none of which may reach this result
    got, want = _both(L, 3, 700, 4, 1, 256, 64, 100, seed=41)
    assert not torch.isnan(got).any()
    assert rel_err(got, want) < 1e-2
    assert torch.equal(got, want)


def test_static_scratch_variant_refuses_what_does_not_fit():
    import paper_2602_03295_b200 as pk
    from paper_2602_03295_b200 import PopError, POP_E_NOSPACE, POP_E_INVALID
    L = pk.lib()
    # 1024 sequences x 32 heads x 1 split x 130 floats = 4.26 M floats > the 4 Mi the library holds.
    # The size check comes before any launch, so the (tiny, unrelated) buffers are never read.
    B, n_q, n_kv, hd, S = 1024, 32, 8, 128, 16384
    q = torch.zeros(B, n_q * hd, dtype=torch.bfloat16, device=DEV)
    pool = torch.zeros(1, 128, n_kv, hd, dtype=torch.bfloat16, device=DEV)
    bt = torch.zeros(B, S // 128, dtype=torch.int32, device=DEV)
    out = torch.zeros_like(q)
    with pytest.raises(PopError) as e:
        L.decode_attention_static(q, pool, pool, bt, out, n_q, n_kv, hd, S, 128, 0)
    assert e.value.code == POP_E_NOSPACE
    with pytest.raises(PopError) as e:
        L.decode_attention_static(q, pool, pool, bt, out, n_q, n_kv, 96, S, 128, 0)
    assert e.value.code == POP_E_INVALID
    assert (out == 0).all()
