"""The seeded input generators: determinism, slicing, value ranges, rough statistics."""
import torch

import pop_synth as ps


def test_normal_is_deterministic_and_sliceable():
    tid = ps.tensor_id("wq", 3)
    a = ps.normal_bf16(7, tid, (64, 48), 0.02)
    b = ps.normal_bf16(7, tid, (64, 48), 0.02)
    assert a.dtype == torch.bfloat16 and torch.equal(a, b)
    part = ps.normal_bf16(7, tid, (64, 48), 0.02, row_start=10, row_count=5)
    assert torch.equal(part, a[10:15])
    other = ps.normal_bf16(8, tid, (64, 48), 0.02)
    assert not torch.equal(a, other)
    other_t = ps.normal_bf16(7, ps.tensor_id("wq", 4), (64, 48), 0.02)
    assert not torch.equal(a, other_t)


def test_normal_statistics():
    x = ps.normal_bf16(1, ps.tensor_id("w_up", 1), (512, 1024), 0.02).double()
    assert abs(x.mean().item()) < 2e-4
    assert abs(x.std().item() - 0.02) < 3e-4
    assert x.abs().max().item() <= 6 * 0.02 * 1.01
    # fourth moment close to a normal's (Irwin-Hall of 12 has kurtosis 3 - 0.1)
    k = (x.pow(4).mean() / x.pow(2).mean() ** 2).item()
    assert 2.8 < k < 3.0


def test_chunk_boundaries_do_not_matter(monkeypatch):
    tid = ps.tensor_id("embed")
    a = ps.normal_bf16(3, tid, (100, 37), 0.02)
    monkeypatch.setattr(ps, "_CHUNK", 1000)
    b = ps.normal_bf16(3, tid, (100, 37), 0.02)
    assert torch.equal(a, b)


def test_tokens_and_gains():
    t = ps.uniform_tokens(5, 3, 1000, 1024)
    assert t.dtype == torch.int32 and t.shape == (3, 1000)
    assert t.min() >= 0 and t.max() < 1024
    assert not torch.equal(t[0], t[1])
    assert len(torch.unique(t[0])) > 500
    g1 = ps.gains(5, 1, 256, False)
    assert torch.all(g1 == 1.0)
    g = ps.gains(5, 1, 4096, True)
    assert g.min() >= 0.5 and g.max() < 1.5
    assert torch.equal(g, g.to(torch.bfloat16).float())
    assert len(torch.unique(g)) > 100


def test_visual_embeds_have_unit_rms():
    e = ps.visual_embeds(5, 1, 16, 256).double()
    rms = e.pow(2).mean(dim=-1).sqrt()
    assert torch.allclose(rms, torch.ones_like(rms), atol=5e-3)


def test_weight_provider_shapes():
    cfg = ps.C1_TINY
    w = ps.SynthWeights(cfg)
    assert w.get("wq", 1).shape == (256, 256)
    assert w.get("wk", 2).shape == (128, 256)
    assert w.get("w_down", 4).shape == (256, 688)
    assert w.get("ln_in", 1).dtype == torch.float32
    ids = torch.tensor([5, 9, 5])
    rows = w.embedding_rows(ids)
    full = w.get("embed")
    assert torch.equal(rows, full[ids])


def test_prompt_recipe_for_embedding_inputs():
    wl = ps.Workload("t", ps.C1_TINY, 2, 12, 3, n_visual=8)
    tok, emb = ps.make_prompt(wl)
    assert (tok[:, :8] == -1).all() and (tok[:, 8:] >= 0).all()
    assert emb.shape == (2, 12, 256) and emb[:, 8:].abs().max() == 0
