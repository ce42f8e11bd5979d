"""The WHOLE oracle against pop_prefill at the benchmark configurations' own sizes (configs 2-4), in
the launch configuration bench.py times: every layer's K and V over all positions, the state H
leaving the kept stack, the boundary token's final state and the logits, element by element.

Config 2 and config 3 run whole (about two minutes of fp32 oracle each on 16 host cores); config 4
(48 layers x 16384 positions, about eight minutes) runs whole when POP_PARITY_FULL=1 and otherwise
on its first 12 layers with L_keep 9, which keeps a kept and a pruned global-attention layer (6, 12)
among the sliding-window ones. The per-layer tables of the whole runs are recorded in the design
notes; set POP_PARITY_DIR to have this test write them.

What is asserted (tests/gpu_util.py states the budgets and where they come from):
  * layers 1..4: the stated tolerance, per tensor max|err| / max|ref| <= 2e-2;
  * every layer: RMS and maximum relative error within the depth budget c * sqrt(l) of a bf16-operand
    pipeline (pruned layers are budgeted at their own depth, although their prompt rows only carry
    the error of H); no non-finite value anywhere;
  * H, the boundary token's final state and the logits within the same budgets;
  * the first token: if the GPU's arg-max differs from the exact oracle's, the oracle's two best
    logits must be closer than twice the measured logits error (a near-tie, not a wrong token).
"""
import os

import pytest
import torch

import pop_synth as ps
from tests import full_parity
from tests.gpu_util import STATED_DEPTH, STATED_KV_TOL, kv_budget, logits_budget

pytestmark = pytest.mark.gpu


def _workload(key):
    wl = ps.WORKLOADS[key]
    if key == "c4" and os.environ.get("POP_PARITY_FULL", "0") != "1":
        wl = ps.Workload("c4", wl.model.replace(n_layers=12), wl.batch, wl.seq_len, 9)
    return wl


@pytest.mark.parametrize("key", ["c2", "c3", "c4"])
def test_whole_oracle_at_the_benchmark_size(key):
    wl = _workload(key)
    L, Lk = wl.model.n_layers, wl.l_keep
    res = full_parity.compare(wl)
    text = f"{key}: {wl.model.name} L={L} L_keep={Lk} N={wl.seq_len}\n" + full_parity.table(res)
    print("\n" + text)
    out_dir = os.environ.get("POP_PARITY_DIR")
    if out_dir:
        with open(os.path.join(out_dir, f"parity_{key}_L{L}.txt"), "w") as f:
            f.write(text + "\n")
    for r in res["rows"]:
        l = r["layer"]
        assert r["finite"], f"layer {l}"
        if l <= STATED_DEPTH:
            assert r["K"] <= STATED_KV_TOL and r["V"] <= STATED_KV_TOL, (l, r["K"], r["V"])
        rms_b, max_b = kv_budget(l)
        assert r["K_rms"] <= rms_b and r["V_rms"] <= rms_b, (l, r["K_rms"], r["V_rms"], rms_b)
        assert r["K"] <= max_b and r["V"] <= max_b, (l, r["K"], r["V"], max_b)
        assert r["K_last"] <= max_b and r["V_last"] <= max_b, (l, r["K_last"], r["V_last"], max_b)
    rms_b, max_b = kv_budget(Lk)
    assert res["H_rms"] <= rms_b and res["H"] <= max_b, (res["H_rms"], res["H"])
    rms_b, max_b = kv_budget(L)
    assert res["x_last_rms"] <= rms_b and res["x_last"] <= max_b, (res["x_last_rms"], res["x_last"])
    rms_b, max_b = logits_budget(L, res["logits_std"])
    assert res["logits_rms"] <= rms_b and res["logits"] <= max_b, (res["logits_rms"], res["logits"], rms_b, max_b)
    for agree, gap in zip(res["argmax_agree"], res["top2_gap"]):
        assert agree or gap <= 2.0 * res["logits"], (gap, res["logits"])
