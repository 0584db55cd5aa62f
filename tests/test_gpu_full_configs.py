"""Parity at the full sizes of the five workloads, in the launch configuration the benchmark times.
The oracle runs on a seeded sample of units (units are independent), the GPU on everything."""
import numpy as np
import pytest
import torch

import paper_2403_09054_b200 as kf
import workloads as W
from workloads.configs import C5_BUDGET_FRACTIONS, c5_budget
from tests import lockstep

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _report(tag, r):
    """One line per workload for the test log: units and steps compared, eviction choices adopted from the GPU
    (decisions inside the tolerance band), largest relative errors seen."""
    print(f"\nLOCKSTEP {tag}: units={r['units']} steps={r['steps']} adoptions={r['adoptions']} "
          f"max_out_err={r['max_out_err']:.3e} max_score_err={r['max_score_err']:.3e}")


def test_config2_gptj_all_units_all_steps():
    wl = W.get_config("c2_gptj")
    r = lockstep.run_workload(wl, check_state_every=32)
    assert r["units"] == 16 and r["steps"] == 256
    _report("c2_gptj", r)


@pytest.mark.parametrize("pos_mode", [0, 1])
def test_config2_gptj_rotation_applied_by_the_library_all_units_all_steps(pos_mode):
    """The rotary workload with Q/K passed unrotated and a cache of unrotated keys: original positions, and positions
    within the reduced cache (section 4.4.2 on a rotary model)."""
    wl = W.get_config("c2_gptj").scaled(rotary_in_library=True)
    r = lockstep.run_workload(wl, check_state_every=64, pos_mode=pos_mode)
    assert r["units"] == 16 and r["steps"] == 256
    _report("c2_gptj, rotation by the library" + (", new positions" if pos_mode else ""), r)


@pytest.mark.parametrize("pos_mode", [0, 1])
def test_config3_mpt_sampled_units_all_steps(pos_mode):
    """The ALiBi workload at full size for all 512 steps, with original positions in the bias and with the bias
    counted in places of the reduced cache (section 4.4.2)."""
    wl = W.get_config("c3_mpt")
    r = lockstep.run_workload(wl, units_per_layer=8, check_state_every=64, pos_mode=pos_mode)
    assert r["units"] == 8 and r["steps"] == 512
    _report("c3_mpt" + (" new positions" if pos_mode else ""), r)


def test_config4_cerebras_three_layers_sampled_units_all_steps():
    """66 units sampled from the first, the middle and the last layer, all 256 steps.  The context is the full
    32-layer one (the launch configuration the benchmark times); only the three layers are given a prompt."""
    wl = W.get_config("c4_cerebras")
    r = lockstep.run_workload(wl, units_per_layer=22, layers=[0, wl.n_layers // 2 - 1, wl.n_layers - 1], check_state_every=64)
    assert r["units"] == 66 and r["steps"] == 256
    _report("c4_cerebras", r)


def test_config4_cerebras_with_shared_key_value_heads_sampled_units_all_steps():
    """The Cerebras-shaped model with its 32 query heads on 8 key/value heads (section 6), 24 caches of three layers,
    all 256 steps."""
    wl = W.get_config("c4_cerebras_gqa8")
    r = lockstep.run_workload(wl, units_per_layer=8, layers=[0, wl.n_layers // 2 - 1, wl.n_layers - 1], check_state_every=64)
    assert r["units"] == 24 and r["steps"] == 256
    _report("c4_cerebras_gqa8", r)


@pytest.mark.parametrize("name", ["c5_prefill_1k", "c5_prefill_2k", "c5_prefill_4k", "c5_prefill_8k"])
def test_config5_prefill_sweep(name):
    base = W.get_config(name)
    n = base.prompt_len
    q, k, v = W.make_prompt(base, 0, DEV)
    units = W.sample_units(base, 16, seed=n, layer=0)
    acc_ref = None
    adoptions = []
    for frac in C5_BUDGET_FRACTIONS:
        kk, w = c5_budget(n, frac)
        wl = base.scaled(budget_k=kk, recent_w=w)
        gpu = lockstep.make_gpu(wl)
        ls = lockstep.LockStep(wl, gpu, 0, units)
        if acc_ref is None:
            acc_ref = ls.prefill(q, k, v)            # scores do not depend on the budget: oracle scores once
        else:
            ls.st.prefill_score = lambda Q, K, _a=acc_ref: _a
            ls.prefill(q, k, v)
        # every unit of the GPU (not only the sampled ones) keeps exactly k entries incl. the recent window
        _, _, pos, _, ln = gpu.kf_view_state(0)
        torch.cuda.synchronize()
        assert (ln == kk).all()
        assert (pos[..., -w:] == torch.arange(n - w, n, device=DEV, dtype=torch.int32)).all()
        assert (pos[..., 1:] > pos[..., :-1]).all()
        adoptions.append(ls.adoptions)
        lockstep.check_guards(gpu)
        gpu.kf_destroy()
    print(f"\nLOCKSTEP {name}: units={len(units)} budgets={list(C5_BUDGET_FRACTIONS)} adoptions={adoptions} "
          f"max_score_err={ls.max_score_err:.3e}")
