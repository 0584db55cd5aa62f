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


def test_config2_gptj_all_units():
    wl = W.get_config("c2_gptj")
    r = lockstep.run_workload(wl, steps=24, check_state_every=8)
    print("c2", r)


def test_config3_mpt_sampled_units():
    wl = W.get_config("c3_mpt")
    r = lockstep.run_workload(wl, units_per_layer=6, steps=12, check_state_every=6)
    print("c3", r)


def test_config3_mpt_new_positions_sampled_units():
    """The ALiBi workload at full size with the bias counted in places of the reduced cache (section 4.4.2)."""
    wl = W.get_config("c3_mpt")
    r = lockstep.run_workload(wl, units_per_layer=4, steps=8, check_state_every=4, pos_mode=1)
    print("c3 new positions", r)


def test_config4_cerebras_first_and_last_layer_sampled_units():
    wl = W.get_config("c4_cerebras")
    r = lockstep.run_workload(wl, units_per_layer=8, steps=6, layers=[0, wl.n_layers - 1], check_state_every=3)
    print("c4", r)


@pytest.mark.parametrize("name", ["c5_prefill_1k", "c5_prefill_2k", "c5_prefill_4k", "c5_prefill_8k"])
def test_config5_prefill_sweep(name):
    base = W.get_config(name)
    n = base.prompt_len
    q, k, v = W.make_prompt(base, 0, DEV)
    units = W.sample_units(base, 4 if n >= 4096 else 8, seed=n, layer=0)
    acc_ref = None
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
        gpu.kf_destroy()
