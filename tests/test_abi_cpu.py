"""CPU-side checks of the boundary: the library loads, exports every declared symbol,
validates configurations on the host and refuses to compute without a device."""
import ctypes as C
import os
import re

import pytest
import torch

import paper_2403_09054_b200 as kf

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "keyformer.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(kf_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    syms = _declared_symbols()
    assert set(kf.EXPORTS) <= set(syms)
    lib = C.CDLL(kf.LIB_PATH)
    for s in syms:
        assert hasattr(lib, s), f"{s} declared in include/keyformer.h but not exported"


def _cfg(**kw):
    base = dict(n_layers=2, batch=2, n_heads=4, head_dim=128, budget_k=64, recent_w=16, max_prompt_len=128, gen_len_T=8)
    base.update(kw)
    return kf.make_config(**base)[0]


def test_workspace_size_covers_the_cache():
    cfg = _cfg()
    nbytes = kf.kf_workspace_bytes(cfg)
    kv = 2 * 2 * 2 * 4 * 64 * 128 * 2
    assert nbytes >= kv and nbytes % 256 == 0


def test_new_positions_cost_one_int32_per_slot():
    base, new = kf.kf_workspace_bytes(_cfg()), kf.kf_workspace_bytes(_cfg(pos_mode=kf.KF_POS_NEW))
    assert new - base == 2 * 2 * 4 * 64 * 4          # layers x batch x heads x k x sizeof(int32), already 256-aligned


@pytest.mark.parametrize("bad", [dict(head_dim=96), dict(budget_k=0), dict(recent_w=65), dict(recent_w=-1),
                                 dict(tau_init=0.0), dict(tau_end=-1.0), dict(n_layers=0), dict(gen_len_T=-1),
                                 dict(noise_mode=7), dict(bias_mode=1), dict(max_prompt_len=0), dict(pos_mode=2),
                                 dict(pos_mode=-1)])
def test_invalid_configurations_are_rejected(bad):
    assert kf.kf_workspace_bytes(_cfg(**bad)) == 0


def test_create_rejects_bad_arguments_on_the_host():
    cfg = _cfg()
    h = C.c_void_p()
    assert kf.LIB.kf_create(C.byref(cfg), None, 1 << 30, None, C.byref(h)) == kf.KF_EINVAL
    assert kf.LIB.kf_create(C.byref(cfg), 256, 16, None, C.byref(h)) == kf.KF_ENOSPC
    assert kf.LIB.kf_create(C.byref(cfg), 257, 1 << 40, None, C.byref(h)) == kf.KF_EINVAL   # misaligned
    assert kf.LIB.kf_destroy(None) == kf.KF_EINVAL
    assert kf.kf_strerror(kf.KF_ESTATE) == "call out of order"


@pytest.mark.skipif(torch.cuda.is_available(), reason="only meaningful without a device")
def test_no_cpu_fallback():
    with pytest.raises(kf.KeyformerError) as e:
        kf.Keyformer(n_layers=1, batch=1, n_heads=1, head_dim=64, budget_k=8, recent_w=2, max_prompt_len=16, gen_len_T=4)
    assert e.value.code == kf.KF_ECUDA
    cfg = _cfg()
    h = C.c_void_p()
    assert kf.LIB.kf_create(C.byref(cfg), 256, 1 << 40, None, C.byref(h)) == kf.KF_ECUDA
