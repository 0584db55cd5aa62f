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


def test_static_step_validates_before_touching_the_device():
    """kf_decode_step_static checks its arguments before its first CUDA call: reserved field, noise mode,
    alignment (all refused with KF_EINVAL and nothing launched; this runs without a device)."""
    a = kf.kf_static_step()
    a.batch, a.n_heads, a.head_dim, a.budget_k, a.recent_w = 1, 2, 64, 32, 8
    a.tau = 1.0
    ok = 4096                                            # a 16-byte aligned (never dereferenced) address
    call = lambda *p: kf.LIB.kf_decode_step_static(C.byref(a), *p, None, None)
    a.reserved = 1
    assert call(ok, ok, ok, ok, ok, ok, ok, ok, ok) == kf.KF_EINVAL
    a.reserved = 0
    a.noise_mode = kf.KF_NOISE_GAUSS
    assert call(ok, ok, ok, ok, ok, ok, ok, ok, ok) == kf.KF_EINVAL
    a.noise_mode = kf.KF_NOISE_GUMBEL
    for i in (0, 1, 5, 6, 7, 8):                         # K, V, q, k_new, v_new, out: 16-byte alignment
        p = [ok] * 9
        p[i] = ok + 2
        assert call(*p) == kf.KF_EINVAL
    for i in (2, 3, 4):                                  # positions, scores, entry counts: 4-byte alignment
        p = [ok] * 9
        p[i] = ok + 2
        assert call(*p) == kf.KF_EINVAL
    a.budget_k = 1 << 22                                 # scratch beyond the built-in block
    assert call(ok, ok, ok, ok, ok, ok, ok, ok, ok) == kf.KF_ENOSPC


def test_error_codes_have_messages():
    for code in (kf.KF_EINVAL, kf.KF_ENOSPC, kf.KF_ESTATE, kf.KF_ECUDA, kf.KF_ETIMEOUT, kf.KF_EBOUNDS):
        assert kf.kf_strerror(code) not in ("ok", "unknown error")
    assert kf.kf_strerror(-99) == "unknown error"


def test_guard_blocks_enlarge_the_workspace():
    base, dbg = kf.kf_workspace_bytes(_cfg()), kf.kf_workspace_bytes(_cfg(debug_canaries=1))
    assert dbg - base == 14 * 256                        # one guard behind each of the 14 sub-buffers (no places)
    assert kf.kf_workspace_bytes(_cfg(debug_canaries=2)) == 0 and kf.kf_workspace_bytes(_cfg(debug_fail_first_wait=3)) == 0


def test_unsupported_group_sizes_are_rejected():
    for hkv in (3, 5, 7):           # 12 / 5, 12 / 7 do not divide; 12 / 3 = 4 is fine
        cfg = kf.make_config(n_layers=1, batch=1, n_heads=12, n_kv_heads=hkv, head_dim=64, budget_k=8, recent_w=2,
                             max_prompt_len=16, gen_len_T=4)[0]
        assert (kf.kf_workspace_bytes(cfg) > 0) == (hkv == 3)
    cfg = kf.make_config(n_layers=1, batch=1, n_heads=32, n_kv_heads=1, head_dim=64, budget_k=8, recent_w=2,
                         max_prompt_len=16, gen_len_T=4)[0]
    assert kf.kf_workspace_bytes(cfg) == 0              # 32 query heads on one cache: more than the kernels are built for


def test_tensor_core_generation_kernel_is_refused_where_it_is_not_built():
    assert kf.kf_workspace_bytes(_cfg(decode_impl=kf.KF_DECODE_TENSOR)) > 0                 # head_dim 128
    assert kf.kf_workspace_bytes(_cfg(decode_impl=kf.KF_DECODE_TENSOR, head_dim=64)) == 0
    assert kf.kf_workspace_bytes(_cfg(decode_impl=3)) == 0


def test_rotary_configuration_limits():
    assert kf.kf_workspace_bytes(_cfg(rotary_dims=64)) > kf.kf_workspace_bytes(_cfg())     # table + rotated prompt copies
    for bad in (dict(rotary_dims=4), dict(rotary_dims=48), dict(rotary_dims=256), dict(rotary_dims=64, rotary_base=1.0),
                dict(rotary_dims=64, decode_impl=kf.KF_DECODE_TENSOR)):
        assert kf.kf_workspace_bytes(_cfg(**bad)) == 0
