"""GPU parity of the prompt-phase attention output (Eq. 1 under the causal mask) against the CPU oracle,
through the C ABI."""
import numpy as np
import pytest
import torch

import paper_2403_09054_b200 as kf
import workloads as W
from oracle import keyformer_oracle as ko
from tests import lockstep

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _check(wl, units=None, edit=None):
    gpu = lockstep.make_gpu(wl)
    q, k, v = W.make_prompt(wl, 0, DEV)
    if edit is not None:
        edit(q, k, v)
    out = torch.empty_like(q)
    gpu.kf_prefill_attend(q, k, v, out)
    assert gpu.kf_poll_error() == 0
    lbh = W.unit_list(wl, 0) if units is None else W.sample_units(wl, units, seed=3, layer=0)
    flat = torch.as_tensor(lbh[:, 1] * wl.kv_heads + lbh[:, 2], dtype=torch.long, device=DEV)
    # one entry per cache; tensors with one entry per query head give [U, g, n, d] when g heads share a cache
    rows = lambda t: t.reshape(wl.batch * wl.kv_heads, -1, wl.prompt_len, wl.head_dim)[flat].squeeze(1).cpu().numpy()
    st = ko.State(lockstep.oracle_params(wl), lbh)
    ref = st.prefill_attend(rows(q), rows(k), rows(v))
    got = rows(out).astype(np.float64)
    scale = np.abs(ref).max(axis=-1, keepdims=True)
    err = np.abs(got - ref) / scale
    assert err.max() <= lockstep.OUT_RTOL, f"attention output off by {err.max():.3e} of the row's largest value"
    lockstep.check_guards(gpu)
    gpu.kf_destroy()
    return float(err.max())


@pytest.mark.parametrize("d", [64, 128, 256])
@pytest.mark.parametrize("n", [1, 57, 64, 65, 128, 129, 300, 641])
def test_prompt_attention_small(n, d):
    _check(W.Workload("attend", 1, 2, 3, d, n, max(1, n // 2), n // 8, 0, data_seed=n + d, noise_seed=1))


@pytest.mark.parametrize("d,positional", [(128, "none"), (64, "alibi"), (128, "alibi")])
def test_prompt_attention_when_late_keys_dwarf_the_early_ones(d, positional):
    """Keys whose logits lie far above everything before them, first met in the third key tile and again, larger still,
    in the seventh: a one-pass kernel has to move the rows' reference exponent (and rescale what it has accumulated)
    in the middle of the walk, twice, and rows that end before a band must not be touched by it."""
    def edit(q, k, v):
        k[..., 300:340, :] *= 14.0       # logits of these keys: standard deviation 14 instead of 1
        k[..., 800:806, :] *= 60.0
        k[..., 1100:1101, :] *= 0.0      # and a key every row is indifferent to
    _check(W.Workload("attend_spikes", 1, 2, 3, d, 1200, 300, 40, 0, data_seed=77, noise_seed=1, positional=positional), edit=edit)


@pytest.mark.parametrize("positional", ["alibi", "rotary"])
def test_prompt_attention_with_positional_structure(positional):
    _check(W.Workload("attend", 1, 2, 4, 128, 333, 100, 10, 0, data_seed=5, positional=positional, rotary_dims=32))


def test_prompt_attention_heavy_hitters_sampled_units():
    wl = W.get_config("c4_cerebras").scaled(n_layers=1, batch=2, n_heads=8, prompt_len=1500, budget_k=512, recent_w=128)
    _check(wl, units=4)


@pytest.mark.parametrize("d,positional", [(128, "none"), (64, "alibi"), (256, "rotary")])
def test_attend_and_score_in_one_call_match_the_separate_calls(d, positional):
    wl = W.Workload("attend", 1, 2, 3, d, 400, 150, 30, 4, data_seed=9, noise_seed=2, positional=positional, rotary_dims=32)
    q, k, v = W.make_prompt(wl, 0, DEV)
    a, b = lockstep.make_gpu(wl), lockstep.make_gpu(wl)
    out_a, out_b = torch.empty_like(q), torch.empty_like(q)
    sc_a = torch.empty(wl.batch, wl.n_heads, wl.prompt_len, device=DEV)
    sc_b = torch.empty_like(sc_a)
    a.kf_prefill_attend_score_prune(0, q, k, v, out_a, score_out=sc_a)
    b.kf_prefill_attend(q, k, v, out_b)
    b.kf_prefill_score_prune(0, q, k, v, score_out=sc_b)
    torch.cuda.synchronize()
    # the one-call form takes the rows' softmax statistics from the scoring sweep (another summation order)
    scale = out_b.float().abs().amax(dim=-1, keepdim=True)
    assert ((out_a.float() - out_b.float()).abs() <= 1e-3 * scale).all()
    assert torch.equal(sc_a, sc_b)
    for x, y in zip(a.kf_view_state(0), b.kf_view_state(0)):
        assert torch.equal(x, y)
    assert a.kf_poll_error() == 0 and b.kf_poll_error() == 0


def test_prompt_attention_gptj_shape_sampled_units():
    wl = W.get_config("c2_gptj").scaled(n_heads=4, prompt_len=1100, budget_k=512, recent_w=128)
    _check(wl, units=2)


@pytest.mark.parametrize("d,g,positional", [(128, 4, "none"), (64, 2, "alibi"), (256, 8, "rotary")])
def test_prompt_attention_with_shared_key_value_heads(d, g, positional):
    """g query heads read the keys and values of one cache (section 6: MQA / GQA)."""
    _check(W.Workload("attend_gqa", 1, 2, 2 * g, d, 333, 100, 10, 0, data_seed=6, positional=positional, rotary_dims=32,
                      n_kv_heads=2))
