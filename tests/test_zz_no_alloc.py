"""kf_decode_step_static: the generation step for callers that cannot allocate device memory
(its scratch is a fixed block inside the library).  Checked through the C ABI, two steps in a row,
against kf_decode_step on the same state and inputs and against the CPU oracle; free device memory
must not move across the calls.  Collected last on purpose."""
import numpy as np
import pytest
import torch

import paper_2403_09054_b200 as kf
import workloads as W
from tests import lockstep

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _tau(wl, step):
    t = min(step, wl.gen_len_T)
    return wl.tau_init + t * ((wl.tau_end - wl.tau_init) / wl.gen_len_T)


def _static_step(wl, mine, step, q, kn, vn, out, score, slopes):
    return kf.kf_decode_step_static(
        batch=wl.batch, n_heads=wl.n_heads, head_dim=wl.head_dim, budget_k=wl.budget_k, recent_w=wl.recent_w,
        layer=0, position=wl.prompt_len + step - 1, tau=_tau(wl, step),
        K=mine[0], V=mine[1], pos=mine[2], acc=mine[3], length=mine[4],
        q=q, knew=kn, vnew=vn, out=out, score_out=score, noise_seed=wl.noise_seed,
        bias_mode=kf.KF_BIAS_ALIBI if slopes is not None else kf.KF_BIAS_NONE, alibi_slopes_dev=slopes)


@pytest.mark.parametrize("d,positional", [(128, "none"), (64, "alibi")])
def test_static_scratch_step_matches_context_step_and_oracle(d, positional):
    wl = W.Workload("static", 1, 2, 3, d, 333, 200, 50, 8, data_seed=21, noise_seed=9, positional=positional)
    gpu = lockstep.make_gpu(wl)
    ls = lockstep.LockStep(wl, gpu, 0, W.unit_list(wl, 0))               # the oracle walks along
    ls.prefill(*W.make_prompt(wl, 0, DEV))
    torch.cuda.synchronize()
    # the caller-held copy of the cache that the static variant works on
    mine = [t.clone() for t in gpu.kf_view_state(0)]
    slopes = torch.tensor(W.alibi_slopes(wl.n_heads), dtype=torch.float32, device=DEV) if positional == "alibi" else None
    # the first call on a device loads the kernels' module (the block is part of it) and looks up the block's address:
    # made here on a throw-away copy of the state, so that the calls below can be watched for allocations
    q, kn, vn = W.make_step(wl, 0, 1, DEV)
    assert _static_step(wl, [t.clone() for t in mine], 1, q, kn, vn, torch.empty_like(q), None, slopes) == kf.KF_OK
    for step in (1, 2):
        q, kn, vn = W.make_step(wl, 0, step, DEV)
        out_new = torch.empty_like(q)
        sc_new = torch.zeros(wl.batch, wl.n_heads, wl.budget_k + 1, device=DEV)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        rc = _static_step(wl, mine, step, q, kn, vn, out_new, sc_new, slopes)
        assert rc == kf.KF_OK
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before               # the call obtained no device memory
        # the context's own step on the same inputs, compared with the oracle by the lock-step driver
        out_ref, sc_ref = ls.decode_step(step, q, kn, vn)
        U = wl.batch * wl.n_heads
        out_n = out_new.reshape(U, d).double().cpu().numpy()
        sc_n = sc_new.reshape(U, -1).double().cpu().numpy()
        scale = np.abs(out_ref).max(axis=-1, keepdims=True)
        assert (np.abs(out_n - out_ref) <= lockstep.OUT_RTOL * scale).all()
        assert (np.abs(sc_n - sc_ref) <= lockstep.SCORE_RTOL * np.abs(sc_ref) + lockstep.SCORE_ATOL).all()
        ref = gpu.kf_view_state(0)
        torch.cuda.synchronize()
        assert torch.equal(mine[2], ref[2]) and torch.equal(mine[4], ref[4])          # positions, lengths
        assert torch.equal(mine[0], ref[0]) and torch.equal(mine[1], ref[1])          # K, V rows
        assert ((mine[3] - ref[3]).abs() <= lockstep.SCORE_RTOL * ref[3].abs() + 1e-6).all()
    lockstep.check_guards(gpu)


def test_static_scratch_is_reused_by_calls_of_different_shapes():
    """A large call leaves its adjusted logits and partials in the block; a small call right after it must not be
    disturbed by them (nothing in the block has to start at zero), and the reverse."""
    big = W.Workload("static_big", 1, 2, 4, 128, 1500, 1200, 100, 4, data_seed=31, noise_seed=3)
    small = W.Workload("static_small", 1, 1, 2, 128, 90, 40, 10, 4, data_seed=32, noise_seed=4)
    state = {}
    for wl in (big, small):
        gpu = lockstep.make_gpu(wl)
        gpu.kf_prefill_score_prune(0, *W.make_prompt(wl, 0, DEV))
        torch.cuda.synchronize()
        state[wl.name] = (gpu, [t.clone() for t in gpu.kf_view_state(0)])
    for step, order in ((1, (big, small)), (2, (small, big))):
        for wl in order:
            gpu, mine = state[wl.name]
            q, kn, vn = W.make_step(wl, 0, step, DEV)
            out_ref, out_new = torch.empty_like(q), torch.empty_like(q)
            gpu.kf_decode_step(0, step, q, kn, vn, out_ref)
            assert _static_step(wl, mine, step, q, kn, vn, out_new, None, None) == kf.KF_OK
            torch.cuda.synchronize()
            assert torch.equal(out_new, out_ref)                         # same kernels, same inputs, same split plan
            assert torch.equal(mine[2], gpu.kf_view_state(0)[2])
    for gpu, _ in state.values():
        lockstep.check_guards(gpu)


def test_static_scratch_rejects_oversized_and_invalid_requests():
    dummy = torch.zeros(16, dtype=torch.float16, device=DEV)
    args = kf.kf_static_step()
    args.batch, args.n_heads, args.head_dim, args.budget_k, args.recent_w = 64, 64, 128, 4096, 16
    args.tau = 1.0
    ptr = dummy.data_ptr()
    # 4096 units x 4097 scores x 4 bytes is far beyond the 16 MiB block: refused before any launch
    rc = kf.LIB.kf_decode_step_static(args, ptr, ptr, ptr, ptr, ptr, ptr, ptr, ptr, ptr, None, None)
    assert rc == kf.KF_ENOSPC
    args.head_dim = 100
    assert kf.LIB.kf_decode_step_static(args, ptr, ptr, ptr, ptr, ptr, ptr, ptr, ptr, ptr, None, None) == kf.KF_EINVAL
    torch.cuda.synchronize()
