"""kf_decode_step_static: the generation step for callers that cannot allocate device memory
(its scratch is a fixed block inside the library).  Checked against kf_decode_step on the same
state and inputs, two steps in a row, through the C ABI.  Collected last on purpose."""
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


@pytest.mark.parametrize("d,positional", [(128, "none"), (64, "alibi")])
def test_static_scratch_step_matches_context_step(d, positional):
    wl = W.Workload("static", 1, 2, 3, d, 333, 200, 50, 8, data_seed=21, noise_seed=9, positional=positional)
    gpu = lockstep.make_gpu(wl)
    Q, K, V = W.make_prompt(wl, 0, DEV)
    gpu.kf_prefill_score_prune(0, Q, K, V)
    torch.cuda.synchronize()
    # the caller-held copy of the cache that the static variant works on
    mine = [t.clone() for t in gpu.kf_view_state(0)]
    slopes = torch.tensor(W.alibi_slopes(wl.n_heads), dtype=torch.float32, device=DEV) if positional == "alibi" else None
    for step in (1, 2):
        q, kn, vn = W.make_step(wl, 0, step, DEV)
        out_ref, out_new = torch.empty_like(q), torch.empty_like(q)
        sc_ref = torch.zeros(wl.batch, wl.n_heads, wl.budget_k + 1, device=DEV)
        sc_new = torch.zeros_like(sc_ref)
        gpu.kf_decode_step(0, step, q, kn, vn, out_ref, score_out=sc_ref)
        rc = kf.kf_decode_step_static(
            batch=wl.batch, n_heads=wl.n_heads, head_dim=d, budget_k=wl.budget_k, recent_w=wl.recent_w,
            layer=0, position=wl.prompt_len + step - 1, tau=_tau(wl, step),
            K=mine[0], V=mine[1], pos=mine[2], acc=mine[3], length=mine[4],
            q=q, knew=kn, vnew=vn, out=out_new, score_out=sc_new, noise_seed=wl.noise_seed,
            bias_mode=kf.KF_BIAS_ALIBI if slopes is not None else kf.KF_BIAS_NONE, alibi_slopes_dev=slopes)
        assert rc == kf.KF_OK
        torch.cuda.synchronize()
        assert gpu.kf_poll_error() == 0
        scale = out_ref.float().abs().amax(dim=-1, keepdim=True)
        assert ((out_new.float() - out_ref.float()).abs() <= lockstep.OUT_RTOL * scale).all()
        assert ((sc_new - sc_ref).abs() <= lockstep.SCORE_RTOL * sc_ref.abs() + lockstep.SCORE_ATOL).all()
        ref = gpu.kf_view_state(0)
        torch.cuda.synchronize()
        assert torch.equal(mine[2], ref[2]) and torch.equal(mine[4], ref[4])          # positions, lengths
        assert torch.equal(mine[0], ref[0]) and torch.equal(mine[1], ref[1])          # K, V rows
        assert ((mine[3] - ref[3]).abs() <= lockstep.SCORE_RTOL * ref[3].abs() + 1e-6).all()


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
