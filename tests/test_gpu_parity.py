"""GPU parity: the CUDA library against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import paper_2403_09054_b200 as kf
import workloads as W
from tests import lockstep

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _wl(**kw):
    base = dict(name="t", n_layers=1, batch=2, n_heads=3, head_dim=64, prompt_len=100, budget_k=40, recent_w=10,
                gen_len_T=12, data_seed=11, noise_seed=5)
    base.update(kw)
    return W.Workload(**base)


@pytest.mark.parametrize("impl", [kf.KF_PREFILL_TENSOR, kf.KF_PREFILL_SIMT])
@pytest.mark.parametrize("d", [64, 128, 256])
def test_small_odd_shapes(d, impl):
    wl = _wl(head_dim=d, prompt_len=157, budget_k=71, recent_w=13)
    r = lockstep.run_workload(wl, gpu_kwargs=dict(prefill_impl=impl))
    assert r["max_out_err"] < 2e-3


@pytest.mark.parametrize("n", [1, 31, 128, 129, 257, 640, 1000])
@pytest.mark.parametrize("noise", ["gumbel", "none"])
def test_prompt_lengths_around_tile_edges(n, noise):
    """Prompt scoring only (T = 0): one row, a partial tile, exact tiles, several tiles with a ragged tail."""
    wl = _wl(head_dim=128, prompt_len=n, budget_k=max(1, n // 2), recent_w=max(0, n // 8), gen_len_T=0)
    lockstep.run_workload(wl, noise=noise)


@pytest.mark.parametrize("impl", [kf.KF_PREFILL_TENSOR, kf.KF_PREFILL_SIMT])
def test_prompts_shorter_than_the_maximum_and_a_context_used_again(impl):
    """A context sized for 700 positions takes prompts of 700, 129 and 300 tokens on the same layer one after
    the other (scratch of a longer prompt must not leak into a shorter one), each followed by decode steps."""
    for n in (700, 129, 300):
        wl = _wl(head_dim=128, prompt_len=n, budget_k=96, recent_w=24, gen_len_T=4, data_seed=100 + n)
        if n == 700:
            gpu = lockstep.make_gpu(wl, max_prompt_len=700, prefill_impl=impl)
        ls = lockstep.LockStep(wl, gpu, 0, W.unit_list(wl, 0))
        ls.prefill(*W.make_prompt(wl, 0, DEV))
        for s in range(1, 5):
            ls.decode_step(s, *W.make_step(wl, 0, s, DEV))
    with pytest.raises(kf.KeyformerError) as e:
        gpu.kf_prefill_score_prune(0, *W.make_prompt(_wl(head_dim=128, prompt_len=701), 0, DEV))
    assert e.value.code == kf.KF_EINVAL
    lockstep.check_guards(gpu)
    gpu.kf_destroy()


@pytest.mark.parametrize("scale", [2.0, 16.0])
def test_prompt_scores_with_extreme_logits(scale):
    """Logits hundreds of units apart (a scale far above 1/sqrt(d)): the prompt softmax must not overflow,
    and rows dominated by a single key must still match the oracle."""
    wl = _wl(head_dim=64, prompt_len=400, budget_k=150, recent_w=20, gen_len_T=2)
    lockstep.run_workload(wl, logit_scale=scale)


def test_prompt_scores_tensor_core_vs_cuda_core():
    """The two scoring implementations agree far inside the oracle tolerance, and the tensor-core
    one is reproducible bit for bit (no atomics)."""
    wl = _wl(head_dim=128, prompt_len=777, budget_k=300, recent_w=50, positional="alibi")
    q, k, v = W.make_prompt(wl, 0, DEV)
    scores = []
    for impl in (kf.KF_PREFILL_TENSOR, kf.KF_PREFILL_TENSOR, kf.KF_PREFILL_SIMT):
        gpu = lockstep.make_gpu(wl, prefill_impl=impl)
        s = torch.empty(wl.batch, wl.n_heads, wl.prompt_len, dtype=torch.float32, device=DEV)
        gpu.kf_prefill_score_prune(0, q, k, v, score_out=s)
        assert gpu.kf_poll_error() == 0
        scores.append(s)
        lockstep.check_guards(gpu)
        gpu.kf_destroy()
    assert torch.equal(scores[0], scores[1])
    assert torch.allclose(scores[0], scores[2], rtol=2e-4, atol=1e-6)
    assert torch.allclose(scores[0].sum(-1), torch.full_like(scores[0].sum(-1), float(wl.prompt_len)), rtol=1e-4)


@pytest.mark.parametrize("k,w,n", [(33, 0, 90), (32, 32, 90), (64, 1, 65), (40, 10, 30), (40, 10, 40), (1, 0, 5), (1, 1, 5)])
def test_edge_budgets(k, w, n):
    wl = _wl(prompt_len=n, budget_k=k, recent_w=w, gen_len_T=14)
    lockstep.run_workload(wl)


@pytest.mark.parametrize("splits", [1, 2, 3, 5])
def test_split_counts(splits):
    wl = _wl(head_dim=128, prompt_len=700, budget_k=517, recent_w=100, gen_len_T=6)
    lockstep.run_workload(wl, gpu_kwargs=dict(decode_splits=splits))


def test_large_budget_many_splits():
    """k = 6200 slots streamed by 48 CTAs per unit: the closing kernel merges more than 32 split partials."""
    wl = _wl(batch=1, n_heads=2, head_dim=64, prompt_len=6500, budget_k=6200, recent_w=100, gen_len_T=3)
    lockstep.run_workload(wl, gpu_kwargs=dict(decode_splits=48))


@pytest.mark.parametrize("impl", [kf.KF_PREFILL_TENSOR, kf.KF_PREFILL_SIMT])
@pytest.mark.parametrize("noise", ["none", "const", "gauss"])
def test_other_adjustments(noise, impl):
    lockstep.run_workload(_wl(head_dim=128, prompt_len=300, budget_k=120, recent_w=30), noise=noise,
                          gpu_kwargs=dict(prefill_impl=impl))


@pytest.mark.parametrize("seed", range(16))
def test_random_small_configurations(seed):
    """Seeded random shapes, budgets, temperatures, adjustments and biases, prompt phase plus a few steps."""
    rng = np.random.default_rng(1000 + seed)
    n = int(rng.integers(1, 420))
    k = int(rng.integers(1, 300))
    w = int(rng.integers(0, k + 1))
    wl = W.Workload(name=f"fuzz{seed}", n_layers=int(rng.integers(1, 3)), batch=int(rng.integers(1, 4)),
                    n_heads=int(rng.integers(1, 5)), head_dim=int(rng.choice([64, 128, 256])), prompt_len=n,
                    budget_k=k, recent_w=w, gen_len_T=int(rng.integers(0, 9)),
                    tau_init=float(rng.choice([0.5, 1.0, 1.5])), tau_end=float(rng.choice([1.0, 2.0, 3.0])),
                    data_seed=seed, noise_seed=int(rng.integers(0, 2 ** 62)),
                    positional=str(rng.choice(["none", "alibi", "rotary"])), rotary_dims=32)
    noise = str(rng.choice(["gumbel", "gumbel", "none", "const", "gauss"]))
    impl = kf.KF_PREFILL_TENSOR if seed % 4 else kf.KF_PREFILL_SIMT
    steps = int(rng.integers(0, 7))          # may run past T: the temperature is clamped there
    lockstep.run_workload(wl, steps=steps, noise=noise, gpu_kwargs=dict(prefill_impl=impl))


def test_zero_noise_tau_one_scores_are_attention_weights():
    wl = _wl(head_dim=128, tau_init=1.0, tau_end=1.0, gen_len_T=3)
    gpu = lockstep.make_gpu(wl, noise_mode=kf.KF_NOISE_NONE)
    q, k, v = W.make_prompt(wl, 0, DEV)
    gpu.kf_prefill_score_prune(0, q, k, v)
    K, V, pos, acc, ln = gpu.kf_view_state(0)
    Kb, Vb = K.clone().float(), V.clone().float()
    qs, kn, vn = W.make_step(wl, 0, 1, DEV)
    out = torch.empty_like(qs)
    score = torch.zeros(wl.batch, wl.n_heads, wl.budget_k + 1, device=DEV)
    gpu.kf_decode_step(0, 1, qs, kn, vn, out, score_out=score)
    torch.cuda.synchronize()
    assert torch.allclose(score.sum(-1), torch.ones_like(score.sum(-1)), atol=1e-5)
    Vall = torch.cat([Vb, vn.float()[:, :, None, :]], dim=2)
    rebuilt = torch.einsum("bhm,bhmd->bhd", score, Vall)
    assert (rebuilt - out.float()).abs().max() < 2e-3 * out.float().abs().max()


def test_alibi_and_rotary_workloads_scaled_down():
    lockstep.run_workload(W.get_config("c3_mpt").scaled(n_heads=4, prompt_len=600, budget_k=300, recent_w=75, gen_len_T=10))
    lockstep.run_workload(W.get_config("c2_gptj").scaled(n_heads=2, prompt_len=300, budget_k=150, recent_w=37, gen_len_T=10))


@pytest.mark.parametrize("d,n,k,w", [(128, 600, 300, 75), (64, 200, 96, 0), (256, 150, 40, 40), (128, 40, 64, 16)])
def test_new_positions_in_the_bias(d, n, k, w):
    """"New Pos" (section 4.4.2) with ALiBi: the bias distance is the place within the reduced cache.  Covers
    several splits, no recent window, window = budget, and a cache that only fills up during generation."""
    wl = W.get_config("c3_mpt").scaled(n_heads=4, head_dim=d, prompt_len=n, budget_k=k, recent_w=w, gen_len_T=30)
    r = lockstep.run_workload(wl, pos_mode=1)
    assert r["steps"] == 30


def test_new_positions_differ_from_original_positions_and_survive_import():
    wl = W.get_config("c3_mpt").scaled(n_heads=4, batch=2, prompt_len=300, budget_k=128, recent_w=32, gen_len_T=12)
    q, k, v = W.make_prompt(wl, 0, DEV)

    def run(gpu, first, last):
        outs = []
        for s in range(first, last + 1):
            qs, kn, vn = W.make_step(wl, 0, s, DEV)
            out = torch.empty_like(qs)
            gpu.kf_decode_step(0, s, qs, kn, vn, out)
            outs.append(out)
        return outs

    org = lockstep.make_gpu(wl)
    org.kf_prefill_score_prune(0, q, k, v)
    with pytest.raises(kf.KeyformerError) as e:
        org.kf_view_place(0)
    assert e.value.code == kf.KF_EINVAL
    new = lockstep.make_gpu(wl, pos_mode=kf.KF_POS_NEW)
    new.kf_prefill_score_prune(0, q, k, v)
    o_org, o_new = run(org, 1, 6), run(new, 1, 6)
    assert not torch.equal(o_org[0], o_new[0])          # 172 prompt tokens are gone: distances shrink
    img = torch.empty(new.kf_state_bytes(), dtype=torch.uint8, device=DEV)
    n_prompt, last_step = new.kf_export_state(0, img)
    rest = run(new, 7, 12)
    again = lockstep.make_gpu(wl, pos_mode=kf.KF_POS_NEW)
    again.kf_import_state(0, img, n_prompt, last_step)     # the places are rebuilt from the positions
    for x, y in zip(run(again, 7, 12), rest):
        assert torch.equal(x, y)
    torch.cuda.synchronize()
    assert torch.equal(again.kf_view_place(0), new.kf_view_place(0))
    pos = new.kf_view_state(0)[2]
    assert torch.equal(new.kf_view_place(0).long(), pos.argsort(-1).argsort(-1))
    for g in (org, new, again):
        lockstep.check_guards(g)


@pytest.mark.parametrize("d,k,order", [(128, 700, "random"), (64, 300, "reverse"), (256, 200, "random"), (128, 700, "rotate"),
                                       (128, 2048, "arrivals"), (256, 333, "arrivals"), (64, 1000, "many arrivals"),
                                       (128, 4096, "arrivals"), (64, 5000, "arrivals")])
def test_compaction_of_arbitrary_slot_orders(d, k, order):
    """kf_compact_layer has two ways through: entries that only move down plus a few that move up (what generation
    steps leave: `rotate`, `arrivals`) are carried over in ascending chunks; anything else (`random`, `reverse`, more
    arrivals than the kernel sets aside) is applied cycle by cycle.  The slots of a freshly filled cache are put
    into the given order here, through the library's own view of its state, and the call must sort them back."""
    wl = W.Workload("compact_orders", 1, 2, 3, d, k + 60, k, k // 4, 4, data_seed=k + d, noise_seed=3)
    gpu = lockstep.make_gpu(wl)
    gpu.kf_prefill_score_prune(0, *W.make_prompt(wl, 0, DEV))
    torch.cuda.synchronize()
    K, V, pos, acc, ln = gpu.kf_view_state(0)
    gen = torch.Generator(device="cpu").manual_seed(k)
    U = wl.batch * wl.n_heads
    if order in ("arrivals", "many arrivals"):
        # entries in scattered slots become tokens that arrived later: larger positions than everything else, in any order
        m = 40 if order == "arrivals" else 150
        for u in range(U):
            b, h = divmod(u, wl.n_heads)
            sel = torch.randperm(k, generator=gen)[:m].to(DEV)
            pos[b, h, sel] = (int(pos[b, h].max()) + 1 + torch.randperm(m, generator=gen)).to(device=DEV, dtype=torch.int32)
    else:
        if order == "random":
            perm = torch.stack([torch.randperm(k, generator=gen) for _ in range(U)])
        elif order == "reverse":
            perm = torch.arange(k - 1, -1, -1).expand(U, k)
        else:
            perm = torch.arange(k).roll(-1).expand(U, k)                 # the first entry sits in the last slot
        perm = perm.reshape(wl.batch, wl.n_heads, k).to(DEV)
        rows = perm[..., None].expand(-1, -1, -1, d)
        K.copy_(K.gather(2, rows)); V.copy_(V.gather(2, rows)); pos.copy_(pos.gather(-1, perm)); acc.copy_(acc.gather(-1, perm))
    torch.cuda.synchronize()
    before = [t.clone() for t in (K, V, pos, acc, ln)]
    gpu.kf_compact_layer(0)
    assert gpu.kf_poll_error() == 0
    srt = before[2].argsort(-1)
    rows = srt[..., None].expand(-1, -1, -1, d)
    assert torch.equal(pos, before[2].gather(-1, srt)) and torch.equal(acc, before[3].gather(-1, srt))
    assert torch.equal(K, before[0].gather(2, rows)) and torch.equal(V, before[1].gather(2, rows))
    assert torch.equal(ln, before[4])
    lockstep.check_guards(gpu)
    gpu.kf_destroy()


@pytest.mark.parametrize("d,pos_mode", [(64, 0), (128, 1), (256, 0)])
def test_compaction_restores_position_order_in_place(d, pos_mode):
    """After enough steps the slots of a unit are a permutation of the position order.  kf_compact_layer must apply
    exactly the sorting permutation to K, V, positions and scores (compared with a gather done here by library
    ops), leave a layer it is not asked about alone, and the generation that follows must still match the oracle."""
    wl = W.get_config("c3_mpt").scaled(n_layers=2, n_heads=3, batch=2, head_dim=d, prompt_len=200, budget_k=77,
                                       recent_w=20, gen_len_T=40)
    gpu = lockstep.make_gpu(wl, pos_mode=pos_mode)
    with pytest.raises(kf.KeyformerError) as e:
        gpu.kf_compact_layer(0)
    assert e.value.code == kf.KF_ESTATE
    drivers = [lockstep.LockStep(wl, gpu, l, W.unit_list(wl, l), pos_mode=pos_mode) for l in range(2)]
    for ls in drivers:
        ls.prefill(*W.make_prompt(wl, ls.layer, DEV))
    for s in range(1, 26):
        for ls in drivers:
            ls.decode_step(s, *W.make_step(wl, ls.layer, s, DEV), check_state=(s == 25))
    before = [[t.clone() for t in gpu.kf_view_state(l)] for l in range(2)]
    assert not torch.equal(before[0][2], before[0][2].sort(-1).values)       # the slots are out of order by now
    gpu.kf_compact_layer(0)
    assert gpu.kf_poll_error() == 0
    K, V, pos, acc, ln = gpu.kf_view_state(0)
    order = before[0][2].argsort(-1)
    assert torch.equal(pos, before[0][2].gather(-1, order)) and torch.equal(acc, before[0][3].gather(-1, order))
    rows = order[..., None].expand(-1, -1, -1, d)
    assert torch.equal(K, before[0][0].gather(2, rows)) and torch.equal(V, before[0][1].gather(2, rows))
    assert torch.equal(ln, before[0][4])
    if pos_mode == 1:
        assert torch.equal(gpu.kf_view_place(0).long(), torch.arange(77, device=DEV).expand(2, 3, 77))
    # the oracle keeps its entries in position order, so after the compaction the GPU's slots line up with it one to one
    st = drivers[0].st
    for u in range(st.U):
        b, h = int(st.lbh[u, 1]), int(st.lbh[u, 2])
        L = int(st.len[u])
        assert int(ln[b, h]) == L and np.array_equal(pos[b, h, :L].cpu().numpy(), st.pos[u, :L])
        a_ref = st.acc[u, :L]
        assert (np.abs(acc[b, h, :L].cpu().numpy() - a_ref) <= lockstep.SCORE_RTOL * np.abs(a_ref) + 1e-6).all()
        assert np.array_equal(K[b, h, :L].cpu().numpy().view(np.uint16), st.K[u, :L])
        assert np.array_equal(V[b, h, :L].cpu().numpy().view(np.uint16), st.V[u, :L])
    for x, y in zip(gpu.kf_view_state(1), before[1]):
        assert torch.equal(x, y)
    gpu.kf_compact_layer(0)                                                   # already in order: nothing moves
    assert torch.equal(gpu.kf_view_state(0)[2], pos) and torch.equal(gpu.kf_view_state(0)[0], K)
    for s in range(26, 41):
        for ls in drivers:
            ls.decode_step(s, *W.make_step(wl, ls.layer, s, DEV))
    lockstep.check_guards(gpu)
    gpu.kf_destroy()


def test_heavy_hitter_multi_layer_scaled_down():
    wl = W.get_config("c4_cerebras").scaled(n_layers=3, batch=2, n_heads=4, prompt_len=400, budget_k=200, recent_w=50, gen_len_T=8)
    lockstep.run_workload(wl)


def test_config1_full():
    wl = W.get_config("c1_tiny")
    r = lockstep.run_workload(wl)
    print("c1", r)


def test_call_order_and_argument_errors():
    wl = _wl()
    gpu = lockstep.make_gpu(wl)
    q, kn, vn = W.make_step(wl, 0, 1, DEV)
    out = torch.empty_like(q)
    with pytest.raises(kf.KeyformerError) as e:
        gpu.kf_decode_step(0, 1, q, kn, vn, out)
    assert e.value.code == kf.KF_ESTATE
    Q, K, V = W.make_prompt(wl, 0, DEV)
    gpu.kf_prefill_score_prune(0, Q, K, V)
    with pytest.raises(kf.KeyformerError) as e:
        gpu.kf_decode_step(0, 2, q, kn, vn, out)
    assert e.value.code == kf.KF_ESTATE
    with pytest.raises(kf.KeyformerError) as e:
        gpu.kf_decode_step(5, 1, q, kn, vn, out)
    assert e.value.code == kf.KF_EINVAL
    gpu.kf_decode_step(0, 1, q, kn, vn, out)
    assert gpu.kf_poll_error() == 0
    assert gpu.kf_launch_count() == 6   # prompt phase: 2 scoring sweeps + select + gather; then the decode step's 2 kernels


def test_export_import_state_resumes_bit_exactly():
    wl = _wl(head_dim=128, n_layers=2, prompt_len=130, budget_k=64, recent_w=16, gen_len_T=10)
    a = lockstep.make_gpu(wl)
    for l in range(2):
        a.kf_prefill_score_prune(l, *W.make_prompt(wl, l, DEV))
    outs = {}

    def step(gpu, l, s):
        q, kn, vn = W.make_step(wl, l, s, DEV)
        out = torch.empty_like(q)
        gpu.kf_decode_step(l, s, q, kn, vn, out)
        return out

    for s in range(1, 4):
        for l in range(2):
            step(a, l, s)
    images = []
    for l in range(2):
        img = torch.empty(a.kf_state_bytes(), dtype=torch.uint8, device=DEV)
        images.append((img, a.kf_export_state(l, img)))
    assert images[0][1] == (130, 3)
    for s in range(4, 8):
        for l in range(2):
            outs[(l, s)] = step(a, l, s)
    b = lockstep.make_gpu(wl)            # a fresh context continues from the images
    with pytest.raises(kf.KeyformerError) as e:
        b.kf_export_state(0, images[0][0])
    assert e.value.code == kf.KF_ESTATE
    for l in range(2):
        img, (n_prompt, last_step) = images[l]
        b.kf_import_state(l, img, n_prompt, last_step)
    for s in range(4, 8):
        for l in range(2):
            assert torch.equal(step(b, l, s), outs[(l, s)])
    torch.cuda.synchronize()
    for l in range(2):
        for x, y in zip(a.kf_view_state(l), b.kf_view_state(l)):
            assert torch.equal(x, y)
    lockstep.check_guards(a)
    lockstep.check_guards(b)


def test_host_buffer_variant_matches_device_variant():
    wl = _wl(head_dim=128)
    a, b = lockstep.make_gpu(wl), lockstep.make_gpu(wl)
    Q, K, V = W.make_prompt(wl, 0, DEV)
    a.kf_prefill_score_prune(0, Q, K, V)
    b.kf_prefill_score_prune(0, Q, K, V)
    for s in range(1, 4):
        q, kn, vn = W.make_step(wl, 0, s, DEV)
        out_a = torch.empty_like(q)
        a.kf_decode_step(0, s, q, kn, vn, out_a)
        hq, hk, hv = (t.cpu().pin_memory() for t in (q, kn, vn))
        out_b = torch.empty_like(hq).pin_memory()
        b.kf_decode_step_host(0, s, hq, hk, hv, out_b, wait=True)
        torch.cuda.synchronize()
        assert torch.equal(out_a.cpu(), out_b)
    # several calls in flight (copies overlapping kernels), one wait at the end
    outs_a, outs_b, keep = [], [], []
    for s in range(4, 10):
        q, kn, vn = W.make_step(wl, 0, s, DEV)
        out_a = torch.empty_like(q)
        a.kf_decode_step(0, s, q, kn, vn, out_a)
        outs_a.append(out_a)
        hq, hk, hv = (t.cpu().pin_memory() for t in (q, kn, vn))
        keep.append((hq, hk, hv))            # host inputs must outlive the copies that read them
        outs_b.append(torch.empty_like(hq).pin_memory())
        b.kf_decode_step_host(0, s, hq, hk, hv, outs_b[-1], wait=(s == 9))
    torch.cuda.synchronize()
    for x, y in zip(outs_a, outs_b):
        assert torch.equal(x.cpu(), y)
    sa, sb = a.kf_view_state(0), b.kf_view_state(0)
    torch.cuda.synchronize()
    for name, x, y in zip("K V pos acc len".split(), sa, sb):
        if name == "acc":   # prompt scores are summed with floating-point atomics: order-dependent rounding
            assert torch.allclose(x, y, rtol=1e-5, atol=1e-6)
        else:
            assert torch.equal(x, y)


# ------------------------------------------------------------------ error paths (nothing here faults or hangs the GPU)
def test_a_wait_that_runs_out_is_reported_and_the_context_survives():
    """debug_fail_first_wait makes every warp of the streaming kernel treat its first wait for a cache tile as
    run out: the warp flags KF_ETIMEOUT, waits (with the full limit) for its copies in flight and leaves.  The
    error word is returned once and cleared; a fresh context on the same device then runs in lock step."""
    wl = _wl(head_dim=128, prompt_len=300, budget_k=200, recent_w=20, gen_len_T=4)
    gpu = lockstep.make_gpu(wl, debug_fail_first_wait=1)
    gpu.kf_prefill_score_prune(0, *W.make_prompt(wl, 0, DEV))
    assert gpu.kf_poll_error() == 0                                     # the prompt phase has no such switch
    q, kn, vn = W.make_step(wl, 0, 1, DEV)
    out = torch.empty_like(q)
    gpu.kf_decode_step(0, 1, q, kn, vn, out)
    assert gpu.kf_poll_error() == kf.KF_ETIMEOUT
    assert kf.kf_strerror(kf.KF_ETIMEOUT) == "a bounded device-side wait ran out"
    assert gpu.kf_poll_error() == 0                                     # read once, then cleared
    rc, bad = gpu.kf_check_canaries()
    assert rc == kf.KF_OK, bad                                          # the aborted step stayed inside its buffers
    gpu.kf_destroy()
    r = lockstep.run_workload(wl)                                       # the device and the library are fine
    assert r["steps"] == 4


@pytest.mark.parametrize("bad_len", [-1, 41, 1 << 20])
def test_a_damaged_entry_count_is_reported_and_the_unit_left_alone(bad_len):
    wl = _wl(prompt_len=100, budget_k=40, recent_w=10)
    gpu = lockstep.make_gpu(wl)
    gpu.kf_prefill_score_prune(0, *W.make_prompt(wl, 0, DEV))
    K, V, pos, acc, ln = gpu.kf_view_state(0)
    torch.cuda.synchronize()
    ln[1, 2] = bad_len                                                  # what a foreign state image could contain
    before = [t.clone() for t in (K, V, pos, acc, ln)]
    q, kn, vn = W.make_step(wl, 0, 1, DEV)
    out = torch.zeros_like(q)
    gpu.kf_decode_step(0, 1, q, kn, vn, out)
    assert gpu.kf_poll_error() == kf.KF_EBOUNDS
    assert kf.kf_strerror(kf.KF_EBOUNDS) == "a device-side bounds check failed"
    after = gpu.kf_view_state(0)
    for x, y in zip(before, after):
        assert torch.equal(x[1, 2], y[1, 2])                            # nothing of the damaged unit was written
    assert (out[1, 2] == 0).all()
    assert (after[4].flatten()[:5] == 40).all() and not torch.equal(before[2][0, 0], after[2][0, 0])   # the others stepped
    lockstep.check_guards(gpu)
    gpu.kf_destroy()


def test_guard_blocks_detect_a_write_past_a_sub_buffer():
    wl = _wl()
    gpu = lockstep.make_gpu(wl)
    assert gpu.kf_check_canaries() == (kf.KF_OK, -1)
    K = gpu.kf_view_state(0)[0]
    off = K.data_ptr() - gpu.workspace.data_ptr() + K.numel() * 2      # first byte behind the K cache (a guard)
    gpu.workspace[off + 7] = 0                                          # a write one row too far would land here
    assert gpu.kf_check_canaries() == (kf.KF_EBOUNDS, 0)
    plain = lockstep.make_gpu(wl, debug_canaries=0)
    assert plain.kf_check_canaries()[0] == kf.KF_EINVAL
    assert gpu.workspace_bytes > plain.workspace_bytes


def test_misaligned_pointers_are_rejected_on_the_host():
    wl = _wl(head_dim=64)
    gpu = lockstep.make_gpu(wl)
    n, d = wl.prompt_len, wl.head_dim
    numel = wl.batch * wl.n_heads * n * d
    big = torch.zeros(numel + 8, dtype=torch.float16, device=DEV)
    Q, K, V = W.make_prompt(wl, 0, DEV)
    odd = big[1:1 + numel].view(Q.shape)                                # contiguous, but 2 bytes off a 16-byte boundary
    launches = gpu.kf_launch_count()
    for args in ((odd, K, V), (Q, odd, V), (Q, K, odd)):
        with pytest.raises(kf.KeyformerError) as e:
            gpu.kf_prefill_score_prune(0, *args)
        assert e.value.code == kf.KF_EINVAL
    gpu.kf_prefill_score_prune(0, Q, K, V)
    q, kn, vn = W.make_step(wl, 0, 1, DEV)
    out = torch.empty_like(q)
    small = big[1:1 + q.numel()].view(q.shape)
    for args in ((small, kn, vn, out), (q, small, vn, out), (q, kn, small, out), (q, kn, vn, small)):
        with pytest.raises(kf.KeyformerError) as e:
            gpu.kf_decode_step(0, 1, *args)
        assert e.value.code == kf.KF_EINVAL
    assert gpu.kf_launch_count() == launches + 4                        # only the accepted prompt call launched
    gpu.kf_decode_step(0, 1, q, kn, vn, out)
    lockstep.check_guards(gpu)


# ------------------------------------------------------------------ query heads sharing a key/value head (section 6)
@pytest.mark.parametrize("impl", [kf.KF_PREFILL_TENSOR, kf.KF_PREFILL_SIMT])
@pytest.mark.parametrize("d,g", [(64, 2), (128, 4), (256, 8), (128, 8), (64, 4)])
def test_shared_key_value_heads(d, g, impl):
    """One cache and one accumulated score per key/value head; every query head of the group has its own logits,
    noise and softmax; the accumulated score receives the group's mean.  Prompt phase plus generation, in lock
    step with the oracle (several splits, a ragged last tile)."""
    wl = _wl(head_dim=d, n_heads=3 * g, n_kv_heads=3, prompt_len=211, budget_k=150, recent_w=20, gen_len_T=10)
    r = lockstep.run_workload(wl, gpu_kwargs=dict(prefill_impl=impl))
    assert r["steps"] == 10 and r["units"] == 2 * 3


@pytest.mark.parametrize("pos_mode", [0, 1])
def test_shared_key_value_heads_with_alibi_slopes_per_query_head(pos_mode):
    wl = W.get_config("c3_mpt").scaled(n_heads=8, n_kv_heads=2, batch=2, prompt_len=300, budget_k=128, recent_w=32, gen_len_T=12)
    lockstep.run_workload(wl, pos_mode=pos_mode)


@pytest.mark.parametrize("noise", ["none", "const", "gauss"])
def test_shared_key_value_heads_other_adjustments(noise):
    lockstep.run_workload(_wl(head_dim=128, n_heads=4, n_kv_heads=1, prompt_len=140, budget_k=60, recent_w=12), noise=noise)


def test_multi_query_attention_filling_cache_and_window_edge_cases():
    """All query heads on one cache (MQA); a prompt shorter than the budget (the cache fills during generation),
    then no recent window, then window = budget."""
    for n, k, w in ((30, 48, 8), (90, 33, 0), (90, 32, 32)):
        lockstep.run_workload(_wl(head_dim=64, n_heads=8, n_kv_heads=1, prompt_len=n, budget_k=k, recent_w=w, gen_len_T=24))


def test_shared_key_value_heads_many_splits_and_host_buffers():
    wl = _wl(batch=1, head_dim=128, n_heads=8, n_kv_heads=2, prompt_len=2300, budget_k=2100, recent_w=100, gen_len_T=3)
    lockstep.run_workload(wl, gpu_kwargs=dict(decode_splits=17))
    a, b = lockstep.make_gpu(wl), lockstep.make_gpu(wl)
    Q, K, V = W.make_prompt(wl, 0, DEV)
    a.kf_prefill_score_prune(0, Q, K, V)
    b.kf_prefill_score_prune(0, Q, K, V)
    for s in range(1, 4):
        q, kn, vn = W.make_step(wl, 0, s, DEV)
        out_a = torch.empty_like(q)
        a.kf_decode_step(0, s, q, kn, vn, out_a)
        hq, hk, hv = (t.cpu().pin_memory() for t in (q, kn, vn))
        out_b = torch.empty_like(hq).pin_memory()
        b.kf_decode_step_host(0, s, hq, hk, hv, out_b, wait=True)
        torch.cuda.synchronize()
        assert torch.equal(out_a.cpu(), out_b)
    lockstep.check_guards(a)
    lockstep.check_guards(b)


# ------------------------------------------------------------------ tensor-core streaming kernel of the generation step
@pytest.mark.parametrize("g", [1, 2, 4, 8])
def test_tensor_core_generation_kernel_in_lock_step(g):
    """tcgen05 logits and value sums (head_dim 128): several splits, a ragged last tile, items of several tiles."""
    wl = _wl(head_dim=128, n_heads=2 * g, n_kv_heads=2, prompt_len=900, budget_k=700, recent_w=60, gen_len_T=8)
    for splits in (0, 1, 2):
        gpu_kwargs = dict(decode_impl=kf.KF_DECODE_TENSOR, decode_splits=splits)
        r = lockstep.run_workload(wl, gpu_kwargs=gpu_kwargs)
        assert r["steps"] == 8
    gpu = lockstep.make_gpu(wl, decode_impl=kf.KF_DECODE_TENSOR)
    assert gpu.kf_describe_decode().startswith(f"decode_tc_kernel<128,{g}>")
    assert lockstep.make_gpu(wl, decode_impl=kf.KF_DECODE_CUDA_CORES).kf_describe_decode().startswith("decode_kernel<128")


@pytest.mark.parametrize("pos_mode,noise", [(0, "gumbel"), (1, "gumbel"), (0, "none"), (0, "gauss")])
def test_tensor_core_generation_kernel_alibi_positions_and_adjustments(pos_mode, noise):
    wl = W.get_config("c3_mpt").scaled(n_heads=8, n_kv_heads=2, batch=2, prompt_len=500, budget_k=300, recent_w=64, gen_len_T=10)
    lockstep.run_workload(wl, pos_mode=pos_mode, noise=noise, gpu_kwargs=dict(decode_impl=kf.KF_DECODE_TENSOR))


@pytest.mark.parametrize("scale", [1.0, 3.0])
def test_tensor_core_generation_kernel_moves_its_reference_exponent(scale):
    """Logits tens of units apart: a later tile of an item exceeds the first tile's maximum by far more than 2^8, so
    the output accumulator is rescaled in tensor memory (one item of six tiles per cache)."""
    wl = _wl(head_dim=128, n_heads=4, n_kv_heads=1, batch=3, prompt_len=800, budget_k=700, recent_w=50, gen_len_T=6)
    lockstep.run_workload(wl, logit_scale=scale, gpu_kwargs=dict(decode_impl=kf.KF_DECODE_TENSOR, decode_splits=1))


def test_tensor_core_generation_kernel_ignores_what_lies_beyond_the_entry_count():
    """A cache that is still filling: the slots past the entry count hold NaN patterns (as uninitialised memory
    may); they must not leak into the output through a zero weight."""
    wl = _wl(head_dim=128, n_heads=4, n_kv_heads=2, prompt_len=70, budget_k=200, recent_w=16, gen_len_T=20)
    gpu = lockstep.make_gpu(wl, decode_impl=kf.KF_DECODE_TENSOR)
    K, V = gpu.kf_view_state(0)[:2]
    K.fill_(float("nan"))
    V.fill_(float("nan"))
    ls = lockstep.LockStep(wl, gpu, 0, W.unit_list(wl, 0))
    ls.prefill(*W.make_prompt(wl, 0, DEV))
    for s in range(1, 21):
        ls.decode_step(s, *W.make_step(wl, 0, s, DEV))
    lockstep.check_guards(gpu)
    gpu.kf_destroy()


def test_tensor_core_and_cuda_core_generation_kernels_agree():
    wl = _wl(head_dim=128, n_heads=8, n_kv_heads=2, prompt_len=600, budget_k=400, recent_w=40, gen_len_T=5)
    Q, K, V = W.make_prompt(wl, 0, DEV)
    outs = []
    for impl in (kf.KF_DECODE_TENSOR, kf.KF_DECODE_CUDA_CORES):
        gpu = lockstep.make_gpu(wl, decode_impl=impl)
        gpu.kf_prefill_score_prune(0, Q, K, V)
        res = []
        for s in range(1, 6):
            q, kn, vn = W.make_step(wl, 0, s, DEV)
            out = torch.empty_like(q)
            sc = torch.zeros(wl.batch, wl.kv_heads, wl.budget_k + 1, device=DEV)
            gpu.kf_decode_step(0, s, q, kn, vn, out, score_out=sc)
            res.append((out, sc))
        torch.cuda.synchronize()
        res.append(tuple(t.clone() for t in gpu.kf_view_state(0)[2:]))
        lockstep.check_guards(gpu)
        outs.append(res)
    for (oa, sa), (ob, sb) in zip(outs[0][:5], outs[1][:5]):
        scale = ob.float().abs().amax(dim=-1, keepdim=True)
        assert ((oa.float() - ob.float()).abs() <= 2e-3 * scale).all()
        assert torch.allclose(sa, sb, rtol=1e-3, atol=1e-7)
    assert torch.equal(outs[0][5][0], outs[1][5][0])        # the same entries were kept


# ------------------------------------------------------------------ rotary embedding applied by the library (section 4.4.2 on rotary models)
def _rot_wl(**kw):
    base = dict(head_dim=128, n_heads=3, prompt_len=300, budget_k=150, recent_w=30, gen_len_T=16, positional="rotary", rotary_dims=64,
                rotary_in_library=True)
    base.update(kw)
    return _wl(**base)


@pytest.mark.parametrize("impl", [kf.KF_PREFILL_TENSOR, kf.KF_PREFILL_SIMT])
@pytest.mark.parametrize("d,R", [(64, 64), (128, 32), (256, 64), (128, 128)])
@pytest.mark.parametrize("pos_mode", [0, 1])
def test_rotary_embedding_applied_at_logit_time(pos_mode, d, R, impl):
    """Q and K come unrotated, the cache keeps keys unrotated; the prompt phase rotates at the tokens' positions, the
    generation phase at original positions (Org Pos) or at places in the reduced cache (New Pos).  Lock step with the
    oracle, which rotates in double precision; several splits and evictions."""
    wl = _rot_wl(head_dim=d, rotary_dims=R)
    r = lockstep.run_workload(wl, pos_mode=pos_mode, gpu_kwargs=dict(prefill_impl=impl))
    assert r["steps"] == 16


def test_rotary_embedding_with_shared_key_value_heads_and_alibi_free_long_positions():
    wl = _rot_wl(n_heads=8, n_kv_heads=2, prompt_len=1500, budget_k=400, recent_w=64, gen_len_T=6, rotary_dims=32)
    for pos_mode in (0, 1):
        lockstep.run_workload(wl, pos_mode=pos_mode)


def test_library_rotation_agrees_with_rotated_inputs_and_keeps_the_cache_unrotated():
    """Org Pos with the embedding applied by the library is the ordinary rotary model: feeding tensors rotated by the
    generator (and rounded to fp16) gives the same outputs within that rounding; the cache rows differ (rotated vs not)."""
    plain = _rot_wl(rotary_in_library=False, gen_len_T=5)
    inlib = _rot_wl(gen_len_T=5)
    a, b = lockstep.make_gpu(plain), lockstep.make_gpu(inlib)
    assert "rot" in b.kf_describe_decode() and "rot" not in a.kf_describe_decode()
    a.kf_prefill_score_prune(0, *W.make_prompt(plain, 0, DEV))
    Qu, Ku, Vu = W.make_prompt(inlib, 0, DEV)
    b.kf_prefill_score_prune(0, Qu, Ku, Vu)
    for s in range(1, 6):
        qa, ka, va = W.make_step(plain, 0, s, DEV)
        qb, kb, vb = W.make_step(inlib, 0, s, DEV)
        oa, ob = torch.empty_like(qa), torch.empty_like(qb)
        a.kf_decode_step(0, s, qa, ka, va, oa)
        b.kf_decode_step(0, s, qb, kb, vb, ob)
        torch.cuda.synchronize()
        scale = oa.float().abs().amax(dim=-1, keepdim=True)
        assert ((oa.float() - ob.float()).abs() <= 1e-2 * scale).all()
    Kb, _, posb, _, _ = b.kf_view_state(0)
    torch.cuda.synchronize()
    rows = Ku.gather(2, posb.clamp(max=inlib.prompt_len - 1).long()[..., None].expand(-1, -1, -1, inlib.head_dim))
    from_prompt = posb < inlib.prompt_len
    assert torch.equal(Kb[from_prompt], rows[from_prompt])            # the caller's unrotated rows, bit for bit
    with pytest.raises(kf.KeyformerError) as e:                        # the table of angles ends at n_max + T - 1
        for s in range(6, 40):
            qb, kb, vb = W.make_step(inlib, 0, s, DEV)
            b.kf_decode_step(0, s, qb, kb, vb, ob)
    assert e.value.code == kf.KF_EINVAL
    lockstep.check_guards(a)
    lockstep.check_guards(b)
