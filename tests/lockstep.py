"""Lock-step parity driver: the CUDA library and the CPU oracle walk the same seeded
workload step by step; after every call the results are compared and, where the GPU's
eviction choice differs only inside the tolerance band, the oracle adopts it so that
later steps stay comparable.

Comparison rules
  out     |gpu - ref| <= 2e-3 * max|ref|           per (batch row, head) vector
  scores  |gpu - ref| <= 2e-3 * |ref| + 1e-7       per entry
  kept    size and recent window exact; with r = k - #recent and theta_in / theta_out the
          r-th / (r+1)-th largest candidate score of the oracle, a candidate above
          theta_out * (1 + 1e-3) must be kept, one below theta_in * (1 - 1e-3) must be
          dropped, the others are free.
"""
from __future__ import annotations

import numpy as np
import torch

import paper_2403_09054_b200 as kf
import workloads as W
from oracle import keyformer_oracle as ko

OUT_RTOL = 2e-3
SCORE_RTOL = 2e-3
SCORE_ATOL = 1e-7
BAND = 1e-3


def oracle_params(wl: W.Workload, noise_mode=ko.NOISE_GUMBEL, logit_scale=0.0, pos_mode=0) -> ko.Params:
    return ko.Params(head_dim=wl.head_dim, n_heads=wl.n_heads, budget_k=wl.budget_k, recent_w=wl.recent_w,
                     gen_len_T=wl.gen_len_T, tau_init=wl.tau_init, tau_end=wl.tau_end,
                     noise_seed=wl.noise_seed, noise_mode=noise_mode, logit_scale=logit_scale, pos_mode=pos_mode,
                     n_kv_heads=wl.n_kv_heads, rotary_dims=wl.rotary_dims if wl.rotary_in_library else 0,
                     bias_mode=1 if wl.positional == "alibi" else 0,
                     alibi_slopes=W.alibi_slopes(wl.n_heads) if wl.positional == "alibi" else None)


def make_gpu(wl: W.Workload, noise_mode=kf.KF_NOISE_GUMBEL, max_prompt_len=None, **kw) -> kf.Keyformer:
    """A context for `wl`.  Unless told otherwise the workspace carries guard blocks between its sub-buffers
    (see check_guards): the kernels and their launch shapes are the same with and without them."""
    kw.setdefault("debug_canaries", 1)
    return kf.Keyformer(n_layers=wl.n_layers, batch=wl.batch, n_heads=wl.n_heads, head_dim=wl.head_dim,
                        n_kv_heads=wl.n_kv_heads, rotary_dims=wl.rotary_dims if wl.rotary_in_library else 0, budget_k=wl.budget_k, recent_w=wl.recent_w,
                        max_prompt_len=max_prompt_len or wl.prompt_len, gen_len_T=wl.gen_len_T,
                        tau_init=wl.tau_init, tau_end=wl.tau_end, noise_seed=wl.noise_seed,
                        noise_mode=noise_mode,
                        bias_mode=kf.KF_BIAS_ALIBI if wl.positional == "alibi" else kf.KF_BIAS_NONE,
                        alibi_slopes=W.alibi_slopes(wl.n_heads) if wl.positional == "alibi" else None, **kw)


def check_guards(gpu: kf.Keyformer):
    """No kernel wrote past the end of a workspace sub-buffer (and no bounded wait ran out)."""
    assert gpu.kf_poll_error() == 0
    rc, bad = gpu.kf_check_canaries()
    assert rc == kf.KF_OK, f"guard behind workspace sub-buffer {bad} was overwritten ({kf.kf_strerror(rc)})"


def check_band(acc_ref, cand_mask, kept_mask, n_keep, what):
    """Band rule on one unit.  acc_ref: oracle scores of the entries; cand_mask: which are
    candidates (outside the recent window); kept_mask: the GPU's decision; n_keep: r."""
    cand = np.flatnonzero(cand_mask)
    assert kept_mask[~cand_mask].all(), f"{what}: a recent-window entry was dropped"
    assert int(kept_mask[cand].sum()) == n_keep, f"{what}: kept {int(kept_mask[cand].sum())} candidates, expected {n_keep}"
    if n_keep == 0 or n_keep == cand.size:
        return
    srt = np.sort(acc_ref[cand])[::-1]
    theta_in, theta_out = srt[n_keep - 1], srt[n_keep]
    must_keep = cand[acc_ref[cand] > theta_out * (1 + BAND)]
    must_drop = cand[acc_ref[cand] < theta_in * (1 - BAND)]
    assert kept_mask[must_keep].all(), f"{what}: dropped an entry whose score is clearly above the threshold"
    assert not kept_mask[must_drop].any(), f"{what}: kept an entry whose score is clearly below the threshold"


class LockStep:
    """One layer of a workload on the GPU next to the oracle on a sample of its units."""

    def __init__(self, wl: W.Workload, gpu: kf.Keyformer, layer: int, units: np.ndarray,
                 noise_mode=ko.NOISE_GUMBEL, logit_scale=0.0, pos_mode=0):
        self.wl, self.gpu, self.layer = wl, gpu, layer
        self.pos_mode = pos_mode
        self.units = np.ascontiguousarray(units, dtype=np.int32).reshape(-1, 3)
        assert (self.units[:, 0] == layer).all()
        self.flat = torch.as_tensor(self.units[:, 1] * wl.kv_heads + self.units[:, 2], dtype=torch.long)
        self.P = oracle_params(wl, noise_mode, logit_scale, pos_mode)
        self.st = ko.State(self.P, self.units)
        self.adoptions = 0
        self.n = None
        self.max_out_err = 0.0
        self.max_score_err = 0.0

    # ------------------------------------------------------------------ helpers
    def _rows(self, t: torch.Tensor) -> np.ndarray:
        """[B, Hkv, ...] device tensor (one entry per cache) -> numpy rows of the sampled units."""
        flat = t.reshape(self.wl.batch * self.wl.kv_heads, *t.shape[2:])
        return flat[self.flat.to(t.device)].cpu().numpy()

    def _qrows(self, t: torch.Tensor) -> np.ndarray:
        """[B, H, ...] device tensor (one entry per query head) -> numpy [U, ...] of the sampled units, or
        [U, g, ...] when g query heads share a cache (the heads of a group are consecutive)."""
        g = self.wl.group
        flat = t.reshape(self.wl.batch * self.wl.kv_heads, g, *t.shape[2:])[self.flat.to(t.device)].cpu().numpy()
        return flat[:, 0] if g == 1 else flat

    def gpu_state(self, rows=True):
        K, V, pos, acc, ln = self.gpu.kf_view_state(self.layer)
        torch.cuda.synchronize()
        if not rows:
            return None, None, self._rows(pos), self._rows(acc), self._rows(ln)
        return self._rows(K), self._rows(V), self._rows(pos), self._rows(acc), self._rows(ln)

    # ------------------------------------------------------------------ prompt phase
    def prefill(self, q, k, v):
        wl, gpu = self.wl, self.gpu
        n = q.shape[-2]
        self.n = n
        score = torch.empty(wl.batch, wl.kv_heads, n, dtype=torch.float32, device=q.device)
        gpu.kf_prefill_score_prune(self.layer, q, k, v, score_out=score)
        assert gpu.kf_poll_error() == 0
        # every unit of the layer, sampled by the oracle or not: each of the n softmax rows adds 1 to the scores,
        # the kept positions ascend and end with the w most recent ones
        kk_, w_ = wl.budget_k, wl.recent_w
        tot = score.double().sum(-1)
        assert ((tot - n).abs() <= 1e-4 * n).all(), "prompt scores do not add up to the number of query rows"
        _, _, pos_all, _, len_all = gpu.kf_view_state(self.layer)
        L_all = min(n, kk_)
        assert (len_all == L_all).all()
        assert (pos_all[..., 1:L_all] > pos_all[..., :L_all - 1]).all() and (pos_all[..., :L_all] >= 0).all()
        n_rec = min(w_, L_all)
        if n_rec > 0:
            assert torch.equal(pos_all[..., L_all - n_rec:L_all].long(),
                               torch.arange(n - n_rec, n, device=pos_all.device).expand(wl.batch, wl.kv_heads, n_rec))
        Qs, Ks, Vs = self._qrows(q), self._rows(k), self._rows(v)
        acc_ref = self.st.prefill_score(Qs, Ks)
        acc_gpu = self._rows(score).astype(np.float64)
        err = np.abs(acc_gpu - acc_ref) - SCORE_RTOL * np.abs(acc_ref)
        self.max_score_err = max(self.max_score_err, float((np.abs(acc_gpu - acc_ref) / np.maximum(acc_ref, 1e-30)).max()))
        assert err.max() <= 1e-6, f"prefill scores off by {err.max():.3e} beyond tolerance"
        Kc, Vc, pos, acc, ln = self.gpu_state()
        kk, w = wl.budget_k, wl.recent_w
        keep_gpu = np.zeros((len(self.units), n), dtype=np.uint8)
        for u in range(len(self.units)):
            L = int(ln[u])
            assert L == min(n, kk)
            p_u = pos[u, :L]
            assert (np.diff(p_u) > 0).all() and p_u.min() >= 0 and p_u.max() < n, "kept positions not ascending / in range"
            assert (pos[u, L:] == -1).all()
            keep_gpu[u, p_u] = 1
            if n > kk:
                cand_mask = np.arange(n) < n - w
                check_band(acc_ref[u], cand_mask, keep_gpu[u].astype(bool), kk - w, f"prefill unit {self.units[u]}")
            # rows and scores stored with the kept positions
            assert (Kc[u, :L].view(np.uint16) == Ks[u][p_u].view(np.uint16)).all()
            assert (Vc[u, :L].view(np.uint16) == Vs[u][p_u].view(np.uint16)).all()
            assert (acc[u, :L] == self._rows(score)[u][p_u]).all()
        ref_keep = np.stack([ko.select(np.arange(n), acc_ref[u], kk, w, n - 1) for u in range(len(self.units))])
        self.adoptions += int((ref_keep != keep_gpu.astype(bool)).any(axis=1).sum())
        self.st.prefill_prune(Ks, Vs, acc_ref, keep_override=keep_gpu)
        return acc_ref

    # ------------------------------------------------------------------ generation phase
    def decode_step(self, step, q, knew, vnew, check_state=True):
        """GPU step + oracle step with adoption of the GPU's (band-checked) eviction."""
        wl = self.wl
        U = len(self.units)
        _, _, pos_before, _, len_before = self.gpu_state(rows=False)
        out = torch.empty(wl.batch, wl.n_heads, wl.head_dim, dtype=torch.float16, device=q.device)
        score = torch.zeros(wl.batch, wl.kv_heads, wl.budget_k + 1, dtype=torch.float32, device=q.device)
        len_all_before = self.gpu.kf_view_state(self.layer)[4].clone()
        self.gpu.kf_decode_step(self.layer, step, q, knew, vnew, out, score_out=score)
        assert self.gpu.kf_poll_error() == 0
        self._check_all_units(step, out, score, len_all_before)
        return self._compare_decode(step, q, knew, vnew, out, score, pos_before, len_before, check_state)

    def _check_all_units(self, step, out, score, len_before):
        """Properties that hold for every unit of the layer, sampled by the oracle or not (computed on the GPU
        with library ops): Eq. 11 is a softmax, one entry at most leaves, positions stay distinct, and the new
        token and the w most recent positions are always in the cache."""
        wl = self.wl
        kk, w = wl.budget_k, wl.recent_w
        p = self.n + step - 1
        _, _, pos, acc, ln = self.gpu.kf_view_state(self.layer)
        m = len_before.long() + 1                                            # entries scored this step
        col = torch.arange(kk + 1, device=score.device)
        zsum = torch.where(col < m[..., None], score, torch.zeros_like(score)).sum(-1)
        assert torch.isfinite(out.float()).all() and (zsum - 1).abs().max().item() < 1e-4, f"step {step}: scores do not sum to 1"
        assert torch.equal(ln.long(), torch.clamp(m, max=kk)), f"step {step}: entry counts"
        valid = torch.arange(kk, device=pos.device) < ln[..., None]
        ps = torch.where(valid, pos, torch.full_like(pos, -1)).long()
        srt = ps.sort(-1).values
        dup = (srt[..., 1:] == srt[..., :-1]) & (srt[..., 1:] >= 0)
        assert not dup.any(), f"step {step}: a position is cached twice"
        assert (ps.max(-1).values == p).all() or w == 0, f"step {step}: the new token is missing"
        recent = ((ps > p - w) & valid).sum(-1)
        assert torch.equal(recent, torch.clamp(ln.long(), max=min(w, p + 1))), f"step {step}: recent window incomplete"
        assert (acc[valid] >= 0).all()

    def _compare_decode(self, step, q, knew, vnew, out, score, pos_before, len_before, check_state):
        wl = self.wl
        kk, w = wl.budget_k, wl.recent_w
        U = len(self.units)
        out_ref, z_ref = self.st.decode_score(step, self._qrows(q), self._rows(knew), self._rows(vnew))
        out_gpu = self._qrows(out).astype(np.float64)
        z_gpu = self._rows(score).astype(np.float64)
        Kc, Vc, pos_after, acc_after, len_after = self.gpu_state(rows=check_state)
        p = self.n + step - 1
        forced = np.full(U, -1, dtype=np.int32)
        own = np.full(U, -1, dtype=np.int32)
        for u in range(U):
            tag = f"step {step} unit {self.units[u]}"
            scale = np.abs(out_ref[u]).max(axis=-1)               # per query head of the unit
            oerr = np.abs(out_gpu[u] - out_ref[u]).max(axis=-1)
            self.max_out_err = max(self.max_out_err, float((oerr / scale).max()))
            assert (oerr <= OUT_RTOL * scale).all(), f"{tag}: attention output off by {oerr.max():.3e} (scale {scale.min():.3e})"
            L = int(len_before[u])
            m = L + 1
            assert int(self.st.len[u]) == m
            ref_pos = self.st.pos[u, :m]                       # the oracle keeps its entries in position order
            gpu_pos = np.concatenate([pos_before[u, :L], [p]])
            assert (np.diff(ref_pos) > 0).all()
            assert np.array_equal(ref_pos, np.sort(gpu_pos)), f"{tag}: cached positions differ"
            perm = np.searchsorted(ref_pos, gpu_pos)
            zr, zg = z_ref[u, perm], z_gpu[u, :m]
            serr = np.abs(zg - zr) - (SCORE_RTOL * np.abs(zr) + SCORE_ATOL)
            self.max_score_err = max(self.max_score_err, float((np.abs(zg - zr) / np.maximum(zr, 1e-6)).max()))
            assert serr.max() <= 0, f"{tag}: score off by {serr.max():.3e} beyond tolerance"
            La = int(len_after[u])
            assert La == min(m, kk), f"{tag}: cache length {La}"
            after = np.sort(pos_after[u, :La])
            assert (np.diff(after) > 0).all() and np.isin(after, ref_pos).all(), f"{tag}: duplicate or foreign positions"
            gone = np.setdiff1d(ref_pos, after)
            if m <= kk:
                assert gone.size == 0
            else:
                assert gone.size == 1, f"{tag}: {gone.size} entries left the cache"
                ev = int(gone[0])
                acc_r = self.st.acc[u, :m]
                cand_mask = ref_pos <= p - w
                check_band(acc_r, cand_mask, ref_pos != ev, kk - int((~cand_mask).sum()), tag)
                forced[u] = ev
                keep = ko.select(ref_pos, acc_r, kk, w, p)
                own[u] = int(ref_pos[~keep][0])
        self.adoptions += int((forced != own).sum())
        self.st.decode_evict(step, force_evict_pos=forced if (forced >= 0).any() else None)
        if check_state and self.pos_mode == 1:
            # the places the bias will use next step: rank of each entry's position within its unit
            place = self._rows(self.gpu.kf_view_place(self.layer))
            for u in range(U):
                La = int(len_after[u])
                assert (place[u, :La] == np.argsort(np.argsort(pos_after[u, :La]))).all(), f"step {step}: places out of order"
        if check_state:
            for u in range(U):
                La = int(len_after[u])
                ref_pos = self.st.pos[u, :La]
                assert np.array_equal(ref_pos, np.sort(pos_after[u, :La]))
                idx = np.searchsorted(ref_pos, pos_after[u, :La])
                a_ref = self.st.acc[u, idx]
                aerr = np.abs(acc_after[u, :La] - a_ref) - (SCORE_RTOL * np.abs(a_ref) + 1e-6)
                assert aerr.max() <= 0, f"step {step}: accumulated score off by {aerr.max():.3e}"
                assert (Kc[u, :La].view(np.uint16) == self.st.K[u, idx]).all(), "K rows differ"
                assert (Vc[u, :La].view(np.uint16) == self.st.V[u, idx]).all(), "V rows differ"
        return out_gpu, z_gpu


def run_workload(wl: W.Workload, units_per_layer=None, steps=None, layers=None, device="cuda:0",
                 sample_seed=0, check_state_every=1, gpu_kwargs=None, noise="gumbel", logit_scale=0.0, pos_mode=0):
    """Prefill + `steps` decode steps of `wl` on the GPU in lock step with the oracle.
    Returns a dict of summary numbers."""
    nm_gpu = {"gumbel": kf.KF_NOISE_GUMBEL, "none": kf.KF_NOISE_NONE, "const": kf.KF_NOISE_CONST, "gauss": kf.KF_NOISE_GAUSS}[noise]
    nm_ref = {"gumbel": ko.NOISE_GUMBEL, "none": ko.NOISE_NONE, "const": ko.NOISE_CONST, "gauss": ko.NOISE_GAUSS}[noise]
    gpu = make_gpu(wl, noise_mode=nm_gpu, logit_scale=logit_scale, pos_mode=pos_mode, **(gpu_kwargs or {}))
    layers = list(range(wl.n_layers)) if layers is None else layers
    steps = wl.gen_len_T if steps is None else steps
    drivers = []
    for l in layers:
        units = W.unit_list(wl, l) if units_per_layer is None else W.sample_units(wl, units_per_layer, sample_seed + l, l)
        ls = LockStep(wl, gpu, l, units, noise_mode=nm_ref, logit_scale=logit_scale, pos_mode=pos_mode)
        q, k, v = W.make_prompt(wl, l, device)
        ls.prefill(q, k, v)
        del q, k, v
        drivers.append(ls)
    for s in range(1, steps + 1):
        for ls in drivers:
            q, kn, vn = W.make_step(wl, ls.layer, s, device)
            ls.decode_step(s, q, kn, vn, check_state=(s % check_state_every == 0 or s == steps))
    res = dict(adoptions=sum(d.adoptions for d in drivers),
               max_out_err=max(d.max_out_err for d in drivers),
               max_score_err=max(d.max_score_err for d in drivers),
               units=sum(len(d.units) for d in drivers), steps=steps)
    check_guards(gpu)
    gpu.kf_destroy()
    return res
