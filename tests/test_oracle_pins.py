"""CPU pins of the oracle: every check compares it with something other than itself
(published vectors, closed forms, library routines, brute force, statistical laws)."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import keyformer_oracle as ko
import workloads as W

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _params(**kw):
    base = dict(head_dim=16, n_heads=2, budget_k=8, recent_w=2, gen_len_T=4)
    base.update(kw)
    return ko.Params(**base)


# ---------------------------------------------------------------- RNG / noise
def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLD, "philox4x32_10_kat.txt")) if not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        w = [int(x, 16) for x in r]
        assert ko.philox4x32_10(w[:4], w[4:6]).tolist() == w[6:]


def test_philox_against_python_bigint_restatement():
    # independent restatement with Python big integers (no uint overflow semantics involved)
    def ref(ctr, key):
        c, k = list(ctr), list(key)
        for _ in range(10):
            pa, pb = 0xD2511F53 * c[0], 0xCD9E8D57 * c[2]
            c = [(pb >> 32) ^ c[1] ^ k[0], pb & 0xFFFFFFFF, (pa >> 32) ^ c[3] ^ k[1], pa & 0xFFFFFFFF]
            k = [(k[0] + 0x9E3779B9) & 0xFFFFFFFF, (k[1] + 0xBB67AE85) & 0xFFFFFFFF]
        return c
    rng = np.random.default_rng(0)
    for _ in range(50):
        ctr = rng.integers(0, 2**32, 4, dtype=np.uint64).tolist()
        key = rng.integers(0, 2**32, 2, dtype=np.uint64).tolist()
        assert ko.philox4x32_10(ctr, key).tolist() == ref(ctr, key)


def test_half_decoding_matches_numpy():
    bits = np.arange(65536, dtype=np.uint16)
    ref = bits.view(np.float16).astype(np.float64)
    got = np.array([ko.half_to_double(int(b)) for b in bits[::7]])
    r = ref[::7]
    ok = (got == r) | (np.isnan(got) & np.isnan(r))
    assert ok.all()


def test_uniform_is_open_interval_and_exact_in_fp32():
    assert ko.uniform_from_word(0) == 2.0 ** -24
    assert ko.uniform_from_word(0xFFFFFFFF) == 1.0 - 2.0 ** -24
    for r in (0, 1, 511, 512, 0x80000000, 0xFFFFFFFF, 123456789):
        u = ko.uniform_from_word(r)
        assert 0.0 < u < 1.0 and float(np.float32(u)) == u


def _gumbel_samples(count, seed=7):
    P = _params(noise_seed=seed)
    # walk the (query i, key j) plane exactly as the method does
    side = int(math.isqrt(count))
    return np.array([ko.noise(P, 0, 1, 1, i, j) for i in range(side) for j in range(side)])


def test_gumbel_moments_match_paper_constants():
    gold = dict(l.split() for l in open(os.path.join(GOLD, "gumbel_constants.txt")) if not l.startswith("#"))
    z = _gumbel_samples(250_000)
    assert abs(z.mean() - float(gold["mean"])) < 0.01
    assert abs(z.std() - float(gold["std"])) < 0.01
    # closed forms: Euler-Mascheroni and pi/sqrt(6)
    assert abs(float(gold["mean"]) - 0.5772156649) < 1e-4
    assert abs(float(gold["std"]) - math.pi / math.sqrt(6)) < 1e-4
    # skewed to the right (a sign error in the transform would flip this)
    assert ((z - z.mean()) ** 3).mean() / z.std() ** 3 > 0.9


def test_gumbel_cdf_matches_eq7():
    # Eq. 7 pdf exp(-z - exp(-z)) integrates to the cdf exp(-exp(-z)): Kolmogorov distance
    z = np.sort(_gumbel_samples(90_000, seed=11))
    cdf = np.exp(-np.exp(-z))
    emp = (np.arange(z.size) + 0.5) / z.size
    assert np.abs(cdf - emp).max() < 0.008


def test_gumbel_max_law():
    # P[argmax_j (x_j + zeta_j) = i] = softmax(x)_i : pins "noise is added to the logits"
    x = np.array([0.0, 1.0, -0.5, 2.0, 0.3])
    target = np.exp(x) / np.exp(x).sum()
    P = _params(noise_seed=3)
    trials = 40_000
    wins = np.zeros(5)
    for i in range(trials):
        zeta = np.array([ko.noise(P, 0, 0, 0, i, j) for j in range(5)])
        wins[np.argmax(x + zeta)] += 1
    assert np.abs(wins / trials - target).max() < 0.01


def test_noise_keying_is_a_pure_function_and_distinguishes_coordinates():
    P = _params(noise_seed=5, n_heads=4)
    base = ko.noise(P, 1, 2, 3, 40, 17)
    assert base == ko.noise(P, 1, 2, 3, 40, 17)
    others = [ko.noise(P, 0, 2, 3, 40, 17), ko.noise(P, 1, 1, 3, 40, 17), ko.noise(P, 1, 2, 2, 40, 17),
              ko.noise(P, 1, 2, 3, 41, 17), ko.noise(P, 1, 2, 3, 40, 16), ko.noise(P, 1, 2, 3, 40, 18),
              ko.noise(_params(noise_seed=6, n_heads=4), 1, 2, 3, 40, 17)]
    assert len(set(others + [base])) == len(others) + 1
    # the four words of one Philox block serve key positions 4q .. 4q+3
    words = ko.philox4x32_10([17 >> 2, 40, 2 * 4 + 3, 1], [5, 0])
    assert base == ko.gumbel_from_word(int(words[17 & 3]))
    assert abs(ko.gumbel_from_word(0) - (-math.log(-math.log(2.0 ** -24)))) < 1e-12


def test_other_adjustments():
    assert ko.noise(_params(noise_mode=ko.NOISE_NONE), 0, 0, 0, 3, 2) == 0.0
    assert ko.noise(_params(noise_mode=ko.NOISE_CONST), 0, 0, 0, 3, 2) == 0.5772
    P = _params(noise_mode=ko.NOISE_GAUSS, noise_seed=9)
    g = np.array([ko.noise(P, 0, 0, 0, i, j) for i in range(300) for j in range(300)])
    assert abs(g.mean() - 0.5772) < 0.02 and abs(g.std() - 1.2825) < 0.02
    assert abs(((g - g.mean()) ** 3).mean()) < 0.05          # symmetric


# ---------------------------------------------------------------- temperature
def test_tau_schedule_closed_form():
    P = _params(gen_len_T=8, tau_init=1.0, tau_end=2.0)
    assert ko.tau(P, 0) == 1.0 and ko.tau(P, 8) == 2.0
    assert ko.tau(P, 2) == 1.25 and ko.tau(P, 4) == 1.5
    assert ko.tau(P, 9) == 2.0 and ko.tau(P, 1000) == 2.0          # clamped past T
    assert ko.tau(_params(gen_len_T=0, tau_init=1.5), 3) == 1.5
    P2 = _params(gen_len_T=5, tau_init=0.5, tau_end=3.0)
    for t in range(6):
        assert abs(ko.tau(P2, t) - (0.5 + t * 0.5)) < 1e-15


# ---------------------------------------------------------------- selection
def _brute_select(pos, acc, k, w, p):
    m = len(pos)
    if m <= k:
        return np.ones(m, bool)
    recent = [j for j in range(m) if pos[j] > p - w]
    rest = [j for j in range(m) if pos[j] <= p - w]
    rest.sort(key=lambda j: (-acc[j], pos[j]))
    keep = np.zeros(m, bool)
    keep[recent] = True
    keep[rest[: k - len(recent)]] = True
    return keep


@pytest.mark.parametrize("seed", range(6))
def test_selection_matches_brute_force_sort(seed):
    rng = np.random.default_rng(seed)
    for _ in range(40):
        m = int(rng.integers(1, 40))
        k = int(rng.integers(1, 40))
        w = int(rng.integers(0, k + 1))
        pos = np.sort(rng.choice(200, size=m, replace=False)).astype(np.int32)
        # recent window is contiguous below p, as in the method
        p = int(pos[-1])
        pos[-min(w, m):] = np.arange(p - min(w, m) + 1, p + 1) if w > 0 else pos[-min(w, m):]
        pos = np.unique(pos).astype(np.int32)
        m = len(pos)
        acc = rng.choice([0.1, 0.2, 0.2, 0.5, 0.7, 1.0], size=m)     # many exact ties
        perm = rng.permutation(m)                                      # slot order is arbitrary
        got = ko.select(pos[perm], acc[perm], k, w, p)
        ref = _brute_select(pos[perm], acc[perm], k, w, p)
        assert (got == ref).all()
        assert got.sum() == min(m, k)
        assert got[pos[perm] > p - w].all()                            # recent window always kept


def test_selection_tie_keeps_lower_position():
    pos = np.array([0, 1, 2, 3, 4, 5], dtype=np.int32)
    acc = np.array([0.3, 0.3, 0.3, 0.3, 9.0, 9.0])
    keep = ko.select(pos, acc, k=4, w=2, p=5)
    assert keep.tolist() == [True, True, False, False, True, True]


def test_window_attention_special_case():
    # w = k: only the k most recent survive, whatever the scores say
    pos = np.arange(10, dtype=np.int32)
    acc = np.linspace(10, 1, 10)
    keep = ko.select(pos, acc, k=4, w=4, p=9)
    assert keep.tolist() == [False] * 6 + [True] * 4


# ---------------------------------------------------------------- prompt phase
def _tiny_prompt(seed, U, n, d):
    g = torch.Generator().manual_seed(seed)
    mk = lambda: torch.randn(U, n, d, generator=g).half().numpy()
    return mk(), mk(), mk()


def _lbh(U, H):
    return np.array([(0, u // H, u % H) for u in range(U)], dtype=np.int32)


def test_prefill_zero_noise_equals_column_sums_of_library_softmax():
    U, n, d = 3, 37, 16
    Q, K, V = _tiny_prompt(0, U, n, d)
    P = _params(noise_mode=ko.NOISE_NONE, budget_k=64, recent_w=4)
    st = ko.State(P, _lbh(U, 2))
    acc = st.prefill_score(Q, K)
    q, k = torch.from_numpy(Q).double(), torch.from_numpy(K).double()
    logits = q @ k.transpose(-1, -2) / math.sqrt(d)
    logits = logits.masked_fill(torch.triu(torch.ones(n, n, dtype=torch.bool), 1), float("-inf"))
    ref = torch.softmax(logits, dim=-1).sum(dim=-2).numpy()
    assert np.abs(acc - ref).max() < 1e-12
    assert np.abs(acc.sum(axis=1) - n).max() < 1e-10             # one unit of mass per query row


def test_prefill_with_noise_conserves_mass_and_uses_tau_init():
    U, n, d = 2, 29, 16
    Q, K, V = _tiny_prompt(1, U, n, d)
    P = _params(budget_k=64, recent_w=4, tau_init=1.3, noise_seed=21)
    st = ko.State(P, _lbh(U, 2))
    acc = st.prefill_score(Q, K)
    assert np.abs(acc.sum(axis=1) - n).max() < 1e-10
    # rebuild unit 1 from Eq. 4 / Eq. 11 with numpy and the noise routine
    u = 1
    l, b, h = st.lbh[u]
    q, k = Q[u].astype(np.float64), K[u].astype(np.float64)
    ref = np.zeros(n)
    for i in range(n):
        y = np.array([(q[i] @ k[j] / math.sqrt(d) + ko.noise(P, b, l, h, i, j)) / 1.3 for j in range(i + 1)])
        e = np.exp(y - y.max())
        ref[: i + 1] += e / e.sum()
    assert np.abs(acc[u] - ref).max() < 1e-12
    # first key column receives the whole first row: bias towards initial tokens
    assert acc[u][0] >= 1.0


def test_prefill_alibi_bias_matches_library_softmax():
    U, n, d, H = 2, 24, 16, 2
    Q, K, V = _tiny_prompt(2, U, n, d)
    slopes = W.alibi_slopes(H)
    P = _params(noise_mode=ko.NOISE_NONE, bias_mode=1, alibi_slopes=slopes, n_heads=H, budget_k=64)
    st = ko.State(P, _lbh(U, H))
    acc = st.prefill_score(Q, K)
    i = torch.arange(n)[:, None].double(); j = torch.arange(n)[None, :].double()
    for u in range(U):
        h = st.lbh[u][2]
        logits = torch.from_numpy(Q[u]).double() @ torch.from_numpy(K[u]).double().T / math.sqrt(d) - slopes[h] * (i - j)
        logits = logits.masked_fill(j > i, float("-inf"))
        ref = torch.softmax(logits, -1).sum(0).numpy()
        assert np.abs(acc[u] - ref).max() < 1e-12


def test_prefill_prune_keeps_recent_plus_top_scores_in_position_order():
    U, n, d = 2, 40, 16
    Q, K, V = _tiny_prompt(3, U, n, d)
    P = _params(budget_k=12, recent_w=5, noise_seed=4)
    st = ko.State(P, _lbh(U, 2))
    acc = st.prefill_score(Q, K)
    st.prefill_prune(K, V, acc)
    for u in range(U):
        assert st.len[u] == 12
        pos = st.pos[u, :12]
        assert (np.diff(pos) > 0).all()
        assert set(range(n - 5, n)) <= set(pos.tolist())
        rest = sorted(range(n - 5), key=lambda j: (-acc[u, j], j))[:7]
        assert set(pos.tolist()) == set(rest) | set(range(n - 5, n))
        assert (st.K[u, :12] == K[u].view(np.uint16)[pos]).all()
        assert (st.V[u, :12] == V[u].view(np.uint16)[pos]).all()
        assert (st.acc[u, :12] == acc[u, pos]).all()


def test_prefill_short_prompt_keeps_everything():
    U, n, d = 1, 6, 16
    Q, K, V = _tiny_prompt(4, U, n, d)
    P = _params(budget_k=8, recent_w=2)
    st = ko.State(P, _lbh(U, 2))
    st.prefill_prune(K, V, st.prefill_score(Q, K))
    assert st.len[0] == 6 and st.pos[0, :6].tolist() == list(range(6))


# ---------------------------------------------------------------- generation phase
def _prefilled(P, U, n, d, seed):
    Q, K, V = _tiny_prompt(seed, U, n, d)
    st = ko.State(P, _lbh(U, P.n_heads))
    st.prefill_prune(K, V, st.prefill_score(Q, K))
    return st


def _step_inputs(seed, U, d):
    g = torch.Generator().manual_seed(1000 + seed)
    mk = lambda: torch.randn(U, d, generator=g).half().numpy()
    return mk(), mk(), mk()


def test_prompt_attention_output_matches_library_causal_attention():
    """Eq. 1 over the prompt with the causal mask, against torch's attention in fp64 (also with ALiBi as a mask)."""
    U, n, d = 4, 37, 16
    Q, K, V = _tiny_prompt(11, U, n, d)
    t = lambda a: torch.from_numpy(a.astype(np.float64))
    for slopes in (None, np.array([0.5, 0.125])):
        P = _params(noise_seed=3, bias_mode=0 if slopes is None else 1, alibi_slopes=slopes)
        lbh = _lbh(U, P.n_heads)
        out = ko.State(P, lbh).prefill_attend(Q, K, V)
        i, j = torch.arange(n)[:, None], torch.arange(n)[None, :]
        mask = torch.zeros(U, n, n, dtype=torch.float64).masked_fill(j > i, float("-inf"))
        if slopes is not None:
            mask = mask - torch.from_numpy(slopes[lbh[:, 2]])[:, None, None] * (i - j).clamp(min=0).to(torch.float64)
        ref = torch.nn.functional.scaled_dot_product_attention(t(Q), t(K), t(V), attn_mask=mask)
        assert np.abs(out - ref.numpy()).max() < 1e-12
    # a transposed operand or a dropped mask would show here: row 0 attends to itself only
    assert np.abs(out[:, 0] - V[:, 0].astype(np.float64)).max() < 1e-12


def test_decode_output_matches_library_attention():
    U, n, d = 3, 30, 16
    P = _params(budget_k=10, recent_w=3, noise_seed=8)
    st = _prefilled(P, U, n, d, 5)
    q, kn, vn = _step_inputs(0, U, d)
    out, z = st.decode_score(1, q, kn, vn)
    m = 11
    Kc = torch.from_numpy(st.K[:, :m].view(np.float16).astype(np.float64))
    Vc = torch.from_numpy(st.V[:, :m].view(np.float16).astype(np.float64))
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q.astype(np.float64))[:, None, :], Kc, Vc)[:, 0]
    assert np.abs(out - ref.numpy()).max() < 1e-12
    # the appended entry is the new token at position n
    assert (st.pos[:, m - 1] == n).all() and (st.K[:, m - 1] == kn.view(np.uint16)).all()
    assert np.abs(z[:, :m].sum(axis=1) - 1.0).max() < 1e-12          # Eq. 11 is a softmax


def test_decode_zero_noise_tau_one_score_is_the_attention_weight():
    U, n, d = 2, 20, 16
    P = _params(budget_k=10, recent_w=3, noise_mode=ko.NOISE_NONE, tau_init=1.0, tau_end=1.0)
    st = _prefilled(P, U, n, d, 6)
    q, kn, vn = _step_inputs(1, U, d)
    out, z = st.decode_score(1, q, kn, vn)
    m = 11
    Vc = st.V[:, :m].view(np.float16).astype(np.float64)
    assert np.abs(np.einsum("um,umd->ud", z[:, :m], Vc) - out).max() < 1e-12
    Kc = st.K[:, :m].view(np.float16).astype(np.float64)
    x = np.einsum("ud,umd->um", q.astype(np.float64), Kc) / math.sqrt(d)
    ref = torch.softmax(torch.from_numpy(x), -1).numpy()
    assert np.abs(z[:, :m] - ref).max() < 1e-12


def test_decode_temperature_limits():
    U, n, d = 1, 20, 16
    q, kn, vn = _step_inputs(2, U, d)
    hot = _params(budget_k=10, recent_w=3, tau_init=1e9, tau_end=1e9, noise_seed=2)
    _, z = _prefilled(hot, U, n, d, 7).decode_score(1, q, kn, vn)
    assert np.abs(z[0, :11] - 1.0 / 11).max() < 1e-6                  # tau -> inf : uniform
    cold = _params(budget_k=10, recent_w=3, tau_init=1e-4, tau_end=1e-4, noise_seed=2)
    st = _prefilled(cold, U, n, d, 7)
    _, z = st.decode_score(1, q, kn, vn)
    Kc = st.K[0, :11].view(np.float16).astype(np.float64)
    y = Kc @ q[0].astype(np.float64) / math.sqrt(d) + np.array(
        [ko.noise(cold, 0, 0, 0, n, int(pj)) for pj in st.pos[0, :11]])
    assert z[0, np.argmax(y)] > 1 - 1e-9                              # tau -> 0 : one-hot at argmax(x+zeta)


def test_decode_score_uses_step_temperature_and_position_keyed_noise():
    U, n, d = 2, 25, 16
    P = _params(budget_k=10, recent_w=3, gen_len_T=4, noise_seed=31)
    st = _prefilled(P, U, n, d, 8)
    for s in (1, 2, 3):
        q, kn, vn = _step_inputs(10 + s, U, d)
        before = st.acc.copy()
        out, z = st.decode_score(s, q, kn, vn)
        m = int(st.len[0])
        p = n + s - 1
        tau = 1.0 + s * 0.25
        for u in range(U):
            l, b, h = st.lbh[u]
            Kc = st.K[u, :m].view(np.float16).astype(np.float64)
            x = Kc @ q[u].astype(np.float64) / math.sqrt(d)
            y = (x + np.array([ko.noise(P, b, l, h, p, int(pj)) for pj in st.pos[u, :m]])) / tau
            ref = np.exp(y - y.max()); ref /= ref.sum()
            assert np.abs(z[u, :m] - ref).max() < 1e-12
            # accumulation: old entries gain z, the new entry starts from zero
            assert np.abs(st.acc[u, : m - 1] - (before[u, : m - 1] + z[u, : m - 1])).max() < 1e-15
            assert st.acc[u, m - 1] == z[u, m - 1]
        total_before = st.acc[:, :m].sum(axis=1)
        ev = st.decode_evict(s)
        assert (st.len == P.budget_k).all() and (ev >= 0).all()
        # recent window survives; exactly one entry left
        for u in range(U):
            pos = st.pos[u, : P.budget_k]
            assert set(range(p - P.recent_w + 1, p + 1)) <= set(pos.tolist())
            assert ev[u] not in pos and ev[u] <= p - P.recent_w


def test_decode_conservation_of_mass_and_single_eviction():
    U, n, d = 2, 30, 16
    P = _params(budget_k=12, recent_w=4, gen_len_T=6, noise_seed=77)
    st = _prefilled(P, U, n, d, 9)
    kept_mass = st.acc[:, :12].sum(axis=1)
    for s in range(1, 7):
        q, kn, vn = _step_inputs(50 + s, U, d)
        st.decode_score(s, q, kn, vn)
        assert (st.len == 13).all()
        mass = st.acc[:, :13].sum(axis=1)
        assert np.abs(mass - (kept_mass + 1.0)).max() < 1e-12          # each step adds one unit
        pos_before = [set(st.pos[u, :13].tolist()) for u in range(U)]
        acc_before = st.acc.copy(); posb = st.pos.copy()
        ev = st.decode_evict(s)
        for u in range(U):
            assert pos_before[u] - set(st.pos[u, :12].tolist()) == {int(ev[u])}
            # evicted entry had the smallest score among the non-recent ones
            p = n + s - 1
            cand = [j for j in range(13) if posb[u, j] <= p - 4]
            jmin = min(cand, key=lambda j: (acc_before[u, j], -posb[u, j]))
            assert posb[u, jmin] == ev[u]
        kept_mass = st.acc[:, :12].sum(axis=1)


def test_decode_window_special_case_is_a_sliding_window():
    U, n, d = 1, 20, 16
    P = _params(budget_k=6, recent_w=6, gen_len_T=5)
    st = _prefilled(P, U, n, d, 10)
    assert st.pos[0, :6].tolist() == list(range(14, 20))
    for s in range(1, 6):
        q, kn, vn = _step_inputs(70 + s, U, d)
        st.decode_score(s, q, kn, vn)
        st.decode_evict(s)
        assert st.pos[0, :6].tolist() == list(range(14 + s, 20 + s))


def test_decode_heavy_hitter_special_case_without_window():
    # w = 0, no noise, tau = 1: the entry with the least accumulated attention leaves (H2O-like)
    U, n, d = 1, 16, 16
    P = _params(budget_k=8, recent_w=0, noise_mode=ko.NOISE_NONE, tau_init=1.0, tau_end=1.0)
    st = _prefilled(P, U, n, d, 11)
    q, kn, vn = _step_inputs(90, U, d)
    st.decode_score(1, q, kn, vn)
    acc = st.acc[0, :9].copy(); pos = st.pos[0, :9].copy()
    ev = st.decode_evict(1)
    assert ev[0] == pos[np.lexsort((-pos, acc))[0]]


def test_decode_growing_cache_without_eviction():
    U, n, d = 1, 5, 16
    P = _params(budget_k=8, recent_w=2)
    st = _prefilled(P, U, n, d, 12)
    for s in range(1, 4):
        q, kn, vn = _step_inputs(95 + s, U, d)
        st.decode_score(s, q, kn, vn)
        ev = st.decode_evict(s)
        assert ev[0] == -1 and st.len[0] == 5 + s
    q, kn, vn = _step_inputs(99, U, d)
    st.decode_score(4, q, kn, vn)
    assert st.decode_evict(4)[0] >= 0 and st.len[0] == 8


def test_forced_eviction_and_forced_keep_are_applied():
    U, n, d = 1, 20, 16
    P = _params(budget_k=8, recent_w=2)
    Q, K, V = _tiny_prompt(13, U, n, d)
    st = ko.State(P, _lbh(U, 2))
    acc = st.prefill_score(Q, K)
    keep = np.zeros((1, n), np.uint8); keep[0, [0, 1, 2, 3, 4, 5, 18, 19]] = 1
    st.prefill_prune(K, V, acc, keep_override=keep)
    assert st.pos[0, :8].tolist() == [0, 1, 2, 3, 4, 5, 18, 19]
    q, kn, vn = _step_inputs(100, U, d)
    st.decode_score(1, q, kn, vn)
    ev = st.decode_evict(1, force_evict_pos=np.array([3], np.int32))
    assert ev[0] == 3 and st.pos[0, :8].tolist() == [0, 1, 2, 4, 5, 18, 19, 20]


# ---------------------------------------------------------------- position variants (section 4.4.2)
def test_decode_new_positions_bias_follows_the_place_in_the_reduced_cache():
    """"New Pos": the ALiBi distance is counted in places of the reduced cache.  The reference is library
    attention with an additive mask built here from the kept positions; with original positions the same
    construction uses the position gaps, so the two variants must differ once tokens have been evicted."""
    U, n, d, H = 2, 40, 16, 2
    slopes = W.alibi_slopes(H)
    outs = {}
    for mode in (0, 1):
        P = _params(budget_k=10, recent_w=3, noise_mode=ko.NOISE_NONE, tau_init=1.0, tau_end=1.0, bias_mode=1,
                    alibi_slopes=slopes, n_heads=H, pos_mode=mode)
        st = _prefilled(P, U, n, d, 21)
        for s in (1, 2, 3):
            q, kn, vn = _step_inputs(40 + s, U, d)
            out, z = st.decode_score(s, q, kn, vn)
            m = 11
            p = n + s - 1
            pos = st.pos[:, :m].astype(np.float64)
            assert (np.diff(pos, axis=1) > 0).all() and (pos[:, -1] == p).all()
            sl = np.array([slopes[st.lbh[u][2]] for u in range(U)])[:, None]
            dist = (m - 1 - np.arange(m, dtype=np.float64))[None, :] if mode == 1 else p - pos
            assert mode == 1 or (dist[:, 0] > m - 1).all()      # something was evicted: gaps exceed places
            mask = torch.from_numpy(-sl * dist)[:, None, :]
            Kc = torch.from_numpy(st.K[:, :m].view(np.float16).astype(np.float64))
            Vc = torch.from_numpy(st.V[:, :m].view(np.float16).astype(np.float64))
            ref = torch.nn.functional.scaled_dot_product_attention(
                torch.from_numpy(q.astype(np.float64))[:, None, :], Kc, Vc, attn_mask=mask)[:, 0]
            assert np.abs(out - ref.numpy()).max() < 1e-12
            # zero noise, temperature 1: the score is the attention weight under the same bias
            x = np.einsum("ud,umd->um", q.astype(np.float64), Kc.numpy()) / math.sqrt(d) - sl * dist
            assert np.abs(z[:, :m] - torch.softmax(torch.from_numpy(x), -1).numpy()).max() < 1e-12
            st.decode_evict(s)
            outs[(mode, s)] = out
    assert np.abs(outs[(0, 1)] - outs[(1, 1)]).max() > 1e-4


def test_new_positions_equal_original_positions_until_something_is_evicted():
    U, n, d, H = 2, 6, 16, 2
    slopes = W.alibi_slopes(H)
    res = []
    for mode in (0, 1):
        P = _params(budget_k=12, recent_w=3, noise_seed=4, bias_mode=1, alibi_slopes=slopes, n_heads=H, pos_mode=mode)
        st = _prefilled(P, U, n, d, 22)
        steps = []
        for s in range(1, 9):
            q, kn, vn = _step_inputs(60 + s, U, d)
            out, z = st.decode_score(s, q, kn, vn)
            st.decode_evict(s)
            steps.append(out.copy())
        res.append(steps)
    for s in range(8):
        if n + s <= 12:                # nothing evicted before this step's scoring: places are positions
            assert np.array_equal(res[0][s], res[1][s])
    assert not np.array_equal(res[0][7], res[1][7])


# ---------------------------------------------------------------- shared key/value heads (section 6: MQA / GQA)
def _grouped_case(seed, B, Hkv, g, n, d):
    """Q [B*Hkv][g][n][d], K, V [B*Hkv][n][d] and the same data laid out for H = Hkv * g independent heads
    (K, V repeated for every query head of a group)."""
    gen = torch.Generator().manual_seed(400 + seed)
    U = B * Hkv
    Q = torch.randn(U, g, n, d, generator=gen).half().numpy()
    K = torch.randn(U, n, d, generator=gen).half().numpy()
    V = torch.randn(U, n, d, generator=gen).half().numpy()
    lbh_kv = np.array([(1, u // Hkv, u % Hkv) for u in range(U)], dtype=np.int32)
    lbh_q = np.array([(1, u // Hkv, (u % Hkv) * g + r) for u in range(U) for r in range(g)], dtype=np.int32)
    return Q, K, V, lbh_kv, lbh_q


@pytest.mark.parametrize("g", [2, 4])
def test_grouped_heads_prompt_scores_are_the_group_mean_of_independent_heads(g):
    """With K/V repeated for every query head, multi-head scoring (pinned above to library softmax) gives each
    query head's f_theta; the shared-head score must be their mean over the group, noise, temperature and ALiBi
    slope of every head being that head's own."""
    B, Hkv, n, d = 2, 3, 29, 16
    H = Hkv * g
    Q, K, V, lbh_kv, lbh_q = _grouped_case(g, B, Hkv, g, n, d)
    slopes = W.alibi_slopes(H)
    common = dict(head_dim=d, n_heads=H, budget_k=12, recent_w=3, gen_len_T=4, noise_seed=77, tau_init=1.3,
                  bias_mode=1, alibi_slopes=slopes)
    grouped = ko.State(ko.Params(n_kv_heads=Hkv, **common), lbh_kv).prefill_score(Q, K)
    single = ko.State(ko.Params(**common), lbh_q).prefill_score(Q.reshape(-1, n, d), np.repeat(K, g, axis=0))
    assert np.abs(grouped - single.reshape(B * Hkv, g, n).mean(axis=1)).max() < 1e-12
    assert np.abs(grouped.sum(axis=1) - n).max() < 1e-9                 # a cache still receives mass 1 per query row
    # and the heads of a group really differ (own noise, own slope): the mean is not one head's score
    assert np.abs(single.reshape(B * Hkv, g, n)[:, 0] - grouped).max() > 1e-3


@pytest.mark.parametrize("g", [2, 8])
def test_grouped_heads_decode_against_library_attention_with_repeated_kv(g):
    B, Hkv, n, d = 1, 2, 26, 16
    H = Hkv * g
    U = B * Hkv
    Q, K, V, lbh_kv, _ = _grouped_case(10 + g, B, Hkv, g, n, d)
    P = ko.Params(head_dim=d, n_heads=H, n_kv_heads=Hkv, budget_k=10, recent_w=3, gen_len_T=4, noise_mode=ko.NOISE_NONE,
                  tau_init=1.0, tau_end=1.0)
    st = ko.State(P, lbh_kv)
    st.prefill_prune(K, V, st.prefill_score(Q, K))
    gen = torch.Generator().manual_seed(5)
    q = torch.randn(U, g, d, generator=gen).half().numpy()
    kn, vn = torch.randn(U, d, generator=gen).half().numpy(), torch.randn(U, d, generator=gen).half().numpy()
    total_before = st.acc[:, :10].sum(axis=1)
    out, z = st.decode_score(1, q, kn, vn)
    m = 11
    Kc = torch.from_numpy(st.K[:, :m].view(np.float16).astype(np.float64))
    Vc = torch.from_numpy(st.V[:, :m].view(np.float16).astype(np.float64))
    qt = torch.from_numpy(q.astype(np.float64))
    # library attention with every key/value head repeated for the g query heads of its group
    ref = torch.nn.functional.scaled_dot_product_attention(
        qt.reshape(1, U * g, 1, d), Kc.repeat_interleave(g, 0)[None], Vc.repeat_interleave(g, 0)[None])
    assert out.shape == (U, g, d) and np.abs(out - ref.reshape(U, g, d).numpy()).max() < 1e-12
    # zero noise, temperature 1: the accumulated score is the mean attention weight of the group
    w = torch.softmax(torch.einsum("ugd,umd->ugm", qt, Kc) / math.sqrt(d), -1).mean(1).numpy()
    assert np.abs(z[:, :m] - w).max() < 1e-12
    assert np.abs(st.acc[:, :m].sum(axis=1) - (total_before + 1.0)).max() < 1e-12      # +1 per step per cache


def test_grouped_heads_decode_noise_is_drawn_per_query_head():
    B, Hkv, g, n, d = 1, 2, 4, 20, 16
    H, U = Hkv * g, B * Hkv
    Q, K, V, lbh_kv, _ = _grouped_case(3, B, Hkv, g, n, d)
    P = ko.Params(head_dim=d, n_heads=H, n_kv_heads=Hkv, budget_k=8, recent_w=2, gen_len_T=4, noise_seed=123)
    st = ko.State(P, lbh_kv)
    st.prefill_prune(K, V, st.prefill_score(Q, K))
    gen = torch.Generator().manual_seed(6)
    q = torch.randn(U, g, d, generator=gen).half().numpy()
    kn, vn = torch.randn(U, d, generator=gen).half().numpy(), torch.randn(U, d, generator=gen).half().numpy()
    _, z = st.decode_score(2, q, kn, vn)
    m, p, tau = 9, n + 1, 1.0 + 2 * 0.25
    for u in range(U):
        l, b, hk = st.lbh[u]
        Kc = st.K[u, :m].view(np.float16).astype(np.float64)
        ref = np.zeros(m)
        for r in range(g):
            x = Kc @ q[u, r].astype(np.float64) / math.sqrt(d)
            y = (x + np.array([ko.noise(P, b, l, hk * g + r, p, int(pj)) for pj in st.pos[u, :m]])) / tau
            e = np.exp(y - y.max())
            ref += e / e.sum() / g
        assert np.abs(z[u, :m] - ref).max() < 1e-12


def test_one_query_head_per_key_value_head_is_the_plain_method_bit_for_bit():
    """n_kv_heads = n_heads (or 0) must not change a single bit of any result."""
    U, n, d = 4, 33, 16
    Q, K, V = _tiny_prompt(21, U, n, d)
    res = []
    for nkv in (0, 2):
        P = _params(budget_k=9, recent_w=2, noise_seed=17, n_kv_heads=nkv)
        st = ko.State(P, _lbh(U, 2))
        acc = st.prefill_score(Q, K)
        st.prefill_prune(K, V, acc)
        outs = [acc, st.prefill_attend(Q, K, V)]
        for s in (1, 2, 3):
            out, z = st.decode_score(s, *_step_inputs(s, U, d))
            st.decode_evict(s)
            outs += [out, z, st.acc.copy(), st.pos.copy()]
        res.append(outs)
    for a, b in zip(*res):
        assert a.shape == b.shape and np.array_equal(a, b)


# ---------------------------------------------------------------- rotary embedding applied at logit time (section 4.4.2 on rotary models)
def _rope_np(x, pos, R, base=10000.0):
    """Independent restatement (numpy, complex arithmetic): pair (2i, 2i+1) is the complex number x_2i + i x_2i+1,
    multiplied by exp(i pos theta_i), theta_i = base^(-2i/R).  x: [..., d] float64, pos: broadcastable to x[..., 0]."""
    x = np.array(x, dtype=np.float64)
    z = x[..., 0:R:2] + 1j * x[..., 1:R:2]
    theta = base ** (-2.0 * np.arange(R // 2) / R)
    z = z * np.exp(1j * np.asarray(pos, dtype=np.float64)[..., None] * theta)
    out = x.copy()
    out[..., 0:R:2], out[..., 1:R:2] = z.real, z.imag
    return out


@pytest.mark.parametrize("R,d", [(16, 16), (8, 16)])
def test_rotary_prompt_scores_and_attention_match_library_routines_on_rotated_inputs(R, d):
    U, n = 3, 33
    Q, K, V = _tiny_prompt(31, U, n, d)
    P = _params(noise_mode=ko.NOISE_NONE, budget_k=64, recent_w=4, rotary_dims=R, head_dim=d)
    st = ko.State(P, _lbh(U, 2))
    acc = st.prefill_score(Q, K)
    pos = np.arange(n)
    q = torch.from_numpy(_rope_np(Q.astype(np.float64), pos[None, :], R))
    k = torch.from_numpy(_rope_np(K.astype(np.float64), pos[None, :], R))
    logits = q @ k.transpose(-1, -2) / math.sqrt(d)
    causal = torch.triu(torch.ones(n, n, dtype=torch.bool), 1)
    ref = torch.softmax(logits.masked_fill(causal, float("-inf")), dim=-1).sum(dim=-2).numpy()
    assert np.abs(acc - ref).max() < 1e-11
    out = st.prefill_attend(Q, K, V)
    ref_o = torch.nn.functional.scaled_dot_product_attention(q, k, torch.from_numpy(V.astype(np.float64)), is_causal=True)
    assert np.abs(out - ref_o.numpy()).max() < 1e-11
    # the rotation matters (a forgotten one would reproduce the unrotated scores)
    plain = ko.State(_params(noise_mode=ko.NOISE_NONE, budget_k=64, recent_w=4, head_dim=d), _lbh(U, 2)).prefill_score(Q, K)
    assert np.abs(plain - acc).max() > 1e-2


@pytest.mark.parametrize("pos_mode", [0, 1])
def test_rotary_decode_uses_original_positions_or_places(pos_mode):
    """After evictions the kept positions have gaps.  Org Pos rotates query and keys at the positions in the text, New
    Pos at the places in the reduced cache; both against library attention on inputs rotated here."""
    U, n, d, R = 2, 40, 16, 16
    P = _params(budget_k=12, recent_w=3, noise_mode=ko.NOISE_NONE, tau_init=1.0, tau_end=1.0, rotary_dims=R, pos_mode=pos_mode)
    st = _prefilled(P, U, n, d, 41)
    for s in (1, 2, 3):
        q, kn, vn = _step_inputs(40 + s, U, d)
        out, z = st.decode_score(s, q, kn, vn)
        m, p = int(st.len[0]), n + s - 1
        kpos = np.tile(np.arange(m), (U, 1)) if pos_mode == 1 else st.pos[:, :m].astype(np.int64)
        qpos = np.full(U, m - 1 if pos_mode == 1 else p)
        assert pos_mode == 1 or (np.diff(kpos, axis=1) > 1).any()        # gaps: the two numberings really differ
        Kc = _rope_np(st.K[:, :m].view(np.float16).astype(np.float64), kpos, R)
        Vc = st.V[:, :m].view(np.float16).astype(np.float64)
        qr = _rope_np(q.astype(np.float64), qpos, R)
        ref = torch.nn.functional.scaled_dot_product_attention(torch.from_numpy(qr)[:, None, :], torch.from_numpy(Kc),
                                                               torch.from_numpy(Vc))[:, 0]
        assert np.abs(out - ref.numpy()).max() < 1e-11
        w = torch.softmax(torch.einsum("ud,umd->um", torch.from_numpy(qr), torch.from_numpy(Kc)) / math.sqrt(d), -1).numpy()
        assert np.abs(z[:, :m] - w).max() < 1e-11                        # zero noise, tau 1: the score is the attention weight
        assert (st.K[:, m - 1] == kn.view(np.uint16)).all()              # the cache keeps the new key as given, without rotation
        st.decode_evict(s)


def test_rotary_logits_depend_on_relative_positions_only():
    """A prompt phase shifted by a constant offset gives the same scores: x_ij depends on i - j (the defining property
    of the embedding); checked by comparing rows/columns of a long prompt's logit structure through two sub-prompts."""
    d, R = 16, 16
    Q, K, V = _tiny_prompt(51, 1, 24, d)
    P = _params(noise_mode=ko.NOISE_NONE, budget_k=64, recent_w=2, rotary_dims=R)
    st = ko.State(P, _lbh(1, 2))
    full = st.prefill_attend(Q, K, V)
    # generation with New Pos on a cache that holds everything equals Org Pos (places = positions), at every step
    a = _prefilled(_params(budget_k=64, recent_w=2, noise_seed=5, rotary_dims=R, pos_mode=0), 2, 20, d, 52)
    b = _prefilled(_params(budget_k=64, recent_w=2, noise_seed=5, rotary_dims=R, pos_mode=1), 2, 20, d, 52)
    for s in (1, 2, 3):
        q, kn, vn = _step_inputs(60 + s, 2, d)
        oa, za = a.decode_score(s, q, kn, vn)
        ob, zb = b.decode_score(s, q, kn, vn)
        assert np.abs(oa - ob).max() < 1e-12 and np.abs(za - zb).max() < 1e-12
        a.decode_evict(s); b.decode_evict(s)
    assert np.isfinite(full).all()


def test_rotary_modes_differ_once_something_is_evicted_and_zero_dims_is_the_plain_method():
    U, n, d = 2, 40, 16
    res = []
    for pm in (0, 1):
        st = _prefilled(_params(budget_k=10, recent_w=3, noise_seed=9, rotary_dims=16, pos_mode=pm), U, n, d, 61)
        q, kn, vn = _step_inputs(70, U, d)
        res.append(st.decode_score(1, q, kn, vn)[0])
    assert np.abs(res[0] - res[1]).max() > 1e-3
    outs = []
    for kw in (dict(), dict(rotary_dims=0, rotary_base=500.0)):
        st = _prefilled(_params(budget_k=10, recent_w=3, noise_seed=9, **kw), U, n, d, 61)
        q, kn, vn = _step_inputs(70, U, d)
        outs.append(st.decode_score(1, q, kn, vn))
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])
