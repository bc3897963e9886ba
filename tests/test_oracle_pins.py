"""Pins of the CPU oracle against what the paper's definitions and plain mathematics fix.

None of these tests touches the CUDA library.  Each one is chosen so that a plausible mistake in
the oracle (a dropped term, a wrong sign or index, a transposed operand, a wrong normaliser)
fails it.  Library routines used as independent references: torch.softmax (fp64),
scipy.stats.skew, numpy sorting, exhaustive enumeration.
"""
import itertools
import math
import os

import numpy as np
import pytest
import scipy.stats
import torch

from workloads import CONFIGS, decode_queries, full_cache, plan, window_queries
from workloads.synth import to_u16

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32/fp64 numpy -> bf16 bit patterns (round to nearest even), as uint16."""
    return to_u16(torch.from_numpy(np.asarray(x, np.float32)).to(torch.bfloat16))


def bf16_val(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def dims_of(oracle, wl, **kw):
    d = dict(n_layers=wl.n_layers, batch=wl.batch, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads,
             head_dim=wl.head_dim, n_visual=wl.n_visual, n_text=wl.n_text, window=wl.window)
    d.update(kw)
    return oracle.Dims(**d)


def rand_case(rng, L=2, B=2, Hq=4, Hkv=2, d=16, Nv=40, Nt=8, W=4):
    k = bf16_bits(rng.standard_normal((L, B, Hkv, Nv + Nt, d)))
    v = bf16_bits(rng.standard_normal((L, B, Hkv, Nv + Nt, d)))
    qw = bf16_bits(rng.standard_normal((L, B, W, Hq, d)))
    return k, v, qw


# ----------------------------------------------------------------------------------------------
# Eq. 4-5: elite observation window
# ----------------------------------------------------------------------------------------------
def test_elite_alpha_zero_keeps_all_and_alpha_one_keeps_argmax(oracle_mod):
    rng = np.random.default_rng(1)
    L, B, Hq, Hkv, d, Nv, Nt, W = 2, 2, 4, 2, 16, 40, 8, 8
    k, _, qw = rand_case(rng, L, B, Hq, Hkv, d, Nv, Nt, W)
    dm = oracle_mod.Dims(L, B, Hq, Hkv, d, Nv, Nt, W)
    scale = 0.25
    m0 = oracle_mod.score(dm, k, qw, scale, 0.0)["elite_mask"]
    assert (m0 == (1 << W) - 1).all()
    out = oracle_mod.score(dm, k, qw, scale, 1.0, want_logits=True)
    # independent logits: last window query against the last W text keys
    kf, qf = bf16_val(k), bf16_val(qw)
    for l, b, h in itertools.product(range(L), range(B), range(Hq)):
        g = h // (Hq // Hkv)
        t = kf[l, b, g, Nv + Nt - W:, :] @ qf[l, b, W - 1, h, :] * scale
        assert np.allclose(out["elite_logits"][l, b, h], t, rtol=1e-6, atol=1e-6)
        assert int(out["elite_mask"][l, b, h]) == 1 << int(np.argmax(t))


def test_elite_matches_literal_softmax_threshold(oracle_mod):
    """Eq. 5 taken literally on the softmax row of Eq. 4 (library softmax, all text tokens as
    candidates) gives the same set as the oracle's log-domain comparison."""
    rng = np.random.default_rng(2)
    L, B, Hq, Hkv, d, Nv, Nt = 3, 2, 6, 2, 32, 24, 20
    W = Nt
    k, _, qw = rand_case(rng, L, B, Hq, Hkv, d, Nv, Nt, W)
    dm = oracle_mod.Dims(L, B, Hq, Hkv, d, Nv, Nt, W)
    scale = 1 / math.sqrt(d)
    kf, qf = bf16_val(k), bf16_val(qw)
    for alpha in (0.3, 0.6, 0.9):
        out = oracle_mod.score(dm, k, qw, scale, alpha)
        checked = 0
        for l, b, h in itertools.product(range(L), range(B), range(Hq)):
            g = h // (Hq // Hkv)
            logits = torch.from_numpy(kf[l, b, g, Nv:, :] @ qf[l, b, W - 1, h, :] * scale)
            a = torch.softmax(logits, 0).numpy()
            rel = a / a.max()
            if np.abs(rel - alpha).min() < 1e-4:      # too close to the threshold to call in fp32
                continue
            want = sum(1 << j for j in range(W) if rel[j] >= alpha)
            assert int(out["elite_mask"][l, b, h]) == want
            # the arg-max is always elite
            assert want >> int(np.argmax(a)) & 1
            checked += 1
        assert checked > 20


def test_window_of_all_text_tokens_beyond_64(oracle_mod):
    """The paper's own window: every text token is a candidate (W = N_t, here 100 > 64, so the elite set takes two
    mask words).  Eq. 5 literally on the library softmax row, and Eq. 6-8 in matrix form on that set."""
    rng = np.random.default_rng(5)
    L, B, Hq, Hkv, d, Nv, Nt = 1, 2, 4, 2, 32, 19, 100
    W = Nt
    k, _, qw = rand_case(rng, L, B, Hq, Hkv, d, Nv, Nt, W)
    dm = oracle_mod.Dims(L, B, Hq, Hkv, d, Nv, Nt, W)
    scale = 1 / math.sqrt(d)
    kf, qf = bf16_val(k), bf16_val(qw)
    for alpha in (0.0, 0.5, 0.9):
        out = oracle_mod.score(dm, k, qw, scale, alpha)
        assert out["elite_mask"].shape == (L, B, Hq, 2)
        for l, b in itertools.product(range(L), range(B)):
            acc = np.zeros(Nv)
            for h in range(Hq):
                g = h // (Hq // Hkv)
                E = int(out["elite_mask"][l, b, h, 0]) | int(out["elite_mask"][l, b, h, 1]) << 64
                a = torch.softmax(torch.from_numpy(kf[l, b, g, Nv:, :] @ qf[l, b, W - 1, h, :] * scale), 0).numpy()
                rel = a / a.max()
                if np.abs(rel - alpha).min() > 1e-4:
                    assert E == sum(1 << j for j in range(W) if rel[j] >= alpha)
                assert E >> W == 0 and E >> int(np.argmax(a)) & 1
                iv, _ = literal_importance(kf[l, b, g], qf[l, b, :, h, :], E, Nv, Nt, W, scale)
                acc += iv
            assert np.allclose(out["scores"][l, b], acc / Hq, rtol=2e-7, atol=0)
        if alpha == 0.0:
            assert (out["elite_mask"][..., 0] == 2 ** 64 - 1).all() and (out["elite_mask"][..., 1] == 2 ** 36 - 1).all()


# ----------------------------------------------------------------------------------------------
# Eq. 6-8: inter-modal attention and importance
# ----------------------------------------------------------------------------------------------
def literal_importance(kf, qf, E, Nv, Nt, W, scale):
    """Eq. 6-8 for one head in matrix form with a library softmax: gather elite queries/keys,
    softmax over Concat(K_v, K_t[k]) with a causal mask among the text columns, mean over rows."""
    N = Nv + Nt
    idx = [w for w in range(W) if E >> w & 1]
    q_tk = qf[idx]                                            # [n_elite, d]
    k_vtk = np.concatenate([kf[:Nv], kf[[N - W + w for w in idx]]], 0)
    logits = torch.from_numpy(q_tk @ k_vtk.T * scale)
    for r, w in enumerate(idx):
        for c, w2 in enumerate(idx):
            if w2 > w:
                logits[r, Nv + c] = -float("inf")
    a = torch.softmax(logits, dim=1).numpy()
    return a[:, :Nv].mean(0), a[:, Nv:].sum(1).mean()


@pytest.mark.parametrize("alpha", [0.0, 0.5, 0.9])
def test_scores_match_matrix_form_and_sum_to_one(oracle_mod, alpha):
    rng = np.random.default_rng(3)
    L, B, Hq, Hkv, d, Nv, Nt, W = 2, 2, 4, 2, 16, 37, 9, 6
    k, _, qw = rand_case(rng, L, B, Hq, Hkv, d, Nv, Nt, W)
    dm = oracle_mod.Dims(L, B, Hq, Hkv, d, Nv, Nt, W)
    scale = 1 / math.sqrt(d)
    out = oracle_mod.score(dm, k, qw, scale, alpha)
    kf, qf = bf16_val(k), bf16_val(qw)
    for l, b in itertools.product(range(L), range(B)):
        acc = np.zeros(Nv)
        for h in range(Hq):
            g = h // (Hq // Hkv)
            E = int(out["elite_mask"][l, b, h])
            iv, tm = literal_importance(kf[l, b, g], qf[l, b, :, h, :], E, Nv, Nt, W, scale)
            acc += iv
            # visual mass + text mass of every softmax row is 1
            assert abs(tm - out["text_mass"][l, b, h]) < 1e-12
        want = acc / Hq
        got = out["scores"][l, b].astype(np.float64)
        assert np.allclose(got, want, rtol=2e-7, atol=0)
        s_t = got.sum()
        assert 0 < s_t <= 1
        assert abs(s_t - (1 - out["text_mass"][l, b].mean())) < 1e-6


def test_system_prompt_prefix_is_kept_and_stays_out_of_the_scores(oracle_mod):
    """A system prompt passed as leading text rows (Section 3.3: it is left out of the window): the scores are the
    ones of the same cache without the prefix, whatever the prefix holds, and every prefix row survives compaction
    in place, in front of the other text rows."""
    rng = np.random.default_rng(21)
    L, B, Hq, Hkv, d, Nv, Nt, W, P = 2, 2, 4, 2, 16, 37, 9, 6, 5
    k, v, qw = rand_case(rng, L, B, Hq, Hkv, d, Nv, Nt, W)
    prefix_k = bf16_bits(rng.standard_normal((L, B, Hkv, P, d)) * 50.0)   # loud rows: they would show in any softmax
    prefix_v = bf16_bits(rng.standard_normal((L, B, Hkv, P, d)))
    k2 = np.concatenate([k[:, :, :, :Nv], prefix_k, k[:, :, :, Nv:]], axis=3)
    v2 = np.concatenate([v[:, :, :, :Nv], prefix_v, v[:, :, :, Nv:]], axis=3)
    dm, dm2 = oracle_mod.Dims(L, B, Hq, Hkv, d, Nv, Nt, W), oracle_mod.Dims(L, B, Hq, Hkv, d, Nv, Nt + P, W)
    a, b2 = oracle_mod.score(dm, k, qw, 0.25, 0.9), oracle_mod.score(dm2, k2, qw, 0.25, 0.9)
    assert np.array_equal(a["scores"], b2["scores"]) and np.array_equal(a["elite_mask"], b2["elite_mask"])
    st, sk = oracle_mod.moments(b2["scores"])
    bud = oracle_mod.allocate(st, sk, Nv, 0.3)
    cc = oracle_mod.compact(dm2, 0, k2, v2, b2["scores"], bud)
    for r in range(L * B):
        l, b = divmod(r, B)
        first_text = int(cc["offsets"][r]) + int(bud[l, b])
        assert np.array_equal(cc["k"][first_text:first_text + P], prefix_k[l, b].transpose(1, 0, 2))
        assert np.array_equal(cc["v"][first_text:first_text + P], prefix_v[l, b].transpose(1, 0, 2))


def test_single_row_reduces_to_textbook_softmax(oracle_mod):
    """One head, W = 1: the only elite row sees all visual keys plus its own text key."""
    rng = np.random.default_rng(4)
    d, Nv, Nt = 8, 50, 3
    k, _, qw = rand_case(rng, 1, 1, 1, 1, d, Nv, Nt, 1)
    dm = oracle_mod.Dims(1, 1, 1, 1, d, Nv, Nt, 1)
    out = oracle_mod.score(dm, k, qw, 0.5, 0.9)
    kf, qf = bf16_val(k)[0, 0, 0], bf16_val(qw)[0, 0, 0, 0]
    keys = np.concatenate([kf[:Nv], kf[Nv + Nt - 1:]], 0)
    p = torch.softmax(torch.from_numpy(keys @ qf * 0.5), 0).numpy()
    assert np.allclose(out["scores"][0, 0], p[:Nv], rtol=2e-7)
    assert abs(out["text_mass"][0, 0, 0] - p[Nv]) < 1e-12


def test_equal_keys_give_uniform_scores_and_permutation_equivariance(oracle_mod):
    rng = np.random.default_rng(5)
    L, B, Hq, Hkv, d, Nv, Nt, W = 1, 1, 2, 1, 16, 30, 6, 4
    k, _, qw = rand_case(rng, L, B, Hq, Hkv, d, Nv, Nt, W)
    dm = oracle_mod.Dims(L, B, Hq, Hkv, d, Nv, Nt, W)
    base = oracle_mod.score(dm, k, qw, 0.25, 0.5)
    perm = rng.permutation(Nv)
    k2 = k.copy()
    k2[:, :, :, :Nv] = k[:, :, :, perm]
    out2 = oracle_mod.score(dm, k2, qw, 0.25, 0.5)
    assert (out2["elite_mask"] == base["elite_mask"]).all()
    assert np.array_equal(out2["scores"][0, 0], base["scores"][0, 0][perm])
    # all visual keys equal -> uniform importance = visual share / Nv
    k3 = k.copy()
    k3[:, :, :, :Nv] = k[:, :, :, :1]
    out3 = oracle_mod.score(dm, k3, qw, 0.25, 0.5)
    s = out3["scores"][0, 0].astype(np.float64)
    assert np.allclose(s, s[0], rtol=1e-7)
    assert abs(s.sum() - (1 - out3["text_mass"][0, 0].mean())) < 1e-6


def test_strided_layouts_agree(oracle_mod):
    """Token-major and head-major storage of the same logical cache give identical results."""
    rng = np.random.default_rng(6)
    L, B, Hq, Hkv, d, Nv, Nt, W = 2, 1, 4, 2, 16, 20, 6, 4
    k, _, qw = rand_case(rng, L, B, Hq, Hkv, d, Nv, Nt, W)
    dm = oracle_mod.Dims(L, B, Hq, Hkv, d, Nv, Nt, W)
    k_tok = np.ascontiguousarray(k.transpose(0, 1, 3, 2, 4)).transpose(0, 1, 3, 2, 4)
    assert k_tok.strides != k.strides
    a = oracle_mod.score(dm, k, qw, 0.25, 0.7)
    b = oracle_mod.score(dm, k_tok, qw, 0.25, 0.7)
    assert np.array_equal(a["scores"], b["scores"]) and (a["elite_mask"] == b["elite_mask"]).all()


# ----------------------------------------------------------------------------------------------
# Eq. 9-10: strength and skewness
# ----------------------------------------------------------------------------------------------
def golden_skew_rows():
    rows = []
    with open(os.path.join(GOLDEN, "skewness_closed_forms.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                kind, n, a, exp = line.split()
                rows.append((kind, int(n), int(a), float(exp)))
    return rows


@pytest.mark.parametrize("kind,n,a,expected", golden_skew_rows())
def test_skewness_closed_forms(oracle_mod, kind, n, a, expected):
    x = np.zeros(n, np.float32)
    if kind in ("onehot", "twopoint"):
        x[np.random.default_rng(n).choice(n, a, replace=False)] = 1.0
    else:
        x[:] = np.arange(n) - (n - 1) / 2
    st, sk = oracle_mod.moments(x)
    assert abs(float(sk) - expected) <= 1e-12 * max(1.0, expected)
    assert abs(float(st) - x.astype(np.float64).sum()) < 1e-12


def test_skewness_matches_library_and_is_affine_invariant(oracle_mod):
    rng = np.random.default_rng(7)
    x = rng.gamma(0.7, size=(5, 1000)).astype(np.float32)
    st, sk = oracle_mod.moments(x)
    ref = scipy.stats.skew(x.astype(np.float64), axis=1, bias=False)
    assert np.allclose(sk, ref, rtol=1e-11)
    assert np.allclose(st, x.astype(np.float64).sum(1), rtol=1e-14)
    y = (x * 4.0 + 2.0).astype(np.float32)            # exact in fp32 for these magnitudes? compare via library
    _, sk2 = oracle_mod.moments(y)
    assert np.allclose(sk2, scipy.stats.skew(y.astype(np.float64), axis=1, bias=False), rtol=1e-11)
    assert np.allclose(sk2, sk, rtol=1e-5)
    _, sk3 = oracle_mod.moments(np.full(10, 0.25, np.float32))
    assert float(sk3) == 0.0                           # sigma = 0
    with pytest.raises(ValueError):
        oracle_mod.moments(np.ones(2, np.float32))


# ----------------------------------------------------------------------------------------------
# Eq. 11 + integer budgets
# ----------------------------------------------------------------------------------------------
def waterfill(w, T, cap):
    """Continuous capped proportional shares by bisection on the multiplier (independent method)."""
    w = np.asarray(w, float)
    lo, hi = 0.0, 1e12
    for _ in range(200):
        mid = 0.5 * (lo + hi)
        if np.minimum(cap, mid * w).sum() < T:
            lo = mid
        else:
            hi = mid
    return np.minimum(cap, hi * w)


def weights_of(st, sk):
    skp = np.maximum(sk, 0)
    nt = st / st.mean() if st.mean() > 0 else np.ones_like(st)
    nk = skp / skp.mean() if skp.mean() > 0 else np.ones_like(st)
    return 0.5 * (nt + nk)


def test_budget_invariants(oracle_mod):
    rng = np.random.default_rng(8)
    for trial in range(200):
        L = int(rng.integers(1, 40))
        B = int(rng.integers(1, 4))
        Nv = int(rng.integers(3, 3000))
        ratio = float(rng.choice([0.01, 0.05, 0.1, 0.25, 0.5, 0.9, 1.0, rng.uniform()]))
        st = rng.uniform(0.1, 1.0, (L, B))
        sk = rng.normal(5, 6, (L, B))
        for mode in range(4):
            n = oracle_mod.allocate(st, sk, Nv, ratio, mode)
            T = math.floor(ratio * (Nv * L) + 0.5)
            assert (n.sum(0) == T).all(), (L, B, Nv, ratio, mode)
            assert n.min() >= 0 and n.max() <= Nv
            assert oracle_mod.total_kept(Nv, L, ratio) == T
            if ratio == 1.0:
                assert (n == Nv).all()
            if mode == 3:                                # uniform: differ by <= 1, +1s on the lowest layers
                for b in range(B):
                    col = n[:, b]
                    assert col.max() - col.min() <= 1
                    assert (np.diff(col) <= 0).all()


def test_budget_equal_layers_uniform_and_mean_preserving(oracle_mod):
    L, Nv = 7, 100
    st = np.full((L, 1), 0.8)
    sk = np.full((L, 1), 3.0)
    n = oracle_mod.allocate(st, sk, Nv, 0.1)[:, 0]
    assert n.sum() == 70 and (n == 10).all()
    n = oracle_mod.allocate(st, sk, Nv, 0.123)[:, 0]       # T = round(86.1) = 86 = 7*12 + 2
    assert n.tolist() == [13, 13, 12, 12, 12, 12, 12]
    # Eq. 11: r_hat_l = w_l * r with mean_l w_l = 1 -> continuous shares Nv * r_hat_l (no cap active)
    rng = np.random.default_rng(9)
    st = rng.uniform(0.5, 1.0, (L, 1))
    sk = rng.uniform(1.0, 9.0, (L, 1))
    w = weights_of(st[:, 0], sk[:, 0])
    assert abs(w.mean() - 1) < 1e-12
    n = oracle_mod.allocate(st, sk, 10000, 0.1)[:, 0]
    assert np.abs(n - 10000 * 0.1 * w).max() < 1.0
    # all skewness negative -> that factor is 1 everywhere -> strength only decides
    n_neg = oracle_mod.allocate(st, -sk, 10000, 0.1)[:, 0]
    assert np.abs(n_neg - 10000 * 0.1 * 0.5 * (st[:, 0] / st.mean() + 1)).max() < 1.0


def test_budget_monotone_in_strength(oracle_mod):
    rng = np.random.default_rng(10)
    for _ in range(50):
        L = int(rng.integers(2, 12))
        st = rng.uniform(0.2, 1.0, (L, 1))
        sk = rng.uniform(0.5, 9.0, (L, 1))
        base = oracle_mod.allocate(st, sk, 500, 0.2)[:, 0]
        j = int(rng.integers(L))
        st2 = st.copy()
        st2[j] *= 1.5
        assert oracle_mod.allocate(st2, sk, 500, 0.2)[j, 0] >= base[j]


def test_budget_is_the_nearest_integer_apportionment_brute_force(oracle_mod):
    """Enumerate every integer vector with 0 <= n_l <= Nv and sum T: the oracle's answer is the one
    closest (L2 and L-infinity) to the continuous capped proportional shares, which are computed
    here by an independent bisection."""
    rng = np.random.default_rng(11)
    n_cases = 0
    for _ in range(60):
        L = int(rng.integers(2, 5))
        Nv = int(rng.integers(3, 9))
        ratio = float(rng.uniform(0.05, 0.95))
        st = rng.uniform(0.05, 1.0, (L, 1))
        sk = rng.uniform(-2.0, 12.0, (L, 1))
        T = math.floor(ratio * Nv * L + 0.5)
        w = weights_of(st[:, 0], sk[:, 0])
        share = waterfill(w, T, Nv)
        frac = share - np.floor(share)
        uncapped = share < Nv - 1e-9
        fr = np.sort(frac[uncapped])
        if len(fr) > 1 and np.min(np.diff(fr)) < 1e-6:
            continue                                           # a tie in the remainders: not unique
        got = oracle_mod.allocate(st, sk, Nv, ratio)[:, 0]
        best, best_d = None, None
        for cand in itertools.product(range(Nv + 1), repeat=L):
            if sum(cand) != T:
                continue
            dist = float(((np.array(cand) - share) ** 2).sum())
            if best_d is None or dist < best_d - 1e-12:
                best, best_d = cand, dist
        assert tuple(got) == best, (st.ravel(), sk.ravel(), Nv, ratio, share, got, best)
        assert np.abs(got - share).max() < 1 + 1e-9
        n_cases += 1
    assert n_cases > 40


def test_budget_cap_redistributes(oracle_mod):
    st = np.array([[10.0], [1.0], [1.0], [1.0]])
    sk = np.array([[10.0], [1.0], [1.0], [1.0]])
    n = oracle_mod.allocate(st, sk, 100, 0.5)[:, 0]            # T = 200; layer 0 would want ~154
    assert n[0] == 100 and n.sum() == 200
    assert n[1:].tolist() == [34, 33, 33]


# ----------------------------------------------------------------------------------------------
# top-k selection
# ----------------------------------------------------------------------------------------------
def test_select_brute_force_subsets(oracle_mod):
    rng = np.random.default_rng(12)
    for _ in range(40):
        n = int(rng.integers(3, 13))
        k = int(rng.integers(0, n + 1))
        s = rng.integers(0, 4, n).astype(np.float32) / 4        # many ties
        got = oracle_mod.select(s, k).tolist()
        best = None
        for sub in itertools.combinations(range(n), k):          # lexicographic order
            tot = float(s[list(sub)].sum())
            if best is None or tot > best[0] + 1e-12:
                best = (tot, sub)
        # among subsets of maximal sum, the lexicographically smallest is found first
        assert tuple(got) == best[1]


def test_select_equal_scores_and_planted_subset(oracle_mod):
    assert oracle_mod.select(np.full(20, 0.5, np.float32), 7).tolist() == list(range(7))
    rng = np.random.default_rng(13)
    s = rng.uniform(0, 0.5, 500).astype(np.float32)
    planted = np.sort(rng.choice(500, 37, replace=False))
    s[planted] += 1.0
    assert oracle_mod.select(s, 37).tolist() == planted.tolist()
    # library cross-check: stable argsort on (-score, index)
    s = rng.integers(0, 50, 3000).astype(np.float32)
    want = np.sort(np.lexsort((np.arange(3000), -s))[:411])
    assert oracle_mod.select(s, 411).tolist() == want.tolist()
    assert oracle_mod.select(s, 0).tolist() == []
    assert oracle_mod.select(s, 3000).tolist() == list(range(3000))
    # the two zeros are one value: among them the lower index wins whatever the sign (float comparison, as in
    # the library's stable sort on the values)
    assert oracle_mod.select(np.array([-0.0, 0.0, -0.0, 0.0], np.float32), 2).tolist() == [0, 1]
    z = np.where(rng.integers(0, 2, 400) == 1, np.float32(-0.0), np.float32(0.0)).astype(np.float32)
    z[rng.choice(400, 60, replace=False)] = rng.choice(np.array([1e-42, -1e-42, 0.5, -0.5], np.float32), 60)
    want = np.sort(np.lexsort((np.arange(400), -z))[:150])
    assert oracle_mod.select(z, 150).tolist() == want.tolist()


# ----------------------------------------------------------------------------------------------
# per-KV-group budgets (Eq. 8-11 and the second loop of Algorithm 1 applied to every KV head on its own)
# ----------------------------------------------------------------------------------------------
def test_group_scores_average_to_the_layer_score_and_match_the_matrix_form(oracle_mod):
    rng = np.random.default_rng(41)
    L, B, Hq, Hkv, d, Nv, Nt, W = 2, 2, 6, 3, 16, 33, 9, 5
    k, _, qw = rand_case(rng, L, B, Hq, Hkv, d, Nv, Nt, W)
    dm = oracle_mod.Dims(L, B, Hq, Hkv, d, Nv, Nt, W)
    scale = 1 / math.sqrt(d)
    whole = oracle_mod.score(dm, k, qw, scale, 0.7)
    grp = oracle_mod.score_groups(dm, k, qw, scale, 0.7)
    assert np.array_equal(whole["elite_mask"], grp["elite_mask"])
    # groups have equal size: the mean over the groups is the mean over all heads (one fp32 rounding apart)
    assert np.allclose(grp["scores"].astype(np.float64).mean(axis=2), whole["scores"], rtol=3e-7, atol=0)
    # and each group's score is the library-softmax matrix form averaged over that group's heads only
    kf, qf = bf16_val(k), bf16_val(qw)
    G = Hq // Hkv
    for l, b, g in itertools.product(range(L), range(B), range(Hkv)):
        acc = np.zeros(Nv)
        for h in range(g * G, (g + 1) * G):
            iv, _ = literal_importance(kf[l, b, g], qf[l, b, :, h, :], int(grp["elite_mask"][l, b, h]), Nv, Nt, W, scale)
            acc += iv
        assert np.allclose(grp["scores"][l, b, g], acc / G, rtol=2e-7, atol=0)
    # heads of different groups do not leak into each other: changing group 1's keys leaves group 0's score alone
    k2 = k.copy()
    k2[:, :, 1] = bf16_bits(rng.standard_normal(k2[:, :, 1].shape))
    grp2 = oracle_mod.score_groups(dm, k2, qw, scale, 0.7)
    assert np.array_equal(grp2["scores"][:, :, 0], grp["scores"][:, :, 0])
    assert not np.array_equal(grp2["scores"][:, :, 1], grp["scores"][:, :, 1])


def test_group_budgets_sum_cap_and_reduce_to_the_layer_rule(oracle_mod):
    rng = np.random.default_rng(42)
    L, B, Hkv, Nv = 5, 3, 4, 50
    for ratio in (0.0, 0.1, 0.37, 0.9, 1.0):
        st = rng.uniform(0.1, 1.0, (L, B, Hkv))
        sk = rng.uniform(-1.0, 6.0, (L, B, Hkv))
        bud = oracle_mod.allocate_groups(st, sk, Nv, ratio)
        assert bud.shape == (L, B, Hkv) and bud.min() >= 0 and bud.max() <= Nv
        T = oracle_mod.total_kept(Nv, L * Hkv, ratio)
        assert (bud.sum(axis=(0, 2)) == T).all()
        # a sequence's cells are apportioned exactly like the layers of a sequence with L * Hkv layers
        for b in range(B):
            flat = oracle_mod.allocate(st[:, b].reshape(L * Hkv, 1), sk[:, b].reshape(L * Hkv, 1), Nv, ratio)
            assert np.array_equal(bud[:, b].reshape(-1), flat[:, 0])
    # one KV head: the per-layer rule itself
    st, sk = rng.uniform(0.1, 1.0, (L, B, 1)), rng.uniform(0.0, 3.0, (L, B, 1))
    assert np.array_equal(oracle_mod.allocate_groups(st, sk, Nv, 0.3)[:, :, 0], oracle_mod.allocate(st[:, :, 0], sk[:, :, 0], Nv, 0.3))
    # equal cells: a uniform split with the spare rows on the lowest cells
    bud = oracle_mod.allocate_groups(np.ones((3, 1, 2)), np.ones((3, 1, 2)), 10, 0.45)   # T = 27 over 6 cells
    assert bud.reshape(-1).tolist() == [5, 5, 5, 4, 4, 4]


def test_group_compaction_keeps_each_heads_own_tokens_and_all_text(oracle_mod):
    rng = np.random.default_rng(43)
    L, B, Hq, Hkv, d, Nv, Nt, W = 2, 2, 4, 2, 16, 40, 6, 4
    k, v, qw = rand_case(rng, L, B, Hq, Hkv, d, Nv, Nt, W)
    dm = oracle_mod.Dims(L, B, Hq, Hkv, d, Nv, Nt, W)
    sc = oracle_mod.score_groups(dm, k, qw, 0.25, 0.9)["scores"]
    st, sk = oracle_mod.moments(sc)
    bud = oracle_mod.allocate_groups(st, sk, Nv, 0.25)
    slack = 2
    cc = oracle_mod.compact_groups(dm, slack, k, v, sc, bud)
    pos = 0
    for c in range(L * B * Hkv):
        l, b, g = c // Hkv // B, c // Hkv % B, c % Hkv
        n = int(bud[l, b, g])
        want = np.sort(np.lexsort((np.arange(Nv), -sc[l, b, g]))[:n])     # library sort: top n, ties to the lower index
        assert cc["kept_idx"][pos:pos + n].tolist() == want.tolist()
        a = int(cc["offsets"][c])
        assert int(cc["lens"][c]) == n + Nt and int(cc["offsets"][c + 1]) - a == n + Nt + slack
        assert np.array_equal(cc["k"][a:a + n, 0], k[l, b, g, want])
        assert np.array_equal(cc["v"][a:a + n, 0], v[l, b, g, want])
        assert np.array_equal(cc["k"][a + n:a + n + Nt, 0], k[l, b, g, Nv:])
        assert np.array_equal(cc["v"][a + n:a + n + Nt, 0], v[l, b, g, Nv:])
        pos += n
    # full retention: decode over the per-group cache equals decode over the full cache
    bud1 = np.full((L, B, Hkv), Nv, np.int32)
    c1 = oracle_mod.compact_groups(dm, 0, k, v, sc, bud1)
    q = bf16_bits(rng.standard_normal((L, B, Hq, d)))
    got = oracle_mod.decode(oracle_mod.group_decode_dims(dm), c1["k"], c1["v"], c1["offsets"], c1["lens"],
                            q.reshape(L * B * Hkv, 1, Hq // Hkv, d), 0.25).reshape(L, B, Hq, d)
    N = Nv + Nt
    kf = np.ascontiguousarray(k.transpose(0, 1, 3, 2, 4)).reshape(L * B * N, Hkv, d)
    vf = np.ascontiguousarray(v.transpose(0, 1, 3, 2, 4)).reshape(L * B * N, Hkv, d)
    want = oracle_mod.decode(dm, kf, vf, (np.arange(L * B + 1) * N).astype(np.int64), np.full(L * B, N, np.int32), q, 0.25)
    assert np.allclose(got, want, rtol=1e-6, atol=1e-7)


# ----------------------------------------------------------------------------------------------
# compaction and decode
# ----------------------------------------------------------------------------------------------
def small_pipeline(oracle_mod, ratio, slack=0, seed=14):
    rng = np.random.default_rng(seed)
    L, B, Hq, Hkv, d, Nv, Nt, W = 3, 2, 4, 2, 16, 40, 8, 4
    k, v, qw = rand_case(rng, L, B, Hq, Hkv, d, Nv, Nt, W)
    dm = oracle_mod.Dims(L, B, Hq, Hkv, d, Nv, Nt, W)
    sc = oracle_mod.score(dm, k, qw, 0.25, 0.9)["scores"]
    st, sk = oracle_mod.moments(sc)
    bud = oracle_mod.allocate(st, sk, Nv, ratio)
    cc = oracle_mod.compact(dm, slack, k, v, sc, bud)
    return dm, k, v, sc, bud, cc, rng


@pytest.mark.parametrize("slack", [0, 3])
def test_compact_text_kept_indices_ascending(oracle_mod, slack):
    dm, k, v, sc, bud, cc, _ = small_pipeline(oracle_mod, 0.3, slack)
    L, B, Nv, Nt = dm.n_layers, dm.batch, dm.n_visual, dm.n_text
    pos = 0
    for l in range(L):
        for b in range(B):
            r = l * B + b
            n = int(bud[l, b])
            off = int(cc["offsets"][r])
            assert cc["lens"][r] == n + Nt
            kept = cc["kept_idx"][pos:pos + n]
            pos += n
            assert (np.diff(kept) > 0).all() and kept.min() >= 0 and kept.max() < Nv
            # kept set = top-n by (score desc, index asc), via a library sort
            want = np.sort(np.lexsort((np.arange(Nv), -sc[l, b]))[:n])
            assert kept.tolist() == want.tolist()
            for g in range(dm.n_kv_heads):
                assert np.array_equal(cc["k"][off:off + n, g], k[l, b, g, kept])
                assert np.array_equal(cc["v"][off:off + n, g], v[l, b, g, kept])
                # every text row survives, in order, byte-identical
                assert np.array_equal(cc["k"][off + n:off + n + Nt, g], k[l, b, g, Nv:])
                assert np.array_equal(cc["v"][off + n:off + n + Nt, g], v[l, b, g, Nv:])
            assert cc["offsets"][r + 1] - off == n + Nt + slack
    assert cc["offsets"][-1] == cc["k"].shape[0]


def test_full_retention_is_identity(oracle_mod):
    dm, k, v, sc, bud, cc, _ = small_pipeline(oracle_mod, 1.0)
    N = dm.n_visual + dm.n_text
    assert (bud == dm.n_visual).all()
    want_k = k.transpose(0, 1, 3, 2, 4).reshape(-1, dm.n_kv_heads, dm.head_dim)
    want_v = v.transpose(0, 1, 3, 2, 4).reshape(-1, dm.n_kv_heads, dm.head_dim)
    assert np.array_equal(cc["k"], want_k) and np.array_equal(cc["v"], want_v)
    assert (cc["lens"] == N).all()


def dense_masked_attention(kf, vf, qf, keep_mask, scale, G):
    """Textbook attention over the FULL cache with -inf on evicted positions (library softmax)."""
    Hq = qf.shape[0]
    out = np.zeros((Hq, kf.shape[-1]))
    for h in range(Hq):
        g = h // G
        logits = torch.from_numpy(kf[g] @ qf[h] * scale)
        logits[~torch.from_numpy(keep_mask)] = -float("inf")
        p = torch.softmax(logits, 0).numpy()
        out[h] = p @ vf[g]
    return out


@pytest.mark.parametrize("ratio", [0.2, 1.0])
def test_decode_equals_masked_dense_attention(oracle_mod, ratio):
    dm, k, v, sc, bud, cc, rng = small_pipeline(oracle_mod, ratio, slack=2)
    L, B, Hq, Hkv, d, Nv, Nt = dm.n_layers, dm.batch, dm.n_q_heads, dm.n_kv_heads, dm.head_dim, dm.n_visual, dm.n_text
    q = bf16_bits(rng.standard_normal((L, B, Hq, d)))
    out = oracle_mod.decode(dm, cc["k"], cc["v"], cc["offsets"], cc["lens"], q, 0.25)
    kf, vf, qf = bf16_val(k), bf16_val(v), bf16_val(q)
    pos = 0
    for l in range(L):
        for b in range(B):
            n = int(bud[l, b])
            keep = np.zeros(Nv + Nt, bool)
            keep[cc["kept_idx"][pos:pos + n]] = True
            keep[Nv:] = True
            pos += n
            want = dense_masked_attention(kf[l, b], vf[l, b], qf[l, b], keep, 0.25, Hq // Hkv)
            assert np.allclose(out[l, b], want, rtol=1e-6, atol=1e-7)


def test_decode_library_sdpa_one_row_and_convexity(oracle_mod):
    rng = np.random.default_rng(15)
    L, B, Hq, Hkv, d = 1, 1, 4, 2, 16
    dm = oracle_mod.Dims(L, B, Hq, Hkv, d, 5, 2, 1)
    rows = 33
    kc = bf16_bits(rng.standard_normal((rows, Hkv, d)))
    vc = bf16_bits(rng.standard_normal((rows, Hkv, d)))
    q = bf16_bits(rng.standard_normal((L, B, Hq, d)))
    offsets = np.array([0, rows], np.int64)
    out = oracle_mod.decode(dm, kc, vc, offsets, np.array([rows], np.int32), q, 0.25)
    kt = torch.from_numpy(bf16_val(kc)).permute(1, 0, 2).repeat_interleave(2, 0)[None]     # [1,Hq,rows,d]
    vt = torch.from_numpy(bf16_val(vc)).permute(1, 0, 2).repeat_interleave(2, 0)[None]
    qt = torch.from_numpy(bf16_val(q))[0, 0][None, :, None, :]                               # [1,Hq,1,d]
    ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, scale=0.25)[0, :, 0].numpy()
    assert np.allclose(out[0, 0], ref, rtol=1e-6, atol=1e-7)
    vf = bf16_val(vc)
    for h in range(Hq):
        g = h // 2
        assert (out[0, 0, h] <= vf[:, g].max(0) + 1e-6).all() and (out[0, 0, h] >= vf[:, g].min(0) - 1e-6).all()
    # one-row cache: the output is that V row
    out1 = oracle_mod.decode(dm, kc, vc, offsets, np.array([1], np.int32), q, 0.25)
    for h in range(Hq):
        assert np.array_equal(out1[0, 0, h], bf16_val(vc)[0, h // 2].astype(np.float32))


# ----------------------------------------------------------------------------------------------
# the synthetic workload end to end (oracle only)
# ----------------------------------------------------------------------------------------------
def test_planted_relevance_is_recovered_on_tiny_config(oracle_mod):
    wl = CONFIGS["c1"].with_(amp_lo=6.0, amp_hi=8.0)
    K, V, Qw = full_cache(wl, "k"), full_cache(wl, "v"), window_queries(wl)
    dm = dims_of(oracle_mod, wl)
    kl, vl = to_u16(K).transpose(0, 1, 3, 2, 4), to_u16(V).transpose(0, 1, 3, 2, 4)
    sc = oracle_mod.score(dm, kl, to_u16(Qw), wl.scale, wl.alpha)["scores"]
    st, sk = oracle_mod.moments(sc)
    assert (st > 0).all() and (st <= 1).all() and (sk > 0).all()      # right-skewed "head effect"
    bud = oracle_mod.allocate(st, sk, wl.n_visual, wl.ratio)
    assert bud.sum() == round(wl.ratio * wl.n_visual * wl.n_layers) == 230
    cc = oracle_mod.compact(dm, 0, kl, vl, sc, bud)
    pl = plan(wl)
    pos = 0
    for l in range(wl.n_layers):
        n = int(bud[l, 0])
        kept = set(cc["kept_idx"][pos:pos + n].tolist())
        pos += n
        planted = set(np.nonzero(pl.planted[l, 0])[0].tolist())
        assert len(planted) == 28
        if n >= len(planted):
            assert planted <= kept
        else:
            assert kept <= planted
    # text rows of every layer are the full text block
    for l in range(wl.n_layers):
        off, n = int(cc["offsets"][l]), int(bud[l, 0])
        assert np.array_equal(cc["k"][off + n:off + n + wl.n_text], to_u16(K)[l, 0, wl.n_visual:])
    q = decode_queries(wl, 0)
    out = oracle_mod.decode(dm, cc["k"], cc["v"], cc["offsets"], cc["lens"], to_u16(q), wl.scale)
    assert np.isfinite(out).all()


def test_generator_is_sliceable_and_deterministic():
    wl = CONFIGS["c1"]
    K = full_cache(wl, "k")
    K2 = full_cache(wl, "k", layers=[2], seqs=[0])
    assert torch.equal(K[2:3], K2)
    assert torch.equal(window_queries(wl)[1:2], window_queries(wl, layers=[1]))
    x = K.float()
    assert abs(float(x.mean())) < 0.02 and abs(float(x[:, :, wl.n_visual:].std()) - 1) < 0.02
    assert not torch.equal(decode_queries(wl, 0), decode_queries(wl, 1))
