"""Pins for the oracle's building blocks: each is checked against something other
than itself -- published vectors, closed forms, scipy/numpy library routines, brute
force on tiny inputs, textbook identities."""
import math
import os

import numpy as np
import pytest
import scipy.special as sps
import scipy.stats as sst

from oracle import oracle as orc
from paper_2511_02017_b200.synth_inputs import bf16_bits_from_float

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ Philox
def test_philox_known_answers():
    n = 0
    for line in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        out = orc.philox4x32_10(w[0:4], w[4:6])
        assert [int(x) for x in out] == w[6:10]
        n += 1
    assert n == 3


def test_rng_counter_layout_and_uniform_mapping():
    seed = 0x1234567890ABCDEF
    # counter = (seq, round, pos, purpose | arm<<4 | draw<<8), key = (seed lo, seed hi)
    raw = orc.philox4x32_10([7, 11, 3, 2 | (5 << 4) | (9 << 8)], [seed & 0xFFFFFFFF, seed >> 32])
    for word in range(4):
        k = orc.rng_u24(seed, 7, 11, 3, 2, 5, 9, word)
        assert k == int(raw[word]) >> 8
        u = orc.rng_uniform(seed, 7, 11, 3, 2, 5, 9, word)
        assert u == k / 2.0 ** 24 and 0.0 <= u < 1.0
    # streams differ in every counter field
    base = orc.rng_u24(seed, 7, 11, 3, 2)
    assert len({base, orc.rng_u24(seed, 8, 11, 3, 2), orc.rng_u24(seed, 7, 12, 3, 2),
                orc.rng_u24(seed, 7, 11, 4, 2), orc.rng_u24(seed, 7, 11, 3, 1),
                orc.rng_u24(seed + 1, 7, 11, 3, 2)}) == 6


def test_rng_uniformity():
    u = np.array([orc.rng_uniform(5, s, 0, 0, orc.RNG_DRAFT) for s in range(20000)])
    assert sst.kstest(u, "uniform").pvalue > 1e-3
    assert abs(u.mean() - 0.5) < 0.01


# --------------------------------------------------------------- row stats
def test_uniform_row_closed_form():
    for V in (1, 2, 7, 1000):
        st = orc.row_stats(np.full(V, 1.25, np.float32))
        assert st.valid
        assert st.p1 == pytest.approx(1.0 / V, rel=1e-14)
        if V > 1:
            assert st.p2 == pytest.approx(1.0 / V, rel=1e-14)
        assert st.H == pytest.approx(math.log(V), rel=1e-13, abs=1e-15)
        assert st.lse == pytest.approx(1.25 + math.log(V), rel=1e-14)
        assert st.argmax == 0


def test_one_hot_over_zeros_closed_form():
    V, L, j = 501, 3.5, 17
    z = np.zeros(V, np.float32)
    z[j] = L
    st = orc.row_stats(z)
    Wn = math.exp(L) + V - 1
    p1, po = math.exp(L) / Wn, 1.0 / Wn
    assert st.argmax == j
    assert st.m == L
    assert st.p1 == pytest.approx(p1, rel=1e-13)
    assert st.p2 == pytest.approx(po, rel=1e-13)
    assert st.lse == pytest.approx(math.log(Wn), rel=1e-13)
    assert st.H == pytest.approx(-(p1 * math.log(p1) + (V - 1) * po * math.log(po)), rel=1e-12)


def test_two_level_row_and_ties():
    z = np.array([0.0, 2.0, 2.0, -1.0, 0.0], np.float32)
    st = orc.row_stats(z)
    W = 2 * math.exp(2) + 2 + math.exp(-1)
    assert st.p1 == pytest.approx(math.exp(2) / W, rel=1e-14)
    assert st.p2 == st.p1                       # duplicated maximum: second largest element equals it
    assert st.argmax == 1                       # lowest index of the maximum


def test_shift_invariance_and_temperature():
    rng = np.random.default_rng(0)
    z = rng.normal(size=300).astype(np.float32) * 2
    a = orc.row_stats(z)
    b = orc.row_stats(z + np.float32(8.0))       # exact in fp32 for these magnitudes? compare loosely
    assert b.p1 == pytest.approx(a.p1, rel=1e-6) and b.H == pytest.approx(a.H, rel=1e-6)
    assert b.lse - a.lse == pytest.approx(8.0, abs=1e-5)
    # temperature: inv_T scales the logits (as a float32 value) before the softmax
    t = np.float32(1.0 / 0.7)
    c = orc.row_stats(z, inv_T=t)
    s = z.astype(np.float64) * float(t)
    q = sps.softmax(s)
    assert c.p1 == pytest.approx(q.max(), rel=1e-13)
    assert c.lse == pytest.approx(sps.logsumexp(s), rel=1e-13)
    assert c.H == pytest.approx(sst.entropy(q), rel=1e-12)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_row_stats_against_scipy(dtype):
    rng = np.random.default_rng(1)
    for V in (2, 33, 1000, 4099):
        z = (rng.normal(size=V) * 3 - 1.1 * np.log1p(rng.permutation(V))).astype(np.float32)
        if dtype == "bf16":
            row = bf16_bits_from_float(z)
            zz = (row.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
        else:
            row, zz = z, z.astype(np.float64)
        st, w = orc.row_stats(row, want_w=True)
        q = sps.softmax(zz)
        srt = np.sort(q)
        assert st.m == zz.max() and st.argmax == int(np.argmax(zz))
        assert st.lse == pytest.approx(sps.logsumexp(zz), rel=1e-13)
        assert st.p1 == pytest.approx(srt[-1], rel=1e-12)
        assert st.p2 == pytest.approx(srt[-2], rel=1e-12)
        assert st.H == pytest.approx(sst.entropy(q), rel=1e-11)
        np.testing.assert_allclose(w, np.exp(zz - zz.max()), rtol=1e-14)
        assert st.W == pytest.approx(np.exp(zz - zz.max()).sum(), rel=1e-13)


def test_minus_inf_entries_and_invalid_rows():
    z = np.array([0.0, -np.inf, 1.0, -np.inf], np.float32)
    st, w = orc.row_stats(z, want_w=True)
    assert st.valid and w[1] == 0.0 and w[3] == 0.0
    assert st.p1 == pytest.approx(math.e / (1 + math.e), rel=1e-14)
    assert not orc.row_stats(np.array([0.0, np.nan, 1.0], np.float32)).valid
    assert not orc.row_stats(np.full(5, -np.inf, np.float32)).valid
    assert not orc.row_stats(np.array([0.0, np.inf], np.float32)).valid


# ---------------------------------------------------------------- sampling
def _brute_sample(w, u):
    c = 0.0
    tot = 0.0
    for x in w:
        tot += x
    for j, x in enumerate(w):
        c += x
        if c > u * tot:
            return j
    return max(j for j, x in enumerate(w) if x > 0)


def test_sample_cdf_brute_force_tiny():
    rng = np.random.default_rng(2)
    for _ in range(200):
        V = int(rng.integers(1, 9))
        w = rng.random(V)
        w[rng.random(V) < 0.3] = 0.0
        if w.sum() == 0:
            w[0] = 1.0
        tot = float(np.add.reduce(w))
        tot = 0.0
        for x in w:
            tot += x
        for u in (0.0, 0.25, 0.5, 0.999999, float(rng.random())):
            x, lo, hi = orc.sample_cdf(w, tot, u)
            assert x == _brute_sample(w, u)
            assert w[x] > 0 and w[lo] > 0 and w[hi] > 0
            assert lo <= x <= hi


def test_sample_cdf_boundaries_and_tolerance_band():
    w = np.array([0.25, 0.0, 0.25, 0.5])
    assert orc.sample_cdf(w, 1.0, 0.0)[0] == 0
    assert orc.sample_cdf(w, 1.0, 0.25)[0] == 2          # c_0 = 0.25 is not > 0.25; token 1 has no mass
    assert orc.sample_cdf(w, 1.0, 0.4999)[0] == 2
    assert orc.sample_cdf(w, 1.0, 0.5)[0] == 3
    x, lo, hi = orc.sample_cdf(w, 1.0, 0.25 - 5e-7, tol=1e-6)
    assert (x, lo, hi) == (0, 0, 2)
    x, lo, hi = orc.sample_cdf(w, 1.0, 0.6, tol=1e-6)
    assert (x, lo, hi) == (3, 3, 3)


def test_sample_cdf_chi_square():
    rng = np.random.default_rng(3)
    V, n = 12, 120000
    w = rng.random(V) ** 3
    w[4] = 0.0
    tot = 0.0
    for x in w:
        tot += x
    cnt = np.zeros(V)
    for s in range(n):
        u = orc.rng_uniform(99, s, 0, 0, orc.RNG_DRAFT)
        cnt[orc.sample_cdf(w, tot, u)[0]] += 1
    assert cnt[4] == 0
    keep = w > 0
    chi = sst.chisquare(cnt[keep], n * w[keep] / tot)
    assert chi.pvalue > 1e-4


# ------------------------------------------------------------------- rules
def test_rule_thresholds_strict():
    e = 1e-9
    R = orc
    # Max-Confidence: stop iff p1 < 0.8
    assert R.rule_stop(R.RULE_MAXCONF, 0.8 - e, 0.1, 1.0)[0] is True
    assert R.rule_stop(R.RULE_MAXCONF, 0.8, 0.1, 1.0)[0] is False
    assert R.rule_stop(R.RULE_MAXCONF, 0.8 + e, 0.1, 1.0)[0] is False
    # SVIP: stop iff sqrt(H) > 0.6  (H = 0.36)
    assert R.rule_stop(R.RULE_SVIP, 0.5, 0.1, 0.36 + e)[0] is True
    assert R.rule_stop(R.RULE_SVIP, 0.5, 0.1, 0.36 - e)[0] is False
    # AdaEDL: stop iff 1 - sqrt(gamma*H) < lambda ; gamma = 0.2, lambda = 0.4 -> H > 1.8
    assert R.rule_stop(R.RULE_ADAEDL, 0.5, 0.1, 1.8 + 1e-6, lam=0.4)[0] is True
    assert R.rule_stop(R.RULE_ADAEDL, 0.5, 0.1, 1.8 - 1e-6, lam=0.4)[0] is False
    # SVIPDifference: stop iff sqrt(H_t) - sqrt(H_{t-1}) > 0.2, never at the first position
    assert R.rule_stop(R.RULE_SVIPDIFF, 0.5, 0.1, 1.0, sqrtH_prev=0.8 - e, has_prev=1)[0] is True
    assert R.rule_stop(R.RULE_SVIPDIFF, 0.5, 0.1, 1.0, sqrtH_prev=0.8 + e, has_prev=1)[0] is False
    assert R.rule_stop(R.RULE_SVIPDIFF, 0.5, 0.1, 9.0, sqrtH_prev=0.0, has_prev=0) == (False, False)
    # LogitMargin: stop iff p1 - p2 < 0.2
    assert R.rule_stop(R.RULE_MARGIN, 0.5, 0.3 + e, 1.0)[0] is True
    assert R.rule_stop(R.RULE_MARGIN, 0.5, 0.3 - e, 1.0)[0] is False
    # fixed-length arm never stops
    assert R.rule_stop(R.RULE_STATIC, 0.0, 0.0, 50.0) == (False, False)


def test_rule_near_flag():
    assert orc.rule_stop(orc.RULE_MAXCONF, 0.8 - 5e-7, 0.0, 1.0)[1] is True
    assert orc.rule_stop(orc.RULE_MAXCONF, 0.8 - 5e-6, 0.0, 1.0)[1] is False
    assert orc.rule_stop(orc.RULE_SVIP, 0.1, 0.0, (0.6 + 5e-7) ** 2)[1] is True


def test_adaedl_lambda_trajectory_by_hand():
    # as printed: lambda' = b2*lambda + (1-b2)*(lambda + eps*sign(alpha - r)) = lambda + (1-b2)*eps*sign(.)
    lam, acc = 0.4, 1.0
    script = [(1, 4), (4, 4), (9, 10), (0, 3), (2, 2)]     # (accepted, drafted); alpha = 0.9
    exp_lam, exp_acc = 0.4, 1.0
    for a, n in script:
        lam, acc = orc.adaedl_update(lam, acc, a, n)
        r = a / n
        sgn = 1 if 0.9 > r else (-1 if 0.9 < r else 0)
        exp_lam = exp_lam + 0.1 * 0.01 * sgn
        exp_acc = 0.5 * exp_acc + 0.5 * r
        assert lam == pytest.approx(exp_lam, rel=1e-14)
        assert acc == pytest.approx(exp_acc, rel=1e-14)
    # signs were +, -, 0, +, - : net zero
    assert lam == pytest.approx(0.4, rel=1e-13)


# ----------------------------------------------------------------- rewards
def test_rewards_exact_rationals():
    assert orc.reward_simple(3, 8) == 0.375
    assert orc.reward_blend(3, 4, 8) == 0.5625            # 0.5*3/8 + 0.5*3/4
    assert orc.reward_blend(8, 8, 8) == 1.0
    assert orc.reward_blend(0, 5, 8) == 0.0
    assert orc.reward_blend(2, 4, 16, alpha=0.25) == 0.25 * 0.125 + 0.75 * 0.5
    for n in range(1, 9):
        for a in range(0, n + 1):
            assert 0.0 <= orc.reward_blend(a, n, 8) <= 1.0


# ------------------------------------------------------------------ bandits
def test_ucb1_unplayed_first_and_hand_indices():
    assert orc.ucb1_select([0, 0, 0], [0, 0, 0])[0] == 0
    assert orc.ucb1_select([1, 0, 0], [0.3, 0, 0])[0] == 1
    assert orc.ucb1_select([1, 2, 0], [0.3, 0.1, 0])[0] == 2
    N, R = [3, 1, 2], [1.5, 0.9, 0.2]
    a, idx, mk = orc.ucb1_select(N, R)
    t = 1 + sum(N)
    want = [R[i] / N[i] + math.sqrt(2 * math.log(t) / N[i]) for i in range(3)]
    np.testing.assert_allclose(idx, want, rtol=1e-14)
    assert a == int(np.argmax(want)) and mk == 1 << a
    # exact tie goes to the lowest index, and both arms are within the band
    a, idx, mk = orc.ucb1_select([2, 2], [1.0, 1.0])
    assert a == 0 and mk == 0b11


def test_ucb1_bernoulli_counts_and_regret():
    # Auer et al. 2002, Thm 1: E[N_a] <= 8 ln T / Delta_a^2 + 1 + pi^2/3 for sub-optimal arms.
    mus = [0.8, 0.6, 0.3]
    T, runs = 4000, 12
    rng = np.random.default_rng(7)
    counts = np.zeros((runs, 3))
    for r in range(runs):
        N = np.zeros(3, np.uint32)
        R = np.zeros(3)
        for _ in range(T):
            a = orc.ucb1_select(N, R)[0]
            N[a] += 1
            R[a] += float(rng.random() < mus[a])
        assert N.sum() == T
        counts[r] = N
    mean = counts.mean(axis=0)
    for a in (1, 2):
        d = mus[0] - mus[a]
        assert mean[a] <= 8 * math.log(T) / d ** 2 + 1 + math.pi ** 2 / 3
    assert mean[0] > 0.6 * T
    regret = sum((mus[0] - mus[a]) * mean[a] for a in range(3))
    assert regret < sum(8 * math.log(T) / (mus[0] - mus[a]) for a in (1, 2)) + (1 + math.pi ** 2 / 3) * 0.7


def test_ucb_tuned_hand_indices():
    N, R, R2 = [4, 2, 3], [2.0, 1.5, 0.6], [1.2, 1.25, 0.2]
    a, idx, _ = orc.ucb_tuned_select(N, R, R2)
    t = 1 + sum(N)
    want = []
    for i in range(3):
        mu = R[i] / N[i]
        var = R2[i] / N[i] - mu * mu
        Va = var + math.sqrt(2 * math.log(t) / N[i])
        want.append(mu + math.sqrt(math.log(t) / N[i] * min(0.25, Va)))
    np.testing.assert_allclose(idx, want, rtol=1e-14)
    assert a == int(np.argmax(want))


def test_beta_order_statistic_matches_beta_cdf():
    # Beta(a, b) for integer a, b is the a-th smallest of a+b-1 uniforms.
    for (a, b) in [(1, 1), (3, 2), (1, 9), (20, 5)]:
        x = np.array([orc.beta_order_stat(a, b, 11, s, 0, 0, 0) for s in range(4000)]) / 2.0 ** 24
        assert sst.kstest(x, sst.beta(a, b).cdf).pvalue > 1e-3
    # brute force: sort the same uniforms by hand (uniform j = word j%4 of draw j//4)
    a, b = 4, 6
    us = sorted(orc.rng_u24(11, 5, 2, 3, orc.RNG_BANDIT, arm=1, draw=j // 4, word=j % 4) for j in range(a + b - 1))
    assert orc.beta_order_stat(a, b, 11, 5, 2, 3, 1) == us[a - 1]


def test_ts_beta_posterior_and_concentration():
    # posterior parameters are 1 + successes, 1 + failures (Beta(1,1) prior)
    N, R = np.array([10, 4], np.uint32), np.array([7.0, 1.0])
    a, smp = orc.ts_beta_select(N, R, 3, 0, 0, 0)
    assert smp[0] == orc.beta_order_stat(1 + 7, 1 + 3, 3, 0, 0, 0, 0)
    assert smp[1] == orc.beta_order_stat(1 + 1, 1 + 3, 3, 0, 0, 0, 1)
    assert a == int(np.argmax(smp))
    mus = [0.75, 0.4, 0.2]
    rng = np.random.default_rng(5)
    N = np.zeros(3, np.uint32)
    R = np.zeros(3)
    for t in range(600):
        a = orc.ts_beta_select(N, R, 17, 0, t, 0)[0]
        N[a] += 1
        R[a] += float(rng.random() < mus[a])
    assert N.sum() == 600 and N[0] > 450


def test_ts_gauss_posterior_and_moments():
    # mu0 = 0, var0 = 1, noise = 1  =>  posterior N(R/(N+1), 1/(N+1))
    N, R = np.array([3, 0], np.uint32), np.array([2.4, 0.0])
    smp = np.array([orc.ts_gauss_select(N, R, 21, s, 0)[1] for s in range(20000)])
    assert smp[:, 0].mean() == pytest.approx(2.4 / 4, abs=0.02)
    assert smp[:, 0].var() == pytest.approx(1 / 4, rel=0.05)
    assert smp[:, 1].mean() == pytest.approx(0.0, abs=0.03)
    assert smp[:, 1].var() == pytest.approx(1.0, rel=0.05)
    z = (smp[:, 1])
    assert sst.kstest(z, "norm").pvalue > 1e-3
    # Box-Muller from the two uniforms of arm a's Philox call, general prior
    a, s, _ = orc.ts_gauss_select(N, R, 21, 4, 9, mu0=0.5, var0=2.0, noise_var=0.25)
    for arm in range(2):
        u1 = orc.rng_uniform(21, 4, 9, 0, orc.RNG_BANDIT, arm, 0, 0)
        u2 = orc.rng_uniform(21, 4, 9, 0, orc.RNG_BANDIT, arm, 0, 1)
        zz = math.sqrt(-2 * math.log(1 - u1)) * math.cos(2 * math.pi * u2)
        var_n = 1 / (1 / 2.0 + N[arm] / 0.25)
        mu_n = var_n * (0.5 / 2.0 + R[arm] / 0.25)
        assert s[arm] == pytest.approx(mu_n + math.sqrt(var_n) * zz, rel=1e-12, abs=1e-14)
    assert a == int(np.argmax(s))
