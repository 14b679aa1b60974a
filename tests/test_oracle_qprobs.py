"""Pins for the oracle's verification when the draft distributions arrive as normalised fp32 probabilities
(instead of logits): hand-computed ratios and residuals, the speculative-sampling identities with an
arbitrary probability vector q, and agreement with the logits format on the same distributions."""
import numpy as np
import scipy.special as sps
import scipy.stats as sst

from oracle import oracle as orc


def _logits_from_probs(p):
    with np.errstate(divide="ignore"):
        return np.log(np.asarray(p, dtype=np.float64)).astype(np.float32)


def test_hand_computed_ratio_and_residual():
    p = np.array([0.5, 0.3, 0.2])
    q = np.array([[0.25, 0.5, 0.25]], np.float32)                   # exact in fp32
    P = np.tile(_logits_from_probs(p), (2, 1))
    n_acc = {0: 0, 1: 0, 2: 0}
    for seq in range(4000):
        u = orc.rng_uniform(3, seq, 0, 0, orc.RNG_ACCEPT)
        for x, ratio in ((0, 2.0), (1, 0.6), (2, 0.8)):             # p(x) / q(x)
            out = orc.verify_sequence_qprobs(q, P, [x], seed=3, seq=seq, rnd=0)
            if abs(u - ratio) < 1e-5:
                continue
            assert out.accept_len == (1 if u < ratio else 0)
            n_acc[x] += out.accept_len
            if out.accept_len == 0:
                assert out.next_token == 0                           # max(0, p - q) = [0.25, 0, 0]
    assert n_acc[0] > n_acc[2] > n_acc[1] > 0


def test_zero_draft_probability():
    P = np.tile(_logits_from_probs([0.5, 0.5, 0.0]), (2, 1))
    q = np.array([[0.0, 1.0, 0.0]], np.float32)
    for seq in range(50):
        assert orc.verify_sequence_qprobs(q, P, [0], seed=1, seq=seq, rnd=0).accept_len == 1   # p > 0 = q: ratio inf
        out = orc.verify_sequence_qprobs(q, P, [2], seed=1, seq=seq, rnd=0)                     # 0 / 0: rejected
        assert out.accept_len == 0 and out.next_token == 0                                     # residual [0.5, 0, 0]


def test_acceptance_frequency_and_first_token_distribution():
    rng = np.random.default_rng(2)
    V = 9
    zp = (rng.normal(size=V) * 1.5).astype(np.float32)
    p = sps.softmax(zp.astype(np.float64))
    q = rng.dirichlet(np.ones(V)).astype(np.float32)
    q64 = q.astype(np.float64)
    P = np.stack([zp, zp])
    N = 60000
    acc = 0
    first = np.zeros(V)
    for seq in range(N):
        u = orc.rng_uniform(7, seq, 5, 0, orc.RNG_DRAFT)
        x = int(np.searchsorted(np.cumsum(q64), u * q64.sum(), side="right"))   # x ~ q, drawn here
        x = min(x, V - 1)
        out = orc.verify_sequence_qprobs(q[None], P, [x], seed=7, seq=seq, rnd=5)
        acc += out.accept_len
        first[x if out.accept_len else out.next_token] += 1
    want = np.minimum(p, q64 / q64.sum()).sum()                      # textbook: P(accept) = sum min(p, q)
    assert abs(acc / N - want) < 4 * np.sqrt(want * (1 - want) / N)
    assert sst.chisquare(first, N * p).pvalue > 1e-4                 # the emitted token is distributed as p


def test_agrees_with_the_logits_format():
    rng = np.random.default_rng(3)
    V, n = 40, 5
    diff = 0
    for seq in range(300):
        zq = (rng.normal(size=(n, V)) * 2).astype(np.float32)
        zp = (zq + rng.normal(size=(n, V)) * 0.7).astype(np.float32)
        zp = np.concatenate([zp, rng.normal(size=(1, V)).astype(np.float32)])
        q = sps.softmax(zq.astype(np.float64), axis=1).astype(np.float32)
        x = [int(rng.choice(V, p=sps.softmax(zq[i].astype(np.float64)))) for i in range(n)]
        lse = [orc.row_stats(zq[i]).lse for i in range(n)]
        a = orc.verify_sequence(zq, zp, x, lse, seed=11, seq=seq, rnd=2)
        b = orc.verify_sequence_qprobs(q, zp, x, seed=11, seq=seq, rnd=2)
        if a.near_accept or b.near_accept:
            continue
        assert a.accept_len == b.accept_len
        if a.next_token != b.next_token:                             # fp32 rounding of q moves a CDF boundary: within the band
            assert a.next_lo <= b.next_token <= a.next_hi
            diff += 1
    assert diff <= 3


def test_engine_uses_the_probabilities():
    rng = np.random.default_rng(4)
    S, V, K = 5, 64, 3
    o = orc.Oracle(S, V, K, 1, orc.UCB1, orc.SEQ, dtype=orc.FP32, seed=6, arms=[orc.RULE_STATIC], q_format=1)
    T = (rng.normal(size=(S, K + 1, V)) * 2).astype(np.float32)
    D = T[:, :K].copy()
    toks = np.full((S, K), -1, np.int32)
    for i in range(K):
        toks[:, i] = o.draft_step(D[:, i])["token"]
    Q = np.zeros((S, K, V), np.float32)
    Q[np.arange(S)[:, None], np.arange(K)[None, :], toks] = 1.0     # q = delta on the drafted token: ratio = p(x) <= 1
    v = o.verify(Q, T, toks)
    p = sps.softmax(T.astype(np.float64), axis=2)
    for s in range(S):
        a = 0
        for i in range(K):
            u = orc.rng_uniform(6, s, 0, i, orc.RNG_ACCEPT)
            if not u < p[s, i, toks[s, i]]:
                break
            a += 1
        assert v["accept_len"][s] == a
        if a < K:
            assert v["next_token"][s] != toks[s, a]                  # the residual is p with the drafted token removed


def test_residual_band_is_measured_in_probability():
    """The set of acceptable residual draws is what a running sum off by 1e-6 of probability could give: with a
    residual mass of 1e-3 that is a thousandth of the mass, not a millionth."""
    p = np.array([0.4, 0.3, 0.3, 0.0])
    q = np.array([[0.3994, 0.2996, 0.3, 0.001]], np.float32)        # residual [6e-4, 4e-4, 0, 0]; token 3 is always rejected
    P = np.tile(_logits_from_probs(p), (2, 1))
    seen = set()
    for seq in range(40000):
        u = orc.rng_uniform(5, seq, 0, 0, orc.RNG_RESAMPLE)
        if 0.6002 < u < 0.6008:
            kind, want = "just above", (1, 0, 1)
        elif 0.5992 < u < 0.5998:
            kind, want = "just below", (0, 0, 1)
        elif 0.30 < u < 0.31:
            kind, want = "far", (0, 0, 0)
        elif 0.80 < u < 0.81:
            kind, want = "far above", (1, 1, 1)
        else:
            continue
        out = orc.verify_sequence_qprobs(q, P, [3], seed=5, seq=seq, rnd=0)
        assert out.accept_len == 0
        assert (out.next_token, out.next_lo, out.next_hi) == want, (kind, u)
        seen.add(kind)
        if len(seen) == 4:
            break
    assert len(seen) == 4
