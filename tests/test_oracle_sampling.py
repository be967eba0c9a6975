"""The fixed-point decision arithmetic pinned to the fp64 definitions of Section 2."""
import math

import numpy as np

from oracle import philox, sampling as S


def _rows(seed, V, std=3.0, bf16=True):
    rng = np.random.default_rng(seed)
    l = rng.normal(0, std, V).astype(np.float32)
    if bf16:
        l = (l.view(np.uint32) & np.uint32(0xFFFF0000)).view(np.float32)
    return l


def test_exp_weights_match_math_exp():
    l = _rows(0, 4096)
    E = S.exp_weights(l)
    m = float(l.max())
    assert int(E.max()) == (1 << 32) - 1                 # the maximum saturates at 2^32 - 1
    for k in range(0, 4096, 7):
        ref = math.exp(float(l[k]) - m) * 2.0 ** 32
        assert abs(int(E[k]) - ref) <= 1.0 + 1.5e-6 * ref
    # far tails and -inf are zero weight, never negative or NaN
    l2 = np.array([0.0, -40.0, -1e30, -np.inf, -16.0], dtype=np.float32)
    E2 = S.exp_weights(l2)
    assert E2.tolist()[:4] == [(1 << 32) - 1, 0, 0, 0]
    assert abs(int(E2[4]) - math.exp(-16.0) * 2 ** 32) < 2


def test_fixed_probs_match_softmax():
    for seed in range(3):
        l = _rows(seed, 1000)
        P, Ssum = S.fixed_probs(S.exp_weights(l))
        p = S.softmax64(l)
        got = P.astype(np.float64) / 2.0 ** 40
        assert np.all(np.abs(got - p) <= 2e-6 * p + 2.0 ** -31)
        assert abs(got.sum() - 1.0) < 1e-6


def test_categorical_counts_are_exact():
    # number of uniforms U mapping to token k must be E_k * 2^24 / S up to rounding
    l = _rows(3, 37, std=2.0)
    E = S.exp_weights(l)
    tot = int(E.sum())
    c = np.concatenate([[0], np.cumsum(E.astype(object))])
    for k in range(37):
        # U maps to k  <=>  c[k] <= (U*tot)>>24 < c[k+1]  <=>  ceil(c[k]*2^24/tot) <= U < ceil(c[k+1]*2^24/tot)
        lo = -((-int(c[k]) << 24) // tot)
        hi = -((-int(c[k + 1]) << 24) // tot)
        for U in {lo, hi - 1} if hi > lo else set():
            assert S.inverse_cdf(E, tot, U) == k
            assert S.inverse_cdf_fast(E, tot, U) == k
        assert abs((hi - lo) - int(E[k]) * 2.0 ** 24 / tot) <= 1.0
    assert S.inverse_cdf_fast(E, tot, 0) == int(np.nonzero(E)[0][0])
    assert S.inverse_cdf_fast(E, tot, (1 << 24) - 1) == int(np.nonzero(E)[0][-1])


def test_zero_weight_tokens_are_never_drawn():
    l = np.array([-50.0, 0.0, -50.0, -1.0, -50.0], dtype=np.float32)
    seen = {S.categorical(l, U) for U in range(0, 1 << 24, 4099)} | {S.categorical(l, (1 << 24) - 1)}
    assert seen == {1, 3}


def _accept_count(Pp_x, Pq_x):
    """#{U in [0,2^24): ((U*Pq)>>24) < Pp} by the closed form, cross-checked at its edges."""
    if Pq_x == 0:
        return (1 << 24) if Pp_x > 0 else 0
    n = min(1 << 24, -((-(Pp_x << 24)) // Pq_x))
    for U in (n - 1, n):
        if 0 <= U < (1 << 24):
            assert S.accept(Pp_x, Pq_x, U) == (U < n)
    return n


def test_accept_probability_is_min_1_p_over_q():
    lp, lq = _rows(5, 300), _rows(6, 300)
    Ep, Eq = S.exp_weights(lp), S.exp_weights(lq)
    Pp, _ = S.fixed_probs(Ep)
    Pq, _ = S.fixed_probs(Eq)
    p, q = S.softmax64(lp), S.softmax64(lq)
    for x in range(300):
        if Pq[x] == 0 or Pp[x] == 0:
            continue
        got = _accept_count(int(Pp[x]), int(Pq[x])) / 2.0 ** 24
        want = S.accept_probability(p, q, x)
        # exp_spec error (~1e-6) + one unit of flooring in each integer weight / probability
        rel = 4e-6 + 2.0 / float(Ep[x]) + 2.0 / float(Eq[x]) + 2.0 / float(Pp[x]) + 2.0 / float(Pq[x])
        assert abs(got - want) <= rel * want + 2.0 ** -23
    assert S.accept(5, 5, (1 << 24) - 1) and S.accept(6, 5, (1 << 24) - 1)   # ratio >= 1 always accepts
    assert not S.accept(0, 5, 0)                                              # p(x) = 0 never accepts


def _emitted_law(lp, lq):
    """Exact law (over U_draft, U_accept, U_final independent) of the token emitted at one
    position: x ~ q accepted w.p. acc(x), else the residual draw."""
    V = len(lp)
    Ep, Eq = S.exp_weights(lp), S.exp_weights(lq)
    Pp, Sp = S.fixed_probs(Ep)
    Pq, Sq = S.fixed_probs(Eq)
    cq = np.concatenate([[0], np.cumsum(Eq.astype(object))])
    draw_q = [(-((-int(cq[k + 1]) << 24) // Sq)) - (-((-int(cq[k]) << 24) // Sq)) for k in range(V)]
    acc = [_accept_count(int(Pp[k]), int(Pq[k])) for k in range(V)]
    r = np.where(Pp > Pq, Pp - Pq, np.uint64(0))
    rt = int(r.sum())
    cr = np.concatenate([[0], np.cumsum(r.astype(object))])
    draw_r = [(-((-int(cr[k + 1]) << 24) // rt)) - (-((-int(cr[k]) << 24) // rt)) for k in range(V)]
    two24 = float(1 << 24)
    p_acc = [draw_q[k] / two24 * acc[k] / two24 for k in range(V)]
    rej = 1.0 - sum(p_acc)
    return np.array([p_acc[k] + rej * draw_r[k] / two24 for k in range(V)]), 1.0 - rej


def test_speculative_sampling_lemma_and_acceptance_rate():
    # Section 2: the emitted token follows p; the acceptance rate is 1 - TV(p, q)
    for seed in range(3):
        lp = _rows(10 + seed, 200, std=2.0)
        lq = (lp + _rows(20 + seed, 200, std=1.0, bf16=False)).astype(np.float32)
        law, alpha = _emitted_law(lp, lq)
        p, q = S.softmax64(lp), S.softmax64(lq)
        assert np.abs(law - p).max() < 2e-6
        assert abs(alpha - S.acceptance_rate(p, q)) < 2e-5
        res = S.residual_distribution(p, q)
        assert abs(res.sum() - 1.0) < 1e-12 and np.all(res[p <= q] == 0)


def test_residual_sample_support_and_fallback():
    lp = np.array([0.0, 1.0, 2.0, -1.0], dtype=np.float32)
    lq = np.array([2.0, 1.0, 0.0, -1.0], dtype=np.float32)
    p, q = S.softmax64(lp), S.softmax64(lq)
    res = S.residual_distribution(p, q)
    counts = np.zeros(4)
    N = 1 << 14
    for i in range(N):
        counts[S.residual_sample(lp, lq, i << 10)] += 1
    assert np.abs(counts / N - res).max() < 2e-3 and counts[0] == 0
    # identical rows: residual is empty, the draw falls back to p
    assert S.residual_distribution(p, p) is None
    for U in (0, 12345678, (1 << 24) - 1):
        assert S.residual_sample(lp, lp, U) == S.categorical(lp, U)


def test_philox_driven_draws_follow_the_softmax():
    l = _rows(42, 16, std=1.5)
    p = S.softmax64(l)
    N = 20000
    counts = np.zeros(16)
    for j in range(N):
        counts[S.categorical(l, philox.uniform24(9, j, 0, 0, 0, 0))] += 1
    chi2 = float((((counts - N * p) ** 2) / (N * p)).sum())
    assert chi2 < 45.0            # 15 degrees of freedom, p-value ~ 1e-4


def test_pairwise_acceptance_matrix():
    """alpha[i][j] of Section 2 between every pair of models: symmetric, ones on the diagonal, equal to the mass
    shared by the two distributions (sum of minima), 1 for identical and 0 for disjoint models, and equal to
    the empirical acceptance frequency of the speculative rule."""
    rng = np.random.default_rng(3)
    logits = rng.normal(0, 2.0, size=(4, 5, 37))
    logits[3] = logits[0]                                   # model 3 = model 0
    a = S.pairwise_acceptance(logits)
    assert a.shape == (4, 4) and np.allclose(a, a.T) and np.allclose(np.diag(a), 1.0)
    assert abs(a[0, 3] - 1.0) < 1e-12 and np.allclose(a[3, 1:3], a[0, 1:3])
    for i in range(3):
        for j in range(i + 1, 3):
            shared = np.mean([np.minimum(S.softmax64(logits[i, r]), S.softmax64(logits[j, r])).sum() for r in range(5)])
            assert abs(a[i, j] - shared) < 1e-12
    disjoint = np.full((2, 1, 8), -1e30)
    disjoint[0, 0, :4] = 0.0
    disjoint[1, 0, 4:] = 0.0
    assert abs(S.pairwise_acceptance(disjoint)[0, 1]) < 1e-12
    # empirical: draft x ~ q, accept with probability min(1, p(x) / q(x))
    q, p = S.softmax64(logits[1, 0]), S.softmax64(logits[2, 0])
    xs = rng.choice(len(q), size=200000, p=q)
    freq = float((rng.random(xs.size) < np.minimum(1.0, p[xs] / q[xs])).mean())
    assert abs(freq - S.pairwise_acceptance(logits[1:3, :1])[0, 1]) < 5e-3
