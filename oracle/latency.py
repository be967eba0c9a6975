"""Expected latency of a hierarchy (Theorem 3.2, Corollary 4.1) and the search of Section 4.

Reading of the garbled indices (the printed product runs over R(alpha_{j-1,j}, j)
with a dummy alpha_{-1,0}; the corollary sums to |sigma|): the proof's recursion,

    cost(0) = T_0 c_0
    cost(k) = gamma(alpha_{k-1,k}, T_{k-1}, T_k) * (cost(k-1) + c_k)       0 < k < K
    L       = (1 - a) / (1 - a^(T_{K-1}+1)) * (cost(K-1) + c_K),  a = alpha_{K-1,K}

gamma(alpha, T_in, T_out) counts, in expectation, the draft-and-verify rounds a
level goes through until it holds the T_out tokens it needs when each round offers
T_in drafts; the paper gives no formula for it (it says the value was measured).
Reading used here: acceptances are IID with rate alpha (the paper's standing assumption),
a round yields Y = k tokens with probability alpha^(k-1) (1 - alpha) for
k = 1..T_in and T_in + 1 with probability alpha^T_in, and gamma is the expected
number of rounds until the yields sum to at least T_out.

Search: the reduction graph of Section 4.2 minus its self-loops is acyclic (edges
go to a strictly smaller model index), so the cheapest augmented path is a
cost-to-go recursion over vertices (M_i, j); edges (M_i, j) -> (M_k, l) exist for
k < i and l <= j, as the paper's edge list says.
"""
from functools import lru_cache
from itertools import combinations, product


@lru_cache(maxsize=None)
def gamma(alpha, T_in, T_out):
    probs = [alpha ** (k - 1) * (1.0 - alpha) for k in range(1, T_in + 1)] + [alpha ** T_in]
    g = [0.0] * (T_out + T_in + 2)          # g[c] = expected further rounds with c tokens in hand
    for c in range(T_out - 1, -1, -1):
        g[c] = 1.0 + sum(p * g[c + k] for k, p in enumerate(probs, start=1))
    return g[0]


def top_multiplier(alpha, T):
    """(1 - alpha) / (1 - alpha^(T+1)): one over the expected tokens per target verification."""
    if alpha >= 1.0:
        return 1.0 / (T + 1)
    return (1.0 - alpha) / (1.0 - alpha ** (T + 1))


def expected_latency(costs, alphas, T):
    """L for the full chain: costs c_0..c_K, alphas[i] = alpha_{i,i+1}, T = T_0..T_{K-1}."""
    K = len(costs) - 1
    assert len(alphas) == K and len(T) == K
    if K == 0:
        return costs[0]
    cost = T[0] * costs[0]
    for k in range(1, K):
        cost = gamma(alphas[k - 1], T[k - 1], T[k]) * (cost + costs[k])
    return top_multiplier(alphas[K - 1], T[K - 1]) * (cost + costs[K])


def literal_latency(costs, alphas, T):
    """Expected cost per token of Algorithm 1 run literally, under the same two assumptions (IID acceptance,
    constant costs).  Theorem 3.2 lets every verifier see exactly T_{k-1} drafts; the algorithm as printed hands
    a verifier everything the level below collected, between T_{k-1} and T_{k-1} + (its own batch) tokens.  This
    is the exact renewal computation for that process:
      level 0 returns t = T_0 tokens at cost T_0 c_0;
      level k, 0 < k < K, repeats (call level k-1, verify: n accepted of t with P(n = j) = a^j (1 - a) for
        j < t and a^t for j = t, yield n + 1) until it holds >= T_k tokens: cost_k = E[rounds] (cost_{k-1} + c_k)
        by Wald's identity, and the distribution of the number it returns feeds level k + 1;
      the target does one such round per call: L = (cost_{K-1} + c_K) / E[yield]  (renewal-reward).
    Equal to Theorem 3.2 for one drafter (K = 1)."""
    K = len(costs) - 1
    assert len(alphas) == K and len(T) == K
    if K == 0:
        return costs[0]
    dist = {T[0]: 1.0}                     # number of tokens the level below returns
    cost = T[0] * costs[0]
    for k in range(1, K + 1):
        a = alphas[k - 1]
        yld = {}
        for t, pt in dist.items():
            for j in range(t):
                yld[j + 1] = yld.get(j + 1, 0.0) + pt * a ** j * (1.0 - a)
            yld[t + 1] = yld.get(t + 1, 0.0) + pt * a ** t
        if k == K:
            return (cost + costs[K]) / sum(y * p for y, p in yld.items())
        need = T[k]
        mass = {0: 1.0}                    # probability of holding c < need tokens before a round
        rounds, out = 0.0, {}
        for c in range(need):
            m = mass.get(c, 0.0)
            if m == 0.0:
                continue
            rounds += m
            for y, p in yld.items():
                tgt = out if c + y >= need else mass
                tgt[c + y] = tgt.get(c + y, 0.0) + m * p
        cost = rounds * (cost + costs[k])
        dist = out


def subset_latency(costs, alpha, sigma, T):
    """Corollary 4.1: L(sigma, T); alpha[i][j] = acceptance rate drafter i -> verifier j."""
    c = [costs[i] for i in sigma]
    a = [alpha[sigma[i]][sigma[i + 1]] for i in range(len(sigma) - 1)]
    return expected_latency(c, a, list(T))


def search_T(costs, alphas, T_max, monotone=True):
    """Best T for a fixed chain; monotone=True keeps the graph's constraint T_{k} >= T_{k-1}."""
    K = len(costs) - 1
    best = (costs[K], ())
    if K == 0:
        return best
    best = None
    for T in product(range(1, T_max + 1), repeat=K):
        if monotone and any(T[k] < T[k - 1] for k in range(1, K)):
            continue
        L = expected_latency(costs, alphas, T)
        if best is None or L < best[0] - 1e-15:
            best = (L, T)
    return best


def search_hierarchy(costs, alpha, T_max):
    """min over ordered subsets ending in K and T in [1, T_max]: returns (L, sigma, T).

    Cost-to-go over the reduction graph: down[i][j] = cheapest way for a
    sub-hierarchy topped by M_i to hand up a batch of j tokens.
    """
    K = len(costs) - 1
    down = [[None] * (T_max + 1) for _ in range(K)]
    for i in range(K):
        for j in range(1, T_max + 1):
            best = (j * costs[i], (i,), (j,))                       # M_i is the bottom level
            for k in range(i):
                for l in range(1, j + 1):
                    sub = down[k][l]
                    c = gamma(alpha[k][i], l, j) * (costs[i] + sub[0])
                    if c < best[0]:
                        best = (c, sub[1] + (i,), sub[2] + (j,))
            down[i][j] = best
    best = (costs[K], (K,), ())
    for i in range(K):
        for j in range(1, T_max + 1):
            sub = down[i][j]
            c = top_multiplier(alpha[i][K], j) * (costs[K] + sub[0])
            if c < best[0]:
                best = (c, sub[1] + (K,), sub[2])
    return best


def brute_force_hierarchy(costs, alpha, T_max):
    """Same minimum by enumerating every (sigma, T) with the monotone constraint."""
    K = len(costs) - 1
    best = (costs[K], (K,), ())
    for r in range(1, K + 1):
        for lower in combinations(range(K), r):
            sigma = lower + (K,)
            for T in product(range(1, T_max + 1), repeat=r):
                if any(T[k] < T[k - 1] for k in range(1, r)):
                    continue
                L = subset_latency(costs, alpha, sigma, T)
                if L < best[0]:
                    best = (L, sigma, T)
    return best
