"""Algorithm 1 + Algorithm 2 pinned by Theorem 3.1 (exact enumeration), the yield bounds of
Section 1, the two-model closed form of Leviathan et al. (used in the proof of Theorem 3.2), and
a sampled chi-square with the real Philox addressing."""
from collections import defaultdict
from fractions import Fraction
from itertools import product

import numpy as np
import pytest

from oracle import sampling
from oracle.hsd import HSD, SpecDecisions, generate
from oracle.verify import verify


# ------------------------------------------------------------------ toy models
class TableModel:
    """Context-dependent toy distributions (exact Fractions) with some zero entries.  Each level
    has its own table; a row depends on the last two tokens and the parity of the length."""

    def __init__(self, n_levels, V, seed, as_logits=False):
        self.n_levels, self.V, self.as_logits = n_levels, V, as_logits
        rng = np.random.default_rng(seed)
        self.w = rng.integers(0, 5, size=(n_levels, 2, V + 1, V + 1, V)).astype(int)
        self.w[..., 0] += (self.w.sum(-1) == 0)        # no all-zero row
        self.w[-1] += 1 if as_logits else 0
        self.calls = []

    def dist(self, level, prefix):
        a = prefix[-1] + 1 if len(prefix) >= 1 else 0
        b = prefix[-2] + 1 if len(prefix) >= 2 else 0
        w = self.w[level, len(prefix) % 2, a, b]
        if self.as_logits:
            return np.log(np.maximum(w, 1e-30)).astype(np.float32)
        tot = int(w.sum())
        return tuple(Fraction(int(x), tot) for x in w)

    def rows(self, level, context, draft_tokens):
        self.calls.append((level, len(context), len(draft_tokens)))
        return [self.dist(level, list(context) + list(draft_tokens[:j])) for j in range(len(draft_tokens) + 1)]


class EnumDecisions:
    """Replays a prefix of choices, then takes option 0 everywhere, recording the branching."""

    def __init__(self, prefix):
        self.prefix, self.path, self.widths, self.prob = list(prefix), [], [], Fraction(1)

    def _choose(self, options):
        """options: list of (outcome, probability) with positive probability."""
        d = len(self.path)
        i = self.prefix[d] if d < len(self.prefix) else 0
        self.path.append(i)
        self.widths.append(len(options))
        self.prob *= options[i][1]
        return options[i][0]

    def draft_sample(self, row, j, serial, level=0):
        return self._choose([(k, p) for k, p in enumerate(row) if p > 0])

    def accept(self, p_row, q_row, x, j, serial, level):
        a = min(Fraction(1), p_row[x] / q_row[x])
        return self._choose([(o, pr) for o, pr in ((True, a), (False, 1 - a)) if pr > 0])

    def final_sample(self, p_row, q_row, serial, level):
        if q_row is None:
            dist = p_row
        else:
            r = [max(Fraction(0), a - b) for a, b in zip(p_row, q_row)]
            tot = sum(r)
            dist = [x / tot for x in r] if tot > 0 else p_row
        return self._choose([(k, p) for k, p in enumerate(dist) if p > 0])


def enumerate_law(run):
    """run(decisions) -> hashable outcome; returns {outcome: exact probability}."""
    law, stack, n = defaultdict(Fraction), [[]], 0
    while stack:
        prefix = stack.pop()
        dec = EnumDecisions(prefix)
        out = run(dec)
        law[out] += dec.prob
        n += 1
        for d in range(len(prefix), len(dec.path)):
            for alt in range(1, dec.widths[d]):
                stack.append(dec.path[:d] + [alt])
    assert sum(law.values()) == 1
    return law, n


def target_law(model, prompt, n):
    K = model.n_levels - 1
    law = {}
    for toks in product(range(model.V), repeat=n):
        p = Fraction(1)
        for i, t in enumerate(toks):
            p *= model.dist(K, list(prompt) + list(toks[:i]))[t]
        if p > 0:
            law[toks] = p
    return law


CASES = [  # (n_levels, V, T, n tokens compared)
    (2, 3, (2,), 3), (2, 3, (1,), 2), (3, 3, (2, 2), 2), (3, 3, (2, 1), 2), (3, 2, (1, 2), 3),
    (3, 2, (3, 2), 2), (4, 2, (1, 1, 1), 2), (4, 2, (2, 1, 2), 2),
]


@pytest.mark.parametrize("n_levels,V,T,n", CASES)
def test_output_law_equals_target_exactly(n_levels, V, T, n):
    # Theorem 3.1: for any models and any parameters the output follows the target model
    model = TableModel(n_levels, V, seed=100 + n_levels * 10 + V)
    prompt = [1, 0]

    def run(dec):
        return tuple(HSD(model, T, dec).generate(prompt, n))

    law, n_paths = enumerate_law(run)
    want = target_law(model, prompt, n)
    assert set(law) == set(want)
    for k in want:
        assert law[k] == want[k], (k, law[k], want[k])


def test_enumeration_has_teeth_wrong_rows_upward_breaks_the_law():
    # handing the drafter's rows upward instead of the verifier's own (a plausible misreading of
    # Algorithm 2's return statement) must be caught by the enumeration
    import oracle.hsd as H
    model = TableModel(3, 3, seed=133)
    prompt = [1, 0]
    orig = H.verify

    def bad_verify(idx, d_tok, d_rows, ctx, mdl, dec, serial):
        toks, rows, tested = orig(idx, d_tok, d_rows, ctx, mdl, dec, serial)
        n = len(toks) - 1
        return toks, list(d_rows[:n]) + [rows[n]], tested

    H.verify = bad_verify
    try:
        law, _ = enumerate_law(lambda dec: tuple(HSD(model, (2, 2), dec).generate(prompt, 2)))
    finally:
        H.verify = orig
    want = target_law(model, prompt, 2)
    assert any(law.get(k, 0) != want[k] for k in want)


def test_verify_yield_bounds_and_returned_rows():
    # every round yields between 1 and t + 1 tokens; returned rows are the verifier's own
    model = TableModel(2, 3, seed=7)
    ctx = [2, 1]
    seen = set()

    def run(dec):
        d_tok, d_rows = [], []
        for j in range(3):
            row = model.dist(0, ctx + d_tok)
            d_tok.append(dec.draft_sample(row, j, 0))
            d_rows.append(row)
        out, rows, tested = verify(1, d_tok, d_rows, ctx, model, dec, 0)
        n = len(out) - 1
        assert 1 <= len(out) <= 4 and out[:n] == d_tok[:n] and len(rows) == n + 1
        assert tested == min(n + 1, 3)
        for k in range(n + 1):
            assert rows[k] == model.dist(1, ctx + d_tok[:k])
        seen.add(len(out))
        return len(out)

    enumerate_law(run)
    assert seen == {1, 2, 3, 4}


def test_level_returns_between_T_and_sum_T():
    model = TableModel(3, 3, seed=5)
    T = (3, 2)
    lens = set()

    def run(dec):
        h = HSD(model, T, dec)
        toks, rows = h.hsd(1, [0, 1])
        assert T[1] <= len(toks) <= T[0] + T[1] and len(rows) == len(toks)
        lens.add(len(toks))
        return len(toks)

    enumerate_law(run)
    assert min(lens) == 2 and max(lens) == 5


class ConstModel:
    """Context-free rows: acceptances are IID with rate 1 - TV(p, q)."""
    n_levels, V = 2, 3
    p = (Fraction(1, 2), Fraction(1, 3), Fraction(1, 6))
    q = (Fraction(1, 4), Fraction(1, 4), Fraction(1, 2))

    def rows(self, level, context, draft_tokens):
        return [(self.q, self.p)[level]] * (len(draft_tokens) + 1)


@pytest.mark.parametrize("T", [1, 2, 4])
def test_two_level_expected_tokens_per_round(T):
    # (1 - alpha^(T+1)) / (1 - alpha) tokens per target verification (Section 3.3, proof)
    m = ConstModel()
    alpha = 1 - sum(abs(a - b) for a, b in zip(m.p, m.q)) / 2
    law, _ = enumerate_law(lambda dec: len(HSD(m, (T,), dec).hsd(1, [0])[0]))
    mean = sum(k * pr for k, pr in law.items())
    assert mean == (1 - alpha ** (T + 1)) / (1 - alpha)


def test_single_level_is_ancestral_sampling():
    model = TableModel(1, 4, seed=3, as_logits=True)
    toks, stats, trace = generate(model, (), [1, 2], 12, seed=77)
    from oracle import philox
    ctx = [1, 2]
    for i, t in enumerate(toks):
        U = philox.uniform24(77, 0, i, 0, philox.PURPOSE_DRAFT, 0)
        assert t == sampling.categorical(model.dist(0, ctx), U)
        ctx.append(int(t))
    assert stats[0][0] == 12 and stats[0][5] == 12


def test_sampled_streams_follow_the_target_law():
    # real Philox addressing + fixed-point decisions, many seeds, first two tokens
    model = TableModel(3, 4, seed=21, as_logits=True)
    prompt = [3, 1]
    want = {}
    for a in range(4):
        pa = sampling.softmax64(model.dist(2, prompt))[a]
        for b in range(4):
            want[(a, b)] = pa * sampling.softmax64(model.dist(2, prompt + [a]))[b]
    N = 6000
    counts = defaultdict(int)
    for seed in range(N):
        toks, _, _ = generate(model, (2, 2), prompt, 2, seed=seed)
        counts[(int(toks[0]), int(toks[1]))] += 1
    cells = [k for k in want if want[k] * N >= 5]
    chi2 = sum((counts[k] - N * want[k]) ** 2 / (N * want[k]) for k in cells)
    assert sum(counts[k] for k in want if k not in cells) <= 40
    assert chi2 < 45.0, chi2          # <= 15 degrees of freedom


def test_stats_and_trace_bookkeeping():
    model = TableModel(3, 4, seed=2, as_logits=True)
    run = HSD(model, (3, 2), SpecDecisions(5))
    out = run.generate([0, 1, 2], 20)
    assert len(out) == 20
    s0, s1, s2 = run.stats
    assert s0.emitted == 3 * s0.calls and s0.rows == s0.emitted
    assert s1.drafted == s0.emitted and s2.drafted == s1.emitted
    for s in (s1, s2):
        assert s.emitted == s.accepted + s.calls and s.accepted <= s.tested <= s.drafted
    assert s2.emitted >= 20
    # serials count calls per level from zero
    for lvl in range(3):
        assert [t[1] for t in run.trace if t[0] == lvl] == list(range(run.stats[lvl].calls))


class FlatModel:
    """Three context-free levels over 5 tokens (stored logits)."""
    n_levels = 3
    tab = np.log(np.array([[.3, .3, .2, .1, .1], [.25, .35, .2, .1, .1], [.2, .4, .2, .1, .1]])).astype(np.float32)

    def rows(self, level, context, draft_tokens):
        return [self.tab[level]] * (len(draft_tokens) + 1)


def test_coin_acceptance_extremes_and_frequency():
    from oracle.hsd import CoinDecisions
    m = FlatModel()
    run = HSD(m, (2, 3), CoinDecisions(1, (1.0, 1.0)))
    run.generate([0], 60)
    assert all(t[4] == t[3] for t in run.trace if t[0] > 0)           # every draft accepted
    run = HSD(m, (2, 3), CoinDecisions(1, (0.0, 0.0)))
    run.generate([0], 30)
    assert all(t[4] == 0 for t in run.trace if t[0] > 0)              # every first draft rejected
    run = HSD(m, (2, 3), CoinDecisions(7, (0.6, 0.8)))
    run.generate([0], 3000)
    for st, a in zip(run.stats[1:], (0.6, 0.8)):
        assert st.tested > 1500
        assert abs(st.accepted / st.tested - a) < 4 * (a * (1 - a) / st.tested) ** 0.5


class FlatModel2(FlatModel):
    n_levels = 2


def _coin_cost_per_token(model, costs, alphas, T, n_new=2500, seeds=4):
    from oracle.hsd import CoinDecisions, artificial_latency
    total, n_tok = 0.0, 0
    for seed in range(seeds):
        run = HSD(model, T, CoinDecisions(seed, alphas))
        run.generate([0], n_new)
        emitted = run.stats[-1].emitted                                # whole rounds: nothing cut off
        total += artificial_latency(run.stats, costs, emitted) * emitted
        n_tok += emitted
    return total / n_tok


def test_coin_acceptance_with_artificial_costs_reproduces_theorem_3_2():
    """The fully simplified setting of the ablation (IID acceptance, constant costs) is the model behind
    Theorem 3.2.  Two levels: the closed form (1 - a) / (1 - a^(T+1)) (T c_0 + c_1) is exact, the simulation
    converges to it.  Three levels: the theorem lets the top verifier see exactly T_1 drafts per round, the
    literal Algorithm 1 hands it everything the level below collected (T_1 .. T_1 + T_0), so the simulated
    cost lies a little below the closed form."""
    from oracle import latency
    sim2 = _coin_cost_per_token(FlatModel2(), (1.0, 10.0), (0.7,), (3,))
    want2 = latency.expected_latency((1.0, 10.0), (0.7,), (3,))
    assert abs(want2 - (1 - 0.7) / (1 - 0.7 ** 4) * 13.0) < 1e-12
    assert abs(sim2 - want2) < 0.02 * want2, (sim2, want2)
    costs, alphas, T = (1.0, 3.0, 10.0), (0.6, 0.8), (2, 3)
    sim3 = _coin_cost_per_token(FlatModel(), costs, alphas, T)
    want3 = latency.expected_latency(costs, alphas, T)
    assert 0.88 * want3 < sim3 < 1.01 * want3, (sim3, want3)
    # and the coins matter: another rate gives another cost
    assert abs(_coin_cost_per_token(FlatModel2(), (1.0, 10.0), (0.4,), (3,), seeds=2) - want2) > 0.1 * want2


def test_literal_latency_model_matches_the_simulated_algorithm():
    """oracle/latency.py: literal_latency is the exact expected cost per token of Algorithm 1 as printed under IID
    acceptance and constant costs: the coin simulation converges to it for three and four levels, and it equals
    Theorem 3.2's closed form for one drafter."""
    from oracle import latency
    assert abs(latency.literal_latency((1.0, 10.0), (0.7,), (3,)) - latency.expected_latency((1.0, 10.0), (0.7,), (3,))) < 1e-12
    costs, alphas, T = (1.0, 3.0, 10.0), (0.6, 0.8), (2, 3)
    sim3 = _coin_cost_per_token(FlatModel(), costs, alphas, T)
    lit3 = latency.literal_latency(costs, alphas, T)
    assert abs(sim3 - lit3) < 0.02 * lit3, (sim3, lit3)
    assert lit3 < latency.expected_latency(costs, alphas, T)          # more drafts per target pass than the theorem grants

    class Flat4(FlatModel):
        n_levels = 4
        tab = np.concatenate([FlatModel.tab, FlatModel.tab[-1:]])
    costs, alphas, T = (1.0, 2.0, 5.0, 20.0), (0.5, 0.7, 0.6), (1, 2, 2)
    sim4 = _coin_cost_per_token(Flat4(), costs, alphas, T)
    lit4 = latency.literal_latency(costs, alphas, T)
    assert abs(sim4 - lit4) < 0.02 * lit4, (sim4, lit4)
