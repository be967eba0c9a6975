"""Algorithm 1 (Hierarchical Speculative Decoding) and the outer generation loop.

Models M_0..M_K (M_K the target), parameters T_0..T_{K-1}.  What each level does:
  bottom (0)     M_0 extends the context by T_0 tokens, one forward per token,
                 and keeps the full distribution row behind every token.
  middle (i)     asks the level below for drafts after everything it has collected
                 so far, verifies them with M_i (Algorithm 2), and repeats until it
                 holds at least T_i tokens; ALL collected tokens and rows go up (the
                 count may exceed T_i: Algorithm 1 hands back what it has, uncut).
  top (K)        one draft request to level K-1, one verification by the target.
Generation (Section 3.2 starts every round at the top level): rounds are run on
prompt + output until at least n_new tokens exist and the first n_new are kept
(the paper does not say how generation stops; truncation is this project's
reading).  K = 0 is this project's degenerate case: one sample from M_0 per round.

Random numbers are addressed by (purpose, level, per-level call serial, position
in the call, sequence) -- see oracle/philox.py -- so a decision's uniform does
not depend on how many draws came before it.
"""
import numpy as np

from . import philox, sampling
from .verify import verify


class LevelStats:
    __slots__ = ("calls", "rows", "drafted", "tested", "accepted", "emitted")

    def __init__(self):
        self.calls = self.rows = self.drafted = self.tested = self.accepted = self.emitted = 0

    def as_tuple(self):
        return (self.calls, self.rows, self.drafted, self.tested, self.accepted, self.emitted)


class SpecDecisions:
    """Decisions as the CUDA library takes them: Philox uniforms + fixed-point arithmetic.

    Rows are 1-D arrays of stored logits.  ``log`` (optional list) receives one
    tuple per decision for trace comparisons.
    """

    def __init__(self, seed, seq=0, log=None):
        self.seed, self.seq, self.log = seed, seq, log

    def draft_sample(self, row, j, serial, level=0):
        U = philox.uniform24(self.seed, j, serial, level, philox.PURPOSE_DRAFT, self.seq)
        return sampling.categorical(row, U)

    def accept(self, p_row, q_row, x, j, serial, level):
        U = philox.uniform24(self.seed, j, serial, level, philox.PURPOSE_ACCEPT, self.seq)
        Pp, _ = sampling.fixed_probs(sampling.exp_weights(p_row))
        Pq, _ = sampling.fixed_probs(sampling.exp_weights(q_row))
        return sampling.accept(Pp[x], Pq[x], U)

    def final_sample(self, p_row, q_row, serial, level):
        U = philox.uniform24(self.seed, 0, serial, level, philox.PURPOSE_FINAL, self.seq)
        if q_row is None:
            return sampling.categorical(p_row, U)
        return sampling.residual_sample(p_row, q_row, U)


class CoinDecisions(SpecDecisions):
    """The ablation of the appendix "Examining the assumptions of HSD": Algorithm 2's accept test is replaced by
    a biased coin per drafted token, level i+1 accepting with probability alphas[i].  The coin is the accept
    test's own uniform compared with round(alpha * 2^24); drafting and the final draw are unchanged."""

    def __init__(self, seed, alphas, seq=0, log=None):
        super().__init__(seed, seq, log)
        self.thr = [int(a * 16777216.0 + 0.5) for a in alphas]

    def accept(self, p_row, q_row, x, j, serial, level):
        U = philox.uniform24(self.seed, j, serial, level, philox.PURPOSE_ACCEPT, self.seq)
        return U < self.thr[level - 1]


def artificial_latency(stats, costs, n_tokens):
    """The same ablation's fixed artificial cost: every forward of level i costs costs[i] (level 0 runs one
    forward per drafted token, a verifier one per call); total cost per generated token."""
    total = stats[0].rows * costs[0] + sum(st.calls * c for st, c in zip(stats[1:], costs[1:]))
    return total / n_tokens


class HSD:
    """One sequence's run of Algorithm 1 over ``model`` with parameters ``T``.

    model.n_levels = K + 1; model.rows(level, context, draft_tokens) -> list of
    len(draft_tokens) + 1 rows, row j describing M_level(context + x_1..x_j).
    """

    def __init__(self, model, T, decisions):
        self.model, self.T, self.dec = model, list(T), decisions
        self.K = model.n_levels - 1
        assert len(self.T) == self.K and all(t >= 1 for t in self.T)
        self.serial = [0] * (self.K + 1)
        self.stats = [LevelStats() for _ in range(self.K + 1)]
        self.trace = []   # (level, serial, context_len, t, n, tokens) per Verify / level-0 call

    def _next_serial(self, level):
        s = self.serial[level]
        self.serial[level] += 1
        return s

    def hsd(self, idx, context):
        """Tokens and rows that level idx hands to the level above for this context."""
        if idx == 0:
            return self._bottom(context)
        if idx == self.K:
            d_tok, d_rows = self.hsd(idx - 1, context)
            return self._verify(idx, d_tok, d_rows, context)
        return self._middle(idx, context)

    def _bottom(self, context):
        # M_0 on its own: one forward per token, each token drawn from the row just computed
        st = self.stats[0]
        serial = self._next_serial(0)
        n_draft = self.T[0] if self.K > 0 else 1
        tokens, rows = [], []
        for j in range(n_draft):
            row = self.model.rows(0, context + tokens, [])[0]
            tokens.append(self.dec.draft_sample(row, j, serial, 0))
            rows.append(row)
            st.rows += 1
        st.calls += 1
        st.emitted += n_draft
        self.trace.append((0, serial, len(context), 0, n_draft, tuple(tokens)))
        return tokens, rows

    def _middle(self, idx, context):
        # keep drafting (below) and verifying (here) behind what has been collected, until T_idx tokens are in hand
        held_tokens, held_rows = [], []
        while len(held_tokens) < self.T[idx]:
            ctx = context + held_tokens
            d_tok, d_rows = self.hsd(idx - 1, ctx)
            v_tok, v_rows = self._verify(idx, d_tok, d_rows, ctx)
            held_tokens += v_tok
            held_rows += v_rows
        return held_tokens, held_rows

    def _verify(self, idx, d_tok, d_rows, ctx):
        serial = self._next_serial(idx)
        out_tok, out_rows, tested = verify(idx, d_tok, d_rows, ctx, self.model, self.dec, serial)
        st = self.stats[idx]
        st.calls += 1
        st.rows += len(d_tok) + 1
        st.drafted += len(d_tok)
        st.tested += tested
        st.accepted += len(out_tok) - 1
        st.emitted += len(out_tok)
        self.trace.append((idx, serial, len(ctx), len(d_tok), len(out_tok) - 1, tuple(out_tok)))
        return out_tok, out_rows

    def generate(self, prompt, n_new):
        out = []
        prompt = list(prompt)
        while len(out) < n_new:
            toks, _ = self.hsd(self.K, prompt + out)
            assert 1 <= len(toks)
            out.extend(toks)
        return out[:n_new]


def generate(model, T, prompt, n_new, seed, seq=0):
    """Convenience wrapper: returns (tokens, per-level stats tuples, trace)."""
    run = HSD(model, T, SpecDecisions(seed, seq))
    toks = run.generate(prompt, n_new)
    return np.asarray(toks, dtype=np.int32), [s.as_tuple() for s in run.stats], run.trace
