"""Algorithm 2 (Token Verification and Correction), step by step.

The verifier M_idx is run on every prefix context, context + x_1, ...,
context + x_1..x_t to give p_1..p_{t+1}; drafted tokens are tested in order
and the loop stops at the first rejection; the final token m comes from the
normalised residual max(0, p_{n+1} - q_{n+1}) after a rejection, or from
p_{t+1} when everything was accepted; the distributions handed upward are the
verifier's own rows p_1..p_{n+1} (also for m, even when m came from the
residual), as Algorithm 2's return statement says.

A "row" is whatever the model returns to describe one next-token distribution
(stored logits for the real models, exact probability vectors for the toy models
of the enumeration tests); only the ``decisions`` object looks inside rows.
"""


def verify(idx, draft_tokens, draft_rows, context, model, decisions, serial):
    """Returns (output_tokens, output_rows, n_tested).

    model.rows(idx, context, draft_tokens) -> the t+1 rows p_1..p_{t+1}
    decisions.accept(p_row, q_row, x, j, serial, idx) -> bool   (j = 0-based position)
    decisions.final_sample(p_row, q_row_or_None, serial, idx) -> token
    """
    t = len(draft_tokens)
    assert len(draft_rows) == t
    p_rows = model.rows(idx, context, draft_tokens)
    assert len(p_rows) == t + 1
    n = t
    tested = 0
    for i in range(1, t + 1):
        tested += 1
        if not decisions.accept(p_rows[i - 1], draft_rows[i - 1], draft_tokens[i - 1], i - 1, serial, idx):
            n = i - 1
            break
    if n < t:
        m = decisions.final_sample(p_rows[n], draft_rows[n], serial, idx)
    else:
        m = decisions.final_sample(p_rows[t], None, serial, idx)
    output_tokens = list(draft_tokens[:n]) + [m]
    output_rows = [p_rows[k] for k in range(n + 1)]
    return output_tokens, output_rows, tested
