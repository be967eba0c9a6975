"""Parity of the sampling kernels with the oracle on identical logits (decisions are bit-exact)."""
import numpy as np
import pytest
import torch

from oracle import philox, sampling
from paper_2510_19705_b200 import inputs

pytestmark = pytest.mark.gpu


def _oracle_draft(logits_np, seed, serial):
    B, R, V = logits_np.shape
    out = np.empty((B, R), dtype=np.int32)
    for b in range(B):
        for j in range(R):
            out[b, j] = sampling.categorical(logits_np[b, j], philox.uniform24(seed, j, serial, 0, philox.PURPOSE_DRAFT, b))
    return out


def _oracle_verify(level, p_np, q_np, x_np, seed, serial):
    """Algorithm 2's decisions on given rows, per sequence."""
    from oracle.hsd import SpecDecisions
    from oracle.verify import verify

    class Rows:
        def __init__(self, rows):
            self.r = rows

        def rows(self, idx, ctx, draft):
            return list(self.r)

    B, tp1, V = p_np.shape
    t = tp1 - 1
    out = np.full((B, t + 1), -1, dtype=np.int32)
    n_acc = np.empty(B, dtype=np.int32)
    for b in range(B):
        toks, _, _ = verify(level, list(x_np[b]), list(q_np[b]), [0], Rows(p_np[b]), SpecDecisions(seed, b), serial)
        out[b, :len(toks)] = toks
        n_acc[b] = len(toks) - 1
    return out, n_acc


@pytest.mark.parametrize("dtype,V,B,R", [("bf16", 32000, 6, 5), ("fp32", 512, 3, 4), ("bf16", 1000, 2, 3),
                                         ("fp32", 33, 2, 2), ("bf16", 50001, 1, 2)])
def test_draft_sample_matches_oracle(lib, dtype, V, B, R):
    _, q = inputs.make_accept_logits(B, R, V, seed=V + B, device="cuda", dtype=dtype)
    for seed, serial in [(0, 0), (12345678901234, 7)]:
        got = lib.hsd_draft_sample(q, seed, serial).cpu().numpy()
        want = _oracle_draft(inputs.logits_to_numpy(q), seed, serial)
        assert np.array_equal(got, want)


@pytest.mark.parametrize("dtype,V,B,t", [("bf16", 32000, 8, 8), ("fp32", 512, 4, 3), ("bf16", 4097, 3, 5),
                                         ("bf16", 32000, 2, 1), ("fp32", 7, 5, 2)])
def test_verify_level_matches_oracle(lib, dtype, V, B, t):
    p, q = inputs.make_accept_logits(B, t, V, seed=3 * V + t, device="cuda", dtype=dtype)
    x = lib.hsd_draft_sample(q, 99, 0)
    p_np, q_np, x_np = inputs.logits_to_numpy(p), inputs.logits_to_numpy(q), x.cpu().numpy()
    seen_n = set()
    for seed, serial, level in [(0, 0, 1), (5, 3, 2), (2 ** 40 + 17, 1000, 1)]:
        out, n = lib.hsd_verify_level(level, p, q, x, seed, serial)
        want_out, want_n = _oracle_verify(level, p_np, q_np, x_np, seed, serial)
        assert np.array_equal(n.cpu().numpy(), want_n)
        assert np.array_equal(out.cpu().numpy(), want_out)
        seen_n.update(want_n.tolist())
    assert len(seen_n) >= 2          # both accepted and rejected positions were exercised


def test_verify_edge_cases(lib):
    V = 64
    # t = 0: only the bonus draw from the single target row
    p, _ = inputs.make_accept_logits(3, 0, V, seed=1, device="cuda", dtype="fp32")
    out, n = lib.hsd_verify_level(1, p, None, None, 4, 2)
    p_np = inputs.logits_to_numpy(p)
    for b in range(3):
        U = philox.uniform24(4, 0, 2, 1, philox.PURPOSE_FINAL, b)
        assert n[b].item() == 0 and out[b, 0].item() == sampling.categorical(p_np[b, 0], U)
    # identical rows: everything is accepted (ratio 1), the bonus comes from the last target row
    p, _ = inputs.make_accept_logits(2, 4, V, seed=2, device="cuda", dtype="bf16")
    q = p[:, :4].contiguous()
    x = lib.hsd_draft_sample(q, 1, 0)
    out, n = lib.hsd_verify_level(1, p, q, x, 1, 0)
    assert n.tolist() == [4, 4] and torch.equal(out[:, :4], x)
    # a drafted token the target gives (almost) no mass is rejected and never re-emitted
    p = torch.zeros(1, 2, V, device="cuda")
    q = torch.zeros(1, 1, V, device="cuda")
    p[0, 0, 5] = -60.0
    x = torch.tensor([[5]], dtype=torch.int32, device="cuda")
    for seed in range(8):
        out, n = lib.hsd_verify_level(1, p, q, x, seed, 0)
        assert n.item() == 0 and out[0, 0].item() != 5 and out[0, 1].item() == -1


def test_acceptance_frequency_is_one_minus_tv(lib):
    # Section 2: P(accept) = 1 - sum |p - q| / 2 when x ~ q; measured over many sequences of the
    # same pair of rows (sequence index and serial vary the uniforms)
    V, B = 4096, 2048
    p1, q1 = inputs.make_accept_logits(1, 1, V, seed=8, device="cuda", dtype="bf16")
    p, q = p1.expand(B, 2, V).contiguous(), q1.expand(B, 1, V).contiguous()
    x = lib.hsd_draft_sample(q, 3, 0)
    _, n = lib.hsd_verify_level(1, p, q, x, 3, 0)
    alpha = sampling.acceptance_rate(sampling.softmax64(inputs.logits_to_numpy(p1)[0, 0]),
                                     sampling.softmax64(inputs.logits_to_numpy(q1)[0, 0]))
    freq = n.float().mean().item()
    assert abs(freq - alpha) < 4.5 * (alpha * (1 - alpha) / B) ** 0.5 + 1e-3


def test_bad_arguments_are_rejected(lib):
    p, q = inputs.make_accept_logits(2, 2, 32, seed=1, device="cuda", dtype="fp32")
    x = lib.hsd_draft_sample(q, 0, 0)
    small = torch.empty(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(lib.HsdError, match="workspace too small"):
        lib.hsd_verify_level(1, p, q, x, 0, 0, workspace=small)
    with pytest.raises(lib.HsdError, match="invalid argument"):
        lib.hsd_verify_level(300, p, q, x, 0, 0)
