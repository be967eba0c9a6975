"""The calibration kernels (pairwise acceptance rates between exit layers) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import sampling as S
from paper_2510_19705_b200 import binding

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("L,R,V,dtype", [(3, 5, 777, torch.float32), (4, 9, 2048, torch.bfloat16), (2, 3, 5000, torch.bfloat16),
                                         (8, 4, 1500, torch.float32), (1, 2, 100, torch.float32)])
def test_pairwise_alpha_matches_oracle(lib, L, R, V, dtype):
    g = torch.Generator().manual_seed(L * 1000 + R)
    base = torch.randn(R, V, generator=g) * 2.5
    logits = torch.stack([base + 0.8 * (m + 1) * torch.randn(R, V, generator=g) for m in range(L)]).to(dtype)
    got = lib.hsd_pairwise_alpha(logits.cuda())
    torch.cuda.synchronize()
    want = S.pairwise_acceptance(logits.float().numpy().astype(np.float64))
    got = got.cpu().numpy()
    assert got.shape == (L, L) and np.array_equal(got, got.T) and np.array_equal(np.diag(got), np.ones(L))
    assert np.abs(got - want).max() < 2e-5, np.abs(got - want).max()
    again = lib.hsd_pairwise_alpha(logits.cuda()).cpu().numpy()          # no atomics: repeatable bit for bit
    assert np.array_equal(got, again)


def test_pairwise_alpha_of_a_model_stack(lib):
    """The rates between the exits of one random-init model on its own drafted positions feed the hierarchy
    search: nearer exits accept each other more often, and the search returns a valid chain."""
    from paper_2510_19705_b200 import inputs
    torch.manual_seed(0)
    R, V = 16, 2048
    h = torch.randn(R, V)
    logits = torch.stack([h + s * torch.randn(R, V) for s in (1.5, 1.0, 0.5, 0.0)]).bfloat16().cuda()
    alpha = lib.hsd_pairwise_alpha(logits).cpu().numpy()
    assert alpha[2, 3] > alpha[1, 3] > alpha[0, 3]
    lat, sigma, T = binding.hsd_search_hierarchy([0.1, 0.3, 1.0, 3.0], alpha.tolist(), 8)
    assert sigma[-1] == 3 and len(T) == len(sigma) - 1 and lat <= 3.0
