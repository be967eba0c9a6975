"""The tensor-core weight-streaming GEMM against a plain fp64 matrix product of the same bf16 inputs."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

SHAPES = [  # (R, N, K): one tile / ragged N / several row paddings / deep split-K / full projection sizes / prompt chunks
    (1, 128, 64), (3, 200, 128), (5, 300, 256), (16, 1024, 512), (17, 520, 320), (40, 257, 192), (100, 1000, 512),
    (128, 384, 1024), (8, 4096, 14336), (6, 6144, 4096), (2, 32000, 4096),
    (129, 384, 512), (200, 1000, 1024), (256, 6144, 4096), (255, 4096, 14336),      # prompt-chunk row counts (256-row padding)
]


@pytest.mark.parametrize("R,N,K", SHAPES)
def test_gemm_matches_fp64_product(lib, R, N, K):
    g = torch.Generator().manual_seed(R * 1000003 + N * 101 + K)
    A = (torch.randn(R, K, generator=g) * 1.0).to(torch.bfloat16)
    W = (torch.randn(N, K, generator=g) * 0.05).to(torch.bfloat16)
    out = lib.hsd_gemm_bf16(A.cuda(), W.cuda()).cpu().numpy()
    ref = A.to(torch.float64).numpy() @ W.to(torch.float64).numpy().T
    scale = np.sqrt(K) * 0.05
    err = np.abs(out - ref).max()
    assert err < 2e-5 * scale * np.sqrt(K) + 1e-6, (err, scale)
    assert np.abs(ref).max() > 0.1 * scale


def test_gemm_is_bit_reproducible_and_row_count_independent(lib):
    # split tiles are summed in a fixed order; a row's result does not depend on how many rows ride along
    g = torch.Generator().manual_seed(5)
    A = torch.randn(8, 4096, generator=g).to(torch.bfloat16).cuda()
    W = (torch.randn(4096, 4096, generator=g) * 0.02).to(torch.bfloat16).cuda()
    a = lib.hsd_gemm_bf16(A, W)
    b = lib.hsd_gemm_bf16(A, W)
    assert torch.equal(a, b)
    one = lib.hsd_gemm_bf16(A[:1].contiguous(), W)
    assert torch.equal(one[0], a[0])


def test_gemm_rejects_bad_shapes(lib):
    A = torch.zeros(4, 100, dtype=torch.bfloat16, device="cuda")
    W = torch.zeros(64, 100, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(lib.HsdError):
        lib.hsd_gemm_bf16(A, W)          # K not a multiple of 64
