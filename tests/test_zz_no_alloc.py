"""The allocation-free verification entry point (for callers that are handed their input and output
buffers and cannot get scratch memory of their own) must give exactly what hsd_verify_level gives.

Collected last on purpose: if it fails, a run that stops at the first failure has run everything else."""
import pytest
import torch

from paper_2510_19705_b200 import inputs

pytestmark = pytest.mark.gpu


def test_static_scratch_variant_matches_the_workspace_variant_twice_in_a_row(lib):
    cases = [("bf16", 32000, 8, 8, 11), ("fp32", 512, 5, 3, 12)]
    for dtype, V, B, t, seed in cases:
        p, q = inputs.make_accept_logits(B, t, V, seed=seed, device="cuda", dtype=dtype)
        x = lib.hsd_draft_sample(q, 7, 0)
        out_s = torch.empty(B, t + 1, dtype=torch.int32, device="cuda")
        n_s = torch.empty(B, dtype=torch.int32, device="cuda")
        # two calls in a row with different uniforms: the second must not see anything of the first
        for call_serial in (0, 1):
            want_out, want_n = lib.hsd_verify_level(1, p, q, x, 7, call_serial)
            out_s.fill_(-7)
            n_s.fill_(-7)
            lib.hsd_verify_level_static(1, p, q, x, 7, call_serial, out_s, n_s)
            torch.cuda.synchronize()
            assert torch.equal(n_s, want_n), (dtype, call_serial)
            assert torch.equal(out_s, want_out), (dtype, call_serial)


def test_static_scratch_variant_rejects_what_does_not_fit(lib):
    # batch * (2 t + 1) rows of statistics must fit the 4096-row built-in array
    B, t, V = 512, 4, 16
    p = torch.zeros(B, t + 1, V, device="cuda")
    q = torch.zeros(B, t, V, device="cuda")
    x = torch.zeros(B, t, dtype=torch.int32, device="cuda")
    out = torch.empty(B, t + 1, dtype=torch.int32, device="cuda")
    n = torch.empty(B, dtype=torch.int32, device="cuda")
    with pytest.raises(lib.HsdError, match="built-in scratch"):
        lib.hsd_verify_level_static(1, p, q, x, 0, 0, out, n)
    lib.hsd_verify_level_static(1, p[:455].contiguous(), q[:455].contiguous(), x[:455].contiguous(), 0, 0, out, n)
    torch.cuda.synchronize()


@pytest.mark.parametrize("dtype,V", [("bf16", 64), ("fp32", 16)])
def test_static_scratch_variant_at_exactly_its_limit_and_without_allocating(lib, dtype, V):
    # batch * (2 t + 1) == 4096: the last row of statistics and the last counter of the built-in array are used
    B, t = 4096, 0
    p, _ = inputs.make_accept_logits(B, 1, V, seed=5, device="cuda", dtype=dtype)
    p = p[:, :1].contiguous()
    out = torch.full((B, 1), -7, dtype=torch.int32, device="cuda")
    n = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    want_out, want_n = lib.hsd_verify_level(1, p, None, None, 3, 0)
    lib.hsd_verify_level_static(1, p, None, None, 3, 0, out, n)          # first use: kernels loaded, address looked up
    torch.cuda.synchronize()
    assert torch.equal(out, want_out) and torch.equal(n, want_n)
    # the device's free memory is the same before and after a call: nothing was allocated (or freed)
    free_before, _ = torch.cuda.mem_get_info()
    lib.hsd_verify_level_static(1, p, None, None, 3, 1, out, n)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    want_out, want_n = lib.hsd_verify_level(1, p, None, None, 3, 1)
    assert torch.equal(out, want_out) and torch.equal(n, want_n)
