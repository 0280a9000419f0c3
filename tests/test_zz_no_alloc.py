"""The allocation-free statistics entry point against the ordinary one.

Some users of the library cannot let it allocate: their device memory belongs to a pool of their
own, or they are inside a section that must not meet the device-wide synchronisation of
cudaMalloc.  abs_test_stats_noalloc serves them with a fixed scratch array inside the library.
This test calls it through the C ABI twice in a row (the second call finds the first call's
partial sums still in the array) and compares each result with abs_test_stats on the same input.
The allocation-free call only has the tiled and the alignment-free kernel, so for bf16 rows with
b <= 256 and for any b > 256 (the second case below) the two entry points run different kernels
and agree to rounding, not to the bit: the check uses the suite's tolerances, 1e-5 for fp32 and
1e-3 for bf16 input.  It also checks that
device memory in use does not change across a call (once the first call has made the runtime
place the fixed array on the GPU) and that oversize problems are refused.
The file sorts last so that a failure here cannot hide the results of the other tests.
"""
import pytest
import torch

import paper_2406_13936_b200 as pkg
from paper_2406_13936_b200 import inputs

pytestmark = pytest.mark.gpu

KEYS = ("gbar_sq", "var_norm", "var_ip", "var_orth", "sum_sq")


def _compare(G, tol=1e-5, check_memory=True):
    M, _, d = G.shape
    ctx = pkg.Context(0)
    try:
        ref_stats, ref_gbar = ctx.new_stats(M), torch.empty((M, d), device="cuda")
        ctx.abs_test_stats(G, ref_stats, ref_gbar)
        torch.cuda.synchronize()
        ref = pkg.stats_to_dicts(ref_stats)
    finally:
        ctx.close()
    stats = torch.zeros((M, 7), dtype=torch.float64, device="cuda")
    gbar = torch.empty((M, d), device="cuda")
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    pkg.abs_test_stats_noalloc(G, stats, gbar)
    torch.cuda.synchronize()
    if check_memory:                                              # nothing was allocated on the device
        assert torch.cuda.mem_get_info()[0] == free_before
    got = pkg.stats_to_dicts(stats)
    for g, r in zip(got, ref):
        assert g["rows"] == r["rows"] and g["status"] == r["status"] == 0
        for key in KEYS:
            assert abs(g[key] - r[key]) <= tol * abs(r[key])
    assert torch.allclose(gbar, ref_gbar, rtol=1e-5, atol=1e-6 * ref_gbar.abs().max().item())


def test_two_calls_in_a_row_match_the_context_entry_point():
    first = inputs.gaussian_rows(41, 3, 64, 30000, 1.0, device="cuda")
    second = inputs.gaussian_rows(42, 2, 300, 5000, 3.0, device="cuda").to(torch.bfloat16)
    # The first call on a device resolves the scratch address; with CUDA's lazy module loading that is
    # also the moment the runtime places the fixed array on the GPU, so free memory is compared
    # from the second call on.
    _compare(first, check_memory=False)
    _compare(second, tol=1e-3)      # different shape: the array still holds the first call's sums
    _compare(first)


def test_unaligned_input_uses_the_same_scratch():
    buf = torch.zeros(2 * 9 * 1001 + 1, device="cuda")
    G = buf[1:].view(2, 9, 1001)
    G.copy_(inputs.gaussian_rows(43, 2, 9, 1001, 1.0, device="cuda"))
    _compare(G)


def test_sizes_beyond_the_fixed_scratch_are_refused():
    stats = torch.zeros((1, 7), dtype=torch.float64, device="cuda")
    with pytest.raises(pkg.AbsError, match="b <= 2048"):
        pkg.abs_test_stats_noalloc(torch.zeros((1, 2049, 8), device="cuda"), stats)
    with pytest.raises(pkg.AbsError, match="M <= 64"):
        pkg.abs_test_stats_noalloc(torch.zeros((65, 2, 8), device="cuda"), torch.zeros((65, 7), dtype=torch.float64, device="cuda"))
    with pytest.raises(pkg.AbsError):
        pkg.abs_test_stats_noalloc(torch.zeros((1, 1, 8), device="cuda"), stats)
