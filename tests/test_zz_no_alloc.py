"""gaf_cosdist_static: the entry point for callers that cannot allocate device
memory (code inside a frozen memory pool, plug-ins called where cudaMalloc would
stall the device).  It must give what gaf_cosdist and the CPU oracle give, call after call, although
its scratch is one array shared by all calls that still holds the previous
call's contents.  This file sorts last on purpose: a run that stops at the first
failure has then already been through every other test."""
import ctypes

import pytest
import torch

import paper_2412_18052_b200 as gaf
from oracle import gaf_oracle as orc
from paper_2412_18052_b200 import workloads
from parity import DIST_ATOL


def test_static_rejects_sizes_beyond_its_limit():
    """Host-side check: nothing is launched and no GPU is needed."""
    L = gaf.binding.lib()
    A = 0x7000_0000_0000
    too_big = (1 << 31) + 1
    assert L.gaf_cosdist_static(A, A + (1 << 36), too_big, 1, A + (1 << 40), None, None) == 8
    assert b"fixed limit" in L.gaf_error_string(8)
    assert L.gaf_cosdist_static(A, A + 4096, -1, 0, A + 8192, None, None) == 1
    assert L.gaf_cosdist_static(A + 4, A + 4096, 10, 0, A + 8192, None, None) == 2


@pytest.mark.gpu
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_static_matches_workspace_entry_point_twice_in_a_row(dtype):
    ws = gaf.new_workspace(2, 1 << 20, gaf.GAF_F32)
    dist_s = torch.empty(1, dtype=torch.float32, device="cuda")
    stats_s = torch.empty(3, dtype=torch.float64, device="cuda")
    # two different problems back to back: the second call meets the first one's leftovers,
    # including a different number of CTAs and a raised zero-norm status
    cases = [workloads.mixture(2, 3_000_017, dtype, [0.7, 0.2], seed=21, device="cuda").grads,
             workloads.mixture(2, 40_003, dtype, [0.1, -0.6], seed=22, device="cuda").grads]
    zero = [cases[1][0], torch.zeros_like(cases[1][0])]
    for x, y in (cases[0], zero, cases[1], cases[0]):
        for _ in range(2):
            want_d, want_s = gaf.gaf_cosdist(x, y, ws)
            gaf.gaf_cosdist_static(x, y, dist_s, stats_s)
            torch.cuda.synchronize()
            assert abs(float(dist_s.item()) - float(want_d.item())) <= DIST_ATOL
            # ... and what the CPU oracle gives for the same bits
            oracle_d, _ = orc.cosdist(workloads.as_numpy_bits(x), workloads.as_numpy_bits(y))
            assert abs(float(dist_s.item()) - oracle_d) <= DIST_ATOL
            scale = float((want_s[1] * want_s[2]).sqrt().item()) + 1e-300
            assert float((stats_s - want_s).abs().max().item()) <= 1e-6 * scale
    # empty input and NULL stats
    e = torch.empty(0, dtype=cases[0][0].dtype, device="cuda")
    gaf.gaf_cosdist_static(e, e, dist_s)
    assert float(dist_s.item()) == 1.0
