"""draco_cyc_project_noalloc: the projection for callers that may not allocate device memory
(their GPU memory belongs to another allocator, or they cannot afford an allocation's implicit
synchronisation inside the step loop).  It keeps its scratch in an array built into the library,
so this test checks, through the C ABI, that it returns what the plan-based entry point returns
and what the CPU oracle's projection gives, on calls in a row with different inputs (a later call
must not see an earlier call's leftovers), up to the largest number of nodes it accepts.
Collected last on purpose: a failure here cannot hide another test's result under `-x`.
"""
import ctypes

import numpy as np
import pytest
import torch

import draco_inputs as di
from oracle import draco_oracle as orc

pytestmark = pytest.mark.gpu


def _project_both_ways(dr, n, s, d, seed):
    Rh = di.complex_rows(seed, n, d, std=3.0)
    fh = di.projection_vector(seed + 1, d)
    R = torch.from_numpy(Rh.view(np.float32)).cuda()
    f = torch.from_numpy(fh).cuda()
    plan = dr.Plan(n, s, d, dr.CYC)
    e_plan = torch.zeros(3 * n, dtype=torch.float64, device="cuda")          # n (re, im) pairs, then n squared norms q_j
    plan.cyc_project(R, f, e_plan)
    e_static = torch.full((3 * n,), float("nan"), dtype=torch.float64, device="cuda")
    dr.cyc_project_noalloc(n, d, R, f, e_static)
    torch.cuda.synchronize()
    return e_plan.cpu().numpy(), e_static.cpu().numpy(), orc.cyc_project(Rh, fh), orc.cyc_project_energy(Rh)


def test_noalloc_projection_matches_plan_projection_and_oracle_on_calls_in_a_row():
    import paper_1803_09877_b200 as dr
    # vector path, the odd-d scalar path of the few-rows kernel, then more than 64 nodes (two launches over half the
    # rows each into the one array), the last at the entry point's limit of 128 nodes
    for call, (n, s, d) in enumerate([(45, 5, 300_004), (15, 2, 4099), (105, 7, 6150), (128, 2, 4099)]):
        want, got, e_oracle, q_oracle = _project_both_ways(dr, n, s, d, seed=100 + call)
        assert np.all(np.isfinite(got))
        # against the oracle's definition e_j = sum_i f_i R[j][i], q_j = sum_i |R[j][i]|^2
        assert np.abs(got[: 2 * n].view(np.complex128) - e_oracle).max() <= 1e-6 * np.abs(e_oracle).max()
        assert np.abs(got[2 * n:] - q_oracle).max() <= 1e-5 * q_oracle.max()
        we, ge = want[: 2 * n].view(np.complex128), got[: 2 * n].view(np.complex128)
        assert np.abs(ge - we).max() <= 1e-6 * np.abs(we).max()                # tolerance of the projection parity tests
        assert np.abs(ge - we).max() <= 1e-12 * np.abs(we).max()               # same kernel; only the number of block partials differs
        # the squared norms are a yardstick (few-row plans add their fp32 terms in fp32): a few digits
        assert np.abs(got[2 * n:] - want[2 * n:]).max() <= 1e-5 * want[2 * n:].max() and want[2 * n:].min() > 0


def test_noalloc_projection_rejects_sizes_beyond_its_fixed_capacity():
    import paper_1803_09877_b200 as dr
    from paper_1803_09877_b200 import binding
    buf = torch.zeros(1024, dtype=torch.float32, device="cuda")
    e = torch.zeros(512, dtype=torch.float64, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    rc = binding.lib.draco_cyc_project_noalloc(129, 4, buf.data_ptr(), buf.data_ptr(), e.data_ptr(), st)
    assert rc == binding.ELIMIT and b"capacity" in binding.lib.draco_strerror(rc)
    assert binding.lib.draco_cyc_project_noalloc(0, 4, buf.data_ptr(), buf.data_ptr(), e.data_ptr(), st) == binding.EINVAL
    assert binding.lib.draco_cyc_project_noalloc(4, 4, None, buf.data_ptr(), e.data_ptr(), st) == binding.EINVAL
