"""The CUDA generator / corruptor produce the same bits as the numpy definition."""
import numpy as np
import pytest
import torch

import draco_inputs as di
from gpu_util import dev, host

pytestmark = pytest.mark.gpu


def test_generate_matches_numpy_bit_for_bit():
    import paper_1803_09877_b200 as dr
    for rows, length, row0, mean, std, seed in [(3, 1000, 0, 0.0, 1.0, 1), (2, 4099, 5, 1.0, 1.0, 0xD2AC0),
                                                (1, 17, 0, 0.25, 0.1, 2 ** 63 + 11)]:
        out = torch.empty((rows, length), dtype=torch.float32, device="cuda")
        dr.generate(out, rows, length, row0=row0, mean=mean, std=std, seed=seed)
        torch.cuda.synchronize()
        want = di.approx_normal_rows(seed, range(row0, row0 + rows), 0, length, mean, std)
        np.testing.assert_array_equal(host(out).view(np.uint32), want.view(np.uint32))


def test_generate_f_and_complex_views():
    import paper_1803_09877_b200 as dr
    d = 3000
    f = torch.empty(d, dtype=torch.float32, device="cuda")
    dr.generate(f, 1, d, mean=1.0, std=1.0, seed=77)
    np.testing.assert_array_equal(host(f), di.projection_vector(77, d))
    R = torch.empty((4, 2 * d), dtype=torch.float32, device="cuda")
    dr.generate(R, 4, 2 * d, std=3.0, seed=78)
    np.testing.assert_array_equal(host(R, complex64=True), di.complex_rows(78, 4, d, std=3.0))


@pytest.mark.parametrize("code", [0, 1])
def test_corrupt_matches_numpy(code):
    import paper_1803_09877_b200 as dr
    n, s, d = 9, 2, 1234
    plan = dr.Plan(n, s, d, code)
    R0 = di.complex_rows(5, n, d) if code == dr.CYC else di.gradient_rows(5, n, d)
    adv, model, param = [1, 4, 8], [dr.ADV_REVGRAD, dr.ADV_CONST, dr.ADV_GAUSS], [100.0, 1e4, 1e3]
    Rd = dev(R0)
    plan.corrupt(Rd, adv, model, param, seed=99)
    torch.cuda.synchronize()
    want = di.apply_adversaries(R0.copy(), adv, model, param, seed=99)
    got = host(Rd, complex64=(code == dr.CYC))
    np.testing.assert_array_equal(got.view(np.uint32), want.view(np.uint32))


def test_corruptor_rejects_duplicate_and_out_of_range_nodes():
    """All adversarial rows are rewritten by one launch, so a node may appear once only."""
    import paper_1803_09877_b200 as dr
    from paper_1803_09877_b200 import binding
    n, s, d = 9, 2, 64
    plan = dr.Plan(n, s, d, dr.REP)
    Z = torch.zeros((n, d), dtype=torch.float32, device="cuda")
    with pytest.raises(binding.DracoError, match="invalid argument"):
        plan.corrupt(Z, [3, 3], [dr.ADV_CONST] * 2, [1.0] * 2)
    with pytest.raises(binding.DracoError, match="invalid argument"):
        plan.corrupt(Z, [9], [dr.ADV_CONST], [1.0])
    with pytest.raises(binding.DracoError, match="invalid argument"):
        plan.corrupt(Z, [1], [7], [1.0])
    torch.cuda.synchronize()
    assert float(Z.abs().max()) == 0.0                     # nothing was launched
    plan.corrupt(Z, [1, 8], [dr.ADV_CONST] * 2, [2.0, 3.0])
    torch.cuda.synchronize()
    assert Z[1].eq(2.0).all() and Z[8].eq(3.0).all() and float(Z[[0, 2, 3, 4, 5, 6, 7]].abs().max()) == 0.0
