"""Repetition code: CUDA path vs the CPU oracle, element by element.

Bars: flags, majority selections and the no-majority count are bit-exact; the
decoded sum is within 1e-5 (max |u - u*| / max |u*|) of the oracle's fp64 sum of
the selections, and bit-equal to their fp32 left-to-right sum; encoded vectors
are within 1e-6 of the oracle's and bit-identical inside a group.
"""
import numpy as np
import pytest
import torch

import draco_inputs as di
from gpu_util import dev, fp32_sequential_sum, host, normwise
from oracle import draco_oracle as orc

pytestmark = pytest.mark.gpu

# (n, s, d): r | n; r does not divide n (groups of 8 and 7); one group of 15 (16-wide path);
# groups of 20 (streamed path); scalar paths (d % 4 != 0); d below one block; s = 0
SHAPES = [(15, 2, 100_000), (45, 3, 40_004), (15, 5, 5000), (40, 9, 3000), (15, 2, 1001), (9, 1, 7), (6, 0, 260),
          (105, 7, 2052)]


def _plan(n, s, d):
    import paper_1803_09877_b200 as dr
    return dr, dr.Plan(n, s, d, dr.REP)


@pytest.mark.parametrize("n,s,d", SHAPES)
def test_groups_match_oracle(n, s, d):
    dr, plan = _plan(n, s, d)
    assert plan.groups() == orc.rep_groups(n, s)


@pytest.mark.parametrize("n,s,d", SHAPES)
def test_encode_parity(n, s, d):
    dr, plan = _plan(n, s, d)
    G = di.gradient_rows(0xD2AC0 + n, n, d)
    Z = torch.empty((n, d), dtype=torch.float32, device="cuda")
    plan.encode(dev(G), Z)
    torch.cuda.synchronize()
    Zg, Zo = host(Z), orc.rep_encode(G, n, s)
    assert normwise(Zg, Zo) <= 1e-6
    for first, size in orc.rep_groups(n, s):
        for j in range(first + 1, first + size):
            np.testing.assert_array_equal(Zg[j].view(np.uint32), Zg[first].view(np.uint32))


def _received(n, s, d, seed, n_adv, models=None):
    G = di.gradient_rows(seed, n, d)
    R = orc.rep_encode(G, n, s)
    adv = di.choose_adversaries(seed + 1, n, n_adv)
    models = models or [di.ADV_REVGRAD]
    model = [models[k % len(models)] for k in range(n_adv)]
    param = [{di.ADV_REVGRAD: 100.0, di.ADV_CONST: 1e4, di.ADV_GAUSS: 1e3}[m] for m in model]
    di.apply_adversaries(R, adv, model, param, seed=seed + 2)
    return G, R, adv


@pytest.mark.parametrize("n,s,d", SHAPES)
@pytest.mark.parametrize("full", [True, False])
def test_decode_parity(n, s, d, full):
    dr, plan = _plan(n, s, d)
    n_adv = s if full else max(s - 1, 0)
    G, R, adv = _received(n, s, d, 31 * n + s, n_adv, [di.ADV_REVGRAD, di.ADV_CONST, di.ADV_GAUSS])
    want = orc.rep_decode(R, n, s)
    Rd = dev(R)
    g = len(orc.rep_groups(n, s))
    u = torch.empty(d, dtype=torch.float32, device="cuda")
    maj = torch.empty((g, d), dtype=torch.float32, device="cuda")
    flags = torch.full((n,), 7, dtype=torch.uint8, device="cuda")
    plan.rep_vote(Rd, u, maj, flags)
    info = plan.info()
    np.testing.assert_array_equal(host(flags).astype(bool), want["flags"])
    assert sorted(np.flatnonzero(host(flags))) == sorted(adv.tolist())
    np.testing.assert_array_equal(host(maj).view(np.uint32), want["maj"].view(np.uint32))
    assert info["no_majority"] == want["no_majority"] == 0 and info["n_flagged"] == n_adv and info["status"] == 0
    assert normwise(host(u), want["u"]) <= 1e-5
    np.testing.assert_array_equal(host(u).view(np.uint32), fp32_sequential_sum(want["maj"]).view(np.uint32))
    exact = G.astype(np.float64).sum(axis=0)
    assert normwise(host(u), exact) <= 1e-5
    # the public entry points give the same answers
    u2 = torch.empty_like(u)
    f2 = torch.empty_like(flags)
    plan.decode(Rd, None, u2)
    plan.locate(Rd, None, f2)
    torch.cuda.synchronize()
    assert torch.equal(u2, u) and torch.equal(f2, flags)
    u3 = torch.empty_like(u)
    f3 = torch.empty_like(flags)
    plan.locate_decode(Rd, None, f3, u3)
    torch.cuda.synchronize()
    assert torch.equal(u3, u) and torch.equal(f3, flags)


def test_beyond_s_is_reported_not_hidden():
    n, s, d = 15, 2, 4096
    dr, plan = _plan(n, s, d)
    G = di.gradient_rows(5, n, d)
    Z = orc.rep_encode(G, n, s)
    # s + 1 identical colluders in one group win the vote (Theorem 1: redundancy 2 s + 1 is not enough)
    R = Z.copy()
    R[[5, 6, 7]] = np.float32(1e4)
    want = orc.rep_decode(R, n, s)
    u = torch.empty(d, dtype=torch.float32, device="cuda")
    flags = torch.empty(n, dtype=torch.uint8, device="cuda")
    plan.locate_decode(dev(R), None, flags, u)
    np.testing.assert_array_equal(host(flags).astype(bool), want["flags"])
    assert normwise(host(u), want["u"]) <= 1e-5
    assert normwise(host(u), G.astype(np.float64).sum(axis=0)) > 1.0
    # s + 1 unrelated noise vectors leave no strict majority: warning status and a count
    R = Z.copy()
    di.apply_adversaries(R, [5, 6, 7], [di.ADV_GAUSS] * 3, [1e3] * 3, seed=8)
    want = orc.rep_decode(R, n, s)
    g = len(orc.rep_groups(n, s))
    maj = torch.empty((g, d), dtype=torch.float32, device="cuda")
    plan.rep_vote(dev(R), u, maj, flags)
    info = plan.info()
    assert info["no_majority"] == want["no_majority"] == d and info["status"] == dr.binding.ENOMAJ
    np.testing.assert_array_equal(host(maj).view(np.uint32), want["maj"].view(np.uint32))
    np.testing.assert_array_equal(host(flags).astype(bool), want["flags"])


def test_bit_pattern_equality_signed_zero_and_nan():
    n, s, d = 3, 1, 64
    dr, plan = _plan(n, s, d)
    R = np.zeros((n, d), dtype=np.float32)
    R[0] = -0.0
    R[:, 32:] = np.nan
    R[2, 32:] = 1.0
    want = orc.rep_decode(R, n, s)
    maj = torch.empty((1, d), dtype=torch.float32, device="cuda")
    flags = torch.empty(n, dtype=torch.uint8, device="cuda")
    plan.rep_vote(dev(R), None, maj, flags)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(host(maj).view(np.uint32), want["maj"].view(np.uint32))
    np.testing.assert_array_equal(host(flags).astype(bool), want["flags"])


def test_full_size_resnet18_config_sampled():
    """n = 45, s = 3, d = 11.7 M, gradients N(0, sigma = 0.1), reversed-gradient and constant
    adversaries mixed: inputs generated on the device, checked on a coordinate sample."""
    import paper_1803_09877_b200 as dr
    n, s, d = 45, 3, 11_700_000
    plan = dr.Plan(n, s, d, dr.REP)
    seed = 0xD2AC0 + 3
    G = torch.empty((n, d), dtype=torch.float32, device="cuda")
    dr.generate(G, n, d, mean=0.0, std=0.1, seed=seed)
    Z = torch.empty_like(G)
    plan.encode(G, Z)
    adv = di.choose_adversaries(seed + 1, n, s)
    model = [di.ADV_REVGRAD, di.ADV_CONST, di.ADV_REVGRAD]
    param = [100.0, 1e4, 100.0]
    plan.corrupt(Z, adv, model, param, seed=seed + 2)
    u = torch.empty(d, dtype=torch.float32, device="cuda")
    flags = torch.empty(n, dtype=torch.uint8, device="cuda")
    plan.locate_decode(Z, None, flags, u)
    info = plan.info()
    assert sorted(np.flatnonzero(host(flags))) == adv.tolist() and info["no_majority"] == 0
    rng = np.random.default_rng(1)
    idx = np.unique(np.concatenate([np.arange(4096), np.arange(d - 4096, d), rng.integers(0, d, 1_000_000)]))
    Gs = di.gradient_rows(seed, n, d, 0.0, 0.1, idx=idx)
    np.testing.assert_array_equal(host(G[:, idx]), Gs)                      # same inputs on both sides
    Rs = orc.rep_encode(Gs, n, s)
    di.apply_adversaries(Rs, adv, model, param, seed=seed + 2, idx=idx)
    assert normwise(host(Z[:, idx]), Rs) <= 1e-6
    want = orc.rep_decode(Rs, n, s)
    assert normwise(host(u[idx]), want["u"]) <= 1e-5
    assert normwise(host(u[idx]), Gs.astype(np.float64).sum(axis=0)) <= 1e-5


def test_decode_fused_with_model_update():
    """w <- w - scale * D(R) in the vote kernel's epilogue (the SGD step of Section 2)."""
    n, s, d = 15, 2, 50_004
    dr, plan = _plan(n, s, d)
    G, R, adv = _received(n, s, d, 77, s)
    want = orc.rep_decode(R, n, s)
    w0 = di.gradient_rows(78, 1, d)[0]
    w = dev(w0)
    scale = np.float32(0.01 / n)
    plan.decode_update(dev(R), None, w, float(scale))
    torch.cuda.synchronize()
    expect = w0.astype(np.float64) - float(scale) * want["u"]
    assert normwise(host(w), expect) <= 1e-6
    u = torch.empty(d, dtype=torch.float32, device="cuda")
    plan.decode(dev(R), None, u)
    step = (w0.astype(np.float64) - np.float64(scale) * host(u).astype(np.float64)).astype(np.float32)
    np.testing.assert_allclose(host(w), step, rtol=2e-7, atol=0)


def test_largest_supported_n():
    n, s, d = 128, 3, 2052                                   # 18 groups of 8 / 7
    dr, plan = _plan(n, s, d)
    G, R, adv = _received(n, s, d, 99, s)
    want = orc.rep_decode(R, n, s)
    u = torch.empty(d, dtype=torch.float32, device="cuda")
    flags = torch.empty(n, dtype=torch.uint8, device="cuda")
    plan.locate_decode(dev(R), None, flags, u)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(host(flags).astype(bool), want["flags"])
    assert normwise(host(u), want["u"]) <= 1e-5
    import ctypes
    h = ctypes.c_void_p()
    assert dr.binding.lib.draco_plan_create(129, 1, 10, dr.REP, ctypes.byref(h)) == dr.binding.EINVAL
