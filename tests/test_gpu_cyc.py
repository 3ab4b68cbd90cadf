"""Cyclic code: CUDA path vs the CPU oracle.

Bars (max |a - b| / max |b| unless said otherwise):
  W table                 <= 1e-12 of max |W|
  encode                  <= 1e-6 per worker vector (fp32 FMA chains of 2 s + 1 terms)
  projection e = f R      <= 1e-6 (fp32 products, fp64 sums)
  flags, locator rank     exact
  decode vector b         <= 1e-9
  decode on identical R, identical flags   <= 1e-4 (the stated tolerance; observed ~1e-7)
  end to end vs the exact sum   <= 1e-4 at (15, 2); at (45, 5) complex64 transport limits any
                          implementation to ~1e-3, so the bar there is 2 x the oracle's own error.
"""
import numpy as np
import pytest
import torch

import draco_inputs as di
from gpu_util import dev, host, normwise
from oracle import draco_oracle as orc

pytestmark = pytest.mark.gpu

# (n, s, d): config-1-like; several tiles + ragged tail; 4 does not divide d (generic encoder,
# scalar projection / recovery); d odd; d below one tile; n = 2 s + 1; s = 0; larger s paths
SHAPES = [(15, 2, 100_000), (45, 5, 20_484), (45, 3, 6150), (15, 2, 4098), (15, 2, 1001), (9, 1, 5), (5, 2, 300),
          (6, 0, 516), (15, 7, 2048), (21, 4, 4100), (33, 6, 2052), (20, 8, 1028)]


def _plan(n, s, d):
    import paper_1803_09877_b200 as dr
    return dr, dr.Plan(n, s, d, dr.CYC)


@pytest.mark.parametrize("n,s", [(4, 1), (15, 2), (45, 3), (45, 5), (15, 7), (105, 7), (20, 8)])
def test_W_table(n, s):
    dr, plan = _plan(n, s, 8)
    W, Wo = plan.cyc_W(), orc.cyc_W(n, s)
    assert np.abs(W - Wo).max() <= 1e-12 * np.abs(Wo).max()


@pytest.mark.parametrize("n,s,d", SHAPES)
def test_encode_parity(n, s, d):
    dr, plan = _plan(n, s, d)
    G = di.gradient_rows(0xD2AC0 + n + s, n, d)
    Z = torch.empty((n, 2 * d), dtype=torch.float32, device="cuda")
    plan.encode(dev(G), Z)
    torch.cuda.synchronize()
    Zg = host(Z, complex64=True)
    Zo = orc.cyc_encode(G, n, s, dtype=np.complex128)
    for j in range(n):
        assert np.abs(Zg[j] - Zo[j]).max() <= 1e-6 * np.abs(Zo[j]).max(), j


def _received(n, s, d, seed, n_adv, model=di.ADV_REVGRAD, param=100.0):
    G = di.gradient_rows(seed, n, d)
    R = orc.cyc_encode(G, n, s)                            # complex64 worker vectors
    adv = di.choose_adversaries(seed + 1, n, n_adv)
    if model == di.ADV_GAUSS:
        param = param * float(np.abs(R).max()) / 1e3      # noise far above the vectors' own scale
    di.apply_adversaries(R, adv, [model] * n_adv, [param] * n_adv, seed=seed + 2)
    return G, R, adv, di.projection_vector(seed + 3, d)


@pytest.mark.parametrize("n,s,d", SHAPES)
@pytest.mark.parametrize("n_adv_mode", ["s", "fewer", "none"])
def test_locate_and_decode_parity_on_identical_R(n, s, d, n_adv_mode):
    dr, plan = _plan(n, s, d)
    n_adv = {"s": s, "fewer": max(s - 1, 0) if s < 3 else s - 2, "none": 0}[n_adv_mode]
    model = di.ADV_GAUSS if (n + s) % 2 else di.ADV_REVGRAD
    G, R, adv, f = _received(n, s, d, 17 * n + s, n_adv, model, 1e3 if model == di.ADV_GAUSS else 100.0)
    want = orc.cyc_locate(R, f, n, s)
    Rd, fd = dev(R), dev(f)
    # projection
    e = torch.empty(3 * n, dtype=torch.float64, device="cuda")        # n (re, im) pairs, then n squared norms q_j
    plan.cyc_project(Rd, fd, e)
    eg = host(e)[: 2 * n].view(np.complex128)
    assert np.abs(eg - want["e"]).max() <= 1e-6 * np.abs(want["e"]).max()
    qo = orc.cyc_project_energy(R)
    assert np.abs(host(e)[2 * n:] - qo).max() <= 1e-5 * qo.max()
    # the device forms every product f_i R[j][i] exactly (fp32 x fp32 in fp64) and adds in fp64: only the order of the
    # additions separates it from the oracle, so its e carries the rounding noise of the complex64 vectors and no more
    assert np.abs(eg - want["e"]).max() <= 1e-11 * np.sqrt(qo.max() * 2 * d)
    assert np.abs(host(e)[2 * n:] - qo).max() <= 1e-12 * qo.max()
    # locator
    flags = torch.full((n,), 9, dtype=torch.uint8, device="cuda")
    plan.locate(Rd, fd, flags)
    info = plan.info()
    fg = host(flags).astype(bool)
    tol = 1e-6 * want["scale"]
    sv = want.get("sv", np.zeros(0))
    assert all(x > 3 * tol or x < tol / 3 for x in sv), "test input sits too close to the rank cutoff"
    assert want["margin"] > 10, "test input: |t| of flagged and unflagged nodes too close"
    np.testing.assert_array_equal(fg, want["flags"])
    assert sorted(np.flatnonzero(fg)) == adv.tolist()
    assert info["locator_rank"] == want["rank"] == n_adv and info["n_flagged"] == n_adv
    assert abs(info["scale"] - want["scale"]) <= 1e-5 * want["scale"]
    # |t| of the weakest flagged node over |t| of the strongest unflagged one
    if 0 < want["rank"] < n:
        assert info["locator_margin"] > 10
        # the denominator is the noise left on an honest node: the same order of magnitude on both sides, no more
        assert 0.1 < info["locator_margin"] / want["margin"] < 10 or min(info["locator_margin"], want["margin"]) > 1e6
    else:
        assert info["locator_margin"] == 1e300
    # split entry points agree with the fused one
    flags2 = torch.empty_like(flags)
    plan.cyc_locate_from_projection(e, flags2)
    torch.cuda.synchronize()
    assert torch.equal(flags, flags2)
    # decode with the same flags on the same R
    u = torch.empty(d, dtype=torch.float32, device="cuda")
    plan.decode(Rd, flags, u)
    info = plan.info()
    assert info["status"] == 0 and info["n_active"] == n - n_adv
    b = plan.cyc_decode_vector()
    bo = orc.cyc_decode_vector(n, s, want["flags"])
    assert np.abs(b - bo).max() <= 1e-9 * np.abs(bo).max()
    uo = orc.cyc_decode(R, n, s, want["flags"])
    assert normwise(host(u), uo) <= 1e-4
    assert normwise(host(u), uo) <= 1e-6                    # what fp64 accumulation actually delivers
    # the decoder's self-check: Im(u-hat) on one 64-coordinate run in eight, against the oracle's u-hat there
    uhat = orc.cyc_recover(R, bo)
    sampled = (np.arange(d) // 64) % 8 == 0
    im_o, re_o = np.abs(uhat.imag[sampled]).max(), np.abs(uhat.real[sampled]).max()
    assert abs(info["re_max"] - re_o) <= 1e-6 * re_o
    assert abs(info["im_residual"] - im_o) <= 1e-3 * im_o + 1e-12 * re_o
    assert info["im_residual"] <= 1e-2 * info["re_max"]       # an honest U: rounding residue only
    u2 = torch.empty_like(u)
    f2 = torch.empty_like(flags)
    plan.locate_decode(Rd, fd, f2, u2)
    torch.cuda.synchronize()
    assert torch.equal(u2, u) and torch.equal(f2, flags)


# odd d: the one-coordinate-per-thread encoder (fp64 taps) and the scalar projection / recovery paths
@pytest.mark.parametrize("n,s,d,bar", [(15, 2, 100_000, 1e-4), (15, 1, 30_000, 1e-4), (45, 5, 30_000, None),
                                        (45, 3, 30_000, None), (45, 3, 20_001, None), (45, 5, 20_001, None),
                                        (20, 8, 10_002, None)])
def test_pipeline_against_exact_sum(n, s, d, bar):
    """encode -> corrupt -> locate -> decode, all on the device, against G 1_P."""
    dr, plan = _plan(n, s, d)
    seed = 900 + n + s
    G = di.gradient_rows(seed, n, d)
    adv = di.choose_adversaries(seed + 1, n, s)
    f = di.projection_vector(seed + 3, d)
    Gd, fd = dev(G), dev(f)
    Z = torch.empty((n, 2 * d), dtype=torch.float32, device="cuda")
    plan.encode(Gd, Z)
    plan.corrupt(Z, adv, [di.ADV_REVGRAD] * s, [100.0] * s, seed=seed + 2)
    flags = torch.empty(n, dtype=torch.uint8, device="cuda")
    u = torch.empty(d, dtype=torch.float32, device="cuda")
    plan.locate_decode(Z, fd, flags, u)
    torch.cuda.synchronize()
    assert sorted(np.flatnonzero(host(flags))) == adv.tolist()
    exact = G.astype(np.float64).sum(axis=0)
    err = normwise(host(u), exact)
    # the oracle's own end-to-end error with complex64 worker vectors
    Ro = orc.cyc_encode(G, n, s)
    di.apply_adversaries(Ro, adv, [di.ADV_REVGRAD] * s, [100.0] * s, seed=seed + 2)
    out = orc.cyc_decode_full(Ro, f, n, s)
    assert sorted(np.flatnonzero(out["flags"])) == adv.tolist()
    floor = normwise(out["u"], exact)
    if bar is not None:
        assert err <= bar and floor <= bar
    else:
        assert err <= 2.0 * floor + 1e-6, (err, floor)
    assert np.abs(host(u)).max() > 0


def test_too_many_flags_is_refused_with_zero_output():
    n, s, d = 15, 2, 2048
    dr, plan = _plan(n, s, d)
    R = di.complex_rows(3, n, d)
    flags = np.zeros(n, dtype=np.uint8)
    flags[: 2 * s + 1] = 1
    u = torch.full((d,), 5.0, dtype=torch.float32, device="cuda")
    plan.decode(dev(R), dev(flags), u)
    info = plan.info()
    assert info["status"] == dr.binding.ETOOMANY and info["n_active"] == 0
    assert float(u.abs().max()) == 0.0
    # 2 s flagged (erasure decoding) still works on any R: u = Re(b^T R)
    flags[2 * s] = 0
    plan.decode(dev(R), dev(flags), u)
    # not refused; R is random rather than a set of coded vectors, so its u-hat is as complex as it is real and the
    # decoder's self-check says so
    assert plan.info()["status"] == dr.binding.EUNSURE
    uo = orc.cyc_decode(R, n, s, flags.astype(bool))
    assert normwise(host(u), uo) <= 1e-6


def test_beyond_s_fails_visibly():
    """s + 1 adversaries: the decoder cannot return the true sum (Theorem 1)."""
    n, s, d = 15, 2, 8192
    dr, plan = _plan(n, s, d)
    G = di.gradient_rows(11, n, d)
    R = orc.cyc_encode(G, n, s)
    adv = [1, 6, 12]
    di.apply_adversaries(R, adv, [di.ADV_REVGRAD] * 3, [100.0] * 3, seed=0)
    f = di.projection_vector(12, d)
    flags = torch.empty(n, dtype=torch.uint8, device="cuda")
    u = torch.empty(d, dtype=torch.float32, device="cuda")
    plan.locate_decode(dev(R), dev(f), flags, u)
    info = plan.info()
    wrong_set = sorted(np.flatnonzero(host(flags))) != adv
    wrong_sum = normwise(host(u), G.astype(np.float64).sum(axis=0)) > 1e-3
    assert wrong_set or wrong_sum
    # and the caller can see it without knowing the truth: an adversary left in U makes u-hat complex
    assert info["im_residual"] > 0.1 * info["re_max"]
    assert info["status"] == dr.binding.EUNSURE


def test_undetected_adversary_shows_in_the_self_checks():
    """Six noise adversaries, three of them two nodes apart, at n = 44: the sixth singular value of the syndrome
    system sinks below the rank cutoff of complex64 vectors, oracle and GPU both end with the same wrong set, and
    the sum is wrong.  The margin between flagged and unflagged |t_j| and the imaginary residue of the decode both say so."""
    n, s, d, seed = 44, 6, 257, 892766506
    dr, plan = _plan(n, s, d)
    G = di.gradient_rows(seed, n, d)
    Z = torch.empty(n, 2 * d, dtype=torch.float32, device="cuda")
    plan.encode(dev(G), Z)
    adv = di.choose_adversaries(seed + 1, n, s)
    plan.corrupt(Z, adv, [di.ADV_GAUSS] * s, [1e3] * s, seed=seed + 2)
    f = di.projection_vector(seed + 3, d)
    flags = torch.empty(n, dtype=torch.uint8, device="cuda")
    u = torch.empty(d, dtype=torch.float32, device="cuda")
    plan.locate_decode(Z, dev(f), flags, u)
    info = plan.info()
    want = orc.cyc_locate(host(Z).view(np.complex64), f, n, s)
    np.testing.assert_array_equal(host(flags).astype(bool), want["flags"])
    # the first pass sees five of the six; the pass with erasures adds one more node, but the set is still not the planted one
    assert want["ranks"][0] == s - 1 and sorted(np.flatnonzero(want["flags"])) != adv.tolist()
    assert info["locator_rank"] == want["rank"]
    assert normwise(host(u), G.astype(np.float64).sum(axis=0)) > 1.0
    assert info["locator_margin"] < 3 and want["margin"] < 3
    assert info["im_residual"] > 0.1 * info["re_max"]
    assert info["status"] == dr.binding.EUNSURE              # the warning a caller acts on
    assert 0 < info["svd_sweeps"] < 60                       # the singular-value iteration itself converged


def test_host_pipeline_matches_device_pipeline():
    n, s, d = 15, 2, 300_000
    dr, plan = _plan(n, s, d)
    seed = 4242
    G = di.gradient_rows(seed, n, d)
    f = di.projection_vector(seed + 3, d)
    adv = di.choose_adversaries(seed + 1, n, s)
    Z = torch.empty((n, 2 * d), dtype=torch.float32, device="cuda")
    u_host = np.empty(d, dtype=np.float32)
    flags_host = np.empty(n, dtype=np.uint8)
    info = plan.pipeline_host(G.ctypes.data, f.ctypes.data, adv, [di.ADV_REVGRAD] * s, [100.0] * s, seed + 2, Z,
                              u_host.ctypes.data, flags_host.ctypes.data)
    assert info["status"] == 0 and sorted(np.flatnonzero(flags_host)) == adv.tolist()
    assert normwise(u_host, G.astype(np.float64).sum(axis=0)) <= 1e-4
    Z2 = torch.empty_like(Z)
    plan.encode(dev(G), Z2)
    plan.corrupt(Z2, adv, [di.ADV_REVGRAD] * s, [100.0] * s, seed=seed + 2)
    flags = torch.empty(n, dtype=torch.uint8, device="cuda")
    u = torch.empty(d, dtype=torch.float32, device="cuda")
    plan.locate_decode(Z2, dev(f), flags, u)
    torch.cuda.synchronize()
    assert torch.equal(Z, Z2)
    np.testing.assert_array_equal(host(u), u_host)


def test_full_size_resnet152_config_sampled():
    """n = 45, s = 5, d = 60.2 M (21.7 GB of complex64 worker vectors), reversed-gradient
    adversaries at random positions; inputs generated on the device, outputs checked on a
    coordinate sample, the projection on sampled rows over all d."""
    import paper_1803_09877_b200 as dr
    n, s, d = 45, 5, 60_200_000
    plan = dr.Plan(n, s, d, dr.CYC)
    seed = 0xD2AC0 + 4
    G = torch.empty((n, d), dtype=torch.float32, device="cuda")
    dr.generate(G, n, d, seed=seed)
    f = torch.empty(d, dtype=torch.float32, device="cuda")
    dr.generate(f, 1, d, mean=1.0, std=1.0, seed=seed + 3)
    Z = torch.empty((n, 2 * d), dtype=torch.float32, device="cuda")
    plan.encode(G, Z)
    adv = di.choose_adversaries(seed + 1, n, s)
    plan.corrupt(Z, adv, [di.ADV_REVGRAD] * s, [100.0] * s, seed=seed + 2)
    flags = torch.empty(n, dtype=torch.uint8, device="cuda")
    u = torch.empty(d, dtype=torch.float32, device="cuda")
    plan.locate_decode(Z, f, flags, u)
    info = plan.info()
    assert sorted(np.flatnonzero(host(flags))) == adv.tolist()            # Lemma 4: V = the corrupted nodes
    assert info["locator_rank"] == s and info["status"] == 0
    rng = np.random.default_rng(2)
    idx = np.unique(np.concatenate([np.arange(4096), np.arange(d - 4096, d), rng.integers(0, d, 1_000_000)]))
    Gs = di.gradient_rows(seed, n, d, idx=idx)
    np.testing.assert_array_equal(host(G[:, idx]), Gs)                     # same inputs on both sides
    # encode on the sample
    Zo = orc.cyc_encode(Gs, n, s, dtype=np.complex128)
    Zg = host(Z.view(n, d, 2)[:, idx, :].contiguous().view(n, -1), complex64=True)
    honest = np.setdiff1d(np.arange(n), adv)
    for j in honest:
        assert np.abs(Zg[j] - Zo[j]).max() <= 1e-6 * np.abs(Zo[j]).max()
    # decode on the sample: identical R (the device's rows), identical flags
    want_flags = np.zeros(n, dtype=bool)
    want_flags[adv] = True
    Ro = Zo.astype(np.complex64)
    di.apply_adversaries(Ro, adv, [di.ADV_REVGRAD] * s, [100.0] * s, seed=seed + 2, idx=idx)
    exact = Gs.astype(np.float64).sum(axis=0)
    floor = normwise(orc.cyc_decode(Ro, n, s, want_flags), exact)
    err = normwise(host(u[idx]), exact)
    assert err <= 2.0 * floor + 1e-6, (err, floor)
    # projection of two honest rows over all d, by the oracle's definition in chunks
    e = torch.empty(3 * n, dtype=torch.float64, device="cuda")
    plan.cyc_project(Z, f, e)
    eg = host(e)[: 2 * n].view(np.complex128)
    W = orc.cyc_W(n, s)
    for j in (int(honest[0]), int(honest[-1])):
        acc = 0.0 + 0.0j
        step = 4_000_000
        for c0 in range(0, d, step):
            c1 = min(d, c0 + step)
            Gc = di.gradient_rows(seed, n, d, i0=c0, i1=c1)
            fc = di.projection_vector(seed + 3, d, i0=c0, i1=c1)
            zj = (W[:, j] @ Gc.astype(np.complex128)).astype(np.complex64)
            acc += orc.cyc_project(zj[None, :], fc)[0]
        assert abs(eg[j] - acc) <= 1e-5 * abs(acc), (j, eg[j], acc)


def test_full_size_decode_on_generated_R_sampled():
    """Recovery kernel alone at full size on a synthetic complex64 matrix that both sides can
    generate: identical R, identical flags, sampled coordinates."""
    import paper_1803_09877_b200 as dr
    n, s, d = 45, 5, 60_200_000
    plan = dr.Plan(n, s, d, dr.CYC)
    R = torch.empty((n, 2 * d), dtype=torch.float32, device="cuda")
    dr.generate(R, n, 2 * d, seed=555)
    flags = np.zeros(n, dtype=np.uint8)
    flags[[3, 11, 12, 30, 44]] = 1
    u = torch.empty(d, dtype=torch.float32, device="cuda")
    plan.decode(R, dev(flags), u)
    torch.cuda.synchronize()
    rng = np.random.default_rng(3)
    idx = np.unique(np.concatenate([np.arange(2048), np.arange(d - 2048, d), rng.integers(0, d, 50_000)]))
    Rs = di.complex_rows(555, n, d, idx=idx)
    uo = orc.cyc_decode(Rs, n, s, flags.astype(bool))
    assert normwise(host(u[idx]), uo) <= 1e-6


# ------------------------------------------------------------------ packed transport (Section 3, last paragraph)
# (n, s, d): d % 8 == 0 takes the streaming kernel and 64-bit stores; the others the generic paths (odd d pads the last imaginary part)
PACKED_SHAPES = [(15, 2, 100_000), (45, 5, 24_592), (45, 3, 6152), (15, 2, 1001), (9, 1, 6), (15, 7, 4100), (20, 8, 1032),
                 (45, 3, 20_001), (45, 5, 20_003)]


def _packed_plan(n, s, d):
    import paper_1803_09877_b200 as dr
    return dr, dr.Plan(n, s, d, dr.CYC_PACKED)


@pytest.mark.parametrize("n,s,d", PACKED_SHAPES)
def test_packed_encode_parity(n, s, d):
    dr, plan = _packed_plan(n, s, d)
    h = (d + 1) // 2
    G = di.gradient_rows(0xD2AC0 + n + s, n, d)
    Z = torch.empty((n, 2 * h), dtype=torch.float32, device="cuda")
    plan.encode(dev(G), Z)
    torch.cuda.synchronize()
    Zg = host(Z, complex64=True)
    Zo = orc.cyc_encode_packed(G, n, s, dtype=np.complex128)
    assert Zg.shape == Zo.shape == (n, h)
    for j in range(n):
        assert np.abs(Zg[j] - Zo[j]).max() <= 1e-6 * np.abs(Zo[j]).max(), j


@pytest.mark.parametrize("n,s,d", PACKED_SHAPES)
def test_packed_locate_decode_parity_and_exact_sum(n, s, d):
    dr, plan = _packed_plan(n, s, d)
    h = (d + 1) // 2
    seed = 23 * n + s
    G = di.gradient_rows(seed, n, d)
    R = orc.cyc_encode_packed(G, n, s)                     # complex64 worker vectors of h entries
    adv = di.choose_adversaries(seed + 1, n, s)
    di.apply_adversaries(R, adv, [di.ADV_REVGRAD] * s, [100.0] * s, seed=seed + 2)
    f = di.projection_vector(seed + 3, h)
    want = orc.cyc_locate(R, f, n, s)
    assert sorted(np.flatnonzero(want["flags"])) == adv.tolist() and want["margin"] > 10
    Rd, fd = dev(R), dev(f)
    flags = torch.empty(n, dtype=torch.uint8, device="cuda")
    u = torch.full((d,), float("nan"), dtype=torch.float32, device="cuda")
    plan.locate_decode(Rd, fd, flags, u)
    info = plan.info()
    np.testing.assert_array_equal(host(flags).astype(bool), want["flags"])
    assert info["status"] == 0 and info["locator_rank"] == s
    uo = orc.cyc_decode_packed(R, n, s, want["flags"], d)
    assert uo.shape == (d,)
    assert normwise(host(u), uo) <= 1e-6                    # identical R, identical flags
    # whole path on the device against G 1_P
    Z = torch.empty((n, 2 * h), dtype=torch.float32, device="cuda")
    plan.encode(dev(G), Z)
    plan.corrupt(Z, adv, [di.ADV_REVGRAD] * s, [100.0] * s, seed=seed + 2)
    plan.locate_decode(Z, fd, flags, u)
    torch.cuda.synchronize()
    assert sorted(np.flatnonzero(host(flags))) == adv.tolist()
    exact = G.astype(np.float64).sum(axis=0)
    floor = normwise(uo, exact)
    assert normwise(host(u), exact) <= max(1e-4 if n <= 21 else 0.0, 2.0 * floor + 1e-6)


def test_packed_host_pipeline():
    n, s, d = 15, 2, 300_008
    dr, plan = _packed_plan(n, s, d)
    h = d // 2
    seed = 5151
    G = di.gradient_rows(seed, n, d)
    f = di.projection_vector(seed + 3, h)
    adv = di.choose_adversaries(seed + 1, n, s)
    Z = torch.empty((n, 2 * h), dtype=torch.float32, device="cuda")
    u_host = np.empty(d, dtype=np.float32)
    flags_host = np.empty(n, dtype=np.uint8)
    info = plan.pipeline_host(G.ctypes.data, f.ctypes.data, adv, [di.ADV_REVGRAD] * s, [100.0] * s, seed + 2, Z,
                              u_host.ctypes.data, flags_host.ctypes.data)
    assert info["status"] == 0 and sorted(np.flatnonzero(flags_host)) == adv.tolist()
    assert normwise(u_host, G.astype(np.float64).sum(axis=0)) <= 1e-4
    Z2 = torch.empty_like(Z)
    plan.encode(dev(G), Z2)
    plan.corrupt(Z2, adv, [di.ADV_REVGRAD] * s, [100.0] * s, seed=seed + 2)
    torch.cuda.synchronize()
    assert torch.equal(Z, Z2)


def test_packed_full_size_resnet152_sampled():
    """Packed transport at n = 45, s = 5, d = 60.2 M: 30.1 M complex entries per worker (10.8 GB instead of 21.7 GB)."""
    import paper_1803_09877_b200 as dr
    n, s, d = 45, 5, 60_200_000
    h = d // 2
    plan = dr.Plan(n, s, d, dr.CYC_PACKED)
    seed = 0xD2AC0 + 6
    G = torch.empty((n, d), dtype=torch.float32, device="cuda")
    dr.generate(G, n, d, seed=seed)
    f = torch.empty(h, dtype=torch.float32, device="cuda")
    dr.generate(f, 1, h, mean=1.0, std=1.0, seed=seed + 3)
    Z = torch.empty((n, 2 * h), dtype=torch.float32, device="cuda")
    plan.encode(G, Z)
    adv = di.choose_adversaries(seed + 1, n, s)
    plan.corrupt(Z, adv, [di.ADV_REVGRAD] * s, [100.0] * s, seed=seed + 2)
    flags = torch.empty(n, dtype=torch.uint8, device="cuda")
    u = torch.empty(d, dtype=torch.float32, device="cuda")
    plan.locate_decode(Z, f, flags, u)
    assert plan.info()["status"] == 0
    assert sorted(np.flatnonzero(host(flags))) == adv.tolist()
    rng = np.random.default_rng(4)
    ci = np.unique(np.concatenate([np.arange(2048), np.arange(h - 2048, h), rng.integers(0, h, 50_000)]))
    both = np.concatenate([ci, h + ci])
    Gs = di.gradient_rows(seed, n, d, idx=both)
    np.testing.assert_array_equal(host(G[:, both]), Gs)
    exact = Gs.astype(np.float64).sum(axis=0)
    Ghat = Gs[:, : len(ci)].astype(np.float64) + 1j * Gs[:, len(ci):].astype(np.float64)
    Zo = orc.cyc_W(n, s).T @ Ghat
    Zg = host(Z.view(n, h, 2)[:, ci, :].contiguous().view(n, -1), complex64=True)
    for j in np.setdiff1d(np.arange(n), adv):
        assert np.abs(Zg[j] - Zo[j]).max() <= 1e-6 * np.abs(Zo[j]).max()
    want_flags = np.zeros(n, dtype=bool)
    want_flags[adv] = True
    Ro = Zo.astype(np.complex64)
    di.apply_adversaries(Ro, adv, [di.ADV_REVGRAD] * s, [100.0] * s, seed=seed + 2, idx=ci)
    uhat = orc.cyc_recover(Ro, orc.cyc_decode_vector(n, s, want_flags))
    floor = normwise(np.concatenate([uhat.real, uhat.imag]), exact)
    assert normwise(host(u[both]), exact) <= 2.0 * floor + 1e-6


@pytest.mark.parametrize("code_name,n,s,d", [("CYC", 15, 2, 40_004), ("CYC_PACKED", 15, 2, 40_008), ("CYC_PACKED", 9, 1, 1001)])
def test_decode_fused_with_model_update(code_name, n, s, d):
    """w <- w - scale * D(R) in the recovery kernel's epilogue (the SGD step of Section 2)."""
    import paper_1803_09877_b200 as dr
    packed = code_name == "CYC_PACKED"
    plan = dr.Plan(n, s, d, getattr(dr, code_name))
    G = di.gradient_rows(61, n, d)
    R = orc.cyc_encode_packed(G, n, s) if packed else orc.cyc_encode(G, n, s)
    adv = di.choose_adversaries(62, n, s)
    di.apply_adversaries(R, adv, [di.ADV_REVGRAD] * s, [100.0] * s, seed=63)
    flags = np.zeros(n, dtype=np.uint8)
    flags[adv] = 1
    uo = orc.cyc_decode_packed(R, n, s, flags.astype(bool), d) if packed else orc.cyc_decode(R, n, s, flags.astype(bool))
    w0 = di.gradient_rows(64, 1, d)[0]
    w = dev(w0)
    scale = np.float32(0.05 / n)
    plan.decode_update(dev(R), dev(flags), w, float(scale))
    torch.cuda.synchronize()
    assert normwise(host(w), w0.astype(np.float64) - float(scale) * uo) <= 1e-6
    u = torch.empty(d, dtype=torch.float32, device="cuda")
    plan.decode(dev(R), dev(flags), u)
    step = (w0.astype(np.float64) - np.float64(scale) * host(u).astype(np.float64)).astype(np.float32)
    np.testing.assert_allclose(host(w), step, rtol=2e-7, atol=1e-12)
    # refused decode (more than 2 s flags) leaves the model untouched
    flags[:] = 0
    flags[: 2 * s + 1] = 1
    w2 = dev(w0)
    plan.decode_update(dev(R), dev(flags), w2, float(scale))
    assert plan.info()["status"] == dr.binding.ETOOMANY
    np.testing.assert_array_equal(host(w2), w0)


def test_largest_supported_n():
    n, s, d = 128, 2, 4100
    dr, plan = _plan(n, s, d)
    W, Wo = plan.cyc_W(), orc.cyc_W(n, s)
    assert np.abs(W - Wo).max() <= 1e-12 * np.abs(Wo).max()
    G = di.gradient_rows(5, n, d)
    Z = torch.empty((n, 2 * d), dtype=torch.float32, device="cuda")
    plan.encode(dev(G), Z)
    torch.cuda.synchronize()
    Zo = orc.cyc_encode(G, n, s, dtype=np.complex128)
    Zg = host(Z, complex64=True)
    for j in (0, 1, 64, 127):
        assert np.abs(Zg[j] - Zo[j]).max() <= 1e-6 * np.abs(Zo[j]).max()
    R = Zo.astype(np.complex64)
    adv = di.choose_adversaries(6, n, s)
    di.apply_adversaries(R, adv, [di.ADV_REVGRAD] * s, [100.0] * s, seed=7)
    f = di.projection_vector(8, d)
    want = orc.cyc_locate(R, f, n, s)
    flags = torch.empty(n, dtype=torch.uint8, device="cuda")
    plan.locate(dev(R), dev(f), flags)
    torch.cuda.synchronize()
    assert sorted(np.flatnonzero(want["flags"])) == adv.tolist() and want["margin"] > 10
    np.testing.assert_array_equal(host(flags).astype(bool), want["flags"])


def test_rank_cutoff_theta_is_adjustable():
    """With an absurdly high cutoff every singular value counts as zero: nobody is flagged."""
    n, s, d = 15, 2, 8192
    dr, plan = _plan(n, s, d)
    G, R, adv, f = _received(n, s, d, 321, s)
    flags = torch.empty(n, dtype=torch.uint8, device="cuda")
    plan.locate(dev(R), dev(f), flags)
    assert sorted(np.flatnonzero(host(flags))) == adv.tolist()
    plan.set_theta(1e9)
    plan.locate(dev(R), dev(f), flags)
    info = plan.info()
    assert info["locator_rank"] == 0 and info["n_flagged"] == 0 and not host(flags).any()
    want = orc.cyc_locate(R, f, n, s, theta=1e9)
    assert want["rank"] == 0 and not want["flags"].any()


def test_decode_with_null_flags_uses_the_plans_last_locate():
    """locate (flags kept by the plan only) then decode(flags = NULL): same u as with the flags handed over."""
    n, s, d = 15, 2, 6150
    dr, plan = _plan(n, s, d)
    G, R, adv, f = _received(n, s, d, 777, s)
    Rd, fd = dev(R), dev(f)
    u0 = torch.empty(d, dtype=torch.float32, device="cuda")
    u1 = torch.full((d,), 7.0, dtype=torch.float32, device="cuda")
    # a plan that has not located yet decodes with nobody flagged
    plan.decode(Rd, None, u1)
    info = plan.info()
    assert info["n_flagged"] == 0 and info["n_active"] == n
    assert info["status"] == dr.binding.EUNSURE              # adversaries left in U: the imaginary residue shows it
    flags = torch.empty(n, dtype=torch.uint8, device="cuda")
    plan.locate(Rd, fd, flags)
    plan.decode(Rd, flags, u0)
    assert plan.info()["status"] == 0
    plan.locate(Rd, fd, None)                                # V stays in the plan
    plan.decode(Rd, None, u1)
    info = plan.info()
    assert info["status"] == 0 and info["n_flagged"] == s
    assert torch.equal(u0, u1)
    assert normwise(host(u1), orc.cyc_decode(R, n, s, host(flags).astype(bool))) <= 1e-6
    w0 = di.gradient_rows(5, 1, d)[0]
    wa, wb = dev(w0), dev(w0)
    plan.decode_update(Rd, flags, wa, 0.01)
    plan.decode_update(Rd, None, wb, 0.01)
    torch.cuda.synchronize()
    assert torch.equal(wa, wb)


@pytest.mark.parametrize("n,s,d", [(15, 2, 6150), (45, 5, 4099)])
def test_adversaries_sending_nan_or_infinities(n, s, d):
    """A vector with NaN or infinite entries is flagged outright (its projection is not finite), the others are
    located as usual, and the sum comes out finite and exact; flags and sum against the oracle on the same R."""
    dr, plan = _plan(n, s, d)
    G = di.gradient_rows(31 * n + s, n, d)
    R = orc.cyc_encode(G, n, s)
    adv = di.choose_adversaries(5 * n + s, n, s)
    R[adv[0], 7] = np.nan                                      # one NaN entry in an otherwise honest vector
    if s > 1:
        R[adv[1], ::3] = np.inf * (1 - 1j)
    for j in adv[2:]:
        R[j] = -100 * R[j]
    f = di.projection_vector(77, d)
    import warnings
    with warnings.catch_warnings():
        warnings.simplefilter("ignore")
        want = orc.cyc_decode_full(R, f, n, s)
    assert sorted(np.flatnonzero(want["flags"])) == adv.tolist() and want["nonfinite"].sum() == min(s, 2)
    flags = torch.empty(n, dtype=torch.uint8, device="cuda")
    u = torch.empty(d, dtype=torch.float32, device="cuda")
    plan.locate_decode(dev(R), dev(f), flags, u)
    info = plan.info()
    np.testing.assert_array_equal(host(flags).astype(bool), want["flags"])
    assert info["status"] == 0 and info["n_flagged"] == s and info["locator_rank"] == want["rank"]
    assert np.all(np.isfinite(host(u)))
    assert normwise(host(u), want["u"]) <= 1e-6
    assert normwise(host(u), G.astype(np.float64).sum(axis=0)) <= (1e-4 if n <= 15 else 1e-2)


def test_host_pipeline_over_several_column_chunks():
    """d large enough that draco_pipeline_host streams G in three column chunks (the last one ragged): the projection
    then accumulates over the chunks' launches.  Same worker vectors, flags and sum as the device-resident path."""
    import paper_1803_09877_b200 as dr
    n, s, d = 45, 3, 3_100_004
    plan = dr.Plan(n, s, d, dr.CYC)
    seed = 777
    G = torch.empty((n, d), dtype=torch.float32, device="cuda")
    dr.generate(G, n, d, seed=seed)
    f = torch.empty(d, dtype=torch.float32, device="cuda")
    dr.generate(f, 1, d, mean=1.0, std=1.0, seed=seed + 3)
    adv = di.choose_adversaries(seed + 1, n, s)
    Gh, fh = G.cpu().numpy(), f.cpu().numpy()
    Z = torch.empty((n, 2 * d), dtype=torch.float32, device="cuda")
    u_host = np.empty(d, dtype=np.float32)
    flags_host = np.empty(n, dtype=np.uint8)
    info = plan.pipeline_host(Gh.ctypes.data, fh.ctypes.data, adv, [di.ADV_REVGRAD] * s, [100.0] * s, seed + 2, Z,
                              u_host.ctypes.data, flags_host.ctypes.data)
    assert info["status"] == 0 and sorted(np.flatnonzero(flags_host)) == adv.tolist() and info["locator_rank"] == s
    Z2 = torch.empty_like(Z)
    plan2 = dr.Plan(n, s, d, dr.CYC)
    plan2.encode(G, Z2)
    plan2.corrupt(Z2, adv, [di.ADV_REVGRAD] * s, [100.0] * s, seed=seed + 2)
    flags = torch.empty(n, dtype=torch.uint8, device="cuda")
    u = torch.empty(d, dtype=torch.float32, device="cuda")
    plan2.locate_decode(Z2, f, flags, u)
    torch.cuda.synchronize()
    assert torch.equal(Z, Z2)
    np.testing.assert_array_equal(host(flags), flags_host)
    np.testing.assert_array_equal(host(u), u_host)             # same flags, same decode vector, same rows: same bits
    # and the sum itself on a sample, against the exact one
    idx = np.unique(np.concatenate([np.arange(64), np.arange(d - 64, d), np.random.default_rng(1).integers(0, d, 5000)]))
    exact = Gh[:, idx].astype(np.float64).sum(axis=0)
    assert normwise(u_host[idx], exact) <= 2e-3                # complex64 floor at (45, 3) is about 2e-4


def test_adjacent_adversaries_at_45_5():
    """Five adversaries side by side at n = 45, s = 5: the placement that one pass of the locator cannot always resolve
    with complex64 vectors.  The passes with erasures end with a set that contains all five (the same set as the
    oracle's, on the same received matrix), and the sum is right to the accuracy of the transport."""
    n, s, d = 45, 5, 4100
    dr, plan = _plan(n, s, d)
    supersets = 0
    for start in (0, 9, 12, 21, 30, 39, 42):
        adv = [(start + k) % n for k in range(s)]
        G = di.gradient_rows(1000 + start, n, d)
        Z = torch.empty((n, 2 * d), dtype=torch.float32, device="cuda")
        plan.encode(dev(G), Z)
        plan.corrupt(Z, adv, [di.ADV_REVGRAD] * s, [100.0] * s, seed=3)
        f = di.projection_vector(2000 + start, d)
        flags = torch.empty(n, dtype=torch.uint8, device="cuda")
        u = torch.empty(d, dtype=torch.float32, device="cuda")
        plan.locate_decode(Z, dev(f), flags, u)
        info = plan.info()
        want = orc.cyc_locate(host(Z).view(np.complex64), f, n, s)
        np.testing.assert_array_equal(host(flags).astype(bool), want["flags"], err_msg=str(start))
        assert info["locator_rank"] == want["rank"]
        found = set(np.flatnonzero(host(flags)).tolist())
        assert found >= set(adv) and len(found) <= 2 * s, (start, sorted(found))
        supersets += found != set(adv)
        exact = G.astype(np.float64).sum(axis=0)
        assert normwise(host(u), exact) <= 2e-2, start
        assert info["im_residual"] <= 1e-2 * info["re_max"]          # nobody adversarial is left among the rows combined
        assert info["status"] == 0                                   # whatever the first pass's margin was
    assert supersets >= 1                                            # at least one of these positions needs the extra pass
