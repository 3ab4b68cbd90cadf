"""Cyclic code on the kernel paths that small shapes do not reach, element by element against the CPU oracle
through the C ABI:

  * more than 64 nodes: the projection runs as two launches of the tile kernel over half the rows each
    (n = 65, 105, 128; ragged d, d not a multiple of 4, packed and unpacked vectors);
  * s >= 17: the s x s syndrome system no longer fits one warp's shared-memory solver and is solved by the
    block-wide Jacobi SVD in the plan's work space;
  * more than 16 flagged nodes (erasure decoding up to 2 s flags): the decode vector's |V| x |V| system is
    eliminated by the whole block in the plan's work space.

Bars (max |a - b| / max |b|): projection e <= 1e-6, squared norms q <= 1e-5, flags and rank exact (inputs are
checked to sit >= 3 x from the rank cutoff), decode vector b <= 1e-9 (erasure cases: see `_b_bar`), u on
identical R and identical flags <= 1e-6 plus the rounding bound of the sum itself (see `_u_bound`): at n = 105
and 128 with s >= 5 the decode vector is as large as 1e9 .. 1e17 and cancels, so the recovered sum carries no
information there (a property of the code with complex64 vectors); what is compared is that both sides
evaluate the same cancelling sum to within its fp64 rounding.
"""
import numpy as np
import pytest
import torch

import draco_inputs as di
from gpu_util import dev, host, normwise
from oracle import draco_oracle as orc

pytestmark = pytest.mark.gpu


def _received(n, s, d, seed, n_adv, model, packed):
    G = di.gradient_rows(seed, n, d)
    R = orc.cyc_encode_packed(G, n, s) if packed else orc.cyc_encode(G, n, s)      # complex64 worker vectors
    adv = di.choose_adversaries(seed + 1, n, n_adv)
    param = 100.0
    if model == di.ADV_GAUSS:
        param = float(np.abs(R).max())                     # noise of the size of the vectors themselves
    di.apply_adversaries(R, adv, [model] * n_adv, [param] * n_adv, seed=seed + 2)
    return G, R, adv, di.projection_vector(seed + 3, R.shape[1])


def _u_bound(b, R, db):
    """What |u_gpu - u_oracle| may be when both add up sum_j b_j R_j in fp64 in different orders and their decode
    vectors differ by db (relative to max |b|): rounding of an n-term sum, plus the decode vectors' difference."""
    n = len(b)
    size = float(np.abs(b).sum() * np.abs(R).max())
    return (4 * n * 2.0 ** -53 + db * n) * size


def _b_bar(n, s, flags):
    """The device forms b from the |V| x |V| system [C_R]_{.,V}^H [C_R]_{.,V}, whose condition number is the square
    of cond([C_L]_{.,U}); Gaussian elimination in fp64 then leaves about cond^2 * 2^-53 in b."""
    U = np.flatnonzero(~flags)
    sv = np.linalg.svd(orc.idft_matrix(n)[: n - 2 * s][:, U], compute_uv=False)
    cond = float(sv[0] / sv[-1])
    return cond, max(1e-9, 50.0 * cond * cond * 2.0 ** -53)


def _check_locate_decode(dr, n, s, d, n_adv, model, packed, seed=None):
    plan = dr.Plan(n, s, d, dr.CYC_PACKED if packed else dr.CYC)
    G, R, adv, f = _received(n, s, d, 1000 * n + 10 * s + n_adv if seed is None else seed, n_adv, model, packed)
    vlen = R.shape[1]
    want = orc.cyc_locate(R, f, n, s)
    Rd, fd = dev(R), dev(f)
    # projection record
    e = torch.full((3 * n,), float("nan"), dtype=torch.float64, device="cuda")
    plan.cyc_project(Rd, fd, e)
    eg = host(e)
    assert np.abs(eg[: 2 * n].view(np.complex128) - want["e"]).max() <= 1e-6 * np.abs(want["e"]).max()
    qo = orc.cyc_project_energy(R)
    assert np.abs(eg[2 * n:] - qo).max() <= 1e-5 * qo.max()
    # exact products, fp64 sums: only the order of the additions differs from the oracle's
    assert np.abs(eg[: 2 * n].view(np.complex128) - want["e"]).max() <= 1e-11 * np.sqrt(qo.max() * 2 * vlen)
    assert np.abs(eg[2 * n:] - qo).max() <= 1e-12 * qo.max()
    # flags and rank
    # The singular values that stand for "zero" are rounding noise.  Both sides see the noise of the complex64
    # vectors; the device adds that of its fp32 products, of the same size, so its noise may be sqrt(2) times
    # the oracle's: inputs whose noise reaches half the cutoff (it grows like sqrt(s): 0.05 of the cutoff at
    # s = 2, 0.3 at s = 20) or whose weakest adversary is within 3 x of it are not used.
    tol = 1e-6 * want["scale"]
    assert all(x > 3 * tol or x < tol / 2 for x in want.get("sv", [])), "test input sits too close to the rank cutoff"
    assert want["rank"] == n_adv and sorted(np.flatnonzero(want["flags"])) == adv.tolist()
    assert n_adv == 0 or want["margin"] > 10
    flags = torch.full((n,), 9, dtype=torch.uint8, device="cuda")
    plan.locate(Rd, fd, flags)
    info = plan.info()
    np.testing.assert_array_equal(host(flags).astype(bool), want["flags"])
    assert info["locator_rank"] == want["rank"] and info["n_flagged"] == n_adv
    assert abs(info["scale"] - want["scale"]) <= 1e-5 * want["scale"]
    # decode vector and recovered sum on the same R with the same flags
    u = torch.full((d,), float("nan"), dtype=torch.float32, device="cuda")
    plan.decode(Rd, flags, u)
    info = plan.info()
    assert info["n_active"] == n - n_adv
    # where the code's cancellation leaves nothing of the sum (its imaginary part is as large as its real part)
    # the decoder says so; otherwise the status is clean
    unsure = (not packed) and not (info["im_residual"] <= 1e-2 * info["re_max"])
    assert info["status"] == (dr.binding.EUNSURE if unsure else 0)
    b, bo = plan.cyc_decode_vector(), orc.cyc_decode_vector(n, s, want["flags"])
    db = float(np.abs(b - bo).max() / np.abs(bo).max())
    assert db <= _b_bar(n, s, want["flags"])[1]
    uhat = orc.cyc_recover(R, bo)
    uo = orc.cyc_unpack(uhat, d) if packed else uhat.real
    ug = host(u).astype(np.float64)
    assert np.all(np.isfinite(ug))
    assert np.abs(ug - uo).max() <= 1e-6 * np.abs(uo).max() + _u_bound(bo, R, db)
    return vlen


# (n, s, d): above 64 nodes; d ragged against the 2048-coordinate tile, odd, and below one tile
LARGE_N = [(65, 2, 4100), (65, 5, 2050), (105, 2, 4099), (105, 7, 6150), (128, 2, 1001), (128, 5, 2049)]


@pytest.mark.parametrize("n,s,d", LARGE_N)
@pytest.mark.parametrize("adversaries", ["s", "none"])
@pytest.mark.parametrize("packed", [False, True])
def test_more_than_64_nodes(n, s, d, adversaries, packed):
    import paper_1803_09877_b200 as dr
    n_adv = s if adversaries == "s" else 0
    _check_locate_decode(dr, n, s, d, n_adv, di.ADV_REVGRAD, packed)


@pytest.mark.parametrize("n,s,d", [(105, 2, 4099), (128, 5, 2049)])
def test_more_than_64_nodes_encode_parity(n, s, d):
    import paper_1803_09877_b200 as dr
    plan = dr.Plan(n, s, d, dr.CYC)
    G = di.gradient_rows(3 * n + s, n, d)
    Z = torch.empty((n, 2 * d), dtype=torch.float32, device="cuda")
    plan.encode(dev(G), Z)
    torch.cuda.synchronize()
    Zg, Zo = host(Z, complex64=True), orc.cyc_encode(G, n, s, dtype=np.complex128)
    for j in range(n):
        assert np.abs(Zg[j] - Zo[j]).max() <= 1e-6 * np.abs(Zo[j]).max(), j


# s >= 17: block-wide Jacobi SVD of the syndrome system.  (n, s, d, adversaries, seed); seeds picked so that the
# oracle itself finds the planted set with a margin: with 20 adversaries among 128 nodes complex64 vectors no
# longer carry the code (the 20th singular value sinks below the cutoff on both sides), so that case has 18.
BIG_S = [(36, 17, 1030, 0, 36170), (36, 17, 1030, 15, 36185), (36, 17, 1030, 17, 36187),
         (40, 18, 4100, 0, 40180), (40, 18, 4100, 16, 40196), (40, 18, 4100, 18, 40198),
         (50, 20, 2049, 0, 50200), (50, 20, 2049, 18, 50218), (50, 20, 2049, 20, 50220),
         (64, 20, 4100, 0, 64200), (64, 20, 4100, 18, 64218), (64, 20, 4100, 20, 80058),
         (128, 20, 2052, 0, 128200), (128, 20, 2052, 18, 128218)]


@pytest.mark.parametrize("n,s,d,n_adv,seed", BIG_S)
def test_syndrome_systems_larger_than_16(n, s, d, n_adv, seed):
    import paper_1803_09877_b200 as dr
    model = di.ADV_GAUSS if n_adv % 2 else di.ADV_REVGRAD
    _check_locate_decode(dr, n, s, d, n_adv, model, packed=False, seed=seed)


# erasure decoding with more than 16 flagged nodes, up to the limit of 2 s
@pytest.mark.parametrize("n,s,d", [(36, 17, 1030), (40, 18, 4100), (64, 20, 2049), (128, 20, 2052), (45, 10, 4100)])
@pytest.mark.parametrize("n_flags", ["17", "2s-3", "2s"])
def test_decode_vector_with_more_than_16_flags(n, s, d, n_flags):
    import paper_1803_09877_b200 as dr
    k = {"17": 17, "2s-3": 2 * s - 3, "2s": 2 * s}[n_flags]
    plan = dr.Plan(n, s, d, dr.CYC)
    rng = np.random.default_rng(100 * n + k)
    flags = np.zeros(n, dtype=np.uint8)
    flags[rng.choice(n, k, replace=False)] = 1
    cond, bar = _b_bar(n, s, flags.astype(bool))
    R = di.complex_rows(7 * n + k, n, d)
    u = torch.full((d,), float("nan"), dtype=torch.float32, device="cuda")
    plan.decode(dev(R), dev(flags), u)
    info = plan.info()
    # R is random, not a set of coded vectors: u-hat comes out as complex as it is real, which the self-check reports
    assert info["status"] == dr.binding.EUNSURE and info["n_active"] == n - k and info["n_flagged"] == k
    b, bo = plan.cyc_decode_vector(), orc.cyc_decode_vector(n, s, flags.astype(bool))
    assert not np.abs(b[flags.astype(bool)]).any()
    db = float(np.abs(b - bo).max() / np.abs(bo).max())
    assert db <= bar, (cond, db, bar)
    # b solves the system it stands for: [C_L]_{.,U} b_U = (0, .., 0, 1)^T, to the same accuracy
    CL = orc.idft_matrix(n)[: n - 2 * s]
    rhs = np.zeros(n - 2 * s)
    rhs[-1] = 1.0
    assert np.abs(CL @ b - rhs).max() <= bar * max(1.0, np.abs(bo).max()) * np.sqrt(n)
    uo = orc.cyc_recover(R, bo).real
    ug = host(u).astype(np.float64)
    assert np.all(np.isfinite(ug))
    assert np.abs(ug - uo).max() <= 1e-6 * np.abs(uo).max() + _u_bound(bo, R, db)
    # one flag more than 2 s is refused
    if k == 2 * s:
        free = np.flatnonzero(flags == 0)
        flags[free[0]] = 1
        plan.decode(dev(R), dev(flags), u)
        assert plan.info()["status"] == dr.binding.ETOOMANY and float(u.abs().max()) == 0.0


# the smallest and the largest shapes the plan accepts: one node, one coordinate, s = (n - 1) / 2 at n = 3 and n = 127 / 128
@pytest.mark.parametrize("n,s,d", [(1, 0, 1), (1, 0, 7), (2, 0, 3), (3, 1, 1), (3, 1, 2), (127, 63, 5), (128, 63, 9)])
@pytest.mark.parametrize("code_name", ["CYC", "CYC_PACKED", "REP"])
def test_degenerate_shapes(n, s, d, code_name):
    import paper_1803_09877_b200 as dr
    plan = dr.Plan(n, s, d, getattr(dr, code_name))
    G = di.gradient_rows(11 * n + d, n, d)
    exact = G.astype(np.float64).sum(axis=0)
    flags = torch.full((n,), 9, dtype=torch.uint8, device="cuda")
    u = torch.full((d,), float("nan"), dtype=torch.float32, device="cuda")
    if code_name == "REP":
        Z = torch.empty((n, d), dtype=torch.float32, device="cuda")
        plan.encode(dev(G), Z)
        torch.cuda.synchronize()
        Zo = orc.rep_encode(G, n, s)                         # fp64 sums rounded once; the device adds in fp32, ascending
        assert np.abs(host(Z) - Zo).max() <= 1e-6 * max(np.abs(Zo).max(), 1e-30)
        for first, size in orc.rep_groups(n, s):
            assert (host(Z)[first:first + size].view(np.uint32) == host(Z)[first].view(np.uint32)).all()
        plan.locate_decode(Z, None, flags, u)
        info = plan.info()
        assert not host(flags).any() and info["status"] == 0 and info["no_majority"] == 0
        assert np.abs(host(u) - exact).max() <= 1e-5 * max(np.abs(exact).max(), 1e-30)
        return
    packed = code_name == "CYC_PACKED"
    h = (d + 1) // 2 if packed else d
    Z = torch.empty((n, 2 * h), dtype=torch.float32, device="cuda")
    plan.encode(dev(G), Z)
    torch.cuda.synchronize()
    Zo = orc.cyc_encode_packed(G, n, s, dtype=np.complex128) if packed else orc.cyc_encode(G, n, s, dtype=np.complex128)
    Zg = host(Z, complex64=True)
    for j in range(n):
        assert np.abs(Zg[j] - Zo[j]).max() <= 1e-6 * max(np.abs(Zo[j]).max(), 1e-30)
    f = di.projection_vector(5, h)
    plan.locate_decode(Z, dev(f), flags, u)
    info = plan.info()
    assert not host(flags).any() and info["locator_rank"] == 0 and info["status"] == 0
    assert np.abs(host(u) - exact).max() <= 1e-5 * max(np.abs(exact).max(), 1e-30)
