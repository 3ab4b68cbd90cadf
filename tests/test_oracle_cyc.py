"""Pins for the cyclic-code oracle: the paper's lemmas, closed forms, brute force."""
import itertools
import os

import numpy as np
import pytest

import draco_inputs as di
from oracle import draco_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _exact_sum(G):
    return G.astype(np.float64).sum(axis=0)


def test_W_matches_hand_derived_table_n4_s1():
    rows = [ln.split() for ln in open(os.path.join(GOLDEN, "cyc_W_n4_s1.txt")) if not ln.startswith("#")]
    table = np.array([[0.5 * (float(r[2 * k]) + 1j * float(r[2 * k + 1])) for k in range(4)] for r in rows])
    np.testing.assert_allclose(orc.cyc_W_by_definition(4, 1), table, atol=1e-15)
    np.testing.assert_allclose(orc.cyc_W_closed_form(4, 1), table, atol=1e-15)


@pytest.mark.parametrize("n,s", [(4, 1), (5, 1), (7, 3), (9, 1), (10, 2), (15, 2), (15, 5), (21, 3)])
def test_W_definition_equals_closed_form(n, s):
    Wd, Wc = orc.cyc_W_by_definition(n, s), orc.cyc_W_closed_form(n, s)
    assert np.abs(Wd - Wc).max() <= 1e-14 * np.abs(Wc).max()


def test_W_definition_equals_closed_form_n45_s5():
    Wd, Wc = orc.cyc_W_by_definition(45, 5, dps=50), orc.cyc_W_closed_form(45, 5)
    assert np.abs(Wd - Wc).max() <= 1e-14 * np.abs(Wc).max()
    assert 1.7e5 < np.abs(Wc).max() < 1.9e5               # entries grow geometrically with n and s


@pytest.mark.parametrize("n,s", [(4, 1), (9, 2), (15, 2), (45, 5)])
def test_lemma3_support_and_span(n, s):
    A, W = orc.cyc_allocation(n, s), orc.cyc_W(n, s)
    assert A.sum() / n == 2 * s + 1                        # redundancy ratio meets Theorem 1 with equality
    assert np.abs(W[A == 0]).max() <= 1e-9 * np.abs(W).max()
    assert np.abs(W[A == 1]).min() > 1e-3
    rng = np.random.default_rng(n)
    for trial in range(6):
        flags = np.zeros(n, dtype=bool)
        flags[rng.choice(n, size=int(rng.integers(0, 2 * s + 1)), replace=False)] = True
        for b in (orc.cyc_decode_vector(n, s, flags), orc.cyc_decode_vector_first(n, s, flags)):
            assert np.all(b[flags] == 0)
            assert np.abs(W @ b - 1.0).max() <= 1e-7 * np.abs(W).max() * max(1.0, np.abs(b).max())
    flags = np.zeros(n, dtype=bool)
    flags[: 2 * s + 1] = True
    with pytest.raises(ValueError):
        orc.cyc_decode_vector(n, s, flags)


def test_min_norm_vector_lies_in_row_space():
    n, s = 15, 2
    flags = np.zeros(n, dtype=bool)
    flags[[2, 9]] = True
    b = orc.cyc_decode_vector(n, s, flags)
    U = np.flatnonzero(~flags)
    A = orc.idft_matrix(n)[: n - 2 * s][:, U]
    null = np.linalg.svd(A)[2][n - 2 * s:].conj().T      # basis of the null space of A
    assert np.abs(null.conj().T @ b[U]).max() < 1e-12      # min-norm <=> orthogonal to the null space
    assert np.linalg.norm(b) <= np.linalg.norm(orc.cyc_decode_vector_first(n, s, flags)) + 1e-12


def test_literal_decode_vector_is_lagrange_closed_form():
    """b_k = sqrt(n) / prod_{l in U-bar, l != k} (w^k - w^l) solves [C_L]_{., U-bar} b = e_last."""
    n, s = 15, 2
    flags = np.zeros(n, dtype=bool)
    flags[[0, 7]] = True
    Ubar = np.flatnonzero(~flags)[: n - 2 * s]
    w = np.exp(2j * np.pi / n)
    expect = np.zeros(n, dtype=complex)
    for k in Ubar:
        expect[k] = np.sqrt(n) / np.prod([w ** k - w ** l for l in Ubar if l != k])
    np.testing.assert_allclose(orc.cyc_decode_vector_first(n, s, flags), expect, rtol=1e-9, atol=1e-12)


@pytest.mark.parametrize("n,s", [(4, 1), (15, 2), (45, 5)])
def test_lemma7_orthogonality_and_clean_syndromes(n, s):
    C = orc.idft_matrix(n)
    np.testing.assert_allclose(C @ C.conj().T, np.eye(n), atol=1e-13)       # unitary
    np.testing.assert_allclose(C, C.T, atol=0)                              # symmetric
    C_L, C_R = C[: n - 2 * s], C[n - 2 * s:]
    assert np.abs(C_L @ C_R.conj().T).max() < 1e-13
    d = 64
    G = di.gradient_rows(1, n, d)
    Z = orc.cyc_encode(G, n, s, dtype=np.complex128)
    synd = Z.T @ C_R.conj().T                                               # R C_R^dagger, per coordinate
    assert np.abs(synd).max() <= 1e-10 * np.abs(Z).max()
    f = di.projection_vector(2, d)
    loc = orc.cyc_locate(Z, f, n, s)
    assert not loc["flags"].any() and loc["rank"] == 0


@pytest.mark.parametrize("n,s", [(4, 1), (15, 2), (45, 5), (45, 3)])
def test_locator_returns_f_times_N_value_for_value(n, s):
    """Proof of Lemma 4: t = C h = gamma = (f N)^T, for 0..s adversaries."""
    d = 200
    G = di.gradient_rows(21, n, d)
    Z = orc.cyc_encode(G, n, s, dtype=np.complex128)
    f = di.projection_vector(22, d)
    rng = np.random.default_rng(5)
    for a in range(s + 1):
        adv = np.sort(rng.choice(n, size=a, replace=False))
        N = np.zeros_like(Z)
        N[adv] = (rng.normal(size=(a, d)) + 1j * rng.normal(size=(a, d))) * 50.0 * np.abs(Z).max()
        loc = orc.cyc_locate(Z + N, f, n, s)
        gamma = N @ f.astype(np.float64)
        assert loc["rank"] == a
        assert set(np.flatnonzero(loc["flags"])) == set(adv.tolist())
        if a:
            assert np.abs(loc["t"] - gamma).max() <= 1e-6 * np.abs(gamma).max()


@pytest.mark.parametrize("n,s", [(3, 1), (4, 1), (5, 1), (5, 2), (6, 2), (7, 3), (9, 2), (10, 1), (15, 2)])
def test_every_placement_of_up_to_s_adversaries_is_corrected(n, s):
    """Definition 2 / Theorem 5 by brute force on tiny n (complex128 transport)."""
    d = 16
    G = di.gradient_rows(31, n, d)
    Z = orc.cyc_encode(G, n, s, dtype=np.complex128)
    f = di.projection_vector(32, d)
    exact = _exact_sum(G)
    attacks = [(di.ADV_REVGRAD, 100.0), (di.ADV_CONST, -100.0), (di.ADV_GAUSS, 1e3)]
    for a in range(s + 1):
        for placement in itertools.combinations(range(n), a):
            for model, param in attacks:
                R = Z.copy().astype(np.complex64)          # the corruptor works on complex64 rows
                di.apply_adversaries(R, placement, [model] * a, [param] * a, seed=3)
                R = R.astype(np.complex128)
                honest = np.setdiff1d(np.arange(n), placement)
                R[honest] = Z[honest]                      # honest rows keep full precision
                out = orc.cyc_decode_full(R, f, n, s)
                assert set(np.flatnonzero(out["flags"])) == set(placement), (placement, model)
                assert np.abs(out["u"] - exact).max() <= 1e-8 * np.abs(exact).max()
    # a single corrupted coordinate on one node
    R = Z.copy()
    R[n - 1, 5] += 3.0
    out = orc.cyc_decode_full(R, f, n, s)
    assert list(np.flatnonzero(out["flags"])) == [n - 1]
    assert np.abs(out["u"] - exact).max() <= 1e-8 * np.abs(exact).max()


def test_failure_beyond_s():
    """Theorem 1 / its corollary: s + 1 colluding adversaries defeat a redundancy-(2 s + 1) code.  The attack of the
    proof: change one gradient g_k by delta; only the 2 s + 1 nodes that hold g_k send something else.  s + 1 of them
    (the adversaries) send what they would send for the changed gradient, the other s stay honest.  The received
    matrix is then s errors away from the coded vectors of the *changed* gradients, which is what any decoder must
    return: the honest s get the blame and the sum is off by delta, with nothing to warn about."""
    n, s, d = 15, 2, 32
    G = di.gradient_rows(41, n, d)
    Z = orc.cyc_encode(G, n, s, dtype=np.complex128)
    W = orc.cyc_W(n, s)
    f = di.projection_vector(42, d)
    exact = _exact_sum(G)
    delta = np.linspace(1.0, 2.0, d)
    for k in (0, 6, 13):
        holders = [(k + t) % n for t in range(2 * s + 1)]          # nodes j with W[k][j] != 0 (z_j uses g_{j-2s..j})
        assert all(abs(W[k, j]) > 0 for j in holders) and np.count_nonzero(np.abs(W[k]) > 1e-12) == 2 * s + 1
        for adversaries in itertools.combinations(holders, s + 1):
            R = Z.copy()
            for j in adversaries:
                R[j] = Z[j] + W[k, j] * delta
            out = orc.cyc_decode_full(R, f, n, s)
            blamed = set(np.flatnonzero(out["flags"]))
            assert blamed == set(holders) - set(adversaries)       # the honest holders of g_k
            assert np.abs(out["u"] - (exact + delta)).max() <= 1e-9 * np.abs(exact).max()
            assert np.abs(out["u"] - exact).max() >= 0.99


def test_n4_any_two_coded_vectors_recover_the_sum():
    """Figure 1: 4 gradients, replication 3, any 2 coded vectors give the sum; a
    majority vote over the 6 pair-decodes survives one adversary."""
    n, s, d = 4, 1, 8
    G = di.gradient_rows(51, n, d)
    Z = orc.cyc_encode(G, n, s, dtype=np.complex128)
    exact = _exact_sum(G)
    pairs = list(itertools.combinations(range(n), 2))
    assert len(pairs) == 6
    for pair in pairs:
        flags = np.ones(n, dtype=bool)
        flags[list(pair)] = False
        np.testing.assert_allclose(orc.cyc_decode(Z, n, s, flags), exact, atol=1e-12)
    R = Z.copy()
    R[2] = -100.0 * R[2]
    decodes = []
    for pair in pairs:
        flags = np.ones(n, dtype=bool)
        flags[list(pair)] = False
        decodes.append(np.round(orc.cyc_decode(R, n, s, flags), 9))
    agree = [sum(np.array_equal(x, y) for y in decodes) for x in decodes]
    assert sorted(agree) == [1, 1, 1, 3, 3, 3]              # 3 clean pairs agree, 3 dirty pairs differ
    winner = decodes[int(np.argmax(agree))]
    np.testing.assert_allclose(winner, exact, atol=1e-8)
    f = di.projection_vector(52, d)
    np.testing.assert_allclose(orc.cyc_decode_full(R, f, n, s)["u"], exact, atol=1e-10)


def test_no_adversary_decode_vector_is_conjugate_idft_row():
    for n, s in [(4, 1), (15, 2), (45, 5)]:
        b = orc.cyc_decode_vector(n, s, np.zeros(n, dtype=bool))
        np.testing.assert_allclose(b, orc.idft_matrix(n)[n - 2 * s - 1].conj(), atol=1e-12)
        G = di.gradient_rows(61, n, 50)
        Z = orc.cyc_encode(G, n, s, dtype=np.complex128)
        uhat = orc.cyc_recover(Z, b)
        scale = np.abs(orc.cyc_W(n, s)).max()
        assert np.abs(uhat.real - _exact_sum(G)).max() <= 1e-12 * scale * 10
        assert np.abs(uhat.imag).max() <= 1e-12 * scale * 10          # Im(u-hat) is rounding residue


def test_full_redundancy_degenerates_to_repetition():
    n, s = 15, 7                                           # r = n: C_L has one row
    W = orc.cyc_W(n, s)
    np.testing.assert_allclose(W, np.full((n, n), 1 / np.sqrt(n)), atol=1e-14)


def test_complex64_transport_floor():
    """With complex64 worker vectors the recovered sum is only as good as the
    code's cancellation allows: tight at (15,2), about 1e-3 at (45,5)."""
    for (n, s, lo, hi) in [(15, 2, 0.0, 5e-6), (45, 5, 1e-4, 1e-2)]:
        d = 4000
        G = di.gradient_rows(71, n, d)
        R = orc.cyc_encode(G, n, s)
        adv = di.choose_adversaries(72, n, s)
        di.apply_adversaries(R, adv, [di.ADV_REVGRAD] * s, [100.0] * s, seed=0)
        out = orc.cyc_decode_full(R, di.projection_vector(73, d), n, s)
        assert list(np.flatnonzero(out["flags"])) == adv.tolist()
        err = np.abs(out["u"] - _exact_sum(G)).max() / np.abs(_exact_sum(G)).max()
        assert lo <= err <= hi, err


@pytest.mark.parametrize("d", [1, 2, 7, 8, 33])
def test_packing_round_trip_and_sum(d):
    n = 5
    G = di.gradient_rows(81, n, d)
    Gh = orc.cyc_pack(G)
    assert Gh.shape == (n, (d + 1) // 2)
    for k in range(n):
        np.testing.assert_array_equal(orc.cyc_unpack(Gh[k], d), G[k].astype(np.float64))
    np.testing.assert_array_equal(orc.cyc_unpack(Gh.sum(axis=0), d), G.astype(np.float64).sum(axis=0))
    if d >= 7:   # the literal "Re + Im" of the text is not the gradient sum
        literal = Gh.sum(axis=0).real + Gh.sum(axis=0).imag
        assert literal.shape[0] != d or np.abs(literal - G.astype(np.float64).sum(axis=0)).max() > 1e-3


@pytest.mark.parametrize("n,s,d", [(4, 1, 9), (7, 2, 16), (9, 2, 31), (15, 2, 40)])
def test_packed_pipeline_corrects_every_placement(n, s, d):
    """Definition 2 through the packed transport: half the complex coordinates, same guarantee."""
    G = di.gradient_rows(91, n, d)
    Z = orc.cyc_encode_packed(G, n, s, dtype=np.complex128)
    h = (d + 1) // 2
    assert Z.shape == (n, h)
    f = di.projection_vector(92, h)
    exact = _exact_sum(G)
    for a in range(s + 1):
        for placement in itertools.combinations(range(n), a):
            R = Z.copy()
            R[list(placement)] *= -100.0
            loc = orc.cyc_locate(R, f, n, s)
            assert set(np.flatnonzero(loc["flags"])) == set(placement)
            u = orc.cyc_decode_packed(R, n, s, loc["flags"], d)
            assert u.shape == (d,)
            assert np.abs(u - exact).max() <= 1e-8 * np.abs(exact).max()


def test_rank_cutoff_is_measured_against_the_size_of_the_vectors_not_of_their_projection():
    """r = n (one row in C_L): every honest node sends the same vector, so all e_j coincide and, for an f that makes
    that one signed sum cancel, median_j |e_j| is tiny while the rounding noise of the vectors is not.  The cutoff
    theta * median_j q_j^(1/2) must still call rounding-level differences between the rows rank 0, and must still
    see real adversaries."""
    n, s, d = 15, 7, 4096
    G = di.gradient_rows(31, n, d)
    Z = orc.cyc_encode(G, n, s)
    rng = np.random.default_rng(5)
    f = di.projection_vector(32, d).astype(np.float64)
    f -= (Z[0].real @ f) / (Z[0].real @ Z[0].real) * Z[0].real * (1 - 1e-3)         # e_j shrinks to 1e-3 of its size
    noisy = (Z * (1 + 2.0 ** -24 * rng.uniform(-1, 1, Z.shape))).astype(np.complex64)   # rows differ by fp32 rounding
    e, q = orc.cyc_project(noisy, f), orc.cyc_project_energy(noisy)
    assert np.median(np.abs(e)) < 0.02 * np.median(np.sqrt(q))                      # the sum did cancel
    loc = orc.cyc_locate(noisy, f, n, s)
    assert loc["rank"] == 0 and not loc["flags"].any()
    assert abs(loc["scale"] - np.median(np.sqrt(q))) <= 1e-12 * loc["scale"]
    # against |e_j| the same rows look like seven adversaries
    assert orc.cyc_locate_from_projection(e, np.abs(e) ** 2, n, s)["rank"] > 0
    # q by its definition, term by term
    j = 3
    assert abs(q[j] - sum(abs(complex(noisy[j, i])) ** 2 for i in range(d))) <= 1e-10 * q[j]
    adv = [2, 9, 13]
    R = noisy.copy()
    R[adv] *= -100
    loc = orc.cyc_locate(R, di.projection_vector(33, d), n, s)
    assert sorted(np.flatnonzero(loc["flags"])) == adv


@pytest.mark.parametrize("n,s", [(5, 1), (7, 2), (9, 2)])
def test_adversaries_sending_nan_or_infinities_are_flagged_and_the_sum_is_exact(n, s):
    """Definition 2 with "arbitrary" taken at its word: vectors holding NaN or infinities, alone or beside an
    ordinary reversed-gradient adversary, at every placement of up to s adversaries."""
    import warnings
    d = 12
    G = di.gradient_rows(3, n, d)
    Z = orc.cyc_encode(G, n, s)
    f = di.projection_vector(4, d)
    exact = G.astype(np.float64).sum(axis=0)
    with warnings.catch_warnings():
        warnings.simplefilter("ignore")                         # numpy warns about inf - inf on the way
        for a in range(1, s + 1):
            for placement in itertools.combinations(range(n), a):
                for kind in range(3):
                    R = Z.copy()
                    for k, j in enumerate(placement):
                        if kind == 0:
                            R[j, 3] = np.nan                     # a single NaN entry
                        elif kind == 1 and k % 2 == 0:
                            R[j] = np.inf * (1 + 1j)
                        elif kind == 1:
                            R[j] = -100 * R[j]                   # an ordinary adversary beside the infinite one
                        else:
                            R[j, ::2] = -np.inf
                            R[j, 1] = np.nan
                    out = orc.cyc_decode_full(R, f, n, s)
                    assert set(np.flatnonzero(out["flags"])) == set(placement)
                    assert np.all(np.isfinite(out["u"]))
                    assert np.abs(out["u"] - exact).max() <= 1e-4 * np.abs(exact).max()
    # a clean matrix reports no such node
    assert not orc.cyc_locate(Z, f, n, s)["nonfinite"].any()


def test_projection_and_energy_closed_forms():
    """e = f R and q_j = sum_i |R[j][i]|^2 on inputs whose sums are known in closed form: rows of unit-modulus
    geometric sequences R[j][i] = exp(2 pi i j i / m) scaled by a_j, with f = 1 and with f = the ramp 0, 1, 2, ..."""
    n, d, m = 6, 40, 8
    a = np.array([1.0, 2.0, 0.5, 3.0, 1.5, 0.25])
    i = np.arange(d)
    z = np.exp(2j * np.pi * np.arange(n) / m)                       # ratio of row j's geometric sequence
    R = a[:, None] * z[:, None] ** i[None, :]
    # q: every entry of row j has modulus a_j
    np.testing.assert_allclose(orc.cyc_project_energy(R), d * a ** 2, rtol=1e-13)
    # f = 1: geometric sum (row 0 has ratio 1); d = 40 is a multiple of m / gcd(j, m) for every j, so the others vanish
    e1 = orc.cyc_project(R, np.ones(d))
    want1 = np.where(np.arange(n) == 0, a * d, 0.0)
    np.testing.assert_allclose(e1, want1, atol=1e-12)
    # f = ramp: sum_i i z^i = z (1 - d z^(d-1) + (d-1) z^d) / (1 - z)^2 for z != 1, d (d - 1) / 2 for z = 1
    e2 = orc.cyc_project(R, i.astype(np.float64))
    zz = z[1:]
    want2 = np.concatenate([[a[0] * d * (d - 1) / 2], a[1:] * zz * (1 - d * zz ** (d - 1) + (d - 1) * zz ** d) / (1 - zz) ** 2])
    np.testing.assert_allclose(e2, want2, rtol=1e-11, atol=1e-11)
    # a transposed or conjugated operand would not pass: the ramp sum of row 1 has a non-zero imaginary part of known sign
    assert want2[1].imag < -1.0 and abs(e2[1].imag - want2[1].imag) < 1e-9


def test_adjacent_adversaries_at_45_5_are_decoded_at_every_position():
    """Definition 2 at the paper's own size with the worst placement for complex64 vectors: five adversaries side by
    side, at each of the 45 positions on the circle.  One pass of the locator misses one of them in about half of the
    positions (the 5 x 5 system's smallest singular value is a few times the cutoff); the passes with erasures find
    a set that contains all five, at most 2 s nodes in all, and the sum comes out to the accuracy of the transport."""
    n, s, d = 45, 5, 1024
    W = orc.cyc_W(n, s)
    worst = 0.0
    supersets = 0
    for start in range(n):
        adv = [(start + k) % n for k in range(s)]
        G = di.gradient_rows(1000 + start, n, d)
        R = orc.cyc_encode(G, n, s, W=W)
        di.apply_adversaries(R, adv, [di.ADV_REVGRAD] * s, [100.0] * s, seed=3)
        f = di.projection_vector(2000 + start, d)
        out = orc.cyc_decode_full(R, f, n, s)
        found = set(np.flatnonzero(out["flags"]))
        assert found >= set(adv) and len(found) <= 2 * s, (start, sorted(found))
        supersets += found != set(adv)
        exact = _exact_sum(G)
        worst = max(worst, np.abs(out["u"] - exact).max() / np.abs(exact).max())
    assert worst <= 2e-2, worst          # complex64 floor at (45, 5) is about 1.5e-3; a sixth erasure costs a little
    assert supersets <= 15               # an honest node is blamed along with the five in about a quarter of the positions


def test_known_bad_nodes_cost_one_syndrome_each():
    """Nodes with a non-finite record are erasures from the start: s of them plus floor(s / 2) ordinary adversaries,
    more than s nodes in all, are still all found and the sum is exact (2 s syndromes = erasures + 2 x errors)."""
    import warnings
    n, s, d = 15, 4, 64
    G = di.gradient_rows(5, n, d)
    Z = orc.cyc_encode(G, n, s)
    f = di.projection_vector(6, d)
    exact = _exact_sum(G)
    rng = np.random.default_rng(0)
    with warnings.catch_warnings():
        warnings.simplefilter("ignore")
        for trial in range(40):
            nodes = rng.choice(n, s + s // 2, replace=False)
            R = Z.copy()
            for j in nodes[:s]:
                R[j, int(rng.integers(0, d))] = np.nan
            for j in nodes[s:]:
                R[j] = -100 * R[j]
            out = orc.cyc_decode_full(R, f, n, s)
            assert set(np.flatnonzero(out["flags"])) == set(nodes.tolist())
            assert np.abs(out["u"] - exact).max() <= 1e-4 * np.abs(exact).max()
