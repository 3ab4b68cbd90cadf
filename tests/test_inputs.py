"""The seeded input generator: published SplitMix64 vectors, moments, and the
random-access property (a slice or sample equals the whole)."""
import numpy as np

import draco_inputs as di


def test_splitmix64_published_vectors():
    # First outputs of SplitMix64 from state 0 (reference implementation by S. Vigna).
    got = [int(di.splitmix64_at(0, c)) for c in range(4)]
    assert got == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F, 0xF88BB8A8724C81EC]


def test_normal_moments():
    x = di.approx_normal_at(123, 5, np.arange(2_000_000)).astype(np.float64)
    assert abs(x.mean()) < 3e-3
    assert abs(x.std() - 1.0) < 3e-3
    assert abs((x ** 3).mean()) < 1e-2
    assert abs((x ** 4).mean() - 3.0 + 0.15) < 3e-2      # Irwin-Hall(8): excess kurtosis -6/40
    assert np.abs(x).max() <= 4.9


def test_slices_and_samples_equal_whole():
    n, d = 5, 1000
    G = di.gradient_rows(7, n, d, mean=0.25, std=0.1)
    assert G.dtype == np.float32 and G.shape == (n, d)
    np.testing.assert_array_equal(G[:, 100:333], di.gradient_rows(7, n, d, 0.25, 0.1, i0=100, i1=333))
    idx = np.array([999, 0, 17, 17, 512])
    np.testing.assert_array_equal(G[:, idx], di.gradient_rows(7, n, d, 0.25, 0.1, idx=idx))
    f = di.projection_vector(3, d)
    assert abs(f.mean() - 1.0) < 0.15
    np.testing.assert_array_equal(f[idx], di.projection_vector(3, d, idx=idx))
    Rc = di.complex_rows(11, n, d, std=2.0)
    assert Rc.dtype == np.complex64 and Rc.shape == (n, d)
    np.testing.assert_array_equal(Rc[:, 10:20], di.complex_rows(11, n, d, 2.0, i0=10, i1=20))
    np.testing.assert_array_equal(Rc[:, idx], di.complex_rows(11, n, d, 2.0, idx=idx))


def test_rows_differ_and_seeds_differ():
    a = di.approx_normal_at(1, 0, np.arange(64))
    assert not np.array_equal(a, di.approx_normal_at(1, 1, np.arange(64)))
    assert not np.array_equal(a, di.approx_normal_at(2, 0, np.arange(64)))


def test_adversaries_models_real_and_complex():
    n, d = 6, 200
    R0 = di.gradient_rows(1, n, d)
    R = R0.copy()
    di.apply_adversaries(R, [1, 4, 5], [di.ADV_REVGRAD, di.ADV_CONST, di.ADV_GAUSS], [100.0, -100.0, 1e3], seed=9)
    np.testing.assert_array_equal(R[1], R0[1] * np.float32(-100.0))
    assert np.all(R[4] == np.float32(-100.0))
    assert np.abs(R[5] - R0[5]).std() > 500
    for j in (0, 2, 3):
        np.testing.assert_array_equal(R[j], R0[j])
    # slice / sample consistency of the corruption
    Rs = R0[:, 50:90].copy()
    di.apply_adversaries(Rs, [1, 4, 5], [0, 1, 2], [100.0, -100.0, 1e3], seed=9, i0=50)
    np.testing.assert_array_equal(Rs, R[:, 50:90])
    C0 = di.complex_rows(2, n, d)
    C = C0.copy()
    di.apply_adversaries(C, [0, 3], [di.ADV_CONST, di.ADV_GAUSS], [1e4, 1e3], seed=5)
    assert np.all(C[0] == np.complex64(1e4))
    idx = np.array([3, 150, 77])
    Cs = C0[:, idx].copy()
    di.apply_adversaries(Cs, [0, 3], [1, 2], [1e4, 1e3], seed=5, idx=idx)
    np.testing.assert_array_equal(Cs, C[:, idx])


def test_choose_adversaries():
    a = di.choose_adversaries(4, 45, 5)
    assert len(set(a.tolist())) == 5 and a.min() >= 0 and a.max() < 45 and np.all(np.diff(a) > 0)
    np.testing.assert_array_equal(a, di.choose_adversaries(4, 45, 5))
