"""Eq. 1 profile fit: pins for the oracle (CPU) and parity of the CUDA fit."""
import numpy as np
import pytest

from paper_2407_14843_b200 import workloads as W
from oracle import profile_fit


def test_oracle_recovers_exact_coefficients():
    """Noise-free samples of a known profile: the fit returns the generating
    coefficients and a table that is the profile itself."""
    sb, sc, lat, true = W.profile_samples(5, 16, noise=0.0)
    coeffs, lat_us, status = profile_fit.fit_profiles(sb, sc, lat, 16, (1, 2, 4, 8, 16))
    assert (status == 0).all()
    assert np.allclose(coeffs, true, rtol=1e-9, atol=1e-9)
    g, e, d, h = true[3]
    assert abs(lat_us[3, 3, 2] - np.ceil(1000 * (g * 4 / 4 + e / 4 + d * 4 + h))) <= 1   # c = 4, b = 4


def test_oracle_residual_is_orthogonal_to_the_regressors():
    """Least squares: X^T (l - X beta) = 0, and no other coefficients fit better."""
    sb, sc, lat, _ = W.profile_samples(6, 8)
    coeffs, _, _ = profile_fit.fit_profiles(sb, sc, lat, 16, (1, 2, 4))
    X = profile_fit.design_matrix(sb, sc)
    for m in range(8):
        r = lat[m] - X @ coeffs[m]
        assert np.abs(X.T @ r).max() < 1e-8 * np.abs(X.T @ lat[m]).max()
        rng = np.random.default_rng(m)
        for _ in range(5):
            other = coeffs[m] * (1 + 1e-3 * rng.standard_normal(4))
            assert np.sum((lat[m] - X @ other) ** 2) >= np.sum(r ** 2)


def test_oracle_flags_underdetermined_samples():
    """All samples on one core: b/c and b coincide, four coefficients are not determined."""
    b = np.asarray([1, 2, 4, 8, 16], np.int32)
    c = np.ones(5, np.int32)
    _, lat_us, status = profile_fit.fit_profiles(b, c, np.ones((2, 5)), 4, (1, 2))
    assert (status == -1).all() and not lat_us.any()


@pytest.mark.gpu
def test_cuda_fit_matches_the_oracle():
    """Coefficients to 1e-8 relative (both sides float64, different elimination
    orders); table entries equal, except that a value within rounding of an integer
    number of microseconds may land on either side (at most 1 us, < 0.1 % of entries)."""
    import torch
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    from paper_2407_14843_b200 import build
    build.build_library()
    from paper_2407_14843_b200 import solver as S
    for n_models, c_max, batches in ((1, 4, (1,)), (37, 16, (1, 2, 4, 8, 16)), (640, 64, (1, 2, 4, 8, 16, 32, 64))):
        sb, sc, lat, _ = W.profile_samples(40 + n_models, n_models)
        ref_c, ref_t, ref_s = profile_fit.fit_profiles(sb, sc, lat, c_max, batches)
        dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
        coeffs = torch.empty((n_models, 4), dtype=torch.float64, device="cuda")
        tab = torch.empty((n_models, c_max, len(batches)), dtype=torch.int32, device="cuda")
        status = torch.empty(n_models, dtype=torch.int32, device="cuda")
        S.themis_fit_profiles_batch(dev(sb), dev(sc), dev(lat), c_max, dev(np.asarray(batches, np.int32)),
                                    coeffs, tab, status)
        torch.cuda.synchronize()
        assert np.array_equal(status.cpu().numpy(), ref_s)
        assert np.allclose(coeffs.cpu().numpy(), ref_c, rtol=1e-8, atol=1e-10)
        diff = np.abs(tab.cpu().numpy().astype(np.int64) - ref_t)
        assert diff.max() <= 1 and (diff != 0).mean() < 1e-3
    # underdetermined samples are reported, not fitted
    b = np.asarray([1, 2, 4, 8, 16], np.int32)
    coeffs = torch.empty((2, 4), dtype=torch.float64, device="cuda")
    tab = torch.empty((2, 4, 2), dtype=torch.int32, device="cuda")
    status = torch.empty(2, dtype=torch.int32, device="cuda")
    S.themis_fit_profiles_batch(dev(b), dev(np.ones(5, np.int32)), dev(np.ones((2, 5))), 4,
                                dev(np.asarray((1, 2), np.int32)), coeffs, tab, status)
    torch.cuda.synchronize()
    assert (status.cpu().numpy() == S.STATUS_BAD_INPUT).all() and not tab.cpu().numpy().any()
