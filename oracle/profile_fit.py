"""CPU oracle for the latency-profile fit (Eq. 1 of Themis, arXiv 2407.14843).

TEST INFRASTRUCTURE ONLY; shares nothing with the CUDA path.  The profile of a
model is l(b, c) = gamma*b/c + epsilon/c + delta*b + eta (milliseconds), fitted
to measured samples by ordinary least squares; numpy's SVD-based ``lstsq`` in
float64 is the solver.  The table the scaling solvers consume is
ceil(1000 * l(b, c)) microseconds, at least 1.
"""
import numpy as np


def design_matrix(sample_b, sample_c):
    b = np.asarray(sample_b, dtype=np.float64)
    c = np.asarray(sample_c, dtype=np.float64)
    return np.stack([b / c, 1.0 / c, b, np.ones_like(b)], axis=1)


def fit_profiles(sample_b, sample_c, latency_ms, c_max, batch_sizes):
    """Returns (coeffs [M][4] = gamma, epsilon, delta, eta; lat_us [M][c_max][n_batch] int32;
    status [M]: 0, or -1 where the samples do not determine four coefficients)."""
    X = design_matrix(sample_b, sample_c)
    lat = np.asarray(latency_ms, dtype=np.float64)
    M = lat.shape[0]
    coeffs = np.zeros((M, 4))
    status = np.zeros(M, np.int32)
    rank = np.linalg.matrix_rank(X)
    for m in range(M):
        if rank < 4:
            status[m] = -1
            continue
        coeffs[m] = np.linalg.lstsq(X, lat[m], rcond=None)[0]
    c = np.arange(1, c_max + 1, dtype=np.float64)[:, None]
    b = np.asarray(batch_sizes, dtype=np.float64)[None, :]
    g, e, d, h = (coeffs[:, i][:, None, None] for i in range(4))
    l_ms = g * b / c + e / c + d * b + h
    lat_us = np.clip(np.ceil(l_ms * 1000.0), 1, 2 ** 31 - 1).astype(np.int32)
    lat_us[status != 0] = 0
    return coeffs, lat_us, status
