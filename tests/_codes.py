"""Test-side builders of valid code matrices (A, w) handed to BOTH the oracle and the
CUDA path. Values come from the float64 design oracle; nothing here is used by
the product."""
import numpy as np

from oracle import design as od


def identity_code(n):
    return (np.arange(n + 1, dtype=np.int32), np.arange(n, dtype=np.int32), np.ones(n, np.float32),
            np.ones(n, np.float32))


def interval_code(p, bits, k, dim):
    alpha = od.interval_alpha(od.optimal_row_sums(p, bits, k, dim), k)
    rp, ci, vals = od.alpha_to_csr(alpha)
    _, w = od.physical_coefficients(alpha, p)
    return rp, ci, vals.astype(np.float32), w.astype(np.float32)


def cyclic_code(p, bits, k, s, dim):
    """Unbiased code on the cyclic-s support: each partition's unit mass is split among
    its holders in proportion to c_i^-1 (the column-normalised closed form)."""
    n = len(p)
    sup = od.cyclic_support(n, k, s)
    cinv = 1.0 / od.c_coeff(p, bits, dim)
    alpha = np.zeros((n, k))
    for i, cols in enumerate(sup):
        alpha[i, cols] = cinv[i]
    alpha /= alpha.sum(0, keepdims=True)
    rp, ci, vals = od.alpha_to_csr(alpha)
    _, w = od.physical_coefficients(alpha, p)
    return rp, ci, vals.astype(np.float32), w.astype(np.float32)
