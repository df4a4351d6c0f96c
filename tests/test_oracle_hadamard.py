"""Pins for the oracle's Hadamard transform: scipy's Sylvester Hadamard matrix is the independent
library reference; orthogonality and Parseval are the mathematical invariants."""
import numpy as np
import pytest
from scipy.linalg import hadamard

import oracle


@pytest.mark.parametrize("h", [2, 4, 64, 256, 1024])
def test_definition_and_butterfly_match_library_matrix(h):
    rng = np.random.default_rng(h)
    x = rng.standard_normal(h)
    ref = hadamard(h).astype(np.float64) @ x
    tol = 1e-12 * np.abs(ref).max() * np.sqrt(h)
    assert np.abs(oracle.hadamard_definition(x) - ref).max() <= tol
    assert np.abs(oracle.hadamard_butterfly(x) - ref).max() <= tol


@pytest.mark.parametrize("h", [64, 1024])
def test_unit_vectors_give_matrix_columns(h):
    # catches a wrong ordering (e.g. sequency order) or a transposed/asymmetric butterfly
    H = hadamard(h)
    for j in (0, 1, 2, 3, 5, h // 2, h - 1):
        e = np.zeros(h)
        e[j] = 1.0
        assert np.array_equal(oracle.hadamard_butterfly(e), H[:, j].astype(np.float64))


@pytest.mark.parametrize("h", [64, 1024])
def test_involution_and_parseval(h):
    rng = np.random.default_rng(3)
    x = rng.standard_normal(h)
    y = oracle.hadamard_butterfly(x) / np.sqrt(h)
    back = oracle.hadamard_butterfly(y) / np.sqrt(h)
    assert np.abs(back - x).max() <= 1e-12          # unquantized round trip (bound 1e-6 needed)
    assert abs(np.dot(y, y) - np.dot(x, x)) <= 1e-10 * np.dot(x, x)
