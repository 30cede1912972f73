"""Pins of the oracle's block-wise Hadamard (App. A transform table; App. D "Hadamard non-powers of
2") against things other than itself: the Kronecker definition, scipy's construction,
orthogonality, invertibility on the full (non-power-of-two) dimension, and the textbook 2- and
4-point values."""
import numpy as np
import pytest
import scipy.linalg

from oracle import hadamard as OH


def test_small_cases_by_hand():
    h2 = OH.hadamard_matrix(2) * np.sqrt(2)
    assert np.array_equal(h2, [[1, 1], [1, -1]])
    x = np.array([[1.0, 2.0, 3.0, 4.0]], dtype=np.float32)
    # H_4 x = 1/2 (10, -2, -4, 0)
    assert np.array_equal(OH.block_hadamard_f32(x, 4), np.array([[5.0, -1.0, -2.0, 0.0]], dtype=np.float32))


@pytest.mark.parametrize("n", [2, 8, 256, 2048])
def test_matrix_is_scipys_and_orthogonal(n):
    h = OH.hadamard_matrix(n)
    assert np.array_equal(h * np.sqrt(n), scipy.linalg.hadamard(n))
    assert np.allclose(h @ h.T, np.eye(n), atol=1e-12) and np.allclose(h, h.T)


@pytest.mark.parametrize("d,block", [(14336, 2048), (28672, 4096), (3584, 512), (768, 256), (96, 32)])
def test_group_size_and_butterflies_match_the_definition(d, block):
    assert OH.largest_pow2_divisor(d) == block
    rng = np.random.default_rng(d)
    x = rng.standard_normal((3, d)).astype(np.float32)
    got = OH.block_hadamard_f32(x)
    hb = OH.hadamard_matrix(block)
    want = (x.astype(np.float64).reshape(3, d // block, block) @ hb.T).reshape(3, d)
    assert np.max(np.abs(got - want)) < 2e-5 * np.max(np.abs(want))
    # groups do not mix: zeroing one group's input changes only that group's output
    x2 = x.copy()
    x2[:, :block] = 0
    got2 = OH.block_hadamard_f32(x2)
    assert np.array_equal(got2[:, block:], got[:, block:]) and not np.any(got2[:, :block])


def test_invertible_on_the_full_dimension_without_padding():
    d = 14336
    rng = np.random.default_rng(0)
    x = rng.standard_normal((2, d)).astype(np.float32)
    y = OH.block_hadamard_f32(x)
    assert y.shape == x.shape                                   # no padded channels to discard
    back = OH.block_hadamard_f32(y)                             # H is its own inverse
    assert np.max(np.abs(back - x)) < 1e-5
    assert np.allclose(np.sum(y.astype(np.float64) ** 2, axis=1), np.sum(x.astype(np.float64) ** 2, axis=1), rtol=1e-5)


def test_exact_on_small_integers_and_stage_order_is_fixed():
    # integers below 2^24 / n: every butterfly is exact, so any stage order gives the same bits ...
    rng = np.random.default_rng(1)
    xi = rng.integers(-50, 50, (4, 1024)).astype(np.float32)
    got = OH.block_hadamard_f32(xi, 1024)
    want = (xi.astype(np.float64) @ (OH.hadamard_matrix(1024) * 32.0).T) * float(np.float32(1 / 32.0))
    assert np.array_equal(got.astype(np.float64), want)
    # ... and for general floats the result is the float32 value sequence of the stated order
    x = rng.standard_normal((1, 8)).astype(np.float32)
    a = x[0].copy()
    for s in (1, 2, 4):
        b = a.copy()
        for i in range(8):
            j = i ^ s
            lo, hi = (i, j) if i < j else (j, i)
            b[i] = np.float32(a[lo] + a[hi]) if i == lo else np.float32(a[lo] - a[hi])
        a = b
    assert np.array_equal(OH.block_hadamard_f32(x, 8)[0], (a * np.float32(1 / np.sqrt(8.0))).astype(np.float32))


def _golden(name):
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", name)
    rows = [ln.split() for ln in open(path) if ln.strip() and not ln.startswith("#")]
    return np.array(rows, dtype=np.float64)


def test_values_the_paper_prints():
    """tests/golden: the group count and size the paper states for Llama-2 7B's FFN width (App. D), and
    H_4 written out from the paper's Kronecker definition."""
    for d, groups, size in _golden("hadamard_groups.txt").astype(np.int64):
        assert OH.largest_pow2_divisor(int(d)) == size and d // size == groups
        m = OH.block_hadamard_matrix(int(d))
        assert m.shape == (d, d)
        assert np.count_nonzero(m[:size, size:]) == 0 and np.count_nonzero(m[size:2 * size, :size]) == 0   # block diagonal
    h4 = _golden("hadamard_h4.txt")
    assert np.array_equal(OH.hadamard_matrix(4) * 2.0, h4)          # the table's factor n^(-1/2) = 1/2 taken out
    x = np.arange(8, dtype=np.float32).reshape(2, 4)
    assert np.array_equal(OH.block_hadamard_f32(x), (x.astype(np.float64) @ h4.T * 0.5).astype(np.float32))
