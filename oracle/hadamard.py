"""Block-wise Hadamard transform at the down-projection input (Sec. 3.1, last paragraph; the
transform table of App. A: H_n = n^(-1/2) (x)_{i=1..log2 n} [[1, 1], [1, -1]]; App. D "Hadamard
non-powers of 2": the channels are split into K groups of a power-of-two size, reshaped to
(K, 2^n), and a standard Hadamard is applied to each group -- never zero padding, which would
not be invertible on the original dimension).

Test infrastructure (see the package header).

What the paper leaves open, and the reading taken here
  * the group size: the largest power of two that divides the dimension (14336 = 7 x 2048);
  * arithmetic: float32 butterflies (a, b) -> (a + b, a - b), one rounding each, taken stage by
    stage with the distance between partners growing 1, 2, 4, ..., n/2 (the Kronecker factors
    from the last to the first), followed by ONE float32 multiply by float32(n^(-1/2));
  * the result stays float32 until the quantiser reads it (no 16-bit rounding in between).

`hadamard_matrix` is the definition written out in float64; the tests pin the butterfly form to
it, to scipy's construction, to orthogonality and to invertibility on the full dimension.
"""
import numpy as np

F32 = np.float32


def largest_pow2_divisor(d):
    return d & (-d)


def hadamard_matrix(n):
    """H_n by its Kronecker definition, float64, with the n^(-1/2) factor."""
    assert n >= 1 and n & (n - 1) == 0
    h = np.ones((1, 1))
    base = np.array([[1.0, 1.0], [1.0, -1.0]])
    while h.shape[0] < n:
        h = np.kron(base, h)
    return h / np.sqrt(n)


def block_hadamard_matrix(d, block=None):
    """blockdiag(H_block, ..., H_block) on d channels, float64."""
    block = block or largest_pow2_divisor(d)
    assert d % block == 0
    return np.kron(np.eye(d // block), hadamard_matrix(block))


def block_hadamard_f32(x, block=None):
    """Rows of x [M, d] transformed group by group with the float32 butterfly sequence above."""
    x = np.ascontiguousarray(x, dtype=F32)
    M, d = x.shape
    block = block or largest_pow2_divisor(d)
    assert d % block == 0 and block & (block - 1) == 0
    y = x.reshape(M, d // block, block).copy()
    s = 1
    while s < block:
        v = y.reshape(M, d // block, block // (2 * s), 2, s)
        a = v[:, :, :, 0, :].copy()
        b = v[:, :, :, 1, :].copy()
        v[:, :, :, 0, :] = (a + b).astype(F32)
        v[:, :, :, 1, :] = (a - b).astype(F32)
        s *= 2
    norm = F32(1.0 / np.sqrt(np.float64(block)))
    return (y * norm).astype(F32).reshape(M, d)
