"""INT4 x INT4 matrix product with an INT32 accumulator (App. J, "Setup").

Test infrastructure (see the package header).

acc[t, n] = sum_k (qa[t, k] - z) * qw[n, k], exactly, as 32-bit integers.  Both
operands are row-major over k (activations [M, K], stored weights [N, K]), so the
product is qa @ qw^T.

`int_matmul` uses the float64 BLAS product as its library step: every operand
is an integer of magnitude < 16, every partial sum stays below 2^53, so the
float64 result is the exact integer.  `int_matmul_bruteforce` is the definition
as a triple loop over Python integers; the tests pin the former to the latter.
"""
import numpy as np


def int_matmul(qa, qw, z=0):
    a = np.asarray(qa).astype(np.float64) - float(z)
    w = np.asarray(qw).astype(np.float64)
    acc = a @ w.T
    assert np.all(np.abs(acc) < 2.0 ** 31), "accumulator leaves the int32 range"
    out = acc.astype(np.int64)
    assert np.array_equal(out.astype(np.float64), acc), "non-integer accumulator"
    return out.astype(np.int32)


def int_matmul_bruteforce(qa, qw, z=0):
    """The same product with arbitrary-precision Python integers (tiny shapes only)."""
    qa = np.asarray(qa)
    qw = np.asarray(qw)
    M, K = qa.shape
    N, K2 = qw.shape
    assert K == K2
    out = [[0] * N for _ in range(M)]
    for t in range(M):
        for n in range(N):
            s = 0
            for k in range(K):
                s += (int(qa[t, k]) - int(z)) * int(qw[n, k])
            out[t][n] = s
    return np.array(out, dtype=np.int64)
