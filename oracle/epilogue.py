"""Floating-point scale factors applied after the integer matmul
(App. B, "Static quantization").

Test infrastructure (see the package header).

    c_t    = D_a * post[t]                     (D_a alone when there is no post vector)
    y[t,n] = bf16( ((float)acc[t,n] * sw[n]) * c_t  [+ res[t,n]] )

All in float32, one rounding per operation, no fused multiply-add; the final
narrowing is round-to-nearest-even.  `post` is the caller's choice of where the
per-token scale ends up (Sec. 3.1.3: the scale commutes with a bias-free linear):
absent (the output stays in the scaled domain), the reciprocal of the
pre-quantisation multiplier (plain-linear semantics), or any vector.
"""
import numpy as np

from .bf16 import round_to_bf16

F32 = np.float32


def dequant_epilogue(acc, sw, act_scale, post=None, residual=None):
    acc = np.asarray(acc)
    assert np.all(np.abs(acc.astype(np.int64)) < (1 << 24)), "(float)acc must be exact"
    sw = np.asarray(sw, dtype=F32)
    M = acc.shape[0]
    if post is None:
        c = np.full(M, F32(act_scale), dtype=F32)
    else:
        c = (F32(act_scale) * np.asarray(post, dtype=F32)).astype(F32)
    y = (acc.astype(F32) * sw[None, :]).astype(F32)
    y = (y * c[:, None]).astype(F32)
    if residual is not None:
        y = (y + np.asarray(residual, dtype=F32)).astype(F32)
    return round_to_bf16(y)


def inverse_of_pre(p):
    """post = 1 / p_t, IEEE float32 division."""
    return (F32(1.0) / np.asarray(p, dtype=F32)).astype(F32)
