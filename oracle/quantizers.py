"""Uniform integer quantisers of the W4A4 path, step by step.

Test infrastructure (see the package header).

What the paper fixes
  * values are mapped to a uniform integer grid (Sec. 1, "Quantization"),
    with round-to-nearest (Sec. 4, "Baselines": RTN) and a scale and offset per
    quantiser (App. D, "General set-up");
  * static quantisation fixes the grid ahead of inference from calibration data
    and applies only floating-point scale factors after the integer matmul
    (App. B, "Static quantization");
  * the initial grid minimises the L_p norm of the quantisation error, p = 3,
    and L_inf is plain min-max (App. D, "Quantizer range setting");
  * the per-token scale is the reciprocal root-mean-square that the existing
    RMSNorm computes, S_n = S_{n-1} / ||Z~_{n-1}||_R (Sec. 3.1.3, Eq. 6-7), and
    it may be applied anywhere along a bias-free linear chain (Sec. 3.1.3);
  * two INT4 codes share one byte (App. J, "Setup").

What the paper leaves open, and the reading taken here (the CUDA library states
the same readings in its header, in its own words)
  * the grid formula: symmetric q = clamp(rne(x/D), -2^(b-1), 2^(b-1)-1),
    x^ = D*q; asymmetric q = clamp(rne(x/D) + z, 0, 2^b - 1), x^ = D*(q - z);
  * rounding is to nearest with ties to even;
  * the static activation scale is one scalar per tensor;
  * the dynamic variant (App. B) uses, per token, the symmetric grid that ends at the
    token's largest magnitude;
  * arithmetic precision: float32 with one rounding per operation and no fused
    multiply-add, except the sum of squares of the RMS, which is accumulated in
    float64 and rounded once;
  * the byte layout: code 2j in bits 0..3 and code 2j+1 in bits 4..7 of byte j,
    two's complement nibbles on the symmetric grid;
  * SiLU uses a fixed polynomial exp2 so that it has one defined float32 result.
"""
from dataclasses import dataclass
import math

import numpy as np

from .bf16 import round_to_bf16

F32 = np.float32


@dataclass(frozen=True)
class QParams:
    """One quantiser: bit-width, grid kind, static scale D, zero point z."""
    bits: int = 4
    symmetric: bool = True
    scale: float = 1.0
    zero_point: int = 0

    @property
    def qmin(self):
        return -(1 << (self.bits - 1)) if self.symmetric else 0

    @property
    def qmax(self):
        return (1 << (self.bits - 1)) - 1 if self.symmetric else (1 << self.bits) - 1

    @property
    def z(self):
        return 0 if self.symmetric else int(self.zero_point)


# --------------------------------------------------------------------------- #
# grid primitives
# --------------------------------------------------------------------------- #
def round_clamp(u, z, qmin, qmax):
    """codes = clamp(rne(u) + z, qmin, qmax); a NaN maps to the lowest code."""
    u = np.asarray(u, dtype=F32)
    v = np.rint(u) + F32(z)                      # rint: ties to even
    v = np.where(np.isnan(v), F32(qmin), v)
    v = np.minimum(np.maximum(v, F32(qmin)), F32(qmax))
    return v.astype(np.int8 if qmin < 0 else np.uint8)


def dequantize(codes, scale, z=0):
    """x^ = D * (q - z) in float64 (used by the invariants, not by the path)."""
    return np.float64(scale) * (np.asarray(codes, dtype=np.float64) - z)


def pack_int4(codes):
    """[R, K] codes -> [R, K/2] bytes; code 2j low nibble, code 2j+1 high nibble."""
    c = np.asarray(codes)
    assert c.shape[-1] % 2 == 0
    n = (c.astype(np.int16) & 0xF).astype(np.uint8)
    return (n[..., 0::2] | (n[..., 1::2] << np.uint8(4))).astype(np.uint8)


def unpack_int4(packed, symmetric=True):
    """Inverse of pack_int4."""
    p = np.asarray(packed, dtype=np.uint8)
    lo = (p & np.uint8(0xF)).astype(np.int16)
    hi = (p >> np.uint8(4)).astype(np.int16)
    out = np.empty(p.shape[:-1] + (p.shape[-1] * 2,), dtype=np.int16)
    out[..., 0::2] = lo
    out[..., 1::2] = hi
    if symmetric:
        out = np.where(out >= 8, out - 16, out)
        return out.astype(np.int8)
    return out.astype(np.uint8)


# --------------------------------------------------------------------------- #
# weight quantiser (offline): per-output-channel symmetric grid
# --------------------------------------------------------------------------- #
RANGE_MINMAX = 0
RANGE_LP = 1


def _store_scale(delta, scale_dtype):
    if scale_dtype == "fp16":
        return delta.astype(np.float16).astype(F32)
    assert scale_dtype == "fp32"
    return delta.astype(F32)


def quantize_weights(w, qp=QParams(), range_mode=RANGE_MINMAX, p=3.0, scale_dtype="fp32"):
    """Per-row (output channel) symmetric quantiser of a stored [N, K] weight.

    MINMAX (the L_inf grid): D_n = max_k|w_nk| / qmax.
    LP: over the candidates D_i = (a_n * (i/100)) / qmax, i = 20..100, the one
        with the least sum_k |w - D*clamp(rne(w/D))|^p, evaluated in float64;
        equal errors go to the larger i.
    The scale is rounded to its storage type before it is used; an all-zero row
    gets D = 1.  Returns (codes int8 [N,K], scales float32 [N], row sums int32).
    """
    assert qp.symmetric, "weights use the symmetric grid"
    w = np.ascontiguousarray(w, dtype=F32)
    qmin, qmax = qp.qmin, qp.qmax
    a = np.max(np.abs(w), axis=1)                                   # [N] float32

    def grid(frac):
        d = (a * F32(frac)) / F32(qmax) if frac is not None else a / F32(qmax)
        d = _store_scale(d.astype(F32), scale_dtype)
        return np.where((a == 0) | (d == 0), F32(1.0), d).astype(F32)

    if range_mode == RANGE_MINMAX:
        delta = grid(None)
    else:
        best_err = np.full(a.shape, np.inf)
        delta = grid(None)
        for i in range(20, 101):
            d = grid(F32(i) / F32(100.0))
            q = round_clamp(w / d[:, None], 0, qmin, qmax)
            e = np.abs(w.astype(np.float64) - d[:, None].astype(np.float64) * q)
            err = np.sum(e ** p, axis=1)
            take = err <= best_err
            best_err = np.where(take, err, best_err)
            delta = np.where(take, d, delta).astype(F32)
    codes = round_clamp(w / delta[:, None], 0, qmin, qmax)          # IEEE float32 division
    wsum = codes.astype(np.int64).sum(axis=1).astype(np.int32)
    return codes, delta, wsum


# --------------------------------------------------------------------------- #
# per-token scale from the RMSNorm, and the static activation quantiser
# --------------------------------------------------------------------------- #
def rms_reciprocal(x, eps):
    """r_t = 1 / sqrt(mean_k x_tk^2 + eps), the factor the RMSNorm applies.

    ||x||_R = ||x||_2 / sqrt(d) (Sec. 3.1.3, Step 1).  Each square is formed in
    float32 (exact for bfloat16 inputs), the sum is taken in float64 and rounded
    once to float32; the mean, the square root and the reciprocal are float32.
    """
    x = np.asarray(x, dtype=F32)
    sq = (x * x).astype(np.float64)
    ss = sq.sum(axis=1).astype(F32)
    ms = ss / F32(x.shape[1])
    rho = np.sqrt(ms + F32(eps))
    return (F32(1.0) / rho).astype(F32)


def act_quant(x, qp, rmsnorm=True, scale_input=False, eps=1e-5, s_in=None):
    """Static activation quantiser with the per-token scale (one row = one token).

      r_t   = RMSNorm reciprocal (rmsnorm) or 1
      p_t   = r_t * s_in[t] if scale_input else r_t        multiplier before the grid
      q_tk  = clamp(rne((x_tk * p_t) * (1/D)) + z)
      S_out = r_t * s_in[t] (s_in given) else r_t          S_n = S_{n-1} / ||Z~_{n-1}||_R

    Block inputs (after the norm) use rmsnorm=True, scale_input=False: the grid
    sees RMSNorm(x) and S_out carries the recursion of Eq. 7.  Sites inside a
    block (attention output, down-projection input) use rmsnorm=False,
    scale_input=True: the grid sees S_n * x.
    Returns (codes, S_out, p, r), float32 vectors of length M.
    """
    x = np.asarray(x, dtype=F32)
    M = x.shape[0]
    r = rms_reciprocal(x, eps) if rmsnorm else np.ones(M, dtype=F32)
    s = None if s_in is None else np.asarray(s_in, dtype=F32)
    p = (r * s).astype(F32) if (scale_input and s is not None) else r
    s_out = (r * s).astype(F32) if s is not None else r
    inv_d = F32(1.0) / F32(qp.scale)
    u = (x * p[:, None]) * inv_d                                   # two roundings, no FMA
    codes = round_clamp(u, qp.z, qp.qmin, qp.qmax)
    return codes, s_out, p, r


def act_quant_dynamic(x, bits=4, rmsnorm=True, scale_input=False, eps=1e-5, s_in=None):
    """Dynamic activation quantiser: one grid per token, computed at run time (App. B, "Dynamic
    quantization": the extreme activation values are reduced over the last dimension for each
    token and the resulting scale factor is applied to each value).

    Reading taken (the paper gives no formula): the symmetric grid whose end is the token's
    largest magnitude,
      v_tk    = x_tk * p_t                          p_t as in act_quant
      m_t     = max_k |v_tk|
      D_t     = m_t / qmax   (float32 division);  D_t = 1 when m_t is zero, infinite or NaN
      q_tk    = clamp(rne(v_tk * (1 / D_t)), qmin, qmax)      (1 / D_t: float32 division)
    Returns (codes, D [M] float32, S_out, p, r).
    """
    x = np.asarray(x, dtype=F32)
    M = x.shape[0]
    qp = QParams(bits, True, 1.0, 0)
    r = rms_reciprocal(x, eps) if rmsnorm else np.ones(M, dtype=F32)
    s = None if s_in is None else np.asarray(s_in, dtype=F32)
    p = (r * s).astype(F32) if (scale_input and s is not None) else r
    s_out = (r * s).astype(F32) if s is not None else r
    v = (x * p[:, None]).astype(F32)
    with np.errstate(invalid="ignore"):
        m = np.max(np.abs(v), axis=1).astype(F32)              # NaN propagates
        ok = np.isfinite(m) & (m > 0)
        delta = np.where(ok, m / F32(qp.qmax), F32(1.0)).astype(F32)
    inv = (F32(1.0) / delta).astype(F32)
    u = (v * inv[:, None]).astype(F32)
    codes = round_clamp(u, 0, qp.qmin, qp.qmax)
    return codes, delta, s_out, p, r


# --------------------------------------------------------------------------- #
# SiLU * mul at the down-projection input
# --------------------------------------------------------------------------- #
_LN2 = math.log(2.0)
_EXP2_COEF = [F32(_LN2 ** k / math.factorial(k)) for k in range(7)]   # Taylor of 2^f
_LOG2E = F32(1.0 / _LN2)


def exp2_spec(t):
    """2^t in float32 with a fixed sequence of roundings.

    t is clamped to [-126, 126]; n = rne(t); f = t - n (exact); 2^f by the
    degree-6 Taylor polynomial of 2^f in Horner form, every multiply and every
    add rounded to float32 separately; the result is scaled by 2^n exactly.
    """
    t = np.minimum(np.maximum(np.asarray(t, dtype=F32), F32(-126.0)), F32(126.0))
    n = np.rint(t)
    f = (t - n).astype(F32)
    acc = np.full(t.shape, _EXP2_COEF[6], dtype=F32)
    for k in range(5, -1, -1):
        acc = (acc * f).astype(F32)
        acc = (acc + _EXP2_COEF[k]).astype(F32)
    two_n = ((n.astype(np.int32) + 127).astype(np.uint32) << np.uint32(23)).view(F32)
    return (acc * two_n).astype(F32)


def silu_spec(g):
    """silu(g) = g / (1 + 2^(-g*log2 e)) in float32, IEEE division."""
    g = np.asarray(g, dtype=F32)
    e = exp2_spec((-g) * _LOG2E)
    return (g / (F32(1.0) + e)).astype(F32)


def silu_mul(g, u):
    """bf16(silu(g) * u): the SwiGLU product, kept in 16-bit as in App. J."""
    return round_to_bf16(silu_spec(g) * np.asarray(u, dtype=F32))


def silu_mul_quant(g, u, qp, s_n=None):
    """Down-projection input: q = clamp(rne((m * S_n[t]) * (1/D)) + z), m = bf16(silu(g)*u)."""
    m = silu_mul(g, u)
    codes, _, p, _ = act_quant(m, qp, rmsnorm=False, scale_input=True, s_in=s_n)
    return codes, m


# --------------------------------------------------------------------------- #
# range setting of the static activation scale (harness side)
# --------------------------------------------------------------------------- #
def calibrate_static_scale(v, qp, p=3.0, steps=100):
    """Static per-tensor scale from a calibration batch (App. D, L_p range setting).

    v holds the values the grid will see (already multiplied by the per-token
    scale).  Candidates D_i = absmax * i / (steps * qmax), i = 1..steps (asymmetric: the
    larger distance from z to a grid end in place of qmax); the
    one with the least sum |v - D*(clamp(rne(v/D)+z) - z)|^p in float64 wins,
    equal errors going to the larger D.  Returns a float32 scalar.
    """
    v = np.asarray(v, dtype=np.float64).ravel()
    amax = float(np.max(np.abs(v)))
    if amax == 0.0:
        return F32(1.0)
    span = qp.qmax if qp.symmetric else max(qp.z - qp.qmin, qp.qmax - qp.z)
    best, best_err = None, np.inf
    for i in range(1, steps + 1):
        d = float(F32(amax * i / (steps * span)))
        q = np.clip(np.rint(v / d) + qp.z, qp.qmin, qp.qmax)
        err = float(np.sum(np.abs(v - d * (q - qp.z)) ** p))
        if err <= best_err:
            best, best_err = d, err
    return F32(best)
