"""Pins for the oracle's quantisers: format definitions, closed forms, invariants,
brute force on tiny inputs.  None of them re-calls the function under test."""
import math

import numpy as np
import pytest
import torch

from oracle import bf16, quantizers as Q
from oracle.quantizers import QParams

F32 = np.float32


# ----------------------------- bfloat16 ------------------------------------ #
def test_bf16_widen_matches_torch_all_patterns():
    bits = np.arange(65536, dtype=np.uint16)
    ours = bf16.bf16_bits_to_f32(bits)
    t = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(ours.view(np.uint32), t.view(np.uint32))


def test_bf16_narrow_matches_torch_random_and_ties():
    rng = np.random.default_rng(1)
    x = rng.standard_normal(200000).astype(F32) * np.exp(rng.uniform(-30, 30, 200000)).astype(F32)
    # exact ties: kept mantissa even and odd, discarded half exactly 0x8000
    base = rng.integers(0, 1 << 16, 4096, dtype=np.uint32)
    ties = ((base << np.uint32(16)) | np.uint32(0x8000)).view(F32)
    x = np.concatenate([x, ties, np.array([0.0, -0.0, np.inf, -np.inf, 3.3895314e38], dtype=F32)])
    ours = bf16.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    finite = ~np.isnan(x)
    assert np.array_equal(ours[finite], ref[finite])
    assert np.isnan(bf16.round_to_bf16(np.array([np.nan], dtype=F32)))[0]


def test_bf16_hand_values():
    # 1 + 2^-8 is a tie between 1.0 (even) and 1 + 2^-7 -> 1.0; 1 + 3*2^-8 -> 1 + 2^-6 (even)
    x = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20], dtype=F32)
    assert bf16.round_to_bf16(x).tolist() == [1.0, 1.0 + 2.0 ** -6, 1.0 + 2.0 ** -7]


# ----------------------------- packing ------------------------------------- #
def test_pack_hand_bytes():
    assert Q.pack_int4(np.array([[-8, 7]], dtype=np.int8)).tolist() == [[0x78]]
    assert Q.pack_int4(np.array([[1, -1, 0, 3]], dtype=np.int8)).tolist() == [[0xF1, 0x30]]
    assert Q.pack_int4(np.array([[15, 0]], dtype=np.uint8)).tolist() == [[0x0F]]


def test_unpack_all_bytes_roundtrip():
    allb = np.arange(256, dtype=np.uint8)[None, :]
    for sym in (True, False):
        c = Q.unpack_int4(allb, sym)
        assert c.shape == (1, 512)
        assert c.min() == (-8 if sym else 0) and c.max() == (7 if sym else 15)
        assert np.array_equal(Q.pack_int4(c), allb)
    # byte 0x8F, symmetric: low nibble F = -1 first, high nibble 8 = -8 second
    assert Q.unpack_int4(np.array([[0x8F]], dtype=np.uint8)).tolist() == [[-1, -8]]


# ----------------------------- grid ---------------------------------------- #
def test_round_ties_to_even_table():
    u = np.array([0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 3.5, 6.5, 7.5, -8.5, 100.0, -100.0], dtype=F32)
    assert Q.round_clamp(u, 0, -8, 7).tolist() == [0, 2, 2, 0, -2, -2, 4, 6, 7, -8, 7, -8]
    assert Q.round_clamp(u, 8, 0, 15).tolist() == [8, 10, 10, 8, 6, 6, 12, 14, 15, 0, 15, 0]
    assert Q.round_clamp(np.array([np.nan], dtype=F32), 0, -8, 7).tolist() == [-8]


@pytest.mark.parametrize("sym,z", [(True, 0), (False, 8), (False, 3)])
def test_idempotence_every_code(sym, z):
    for scale in (0.0371, 1.0, 2.0 ** -5, 13.7):
        qp = QParams(4, sym, scale, z)
        codes = np.arange(qp.qmin, qp.qmax + 1)
        xhat = Q.dequantize(codes, scale, qp.z).astype(F32)[None, :]
        got, _, _, _ = Q.act_quant(xhat, qp, rmsnorm=False)
        assert got[0].tolist() == codes.tolist()


def test_error_bound_clamp_and_monotone():
    rng = np.random.default_rng(2)
    qp = QParams(4, True, 0.173)
    x = np.sort((rng.standard_normal(4096) * 0.6).astype(F32))[None, :]
    codes, _, _, _ = Q.act_quant(x, qp, rmsnorm=False)
    c = codes[0].astype(np.int64)
    assert c.min() >= -8 and c.max() <= 7
    assert np.all(np.diff(c) >= 0)                                  # monotone
    xh = Q.dequantize(c, qp.scale)
    inside = (x[0] >= (qp.qmin - 0.5) * qp.scale) & (x[0] <= (qp.qmax + 0.5) * qp.scale)
    assert inside.sum() > 3000
    assert np.all(np.abs(x[0][inside] - xh[inside]) <= qp.scale / 2 * (1 + 1e-6))
    assert np.all(c[x[0] > 7.5 * qp.scale * 1.001] == 7)
    assert np.all(c[x[0] < -8.5 * qp.scale * 1.001] == -8)


# ----------------------------- per-token scale ----------------------------- #
def test_rms_closed_forms():
    x = np.zeros((3, 4), dtype=F32)
    x[0] = [3, 4, 0, 0]            # mean square 25/4 -> rms 2.5
    x[1] = [-2, -2, -2, -2]        # rms 2
    x[2] = [0.5, -0.5, 0.5, -0.5]  # rms 0.5
    r = Q.rms_reciprocal(x, 0.0)
    assert r.tolist() == [F32(0.4), 0.5, 2.0]
    # eps enters under the root: x = 0 gives 1/sqrt(eps)
    r0 = Q.rms_reciprocal(np.zeros((1, 8), dtype=F32), 1e-6)
    assert abs(float(r0[0]) - 1000.0) < 1e-3


def test_rms_against_float64_formula():
    rng = np.random.default_rng(3)
    x = bf16.round_to_bf16((rng.standard_normal((64, 4096)) * 3).astype(F32))
    r = Q.rms_reciprocal(x, 1e-5).astype(np.float64)
    ref = 1.0 / np.sqrt(np.mean(x.astype(np.float64) ** 2, axis=1) + 1e-5)
    assert np.max(np.abs(r / ref - 1.0)) < 3 * 2.0 ** -24


def test_scale_recursion_and_sites():
    rng = np.random.default_rng(4)
    x = bf16.round_to_bf16(rng.standard_normal((16, 256)).astype(F32) * 5)
    s_in = np.exp(rng.standard_normal(16)).astype(F32)
    qp = QParams(4, True, 0.25)
    r = Q.rms_reciprocal(x, 1e-5)
    # block input: grid sees RMSNorm(x) whatever S_{n-1} is; S_n = S_{n-1} * r   (Eq. 7)
    c1, s1, p1, r1 = Q.act_quant(x, qp, True, False, 1e-5, s_in)
    c0, s0, _, _ = Q.act_quant(x, qp, True, False, 1e-5, None)
    assert np.array_equal(c1, c0) and np.array_equal(p1, r) and np.array_equal(s0, r)
    assert np.array_equal(s1, (r * s_in).astype(F32))
    # inner site: grid sees S_n * x and nothing is normalised
    c2, s2, p2, _ = Q.act_quant(x, qp, False, True, 0.0, s_in)
    assert np.array_equal(p2, s_in) and np.array_equal(s2, s_in)
    expect = np.clip(np.rint((x * s_in[:, None]).astype(F32) * F32(4.0)), -8, 7)
    assert np.array_equal(c2, expect.astype(np.int8))


def test_power_of_two_equivariance_under_rmsnorm():
    rng = np.random.default_rng(5)
    x = bf16.round_to_bf16(rng.standard_normal((32, 512)).astype(F32))
    qp = QParams(4, True, 0.31)
    base, _, _, _ = Q.act_quant(x, qp, True, False, 0.0)
    for j in (-7, 3, 11):
        c, _, _, _ = Q.act_quant((x * F32(2.0 ** j)).astype(F32), qp, True, False, 0.0)
        assert np.array_equal(c, base)


def test_act_quant_matches_scalar_brute_force():
    """Same recipe with Python scalars through struct-rounded float32 (no numpy ufuncs)."""
    import struct

    def f(v):
        return struct.unpack("f", struct.pack("f", v))[0]

    rng = np.random.default_rng(6)
    x = bf16.round_to_bf16(rng.standard_normal((5, 64)).astype(F32) * 2)
    s_in = np.exp(rng.standard_normal(5)).astype(F32)
    qp = QParams(4, False, 0.21, 7)
    codes, s_out, _, _ = Q.act_quant(x, qp, True, True, 1e-5, s_in)
    inv = f(1.0 / f(0.21))
    for t in range(5):
        ss = f(math.fsum(float(v) * float(v) for v in x[t]))
        rho = f(math.sqrt(f(f(ss / 64.0) + f(1e-5))))
        r = f(1.0 / rho)
        p = f(r * float(s_in[t]))
        assert f(s_out[t]) == p
        for k in range(64):
            u = f(f(float(x[t, k]) * p) * inv)
            q = min(max(round(u) + 7, 0), 15)       # Python round(): ties to even
            assert q == int(codes[t, k])


# ----------------------------- weights ------------------------------------- #
def test_weight_minmax_closed_form():
    w = np.array([[0.7, -0.1, 0.35, 0.0], [-1.4, 0.2, 0.2, 0.1], [0, 0, 0, 0]], dtype=F32)
    codes, d, wsum = Q.quantize_weights(w)
    assert d[0] == F32(F32(0.7) / F32(7)) and d[1] == F32(F32(1.4) / F32(7)) and d[2] == 1.0
    assert codes.tolist() == [[7, -1, 4, 0], [-7, 1, 1, 0], [0, 0, 0, 0]]   # 3.5 -> 4 (even)
    assert wsum.tolist() == [10, -5, 0]


def test_weight_scale_storage_dtype_is_used_for_codes():
    rng = np.random.default_rng(7)
    w = bf16.round_to_bf16((rng.standard_normal((32, 256)) * 0.02).astype(F32))
    c32, d32, _ = Q.quantize_weights(w, scale_dtype="fp32")
    c16, d16, _ = Q.quantize_weights(w, scale_dtype="fp16")
    assert np.array_equal(d16, d16.astype(np.float16).astype(F32))
    assert np.array_equal(c16, np.clip(np.rint(w / d16[:, None]), -8, 7).astype(np.int8))
    assert not np.array_equal(d16, d32)


def test_weight_lp_range_bruteforce_and_properties():
    rng = np.random.default_rng(8)
    w = (rng.standard_t(3, size=(6, 128)) * 0.02).astype(F32)
    codes, d, _ = Q.quantize_weights(w, range_mode=Q.RANGE_LP, p=3.0)
    _, dmm, _ = Q.quantize_weights(w)
    for n in range(6):
        a = float(np.max(np.abs(w[n])))
        best, best_i = None, None
        for i in range(20, 101):
            di = float(F32(F32(F32(a) * F32(F32(i) / F32(100))) / F32(7)))
            q = np.clip(np.rint(w[n] / F32(di)), -8, 7)
            err = sum(abs(float(w[n, k]) - di * float(q[k])) ** 3 for k in range(128))
            if best is None or err <= best:
                best, best_i, best_d = err, i, di
        assert float(d[n]) == best_d
        e_lp = np.sum(np.abs(w[n] - d[n] * codes[n]) ** 3)
        qmm = np.clip(np.rint(w[n] / dmm[n]), -8, 7)
        assert e_lp <= np.sum(np.abs(w[n] - dmm[n] * qmm) ** 3) + 1e-18
    assert np.any(d < dmm)              # heavy tails: clipping pays under L_3
    # a row that already lies on a grid keeps the full range (zero error, ties -> larger)
    grid = (np.arange(-7, 8).repeat(4)[None, :] * F32(0.125)).astype(F32)
    cg, dg, _ = Q.quantize_weights(grid, range_mode=Q.RANGE_LP)
    assert dg[0] == 0.125 and np.array_equal(cg[0], np.arange(-7, 8).repeat(4))


# ----------------------------- SiLU ---------------------------------------- #
def test_exp2_spec_exact_at_integers_and_accurate():
    n = np.arange(-126, 127).astype(F32)
    assert np.array_equal(Q.exp2_spec(n), np.exp2(n.astype(np.float64)).astype(F32))
    t = np.linspace(-60, 60, 200001).astype(F32)
    rel = np.abs(Q.exp2_spec(t).astype(np.float64) / np.exp2(t.astype(np.float64)) - 1.0)
    assert rel.max() < 4 * 2.0 ** -23


def test_silu_against_float64_on_all_bf16_values():
    bits = np.arange(65536, dtype=np.uint16)
    g = bf16.bf16_bits_to_f32(bits)
    g = g[np.isfinite(g) & (np.abs(g) < 80)]
    s = Q.silu_spec(g).astype(np.float64)
    g64 = g.astype(np.float64)
    ref = g64 / (1.0 + np.exp(-g64))
    nz = np.abs(ref) > 1e-30
    rel = np.abs(s[nz] / ref[nz] - 1.0)
    # the float32 product g*log2(e) carries half an ulp of |g|*1.44 into the exponent,
    # so the relative error grows with |g| for negative g (where silu is tiny anyway)
    assert np.max(rel[np.abs(g[nz]) <= 8]) < 6 * 2.0 ** -23
    assert np.max(rel) < 1e-5
    assert np.max(np.abs(s - ref)) < 2.0 ** -22 * np.max(np.abs(ref))
    assert Q.silu_spec(np.array([0.0], dtype=F32))[0] == 0.0
    assert Q.silu_spec(np.array([40.0], dtype=F32))[0] == 40.0
    assert abs(Q.silu_spec(np.array([-40.0], dtype=F32))[0]) < 1e-15


def test_silu_mul_quant_composition():
    rng = np.random.default_rng(9)
    g = bf16.round_to_bf16(rng.standard_normal((8, 64)).astype(F32) * 3)
    u = bf16.round_to_bf16(rng.standard_normal((8, 64)).astype(F32) * 3)
    s = np.exp(rng.standard_normal(8)).astype(F32)
    qp = QParams(4, True, 0.4)
    codes, m = Q.silu_mul_quant(g, u, qp, s)
    assert np.array_equal(m, bf16.round_to_bf16(m))                  # product is held in bf16
    g64, u64 = g.astype(np.float64), u.astype(np.float64)
    ref = g64 / (1 + np.exp(-g64)) * u64
    assert np.max(np.abs(m - ref) <= np.abs(ref) * 2.0 ** -8 + 1e-30)
    val = ref * s[:, None] / 0.4
    far = np.abs(val - np.floor(val) - 0.5) > 0.02                    # away from rounding edges
    assert np.array_equal(codes[far], np.clip(np.rint(val), -8, 7).astype(np.int8)[far])


# ----------------------------- calibration --------------------------------- #
def test_calibration_recovers_an_exact_grid_and_clips_tails():
    qp = QParams(4, True, 1.0)
    v = np.arange(-7, 8).repeat(10) * 0.5
    assert Q.calibrate_static_scale(v, qp) == F32(0.5)
    rng = np.random.default_rng(10)
    t = rng.standard_t(3, size=20000)
    d = float(Q.calibrate_static_scale(t, qp))
    assert d < np.max(np.abs(t)) / 8          # L_3 clips far inside the min-max range
    # brute force over the same candidate list with plain loops on a small sample
    small = t[:300]
    amax = np.max(np.abs(small))
    errs = []
    for i in range(1, 101):
        di = float(F32(amax * i / 700.0))
        e = 0.0
        for x in small:
            q = min(max(round(x / di), -8), 7)
            e += abs(x - di * q) ** 3
        errs.append((e, di))
    best = min(errs, key=lambda p: (p[0], -p[1]))[1]
    assert float(Q.calibrate_static_scale(small, qp)) == pytest.approx(best, rel=1e-6)


# --------------------------------------------------------------------------- #
# dynamic (per-token) quantiser, 4 and 8 bits
# --------------------------------------------------------------------------- #
@pytest.mark.parametrize("bits", [4, 8])
def test_dynamic_quantiser_grid_ends_at_the_token_maximum(bits):
    rng = np.random.default_rng(31)
    M, K = 64, 256
    x = bf16.round_to_bf16((rng.standard_normal((M, K)) * np.exp(rng.standard_normal((M, 1)) * 2)).astype(F32))
    s_in = np.exp(rng.standard_normal(M)).astype(F32)
    qmax = 2 ** (bits - 1) - 1
    for rmsnorm, scale_input in ((True, False), (False, True), (True, True), (False, False)):
        codes, delta, s_out, p, r = Q.act_quant_dynamic(x, bits, rmsnorm, scale_input, 1e-5, s_in)
        # the scale is the token's largest magnitude over qmax (float64 restatement, float32 tolerance)
        m64 = np.max(np.abs(x.astype(np.float64)), axis=1) * p.astype(np.float64)
        assert np.allclose(delta, m64 / qmax, rtol=3e-7)
        # so the largest element sits on the last code, nothing is clipped, and the error is half a step
        assert np.array_equal(np.max(np.abs(codes.astype(np.int32)), axis=1), np.full(M, qmax))
        v = x.astype(np.float64) * p.astype(np.float64)[:, None]
        err = np.abs(v - delta.astype(np.float64)[:, None] * codes)
        assert np.all(err <= 0.5 * delta.astype(np.float64)[:, None] * (1 + 1e-5))
        # per row it is the static quantiser with that row's scale
        for t in (0, 17, M - 1):
            ref, _, _, _ = Q.act_quant(x[t:t + 1], QParams(bits, True, float(delta[t])), rmsnorm, scale_input, 1e-5,
                                       s_in[t:t + 1])
            assert np.array_equal(ref[0], codes[t])
        # bookkeeping identical to the static quantiser
        _, s_ref, p_ref, r_ref = Q.act_quant(x, QParams(4, True, 1.0), rmsnorm, scale_input, 1e-5, s_in)
        assert np.array_equal(s_out, s_ref) and np.array_equal(p, p_ref) and np.array_equal(r, r_ref)


@pytest.mark.parametrize("bits", [4, 8])
def test_dynamic_quantiser_equivariance_and_degenerate_rows(bits):
    rng = np.random.default_rng(32)
    x = bf16.round_to_bf16(rng.standard_normal((8, 128)).astype(F32))
    c0, d0, _, _, _ = Q.act_quant_dynamic(x, bits, rmsnorm=False)
    c1, d1, _, _, _ = Q.act_quant_dynamic(x * F32(8.0), bits, rmsnorm=False)
    assert np.array_equal(c0, c1) and np.array_equal(d1, d0 * F32(8.0))      # powers of two move into the scale
    c2, d2, _, _, _ = Q.act_quant_dynamic(-x, bits, rmsnorm=False)
    assert np.array_equal(d2, d0)                                            # the grid depends on magnitudes only
    qmax = 2 ** (bits - 1) - 1
    assert np.array_equal(np.clip(-c0.astype(np.int32), -qmax - 1, qmax), c2.astype(np.int32))
    # with the RMSNorm in front, a per-token factor on the input changes nothing at all (eps = 0)
    f = np.exp2(rng.integers(-3, 4, 8)).astype(F32)
    c3, d3, _, _, _ = Q.act_quant_dynamic(x, bits, rmsnorm=True, eps=0.0)
    c4, d4, _, _, _ = Q.act_quant_dynamic(x * f[:, None], bits, rmsnorm=True, eps=0.0)
    assert np.array_equal(c3, c4) and np.array_equal(d3, d4)
    # an outlier token gets a wider grid than its neighbours, the others keep theirs
    y = x.copy()
    y[3, 5] = F32(1000.0)
    c5, d5, _, _, _ = Q.act_quant_dynamic(y, bits, rmsnorm=False)
    assert d5[3] == F32(1000.0) / F32(qmax) and np.array_equal(np.delete(d5, 3), np.delete(d0, 3))
    assert np.array_equal(np.delete(c5, 3, axis=0), np.delete(c0, 3, axis=0))
    # degenerate rows: all zero -> scale 1, codes 0; Inf or NaN in the row -> scale 1, saturated / lowest code
    z = np.zeros((3, 128), dtype=F32)
    z[1, 0], z[1, 1], z[1, 2] = np.inf, -np.inf, 3.0
    z[2, 0], z[2, 1] = np.nan, -2.0
    c6, d6, _, _, _ = Q.act_quant_dynamic(z, bits, rmsnorm=False)
    assert np.array_equal(d6, np.ones(3, dtype=F32)) and not c6[0].any()
    assert c6[1, 0] == qmax and c6[1, 1] == -qmax - 1 and c6[1, 2] == 3
    assert c6[2, 0] == -qmax - 1 and c6[2, 1] == -2


# --------------------------------------------------------------------------- #
# 8-bit activation grid (the W4A8 setting)
# --------------------------------------------------------------------------- #
def test_eight_bit_grid_idempotence_ties_clamp_and_scalar_brute_force():
    import struct

    def f(v):
        return struct.unpack("f", struct.pack("f", v))[0]

    for scale in (0.0371, 1.0, 2.0 ** -5):
        qp = QParams(8, True, scale)
        assert (qp.qmin, qp.qmax) == (-128, 127)
        codes = np.arange(-128, 128)
        got, _, _, _ = Q.act_quant(Q.dequantize(codes, scale).astype(F32)[None, :], qp, rmsnorm=False)
        assert got.dtype == np.int8 and got[0].tolist() == codes.tolist()
    u = np.array([0.5, 1.5, 126.5, 127.5, -127.5, -128.5, 1e9, -1e9, np.nan], dtype=F32)
    assert Q.round_clamp(u, 0, -128, 127).tolist() == [0, 2, 126, 127, -128, -128, 127, -128, -128]
    rng = np.random.default_rng(41)
    x = bf16.round_to_bf16(rng.standard_normal((4, 64)).astype(F32) * 3)
    s_in = np.exp(rng.standard_normal(4)).astype(F32)
    qp = QParams(8, True, 0.013)
    codes, s_out, _, _ = Q.act_quant(x, qp, True, True, 1e-5, s_in)
    inv = f(1.0 / f(0.013))
    for t in range(4):
        ss = f(math.fsum(float(v) * float(v) for v in x[t]))
        p = f(f(1.0 / f(math.sqrt(f(f(ss / 64.0) + f(1e-5))))) * float(s_in[t]))
        for k in range(64):
            q = min(max(round(f(f(float(x[t, k]) * p) * inv)), -128), 127)
            assert q == int(codes[t, k])
    assert np.abs(codes.astype(np.int32)).max() > 64          # the wide grid is used
