"""Pins for the integer matmul, the scale-factor epilogue and the composed linear."""
import numpy as np
import pytest

from oracle import bf16, quantizers as Q
from oracle.quantizers import QParams
from oracle.int_matmul import int_matmul, int_matmul_bruteforce
from oracle.epilogue import dequant_epilogue, inverse_of_pre
from oracle import linear as L
from oracle import transforms as T

F32 = np.float32


@pytest.mark.parametrize("M,N,K", [(1, 1, 128), (3, 5, 128), (8, 8, 256), (2, 7, 64)])
@pytest.mark.parametrize("z", [0, 8])
def test_int_matmul_equals_bruteforce(M, N, K, z):
    rng = np.random.default_rng(M * 100 + N * 10 + K + z)
    lo, hi = (-8, 8) if z == 0 else (0, 16)
    qa = rng.integers(lo, hi, (M, K))
    qw = rng.integers(-8, 8, (N, K))
    assert np.array_equal(int_matmul(qa, qw, z).astype(np.int64), int_matmul_bruteforce(qa, qw, z))


def test_int_matmul_extreme_codes():
    K = 256
    qa = np.array([[-8] * K, [7] * K, [-8] * K])
    qw = np.array([[-8] * K, [7] * K])
    got = int_matmul(qa, qw)
    assert got.tolist() == [[64 * K, -56 * K], [-56 * K, 49 * K], [64 * K, -56 * K]]
    assert got.dtype == np.int32
    # the weight operand is indexed [n, k] (a transposed operand would change the shape)
    assert int_matmul(np.ones((2, 128), int), np.ones((5, 128), int)).shape == (2, 5)
    # asymmetric zero point is subtracted from the activation codes only
    a = np.full((1, 128), 15)
    w = np.full((1, 128), -8)
    assert int_matmul(a, w, 8)[0, 0] == (15 - 8) * (-8) * 128


def test_epilogue_on_grid_reduces_to_float64_matmul():
    """Power-of-two scales and on-grid inputs: the whole W4A4 linear must equal X W^T."""
    rng = np.random.default_rng(11)
    M, N, K = 24, 40, 256
    qa = rng.integers(-8, 8, (M, K))
    qw = rng.integers(-7, 8, (N, K))
    qw[:, 0] = 7                                      # every row reaches max code: D_w = exact
    da = 2.0 ** -3
    dw = (2.0 ** -rng.integers(2, 6, N)).astype(F32)
    X = (qa * da).astype(F32)
    W = (qw * dw[:, None]).astype(F32)
    cw, sw, _ = Q.quantize_weights(W)
    assert np.array_equal(cw, qw)
    # 7*dw/7 may round; rebuild the exact scale for the equality below
    out = L.w4a4_linear(X, cw, dw, QParams(4, True, da), rmsnorm=False)
    assert np.array_equal(out["codes"], qa)
    ref = X.astype(np.float64) @ W.astype(np.float64).T
    assert np.array_equal(out["y"], bf16.round_to_bf16(ref.astype(F32)))
    assert np.array_equal(out["acc"], (ref / (da * dw[None, :].astype(np.float64))).astype(np.int64))


def test_epilogue_scale_order_and_post_modes():
    acc = np.array([[1000, -3, 0], [7, 123456, -99999]], dtype=np.int32)
    sw = np.array([0.013, 0.5, 1.7], dtype=F32)
    da = F32(0.37)
    post = np.array([2.5, 0.3], dtype=F32)
    y = dequant_epilogue(acc, sw, da, post).astype(np.float64)
    ref = acc.astype(np.float64) * sw[None, :].astype(np.float64) * float(da) * post[:, None].astype(np.float64)
    # three float32 roundings and one bfloat16 rounding
    assert np.all(np.abs(y - ref) <= np.abs(ref) * (2.0 ** -8 + 4 * 2.0 ** -24))
    y0 = dequant_epilogue(acc, sw, da, None).astype(np.float64)
    ref0 = acc.astype(np.float64) * sw[None, :] * float(da)
    assert np.all(np.abs(y0 - ref0) <= np.abs(ref0) * (2.0 ** -8 + 3 * 2.0 ** -24))
    # residual joins before the single final rounding
    res = np.array([[1.0, 2.0, -3.0], [0.5, 0.25, 8.0]], dtype=F32)
    y1 = dequant_epilogue(acc, sw, da, None, res).astype(np.float64)
    assert np.all(np.abs(y1 - (ref0 + res)) <= np.abs(ref0 + res) * 2.0 ** -8 + np.abs(ref0) * 2.0 ** -22)
    assert inverse_of_pre(np.array([4.0, 0.5], dtype=F32)).tolist() == [0.25, 2.0]


def test_inverse_of_pre_gives_plain_linear_semantics():
    """With post = 1/p the output approximates X W^T itself, whatever the token norms."""
    rng = np.random.default_rng(12)
    M, N, K = 64, 96, 512
    x = bf16.round_to_bf16(rng.standard_normal((M, K)).astype(F32) * np.exp(rng.standard_normal((M, 1))).astype(F32))
    w = bf16.round_to_bf16((rng.standard_normal((N, K)) * 0.02).astype(F32))
    cw, sw, _ = Q.quantize_weights(w)
    r = Q.rms_reciprocal(x, 1e-5)
    da = Q.calibrate_static_scale(x * r[:, None], QParams())
    out = L.w4a4_linear(x, cw, sw, QParams(4, True, float(da)), rmsnorm=True, post_mode=L.POST_INVERSE_OF_PRE)
    ref = x.astype(np.float64) @ w.astype(np.float64).T
    rel = np.linalg.norm(out["y"] - ref) / np.linalg.norm(ref)
    assert rel < 0.25                                     # 4-bit x 4-bit: coarse but unbiased
    # and a loose element-wise bound from the two half-step errors (unclipped inputs only)
    xn = x * r[:, None]
    unclipped = np.all(np.abs(xn) <= 7.5 * float(da), axis=1)
    bound = (float(da) / 2 * np.abs(w).sum(axis=1)[None, :] + (sw / 2)[None, :] * np.abs(xn).sum(axis=1)[:, None]
             + float(da) / 2 * (sw / 2)[None, :] * K) / r[:, None]
    err = np.abs(out["y"] - ref)
    assert np.all(err[unclipped] <= bound[unclipped] * 1.02 + 1e-6)
    # without the post factor the output is the normalised-domain result
    out2 = L.w4a4_linear(x, cw, sw, QParams(4, True, float(da)), rmsnorm=True)
    refn = (x * r[:, None]).astype(np.float64) @ w.astype(np.float64).T
    assert np.linalg.norm(out2["y"] - refn) / np.linalg.norm(refn) < 0.25
    assert np.array_equal(out2["codes"], out["codes"]) and np.array_equal(out2["acc"], out["acc"])


def test_decoder_mlp_tracks_float64_block_and_scale_bookkeeping():
    rng = np.random.default_rng(13)
    M, d, dff = 48, 256, 512
    x = bf16.round_to_bf16(rng.standard_normal((M, d)).astype(F32) * 3)
    s_prev = np.exp(rng.standard_normal(M) * 0.5).astype(F32)
    wg, wu = (bf16.round_to_bf16((rng.standard_normal((dff, d)) * 0.06).astype(F32)) for _ in range(2))
    wd = bf16.round_to_bf16((rng.standard_normal((d, dff)) * 0.04).astype(F32))
    (cg, sg, _), (cu, su, _), (cd, sd, _) = (Q.quantize_weights(w) for w in (wg, wu, wd))
    r = Q.rms_reciprocal(x, 1e-5)
    xn = (x * r[:, None]).astype(np.float64)
    g = xn @ wg.astype(np.float64).T
    u = xn @ wu.astype(np.float64).T
    h = g / (1 + np.exp(-g)) * u
    s_n = (s_prev * r).astype(np.float64)
    qp_in = QParams(4, True, float(Q.calibrate_static_scale(xn, QParams())))
    qp_mid = QParams(4, True, float(Q.calibrate_static_scale(h * s_n[:, None], QParams())))
    out = L.decoder_mlp(x, cg, sg, cu, su, cd, sd, qp_in, qp_mid, 1e-5, s_prev, add_residual=True)
    assert np.array_equal(out["s_out"], (r * s_prev).astype(F32))           # Eq. 7
    y_ref = (h * s_n[:, None]) @ wd.astype(np.float64).T                    # S_n * Y_n  (Eq. 5)
    z_ref = xn + y_ref                                                     # Z~_n = X~_n + Y~_n
    assert np.linalg.norm(out["y"] - z_ref) / np.linalg.norm(z_ref) < 0.2
    out_nr = L.decoder_mlp(x, cg, sg, cu, su, cd, sd, qp_in, qp_mid, 1e-5, s_prev, add_residual=False)
    assert np.linalg.norm(out_nr["y"] - y_ref) / np.linalg.norm(y_ref) < 0.45
    # exact integer accumulators whichever way they are computed
    assert np.array_equal(out["acc_d"][:2, :3].astype(np.int64), int_matmul_bruteforce(out["mq"][:2], cd[:3]))


def _attention_core_f64(q, k, v, d_head, m, thetas):
    """softmax(rope(q) rope(k)^T / sqrt(d)) v per head, causal, grouped-query; float64."""
    Lq = q.shape[0]
    pos = np.arange(Lq)
    mask = np.triu(np.ones((Lq, Lq), dtype=bool), k=1)
    heads = []
    for j in range(q.shape[1] // d_head):
        h = j // m
        qj = T.apply_rope(q[:, j * d_head:(j + 1) * d_head], pos, thetas, "half")
        kh = T.apply_rope(k[:, h * d_head:(h + 1) * d_head], pos, thetas, "half")
        lg = np.where(mask, -np.inf, qj @ kh.T / np.sqrt(d_head))
        a = np.exp(lg - lg.max(axis=-1, keepdims=True))
        heads.append((a / a.sum(axis=-1, keepdims=True)) @ v[:, h * d_head:(h + 1) * d_head])
    return np.concatenate(heads, axis=1)


def test_decoder_attention_projections_track_float64_block_and_scale_bookkeeping():
    """The two halves of the attention block around a float64 attention core: S_n bookkeeping exact
    (Eq. 7), Z~_n = X~_n + S_n * Y_n (Eq. 5) within what two 4-bit grids allow, the scaler at the
    attention output commutes with the output projection, integer accumulators by brute force."""
    rng = np.random.default_rng(21)
    M, d, d_head, n_kv, m = 40, 256, 32, 2, 4
    n_q = n_kv * m
    x = bf16.round_to_bf16(rng.standard_normal((M, d)).astype(F32) * np.exp(rng.standard_normal((M, 1))).astype(F32))
    s_prev = np.exp(rng.standard_normal(M) * 0.5).astype(F32)
    wq, wk, wv = (bf16.round_to_bf16((rng.standard_normal((n, d)) * 0.06).astype(F32))
                  for n in (n_q * d_head, n_kv * d_head, n_kv * d_head))
    wo = bf16.round_to_bf16((rng.standard_normal((d, n_q * d_head)) * 0.06).astype(F32))
    wqkv = np.concatenate([wq, wk, wv], axis=0)
    cqkv, sqkv, _ = Q.quantize_weights(wqkv)
    co, so, _ = Q.quantize_weights(wo)
    r = Q.rms_reciprocal(x, 1e-5)
    xn = (x * r[:, None]).astype(np.float64)
    qp_in = QParams(4, True, float(Q.calibrate_static_scale(xn, QParams())))
    first = L.decoder_attn_qkv(x, cqkv, sqkv, qp_in, 1e-5, s_prev)
    assert np.array_equal(first["s_out"], (r * s_prev).astype(F32))          # Eq. 7
    assert np.array_equal(first["r"], r)
    qkv_ref = xn @ wqkv.astype(np.float64).T
    assert np.linalg.norm(first["qkv"] - qkv_ref) / np.linalg.norm(qkv_ref) < 0.25
    assert np.array_equal(first["acc"][:2, :3].astype(np.int64), int_matmul_bruteforce(first["xq"][:2], cqkv[:3]))
    # QKV carries no per-token scale: another S_{n-1} changes S_n only
    again = L.decoder_attn_qkv(x, cqkv, sqkv, qp_in, 1e-5, None)
    assert np.array_equal(again["qkv"], first["qkv"]) and np.array_equal(again["s_out"], r)
    # the caller's attention (float64 here) on the reference projections
    thetas = 10000.0 ** (-np.arange(d_head // 2) / (d_head // 2))
    nq, nk = n_q * d_head, n_kv * d_head
    a_ref = _attention_core_f64(qkv_ref[:, :nq], qkv_ref[:, nq:nq + nk], qkv_ref[:, nq + nk:], d_head, m, thetas)
    a = bf16.round_to_bf16(a_ref.astype(F32))
    s_n = first["s_out"]
    qp_ap = QParams(4, True, float(Q.calibrate_static_scale(a_ref * s_n[:, None].astype(np.float64), QParams())))
    second = L.decoder_attn_out(a, co, so, qp_ap, s_n, x, r)
    y_ref = (a_ref * s_n[:, None].astype(np.float64)) @ wo.astype(np.float64).T     # S_n * Y_n  (Eq. 5)
    z_ref = xn + y_ref                                                               # Z~_n = X~_n + Y~_n
    err = np.linalg.norm(second["y"] - z_ref) / np.linalg.norm(z_ref)
    assert err < 0.35
    # ... and nowhere near the block with the scaler left out, or the residual left unnormalised
    assert np.linalg.norm(second["y"] - (xn + a_ref @ wo.astype(np.float64).T)) / np.linalg.norm(z_ref) > 2 * err
    assert np.linalg.norm(second["y"] - (x.astype(np.float64) + y_ref)) / np.linalg.norm(z_ref) > 2 * err
    no_res = L.decoder_attn_out(a, co, so, qp_ap, s_n)
    assert np.linalg.norm(no_res["y"] - y_ref) / np.linalg.norm(y_ref) < 0.45
    assert np.array_equal(second["acc"], no_res["acc"])
    assert np.array_equal(second["acc"][:2, :3].astype(np.int64), int_matmul_bruteforce(second["aq"][:2], co[:3]))
    # the scaler commutes with the projection: powers of two move through the grid exactly
    two = np.full(M, 4.0, dtype=F32)
    scaled = L.decoder_attn_out(a, co, so, QParams(4, True, qp_ap.scale * 4.0), s_n * two)
    assert np.array_equal(scaled["aq"], second["aq"])
    assert np.array_equal(scaled["y"], (no_res["y"] * 4.0).astype(F32))
    # and it matters where the scale is: without S_n the same grid clips differently
    unscaled = L.decoder_attn_out(a, co, so, qp_ap, np.ones(M, dtype=F32))
    assert not np.array_equal(unscaled["aq"], second["aq"])


@pytest.mark.parametrize("bits", [4, 8])
def test_dynamic_linear_on_grid_inputs_reduce_to_a_float64_matmul(bits):
    """Rows that lie on their own dynamic grid (x = c_t * q, |q| reaching qmax, c_t a power of two)
    are quantised without error, so the whole dynamic linear equals the float64 product."""
    rng = np.random.default_rng(33)
    M, K, N = 24, 256, 40
    qmax = 2 ** (bits - 1) - 1
    qa = rng.integers(-qmax, qmax + 1, (M, K))
    qa[np.arange(M), rng.integers(0, K, M)] = qmax * rng.choice([-1, 1], M)
    c = np.exp2(rng.integers(-6, 3, M))
    x = (qa * c[:, None]).astype(F32)
    qw = rng.integers(-8, 8, (N, K)).astype(np.int8)
    sw = np.exp2(rng.integers(-8, -3, N)).astype(F32)
    out = L.w4a4_linear_dynamic(x, qw, sw, bits, rmsnorm=False)
    assert np.array_equal(out["codes"], qa) and np.array_equal(out["delta"], c.astype(F32))
    ref = x.astype(np.float64) @ (qw * sw[:, None].astype(np.float64)).T
    assert np.array_equal(out["y"], bf16.round_to_bf16(ref.astype(F32)))
    assert np.array_equal(out["acc"][:2, :3].astype(np.int64), int_matmul_bruteforce(qa[:2], qw[:3]))


def test_dynamic_linear_post_modes_and_gain_over_static_on_outlier_tokens():
    rng = np.random.default_rng(34)
    M, K, N = 64, 512, 48
    x = bf16.round_to_bf16((rng.standard_normal((M, K)) * np.exp(rng.standard_normal((M, 1)) * 1.5)).astype(F32))
    w = bf16.round_to_bf16((rng.standard_normal((N, K)) * 0.05).astype(F32))
    cw, sw, _ = Q.quantize_weights(w)
    ref = x.astype(np.float64) @ w.astype(np.float64).T
    dyn = L.w4a4_linear_dynamic(x, cw, sw, 4, rmsnorm=False)
    e_dyn = np.linalg.norm(dyn["y"] - ref) / np.linalg.norm(ref)
    d_static = float(Q.calibrate_static_scale(x.astype(np.float64), QParams()))
    sta = L.w4a4_linear(x, cw, sw, QParams(4, True, d_static), rmsnorm=False)
    e_sta = np.linalg.norm(sta["y"] - ref) / np.linalg.norm(ref)
    assert e_dyn < 0.3 and e_dyn < 0.7 * e_sta             # per-token grids absorb the norm disparity (App. B)
    y8 = L.w4a4_linear_dynamic(x, cw, sw, 8, rmsnorm=False)["y"]
    assert np.linalg.norm(y8 - ref) / np.linalg.norm(ref) < e_dyn
    ref_wq = x.astype(np.float64) @ (cw.astype(np.float64) * sw[:, None].astype(np.float64)).T
    assert np.linalg.norm(y8 - ref_wq) / np.linalg.norm(ref_wq) < 0.02    # 8-bit activations: only the weight grid's error remains
    # post modes: with the RMSNorm in front, INVERSE_OF_PRE undoes the normalisation, VECTOR applies any vector
    r = Q.rms_reciprocal(x, 1e-5)
    inv = L.w4a4_linear_dynamic(x, cw, sw, 4, rmsnorm=True, post_mode=L.POST_INVERSE_OF_PRE)
    assert np.linalg.norm(inv["y"] - ref) / np.linalg.norm(ref) < 0.3
    vec = L.w4a4_linear_dynamic(x, cw, sw, 4, rmsnorm=True, post_mode=L.POST_VECTOR, post=np.full(M, 2.0, dtype=F32))
    non = L.w4a4_linear_dynamic(x, cw, sw, 4, rmsnorm=True)
    assert np.array_equal(vec["y"], (non["y"] * F32(2.0)).astype(F32))
    assert np.array_equal(non["codes"], inv["codes"]) and np.array_equal(non["s_out"], r)
