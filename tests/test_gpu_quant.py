"""GPU parity of the quantise kernels against the oracle: packed codes, scales and row
sums must match bit for bit."""
import numpy as np
import pytest
import torch

from oracle import quantizers as OQ
from paper_2506_04985_b200 import binding as B, synth
from helpers import dev, host, oqp, bf16_host

pytestmark = pytest.mark.gpu


def _acts(M, K, seed, law="student_t3"):
    return synth.activations(M, K, seed, f"x{M}x{K}", law=law, outlier_frac=0.005, outlier_gain=50.0,
                             token_log_std=0.7)


@pytest.mark.parametrize("M,K", [(128, 1024), (37, 4096), (5, 14336), (3, 28672), (130, 128), (2, 32), (9, 8192),
                                 (4, 2048), (1, 65536 - 32)])
@pytest.mark.parametrize("mode", ["norm", "norm_sin", "scale", "norm_scale", "asym"])
def test_act_quant_codes_bit_exact(M, K, mode):
    x = _acts(M, K, 3)
    s_in = synth.per_token_scale(M, 3, "s_in")
    flags = {"norm": B.RMSNORM, "norm_sin": B.RMSNORM, "scale": B.SCALE_INPUT,
             "norm_scale": B.RMSNORM | B.SCALE_INPUT, "asym": B.RMSNORM}[mode]
    use_s = mode in ("norm_sin", "scale", "norm_scale")
    qp = B.QParams(4, mode != "asym", 0.37 if flags & B.RMSNORM else 1.9, 7)
    xq, s_out = B.fpt_act_quant(dev(x), qp, flags, 1e-5, s_in=dev(s_in) if use_s else None)
    codes, so, _, _ = OQ.act_quant(synth.f32(x), oqp(qp), bool(flags & B.RMSNORM), bool(flags & B.SCALE_INPUT),
                                   1e-5, s_in.numpy() if use_s else None)
    assert np.array_equal(host(xq), OQ.pack_int4(codes))
    assert np.array_equal(host(s_out).view(np.uint32), so.view(np.uint32))
    assert len(np.unique(codes)) >= 8 or K < 64        # the grid is actually exercised


@pytest.mark.parametrize("M,K,ld", [(600, 1024, 1024), (1500, 4096, 4096), (777, 8192, 8200), (513, 16384, 16384)])
@pytest.mark.parametrize("mode", ["norm", "scale", "asym"])
def test_act_quant_many_tokens_streaming_kernel(M, K, ld, mode):
    """Enough tokens for the persistent double-buffered kernel: every warp walks over several rows,
    some rows carry Inf / NaN / zeros, rows may be strided."""
    x = torch.zeros((M, ld), dtype=torch.bfloat16)
    x[:, :K] = _acts(M, K, 8)
    x[:, K:] = -777.0
    x[3, :K] = 0.0
    x[M // 2, 11] = float("nan")
    x[M - 1, K - 1] = float("inf")
    s_in = synth.per_token_scale(M, 8, "s_in")
    flags = B.SCALE_INPUT if mode == "scale" else B.RMSNORM
    qp = B.QParams(4, mode != "asym", 0.37 if flags & B.RMSNORM else 1.9, 9)
    xq, s_out = B.fpt_act_quant(dev(x), qp, flags, 1e-5, s_in=dev(s_in), K=K)
    with np.errstate(all="ignore"):
        codes, so, _, _ = OQ.act_quant(synth.f32(x)[:, :K], oqp(qp), bool(flags & B.RMSNORM),
                                       bool(flags & B.SCALE_INPUT), 1e-5, s_in.numpy())
    assert np.array_equal(host(xq), OQ.pack_int4(codes))
    assert np.array_equal(host(s_out), so, equal_nan=True)


def test_act_quant_strided_rows_and_edge_values():
    M, K, ld = 6, 256, 384
    x = torch.zeros((M, ld), dtype=torch.bfloat16)
    x[:, :K] = _acts(M, K, 4)
    x[:, K:] = 1000.0                                # must be ignored
    x[1, :K] = 0.0                                   # zero row: r = 1/sqrt(eps)
    x[2, 5] = float("nan")
    x[3, 7] = float("inf")
    x[4, :K] = 3.0e38                                # squares overflow float32
    x[5, 9] = 3.0e38                                 # finite, but far beyond the exact range of the rounding trick
    x[5, 10] = -3.0e38
    qp = B.QParams(4, True, 0.41, 0)
    xq, s_out = B.fpt_act_quant(dev(x), qp, B.RMSNORM, 1e-6, K=K)
    with np.errstate(all="ignore"):
        codes, so, _, _ = OQ.act_quant(synth.f32(x)[:, :K], oqp(qp), True, False, 1e-6)
    assert np.array_equal(host(xq), OQ.pack_int4(codes))
    assert np.array_equal(host(s_out), so, equal_nan=True)           # NaN payloads may differ
    assert np.isnan(so[2]) and so[3] == 0.0 and so[4] == 0.0


@pytest.mark.parametrize("M,K", [(64, 1024), (7, 14336), (3, 256)])
@pytest.mark.parametrize("inter", [False, True])
def test_silu_mul_quant_bit_exact(M, K, inter):
    g = synth.activations(M, K, 5, "g", law="normal", outlier_frac=0.01, outlier_gain=6.0)
    u = synth.activations(M, K, 5, "u", law="student_t3", outlier_frac=0.0)
    g.view(-1)[:256] = torch.linspace(-90, 90, 256).to(torch.bfloat16)   # exp2 range reduction edges
    s_n = synth.per_token_scale(M, 5, "s_n")
    qp = B.QParams(4, True, 0.23, 0)
    if inter:
        gu = torch.empty((M, 2 * K), dtype=torch.bfloat16)
        gu.view(M, K // 64, 2, 64)[:, :, 0, :] = g.view(M, K // 64, 64)
        gu.view(M, K // 64, 2, 64)[:, :, 1, :] = u.view(M, K // 64, 64)
        xq, _ = B.fpt_act_quant(dev(gu), qp, B.SILU_MUL | B.GU_INTERLEAVED | B.SCALE_INPUT, 0.0, s_in=dev(s_n))
    else:
        xq, _ = B.fpt_act_quant(dev(g), qp, B.SILU_MUL | B.SCALE_INPUT, 0.0, X2=dev(u), s_in=dev(s_n))
    codes, _ = OQ.silu_mul_quant(synth.f32(g), synth.f32(u), oqp(qp), s_n.numpy())
    assert np.array_equal(host(xq), OQ.pack_int4(codes))


@pytest.mark.parametrize("N,K", [(64, 1024), (33, 4096), (8, 14336), (300, 128)])
@pytest.mark.parametrize("mode", ["minmax32", "minmax16", "lp32", "lp16_f32in"])
def test_weight_quant_bit_exact(N, K, mode):
    w = synth.weights(N, K, 0.02, 6, f"w{N}x{K}", outlier_row_frac=0.02, outlier_row_gain=20.0)
    if N > 2:
        w[2] = 0.0                                    # all-zero row: scale 1
    wf = synth.f32(w)
    sd = torch.float16 if "16" in mode else torch.float32
    rm = B.RANGE_LP if mode.startswith("lp") else B.RANGE_MINMAX
    wd = dev(w).float() if mode.endswith("f32in") else dev(w)
    wq, sw, wsum = B.fpt_quantize_weights(wd, None, rm, 3.0, sd)
    codes, d, ws = OQ.quantize_weights(wf, range_mode=OQ.RANGE_LP if rm else OQ.RANGE_MINMAX, p=3.0,
                                       scale_dtype="fp16" if sd == torch.float16 else "fp32")
    assert np.array_equal(host(sw.float()).view(np.uint32), d.view(np.uint32))
    assert np.array_equal(host(wq), OQ.pack_int4(codes))
    assert np.array_equal(host(wsum), ws)


def test_interleave_gate_up_layout():
    d_ff, K = 384, 256
    rng = np.random.default_rng(0)
    g = torch.from_numpy(rng.integers(0, 256, (d_ff, K // 2), dtype=np.uint8))
    u = torch.from_numpy(rng.integers(0, 256, (d_ff, K // 2), dtype=np.uint8))
    sg = torch.from_numpy(rng.standard_normal(d_ff).astype(np.float32))
    su = torch.from_numpy(rng.standard_normal(d_ff).astype(np.float32))
    wgu, sw = B.fpt_interleave_gate_up(dev(g), dev(u), dev(sg), dev(su))
    wgu, sw = host(wgu), host(sw)
    for r in range(d_ff // 64):
        assert np.array_equal(wgu[128 * r:128 * r + 64], g[64 * r:64 * r + 64].numpy())
        assert np.array_equal(wgu[128 * r + 64:128 * r + 128], u[64 * r:64 * r + 64].numpy())
        assert np.array_equal(sw[128 * r:128 * r + 64], sg[64 * r:64 * r + 64].numpy())
        assert np.array_equal(sw[128 * r + 64:128 * r + 128], su[64 * r:64 * r + 64].numpy())


def _rows_with_products_that_round_to_a_tie(scale, n_rows, K, seed):
    """Per-token multipliers p and bf16 inputs for which (x * p) * (1/D) is exactly k + 1/2 after its
    two roundings while the unrounded product is not: a kernel that contracts the second multiply
    with anything that follows takes the other code there.  Found by search over all bf16 values."""
    rng = np.random.default_rng(seed)
    F = np.float32
    inv = F(1.0) / F(scale)
    vals = np.arange(0x3C00, 0x4300, dtype=np.uint32)                       # bf16 patterns of about 0.008 .. 128
    xs = (vals << 16).view(F)
    rows, ps, hits = [], [], 0
    while len(rows) < n_rows:
        cand = np.exp(rng.uniform(-3.0, 0.5, 4096)).astype(F)                # many multipliers at once
        v = (xs[None, :] * cand[:, None]).astype(F)
        u = (v * inv).astype(F)
        tie = (np.abs(u) < 8) & (u - np.floor(u) == F(0.5))
        off = v.astype(np.float64) * np.float64(inv) != u.astype(np.float64)
        good = tie & off
        for i in np.nonzero(good.any(axis=1))[0]:
            if len(rows) == n_rows:
                break
            sel = xs[good[i]]
            row = rng.choice(xs, K).astype(F) * rng.choice([-1, 1], K).astype(F)
            row[:sel.size] = sel
            row[sel.size:2 * sel.size] = -sel
            hits += 2 * sel.size
            rows.append(row)
            ps.append(cand[i])
    return np.stack(rows), np.array(ps, dtype=F), hits


@pytest.mark.parametrize("K", [256, 4096])
def test_act_quant_products_that_round_to_a_tie(K):
    scale = 0.62
    x, p, hits = _rows_with_products_that_round_to_a_tie(scale, 60, K, 9)
    assert hits >= 100
    x, p = np.tile(x, (10, 1)), np.tile(p, 10)           # 600 tokens: enough for the many-token kernels
    xb = synth.to_bf16(x)
    qp = B.QParams(4, True, scale, 0)
    for M in (600, 24):                                  # the many-token and the few-token kernels
        xq, _ = B.fpt_act_quant(dev(xb[:M]), qp, B.SCALE_INPUT, 0.0, s_in=dev(torch.from_numpy(p[:M])))
        codes, _, _, _ = OQ.act_quant(synth.f32(xb[:M]), oqp(qp), False, True, 0.0, p[:M])
        assert np.array_equal(host(xq), OQ.pack_int4(codes))
