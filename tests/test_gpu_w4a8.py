"""GPU parity of the W4A8 path (8-bit activation codes, 4-bit weights) against the oracle: integer
accumulators and codes bit for bit, outputs within one bf16 ulp.  Both routes are covered: the
CTA-pair kernel with an int8 activation tile and the split a = 16 (a >> 4) + (a & 15) for small shapes."""
import numpy as np
import pytest
import torch

from oracle import quantizers as OQ, linear as OL
from oracle.int_matmul import int_matmul
from oracle.epilogue import dequant_epilogue
from paper_2506_04985_b200 import binding as B, synth
from helpers import dev, host, oqp, bf16_host, assert_bf16_close, random_codes, packed_dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("M,N,K", [(1, 256, 128), (8, 1024, 1024), (16, 512, 4096), (40, 1024, 2048), (64, 264, 512),
                                   (100, 512, 1024), (128, 4096, 256), (300, 128, 1024), (129, 136, 128),
                                   (256, 256, 128), (384, 520, 1024), (513, 1024, 4096), (300, 2048, 14336),
                                   (2048, 2048, 4096)])
@pytest.mark.parametrize("extras", [False, True])
def test_w4a8_gemm_exact_accumulators_and_outputs(M, N, K, extras):
    if extras and M * N * K > 2 ** 31:
        pytest.skip("large shapes once")
    rng = np.random.default_rng(M * 7 + N)
    qa = rng.integers(-128, 128, (M, K)).astype(np.int8)
    qa[0, :] = -128 if M > 1 else qa[0, :]                   # extreme rows: the largest accumulators there are
    qw = random_codes(rng, (N, K))
    qw[0, :] = -8
    sw = (rng.uniform(0.5, 1.5, N) * 2e-3).astype(np.float32)
    post = rng.uniform(0.5, 2.0, M).astype(np.float32) if extras else None
    res = synth.to_bf16(rng.standard_normal((M, N)).astype(np.float32)) if extras else None
    rs = rng.uniform(0.5, 2.0, M).astype(np.float32) if extras else None
    Y, acc = B.fpt_w4a8_gemm(dev(qa), packed_dev(qw), dev(sw), 0.031, post=None if post is None else dev(post),
                             residual=None if res is None else dev(res), res_scale=None if rs is None else dev(rs),
                             want_acc=True)
    ws = B.new_workspace(B.OP_GEMM_A8, M, N, K)
    assert B.lib().fpt_check_status(None, B._ptr(ws)) == 0
    rows = np.arange(M) if M * N * K <= 2 ** 31 else np.unique(np.r_[0:3, 127:130, 255:258, M - 2:M])
    ref_acc = int_matmul(qa[rows], qw, 0)
    assert np.array_equal(host(acc)[rows], ref_acc)
    resid = None if res is None else (synth.f32(res)[rows] * rs[rows, None]).astype(np.float32)
    ref_y = dequant_epilogue(ref_acc, sw, 0.031, None if post is None else post[rows], resid)
    assert assert_bf16_close(bf16_host(Y)[rows], ref_y, "w4a8 Y") == 0


@pytest.mark.parametrize("M,K", [(128, 1024), (37, 4096), (5, 14336), (130, 128), (2, 32), (600, 2048)])
@pytest.mark.parametrize("mode", ["norm", "scale", "norm_scale"])
def test_static_eight_bit_quantiser_bit_exact(M, K, mode):
    x = synth.activations(M, K, 3, f"a8{M}x{K}", law="student_t3", outlier_frac=0.005, outlier_gain=50.0, token_log_std=0.7)
    s_in = synth.per_token_scale(M, 3, "s_in")
    flags = {"norm": B.RMSNORM, "scale": B.SCALE_INPUT, "norm_scale": B.RMSNORM | B.SCALE_INPUT}[mode]
    qp = B.QParams(8, True, 0.031 if flags & B.RMSNORM else 0.11, 0)
    xq, s_out = B.fpt_act_quant(dev(x), qp, flags, 1e-5, s_in=dev(s_in) if flags & B.SCALE_INPUT else None)
    codes, so, _, _ = OQ.act_quant(synth.f32(x), oqp(qp), bool(flags & B.RMSNORM), bool(flags & B.SCALE_INPUT), 1e-5,
                                   s_in.numpy() if flags & B.SCALE_INPUT else None)
    assert xq.dtype == torch.int8 and np.array_equal(host(xq), codes)
    assert np.array_equal(host(s_out).view(np.uint32), so.view(np.uint32))
    assert np.abs(codes.astype(np.int32)).max() == 128 or len(np.unique(codes)) > 100


@pytest.mark.parametrize("M,N,K", [(8, 1024, 1024), (100, 512, 2048), (300, 1024, 4096), (2048, 6144, 4096)])
@pytest.mark.parametrize("dynamic", [False, True])
@pytest.mark.parametrize("post_mode", [B.POST_NONE, B.POST_INVERSE_OF_PRE])
def test_w4a8_linear_parity(M, N, K, dynamic, post_mode):
    x = synth.activations(M, K, 6, f"a8lin{M}", law="student_t3", outlier_frac=0.005, outlier_gain=50.0, token_log_std=0.7)
    w = synth.weights(N, K, 0.02, 6, "a8/w")
    wq, sw, _ = B.fpt_quantize_weights(dev(w))
    cw, d, _ = OQ.quantize_weights(synth.f32(w))
    rows = np.arange(M) if M <= 300 else np.array([0, 1, 127, 128, 255, 256, 1023, 1024, 2046, 2047])
    xf = synth.f32(x)
    if dynamic:
        Y, s_out = B.fpt_w4a4_linear_dynamic(dev(x), wq, sw, 8, B.RMSNORM, 1e-5, post_mode=post_mode)
        ref = OL.w4a4_linear_dynamic(xf[rows], cw, d, 8, True, False, 1e-5, None, post_mode)
    else:
        qp = B.QParams(8, True, 0.04, 0)
        Y, s_out = B.fpt_w4a4_linear(dev(x), wq, sw, qp, B.RMSNORM, 1e-5, post_mode=post_mode)
        ref = OL.w4a4_linear(xf[rows], cw, d, oqp(qp), True, False, 1e-5, None, post_mode)
        assert len(np.unique(ref["codes"])) > 60
    assert np.array_equal(host(s_out)[rows], ref["s_out"])
    assert assert_bf16_close(bf16_host(Y)[rows], ref["y"], "w4a8 linear Y") == 0
