"""GPU parity of the dynamic (per-token grid) quantiser and linear against the oracle: codes, scales
and per-token vectors bit for bit, outputs within one bf16 ulp."""
import numpy as np
import pytest
import torch

from oracle import quantizers as OQ, linear as OL
from paper_2506_04985_b200 import binding as B, synth
from helpers import dev, host, bf16_host, assert_bf16_close

pytestmark = pytest.mark.gpu


def _acts(M, K, seed):
    return synth.activations(M, K, seed, f"dyn{M}x{K}", law="student_t3", outlier_frac=0.005, outlier_gain=50.0,
                             token_log_std=0.7)


def _codes_host(xq, bits):
    return host(xq) if bits == 8 else OQ.unpack_int4(host(xq), True)


@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("M,K", [(128, 1024), (37, 4096), (5, 14336), (3, 28672), (130, 128), (2, 32), (9, 8192),
                                 (300, 2048), (1, 65536 - 32)])
@pytest.mark.parametrize("mode", ["norm", "norm_sin", "scale", "norm_scale", "plain"])
def test_dynamic_quantiser_bit_exact(bits, M, K, mode):
    x = _acts(M, K, 3)
    s_in = synth.per_token_scale(M, 3, "s_in")
    flags = {"norm": B.RMSNORM, "norm_sin": B.RMSNORM, "scale": B.SCALE_INPUT,
             "norm_scale": B.RMSNORM | B.SCALE_INPUT, "plain": 0}[mode]
    use_s = mode in ("norm_sin", "scale", "norm_scale")
    xq, s_out, delta = B.fpt_act_quant_dynamic(dev(x), bits, flags, 1e-5, s_in=dev(s_in) if use_s else None)
    codes, d, so, _, _ = OQ.act_quant_dynamic(synth.f32(x), bits, bool(flags & B.RMSNORM), bool(flags & B.SCALE_INPUT),
                                              1e-5, s_in.numpy() if use_s else None)
    assert np.array_equal(host(delta).view(np.uint32), d.view(np.uint32))
    assert np.array_equal(host(s_out).view(np.uint32), so.view(np.uint32))
    assert np.array_equal(_codes_host(xq, bits), codes)
    assert np.abs(codes.astype(np.int32)).max() == (7 if bits == 4 else 127)


@pytest.mark.parametrize("bits", [4, 8])
def test_dynamic_quantiser_degenerate_rows(bits):
    """All-zero rows, rows with Inf / NaN (scale 1), ties exactly between two codes, a strided input."""
    K = 256
    x = np.zeros((6, K), dtype=np.float32)
    x[1, 0], x[1, 1], x[1, 2] = np.inf, -np.inf, 3.0
    x[2, 0], x[2, 1] = np.nan, -2.0
    qmax = 7 if bits == 4 else 127
    x[3, :8] = np.array([qmax, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 3.5], dtype=np.float32)   # D = 1: ties to even
    x[4] = np.linspace(-1, 1, K).astype(np.float32)
    x[5, 7] = -1e-30
    xb = synth.to_bf16(x)
    wide = torch.zeros((6, K + 64), dtype=torch.bfloat16)
    wide[:, :K] = xb
    xd = dev(wide)[:, :K]
    xq, _, delta = B.fpt_act_quant_dynamic(xd, bits, 0, 0.0)
    codes, d, _, _, _ = OQ.act_quant_dynamic(synth.f32(xb), bits, False, False, 0.0, None)
    assert np.array_equal(host(delta).view(np.uint32), d.view(np.uint32))
    assert np.array_equal(_codes_host(xq, bits), codes)
    assert d[0] == 1 and d[1] == 1 and d[2] == 1 and d[3] == 1
    assert list(codes[3, :8]) == [qmax, 0, 2, 2, 0, -2, -2, 4]


@pytest.mark.parametrize("M,N,K", [(128, 1024, 1024), (300, 512, 4096), (8, 4096, 4096), (40, 1024, 2048),
                                   (2048, 6144, 4096)])
@pytest.mark.parametrize("post_mode", [B.POST_NONE, B.POST_INVERSE_OF_PRE, B.POST_VECTOR])
def test_dynamic_linear_parity(M, N, K, post_mode):
    if M == 2048 and post_mode != B.POST_INVERSE_OF_PRE:
        pytest.skip("the large shape once")
    x = _acts(M, K, 4)
    w = synth.weights(N, K, 0.02, 4, "dyn/w")
    s_in = synth.per_token_scale(M, 4, "dyn/s")
    post = synth.per_token_scale(M, 4, "dyn/post")
    wq, sw, _ = B.fpt_quantize_weights(dev(w))
    cw, d, _ = OQ.quantize_weights(synth.f32(w))
    flags = B.RMSNORM | (B.SCALE_INPUT if post_mode == B.POST_VECTOR else 0)
    Y, s_out = B.fpt_w4a4_linear_dynamic(dev(x), wq, sw, 4, flags, 1e-5, s_in=dev(s_in), post_mode=post_mode,
                                         post=dev(post) if post_mode == B.POST_VECTOR else None)
    rows = np.arange(M) if M <= 300 else np.array([0, 1, 127, 128, 255, 256, 1023, 1024, 2046, 2047])
    ref = OL.w4a4_linear_dynamic(synth.f32(x)[rows], cw, d, 4, True, bool(flags & B.SCALE_INPUT), 1e-5,
                                 s_in.numpy()[rows], post_mode, post.numpy()[rows])
    assert np.array_equal(host(s_out)[rows], ref["s_out"])
    assert assert_bf16_close(bf16_host(Y)[rows], ref["y"], "dynamic linear Y") == 0
