"""Full-size launches of the remaining benchmark configurations on the GPU, checked against the
oracle on sampled token rows (first / last rows of several 256-row tiles) over all output columns.
Codes and accumulators are integers, so the sampled rows must match bit for bit; the bf16
outputs are expected to be identical too (same operation order)."""
import numpy as np
import pytest
import torch

from oracle import quantizers as OQ, linear as OL
from paper_2506_04985_b200 import binding as B, synth
from helpers import dev, host, oqp, bf16_host, assert_bf16_close

pytestmark = pytest.mark.gpu


def _rows(M, n=10):
    base = [0, 1, 127, 128, 255, 256, 257, M // 2 - 1, M // 2, M - 257, M - 256, M - 129, M - 2, M - 1]
    return np.unique(np.clip(np.array(base), 0, M - 1))


def test_config3_mlp_block_4096_tokens_sampled():
    """Llama-3-8B-shaped SwiGLU MLP at 4096 tokens: RMSNorm quantise -> gate/up (14336) -> SiLU*mul,
    per-token scale, quantise -> down (4096), with the normalised residual."""
    M, d, d_ff = 4096, 4096, 14336
    x = synth.activations(M, d, 0, "cfg3/x", law="student_t3", outlier_frac=0.005, outlier_gain=50.0)
    wg = synth.weights(d_ff, d, 0.02, 0, "cfg3/wg")
    wu = synth.weights(d_ff, d, 0.02, 0, "cfg3/wu")
    wd = synth.weights(d, d_ff, 0.02, 0, "cfg3/wd")
    rows = _rows(M)
    xf = synth.f32(x)[rows]
    (cg, sg, _), (cu, su, _), (cd, sd, _) = (OQ.quantize_weights(synth.f32(w)) for w in (wg, wu, wd))
    r = OQ.rms_reciprocal(xf, 1e-5)
    qp_in = B.QParams(4, True, float(OQ.calibrate_static_scale(xf * r[:, None], OQ.QParams())), 0)
    pre = OL.decoder_mlp(xf, cg, sg, cu, su, cd, sd, oqp(qp_in), OQ.QParams(4, True, 1.0), 1e-5)
    qp_mid = B.QParams(4, True, float(OQ.calibrate_static_scale(pre["m"] * pre["s_out"][:, None], OQ.QParams())), 0)
    gq, gs, _ = B.fpt_quantize_weights(dev(wg))
    uq, us, _ = B.fpt_quantize_weights(dev(wu))
    dq, ds, _ = B.fpt_quantize_weights(dev(wd))
    assert np.array_equal(host(dq), OQ.pack_int4(cd))
    wgu, swgu = B.fpt_interleave_gate_up(gq, uq, gs, us)
    ws = B.new_workspace(B.OP_MLP, M, d_ff, d)
    Y, s_out = B.fpt_decoder_mlp(dev(x), wgu, swgu, dq, ds, qp_in, qp_mid, 1e-5, None, True, ws=ws)
    assert B.fpt_check_status(ws) == B.OK
    ref = OL.decoder_mlp(xf, cg, sg, cu, su, cd, sd, oqp(qp_in), oqp(qp_mid), 1e-5, None, True)
    assert np.array_equal(host(s_out)[rows], ref["s_out"])
    assert len(np.unique(ref["mq"])) >= 8
    assert assert_bf16_close(bf16_host(Y)[rows], ref["y"], "cfg3 Y") == 0


@pytest.mark.parametrize("tokens", [512, 2048])
def test_config5_70b_class_linears_sampled(tokens):
    """hidden 8192, MLP 28672, 8 kv heads x 128: fused QKV (10240), O, gate||up as two linears, down;
    weights with outlier rows, activations with outlier channels x60."""
    M, h, d_ff = tokens, 8192, 28672
    rows = _rows(M)

    def run(K, N, name, flags, scale):
        x = synth.activations(M, K, 0, f"cfg5/x{name}", law="student_t3", outlier_frac=0.005, outlier_gain=60.0)
        w = synth.weights(N, K, 0.015, 0, f"cfg5/w{name}", outlier_row_frac=0.002, outlier_row_gain=20.0)
        s_in = synth.per_token_scale(M, 0, f"cfg5/s{name}")
        qp = B.QParams(4, True, scale, 0)
        wq, sw, _ = B.fpt_quantize_weights(dev(w))
        cw, d, _ = OQ.quantize_weights(synth.f32(w))
        assert np.array_equal(host(sw), d)
        ws = B.new_workspace(B.OP_LINEAR, M, N, K)
        Y, s_out = B.fpt_w4a4_linear(dev(x), wq, sw, qp, flags, 1e-5, s_in=dev(s_in), ws=ws)
        assert B.fpt_check_status(ws) == B.OK
        ref = OL.w4a4_linear(synth.f32(x)[rows], cw, d, oqp(qp), bool(flags & B.RMSNORM), bool(flags & B.SCALE_INPUT),
                             1e-5, s_in.numpy()[rows])
        assert len(np.unique(ref["codes"])) >= 8
        assert np.array_equal(host(s_out)[rows], ref["s_out"])
        assert assert_bf16_close(bf16_host(Y)[rows], ref["y"], f"cfg5 {name}") == 0
        del x, w
        torch.cuda.empty_cache()

    run(h, 10240, "qkv", B.RMSNORM, 0.45)
    run(h, h, "o", B.SCALE_INPUT, 2.5)
    if tokens == 512:                      # the wide MLP matrices once: their oracle side is the slow part
        run(h, d_ff, "gate", B.RMSNORM, 0.45)
        run(d_ff, h, "down", B.SCALE_INPUT, 2.5)
