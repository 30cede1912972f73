"""The library's offline fold helper (float64) against the oracle's independent construction and
against the float64 reference model: merged and unmerged networks must compute the same function
(Theorem 1; Sec. 3.1.2; Sec. 3.1 last paragraph), within 1e-5 relative."""
import numpy as np
import pytest

from oracle import hadamard as OH
from oracle import transforms as OT
from paper_2506_04985_b200 import fold, synth


def _model(seed, d_model=96, d_head=16, H=2, m=3, L=10):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((L, d_model))
    wq = rng.standard_normal((H * m * d_head, d_model)) * 0.1
    wk = rng.standard_normal((H * d_head, d_model)) * 0.1
    wv = rng.standard_normal((H * d_head, d_model)) * 0.1
    wo = rng.standard_normal((d_model, H * m * d_head)) * 0.1
    thetas = 10000.0 ** (-np.arange(d_head // 2) / (d_head // 2))
    return rng, x, wq, wk, wv, wo, thetas


def _rel(a, b):
    return np.max(np.abs(a - b)) / np.max(np.abs(b))


@pytest.mark.parametrize("pairing", ["interleaved", "half"])
@pytest.mark.parametrize("m,H", [(1, 4), (4, 2)])
def test_pre_rope_fold_matches_oracle_and_keeps_the_logits(pairing, m, H):
    d_head = 16
    rng, x, wq, wk, wv, wo, thetas = _model(1, d_head=d_head, H=H, m=m)
    phi, s = synth.tk_params(H, d_head, 3, "fold/tk")
    wq2, wk2 = fold.fold_pre_rope(wq, wk, phi, s, H, d_head, pairing)
    blocks = [OT.make_tk_head(phi[h], s[h], pairing) for h in range(H)]
    wq_o, wk_o, _, _ = OT.fold_attention(wq, wk, wv, wo, d_head, m, tk=[b[0] for b in blocks], tkbar=[b[1] for b in blocks])
    assert np.allclose(wq2, wq_o, rtol=1e-12, atol=1e-14) and np.allclose(wk2, wk_o, rtol=1e-12, atol=1e-14)
    pos = np.array([0, 1, 2, 5, 17, 100, 1000, 2047, 4095, 3])
    ref = OT.attention_logits(x, wq, wk, d_head, m, pos, thetas, pairing)
    got = OT.attention_logits(x, wq2, wk2, d_head, m, pos, thetas, pairing)
    assert _rel(got, ref) < 1e-10
    # the wrong pairing must NOT preserve the logits (the transform has to match the RoPE in use)
    other = "half" if pairing == "interleaved" else "interleaved"
    bad = OT.attention_logits(x, *fold.fold_pre_rope(wq, wk, phi, s, H, d_head, other), d_head, m, pos, thetas, pairing)
    assert _rel(bad, ref) > 1e-3


@pytest.mark.parametrize("m,H", [(1, 3), (4, 2)])
def test_value_fold_matches_oracle_and_keeps_the_block_output(m, H):
    d_head = 16
    rng, x, wq, wk, wv, wo, thetas = _model(2, d_head=d_head, H=H, m=m)
    tv = synth.tv_params(H, d_head, 5, "fold/tv") + 0.3 * rng.standard_normal((H, d_head, d_head)) / np.sqrt(d_head)
    wv2, wo2 = fold.fold_value(wv, wo, tv, H, d_head)
    _, _, wv_o, wo_o = OT.fold_attention(wq, wk, wv, wo, d_head, m, tv=list(tv))
    assert np.allclose(wv2, wv_o, rtol=1e-11, atol=1e-13) and np.allclose(wo2, wo_o, rtol=1e-9, atol=1e-12)
    pos = np.arange(x.shape[0])
    ref = OT.attention_block(x, wq, wk, wv, wo, d_head, m, pos, thetas, "half")
    got = OT.attention_block(x, wq, wk, wv2, wo2, d_head, m, pos, thetas, "half")
    assert _rel(got, ref) < 1e-5


def test_up_down_scaler_and_norm_weight_keep_the_mlp():
    rng = np.random.default_rng(4)
    d, dff, L = 48, 160, 9
    x = rng.standard_normal((L, d))
    gamma = np.exp(0.3 * rng.standard_normal(d))
    wg, wu, wd = (rng.standard_normal(s) * 0.2 for s in ((dff, d), (dff, d), (d, dff)))
    xn = x / OT.rms(x)[:, None]
    ref = OT.swiglu_mlp(xn * gamma[None, :], wg, wu, wd)
    t = np.exp(rng.standard_normal(dff)) * rng.choice([-1.0, 1.0], dff)
    wu2, wd2 = fold.fold_up_down_scaler(fold.fold_norm_weight(wu, gamma), wd, t)
    got = OT.swiglu_mlp(xn, fold.fold_norm_weight(wg, gamma), wu2, wd2)
    assert _rel(got, ref) < 1e-10


def test_residual_rotation_keeps_a_two_block_network():
    rng = np.random.default_rng(6)
    d, dff, L = 32, 96, 7
    x = rng.standard_normal((L, d)) * 3.0
    rot, _ = np.linalg.qr(rng.standard_normal((d, d)))
    layers = [tuple(rng.standard_normal(s) * 0.2 for s in ((dff, d), (dff, d), (d, dff))) for _ in range(2)]

    def net(x0, ls):
        return OT.plain_forward(x0, [lambda xn, s, l=l: OT.swiglu_mlp(xn, *l) for l in ls])[-1]

    ref = net(x, layers)
    rotated = []
    for wg, wu, wd in layers:
        (wg2, wu2), (wd2,) = fold.fold_residual_rotation([wg, wu], [wd], rot)
        rotated.append((wg2, wu2, wd2))
    got = net(x @ rot, rotated)                   # the embedding is rotated once; so is the output
    assert _rel(got, ref @ rot) < 1e-10
    with pytest.raises(AssertionError):
        fold.fold_residual_rotation([layers[0][0]], [layers[0][2]], rot * 1.01)


@pytest.mark.parametrize("dff", [96, 224, 1024])
def test_down_hadamard_fold_matches_the_definition_and_keeps_the_mlp(dff):
    rng = np.random.default_rng(8)
    d, L = 40, 6
    wg, wu, wd = (rng.standard_normal(s) * 0.2 for s in ((dff, d), (dff, d), (d, dff)))
    hb = OH.block_hadamard_matrix(dff)
    assert fold.hadamard_block_size(dff) == OH.largest_pow2_divisor(dff)
    wd2 = fold.fold_down_hadamard(wd)
    assert np.allclose(wd2, wd @ hb, rtol=1e-12, atol=1e-13)
    # the network with the online transform in front of the merged weight computes the same function
    xn = rng.standard_normal((L, d))
    g = xn @ wg.T
    m = g / (1.0 + np.exp(-g)) * (xn @ wu.T)
    ref = m @ wd.T
    got = (m @ hb.T) @ wd2.T
    assert _rel(got, ref) < 1e-10
