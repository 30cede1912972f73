"""Function preservation of the merged transforms, in float64 (Theorem 1, Sec. 3.1.2, 3.1.3)."""
import numpy as np
import pytest

from oracle import transforms as T


def _setup(seed, d_model=96, d_head=16, H=2, m=3, L=12):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((L, d_model))
    wq = rng.standard_normal((m * H * d_head, d_model)) / np.sqrt(d_model)
    wk = rng.standard_normal((H * d_head, d_model)) / np.sqrt(d_model)
    wv = rng.standard_normal((H * d_head, d_model)) / np.sqrt(d_model)
    wo = rng.standard_normal((d_model, m * H * d_head)) / np.sqrt(m * H * d_head)
    thetas = 10000.0 ** (-np.arange(d_head // 2) / (d_head // 2))
    pos = rng.integers(0, 4096, L)
    return rng, x, wq, wk, wv, wo, thetas, pos


def _tk(rng, H, d_head, pairing, **kw):
    out = [T.make_tk_head(rng.uniform(-np.pi, np.pi, d_head // 2),
                          np.exp(rng.standard_normal(d_head // 2) * 0.5), pairing, **kw) for _ in range(H)]
    return [a for a, _ in out], [b for _, b in out]


def test_rope_depends_on_relative_position_only():
    rng = np.random.default_rng(0)
    d = 8
    thetas = 10000.0 ** (-np.arange(d // 2) / (d // 2))
    q, k = rng.standard_normal((1, d)), rng.standard_normal((1, d))
    for pairing in ("interleaved", "half"):
        a = T.apply_rope(q, [17], thetas, pairing) @ T.apply_rope(k, [5], thetas, pairing).T
        b = T.apply_rope(q, [112], thetas, pairing) @ T.apply_rope(k, [100], thetas, pairing).T
        assert abs(a - b) < 1e-12
        R = T.rope_matrix(d, 3, thetas, pairing)
        assert np.allclose(R @ R.T, np.eye(d), atol=1e-14) and np.linalg.det(R) > 0


@pytest.mark.parametrize("pairing", ["interleaved", "half"])
@pytest.mark.parametrize("m,H", [(1, 2), (4, 2), (3, 1)])
def test_theorem1_logits_unchanged(pairing, m, H):
    rng, x, wq, wk, wv, wo, thetas, pos = _setup(1, H=H, m=m)
    tk, tkb = _tk(rng, H, 16, pairing)
    wq2, wk2, _, _ = T.fold_attention(wq, wk, wv, wo, 16, m, tk=tk, tkbar=tkb)
    assert np.linalg.norm(wk2 - wk) > 0.1 * np.linalg.norm(wk)            # the merge is not a no-op
    a = T.attention_logits(x, wq, wk, 16, m, pos, thetas, pairing)
    b = T.attention_logits(x, wq2, wk2, 16, m, pos, thetas, pairing)
    assert np.max(np.abs(a - b)) <= 1e-10 * np.max(np.abs(a))


def test_tkbar_times_tk_transposed_is_identity_but_not_inverse_under_gqa():
    rng = np.random.default_rng(2)
    for pairing in ("interleaved", "half"):
        Tk, Tb = T.make_tk_head(rng.uniform(-3, 3, 8), np.exp(rng.standard_normal(8)), pairing)
        assert np.allclose(Tb @ Tk.T, np.eye(16), atol=1e-13)
        assert np.allclose(Tb, np.linalg.inv(Tk).T, atol=1e-12)
        assert not np.allclose(Tb, np.linalg.inv(Tk), atol=1e-3)          # T-bar is the inverse TRANSPOSE
        R = T.rope_matrix(16, 77, 10000.0 ** (-np.arange(8) / 8), pairing)
        assert np.allclose(R @ Tk, Tk @ R, atol=1e-13)                    # commutes with RoPE


def test_reflection_or_unequal_pair_scales_break_theorem1():
    rng, x, wq, wk, wv, wo, thetas, pos = _setup(3, H=1, m=1)
    a = T.attention_logits(x, wq, wk, 16, 1, pos, thetas, "interleaved")
    refl = np.zeros(8, bool)
    refl[2] = True
    Tk, Tb = T.make_tk_head(rng.uniform(-3, 3, 8), np.ones(8), "interleaved", reflect=refl)
    wq2, wk2, _, _ = T.fold_attention(wq, wk, wv, wo, 16, 1, tk=[Tk], tkbar=[Tb])
    b = T.attention_logits(x, wq2, wk2, 16, 1, pos, thetas, "interleaved")
    assert np.max(np.abs(a - b)) > 1e-3 * np.max(np.abs(a))
    s = np.exp(rng.standard_normal(16))                                   # one scale per coordinate
    Tk, Tb = T.make_tk_head(rng.uniform(-3, 3, 8), s, "interleaved")
    wq2, wk2, _, _ = T.fold_attention(wq, wk, wv, wo, 16, 1, tk=[Tk], tkbar=[Tb])
    b = T.attention_logits(x, wq2, wk2, 16, 1, pos, thetas, "interleaved")
    assert np.max(np.abs(a - b)) > 1e-3 * np.max(np.abs(a))
    # and a transform built for the wrong pairing does not commute with RoPE either
    Tk, Tb = T.make_tk_head(rng.uniform(-3, 3, 8), np.ones(8), "half")
    wq2, wk2, _, _ = T.fold_attention(wq, wk, wv, wo, 16, 1, tk=[Tk], tkbar=[Tb])
    b = T.attention_logits(x, wq2, wk2, 16, 1, pos, thetas, "interleaved")
    assert np.max(np.abs(a - b)) > 1e-3 * np.max(np.abs(a))


def test_wrong_gqa_repeat_is_detected():
    """Query heads j use kv head j // m; pairing consecutive blocks differently must fail."""
    rng, x, wq, wk, wv, wo, thetas, pos = _setup(4, H=2, m=2)
    tk, tkb = _tk(rng, 2, 16, "interleaved")
    wk2 = T.fold_rows(wk, tk, 16, 1)
    wq_bad = T.fold_rows(wq, [tkb[0], tkb[1], tkb[0], tkb[1]], 16, 1)     # interleaved, not repeated
    a = T.attention_logits(x, wq, wk, 16, 2, pos, thetas, "interleaved")
    b = T.attention_logits(x, wq_bad, wk2, 16, 2, pos, thetas, "interleaved")
    assert np.max(np.abs(a - b)) > 1e-3 * np.max(np.abs(a))


@pytest.mark.parametrize("m,H", [(1, 2), (4, 2)])
def test_value_transform_preserves_attention_output(m, H):
    rng, x, wq, wk, wv, wo, thetas, pos = _setup(5, H=H, m=m)
    pos = np.arange(x.shape[0])
    tv = [np.eye(16) + 0.3 * rng.standard_normal((16, 16)) for _ in range(H)]
    tk, tkb = _tk(rng, H, 16, "half")
    y0 = T.attention_block(x, wq, wk, wv, wo, 16, m, pos, thetas, "half")
    w2 = T.fold_attention(wq, wk, wv, wo, 16, m, tk=tk, tkbar=tkb, tv=tv)
    y1 = T.attention_block(x, *w2, 16, m, pos, thetas, "half")
    assert np.linalg.norm(w2[2] - wv) > 0.05 * np.linalg.norm(wv)
    assert np.max(np.abs(y0 - y1)) <= 1e-5 * np.max(np.abs(y0))          # bound asked of the build
    assert np.max(np.abs(y0 - y1)) <= 1e-9 * np.max(np.abs(y0))          # what float64 delivers
    # merging T_v into W_o without inverting it is not function preserving
    wo_bad = T.fold_cols(wo, tv, 16, m)
    y2 = T.attention_block(x, w2[0], w2[1], w2[2], wo_bad, 16, m, pos, thetas, "half")
    assert np.max(np.abs(y0 - y2)) > 1e-2 * np.max(np.abs(y0))


def test_residual_scaling_recursion():
    """Z~_n = S_n * Z_n, S_n = 1/||X_n||_R, and the final RMSNorm removes S_N (Sec. 3.1.3)."""
    rng = np.random.default_rng(6)
    L, d, dff, nblk = 10, 32, 64, 4
    x1 = rng.standard_normal((L, d)) * np.exp(rng.standard_normal((L, 1)) * 2)   # wild token norms
    ws = [(rng.standard_normal((dff, d)) / 5, rng.standard_normal((dff, d)) / 5,
           rng.standard_normal((d, dff)) / 5) for _ in range(nblk)]
    blocks = [lambda xn, s, w=w: T.swiglu_mlp(xn, *w, mid_scale=s) for w in ws]
    zs = T.plain_forward(x1, blocks)
    zts, ss = T.residual_scaling_forward(x1, blocks)
    xs = [x1] + zs[:-1]
    for n in range(nblk):
        assert np.allclose(ss[n], 1.0 / T.rms(xs[n]), rtol=1e-12)
        assert np.allclose(zts[n], ss[n][:, None] * zs[n], rtol=1e-10, atol=1e-12)
    fin0 = zs[-1] / T.rms(zs[-1])[:, None]
    fin1 = zts[-1] / T.rms(zts[-1])[:, None]
    assert np.max(np.abs(fin0 - fin1)) < 1e-10
    # the first normalised residual has unit RMS per token while the plain one does not
    assert np.allclose(T.rms(zts[0] - blocks[0](x1 / T.rms(x1)[:, None], ss[0])), 1.0)
    assert T.rms(x1).max() / T.rms(x1).min() > 50
    # a per-token scaler commutes with a bias-free linear
    w = rng.standard_normal((7, d))
    s = np.exp(rng.standard_normal(L))
    assert np.allclose((s[:, None] * x1) @ w.T, s[:, None] * (x1 @ w.T), rtol=1e-13)
