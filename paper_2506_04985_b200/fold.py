"""Offline merge of the function-preserving transforms into stored weights, in float64.

This is the step that comes before `fpt_quantize_weights`: the transforms that can be merged
cost nothing at inference time once they are part of the weights (Sec. 3.1, "mergeable").
Weights are stored [out_features, in_features] (y = x @ W.T); the paper writes row vectors times
W of shape [d_in, d_out], so a paper merge "W T" acts on the ROWS of the stored matrix and a merge
"T W" on its COLUMNS.  Everything is numpy float64 (App. D keeps all transforms in double
precision); round to the storage type afterwards.

    fold_pre_rope          Sec. 3.1.1, Theorem 1, Eq. 1-4: W_k <- W_k T_k, W_q <- W_q T-bar_k
    fold_value             Sec. 3.1.2, Eq. 5: W_v <- W_v T_v, W_o <- T_v^-1 W_o per head
    fold_norm_weight       RMSNorm weight gamma into the linears that read the normalised vector
    fold_up_down_scaler    Sec. 3.1 (last paragraph): per-channel scaler between up and down projection
    fold_residual_rotation Sec. 3.1 (last paragraph): one orthogonal matrix on the residual stream
    fold_down_hadamard     Sec. 3.1 (last paragraph), App. D: inverse of the online block-wise Hadamard
                           transform at the down-projection input, merged into the down projection

Readings of the paper used here (the same as everywhere in this package): every 2x2 block of
T_k is a proper rotation times ONE scale shared by its two coordinates; under grouped-query
attention the block of kv head h applies to each of its m query heads; the pairing of
coordinates is the one RoPE uses.
"""
import numpy as np


def _pair_index(d_head, pairing):
    n = d_head // 2
    if pairing == "interleaved":          # (2n, 2n+1), the layout of App. C
        return np.arange(0, d_head, 2), np.arange(1, d_head, 2)
    if pairing == "half":                 # (n, n + d/2), the layout most Llama code uses
        return np.arange(n), np.arange(n, d_head)
    raise ValueError(f"unknown RoPE pairing {pairing!r}")


def _rotate_scale_rows(w, heads, d_head, phi, scale, pairing):
    """Rows of every head h, taken in RoPE pairs (a, b), become scale * R(phi)^T (row_a, row_b)."""
    w = np.array(w, dtype=np.float64).reshape(heads, d_head, -1)
    ia, ib = _pair_index(d_head, pairing)
    c = (np.cos(phi) * scale)[:, :, None]
    s = (np.sin(phi) * scale)[:, :, None]
    a, b = w[:, ia, :], w[:, ib, :]
    out = np.empty_like(w)
    out[:, ia, :] = c * a + s * b
    out[:, ib, :] = -s * a + c * b
    return out.reshape(heads * d_head, -1)


def fold_pre_rope(wq, wk, phi, s, n_kv_heads, d_head, pairing="half"):
    """phi, s: [n_kv_heads, d_head / 2] angles and positive scales.  Returns (W_q', W_k').

    Keys get T_k = s * R(phi) per pair, queries get T-bar_k = R(phi) / s, so that every
    query-key product after RoPE is unchanged (Theorem 1)."""
    phi = np.asarray(phi, dtype=np.float64)
    s = np.asarray(s, dtype=np.float64)
    assert phi.shape == s.shape == (n_kv_heads, d_head // 2) and np.all(s > 0)
    n_q_heads = wq.shape[0] // d_head
    assert wk.shape[0] == n_kv_heads * d_head and n_q_heads % n_kv_heads == 0
    m = n_q_heads // n_kv_heads
    wk2 = _rotate_scale_rows(wk, n_kv_heads, d_head, phi, s, pairing)
    wq2 = _rotate_scale_rows(wq, n_q_heads, d_head, np.repeat(phi, m, axis=0), np.repeat(1.0 / s, m, axis=0), pairing)
    return wq2, wk2


def fold_value(wv, wo, tv, n_kv_heads, d_head):
    """tv: [n_kv_heads, d_head, d_head], invertible.  Returns (W_v', W_o').

    Value head h is multiplied by T_v^(h); the d_head input columns of the output projection that
    belong to each of its m query heads by the inverse, so attention-times-value-times-output is
    unchanged whatever the attention probabilities are."""
    tv = np.asarray(tv, dtype=np.float64)
    assert tv.shape == (n_kv_heads, d_head, d_head)
    n_q_heads = wo.shape[1] // d_head
    m = n_q_heads // n_kv_heads
    v = np.array(wv, dtype=np.float64).reshape(n_kv_heads, d_head, -1)
    wv2 = np.einsum("hij,hik->hjk", tv, v).reshape(n_kv_heads * d_head, -1)        # T^T rows
    o = np.array(wo, dtype=np.float64).reshape(wo.shape[0], n_q_heads, d_head)
    # columns of head j become cols @ (T^-1)^T, i.e. the solution Z of Z T^T = cols
    t_rep = np.repeat(tv, m, axis=0)
    wo2 = np.stack([np.linalg.solve(t_rep[j], o[:, j, :].T).T for j in range(n_q_heads)], axis=1)
    return wv2, wo2.reshape(wo.shape[0], n_q_heads * d_head)


def fold_norm_weight(w, gamma):
    """Linear that reads RMSNorm(x) * gamma: the weight of the norm moves into its input columns."""
    return np.asarray(w, dtype=np.float64) * np.asarray(gamma, dtype=np.float64)[None, :]


def fold_up_down_scaler(wu, wd, t):
    """Per-channel scaler t (non-zero) on the up projection's outputs, undone on the down
    projection's inputs: silu(g) * (t u) then / t is the same product."""
    t = np.asarray(t, dtype=np.float64)
    assert np.all(t != 0)
    return np.asarray(wu, dtype=np.float64) * t[:, None], np.asarray(wd, dtype=np.float64) / t[None, :]


def fold_residual_rotation(readers, writers, rot):
    """One orthogonal matrix on the residual stream (x' = x R): linears that READ the (normalised)
    residual get W <- W R, linears that WRITE to it W <- R^T W.  RMSNorm commutes with R only
    without a per-channel weight: fold the norm weights first (`fold_norm_weight`)."""
    rot = np.asarray(rot, dtype=np.float64)
    assert np.allclose(rot @ rot.T, np.eye(rot.shape[0]), atol=1e-10), "R must be orthogonal"
    return ([np.asarray(w, dtype=np.float64) @ rot for w in readers],
            [rot.T @ np.asarray(w, dtype=np.float64) for w in writers])


def hadamard_block_size(d):
    """Group size of the block-wise Hadamard on d channels: the largest power of two dividing d
    (App. D "Hadamard non-powers of 2": groups of a power-of-two size, no zero padding)."""
    return d & (-d)


def _fwht_last_axis(a):
    """Unnormalised Walsh-Hadamard transform (Sylvester order) along the last axis, float64."""
    n = a.shape[-1]
    if n == 1:
        return a
    half = n // 2
    top, bot = _fwht_last_axis(a[..., :half]), _fwht_last_axis(a[..., half:])
    return np.concatenate([top + bot, top - bot], axis=-1)


def fold_down_hadamard(wd, block=None):
    """The activations entering the down projection are transformed online, group by group, with the
    orthonormal Hadamard matrix H (fpt_decoder_mlp with mid_hadamard = 1); H is symmetric and its own
    inverse, so the merged weight is W_d <- W_d blockdiag(H, ..., H) on the input columns."""
    wd = np.asarray(wd, dtype=np.float64)
    d = wd.shape[1]
    block = block or hadamard_block_size(d)
    assert d % block == 0 and block & (block - 1) == 0
    g = wd.reshape(wd.shape[0], d // block, block)
    return (_fwht_last_axis(g) / np.sqrt(block)).reshape(wd.shape[0], d)
