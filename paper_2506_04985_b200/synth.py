"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws numbers.  It holds none of the method's arithmetic (no
quantiser, no scale, no transform maths) so that the CUDA library's tests and an
independent checker can both be fed from it.

The paper measures on Llama / Qwen weights and on activations of Wikitext-2
sequences; neither is available offline, so the tensors below copy the structure
the paper describes: roughly Gaussian weights, activations with heavy tails, a
few outlier channels that are much larger than the rest (Sec. 1; App. E), and
tokens whose norms differ widely (Sec. 3.1.3).

Every tensor is a CPU torch.bfloat16 tensor drawn from a Philox stream keyed by
(seed, tensor name); `f32` gives the exact float32 view of one as numpy.
"""
import zlib

import numpy as np
import torch


def _rng(seed, name):
    key = (int(seed) << 32) ^ zlib.crc32(name.encode())
    return np.random.Generator(np.random.Philox(key=key))


def to_bf16(a):
    """numpy float array -> CPU bfloat16 tensor (round-to-nearest-even)."""
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16)


def f32(t):
    """bfloat16 tensor -> numpy float32 with the same values."""
    return t.detach().cpu().to(torch.float32).numpy()


def outlier_channels(k, frac, seed, name):
    """Indices of ceil(frac*k) outlier channels (a seeded permutation's head)."""
    n = int(np.ceil(frac * k))
    return np.sort(_rng(seed, name + "/outliers").permutation(k)[:n])


def normal(shape, std, seed, name):
    r = _rng(seed, name)
    return to_bf16(r.standard_normal(shape, dtype=np.float32) * np.float32(std))


def student_t(shape, nu, seed, name):
    """Student-t(nu) as Z / sqrt(chi2_nu / nu), float32."""
    r = _rng(seed, name)
    z = r.standard_normal(shape, dtype=np.float32)
    c = r.chisquare(nu, size=shape).astype(np.float32)
    return z / np.sqrt(c / np.float32(nu))


def activations(m, k, seed, name, law="normal", outlier_frac=0.01, outlier_gain=40.0,
                token_log_std=0.0):
    """[m, k] activations: base law, some channels multiplied by a gain, and an
    optional log-normal factor per token (norm disparity between tokens)."""
    if law == "normal":
        a = _rng(seed, name).standard_normal((m, k), dtype=np.float32)
    elif law == "student_t3":
        a = student_t((m, k), 3.0, seed, name)
    else:
        raise ValueError(law)
    idx = outlier_channels(k, outlier_frac, seed, name)
    a[:, idx] *= np.float32(outlier_gain)
    if token_log_std > 0.0:
        f = np.exp(_rng(seed, name + "/tok").standard_normal(m) * token_log_std)
        a *= f.astype(np.float32)[:, None]
    return to_bf16(a)


def weights(n, k, std, seed, name, outlier_row_frac=0.0, outlier_row_gain=1.0):
    """[n, k] stored weight (out x in), N(0, std), some rows multiplied by a gain."""
    r = _rng(seed, name)
    w = r.standard_normal((n, k), dtype=np.float32) * np.float32(std)
    if outlier_row_frac > 0.0:
        idx = outlier_channels(n, outlier_row_frac, seed, name + "/rows")
        w[idx, :] *= np.float32(outlier_row_gain)
    return to_bf16(w)


def per_token_scale(m, seed, name, log_std=0.5):
    """Positive per-token scale vector, log-normal, float32 torch tensor."""
    v = np.exp(_rng(seed, name).standard_normal(m) * log_std).astype(np.float32)
    return torch.from_numpy(v)


def tk_params(n_kv_heads, d_head, seed, name):
    """Angles ~ U(-pi, pi) and log-scales ~ N(0, 0.25) for every kv head and 2x2 block."""
    r = _rng(seed, name)
    phi = r.uniform(-np.pi, np.pi, size=(n_kv_heads, d_head // 2))
    s = np.exp(r.standard_normal((n_kv_heads, d_head // 2)) * 0.5)
    return phi, s


def tv_params(n_kv_heads, d_head, seed, name):
    """I + 0.1 * N(0,1)/sqrt(d_head) per kv head: invertible and well conditioned."""
    r = _rng(seed, name)
    g = r.standard_normal((n_kv_heads, d_head, d_head)) * (0.1 / np.sqrt(d_head))
    return np.eye(d_head)[None] + g
