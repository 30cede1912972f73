"""Function-preserving transforms that are merged into the weights, in float64.

Test infrastructure (see the package header).

Storage convention: a weight is stored [out, in] (y = x @ W_stored^T), whereas the
paper writes row vectors times W in R^{d_in x d_out}; so paper-W = W_stored^T and a
paper merge "W T" acts on the ROWS (output features) of the stored matrix, a
merge "T W" on its COLUMNS (input features).

Pre-RoPE transform (Sec. 3.1.1, Theorem 1, Eq. 1-4)
    T_k^(h)    = diag(s^(h)) diag({R_n^(h)}),  T-bar_k^(h) = diag(1/s^(h)) diag({R_n^(h)})
    W~_k = W_k T_k,  W~_q = W_q T-bar_k, the block of kv head h repeated over its m
    query heads.  Readings: R_n is a proper rotation (the remark after the proof
    rules reflections out); there is one scale per 2x2 block, shared by its two
    coordinates (the proof writes each block as w_n R_phi_n); every head's block
    is repeated m times under grouped-query attention; the pairing of
    coordinates is the one RoPE uses ("interleaved": (2n, 2n+1), as in App. C,
    or "half": (n, n + d/2)).

Multi-head value transform (Sec. 3.1.2, Eq. 5)
    W~_v = W_v T_v,  W~_o = T-bar_v W_o with T-bar_v holding each (T_v^(h))^-1 m times.

Per-token residual scaling (Sec. 3.1.3, Eq. 6-7) is simulated by
`residual_scaling_forward` against the plain pre-norm transformer recursion.

Everything here is double precision (App. D, "FPT Parametrization").
"""
import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------- #
# RoPE (App. C, "RoPE background"): f(x, i) = x R_{Theta,i}, row-vector form
# --------------------------------------------------------------------------- #
def rope_pairs(d_head, pairing):
    n = d_head // 2
    if pairing == "interleaved":
        return [(2 * i, 2 * i + 1) for i in range(n)]
    if pairing == "half":
        return [(i, i + n) for i in range(n)]
    raise ValueError(pairing)


def rot2(phi):
    c, s = np.cos(phi), np.sin(phi)
    return np.array([[c, -s], [s, c]], dtype=F64)


def rope_matrix(d_head, pos, thetas, pairing):
    """R_{Theta,pos}: block n is the 2-D rotation by pos * theta_n."""
    R = np.zeros((d_head, d_head), dtype=F64)
    for n, (a, b) in enumerate(rope_pairs(d_head, pairing)):
        blk = rot2(pos * thetas[n])
        R[np.ix_([a, b], [a, b])] = blk
    return R


def apply_rope(x, positions, thetas, pairing):
    """x: [L, d_head] rows; row i is multiplied by R_{Theta, positions[i]}."""
    out = np.empty_like(x, dtype=F64)
    for i, pos in enumerate(positions):
        out[i] = x[i] @ rope_matrix(x.shape[1], pos, thetas, pairing)
    return out


# --------------------------------------------------------------------------- #
# building the transforms
# --------------------------------------------------------------------------- #
def make_tk_head(phi, s, pairing, reflect=None):
    """(T_k^(h), T-bar_k^(h)) for one kv head.

    phi, s: N = d_head/2 angles and scales.  `s` may also have length d_head
    (one scale per coordinate) and `reflect` may mark blocks to build as
    reflections: both break Theorem 1 and exist for the negative tests.
    """
    phi = np.asarray(phi, dtype=F64)
    s = np.asarray(s, dtype=F64)
    n = phi.shape[0]
    d = 2 * n
    T = np.zeros((d, d), dtype=F64)
    Tb = np.zeros((d, d), dtype=F64)
    for i, (a, b) in enumerate(rope_pairs(d, pairing)):
        blk = rot2(phi[i])
        if reflect is not None and reflect[i]:
            blk = blk @ np.array([[1.0, 0.0], [0.0, -1.0]])
        sa, sb = (s[i], s[i]) if s.shape[0] == n else (s[a], s[b])
        S = np.diag([sa, sb])
        Si = np.diag([1.0 / sa, 1.0 / sb])
        T[np.ix_([a, b], [a, b])] = S @ blk
        Tb[np.ix_([a, b], [a, b])] = Si @ blk
    return T, Tb


def fold_rows(w_stored, blocks, d_head, repeat=1):
    """paper W <- W blockdiag(blocks, each repeated `repeat` times).

    On the stored [out, in] matrix head j's d_head rows become B^T @ rows with
    B = blocks[j // repeat].
    """
    w = np.array(w_stored, dtype=F64, copy=True)
    heads = w.shape[0] // d_head
    assert heads == len(blocks) * repeat
    for j in range(heads):
        B = np.asarray(blocks[j // repeat], dtype=F64)
        rows = slice(j * d_head, (j + 1) * d_head)
        w[rows] = B.T @ w[rows]
    return w


def fold_cols(w_stored, blocks, d_head, repeat=1):
    """paper W <- blockdiag(blocks, each repeated) W.

    On the stored [out, in] matrix head j's d_head columns become cols @ B^T.
    """
    w = np.array(w_stored, dtype=F64, copy=True)
    heads = w.shape[1] // d_head
    assert heads == len(blocks) * repeat
    for j in range(heads):
        B = np.asarray(blocks[j // repeat], dtype=F64)
        cols = slice(j * d_head, (j + 1) * d_head)
        w[:, cols] = w[:, cols] @ B.T
    return w


def fold_attention(wq, wk, wv, wo, d_head, m, tk=None, tkbar=None, tv=None):
    """Merge (T_k, T-bar_k) into (W_k, W_q) and (T_v, T_v^-1) into (W_v, W_o)."""
    wq2, wk2, wv2, wo2 = (np.array(a, dtype=F64, copy=True) for a in (wq, wk, wv, wo))
    if tk is not None:
        wk2 = fold_rows(wk2, tk, d_head, 1)
        wq2 = fold_rows(wq2, tkbar, d_head, m)
    if tv is not None:
        wv2 = fold_rows(wv2, tv, d_head, 1)
        inv = [np.linalg.inv(np.asarray(t, dtype=F64)) for t in tv]
        wo2 = fold_cols(wo2, inv, d_head, m)
    return wq2, wk2, wv2, wo2


# --------------------------------------------------------------------------- #
# float64 references used to show function preservation
# --------------------------------------------------------------------------- #
def attention_logits(x, wq, wk, d_head, m, positions, thetas, pairing):
    """[mH, L, L] pre-softmax logits <f(x_i W_q, i), f(x_j W_k, j)> (unscaled)."""
    x = np.asarray(x, dtype=F64)
    q = x @ np.asarray(wq, dtype=F64).T
    k = x @ np.asarray(wk, dtype=F64).T
    n_q = q.shape[1] // d_head
    out = []
    for j in range(n_q):
        h = j // m
        qj = apply_rope(q[:, j * d_head:(j + 1) * d_head], positions, thetas, pairing)
        kh = apply_rope(k[:, h * d_head:(h + 1) * d_head], positions, thetas, pairing)
        out.append(qj @ kh.T)
    return np.stack(out)


def attention_block(x, wq, wk, wv, wo, d_head, m, positions, thetas, pairing, causal=True):
    """softmax(QK^T / sqrt(d)) V W_o with grouped-query heads, float64."""
    x = np.asarray(x, dtype=F64)
    L = x.shape[0]
    logits = attention_logits(x, wq, wk, d_head, m, positions, thetas, pairing) / np.sqrt(d_head)
    if causal:
        mask = np.triu(np.ones((L, L), dtype=bool), k=1)
        logits = np.where(mask[None], -np.inf, logits)
    logits = logits - logits.max(axis=-1, keepdims=True)
    a = np.exp(logits)
    a = a / a.sum(axis=-1, keepdims=True)
    v = x @ np.asarray(wv, dtype=F64).T
    heads = []
    for j in range(a.shape[0]):
        h = j // m
        heads.append(a[j] @ v[:, h * d_head:(h + 1) * d_head])
    o = np.concatenate(heads, axis=1)
    return o @ np.asarray(wo, dtype=F64).T


def rms(x, eps=0.0):
    """||x||_R per row (with an optional eps under the root)."""
    x = np.asarray(x, dtype=F64)
    return np.sqrt(np.mean(x * x, axis=1) + eps)


def swiglu_mlp(xn, wg, wu, wd, mid_scale=None):
    """down(silu(gate(x)) * up(x)); `mid_scale` multiplies the product per token."""
    g = xn @ np.asarray(wg, dtype=F64).T
    u = xn @ np.asarray(wu, dtype=F64).T
    h = g / (1.0 + np.exp(-g)) * u
    if mid_scale is not None:
        h = h * mid_scale[:, None]
    return h @ np.asarray(wd, dtype=F64).T


def plain_forward(x1, blocks):
    """Pre-norm residual network: X_{n+1} = Z_n = X_n + F_n(RMSNorm(X_n)).  Returns all Z_n."""
    x = np.asarray(x1, dtype=F64)
    zs = []
    for f in blocks:
        xn = x / rms(x)[:, None]
        x = x + f(xn, None)
        zs.append(x)
    return zs


def residual_scaling_forward(x1, blocks):
    """The same network in the normalised-residual form (Sec. 3.1.3).

    Z~_0 = X_1, S_0 = 1; S_n = S_{n-1} / ||Z~_{n-1}||_R; X~_n = Z~_{n-1} / ||Z~_{n-1}||_R;
    the block output is produced already multiplied by S_n (each block applies
    the scale inside itself, where it commutes with the bias-free linear);
    Z~_n = X~_n + Y~_n.  Returns ([Z~_n], [S_n]).
    """
    zt = np.asarray(x1, dtype=F64)
    s = np.ones(zt.shape[0], dtype=F64)
    zts, ss = [], []
    for f in blocks:
        rho = rms(zt)
        xt = zt / rho[:, None]
        s = s / rho
        zt = xt + f(xt, s)
        zts.append(zt)
        ss.append(s)
    return zts, ss
