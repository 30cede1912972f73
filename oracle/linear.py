"""The composed entry points of the path, built from the single steps.

Test infrastructure (see the package header).

w4a4_linear : per-token scale + static quantise -> INT4 matmul -> scale factors
              (Sec. 3.1.3; App. B "Static quantization"; App. J "Setup")
decoder_mlp : one SwiGLU MLP block in the normalised-residual form of Sec. 3.1.3
              X~_n = RMSNorm(Z~_{n-1}),  S_n = S_{n-1} / ||Z~_{n-1}||_R   (Eq. 7)
              g, u = W4A4 linears of X~_n
              m    = bf16(silu(g) * u), quantised after the multiply by S_n
                     (the scaler placed at the down-projection input)
              Y~_n = W4A4 down projection of S_n * m  (= S_n * Y_n, Eq. 5)
              Z~_n = X~_n + Y~_n   when the residual is requested
decoder_attn_qkv / decoder_attn_out : the attention block in the same form, split around the
              attention itself (which stays in 16-bit floating point, App. J "Setup"):
              X~_n = RMSNorm(Z~_{n-1}),  S_n = S_{n-1} / ||Z~_{n-1}||_R,  QKV = W4A4 linear of X~_n;
              then, with the scaler at the attention output ("ap", App. A placement table):
              Y~_n = W4A4 output projection of S_n * A  (= S_n * Y_n, Eq. 5),  Z~_n = X~_n + Y~_n
"""
import numpy as np

from .quantizers import QParams, act_quant, act_quant_dynamic, silu_mul_quant
from .int_matmul import int_matmul
from .epilogue import dequant_epilogue, inverse_of_pre
from .hadamard import block_hadamard_f32

F32 = np.float32

POST_NONE = 0
POST_INVERSE_OF_PRE = 1
POST_VECTOR = 2


def w4a4_linear(x, wq, sw, qp, rmsnorm=True, scale_input=False, eps=1e-5, s_in=None,
                post_mode=POST_NONE, post=None):
    """Returns dict(codes, acc, y, s_out, p)."""
    codes, s_out, p, r = act_quant(x, qp, rmsnorm, scale_input, eps, s_in)
    acc = int_matmul(codes, wq, qp.z)
    if post_mode == POST_NONE:
        pv = None
    elif post_mode == POST_INVERSE_OF_PRE:
        pv = inverse_of_pre(p)
    else:
        pv = np.asarray(post, dtype=F32)
    y = dequant_epilogue(acc, sw, qp.scale, pv)
    return dict(codes=codes, acc=acc, y=y, s_out=s_out, p=p, r=r)


def decoder_mlp(x, wg_q, sw_g, wu_q, sw_u, wd_q, sw_d, qp_in, qp_mid, eps=1e-5,
                s_prev=None, add_residual=False, hadamard=False):
    """Returns dict(xq, g, u, m, mq, y, s_out).

    hadamard=True inserts the online block-wise Hadamard transform at the down-projection input
    (Sec. 3.1, last paragraph): the grid sees S_n * H(m) instead of S_n * m; `wd_q` must then be
    the quantised down projection with the inverse transform merged into it."""
    xq, s_n, p, r = act_quant(x, qp_in, rmsnorm=True, scale_input=False, eps=eps, s_in=s_prev)
    g = dequant_epilogue(int_matmul(xq, wg_q, qp_in.z), sw_g, qp_in.scale)
    u = dequant_epilogue(int_matmul(xq, wu_q, qp_in.z), sw_u, qp_in.scale)
    mq, m = silu_mul_quant(g, u, qp_mid, s_n)
    if hadamard:
        h = block_hadamard_f32(m)
        mq, _, _, _ = act_quant(h, qp_mid, rmsnorm=False, scale_input=True, s_in=s_n)
    acc_d = int_matmul(mq, wd_q, qp_mid.z)
    res = None
    if add_residual:
        res = (np.asarray(x, dtype=F32) * r[:, None]).astype(F32)     # X~_n = Z~_{n-1} / rho
    y = dequant_epilogue(acc_d, sw_d, qp_mid.scale, None, res)
    return dict(xq=xq, g=g, u=u, m=m, mq=mq, acc_d=acc_d, y=y, s_out=s_n, r=r)


def decoder_attn_qkv(x, wqkv_q, sw_qkv, qp_in, eps=1e-5, s_prev=None, wsum=None):
    """Returns dict(xq, acc, qkv, s_out, r).  `wqkv_q` holds the query, key and value rows with the
    mergeable transforms (Sec. 3.1.1, 3.1.2) already folded in; RMSNorm's output carries no
    per-token scale, so neither does QKV."""
    xq, s_n, p, r = act_quant(x, qp_in, rmsnorm=True, scale_input=False, eps=eps, s_in=s_prev)
    acc = int_matmul(xq, wqkv_q, qp_in.z)
    qkv = dequant_epilogue(acc, sw_qkv, qp_in.scale)
    return dict(xq=xq, acc=acc, qkv=qkv, s_out=s_n, r=r)


def decoder_attn_out(a, wo_q, sw_o, qp_ap, s_n, x=None, r=None):
    """Returns dict(aq, acc, y).  `a` is the attention output (bf16 values); the grid sees
    a * S_n; with `x` (the Z~_{n-1} that entered the block) and its `r`, the normalised residual
    X~_n = x * r is added in float32 before the one rounding to bf16."""
    aq, _, _, _ = act_quant(a, qp_ap, rmsnorm=False, scale_input=True, s_in=s_n)
    acc = int_matmul(aq, wo_q, qp_ap.z)
    res = None
    if x is not None:
        res = (np.asarray(x, dtype=F32) * np.asarray(r, dtype=F32)[:, None]).astype(F32)
    y = dequant_epilogue(acc, sw_o, qp_ap.scale, None, res)
    return dict(aq=aq, acc=acc, y=y)


def w4a4_linear_dynamic(x, wq, sw, bits=4, rmsnorm=True, scale_input=False, eps=1e-5, s_in=None,
                        post_mode=POST_NONE, post=None):
    """The linear with the dynamic activation quantiser (App. B "Dynamic quantization"; the second
    timing table of App. J): per-token grid D_t, integer matmul, and the scale factors
    y = bf16(((float)acc * sw[n]) * c_t) with c_t = D_t, D_t * (1/p_t) or D_t * post[t].
    Returns dict(codes, delta, acc, y, s_out, p, r)."""
    codes, delta, s_out, p, r = act_quant_dynamic(x, bits, rmsnorm, scale_input, eps, s_in)
    acc = int_matmul(codes, wq, 0)
    if post_mode == POST_NONE:
        c = delta
    elif post_mode == POST_INVERSE_OF_PRE:
        c = (delta * inverse_of_pre(p)).astype(F32)
    else:
        c = (delta * np.asarray(post, dtype=F32)).astype(F32)
    y = dequant_epilogue(acc, sw, 1.0, c)
    return dict(codes=codes, delta=delta, acc=acc, y=y, s_out=s_out, p=p, r=r)
