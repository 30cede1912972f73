"""ctypes binding of the C-ABI library (include/fpt.h): argument marshalling only.

Every function has the name of the C entry point it calls and takes torch CUDA tensors
where the C function takes device pointers.  torch is used for device memory and the
current stream, nothing else; no step of the path runs in Python or in torch ops.
A missing or unloadable library raises at first use: there is no fallback.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfpt_b200.so")

OK = 0
ERR_BAD_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = -1, -2, -3, -4, -5, -6
DTYPE_BF16, DTYPE_F32, DTYPE_F16 = 0, 1, 2
RANGE_MINMAX, RANGE_LP = 0, 1
RMSNORM, SCALE_INPUT, SILU_MUL, GU_INTERLEAVED = 1, 2, 4, 8
POST_NONE, POST_INVERSE_OF_PRE, POST_VECTOR = 0, 1, 2
OP_LINEAR, OP_MLP, OP_GEMM, OP_GEMM_A8, OP_LINEAR_A8, OP_MLP_HADAMARD = 0, 1, 2, 3, 4, 5

EXPORTS = ["fpt_version", "fpt_strerror", "fpt_quantize_weights", "fpt_interleave_gate_up", "fpt_act_quant", "fpt_hadamard_quant",
           "fpt_w4a4_gemm", "fpt_w4a4_linear", "fpt_w4a4_linear_static", "fpt_decoder_mlp", "fpt_decoder_attn_qkv",
           "fpt_decoder_attn_out", "fpt_act_quant_dynamic", "fpt_w4a4_linear_dynamic", "fpt_w4a8_gemm", "fpt_workspace_bytes",
           "fpt_reset_status",
           "fpt_check_status", "fpt_probe_mma", "fpt_set_programmatic_launch", "fpt_selftest_wait_timeout"]


class QParams(ctypes.Structure):
    """Mirror of `fpt_qparams`."""
    _fields_ = [("bits", ctypes.c_int), ("symmetric", ctypes.c_int), ("scale", ctypes.c_float),
                ("zero_point", ctypes.c_int)]

    def __init__(self, bits=4, symmetric=True, scale=1.0, zero_point=0):
        super().__init__(int(bits), int(bool(symmetric)), float(scale), int(zero_point))


class FptError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


_lib = None
_allocator = None


def set_allocator(fn):
    """Routes every device allocation of this module through `fn(shape, dtype, device) -> tensor`
    (None: plain torch.empty).  The GPU tests install one that surrounds each buffer with guard bands."""
    global _allocator
    _allocator = fn


def _empty(shape, dtype, device):
    if _allocator is not None:
        return _allocator(shape, dtype, device)
    return torch.empty(shape, dtype=dtype, device=device)


def lib():
    """The loaded shared library (loads it on first use; raises if it is not there)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2506_04985_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        vp, ci, cf, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
        qp = ctypes.POINTER(QParams)
        L.fpt_version.restype = ci
        L.fpt_strerror.restype = ctypes.c_char_p
        L.fpt_strerror.argtypes = [ci]
        L.fpt_quantize_weights.argtypes = [vp, vp, ci, ci, ci, qp, ci, cf, ci, vp, vp, vp]
        L.fpt_interleave_gate_up.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, vp, vp]
        L.fpt_act_quant.argtypes = [vp, vp, ci, ci, ci, qp, ci, cf, vp, vp, vp, vp]
        L.fpt_w4a4_gemm.argtypes = [vp, vp, vp, ci, ci, ci, vp, ci, vp, cf, ci, ci, vp, vp, vp, vp, vp, vp, sz]
        L.fpt_w4a4_linear.argtypes = [vp, vp, ci, ci, vp, vp, ci, vp, ci, qp, ci, cf, vp, ci, vp, vp, vp, vp, sz]
        L.fpt_w4a4_linear_static.argtypes = [vp, vp, ci, ci, vp, vp, ci, vp, ci, qp, ci, cf, vp, ci, vp, vp, vp]
        L.fpt_decoder_mlp.argtypes = [vp, vp, ci, ci, ci, vp, vp, vp, vp, ci, qp, qp, cf, vp, vp, ci, ci, vp, vp, sz]
        L.fpt_hadamard_quant.argtypes = [vp, vp, ci, ci, ci, qp, ci, vp, vp]
        L.fpt_w4a8_gemm.argtypes = [vp, vp, vp, ci, ci, ci, vp, ci, cf, vp, vp, vp, vp, vp, vp, sz]
        L.fpt_act_quant_dynamic.argtypes = [vp, vp, ci, ci, ci, ci, ci, cf, vp, vp, vp, vp]
        L.fpt_w4a4_linear_dynamic.argtypes = [vp, vp, ci, ci, vp, vp, ci, ci, ci, ci, cf, vp, ci, vp, vp, vp, vp, sz]
        L.fpt_decoder_attn_qkv.argtypes = [vp, vp, ci, ci, vp, vp, ci, vp, ci, qp, cf, vp, vp, vp, vp, vp, sz]
        L.fpt_decoder_attn_out.argtypes = [vp, vp, ci, ci, vp, vp, ci, vp, ci, qp, vp, vp, vp, vp, vp, sz]
        L.fpt_workspace_bytes.restype = sz
        L.fpt_workspace_bytes.argtypes = [ci, ci, ci, ci]
        L.fpt_reset_status.argtypes = [vp, vp]
        L.fpt_check_status.argtypes = [vp, vp]
        L.fpt_set_programmatic_launch.argtypes = [ci]
        L.fpt_selftest_wait_timeout.argtypes = [vp, vp, ctypes.c_uint, vp]
        L.fpt_probe_mma.argtypes = [vp, ci, ci, ci, ci, ci, ci, vp, vp]
        for name in EXPORTS:
            if name not in ("fpt_strerror", "fpt_workspace_bytes", "fpt_version"):
                getattr(L, name).restype = ci
        _lib = L
    return _lib


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(code, where):
    if code != OK:
        raise FptError(code, where)


def _scale_dtype(t):
    return {torch.float32: DTYPE_F32, torch.float16: DTYPE_F16}[t.dtype]


def fpt_version():
    return lib().fpt_version()


def strerror(code):
    return lib().fpt_strerror(code).decode()


def fpt_workspace_bytes(op, M, N, K):
    return int(lib().fpt_workspace_bytes(op, M, N, K))


def new_workspace(op, M, N, K, device="cuda"):
    """Allocates a workspace of the required size and clears its status word."""
    ws = _empty(max(fpt_workspace_bytes(op, M, N, K), 256), dtype=torch.uint8, device=device)
    _check(lib().fpt_reset_status(_stream(), _ptr(ws)), "fpt_reset_status")
    return ws


def fpt_check_status(ws):
    return lib().fpt_check_status(_stream(), _ptr(ws))


def fpt_quantize_weights(W, qp=None, range_mode=RANGE_MINMAX, p=3.0, scale_dtype=torch.float32, want_wsum=True):
    """W [N, K] bf16/f32 -> (Wq uint8 [N, K/2], sw [N], wsum int32 [N] or None)."""
    qp = qp or QParams()
    N, K = W.shape
    Wq = _empty((N, K // 2), dtype=torch.uint8, device=W.device)
    sw = _empty((N,), dtype=scale_dtype, device=W.device)
    wsum = _empty((N,), dtype=torch.int32, device=W.device) if want_wsum else None
    wd = {torch.bfloat16: DTYPE_BF16, torch.float32: DTYPE_F32}[W.dtype]
    _check(lib().fpt_quantize_weights(_stream(), _ptr(W), wd, N, K, ctypes.byref(qp), range_mode, p,
                                      _scale_dtype(sw), _ptr(Wq), _ptr(sw), _ptr(wsum)), "fpt_quantize_weights")
    return Wq, sw, wsum


def fpt_interleave_gate_up(Wg_q, Wu_q, sw_g, sw_u):
    d_ff, kb = Wg_q.shape
    Wgu = _empty((2 * d_ff, kb), dtype=torch.uint8, device=Wg_q.device)
    sw = _empty((2 * d_ff,), dtype=sw_g.dtype, device=Wg_q.device)
    _check(lib().fpt_interleave_gate_up(_stream(), _ptr(Wg_q), _ptr(Wu_q), _ptr(sw_g), _ptr(sw_u),
                                        _scale_dtype(sw_g), d_ff, kb * 2, _ptr(Wgu), _ptr(sw)),
           "fpt_interleave_gate_up")
    return Wgu, sw


def fpt_act_quant(X, qp, flags=RMSNORM, eps=1e-5, X2=None, s_in=None, K=None, want_s_out=True, out=None):
    """X [M, ldx] bf16 -> (Xq uint8 [M, K/2], s_out f32 [M] or None)."""
    M, ldx = X.shape
    if K is None:
        K = ldx // 2 if (flags & GU_INTERLEAVED) else ldx
    if out is not None:
        Xq = out
    elif qp.bits == 8:
        Xq = _empty((M, K), dtype=torch.int8, device=X.device)
    else:
        Xq = _empty((M, K // 2), dtype=torch.uint8, device=X.device)
    s_out = _empty((M,), dtype=torch.float32, device=X.device) if want_s_out else None
    _check(lib().fpt_act_quant(_stream(), _ptr(X), M, K, ldx, ctypes.byref(qp), flags, eps, _ptr(X2), _ptr(s_in),
                               _ptr(Xq), _ptr(s_out)), "fpt_act_quant")
    return Xq, s_out


def fpt_w4a4_gemm(Xq, Wq, sw, act_scale, wsum=None, act_symmetric=True, act_zero_point=0, post=None, residual=None,
                  res_scale=None, want_y=True, want_acc=False, ws=None, Y=None):
    """Packed x packed matmul + scale factors -> (Y bf16 [M, N] or None, acc int32 [M, N] or None)."""
    M, kb = Xq.shape
    N = Wq.shape[0]
    K = kb * 2
    if ws is None:
        ws = new_workspace(OP_GEMM, M, N, K, Xq.device)
    if Y is None and want_y:
        Y = _empty((M, N), dtype=torch.bfloat16, device=Xq.device)
    acc = _empty((M, N), dtype=torch.int32, device=Xq.device) if want_acc else None
    _check(lib().fpt_w4a4_gemm(_stream(), _ptr(Xq), _ptr(Wq), M, N, K, _ptr(sw), _scale_dtype(sw), _ptr(wsum),
                               float(act_scale), int(bool(act_symmetric)), int(act_zero_point), _ptr(post),
                               _ptr(residual), _ptr(res_scale), _ptr(Y), _ptr(acc), _ptr(ws), ws.numel()),
           "fpt_w4a4_gemm")
    return Y, acc


def fpt_w4a4_linear(X, Wq, sw, qp, flags=RMSNORM, eps=1e-5, s_in=None, post_mode=POST_NONE, post=None, wsum=None,
                    want_s_out=True, ws=None, Y=None):
    """One W4A4 linear on bf16 activations -> (Y bf16 [M, N], s_out f32 [M] or None)."""
    M, K = X.shape
    N = Wq.shape[0]
    if ws is None:
        ws = new_workspace(OP_LINEAR_A8 if qp.bits == 8 else OP_LINEAR, M, N, K, X.device)
    if Y is None:
        Y = _empty((M, N), dtype=torch.bfloat16, device=X.device)
    s_out = _empty((M,), dtype=torch.float32, device=X.device) if want_s_out else None
    _check(lib().fpt_w4a4_linear(_stream(), _ptr(X), M, K, _ptr(Wq), _ptr(sw), _scale_dtype(sw), _ptr(wsum), N,
                                 ctypes.byref(qp), flags, eps, _ptr(s_in), post_mode, _ptr(post), _ptr(Y),
                                 _ptr(s_out), _ptr(ws), ws.numel()), "fpt_w4a4_linear")
    return Y, s_out


STATIC_SCRATCH_BYTES = 17 * 1024 * 1024


def fpt_w4a4_linear_static(X, Wq, sw, qp, flags=RMSNORM, eps=1e-5, s_in=None, post_mode=POST_NONE, post=None,
                           wsum=None, Y=None, s_out=None):
    """fpt_w4a4_linear on the library's built-in scratch: the call allocates nothing, so the
    caller passes every output (Y bf16 [M, N]; s_out f32 [M] or None).  For callers that cannot
    allocate device memory; M x K is limited by STATIC_SCRATCH_BYTES and calls must not overlap
    on the GPU.  Returns (Y, s_out)."""
    M, K = X.shape
    N = Wq.shape[0]
    _check(lib().fpt_w4a4_linear_static(_stream(), _ptr(X), M, K, _ptr(Wq), _ptr(sw), _scale_dtype(sw), _ptr(wsum),
                                        N, ctypes.byref(qp), flags, eps, _ptr(s_in), post_mode, _ptr(post), _ptr(Y),
                                        _ptr(s_out)), "fpt_w4a4_linear_static")
    return Y, s_out


def fpt_hadamard_quant(X, qp, flags=SCALE_INPUT, s_in=None, K=None, out=None):
    """X [M, ldx] bf16 (products, or gate||up with SILU_MUL | GU_INTERLEAVED) -> Xq uint8 [M, K/2]."""
    M, ldx = X.shape
    if K is None:
        K = ldx // 2 if (flags & GU_INTERLEAVED) else ldx
    Xq = out if out is not None else _empty((M, K // 2), dtype=torch.uint8, device=X.device)
    _check(lib().fpt_hadamard_quant(_stream(), _ptr(X), M, K, ldx, ctypes.byref(qp), flags, _ptr(s_in), _ptr(Xq)),
           "fpt_hadamard_quant")
    return Xq


def fpt_decoder_mlp(X, Wgu_q, sw_gu, Wd_q, sw_d, qp_in, qp_mid, eps=1e-5, s_prev=None, add_residual=False,
                    want_s_out=True, ws=None, Y=None, mid_hadamard=False):
    """One SwiGLU MLP block -> (Y bf16 [M, d], s_out f32 [M] or None)."""
    M, d = X.shape
    d_ff = Wgu_q.shape[0] // 2
    if ws is None:
        ws = new_workspace(OP_MLP_HADAMARD if mid_hadamard else OP_MLP, M, d_ff, d, X.device)
    if Y is None:
        Y = _empty((M, d), dtype=torch.bfloat16, device=X.device)
    s_out = _empty((M,), dtype=torch.float32, device=X.device) if want_s_out else None
    _check(lib().fpt_decoder_mlp(_stream(), _ptr(X), M, d, d_ff, _ptr(Wgu_q), _ptr(sw_gu), _ptr(Wd_q), _ptr(sw_d),
                                 _scale_dtype(sw_gu), ctypes.byref(qp_in), ctypes.byref(qp_mid), eps, _ptr(s_prev),
                                 _ptr(s_out), int(bool(add_residual)), int(bool(mid_hadamard)), _ptr(Y), _ptr(ws),
                                 ws.numel()),
           "fpt_decoder_mlp")
    return Y, s_out


def fpt_decoder_attn_qkv(X, Wqkv_q, sw_qkv, qp_in, eps=1e-5, s_prev=None, wsum=None, ws=None, QKV=None):
    """First half of the attention block -> (QKV bf16 [M, n_qkv], S_n f32 [M], r f32 [M])."""
    M, d = X.shape
    n_qkv = Wqkv_q.shape[0]
    if ws is None:
        ws = new_workspace(OP_LINEAR, M, n_qkv, d, X.device)
    if QKV is None:
        QKV = _empty((M, n_qkv), dtype=torch.bfloat16, device=X.device)
    s_out = _empty((M,), dtype=torch.float32, device=X.device)
    r_out = _empty((M,), dtype=torch.float32, device=X.device)
    _check(lib().fpt_decoder_attn_qkv(_stream(), _ptr(X), M, d, _ptr(Wqkv_q), _ptr(sw_qkv), _scale_dtype(sw_qkv),
                                      _ptr(wsum), n_qkv, ctypes.byref(qp_in), eps, _ptr(s_prev), _ptr(s_out),
                                      _ptr(r_out), _ptr(QKV), _ptr(ws), ws.numel()), "fpt_decoder_attn_qkv")
    return QKV, s_out, r_out


def fpt_decoder_attn_out(A, Wo_q, sw_o, qp_ap, s_n, X=None, r=None, wsum=None, ws=None, Y=None):
    """Second half of the attention block: scaler at the attention output, output projection,
    optional normalised residual -> Y bf16 [M, d]."""
    M, k_o = A.shape
    d = Wo_q.shape[0]
    if ws is None:
        ws = new_workspace(OP_LINEAR, M, d, k_o, A.device)
    if Y is None:
        Y = _empty((M, d), dtype=torch.bfloat16, device=A.device)
    _check(lib().fpt_decoder_attn_out(_stream(), _ptr(A), M, k_o, _ptr(Wo_q), _ptr(sw_o), _scale_dtype(sw_o), _ptr(wsum),
                                      d, ctypes.byref(qp_ap), _ptr(s_n), _ptr(X), _ptr(r), _ptr(Y), _ptr(ws),
                                      ws.numel()), "fpt_decoder_attn_out")
    return Y


def fpt_act_quant_dynamic(X, bits=4, flags=RMSNORM, eps=1e-5, s_in=None, want_s_out=True, out=None):
    """Dynamic per-token grid -> (codes uint8 [M, K/2] or int8 [M, K], s_out f32 [M] or None, delta f32 [M])."""
    M, K = X.shape
    if out is None:
        out = (_empty((M, K // 2), dtype=torch.uint8, device=X.device) if bits == 4
               else _empty((M, K), dtype=torch.int8, device=X.device))
    s_out = _empty((M,), dtype=torch.float32, device=X.device) if want_s_out else None
    delta = _empty((M,), dtype=torch.float32, device=X.device)
    _check(lib().fpt_act_quant_dynamic(_stream(), _ptr(X), M, K, X.stride(0), bits, flags, eps, _ptr(s_in), _ptr(out),
                                       _ptr(s_out), _ptr(delta)), "fpt_act_quant_dynamic")
    return out, s_out, delta


def fpt_w4a4_linear_dynamic(X, Wq, sw, bits=4, flags=RMSNORM, eps=1e-5, s_in=None, post_mode=POST_NONE, post=None,
                            want_s_out=True, ws=None, Y=None):
    """One linear with the dynamic activation grid -> (Y bf16 [M, N], s_out f32 [M] or None)."""
    M, K = X.shape
    N = Wq.shape[0]
    if ws is None:
        ws = new_workspace(OP_LINEAR_A8 if bits == 8 else OP_LINEAR, M, N, K, X.device)
    if Y is None:
        Y = _empty((M, N), dtype=torch.bfloat16, device=X.device)
    s_out = _empty((M,), dtype=torch.float32, device=X.device) if want_s_out else None
    _check(lib().fpt_w4a4_linear_dynamic(_stream(), _ptr(X), M, K, _ptr(Wq), _ptr(sw), _scale_dtype(sw), N, bits, flags,
                                         eps, _ptr(s_in), post_mode, _ptr(post), _ptr(Y), _ptr(s_out), _ptr(ws),
                                         ws.numel()), "fpt_w4a4_linear_dynamic")
    return Y, s_out


def fpt_w4a8_gemm(Xq8, Wq, sw, act_scale, post=None, residual=None, res_scale=None, want_y=True, want_acc=False,
                  ws=None, Y=None):
    """int8 [M, K] x packed 4-bit [N, K/2] matmul + scale factors -> (Y bf16 or None, acc int32 or None)."""
    M, K = Xq8.shape
    N = Wq.shape[0]
    if ws is None:
        ws = new_workspace(OP_GEMM_A8, M, N, K, Xq8.device)
    if Y is None and want_y:
        Y = _empty((M, N), dtype=torch.bfloat16, device=Xq8.device)
    acc = _empty((M, N), dtype=torch.int32, device=Xq8.device) if want_acc else None
    _check(lib().fpt_w4a8_gemm(_stream(), _ptr(Xq8), _ptr(Wq), M, N, K, _ptr(sw), _scale_dtype(sw), float(act_scale),
                               _ptr(post), _ptr(residual), _ptr(res_scale), _ptr(Y), _ptr(acc), _ptr(ws), ws.numel()),
           "fpt_w4a8_gemm")
    return Y, acc


def fpt_probe_mma(pair, n, n_acc, a_in_tmem, iters, ctas, ws=None, want_cycles=True):
    """Measurement aid: bare 8-bit integer tensor-core instructions (see fpt.h) -> cycles uint64 per CTA (pair) or None."""
    dev = torch.device("cuda", torch.cuda.current_device())
    if ws is None:
        ws = torch.zeros((8192,), dtype=torch.uint8, device=dev)
    cyc = torch.zeros((ctas // 2 if pair else ctas,), dtype=torch.int64, device=dev) if want_cycles else None
    _check(lib().fpt_probe_mma(_stream(), int(pair), n, n_acc, int(a_in_tmem), iters, ctas, _ptr(cyc), _ptr(ws)),
           "fpt_probe_mma")
    return cyc


def fpt_set_programmatic_launch(enabled):
    """Switches programmatic dependent launch of the library's kernels on or off; returns the previous setting."""
    return lib().fpt_set_programmatic_launch(int(bool(enabled)))


def fpt_selftest_wait_timeout(ws, limit_us=1000):
    """Runs the library's bounded wait on a barrier nothing arrives at -> uint32 tensor [1]: 1 if it gave up."""
    flag = torch.zeros((1,), dtype=torch.int32, device=ws.device)
    _check(lib().fpt_selftest_wait_timeout(_stream(), _ptr(ws), int(limit_us), _ptr(flag)), "fpt_selftest_wait_timeout")
    return flag
