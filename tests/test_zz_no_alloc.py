"""fpt_w4a4_linear_static, the entry point for callers that cannot allocate device memory
(a runtime plug-in that only receives input/output pointers, a server whose memory pool is
frozen): it must give exactly what fpt_w4a4_linear gives -- and what the CPU oracle gives --
call after call, although its scratch is one array shared by every call and never cleared
between them.  The cases walk through every matmul route behind the entry point (CTA pairs,
one-CTA tiles, the 17..64-token weight-streaming kernel whose tile counters and partial sums
live in the shared array, the register kernel for at most 16 tokens), each right after a
larger call that left the array full of stale codes, counters and partial sums.

Collected last on purpose (file name): a run that stops at the first failure has then already
run every other test."""
import numpy as np
import pytest
import torch

from oracle import quantizers as OQ, linear as OL
from paper_2506_04985_b200 import binding as B, synth
from helpers import dev, host, oqp, bf16_host, assert_bf16_close, guarded_empty

pytestmark = pytest.mark.gpu


def _case(M, K, N, seed, flags, post_mode, symmetric, f16=False):
    x = synth.activations(M, K, seed, "noalloc/x", law="student_t3", outlier_frac=0.01, outlier_gain=40.0)
    w = synth.weights(N, K, 0.02, seed, "noalloc/w")
    s_in = synth.per_token_scale(M, seed, "noalloc/s")
    sdt = torch.float16 if f16 else torch.float32
    wq, sw, wsum = B.fpt_quantize_weights(dev(w), scale_dtype=sdt)
    qp = B.QParams(4, symmetric, 0.4 if flags & B.RMSNORM else 2.0, 0 if symmetric else 8)
    xd, sd = dev(x), dev(s_in)
    want_y, want_s = B.fpt_w4a4_linear(xd, wq, sw, qp, flags, 1e-5, s_in=sd, post_mode=post_mode, wsum=wsum)
    # outputs are the caller's; poisoned and between guard bands, so that a call that wrote nothing, or
    # past the end, is caught
    y = guarded_empty((M, N), torch.bfloat16)
    s = guarded_empty((M,), torch.float32)
    B.fpt_w4a4_linear_static(xd, wq, sw, qp, flags, 1e-5, s_in=sd, post_mode=post_mode, wsum=wsum, Y=y, s_out=s)
    torch.cuda.synchronize()
    assert np.array_equal(host(s), host(want_s))
    assert assert_bf16_close(bf16_host(y), bf16_host(want_y), "static-scratch linear vs workspace linear") == 0
    # ... and against the CPU oracle
    cw, d, _ = OQ.quantize_weights(synth.f32(w), scale_dtype="fp16" if f16 else "fp32")
    ref = OL.w4a4_linear(synth.f32(x), cw, d.astype(np.float32), oqp(qp), bool(flags & B.RMSNORM),
                         bool(flags & B.SCALE_INPUT), 1e-5, s_in.numpy(), post_mode)
    assert np.array_equal(host(s), ref["s_out"])
    assert assert_bf16_close(bf16_host(y), ref["y"], "static-scratch linear vs oracle") == 0


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    # first call fills the shared scratch with 300 x 1024 codes ...
    _case(300, 1024, 520, 3, B.RMSNORM, B.POST_INVERSE_OF_PRE, True)
    # ... the second, smaller and differently shaped, finds them there and must not be disturbed
    _case(130, 512, 264, 4, B.RMSNORM | B.SCALE_INPUT, B.POST_NONE, False)


def test_every_matmul_route_on_stale_scratch():
    _case(300, 4096, 520, 5, B.RMSNORM, B.POST_NONE, True)                     # CTA pairs; leaves 600 KB of codes
    _case(40, 4096, 1024, 6, B.RMSNORM, B.POST_INVERSE_OF_PRE, True)           # 17..64 tokens: ranges split tiles
    _case(40, 4096, 1024, 6, B.RMSNORM, B.POST_INVERSE_OF_PRE, True)           # the same again: counters back at zero
    _case(300, 1024, 264, 7, B.SCALE_INPUT, B.POST_NONE, False)
    _case(8, 2048, 1040, 8, B.RMSNORM | B.SCALE_INPUT, B.POST_NONE, True, f16=True)   # register kernel, fp16 scales
    _case(64, 1024, 136, 9, B.RMSNORM, B.POST_NONE, False)
    _case(100, 1024, 264, 10, B.RMSNORM, B.POST_NONE, True)                    # 65..128 tokens
    _case(100, 512, 128, 11, B.SCALE_INPUT, B.POST_INVERSE_OF_PRE, True, f16=True)    # one-CTA tiles (N <= 128)
    _case(17, 14336, 512, 12, B.RMSNORM, B.POST_NONE, True)                    # long rows, few tiles: many partial sums


def test_size_beyond_the_built_in_scratch_is_refused_before_any_launch():
    M, K, N = 8192, 8192, 8          # 32 MiB of codes: more than the array holds
    assert B.fpt_workspace_bytes(B.OP_LINEAR, M, N, K) > B.STATIC_SCRATCH_BYTES
    x = torch.zeros((M, K), dtype=torch.bfloat16, device="cuda")
    wq = torch.zeros((N, K // 2), dtype=torch.uint8, device="cuda")
    sw = torch.ones((N,), dtype=torch.float32, device="cuda")
    y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.FptError) as e:
        B.fpt_w4a4_linear_static(x, wq, sw, B.QParams(4, True, 1.0, 0), Y=y)
    assert e.value.code == B.ERR_WORKSPACE
