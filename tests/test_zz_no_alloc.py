"""fpt_w4a4_linear_static, the entry point for callers that cannot allocate device memory
(a runtime plug-in that only receives input/output pointers, a server whose memory pool is
frozen): it must give exactly what fpt_w4a4_linear gives, call after call, although its
scratch is one array shared by every call and never cleared between them.

Collected last on purpose (file name): a run that stops at the first failure has then already
run every other test."""
import numpy as np
import pytest
import torch

from paper_2506_04985_b200 import binding as B, synth
from helpers import dev, host, bf16_host, assert_bf16_close

pytestmark = pytest.mark.gpu


def _case(M, K, N, seed, flags, post_mode, symmetric):
    x = dev(synth.activations(M, K, seed, "noalloc/x", law="student_t3", outlier_frac=0.01, outlier_gain=40.0))
    w = dev(synth.weights(N, K, 0.02, seed, "noalloc/w"))
    s_in = dev(synth.per_token_scale(M, seed, "noalloc/s"))
    wq, sw, wsum = B.fpt_quantize_weights(w)
    qp = B.QParams(4, symmetric, 0.4 if flags & B.RMSNORM else 2.0, 0 if symmetric else 8)
    want_y, want_s = B.fpt_w4a4_linear(x, wq, sw, qp, flags, 1e-5, s_in=s_in, post_mode=post_mode, wsum=wsum)
    # outputs are allocated here, by the caller; poison them so that a call that wrote nothing is caught
    y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    s = torch.full((M,), float("nan"), dtype=torch.float32, device="cuda")
    B.fpt_w4a4_linear_static(x, wq, sw, qp, flags, 1e-5, s_in=s_in, post_mode=post_mode, wsum=wsum, Y=y, s_out=s)
    torch.cuda.synchronize()
    assert np.array_equal(host(s), host(want_s))
    assert assert_bf16_close(bf16_host(y), bf16_host(want_y), "static-scratch linear") == 0


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    # first call fills the shared scratch with 300 x 1024 codes ...
    _case(300, 1024, 520, 3, B.RMSNORM, B.POST_INVERSE_OF_PRE, True)
    # ... the second, smaller and differently shaped, finds them there and must not be disturbed
    _case(130, 512, 264, 4, B.RMSNORM | B.SCALE_INPUT, B.POST_NONE, False)


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
