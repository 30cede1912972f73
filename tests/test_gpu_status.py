"""The status word of a workspace, host half: a kernel whose bounded wait gives up writes a non-zero
word at the head of the workspace; fpt_check_status turns that into FPT_ERR_TIMEOUT and
fpt_reset_status clears it.  Here the word is planted from the host: no device-side wait is made
to run out."""
import pytest
import torch

from paper_2506_04985_b200 import binding as B

pytestmark = pytest.mark.gpu


def test_planted_status_word_reads_as_timeout_and_reset_clears_it():
    ws = B.new_workspace(B.OP_GEMM, 300, 512, 256)
    assert B.fpt_check_status(ws) == B.OK
    ws[:4] = torch.tensor([0x05, 0x71, 0, 0], dtype=torch.uint8, device=ws.device)     # 0x7105: "role 5 gave up"
    torch.cuda.synchronize()
    assert B.fpt_check_status(ws) == B.ERR_TIMEOUT
    assert "wait" in B.strerror(B.ERR_TIMEOUT)
    assert B.lib().fpt_reset_status(B._stream(), B._ptr(ws)) == B.OK
    assert B.fpt_check_status(ws) == B.OK
    # the word alone decides: anything behind it (tile counters, scratch) does not
    ws[8:16] = 0xFF
    torch.cuda.synchronize()
    assert B.fpt_check_status(ws) == B.OK


def test_status_calls_refuse_a_null_workspace():
    assert B.lib().fpt_check_status(B._stream(), None) == B.ERR_BAD_ARG
    assert B.lib().fpt_reset_status(B._stream(), None) == B.ERR_BAD_ARG


def test_a_wait_that_runs_out_ends_the_kernel_and_sets_the_status_word():
    """The device half of the time-out path: the library's own wait routine, on a barrier nothing arrives
    at, with a 2 ms limit.  The kernel must end by itself, report that it gave up, and leave a code in the
    status word; the context stays usable."""
    import time
    ws = B.new_workspace(B.OP_GEMM, 300, 512, 256)
    t0 = time.perf_counter()
    flag = B.fpt_selftest_wait_timeout(ws, limit_us=2000)
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    assert int(flag.item()) == 1
    assert 0.0015 < dt < 1.0, dt
    assert B.fpt_check_status(ws) == B.ERR_TIMEOUT
    word = int(ws[:4].view(torch.int32).item())
    assert word == (0x7100 | 14)
    assert B.lib().fpt_reset_status(B._stream(), B._ptr(ws)) == B.OK
    assert B.fpt_check_status(ws) == B.OK
    # the context is fine: a real matmul right after
    x = torch.randint(0, 256, (300, 128), dtype=torch.uint8, device="cuda")
    w = torch.randint(0, 256, (512, 128), dtype=torch.uint8, device="cuda")
    sw = torch.ones((512,), dtype=torch.float32, device="cuda")
    B.fpt_w4a4_gemm(x, w, sw, 1.0, ws=ws)
    assert B.fpt_check_status(ws) == B.OK
