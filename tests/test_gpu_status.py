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
