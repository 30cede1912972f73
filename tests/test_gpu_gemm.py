"""GPU parity of the packed INT4 matmul and its scale-factor epilogue against the oracle:
int32 accumulators bit-exact, bf16 outputs within 1 bf16 ulp (they are expected to be
identical, the operation order being the same)."""
import numpy as np
import pytest
import torch

from oracle import quantizers as OQ
from oracle.int_matmul import int_matmul
from oracle.epilogue import dequant_epilogue
from paper_2506_04985_b200 import binding as B
from helpers import dev, host, bf16_host, random_codes, packed_dev, assert_bf16_close

pytestmark = pytest.mark.gpu

SHAPES = [(128, 256, 128), (1, 8, 128), (64, 64, 128), (200, 384, 256), (129, 264, 512), (300, 1024, 1024),
          (17, 128, 384), (128, 72, 256), (257, 520, 128), (512, 768, 2048), (8, 14336, 1024), (130, 4096, 14336)]


def _run(M, N, K, symmetric=True, z=0, seed=0, post=False, residual=False, f16=False):
    rng = np.random.default_rng(seed + M + N + K)
    qa = random_codes(rng, (M, K), symmetric)
    qw = random_codes(rng, (N, K), True)
    sw = (np.exp(rng.standard_normal(N)) * 0.01).astype(np.float16 if f16 else np.float32)
    act_scale = np.float32(0.173)
    pv = np.exp(rng.standard_normal(M)).astype(np.float32) if post else None
    res = rs = None
    if residual:
        res = torch.from_numpy(rng.standard_normal((M, N)).astype(np.float32)).to(torch.bfloat16)
        rs = np.exp(rng.standard_normal(M)).astype(np.float32)
    wsum = qw.astype(np.int64).sum(axis=1).astype(np.int32)
    Y, acc = B.fpt_w4a4_gemm(packed_dev(qa), packed_dev(qw), dev(sw), float(act_scale),
                             wsum=None if symmetric else dev(wsum), act_symmetric=symmetric, act_zero_point=z,
                             post=None if pv is None else dev(pv), residual=None if res is None else dev(res),
                             res_scale=None if rs is None else dev(rs), want_acc=True)
    ref_acc = int_matmul(qa, qw, z)
    assert np.array_equal(host(acc), ref_acc), "int32 accumulators differ"
    rres = None
    if residual:
        rres = (res.float().numpy() * rs[:, None]).astype(np.float32)
    ref_y = dequant_epilogue(ref_acc, sw.astype(np.float32), act_scale, pv, rres)
    nd = assert_bf16_close(bf16_host(Y), ref_y, f"Y {M}x{N}x{K}")
    assert nd == 0, f"{nd} outputs differ by one ulp although the operation order is the same"


@pytest.mark.parametrize("M,N,K", SHAPES)
def test_gemm_symmetric(M, N, K):
    _run(M, N, K)


@pytest.mark.parametrize("M,N,K", [(200, 384, 256), (64, 64, 128), (129, 264, 512)])
@pytest.mark.parametrize("z", [8, 3, 15, 0])
def test_gemm_asymmetric_activations(M, N, K, z):
    _run(M, N, K, symmetric=False, z=z)


@pytest.mark.parametrize("M,N,K", [(200, 384, 256), (33, 1024, 512)])
def test_gemm_post_residual_and_fp16_scales(M, N, K):
    _run(M, N, K, post=True)
    _run(M, N, K, post=True, residual=True)
    _run(M, N, K, residual=True, f16=True)


@pytest.mark.parametrize("M,N,K", [(256, 15392, 128), (256, 16576, 128), (256, 17760, 128), (300, 17768, 256),
                                   (200, 6152, 128), (513, 248, 256), (2048, 6144, 128)])
@pytest.mark.parametrize("extras", [False, True])
def test_gemm_wide_outputs_ragged_column_tiles(M, N, K, extras):
    """Wide outputs whose width is not a multiple of the 256-column tile (ragged last column tile, more
    column tiles than CTA pairs), with and without post scale, residual and the asymmetric grid."""
    _run(M, N, K, seed=5, post=extras, residual=extras, symmetric=not extras, z=9 if extras else 0)


def test_gemm_extreme_codes_reach_the_accumulator_bound():
    M, N, K = 130, 264, 28672
    qa = np.full((M, K), -8, dtype=np.int8)
    qw = np.full((N, K), -8, dtype=np.int8)
    qw[1::2] = 7
    sw = np.full(N, 2.0 ** -10, dtype=np.float32)
    _, acc = B.fpt_w4a4_gemm(packed_dev(qa), packed_dev(qw), dev(sw), 1.0, want_acc=True, want_y=False)
    acc = host(acc)
    assert np.all(acc[:, 0::2] == 64 * K) and np.all(acc[:, 1::2] == -56 * K)


def test_gemm_persistent_many_tiles_and_status_word():
    M, N, K = 1500, 2304, 512           # 12 x 9 tiles of 128 x 256: several per CTA is not reached on 148 SMs...
    _run(M, N, K, seed=5)
    M, N, K = 2200, 4352, 256           # 18 x 17 = 306 tiles: every CTA loops over at least two
    rng = np.random.default_rng(9)
    qa, qw = random_codes(rng, (M, K)), random_codes(rng, (N, K))
    sw = np.ones(N, dtype=np.float32)
    ws = B.new_workspace(B.OP_GEMM, M, N, K)
    _, acc = B.fpt_w4a4_gemm(packed_dev(qa), packed_dev(qw), dev(sw), 1.0, want_acc=True, want_y=False, ws=ws)
    assert B.fpt_check_status(ws) == B.OK
    assert np.array_equal(host(acc), int_matmul(qa, qw))


@pytest.mark.parametrize("residual", [False, True])
def test_gemm_many_rounds_per_cta_pair_repeatable_and_exact(residual):
    """Several tiles per CTA pair with the slow (residual) epilogue: results must not depend on timing
    (a register holding an in-flight tensor-memory load must never be spilled before its wait), and
    sampled rows must match the oracle."""
    M, N, K = 2048, 6144, 4096
    rng = np.random.default_rng(17)
    qa, qw = random_codes(rng, (M, K)), random_codes(rng, (N, K))
    sw = (np.exp(rng.standard_normal(N)) * 0.01).astype(np.float32)
    res = torch.from_numpy(rng.standard_normal((M, N)).astype(np.float32)).to(torch.bfloat16) if residual else None
    rs = np.exp(rng.standard_normal(M)).astype(np.float32) if residual else None
    xa, xw, xs = packed_dev(qa), packed_dev(qw), dev(sw)
    dres, drs = (dev(res), dev(rs)) if residual else (None, None)
    ws = B.new_workspace(B.OP_GEMM, M, N, K)
    outs = []
    for _ in range(4):
        Y, _ = B.fpt_w4a4_gemm(xa, xw, xs, 0.31, residual=dres, res_scale=drs, ws=ws)
        outs.append(Y.view(torch.int16).clone())
    assert B.fpt_check_status(ws) == B.OK
    for o in outs[1:]:
        assert torch.equal(o, outs[0]), "two launches on the same inputs gave different outputs"
    rows = np.array([0, 127, 128, 255, 256, 1023, 1024, 1791, 1792, 2047])
    acc = int_matmul(qa[rows], qw)
    rres = (res.float().numpy()[rows] * rs[rows, None]).astype(np.float32) if residual else None
    ref = dequant_epilogue(acc, sw, np.float32(0.31), None, rres)
    assert assert_bf16_close(bf16_host(outs[0].view(torch.bfloat16))[rows], ref, "Y rows") == 0


def test_gemm_random_shapes_all_kernels():
    """150 seeded random shapes (1 to 700 tokens, ragged widths, every K from 128 to 1536), symmetric and
    asymmetric grids, with and without post scale and residual: whichever kernel the dispatch picks, the
    accumulators equal the oracle's and the outputs match bit for bit."""
    rng = np.random.default_rng(77)
    for _ in range(150):
        M = int(rng.integers(1, 700))
        N = int(rng.integers(1, 90)) * 8
        K = int(rng.integers(1, 13)) * 128
        sym = bool(rng.integers(0, 3))
        _run(M, N, K, symmetric=sym, z=0 if sym else int(rng.integers(0, 16)), seed=int(rng.integers(0, 1000)),
             post=bool(rng.integers(0, 2)), residual=bool(rng.integers(0, 2)), f16=bool(rng.integers(0, 2)))
