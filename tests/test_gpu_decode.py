"""GPU parity of the decode-size matmul (at most 64 tokens; weights streamed once, work split
evenly over the SMs, partial sums added as integers) against the oracle: int32 accumulators
bit-exact, bf16 outputs identical."""
import numpy as np
import pytest
import torch

from oracle.int_matmul import int_matmul
from oracle.epilogue import dequant_epilogue
from paper_2506_04985_b200 import binding as B
from helpers import dev, host, bf16_host, random_codes, packed_dev, assert_bf16_close

pytestmark = pytest.mark.gpu


def _run(M, N, K, symmetric=True, z=0, seed=0, post=False, residual=False, f16=True, ws=None, reps=1):
    rng = np.random.default_rng(seed + 7 * M + N + K)
    qa = random_codes(rng, (M, K), symmetric)
    qw = random_codes(rng, (N, K), True)
    sw = (np.exp(rng.standard_normal(N)) * 0.01).astype(np.float16 if f16 else np.float32)
    act_scale = np.float32(0.311)
    pv = np.exp(rng.standard_normal(M)).astype(np.float32) if post else None
    res = rs = None
    if residual:
        res = torch.from_numpy(rng.standard_normal((M, N)).astype(np.float32)).to(torch.bfloat16)
        rs = np.exp(rng.standard_normal(M)).astype(np.float32)
    wsum = qw.astype(np.int64).sum(axis=1).astype(np.int32)
    ref_acc = int_matmul(qa, qw, z)
    rres = (res.float().numpy() * rs[:, None]).astype(np.float32) if residual else None
    ref_y = dequant_epilogue(ref_acc, sw.astype(np.float32), act_scale, pv, rres)
    xa, xw, xs = packed_dev(qa), packed_dev(qw), dev(sw)
    for _ in range(reps):          # the same workspace again: its tile counters must be back at zero
        Y, acc = B.fpt_w4a4_gemm(xa, xw, xs, float(act_scale), wsum=None if symmetric else dev(wsum),
                                 act_symmetric=symmetric, act_zero_point=z, post=None if pv is None else dev(pv),
                                 residual=None if res is None else dev(res), res_scale=None if rs is None else dev(rs),
                                 want_acc=True, ws=ws)
        assert np.array_equal(host(acc), ref_acc), f"int32 accumulators differ {M}x{N}x{K}"
        assert assert_bf16_close(bf16_host(Y), ref_y, f"Y {M}x{N}x{K}") == 0
    if ws is not None:
        assert B.fpt_check_status(ws) == B.OK


@pytest.mark.parametrize("M", [1, 2, 8, 16, 17, 32, 33, 64])
@pytest.mark.parametrize("N,K", [(128, 128), (264, 512), (1024, 2048), (72, 384)])
def test_decode_shapes(M, N, K):
    _run(M, N, K)


@pytest.mark.parametrize("M", [1, 8, 32, 64])
@pytest.mark.parametrize("N,K", [(14336, 4096), (4096, 14336)])
def test_decode_llama_mlp_shapes_full_size(M, N, K):
    """Decode configuration: every output of the full-size launch is checked."""
    _run(M, N, K, seed=3)


@pytest.mark.parametrize("M,N,K", [(8, 520, 1024), (64, 4096, 1024), (40, 1032, 256)])
@pytest.mark.parametrize("z", [8, 15])
def test_decode_asymmetric_activations(M, N, K, z):
    _run(M, N, K, symmetric=False, z=z)


def test_decode_post_residual_and_f32_scales():
    _run(24, 1024, 1024, post=True)
    _run(64, 2048, 512, post=True, residual=True, f16=False)
    _run(3, 136, 256, residual=True)


def test_decode_same_workspace_many_launches():
    M, N, K = 64, 4096, 2048
    ws = B.new_workspace(B.OP_GEMM, M, N, K)
    _run(M, N, K, ws=ws, reps=5)
    _run(9, 8192, 1024, ws=B.new_workspace(B.OP_GEMM, 9, 8192, 1024), reps=3)


def test_decode_extreme_codes_and_long_k():
    M, N, K = 64, 264, 28672
    qa = np.full((M, K), -8, dtype=np.int8)
    qw = np.full((N, K), -8, dtype=np.int8)
    qw[1::2] = 7
    sw = np.full(N, 2.0 ** -10, dtype=np.float32)
    _, acc = B.fpt_w4a4_gemm(packed_dev(qa), packed_dev(qw), dev(sw), 1.0, want_acc=True, want_y=False)
    acc = host(acc)
    assert np.all(acc[:, 0::2] == 64 * K) and np.all(acc[:, 1::2] == -56 * K)


def test_decode_many_tiles_without_counters():
    """More 128-row tiles than the control block has counters: ranges then end on tile boundaries."""
    _run(8, 64000, 128, seed=11)


@pytest.mark.parametrize("M,N,K,what", [
    (40, 8192, 2048, "64 tiles cut in 2: clusters of two CTAs"),
    (33, 2048, 4096, "16 tiles cut in 8: clusters of eight CTAs"),
    (64, 4096, 2048, "32 tiles cut in 4, asymmetric grid and residual below"),
    (64, 1024, 8192, "8 tiles cut in 16 ranges: no cluster that size, partial sums through the scratch slots"),
    (20, 1152, 1280, "9 tiles, 5 k-blocks: ranges that do not end on tile boundaries")])
def test_decode_split_tiles_cluster_and_slot_paths(M, N, K, what):
    """Few tiles and long rows: every tile is cut into ranges whose partial sums are exchanged through a
    cluster's shared memory (2, 4, 8 CTAs) or through scratch slots; twice on one workspace."""
    ws = B.new_workspace(B.OP_GEMM, M, N, K)
    _run(M, N, K, seed=21, ws=ws, reps=2)
    _run(M, N, K, symmetric=False, z=9, seed=22, post=True, residual=True, f16=False, ws=ws, reps=2)
