"""Times one entry point of the library on one shape, with CUDA events.

    python -m paper_2506_04985_b200.microbench gemm      --M 2048 --N 6144 --K 4096
    python -m paper_2506_04985_b200.microbench act_quant --M 2048 --K 4096
    python -m paper_2506_04985_b200.microbench silu_quant --M 4096 --K 14336
    python -m paper_2506_04985_b200.microbench linear    --M 64 --N 14336 --K 4096
    python -m paper_2506_04985_b200.microbench hadamard_quant --M 4096 --K 14336
    python -m paper_2506_04985_b200.microbench mlp       --M 4096 --K 4096 --N 14336      (mlp_hadamard: with the online transform)
    python -m paper_2506_04985_b200.microbench attn_proj --M 2048 --N 6144 --K 4096       (QKV and output projections with the residual)
    python -m paper_2506_04985_b200.microbench gemm_a8   --M 2048 --N 6144 --K 4096       (int8 activation codes)
    python -m paper_2506_04985_b200.microbench linear_dynamic --M 2048 --N 6144 --K 4096 --bits 4
    python -m paper_2506_04985_b200.microbench act_quant_dynamic --M 2048 --K 4096 --bits 4
    python -m paper_2506_04985_b200.microbench mma_probe                                  (bare tensor-core instruction rates)

Operands are random packed codes / random bf16 values made on the device (timing does
not depend on the values).  `--sets S` rotates S independent operand sets so that every
launch reads HBM rather than the L2 (pick S so that S x bytes-per-set exceeds 126 MB);
`--reps R` launches are timed back to back between two events on the launching stream
(`--graph`: captured once in a CUDA graph and replayed, for kernels shorter than a launch).
Prints one JSON line: microseconds per launch, TOP/s, GB/s of algorithmic bytes.
The same command with small `--reps` is what the profiler captures.
"""
import argparse
import json

import torch

from . import binding as B


def _codes(rows, kb, dev):
    return torch.randint(0, 256, (rows, kb), dtype=torch.uint8, device=dev)


def _bf16(rows, cols, dev):
    return torch.randn((rows, cols), dtype=torch.float32, device=dev).to(torch.bfloat16)


def make_case(kind, M, N, K, sets, dev, f16_scales=False, bits=4):
    """Returns (list of zero-argument launchers, algorithmic ops, algorithmic bytes)."""
    sdt = torch.float16 if f16_scales else torch.float32
    ssz = 2 if f16_scales else 4
    qp = B.QParams(4, True, 0.45, 0)
    runs = []
    if kind == "gemm":
        ws = B.new_workspace(B.OP_GEMM, M, N, K, dev)
        for _ in range(sets):
            xq, wq = _codes(M, K // 2, dev), _codes(N, K // 2, dev)
            sw = torch.rand((N,), device=dev).to(sdt) * 0.01 + 0.001
            y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
            runs.append(lambda xq=xq, wq=wq, sw=sw, y=y: B.fpt_w4a4_gemm(xq, wq, sw, 0.45, ws=ws, Y=y))
        return runs, 2.0 * M * N * K, M * K / 2 + N * K / 2 + N * ssz + 2.0 * M * N
    if kind == "act_quant":
        for _ in range(sets):
            x = _bf16(M, K, dev)
            out = torch.empty((M, K // 2), dtype=torch.uint8, device=dev)
            runs.append(lambda x=x, out=out: B.fpt_act_quant(x, qp, B.RMSNORM, 1e-5, out=out))
        return runs, 0.0, 2.5 * M * K + 4.0 * M
    if kind == "silu_quant":
        for _ in range(sets):
            gu = _bf16(M, 2 * K, dev)
            s = torch.rand((M,), device=dev) + 0.5
            out = torch.empty((M, K // 2), dtype=torch.uint8, device=dev)
            runs.append(lambda gu=gu, s=s, out=out: B.fpt_act_quant(
                gu, qp, B.SILU_MUL | B.GU_INTERLEAVED | B.SCALE_INPUT, 0.0, s_in=s, K=K, want_s_out=False, out=out))
        return runs, 0.0, 4.5 * M * K + 4.0 * M
    if kind == "hadamard_quant":            # products m [M, K] bf16 -> block Hadamard -> codes
        for _ in range(sets):
            m = _bf16(M, K, dev)
            s = torch.rand((M,), device=dev) + 0.5
            out = torch.empty((M, K // 2), dtype=torch.uint8, device=dev)
            runs.append(lambda m=m, s=s, out=out: B.fpt_hadamard_quant(m, qp, B.SCALE_INPUT, s_in=s, out=out))
        return runs, 0.0, 2.5 * M * K + 4.0 * M
    if kind == "gemm_a8":
        ws = B.new_workspace(B.OP_GEMM_A8, M, N, K, dev)
        for _ in range(sets):
            xq = torch.randint(-128, 128, (M, K), dtype=torch.int8, device=dev)
            wq = _codes(N, K // 2, dev)
            sw = torch.rand((N,), device=dev).to(sdt) * 0.01 + 0.001
            y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
            runs.append(lambda xq=xq, wq=wq, sw=sw, y=y: B.fpt_w4a8_gemm(xq, wq, sw, 0.45, ws=ws, Y=y))
        return runs, 2.0 * M * N * K, M * K + N * K / 2 + N * ssz + 2.0 * M * N
    if kind == "act_quant_dynamic":
        for _ in range(sets):
            x = _bf16(M, K, dev)
            out = (torch.empty((M, K // 2), dtype=torch.uint8, device=dev) if bits == 4
                   else torch.empty((M, K), dtype=torch.int8, device=dev))
            runs.append(lambda x=x, out=out: B.fpt_act_quant_dynamic(x, bits, B.RMSNORM, 1e-5, want_s_out=False, out=out))
        return runs, 0.0, (2.0 + bits / 8.0) * M * K + 8.0 * M
    if kind == "linear_dynamic":
        for _ in range(sets):
            x, wq = _bf16(M, K, dev), _codes(N, K // 2, dev)
            sw = torch.rand((N,), device=dev).to(sdt) * 0.01 + 0.001
            y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
            ws = B.new_workspace(B.OP_LINEAR_A8 if bits == 8 else B.OP_LINEAR, M, N, K, dev)
            runs.append(lambda x=x, wq=wq, sw=sw, y=y, ws=ws: B.fpt_w4a4_linear_dynamic(
                x, wq, sw, bits, B.RMSNORM, 1e-5, want_s_out=False, ws=ws, Y=y))
        return runs, 2.0 * M * N * K, 2.0 * M * K + N * K / 2 + N * ssz + 2.0 * M * N
    if kind == "linear":
        for _ in range(sets):
            x, wq = _bf16(M, K, dev), _codes(N, K // 2, dev)
            sw = torch.rand((N,), device=dev).to(sdt) * 0.01 + 0.001
            y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
            ws = B.new_workspace(B.OP_LINEAR, M, N, K, dev)
            runs.append(lambda x=x, wq=wq, sw=sw, y=y, ws=ws: B.fpt_w4a4_linear(
                x, wq, sw, qp, B.RMSNORM, 1e-5, want_s_out=False, ws=ws, Y=y))
        return runs, 2.0 * M * N * K, 2.0 * M * K + N * K / 2 + N * ssz + 2.0 * M * N
    if kind == "attn_proj":                 # K = d (= query width), N = fused QKV width; both halves of the attention block
        d, nqkv = K, N
        for _ in range(sets):
            x, a = _bf16(M, d, dev), _bf16(M, d, dev)          # a stands for the caller's attention output
            wqkv, wo = _codes(nqkv, d // 2, dev), _codes(d, d // 2, dev)
            sqkv = torch.rand((nqkv,), device=dev).to(sdt) * 0.01 + 0.001
            so = torch.rand((d,), device=dev).to(sdt) * 0.01 + 0.001
            qkv = torch.empty((M, nqkv), dtype=torch.bfloat16, device=dev)
            y = torch.empty((M, d), dtype=torch.bfloat16, device=dev)
            ws = B.new_workspace(B.OP_LINEAR, M, max(nqkv, d), d, dev)

            def run(x=x, a=a, wqkv=wqkv, wo=wo, sqkv=sqkv, so=so, qkv=qkv, y=y, ws=ws):
                _, s_n, r = B.fpt_decoder_attn_qkv(x, wqkv, sqkv, qp, 1e-5, ws=ws, QKV=qkv)
                B.fpt_decoder_attn_out(a, wo, so, qp, s_n, X=x, r=r, ws=ws, Y=y)
            runs.append(run)
        return runs, 2.0 * M * d * (nqkv + d), 6.0 * M * d + (nqkv + d) * d / 2 + 2.0 * M * nqkv + 2.0 * M * d
    if kind in ("mlp", "mlp_hadamard"):    # K = d, N = d_ff
        d, dff = K, N
        for _ in range(sets):
            x = _bf16(M, d, dev)
            wgu, wd = _codes(2 * dff, d // 2, dev), _codes(d, dff // 2, dev)
            sgu = torch.rand((2 * dff,), device=dev).to(sdt) * 0.01 + 0.001
            sd = torch.rand((d,), device=dev).to(sdt) * 0.01 + 0.001
            y = torch.empty((M, d), dtype=torch.bfloat16, device=dev)
            ws = B.new_workspace(B.OP_MLP_HADAMARD if kind == "mlp_hadamard" else B.OP_MLP, M, dff, d, dev)
            runs.append(lambda x=x, wgu=wgu, sgu=sgu, wd=wd, sd=sd, y=y, ws=ws: B.fpt_decoder_mlp(
                x, wgu, sgu, wd, sd, qp, qp, 1e-5, want_s_out=False, ws=ws, Y=y, mid_hadamard=kind == "mlp_hadamard"))
        return runs, 6.0 * M * d * dff, 4.0 * M * d + 1.5 * d * dff + 3 * dff * ssz
    raise ValueError(kind)


def time_case(runs, reps, warmup=3):
    for i in range(max(warmup, 1)):
        runs[i % len(runs)]()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(reps):
        runs[i % len(runs)]()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e3 / reps


def time_case_graph(runs, reps, warmup=3, replays=5):
    """The same `reps` launches captured once in a CUDA graph and replayed: removes the host's
    launch cost (argument marshalling, tensor-map encoding) from kernels of a few microseconds."""
    for i in range(max(warmup, 1)):
        runs[i % len(runs)]()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i in range(reps):
            runs[i % len(runs)]()
    g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(replays):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e3 / (reps * replays)


def mma_rate(pair, n, n_acc, a_in_tmem, iters=4096, ctas=None, repeats=5):
    """Rate of bare 8-bit integer tensor-core instructions (fpt_probe_mma) over all SMs: best of `repeats`
    launches, CUDA events on the launching stream -> dict with TOP/s and SM cycles per instruction."""
    dev = torch.device("cuda", torch.cuda.current_device())
    if ctas is None:
        ctas = torch.cuda.get_device_properties(dev).multi_processor_count
        if pair:
            ctas -= ctas & 1
    ws = torch.zeros((8192,), dtype=torch.uint8, device=dev)
    B.fpt_probe_mma(pair, n, n_acc, a_in_tmem, 64, ctas, ws)
    torch.cuda.synchronize()
    best, cyc = None, None
    for _ in range(repeats):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        c = B.fpt_probe_mma(pair, n, n_acc, a_in_tmem, iters, ctas, ws)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        if best is None or ms < best:
            best, cyc = ms, c
    assert B.fpt_check_status(ws) == B.OK
    rows = 256 if pair else 128
    units = ctas // 2 if pair else ctas
    ops = 2.0 * rows * n * 32 * 4 * iters * units
    return {"pair": int(pair), "n": n, "n_acc": n_acc, "a_in_tmem": int(a_in_tmem), "ctas": ctas, "iters": iters,
            "us": best * 1e3, "tops": ops / (best * 1e-3) / 1e12,
            "cycles_per_instruction": float(cyc.double().median().item()) / (4 * iters)}


def main():
    if len(__import__("sys").argv) > 1 and __import__("sys").argv[1] == "mma_probe":
        B.lib()
        torch.cuda.set_device(0)
        for pair, n, n_acc, atm in ((1, 256, 1, 1), (1, 256, 1, 0), (1, 240, 1, 1), (0, 256, 1, 1), (0, 256, 1, 0),
                                    (0, 64, 1, 1), (0, 64, 2, 1), (0, 64, 4, 1), (0, 64, 7, 1), (0, 64, 1, 0), (0, 64, 4, 0),
                                    (0, 32, 1, 1), (0, 32, 4, 1), (0, 32, 8, 1), (0, 16, 1, 1), (0, 16, 4, 1), (0, 16, 8, 1),
                                    (0, 128, 1, 1), (0, 128, 2, 1), (1, 64, 1, 1), (1, 64, 4, 1), (1, 128, 1, 1), (1, 128, 2, 1)):
            print(json.dumps(mma_rate(pair, n, n_acc, atm)))
        return
    ap = argparse.ArgumentParser()
    ap.add_argument("kind", choices=["gemm", "act_quant", "silu_quant", "hadamard_quant", "linear", "mlp", "mlp_hadamard",
                                     "gemm_a8", "act_quant_dynamic", "linear_dynamic", "attn_proj"])
    ap.add_argument("--M", type=int, default=2048)
    ap.add_argument("--N", type=int, default=4096)
    ap.add_argument("--K", type=int, default=4096)
    ap.add_argument("--sets", type=int, default=4)
    ap.add_argument("--reps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--f16-scales", action="store_true")
    ap.add_argument("--bits", type=int, default=4, help="activation bits of the dynamic kinds")
    ap.add_argument("--graph", action="store_true", help="replay the launches from a CUDA graph")
    a = ap.parse_args()
    B.lib()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    runs, ops, nbytes = make_case(a.kind, a.M, a.N, a.K, a.sets, dev, a.f16_scales, a.bits)
    us = time_case_graph(runs, a.reps, a.warmup) if a.graph else time_case(runs, a.reps, a.warmup)
    print(json.dumps({"kind": a.kind, "M": a.M, "N": a.N, "K": a.K, "sets": a.sets, "reps": a.reps,
                      "us": us, "tops": ops / us / 1e6, "gbs": nbytes / us / 1e3}))


if __name__ == "__main__":
    main()
