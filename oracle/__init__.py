"""CPU oracle for the statically quantised W4A4 linear path of FPTQuant.

THIS PACKAGE IS TEST INFRASTRUCTURE.  It is a plain, slow, numpy restatement of
what the hot path computes, written from the paper, and exists only so that the
CUDA library can be checked against it.  Only the test-suite, the smoke check
and the CPU-baseline leg of the benchmark may import it; the product path never
does.  It shares no code, table or constant with the CUDA sources.

Modules and the passages they follow
    bf16        bfloat16 <-> float32 conversion (format definition)
    quantizers  uniform integer grids: weight quantiser, static activation
                quantiser with the RMSNorm-derived per-token scale S_n
                (Sec. 3.1.3, App. B "Static quantization", App. D "Quantizer
                range setting"), SiLU*mul variant at the down-projection input
    int_matmul  INT4 x INT4 product with INT32 accumulator (App. J "Setup")
    epilogue    floating-point scale factors applied after the integer matmul
                (App. B "Static quantization")
    transforms  pre-RoPE transform (Sec. 3.1.1, Theorem 1, Eq. 1-4), multi-head
                value transform (Sec. 3.1.2), per-token residual scaling
                (Sec. 3.1.3), fp64 attention / MLP references used to prove
                function preservation
    hadamard    block-wise Hadamard transform at the down-projection input (Sec. 3.1 last
                paragraph; App. A transform table; App. D "Hadamard non-powers of 2")
    linear      the composed entry points (one W4A4 linear; one SwiGLU MLP block; the attention
                block's two projections around the caller's attention)

Parity status: every function is pinned by a CPU test (tests/test_oracle_*.py)
against something other than itself, with two exceptions that cannot be pinned
here: the paper's accuracy tables and its speed-up ratios ("parity unpinned":
they need model weights, datasets and an RTX 3080 Ti).
"""
