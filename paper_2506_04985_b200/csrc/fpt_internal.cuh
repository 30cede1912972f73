// Declarations shared between the translation units of the library (host side).
#pragma once

#include "fpt_common.cuh"
#include "fpt_host.cuh"

namespace fpt {

struct GemmParams {
  int M, N, K;
  int tiles_m, num_tiles, kblocks;
  const void* sw;
  int scale_dtype;
  const int32_t* wsum;
  int zero_point;              // 0 when the activation grid is symmetric
  int a_unsigned;              // activation codes are unsigned nibbles (asymmetric grid)
  int a_bits;                  // 8: the activation operand is int8 [M, K] (CTA-pair kernel only); otherwise packed 4-bit
  float act_scale;
  const float* post;
  const __nv_bfloat16* residual;
  const float* res_scale;
  __nv_bfloat16* Y;
  int32_t* acc_out;
  // SwiGLU + quantise fused into the epilogue (gate||up matmul of the MLP block, CTA-pair kernel
  // only): with Mq set, the columns are 64 gate | 64 up | ... output features, no bf16 tile is
  // written, and m = bf16(silu(g) * u) is quantised with the per-token multiplier mid_scale[t]
  int swiglu_bf16;             // with Y set and Mq null: Y [M, N/2] receives m itself (bf16), nothing is quantised
  uint8_t* Mq;                 // [M, N/4] packed codes of the N/2 products, or nullptr
  const float* mid_scale;      // [M] S_n
  float mid_inv_delta;         // 1/D of the grid at the down-projection input
  int mid_qmax_minus_z;
  uint32_t mid_flip;
  uint32_t* status;            // control block of the workspace (status word, decode counters)
  void* scratch;               // gemm_scratch_bytes(M) bytes behind the control block (decode partial sums)
};

// gemm_a8.cu: scratch bytes fpt_w4a8_gemm needs behind the control block and the matmul scratch.
size_t gemm_a8_scratch_bytes(int M, int N, int K);

// act_quant.cu: validated arguments only; also fills 1/p_t and r_t for the composed calls.
cudaError_t act_quant_launch(cudaStream_t st, const void* X, int M, int K, int ldx, const fpt_qparams* qp,
                             int flags, float eps, const void* X2, const float* s_in, uint8_t* Xq,
                             float* s_out, float* post_inv, float* r_out);
// Dynamic (per-token grid) and 8-bit forms of the same step (act_quant_dynamic.cu).
cudaError_t act_quant_dyn_launch(cudaStream_t st, const void* X, int M, int K, int ldx, int bits, int dynamic,
                                 float qp_scale, int flags, float eps, const float* s_in, int post_mode,
                                 const float* post, void* Xq, float* s_out, float* c_out, float* delta_out,
                                 float* r_out);

// hadamard_quant.cu: block-wise Hadamard + per-token scale + quantise (validated arguments only).
int hadamard_block(int K);
cudaError_t hadamard_quant_launch(cudaStream_t st, const void* X, int M, int K, int ldx, const fpt_qparams* qp,
                                  int silu_inter, const float* s_in, uint8_t* Xq);

// gemm_w4a4.cu: validated arguments only; returns an FPT_* code.
int gemm_launch(cudaStream_t st, const uint8_t* Xq, const uint8_t* Wq, const GemmParams& P);

// gemm_decode.cu: the weight-streaming kernel for M <= 64 and the scratch it needs.
size_t gemm_decode_scratch_bytes(int M);
int gemm_decode_launch(cudaStream_t st, const uint8_t* Xq, const uint8_t* Wq, const GemmParams& P, void* scratch);
inline size_t gemm_scratch_bytes(int M) { return M <= 64 ? gemm_decode_scratch_bytes(M) : 0; }

// gemm_decode_small.cu: register-only weight streaming for M <= 16 (no scratch).
int gemm_decode_small_launch(cudaStream_t st, const uint8_t* Xq, const uint8_t* Wq, const GemmParams& P);

// gemm_w4a4_2cta.cu: the CTA-pair kernel (256 x 256 tiles) behind gemm_launch for prefill sizes.
int gemm_pair_launch(cudaStream_t st, const uint8_t* Xq, const uint8_t* Wq, const GemmParams& P);

// api.cu: argument checks and body of the 4-bit static linear on a workspace of
// fpt_workspace_bytes(FPT_OP_LINEAR, M, N, K) bytes whose control block is zero (shared by
// fpt_w4a4_linear and fpt_w4a4_linear_static).
int linear4_check(const void* X, const uint8_t* Wq, const void* sw, int scale_dtype, const int32_t* wsum, const void* Y,
                  const fpt_qparams* act_qp, int M, int N, int K, int flags, const float* s_in, int post_mode,
                  const float* post);
int linear4_run(cudaStream_t st, const void* X, int M, int K, const uint8_t* Wq, const void* sw, int scale_dtype,
                const int32_t* wsum, int N, const fpt_qparams* act_qp, int flags, float eps, const float* s_in,
                int post_mode, const float* post, void* Y, float* s_out, uint8_t* ws);

}  // namespace fpt
