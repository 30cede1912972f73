/*
 * fpt.h -- C ABI of the B200 (sm_100a) statically quantised W4A4 linear path.
 *
 * The path is the transformer linear layer that FPTQuant makes viable with static
 * INT4 activations: once the mergeable transforms are folded into the weights
 * (Sec. 3.1.1, 3.1.2), every projection is
 *   (1) RMSNorm-derived per-token scale + static INT4 quantise + pack   (Sec. 3.1.3, App. B)
 *   (2) packed-INT4 x packed-INT4 matmul with an exact INT32 accumulator (App. J)
 *   (3) floating-point scale factors applied after the integer matmul   (App. B)
 *
 * General rules
 *   - Every pointer is a DEVICE pointer unless it is a `const fpt_qparams*` (HOST).
 *   - The caller owns every buffer.  The library allocates no device memory and keeps
 *     no state between calls except a per-process cache of driver entry points.
 *   - `stream` is a cudaStream_t passed as void*.  Work is enqueued on it and the call
 *     returns without synchronising, except fpt_check_status.
 *   - Row-major, contiguous tensors.  Activations are X[M, K] (one row per token);
 *     weights are stored W[N, K] = [out features, in features], so Y = X W^T.
 *   - Packed INT4: byte j of a row holds code 2j in bits 0..3 and code 2j+1 in bits
 *     4..7 ("double-packed", App. J); symmetric grids store two's complement nibbles,
 *     asymmetric grids store unsigned nibbles.
 *   - Pointers to packed tensors, bf16 tensors and workspaces are 16-byte aligned;
 *     K is a multiple of 32 (fpt_act_quant, fpt_quantize_weights) and of 128 for the
 *     matmul entry points; N is a multiple of 8.
 *   - Every function returns FPT_OK (0) or a negative error code; nothing throws,
 *     aborts or traps.  Argument errors are detected before anything is enqueued.
 *   - Floating point is float32 with one rounding per operation (no fused
 *     multiply-add on the quantisation path); bf16 narrowing is round-to-nearest-even.
 *
 * Quantiser grid (the paper states "uniform integer grid", Sec. 1, with scale and
 * offset as parameters, App. D; the formula is this library's reading):
 *   symmetric : q = clamp(rne(v / D), -2^(b-1), 2^(b-1)-1)        v^ = D q
 *   asymmetric: q = clamp(rne(v / D) + z, 0, 2^b - 1)             v^ = D (q - z)
 * rne = round to nearest, ties to even.  v / D is evaluated as v * (1/D) with 1/D
 * rounded once to float32 on the host.  A NaN maps to the lowest code.
 */
#ifndef FPT_H_
#define FPT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- error codes -------------------------------------------------------------- */
#define FPT_OK                0
#define FPT_ERR_BAD_ARG      -1   /* null pointer, non-positive size, bad enum          */
#define FPT_ERR_UNSUPPORTED  -2   /* bits != 4, K or N not a supported multiple, ...    */
#define FPT_ERR_ALIGNMENT    -3   /* a pointer or leading dimension is misaligned       */
#define FPT_ERR_WORKSPACE    -4   /* workspace missing or smaller than required         */
#define FPT_ERR_CUDA         -5   /* a CUDA runtime / driver call failed                */
#define FPT_ERR_TIMEOUT      -6   /* a device-side wait gave up (see fpt_check_status)  */

/* ---- enums -------------------------------------------------------------------- */
#define FPT_DTYPE_BF16 0
#define FPT_DTYPE_F32  1
#define FPT_DTYPE_F16  2

#define FPT_RANGE_MINMAX 0        /* L_inf range setting: D = max|w| / qmax             */
#define FPT_RANGE_LP     1        /* L_p range setting (App. D): least sum |w - w^|^p   */

/* flags of fpt_act_quant / fpt_w4a4_linear */
#define FPT_RMSNORM         1     /* r_t = 1/sqrt(mean_k x^2 + eps); the grid sees x * r_t        */
#define FPT_SCALE_INPUT     2     /* the grid sees x * s_in[t] (times r_t when FPT_RMSNORM too)   */
#define FPT_SILU_MUL        4     /* x := bf16(silu(X) * X2) before anything else (no RMSNORM)    */
#define FPT_GU_INTERLEAVED  8     /* with FPT_SILU_MUL: X holds gate||up in 64-column groups      */

/* where the per-token scale ends up after the matmul (Sec. 3.1.3: the scale commutes
 * with a bias-free linear, so the caller chooses) */
#define FPT_POST_NONE            0   /* y = (acc * sw[n]) * D_a                                   */
#define FPT_POST_INVERSE_OF_PRE  1   /* ... * (D_a * (1 / p_t)), p_t the multiplier used in (1)   */
#define FPT_POST_VECTOR          2   /* ... * (D_a * post[t])                                     */

#define FPT_OP_LINEAR 0
#define FPT_OP_MLP    1
#define FPT_OP_GEMM   2
#define FPT_OP_GEMM_A8   3     /* fpt_w4a8_gemm                                   */
#define FPT_OP_LINEAR_A8 4     /* fpt_w4a4_linear / _dynamic with 8-bit activations */
#define FPT_OP_MLP_HADAMARD 5  /* fpt_decoder_mlp with mid_hadamard = 1              */

/* One quantiser, as the paper parametrises it: bit-width, grid kind, static scale and
 * offset (App. D "General set-up"). HOST struct. */
typedef struct fpt_qparams {
  int   bits;        /* 4; 8 for activations where an entry point says so (symmetric only) */
  int   symmetric;   /* 1: codes in [-8, 7], zero_point ignored; 0: codes in [0, 15]     */
  float scale;       /* static per-tensor scale D (activations); ignored for weights,    */
                     /* whose per-output-channel scales are computed                     */
  int   zero_point;  /* z of the asymmetric grid                                          */
} fpt_qparams;

int         fpt_version(void);
const char* fpt_strerror(int code);

/*
 * Kernels of steps (1)-(3) are launched so that each may start (set up its barriers and tensor
 * memory, and wait) while the kernel before it in the stream is still draining; each orders itself
 * behind that kernel before it touches any operand, so results and stream semantics are unchanged
 * (no counterpart in the paper: a launch mode).  enabled = 0 switches back to plain launches for
 * every later call of the process, e.g. under a tool that does not follow such launches.
 * Returns the previous setting.  Not synchronised with concurrent calls of the other entry points.
 */
int fpt_set_programmatic_launch(int enabled);

/*
 * Offline weight quantiser (uniform grid, round-to-nearest, per-output-channel scale;
 * Sec. 4 "Quantization Setup", App. D "Quantizer range setting").
 *   W        [N, K] device, bf16 or f32 (w_dtype)
 *   qp       host; bits = 4, symmetric = 1 (weights always use the symmetric grid)
 *   range    FPT_RANGE_MINMAX: D_n = max_k|w_nk| / 7
 *            FPT_RANGE_LP    : D_n = (a_n * (i/100)) / 7 for the i in 20..100 with the least
 *                              sum_k |w - D clamp(rne(w/D))|^p (float64), ties to larger i
 *   scale_dtype  FPT_DTYPE_F32 or FPT_DTYPE_F16: D_n is rounded to it BEFORE the codes
 *            are computed; an all-zero row gets D_n = 1
 *   Wq       [N, K/2] out, packed codes q = clamp(rne(w / D_n), -8, 7) (IEEE division)
 *   sw       [N] out, scale_dtype
 *   wsum     [N] out int32, sum_k q_nk; may be NULL (needed only for asymmetric activations)
 */
int fpt_quantize_weights(void* stream, const void* W, int w_dtype, int N, int K,
                         const fpt_qparams* qp, int range_mode, float p, int scale_dtype,
                         uint8_t* Wq, void* sw, int32_t* wsum);

/*
 * Copies separately quantised gate and up matrices into the row-interleaved layout that
 * fpt_decoder_mlp expects: for every group r of 64 output features, rows
 * [128 r, 128 r + 64) of Wgu_q are gate rows [64 r, 64 r + 64) and rows
 * [128 r + 64, 128 r + 128) are the matching up rows; sw_gu follows the same order.
 * d_ff must be a multiple of 64.  (No counterpart in the paper: it is a storage choice
 * that puts a gate column and its up column into the registers of one epilogue thread, so
 * that the SwiGLU product and the next quantiser run inside the matmul.)
 */
int fpt_interleave_gate_up(void* stream, const uint8_t* Wg_q, const uint8_t* Wu_q,
                           const void* sw_g, const void* sw_u, int scale_dtype,
                           int d_ff, int K, uint8_t* Wgu_q, void* sw_gu);

/*
 * Step (1): per-token scale + static quantise + pack (Sec. 3.1.3 Eq. 6-7; App. B).
 * Per token t (row of X):
 *   x_tk  = X[t,k]                                   (FPT_SILU_MUL: bf16(silu(X[t,k]) * X2[t,k]))
 *   r_t   = 1 / sqrt( (float)(sum_k x_tk^2 in float64) / K + eps )      if FPT_RMSNORM else 1
 *   p_t   = r_t * s_in[t]   if FPT_SCALE_INPUT (s_in required)          else r_t
 *   q_tk  = clamp(rne((x_tk * p_t) * (1/D)) + z)
 *   s_out[t] = r_t * s_in[t] if s_in != NULL else r_t      -- S_n = S_{n-1} / ||Z~_{n-1}||_R
 * A block input uses FPT_RMSNORM alone (the grid sees RMSNorm(x), s_out carries the
 * recursion); a site inside a block (attention output, down-projection input) uses
 * FPT_SCALE_INPUT alone (the grid sees S_n x).
 *   X      [M, ldx] bf16, ldx >= K elements, ldx % 8 == 0
 *   X2     second operand of FPT_SILU_MUL, same layout as X; with FPT_GU_INTERLEAVED X2 is
 *          ignored, X is [M, 2K] (ldx >= 2K) and logical column k lives at
 *          gate: (k/64)*128 + k%64, up: gate + 64
 *   s_in   [M] f32 or NULL;  s_out [M] f32 or NULL
 *   Xq     [M, K/2] packed codes out;  qp->bits == 8 (symmetric grid, no FPT_SILU_MUL): [M, K] int8 codes
 *          q = clamp(rne((x * p) * (1/D)), -128, 127)
 * silu(g) = g / (1 + 2^(-g*log2 e)) with a fixed float32 polynomial for 2^f (degree 6
 * Taylor, Horner, separately rounded multiply and add), so that the result is one
 * defined float32 value.
 */
int fpt_act_quant(void* stream, const void* X, int M, int K, int ldx,
                  const fpt_qparams* qp, int flags, float eps,
                  const void* X2, const float* s_in, uint8_t* Xq, float* s_out);

/*
 * Step (1) with a DYNAMIC grid (App. B "Dynamic quantization": for each token the extreme
 * activation values are reduced over the last dimension and the resulting scale factor is applied
 * to every value).  The paper prints no formula; this library's reading is the symmetric grid that
 * ends at the token's largest magnitude.  Per token t, with r_t, p_t, s_out as in fpt_act_quant:
 *   m_t  = max_k |x_tk * p_t|
 *   D_t  = m_t / qmax            (float32 division; qmax = 7 or 127)
 *          D_t = 1 when m_t is zero, infinite or NaN
 *   q_tk = clamp(rne((x_tk * p_t) * (1 / D_t)), -qmax - 1, qmax)      (1 / D_t: float32 division)
 *   bits = 4: Xq [M, K/2] packed codes;  bits = 8: Xq [M, K] int8 codes
 *   delta_out [M] f32 out: D_t (required);  s_in, s_out as in fpt_act_quant.
 * flags: FPT_RMSNORM, FPT_SCALE_INPUT.
 */
int fpt_act_quant_dynamic(void* stream, const void* X, int M, int K, int ldx, int bits, int flags, float eps,
                          const float* s_in, void* Xq, float* s_out, float* delta_out);

/*
 * Online block-wise Hadamard transform + per-token scale + static quantise + pack, for the input of
 * the down projection (Sec. 3.1, last paragraph; App. A transform table: H_n = n^(-1/2) (x) [[1,1],[1,-1]];
 * App. D "Hadamard non-powers of 2").  The K channels are split into K / B groups of
 * B = largest power of two dividing K (256 <= B <= 4096), each group is multiplied by H_B; there is no
 * zero padding.  Per token t:
 *   m_tk = X[t,k]                    (FPT_SILU_MUL | FPT_GU_INTERLEAVED: bf16(silu(g) * u) from the
 *                                     64-column gate||up layout, X is [M, 2K])
 *   h    = H_B applied group-wise, float32 butterflies (a, b) -> (a + b, a - b) with partner distance
 *          1, 2, 4, ..., B/2 in this order, then one multiply by float32(B^(-1/2))
 *   q_tk = clamp(rne((h_tk * p_t) * (1/D)) + z),  p_t = s_in[t] with FPT_SCALE_INPUT, else 1
 * The weight that consumes the codes must have the inverse transform merged into its input columns
 * (W <- W blockdiag(H_B); H_B is symmetric and orthogonal).
 *   X [M, ldx] bf16;  Xq [M, K/2] packed codes out;  K % 256 == 0.
 */
int fpt_hadamard_quant(void* stream, const void* X, int M, int K, int ldx,
                       const fpt_qparams* qp, int flags, const float* s_in, uint8_t* Xq);

/*
 * Steps (2)+(3) on already packed operands (App. J "Setup"; App. B "Static quantization"):
 *   acc[t,n] = sum_k (qa[t,k] - z) * qw[n,k]                 exact int32
 *   y[t,n]   = bf16( ((float)acc * sw[n]) * c_t  [+ res[t,n] * res_scale[t]] )
 *   c_t      = act_scale * post[t]  (post != NULL)  else act_scale
 *   Xq [M, K/2], Wq [N, K/2] packed; sw [N] (scale_dtype); wsum [N] int32, required
 *   when act_symmetric == 0; post [M] f32 or NULL.
 *   residual [M, N] bf16 or NULL, added in float32 before the single bf16 rounding;
 *   res_scale [M] f32 or NULL (1).
 *   Y [M, N] bf16 out (may be NULL when acc_out is given)
 *   acc_out [M, N] int32 or NULL: debugging aid, the raw accumulators.
 *   workspace: fpt_workspace_bytes(FPT_OP_GEMM, M, N, K) bytes; it starts with an 8 KiB control
 *   block (status word read by fpt_check_status, tile counters) that fpt_reset_status zeroes.
 * M >= 1; K % 128 == 0; N % 8 == 0.  For M <= 64 a weight-streaming kernel is used: it splits
 * the weight stream evenly over the SMs and adds the partial sums up as exact integers.
 */
int fpt_w4a4_gemm(void* stream, const uint8_t* Xq, const uint8_t* Wq, int M, int N, int K,
                  const void* sw, int scale_dtype, const int32_t* wsum,
                  float act_scale, int act_symmetric, int act_zero_point,
                  const float* post, const void* residual, const float* res_scale,
                  void* Y, int32_t* acc_out, void* workspace, size_t workspace_bytes);

/*
 * The same two steps with 8-bit activation codes and 4-bit weights (the W4A8 setting, Sec. 4):
 *   acc[t,n] = sum_k qa[t,k] * qw[n,k]      exact int32;  qa int8 in [-128, 127] (symmetric grid)
 *   y[t,n]   as in fpt_w4a4_gemm.
 *   Xq8 [M, K] int8;  K % 128 == 0, K <= 16384 (so that (float)acc is exact), N % 8 == 0.
 *   workspace: fpt_workspace_bytes(FPT_OP_GEMM_A8, M, N, K) bytes.
 * More than 16 tokens and 128 outputs, or at most 16 tokens: kernels that read the int8 codes as they are.
 * What is left (more than 16 tokens, at most 128 outputs): the codes are split as a = 16 (a >> 4) + (a & 15) and two 4-bit matmuls are
 * combined exactly in int32 before the scale factors (same result, twice the matmul work).
 */
int fpt_w4a8_gemm(void* stream, const int8_t* Xq8, const uint8_t* Wq, int M, int N, int K,
                  const void* sw, int scale_dtype, float act_scale,
                  const float* post, const void* residual, const float* res_scale,
                  void* Y, int32_t* acc_out, void* workspace, size_t workspace_bytes);

/*
 * Steps (1)+(2)+(3): one W4A4 linear on bf16 activations.
 *   X [M, K] bf16; flags / eps / s_in / s_out as in fpt_act_quant (FPT_SILU_MUL not allowed);
 *   post_mode selects c_t (see FPT_POST_*); post [M] only for FPT_POST_VECTOR.
 *   workspace: fpt_workspace_bytes(FPT_OP_LINEAR, M, N, K) bytes (packed activations,
 *   the per-token vectors and the status word live there).
 * act_qp->bits == 8 (symmetric grid only): int8 codes q = clamp(rne((x * p) * (1/D)), -128, 127) and
 *   the matmul of fpt_w4a8_gemm; workspace: fpt_workspace_bytes(FPT_OP_LINEAR_A8, M, N, K) bytes.
 */
int fpt_w4a4_linear(void* stream, const void* X, int M, int K,
                    const uint8_t* Wq, const void* sw, int scale_dtype, const int32_t* wsum, int N,
                    const fpt_qparams* act_qp, int flags, float eps, const float* s_in,
                    int post_mode, const float* post,
                    void* Y, float* s_out, void* workspace, size_t workspace_bytes);

/*
 * The same linear with the dynamic activation grid of fpt_act_quant_dynamic (the paper's second
 * timing table, App. J "Dynamic INT4 runtime"):
 *   codes, D_t as in fpt_act_quant_dynamic;  acc as in fpt_w4a4_gemm (symmetric codes);
 *   y[t,n] = bf16( ((float)acc * sw[n]) * c_t ),
 *   c_t = D_t (FPT_POST_NONE), D_t * (1 / p_t) (FPT_POST_INVERSE_OF_PRE), D_t * post[t] (FPT_POST_VECTOR).
 *   bits = 4: workspace fpt_workspace_bytes(FPT_OP_LINEAR, M, N, K) bytes;
 *   bits = 8: int8 codes, matmul of fpt_w4a8_gemm, workspace fpt_workspace_bytes(FPT_OP_LINEAR_A8, M, N, K).
 */
int fpt_w4a4_linear_dynamic(void* stream, const void* X, int M, int K,
                            const uint8_t* Wq, const void* sw, int scale_dtype, int N,
                            int bits, int flags, float eps, const float* s_in,
                            int post_mode, const float* post,
                            void* Y, float* s_out, void* workspace, size_t workspace_bytes);

/*
 * fpt_w4a4_linear without a caller workspace.  (The paper has no counterpart: this is a
 * packaging variant of fpt_w4a4_linear, same arithmetic, same results.)
 *
 * For callers that cannot allocate device memory: a plug-in that a host runtime calls with
 * input and output pointers only, a serving loop whose pool was frozen at start-up, code that
 * must not trigger the device-wide synchronisation an allocation can cause.  The scratch that
 * fpt_w4a4_linear takes from its workspace (packed activation codes, one float per token, the
 * status block) lives in a __device__ array inside the library, FPT_STATIC_SCRATCH_BYTES long;
 * every GPU that loads the library holds that much until the process ends.  The call itself
 * performs no device allocation or free of any kind.
 *
 * Arguments as fpt_w4a4_linear, minus workspace / workspace_bytes.
 * Limit: fpt_workspace_bytes(FPT_OP_LINEAR, M, N, K) <= FPT_STATIC_SCRATCH_BYTES (about
 * M*K/2 + 4*M + 8 KiB, plus up to 10 MiB of matmul scratch when M <= 64), otherwise
 * FPT_ERR_WORKSPACE is returned and nothing is enqueued (e.g. 4096 tokens x 8192 features fit).
 * First call on a device: looks up the array's device address (cudaGetSymbolAddress, with that
 * device current) and caches it; make this first call outside any stream capture.
 * The array is shared by every call in the process and keeps the previous call's contents;
 * the status word is cleared on `stream` at the start of each call.  Two calls that can
 * overlap on the GPU (different streams, no dependency) race on it: serialise them.
 * A bounded device-side wait that gave up cannot be read back through this entry point; use
 * fpt_w4a4_linear with a workspace where that matters.
 */
#define FPT_STATIC_SCRATCH_BYTES (17u * 1024u * 1024u)
int fpt_w4a4_linear_static(void* stream, const void* X, int M, int K,
                           const uint8_t* Wq, const void* sw, int scale_dtype, const int32_t* wsum, int N,
                           const fpt_qparams* act_qp, int flags, float eps, const float* s_in,
                           int post_mode, const float* post, void* Y, float* s_out);

/*
 * One SwiGLU MLP block in the normalised-residual form of Sec. 3.1.3:
 *   X~ = RMSNorm(X),  S_n = S_{n-1} * r                       (X is Z~_{n-1}; Eq. 7)
 *   g, u = W4A4 linears of X~ (bf16)                          grid qp_in
 *   m = bf16(silu(g) * u);  quantise m * S_n                  grid qp_mid (scaler at the
 *                                                              down-projection input)
 *        with mid_hadamard = 1 the grid sees S_n * H(m) (fpt_hadamard_quant) and Wd_q must be the
 *        quantised W_d blockdiag(H) (Sec. 3.1 last paragraph: the one online transform)
 *   Y~ = W4A4 down projection  (= S_n * Y_n, Eq. 5)
 *   Y  = bf16(Y~ + X * r)  if add_residual  (Z~_n = X~_n + Y~_n)   else bf16(Y~)
 *   Wgu_q [2 d_ff, d/2] and sw_gu [2 d_ff] in the layout of fpt_interleave_gate_up;
 *   Wd_q [d, d_ff/2], sw_d [d]; s_prev [M] or NULL (= 1); s_out [M] or NULL.
 *   d % 128 == 0, d_ff % 128 == 0.  Both grids symmetric in this version.
 *   workspace: fpt_workspace_bytes(FPT_OP_MLP, M, d_ff, d) bytes, or (FPT_OP_MLP_HADAMARD, M, d_ff, d)
 *   with mid_hadamard = 1.  A 16-bit buffer between the two matmuls is part of it only where a route
 *   uses one: none with more than 128 tokens and no transform (the gate||up matmul quantises the
 *   products itself), the products [M, d_ff] with the transform, gate||up [M, 2 d_ff] up to 128 tokens.
 */
int fpt_decoder_mlp(void* stream, const void* X, int M, int d, int d_ff,
                    const uint8_t* Wgu_q, const void* sw_gu, const uint8_t* Wd_q, const void* sw_d,
                    int scale_dtype, const fpt_qparams* qp_in, const fpt_qparams* qp_mid, float eps,
                    const float* s_prev, float* s_out, int add_residual, int mid_hadamard,
                    void* Y, void* workspace, size_t workspace_bytes);

/*
 * The attention block of a decoder layer in the normalised-residual form of Sec. 3.1.3, as two
 * calls around the caller's own attention (RoPE, softmax(QK^T) V; kept in 16-bit floating point
 * in the paper's timing runs, App. J "Setup").  The sequence scaler S_n sits at the attention
 * output ("ap" in the placement table of App. A): a per-token scale commutes with the BMMs and
 * with the bias-free output projection (Sec. 3.1.3, after Eq. 5).
 *
 * fpt_decoder_attn_qkv:
 *   X~ = RMSNorm(X),  S_n = S_{n-1} * r,  r = 1 / sqrt(mean_k X^2 + eps)    (X is Z~_{n-1}; Eq. 7)
 *   QKV = W4A4 linear of X~ with the fused weight Wqkv_q [n_qkv, d/2]        grid qp_in
 *         (query || key || value rows, the pre-RoPE and value transforms of Sec. 3.1.1-3.1.2
 *         already merged into it); QKV [M, n_qkv] bf16 carries no S_n: RMSNorm removed it.
 *   s_prev [M] or NULL (= 1); s_out [M] out: S_n;  r_out [M] out: r (scales the residual later).
 * fpt_decoder_attn_out:
 *   A [M, k_o] bf16: the caller's attention output (heads concatenated)
 *   codes = grid_qp_ap(A * S_n)                                             (scaler at "ap")
 *   Y~ = W4A4 output projection with Wo_q [d, k_o/2]  (= S_n * Y_n, Eq. 5)
 *   Y  = bf16(Y~ + X * r)  if X != NULL   (Z~_n = X~_n + Y~_n;  X is the Z~_{n-1} given to
 *        fpt_decoder_attn_qkv, r its r_out)                     else bf16(Y~)
 * wsum_* [N] int32: required when the grid is asymmetric, else NULL.
 * Shapes as fpt_w4a4_linear; workspace: fpt_workspace_bytes(FPT_OP_LINEAR, M, n_qkv, d) resp.
 * (FPT_OP_LINEAR, M, d, k_o) bytes.  The two calls may share one workspace.
 */
int fpt_decoder_attn_qkv(void* stream, const void* X, int M, int d,
                         const uint8_t* Wqkv_q, const void* sw_qkv, int scale_dtype, const int32_t* wsum_qkv,
                         int n_qkv, const fpt_qparams* qp_in, float eps, const float* s_prev,
                         float* s_out, float* r_out, void* QKV, void* workspace, size_t workspace_bytes);
int fpt_decoder_attn_out(void* stream, const void* A, int M, int k_o,
                         const uint8_t* Wo_q, const void* sw_o, int scale_dtype, const int32_t* wsum_o, int d,
                         const fpt_qparams* qp_ap, const float* s_n, const void* X, const float* r,
                         void* Y, void* workspace, size_t workspace_bytes);

/*
 * Measurement aid; the paper has no counterpart.  Runs nothing of the path: one thread per CTA
 * (pair = 0) or per pair of CTAs (pair = 1, `ctas` even) issues 4 * iters 8-bit integer
 * tensor-core instructions of 128 (pair: 256) rows x n columns x 32 codes on operand tiles that
 * never move, rotating over n_acc accumulators (n_acc * n <= 480), with the row operand read
 * from tensor memory (a_in_tmem = 1) or from shared memory.  2 * rows * n * 32 * 4 * iters * CTAs
 * (pairs) integer operations per launch; the rate it reaches is the ceiling the matmul kernels
 * are compared with.
 *   n       multiple of 16 in [16, 256]
 *   cycles  device [ctas] (pair: [ctas / 2]) out, may be NULL: SM clock ticks from the first issue
 *           to the completion of the last instruction
 *   workspace  device, 16-byte aligned, at least 8192 bytes: status block (fpt_check_status)
 */
int fpt_probe_mma(void* stream, int pair, int n, int n_acc, int a_in_tmem, int iters, int ctas,
                  unsigned long long* cycles, void* workspace);

/*
 * Self-test of the bounded device-side wait (the paper has no counterpart).  Every wait inside the
 * kernels gives up after a time limit, records a code in the status word of the workspace and lets
 * the kernel end normally (FPT_ERR_TIMEOUT from fpt_check_status).  This call runs that very wait
 * routine in a one-warp kernel on a barrier nothing ever arrives at, with a limit of limit_us
 * microseconds (1 .. 100000): the kernel ends by itself after that time.
 *   workspace  device, 16-byte aligned, at least 8192 bytes, status word zero (fpt_reset_status)
 *   gave_up    device, may be NULL: 1 if the wait returned "gave up"
 * Afterwards fpt_check_status(stream, workspace) returns FPT_ERR_TIMEOUT until fpt_reset_status.
 */
int fpt_selftest_wait_timeout(void* stream, void* workspace, unsigned int limit_us, unsigned int* gave_up);

/* Bytes of caller-provided scratch an entry point needs (op = FPT_OP_*).
 * FPT_OP_LINEAR / FPT_OP_GEMM / FPT_OP_GEMM_A8 / FPT_OP_LINEAR_A8: (M, N, K); FPT_OP_MLP: (M, d_ff, d). */
size_t fpt_workspace_bytes(int op, int M, int N, int K);

/* Zeroes the control block (first 8 KiB: status word, tile counters) of a workspace.  Call once
 * after allocating it, and again after a call that ended in FPT_ERR_TIMEOUT. */
int fpt_reset_status(void* stream, void* workspace);

/* Synchronises `stream`, reads the status word at the start of `workspace` and returns
 * FPT_OK, FPT_ERR_TIMEOUT (a bounded device-side wait expired; the kernel released its
 * resources and returned, outputs are invalid) or FPT_ERR_CUDA. */
int fpt_check_status(void* stream, void* workspace);

#ifdef __cplusplus
}
#endif
#endif /* FPT_H_ */
