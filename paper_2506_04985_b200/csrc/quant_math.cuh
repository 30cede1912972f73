// Device arithmetic shared by the kernels that quantise activations: the float32 SiLU with one
// defined result, and the uniform-grid quantiser of a 16-byte chunk of bf16 values
// (App. B "Static quantization"; Sec. 3.1.3 for the per-token multiplier).
#pragma once

#include "fpt_common.cuh"

namespace fpt {

// 2^f on [-0.5, 0.5]: degree-6 Taylor coefficients (ln 2)^k / k!, rounded to float32.
__device__ __forceinline__ float exp2_spec(float t) {
  t = fminf(fmaxf(t, -126.0f), 126.0f);
  const float n = rintf(t);
  const float f = __fsub_rn(t, n);
  float a = 0x1.430912p-13f;                               // (ln2)^6 / 720
  a = __fadd_rn(__fmul_rn(a, f), 0x1.5d87fep-10f);         // (ln2)^5 / 120
  a = __fadd_rn(__fmul_rn(a, f), 0x1.3b2ab6p-7f);          // (ln2)^4 / 24
  a = __fadd_rn(__fmul_rn(a, f), 0x1.c6b08ep-5f);          // (ln2)^3 / 6
  a = __fadd_rn(__fmul_rn(a, f), 0x1.ebfbep-3f);           // (ln2)^2 / 2
  a = __fadd_rn(__fmul_rn(a, f), 0x1.62e43p-1f);           // ln2
  a = __fadd_rn(__fmul_rn(a, f), 1.0f);
  const float two_n = __int_as_float(((int)n + 127) << 23);
  return __fmul_rn(a, two_n);
}

__device__ __forceinline__ float silu_spec(float g) {
  const float e = exp2_spec(__fmul_rn(-g, 0x1.715476p+0f));   // log2(e)
  return __fdiv_rn(g, __fadd_rn(1.0f, e));
}

// bf16(silu(g) * u) for a packed pair of bf16 values.
__device__ __forceinline__ uint32_t silu_mul_pair(uint32_t g, uint32_t u) {
  const float lo = __fmul_rn(silu_spec(bf16lo_to_f32(g)), bf16lo_to_f32(u));
  const float hi = __fmul_rn(silu_spec(bf16hi_to_f32(g)), bf16hi_to_f32(u));
  return f32_to_bf16_bits(lo) | (f32_to_bf16_bits(hi) << 16);
}

// Two float32 lanes in one 64-bit register: sm_100 multiplies both with one instruction, each
// lane rounded to nearest even on its own (the same result as two scalar multiplies).
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t mul_f32x2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
// Packed add / subtract: used only where no multiply feeds them (the butterflies of the Hadamard
// kernel), so there is nothing a compiler could contract them with.
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint64_t sub_f32x2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
// (There is no packed add in the quantiser on purpose.  The quantiser needs the product (x * p) * (1/D) ROUNDED
// before the rounding constant is added; a packed multiply followed by a packed add was contracted
// into one fused multiply-add -- the explicit .rn of the packed forms does not stop that -- and a
// product that rounds to exactly k + 1/2 from slightly off it then took the other code.  The scalar
// add intrinsic is never contracted.)

// Quantiser arithmetic of one 16-byte chunk (8 values), in the order the header states:
//   u = (x * p) * (1/D)          two separately rounded float32 multiplies
//   q = clamp(rne(u) + z)        a NaN maps to the lowest code
// evaluated on the NEGATED value v = (x * -p) * (1/D) = -u (negation is exact and rounding to
// nearest even is symmetric): adding 1.5 * 2^23 leaves -rne(u) in the low mantissa bits, and the
// float's bit pattern is monotone in v, also beyond the exact range and for +Inf and NaN, which
// are the largest patterns.  One integer add-min-relu then yields qmax - q in [0, 15] with the
// NaN at qmax - qmin = 15, i.e. the lowest code; the nibbles are flipped back by one XOR per
// word (15 - c = c ^ 15; on the symmetric grid the two's complement nibble of 7 - c is c ^ 7).
struct QuantConsts {
  uint64_t np2, d2;       // (-p, -p), (1/D, 1/D)
  int bias;               // -(bits of magic) + (qmax - z)
  uint32_t flip;          // 0x77777777 symmetric, 0xFFFFFFFF asymmetric
};

// p: per-token multiplier; inv_delta: 1/D rounded once on the host; qmax_minus_z: upper end of the
// grid minus the zero point; flip: 0x77777777 (symmetric) or 0xFFFFFFFF (asymmetric).
__device__ __forceinline__ QuantConsts quant_consts(float p, float inv_delta, int qmax_minus_z, uint32_t flip) {
  QuantConsts c;
  c.np2 = pack_f32x2(-p, -p);
  c.d2 = pack_f32x2(inv_delta, inv_delta);
  c.bias = -0x4B400000 + qmax_minus_z;
  c.flip = flip;
  return c;
}

// Two values of one 32-bit word -> (15 - code) each, the second in front: returns c0 + 16 * c1 + 256 * prev.
__device__ __forceinline__ uint32_t quant_pair(uint32_t w, const QuantConsts& c, uint32_t prev) {
  float v0, v1;
  unpack_f32x2(mul_f32x2(mul_f32x2(pack_f32x2(bf16lo_to_f32(w), bf16hi_to_f32(w)), c.np2), c.d2), v0, v1);
  v0 = __fadd_rn(v0, 12582912.0f);
  v1 = __fadd_rn(v1, 12582912.0f);
  // (a negative sum -- u beyond 1.2e7 -- has a negative pattern; max(., 0) keeps the add below from wrapping)
  const uint32_t c0 = (uint32_t)__viaddmin_s32_relu(max(__float_as_int(v0), 0), c.bias, 15);
  const uint32_t c1 = (uint32_t)__viaddmin_s32_relu(max(__float_as_int(v1), 0), c.bias, 15);
  return (prev * 16u + c1) * 16u + c0;
}

// The same for two float32 values (no 16-bit rounding in front of the grid).
__device__ __forceinline__ uint32_t quant_pair_f32(float x0, float x1, const QuantConsts& c, uint32_t prev) {
  float v0, v1;
  unpack_f32x2(mul_f32x2(mul_f32x2(pack_f32x2(x0, x1), c.np2), c.d2), v0, v1);
  v0 = __fadd_rn(v0, 12582912.0f);
  v1 = __fadd_rn(v1, 12582912.0f);
  const uint32_t c0 = (uint32_t)__viaddmin_s32_relu(max(__float_as_int(v0), 0), c.bias, 15);
  const uint32_t c1 = (uint32_t)__viaddmin_s32_relu(max(__float_as_int(v1), 0), c.bias, 15);
  return (prev * 16u + c1) * 16u + c0;
}

// The same for a packed pair that is first multiplied by `pre2` (each lane rounded on its own): three
// packed multiplies, nothing a compiler could contract.
__device__ __forceinline__ uint32_t quant_pair_f32_pre(uint64_t x2, uint64_t pre2, const QuantConsts& c, uint32_t prev) {
  float v0, v1;
  unpack_f32x2(mul_f32x2(mul_f32x2(mul_f32x2(x2, pre2), c.np2), c.d2), v0, v1);
  v0 = __fadd_rn(v0, 12582912.0f);
  v1 = __fadd_rn(v1, 12582912.0f);
  const uint32_t c0 = (uint32_t)__viaddmin_s32_relu(max(__float_as_int(v0), 0), c.bias, 15);
  const uint32_t c1 = (uint32_t)__viaddmin_s32_relu(max(__float_as_int(v1), 0), c.bias, 15);
  return (prev * 16u + c1) * 16u + c0;
}

// Eight float32 values -> eight packed codes (value 0 in bits 0-3).
__device__ __forceinline__ uint32_t quant_word_f32(const float (&x)[8], const QuantConsts& c) {
  uint32_t w = quant_pair_f32(x[6], x[7], c, 0u);
  w = quant_pair_f32(x[4], x[5], c, w);
  w = quant_pair_f32(x[2], x[3], c, w);
  w = quant_pair_f32(x[0], x[1], c, w);
  return w ^ c.flip;
}

__device__ __forceinline__ uint32_t quant_word(const uint4& v, const QuantConsts& c) {
  uint32_t w = quant_pair(v.w, c, 0u);
  w = quant_pair(v.z, c, w);
  w = quant_pair(v.y, c, w);
  w = quant_pair(v.x, c, w);
  return w ^ c.flip;
}

// acc + the 8 squares of a chunk in float64.  The bf16 magnitude bits, moved to the top of a
// float64's high word, are the value times 2^-896 for every finite input (normal, subnormal or
// zero alike); one exact multiply by 2^896 restores it, the square is exact in float64 and the
// fused add rounds once.  Inf and NaN inputs come out as huge finite numbers here: the caller
// recognises them by the overflowing float32 sum and redoes the row with sumsq_exact.
__device__ __forceinline__ double sumsq(const uint4& v, double acc) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
  const double rebias = __hiloint2double(0x77F00000, 0);            // 2^896
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const double a = __hiloint2double((int)((w[i] & 0x7FFFu) << 13), 0) * rebias;
    const double b = __hiloint2double((int)((w[i] >> 3) & 0x0FFFE000u), 0) * rebias;
    acc = fma(a, a, acc);
    acc = fma(b, b, acc);
  }
  return acc;
}

// The same sum by the definition (float32 square, widened, added): used for rows with Inf / NaN.
__device__ __forceinline__ double sumsq_exact(const uint4& v, double acc) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float a = bf16lo_to_f32(w[i]), b = bf16hi_to_f32(w[i]);
    acc += (double)__fmul_rn(a, a);
    acc += (double)__fmul_rn(b, b);
  }
  return acc;
}

}  // namespace fpt
