// Sigmoid evaluation shared by the bf16 forward and backward kernels.
//
// With a = log2(e) * x and u = 2^a the weight is P = u / (1 + u) and 1 - P = 1 / (1 + u).
// Both kernels work on a block of 32 or 64 logits of one thread at a time and evaluate
//
//   common path  P = u - u^2 + u^3, the alternating series of u / (1 + u) (relative error
//                u^3 <= 2^-12 for a <= -4, below bf16 resolution), and P (1 - P) = P - P^2;
//                one exponential per element; where the MUFU pipe is the bound (forward at
//                D = 64) a fixed share of them is evaluated on the FMA pipe (ex2_emulated).
//   exact path   e = 2^-a,  r = 1 / (1 + e),  P = r,  P (1 - P) = r e r, taken if any logit of
//                the block has a > -4.  In the forward the reciprocal is formed on the FMA and ALU
//                pipes (an integer first guess and two Newton steps, see rcp_newton), so this path
//                also costs one MUFU op per element there (measured: +13 % on the ViT shape, +9 % at
//                b = 0); the backward, whose activation is not MUFU-bound, keeps the MUFU reciprocal
//                (the Newton form measured 3-8 % slower there).  At b = -log n with normalised q, k almost no
//                block needs it; with unnormalised inputs of unit variance at n = 197 (the ViT
//                shape) about one thread in five does, and since the threads of a warp decide
//                one by one, most warps then run both paths.
//
// The paper evaluates sigmoid as 0.5 (1 + tanh(x / 2)) with the hardware tanh (Section 4).
// On B200 tanh.approx.f32 followed by 0.5 + 0.5 t loses P's relative accuracy for x << 0
// (measured: 1 % at x = -9, 100 % below x = -16), which at b = -log n is where all the
// mass is, so the exponential form is used instead; it costs the same single MUFU op.
#pragma once

#include "sm100_primitives.cuh"

namespace sigattn {

constexpr float kFastPathMaxA = -4.0f;

// max of N values (N = 32 or 64) as a tree of 3-input max ops
template <int N>
__device__ __forceinline__ float max_tree(const float (&a)[N]) {
  static_assert(N == 32 || N == 64, "unsupported width");
  float m[N / 2];
  // level 1: N values -> ceil(N / 3) partial maxima
  constexpr int L1 = (N + 2) / 3;
#pragma unroll
  for (int i = 0; i < N / 3; ++i) m[i] = sm100::fmax3(a[3 * i], a[3 * i + 1], a[3 * i + 2]);
  if (N % 3 == 2) m[L1 - 1] = fmaxf(a[N - 2], a[N - 1]);
  if (N % 3 == 1) m[L1 - 1] = a[N - 1];
  int n = L1;  // 11 or 22
#pragma unroll
  for (int level = 0; level < 4; ++level) {
    if (n > 1) {
      const int groups = n / 3, rest = n % 3;
#pragma unroll
      for (int i = 0; i < groups; ++i) m[i] = sm100::fmax3(m[3 * i], m[3 * i + 1], m[3 * i + 2]);
      if (rest == 2) m[groups] = fmaxf(m[n - 2], m[n - 1]);
      if (rest == 1) m[groups] = m[n - 1];
      n = groups + (rest ? 1 : 0);
    }
  }
  return m[0];
}

// 2^a on the FMA and ALU pipes instead of the MUFU pipe: a = n + f with n = round(a),
// 2^f from a cubic on [-0.5, 0.5] (relative error 7.5e-5 = 2^-13.7, fitted for this
// interval), 2^n by adding n to the exponent field.  Valid for -120 <= a (clamped) and
// a < 100.  Used for a fixed share of the elements to take load off the MUFU pipe, which
// otherwise bounds the activation at 16 elements per clock per SM.
__device__ __forceinline__ float ex2_emulated(float a) {
  a = fmaxf(a, -120.0f);
  const float t = a + 12582912.0f;  // 1.5 * 2^23: the rounded integer lands in the low mantissa bits
  const float f = a - (t - 12582912.0f);
  float p = fmaf(0.05517145885f, f, 0.2426108620f);
  p = fmaf(p, f, 0.6932609924f);
  p = fmaf(p, f, 0.9999280895f);
  return __int_as_float(__float_as_int(p) + (__float_as_int(t) << 23));
}

// Common path: u / (1 + u) = u - u^2 + u^3 - ..., cut after u^3 and evaluated as
// u - u (u - u^2): two FMAs; relative error u^3 <= 2^-12 for a <= -4.
// EMULATE_EVERY = m > 0 evaluates every m-th exponential on the FMA pipe, 0 none.
template <int N, bool WITH_SLOPE, int EMULATE_EVERY>
__device__ __forceinline__ void sigmoid_common(const float (&a)[N], float (&pr)[N], float* pp) {
#pragma unroll
  for (int i = 0; i < N; ++i) {
    const bool emulate = EMULATE_EVERY > 0 && i % (EMULATE_EVERY > 0 ? EMULATE_EVERY : 1) == EMULATE_EVERY - 1;
    const float u = emulate ? ex2_emulated(a[i]) : sm100::ex2_approx(a[i]);
    const float w = fmaf(-u, u, u);
    pr[i] = fmaf(-u, w, u);
    if (WITH_SLOPE) pp[i] = fmaf(-pr[i], pr[i], pr[i]);  // P <= 1/17 here: no cancellation in P - P^2
  }
}

// 1 / y for 1 <= y < 2^126 without the MUFU pipe: the bit pattern of y subtracted from a constant
// gives a first guess within 5 %, and two Newton steps r <- r (2 - y r) bring the relative error to
// 7e-6 (checked over [1, 2) times every power of two used; the error pattern repeats per binade).
__device__ __forceinline__ float rcp_newton(float y) {
  float r = __int_as_float(0x7EF311C7 - __float_as_int(y));
  r = r * fmaf(-y, r, 2.0f);
  r = r * fmaf(-y, r, 2.0f);
  return r;
}

// Exact path: r = 1 / (1 + 2^-a) = P, and 1 - P = 2^-a r (no subtraction from a rounded P).
template <int N, bool WITH_SLOPE>
__device__ __forceinline__ void sigmoid_exact(const float (&a)[N], float (&pr)[N], float* pp) {
#pragma unroll
  for (int i = 0; i < N; ++i) {
    const float e = sm100::ex2_approx(fminf(-a[i], 120.0f));
    const float r = WITH_SLOPE ? sm100::rcp_approx(1.0f + e) : rcp_newton(1.0f + e);
    pr[i] = r;
    if (WITH_SLOPE) pp[i] = r * (e * r);
  }
}

// a[N] (already scaled by log2 e) -> P[N]; if WITH_SLOPE also P (1 - P) in pp[N].
// The block's largest a decides between the two paths before anything else is evaluated.
template <int N, bool WITH_SLOPE, int EMULATE_EVERY>
__device__ __forceinline__ void sigmoid_block(const float (&a)[N], float (&pr)[N], float* pp) {
  if (max_tree<N>(a) <= kFastPathMaxA) sigmoid_common<N, WITH_SLOPE, EMULATE_EVERY>(a, pr, pp);
  else sigmoid_exact<N, WITH_SLOPE>(a, pr, pp);
}

}  // namespace sigattn
