// Sigmoid evaluation shared by the bf16 forward and backward kernels.
//
// With a = log2(e) * x and u = 2^a the weight is P = u / (1 + u) and 1 - P = 1 / (1 + u).
// Both kernels work on a block of 32 or 64 logits of one thread at a time and evaluate
//
//   fast path   t = 1 - u + u^2,  P = u t,  P (1 - P) = P t
//               (the alternating series of 1 / (1 + u) cut after u^2: relative error
//               u^3 <= 2^-12 for a <= -4, i.e. below bf16 resolution; one MUFU op per
//               element).  It is computed unconditionally, so that nothing waits on the
//               reduction that decides whether it was allowed.
//   exact path  e = 2^-a,  r = 1 / (1 + e),  P = r,  P (1 - P) = r e r  (two MUFU ops),
//               taken afterwards if any logit of the block has a > -4.  At b = -log n almost
//               no chunk needs it.
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

// a[N] (already scaled by log2 e) -> P[N]; if WITH_SLOPE also P (1 - P) in pp[N].
// SPECULATE = true evaluates the fast path before the decision is known (shortest
// dependency chain, more live registers); false decides first.
template <int N, bool WITH_SLOPE, bool SPECULATE>
__device__ __forceinline__ void sigmoid_block(const float (&a)[N], float (&pr)[N], float* pp) {
  bool exact;
  if (!SPECULATE) exact = max_tree<N>(a) > kFastPathMaxA;
  if (SPECULATE || !exact) {
#pragma unroll
    for (int i = 0; i < N; ++i) {
      const float u = sm100::ex2_approx(a[i]);
      float t = 1.0f - u;
      t = fmaf(u, u, t);
      pr[i] = u * t;
      if (WITH_SLOPE) pp[i] = pr[i] * t;
    }
  }
  if (SPECULATE) exact = max_tree<N>(a) > kFastPathMaxA;
  if (exact) {
#pragma unroll
    for (int i = 0; i < N; ++i) {
      const float e = sm100::ex2_approx(fminf(-a[i], 120.0f));
      const float r = sm100::rcp_approx(1.0f + e);
      pr[i] = r;
      if (WITH_SLOPE) pp[i] = r * (e * r);
    }
  }
}

}  // namespace sigattn
