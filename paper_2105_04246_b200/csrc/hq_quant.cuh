// Requantization arithmetic shared by every kernel that produces int8 codes.
//   y = fl(float(acc) * s_acc);  u = fl(y * inv_scale);  q = sat8(rint(u) + zero_point)
// one binary32 round-to-nearest-even per step, never fused (arxiv 2105.04246, Sec. 3.2: each accumulator
// output is quantized directly with a range known in advance).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace hq {

struct QParams {
  float s_acc, inv_scale;
  int zx, zp;
  int magic_sub;   // 0x4B400000 - zp
  int fast;        // parameters finite and inv_scale != 0: u can never be NaN, so the magic-number rounding is exact
};

__device__ __forceinline__ void qparams_finish(QParams& q) {
  q.magic_sub = 0x4B400000 - q.zp;
  q.fast = (isfinite(q.inv_scale) && q.inv_scale != 0.0f && isfinite(q.s_acc)) ? 1 : 0;
}

// rint(u) + zp without the (slow) float-to-int conversion pipe: add 1.5 * 2^23 (for |u| <= 2^22 the sum is rounded to
// an integer, ties to even) and read the integer out of the mantissa.  Only a lower clamp is needed: it keeps the sum
// positive, and bit patterns of positive floats are ordered like their values, so any u above the exact range yields
// an integer above 127 (up to +inf, no wrap) and any u below it an integer below -128 -- the saturating pack that
// follows gives the same code as the reference form.
__device__ __forceinline__ int round_add_zp_fast(float u, const QParams& q) {
  u = fmaxf(u, -4194304.0f);
  const float rf = __fadd_rn(u, 12582912.0f);
  return __float_as_int(rf) - q.magic_sub;
}
// reference form: saturating conversion (NaN -> 0) and saturating add
__device__ __forceinline__ int round_add_zp_slow(float u, const QParams& q) {
  const int r = __float2int_rn(u);
  int s;
  asm("add.sat.s32 %0, %1, %2;" : "=r"(s) : "r"(r), "r"(q.zp));
  return s;
}

template <bool kFast>
__device__ __forceinline__ int requant_real(float y, const QParams& q) {
  const float u = __fmul_rn(y, q.inv_scale);
  return kFast ? round_add_zp_fast(u, q) : round_add_zp_slow(u, q);
}
template <bool kFast>
__device__ __forceinline__ int requant_acc(int a, const QParams& q) {
  return requant_real<kFast>(__fmul_rn(__int2float_rn(a), q.s_acc), q);
}

// four values -> four saturated int8 codes in one word, element 0 in the lowest byte
__device__ __forceinline__ uint32_t pack_sat4(int q0, int q1, int q2, int q3) {
  uint32_t hi, d;
  asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(q3), "r"(q2), "r"(0));
  asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(q1), "r"(q0), "r"(hi));
  return d;
}

}  // namespace hq
