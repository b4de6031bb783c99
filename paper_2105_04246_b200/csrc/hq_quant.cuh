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
  int sr;          // stochastic rounding (the output state's `rounding`); draws keyed on (sr_seed, sr_iter, element index)
  uint32_t sr_seed, sr_iter;
};

__device__ __forceinline__ void qparams_finish(QParams& q) {
  q.sr = 0;
  q.sr_seed = q.sr_iter = 0u;
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

// ---- stochastic rounding (the paper's rounding for gradients) ----------------------------------------------------
// code = sat8(floor(fl(u + r)) + zp), r = h / 65536 with h a 16-bit draw of the counter-based generator
// Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11): ten rounds of two 32x32 -> 64-bit multiplications by fixed
// odd constants whose high halves are crossed into the other lane pair together with the round key.
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1, uint32_t (&out)[4]) {
#pragma unroll
  for (int round = 0; round < 10; ++round) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0;
    c1 = lo1;
    c2 = n2;
    c3 = lo0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  out[0] = c0;
  out[1] = c1;
  out[2] = c2;
  out[3] = c3;
}
// the eight 16-bit draws of the elements 8*block .. 8*block + 7 (low half of each word first)
__device__ __forceinline__ void sr_draws8(const QParams& q, uint64_t block, uint32_t (&h)[8]) {
  uint32_t w[4];
  philox4x32_10((uint32_t)block, (uint32_t)(block >> 32), q.sr_iter, 0u, q.sr_seed, 0u, w);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    h[2 * i] = w[i] & 0xFFFFu;
    h[2 * i + 1] = w[i] >> 16;
  }
}
__device__ __forceinline__ uint32_t sr_draw1(const QParams& q, int64_t e) {
  uint32_t w[4];
  const uint64_t block = (uint64_t)e >> 3;
  philox4x32_10((uint32_t)block, (uint32_t)(block >> 32), q.sr_iter, 0u, q.sr_seed, 0u, w);
  const uint32_t word = w[((uint32_t)e & 7u) >> 1];
  return (e & 1) ? (word >> 16) : (word & 0xFFFFu);
}
// floor(t) + zp for t = fl(u + r).  Fast form: the magic-number sum gives rint(t) (exact for |t| < 2^22), one less
// where that lies above t; outside that range the result only has to saturate the right way, as for nearest-even.
template <bool kFast>
__device__ __forceinline__ int requant_real_sr(float y, uint32_t h, const QParams& q) {
  const float u = __fmul_rn(y, q.inv_scale);
  const float r = __fmul_rn(__uint2float_rn(h), 1.52587890625e-05f);   // h / 65536, exact
  float t = __fadd_rn(u, r);
  if (kFast) {
    t = fmaxf(t, -4194304.0f);
    const float rf = __fadd_rn(t, 12582912.0f);
    const float nf = __fsub_rn(rf, 12582912.0f);
    return __float_as_int(rf) - q.magic_sub - (nf > t ? 1 : 0);
  }
  const int fl = __float2int_rd(t);   // saturating, NaN -> 0
  int s;
  asm("add.sat.s32 %0, %1, %2;" : "=r"(s) : "r"(fl), "r"(q.zp));
  return s;
}
template <bool kFast>
__device__ __forceinline__ int requant_acc_sr(int a, uint32_t h, const QParams& q) {
  return requant_real_sr<kFast>(__fmul_rn(__int2float_rn(a), q.s_acc), h, q);
}

// four values -> four saturated int8 codes in one word, element 0 in the lowest byte
__device__ __forceinline__ uint32_t pack_sat4(int q0, int q1, int q2, int q3) {
  uint32_t hi, d;
  asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(q3), "r"(q2), "r"(0));
  asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(q1), "r"(q0), "r"(hi));
  return d;
}

// four accumulators whose first element has linear index e (a multiple of 4) -> four codes with stochastic rounding
__device__ __forceinline__ uint32_t pack4_sr(int a0, int a1, int a2, int a3, int64_t e, const QParams& q) {
  uint32_t h[8];
  sr_draws8(q, (uint64_t)e >> 3, h);
  const int o = (int)(e & 4);
  return q.fast ? pack_sat4(requant_acc_sr<true>(a0, h[o], q), requant_acc_sr<true>(a1, h[o + 1], q), requant_acc_sr<true>(a2, h[o + 2], q),
                            requant_acc_sr<true>(a3, h[o + 3], q))
                : pack_sat4(requant_acc_sr<false>(a0, h[o], q), requant_acc_sr<false>(a1, h[o + 1], q),
                            requant_acc_sr<false>(a2, h[o + 2], q), requant_acc_sr<false>(a3, h[o + 3], q));
}

}  // namespace hq
