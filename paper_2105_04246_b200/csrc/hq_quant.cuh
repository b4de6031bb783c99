// Requantization arithmetic shared by every kernel that produces int8 codes.
//   y = fl(float(acc) * s_acc);  u = fl(y * inv_scale);  q = sat8(rint(u) + zero_point)
// one binary32 round-to-nearest-even per step, never fused (arxiv 2105.04246, Sec. 3.2: each accumulator
// output is quantized directly with a range known in advance).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "hq.h"

namespace hq {

struct QParams {
  float s_acc, inv_scale;
  int zx, zp;
  int magic_sub;   // 0x4B400000 - zp
  int fast;        // parameters finite and inv_scale != 0: u can never be NaN, so the magic-number rounding is exact
  int noclamp;     // fast, and |u| < 2^22 for every accumulator the layer can produce: the lower clamp is not needed
  int sr;          // stochastic rounding (the output state's `rounding`); draws keyed on (sr_seed, sr_iter, element index)
  uint32_t sr_seed, sr_iter;
  int count_sat;   // count the outputs the clamp changes (the output state's HQ_COUNT_SATURATION flag)
};

__device__ __forceinline__ void qparams_finish(QParams& q) {
  q.sr = 0;
  q.sr_seed = q.sr_iter = 0u;
  q.count_sat = 0;
  q.magic_sub = 0x4B400000 - q.zp;
  q.fast = (isfinite(q.inv_scale) && q.inv_scale != 0.0f && isfinite(q.s_acc)) ? 1 : 0;
  q.noclamp = 0;
}
// acc_bound: an upper bound of |accumulator| over every input the layer can see (reduction length x 255 x 128).
// |y| <= fl(acc_bound * |s_acc|) (1 + 2^-23) and |u| <= that * |inv_scale| (1 + 2^-23); a margin of 2 covers the roundings.
__device__ __forceinline__ void qparams_bound(QParams& q, float acc_bound) {
  q.noclamp = (q.fast && fabsf(q.s_acc) * acc_bound * fabsf(q.inv_scale) * 2.0f < 4194304.0f) ? 1 : 0;
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

// Two accumulators at once with the packed binary32 instructions of sm_100 (mul.rn.f32x2 / fma.rn.f32x2: per lane
// the same single round-to-nearest-even operation as the scalar forms, half the instruction slots).  kClamp as in
// round_add_zp_fast; without it the caller guarantees |u| < 2^22 (QParams::noclamp).
// The rounding add is written as fma(u, 1, magic): one rounding of u + magic, like the add, but a form the assembler
// cannot merge with the multiplication before it (it was seen to turn mul.rn.f32x2 followed by add.rn.f32x2 into one
// fused operation, which rounds once instead of twice and moves ties).
struct QPacked {
  unsigned long long s_acc2, inv2, magic2, one2;
};
__device__ __forceinline__ unsigned long long pack_f32x2(float lo, float hi) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ QPacked qpacked(const QParams& q) {
  QPacked k;
  k.s_acc2 = pack_f32x2(q.s_acc, q.s_acc);
  k.inv2 = pack_f32x2(q.inv_scale, q.inv_scale);
  k.magic2 = pack_f32x2(12582912.0f, 12582912.0f);
  k.one2 = pack_f32x2(1.0f, 1.0f);
  return k;
}
template <bool kClamp>
__device__ __forceinline__ void requant_acc2(int a0, int a1, const QParams& q, const QPacked& k, int& r0, int& r1) {
  unsigned long long x = pack_f32x2(__int2float_rn(a0), __int2float_rn(a1)), y, u, t;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(y) : "l"(x), "l"(k.s_acc2));
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(u) : "l"(y), "l"(k.inv2));
  if constexpr (kClamp) {
    float u0, u1;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(u0), "=f"(u1) : "l"(u));
    u = pack_f32x2(fmaxf(u0, -4194304.0f), fmaxf(u1, -4194304.0f));
  }
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(t) : "l"(u), "l"(k.one2), "l"(k.magic2));
  int b0, b1;
  asm("mov.b64 {%0, %1}, %2;" : "=r"(b0), "=r"(b1) : "l"(t));
  r0 = b0 - q.magic_sub;
  r1 = b1 - q.magic_sub;
}
template <bool kClamp>
__device__ __forceinline__ uint32_t requant_pack4(int a0, int a1, int a2, int a3, const QParams& q, const QPacked& k);

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

// rounding mode and statistics flags of the tensor a kernel writes (`rounding` word of its range state; `step` = the
// state's update count at the time the draws are taken)
__device__ __forceinline__ void qparams_output_mode(QParams& q, uint32_t rounding, uint32_t seed, uint32_t step) {
  if ((rounding & HQ_ROUND_MODE_MASK) == HQ_ROUND_STOCHASTIC) {
    q.sr = 1;
    q.sr_seed = seed;
    q.sr_iter = step;
  }
  q.count_sat = (rounding & HQ_COUNT_SATURATION) ? 1 : 0;
}

// Saturation statistic (Sec. 4: "the proportion of values that lie outside the quantization grid", as counts): r is the
// rounded grid coordinate plus the zero point, before the saturating pack; counted when the pack changes it.
__device__ __forceinline__ void count_clipped(int r, int& below, int& above) {
  below += r < -128 ? 1 : 0;
  above += r > 127 ? 1 : 0;
}
// four rounded values -> four codes; counts the clipped ones when the tensor asks for it
__device__ __forceinline__ uint32_t finish4(int r0, int r1, int r2, int r3, const QParams& q, int& below, int& above) {
  if (q.count_sat) {
    count_clipped(r0, below, above);
    count_clipped(r1, below, above);
    count_clipped(r2, below, above);
    count_clipped(r3, below, above);
  }
  return pack_sat4(r0, r1, r2, r3);
}

template <bool kClamp>
__device__ __forceinline__ uint32_t requant_pack4(int a0, int a1, int a2, int a3, const QParams& q, const QPacked& k) {
  int r0, r1, r2, r3;
  requant_acc2<kClamp>(a0, a1, q, k, r0, r1);
  requant_acc2<kClamp>(a2, a3, q, k, r2, r3);
  return pack_sat4(r0, r1, r2, r3);
}

// The straight-line epilogue pass over eight accumulators of one output row: zero-point correction from the shared
// table (already multiplied by the input zero point), running min/max, requantization, two words of codes.
// zrow: the eight corrections of these columns; elem: linear index of the first element in the output tensor (a multiple
// of 8: one generator call covers the eight draws of stochastic rounding).  Requires q.fast.
// kMode selects the rounding at compile time, so that a kernel's tile loop holds one variant only:
//   kLeanNoClamp  nearest even, |u| < 2^22 guaranteed (QParams::noclamp)   kLeanClamp  nearest even   kLeanSr  stochastic
enum LeanMode : int { kLeanNoClamp = 0, kLeanClamp = 1, kLeanSr = 2 };
__device__ __forceinline__ int lean_mode(const QParams& q) { return q.sr ? kLeanSr : (q.noclamp ? kLeanNoClamp : kLeanClamp); }
template <int kMode>
__device__ __forceinline__ void lean_half8c(int (&x)[8], int4 ca, int4 cb, int& tmn, int& tmx, const QParams& q, const QPacked& qk, int64_t elem,
                                            uint32_t& w0, uint32_t& w1);
template <int kMode>
__device__ __forceinline__ void lean_half8m(int (&x)[8], const int32_t* zrow, int& tmn, int& tmx, const QParams& q, const QPacked& qk, int64_t elem,
                                            uint32_t& w0, uint32_t& w1) {
  lean_half8c<kMode>(x, *reinterpret_cast<const int4*>(zrow), *reinterpret_cast<const int4*>(zrow + 4), tmn, tmx, q, qk, elem, w0, w1);
}
// the same with the eight corrections already in registers (callers that fetch them ahead of the accumulators)
template <int kMode>
__device__ __forceinline__ void lean_half8c(int (&x)[8], int4 ca, int4 cb, int& tmn, int& tmx, const QParams& q, const QPacked& qk, int64_t elem,
                                            uint32_t& w0, uint32_t& w1) {
  x[0] -= ca.x; x[1] -= ca.y; x[2] -= ca.z; x[3] -= ca.w;
  x[4] -= cb.x; x[5] -= cb.y; x[6] -= cb.z; x[7] -= cb.w;
  tmn = __vimin3_s32(tmn, x[0], x[1]); tmx = __vimax3_s32(tmx, x[0], x[1]);
  tmn = __vimin3_s32(tmn, x[2], x[3]); tmx = __vimax3_s32(tmx, x[2], x[3]);
  tmn = __vimin3_s32(tmn, x[4], x[5]); tmx = __vimax3_s32(tmx, x[4], x[5]);
  tmn = __vimin3_s32(tmn, x[6], x[7]); tmx = __vimax3_s32(tmx, x[6], x[7]);
  if constexpr (kMode == kLeanSr) {   // stochastic rounding: one aligned block of eight elements, one generator call
    uint32_t h[8];
    sr_draws8(q, (uint64_t)elem >> 3, h);
    w0 = pack_sat4(requant_acc_sr<true>(x[0], h[0], q), requant_acc_sr<true>(x[1], h[1], q), requant_acc_sr<true>(x[2], h[2], q),
                   requant_acc_sr<true>(x[3], h[3], q));
    w1 = pack_sat4(requant_acc_sr<true>(x[4], h[4], q), requant_acc_sr<true>(x[5], h[5], q), requant_acc_sr<true>(x[6], h[6], q),
                   requant_acc_sr<true>(x[7], h[7], q));
  } else if constexpr (kMode == kLeanNoClamp) {
    w0 = requant_pack4<false>(x[0], x[1], x[2], x[3], q, qk);
    w1 = requant_pack4<false>(x[4], x[5], x[6], x[7], q, qk);
  } else {
    w0 = requant_pack4<true>(x[0], x[1], x[2], x[3], q, qk);
    w1 = requant_pack4<true>(x[4], x[5], x[6], x[7], q, qk);
  }
}
// the same with the rounding chosen at run time
__device__ __forceinline__ void lean_half8(int (&x)[8], const int32_t* zrow, int& tmn, int& tmx, const QParams& q, const QPacked& qk, int64_t elem,
                                           uint32_t& w0, uint32_t& w1) {
  if (q.sr) lean_half8m<kLeanSr>(x, zrow, tmn, tmx, q, qk, elem, w0, w1);
  else if (q.noclamp) lean_half8m<kLeanNoClamp>(x, zrow, tmn, tmx, q, qk, elem, w0, w1);
  else lean_half8m<kLeanClamp>(x, zrow, tmn, tmx, q, qk, elem, w0, w1);
}

// four accumulators whose first element has linear index e (a multiple of 4) -> four codes, whatever the rounding mode
__device__ __forceinline__ uint32_t quant4_acc(int a0, int a1, int a2, int a3, int64_t e, const QParams& q, int& below, int& above) {
  int r0, r1, r2, r3;
  if (q.sr) {
    uint32_t h[8];
    sr_draws8(q, (uint64_t)e >> 3, h);
    const int o = (int)(e & 4);
    if (q.fast) {
      r0 = requant_acc_sr<true>(a0, h[o], q); r1 = requant_acc_sr<true>(a1, h[o + 1], q);
      r2 = requant_acc_sr<true>(a2, h[o + 2], q); r3 = requant_acc_sr<true>(a3, h[o + 3], q);
    } else {
      r0 = requant_acc_sr<false>(a0, h[o], q); r1 = requant_acc_sr<false>(a1, h[o + 1], q);
      r2 = requant_acc_sr<false>(a2, h[o + 2], q); r3 = requant_acc_sr<false>(a3, h[o + 3], q);
    }
  } else if (q.fast) {
    r0 = requant_acc<true>(a0, q); r1 = requant_acc<true>(a1, q); r2 = requant_acc<true>(a2, q); r3 = requant_acc<true>(a3, q);
  } else {
    r0 = requant_acc<false>(a0, q); r1 = requant_acc<false>(a1, q); r2 = requant_acc<false>(a2, q); r3 = requant_acc<false>(a3, q);
  }
  return finish4(r0, r1, r2, r3, q, below, above);
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
