// Small kernels around the layer kernels: range update (Eq. 2-3), the dynamic path's derive and
// quantize passes (Eq. 1), weight preparation, and the depthwise convolution on CUDA cores.
// arxiv 2105.04246; equation numbers refer to that paper.
#include <cuda_runtime.h>
#include <stdint.h>

#include <algorithm>

#include "hq_device.cuh"
#include "hq_internal.h"
#include "hq_quant.cuh"

namespace hq {
namespace {

// Grid derived from the running range: the range is widened to contain 0, split into 255 steps.
__device__ __forceinline__ void derive_grid(hq_range_state* s) {
  const float lo = s->q_min < 0.0f ? s->q_min : 0.0f;
  const float hi = s->q_max > 0.0f ? s->q_max : 0.0f;
  float scale = __fdiv_rn(__fsub_rn(hi, lo), 255.0f);
  if (!(scale > 0.0f)) scale = 1.0f;
  s->scale = scale;
  s->inv_scale = __fdiv_rn(1.0f, scale);
  const long long r = (long long)__float2int_rn(__fdiv_rn(lo, scale));
  long long z = -128ll - r;
  z = z < -128 ? -128 : (z > 127 ? 127 : z);
  s->zero_point = (int32_t)z;
}

__global__ void range_update_kernel(hq_range_state* st, int count, float eta) {
  grid_dependency_wait();   // launched ahead of its predecessor's end: see launch_overlapped
  grid_launch_dependents();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= count) return;
  hq_range_state* s = st + i;
  const int mn = s->acc_min, mx = s->acc_max;
  if (mn > mx) return;  // no layer wrote statistics: leave the state alone
  const float m_lo = __fmul_rn(__int2float_rn(mn), s->acc_scale);
  const float m_hi = __fmul_rn(__int2float_rn(mx), s->acc_scale);
  if (s->step == 0) {  // t = 0: the range is the first tensor's min/max
    s->q_min = m_lo;
    s->q_max = m_hi;
  } else {  // Eq. 2-3
    const float ome = __fsub_rn(1.0f, eta);
    s->q_min = __fadd_rn(__fmul_rn(ome, m_lo), __fmul_rn(eta, s->q_min));
    s->q_max = __fadd_rn(__fmul_rn(ome, m_hi), __fmul_rn(eta, s->q_max));
  }
  s->step += 1;
  derive_grid(s);
  s->acc_min = INT32_MAX;
  s->acc_max = INT32_MIN;
  s->last_sat_below = s->sat_below;   // the saturation counts of the tensor just finished
  s->last_sat_above = s->sat_above;
  s->sat_below = 0u;
  s->sat_above = 0u;
}

// Batch-sharded data parallelism: the only exchange of the method is the statistics.  pack writes {acc_min, ~acc_max}
// of every state into one int32 array (the complement reverses the order without overflow, so ONE element-wise MIN
// all-reduce over the ranks serves both columns; an empty slot {INT32_MAX, INT32_MIN} is its identity); unpack puts the
// reduced pair back, after which every rank applies Eq. 2-3 to identical numbers.
__global__ void stats_pack_kernel(const hq_range_state* st, int count, int32_t* buf) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= count) return;
  buf[i] = st[i].acc_min;
  buf[count + i] = ~st[i].acc_max;
}
__global__ void stats_unpack_kernel(hq_range_state* st, int count, const int32_t* buf) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= count) return;
  st[i].acc_min = buf[i];
  st[i].acc_max = ~buf[count + i];
}

// Eq. 1: the range is the min/max of the tensor that was just written; with dynamic_eta > 0, its moving average.
__global__ void dynamic_derive_kernel(hq_range_state* s) {
  grid_dependency_wait();   // launched ahead of its predecessor's end: see launch_overlapped
  grid_launch_dependents();
  const int mn = s->acc_min, mx = s->acc_max;
  if (mn > mx) return;
  const float m_lo = __fmul_rn(__int2float_rn(mn), s->acc_scale);
  const float m_hi = __fmul_rn(__int2float_rn(mx), s->acc_scale);
  const float eta = s->dynamic_eta;
  if (s->step == 0 || eta == 0.0f) {   // current min-max
    s->q_min = m_lo;
    s->q_max = m_hi;
  } else {   // running min-max (Sec. 4.1): Eq. 2-3 over the current tensor's statistics
    const float ome = __fsub_rn(1.0f, eta);
    s->q_min = __fadd_rn(__fmul_rn(ome, m_lo), __fmul_rn(eta, s->q_min));
    s->q_max = __fadd_rn(__fmul_rn(ome, m_hi), __fmul_rn(eta, s->q_max));
  }
  s->step += 1;
  derive_grid(s);
  s->acc_min = INT32_MAX;
  s->acc_max = INT32_MIN;
  s->last_sat_below = 0u;   // the quantize pass that follows counts this tensor's clipped outputs straight into these
  s->last_sat_above = 0u;
  s->sat_below = 0u;
  s->sat_above = 0u;
}

// second pass of the dynamic path: read the binary32 output back and quantize it
__global__ void quantize_pass_kernel(const float* __restrict__ y, int8_t* __restrict__ out, int64_t count, hq_range_state* st) {
  grid_dependency_wait();   // launched ahead of its predecessor's end: see launch_overlapped
  QParams q;
  q.s_acc = 1.0f;
  q.zx = 0;
  q.inv_scale = st->inv_scale;
  q.zp = st->zero_point;
  qparams_finish(q);
  qparams_output_mode(q, st->rounding, st->seed, st->step - 1u);   // the derive kernel has already counted this iteration
  int sat_below = 0, sat_above = 0;
  const int64_t groups = count / 16;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; g < groups; g += stride) {
    const float4* src = reinterpret_cast<const float4*>(y) + 4 * g;
    uint32_t w[4];
    if (q.sr) {   // elements 16g .. 16g + 15: two blocks of eight draws
#pragma unroll
      for (int b = 0; b < 2; ++b) {
        uint32_t h[8];
        sr_draws8(q, (uint64_t)(2 * g + b), h);
        const float4 f0 = __ldcs(src + 2 * b), f1 = __ldcs(src + 2 * b + 1);
        w[2 * b] = q.fast ? finish4(requant_real_sr<true>(f0.x, h[0], q), requant_real_sr<true>(f0.y, h[1], q),
                                    requant_real_sr<true>(f0.z, h[2], q), requant_real_sr<true>(f0.w, h[3], q), q, sat_below, sat_above)
                          : finish4(requant_real_sr<false>(f0.x, h[0], q), requant_real_sr<false>(f0.y, h[1], q),
                                    requant_real_sr<false>(f0.z, h[2], q), requant_real_sr<false>(f0.w, h[3], q), q, sat_below, sat_above);
        w[2 * b + 1] = q.fast ? finish4(requant_real_sr<true>(f1.x, h[4], q), requant_real_sr<true>(f1.y, h[5], q),
                                        requant_real_sr<true>(f1.z, h[6], q), requant_real_sr<true>(f1.w, h[7], q), q, sat_below, sat_above)
                              : finish4(requant_real_sr<false>(f1.x, h[4], q), requant_real_sr<false>(f1.y, h[5], q),
                                        requant_real_sr<false>(f1.z, h[6], q), requant_real_sr<false>(f1.w, h[7], q), q, sat_below, sat_above);
      }
    } else {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float4 f = __ldcs(src + e);
        w[e] = q.fast ? finish4(requant_real<true>(f.x, q), requant_real<true>(f.y, q), requant_real<true>(f.z, q), requant_real<true>(f.w, q), q,
                                sat_below, sat_above)
                      : finish4(requant_real<false>(f.x, q), requant_real<false>(f.y, q), requant_real<false>(f.z, q), requant_real<false>(f.w, q), q,
                                sat_below, sat_above);
      }
    }
    reinterpret_cast<uint4*>(out)[g] = make_uint4(w[0], w[1], w[2], w[3]);
  }
  grid_launch_dependents();   // the successor may take the SMs that free up from here on
  if (blockIdx.x == 0) {
    for (int64_t i = groups * 16 + threadIdx.x; i < count; i += blockDim.x) {
      const int r = q.sr ? requant_real_sr<false>(y[i], sr_draw1(q, i), q) : requant_real<false>(y[i], q);
      if (q.count_sat) count_clipped(r, sat_below, sat_above);
      out[i] = (int8_t)min(max(r, -128), 127);
    }
  }
  if (q.count_sat) {   // this tensor's clipped outputs (the derive kernel cleared the pair)
    sat_below = __reduce_add_sync(0xffffffffu, sat_below);
    sat_above = __reduce_add_sync(0xffffffffu, sat_above);
    if ((threadIdx.x & 31) == 0) {
      if (sat_below) atomicAdd(&st->last_sat_below, (uint32_t)sat_below);
      if (sat_above) atomicAdd(&st->last_sat_above, (uint32_t)sat_above);
    }
  }
}

// ---- weight preparation -----------------------------------------------------------------------
struct TapList {
  int8_t r[kMaxTaps], s[kMaxTaps];
};
struct ClassMasks {
  uint32_t row[16], col[16];
};

// Wmat[n][t][c] (row length ntaps*Cpad, zero padded) from the forward filter W[Ksrc][R][S][Csrc]:
//   plain      : W[n][r_t][s_t][c]
//   transposed : W[c][r_t][s_t][n]                       (backward data: rows are input channels)
//   g > 1      : g copies of that matrix on the block diagonal (g pixels folded into one GEMM row)
__global__ void prep_weights_kernel(const int8_t* __restrict__ W, int8_t* __restrict__ Wmat, int Nout, int ntaps, int Cpad, int Ksrc, int R, int S,
                                    int Csrc, TapList taps, int transposed, int g) {
  const int64_t total = (int64_t)Nout * ntaps * Cpad;
  for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
    const int c = (int)(idx % Cpad);
    const int t = (int)((idx / Cpad) % ntaps);
    const int n = (int)(idx / ((int64_t)Cpad * ntaps));
    int8_t v = 0;
    const int r = taps.r[t], s = taps.s[t];
    const int rows_per = transposed ? Csrc : Ksrc;   // GEMM rows of one block
    const int cols_per = transposed ? Ksrc : Csrc;   // GEMM columns (reduction) of one block
    int nn = n, cc = c;
    if (g > 1) {
      const int j = n / rows_per;
      nn = n % rows_per;
      cc = c - j * cols_per;
    }
    if (cc >= 0 && cc < cols_per)
      v = transposed ? W[(((int64_t)cc * R + r) * S + s) * Csrc + nn] : W[(((int64_t)nn * R + r) * S + s) * Csrc + cc];
    Wmat[idx] = v;
  }
}

// corr[(rc*ncolcls + cc)*corr_ld + n] = sum of Wmat[n][t][:] over the taps t = (ri, si) that are inside
// the image for border class (rc, cc).  Multiplied by the input zero point in the epilogue, this is
// what the zero-filled padding taps did NOT contribute.
__global__ void corr_kernel(const int8_t* __restrict__ Wmat, int32_t* __restrict__ corr, int Nout, int ntaps, int Cpad, int nrowtaps, int ncoltaps,
                            ClassMasks m, int nrowcls, int ncolcls, int corr_ld) {
  // one warp per (class, output channel); Cpad is a multiple of 16, rows are 16-byte aligned
  const int idx = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (idx >= nrowcls * ncolcls * Nout) return;
  const int n = idx % Nout;
  const int cls = idx / Nout;
  const int rc = cls / ncolcls, cc = cls % ncolcls;
  int32_t sum = 0;
  for (int ri = 0; ri < nrowtaps; ++ri) {
    if (!((m.row[rc] >> ri) & 1u)) continue;
    for (int si = 0; si < ncoltaps; ++si) {
      if (!((m.col[cc] >> si) & 1u)) continue;
      const uint4* w = reinterpret_cast<const uint4*>(Wmat + ((int64_t)n * ntaps + (ri * ncoltaps + si)) * Cpad);
      for (int c = lane; c < Cpad / 16; c += 32) {
        const uint4 q = w[c];
        sum = __dp4a((int)q.x, 0x01010101, sum);
        sum = __dp4a((int)q.y, 0x01010101, sum);
        sum = __dp4a((int)q.z, 0x01010101, sum);
        sum = __dp4a((int)q.w, 0x01010101, sum);
      }
    }
  }
  sum = __reduce_add_sync(0xffffffffu, sum);
  if (lane == 0) corr[(int64_t)cls * corr_ld + n] = sum;
}

// depthwise: weights to tap-major [R*S][C]; corr[cls][c] = sum of valid taps
// flip: tap t of the prepared filter is tap R*S-1-t of W (the filter turned by 180 degrees, which makes backward data
// of a stride-1 depthwise layer a forward depthwise layer over the output gradient)
__global__ void dw_prep_kernel(const int8_t* __restrict__ W, int8_t* __restrict__ Wt, int32_t* __restrict__ corr, int C, int R, int S, ClassMasks m,
                               int nrowcls, int ncolcls, int flip) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx < C * R * S) {
    const int c = idx % C, t = idx / C;
    Wt[idx] = W[c * R * S + (flip ? R * S - 1 - t : t)];
  }
  if (idx < nrowcls * ncolcls * C) {
    const int c = idx % C, cls = idx / C;
    const int rc = cls / ncolcls, cc = cls % ncolcls;
    int32_t sum = 0;
    for (int r = 0; r < R; ++r)
      for (int s = 0; s < S; ++s)
        if (((m.row[rc] >> r) & 1u) && ((m.col[cc] >> s) & 1u)) sum += W[c * R * S + (flip ? R * S - 1 - (r * S + s) : r * S + s)];
    corr[idx] = sum;
  }
}

// dense form of the depthwise filter of channels [c0, c0 + cw): Wd[k][tap][c] = (c == k) ? W[c0 + k][tap] : 0
__global__ void dw_dense_kernel(const int8_t* __restrict__ W, int8_t* __restrict__ Wd, int taps, int c0, int cw) {
  const int total = cw * taps * cw;
  for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
    const int c = idx % cw;
    const int kt = idx / cw;
    const int k = kt / taps, t = kt - k * taps;
    Wd[idx] = c == k ? W[(int64_t)(c0 + k) * taps + t] : (int8_t)0;
  }
}

// ---- operand repacking for shapes no TMA box can address ------------------------------------------
// A[m][r*RP + j], j = s*C + c < S*C: the filter window of output pixel m, one filter row per RP-byte slot
// (RP = S*C rounded up to 8).  Taps on padding hold the input zero point (real zero); slot bytes beyond S*C hold
// whatever follows in the input row -- their weights are zero.  For a fixed filter row the S*C input bytes are
// contiguous in NHWC, so thread (pixel, r) moves that run with aligned 32-bit loads and a funnel shift into the
// pixel's row in shared memory; the block then writes its rows out with 16-byte stores.
constexpr int kPatchPixels = 32;   // output pixels per block iteration
__global__ void __launch_bounds__(256) patch_matrix_kernel(const int8_t* __restrict__ x, int8_t* __restrict__ A, const hq_range_state* xq, int N,
                                                           int H, int W, int C, int Ho, int Wo, int R, int S, int stride_h, int stride_w,
                                                           int pad_h, int pad_w, int Kp, int RP) {
  extern __shared__ __align__(16) int8_t rows_s[];   // [kPatchPixels][Kp]
  const int zx = xq->zero_point;
  const uint32_t zx4 = ((uint32_t)zx & 0xffu) * 0x01010101u;
  const int sc = S * C, used = R * RP, nw = RP / 4;
  const int64_t M = (int64_t)N * Ho * Wo;
  const int8_t* x_end = x + (int64_t)N * H * W * C;   // no load starts at or beyond this address
  for (int64_t m0 = (int64_t)blockIdx.x * kPatchPixels; m0 < M; m0 += (int64_t)gridDim.x * kPatchPixels) {
    for (int t = threadIdx.x; t < kPatchPixels * (Kp - used); t += blockDim.x)   // columns after the last slot
      rows_s[(t / (Kp - used)) * Kp + used + t % (Kp - used)] = 0;
    for (int t = threadIdx.x; t < kPatchPixels * R; t += blockDim.x) {
      const int pl = t / R, r = t - pl * R;
      const int64_t m = m0 + pl;
      if (m >= M) continue;
      const int wo = (int)(m % Wo);
      const int ho = (int)((m / Wo) % Ho);
      const int n = (int)(m / ((int64_t)Wo * Ho));
      const int hi = ho * stride_h - pad_h + r;
      const int wi0 = wo * stride_w - pad_w;
      int8_t* dst = rows_s + pl * Kp + r * RP;   // 8-byte aligned
      uint32_t* dst4 = reinterpret_cast<uint32_t*>(dst);
      if (hi < 0 || hi >= H) {
        for (int i = 0; i < nw; ++i) dst4[i] = zx4;
      } else if (wi0 >= 0 && wi0 + S <= W) {
        const int8_t* src = x + (((int64_t)n * H + hi) * W + wi0) * C;
        const uint32_t sh = (uint32_t)(reinterpret_cast<uintptr_t>(src) & 3u) * 8u;
        const uint32_t* a4 = reinterpret_cast<const uint32_t*>(reinterpret_cast<uintptr_t>(src) & ~(uintptr_t)3);
        uint32_t prev = *a4;
        for (int i = 0; i < nw; ++i) {
          const uint32_t* nxt = a4 + i + 1;
          // an aligned word that starts inside the tensor is readable to its end (the base is 16-byte aligned)
          const uint32_t next = (reinterpret_cast<const int8_t*>(nxt) < x_end) ? *nxt : 0u;
          dst4[i] = __funnelshift_r(prev, next, sh);
          prev = next;
        }
      } else {
        const int8_t* src = x + (((int64_t)n * H + hi) * W + wi0) * C;
        for (int q = 0; q < S; ++q) {
          const bool in = (wi0 + q >= 0) && (wi0 + q < W);
          for (int c = 0; c < C; ++c) dst[q * C + c] = in ? src[q * C + c] : (int8_t)zx;
        }
        for (int b = sc; b < RP; ++b) dst[b] = 0;
      }
    }
    __syncthreads();
    const int chunks = kPatchPixels * Kp / 16;
    for (int t = threadIdx.x; t < chunks; t += blockDim.x) {
      const int64_t byte = (int64_t)t * 16;
      if (m0 * Kp + byte < M * Kp) *reinterpret_cast<uint4*>(A + m0 * Kp + byte) = *reinterpret_cast<const uint4*>(rows_s + byte);
    }
    __syncthreads();
  }
}

// Second repacking for spatial filters over few channels (the RGB stem), cheaper than whole patch rows:
// X2[n][m][j][u*SB + b], b = s*C + c < S*C, holds for output column j the horizontal filter window of input row
// m*sh + u (sh = vertical stride; rows beyond the image and taps on horizontal padding hold the input zero point).
// Over X2 the layer is a stride-1 convolution with ceil-range(R/sh) vertical taps, one output column wide, with
// sh*SB "channels" -- a shape the tensor-core kernel stages by itself.  X2 is about the size of the layer's output.
// Thread = one SB-byte slot: the S*C input bytes are contiguous, moved with aligned word loads and a funnel shift.
// Slot indices fit 32 bits (checked by the launcher); kWords = SB / 4 is a compile-time constant so that the slot
// stays in registers.
template <int kWords>
__global__ void __launch_bounds__(256) row_window_kernel(const int8_t* __restrict__ x, int8_t* __restrict__ X2, const hq_range_state* xq, int N,
                                                         int H, int W, int C, int Hg, int Wo, int S, int sh, int stride_w, int pad_w) {
  constexpr int SB = 4 * kWords;
  const int zx = xq->zero_point;
  const uint32_t zx4 = ((uint32_t)zx & 0xffu) * 0x01010101u;
  const int sc = S * C;
  const int nload = (sc + 3) / 4 + 1;                       // aligned words that can hold window bytes
  const int64_t total_words = ((int64_t)N * H * W * C + 3) >> 2;   // aligned words that start inside the tensor
  const uint32_t per_row = (uint32_t)Wo * sh;             // slots of one (image, row group)
  const int sh_log2 = 31 - __clz(sh);                     // sh is a power of two (checked when the layer is prepared)
  // block = one (image, row group) at a time; thread = slot (output column j, sub-row u)
  for (uint32_t rowi = blockIdx.x, rem = threadIdx.x; rowi < (uint32_t)N * Hg;) {
    if (rem >= per_row) {   // next row group of this block
      rowi += gridDim.x;
      rem = threadIdx.x;
      continue;
    }
    const uint32_t idx = rowi * per_row + rem;
    const int j = (int)(rem >> sh_log2);
    const int u = (int)(rem & (uint32_t)(sh - 1));
    const int n = (int)(rowi / (uint32_t)Hg);
    const int m = (int)(rowi - (uint32_t)n * Hg);
    rem += blockDim.x;
    const int hi = m * sh + u;
    const int wi0 = j * stride_w - pad_w;
    uint32_t w[kWords];
    if (hi >= H) {
#pragma unroll
      for (int i = 0; i < kWords; ++i) w[i] = zx4;
    } else {
      // byte offset of the window's first tap from the tensor base (negative for windows that start on left padding of
      // the first row), split into an aligned word index and a shift
      const int64_t off = (((int64_t)n * H + hi) * W + wi0) * C;
      const int64_t woff = off >> 2;                          // floor
      const uint32_t shb = (uint32_t)(off & 3) * 8u;
      const uint32_t* a4 = reinterpret_cast<const uint32_t*>(x) + woff;
      // words [first, last) of this run exist in the tensor (an aligned word that starts inside it is readable)
      const int first = woff < 0 ? (int)-woff : 0;
      const int64_t left = total_words - woff;
      const int last = left < (int64_t)nload ? (int)left : nload;
      uint32_t ld[kWords + 1];
#pragma unroll
      for (int i = 0; i <= kWords; ++i) ld[i] = (i >= first && i < last) ? __ldg(a4 + i) : 0u;
#pragma unroll
      for (int i = 0; i < kWords; ++i) w[i] = __funnelshift_r(ld[i], ld[i + 1], shb);
      // taps on horizontal padding: bytes outside [lo_b, hi_b) of the slot hold the zero point
      const int lo_b = (wi0 < 0 ? -wi0 : 0) * C;
      const int hi_b = (wi0 + S > W ? W - wi0 : S) * C;
      if (lo_b > 0 || hi_b < sc) {
#pragma unroll
        for (int i = 0; i < kWords; ++i) {
          const int klo = min(max(lo_b - 4 * i, 0), 4), khi = min(max(hi_b - 4 * i, 0), 4);   // valid bytes: [klo, khi)
          const uint32_t below_hi = khi >= 4 ? 0xffffffffu : ((1u << (8 * khi)) - 1u);
          const uint32_t below_lo = klo >= 4 ? 0xffffffffu : ((1u << (8 * klo)) - 1u);
          const uint32_t keep = below_hi & ~below_lo;
          w[i] = (w[i] & keep) | (zx4 & ~keep);
        }
      }
    }
    uint4* dst = reinterpret_cast<uint4*>(X2 + (size_t)idx * SB);
#pragma unroll
    for (int i = 0; i < kWords / 4; ++i) dst[i] = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
  }
}

// weight matrix over the window tensor: Wmat[k][t][u*SB + b] = W[k][r][b] with r = (dh_min + t)*sh + u + pad_h, zero
// where r is outside the filter or b >= S*C
__global__ void prep_window_weights_kernel(const int8_t* __restrict__ W, int8_t* __restrict__ Wmat, int K, int R, int SC, int sh, int SB, int ntaps,
                                           int dh_min, int pad_h) {
  const int Cg = sh * SB, ld = ntaps * Cg;
  const int64_t total = (int64_t)K * ld;
  for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
    const int col = (int)(idx % ld);
    const int k = (int)(idx / ld);
    const int t = col / Cg, within = col - t * Cg;
    const int u = within / SB, b = within - u * SB;
    const int r = (dh_min + t) * sh + u + pad_h;
    Wmat[idx] = (r >= 0 && r < R && b < SC) ? W[((int64_t)k * R + r) * SC + b] : (int8_t)0;
  }
}

// weight matrix for the patch layout: Wmat[k][r*RP + j] = W[k][r][j], zero elsewhere (row pitch `ld` bytes)
__global__ void prep_patch_weights_kernel(const int8_t* __restrict__ W, int8_t* __restrict__ Wmat, int K, int R, int SC, int RP, int ld) {
  const int64_t total = (int64_t)K * ld;
  for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
    const int j = (int)(idx % ld);
    const int k = (int)(idx / ld);
    const int r = j / RP, b = j - r * RP;
    Wmat[idx] = (r < R && b < SC) ? W[((int64_t)k * R + r) * SC + b] : (int8_t)0;
  }
}

__global__ void pad_rows_kernel(const int8_t* __restrict__ src, int8_t* __restrict__ dst, int rows, int K, int Kp) {
  const int64_t total = (int64_t)rows * Kp;
  for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
    const int j = (int)(idx % Kp);
    const int64_t r = idx / Kp;
    dst[idx] = j < K ? src[r * K + j] : (int8_t)0;
  }
}

// ---- weight gradient of a linear layer: operand transposition and the final correction ---------------------------
// out[c][r] = in[r][c] for r < R, c < C; every output row is Rp long (zeros from R on).  With `ones_row`, output row C
// holds 1 for r < R and rows C+1 .. C+15 hold zeros (not used at present).
__global__ void __launch_bounds__(256) transpose_rows_kernel(const int8_t* __restrict__ in, int8_t* __restrict__ out, int R, int C, int Rp,
                                                              int ones_row) {
  __shared__ int8_t tile[32][33];
  const int r0 = blockIdx.x * 32, c0 = blockIdx.y * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;   // 32 x 8 threads
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int r = r0 + ty + 8 * j, c = c0 + tx;
    int8_t v = 0;
    if (r < R) {
      if (c < C) v = in[(int64_t)r * C + c];
      else if (ones_row && c == C) v = 1;
    }
    tile[ty + 8 * j][tx] = v;
  }
  __syncthreads();
  const int Ctot = C + (ones_row ? 16 : 0);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int c = c0 + ty + 8 * j, r = r0 + tx;
    if (c < Ctot && r < Rp) out[(int64_t)c * Rp + r] = tile[tx][ty + 8 * j];
  }
}
// Weight gradient of a convolution: the second GEMM operand, transposed.  Bt[(r*S + s)*C + c][m] = x(n, hi, wi, c) for
// output pixel m = (n, ho, wo) and hi = ho*stride_h - pad_h + r (wi alike); the input zero point where (hi, wi) lies
// outside the image (real zero, which the zero-point correction then turns into no contribution); 0 for m >= M.
// One block: 128 output pixels x 32 channels of one filter tap, transposed through shared memory (reads of four
// channels per thread, writes of whole 128-byte runs); it also adds its part of the row sums of Bt (colsum, zeroed by
// the caller), which the zero point of dY needs.
__global__ void __launch_bounds__(256) im2col_t_kernel(const int8_t* __restrict__ X, int8_t* __restrict__ Bt, const hq_range_state* __restrict__ xq,
                                                        hq_conv_desc d, int Ho, int Wo, int M, int Mp, int tiles_per_block,
                                                        FastDiv fd_wo, FastDiv fd_ho, int32_t* __restrict__ colsum) {
  // [round parity][channel][4-pixel word]; 33: both phases hit 32 different banks.  Two tiles: a round writes the one the
  // round before last read, which every thread has left once it reaches this round's barrier -- one barrier per round.
  __shared__ __align__(16) uint32_t tiles[2][32][33];
  const int c0 = blockIdx.y * 32;
  int acc[4] = {0, 0, 0, 0};   // this lane's part of the row sums of its warp's four channel rows
  const int tap = blockIdx.z, r = tap / d.S, s = tap - r * d.S;
  const uint32_t zx = (uint32_t)(uint8_t)(int8_t)xq->zero_point;
  const bool vec = (d.C & 3) == 0;   // four channels of a pixel are one aligned word
  const int cg = threadIdx.x & 7, pg = threadIdx.x >> 3;   // channel group (4 channels) and pixel group (4 pixels)
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int c = c0 + cg * 4;
  for (int mt = 0; mt < tiles_per_block; ++mt) {
    const int m0 = (blockIdx.x * tiles_per_block + mt) * 128;
    if (m0 >= Mp) break;   // the same for every thread of the block
    uint32_t (*tile)[33] = tiles[mt & 1];
    // read: four consecutive output pixels x four channels, one word per pixel
    uint32_t w[4];
    // output pixel of the first of the four, then stepped (divisions by multiplication: the divisors are launch constants)
    int wo, ho, n;
    {
      const int m = m0 + pg * 4;
      const int t = fdiv(m, fd_wo);
      wo = m - t * Wo;
      n = fdiv(t, fd_ho);
      ho = t - n * Ho;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int m = m0 + pg * 4 + j;
      uint32_t v = 0;
      if (m < M && c < d.C) {
        const int hi = ho * d.stride_h - d.pad_h + r, wi = wo * d.stride_w - d.pad_w + s;
        const bool inside = hi >= 0 && hi < d.H && wi >= 0 && wi < d.W;
        if (inside) {
          const int8_t* src = X + (((int64_t)n * d.H + hi) * d.W + wi) * d.C + c;
          if (vec) {
            v = *reinterpret_cast<const uint32_t*>(src);
          } else {
#pragma unroll
            for (int k = 0; k < 4; ++k)
              if (c + k < d.C) v |= (uint32_t)(uint8_t)src[k] << (8 * k);
          }
        } else {
#pragma unroll
          for (int k = 0; k < 4; ++k)
            if (c + k < d.C) v |= zx << (8 * k);
        }
      }
      w[j] = v;
      if (++wo == Wo) {
        wo = 0;
        if (++ho == Ho) {
          ho = 0;
          ++n;
        }
      }
    }
    // 4x4 byte transposition in registers: t[k] = channel k of pixels 0..3
    const uint32_t a0 = __byte_perm(w[0], w[1], 0x5140), a1 = __byte_perm(w[0], w[1], 0x7362);   // ch0|ch1 and ch2|ch3 of pixels 0,1
    const uint32_t b0 = __byte_perm(w[2], w[3], 0x5140), b1 = __byte_perm(w[2], w[3], 0x7362);   // the same of pixels 2,3
    tile[cg * 4 + 0][pg] = __byte_perm(a0, b0, 0x5410);
    tile[cg * 4 + 1][pg] = __byte_perm(a0, b0, 0x7632);
    tile[cg * 4 + 2][pg] = __byte_perm(a1, b1, 0x5410);
    tile[cg * 4 + 3][pg] = __byte_perm(a1, b1, 0x7632);
    __syncthreads();
#pragma unroll
    for (int pass = 0; pass < 4; ++pass) {
      const int cl = pass * 8 + warp;   // channel row of the tile
      const uint32_t v = tile[cl][lane];
      acc[pass] = __dp4a((int)v, 0x01010101, acc[pass]);
      const int m = m0 + lane * 4;
      if (c0 + cl < d.C && m < Mp) *reinterpret_cast<uint32_t*>(Bt + ((int64_t)tap * d.C + c0 + cl) * Mp + m) = v;   // Mp is a multiple of 128
    }
  }
#pragma unroll
  for (int pass = 0; pass < 4; ++pass) {
    const int cc = c0 + pass * 8 + warp;
    const int part = __reduce_add_sync(0xffffffffu, acc[pass]);
    if (lane == 0 && cc < d.C) atomicAdd(&colsum[tap * d.C + cc], part);
  }
}
// The reduction was cut into slices that accumulated into slabs of their own: sum them (modulo 2^32, like everything
// before), take out both zero points -- sum (a - za)(b - zb) = sum a b - za * sum b - zb * (sum a - za * M), with sum b
// the row sums of the second operand (colsum) and sum a those of the first (rowsum) -- and convert:
// G = fl(float(g) * fl(s_dy * s_x)).
__global__ void wgrad_reduce_kernel(const int32_t* __restrict__ slabs, int nslabs, int rows, int cols, const int32_t* __restrict__ colsum,
                                    const int32_t* __restrict__ rowsum, int M, const hq_range_state* __restrict__ dyq,
                                    const hq_range_state* __restrict__ xq, float* __restrict__ G) {
  const float sc = __fmul_rn(dyq->scale, xq->scale);
  const int zdy = dyq->zero_point, zx = xq->zero_point;
  const int64_t total = (int64_t)rows * cols;
  for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
    const int row = (int)(idx / cols), col = (int)(idx - (int64_t)row * cols);
    uint32_t g = 0;
    for (int sl = 0; sl < nslabs; ++sl) g += (uint32_t)slabs[(int64_t)sl * total + idx];
    g -= (uint32_t)zdy * (uint32_t)colsum[col];
    g -= (uint32_t)zx * ((uint32_t)rowsum[row] - (uint32_t)zdy * (uint32_t)M);
    G[idx] = __fmul_rn(__int2float_rn((int)g), sc);
  }
}

// The same for the stride-1 form, where image padding is left out of the sums instead of being filled with the zero
// point: per filter tap t = (r, s), with sums over the output pixels whose tap lies inside the image,
//   sum (dy - z_dy)(x - z_x) = sum dy x - z_dy * colsum[t][c] - z_x * (rowsum[t][k] - z_dy * count[t]).
// Slabs have slab_rows rows of which the first `rows` are output channels.
__global__ void __launch_bounds__(256) wgrad_reduce_taps_kernel(const int32_t* __restrict__ slabs, int nslabs, int rows, int slab_rows, int cols,
                                                                 int C, const int32_t* __restrict__ colsum, const int32_t* __restrict__ rowsum,
                                                                 TapCounts mvalid, const hq_range_state* __restrict__ dyq,
                                                                 const hq_range_state* __restrict__ xq, float* __restrict__ G) {
  // a block: 32 consecutive outputs (lanes) x 8 groups of slabs (warps), joined through shared memory
  __shared__ uint32_t part_s[8][32];
  const float sc = __fmul_rn(dyq->scale, xq->scale);
  const int zdy = dyq->zero_point, zx = xq->zero_point;
  const int64_t total = (int64_t)rows * cols, slab = (int64_t)slab_rows * cols;
  const int lane = threadIdx.x & 31, grp = threadIdx.x >> 5;
  for (int64_t base = (int64_t)blockIdx.x * 32; base < total; base += (int64_t)gridDim.x * 32) {
    const int64_t idx = base + lane;
    uint32_t g = 0;
    if (idx < total)
      for (int sl = grp; sl < nslabs; sl += 8) g += (uint32_t)slabs[(int64_t)sl * slab + idx];
    part_s[grp][lane] = g;
    __syncthreads();
    if (grp == 0 && idx < total) {
#pragma unroll
      for (int k = 1; k < 8; ++k) g += part_s[k][lane];
      const int row = (int)(idx / cols), col = (int)(idx - (int64_t)row * cols);
      const int tap = col / C;
      g -= (uint32_t)zdy * (uint32_t)colsum[col];
      g -= (uint32_t)zx * ((uint32_t)rowsum[tap * rows + row] - (uint32_t)zdy * (uint32_t)mvalid.v[tap]);
      G[idx] = __fmul_rn(__int2float_rn((int)g), sc);
    }
    __syncthreads();
  }
}

// Packs one NHWC tensor for the stride-1 weight-gradient GEMM (reduction over pixels): dst[copy][c][m] with
// m = (n * Hp + row_off + h) * P + w holds src(n, h, w + shift, c), 0 where that column lies outside the source row, in
// the rows of the padded index space that no source row maps to, and for w >= the source width.  In this index space a
// vertical filter offset is a shift by a multiple of P (16-byte aligned, which a TMA coordinate needs), the horizontal
// offsets are the copies, and image padding is real zeros.
// The kernel forms `ns` shifted views of every source row, shift_j = sign * (j - pad): the input (sign +1) writes all of
// them (copy j); the output gradient (sign -1) writes only the unshifted one (as copy 0).  The sum of view j over its
// first `limit` columns is the sum of the source row over the columns that filter column j pairs with a pixel inside
// the other tensor's row; it is added to sums[(r * ns + j) * Cs + c] (zeroed by the caller) for every filter row r whose
// row range rg.row_* contains the source row.
// One block: 32 channels of kPackRows padded rows of one image, all rows at once: the source rows go to shared memory
// transposed (4x4 byte blocks turned in registers; channel-major words behind 16 zero bytes, zeros after), each view is
// read from there as aligned words and funnel-shifted, written in 16-byte pieces and summed with dp4a.
constexpr int kPackRows = 8;   // x 32 channels = the 256 threads of a block
constexpr int kPackMaxP = 256;
// words per channel row of the tile: 16 zero bytes, the row, room for the shifted reads past its end; odd, so that the
// transposing stores spread over the banks
static int pack_tile_pitch(int P, int Ws, int limit) { return ((std::max(std::max(P, limit), Ws) + 64) / 4) | 1; }
__global__ void __launch_bounds__(256) wgrad_pack_kernel(const int8_t* __restrict__ src, int8_t* __restrict__ dst, int Hs, int Ws, int Cs, int Hp,
                                                          int P, int row_off, int sign, int pad, int limit, int64_t pitch, PackRanges rg,
                                                          int32_t* __restrict__ sums, int tp) {
  extern __shared__ uint32_t pack_tile[];   // [kPackRows][32][tp]
  auto tile = [&](int rl, int c) { return pack_tile + (rl * 32 + c) * tp; };
  __shared__ int acc_s[64][32];    // [filter row * ns + view][channel of the block]
  const int n = blockIdx.z, c0 = blockIdx.y * 32, pr0 = blockIdx.x * kPackRows;
  const int tid = threadIdx.x;
  for (int i = tid; i < rg.nr * rg.ns * 32; i += 256) acc_s[i >> 5][i & 31] = 0;
  for (int i = tid; i < kPackRows * 32 * tp; i += 256) pack_tile[i] = 0u;   // margins and missing rows stay zero
  const int wgroups = (Ws + 3) / 4;                // groups of 4 source pixels
  __syncthreads();
  for (int i = tid; i < kPackRows * wgroups * 8; i += 256) {   // (row of the block, pixel group, channel word)
    const int cg = i & 7, wg = (i >> 3) % wgroups, rl = (i >> 3) / wgroups;
    const int h = pr0 + rl - row_off;
    if (pr0 + rl >= Hp || h < 0 || h >= Hs || c0 + cg * 4 >= Cs) continue;   // Cs is a multiple of 4
    const int8_t* row = src + (((int64_t)n * Hs + h) * Ws) * Cs + c0;
    uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
    for (int j = 0; j < 4; ++j)
      if (wg * 4 + j < Ws) w[j] = *reinterpret_cast<const uint32_t*>(row + (int64_t)(wg * 4 + j) * Cs + cg * 4);
    const uint32_t a0 = __byte_perm(w[0], w[1], 0x5140), a1 = __byte_perm(w[0], w[1], 0x7362);
    const uint32_t b0 = __byte_perm(w[2], w[3], 0x5140), b1 = __byte_perm(w[2], w[3], 0x7362);
    tile(rl, cg * 4 + 0)[4 + wg] = __byte_perm(a0, b0, 0x5410);
    tile(rl, cg * 4 + 1)[4 + wg] = __byte_perm(a0, b0, 0x7632);
    tile(rl, cg * 4 + 2)[4 + wg] = __byte_perm(a1, b1, 0x5410);
    tile(rl, cg * 4 + 3)[4 + wg] = __byte_perm(a1, b1, 0x7632);
  }
  __syncthreads();
  // One thread = one (row of the block, channel): the lanes of a warp are 32 channels (conflict-free shared-memory reads).
  // It sums the row once, then for every view takes out the few bytes the view's window leaves, and, for a stored view,
  // walks along the row in 16-byte pieces, two pieces per store where rows allow 32 bytes.
  const bool wide = (P & 31) == 0 && (pitch & 31) == 0 && (reinterpret_cast<uintptr_t>(dst) & 31u) == 0;
  {
    const int rl = tid >> 5, c = tid & 31;   // kPackRows * 32 == 256 threads
    const int pr = pr0 + rl, h = pr - row_off;
    if (pr < Hp && c0 + c < Cs) {
      const uint32_t* trow = tile(rl, c);
      const bool has = h >= 0 && h < Hs;
      int total = 0;
      if (has)
        for (int g = 0; g < wgroups; ++g) total = __dp4a((int)trow[4 + g], 0x01010101, total);
      const int8_t* bytes = reinterpret_cast<const int8_t*>(trow) + 16;
      for (int j = 0; j < rg.ns; ++j) {
        const int shift = sign * (j - pad);
        if (has) {   // sum of the view's first `limit` columns = row total minus what the window [shift, shift + limit) leaves out
          int part = total;
          for (int i = 0; i < min(shift, Ws); ++i) part -= bytes[i];
          for (int i = max(0, shift + limit); i < Ws; ++i) part -= bytes[i];
          if (part != 0)
            for (int r = 0; r < rg.nr; ++r)
              if (h >= rg.row_lo[r] && h < rg.row_hi[r]) atomicAdd(&acc_s[r * rg.ns + j][c], part);
        }
        if (!(sign > 0 || shift == 0)) continue;   // this view is only summed
        const int b0 = 16 + shift;                 // first byte of the view in the tile row (>= 0)
        const uint32_t* wp = trow + (b0 >> 2);
        const uint32_t sh = (uint32_t)(b0 & 3) * 8u;
        int8_t* out = dst + ((int64_t)(sign > 0 ? j : 0) * Cs + c0 + c) * pitch + ((int64_t)n * Hp + pr) * P;
        uint32_t lo = wp[0];
        uint32_t prev[4];
        for (int q = 0; q * 16 < P; ++q) {
          uint32_t w4[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const uint32_t hi = wp[q * 4 + e + 1];
            w4[e] = __funnelshift_r(lo, hi, sh);
            lo = hi;
          }
          if (wide) {
            if (q & 1) {
              const uint32_t w8[8] = {prev[0], prev[1], prev[2], prev[3], w4[0], w4[1], w4[2], w4[3]};
              st_global_v8(reinterpret_cast<uint32_t*>(out + (q - 1) * 16), w8);
            } else {
#pragma unroll
              for (int e = 0; e < 4; ++e) prev[e] = w4[e];
            }
          } else {
            *reinterpret_cast<uint4*>(out + q * 16) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
          }
        }
      }
    }
  }
  __syncthreads();
  for (int i = tid; i < rg.nr * rg.ns * 32; i += 256) {
    const int c = i & 31, t = i >> 5;
    if (c0 + c < Cs && acc_s[t][c] != 0) atomicAdd(&sums[t * Cs + c0 + c], acc_s[t][c]);
  }
}
__global__ void zero_tail_kernel(int8_t* base, int rows, int64_t pitch, int64_t from) {   // bytes [from, pitch) of every row; both multiples of 16
  const int64_t per_row = (pitch - from) / 16;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < per_row * rows; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = i / per_row, q = i - r * per_row;
    *reinterpret_cast<uint4*>(base + r * pitch + from + q * 16) = make_uint4(0u, 0u, 0u, 0u);
  }
}

// sum_m (dy - z_dy)(x - z_x) = sum_m (dy - z_dy) x  -  z_x * sum_m (dy - z_dy): the second term, one number per output
// row n, which the layer kernel's epilogue subtracts from every accumulator of that row.
// Reads the transposed copy dY^T [N][Mp] (rows zero-filled beyond M): one warp per row, 16 bytes per lane and step.
__global__ void __launch_bounds__(256) wgrad_row_terms_kernel(const int8_t* __restrict__ dYt, int M, int Mp, int N,
                                                               const hq_range_state* __restrict__ dyq, const hq_range_state* __restrict__ xq,
                                                               int32_t* __restrict__ terms) {
  const int n = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (n >= N) return;
  const uint4* row = reinterpret_cast<const uint4*>(dYt + (int64_t)n * Mp);   // Mp is a multiple of 16
  int sum = 0;
  for (int i = lane; i < Mp / 16; i += 32) {
    const uint4 v = row[i];
    sum = __dp4a((int)v.x, 0x01010101, sum);
    sum = __dp4a((int)v.y, 0x01010101, sum);
    sum = __dp4a((int)v.z, 0x01010101, sum);
    sum = __dp4a((int)v.w, 0x01010101, sum);
  }
  sum = __reduce_add_sync(0xffffffffu, sum);
  if (lane == 0) terms[n] = xq->zero_point * (sum - dyq->zero_point * M);
}

// ---- weight gradient of a depthwise layer (CUDA cores) -----------------------------------------------------------
// g[c][r][s] = sum over output pixels of (dy(.., c) - z_dy) * (x(hi, wi, c) - z_x), padded taps skipped.  A thread owns
// four channels (one word) and every `lanes`-th output pixel of its block's range; its RS*RS*4 sums stay in registers,
// are gathered per block in shared memory and leave as integer atomics on acc[c][tap] (zeroed by the caller).
template <int RS>
__global__ void __launch_bounds__(256) dw_wgrad_kernel(const int8_t* __restrict__ dY, const int8_t* __restrict__ X, const hq_range_state* __restrict__ dyq,
                                                        const hq_range_state* __restrict__ xq, hq_conv_desc d, int Ho, int Wo, int M,
                                                        int pixels_per_block, FastDiv fd_wo, FastDiv fd_ho, int32_t* __restrict__ acc_out) {
  extern __shared__ int32_t sacc[];   // [C][RS*RS]
  constexpr int T = RS * RS;
  const int CW = d.C / 4;
  for (int i = threadIdx.x; i < d.C * T; i += blockDim.x) sacc[i] = 0;
  __syncthreads();
  const int lanes = (int)blockDim.x / CW;   // C <= 1024
  const int cw = (int)threadIdx.x % CW, pl = (int)threadIdx.x / CW;
  const int zdy = dyq->zero_point, zx = xq->zero_point;
  if (pl < lanes) {
    int acc[T][4];
#pragma unroll
    for (int t = 0; t < T; ++t)
#pragma unroll
      for (int k = 0; k < 4; ++k) acc[t][k] = 0;
    const int m_begin = blockIdx.x * pixels_per_block;
    const int m_end = min(M, m_begin + pixels_per_block);
    for (int m = m_begin + pl; m < m_end; m += lanes) {
      const int t0 = fdiv(m, fd_wo);
      const int wo = m - t0 * Wo;
      const int n = fdiv(t0, fd_ho);
      const int ho = t0 - n * Ho;
      const uint32_t gw = *reinterpret_cast<const uint32_t*>(dY + (int64_t)m * d.C + cw * 4);
      int g[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) g[k] = (int)(int8_t)((gw >> (8 * k)) & 0xffu) - zdy;
#pragma unroll
      for (int r = 0; r < RS; ++r) {
        const int hi = ho * d.stride_h - d.pad_h + r;
        if (hi < 0 || hi >= d.H) continue;
#pragma unroll
        for (int s = 0; s < RS; ++s) {
          const int wi = wo * d.stride_w - d.pad_w + s;
          if (wi < 0 || wi >= d.W) continue;
          const uint32_t xw = *reinterpret_cast<const uint32_t*>(X + (((int64_t)n * d.H + hi) * d.W + wi) * d.C + cw * 4);
#pragma unroll
          for (int k = 0; k < 4; ++k) acc[r * RS + s][k] += g[k] * ((int)(int8_t)((xw >> (8 * k)) & 0xffu) - zx);
        }
      }
    }
#pragma unroll
    for (int t = 0; t < T; ++t)
#pragma unroll
      for (int k = 0; k < 4; ++k) atomicAdd(&sacc[(cw * 4 + k) * T + t], acc[t][k]);
  }
  __syncthreads();
  for (int i = threadIdx.x; i < d.C * T; i += blockDim.x) {
    const int v = sacc[i];
    if (v != 0) atomicAdd(&acc_out[i], v);
  }
}
__global__ void scale_to_real_kernel(const int32_t* __restrict__ acc, int count, const hq_range_state* __restrict__ dyq,
                                     const hq_range_state* __restrict__ xq, float* __restrict__ G) {
  const float sc = __fmul_rn(dyq->scale, xq->scale);
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < count; i += gridDim.x * blockDim.x) G[i] = __fmul_rn(__int2float_rn(acc[i]), sc);
}

// ---- depthwise convolution on CUDA cores --------------------------------------------------------
// One thread: one output pixel x 16 consecutive channels.  Same epilogue as the tensor-core kernel.
__device__ __forceinline__ int sx8(uint32_t w, int k) { return (int)(int8_t)((w >> (8 * k)) & 0xffu); }

template <int kOut>
__global__ void __launch_bounds__(256) depthwise_kernel(const DwParams p) {
  __shared__ int red_min[8], red_max[8];
  grid_dependency_wait();   // launched ahead of its predecessor's end: see launch_overlapped
  QParams q;
  q.s_acc = __fmul_rn(p.xq->scale, *p.w_scale);
  q.zx = p.xq->zero_point;
  q.inv_scale = (kOut == kOutInt8) ? p.yq->inv_scale : 1.0f;
  q.zp = (kOut == kOutInt8) ? p.yq->zero_point : 0;
  qparams_finish(q);
  if (kOut == kOutInt8) qparams_output_mode(q, p.yq->rounding, p.yq->seed, p.yq->step);
  int sat_below = 0, sat_above = 0;
  const float s_acc = q.s_acc;
  const int zx = q.zx;
  if (blockIdx.x == 0 && threadIdx.x == 0) p.yq->acc_scale = s_acc;
  const int cgs = p.C / 16;
  const int64_t total = (int64_t)p.N * p.Ho * p.Wo * cgs;
  int mn = INT32_MAX, mx = INT32_MIN;
  for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
    const int cg = (int)(idx % cgs);
    int64_t t = idx / cgs;
    const int wo = (int)(t % p.Wo);
    t /= p.Wo;
    const int ho = (int)(t % p.Ho);
    const int n = (int)(t / p.Ho);
    int acc[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) acc[e] = 0;
    for (int r = 0; r < p.R; ++r) {
      const int hi = ho * p.stride_h - p.pad_h + r;
      if (hi < 0 || hi >= p.H) continue;
      for (int s = 0; s < p.S; ++s) {
        const int wi = wo * p.stride_w - p.pad_w + s;
        if (wi < 0 || wi >= p.W) continue;
        const uint4 xv = *reinterpret_cast<const uint4*>(p.x + (((int64_t)n * p.H + hi) * p.W + wi) * p.C + cg * 16);
        const uint4 wv = *reinterpret_cast<const uint4*>(p.w + (int64_t)(r * p.S + s) * p.C + cg * 16);
        const uint32_t xa[4] = {xv.x, xv.y, xv.z, xv.w};
        const uint32_t wa[4] = {wv.x, wv.y, wv.z, wv.w};
        if (p.w_zp != 0) {   // asymmetric weights: both zero points taken out term by term (padded taps were skipped above)
#pragma unroll
          for (int e = 0; e < 16; ++e) acc[e] += (sx8(xa[e >> 2], e & 3) - zx) * (sx8(wa[e >> 2], e & 3) - p.w_zp);
        } else {
#pragma unroll
          for (int e = 0; e < 16; ++e) acc[e] += sx8(xa[e >> 2], e & 3) * sx8(wa[e >> 2], e & 3);
        }
      }
    }
    if (zx != 0 && p.w_zp == 0) {
      const int cls = p.rowcls[ho] * p.ncolcls + p.colcls[wo];
      const int32_t* cr = p.corr + (int64_t)cls * p.C + cg * 16;
#pragma unroll
      for (int e = 0; e < 16; ++e) acc[e] -= zx * cr[e];
    }
#pragma unroll
    for (int e = 0; e < 16; ++e) {
      mn = min(mn, acc[e]);
      mx = max(mx, acc[e]);
    }
    const int64_t o = (((int64_t)n * p.Ho + ho) * p.Wo + wo) * p.C + cg * 16;
    if constexpr (kOut == kOutInt8) {
      uint32_t w[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) w[e] = quant4_acc(acc[4 * e], acc[4 * e + 1], acc[4 * e + 2], acc[4 * e + 3], o + 4 * e, q, sat_below, sat_above);
      *reinterpret_cast<uint4*>(reinterpret_cast<int8_t*>(p.out) + o) = make_uint4(w[0], w[1], w[2], w[3]);
    } else {
      uint32_t* dst = reinterpret_cast<uint32_t*>(p.out) + o;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        uint32_t w[4];
#pragma unroll
        for (int k = 0; k < 4; ++k)
          w[k] = (kOut == kOutF32) ? __float_as_uint(__fmul_rn(__int2float_rn(acc[4 * e + k]), s_acc)) : (uint32_t)acc[4 * e + k];
        *reinterpret_cast<uint4*>(dst + 4 * e) = make_uint4(w[0], w[1], w[2], w[3]);
      }
    }
  }
  grid_launch_dependents();   // the successor may take the SMs that free up from here on
  if (q.count_sat) {   // clipped outputs: one atomic pair per warp that saw any
    sat_below = __reduce_add_sync(0xffffffffu, sat_below);
    sat_above = __reduce_add_sync(0xffffffffu, sat_above);
    if ((threadIdx.x & 31) == 0) {
      if (sat_below) atomicAdd(&p.yq->sat_below, (uint32_t)sat_below);
      if (sat_above) atomicAdd(&p.yq->sat_above, (uint32_t)sat_above);
    }
  }
  mn = __reduce_min_sync(0xffffffffu, mn);
  mx = __reduce_max_sync(0xffffffffu, mx);
  const int warp = threadIdx.x >> 5;
  if ((threadIdx.x & 31) == 0) {
    red_min[warp] = mn;
    red_max[warp] = mx;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int e = 1; e < (int)(blockDim.x >> 5); ++e) {
      mn = min(mn, red_min[e]);
      mx = max(mx, red_max[e]);
    }
    if (mn <= mx) {
      atomicMin(&p.yq->acc_min, mn);
      atomicMax(&p.yq->acc_max, mx);
    }
  }
}


// Backward data of a depthwise layer, any stride (Sec. 3.1, backward pass), by the definition:
//   dx(n,hi,wi,c) = sum over (r,s) with ho = (hi + pad_h - r) / stride_h, wo = (wi + pad_w - s) / stride_w integral and
//   inside the output image of (dy(n,ho,wo,c) - z_dy) * (w(c,r,s) - z_w).
// One thread: one input pixel x 16 channels; p describes the FORWARD layer (H x W input, Ho x Wo output), p.x is dY,
// p.w the weights tap-major [R*S][C] (not turned).  Same epilogue as every other kernel.
template <int kOut>
__global__ void __launch_bounds__(256) depthwise_bwd_kernel(const DwParams p) {
  __shared__ int red_min[8], red_max[8];
  QParams q;
  q.s_acc = __fmul_rn(p.xq->scale, *p.w_scale);
  q.zx = p.xq->zero_point;
  q.inv_scale = (kOut == kOutInt8) ? p.yq->inv_scale : 1.0f;
  q.zp = (kOut == kOutInt8) ? p.yq->zero_point : 0;
  qparams_finish(q);
  if (kOut == kOutInt8) qparams_output_mode(q, p.yq->rounding, p.yq->seed, p.yq->step);
  int sat_below = 0, sat_above = 0;
  const int zdy = q.zx;
  if (blockIdx.x == 0 && threadIdx.x == 0) p.yq->acc_scale = q.s_acc;
  const int cgs = p.C / 16;
  const int64_t total = (int64_t)p.N * p.H * p.W * cgs;
  int mn = INT32_MAX, mx = INT32_MIN;
  for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
    const int cg = (int)(idx % cgs);
    int64_t t = idx / cgs;
    const int wi = (int)(t % p.W);
    t /= p.W;
    const int hi = (int)(t % p.H);
    const int n = (int)(t / p.H);
    int acc[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) acc[e] = 0;
    for (int r = 0; r < p.R; ++r) {
      const int th = hi + p.pad_h - r;
      if (th < 0 || th % p.stride_h != 0) continue;
      const int ho = th / p.stride_h;
      if (ho >= p.Ho) continue;
      for (int s = 0; s < p.S; ++s) {
        const int tw = wi + p.pad_w - s;
        if (tw < 0 || tw % p.stride_w != 0) continue;
        const int wo = tw / p.stride_w;
        if (wo >= p.Wo) continue;
        const uint4 gv = *reinterpret_cast<const uint4*>(p.x + (((int64_t)n * p.Ho + ho) * p.Wo + wo) * p.C + cg * 16);
        const uint4 wv = *reinterpret_cast<const uint4*>(p.w + (int64_t)(r * p.S + s) * p.C + cg * 16);
        const uint32_t ga[4] = {gv.x, gv.y, gv.z, gv.w};
        const uint32_t wa[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
        for (int e = 0; e < 16; ++e) acc[e] += (sx8(ga[e >> 2], e & 3) - zdy) * (sx8(wa[e >> 2], e & 3) - p.w_zp);
      }
    }
#pragma unroll
    for (int e = 0; e < 16; ++e) {
      mn = min(mn, acc[e]);
      mx = max(mx, acc[e]);
    }
    const int64_t o = (((int64_t)n * p.H + hi) * p.W + wi) * p.C + cg * 16;
    if constexpr (kOut == kOutInt8) {
      uint32_t w[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) w[e] = quant4_acc(acc[4 * e], acc[4 * e + 1], acc[4 * e + 2], acc[4 * e + 3], o + 4 * e, q, sat_below, sat_above);
      *reinterpret_cast<uint4*>(reinterpret_cast<int8_t*>(p.out) + o) = make_uint4(w[0], w[1], w[2], w[3]);
    } else {
      uint32_t* dst = reinterpret_cast<uint32_t*>(p.out) + o;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        uint32_t w[4];
#pragma unroll
        for (int k = 0; k < 4; ++k)
          w[k] = (kOut == kOutF32) ? __float_as_uint(__fmul_rn(__int2float_rn(acc[4 * e + k]), q.s_acc)) : (uint32_t)acc[4 * e + k];
        *reinterpret_cast<uint4*>(dst + 4 * e) = make_uint4(w[0], w[1], w[2], w[3]);
      }
    }
  }
  if (q.count_sat) {
    sat_below = __reduce_add_sync(0xffffffffu, sat_below);
    sat_above = __reduce_add_sync(0xffffffffu, sat_above);
    if ((threadIdx.x & 31) == 0) {
      if (sat_below) atomicAdd(&p.yq->sat_below, (uint32_t)sat_below);
      if (sat_above) atomicAdd(&p.yq->sat_above, (uint32_t)sat_above);
    }
  }
  mn = __reduce_min_sync(0xffffffffu, mn);
  mx = __reduce_max_sync(0xffffffffu, mx);
  const int warp = threadIdx.x >> 5;
  if ((threadIdx.x & 31) == 0) {
    red_min[warp] = mn;
    red_max[warp] = mx;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int e = 1; e < (int)(blockDim.x >> 5); ++e) {
      mn = min(mn, red_min[e]);
      mx = max(mx, red_max[e]);
    }
    if (mn <= mx) {
      atomicMin(&p.yq->acc_min, mn);
      atomicMax(&p.yq->acc_max, mx);
    }
  }
}

// Asymmetric weights (z_w != 0): sum (a - z_a)(w - z_w) = [sum (a - z_a) w] - z_w * sum (a - z_a), the sums over the taps
// inside the image and all channels.  The bracket is what the layer kernels form; this pre-pass writes the second term,
// one number per output pixel, which their epilogue subtracts.  bwd = 0: pixel (n,ho,wo) of the forward output, sum
// over its input window; bwd = 1: pixel (n,hi,wi) of the input gradient, sum over the output-gradient pixels that reach it.
__global__ void __launch_bounds__(256) rowsum_kernel(const int8_t* __restrict__ a, const hq_range_state* __restrict__ aq, hq_conv_desc d, int Ho, int Wo,
                                                     int bwd, int zw, int32_t* __restrict__ out, int64_t total) {
  const int za = aq->zero_point;
  const int Ca = bwd ? d.K : d.C;                 // channels of the operand that is summed
  const int Ha = bwd ? Ho : d.H, Wa = bwd ? Wo : d.W;
  const int PH = bwd ? d.H : Ho, PW = bwd ? d.W : Wo;   // image of the pixels the sums are for
  const bool vec = (Ca & 3) == 0;
  for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
    const int pw_ = (int)(idx % PW);
    const int ph_ = (int)((idx / PW) % PH);
    const int n = (int)(idx / ((int64_t)PW * PH));
    int sum = 0, cnt = 0;
    for (int r = 0; r < d.R; ++r) {
      int ah;
      if (bwd) {
        const int th = ph_ + d.pad_h - r;
        if (th < 0 || th % d.stride_h != 0) continue;
        ah = th / d.stride_h;
      } else {
        ah = ph_ * d.stride_h - d.pad_h + r;
      }
      if (ah < 0 || ah >= Ha) continue;
      for (int s = 0; s < d.S; ++s) {
        int aw;
        if (bwd) {
          const int tw = pw_ + d.pad_w - s;
          if (tw < 0 || tw % d.stride_w != 0) continue;
          aw = tw / d.stride_w;
        } else {
          aw = pw_ * d.stride_w - d.pad_w + s;
        }
        if (aw < 0 || aw >= Wa) continue;
        const int8_t* src = a + (((int64_t)n * Ha + ah) * Wa + aw) * Ca;
        if (vec) {
          for (int c = 0; c < Ca; c += 4) sum = __dp4a(*reinterpret_cast<const int*>(src + c), 0x01010101, sum);
        } else {
          for (int c = 0; c < Ca; ++c) sum += src[c];
        }
        ++cnt;
      }
    }
    out[idx] = zw * (sum - za * cnt * Ca);
  }
}

// 3x3, stride 1: thread = one 32-bit word of channels (4 channels) x 8 consecutive output pixels of a row.
// The 36 weights of its channels stay in registers, each already shifted into its byte lane so that one dp4a
// against the input word multiplies exactly one channel (the other three lanes meet zeros).  Input words are
// read once per row of the window and reused by the three taps and the neighbouring pixels; a warp's lanes hold
// consecutive channel words, so loads and stores are contiguous.  Out-of-image taps read as 0 and are settled by
// the same border-class correction as in the tensor-core kernel.
constexpr int kDwPix = 8;
template <int kOut>
__global__ void __launch_bounds__(256) depthwise3x3_kernel(const DwParams p, int slots, int groups_w) {
  __shared__ int red_min[8], red_max[8];
  grid_dependency_wait();   // launched ahead of its predecessor's end: see launch_overlapped
  QParams q;
  q.s_acc = __fmul_rn(p.xq->scale, *p.w_scale);
  q.zx = p.xq->zero_point;
  q.inv_scale = (kOut == kOutInt8) ? p.yq->inv_scale : 1.0f;
  q.zp = (kOut == kOutInt8) ? p.yq->zero_point : 0;
  qparams_finish(q);
  if (kOut == kOutInt8) qparams_output_mode(q, p.yq->rounding, p.yq->seed, p.yq->step);
  int sat_below = 0, sat_above = 0;
  if (blockIdx.x == 0 && threadIdx.x == 0) p.yq->acc_scale = q.s_acc;
  const int CW = p.C / 4;
  const int cw = threadIdx.x % CW, slot = threadIdx.x / CW;
  int mn = INT32_MAX, mx = INT32_MIN;
  if (slot < slots) {
    int wsel[9][4];   // weight of (tap, channel k) in byte lane k
#pragma unroll
    for (int t = 0; t < 9; ++t) {
      const uint32_t w4 = *reinterpret_cast<const uint32_t*>(p.w + (int64_t)t * p.C + cw * 4);
#pragma unroll
      for (int k = 0; k < 4; ++k) wsel[t][k] = (int)(w4 & (0xffu << (8 * k)));
    }
    const int64_t items = (int64_t)p.N * p.Ho * groups_w;
    const int cstride = p.C;
    for (int64_t item = (int64_t)blockIdx.x * slots + slot; item < items; item += (int64_t)gridDim.x * slots) {
      const int pg = (int)(item % groups_w);
      const int ho = (int)((item / groups_w) % p.Ho);
      const int n = (int)(item / ((int64_t)groups_w * p.Ho));
      const int wo0 = pg * kDwPix;
      int acc[kDwPix][4];
#pragma unroll
      for (int j = 0; j < kDwPix; ++j)
#pragma unroll
        for (int k = 0; k < 4; ++k) acc[j][k] = 0;
#pragma unroll
      for (int r = 0; r < 3; ++r) {
        const int hi = ho - p.pad_h + r;
        if (hi < 0 || hi >= p.H) continue;
        const int wi0 = wo0 - p.pad_w;
        const int8_t* pj = p.x + (((int64_t)n * p.H + hi) * p.W + wi0) * p.C + cw * 4;   // not dereferenced where masked
        int xw[kDwPix + 2];
        if (wi0 >= 0 && wi0 + kDwPix + 2 <= p.W) {   // whole window inside the row: no per-pixel tests
#pragma unroll
          for (int j = 0; j < kDwPix + 2; ++j) {
            xw[j] = *reinterpret_cast<const int*>(pj);
            pj += cstride;
          }
        } else {
#pragma unroll
          for (int j = 0; j < kDwPix + 2; ++j) {
            const int wi = wi0 + j;
            xw[j] = (wi >= 0 && wi < p.W) ? *reinterpret_cast<const int*>(pj) : 0;
            pj += cstride;
          }
        }
#pragma unroll
        for (int s = 0; s < 3; ++s)
#pragma unroll
          for (int j = 0; j < kDwPix; ++j)
#pragma unroll
            for (int k = 0; k < 4; ++k) acc[j][k] = __dp4a(xw[j + s], wsel[r * 3 + s][k], acc[j][k]);
      }
      const int rcls = q.zx != 0 ? p.rowcls[ho] * p.ncolcls : 0;
#pragma unroll
      for (int j = 0; j < kDwPix; ++j) {
        const int wo = wo0 + j;
        if (wo >= p.Wo) break;
        if (q.zx != 0) {
          const int4 cr = *reinterpret_cast<const int4*>(p.corr + (int64_t)(rcls + p.colcls[wo]) * p.C + cw * 4);
          acc[j][0] -= q.zx * cr.x;
          acc[j][1] -= q.zx * cr.y;
          acc[j][2] -= q.zx * cr.z;
          acc[j][3] -= q.zx * cr.w;
        }
        mn = min(__vimin3_s32(mn, acc[j][0], acc[j][1]), min(acc[j][2], acc[j][3]));
        mx = max(__vimax3_s32(mx, acc[j][0], acc[j][1]), max(acc[j][2], acc[j][3]));
        const int64_t o = (((int64_t)n * p.Ho + ho) * p.Wo + wo) * p.C + cw * 4;
        if constexpr (kOut == kOutInt8) {
          const uint32_t w = quant4_acc(acc[j][0], acc[j][1], acc[j][2], acc[j][3], o, q, sat_below, sat_above);
          *reinterpret_cast<uint32_t*>(reinterpret_cast<int8_t*>(p.out) + o) = w;
        } else {
          uint32_t w[4];
#pragma unroll
          for (int k = 0; k < 4; ++k)
            w[k] = (kOut == kOutF32) ? __float_as_uint(__fmul_rn(__int2float_rn(acc[j][k]), q.s_acc)) : (uint32_t)acc[j][k];
          *reinterpret_cast<uint4*>(reinterpret_cast<uint32_t*>(p.out) + o) = make_uint4(w[0], w[1], w[2], w[3]);
        }
      }
    }
  }
  grid_launch_dependents();   // the successor may take the SMs that free up from here on
  if (q.count_sat) {   // clipped outputs: one atomic pair per warp that saw any
    sat_below = __reduce_add_sync(0xffffffffu, sat_below);
    sat_above = __reduce_add_sync(0xffffffffu, sat_above);
    if ((threadIdx.x & 31) == 0) {
      if (sat_below) atomicAdd(&p.yq->sat_below, (uint32_t)sat_below);
      if (sat_above) atomicAdd(&p.yq->sat_above, (uint32_t)sat_above);
    }
  }
  mn = __reduce_min_sync(0xffffffffu, mn);
  mx = __reduce_max_sync(0xffffffffu, mx);
  const int warp = threadIdx.x >> 5;
  if ((threadIdx.x & 31) == 0) {
    red_min[warp] = mn;
    red_max[warp] = mx;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int e = 1; e < (int)((blockDim.x + 31) >> 5); ++e) {
      mn = min(mn, red_min[e]);
      mx = max(mx, red_max[e]);
    }
    if (mn <= mx) {
      atomicMin(&p.yq->acc_min, mn);
      atomicMax(&p.yq->acc_max, mx);
    }
  }
}

// 3x3 stride-1 depthwise with the input staged in shared memory.  A CTA walks over output tiles of TR rows x TWt
// columns; one TMA box brings the (TR + 2) x (TWt + 2) pixel patch of all C channels (padding pixels arrive as
// zeros), double buffered, so the loads of the next tile run under the arithmetic of this one.  Thread = one
// 32-bit channel word (4 channels) x strips of 8 consecutive output pixels of one row; its 36 weights stay in
// registers, each pre-shifted into its byte lane so that one dp4a against an input word multiplies exactly one
// channel.  The accumulators start at minus the zero-point correction of the pixel's border class (table in
// shared memory, already multiplied by the input zero point), so the epilogue is statistics, requantization, store.
template <int kOut>
__global__ void __launch_bounds__(512) depthwise3x3_tiled_kernel(const DwParams p, const __grid_constant__ CUtensorMap tmap) {
  extern __shared__ uint8_t dsm_raw[];
  __shared__ __align__(8) uint64_t full_bar[2];
  __shared__ int abort_s;
  __shared__ int red_min[16], red_max[16];
  const uint32_t patch0 = (smem_u32(dsm_raw) + 127u) & ~127u;
  uint8_t* gen = dsm_raw + (patch0 - smem_u32(dsm_raw));
  int32_t* zc_s = reinterpret_cast<int32_t*>(gen + 2u * p.patch_stride);
  uint8_t* rcls_s = reinterpret_cast<uint8_t*>(zc_s + p.ncls * p.C);
  uint8_t* ccls_s = rcls_s + p.Ho;
  volatile int* abort_flag = &abort_s;
  const int CW = p.C / 4;
  const int cw = threadIdx.x % CW, slot = threadIdx.x / CW;
  const uint32_t bar0 = smem_u32(full_bar);
  if (threadIdx.x == 0) {
    abort_s = 0;
    mbar_init(bar0, 1);
    mbar_init(bar0 + 8u, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&tmap) : "memory");
  }
  __syncthreads();
  grid_dependency_wait();   // launched ahead of its predecessor's end: see launch_overlapped

  const int total = p.N * p.tiles_h * p.tiles_w;
  int armed[2] = {0, 0};   // thread 0: copies issued into each buffer (for the drain of a CTA that gave up)
  auto issue = [&](int tile, int buf) {   // one thread: the patch of `tile` into buffer `buf`
    const int tw = tile % p.tiles_w;
    const int th = (tile / p.tiles_w) % p.tiles_h;
    const int n = tile / (p.tiles_w * p.tiles_h);
    ++armed[buf];
    mbar_expect_tx(bar0 + 8u * buf, p.patch_bytes);
    tma_load_4d(patch0 + buf * p.patch_stride, &tmap, 0, tw * p.TWt - p.pad_w, th * p.TR - p.pad_h, n, bar0 + 8u * buf);
  };
  if (threadIdx.x == 0) {
    if ((int)blockIdx.x < total) issue(blockIdx.x, 0);
    if ((int)(blockIdx.x + gridDim.x) < total) issue(blockIdx.x + gridDim.x, 1);
  }
  QParams q;
  q.s_acc = __fmul_rn(p.xq->scale, *p.w_scale);
  q.zx = p.xq->zero_point;
  q.inv_scale = (kOut == kOutInt8) ? p.yq->inv_scale : 1.0f;
  q.zp = (kOut == kOutInt8) ? p.yq->zero_point : 0;
  qparams_finish(q);
  if (kOut == kOutInt8) qparams_output_mode(q, p.yq->rounding, p.yq->seed, p.yq->step);
  int sat_below = 0, sat_above = 0;
  if (blockIdx.x == 0 && threadIdx.x == 0) p.yq->acc_scale = q.s_acc;
  for (int i = threadIdx.x; i < p.ncls * p.C; i += blockDim.x) zc_s[i] = q.zx * p.corr[i];
  for (int i = threadIdx.x; i < p.Ho; i += blockDim.x) rcls_s[i] = p.rowcls[i];
  for (int i = threadIdx.x; i < p.Wo; i += blockDim.x) ccls_s[i] = p.colcls[i];
  int wsel[9][4];   // weight of (tap, channel k) in byte lane k
  const bool worker = slot < p.slots;
  if (worker) {
#pragma unroll
    for (int t = 0; t < 9; ++t) {
      const uint32_t w4 = *reinterpret_cast<const uint32_t*>(p.w + (int64_t)t * p.C + cw * 4);
#pragma unroll
      for (int k = 0; k < 4; ++k) wsel[t][k] = (int)(w4 & (0xffu << (8 * k)));
    }
  }
  __syncthreads();   // tables complete

  int mn = INT32_MAX, mx = INT32_MIN;
  const int box_w = p.TWt + 2;
  const int ngw = p.TWt / kDwPix;
  const int strips = p.TR * ngw;
  const int pix_stride = p.C;   // bytes from one patch pixel to the next
  int it = 0;
  for (int tile = blockIdx.x; tile < total; tile += gridDim.x, ++it) {
    const int buf = it & 1;
    bool ok = mbar_wait(bar0 + 8u * buf, (uint32_t)(it >> 1) & 1u, abort_flag, p.status, kAsyncDepthwiseFullWait, 1000u);
    ok = __syncthreads_and(ok) != 0;   // one decision for the whole CTA
    if (!ok) break;
    const int tw = tile % p.tiles_w;
    const int th = (tile / p.tiles_w) % p.tiles_h;
    const int n = tile / (p.tiles_w * p.tiles_h);
    const uint8_t* patch = gen + buf * p.patch_stride + cw * 4;
    if (worker) {
      for (int s = slot; s < strips; s += p.slots) {
        const int row = s / ngw, g = s - row * ngw;
        const int ho = th * p.TR + row;
        const int wo0 = tw * p.TWt + g * kDwPix;
        if (ho >= p.Ho || wo0 >= p.Wo) continue;
        const int rc = rcls_s[ho] * p.ncolcls;
        int acc[kDwPix][4];
#pragma unroll
        for (int j = 0; j < kDwPix; ++j) {
          const int wo = min(wo0 + j, p.Wo - 1);
          const int4 zc = *reinterpret_cast<const int4*>(zc_s + (rc + ccls_s[wo]) * p.C + cw * 4);
          acc[j][0] = -zc.x;
          acc[j][1] = -zc.y;
          acc[j][2] = -zc.z;
          acc[j][3] = -zc.w;
        }
#pragma unroll
        for (int r = 0; r < 3; ++r) {
          const uint8_t* pr = patch + ((row + r) * box_w + g * kDwPix) * pix_stride;
          int xw[kDwPix + 2];
#pragma unroll
          for (int j = 0; j < kDwPix + 2; ++j) xw[j] = *reinterpret_cast<const int*>(pr + j * pix_stride);
#pragma unroll
          for (int sx = 0; sx < 3; ++sx)
#pragma unroll
            for (int j = 0; j < kDwPix; ++j)
#pragma unroll
              for (int k = 0; k < 4; ++k) acc[j][k] = __dp4a(xw[j + sx], wsel[r * 3 + sx][k], acc[j][k]);
        }
        const int64_t o0 = (((int64_t)n * p.Ho + ho) * p.Wo + wo0) * p.C + cw * 4;
#pragma unroll
        for (int j = 0; j < kDwPix; ++j) {
          if (wo0 + j < p.Wo) {
            mn = min(__vimin3_s32(mn, acc[j][0], acc[j][1]), min(acc[j][2], acc[j][3]));
            mx = max(__vimax3_s32(mx, acc[j][0], acc[j][1]), max(acc[j][2], acc[j][3]));
            const int64_t o = o0 + (int64_t)j * p.C;
            if constexpr (kOut == kOutInt8) {
              const uint32_t w = quant4_acc(acc[j][0], acc[j][1], acc[j][2], acc[j][3], o, q, sat_below, sat_above);
              *reinterpret_cast<uint32_t*>(reinterpret_cast<int8_t*>(p.out) + o) = w;
            } else {
              uint32_t w[4];
#pragma unroll
              for (int k = 0; k < 4; ++k)
                w[k] = (kOut == kOutF32) ? __float_as_uint(__fmul_rn(__int2float_rn(acc[j][k]), q.s_acc)) : (uint32_t)acc[j][k];
              *reinterpret_cast<uint4*>(reinterpret_cast<uint32_t*>(p.out) + o) = make_uint4(w[0], w[1], w[2], w[3]);
            }
          }
        }
      }
    }
    __syncthreads();   // every thread is done with this buffer
    if (threadIdx.x == 0 && tile + 2 * (int)gridDim.x < total) issue(tile + 2 * gridDim.x, buf);
  }
  grid_launch_dependents();   // the successor may take the SMs that free up from here on
  if (*abort_flag != 0 && threadIdx.x == 0) {   // gave up: wait, bounded, for the patches still on their way
    for (int b = 0; b < 2; ++b)
      if (armed[b] > 0) mbar_drain(bar0 + 8u * b, (uint32_t)(armed[b] - 1) & 1u);
  }
  if (q.count_sat) {   // clipped outputs: one atomic pair per warp that saw any
    sat_below = __reduce_add_sync(0xffffffffu, sat_below);
    sat_above = __reduce_add_sync(0xffffffffu, sat_above);
    if ((threadIdx.x & 31) == 0) {
      if (sat_below) atomicAdd(&p.yq->sat_below, (uint32_t)sat_below);
      if (sat_above) atomicAdd(&p.yq->sat_above, (uint32_t)sat_above);
    }
  }
  mn = __reduce_min_sync(0xffffffffu, mn);
  mx = __reduce_max_sync(0xffffffffu, mx);
  const int warp = threadIdx.x >> 5;
  if ((threadIdx.x & 31) == 0) {
    red_min[warp] = mn;
    red_max[warp] = mx;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int e = 1; e < (int)((blockDim.x + 31) >> 5); ++e) {
      mn = min(mn, red_min[e]);
      mx = max(mx, red_max[e]);
    }
    if (mn <= mx) {
      atomicMin(&p.yq->acc_min, mn);
      atomicMax(&p.yq->acc_max, mx);
    }
  }
}

}  // namespace

cudaError_t launch_range_update(hq_range_state* st, int count, float eta, cudaStream_t s, bool overlap) {
  return launch_overlapped(range_update_kernel, (count + 127) / 128, 128, 0, s, overlap, st, count, eta);
}

cudaError_t launch_stats_pack(const hq_range_state* st, int count, int32_t* buf, cudaStream_t s) {
  stats_pack_kernel<<<(count + 127) / 128, 128, 0, s>>>(st, count, buf);
  return cudaGetLastError();
}
cudaError_t launch_stats_unpack(hq_range_state* st, int count, const int32_t* buf, cudaStream_t s) {
  stats_unpack_kernel<<<(count + 127) / 128, 128, 0, s>>>(st, count, buf);
  return cudaGetLastError();
}

cudaError_t launch_dynamic_derive(hq_range_state* st, cudaStream_t s, bool overlap) {
  return launch_overlapped(dynamic_derive_kernel, 1, 1, 0, s, overlap, st);
}

cudaError_t launch_quantize_pass(const float* y, int8_t* out, int64_t count, hq_range_state* st, int num_sms, cudaStream_t s,
                                 bool overlap) {
  const int threads = 256;
  int64_t want = (count / 16 + threads - 1) / threads;
  int blocks = (int)(want < 1 ? 1 : (want > (int64_t)num_sms * 8 ? (int64_t)num_sms * 8 : want));
  return launch_overlapped(quantize_pass_kernel, blocks, threads, 0, s, overlap, y, out, count, st);
}

cudaError_t launch_prep_weights(const int8_t* W, int8_t* Wmat, int Nout, int ntaps, int Cpad, int Ksrc, int R, int S, int Csrc,
                                const int8_t* tap_r, const int8_t* tap_s, int transposed, int blockdiag_g, cudaStream_t s) {
  TapList tl{};
  for (int t = 0; t < ntaps; ++t) {
    tl.r[t] = tap_r[t];
    tl.s[t] = tap_s[t];
  }
  const int64_t total = (int64_t)Nout * ntaps * Cpad;
  int blocks = (int)((total + 255) / 256);
  if (blocks > 4096) blocks = 4096;
  prep_weights_kernel<<<blocks, 256, 0, s>>>(W, Wmat, Nout, ntaps, Cpad, Ksrc, R, S, Csrc, tl, transposed, blockdiag_g);
  return cudaGetLastError();
}

cudaError_t launch_corr(const int8_t* Wmat, int32_t* corr, int Nout, int ntaps, int Cpad, int nrowtaps, int ncoltaps, const uint32_t* rowmasks,
                        int nrowcls, const uint32_t* colmasks, int ncolcls, int corr_ld, cudaStream_t s) {
  ClassMasks m{};
  for (int i = 0; i < nrowcls; ++i) m.row[i] = rowmasks[i];
  for (int i = 0; i < ncolcls; ++i) m.col[i] = colmasks[i];
  const int total = nrowcls * ncolcls * Nout;
  corr_kernel<<<(total + 7) / 8, 256, 0, s>>>(Wmat, corr, Nout, ntaps, Cpad, nrowtaps, ncoltaps, m, nrowcls, ncolcls, corr_ld);
  return cudaGetLastError();
}

cudaError_t launch_dw_dense(const int8_t* W, int8_t* Wd, int taps, int c0, int cw, cudaStream_t s) {
  const int total = cw * taps * cw;
  dw_dense_kernel<<<std::min((total + 255) / 256, 1024), 256, 0, s>>>(W, Wd, taps, c0, cw);
  return cudaGetLastError();
}

cudaError_t launch_dw_prep(const int8_t* W, int8_t* Wt, int32_t* corr, int C, int R, int S, const uint32_t* rowmasks, int nrowcls,
                           const uint32_t* colmasks, int ncolcls, int flip, cudaStream_t s) {
  ClassMasks m{};
  for (int i = 0; i < nrowcls; ++i) m.row[i] = rowmasks[i];
  for (int i = 0; i < ncolcls; ++i) m.col[i] = colmasks[i];
  int total = nrowcls * ncolcls * C;
  if (C * R * S > total) total = C * R * S;
  dw_prep_kernel<<<(total + 127) / 128, 128, 0, s>>>(W, Wt, corr, C, R, S, m, nrowcls, ncolcls, flip);
  return cudaGetLastError();
}

cudaError_t launch_prep_patch_weights(const int8_t* W, int8_t* Wmat, int K, int R, int SC, int RP, int ld, cudaStream_t s) {
  const int64_t total = (int64_t)K * ld;
  prep_patch_weights_kernel<<<(int)std::min<int64_t>((total + 255) / 256, 1024), 256, 0, s>>>(W, Wmat, K, R, SC, RP, ld);
  return cudaGetLastError();
}

cudaError_t launch_patch_matrix(const int8_t* x, int8_t* A, const hq_range_state* xq, int N, int H, int W, int C, int Ho, int Wo, int R, int S,
                                int stride_h, int stride_w, int pad_h, int pad_w, int Kp, int RP, cudaStream_t s) {
  const int64_t groups = ((int64_t)N * Ho * Wo + kPatchPixels - 1) / kPatchPixels;
  int blocks = (int)std::min<int64_t>(groups, 148 * 8);
  if (blocks < 1) blocks = 1;
  patch_matrix_kernel<<<blocks, 256, (size_t)kPatchPixels * Kp, s>>>(x, A, xq, N, H, W, C, Ho, Wo, R, S, stride_h, stride_w, pad_h, pad_w, Kp, RP);
  return cudaGetLastError();
}

cudaError_t launch_row_window(const int8_t* x, int8_t* X2, const hq_range_state* xq, int N, int H, int W, int C, int Hg, int Wo, int S, int sh,
                              int stride_w, int pad_w, int SB, cudaStream_t s) {
  const int64_t total = (int64_t)N * Hg * Wo * sh;
  if (total >= (int64_t)1 << 31) return cudaErrorInvalidValue;   // checked when the layer is prepared
  if ((sh & (sh - 1)) != 0) return cudaErrorInvalidValue;
  int blocks = (int)std::min<int64_t>((int64_t)N * Hg, 148 * 64);
  if (blocks < 1) blocks = 1;
  switch (SB) {
    case 16: row_window_kernel<4><<<blocks, 256, 0, s>>>(x, X2, xq, N, H, W, C, Hg, Wo, S, sh, stride_w, pad_w); break;
    case 32: row_window_kernel<8><<<blocks, 256, 0, s>>>(x, X2, xq, N, H, W, C, Hg, Wo, S, sh, stride_w, pad_w); break;
    case 64: row_window_kernel<16><<<blocks, 256, 0, s>>>(x, X2, xq, N, H, W, C, Hg, Wo, S, sh, stride_w, pad_w); break;
    case 128: row_window_kernel<32><<<blocks, 256, 0, s>>>(x, X2, xq, N, H, W, C, Hg, Wo, S, sh, stride_w, pad_w); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

cudaError_t launch_prep_window_weights(const int8_t* W, int8_t* Wmat, int K, int R, int SC, int sh, int SB, int ntaps, int dh_min, int pad_h,
                                       cudaStream_t s) {
  const int64_t total = (int64_t)K * ntaps * sh * SB;
  prep_window_weights_kernel<<<(int)std::min<int64_t>((total + 255) / 256, 1024), 256, 0, s>>>(W, Wmat, K, R, SC, sh, SB, ntaps, dh_min, pad_h);
  return cudaGetLastError();
}

cudaError_t launch_pad_rows(const int8_t* src, int8_t* dst, int rows, int K, int Kp, cudaStream_t s) {
  const int64_t total = (int64_t)rows * Kp;
  int blocks = (int)std::min<int64_t>((total + 255) / 256, 148 * 16);
  if (blocks < 1) blocks = 1;
  pad_rows_kernel<<<blocks, 256, 0, s>>>(src, dst, rows, K, Kp);
  return cudaGetLastError();
}

cudaError_t launch_transpose_rows(const int8_t* in, int8_t* out, int R, int C, int Rp, int ones_row, cudaStream_t s) {
  dim3 grid((unsigned)((Rp + 31) / 32), (unsigned)((C + (ones_row ? 16 : 0) + 31) / 32));
  transpose_rows_kernel<<<grid, 256, 0, s>>>(in, out, R, C, Rp, ones_row);
  return cudaGetLastError();
}
cudaError_t launch_im2col_t(const int8_t* X, int8_t* Bt, const hq_range_state* xq, const hq_conv_desc& d, int Ho, int Wo, int64_t Mp, int32_t* colsum,
                            FastDiv fd_wo, FastDiv fd_ho, cudaStream_t s) {
  const int64_t M = (int64_t)d.N * Ho * Wo;
  const int tiles = (int)((Mp + 127) / 128), tiles_per_block = tiles >= 4096 ? 16 : (tiles >= 256 ? 8 : 1);
  dim3 grid((unsigned)((tiles + tiles_per_block - 1) / tiles_per_block), (unsigned)((d.C + 31) / 32), (unsigned)(d.R * d.S));
  im2col_t_kernel<<<grid, 256, 0, s>>>(X, Bt, xq, d, Ho, Wo, (int)M, (int)Mp, tiles_per_block, fd_wo, fd_ho, colsum);
  return cudaGetLastError();
}
cudaError_t launch_dw_wgrad(const int8_t* dY, const int8_t* X, const hq_range_state* dyq, const hq_range_state* xq, const hq_conv_desc& d, int Ho,
                            int Wo, int num_sms, FastDiv fd_wo, FastDiv fd_ho, int32_t* acc, float* G, cudaStream_t s) {
  const int M = d.N * Ho * Wo, T = d.R * d.S;
  int blocks = std::max(1, std::min(num_sms * 4, (M + 255) / 256));
  const int pixels_per_block = (M + blocks - 1) / blocks;
  blocks = (M + pixels_per_block - 1) / pixels_per_block;
  const size_t smem = (size_t)d.C * T * sizeof(int32_t);
  if (d.R == 3)
    dw_wgrad_kernel<3><<<blocks, 256, smem, s>>>(dY, X, dyq, xq, d, Ho, Wo, M, pixels_per_block, fd_wo, fd_ho, acc);
  else
    dw_wgrad_kernel<5><<<blocks, 256, smem, s>>>(dY, X, dyq, xq, d, Ho, Wo, M, pixels_per_block, fd_wo, fd_ho, acc);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  scale_to_real_kernel<<<std::max(1, std::min(64, (d.C * T + 255) / 256)), 256, 0, s>>>(acc, d.C * T, dyq, xq, G);
  return cudaGetLastError();
}
cudaError_t launch_wgrad_reduce(const int32_t* slabs, int nslabs, int rows, int cols, const int32_t* colsum, const int32_t* rowsum, int M,
                                const hq_range_state* dyq, const hq_range_state* xq, float* G, cudaStream_t s) {
  const int64_t total = (int64_t)rows * cols;
  const int blocks = (int)std::max<int64_t>(1, std::min<int64_t>((total + 255) / 256, 148 * 16));
  wgrad_reduce_kernel<<<blocks, 256, 0, s>>>(slabs, nslabs, rows, cols, colsum, rowsum, M, dyq, xq, G);
  return cudaGetLastError();
}
cudaError_t launch_wgrad_pack(const int8_t* src, int8_t* dst, int N, int Hs, int Ws, int Cs, int Hp, int P, int row_off, int sign, int pad, int limit,
                              int64_t pitch, const PackRanges& rg, int32_t* sums, cudaStream_t s) {
  if (P > kPackMaxP || P % 16 != 0 || Ws > kPackMaxP || rg.nr * rg.ns > 64 || rg.ns > 8 || pad > 16 || rg.ns - 1 - pad > 16 || Cs % 4 != 0)
    return cudaErrorInvalidValue;
  dim3 grid((unsigned)((Hp + kPackRows - 1) / kPackRows), (unsigned)((Cs + 31) / 32), (unsigned)N);
  const int tp = pack_tile_pitch(P, Ws, limit);
  wgrad_pack_kernel<<<grid, 256, (size_t)kPackRows * 32 * tp * sizeof(uint32_t), s>>>(src, dst, Hs, Ws, Cs, Hp, P, row_off, sign, pad, limit, pitch, rg, sums, tp);
  return cudaGetLastError();
}
cudaError_t launch_zero_tail(int8_t* base, int rows, int64_t pitch, int64_t from, cudaStream_t s) {
  if (from >= pitch) return cudaSuccess;
  const int64_t total = (pitch - from) / 16 * rows;
  zero_tail_kernel<<<(int)std::max<int64_t>(1, std::min<int64_t>((total + 255) / 256, 148 * 8)), 256, 0, s>>>(base, rows, pitch, from);
  return cudaGetLastError();
}
cudaError_t launch_wgrad_reduce_taps(const int32_t* slabs, int nslabs, int rows, int slab_rows, int cols, int C, const int32_t* colsum,
                                     const int32_t* rowsum, const TapCounts& mvalid, const hq_range_state* dyq, const hq_range_state* xq, float* G,
                                     cudaStream_t s) {
  const int64_t total = (int64_t)rows * cols;
  const int blocks = (int)std::max<int64_t>(1, std::min<int64_t>((total + 31) / 32, 148 * 16));
  wgrad_reduce_taps_kernel<<<blocks, 256, 0, s>>>(slabs, nslabs, rows, slab_rows, cols, C, colsum, rowsum, mvalid, dyq, xq, G);
  return cudaGetLastError();
}
cudaError_t launch_wgrad_row_terms(const int8_t* dYt, int M, int Mp, int N, const hq_range_state* dyq, const hq_range_state* xq, int32_t* terms,
                                   cudaStream_t s) {
  wgrad_row_terms_kernel<<<(N + 7) / 8, 256, 0, s>>>(dYt, M, Mp, N, dyq, xq, terms);
  return cudaGetLastError();
}

cudaError_t launch_rowsum(const int8_t* a, const hq_range_state* aq, const hq_conv_desc& d, int Ho, int Wo, int bwd, int zw, int32_t* out,
                          cudaStream_t s) {
  const int64_t total = bwd ? (int64_t)d.N * d.H * d.W : (int64_t)d.N * Ho * Wo;
  const int blocks = (int)std::max<int64_t>(1, std::min<int64_t>((total + 255) / 256, 148 * 16));
  rowsum_kernel<<<blocks, 256, 0, s>>>(a, aq, d, Ho, Wo, bwd, zw, out, total);
  return cudaGetLastError();
}

cudaError_t launch_depthwise_bwd(const DwParams& p, int out_mode, int num_sms, cudaStream_t s) {
  const int64_t total = (int64_t)p.N * p.H * p.W * (p.C / 16);
  int64_t want = (total + 255) / 256;
  int blocks = (int)(want > (int64_t)num_sms * 8 ? (int64_t)num_sms * 8 : want);
  if (blocks < 1) blocks = 1;
  switch (out_mode) {
    case kOutInt8: depthwise_bwd_kernel<kOutInt8><<<blocks, 256, 0, s>>>(p); break;
    case kOutF32: depthwise_bwd_kernel<kOutF32><<<blocks, 256, 0, s>>>(p); break;
    default: depthwise_bwd_kernel<kOutAcc><<<blocks, 256, 0, s>>>(p); break;
  }
  return cudaGetLastError();
}

uint32_t depthwise_tiled_smem_bytes(const DwParams& p) {
  return 2u * p.patch_stride + (uint32_t)p.ncls * p.C * 4u + (uint32_t)p.Ho + (uint32_t)p.Wo + 256u;
}

cudaError_t depthwise_tiled_set_smem_attr(uint32_t smem_bytes) {
  cudaError_t e = cudaFuncSetAttribute(depthwise3x3_tiled_kernel<kOutInt8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(depthwise3x3_tiled_kernel<kOutF32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(depthwise3x3_tiled_kernel<kOutAcc>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
}

cudaError_t launch_depthwise_tiled(const DwParams& p, const CUtensorMap& tmap, int out_mode, int num_sms, cudaStream_t s) {
  const int total = p.N * p.tiles_h * p.tiles_w;
  const uint32_t smem = depthwise_tiled_smem_bytes(p);
  const int per_sm = smem <= 110u * 1024u ? 2 : 1;
  const int grid = std::max(1, std::min(total, num_sms * per_sm));
  const int threads = ((p.C / 4) * p.slots + 31) / 32 * 32;
  switch (out_mode) {
    case kOutInt8: depthwise3x3_tiled_kernel<kOutInt8><<<grid, threads, smem, s>>>(p, tmap); break;
    case kOutF32: depthwise3x3_tiled_kernel<kOutF32><<<grid, threads, smem, s>>>(p, tmap); break;
    default: depthwise3x3_tiled_kernel<kOutAcc><<<grid, threads, smem, s>>>(p, tmap); break;
  }
  return cudaGetLastError();
}

cudaError_t launch_depthwise(const DwParams& p, int out_mode, int num_sms, cudaStream_t s, bool overlap) {
  const int CW = p.C / 4;
  if (p.R == 3 && p.S == 3 && p.stride_h == 1 && p.stride_w == 1 && CW <= 256 && p.w_zp == 0) {
    const int slots = 256 / CW;                           // pixel groups per block
    const int threads = ((slots * CW + 31) / 32) * 32;
    const int groups_w = (p.Wo + kDwPix - 1) / kDwPix;
    const int64_t items = (int64_t)p.N * p.Ho * groups_w;
    int blocks = (int)std::min<int64_t>((items + slots - 1) / slots, (int64_t)num_sms * 8);
    if (blocks < 1) blocks = 1;
    switch (out_mode) {
      case kOutInt8: return launch_overlapped(depthwise3x3_kernel<kOutInt8>, blocks, threads, 0, s, overlap, p, slots, groups_w);
      case kOutF32: return launch_overlapped(depthwise3x3_kernel<kOutF32>, blocks, threads, 0, s, overlap, p, slots, groups_w);
      default: return launch_overlapped(depthwise3x3_kernel<kOutAcc>, blocks, threads, 0, s, overlap, p, slots, groups_w);
    }
  }
  const int64_t total = (int64_t)p.N * p.Ho * p.Wo * (p.C / 16);
  int64_t want = (total + 255) / 256;
  int blocks = (int)(want > (int64_t)num_sms * 8 ? (int64_t)num_sms * 8 : want);
  if (blocks < 1) blocks = 1;
  switch (out_mode) {
    case kOutInt8: return launch_overlapped(depthwise_kernel<kOutInt8>, blocks, 256, 0, s, overlap, p);
    case kOutF32: return launch_overlapped(depthwise_kernel<kOutF32>, blocks, 256, 0, s, overlap, p);
    default: return launch_overlapped(depthwise_kernel<kOutAcc>, blocks, 256, 0, s, overlap, p);
  }
}

}  // namespace hq
