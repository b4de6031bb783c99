// hq_oracle.cpp -- CPU oracle for the in-hindsight int8 quantized layer.
//
// THIS IS TEST INFRASTRUCTURE.  It is a plain, slow, literal restatement of what
// the paper's hot path computes, written to be checked against the paper by eye.
// Nothing in the product library links, includes, imports or calls it; it shares
// no code, table or constant generator with the CUDA kernels.
//
// What it follows (arxiv 2105.04246):
//   Sec. 3.1        quantized layer: 8-bit X~ and W~ feed the MAC array, the output Y
//                   is held in 32-bit accumulators and then quantized by Q_Y; backward,
//                   the 8-bit output gradient and the weights give the input gradient
//                   G_X, which is quantized by Q_G.
//   Sec. 3.1        weight gradient of a linear layer from the quantized output gradient and
//                   the quantized input, kept in binary32 (hqo_linear_wgrad_acc).
//   Sec. 3.2, Eq. 1 dynamic quantization: range = (min G, max G) of the current tensor;
//                   the 32-bit output is written out, reduced, read back and quantized.
//   Sec. 3.2        static quantization: the range is known in advance, each
//                   accumulator output is quantized directly.
//   Sec. 4 / 4.1    in-hindsight min-max: quantize iteration t with the range estimated
//                   up to t-1; record min/max of the unquantized output at the
//                   accumulator; Eq. 2-3 moving average; initialisation at t = 0 by the
//                   min-max of the first tensor.
//
// Readings taken where the paper is silent (the paper names "asymmetric uniform
// quantization" without an equation, so these are conventions, not citations):
//   R-1  affine quantizer on 2^8 levels: s = (hi - lo)/255, integer zero point,
//        q = clamp(round(y/s) + z).
//   R-2  signed storage, levels -128..127.
//   R-3  the derived grid is widened to contain 0 (lo = min(q_min,0), hi = max(q_max,0));
//        the running (q_min,q_max) of Eq. 2-3 stay un-widened.
//   R-4  round half to even; y/s is evaluated as y * (1/s) with 1/s rounded once; every
//        floating-point step is one binary32 round-to-nearest-even operation, never fused.
//   R-5  weights symmetric by default (z_w = 0); every accumulator loop takes z_w, pinned with non-zero
//        values against int64 matrix products, scatter-form loops and library convolutions in float64.
//   R-6  deterministic rounding for gradients as well.
//   R-7  statistics are taken on the zero-point-corrected int32 accumulator (+ int32
//        bias), before any clamping; float(min acc) * s_acc is then the exact minimum of
//        the binary32 output because the map is monotone.
//   R-8  padding is zero in the real domain: padded taps are skipped.
//   R-9  t = 0 runs the dynamic path; from t = 1 the range of t-1 is used.
//   R-13 a degenerate range (hi - lo not > 0) gives s = 1.
//   R-15 the dynamic path materialises binary32 y = fl(float(acc) * s_acc).
//   R-18..R-20 stochastic rounding for gradients: see the section further down.
//   R-22 saturation statistic: see hqo_saturation.
//
// Pins (tests/ -m "not gpu"): brute-force and readable-by-eye cases for the index
// arithmetic, the forward/backward adjoint identity, the trace identity <dY, X W^T> = <dY^T X, W>
// that ties the weight gradient to the forward layer, library convolutions in float64,
// the closed form of the Eq. 2-3 recurrence, grid invariants of the quantizer, and
// static == dynamic when the ranges coincide; the stochastic dynamic path is tied to the
// deterministic one (range) and to the static stochastic quantizer (codes, draw count).
// PARITY UNPINNED: the tie rule of the rounding (R-4), the zero-point formula of
// hqo_derive beyond its grid invariants, and symmetric weights (R-5) are fixed by the
// readings above only -- the paper prints no formula or worked example for them.
//
// Build: g++ -O2 -std=c++17 -ffp-contract=off -fopenmp -shared -fPIC hq_oracle.cpp

#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>

extern "C" {

// ------------------------------------------------------------------------------------
// Per-tensor quantizer state (Sec. 4.1: the running range; plus what is derived from it)
// ------------------------------------------------------------------------------------
typedef struct {
  float q_min, q_max;      // running range, Eq. 2-3 (un-widened)
  float scale, inv_scale;  // s and fl(1/s) of the derived grid
  int32_t zero_point;      // z in [-128,127]
  uint32_t step;           // 0 = not initialised (t = 0 not seen yet)
} hqo_range;

typedef struct {
  int32_t N, H, W, C;      // input  NHWC
  int32_t K;               // output channels (== C when depthwise)
  int32_t R, S;            // filter height, width
  int32_t stride_h, stride_w, pad_h, pad_w;
  int32_t groups;          // 1, or C for depthwise
} hqo_conv;

static inline int out_dim(int in, int pad, int k, int stride) { return (in + 2 * pad - k) / stride + 1; }
int32_t hqo_out_h(const hqo_conv* d) { return out_dim(d->H, d->pad_h, d->R, d->stride_h); }
int32_t hqo_out_w(const hqo_conv* d) { return out_dim(d->W, d->pad_w, d->S, d->stride_w); }

// round to nearest integer, ties to even, then to int32 with saturation; NaN -> 0.
static inline int32_t round_half_even_to_i32(float u) {
  if (u != u) return 0;
  float r = std::nearbyintf(u);  // default rounding mode = to nearest even
  if (r >= 2147483648.0f) return std::numeric_limits<int32_t>::max();
  if (r <= -2147483648.0f) return std::numeric_limits<int32_t>::min();
  return (int32_t)r;
}
static inline int32_t clamp_i64(int64_t v, int32_t lo, int32_t hi) { return v < lo ? lo : (v > hi ? hi : (int32_t)v); }

// DERIVE (R-1, R-2, R-3, R-13): grid parameters from the running range.
void hqo_derive(hqo_range* q) {
  float lo = q->q_min < 0.0f ? q->q_min : 0.0f;
  float hi = q->q_max > 0.0f ? q->q_max : 0.0f;
  float width = hi - lo;
  float scale = width / 255.0f;
  if (!(scale > 0.0f)) scale = 1.0f;
  q->scale = scale;
  q->inv_scale = 1.0f / scale;
  float zl = lo / scale;
  q->zero_point = clamp_i64((int64_t)-128 - (int64_t)round_half_even_to_i32(zl), -128, 127);
}

// ------------------------------------------------------------------------------------
// O1: the 32-bit accumulator (Sec. 3.1 / 3.2).  Each *_point function is the definition
// of one output element, summed in int64; the tensor functions call it for every
// element and report (return value 1) if anything left the int32 range.
// ------------------------------------------------------------------------------------

// linear: acc[m,n] = sum_k (x[m,k] - z_x) * (w[n,k] - z_w) (+ bias[n])
static inline int64_t linear_point(int K, const int8_t* X, int zx, const int8_t* W, int zw, const int32_t* bias, int m, int n) {
  int64_t a = 0;
  for (int k = 0; k < K; ++k) a += (int64_t)((int)X[(int64_t)m * K + k] - zx) * ((int)W[(int64_t)n * K + k] - zw);
  if (bias) a += bias[n];
  return a;
}

int hqo_linear_acc(int M, int N, int K, const int8_t* X, int zx, const int8_t* W, int zw, const int32_t* bias, int32_t* acc) {
  int ovf = 0;
#pragma omp parallel for reduction(| : ovf)
  for (int m = 0; m < M; ++m)
    for (int n = 0; n < N; ++n) {
      int64_t a = linear_point(K, X, zx, W, zw, bias, m, n);
      if (a > INT32_MAX || a < INT32_MIN) ovf |= 1;
      acc[(int64_t)m * N + n] = (int32_t)a;
    }
  return ovf;
}

// weight gradient of a linear layer (Sec. 3.1, backward pass: the quantized output gradient G~_Y and the quantized layer
// input X~ give G_W, which stays in binary32):  g[n,k] = sum_m (dy[m,n] - z_dy) * (x[m,k] - z_x)  in int32, and
// G_W[n,k] = fl(float(g[n,k]) * fl(s_dy * s_x)).  dY is [M][N], X is [M][K], G_W is [N][K] like the weights.
int hqo_linear_wgrad_acc(int M, int N, int K, const int8_t* dY, int zdy, const int8_t* X, int zx, int32_t* g) {
  int ovf = 0;
#pragma omp parallel for reduction(| : ovf)
  for (int n = 0; n < N; ++n)
    for (int k = 0; k < K; ++k) {
      int64_t a = 0;
      for (int m = 0; m < M; ++m) a += (int64_t)((int)dY[(int64_t)m * N + n] - zdy) * ((int)X[(int64_t)m * K + k] - zx);
      if (a > INT32_MAX || a < INT32_MIN) ovf |= 1;
      g[(int64_t)n * K + k] = (int32_t)a;
    }
  return ovf;
}
// weight gradient of a convolution (Sec. 3.1, backward pass), W layout [K][R][S][C]:
//   g(k,r,s,c) = sum over n,ho,wo of (dy(n,ho,wo,k) - z_dy) * (x(n,hi,wi,c) - z_x),  hi = ho*stride_h - pad_h + r (wi alike),
//   over those output pixels whose (hi,wi) lies inside the image: padding is zero in the real domain (R-8), so a padded
//   tap contributes nothing.  G_W = fl(float(g) * fl(s_dy * s_x)).  Dense layers, or depthwise (groups == C == K).
int hqo_conv_wgrad_acc(const hqo_conv* d, const int8_t* dY, int zdy, const int8_t* X, int zx, int32_t* g) {
  const int Ho = hqo_out_h(d), Wo = hqo_out_w(d);
  int ovf = 0;
  if (d->groups != 1) {   // depthwise (K == C), W layout [C][R][S]: the same sum with k == c and no sum over channels
#pragma omp parallel for collapse(2) reduction(| : ovf)
    for (int c = 0; c < d->C; ++c)
      for (int r = 0; r < d->R; ++r)
        for (int s = 0; s < d->S; ++s) {
          int64_t a = 0;
          for (int n = 0; n < d->N; ++n)
            for (int ho = 0; ho < Ho; ++ho) {
              const int hi = ho * d->stride_h - d->pad_h + r;
              if (hi < 0 || hi >= d->H) continue;
              for (int wo = 0; wo < Wo; ++wo) {
                const int wi = wo * d->stride_w - d->pad_w + s;
                if (wi < 0 || wi >= d->W) continue;
                a += (int64_t)((int)dY[(((int64_t)n * Ho + ho) * Wo + wo) * d->K + c] - zdy) *
                     ((int)X[(((int64_t)n * d->H + hi) * d->W + wi) * d->C + c] - zx);
              }
            }
          if (a > INT32_MAX || a < INT32_MIN) ovf |= 1;
          g[((int64_t)c * d->R + r) * d->S + s] = (int32_t)a;
        }
    return ovf;
  }
#pragma omp parallel for collapse(2) reduction(| : ovf)
  for (int k = 0; k < d->K; ++k)
    for (int r = 0; r < d->R; ++r)
      for (int s = 0; s < d->S; ++s)
        for (int c = 0; c < d->C; ++c) {
          int64_t a = 0;
          for (int n = 0; n < d->N; ++n)
            for (int ho = 0; ho < Ho; ++ho) {
              const int hi = ho * d->stride_h - d->pad_h + r;
              if (hi < 0 || hi >= d->H) continue;
              for (int wo = 0; wo < Wo; ++wo) {
                const int wi = wo * d->stride_w - d->pad_w + s;
                if (wi < 0 || wi >= d->W) continue;
                a += (int64_t)((int)dY[(((int64_t)n * Ho + ho) * Wo + wo) * d->K + k] - zdy) *
                     ((int)X[(((int64_t)n * d->H + hi) * d->W + wi) * d->C + c] - zx);
              }
            }
          if (a > INT32_MAX || a < INT32_MIN) ovf |= 1;
          g[(((int64_t)k * d->R + r) * d->S + s) * d->C + c] = (int32_t)a;
        }
  return ovf;
}

void hqo_scale_to_real(const int32_t* acc, int64_t count, float s_acc, float* out) {
  for (int64_t i = 0; i < count; ++i) out[i] = (float)acc[i] * s_acc;
}

// forward convolution, X NHWC, W [K][R][S][C/groups], Y [N][Ho][Wo][K]:
//   y(n,ho,wo,k) = sum over r,s,c of (x(n,hi,wi,c) - z_x) * (w(k,r,s,c) - z_w)
//   with hi = ho*stride_h - pad_h + r, wi = wo*stride_w - pad_w + s inside the image;
//   taps that fall on padding contribute nothing (R-8).  Depthwise: c == k only.
static inline int64_t conv_fwd_point(const hqo_conv* d, const int8_t* X, int zx, const int8_t* W, int zw, int n, int ho, int wo, int k) {
  const bool dw = d->groups != 1;
  const int Cg = dw ? 1 : d->C;
  int64_t a = 0;
  for (int r = 0; r < d->R; ++r) {
    int hi = ho * d->stride_h - d->pad_h + r;
    if (hi < 0 || hi >= d->H) continue;
    for (int s = 0; s < d->S; ++s) {
      int wi = wo * d->stride_w - d->pad_w + s;
      if (wi < 0 || wi >= d->W) continue;
      const int8_t* xp = X + (((int64_t)n * d->H + hi) * d->W + wi) * d->C + (dw ? k : 0);
      const int8_t* wp = W + (((int64_t)k * d->R + r) * d->S + s) * Cg;
      int32_t p = 0;  // at most 2^9 channels * 2^8 * 2^8: no overflow
      for (int c = 0; c < Cg; ++c) p += ((int)xp[c] - zx) * ((int)wp[c] - zw);
      a += p;
    }
  }
  return a;
}

int hqo_conv_fwd_acc(const hqo_conv* d, const int8_t* X, int zx, const int8_t* W, int zw, int32_t* acc) {
  const int Ho = hqo_out_h(d), Wo = hqo_out_w(d);
  int ovf = 0;
#pragma omp parallel for collapse(2) reduction(| : ovf)
  for (int n = 0; n < d->N; ++n)
    for (int ho = 0; ho < Ho; ++ho)
      for (int wo = 0; wo < Wo; ++wo)
        for (int k = 0; k < d->K; ++k) {
          int64_t a = conv_fwd_point(d, X, zx, W, zw, n, ho, wo, k);
          if (a > INT32_MAX || a < INT32_MIN) ovf |= 1;
          acc[(((int64_t)n * Ho + ho) * Wo + wo) * d->K + k] = (int32_t)a;
        }
  return ovf;
}

// backward data (input gradient), dY [N][Ho][Wo][K], W in the FORWARD layout, dX NHWC:
//   dx(n,hi,wi,c) = sum over r,s,k of (dy(n,ho,wo,k) - z_dy) * (w(k,r,s,c) - z_w)
//   over those (r,s) for which ho = (hi + pad_h - r)/stride_h and
//   wo = (wi + pad_w - s)/stride_w are integers inside the output image.
//   This is the transpose of the forward map x -> y.  Depthwise: k == c only.
static inline int64_t conv_bwd_point(const hqo_conv* d, int Ho, int Wo, const int8_t* dY, int zdy, const int8_t* W, int zw, int n, int hi, int wi, int c) {
  const bool dw = d->groups != 1;
  const int Cg = dw ? 1 : d->C;
  int64_t a = 0;
  for (int r = 0; r < d->R; ++r) {
    int th = hi + d->pad_h - r;
    if (th < 0 || th % d->stride_h != 0) continue;
    int ho = th / d->stride_h;
    if (ho >= Ho) continue;
    for (int s = 0; s < d->S; ++s) {
      int tw = wi + d->pad_w - s;
      if (tw < 0 || tw % d->stride_w != 0) continue;
      int wo = tw / d->stride_w;
      if (wo >= Wo) continue;
      const int8_t* gp = dY + (((int64_t)n * Ho + ho) * Wo + wo) * d->K;
      if (dw) {
        a += (int64_t)((int)gp[c] - zdy) * ((int)W[((int64_t)c * d->R + r) * d->S + s] - zw);
      } else {
        int32_t p = 0;
        for (int k = 0; k < d->K; ++k) p += ((int)gp[k] - zdy) * ((int)W[(((int64_t)k * d->R + r) * d->S + s) * Cg + c] - zw);
        a += p;
      }
    }
  }
  return a;
}

int hqo_conv_bwd_data_acc(const hqo_conv* d, const int8_t* dY, int zdy, const int8_t* W, int zw, int32_t* acc) {
  const int Ho = hqo_out_h(d), Wo = hqo_out_w(d);
  int ovf = 0;
#pragma omp parallel for collapse(2) reduction(| : ovf)
  for (int n = 0; n < d->N; ++n)
    for (int hi = 0; hi < d->H; ++hi)
      for (int wi = 0; wi < d->W; ++wi)
        for (int c = 0; c < d->C; ++c) {
          int64_t a = conv_bwd_point(d, Ho, Wo, dY, zdy, W, zw, n, hi, wi, c);
          if (a > INT32_MAX || a < INT32_MIN) ovf |= 1;
          acc[(((int64_t)n * d->H + hi) * d->W + wi) * d->C + c] = (int32_t)a;
        }
  return ovf;
}

// The same definitions at a list of flat output indices (for checking sampled outputs
// of tensors too large to evaluate in full).  kind: 0 linear, 1 conv fwd, 2 conv bwd-data.
void hqo_linear_acc_at(int M, int N, int K, const int8_t* X, int zx, const int8_t* W, int zw, const int32_t* bias, const int64_t* idx, int64_t count, int64_t* out) {
  (void)M;
#pragma omp parallel for
  for (int64_t i = 0; i < count; ++i) out[i] = linear_point(K, X, zx, W, zw, bias, (int)(idx[i] / N), (int)(idx[i] % N));
}
void hqo_conv_fwd_acc_at(const hqo_conv* d, const int8_t* X, int zx, const int8_t* W, int zw, const int64_t* idx, int64_t count, int64_t* out) {
  const int Ho = hqo_out_h(d), Wo = hqo_out_w(d);
#pragma omp parallel for
  for (int64_t i = 0; i < count; ++i) {
    int64_t t = idx[i];
    int k = (int)(t % d->K); t /= d->K;
    int wo = (int)(t % Wo); t /= Wo;
    int ho = (int)(t % Ho); t /= Ho;
    out[i] = conv_fwd_point(d, X, zx, W, zw, (int)t, ho, wo, k);
  }
}
void hqo_conv_bwd_data_acc_at(const hqo_conv* d, const int8_t* dY, int zdy, const int8_t* W, int zw, const int64_t* idx, int64_t count, int64_t* out) {
  const int Ho = hqo_out_h(d), Wo = hqo_out_w(d);
#pragma omp parallel for
  for (int64_t i = 0; i < count; ++i) {
    int64_t t = idx[i];
    int c = (int)(t % d->C); t /= d->C;
    int wi = (int)(t % d->W); t /= d->W;
    int hi = (int)(t % d->H); t /= d->H;
    out[i] = conv_bwd_point(d, Ho, Wo, dY, zdy, W, zw, (int)t, hi, wi, c);
  }
}

// ------------------------------------------------------------------------------------
// O2: statistics taken at the accumulator, before quantization (Sec. 4.1, R-7)
// ------------------------------------------------------------------------------------
void hqo_minmax(const int32_t* acc, int64_t count, int32_t* mn, int32_t* mx) {
  int32_t lo = INT32_MAX, hi = INT32_MIN;  // the "nothing seen" values
  for (int64_t i = 0; i < count; ++i) {
    if (acc[i] < lo) lo = acc[i];
    if (acc[i] > hi) hi = acc[i];
  }
  *mn = lo;
  *mx = hi;
}

// ------------------------------------------------------------------------------------
// O4: static quantization with a range known in advance (Sec. 3.2; Sec. 4 step 1)
// ------------------------------------------------------------------------------------
static inline int8_t quantize_real(float y, const hqo_range* q) {
  float u = y * q->inv_scale;
  int32_t r = round_half_even_to_i32(u);
  return (int8_t)clamp_i64((int64_t)r + q->zero_point, -128, 127);
}

void hqo_quantize(const int32_t* acc, int64_t count, float s_acc, const hqo_range* q, int8_t* out) {
  for (int64_t i = 0; i < count; ++i) {
    float y = (float)acc[i] * s_acc;
    out[i] = quantize_real(y, q);
  }
}

// ------------------------------------------------------------------------------------
// O5: range update after the whole tensor is done (Sec. 4.1, Eq. 2-3; t = 0 rule)
//   mn > mx (the "nothing seen" pair) means no layer ran: the state is left alone.
// ------------------------------------------------------------------------------------
void hqo_range_update(hqo_range* q, int32_t mn, int32_t mx, float s_acc, float eta) {
  if (mn > mx) return;
  float m_lo = (float)mn * s_acc;
  float m_hi = (float)mx * s_acc;
  if (q->step == 0) {  // q^0 = min/max of the first tensor
    q->q_min = m_lo;
    q->q_max = m_hi;
  } else {
    float one_minus_eta = 1.0f - eta;
    float a_lo = one_minus_eta * m_lo, b_lo = eta * q->q_min;
    float a_hi = one_minus_eta * m_hi, b_hi = eta * q->q_max;
    q->q_min = a_lo + b_lo;
    q->q_max = a_hi + b_hi;
  }
  q->step += 1;
  hqo_derive(q);
}

// ------------------------------------------------------------------------------------
// Dynamic path (Sec. 3.2, Eq. 1): write the 32-bit output, take min/max of the CURRENT
// tensor, derive the grid, read the output back and quantize it.  Leaves the state
// initialised, which makes it the t = 0 step of the in-hindsight scheme (R-9).
// ------------------------------------------------------------------------------------
void hqo_dynamic(const int32_t* acc, int64_t count, float s_acc, hqo_range* q, float* yf, int8_t* out) {
  for (int64_t i = 0; i < count; ++i) yf[i] = (float)acc[i] * s_acc;
  float lo = std::numeric_limits<float>::infinity(), hi = -lo;
  for (int64_t i = 0; i < count; ++i) {
    if (yf[i] < lo) lo = yf[i];
    if (yf[i] > hi) hi = yf[i];
  }
  if (count == 0) return;
  q->q_min = lo;
  q->q_max = hi;
  q->step += 1;
  hqo_derive(q);
  for (int64_t i = 0; i < count; ++i) out[i] = quantize_real(yf[i], q);
}

// ------------------------------------------------------------------------------------
// Stochastic rounding for gradients (the paper quantizes gradients with stochastic rounding;
// it gives no formula, so the conventions below are readings):
//   R-18  q = sat8(floor(fl(u + r)) + z) with u as in O4 (R-4) and r uniform in [0,1);
//         the sum is one binary32 round-to-nearest-even addition.
//   R-19  r = h / 65536 with h a 16-bit draw, so r is exact in binary32.
//   R-20  draws come from the counter-based generator Philox4x32-10 (Salmon, Moraes, Dror,
//         Shaw: "Parallel random numbers: as easy as 1, 2, 3", SC'11): key = (seed, 0),
//         counter = (low and high word of e >> 3, iteration, 0) for the element with linear
//         index e in the output tensor; of the call's four 32-bit words, element e takes half
//         number (e & 7): word (e & 7) >> 1, low half when e is even, high half when odd.
//         `iteration` is the number of range updates the output's state has seen.
// Pins: the generator against the known-answer vectors published with it; floor(u+r) is one
// of the two neighbours of u; exact for integer u; unbiased over draws; reproducible.
// ------------------------------------------------------------------------------------
static inline void mulhilo32(uint32_t a, uint32_t b, uint32_t* hi, uint32_t* lo) {
  uint64_t p = (uint64_t)a * (uint64_t)b;
  *hi = (uint32_t)(p >> 32);
  *lo = (uint32_t)p;
}

void hqo_philox4x32_10(const uint32_t counter[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t c0 = counter[0], c1 = counter[1], c2 = counter[2], c3 = counter[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    uint32_t hi0, lo0, hi1, lo1;
    mulhilo32(0xD2511F53u, c0, &hi0, &lo0);
    mulhilo32(0xCD9E8D57u, c2, &hi1, &lo1);
    uint32_t n0 = hi1 ^ c1 ^ k0, n1 = lo1, n2 = hi0 ^ c3 ^ k1, n3 = lo0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += 0x9E3779B9u;   // key schedule: golden-ratio and sqrt(3)-1 Weyl constants
    k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// the 16-bit draw of element e (R-20)
uint32_t hqo_draw16(uint32_t seed, uint32_t iteration, int64_t e) {
  uint64_t block = (uint64_t)e >> 3;
  uint32_t counter[4] = {(uint32_t)block, (uint32_t)(block >> 32), iteration, 0u};
  uint32_t key[2] = {seed, 0u};
  uint32_t w[4];
  hqo_philox4x32_10(counter, key, w);
  uint32_t word = w[((uint32_t)e & 7u) >> 1];
  return (e & 1) ? (word >> 16) : (word & 0xFFFFu);
}

static inline int32_t floor_to_i32(float t) {   // floor, then to int32 with saturation; NaN -> 0
  if (t != t) return 0;
  float f = std::floor(t);
  if (f >= 2147483648.0f) return std::numeric_limits<int32_t>::max();
  if (f <= -2147483648.0f) return std::numeric_limits<int32_t>::min();
  return (int32_t)f;
}

static inline int8_t quantize_real_sr(float y, const hqo_range* q, uint32_t seed, uint32_t iteration, int64_t e) {
  float u = y * q->inv_scale;
  float r = (float)hqo_draw16(seed, iteration, e) * (1.0f / 65536.0f);
  float t = u + r;
  return (int8_t)clamp_i64((int64_t)floor_to_i32(t) + q->zero_point, -128, 127);
}

// static quantization with stochastic rounding; element i of `acc` has linear index first + i
void hqo_quantize_sr(const int32_t* acc, int64_t count, float s_acc, const hqo_range* q, uint32_t seed, uint32_t iteration, int64_t first,
                     int8_t* out) {
  for (int64_t i = 0; i < count; ++i) out[i] = quantize_real_sr((float)acc[i] * s_acc, q, seed, iteration, first + i);
}

// ------------------------------------------------------------------------------------
// Saturation statistic (Sec. 4: besides min and max the statistic may be "the saturation ratio", the proportion
// of values that lie outside the quantization grid).  The final text of the paper gives no formula; the reading taken
// (R-22) is "clipped by the quantization operation": an output is counted when its rounded grid coordinate plus the zero
// point falls outside the 2^8 levels, i.e. when the clamp of O4 changes it:
//   c = rint(u) + z   (stochastic rounding: floor(fl(u + r)) + z),   below: c < -128,   above: c > 127,
// with u = fl(fl(float(acc) * s_acc) * inv_scale) as in O4.  Counts, not the ratio: the caller divides by the element
// count.  sr = 0: round half to even; sr = 1: stochastic rounding with (seed, iteration), element i having index first + i.
// ------------------------------------------------------------------------------------
void hqo_saturation(const int32_t* acc, int64_t count, float s_acc, const hqo_range* q, int sr, uint32_t seed, uint32_t iteration, int64_t first,
                    int64_t* below, int64_t* above) {
  int64_t b = 0, a = 0;
  for (int64_t i = 0; i < count; ++i) {
    float y = (float)acc[i] * s_acc;
    float u = y * q->inv_scale;
    int64_t c;
    if (sr) {
      float r = (float)hqo_draw16(seed, iteration, first + i) * (1.0f / 65536.0f);
      float t = u + r;
      c = (int64_t)floor_to_i32(t) + q->zero_point;
    } else {
      c = (int64_t)round_half_even_to_i32(u) + q->zero_point;
    }
    if (c < -128) ++b;
    if (c > 127) ++a;
  }
  *below = b;
  *above = a;
}

// dynamic path with stochastic rounding: as hqo_dynamic; the draws use the iteration count before this call
void hqo_dynamic_sr(const int32_t* acc, int64_t count, float s_acc, hqo_range* q, uint32_t seed, float* yf, int8_t* out) {
  for (int64_t i = 0; i < count; ++i) yf[i] = (float)acc[i] * s_acc;
  float lo = std::numeric_limits<float>::infinity(), hi = -lo;
  for (int64_t i = 0; i < count; ++i) {
    if (yf[i] < lo) lo = yf[i];
    if (yf[i] > hi) hi = yf[i];
  }
  if (count == 0) return;
  const uint32_t iteration = q->step;
  q->q_min = lo;
  q->q_max = hi;
  q->step += 1;
  hqo_derive(q);
  for (int64_t i = 0; i < count; ++i) out[i] = quantize_real_sr(yf[i], q, seed, iteration, i);
}

// ------------------------------------------------------------------------------------
// Running min-max (Sec. 4.1, last sentences): Eq. 2-3 with the statistics of the CURRENT tensor
// G^t in place of G^{t-1}: the range that quantizes tensor t is (1-eta) * minmax(G^t) +
// eta * q^{t-1}.  It is a dynamic method (the tensor's min/max must be known before it can be
// quantized), so it runs on the dynamic path; eta = 0 is current min-max (Eq. 1); t = 0 takes
// the min/max of the first tensor.  Same binary32 op order as hqo_range_update.
// ------------------------------------------------------------------------------------
void hqo_dynamic_running(const int32_t* acc, int64_t count, float s_acc, hqo_range* q, float eta, float* yf, int8_t* out) {
  for (int64_t i = 0; i < count; ++i) yf[i] = (float)acc[i] * s_acc;
  float lo = std::numeric_limits<float>::infinity(), hi = -lo;
  for (int64_t i = 0; i < count; ++i) {
    if (yf[i] < lo) lo = yf[i];
    if (yf[i] > hi) hi = yf[i];
  }
  if (count == 0) return;
  if (q->step == 0 || eta == 0.0f) {
    q->q_min = lo;
    q->q_max = hi;
  } else {
    float one_minus_eta = 1.0f - eta;
    float a_lo = one_minus_eta * lo, b_lo = eta * q->q_min;
    float a_hi = one_minus_eta * hi, b_hi = eta * q->q_max;
    q->q_min = a_lo + b_lo;
    q->q_max = a_hi + b_hi;
  }
  q->step += 1;
  hqo_derive(q);
  for (int64_t i = 0; i < count; ++i) out[i] = quantize_real(yf[i], q);
}

// s_acc = fl(s_x * s_w): scale of one accumulator unit in real terms
float hqo_acc_scale(float s_x, float s_w) { return s_x * s_w; }

// dequantized value of a code, s * (q - z) (for the grid-invariant tests)
float hqo_dequant(int8_t code, const hqo_range* q) { return q->scale * (float)((int)code - q->zero_point); }

}  // extern "C"
