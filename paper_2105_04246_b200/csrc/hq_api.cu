// C ABI of libhq: argument validation, launch planning, TMA descriptor encoding.
// No arithmetic of the method lives here; every step runs in the kernels of hq_gemm.cu / hq_aux.cu.
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdarg.h>
#include <stddef.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <functional>
#include <new>
#include <string>
#include <vector>

#include "hq.h"
#include "hq_internal.h"

using namespace hq;

namespace {

hq_status fail(hq_ctx* ctx, hq_status s, const char* fmt, ...) {
  if (ctx) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(ctx->err, sizeof(ctx->err), fmt, ap);
    va_end(ap);
  }
  return s;
}

#define HQ_CUDA(ctx, expr)                                                                                   \
  do {                                                                                                       \
    cudaError_t e__ = (expr);                                                                                \
    if (e__ != cudaSuccess) return fail(ctx, HQ_ERR_CUDA, "%s failed: %s", #expr, cudaGetErrorString(e__)); \
  } while (0)

// Every launching entry point runs on the context's device: with another device current the kernels would be launched
// there, against pointers that device may not even map.  A host-side query, no launch.
hq_status check_device(hq_ctx* ctx) {
  int cur = -1;
  HQ_CUDA(ctx, cudaGetDevice(&cur));
  if (cur != ctx->device) return fail(ctx, HQ_ERR_INVALID_ARG, "device %d must be current (device %d is)", ctx->device, cur);
  return HQ_OK;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
inline int round_up(int a, int b) { return ceil_div(a, b) * b; }

int out_dim(int in, int pad, int k, int stride) { return (in + 2 * pad - k) / stride + 1; }

hq_status check_desc(hq_ctx* ctx, const hq_conv_desc* d) {
  if (!d) return fail(ctx, HQ_ERR_INVALID_ARG, "conv descriptor is null");
  if (d->N <= 0 || d->H <= 0 || d->W <= 0 || d->C <= 0 || d->K <= 0 || d->R <= 0 || d->S <= 0 || d->stride_h <= 0 || d->stride_w <= 0 ||
      d->pad_h < 0 || d->pad_w < 0)
    return fail(ctx, HQ_ERR_INVALID_ARG, "conv descriptor has a non-positive size");
  if (d->groups != 1 && !(d->groups == d->C && d->K == d->C)) return fail(ctx, HQ_ERR_UNSUPPORTED, "groups must be 1 or C (depthwise, K == C)");
  if (d->H + 2 * d->pad_h < d->R || d->W + 2 * d->pad_w < d->S) return fail(ctx, HQ_ERR_INVALID_ARG, "filter larger than padded input");
  if (d->R > 7 || d->S > 7) return fail(ctx, HQ_ERR_UNSUPPORTED, "filters larger than 7x7 are not supported");
  if (d->pad_h >= d->R || d->pad_w >= d->S) return fail(ctx, HQ_ERR_UNSUPPORTED, "padding must be smaller than the filter");
  return HQ_OK;
}

bool same_desc(const hq_conv_desc& a, const hq_conv_desc& b) {
  return a.N == b.N && a.H == b.H && a.W == b.W && a.C == b.C && a.K == b.K && a.R == b.R && a.S == b.S && a.stride_h == b.stride_h &&
         a.stride_w == b.stride_w && a.pad_h == b.pad_h && a.pad_w == b.pad_w && a.groups == b.groups;
}

// border classes of one tile-space axis: which taps of `d` fall inside [0, a_dim) at position i
void border_classes(int T, int in_mul, const TapVec& d, int a_dim, std::vector<uint8_t>& cls, MaskVec& masks) {
  cls.assign(T, 0);
  masks.clear();
  for (int i = 0; i < T; ++i) {
    uint32_t m = 0;
    for (size_t t = 0; t < d.size(); ++t) {
      const int x = i * in_mul + d[t];
      if (x >= 0 && x < a_dim) m |= 1u << t;
    }
    size_t k = 0;
    while (k < masks.size() && masks[k] != m) ++k;
    if (k == masks.size()) masks.push_back(m);
    cls[i] = (uint8_t)k;
  }
  if (masks.empty()) masks.push_back(0);
}

// 128 = Nt*Ht*Wt with powers of two; the split that covers the tile space with least waste
void pick_tile(int n_img, int TH, int TW, int in_mul_h, int in_mul_w, int& Nt, int& Ht, int& Wt) {
  double best = -1.0;
  for (int a = 7; a >= 0; --a)
    for (int b = 7 - a; b >= 0; --b) {
      const int wt = 1 << a, ht = 1 << b, nt = kTileM / (wt * ht);
      if (wt * in_mul_w > 256 || ht * in_mul_h > 256) continue;
      const double covered = (double)round_up(TW, wt) * round_up(TH, ht) * round_up(n_img, nt);
      const double util = (double)TW * TH * n_img / covered;
      if (util > best + 1e-12) {
        best = util;
        Nt = nt;
        Ht = ht;
        Wt = wt;
      }
    }
}

FastDiv make_fastdiv(int d) {
  FastDiv f{1u, 0u};
  if (d <= 1) return f;
  uint32_t l = 0;
  while ((1ull << l) < (uint64_t)d) ++l;
  f.l = l;
  f.m = (uint32_t)(((1ull << 32) * ((1ull << l) - (uint64_t)d)) / (uint64_t)d + 1ull);
  return f;
}

struct SubSpec {            // geometry of one launch, before tiling
  int n_img, TH, TW;
  int in_mul_h, in_mul_w;
  TapVec dh, dw;            // tap offsets per axis (taps = product, row-major)
  int a_H, a_W;             // image size of operand A (for border classes)
  int Cin;                  // reduction length per tap
  int Nout;
  int out_H, out_W, os_h, os_w, oa_h, oa_w;
  int64_t ldY;
  bool flat;
  bool whole_gpu = true;    // false: the launch shares the SMs with other launches of the same call
  int slices = 0;           // flat GEMM whose reduction is cut into `slices` pieces of `slice_len` bytes: n_img == slices, image n
  int slice_len = 0;        // of the tile space multiplies reduction range [n * slice_len, (n + 1) * slice_len) into its own output slab
};

// fills everything in sub.p that does not depend on per-call pointers, for a given number of column tiles
// (ncol_req = 0: as few as the MMA allows) and a given answer to "CTA pairs?" (pair_req: 0 no, 1 where the layer allows)
hq_status plan_sub_fixed(hq_ctx* ctx, const SubSpec& sp, hq_sub_problem& sub, std::vector<uint8_t>& rowcls, std::vector<uint8_t>& colcls,
                         MaskVec& rowmasks, MaskVec& colmasks, int ncol_req, int pair_req) {
  GemmParams& p = sub.p;
  p.n_img = sp.n_img;
  p.TH = sp.TH;
  p.TW = sp.TW;
  p.in_mul_h = sp.in_mul_h;
  p.in_mul_w = sp.in_mul_w;
  auto tile_shape = [&]() {
    pick_tile(sp.n_img, sp.TH, sp.TW, sp.in_mul_h, sp.in_mul_w, p.Nt, p.Ht, p.Wt);
    if (sp.slices > 0) {   // one slice per tile: rows only
      p.Nt = 1;
      p.Ht = 1;
      p.Wt = kTileM;
    }
  };
  tile_shape();
  p.b_slice = sp.slices > 0 ? sp.slice_len : 0;
  p.tiles_n = ceil_div(sp.n_img, p.Nt);
  p.tiles_h = ceil_div(sp.TH, p.Ht);
  p.tiles_w = ceil_div(sp.TW, p.Wt);
  p.ntaps = (int)(sp.dh.size() * sp.dw.size());
  if (p.ntaps > kMaxTaps) return fail(ctx, HQ_ERR_UNSUPPORTED, "too many filter taps");
  for (size_t a = 0; a < sp.dh.size(); ++a)
    for (size_t b = 0; b < sp.dw.size(); ++b) {
      p.tap_dh[a * sp.dw.size() + b] = (int8_t)sp.dh[a];
      p.tap_dw[a * sp.dw.size() + b] = (int8_t)sp.dw[b];
    }
  if (sp.Cin % 16 != 0) return fail(ctx, HQ_ERR_UNSUPPORTED, "reduction length per tap (%d) must be a multiple of 16", sp.Cin);
  p.BK = (sp.Cin % 128 == 0) ? 128 : 64;
  // a single-tap layer moves few bytes per copy-engine request: prefer 128-byte rows when that takes fewer copies
  // (the padded reduction steps meet zero weights and zero-filled operand bytes)
  if (p.ntaps == 1 && ceil_div(sp.Cin, 128) < ceil_div(sp.Cin, 64)) p.BK = 128;
  p.swizzle64 = p.BK == 64;
  p.Cpad = round_up(sp.Cin, p.BK);
  p.chunks_per_tap = p.Cpad / p.BK;
  p.Nout = sp.Nout;
  p.rt_fold = 1;
  p.rt_cols = sp.Nout;
  // column tiles: as wide as the MMA allows, except for very short reductions, where the epilogue is the bottleneck and
  // narrower tiles give it four or more accumulator buffers to work on
  const int ncol = std::max(ncol_req, ceil_div(sp.Nout, p.ntaps * p.Cpad <= 128 ? 128 : 256));
  p.BN = round_up(ceil_div(sp.Nout, ncol), 16);
  p.tiles_col = ceil_div(sp.Nout, p.BN);
  const int64_t nt = (int64_t)p.tiles_n * p.tiles_h * p.tiles_w * p.tiles_col;
  if (nt > INT32_MAX) return fail(ctx, HQ_ERR_UNSUPPORTED, "too many tiles");
  p.num_tiles = (int)nt;
  p.out_H = sp.out_H;
  p.out_W = sp.out_W;
  p.os_h = sp.os_h;
  p.os_w = sp.os_w;
  p.oa_h = sp.oa_h;
  p.oa_w = sp.oa_w;
  p.ldY = sp.ldY;
  p.corr_ld = p.tiles_col * p.BN;
  // instruction descriptor: D = s32, A = B = signed 8-bit, both K-major, N = BN, M = 128
  p.idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.BN >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
  {
    uint32_t s = 32;
    while ((int)s < p.BN) s <<= 1;
    p.tmem_buf_stride = s;
    p.tmem_bufs = (int)std::min<uint32_t>(8, 512 / s);
    p.tmem_bufs_log2 = p.tmem_bufs == 8 ? 3 : (p.tmem_bufs == 4 ? 2 : 1);
    p.tmem_cols = (uint32_t)p.tmem_bufs * s;
  }
  // border classes first: the size of the correction table decides how much shared memory the rings get
  if (sp.flat) {
    rowcls.clear();
    colcls.clear();
    rowmasks.assign(1, 1u);
    colmasks.assign(1, 1u);
  } else {
    border_classes(sp.TH, sp.in_mul_h, sp.dh, sp.a_H, rowcls, rowmasks);
    border_classes(sp.TW, sp.in_mul_w, sp.dw, sp.a_W, colcls, colmasks);
    if (rowmasks.size() > 16 || colmasks.size() > 16) return fail(ctx, HQ_ERR_UNSUPPORTED, "too many border classes");
  }
  p.ncolcls = (int)colmasks.size();
  p.zc_elems = (int)(rowmasks.size() * colmasks.size()) * p.corr_ld;
  p.zc_in_smem = ((uint32_t)p.zc_elems * 4u <= kMaxZcBytes && p.ntaps > 0) ? 1 : 0;
  const uint32_t zc_bytes = p.zc_in_smem ? (((uint32_t)p.zc_elems * 4u + 1023u) & ~1023u) : 0u;
  const uint32_t ring_budget = kSmemBudget - zc_bytes;
  p.zc_offset = ring_budget;
  // ---- operand staging: resident input rows (kModeHalo) where the tile space is stride-1, else one box per tap ----
  // With CTA pairs (b_rows = BN / 2) each CTA stages half of the rows of B; resident weights are never paired.
  auto plan_staging = [&](bool pair) -> hq_status {
  p.mode = kModeTap;
  p.b_resident = 0;
  const uint32_t full_stage_b = (uint32_t)p.BN * p.BK;
  p.stage_bytes_b = pair ? full_stage_b / 2 : full_stage_b;
  bool halo = !sp.flat && sp.in_mul_h == 1 && sp.in_mul_w == 1 && p.ntaps >= 2 && ctx->force_mode != kModeTap;
  if (halo) {
    const int dh_min = *std::min_element(sp.dh.begin(), sp.dh.end()), dh_max = *std::max_element(sp.dh.begin(), sp.dh.end());
    const int dw_min = *std::min_element(sp.dw.begin(), sp.dw.end()), dw_max = *std::max_element(sp.dw.begin(), sp.dw.end());
    const int dh_span = dh_max - dh_min, dw_span = dw_max - dw_min;
    const int P = sp.TW + dw_span;
    const int L = sp.TH * P;
    const int tiles_per_img = ceil_div(L, kTileM);
    int NR = 0;
    for (int lt = 0; lt < tiles_per_img; ++lt) NR = std::max(NR, ((lt * kTileM) % P + kTileM - 1 + dh_span * P + dw_span) / P + 1);
    const uint32_t box = (uint32_t)p.BK * P * NR;
    const uint32_t stride = (box + 1023u) & ~1023u;
    const double util = (double)sp.TH * sp.TW / ((double)tiles_per_img * kTileM);
    const int kiters = p.ntaps * p.chunks_per_tap;
    halo = (int)sp.dh.size() == dh_span + 1 && (int)sp.dw.size() == dw_span + 1 && P <= 256 && NR <= 256 &&
           (util >= 0.6 || ctx->force_mode == kModeHalo);
    int stages_a = 0, stages_b = 0, resident = 0;
    if (halo) {
      if (kiters <= kMaxStagesB && p.tiles_col == 1 && (uint64_t)kiters * full_stage_b + 2ull * stride <= ring_budget) {
        resident = 1;
        stages_b = kiters;
        stages_a = (int)std::min<uint64_t>(kMaxStagesA, (ring_budget - (uint64_t)kiters * full_stage_b) / stride);
      } else {
        stages_a = 2;
        while (stages_a < 4 && (uint64_t)(stages_a + 1) * stride + 4ull * p.stage_bytes_b <= ring_budget) ++stages_a;
        if ((uint64_t)stages_a * stride < ring_budget)
          stages_b = (int)std::min<uint64_t>(pair ? 12 : 8, (ring_budget - (uint64_t)stages_a * stride) / p.stage_bytes_b);
        if (stages_b < 2) halo = false;
      }
    }
    if (halo) {
      p.mode = kModeHalo;
      p.P = P;
      p.L = L;
      p.NR = NR;
      p.tiles_per_img = tiles_per_img;
      p.dh_min = dh_min;
      p.dw_min = dw_min;
      p.patch_box_bytes = box;
      p.patch_chunk_stride = stride;
      p.stage_bytes_a = stride;
      p.stages_a = stages_a;
      p.stages_b = stages_b;
      p.b_resident = resident;
      p.Nt = 1;
      p.Ht = 1;
      p.Wt = kTileM;
      p.num_tiles = sp.n_img * tiles_per_img * p.tiles_col;
      p.num_pair_tiles = ceil_div(sp.n_img, 2) * tiles_per_img * p.tiles_col;
      p.producer_lanes = 1;
    }
  }
  if (p.mode == kModeTap) {
    tile_shape();
    p.num_tiles = (int)nt;
    p.num_pair_tiles = ceil_div(p.tiles_n * p.tiles_h * p.tiles_w, 2) * p.tiles_col;
    p.stage_bytes_a = (uint32_t)kTileM * p.BK;
    // a small weight matrix stays in shared memory for the whole kernel; the ring then carries operand A only
    const int kiters = p.ntaps * p.chunks_per_tap;
    const uint64_t b_all = (uint64_t)p.tiles_col * kiters * full_stage_b;
    if (kiters > 0 && sp.slices == 0 && p.tiles_col * kiters <= kMaxStagesB && b_all <= 64u * 1024u &&
        b_all + 6ull * p.stage_bytes_a <= ring_budget) {
      p.b_resident = 1;
      p.stages_b = p.tiles_col * kiters;
      p.stages_a = (int)std::min<uint64_t>(kMaxStagesA, (ring_budget - b_all) / p.stage_bytes_a);
    } else {
      p.stages_a = (int)std::min<uint32_t>(kMaxStagesA, ring_budget / (p.stage_bytes_a + p.stage_bytes_b));
      p.stages_b = 0;
    }
    if (p.stages_a < 2) return fail(ctx, HQ_ERR_UNSUPPORTED, "operand tiles do not fit in shared memory");
    p.producer_lanes = std::min(4, p.stages_a);
  }
  return HQ_OK;
  };
  // CTA pairs pay where the weights stream through shared memory and the tile is wide: each CTA then copies and reads
  // half of the rows of B per 128 rows of output.  Never for flat (1x1 / linear) layers, which the epilogue bounds.
  bool want_pair = pair_req != 0 && !sp.flat && p.ntaps >= 1 && p.tiles_n * p.tiles_h * p.tiles_w >= 2;
  {
    hq_status pst = plan_staging(want_pair);
    if (pst != HQ_OK) return pst;
    if (want_pair && (p.b_resident || (p.mode == kModeHalo && sp.n_img < 2))) {
      want_pair = false;
      pst = plan_staging(false);
      if (pst != HQ_OK) return pst;
    }
  }
  p.pair = want_pair ? 1 : 0;
  if (p.pair) p.idesc = (p.idesc & ~(0x1Fu << 24)) | ((uint32_t)(2 * kTileM >> 4) << 24);   // M = 256 across the pair
  sub.smem_bytes = kSmemBudget + 1024;
  sub.a_flat = sp.flat;
  sub.a_stride_h = sp.in_mul_h;
  sub.a_stride_w = sp.in_mul_w;
  p.status = ctx->d_status;
  {
    // Two MMA issuer warps alternate tiles.  An issuer that waits for ring iteration `it` must find iteration
    // `it - stages` already delivered, or the phase parity of an older delivery would satisfy its wait; that holds
    // when the issuer's own previous tile covers it: two tiles' worth of stages must fit in the ring.
    const int kiters = p.ntaps * p.chunks_per_tap;
    const int a_per_tile = p.mode == kModeHalo ? p.chunks_per_tap : kiters;
    const int b_per_tile = (p.mode == kModeHalo && !p.b_resident) ? kiters : 0;
    const bool rings_ok = 2 * a_per_tile <= p.stages_a && (b_per_tile == 0 || 2 * b_per_tile <= p.stages_b);
    p.mma_issuers = (rings_ok && kiters > 0 && p.num_tiles >= 2 * ctx->num_sms && !p.pair) ? 2 : 1;
    // narrow tiles (64 columns or fewer) keep the tensor core busy for so short a time per tile that a third issuer pays;
    // the weight producer's warp takes that part once resident weights are on their way
    // Three issuers share the accumulator buffers unevenly (three does not divide their number), and an issuer's wait for
    // a drained buffer is only sound when the buffer's previous tile has already been issued, possibly by another issuer.
    // The kernel gets that from the operand ring (see its issuer loop), provided the ring holds no more than as many tiles
    // as there are buffers: the ring is shortened to that where needed.
    const int ring3 = std::min(p.stages_a, p.tmem_bufs * a_per_tile);
    p.a_producers = 1;
    const bool two_prod_ok = p.mode == kModeTap && p.b_resident && !p.pair && p.b_group_tiles == 0 && rings_ok && kiters > 0;
    if (p.mma_issuers == 2 && ctx->max_issuers >= 3 && p.b_resident && p.BN <= 64 && 3 * a_per_tile <= ring3 && ring3 >= 6 &&
        p.num_tiles >= 3 * ctx->num_sms && p.tmem_bufs >= 4) {
      // Such layers (1x1 with few channels on either side) were measured to wait for operand A: one warp gets a copy
      // under way about every 0.5-0.7 us whatever its size.  Up to 192 input channels a second producer (the weight
      // producer's warp, with two issuers) beats a third issuer: 64 -> 32 channels 31 -> 25 us, 144 -> 24 44.8 -> 38.6 us,
      // 192 -> 32 41.7 -> 36.4 us per 800k pixels; at 256 input channels the layer is close to the HBM bound either way.
      if (two_prod_ok && ctx->a_producers != 1 && sp.Cin <= 192) {
        p.a_producers = 2;
      } else {
        p.mma_issuers = 3;
        p.stages_a = ring3;
        if (p.mode == kModeTap) p.producer_lanes = std::min(p.producer_lanes, p.stages_a);
      }
    }
    if (two_prod_ok && ctx->a_producers == 2 && p.mma_issuers <= 2) p.a_producers = 2;
    p.mma_issuers = std::min(p.mma_issuers, ctx->max_issuers);
    // Several tiles per CTA: as many epilogue groups as there are accumulator buffers (at most four), so that a warp
    // pays its per-tile set-up once per several column passes; one or two tiles per CTA: all warps on every tile (the
    // epilogue of the last tile, which nothing overlaps, is then shortest).  Measured on the ResNet-18 shapes.
    const int tiles_per_cta = ceil_div(p.num_tiles, ctx->num_sms);
    p.epi_groups_log2 = tiles_per_cta >= 3 ? std::min(2, p.tmem_bufs_log2) : 0;
    if (ctx->force_epi_groups >= 0) p.epi_groups_log2 = std::min(ctx->force_epi_groups, p.tmem_bufs_log2);
  }
  p.fd_tiles_col = make_fastdiv(p.tiles_col);
  p.fd_tiles_per_img = make_fastdiv(p.mode == kModeHalo ? p.tiles_per_img : 1);
  p.fd_tiles_w = make_fastdiv(p.tiles_w);
  p.fd_tiles_h = make_fastdiv(p.tiles_h);
  p.fd_P = make_fastdiv(p.mode == kModeHalo ? p.P : 1);
  return HQ_OK;
}

// Chooses the number of column tiles and single CTAs or CTA pairs, by rules taken from measurements on B200:
//  * CTA pairs pay where the input rows are resident and the weights stream through shared memory (each SM then copies
//    half of the weight rows per 128 rows of output); with one copy per filter tap they do not, and on strided or
//    single-tap layers they cost time;
//  * narrower column tiles only pay where the widest ones leave SMs without any tile (few row tiles: 7x7 images): then
//    as many column tiles as still fit in one round, none narrower than 64 columns.  Everywhere else splitting the
//    columns multiplies the traffic of operand A and is much slower.
hq_status plan_sub(hq_ctx* ctx, const SubSpec& sp, hq_sub_problem& sub, std::vector<uint8_t>& rowcls, std::vector<uint8_t>& colcls,
                   MaskVec& rowmasks, MaskVec& colmasks) {
  if (sp.flat) return plan_sub_fixed(ctx, sp, sub, rowcls, colcls, rowmasks, colmasks, std::max(0, ctx->force_cols), 0);
  int ncol = std::max(0, ctx->force_cols);
  int pair = ctx->force_pair;
  if (ctx->force_cols < 0 || ctx->force_pair < 0) {
    hq_sub_problem trial = sub;
    std::vector<uint8_t> rc, cc;
    MaskVec rm, cm;
    hq_status st = plan_sub_fixed(ctx, sp, trial, rc, cc, rm, cm, ncol, 0);
    if (st != HQ_OK) return st;
    const GemmParams& t = trial.p;
    if (ctx->force_pair < 0) pair = (t.mode == kModeHalo && !t.b_resident && sp.Nout >= 128) ? 1 : 0;
    // Small images fill the 128-row tiles of the resident-row numbering badly (14x14: 77 %).  With one copy per filter
    // tap the tiles are full; where that saves a fifth of the rounds or more, pairs with one copy per tap are faster
    // (each SM then still copies only half of the weight rows).
    if (ctx->force_pair < 0 && ctx->force_mode < 0 && pair == 1) {
      hq_sub_problem halo_trial = sub, tap_trial = sub;
      const int pairs = std::max(1, ctx->num_sms / 2);
      if (plan_sub_fixed(ctx, sp, halo_trial, rc, cc, rm, cm, ncol, 1) == HQ_OK && halo_trial.p.pair) {
        ctx->force_mode = kModeTap;
        const hq_status ts = plan_sub_fixed(ctx, sp, tap_trial, rc, cc, rm, cm, ncol, 1);
        ctx->force_mode = -1;
        if (ts == HQ_OK && tap_trial.p.pair &&
            5 * ceil_div(tap_trial.p.num_pair_tiles, pairs) <= 4 * ceil_div(halo_trial.p.num_pair_tiles, pairs)) {
          ctx->force_mode = kModeTap;
          const hq_status fs = plan_sub_fixed(ctx, sp, sub, rowcls, colcls, rowmasks, colmasks, ncol, 1);
          ctx->force_mode = -1;
          return fs;
        }
      }
    }
    if (ctx->force_cols < 0 && sp.whole_gpu && pair == 0 && t.ntaps > 0 && t.num_tiles < ctx->num_sms) {
      const int row_tiles = t.num_tiles / t.tiles_col;
      for (int k = t.tiles_col + 1; k <= 16 && row_tiles * k <= ctx->num_sms && ceil_div(sp.Nout, k) >= 64; ++k) ncol = k;
    }
  }
  return plan_sub_fixed(ctx, sp, sub, rowcls, colcls, rowmasks, colmasks, ncol, pair);
}

hq_status encode_map(hq_ctx* ctx, CUtensorMap* m, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                     const uint32_t* box, const uint32_t* estr, bool sw64, bool weights) {
  CUresult r = ctx->encode(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, (cuuint32_t)rank, const_cast<void*>(base), dims, strides_bytes, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, sw64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                           weights ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(ctx, HQ_ERR_CUDA, "tensor map encoding failed (CUresult %d)", (int)r);
  return HQ_OK;
}

hq_status encode_b(hq_ctx* ctx, const hq_sub_problem& sub, const int8_t* wmat, int64_t row_bytes, CUtensorMap* m) {
  const GemmParams& p = sub.p;
  uint64_t dims[2] = {(uint64_t)row_bytes, (uint64_t)p.Nout};
  uint64_t strides[1] = {(uint64_t)row_bytes};
  uint32_t box[2] = {(uint32_t)p.BK, (uint32_t)(p.pair ? p.BN / 2 : p.BN)};   // a pair's CTAs fetch half of the rows each
  uint32_t es[2] = {1, 1};
  return encode_map(ctx, m, wmat, 2, dims, strides, box, es, p.swizzle64, true);
}

// operand A: flat [rows][C] view, or NHWC image with one box per tile (traversal strides for strided layers)
hq_status encode_a(hq_ctx* ctx, const hq_sub_problem& sub, const int8_t* base, int C, int W, int H, int N, CUtensorMap* m, int pitch = 0) {
  const GemmParams& p = sub.p;
  if (pitch == 0) pitch = C;   // bytes from one pixel to the next (a channel slice of a wider tensor has pitch > C)
  uint64_t dims[4] = {(uint64_t)C, (uint64_t)W, (uint64_t)H, (uint64_t)N};
  uint64_t strides[3] = {(uint64_t)pitch, (uint64_t)pitch * W, (uint64_t)pitch * W * H};
  uint32_t box[4] = {(uint32_t)p.BK, (uint32_t)(p.Wt * sub.a_stride_w), (uint32_t)(p.Ht * sub.a_stride_h), (uint32_t)p.Nt};
  uint32_t es[4] = {1, (uint32_t)sub.a_stride_w, (uint32_t)sub.a_stride_h, 1};
  if (p.mode == kModeHalo) {  // NR padded rows of P pixels of one image
    box[1] = (uint32_t)p.P;
    box[2] = (uint32_t)p.NR;
    box[3] = 1;
  }
  return encode_map(ctx, m, base, 4, dims, strides, box, es, p.swizzle64, false);
}

hq_status dev_alloc(hq_ctx* ctx, hq_prepared_weights* pw, void** p, size_t bytes) {
  HQ_CUDA(ctx, cudaMalloc(p, bytes ? bytes : 16));
  pw->allocs.push_back(*p);
  return HQ_OK;
}

hq_status upload(hq_ctx* ctx, hq_prepared_weights* pw, const std::vector<uint8_t>& v, uint8_t** out, cudaStream_t s) {
  if (v.empty()) {
    *out = nullptr;
    return HQ_OK;
  }
  void* d = nullptr;
  hq_status st = dev_alloc(ctx, pw, &d, v.size());
  if (st != HQ_OK) return st;
  HQ_CUDA(ctx, cudaMemcpyAsync(d, v.data(), v.size(), cudaMemcpyHostToDevice, s));
  HQ_CUDA(ctx, cudaStreamSynchronize(s));  // v is a temporary on the host
  *out = (uint8_t*)d;
  return HQ_OK;
}

// builds weight matrix, correction table and class maps of one sub-problem; `custom` replaces the standard
// [Nout][tap][Cpad] weight layout (repacked operands), the correction table is always summed from the matrix
using WeightPrep = std::function<cudaError_t(hq_sub_problem&)>;
hq_status build_sub(hq_ctx* ctx, hq_prepared_weights* pw, cudaStream_t s, const SubSpec& sp, const hq_conv_desc& d, const int8_t* W,
                    const std::vector<int>& tap_r, const std::vector<int>& tap_s, bool transposed, int gfold,
                    const WeightPrep* custom = nullptr) {
  pw->subs.emplace_back();
  hq_sub_problem& sub = pw->subs.back();
  sub.gfold = gfold;
  std::vector<uint8_t> rowcls, colcls;
  MaskVec rowmasks, colmasks;
  hq_status st = plan_sub(ctx, sp, sub, rowcls, colcls, rowmasks, colmasks);
  if (st != HQ_OK) return st;
  GemmParams& p = sub.p;
  if (p.ntaps == 0) return HQ_OK;  // nothing to multiply: the epilogue stores the code of real zero
  const size_t wbytes = (size_t)p.Nout * p.ntaps * p.Cpad;
  st = dev_alloc(ctx, pw, (void**)&sub.wmat, wbytes);
  if (st != HQ_OK) return st;
  st = dev_alloc(ctx, pw, (void**)&sub.corr, (size_t)rowmasks.size() * colmasks.size() * p.corr_ld * sizeof(int32_t));
  if (st != HQ_OK) return st;
  HQ_CUDA(ctx, cudaMemsetAsync(sub.corr, 0, (size_t)rowmasks.size() * colmasks.size() * p.corr_ld * sizeof(int32_t), s));
  if (custom != nullptr) {
    HQ_CUDA(ctx, (*custom)(sub));
  } else {
    int8_t tr[kMaxTaps], ts[kMaxTaps];
    for (int t = 0; t < p.ntaps; ++t) {
      tr[t] = (int8_t)tap_r[t / (int)sp.dw.size()];
      ts[t] = (int8_t)tap_s[t % (int)sp.dw.size()];
    }
    HQ_CUDA(ctx, launch_prep_weights(W, sub.wmat, p.Nout, p.ntaps, p.Cpad, d.K, d.R, d.S, d.C, tr, ts, transposed ? 1 : 0, gfold, s));
  }
  HQ_CUDA(ctx, launch_corr(sub.wmat, sub.corr, p.Nout, p.ntaps, p.Cpad, (int)sp.dh.size(), (int)sp.dw.size(), rowmasks.data(),
                           (int)rowmasks.size(), colmasks.data(), (int)colmasks.size(), p.corr_ld, s));
  ctx->launches += 2;
  st = upload(ctx, pw, rowcls, &sub.rowcls, s);
  if (st != HQ_OK) return st;
  st = upload(ctx, pw, colcls, &sub.colcls, s);
  if (st != HQ_OK) return st;
  p.corr = sub.corr;
  p.rowcls = sub.rowcls;
  p.colcls = sub.colcls;
  p.cls_in_smem = (sub.rowcls && sub.colcls && p.TH <= 512 && p.TW <= 512) ? 1 : 0;
  return encode_b(ctx, sub, sub.wmat, (int64_t)p.ntaps * p.Cpad, &sub.tmap_b);
}

int fold_factor(int channels, int64_t pixels) {
  for (int g = 1; g <= 16; g *= 2)
    if ((g * channels) % 16 == 0 && pixels % g == 0) return g;
  return 0;
}

hq_status launch_sub(hq_ctx* ctx, cudaStream_t s, const hq_sub_problem& sub, const CUtensorMap& ta, const CUtensorMap& tb, const hq_range_state* xq,
                     const float* w_scale, const int32_t* bias, void* out, hq_range_state* yq, int out_mode, int max_ctas = 0,
                     bool weights_early = false, const int32_t* row_term = nullptr) {
  GemmParams p = sub.p;
  p.row_term = row_term;
  if (row_term != nullptr && sub.gfold > 1) {   // a GEMM row of a folded 1x1 layer holds gfold pixels side by side
    p.rt_fold = sub.gfold;
    p.rt_cols = p.Nout / sub.gfold;
  }
  p.out_col0 = sub.chan0;
  p.weights_early = weights_early ? 1 : 0;
  p.xq = xq;
  p.w_scale = w_scale;
  p.bias = bias;
  p.acc_bound = (float)p.ntaps * (float)p.Cpad * 255.0f * 128.0f;
  p.out = out;
  p.yq = yq;
  int grid = std::max(1, std::min(p.num_tiles, max_ctas > 0 ? max_ctas : ctx->num_sms));
  if (p.pair) {   // clusters of two: one pair per two SMs
    const int pairs = std::max(1, (max_ctas > 0 ? max_ctas : ctx->num_sms) / 2);
    grid = 2 * std::max(1, std::min(p.num_pair_tiles, pairs));
  }
  {
    const cudaError_t le = launch_gemm(p, ta, tb, out_mode, grid, sub.smem_bytes, s, ctx->overlap);
    if (le != cudaSuccess) {
      (void)cudaGetLastError();   // a rejected launch leaves no work behind; clear it so that later calls start clean
      return fail(ctx, HQ_ERR_CUDA, "layer kernel launch failed: %s (grid %d, pair %d, tiles %d, pair tiles %d, mode %d, BN %d)",
                  cudaGetErrorString(le), grid, p.pair, p.num_tiles, p.num_pair_tiles, p.mode, p.BN);
    }
  }
  ctx->launches += 1;
  ctx->pair_launches += p.pair ? 1 : 0;
  return HQ_OK;
}

hq_status run_conv(hq_ctx* ctx, cudaStream_t s, const hq_conv_desc* desc, hq_direction dir, const int8_t* in, const hq_range_state* inq,
                   const hq_prepared_weights* pw, const float* w_scale, void* out, hq_range_state* outq, int out_mode) {
  hq_status st = check_desc(ctx, desc);
  if (st != HQ_OK) return st;
  if (!in || !inq || !pw || !w_scale || !out || !outq) return fail(ctx, HQ_ERR_INVALID_ARG, "null pointer argument");
  if (!aligned16(in) || !aligned16(out) || !aligned16(inq) || !aligned16(outq))
    return fail(ctx, HQ_ERR_ALIGNMENT, "tensors and range states must be 16-byte aligned");
  if (pw->linear || pw->dir != dir || !same_desc(pw->desc, *desc)) return fail(ctx, HQ_ERR_INVALID_ARG, "prepared weights were built for another layer");
  if (pw->depthwise) {
    // the geometry the kernel runs (see hq_weights_prepare): for backward data the forward layer over the output gradient
    const hq_conv_desc* const caller_desc = desc;
    desc = &pw->dw_run;
    const int Ho = out_dim(desc->H, desc->pad_h, desc->R, desc->stride_h), Wo = out_dim(desc->W, desc->pad_w, desc->S, desc->stride_w);
    DwParams p{};
    p.N = desc->N; p.H = desc->H; p.W = desc->W; p.C = desc->C; p.Ho = Ho; p.Wo = Wo; p.R = desc->R; p.S = desc->S;
    p.stride_h = desc->stride_h; p.stride_w = desc->stride_w; p.pad_h = desc->pad_h; p.pad_w = desc->pad_w;
    p.x = in; p.w = pw->dw_w; p.corr = pw->dw_corr; p.rowcls = pw->dw_rowcls; p.colcls = pw->dw_colcls; p.ncolcls = pw->dw_ncolcls;
    p.xq = inq; p.w_scale = w_scale; p.yq = outq; p.out = out;
    p.status = ctx->d_status;
    p.w_zp = pw->w_zp;
    if (pw->dw_bwd_direct) {   // backward data by the definition (strided layers, asymmetric weights): the forward geometry, dY in p.x
      const hq_conv_desc* f = caller_desc;
      p.N = f->N; p.H = f->H; p.W = f->W; p.C = f->C; p.R = f->R; p.S = f->S;
      p.Ho = out_dim(f->H, f->pad_h, f->R, f->stride_h); p.Wo = out_dim(f->W, f->pad_w, f->S, f->stride_w);
      p.stride_h = f->stride_h; p.stride_w = f->stride_w; p.pad_h = f->pad_h; p.pad_w = f->pad_w;
      p.w = pw->dw_w_plain;
      HQ_CUDA(ctx, launch_depthwise_bwd(p, out_mode, ctx->num_sms, s));
      ctx->launches += 1;
      return HQ_OK;
    }
    // 3x3 stride 1 with at most 256 channels, transposing kernel: tiles of kDwColRows rows x up to 28 columns, one thread per
    // channel word and group of 4 columns (see hq_dw3x3.cu)
    if (desc->R == 3 && desc->S == 3 && desc->stride_h == 1 && desc->stride_w == 1 && desc->C <= 256 && desc->C % 16 == 0 &&
        (ctx->force_dw_tiled < 0 || ctx->force_dw_tiled == 2) && pw->w_zp == 0) {
      const int cwords = desc->C / 4;
      const int groups = std::min(std::min(round_up(Wo, 4) / 4, 7), kDwColMaxThreads / cwords);
      p.TR = kDwColRows;
      p.TWt = 4 * groups;
      p.tiles_h = ceil_div(Ho, p.TR);
      p.tiles_w = ceil_div(Wo, p.TWt);
      p.ncls = pw->dw_ncls;
      p.patch_bytes = (uint32_t)desc->C * (uint32_t)(p.TWt + 2) * (uint32_t)(p.TR + 2);
      p.patch_stride = (p.patch_bytes + 127u) & ~127u;
      const int64_t n_tiles = (int64_t)desc->N * p.tiles_h * p.tiles_w;
      const uint32_t smem = depthwise_col_smem_bytes(p);
      if (groups >= 1 && groups * cwords >= 64 && n_tiles <= INT32_MAX && smem <= 200u * 1024u) {
        CUtensorMap tm;
        uint64_t dims[4] = {(uint64_t)desc->C, (uint64_t)desc->W, (uint64_t)desc->H, (uint64_t)desc->N};
        uint64_t strides[3] = {(uint64_t)desc->C, (uint64_t)desc->C * desc->W, (uint64_t)desc->C * desc->W * desc->H};
        uint32_t box[4] = {(uint32_t)desc->C, (uint32_t)(p.TWt + 2), (uint32_t)(p.TR + 2), 1u};
        uint32_t es[4] = {1, 1, 1, 1};
        CUresult r = ctx->encode(&tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<int8_t*>(in), dims, strides, box, es,
                                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return fail(ctx, HQ_ERR_CUDA, "tensor map encoding failed (CUresult %d)", (int)r);
        // CTAs per SM: by registers (128 per thread, whole warps) and by shared memory (1 KB per CTA is the system's)
        const int warps = ceil_div(groups * cwords, 32);
        const int by_regs = 65536 / (warps * 32 * 128), by_smem = (int)((228u * 1024u) / (smem + 1024u));
        const int per_sm = std::max(1, std::min(std::min(by_regs, by_smem), 8));
        HQ_CUDA(ctx, launch_depthwise_col(p, tm, out_mode, ctx->num_sms, per_sm, s, false));
        ctx->launches += 1;
        return HQ_OK;
      }
    }
    // the same shapes with strips of 8 pixels per thread and one multiply-accumulate per dp4a: output tiles of 4 rows
    if (desc->R == 3 && desc->S == 3 && desc->stride_h == 1 && desc->stride_w == 1 && desc->C <= 256 && ctx->force_dw_tiled != 0 && pw->w_zp == 0) {
      p.TR = 4;
      const int budget = 50 * 1024;   // two patches + tables per CTA, two CTAs per SM
      int twt = (budget / (desc->C * (p.TR + 2)) - 2) / 8 * 8;
      twt = std::min(twt, std::min(round_up(Wo, 8), 248));
      if (twt >= 8) {
        p.TWt = twt;
        p.tiles_h = ceil_div(Ho, p.TR);
        p.tiles_w = ceil_div(Wo, p.TWt);
        p.ncls = pw->dw_ncls;
        p.patch_bytes = (uint32_t)desc->C * (uint32_t)(p.TWt + 2) * (uint32_t)(p.TR + 2);
        p.patch_stride = (p.patch_bytes + 127u) & ~127u;
        // strips of 8 pixels per tile are dealt to `slots` thread groups: the divisor of the strip count that gives
        // the most threads within 512
        const int strips = p.TR * (p.TWt / 8), cwords = desc->C / 4;
        p.slots = 1;
        for (int k = 1; k <= strips; ++k)
          if (strips % k == 0 && k * cwords <= 512 && k * cwords <= 320) p.slots = k;
        if (p.slots * cwords < 128)
          for (int k = 1; k <= strips; ++k)
            if (k * cwords <= 512) p.slots = k;
        const int64_t n_tiles = (int64_t)desc->N * p.tiles_h * p.tiles_w;
        if (n_tiles <= INT32_MAX && depthwise_tiled_smem_bytes(p) <= 200u * 1024u) {
          CUtensorMap tm;
          uint64_t dims[4] = {(uint64_t)desc->C, (uint64_t)desc->W, (uint64_t)desc->H, (uint64_t)desc->N};
          uint64_t strides[3] = {(uint64_t)desc->C, (uint64_t)desc->C * desc->W, (uint64_t)desc->C * desc->W * desc->H};
          uint32_t box[4] = {(uint32_t)desc->C, (uint32_t)(p.TWt + 2), (uint32_t)(p.TR + 2), 1u};
          uint32_t es[4] = {1, 1, 1, 1};
          CUresult r = ctx->encode(&tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<int8_t*>(in), dims, strides, box, es,
                                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
          if (r != CUDA_SUCCESS) return fail(ctx, HQ_ERR_CUDA, "tensor map encoding failed (CUresult %d)", (int)r);
          HQ_CUDA(ctx, launch_depthwise_tiled(p, tm, out_mode, ctx->num_sms, s));
          ctx->launches += 1;
          return HQ_OK;
        }
      }
    }
    HQ_CUDA(ctx, launch_depthwise(p, out_mode, ctx->num_sms, s, false));
    ctx->launches += 1;
    return HQ_OK;
  }
  const int Ho = out_dim(desc->H, desc->pad_h, desc->R, desc->stride_h), Wo = out_dim(desc->W, desc->pad_w, desc->S, desc->stride_w);
  if (pw->gather) {   // few input channels: the fused kernel; the image as {W*C/4 words, H, N}, one box of R rows per tile
    GatherParams g = pw->gp;
    g.xq = inq; g.w_scale = w_scale; g.yq = outq; g.out = out;
    g.weights_early = (ctx->overlap && pw->used) ? 1 : 0;
    pw->used = true;
    CUtensorMap tm;
    const uint64_t row_bytes = (uint64_t)desc->W * desc->C;
    uint64_t dims[3] = {row_bytes / 4, (uint64_t)desc->H, (uint64_t)desc->N};
    uint64_t strides[2] = {row_bytes, row_bytes * desc->H};
    uint32_t box[3] = {g.raw_pitch / 4, (uint32_t)g.box_rows, 1u};
    uint32_t es[3] = {1, 1, 1};
    CUresult r = ctx->encode(&tm, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, const_cast<int8_t*>(in), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                             CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(ctx, HQ_ERR_CUDA, "tensor map encoding failed (CUresult %d)", (int)r);
    const int grid = std::max(1, std::min(g.num_tiles, ctx->num_sms));
    HQ_CUDA(ctx, launch_gather_conv(g, tm, out_mode, grid, pw->gather_smem, s, ctx->overlap));
    ctx->launches += 1;
    return HQ_OK;
  }
  // operand A is the forward input (fwd) or the output gradient (bwd data)
  const int aC = dir == HQ_DIR_FWD ? desc->C : desc->K;
  const int aH = dir == HQ_DIR_FWD ? desc->H : Ho;
  const int aW = dir == HQ_DIR_FWD ? desc->W : Wo;
  // Several launches of one call (parity classes of a strided backward pass, channel slices) write disjoint outputs:
  // they run side by side, each on its share of the SMs (every CTA needs a whole SM's shared memory), forked from and
  // joined back into the caller's stream with events.
  const bool weights_early = ctx->overlap && pw->used;
  pw->used = true;
  // asymmetric weights: z_w times the input sum of every output pixel, subtracted by the layer kernels' epilogue
  const int32_t* row_term = nullptr;
  if (pw->w_zp != 0) {
    HQ_CUDA(ctx, launch_rowsum(in, inq, *desc, Ho, Wo, dir == HQ_DIR_BWD_DATA ? 1 : 0, pw->w_zp, pw->row_term, s));
    ctx->launches += 1;
    row_term = pw->row_term;
  }
  const int nsub = (int)pw->subs.size();
  constexpr int kMaxSideBySide = 64;
  bool side_by_side = nsub > 1 && nsub <= kMaxSideBySide && ctx->parallel_subs;
  int share[kMaxSideBySide] = {0};
  if (side_by_side) {
    double total = 0.0;
    double cost[kMaxSideBySide];
    for (int i = 0; i < nsub; ++i) {
      const GemmParams& gp = pw->subs[i].p;
      cost[i] = (double)gp.num_tiles * (6.0 + (double)gp.ntaps * gp.chunks_per_tap * (gp.BK / 64.0) * (gp.BN / 128.0));
      total += cost[i];
    }
    int used = 0;
    for (int i = 0; i < nsub; ++i) {
      share[i] = std::max(1, (int)(ctx->num_sms * cost[i] / total));
      used += share[i];
    }
    for (int i = 0; used < ctx->num_sms; i = (i + 1) % nsub, ++used) ++share[i];
    HQ_CUDA(ctx, cudaEventRecord(ctx->ev_fork, s));
  }
  int sub_index = -1;
  int forked = 0;   // side streams that wait on the fork event so far
  auto join = [&]() -> hq_status {
    if (!side_by_side) return HQ_OK;
    for (int k = 0; k < forked; ++k) {
      HQ_CUDA(ctx, cudaEventRecord(ctx->ev_join[k], ctx->side[k]));
      HQ_CUDA(ctx, cudaStreamWaitEvent(s, ctx->ev_join[k], 0));
    }
    return HQ_OK;
  };
  // A failure after the fork still joins the side streams first: what they already run is then ordered before the
  // caller's later work on `stream`, and a stream capture is not left with an unjoined branch.  The first error is
  // the one reported (its text is kept across the join).
  auto join_after = [&](hq_status e) -> hq_status {
    char keep[sizeof(ctx->err)];
    memcpy(keep, ctx->err, sizeof(keep));
    (void)join();
    memcpy(ctx->err, keep, sizeof(keep));
    return e;
  };
  for (const hq_sub_problem& sub : pw->subs) {
    ++sub_index;
    cudaStream_t ss = s;
    if (side_by_side && sub_index > 0) {
      ss = ctx->side[(sub_index - 1) % 3];
      if (sub_index <= 3) {
        const cudaError_t we = cudaStreamWaitEvent(ss, ctx->ev_fork, 0);
        if (we != cudaSuccess) return join_after(fail(ctx, HQ_ERR_CUDA, "cudaStreamWaitEvent failed: %s", cudaGetErrorString(we)));
        ++forked;
      }
    }
    const int max_ctas = side_by_side ? share[sub_index] : 0;
    CUtensorMap ta;
    if (sub.p.ntaps == 0) {
      ta = CUtensorMap{};
    } else if (sub.patch_matrix != nullptr) {
      // channel counts that no TMA box can address (C = 3): gather the filter windows into rows first
      const cudaError_t pe = launch_patch_matrix(in, sub.patch_matrix, inq, desc->N, desc->H, desc->W, desc->C, Ho, Wo, desc->R, desc->S,
                                                 desc->stride_h, desc->stride_w, desc->pad_h, desc->pad_w, sub.patch_K, sub.patch_RP, s);
      if (pe != cudaSuccess) return join_after(fail(ctx, HQ_ERR_CUDA, "patch gather launch failed: %s", cudaGetErrorString(pe)));
      ctx->launches += 1;
      st = encode_a(ctx, sub, sub.patch_matrix, sub.patch_K, desc->N * Ho * Wo, 1, 1, &ta);
    } else if (sub.window != nullptr) {
      const cudaError_t we = launch_row_window(in, sub.window, inq, desc->N, desc->H, desc->W, desc->C, sub.win_Hg, Wo, desc->S, sub.win_sh,
                                               desc->stride_w, desc->pad_w, sub.win_SB, s);
      if (we != cudaSuccess) return join_after(fail(ctx, HQ_ERR_CUDA, "window gather launch failed: %s", cudaGetErrorString(we)));
      ctx->launches += 1;
      st = encode_a(ctx, sub, sub.window, sub.win_sh * sub.win_SB, Wo, sub.win_Hg, desc->N, &ta);
    } else if (sub.chans > 0) {
      // depthwise: this launch is the dense layer over the channel slice [chan0, chan0 + chans) of input and output
      st = encode_a(ctx, sub, in + sub.chan0, sub.chans, aW, aH, desc->N, &ta, desc->C);
      if (st != HQ_OK) return join_after(st);
      void* o = out_mode == kOutInt8 ? (void*)((int8_t*)out + sub.chan0) : (void*)((uint32_t*)out + sub.chan0);
      st = launch_sub(ctx, ss, sub, ta, sub.tmap_b, inq, w_scale, nullptr, o, outq, out_mode, max_ctas, weights_early, row_term);
      if (st != HQ_OK) return join_after(st);
      continue;
    } else if (sub.a_flat) {
      const int64_t rows = (int64_t)desc->N * aH * aW / sub.gfold;
      st = encode_a(ctx, sub, in, aC * sub.gfold, (int)rows, 1, 1, &ta);
    } else {
      st = encode_a(ctx, sub, in, aC, aW, aH, desc->N, &ta);
    }
    if (st == HQ_OK) st = launch_sub(ctx, ss, sub, ta, sub.tmap_b, inq, w_scale, nullptr, out, outq, out_mode, max_ctas, weights_early, row_term);
    if (st != HQ_OK) return join_after(st);
  }
  return join();
}

hq_status run_linear(hq_ctx* ctx, cudaStream_t s, int M, int N, int K, const int8_t* X, const hq_range_state* xq, const int8_t* W,
                     const float* w_scale, const int32_t* bias, void* out, hq_range_state* yq, int out_mode, const int32_t* row_term = nullptr,
                     bool no_grow = false, const hq_prepared_weights* lpw = nullptr) {
  // no_grow: the call may not allocate; shapes that would need larger context scratch are refused instead
  // lpw: weights prepared by hq_linear_prepare (padded copy, cached column sums, weight zero point); N, K and W then come from it
  if (lpw != nullptr) {
    if (!lpw->linear) return fail(ctx, HQ_ERR_INVALID_ARG, "prepared weights do not belong to a linear layer");
    N = lpw->lin_N;
    K = lpw->lin_K;
    W = lpw->lin_w;
  }
  if (M <= 0 || N <= 0 || K <= 0) return fail(ctx, HQ_ERR_INVALID_ARG, "linear sizes must be positive");
  if (!X || !xq || !W || !w_scale || !out || !yq) return fail(ctx, HQ_ERR_INVALID_ARG, "null pointer argument");
  if (!aligned16(X) || !aligned16(W) || !aligned16(out) || !aligned16(xq) || !aligned16(yq))
    return fail(ctx, HQ_ERR_ALIGNMENT, "tensors and range states must be 16-byte aligned");
  if (lpw != nullptr) {
    if ((lpw->lin_Kp != K || lpw->w_zp != 0) && M > lpw->lin_maxM)
      return fail(ctx, HQ_ERR_UNSUPPORTED, "M = %d exceeds the max_M = %d these weights were prepared for", M, lpw->lin_maxM);
    if (lpw->w_zp != 0) {   // z_w times the row sums of the (unpadded) input
      hq_conv_desc rd{};
      rd.N = 1; rd.H = 1; rd.W = M; rd.C = K; rd.K = N; rd.R = 1; rd.S = 1; rd.stride_h = rd.stride_w = 1; rd.groups = 1;
      HQ_CUDA(ctx, launch_rowsum(X, xq, rd, 1, M, 0, lpw->w_zp, lpw->row_term, s));
      ctx->launches += 1;
      row_term = lpw->row_term;
    }
    if (lpw->lin_Kp != K) {
      HQ_CUDA(ctx, launch_pad_rows(X, lpw->lin_xpad, M, K, lpw->lin_Kp, s));
      ctx->launches += 1;
      X = lpw->lin_xpad;
      K = lpw->lin_Kp;
    }
  } else if (K % 16 != 0) {
    // rows whose length no TMA box can address: zero-padded copies of both operands in context-owned scratch
    const int Kp = round_up(K, 16);
    const size_t need = ((size_t)M + (size_t)N) * Kp;
    if (need > ctx->pad_bytes && no_grow)
      return fail(ctx, HQ_ERR_UNSUPPORTED, "K = %d: rows that are not a multiple of 16 bytes need %zu bytes of padded copies; the context holds %zu and this call may not allocate", K, need, ctx->pad_bytes);
    if (need > ctx->pad_bytes) {
      if (ctx->d_pad) HQ_CUDA(ctx, cudaFree(ctx->d_pad));
      ctx->d_pad = nullptr;
      ctx->pad_bytes = 0;
      HQ_CUDA(ctx, cudaMalloc((void**)&ctx->d_pad, need));
      ctx->pad_bytes = need;
    }
    int8_t* Xp = ctx->d_pad;
    int8_t* Wp = ctx->d_pad + (size_t)M * Kp;
    HQ_CUDA(ctx, launch_pad_rows(X, Xp, M, K, Kp, s));
    HQ_CUDA(ctx, launch_pad_rows(W, Wp, N, K, Kp, s));
    ctx->launches += 2;
    X = Xp;
    W = Wp;
    K = Kp;
  }
  SubSpec sp{};
  sp.n_img = 1; sp.TH = 1; sp.TW = M; sp.in_mul_h = 1; sp.in_mul_w = 1;
  sp.dh = {0}; sp.dw = {0}; sp.a_H = 1; sp.a_W = M; sp.Cin = K; sp.Nout = N;
  sp.out_H = 1; sp.out_W = M; sp.os_h = 1; sp.os_w = 1; sp.oa_h = 0; sp.oa_w = 0; sp.ldY = N; sp.flat = true;
  hq_sub_problem sub;
  std::vector<uint8_t> rc, cc;
  MaskVec rm, cm;
  hq_status st = plan_sub(ctx, sp, sub, rc, cc, rm, cm);
  if (st != HQ_OK) return st;
  if (lpw != nullptr) {   // column sums cached with the weights (zero padded well beyond the widest column tiling)
    sub.p.corr = lpw->lin_corr;
    sub.p.Cpad = K;
    CUtensorMap pta, ptb;
    st = encode_a(ctx, sub, X, K, M, 1, 1, &pta);
    if (st != HQ_OK) return st;
    st = encode_b(ctx, sub, W, K, &ptb);
    if (st != HQ_OK) return st;
    const bool weights_early = ctx->overlap && lpw->used;   // the library's copy of the weights is older than any kernel in flight
    lpw->used = true;
    return launch_sub(ctx, s, sub, pta, ptb, xq, w_scale, bias, out, yq, out_mode, 0, weights_early, row_term);
  }
  if ((size_t)sub.p.corr_ld > ctx->scratch_elems && no_grow)
    return fail(ctx, HQ_ERR_UNSUPPORTED, "N = %d needs %d column sums; the context holds %zu and this call may not allocate", N, sub.p.corr_ld,
                ctx->scratch_elems);
  if ((size_t)sub.p.corr_ld > ctx->scratch_elems) {
    if (ctx->d_scratch) HQ_CUDA(ctx, cudaFree(ctx->d_scratch));
    ctx->d_scratch = nullptr;
    ctx->scratch_elems = 0;
    HQ_CUDA(ctx, cudaMalloc((void**)&ctx->d_scratch, (size_t)sub.p.corr_ld * sizeof(int32_t)));
    ctx->scratch_elems = sub.p.corr_ld;
  }
  // column sums of W for the input zero point (weights may change between calls, so per call)
  const uint32_t one = 1u;
  HQ_CUDA(ctx, launch_corr(W, ctx->d_scratch, N, 1, K, 1, 1, &one, 1, &one, 1, sub.p.corr_ld, s));
  ctx->launches += 1;
  sub.p.corr = ctx->d_scratch;
  sub.p.Cpad = K;  // the caller's matrix is used as is; the K tail is zero-filled by the copy engine
  CUtensorMap ta, tb;
  st = encode_a(ctx, sub, X, K, M, 1, 1, &ta);
  if (st != HQ_OK) return st;
  st = encode_b(ctx, sub, W, K, &tb);
  if (st != HQ_OK) return st;
  return launch_sub(ctx, s, sub, ta, tb, xq, w_scale, bias, out, yq, out_mode, 0, false, row_term);
}

hq_status run_op(hq_ctx* ctx, cudaStream_t s, const hq_op_desc* op, void* out, hq_range_state* yq, int out_mode, bool no_grow = false) {
  if (!op) return fail(ctx, HQ_ERR_INVALID_ARG, "operation descriptor is null");
  switch (op->kind) {
    case HQ_OP_LINEAR:   // pw set: weights prepared by hq_linear_prepare (N, K and w of the descriptor are then ignored)
      return run_linear(ctx, s, op->M, op->N, op->K, op->x, op->xq, op->w, op->w_scale, op->bias, out, yq, out_mode, nullptr, no_grow, op->pw);
    case HQ_OP_CONV_FWD: return run_conv(ctx, s, op->conv, HQ_DIR_FWD, op->x, op->xq, op->pw, op->w_scale, out, yq, out_mode);
    case HQ_OP_CONV_BWD_DATA: return run_conv(ctx, s, op->conv, HQ_DIR_BWD_DATA, op->x, op->xq, op->pw, op->w_scale, out, yq, out_mode);
    default: return fail(ctx, HQ_ERR_INVALID_ARG, "unknown operation kind %d", op->kind);
  }
}

int64_t op_out_elems(const hq_op_desc* op) {
  if (op->kind == HQ_OP_LINEAR) return (int64_t)op->M * (op->pw ? op->pw->lin_N : op->N);
  const hq_conv_desc* d = op->conv;
  if (op->kind == HQ_OP_CONV_FWD)
    return (int64_t)d->N * out_dim(d->H, d->pad_h, d->R, d->stride_h) * out_dim(d->W, d->pad_w, d->S, d->stride_w) * d->K;
  return (int64_t)d->N * d->H * d->W * d->C;
}

}  // namespace

extern "C" {

__attribute__((visibility("default"))) const char* hq_status_string(hq_status s) {
  switch (s) {
    case HQ_OK: return "ok";
    case HQ_ERR_INVALID_ARG: return "invalid argument";
    case HQ_ERR_UNSUPPORTED: return "unsupported shape";
    case HQ_ERR_ALIGNMENT: return "alignment rule violated";
    case HQ_ERR_CUDA: return "CUDA call failed";
    case HQ_ERR_NOT_INITIALIZED: return "not initialised";
    case HQ_ERR_TIMEOUT: return "a bounded device-side wait expired";
  }
  return "unknown status";
}

static bool make_side_streams(hq_ctx* ctx) {
  if (cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming) != cudaSuccess) return false;
  for (int k = 0; k < 3; ++k) {
    if (cudaStreamCreateWithFlags(&ctx->side[k], cudaStreamNonBlocking) != cudaSuccess) return false;
    if (cudaEventCreateWithFlags(&ctx->ev_join[k], cudaEventDisableTiming) != cudaSuccess) return false;
  }
  return true;
}
static void free_side_streams(hq_ctx* ctx) {
  if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
  for (int k = 0; k < 3; ++k) {
    if (ctx->ev_join[k]) cudaEventDestroy(ctx->ev_join[k]);
    if (ctx->side[k]) cudaStreamDestroy(ctx->side[k]);
  }
}

__attribute__((visibility("default"))) hq_status hq_create(hq_ctx** out, int device) {
  if (!out) return HQ_ERR_INVALID_ARG;
  *out = nullptr;
  hq_ctx* ctx = new (std::nothrow) hq_ctx();
  if (!ctx) return HQ_ERR_CUDA;
  ctx->device = device;
  cudaDeviceProp prop{};
  if (cudaSetDevice(device) != cudaSuccess || cudaGetDeviceProperties(&prop, device) != cudaSuccess) {
    delete ctx;
    return HQ_ERR_CUDA;
  }
  if (prop.major != 10) {
    delete ctx;
    return HQ_ERR_UNSUPPORTED;
  }
  ctx->num_sms = prop.multiProcessorCount;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || qres != cudaDriverEntryPointSuccess ||
      !fn) {
    delete ctx;
    return HQ_ERR_NOT_INITIALIZED;
  }
  ctx->encode = (EncodeTiledFn)fn;
  ctx->scratch_elems = 4096;
  if (cudaMalloc((void**)&ctx->d_status, sizeof(int32_t)) != cudaSuccess || cudaMemset(ctx->d_status, 0, sizeof(int32_t)) != cudaSuccess ||
      cudaMalloc((void**)&ctx->d_scratch, ctx->scratch_elems * sizeof(int32_t)) != cudaSuccess ||
      gemm_set_smem_attr(kSmemBudget + 1024) != cudaSuccess || depthwise_tiled_set_smem_attr(200u * 1024u) != cudaSuccess || depthwise_col_set_smem_attr(200u * 1024u) != cudaSuccess || dw_wgrad3x3_set_smem_attr(200u * 1024u) != cudaSuccess ||
      !make_side_streams(ctx)) {
    if (ctx->d_status) cudaFree(ctx->d_status);
    if (ctx->d_scratch) cudaFree(ctx->d_scratch);
    free_side_streams(ctx);
    delete ctx;
    return HQ_ERR_CUDA;
  }
  *out = ctx;
  return HQ_OK;
}

__attribute__((visibility("default"))) hq_status hq_destroy(hq_ctx* ctx) {
  if (!ctx) return HQ_ERR_INVALID_ARG;
  cudaFree(ctx->d_status);
  cudaFree(ctx->d_scratch);
  if (ctx->d_pad) cudaFree(ctx->d_pad);
  if (ctx->d_wgrad) cudaFree(ctx->d_wgrad);
  free_side_streams(ctx);
  delete ctx;
  return HQ_OK;
}

__attribute__((visibility("default"))) const char* hq_last_error(const hq_ctx* ctx) { return ctx ? ctx->err : "null context"; }

__attribute__((visibility("default"))) uint64_t hq_launch_count(const hq_ctx* ctx) { return ctx ? ctx->launches : 0; }
__attribute__((visibility("default"))) uint64_t hq_pair_launch_count(const hq_ctx* ctx) { return ctx ? ctx->pair_launches : 0; }

__attribute__((visibility("default"))) hq_status hq_set_option(hq_ctx* ctx, const char* key, int32_t value) {
  if (!ctx || !key) return HQ_ERR_INVALID_ARG;
  if (std::string(key) == "staging") {
    if (value < -1 || value > 1) return fail(ctx, HQ_ERR_INVALID_ARG, "staging must be -1, 0 or 1");
    ctx->force_mode = value;
    return HQ_OK;
  }
  if (std::string(key) == "side_by_side") {
    if (value < 0 || value > 1) return fail(ctx, HQ_ERR_INVALID_ARG, "side_by_side must be 0 or 1");
    ctx->parallel_subs = value != 0;
    return HQ_OK;
  }
  if (std::string(key) == "depthwise_staging") {
    if (value < -1 || value > 2) return fail(ctx, HQ_ERR_INVALID_ARG, "depthwise_staging must be -1, 0, 1 or 2");
    ctx->force_dw_tiled = value;
    return HQ_OK;
  }
  if (std::string(key) == "depthwise") {
    if (value < -1 || value > 1) return fail(ctx, HQ_ERR_INVALID_ARG, "depthwise must be -1, 0 or 1");
    ctx->force_depthwise = value;
    return HQ_OK;
  }
  if (std::string(key) == "repack") {
    if (value < -1 || value > 2) return fail(ctx, HQ_ERR_INVALID_ARG, "repack must be -1, 0, 1 or 2");
    ctx->force_repack = value;
    return HQ_OK;
  }
  if (std::string(key) == "gather_span") {
    if (value < 0 || value > 1) return fail(ctx, HQ_ERR_INVALID_ARG, "gather_span must be 0 or 1");
    ctx->gather_span = value;
    return HQ_OK;
  }
  if (std::string(key) == "epilogue_groups") {
    if (value < -1 || value > 2) return fail(ctx, HQ_ERR_INVALID_ARG, "epilogue_groups must be -1, 0, 1 or 2");
    ctx->force_epi_groups = value;
    return HQ_OK;
  }
  if (std::string(key) == "col_tiles") {
    if (value < -1 || value > 16) return fail(ctx, HQ_ERR_INVALID_ARG, "col_tiles must be -1 .. 16");
    ctx->force_cols = value;
    return HQ_OK;
  }
  if (std::string(key) == "pair") {
    if (value < -1 || value > 1) return fail(ctx, HQ_ERR_INVALID_ARG, "pair must be -1, 0 or 1");
    ctx->force_pair = value;
    return HQ_OK;
  }
  if (std::string(key) == "wgrad_windows") {
    if (value < -1 || value > 1) return fail(ctx, HQ_ERR_INVALID_ARG, "wgrad_windows must be -1, 0 or 1");
    ctx->wgrad_windows = value;
    return HQ_OK;
  }
  if (std::string(key) == "a_producers") {
    if (value < -1 || value > 2 || value == 0) return fail(ctx, HQ_ERR_INVALID_ARG, "a_producers must be -1, 1 or 2");
    ctx->a_producers = value;
    return HQ_OK;
  }
  if (std::string(key) == "issuers") {
    if (value < 1 || value > 3) return fail(ctx, HQ_ERR_INVALID_ARG, "issuers must be 1, 2 or 3");
    ctx->max_issuers = value;
    return HQ_OK;
  }
  if (std::string(key) == "overlap_launches") {
    if (value < 0 || value > 1) return fail(ctx, HQ_ERR_INVALID_ARG, "overlap_launches must be 0 or 1");
    ctx->overlap = value != 0;
    return HQ_OK;
  }
  return fail(ctx, HQ_ERR_INVALID_ARG, "unknown option '%s'", key);
}

__attribute__((visibility("default"))) hq_status hq_get_async_error(hq_ctx* ctx, void* stream, int32_t* code) {
  if (!ctx || !code) return HQ_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  HQ_CUDA(ctx, cudaStreamSynchronize(s));
  HQ_CUDA(ctx, cudaMemcpy(code, ctx->d_status, sizeof(int32_t), cudaMemcpyDeviceToHost));
  if (*code != 0) {
    HQ_CUDA(ctx, cudaMemset(ctx->d_status, 0, sizeof(int32_t)));
    return fail(ctx, HQ_ERR_TIMEOUT, "device-side wait %d expired", *code);
  }
  return HQ_OK;
}

}  // extern "C"

namespace {
hq_status prepare_conv_body(hq_ctx* ctx, void* stream, const hq_conv_desc* desc, hq_direction dir, const int8_t* W, int32_t w_zero_point,
                            hq_prepared_weights** out) {
  if (!ctx) return HQ_ERR_INVALID_ARG;
  if (hq_status ds = check_device(ctx); ds != HQ_OK) return ds;
  if (!out) return fail(ctx, HQ_ERR_INVALID_ARG, "out is null");
  *out = nullptr;
  if (w_zero_point < -128 || w_zero_point > 127) return fail(ctx, HQ_ERR_INVALID_ARG, "weight zero point %d is not an int8 code", w_zero_point);
  hq_status st = check_desc(ctx, desc);
  if (st != HQ_OK) return st;
  if (!W) return fail(ctx, HQ_ERR_INVALID_ARG, "W is null");
  if (dir != HQ_DIR_FWD && dir != HQ_DIR_BWD_DATA) return fail(ctx, HQ_ERR_INVALID_ARG, "unknown direction");
  cudaStream_t s = (cudaStream_t)stream;
  const hq_conv_desc& d = *desc;
  const int Ho = out_dim(d.H, d.pad_h, d.R, d.stride_h), Wo = out_dim(d.W, d.pad_w, d.S, d.stride_w);
  hq_prepared_weights* pw = new (std::nothrow) hq_prepared_weights();
  if (!pw) return fail(ctx, HQ_ERR_CUDA, "out of host memory");
  pw->desc = d;
  pw->dir = dir;
  pw->w_zp = w_zero_point;
  auto bail = [&](hq_status e) {
    for (void* p : pw->allocs) cudaFree(p);
    delete pw;
    return e;
  };

  // Backward data of a stride-1 depthwise layer is a forward depthwise layer over the output gradient (Ho x Wo) with the
  // filter turned by 180 degrees and padding R-1-pad: dx(hi) = sum_r dy(hi + pad - r) w(r) = sum_r' dy(hi - (R-1-pad) + r') w(R-1-r').
  // Strided depthwise layers, and any depthwise layer with a non-zero weight zero point, run backward data by the
  // definition instead (depthwise_bwd_kernel).
  const bool dw_bwd = d.groups != 1 && dir == HQ_DIR_BWD_DATA;
  const bool dw_bwd_direct = dw_bwd && (d.stride_h != 1 || d.stride_w != 1 || w_zero_point != 0);
  hq_conv_desc dwd = d;
  if (d.groups != 1) {
    if (d.C % 16 != 0) return bail(fail(ctx, HQ_ERR_UNSUPPORTED, "depthwise needs C %% 16 == 0"));
    if (dw_bwd_direct) {
      pw->depthwise = true;
      pw->dw_bwd_direct = true;
      pw->dw_run = d;
      int32_t* unused_corr = nullptr;
      const uint32_t all = 0xFFFFFFFFu;
      if ((st = dev_alloc(ctx, pw, (void**)&pw->dw_w_plain, (size_t)d.C * d.R * d.S)) != HQ_OK) return bail(st);
      if ((st = dev_alloc(ctx, pw, (void**)&unused_corr, (size_t)d.C * sizeof(int32_t))) != HQ_OK) return bail(st);
      cudaError_t e = launch_dw_prep(W, pw->dw_w_plain, unused_corr, d.C, d.R, d.S, &all, 1, &all, 1, 0, s);   // tap-major copy, not turned
      if (e != cudaSuccess) return bail(fail(ctx, HQ_ERR_CUDA, "depthwise weight preparation failed: %s", cudaGetErrorString(e)));
      ctx->launches += 1;
      *out = pw;
      return HQ_OK;
    }
    if (dw_bwd) {
      dwd.H = Ho;
      dwd.W = Wo;
      dwd.pad_h = d.R - 1 - d.pad_h;
      dwd.pad_w = d.S - 1 - d.pad_w;
    }
  }
  pw->dw_run = dwd;
  // Optional form of a depthwise layer on the tensor cores: ceil(C / 64) dense layers, one per 64-channel slice of
  // input and output, each with a weight matrix that is zero off the channel diagonal (the int32 sums are the same).
  // Measured on the 56x56x144 layer it is only on a par with the CUDA-core kernel (N = 64 MMAs are bound by
  // shared-memory reads of the pixel operand), so it is not chosen by default.
  const bool dw_dense = d.groups != 1 && ctx->force_depthwise == 1 && !dw_bwd && w_zero_point == 0;
  if (dw_dense) {
    for (int c0 = 0; c0 < d.C; c0 += 64) {
      const int cw = std::min(64, d.C - c0);
      int8_t* Wd = nullptr;
      if ((st = dev_alloc(ctx, pw, (void**)&Wd, (size_t)cw * d.R * d.S * cw)) != HQ_OK) return bail(st);
      cudaError_t e = launch_dw_dense(W, Wd, d.R * d.S, c0, cw, s);
      if (e != cudaSuccess) return bail(fail(ctx, HQ_ERR_CUDA, "depthwise weight expansion failed: %s", cudaGetErrorString(e)));
      ctx->launches += 1;
      hq_conv_desc dd = d;
      dd.C = dd.K = cw;
      dd.groups = 1;
      SubSpec sp{};
      std::vector<int> tr, ts;
      sp.n_img = d.N; sp.TH = Ho; sp.TW = Wo; sp.in_mul_h = d.stride_h; sp.in_mul_w = d.stride_w;
      for (int r = 0; r < d.R; ++r) { sp.dh.push_back(r - d.pad_h); tr.push_back(r); }
      for (int q = 0; q < d.S; ++q) { sp.dw.push_back(q - d.pad_w); ts.push_back(q); }
      sp.a_H = d.H; sp.a_W = d.W; sp.Cin = cw; sp.Nout = cw;
      sp.out_H = Ho; sp.out_W = Wo; sp.os_h = sp.os_w = 1; sp.oa_h = sp.oa_w = 0; sp.ldY = d.C; sp.flat = false;
      if ((st = build_sub(ctx, pw, s, sp, dd, Wd, tr, ts, false, 1)) != HQ_OK) return bail(st);
      pw->subs.back().chan0 = c0;
      pw->subs.back().chans = cw;
    }
    *out = pw;
    return HQ_OK;
  }
  if (d.groups != 1 && !dw_dense) {
    pw->depthwise = true;
    TapVec dh, dw;
    for (int r = 0; r < d.R; ++r) dh.push_back(r - dwd.pad_h);
    for (int q = 0; q < d.S; ++q) dw.push_back(q - dwd.pad_w);
    std::vector<uint8_t> rowcls, colcls;
    MaskVec rm, cm;
    // output rows / columns of the layer the kernel runs (backward data: the input image of the original layer)
    const int run_Ho = out_dim(dwd.H, dwd.pad_h, dwd.R, dwd.stride_h), run_Wo = out_dim(dwd.W, dwd.pad_w, dwd.S, dwd.stride_w);
    border_classes(run_Ho, dwd.stride_h, dh, dwd.H, rowcls, rm);
    border_classes(run_Wo, dwd.stride_w, dw, dwd.W, colcls, cm);
    if (rm.size() > 16 || cm.size() > 16) return bail(fail(ctx, HQ_ERR_UNSUPPORTED, "too many border classes"));
    pw->dw_ncolcls = (int)cm.size();
    pw->dw_ncls = (int)(rm.size() * cm.size());
    if ((st = dev_alloc(ctx, pw, (void**)&pw->dw_w, (size_t)d.C * d.R * d.S)) != HQ_OK) return bail(st);
    if ((st = dev_alloc(ctx, pw, (void**)&pw->dw_corr, rm.size() * cm.size() * d.C * sizeof(int32_t))) != HQ_OK) return bail(st);
    cudaError_t e = launch_dw_prep(W, pw->dw_w, pw->dw_corr, d.C, d.R, d.S, rm.data(), (int)rm.size(), cm.data(), (int)cm.size(), dw_bwd ? 1 : 0, s);
    if (e != cudaSuccess) return bail(fail(ctx, HQ_ERR_CUDA, "depthwise weight preparation failed: %s", cudaGetErrorString(e)));
    ctx->launches += 1;
    if ((st = upload(ctx, pw, rowcls, &pw->dw_rowcls, s)) != HQ_OK) return bail(st);
    if ((st = upload(ctx, pw, colcls, &pw->dw_colcls, s)) != HQ_OK) return bail(st);
    *out = pw;
    return HQ_OK;
  }

  const bool pointwise = d.R == 1 && d.S == 1 && d.stride_h == 1 && d.stride_w == 1 && d.pad_h == 0 && d.pad_w == 0;
  if (dir == HQ_DIR_FWD) {
    SubSpec sp{};
    std::vector<int> tr, ts;
    int g = 1;
    if (pointwise) {
      g = fold_factor(d.C, (int64_t)d.N * d.H * d.W);
      if (g == 0) return bail(fail(ctx, HQ_ERR_UNSUPPORTED, "C = %d cannot be folded to a 16-byte multiple", d.C));
      const int64_t rows = (int64_t)d.N * d.H * d.W / g;
      if (rows > INT32_MAX) return bail(fail(ctx, HQ_ERR_UNSUPPORTED, "too many pixels"));
      sp.n_img = 1; sp.TH = 1; sp.TW = (int)rows; sp.in_mul_h = sp.in_mul_w = 1; sp.dh = {0}; sp.dw = {0};
      sp.a_H = 1; sp.a_W = (int)rows; sp.Cin = g * d.C; sp.Nout = g * d.K;
      sp.out_H = 1; sp.out_W = (int)rows; sp.os_h = sp.os_w = 1; sp.oa_h = sp.oa_w = 0; sp.ldY = (int64_t)g * d.K; sp.flat = true;
      tr = {0}; ts = {0};
    } else {
      if (d.C % 16 != 0) {
        // Channel counts no TMA box can address (the RGB stem).  Preferred: a pre-pass gathers, per output column, the
        // horizontal filter windows of stride_h consecutive input rows into a library-owned tensor X2 of
        // Cg = stride_h * SB bytes per pixel; over X2 the layer is a stride-1 convolution with vertical taps only.
        // Preferred where the shape allows: the fused kernel that gathers the filter windows in shared memory (no repacked
        // copy of the input in global memory).  Needs image rows that a TMA box can address (W*C a multiple of 16), one
        // column tile (K a multiple of 16, at most 256), an instantiated (R, S*C) and symmetric weights.
        {
          const int SC = d.S * d.C, Kp = round_up(d.R * SC, 32);
          const uint32_t pitch = (uint32_t)round_up((127 * d.stride_w + d.S) * d.C + 15 + 8, 16);
          std::vector<uint8_t> grc, gcc;
          MaskVec grm, gcm;
          TapVec gdh, gdw;
          for (int r = 0; r < d.R; ++r) gdh.push_back(r - d.pad_h);
          for (int q = 0; q < d.S; ++q) gdw.push_back(q - d.pad_w);
          border_classes(Ho, d.stride_h, gdh, d.H, grc, grm);
          border_classes(Wo, d.stride_w, gdw, d.W, gcc, gcm);
          const int corr_ld = round_up(d.K, 16);
          const size_t zc_bytes = grm.size() * gcm.size() * (size_t)corr_ld * 4;
          if (gather_conv_supported(d.R, SC) && (d.W * d.C) % 16 == 0 && d.K % 16 == 0 && d.K <= 256 && pitch <= 1024 && grm.size() <= 16 &&
              gcm.size() <= 16 && zc_bytes <= kMaxZcBytes && w_zero_point == 0 && (ctx->force_repack < 0 || ctx->force_repack == 2) &&
              (int64_t)d.N * Ho * ceil_div(Wo, kTileM) < INT32_MAX) {
            GatherParams& g = pw->gp;
            g.N = d.N; g.H = d.H; g.W = d.W; g.C = d.C; g.Ho = Ho; g.Wo = Wo; g.R = d.R; g.S = d.S;
            g.stride_h = d.stride_h; g.stride_w = d.stride_w; g.pad_h = d.pad_h; g.pad_w = d.pad_w;
            g.BN = d.K;
            g.tiles_w = ceil_div(Wo, kTileM);
            g.num_tiles = d.N * Ho * g.tiles_w;
            g.span = 0;
            g.tiles_img = Ho * g.tiles_w;
            g.box_rows = d.R;
            // Output rows shorter than a tile would leave tile rows unused (Wo = 112: an eighth of every MMA and epilogue
            // pass).  Tiles then run over the pixels of an image in row-major order, across row ends, and the raw box holds
            // the input rows under every output row a tile touches (the box is as wide as the image row either way).
            if (Wo < kTileM && ctx->gather_span != 0) {
              const int HW = Ho * Wo, tiles_img = ceil_div(HW, kTileM);
              int rows_max = 1;
              for (int t = 0; t < tiles_img; ++t) {
                const int f0 = t * kTileM, f1 = std::min(f0 + kTileM, HW) - 1;
                rows_max = std::max(rows_max, f1 / Wo - f0 / Wo + 1);
              }
              const int box_rows = (rows_max - 1) * d.stride_h + d.R;
              if (box_rows <= 256 && tiles_img < Ho && (uint64_t)pitch * box_rows <= 32u * 1024u) {
                g.span = 1;
                g.tiles_img = tiles_img;
                g.box_rows = box_rows;
                g.num_tiles = d.N * tiles_img;
              }
            }
            g.raw_pitch = pitch;
            g.raw_box_bytes = pitch * (uint32_t)g.box_rows;
            g.raw_stage_stride = (g.raw_box_bytes + 127u) & ~127u;
            g.a_stage_bytes = (uint32_t)kTileM * (uint32_t)Kp;
            g.stages_raw = g.raw_stage_stride * 4u <= 48u * 1024u ? 4 : 2;
            g.off_w = 0;
            g.off_zc = (uint32_t)round_up(d.K * Kp, 128);
            g.off_raw = (uint32_t)round_up((int)(g.off_zc + zc_bytes), 1024);
            g.off_a = (uint32_t)round_up((int)(g.off_raw + g.stages_raw * g.raw_stage_stride + 64), 1024);
            const uint32_t budget = 200u * 1024u;
            g.stages_a = (int)std::min<uint32_t>(8u, (budget - g.off_a) / g.a_stage_bytes);
            if (g.stages_a >= 2) {
              pw->gather_smem = g.off_a + (uint32_t)g.stages_a * g.a_stage_bytes + 1024u;
              g.corr_ld = corr_ld;
              g.ncolcls = (int)gcm.size();
              g.zc_elems = (int)(grm.size() * gcm.size()) * corr_ld;
              g.cls_in_smem = (Ho <= 512 && Wo <= 512) ? 1 : 0;
              g.idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(d.K >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
              uint32_t stride = 32;
              while ((int)stride < d.K) stride <<= 1;
              g.tmem_buf_stride = stride;
              g.tmem_bufs = (int)std::min<uint32_t>(8, 512 / stride);
              g.tmem_cols = (uint32_t)g.tmem_bufs * stride;
              g.epi_groups = std::min(3, g.tmem_bufs);
              g.tmem_bufs_log2 = g.tmem_bufs == 8 ? 3 : (g.tmem_bufs == 4 ? 2 : 1);
              g.epi_groups_log2 = g.epi_groups == 4 ? 2 : 1;
              g.fd_tiles_w = make_fastdiv(g.tiles_w);
              g.fd_Ho = make_fastdiv(Ho);
              g.fd_Wo = make_fastdiv(Wo);
              g.fd_tiles_img = make_fastdiv(g.tiles_img);
              g.status = ctx->d_status;
              g.acc_bound = (float)(d.R * SC) * 255.0f * 128.0f;
              int8_t* wm = nullptr;
              int32_t* corr = nullptr;
              if ((st = dev_alloc(ctx, pw, (void**)&wm, (size_t)d.K * Kp)) != HQ_OK) return bail(st);
              if ((st = dev_alloc(ctx, pw, (void**)&corr, zc_bytes)) != HQ_OK) return bail(st);
              cudaError_t e = cudaMemsetAsync(corr, 0, zc_bytes, s);
              if (e == cudaSuccess) e = launch_pad_rows(W, wm, d.K, d.R * SC, Kp, s);   // the filter's own order, rows padded to Kp
              if (e == cudaSuccess) e = launch_gather_corr(W, corr, d.K, d.R, d.S, d.C, grm.data(), (int)grm.size(), gcm.data(), (int)gcm.size(), corr_ld, s);
              if (e != cudaSuccess) return bail(fail(ctx, HQ_ERR_CUDA, "weight preparation failed: %s", cudaGetErrorString(e)));
              ctx->launches += 2;
              g.wmat = wm;
              g.corr = corr;
              uint8_t *drc = nullptr, *dcc = nullptr;
              if ((st = upload(ctx, pw, grc, &drc, s)) != HQ_OK) return bail(st);
              if ((st = upload(ctx, pw, gcc, &dcc, s)) != HQ_OK) return bail(st);
              g.rowcls = drc;
              g.colcls = dcc;
              pw->gather = true;
              *out = pw;
              return HQ_OK;
            }
          }
        }
        const int sh = d.stride_h, sc = d.S * d.C;
        int SB = round_up(sc, 16), Cg = 0;
        if (64 % sh == 0 && sh * SB <= 64) { SB = 64 / sh; Cg = 64; }
        else if (128 % sh == 0 && sh * SB <= 128) { SB = 128 / sh; Cg = 128; }
        auto floordiv = [](int a, int b) { return a >= 0 ? a / b : -((-a + b - 1) / b); };
        const int dh_min = floordiv(-d.pad_h, sh), dh_max = floordiv(d.R - 1 - d.pad_h, sh);
        const int Hg = (d.H + sh - 1) / sh;
        if (Cg != 0 && dh_max - dh_min + 1 <= kMaxTaps && ctx->force_repack != 0 && (int64_t)d.N * Hg * Wo * sh < ((int64_t)1 << 31)) {
          sp.n_img = d.N; sp.TH = Ho; sp.TW = Wo; sp.in_mul_h = sp.in_mul_w = 1;
          for (int t = dh_min; t <= dh_max; ++t) sp.dh.push_back(t);
          sp.dw = {0};
          sp.a_H = Hg; sp.a_W = Wo; sp.Cin = Cg; sp.Nout = d.K;
          sp.out_H = Ho; sp.out_W = Wo; sp.os_h = sp.os_w = 1; sp.oa_h = sp.oa_w = 0; sp.ldY = d.K; sp.flat = false;
          const int ntaps = dh_max - dh_min + 1;
          const WeightPrep prep = [&](hq_sub_problem& sub) {
            ctx->launches += 1;
            return launch_prep_window_weights(W, sub.wmat, d.K, d.R, sc, sh, SB, ntaps, dh_min, d.pad_h, s);
          };
          if ((st = build_sub(ctx, pw, s, sp, d, W, std::vector<int>(ntaps, 0), {0}, false, 1, &prep)) != HQ_OK) return bail(st);
          hq_sub_problem& sub = pw->subs.back();
          sub.win_sh = sh;
          sub.win_SB = SB;
          sub.win_Hg = Hg;
          if ((st = dev_alloc(ctx, pw, (void**)&sub.window, (size_t)d.N * Hg * Wo * Cg)) != HQ_OK) return bail(st);
          *out = pw;
          return HQ_OK;
        }
        // Fallback: whole patch rows of [R*S*C] input bytes (one filter row per 8-byte aligned slot, padded to a multiple
        // of 16, padding taps holding the input zero point) in a library-owned matrix; the layer is a flat GEMM over it
        const int64_t rows = (int64_t)d.N * Ho * Wo;
        const int RP = round_up(d.S * d.C, 8);
        const int Kp = round_up(d.R * RP, 16);
        if (rows > INT32_MAX) return bail(fail(ctx, HQ_ERR_UNSUPPORTED, "too many pixels"));
        sp.n_img = 1; sp.TH = 1; sp.TW = (int)rows; sp.in_mul_h = sp.in_mul_w = 1; sp.dh = {0}; sp.dw = {0};
        sp.a_H = 1; sp.a_W = (int)rows; sp.Cin = Kp; sp.Nout = d.K;
        sp.out_H = 1; sp.out_W = (int)rows; sp.os_h = sp.os_w = 1; sp.oa_h = sp.oa_w = 0; sp.ldY = d.K; sp.flat = true;
        const WeightPrep prep = [&](hq_sub_problem& sub) {
          ctx->launches += 1;
          return launch_prep_patch_weights(W, sub.wmat, d.K, d.R, d.S * d.C, RP, sub.p.Cpad, s);
        };
        if ((st = build_sub(ctx, pw, s, sp, d, W, {0}, {0}, false, 1, &prep)) != HQ_OK) return bail(st);
        hq_sub_problem& sub = pw->subs.back();
        sub.patch_K = Kp;
        sub.patch_RP = RP;
        if ((st = dev_alloc(ctx, pw, (void**)&sub.patch_matrix, (size_t)rows * Kp)) != HQ_OK) return bail(st);
        *out = pw;
        return HQ_OK;
      }
      sp.n_img = d.N; sp.TH = Ho; sp.TW = Wo; sp.in_mul_h = d.stride_h; sp.in_mul_w = d.stride_w;
      for (int r = 0; r < d.R; ++r) { sp.dh.push_back(r - d.pad_h); tr.push_back(r); }
      for (int q = 0; q < d.S; ++q) { sp.dw.push_back(q - d.pad_w); ts.push_back(q); }
      sp.a_H = d.H; sp.a_W = d.W; sp.Cin = d.C; sp.Nout = d.K;
      sp.out_H = Ho; sp.out_W = Wo; sp.os_h = sp.os_w = 1; sp.oa_h = sp.oa_w = 0; sp.ldY = d.K; sp.flat = false;
    }
    if ((st = build_sub(ctx, pw, s, sp, d, W, tr, ts, false, g)) != HQ_OK) return bail(st);
  } else {
    if (pointwise) {
      const int g = fold_factor(d.K, (int64_t)d.N * d.H * d.W);
      if (g == 0) return bail(fail(ctx, HQ_ERR_UNSUPPORTED, "K = %d cannot be folded to a 16-byte multiple", d.K));
      const int64_t rows = (int64_t)d.N * d.H * d.W / g;
      if (rows > INT32_MAX) return bail(fail(ctx, HQ_ERR_UNSUPPORTED, "too many pixels"));
      SubSpec sp{};
      sp.n_img = 1; sp.TH = 1; sp.TW = (int)rows; sp.in_mul_h = sp.in_mul_w = 1; sp.dh = {0}; sp.dw = {0};
      sp.a_H = 1; sp.a_W = (int)rows; sp.Cin = g * d.K; sp.Nout = g * d.C;
      sp.out_H = 1; sp.out_W = (int)rows; sp.os_h = sp.os_w = 1; sp.oa_h = sp.oa_w = 0; sp.ldY = (int64_t)g * d.C; sp.flat = true;
      if ((st = build_sub(ctx, pw, s, sp, d, W, {0}, {0}, true, g)) != HQ_OK) return bail(st);
    } else {
      if (d.K % 16 != 0) return bail(fail(ctx, HQ_ERR_UNSUPPORTED, "K = %d: backward data needs K %% 16 == 0", d.K));
      // one dense stride-1 problem per output parity class (a, b): hi = i*stride_h + a, wi = j*stride_w + b
      for (int a = 0; a < d.stride_h; ++a)
        for (int b = 0; b < d.stride_w; ++b) {
          SubSpec sp{};
          sp.n_img = d.N;
          sp.TH = (d.H - a + d.stride_h - 1) / d.stride_h;
          sp.TW = (d.W - b + d.stride_w - 1) / d.stride_w;
          if (sp.TH <= 0 || sp.TW <= 0) continue;
          sp.in_mul_h = sp.in_mul_w = 1;
          std::vector<int> tr, ts;
          for (int r = 0; r < d.R; ++r) {
            const int x = a + d.pad_h - r;
            if (((x % d.stride_h) + d.stride_h) % d.stride_h == 0) { sp.dh.push_back(x / d.stride_h); tr.push_back(r); }
          }
          for (int q = 0; q < d.S; ++q) {
            const int x = b + d.pad_w - q;
            if (((x % d.stride_w) + d.stride_w) % d.stride_w == 0) { sp.dw.push_back(x / d.stride_w); ts.push_back(q); }
          }
          sp.a_H = Ho; sp.a_W = Wo; sp.Cin = d.K; sp.Nout = d.C;
          sp.out_H = d.H; sp.out_W = d.W; sp.os_h = d.stride_h; sp.os_w = d.stride_w; sp.oa_h = a; sp.oa_w = b; sp.ldY = d.C; sp.flat = false;
          sp.whole_gpu = d.stride_h * d.stride_w == 1;   // the parity classes of a strided layer run side by side
          if ((st = build_sub(ctx, pw, s, sp, d, W, tr, ts, true, 1)) != HQ_OK) return bail(st);
        }
    }
  }
  *out = pw;
  return HQ_OK;
}

hq_status prepare_conv(hq_ctx* ctx, void* stream, const hq_conv_desc* desc, hq_direction dir, const int8_t* W, int32_t w_zero_point,
                       hq_prepared_weights** out) {
  hq_status st = prepare_conv_body(ctx, stream, desc, dir, W, w_zero_point, out);
  if (st != HQ_OK) return st;
  hq_prepared_weights* pw = *out;
  if (w_zero_point != 0 && !pw->depthwise) {
    // room for the weight-zero-point term of every output pixel (forward: N x Ho x Wo, backward data: N x H x W)
    const hq_conv_desc& d = pw->desc;
    const int Ho = out_dim(d.H, d.pad_h, d.R, d.stride_h), Wo = out_dim(d.W, d.pad_w, d.S, d.stride_w);
    pw->row_term_elems = dir == HQ_DIR_FWD ? (size_t)d.N * Ho * Wo : (size_t)d.N * d.H * d.W;
    st = dev_alloc(ctx, pw, (void**)&pw->row_term, pw->row_term_elems * sizeof(int32_t));
    if (st != HQ_OK) {
      for (void* p : pw->allocs) cudaFree(p);
      delete pw;
      *out = nullptr;
      return st;
    }
  }
  return HQ_OK;
}
}  // namespace

extern "C" {

__attribute__((visibility("default"))) hq_status hq_weights_prepare(hq_ctx* ctx, void* stream, const hq_conv_desc* desc, hq_direction dir, const int8_t* W,
                                                                    hq_prepared_weights** out) {
  return prepare_conv(ctx, stream, desc, dir, W, 0, out);
}

__attribute__((visibility("default"))) hq_status hq_weights_prepare_zp(hq_ctx* ctx, void* stream, const hq_conv_desc* desc, hq_direction dir, const int8_t* W,
                                                                       int32_t w_zero_point, hq_prepared_weights** out) {
  return prepare_conv(ctx, stream, desc, dir, W, w_zero_point, out);
}

__attribute__((visibility("default"))) hq_status hq_linear_prepare(hq_ctx* ctx, void* stream, int32_t N, int32_t K, const int8_t* W, int32_t w_zero_point,
                                                                   int32_t max_M, hq_prepared_weights** out) {
  if (!ctx) return HQ_ERR_INVALID_ARG;
  if (hq_status ds = check_device(ctx); ds != HQ_OK) return ds;
  if (!out) return fail(ctx, HQ_ERR_INVALID_ARG, "out is null");
  *out = nullptr;
  if (N <= 0 || K <= 0 || max_M < 0) return fail(ctx, HQ_ERR_INVALID_ARG, "linear sizes must be positive");
  if (!W || !aligned16(W)) return fail(ctx, W ? HQ_ERR_ALIGNMENT : HQ_ERR_INVALID_ARG, "W is null or not 16-byte aligned");
  if (w_zero_point < -128 || w_zero_point > 127) return fail(ctx, HQ_ERR_INVALID_ARG, "weight zero point %d is not an int8 code", w_zero_point);
  const int Kp = round_up(K, 16);
  if ((Kp != K || w_zero_point != 0) && max_M <= 0)
    return fail(ctx, HQ_ERR_INVALID_ARG, "max_M must be given when K is not a multiple of 16 or the weights have a zero point");
  cudaStream_t s = (cudaStream_t)stream;
  hq_prepared_weights* pw = new (std::nothrow) hq_prepared_weights();
  if (!pw) return fail(ctx, HQ_ERR_CUDA, "out of host memory");
  auto bail = [&](hq_status e) {
    for (void* p : pw->allocs) cudaFree(p);
    delete pw;
    return e;
  };
  pw->linear = true;
  pw->lin_N = N; pw->lin_K = K; pw->lin_Kp = Kp; pw->lin_maxM = max_M;
  pw->w_zp = w_zero_point;
  hq_status st;
  if ((st = dev_alloc(ctx, pw, (void**)&pw->lin_w, (size_t)N * Kp)) != HQ_OK) return bail(st);
  const size_t corr_elems = (size_t)N + 512;   // every column tiling pads N by less than this
  if ((st = dev_alloc(ctx, pw, (void**)&pw->lin_corr, corr_elems * sizeof(int32_t))) != HQ_OK) return bail(st);
  cudaError_t e = cudaMemsetAsync(pw->lin_corr, 0, corr_elems * sizeof(int32_t), s);
  if (e == cudaSuccess) e = launch_pad_rows(W, pw->lin_w, N, K, Kp, s);
  const uint32_t one = 1u;
  if (e == cudaSuccess) e = launch_corr(pw->lin_w, pw->lin_corr, N, 1, Kp, 1, 1, &one, 1, &one, 1, (int)corr_elems, s);
  if (e != cudaSuccess) return bail(fail(ctx, HQ_ERR_CUDA, "linear weight preparation failed: %s", cudaGetErrorString(e)));
  ctx->launches += 2;
  if (Kp != K && (st = dev_alloc(ctx, pw, (void**)&pw->lin_xpad, (size_t)max_M * Kp)) != HQ_OK) return bail(st);
  if (w_zero_point != 0) {
    pw->row_term_elems = (size_t)max_M;
    if ((st = dev_alloc(ctx, pw, (void**)&pw->row_term, pw->row_term_elems * sizeof(int32_t))) != HQ_OK) return bail(st);
  }
  *out = pw;
  return HQ_OK;
}

__attribute__((visibility("default"))) hq_status hq_linear_fwd_prepared(hq_ctx* ctx, void* stream, int32_t M, const int8_t* X, const hq_range_state* xq,
                                                                        const hq_prepared_weights* pw, const float* w_scale, const int32_t* bias,
                                                                        int8_t* Y, hq_range_state* yq) {
  if (!ctx) return HQ_ERR_INVALID_ARG;
  if (hq_status ds = check_device(ctx); ds != HQ_OK) return ds;
  if (!pw) return fail(ctx, HQ_ERR_INVALID_ARG, "prepared weights are null");
  return run_linear(ctx, (cudaStream_t)stream, M, 0, 0, X, xq, nullptr, w_scale, bias, Y, yq, kOutInt8, nullptr, false, pw);
}

__attribute__((visibility("default"))) hq_status hq_weights_release(hq_ctx* ctx, hq_prepared_weights* pw) {
  if (!ctx || !pw) return HQ_ERR_INVALID_ARG;
  for (void* p : pw->allocs) cudaFree(p);
  delete pw;
  return HQ_OK;
}

__attribute__((visibility("default"))) hq_status hq_linear_fwd(hq_ctx* ctx, void* stream, int32_t M, int32_t N, int32_t K, const int8_t* X, const hq_range_state* xq, const int8_t* W,
                        const float* w_scale, const int32_t* bias, int8_t* Y, hq_range_state* yq) {
  if (!ctx) return HQ_ERR_INVALID_ARG;
  if (hq_status ds = check_device(ctx); ds != HQ_OK) return ds;
  return run_linear(ctx, (cudaStream_t)stream, M, N, K, X, xq, W, w_scale, bias, Y, yq, kOutInt8);
}

__attribute__((visibility("default"))) hq_status hq_conv_fwd(hq_ctx* ctx, void* stream, const hq_conv_desc* desc, const int8_t* X, const hq_range_state* xq,
                      const hq_prepared_weights* pw, const float* w_scale, int8_t* Y, hq_range_state* yq) {
  if (!ctx) return HQ_ERR_INVALID_ARG;
  if (hq_status ds = check_device(ctx); ds != HQ_OK) return ds;
  return run_conv(ctx, (cudaStream_t)stream, desc, HQ_DIR_FWD, X, xq, pw, w_scale, Y, yq, kOutInt8);
}

__attribute__((visibility("default"))) hq_status hq_conv_bwd_data(hq_ctx* ctx, void* stream, const hq_conv_desc* desc, const int8_t* dY, const hq_range_state* dyq,
                           const hq_prepared_weights* pw, const float* w_scale, int8_t* dX, hq_range_state* dxq) {
  if (!ctx) return HQ_ERR_INVALID_ARG;
  if (hq_status ds = check_device(ctx); ds != HQ_OK) return ds;
  return run_conv(ctx, (cudaStream_t)stream, desc, HQ_DIR_BWD_DATA, dY, dyq, pw, w_scale, dX, dxq, kOutInt8);
}

__attribute__((visibility("default"))) hq_status hq_range_update(hq_ctx* ctx, void* stream, hq_range_state* states, int32_t count, float eta) {
  if (!ctx) return HQ_ERR_INVALID_ARG;
  if (hq_status ds = check_device(ctx); ds != HQ_OK) return ds;
  if (!states || count <= 0) return fail(ctx, HQ_ERR_INVALID_ARG, "states is null or count is not positive");
  if (!aligned16(states)) return fail(ctx, HQ_ERR_ALIGNMENT, "range states must be 16-byte aligned");
  if (!(eta >= 0.0f && eta <= 1.0f)) return fail(ctx, HQ_ERR_INVALID_ARG, "eta must lie in [0, 1]");
  HQ_CUDA(ctx, launch_range_update(states, count, eta, (cudaStream_t)stream, ctx->overlap));
  ctx->launches += 1;
  return HQ_OK;
}

__attribute__((visibility("default"))) hq_status hq_stats_pack(hq_ctx* ctx, void* stream, const hq_range_state* states, int32_t count, int32_t* buf) {
  if (!ctx) return HQ_ERR_INVALID_ARG;
  if (hq_status ds = check_device(ctx); ds != HQ_OK) return ds;
  if (!states || !buf || count <= 0) return fail(ctx, HQ_ERR_INVALID_ARG, "states or buf is null, or count is not positive");
  if (!aligned16(states)) return fail(ctx, HQ_ERR_ALIGNMENT, "range states must be 16-byte aligned");
  HQ_CUDA(ctx, launch_stats_pack(states, count, buf, (cudaStream_t)stream));
  ctx->launches += 1;
  return HQ_OK;
}

__attribute__((visibility("default"))) hq_status hq_stats_unpack(hq_ctx* ctx, void* stream, hq_range_state* states, int32_t count, const int32_t* buf) {
  if (!ctx) return HQ_ERR_INVALID_ARG;
  if (hq_status ds = check_device(ctx); ds != HQ_OK) return ds;
  if (!states || !buf || count <= 0) return fail(ctx, HQ_ERR_INVALID_ARG, "states or buf is null, or count is not positive");
  if (!aligned16(states)) return fail(ctx, HQ_ERR_ALIGNMENT, "range states must be 16-byte aligned");
  HQ_CUDA(ctx, launch_stats_unpack(states, count, buf, (cudaStream_t)stream));
  ctx->launches += 1;
  return HQ_OK;
}

__attribute__((visibility("default"))) hq_status hq_mma_peak_probe(hq_ctx* ctx, void* stream, int32_t pair, int32_t bn, int32_t chunks, uint64_t* ops) {
  if (!ctx) return HQ_ERR_INVALID_ARG;
  if (hq_status ds = check_device(ctx); ds != HQ_OK) return ds;
  if (pair < 0 || pair > 1 || chunks <= 0 || chunks > (1 << 20)) return fail(ctx, HQ_ERR_INVALID_ARG, "pair must be 0 or 1, chunks in [1, 2^20]");
  if (bn < 32 || bn > 256 || bn % 32 != 0) return fail(ctx, HQ_ERR_INVALID_ARG, "bn must be a multiple of 32 in [32, 256]");
  HQ_CUDA(ctx, launch_mma_peak(pair, bn, chunks, ctx->num_sms, ctx->d_status, (cudaStream_t)stream, ops));
  ctx->launches += 1;
  return HQ_OK;
}

__attribute__((visibility("default"))) hq_status hq_dynamic_quant(hq_ctx* ctx, void* stream, const hq_op_desc* op, float* workspace, int8_t* Y, hq_range_state* yq) {
  if (!ctx) return HQ_ERR_INVALID_ARG;
  if (hq_status ds = check_device(ctx); ds != HQ_OK) return ds;
  if (!op || !workspace || !Y || !yq) return fail(ctx, HQ_ERR_INVALID_ARG, "null pointer argument");
  if (!aligned16(workspace) || !aligned16(Y)) return fail(ctx, HQ_ERR_ALIGNMENT, "workspace and Y must be 16-byte aligned");
  cudaStream_t s = (cudaStream_t)stream;
  hq_status st = run_op(ctx, s, op, workspace, yq, kOutF32);
  if (st != HQ_OK) return st;
  HQ_CUDA(ctx, launch_dynamic_derive(yq, s, ctx->overlap));
  HQ_CUDA(ctx, launch_quantize_pass(workspace, Y, op_out_elems(op), yq, ctx->num_sms, s, false));
  ctx->launches += 2;
  return HQ_OK;
}

__attribute__((visibility("default"))) hq_status hq_linear_wgrad(hq_ctx* ctx, void* stream, int32_t M, int32_t N, int32_t K, const int8_t* dY,
                                                                 const hq_range_state* dyq, const int8_t* X, const hq_range_state* xq, float* GW) {
  if (!ctx) return HQ_ERR_INVALID_ARG;
  if (hq_status ds = check_device(ctx); ds != HQ_OK) return ds;
  if (M <= 0 || N <= 0 || K <= 0) return fail(ctx, HQ_ERR_INVALID_ARG, "linear sizes must be positive");
  if (!dY || !dyq || !X || !xq || !GW) return fail(ctx, HQ_ERR_INVALID_ARG, "null pointer argument");
  if (!aligned16(dY) || !aligned16(X) || !aligned16(GW) || !aligned16(dyq) || !aligned16(xq))
    return fail(ctx, HQ_ERR_ALIGNMENT, "tensors and range states must be 16-byte aligned");
  // The accumulator, the column-sum correction and the per-row term are all added modulo 2^32 (the MMA is issued without
  // saturation), so a partial sum that leaves the int32 range does no harm as long as the gradient itself fits.
  if (M > (1 << 24)) return fail(ctx, HQ_ERR_UNSUPPORTED, "weight gradient over more than 2^24 rows (M = %d)", M);
  cudaStream_t s = (cudaStream_t)stream;
  // The reduction runs over the rows (the batch), so both operands are transposed first: A = dY^T [N][Mp] and
  // B = X^T [K][Mp] (Mp = M rounded up to 16, zero filled).  The layer kernel removes the zero point of its first
  // operand (dY) through the column sums of the second; the zero point of X costs one number per output row,
  // z_x * sum_m (dy - z_dy), which a small kernel prepares and the epilogue subtracts before the conversion to binary32.
  const int Mp = round_up(M, 16);
  const size_t a_bytes = ((size_t)N * Mp + 255) & ~(size_t)255, b_bytes = ((size_t)K * Mp + 255) & ~(size_t)255;
  const size_t t_bytes = ((size_t)N * sizeof(int32_t) + 255) & ~(size_t)255;
  const size_t need = a_bytes + b_bytes + t_bytes + 256;
  if (need > ctx->wgrad_bytes) {
    if (ctx->d_wgrad) HQ_CUDA(ctx, cudaFree(ctx->d_wgrad));
    ctx->d_wgrad = nullptr;
    ctx->wgrad_bytes = 0;
    HQ_CUDA(ctx, cudaMalloc((void**)&ctx->d_wgrad, need));
    ctx->wgrad_bytes = need;
  }
  int8_t* At = reinterpret_cast<int8_t*>(ctx->d_wgrad);
  int8_t* Bt = At + a_bytes;
  int32_t* terms = reinterpret_cast<int32_t*>(ctx->d_wgrad + a_bytes + b_bytes);
  hq_range_state* tmp = reinterpret_cast<hq_range_state*>(ctx->d_wgrad + a_bytes + b_bytes + t_bytes);
  HQ_CUDA(ctx, launch_transpose_rows(dY, At, M, N, Mp, 0, s));
  HQ_CUDA(ctx, launch_transpose_rows(X, Bt, M, K, Mp, 0, s));
  HQ_CUDA(ctx, launch_wgrad_row_terms(At, M, Mp, N, dyq, xq, terms, s));   // row sums of dY^T, from the transposed copy
  ctx->launches += 3;
  // GW[n][k] = fl(float(acc) * fl(s_dy * s_x)): the layer kernel's binary32 output mode; its "weight scale" is the scale of X
  const float* x_scale = reinterpret_cast<const float*>(reinterpret_cast<const char*>(xq) + offsetof(hq_range_state, scale));
  return run_linear(ctx, s, N, K, Mp, At, dyq, Bt, x_scale, nullptr, GW, tmp, kOutF32, terms);
}

}  // extern "C"

// Weight gradient of a dense stride-1 convolution without filter-window copies of the input.  Both tensors are packed
// channel-major over one padded pixel index m = (n * Hp + pad_h + h) * P + w (Hp = Ho + R - 1 rows per image, P = Wo rounded
// up to 16): dY once, X once per horizontal filter offset (shifted by it); a vertical offset is then a shift of the
// reduction index by a multiple of P, which a TMA coordinate can carry, and padding is zeros in both.  The GEMM is the
// layer kernel over slices of m (int32 slabs, as in the general form) with column tiles grouped by filter row: the tiles
// of filter row r read the same rows of the packed input at reduction offset (r - pad_h) * P.  The zero-point terms need
// sums over the output pixels whose tap lies inside the image; the packing kernels take them on the way.
// *done = false (and HQ_OK) when the shape is left to the general form.
static hq_status conv_wgrad_stride1(hq_ctx* ctx, cudaStream_t s, const hq_conv_desc& d, int Ho, int Wo, const int8_t* dY, const hq_range_state* dyq,
                                    const int8_t* X, const hq_range_state* xq, float* GW, bool* done) {
  *done = false;
  const int P = round_up(Wo, 16), Hp = Ho + d.R - 1, RS = d.R * d.S;
  if (d.stride_h != 1 || d.stride_w != 1 || d.R > 8 || d.S > 8 || RS > kMaxTaps || d.C % 16 != 0 || d.K % 4 != 0 || P > 256 || d.W > 256 ||
      d.pad_w > 16 || d.S - 1 - d.pad_w > 16 || d.pad_h >= d.R || d.pad_w >= d.S)
    return HQ_OK;
  const int brows = d.S * d.C;   // rows of the packed input: (horizontal offset, channel)
  int per_row = 0;               // column tiles per filter row: the fewest that divide brows into multiples of 16 of at most 256
  for (int t = 1; t <= brows / 16; ++t)
    if (brows % t == 0 && (brows / t) % 16 == 0 && brows / t <= 256) {
      per_row = t;
      break;
    }
  if (per_row == 0) return HQ_OK;
  const int rows = d.K, cols = RS * d.C;
  const int64_t Mv = (int64_t)d.N * Hp * P;   // padded reduction length
  if (Mv > (1 << 26)) return HQ_OK;
  const int tiles_one = ceil_div(rows, kTileM) * d.R * per_row;
  // one tile per SM, none left over for a second round: fewer slices also mean fewer slab bytes for the last pass
  const int want_slices = std::max(1, ctx->num_sms / tiles_one);
  const int slice_len = (int)std::max<int64_t>(128, round_up((int)ceil_div((int)Mv, want_slices), 128));
  const int slices = ceil_div((int)Mv, slice_len);
  const int64_t Mp = (int64_t)slices * slice_len;
  const size_t a_bytes = (size_t)rows * Mp, b_bytes = (size_t)brows * Mp;
  const size_t ab_bytes = (a_bytes + b_bytes + 255) & ~(size_t)255;
  const size_t slab_bytes = ((size_t)slices * rows * cols * sizeof(int32_t) + 255) & ~(size_t)255;
  const size_t sum_bytes = ((size_t)RS * (rows + d.C) * sizeof(int32_t) + 255) & ~(size_t)255;
  const size_t need = ab_bytes + slab_bytes + sum_bytes + 256;
  if (need > ctx->wgrad_bytes) {
    if (ctx->d_wgrad) HQ_CUDA(ctx, cudaFree(ctx->d_wgrad));
    ctx->d_wgrad = nullptr;
    ctx->wgrad_bytes = 0;
    HQ_CUDA(ctx, cudaMalloc((void**)&ctx->d_wgrad, need));
    ctx->wgrad_bytes = need;
  }
  int8_t* At = reinterpret_cast<int8_t*>(ctx->d_wgrad);
  int8_t* Bs = At + a_bytes;   // the same pitch: the rows of both lie back to back
  int32_t* slabs = reinterpret_cast<int32_t*>(ctx->d_wgrad + ab_bytes);
  int32_t* rowsum = reinterpret_cast<int32_t*>(ctx->d_wgrad + ab_bytes + slab_bytes);   // [tap][K]
  int32_t* colsum = rowsum + (size_t)RS * rows;                                         // [tap][C]
  hq_range_state* tmp = reinterpret_cast<hq_range_state*>(ctx->d_wgrad + ab_bytes + slab_bytes + sum_bytes);
  HQ_CUDA(ctx, cudaMemsetAsync(rowsum, 0, (size_t)RS * (rows + d.C) * sizeof(int32_t), s));
  // output pixels whose tap (r, s) lies inside the image: rows [pad_h - r, H + pad_h - r) and columns alike, cut to the output
  PackRanges ry{}, rx{};
  TapCounts mvalid{};
  ry.nr = rx.nr = d.R;
  ry.ns = rx.ns = d.S;
  for (int r = 0; r < d.R; ++r) {
    ry.row_lo[r] = (int16_t)std::max(0, d.pad_h - r);
    ry.row_hi[r] = (int16_t)std::min(Ho, d.H + d.pad_h - r);
    rx.row_lo[r] = (int16_t)std::max(0, r - d.pad_h);            // the input rows those outputs read through filter row r
    rx.row_hi[r] = (int16_t)std::min(d.H, Ho + r - d.pad_h);
  }
  for (int r = 0; r < d.R; ++r)
    for (int c = 0; c < d.S; ++c) {
      const int cols_in = std::max(0, std::min(Wo, d.W + d.pad_w - c) - std::max(0, d.pad_w - c));
      mvalid.v[r * d.S + c] = d.N * std::max(0, ry.row_hi[r] - ry.row_lo[r]) * cols_in;
    }
  // dY: views shifted by pad_w - s, summed over the first W columns (the pixels of the input row they pair with); X: views
  // shifted by s - pad_w, summed over the first Wo columns
  // the two packing kernels are independent: the smaller one (dY) runs on a side stream next to the other, forked from
  // and joined into the caller's stream with events (as the parity classes of a strided backward pass do)
  const bool side = ctx->parallel_subs && ctx->side[0] != nullptr;
  cudaStream_t s_dy = side ? ctx->side[0] : s;
  if (side) {
    HQ_CUDA(ctx, cudaEventRecord(ctx->ev_fork, s));
    HQ_CUDA(ctx, cudaStreamWaitEvent(s_dy, ctx->ev_fork, 0));
  }
  cudaError_t pe = launch_wgrad_pack(dY, At, d.N, Ho, Wo, d.K, Hp, P, d.pad_h, -1, d.pad_w, d.W, Mp, ry, rowsum, s_dy);
  const cudaError_t xe = launch_wgrad_pack(X, Bs, d.N, d.H, d.W, d.C, Hp, P, d.pad_h, +1, d.pad_w, Wo, Mp, rx, colsum, s);
  if (side) {   // joined whatever happened, so that the side stream never stays forked
    const cudaError_t re = cudaEventRecord(ctx->ev_join[0], s_dy);
    const cudaError_t we = re == cudaSuccess ? cudaStreamWaitEvent(s, ctx->ev_join[0], 0) : re;
    if (pe == cudaSuccess) pe = we;
  }
  HQ_CUDA(ctx, pe);
  HQ_CUDA(ctx, xe);
  HQ_CUDA(ctx, launch_zero_tail(At, rows + brows, Mp, Mv, s));
  ctx->launches += Mp > Mv ? 3 : 2;
  SubSpec sp{};
  sp.n_img = slices; sp.TH = 1; sp.TW = rows; sp.in_mul_h = 1; sp.in_mul_w = 1;
  sp.dh = {0}; sp.dw = {0}; sp.a_H = 1; sp.a_W = rows; sp.Cin = slice_len; sp.Nout = cols;
  sp.out_H = 1; sp.out_W = rows; sp.os_h = 1; sp.os_w = 1; sp.oa_h = 0; sp.oa_w = 0; sp.ldY = cols; sp.flat = true;
  sp.slices = slices; sp.slice_len = slice_len;
  hq_sub_problem sub;
  std::vector<uint8_t> rc, cc;
  MaskVec rm, cm;
  hq_status st = plan_sub_fixed(ctx, sp, sub, rc, cc, rm, cm, d.R * per_row, 0);
  if (st != HQ_OK) return st;
  if (sub.p.BN != brows / per_row || sub.p.tiles_col != d.R * per_row || sub.p.b_resident || sub.p.pair)
    return HQ_OK;   // not the tiling this form needs: the general form takes the layer
  sub.p.corr = nullptr;       // both zero points are taken out after the slabs are summed
  sub.p.zc_in_smem = 0;
  sub.p.zc_elems = 0;
  sub.p.Cpad = slice_len;
  sub.p.b_group_tiles = per_row;
  sub.p.b_k_base = -d.pad_h * P;
  sub.p.b_k_step = P;
  CUtensorMap ta, tb;
  {   // operand A: [rows][Mp] seen as (reduction byte within the slice, row, 1, slice)
    uint64_t dims[4] = {(uint64_t)slice_len, (uint64_t)rows, 1, (uint64_t)slices};
    uint64_t strides[3] = {(uint64_t)Mp, (uint64_t)Mp * rows, (uint64_t)slice_len};
    uint32_t box[4] = {(uint32_t)sub.p.BK, (uint32_t)sub.p.Wt, 1, 1};
    uint32_t es[4] = {1, 1, 1, 1};
    st = encode_map(ctx, &ta, At, 4, dims, strides, box, es, sub.p.swizzle64, false);
    if (st != HQ_OK) return st;
  }
  {   // operand B: [brows][Mp]; coordinates left of 0 and right of Mp read as zeros
    uint64_t dims[2] = {(uint64_t)Mp, (uint64_t)brows};
    uint64_t strides[1] = {(uint64_t)Mp};
    uint32_t box[2] = {(uint32_t)sub.p.BK, (uint32_t)sub.p.BN};
    uint32_t es[2] = {1, 1};
    st = encode_map(ctx, &tb, Bs, 2, dims, strides, box, es, sub.p.swizzle64, true);
    if (st != HQ_OK) return st;
  }
  const float* x_scale = reinterpret_cast<const float*>(reinterpret_cast<const char*>(xq) + offsetof(hq_range_state, scale));
  st = launch_sub(ctx, s, sub, ta, tb, dyq, x_scale, nullptr, slabs, tmp, kOutAcc);
  if (st != HQ_OK) return st;
  HQ_CUDA(ctx, launch_wgrad_reduce_taps(slabs, slices, rows, rows, cols, d.C, colsum, rowsum, mvalid, dyq, xq, GW, s));
  ctx->launches += 1;
  *done = true;
  return HQ_OK;
}

extern "C" {

__attribute__((visibility("default"))) hq_status hq_conv_wgrad(hq_ctx* ctx, void* stream, const hq_conv_desc* desc, const int8_t* dY,
                                                               const hq_range_state* dyq, const int8_t* X, const hq_range_state* xq, float* GW) {
  if (!ctx) return HQ_ERR_INVALID_ARG;
  if (hq_status ds = check_device(ctx); ds != HQ_OK) return ds;
  hq_status st = check_desc(ctx, desc);
  if (st != HQ_OK) return st;
  if (!dY || !dyq || !X || !xq || !GW) return fail(ctx, HQ_ERR_INVALID_ARG, "null pointer argument");
  if (!aligned16(dY) || !aligned16(X) || !aligned16(GW) || !aligned16(dyq) || !aligned16(xq))
    return fail(ctx, HQ_ERR_ALIGNMENT, "tensors and range states must be 16-byte aligned");
  const hq_conv_desc& d = *desc;
  cudaStream_t s = (cudaStream_t)stream;
  const int Ho = out_dim(d.H, d.pad_h, d.R, d.stride_h), Wo = out_dim(d.W, d.pad_w, d.S, d.stride_w);
  const int64_t M64 = (int64_t)d.N * Ho * Wo;
  if (d.groups != 1) {   // depthwise (check_desc admits groups == C == K only): a CUDA-core kernel, GW is [C][R][S]
    if (!(d.R == d.S && (d.R == 3 || d.R == 5))) return fail(ctx, HQ_ERR_UNSUPPORTED, "depthwise weight gradient: 3x3 and 5x5 filters only");
    if (d.C % 4 != 0 || d.C > 1024 || (size_t)d.C * d.R * d.S * sizeof(int32_t) > 48u * 1024u)
      return fail(ctx, HQ_ERR_UNSUPPORTED, "depthwise weight gradient needs C %% 4 == 0, C <= 1024 and C * R * S <= 12288");
    if (M64 > (1 << 30)) return fail(ctx, HQ_ERR_UNSUPPORTED, "weight gradient: too many output pixels");
    // 3x3, stride 1, padding 1: four pixels per dp4a on transposed words, zero points taken out from border sums
    if (d.R == 3 && d.S == 3 && d.stride_h == 1 && d.stride_w == 1 && d.pad_h == 1 && d.pad_w == 1 && d.C % 16 == 0 && d.C <= 256 &&
        d.H >= 2 && d.W >= 2 && ctx->wgrad_windows != 1) {
      DwWgradParams p{};
      p.N = d.N; p.H = d.H; p.W = d.W; p.C = d.C;
      const int cwords = d.C / 4;
      int cols4 = std::min(std::min(round_up(d.W, 4) / 4, 7), kDwColMaxThreads / cwords);
      for (;; --cols4) {   // the widest tile whose two buffers and sums fit
        p.TWt = 4 * std::max(cols4, 1);
        p.x_bytes = (uint32_t)d.C * (uint32_t)(p.TWt + 2) * (uint32_t)(kDwColRows + 2);
        p.dy_bytes = (uint32_t)d.C * (uint32_t)p.TWt * (uint32_t)kDwColRows;
        p.dy_offset = (p.x_bytes + 127u) & ~127u;
        p.buf_stride = p.dy_offset + ((p.dy_bytes + 127u) & ~127u);
        if (dw_wgrad3x3_smem_bytes(p) <= 200u * 1024u || cols4 <= 1) break;
      }
      p.tiles_h = ceil_div(d.H, kDwColRows);
      p.tiles_w = ceil_div(d.W, p.TWt);
      const int64_t n_tiles = (int64_t)d.N * p.tiles_h * p.tiles_w;
      if (cols4 >= 1 && cwords * (p.TWt / 4) >= 64 && n_tiles <= INT32_MAX && dw_wgrad3x3_smem_bytes(p) <= 200u * 1024u) {
        const size_t need = (size_t)kDwWgSlots * d.C * sizeof(int32_t) + 256;
        if (need > ctx->wgrad_bytes) {
          if (ctx->d_wgrad) HQ_CUDA(ctx, cudaFree(ctx->d_wgrad));
          ctx->d_wgrad = nullptr;
          ctx->wgrad_bytes = 0;
          HQ_CUDA(ctx, cudaMalloc((void**)&ctx->d_wgrad, need));
          ctx->wgrad_bytes = need;
        }
        p.sums = reinterpret_cast<int32_t*>(ctx->d_wgrad);
        p.status = ctx->d_status;
        HQ_CUDA(ctx, cudaMemsetAsync(p.sums, 0, (size_t)kDwWgSlots * d.C * sizeof(int32_t), s));
        CUtensorMap tx, ty;
        uint64_t dims[4] = {(uint64_t)d.C, (uint64_t)d.W, (uint64_t)d.H, (uint64_t)d.N};
        uint64_t strides[3] = {(uint64_t)d.C, (uint64_t)d.C * d.W, (uint64_t)d.C * d.W * d.H};
        uint32_t es[4] = {1, 1, 1, 1};
        uint32_t box_x[4] = {(uint32_t)d.C, (uint32_t)(p.TWt + 2), (uint32_t)(kDwColRows + 2), 1u};
        uint32_t box_y[4] = {(uint32_t)d.C, (uint32_t)p.TWt, (uint32_t)kDwColRows, 1u};
        CUresult r1 = ctx->encode(&tx, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<int8_t*>(X), dims, strides, box_x, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                  CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        CUresult r2 = ctx->encode(&ty, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<int8_t*>(dY), dims, strides, box_y, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                  CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r1 != CUDA_SUCCESS || r2 != CUDA_SUCCESS) return fail(ctx, HQ_ERR_CUDA, "tensor map encoding failed (CUresult %d, %d)", (int)r1, (int)r2);
        HQ_CUDA(ctx, launch_dw_wgrad3x3(p, tx, ty, ctx->num_sms, dyq, xq, GW, s));
        ctx->launches += 3;
        return HQ_OK;
      }
    }
    const size_t need = (size_t)d.C * d.R * d.S * sizeof(int32_t) + 256;
    if (need > ctx->wgrad_bytes) {
      if (ctx->d_wgrad) HQ_CUDA(ctx, cudaFree(ctx->d_wgrad));
      ctx->d_wgrad = nullptr;
      ctx->wgrad_bytes = 0;
      HQ_CUDA(ctx, cudaMalloc((void**)&ctx->d_wgrad, need));
      ctx->wgrad_bytes = need;
    }
    int32_t* acc = reinterpret_cast<int32_t*>(ctx->d_wgrad);
    HQ_CUDA(ctx, cudaMemsetAsync(acc, 0, (size_t)d.C * d.R * d.S * sizeof(int32_t), s));
    HQ_CUDA(ctx, launch_dw_wgrad(dY, X, dyq, xq, d, Ho, Wo, ctx->num_sms, make_fastdiv(Wo), make_fastdiv(Ho), acc, GW, s));
    ctx->launches += 2;
    return HQ_OK;
  }
  const int64_t cols64 = (int64_t)d.R * d.S * d.C;
  if (M64 > (1 << 24) || cols64 > (1 << 20)) return fail(ctx, HQ_ERR_UNSUPPORTED, "weight gradient: too many output pixels or filter elements");
  if (ctx->wgrad_windows != 1) {
    bool done = false;
    st = conv_wgrad_stride1(ctx, s, d, Ho, Wo, dY, dyq, X, xq, GW, &done);
    if (st != HQ_OK || done) return st;
  }
  const int M = (int)M64, rows = d.K, cols = (int)cols64;
  // G_W as one GEMM over the output pixels m: rows k (dY^T [K][M]) x columns (r,s,c) (the filter windows of X,
  // transposed: Bt [(r,s,c)][M]).  The output is as small as the weights while the reduction is long, so the reduction is
  // cut into slices that run as the "images" of the layer kernel's tile space, each into an int32 slab of its own; a last
  // pass sums the slabs, takes out both zero points and converts.  Slice length: a multiple of 128 bytes that gives the
  // SMs about two tiles each.
  const int tiles_one = ceil_div(rows, kTileM) * ceil_div(cols, 256);
  int want_slices = std::max(1, (2 * ctx->num_sms + tiles_one - 1) / tiles_one);
  int slice_len = std::max(128, round_up(ceil_div(M, want_slices), 128));
  const int slices = ceil_div(M, slice_len);
  const int64_t Mp = (int64_t)slices * slice_len;
  const size_t a_bytes = ((size_t)rows * Mp + 255) & ~(size_t)255, b_bytes = ((size_t)cols * Mp + 255) & ~(size_t)255;
  const size_t slab_bytes = ((size_t)slices * rows * cols * sizeof(int32_t) + 255) & ~(size_t)255;
  const size_t sum_bytes = (((size_t)rows + cols) * sizeof(int32_t) + 255) & ~(size_t)255;
  const size_t need = a_bytes + b_bytes + slab_bytes + sum_bytes + 256;
  if (need > ctx->wgrad_bytes) {
    if (ctx->d_wgrad) HQ_CUDA(ctx, cudaFree(ctx->d_wgrad));
    ctx->d_wgrad = nullptr;
    ctx->wgrad_bytes = 0;
    HQ_CUDA(ctx, cudaMalloc((void**)&ctx->d_wgrad, need));
    ctx->wgrad_bytes = need;
  }
  int8_t* At = reinterpret_cast<int8_t*>(ctx->d_wgrad);
  int8_t* Bt = At + a_bytes;
  int32_t* slabs = reinterpret_cast<int32_t*>(ctx->d_wgrad + a_bytes + b_bytes);
  int32_t* rowsum = reinterpret_cast<int32_t*>(ctx->d_wgrad + a_bytes + b_bytes + slab_bytes);
  int32_t* colsum = rowsum + rows;
  hq_range_state* tmp = reinterpret_cast<hq_range_state*>(ctx->d_wgrad + a_bytes + b_bytes + slab_bytes + sum_bytes);
  if (Mp > INT32_MAX) return fail(ctx, HQ_ERR_UNSUPPORTED, "weight gradient: too many output pixels");
  // row sums of both operands (for the zero points), accumulated with integer atomics by the kernels that read the data anyway
  HQ_CUDA(ctx, cudaMemsetAsync(rowsum, 0, ((size_t)rows + cols) * sizeof(int32_t), s));
  {   // dY^T and its row sums: the same kernel, dY taken as the input of a 1x1 stride-1 layer (no padding, so no zero point is used)
    hq_conv_desc t{};
    t.N = d.N; t.H = Ho; t.W = Wo; t.C = d.K; t.K = d.K; t.R = 1; t.S = 1; t.stride_h = 1; t.stride_w = 1; t.pad_h = 0; t.pad_w = 0; t.groups = 1;
    HQ_CUDA(ctx, launch_im2col_t(dY, At, dyq, t, Ho, Wo, Mp, rowsum, make_fastdiv(Wo), make_fastdiv(Ho), s));
  }
  HQ_CUDA(ctx, launch_im2col_t(X, Bt, xq, d, Ho, Wo, Mp, colsum, make_fastdiv(Wo), make_fastdiv(Ho), s));
  ctx->launches += 2;
  SubSpec sp{};
  sp.n_img = slices; sp.TH = 1; sp.TW = rows; sp.in_mul_h = 1; sp.in_mul_w = 1;
  sp.dh = {0}; sp.dw = {0}; sp.a_H = 1; sp.a_W = rows; sp.Cin = slice_len; sp.Nout = cols;
  sp.out_H = 1; sp.out_W = rows; sp.os_h = 1; sp.os_w = 1; sp.oa_h = 0; sp.oa_w = 0; sp.ldY = cols; sp.flat = true;
  sp.slices = slices; sp.slice_len = slice_len;
  hq_sub_problem sub;
  std::vector<uint8_t> rc, cc;
  MaskVec rm, cm;
  st = plan_sub(ctx, sp, sub, rc, cc, rm, cm);
  if (st != HQ_OK) return st;
  sub.p.corr = nullptr;       // both zero points are taken out after the slabs are summed
  sub.p.zc_in_smem = 0;       // no correction table: nothing to copy into shared memory
  sub.p.zc_elems = 0;
  sub.p.Cpad = slice_len;
  CUtensorMap ta, tb;
  {   // operand A: [rows][Mp] seen as (reduction byte within the slice, row, 1, slice)
    uint64_t dims[4] = {(uint64_t)slice_len, (uint64_t)rows, 1, (uint64_t)slices};
    uint64_t strides[3] = {(uint64_t)Mp, (uint64_t)Mp * rows, (uint64_t)slice_len};
    uint32_t box[4] = {(uint32_t)sub.p.BK, (uint32_t)sub.p.Wt, 1, 1};
    uint32_t es[4] = {1, 1, 1, 1};
    st = encode_map(ctx, &ta, At, 4, dims, strides, box, es, sub.p.swizzle64, false);
    if (st != HQ_OK) return st;
  }
  st = encode_b(ctx, sub, Bt, Mp, &tb);
  if (st != HQ_OK) return st;
  const float* x_scale = reinterpret_cast<const float*>(reinterpret_cast<const char*>(xq) + offsetof(hq_range_state, scale));
  st = launch_sub(ctx, s, sub, ta, tb, dyq, x_scale, nullptr, slabs, tmp, kOutAcc);
  if (st != HQ_OK) return st;
  HQ_CUDA(ctx, launch_wgrad_reduce(slabs, slices, rows, cols, colsum, rowsum, M, dyq, xq, GW, s));
  ctx->launches += 1;
  return HQ_OK;
}

__attribute__((visibility("default"))) hq_status hq_debug_accumulate(hq_ctx* ctx, void* stream, const hq_op_desc* op, int32_t* acc, hq_range_state* yq) {
  if (!ctx) return HQ_ERR_INVALID_ARG;
  if (hq_status ds = check_device(ctx); ds != HQ_OK) return ds;
  if (!op || !acc || !yq) return fail(ctx, HQ_ERR_INVALID_ARG, "null pointer argument");
  return run_op(ctx, (cudaStream_t)stream, op, acc, yq, kOutAcc);
}

}  // extern "C"

// ---- dynamic quantization without any allocation ------------------------------------------------
// Some callers cannot allocate device memory around a call: allocator or profiler callbacks,
// latency-critical loops that must stay out of the allocator (cudaMalloc / cudaFree synchronise the
// device), or embedders whose memory budget is fixed at start-up.  For them the binary32 workspace of the dynamic path lives in this file-scope device
// array.  In host code the array's name is only a stand-in; the device address is looked up once
// per device with cudaGetSymbolAddress and handed to the kernels.
static __device__ __align__(256) float hq_static_workspace[HQ_STATIC_WORKSPACE_ELEMS];

namespace {
constexpr int kMaxDevices = 64;
// Written without a lock: two host threads that make the first call on a device at the same time both store the same
// address (the symbol's address on that device never changes), so the race is benign.
float* g_static_ws[kMaxDevices] = {};

hq_status static_workspace(hq_ctx* ctx, float** out) {
  int cur = -1;
  HQ_CUDA(ctx, cudaGetDevice(&cur));
  if (cur != ctx->device) return fail(ctx, HQ_ERR_INVALID_ARG, "device %d must be current (device %d is)", ctx->device, cur);
  if (cur < 0 || cur >= kMaxDevices) return fail(ctx, HQ_ERR_UNSUPPORTED, "device index %d out of range", cur);
  if (g_static_ws[cur] == nullptr) {
    void* p = nullptr;
    HQ_CUDA(ctx, cudaGetSymbolAddress(&p, hq_static_workspace));
    g_static_ws[cur] = static_cast<float*>(p);
  }
  *out = g_static_ws[cur];
  return HQ_OK;
}
}  // namespace

extern "C" __attribute__((visibility("default"))) hq_status hq_dynamic_quant_static(hq_ctx* ctx, void* stream, const hq_op_desc* op, int8_t* Y,
                                                                                   hq_range_state* yq) {
  if (!ctx) return HQ_ERR_INVALID_ARG;
  if (!op || !Y || !yq) return fail(ctx, HQ_ERR_INVALID_ARG, "null pointer argument");
  if (op->kind != HQ_OP_LINEAR && op->kind != HQ_OP_CONV_FWD && op->kind != HQ_OP_CONV_BWD_DATA)
    return fail(ctx, HQ_ERR_INVALID_ARG, "unknown operation kind %d", op->kind);
  if (op->kind != HQ_OP_LINEAR) {
    hq_status st = check_desc(ctx, op->conv);
    if (st != HQ_OK) return st;
  } else if (op->M <= 0 || op->N <= 0 || op->K <= 0) {
    return fail(ctx, HQ_ERR_INVALID_ARG, "linear sizes must be positive");
  }
  const int64_t elems = op_out_elems(op);
  if (elems > (int64_t)HQ_STATIC_WORKSPACE_ELEMS)
    return fail(ctx, HQ_ERR_UNSUPPORTED, "output has %lld elements; the built-in workspace holds at most %lld", (long long)elems,
                (long long)HQ_STATIC_WORKSPACE_ELEMS);
  if (!aligned16(Y)) return fail(ctx, HQ_ERR_ALIGNMENT, "Y must be 16-byte aligned");
  float* ws = nullptr;
  hq_status st = static_workspace(ctx, &ws);
  if (st != HQ_OK) return st;
  cudaStream_t s = (cudaStream_t)stream;
  // the planner decides what the layer needs; with no_grow it refuses, before any launch, whatever the context's scratch
  // (column sums of a linear layer's weights, padded operand copies) cannot hold as it stands
  st = run_op(ctx, s, op, ws, yq, kOutF32, true);
  if (st != HQ_OK) return st;
  HQ_CUDA(ctx, launch_dynamic_derive(yq, s, ctx->overlap));
  HQ_CUDA(ctx, launch_quantize_pass(ws, Y, elems, yq, ctx->num_sms, s, false));
  ctx->launches += 2;
  return HQ_OK;
}
