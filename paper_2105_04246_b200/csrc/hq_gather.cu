// Forward convolution with a spatial filter over FEW input channels (the RGB stem of a network: 7x7, stride 2, 3 -> 64),
// fused: no repacked copy of the input ever reaches global memory (arxiv 2105.04246, Sec. 3.1: the 8-bit input is brought
// to the MAC array in slices; Sec. 3.2 / Sec. 4: the accumulator output is quantized directly and min/max are taken there).
//
// For such layers the channel run of one pixel (3 bytes) is far below anything a TMA box or a 32-byte MMA step can
// address, but for a fixed filter row r the S*C input bytes under the filter are contiguous in NHWC.  One CTA per SM
// walks over tiles of up to 128 consecutive output pixels of one output row:
//   warp 0        copies the R input rows the tile touches into shared memory with ONE TMA box (rows above / below the
//                 image and the horizontal margins arrive as zeros);
//   warps 2..5    one thread per output pixel: gathers its R runs of S*C bytes from the raw rows (aligned word loads +
//                 funnel shifts), concatenated in the weights' own (r, s, c) order and zero padded to a multiple of 32 bytes,
//                 and writes that im2col row into the operand tile the tensor core reads (K-major, no swizzle: 8 x 16-byte
//                 core matrices);
//   warp 1        issues the int8 MMAs (tcgen05 kind::i8, accumulators in TMEM) against the weight matrix, which stays
//                 resident in shared memory;
//   warps 10..21  the requantization + min/max epilogue, the same arithmetic as the other layer kernels.
// Zero-filled taps are settled by the border-class correction z_x * (sum of the in-image weights), as everywhere else.
// Every wait is bounded (mbar_wait).
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <type_traits>

#include "hq_device.cuh"
#include "hq_internal.h"
#include "hq_quant.cuh"
#include "hq_tc.cuh"

namespace hq {
namespace {

// A gather warp works through a long dependent instruction stream per tile (shared-memory loads, shifts, stores), so one
// set of four warps cannot keep up with the tensor core and the epilogue: two sets take alternate tiles.  The epilogue
// warps form up to three groups of four (one warp per TMEM lane quarter) that take tiles in turn.
constexpr int kGatherSets = 2;
constexpr int kGatherWarps = 4 * kGatherSets;   // a set = 128 pixels, one per thread
constexpr int kGatherFirstWarp = 2;
constexpr int kGatherEpiFirstWarp = kGatherFirstWarp + kGatherWarps;
constexpr int kGatherEpiWarps = 12;
constexpr int kGatherThreads = 32 * (kGatherEpiFirstWarp + kGatherEpiWarps);   // 704
constexpr int kGatherMaxStages = 8;

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
               "l"((uint64_t)map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
               : "memory");
}
__device__ __forceinline__ uint32_t lds32(uint32_t saddr) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(saddr));
  return v;
}
__device__ __forceinline__ void sts128(uint32_t saddr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(saddr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// The im2col row of one output pixel: R runs of SC bytes, run r read from raw row r at byte offset src0, written to the
// row at byte r * SC.  Source and destination alignments differ by a per-pixel amount, so every destination word is a
// funnel shift of two aligned source words; the first and last word of a run are merged with their neighbours' bytes.
// The loads of run r + 1 are issued before the shifts of run r, so a thread waits for shared memory once per row, not
// once per word.
template <int SC>
struct RunWords {
  static constexpr int kMax = (SC + 3) / 4 + 2;   // destination words a run can touch, plus the look-ahead word
  uint32_t w[kMax];
  uint32_t sh;
};
template <int R, int SC, int r>
__device__ __forceinline__ void load_run(uint32_t raw_stage, uint32_t raw_pitch, uint32_t src0, RunWords<SC>& L) {
  constexpr int d0 = r * SC;
  constexpr int nw = ((d0 + SC - 1) >> 2) - (d0 >> 2) + 1;
  const uint32_t t = raw_stage + (uint32_t)r * raw_pitch + src0 - (uint32_t)(d0 & 3);   // its word stream lines up with word d0 / 4
  const uint32_t wb = t & ~3u;
  L.sh = (t & 3u) * 8u;
#pragma unroll
  for (int k = 0; k <= nw; ++k) L.w[k] = lds32(wb + 4u * (uint32_t)k);
}
template <int R, int SC, int r>
__device__ __forceinline__ void place_run(const RunWords<SC>& L, uint32_t (&D)[((R * SC + 31) / 32) * 8]) {
  constexpr int d0 = r * SC;
  constexpr int j0 = d0 >> 2, nw = ((d0 + SC - 1) >> 2) - j0 + 1;
#pragma unroll
  for (int k = 0; k < nw; ++k) {
    const uint32_t v = __funnelshift_r(L.w[k], L.w[k + 1], L.sh);
    uint32_t mask = 0xFFFFFFFFu;
    if (k == 0) mask &= 0xFFFFFFFFu << (8 * (d0 & 3));
    if (k == nw - 1) mask &= 0xFFFFFFFFu >> (8 * (3 - ((d0 + SC - 1) & 3)));
    if (mask == 0xFFFFFFFFu) D[j0 + k] = v;      // a word this run owns alone
    else D[j0 + k] |= v & mask;
  }
}
template <int R, int SC, int r>
__device__ __forceinline__ void gather_runs(uint32_t raw_stage, uint32_t raw_pitch, uint32_t src0, RunWords<SC>& cur, RunWords<SC>& nxt,
                                            uint32_t (&D)[((R * SC + 31) / 32) * 8]) {
  if constexpr (r < R) {
    if constexpr (r + 1 < R) load_run<R, SC, r + 1>(raw_stage, raw_pitch, src0, nxt);
    place_run<R, SC, r>(cur, D);
    gather_runs<R, SC, r + 1>(raw_stage, raw_pitch, src0, nxt, cur, D);
  }
}
template <int R, int SC>
__device__ __forceinline__ void gather_row(uint32_t raw_stage, uint32_t raw_pitch, uint32_t src0, uint32_t (&D)[((R * SC + 31) / 32) * 8]) {
  constexpr int KW = ((R * SC + 31) / 32) * 8;
#pragma unroll
  for (int j = 0; j < KW; ++j) D[j] = 0u;
  RunWords<SC> a, b;
  load_run<R, SC, 0>(raw_stage, raw_pitch, src0, a);
  gather_runs<R, SC, 0>(raw_stage, raw_pitch, src0, a, b, D);
}

template <int kOut, int R, int SC>
__global__ void __launch_bounds__(kGatherThreads, 1) hq_gather_conv_kernel(const __grid_constant__ GatherParams p, const __grid_constant__ CUtensorMap tmap) {
  constexpr int Kp = ((R * SC + 31) / 32) * 32;
  constexpr int KW = Kp / 4, KPIECES = Kp / 16, KSTEPS = Kp / 32;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[4 * kGatherMaxStages + 16];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag_s;
  __shared__ int red_min[kEpilogueWarps], red_max[kEpilogueWarps];
  __shared__ uint8_t cls_s[1024];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &abort_flag_s;
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* const base_gen = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t w_s = base + p.off_w, raw_s = base + p.off_raw, a_s = base + p.off_a;
  int32_t* const zc_s = reinterpret_cast<int32_t*>(base_gen + p.off_zc);
  const uint32_t bar0 = smem_u32(bars);
  auto raw_full = [&](int s) { return bar0 + 8u * s; };
  auto raw_empty = [&](int s) { return bar0 + 8u * (kGatherMaxStages + s); };
  auto a_full = [&](int s) { return bar0 + 8u * (2 * kGatherMaxStages + s); };
  auto a_empty = [&](int s) { return bar0 + 8u * (3 * kGatherMaxStages + s); };
  auto tfull_bar = [&](int b) { return bar0 + 8u * (4 * kGatherMaxStages + b); };
  auto tempty_bar = [&](int b) { return bar0 + 8u * (4 * kGatherMaxStages + 8 + b); };
  const int nbuf = p.tmem_bufs, ngroups = p.epi_groups;

  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    for (int s = 0; s < p.stages_raw; ++s) {
      mbar_init(raw_full(s), 1);
      mbar_init(raw_empty(s), 4);
    }
    for (int s = 0; s < p.stages_a; ++s) {
      mbar_init(a_full(s), 4);
      mbar_init(a_empty(s), 1);
    }
    for (int b = 0; b < nbuf; ++b) {
      mbar_init(tfull_bar(b), 1);
      mbar_init(tempty_bar(b), 4);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&tmap) : "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(p.tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;

  // divisions by launch constants: multiplier and shift prepared on the host; the buffer and group counts are powers of two
  // span = 0: tile -> image n, output row ho, first output column wo0.  span = 1 (tiles run across the ends of short output
  // rows): image n, wo0 = row-major index of the tile's first pixel in the image, ho = the output row that pixel lies in.
  const int span = p.span;
  const int HW = p.Ho * p.Wo;
  auto decode = [&](int tile, int& n, int& ho, int& wo0) {
    if (span) {
      n = fdiv(tile, p.fd_tiles_img);
      wo0 = (tile - n * p.tiles_img) * kTileM;
      ho = fdiv(wo0, p.fd_Wo);
      return;
    }
    const int t2 = fdiv(tile, p.fd_tiles_w);
    wo0 = (tile - t2 * p.tiles_w) * kTileM;
    n = fdiv(t2, p.fd_Ho);
    ho = t2 - n * p.Ho;
  };
  const int nbuf_log2 = p.tmem_bufs_log2;
  // first byte (in the image row) of the tile's raw box: the leftmost filter tap of its first pixel, rounded down to 16
  auto box_start = [&](int wo0) { return ((wo0 * p.stride_w - p.pad_w) * p.C) & ~15; };   // arithmetic on negative values: & rounds towards -inf

  __shared__ int fin_s[2];    // the raw-row producer's ring position when it stopped (see the end of the kernel)
  if (warp == 0) {
    // ------------------------------ raw rows: one TMA box per tile ------------------------------
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int it = 0; ok; ++it) {
      const int tile = (int)blockIdx.x + it * (int)gridDim.x;
      if (tile >= p.num_tiles) break;
      int n, ho, wo0;
      decode(tile, n, ho, wo0);
      if (it == 0) grid_dependency_wait();   // the input may come from the previous kernel in the stream
      ok = warp_wait(raw_empty(stage), phase ^ 1u, abort_flag, p.status, kAsyncProducerEmptyWait, 8000u);
      if (!ok) break;
      if (elect_one()) {
        mbar_expect_tx(raw_full(stage), p.raw_box_bytes);
        tma_load_3d(raw_s + stage * p.raw_stage_stride, &tmap, box_start(span ? 0 : wo0) >> 2, ho * p.stride_h - p.pad_h, n, raw_full(stage));
      }
      if (++stage == p.stages_raw) {
        stage = 0;
        phase ^= 1u;
      }
    }
    if (lane == 0) {   // where the ring stands, for the drain of a CTA that gave up
      fin_s[0] = stage;
      fin_s[1] = (int)phase;
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    grid_dependency_wait();
    // the weights are written to shared memory by the gather warps before their first tile; their first a_full arrival
    // comes after that (and after the fence that makes generic-proxy writes visible to the tensor core)
    for (int it = 0; ok; ++it) {
      const int tile = (int)blockIdx.x + it * (int)gridDim.x;
      if (tile >= p.num_tiles) break;
      const int buf = it & (nbuf - 1);
      const uint32_t tph = (uint32_t)(it >> nbuf_log2) & 1u;
      // the rings on both sides are several tiles deep, so none of these waits is latency critical: long pauses between
      // polls keep the waiting warps out of the issue slots the epilogue and gather warps need
      ok = warp_wait(tempty_bar(buf), tph ^ 1u, abort_flag, p.status, kAsyncMmaTmemEmptyWait, 2000u);
      if (!ok) break;
      ok = warp_wait(a_full(stage), phase, abort_flag, p.status, kAsyncMmaFullWait, 1000u);
      if (!ok) break;
      tc_fence_after();
      const uint32_t d_tmem = tmem_base + buf * p.tmem_buf_stride;
      const uint32_t a0 = a_s + stage * p.a_stage_bytes;
      if (elect_one()) {
#pragma unroll
        for (int k = 0; k < KSTEPS; ++k) {
          const uint64_t adesc = make_smem_desc_plain(a0 + (uint32_t)(2 * k) * (kTileM * 16u), kTileM * 16u, 128u);
          const uint64_t bdesc = make_smem_desc_plain(w_s + (uint32_t)(2 * k) * ((uint32_t)p.BN * 16u), (uint32_t)p.BN * 16u, 128u);
          umma_i8(d_tmem, adesc, bdesc, p.idesc, k == 0 ? 0u : 1u);
        }
        umma_commit(a_empty(stage));
        umma_commit(tfull_bar(buf));
      }
      __syncwarp();
      if (++stage == p.stages_a) {
        stage = 0;
        phase ^= 1u;
      }
    }
    __syncwarp();
    grid_launch_dependents();
  } else if (warp < kGatherEpiFirstWarp) {
    // ------------------------------ gather: raw rows -> im2col operand tile ------------------------------
    const int gset = (warp - kGatherFirstWarp) >> 2;                              // which set: tiles gset, gset + kGatherSets, ...
    const int gt = ((int)threadIdx.x - kGatherFirstWarp * 32) & 127;             // pixel of the tile
    const int gall = (int)threadIdx.x - kGatherFirstWarp * 32;
    if (!p.weights_early) grid_dependency_wait();
    {   // weight matrix [BN][Kp] (global, zero padded) -> core-matrix layout: piece q of row n at q * BN*16 + n * 16
      const uint4* wsrc = reinterpret_cast<const uint4*>(p.wmat);
      for (int i = gall; i < p.BN * KPIECES; i += kGatherWarps * 32) {
        const int n = i / KPIECES, q = i - n * KPIECES;
        const uint4 v = wsrc[i];
        sts128(w_s + (uint32_t)q * ((uint32_t)p.BN * 16u) + (uint32_t)n * 16u, v.x, v.y, v.z, v.w);
      }
    }
    if (p.weights_early) grid_dependency_wait();
    // the weights must be in place before the first MMA: every gather warp's first arrival on an a_full barrier follows its
    // own weight writes, and the issuer's second tile needs the other set's arrival as well, so a named barrier joins the sets
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("bar.sync 2, %0;" ::"r"(kGatherWarps * 32) : "memory");
    // ring positions are global over the CTA's tiles; this set starts at tile `gset` and steps over the other set's tiles
    int rs = gset % p.stages_raw, as = gset % p.stages_a;
    uint32_t rph = (uint32_t)(gset / p.stages_raw) & 1u, aph = (uint32_t)(gset / p.stages_a) & 1u;
    bool ok = true;
    for (int it = gset; ok; it += kGatherSets) {
      const int tile = (int)blockIdx.x + it * (int)gridDim.x;
      if (tile >= p.num_tiles) break;
      int n, ho, wo0;
      decode(tile, n, ho, wo0);
      ok = warp_wait(raw_full(rs), rph, abort_flag, p.status, kAsyncMmaFullWait, 2000u);
      if (!ok) break;
      uint32_t D[KW];
      uint32_t src0;
      if (span) {   // pixels beyond the image's end gather the last pixel's runs, their results are dropped
        const int f = min(wo0 + gt, HW - 1);
        const int fh = fdiv(f, p.fd_Wo);
        src0 = (uint32_t)((fh - ho) * p.stride_h) * p.raw_pitch + (uint32_t)(((f - fh * p.Wo) * p.stride_w - p.pad_w) * p.C - box_start(0));
      } else {
        src0 = (uint32_t)(((wo0 + gt) * p.stride_w - p.pad_w) * p.C - box_start(wo0));
      }
      // pixels beyond the row's end gather from inside the box as well (clamped), their results are dropped
      const uint32_t src0c = span ? src0 : min(src0, p.raw_pitch - (uint32_t)SC - 4u);
      gather_row<R, SC>(raw_s + rs * p.raw_stage_stride, p.raw_pitch, src0c, D);
      ok = warp_wait(a_empty(as), aph ^ 1u, abort_flag, p.status, kAsyncProducerEmptyWait, 4000u);
      if (!ok) break;
      const uint32_t dst = a_s + as * p.a_stage_bytes + (uint32_t)(gt >> 3) * 128u + (uint32_t)(gt & 7) * 16u;
#pragma unroll
      for (int q = 0; q < KPIECES; ++q) sts128(dst + (uint32_t)q * (kTileM * 16u), D[4 * q], D[4 * q + 1], D[4 * q + 2], D[4 * q + 3]);
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // these writes are read by the tensor core (async proxy)
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(a_full(as));
        mbar_arrive(raw_empty(rs));
      }
      rs += kGatherSets;
      while (rs >= p.stages_raw) {
        rs -= p.stages_raw;
        rph ^= 1u;
      }
      as += kGatherSets;
      while (as >= p.stages_a) {
        as -= p.stages_a;
        aph ^= 1u;
      }
    }
    __syncwarp();
  } else {
    // ------------------------------ epilogue ------------------------------
    const int quarter = warp & 3;
    const int ew = warp - kGatherEpiFirstWarp;
    const int et = (int)threadIdx.x - kGatherEpiFirstWarp * 32;
    constexpr int kEpiThreads = kGatherEpiWarps * 32;
    const int group = ew >> 2;               // warps beyond the groups in use only help with the tables
    const int row = quarter * 32 + lane;
    grid_dependency_wait();
    QParams q;
    q.s_acc = __fmul_rn(p.xq->scale, *p.w_scale);
    q.zx = p.xq->zero_point;
    q.inv_scale = (kOut == kOutInt8) ? p.yq->inv_scale : 1.0f;
    q.zp = (kOut == kOutInt8) ? p.yq->zero_point : 0;
    qparams_finish(q);
    qparams_bound(q, p.acc_bound);
    if (kOut == kOutInt8) qparams_output_mode(q, p.yq->rounding, p.yq->seed, p.yq->step);
    if (blockIdx.x == 0 && et == 0) p.yq->acc_scale = q.s_acc;
    for (int i = et; i < p.zc_elems; i += kEpiThreads) zc_s[i] = q.zx * p.corr[i];
    if (p.cls_in_smem) {   // Ho, Wo <= 512
      for (int i = et; i < p.Ho; i += kEpiThreads) cls_s[i] = p.rowcls[i];
      for (int i = et; i < p.Wo; i += kEpiThreads) cls_s[512 + i] = p.colcls[i];
    }
    asm volatile("bar.sync 1, %0;" ::"r"(kEpiThreads) : "memory");
    int mn = INT32_MAX, mx = INT32_MIN;
    int sat_below = 0, sat_above = 0;
    const int c_begin = 0, c_end = p.BN / 16;   // a warp drains all columns of its 32 rows
    const QPacked qk = qpacked(q);
    const bool lean = kOut == kOutInt8 && q.fast && !q.count_sat;
    // 32-byte stores of the 4-byte output forms where every output row starts on a 32-byte boundary
    const bool base32 = (reinterpret_cast<uintptr_t>(p.out) & 31u) == 0;
    [[maybe_unused]] const bool wide32 = base32 && (p.BN & 7) == 0;
    // The tile loop, instantiated per epilogue variant (kMode >= 0: straight-line int8 pass with that rounding; -1: the
    // general pass), so that the loop a warp actually runs holds one variant's code only.
    auto run_tiles = [&](auto mode_tag) {
      constexpr int kMode = decltype(mode_tag)::value;
      for (int it = group; group < ngroups; it += ngroups) {
        const int tile = (int)blockIdx.x + it * (int)gridDim.x;
        if (tile >= p.num_tiles) break;
        int n, ho, wo0;
        decode(tile, n, ho, wo0);
        int wo = wo0 + row;
        bool row_valid = wo < p.Wo;
        if (span) {
          row_valid = wo < HW;
          const int f = min(wo, HW - 1);
          ho = fdiv(f, p.fd_Wo);
          wo = f - ho * p.Wo;
        }
        const int64_t pix = ((int64_t)n * p.Ho + ho) * p.Wo + wo;
        int zoff = 0;
        if (row_valid) {
          const int rc = p.cls_in_smem ? cls_s[ho] : p.rowcls[ho];
          const int cc = p.cls_in_smem ? cls_s[512 + wo] : p.colcls[wo];
          zoff = (rc * p.ncolcls + cc) * p.corr_ld;
        }
        const int32_t* zrow = zc_s + zoff;
        const int buf = it & (nbuf - 1);
        const uint32_t tph = (uint32_t)(it >> nbuf_log2) & 1u;
        int w = 1;
        if (lane == 0) w = mbar_wait(tfull_bar(buf), tph, abort_flag, p.status, kAsyncEpilogueTmemFullWait, 2000u) ? 1 : 0;
        w = __shfl_sync(0xffffffffu, w, 0);
        if (!w) break;
        tc_fence_after();
        const uint32_t taddr = tmem_base + buf * p.tmem_buf_stride + ((uint32_t)(quarter * 32) << 16);
        if constexpr (kMode >= 0) {
          int8_t* dst_row = reinterpret_cast<int8_t*>(p.out) + pix * p.BN;
          const int64_t elem_row = pix * p.BN;
          int tmn = INT32_MAX, tmx = INT32_MIN;
          // sixteen columns per load, two register sets: the next load is in flight while a set is processed
          int va[16], vb[16];
          tmem_ld16r(taddr, va);
          auto pass16 = [&](int (&v)[16], int c0, uint32_t* wd) {
            int lo[8], hi[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              lo[e] = v[e];
              hi[e] = v[8 + e];
            }
            lean_half8m<kMode>(lo, zrow + c0, tmn, tmx, q, qk, elem_row + c0, wd[0], wd[1]);
            lean_half8m<kMode>(hi, zrow + c0 + 8, tmn, tmx, q, qk, elem_row + c0 + 8, wd[2], wd[3]);
          };
          for (int ch = 0; ch < c_end; ch += 2) {   // chunks ch (in va) and, if there is one, ch + 1 (in vb)
            const bool last = ch + 1 == c_end;
            tmem_ld_wait16(va);
            if (!last) tmem_ld16r(taddr + (ch + 1) * 16, vb);
            uint32_t wd[8];
            pass16(va, ch * 16, wd);
            if (!last) {
              tmem_ld_wait16(vb);
              if (ch + 2 < c_end) tmem_ld16r(taddr + (ch + 2) * 16, va);
              pass16(vb, (ch + 1) * 16, wd + 4);
            }
            if (row_valid) {
              // 16-byte stores: one 32-byte store per two passes was measured 1 us slower on the stem (register pressure)
              *reinterpret_cast<uint4*>(dst_row + ch * 16) = make_uint4(wd[0], wd[1], wd[2], wd[3]);
              if (!last) *reinterpret_cast<uint4*>(dst_row + (ch + 1) * 16) = make_uint4(wd[4], wd[5], wd[6], wd[7]);
            }
          }
          if (row_valid) {
            mn = min(mn, tmn);
            mx = max(mx, tmx);
          }
        } else {
          for (int ch = c_begin; ch < c_end; ++ch) {
            const int c0 = ch * 16;
            int v[16];
            tmem_ld16(taddr + c0, v);
            tmem_ld_wait();
            if (row_valid) {
#pragma unroll
              for (int e = 0; e < 16; ++e) {
                v[e] -= zrow[c0 + e];
                mn = min(mn, v[e]);
                mx = max(mx, v[e]);
              }
              if constexpr (kOut == kOutInt8) {
                uint32_t wd[4];
#pragma unroll
                for (int e = 0; e < 4; ++e)
                  wd[e] = quant4_acc(v[4 * e], v[4 * e + 1], v[4 * e + 2], v[4 * e + 3], pix * p.BN + c0 + 4 * e, q, sat_below, sat_above);
                *reinterpret_cast<uint4*>(reinterpret_cast<int8_t*>(p.out) + pix * p.BN + c0) = make_uint4(wd[0], wd[1], wd[2], wd[3]);
              } else {
                uint32_t* dst = reinterpret_cast<uint32_t*>(p.out) + pix * p.BN + c0;
                uint32_t wd[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) wd[e] = (kOut == kOutF32) ? __float_as_uint(__fmul_rn(__int2float_rn(v[e]), q.s_acc)) : (uint32_t)v[e];
                if (wide32) {   // rows of 4-byte values start on 32-byte boundaries
                  st_global_v8(dst, wd);
                  st_global_v8(dst + 8, wd + 8);
                } else {
#pragma unroll
                  for (int e = 0; e < 4; ++e) *reinterpret_cast<uint4*>(dst + 4 * e) = make_uint4(wd[4 * e], wd[4 * e + 1], wd[4 * e + 2], wd[4 * e + 3]);
                }
              }
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(tempty_bar(buf));
      }
    };
    if (!lean) run_tiles(std::integral_constant<int, -1>{});
    else if (q.sr) run_tiles(std::integral_constant<int, kLeanSr>{});
    else if (q.noclamp) run_tiles(std::integral_constant<int, kLeanNoClamp>{});
    else run_tiles(std::integral_constant<int, kLeanClamp>{});
    if (q.count_sat) {
      sat_below = __reduce_add_sync(0xffffffffu, sat_below);
      sat_above = __reduce_add_sync(0xffffffffu, sat_above);
      if (lane == 0) {
        if (sat_below) atomicAdd(&p.yq->sat_below, (uint32_t)sat_below);
        if (sat_above) atomicAdd(&p.yq->sat_above, (uint32_t)sat_above);
      }
    }
    mn = __reduce_min_sync(0xffffffffu, mn);
    mx = __reduce_max_sync(0xffffffffu, mx);
    if (lane == 0) {
      red_min[ew] = mn;
      red_max[ew] = mx;
    }
    asm volatile("bar.sync 1, %0;" ::"r"(kEpiThreads) : "memory");
    if (ew == 0 && lane == 0) {
      for (int e = 1; e < kGatherEpiWarps; ++e) {
        mn = min(mn, red_min[e]);
        mx = max(mx, red_max[e]);
      }
      if (mn <= mx) {
        atomicMin(&p.yq->acc_min, mn);
        atomicMax(&p.yq->acc_max, mx);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (*abort_flag != 0) {   // gave up: the thread that issued the raw-row copies waits, bounded, for those still in flight
    if (warp == 0 && lane == 0) ring_drain(raw_full, p.stages_raw, fin_s[0], (uint32_t)fin_s[1]);
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(p.tmem_cols) : "memory");
  }
}

// corr[(rc * ncolcls + cc) * corr_ld + k] = sum of W[k][r][s][c] over the filter taps inside the image for border class (rc, cc)
__global__ void gather_corr_kernel(const int8_t* __restrict__ W, int32_t* __restrict__ corr, int K, int R, int S, int C, ClassMasksG m, int nrowcls,
                                   int ncolcls, int corr_ld) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= nrowcls * ncolcls * K) return;
  const int k = idx % K, cls = idx / K;
  const int rc = cls / ncolcls, cc = cls % ncolcls;
  int sum = 0;
  for (int r = 0; r < R; ++r)
    for (int s = 0; s < S; ++s)
      if (((m.row[rc] >> r) & 1u) && ((m.col[cc] >> s) & 1u))
        for (int c = 0; c < C; ++c) sum += W[(((int64_t)k * R + r) * S + s) * C + c];
  corr[(int64_t)cls * corr_ld + k] = sum;
}

template <int R, int SC>
cudaError_t launch_one(const GatherParams& p, const CUtensorMap& tm, int out_mode, int grid, uint32_t smem, cudaStream_t s, bool overlap) {
  cudaError_t e;
  switch (out_mode) {
    case kOutInt8:
      if ((e = cudaFuncSetAttribute(hq_gather_conv_kernel<kOutInt8, R, SC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
      return launch_overlapped(hq_gather_conv_kernel<kOutInt8, R, SC>, grid, kGatherThreads, smem, s, overlap, p, tm);
    case kOutF32:
      if ((e = cudaFuncSetAttribute(hq_gather_conv_kernel<kOutF32, R, SC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
      return launch_overlapped(hq_gather_conv_kernel<kOutF32, R, SC>, grid, kGatherThreads, smem, s, overlap, p, tm);
    default:
      if ((e = cudaFuncSetAttribute(hq_gather_conv_kernel<kOutAcc, R, SC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
      return launch_overlapped(hq_gather_conv_kernel<kOutAcc, R, SC>, grid, kGatherThreads, smem, s, overlap, p, tm);
  }
}

}  // namespace

bool gather_conv_supported(int R, int SC) {
  return (R == 7 && SC == 21) || (R == 3 && SC == 9) || (R == 5 && SC == 15) || (R == 3 && SC == 15) || (R == 5 && SC == 20) || (R == 3 && SC == 12);
}

cudaError_t launch_gather_conv(const GatherParams& p, const CUtensorMap& tm, int out_mode, int grid, uint32_t smem, cudaStream_t s, bool overlap) {
  const int SC = p.S * p.C;
  if (p.R == 7 && SC == 21) return launch_one<7, 21>(p, tm, out_mode, grid, smem, s, overlap);
  if (p.R == 3 && SC == 9) return launch_one<3, 9>(p, tm, out_mode, grid, smem, s, overlap);
  if (p.R == 5 && SC == 15) return launch_one<5, 15>(p, tm, out_mode, grid, smem, s, overlap);
  if (p.R == 3 && SC == 15) return launch_one<3, 15>(p, tm, out_mode, grid, smem, s, overlap);
  if (p.R == 5 && SC == 20) return launch_one<5, 20>(p, tm, out_mode, grid, smem, s, overlap);
  if (p.R == 3 && SC == 12) return launch_one<3, 12>(p, tm, out_mode, grid, smem, s, overlap);
  return cudaErrorInvalidValue;
}

cudaError_t launch_gather_corr(const int8_t* W, int32_t* corr, int K, int R, int S, int C, const uint32_t* rowmasks, int nrowcls, const uint32_t* colmasks,
                               int ncolcls, int corr_ld, cudaStream_t s) {
  ClassMasksG m{};
  for (int i = 0; i < nrowcls; ++i) m.row[i] = rowmasks[i];
  for (int i = 0; i < ncolcls; ++i) m.col[i] = colmasks[i];
  const int total = nrowcls * ncolcls * K;
  gather_corr_kernel<<<(total + 127) / 128, 128, 0, s>>>(W, corr, K, R, S, C, m, nrowcls, ncolcls, corr_ld);
  return cudaGetLastError();
}

}  // namespace hq
