// Tensor-core layer kernel: implicit GEMM on tcgen05 (kind::i8, int32 accumulators in TMEM),
// operands staged by TMA, with the requantization + min/max epilogue of the in-hindsight
// scheme (arxiv 2105.04246, Sec. 3.1, Sec. 3.2 "static quantization", Sec. 4 steps 1 and 2).
//
// One persistent CTA per SM walks over 128-row output tiles (or a pair of CTAs on neighbouring SMs over 256-row tiles:
// the kPairK instantiation).  Roles: warp 0 feeds operand A (kModeTap: one box of A and one of B per filter tap and
// channel chunk; kModeHalo: the padded input rows of the tile, once), warp 2 feeds the weights (streamed in kModeHalo,
// or once when they stay resident), warp 1 -- and warps 3 and 2 where the planner says so -- issue the MMAs, sixteen
// epilogue warps in 1, 2 or 4 groups drain 2 to 8 accumulator buffers in TMEM, so the epilogue of a tile overlaps
// the MAC loops of the following ones.  Every wait is bounded (see mbar_wait).
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

template <int V>
__device__ __forceinline__ void store_bytes16(int8_t* p, const uint32_t* w, int nvalid) {
  // w: 4 words = 16 output bytes; store the first nvalid bytes in pieces of V bytes
  if constexpr (V == 16) {
    if (nvalid >= 16) *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
  } else if constexpr (V == 8) {
#pragma unroll
    for (int g = 0; g < 2; ++g)
      if ((g + 1) * 8 <= nvalid) *reinterpret_cast<uint2*>(p + 8 * g) = make_uint2(w[2 * g], w[2 * g + 1]);
  } else if constexpr (V == 4) {
#pragma unroll
    for (int g = 0; g < 4; ++g)
      if ((g + 1) * 4 <= nvalid) *reinterpret_cast<uint32_t*>(p + 4 * g) = w[g];
  } else {
#pragma unroll
    for (int g = 0; g < 16; ++g)
      if (g < nvalid) p[g] = (int8_t)((w[g >> 2] >> (8 * (g & 3))) & 0xffu);
  }
}

// kPairK: the instantiation that runs as clusters of two CTAs (its cta_group::2 instructions make the launch
// require an even cluster size, so single-CTA launches use the other instantiation).
template <int kOut, bool kPairK>
__global__ void __launch_bounds__(kGemmThreads, 1)
hq_gemm_kernel(const __grid_constant__ GemmParams p, const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
               int out_vec) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[2 * kMaxStagesA + 2 * kMaxStagesB + 16];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag_s;
  __shared__ int red_min[kEpilogueWarps], red_max[kEpilogueWarps];
  __shared__ int red_below[kEpilogueWarps], red_above[kEpilogueWarps];   // saturation counts (tensors that ask for them)
  __shared__ uint32_t tapoff_s[kMaxTaps];      // kModeHalo: start shift of tap t in 16-byte units
  __shared__ uint8_t cls_s[1024];              // border classes of rows [0,512) and columns [512,1024) when they fit

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  volatile int* abort_flag = &abort_flag_s;

  const uint32_t ring_a = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const bool halo = p.mode == kModeHalo;
  // kModeTap: one ring, stage = [A tile | B tile] (A tile alone when the weights are resident, which then follow
  // the ring); kModeHalo: patch ring, then weight ring
  const uint32_t a_stride = (halo || p.b_resident) ? p.stage_bytes_a : p.stage_bytes_a + p.stage_bytes_b;
  const uint32_t ring_b = ring_a + (uint32_t)p.stages_a * a_stride;
  const uint32_t bar0 = smem_u32(bars);
  auto a_full = [&](int s) { return bar0 + 8u * s; };
  auto a_empty = [&](int s) { return bar0 + 8u * (kMaxStagesA + s); };
  auto b_full = [&](int s) { return bar0 + 8u * (2 * kMaxStagesA + s); };
  auto b_empty = [&](int s) { return bar0 + 8u * (2 * kMaxStagesA + kMaxStagesB + s); };
  auto tfull_bar = [&](int b) { return bar0 + 8u * (2 * kMaxStagesA + 2 * kMaxStagesB + b); };
  auto tempty_bar = [&](int b) { return bar0 + 8u * (2 * kMaxStagesA + 2 * kMaxStagesB + 8 + b); };
  const int nbuf = p.tmem_bufs, nbuf_log2 = p.tmem_bufs_log2;   // accumulator buffers in TMEM (2 or 4)
  // CTA pair (cluster of two): both CTAs walk over the same sequence of 256-row pair tiles, each with its own 128 rows
  // of A and half of the rows of B; the MMA issuer of rank 0 drives both tensor cores.  "Full" barriers and the
  // accumulator's "empty" barriers are those of rank 0 (the peer reports to them remotely); operand "empty" and
  // accumulator "full" barriers are local in both CTAs and receive the issuer's multicast commits.
  constexpr bool pair = kPairK;
  uint32_t crank = 0u, bar0_lead = bar0;
  if constexpr (kPairK) {
    crank = cluster_cta_rank();
    bar0_lead = map_to_cta(bar0, 0u);
  }
  auto a_full_lead = [&](int s) { return bar0_lead + 8u * s; };
  auto b_full_lead = [&](int s) { return bar0_lead + 8u * (2 * kMaxStagesA + s); };
  auto tempty_lead = [&](int b) { return bar0_lead + 8u * (2 * kMaxStagesA + 2 * kMaxStagesB + 8 + b); };
  const int ncta = pair ? 2 : 1;

  const int kiters = p.ntaps * p.chunks_per_tap;

  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    for (int s = 0; s < p.stages_a; ++s) {
      mbar_init(a_full(s), ncta);   // one arrival (with its byte count) per producing CTA
      mbar_init(a_empty(s), 1);
    }
    for (int s = 0; s < p.stages_b; ++s) {
      mbar_init(b_full(s), ncta);
      mbar_init(b_empty(s), 1);
    }
    for (int b = 0; b < nbuf; ++b) {
      mbar_init(tfull_bar(b), 1);
      mbar_init(tempty_bar(b), ncta * (kEpilogueWarps >> p.epi_groups_log2));   // one arrival per warp of the group(s) that drain it
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (threadIdx.x < (unsigned)p.ntaps && p.mode == kModeHalo)
    tapoff_s[threadIdx.x] =
        (uint32_t)(((p.tap_dh[threadIdx.x] - p.dh_min) * p.P + (p.tap_dw[threadIdx.x] - p.dw_min)) * p.BK) >> 4;
  int32_t* zc_s = reinterpret_cast<int32_t*>(smem_raw + ((ring_a - smem_u32(smem_raw)) + p.zc_offset));
  if (warp == 0 && lane == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&tmap_a) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&tmap_b) : "memory");
  }
  if (warp == 1) {
    if constexpr (kPairK) {   // the pair's accumulators: the same columns in both CTAs' tensor memory
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(p.tmem_cols)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(p.tmem_cols)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  if constexpr (kPairK) cluster_sync_all();   // the peer's barriers exist before anything arrives on them
  else __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  // Everything above touched only kernel parameters and this CTA's own resources.  What earlier kernels in the stream
  // wrote (operands, range states) is read by the operand producers and the epilogue warps; each of them waits for
  // those kernels (grid_dependency_wait) right before its first access to global memory, after its own set-up, so that
  // the set-up runs while the previous kernel drains (the MMA issuers, which touch shared and tensor memory only, wait
  // before their first barrier).  The weight producer reads nothing but the prepared weight matrix; where the host knows that matrix to be
  // older than the previous kernel (any call after the first with these prepared weights) it starts copying at once.

  // tile index -> origin.  kModeTap: (n0, h0, w0) of the pixel box; kModeHalo: image n0, first linear pixel h0
  auto decode = [&](int tile, int& n0, int& h0, int& w0, int& col0) {
    int t = fdiv(tile, p.fd_tiles_col);
    col0 = (tile - t * p.tiles_col) * p.BN;
    if (halo) {
      n0 = fdiv(t, p.fd_tiles_per_img);
      h0 = (t - n0 * p.tiles_per_img) * kTileM;
      w0 = 0;
    } else {
      const int t2 = fdiv(t, p.fd_tiles_w);
      w0 = (t - t2 * p.tiles_w) * p.Wt;
      const int t3 = fdiv(t2, p.fd_tiles_h);
      h0 = (t2 - t3 * p.tiles_h) * p.Ht;
      n0 = t3 * p.Nt;
    }
  };
  // The CTA's it-th tile, or -1 when it has none left.  A pair takes pair tile (pair index + it * pairs): rank r gets
  // row tile 2q + r (kModeTap) or the same tile of image 2a + r (kModeHalo: both halves of the pair then start at the
  // same pixel of their patch, as the shared matrix descriptor requires).  Row tiles past the end are computed on
  // zero-filled operands and dropped by the epilogue.
  auto own_tile = [&](int it) -> int {
    if (!pair) {
      const int tile = (int)blockIdx.x + it * (int)gridDim.x;
      return tile < p.num_tiles ? tile : -1;
    }
    const int pt = (int)(blockIdx.x >> 1) + it * (int)(gridDim.x >> 1);
    if (pt >= p.num_pair_tiles) return -1;
    const int q = fdiv(pt, p.fd_tiles_col);
    const int ct = pt - q * p.tiles_col;
    int mt;
    if (halo) {
      const int a = fdiv(q, p.fd_tiles_per_img);
      mt = (2 * a + (int)crank) * p.tiles_per_img + (q - a * p.tiles_per_img);
    } else {
      mt = 2 * q + (int)crank;
    }
    return mt * p.tiles_col + ct;
  };
  const int my_tiles = own_tile(0) >= 0 ? 1 : 0;   // only "has any" is used
  int fin_stage = 0;          // the producers' ring position when they stopped (see the end of the kernel)
  uint32_t fin_phase = 0;
  int fin_passed = 0;         // two operand producers: how many ring stages this one got through

  // The three single-issuer roles below are executed by their WHOLE warp with warp-uniform control flow and
  // values; only the copy / MMA / commit instructions themselves sit under a one-lane predicate (elect.sync).
  // Uniform values stay in uniform registers, which is what the TMA and MMA instructions take their operands from.
  auto run_issuer = [&](const int issuer) __attribute__((always_inline)) {
    // ------------------------------ MMA issuer(s) ------------------------------
    // With several issuers (warps 1, 3 and, once resident weights are on their way, 2) issuer i takes the CTA's tiles
    // i, i + n, ...: the fixed per-tile latency of one issuer (decode, waits, commits) hides behind the others' MMA
    // streams.
    const int nissuers = p.mma_issuers;
    // The k-steps of one operand stage are issued from a compile-time unrolled group: a run-time inner loop
    // around the MMA instruction was measured to cost several hundred cycles per iteration.
    auto mma_role = [&](auto kk_tag, auto pair_tag, auto nt_tag) {
      constexpr int KK = decltype(kk_tag)::value;
      constexpr bool kPair = decltype(pair_tag)::value;
      // NT > 0: resident-row layers with exactly NT filter taps (3x3: 9).  Their tap loop is unrolled at compile time with
      // the tap offsets in registers: as a run-time loop (shared-memory load of the offset, branch, descriptor arithmetic
      // in per-thread registers) it cost about 200 clocks per tap, more than the MMAs of a tap on a 64-column tile take.
      constexpr int NT = decltype(nt_tag)::value;
      uint32_t toff[NT > 0 ? NT : 1];
      if constexpr (NT > 0) {
#pragma unroll
        for (int t = 0; t < NT; ++t) toff[t] = tapoff_s[t];
      }
      int stage = 0, bstage = 0;
      uint32_t phase = 0, bphase = 0;
      bool ok = true;
      // ring positions are global over the CTA's tiles: skipping a tile advances them by that tile's stage count
      auto advance = [](int& st, uint32_t& ph, int n, int stages) {
        st += n;
        while (st >= stages) {
          st -= stages;
          ph ^= 1u;
        }
      };
      const int a_per_tile = halo ? p.chunks_per_tap : kiters;
      const int b_per_tile = (halo && !p.b_resident) ? kiters : 0;
      if (issuer > 0) {
        advance(stage, phase, issuer * a_per_tile, p.stages_a);
        if (b_per_tile) advance(bstage, bphase, issuer * b_per_tile, p.stages_b);
      }
      bool first = true;
      const bool sw64 = p.swizzle64 != 0;
      const uint64_t bdesc0 = make_smem_desc(ring_b, sw64);
      const int ntaps = p.ntaps, stages_b = p.stages_b;
      const bool resident = p.b_resident != 0;
      const uint32_t idesc = p.idesc;
      const uint32_t bstep16 = p.stage_bytes_b >> 4;
      // nothing can arrive before the operand producers have passed the same point; waiting here keeps the bounded waits
      // below from counting time that belongs to an earlier kernel
      grid_dependency_wait();
      for (int local_tile = issuer; ok; local_tile += nissuers) {
        const int tile = own_tile(local_tile);
        if (tile < 0) break;
        const int buf = local_tile & (nbuf - 1);
        const uint32_t tph = (uint32_t)(local_tile >> nbuf_log2) & 1u;
        // A parity wait cannot tell "the previous use of this buffer was drained" from "the use before that was drained
        // and the previous one has not even been issued": the wait below is only sound once tile local_tile - nbuf has
        // passed this point.  With one or two issuers that tile is this issuer's own (nbuf is a multiple of two).  With
        // three it belongs to another issuer, which may lag behind this one; then the tile's first operand stage has to be
        // there first: the producer fills stages in order and reuses a stage only after the MMAs that read it, and the
        // host keeps the ring no deeper than nbuf tiles, so a filled first stage means tile local_tile - nbuf was issued.
        if (nissuers > 2) {
          ok = warp_wait(a_full(stage), phase, abort_flag, p.status, kAsyncMmaFullWait, 200u);
          if (!ok) break;
        }
        ok = warp_wait(tempty_bar(buf), tph ^ 1u, abort_flag, p.status, kAsyncMmaTmemEmptyWait, 200u);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * p.tmem_buf_stride;
        uint32_t acc = 0;
        if (resident && first) {   // the whole weight matrix arrives once
          ok = warp_wait(b_full(0), 0u, abort_flag, p.status, kAsyncMmaBFullWait, 200u);
          if (!ok) break;
          tc_fence_after();
        }
        if (halo) {
          int n0, o0, w0, col0;
          decode(tile, n0, o0, w0, col0);
          const uint32_t rel_bytes = (uint32_t)(o0 - fdiv(o0, p.fd_P) * p.P) * (uint32_t)p.BK;
          uint64_t bres = bdesc0;
          for (int cc = 0; cc < p.chunks_per_tap && ok; ++cc) {
            ok = warp_wait(a_full(stage), phase, abort_flag, p.status, kAsyncMmaFullWait, 200u);
            if (!ok) break;
            tc_fence_after();
            const uint64_t abase = make_smem_desc(ring_a + stage * a_stride + rel_bytes, sw64);
            if (resident) {
              if constexpr (NT > 0) {
#pragma unroll
                for (int t = 0; t < NT; ++t) {
                  const uint64_t adesc = abase + toff[t];
                  const uint64_t bdesc = bres + (uint64_t)(t * bstep16);
                  if (elect_one()) {
#pragma unroll
                    for (int k = 0; k < KK; ++k) mma_any<kPair>(d_tmem, adesc + 2u * k, bdesc + 2u * k, idesc, (k == 0 && t == 0) ? acc : 1u);
                  }
                }
                bres += (uint64_t)(NT * bstep16);
              } else {
                if (elect_one()) {
                  for (int t = 0; t < ntaps; ++t) {
                    const uint64_t adesc = abase + tapoff_s[t];
#pragma unroll
                    for (int k = 0; k < KK; ++k) mma_any<kPair>(d_tmem, adesc + 2u * k, bres + 2u * k, idesc, (k == 0 && t == 0) ? acc : 1u);
                    bres += bstep16;
                  }
                }
              }
              __syncwarp();
              acc = 1;
            } else if constexpr (NT > 0) {
#pragma unroll
              for (int t = 0; t < NT; ++t) {
                if (ok) {
                  ok = warp_wait(b_full(bstage), bphase, abort_flag, p.status, kAsyncMmaBFullWait, 200u);
                  if (ok) {
                    tc_fence_after();
                    const uint64_t bdesc = bdesc0 + (uint64_t)bstage * bstep16;
                    const uint64_t adesc = abase + toff[t];
                    if (elect_one()) {
#pragma unroll
                      for (int k = 0; k < KK; ++k) mma_any<kPair>(d_tmem, adesc + 2u * k, bdesc + 2u * k, idesc, k == 0 ? acc : 1u);
                      commit_any<kPair>(b_empty(bstage));
                    }
                    acc = 1;
                    if (++bstage == stages_b) {
                      bstage = 0;
                      bphase ^= 1u;
                    }
                  }
                }
              }
            } else {
              for (int t = 0; t < ntaps; ++t) {
                ok = warp_wait(b_full(bstage), bphase, abort_flag, p.status, kAsyncMmaBFullWait, 200u);
                if (!ok) break;
                tc_fence_after();
                const uint64_t bdesc = bdesc0 + (uint64_t)bstage * bstep16;
                const uint64_t adesc = abase + tapoff_s[t];
                if (elect_one()) {
#pragma unroll
                  for (int k = 0; k < KK; ++k) mma_any<kPair>(d_tmem, adesc + 2u * k, bdesc + 2u * k, idesc, k == 0 ? acc : 1u);
                  commit_any<kPair>(b_empty(bstage));
                }
                acc = 1;
                if (++bstage == stages_b) {
                  bstage = 0;
                  bphase ^= 1u;
                }
              }
            }
            if (!ok) break;
            if (elect_one()) commit_any<kPair>(a_empty(stage));
            if (++stage == p.stages_a) {
              stage = 0;
              phase ^= 1u;
            }
          }
          if (!ok) break;
        } else {
          uint64_t bres = bdesc0;
          if (resident) {
            const int t0 = fdiv(tile, p.fd_tiles_col);
            bres += (uint64_t)((tile - t0 * p.tiles_col) * kiters) * bstep16;
          }
          for (int ki = 0; ki < kiters; ++ki) {
            ok = warp_wait(a_full(stage), phase, abort_flag, p.status, kAsyncMmaFullWait, 200u);
            if (!ok) break;
            tc_fence_after();
            const uint32_t sa = ring_a + stage * a_stride;
            const uint64_t adesc = make_smem_desc(sa, sw64);
            const uint64_t bdesc = resident ? bres + (uint64_t)ki * bstep16 : make_smem_desc(sa + p.stage_bytes_a, sw64);
            if (elect_one()) {
#pragma unroll
              for (int k = 0; k < KK; ++k) mma_any<kPair>(d_tmem, adesc + 2u * k, bdesc + 2u * k, idesc, k == 0 ? acc : 1u);
              commit_any<kPair>(a_empty(stage));
            }
            acc = 1;
            if (++stage == p.stages_a) {
              stage = 0;
              phase ^= 1u;
            }
          }
          if (!ok) break;
        }
        if (elect_one()) commit_any<kPair>(tfull_bar(buf));
        first = false;
        if (nissuers > 1) {   // step over the other issuer's tile
          advance(stage, phase, (nissuers - 1) * a_per_tile, p.stages_a);
          if (b_per_tile) advance(bstage, bphase, (nissuers - 1) * b_per_tile, p.stages_b);
        }
      }
    };
    if (kiters > 0 && crank == 0) {   // in a pair, rank 0 issues for both CTAs
      using PairTag = std::integral_constant<bool, kPairK>;
      using T9 = std::integral_constant<int, 9>;
      using T0 = std::integral_constant<int, 0>;
      const bool nine = halo && p.ntaps == 9;
      if (p.BK == 64) {
        if (nine) mma_role(std::integral_constant<int, 2>{}, PairTag{}, T9{});
        else mma_role(std::integral_constant<int, 2>{}, PairTag{}, T0{});
      } else {
        if (nine) mma_role(std::integral_constant<int, 4>{}, PairTag{}, T9{});
        else mma_role(std::integral_constant<int, 4>{}, PairTag{}, T0{});
      }
    }
  };
  // kModeTap, two operand producers (resident weights): producer `first` of `nprod` copies operand A for the CTA's tiles
  // first, first + nprod, ...  Ring positions are global over the CTA's tiles, so a producer steps over the other's
  // stages.  A producer never runs more than a lap ahead of the other at any stage: it passed the stages of its own
  // previous tile, whose release implies that everything one lap before them was consumed, hence filled (the host
  // allows two producers only where the ring holds at least two tiles).  Returns the number of stages it got through.
  __shared__ int fin2_s[3];   // the second producer's ring position when it stopped: stages passed, stage, phase
  auto produce_tap = [&](int first, int nprod, int& stage, uint32_t& phase) -> int {
    bool ok = true;
    int passed = 0;
    auto advance = [&](int n) {
      passed += n;
      stage += n;
      while (stage >= p.stages_a) {
        stage -= p.stages_a;
        phase ^= 1u;
      }
    };
    advance(first * kiters);
    for (int it = first; ok; it += nprod) {
      const int tile = own_tile(it);
      if (tile < 0) break;
      int n0, h0, w0, col0;
      decode(tile, n0, h0, w0, col0);
      if (it == first) grid_dependency_wait();   // the first copy reads what the previous kernel may have written
      for (int t = 0; t < p.ntaps && ok; ++t) {
        const int ch = h0 * p.in_mul_h + p.tap_dh[t];
        const int cw = w0 * p.in_mul_w + p.tap_dw[t];
        for (int cc = 0; cc < p.chunks_per_tap; ++cc) {
          ok = warp_wait(a_empty(stage), phase ^ 1u, abort_flag, p.status, kAsyncProducerEmptyWait, 1000u);
          if (!ok) break;
          if (elect_one()) {
            mbar_expect_tx(a_full(stage), a_stride);
            tma_load_4d(ring_a + stage * a_stride, &tmap_a, cc * p.BK, cw, ch, n0, a_full(stage));
          }
          advance(1);
        }
      }
      if (ok) advance((nprod - 1) * kiters);
    }
    return passed;
  };
  const bool two_producers = !kPairK && !halo && p.a_producers == 2 && kiters > 0;
  if (warp == 0) {
    // ------------------------------ operand A producer ------------------------------
    if (two_producers) {
      fin_passed = produce_tap(0, 2, fin_stage, fin_phase);
    } else if (kiters > 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      const int b_row_off = (int)crank * (p.BN >> 1);   // pair: this CTA's half of the rows of B
      for (int it = 0; ok; ++it) {
        const int tile = own_tile(it);
        if (tile < 0) break;
        int n0, h0, w0, col0;
        decode(tile, n0, h0, w0, col0);
        if (it == 0) grid_dependency_wait();   // the first copy reads what the previous kernel may have written
        if (halo) {
          const int hp0 = fdiv(h0, p.fd_P);   // h0 is the tile's first linear pixel
          for (int cb = 0; cb < p.chunks_per_tap; ++cb) {   // one ring stage per channel chunk of the patch
            ok = warp_wait(a_empty(stage), phase ^ 1u, abort_flag, p.status, kAsyncProducerEmptyWait, 1000u);
            if (!ok) break;
            if (elect_one()) {
              if constexpr (kPairK) {
                mbar_expect_tx_remote(a_full_lead(stage), p.patch_box_bytes);
                tma_load_4d_pair(ring_a + stage * a_stride, &tmap_a, cb * p.BK, p.dw_min, hp0 + p.dh_min, n0, a_full_lead(stage));
              } else {
                mbar_expect_tx(a_full(stage), p.patch_box_bytes);
                tma_load_4d(ring_a + stage * a_stride, &tmap_a, cb * p.BK, p.dw_min, hp0 + p.dh_min, n0, a_full(stage));
              }
            }
            if (++stage == p.stages_a) {
              stage = 0;
              phase ^= 1u;
            }
          }
        } else {
          // rows and reduction offset of operand B: the tile's own columns, or (column tiles that share rows of B, each
          // group of them at its own shift along the reduction) the group's
          int b_row = col0, b_k_shift = 0;
          if (p.b_group_tiles > 0) {
            const int ct = col0 / p.BN, grp = ct / p.b_group_tiles;
            b_row = (ct - grp * p.b_group_tiles) * p.BN;
            b_k_shift = p.b_k_base + grp * p.b_k_step;
          }
          for (int t = 0; t < p.ntaps && ok; ++t) {
            const int ch = h0 * p.in_mul_h + p.tap_dh[t];
            const int cw = w0 * p.in_mul_w + p.tap_dw[t];
            for (int cc = 0; cc < p.chunks_per_tap; ++cc) {
              ok = warp_wait(a_empty(stage), phase ^ 1u, abort_flag, p.status, kAsyncProducerEmptyWait, 1000u);
              if (!ok) break;
              const uint32_t sa = ring_a + stage * a_stride;
              if (elect_one()) {
                if constexpr (kPairK) {   // never with resident weights
                  mbar_expect_tx_remote(a_full_lead(stage), a_stride);
                  tma_load_4d_pair(sa, &tmap_a, cc * p.BK, cw, ch, n0, a_full_lead(stage));
                  tma_load_2d_pair(sa + p.stage_bytes_a, &tmap_b, t * p.Cpad + cc * p.BK + n0 * p.b_slice, col0 + b_row_off, a_full_lead(stage));
                } else {
                  mbar_expect_tx(a_full(stage), a_stride);
                  tma_load_4d(sa, &tmap_a, cc * p.BK, cw, ch, n0, a_full(stage));
                  if (!p.b_resident) tma_load_2d(sa + p.stage_bytes_a, &tmap_b, t * p.Cpad + cc * p.BK + n0 * p.b_slice + b_k_shift, b_row, a_full(stage));
                }
              }
              if (++stage == p.stages_a) {
                stage = 0;
                phase ^= 1u;
              }
            }
          }
        }
      }
      fin_stage = stage;   // where the ring stands, for the drain of a CTA that gave up
      fin_phase = phase;
    }
    __syncwarp();
  } else if (warp == 2) {
    // ------------------------------ weight producer (kModeHalo) ------------------------------
    if (!p.weights_early) grid_dependency_wait();
    if (!halo && p.b_resident && kiters > 0) {
      // kModeTap with a small weight matrix: every (column tile, tap, chunk) box once, in the order the issuer uses them
      if (my_tiles > 0) {   // all of them report to barrier 0: the issuer waits once
        if (elect_one()) mbar_expect_tx(b_full(0), (uint32_t)(p.tiles_col * kiters) * p.stage_bytes_b);
        __syncwarp();
        for (int ct = 0; ct < p.tiles_col; ++ct)
          for (int ki = 0; ki < kiters; ++ki) {
            const int t = ki / p.chunks_per_tap, cc = ki - t * p.chunks_per_tap;
            const int slot = ct * kiters + ki;
            if (elect_one()) tma_load_2d(ring_b + slot * p.stage_bytes_b, &tmap_b, t * p.Cpad + cc * p.BK, ct * p.BN, b_full(0));
          }
      }
    } else if (halo && kiters > 0) {
      if (p.b_resident) {
        if (my_tiles > 0) {
          if (elect_one()) mbar_expect_tx(b_full(0), (uint32_t)kiters * p.stage_bytes_b);
          __syncwarp();
          for (int ki = 0; ki < kiters; ++ki) {   // chunk-major order, as the MMA issuer consumes them
            const int cc = ki / p.ntaps, t = ki - cc * p.ntaps;
            if (elect_one()) tma_load_2d(ring_b + ki * p.stage_bytes_b, &tmap_b, t * p.Cpad + cc * p.BK, 0, b_full(0));
          }
        }
      } else {
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        for (int it = 0; ok; ++it) {
          const int tile = own_tile(it);
          if (tile < 0) break;
          const int col0 = (tile % p.tiles_col) * p.BN + (int)crank * (p.BN >> 1);   // pair: this CTA's half of the rows of B
          for (int cc = 0; cc < p.chunks_per_tap && ok; ++cc) {
            for (int t = 0; t < p.ntaps; ++t) {
              ok = warp_wait(b_empty(stage), phase ^ 1u, abort_flag, p.status, kAsyncProducerBEmptyWait, 1000u);
              if (!ok) break;
              if (elect_one()) {
                if constexpr (kPairK) {
                  mbar_expect_tx_remote(b_full_lead(stage), p.stage_bytes_b);
                  tma_load_2d_pair(ring_b + stage * p.stage_bytes_b, &tmap_b, t * p.Cpad + cc * p.BK, col0, b_full_lead(stage));
                } else {
                  mbar_expect_tx(b_full(stage), p.stage_bytes_b);
                  tma_load_2d(ring_b + stage * p.stage_bytes_b, &tmap_b, t * p.Cpad + cc * p.BK, col0, b_full(stage));
                }
              }
              if (++stage == p.stages_b) {
                stage = 0;
                phase ^= 1u;
              }
            }
          }
        }
        fin_stage = stage;
        fin_phase = phase;
      }
    }
    __syncwarp();
    if (two_producers) {   // the weights are on their way: this warp copies operand A for the odd tiles
      int st2 = 0;
      uint32_t ph2 = 0;
      const int passed = produce_tap(1, 2, st2, ph2);
      if (lane == 0) {
        fin2_s[0] = passed;
        fin2_s[1] = st2;
        fin2_s[2] = (int)ph2;
      }
      __syncwarp();
    }
    if (p.mma_issuers == 3) {   // the weights are on their way and stay: nothing more to copy
      run_issuer(2);
      __syncwarp();
      grid_launch_dependents();
    }
  } else if (warp == 1 || (warp == 3 && p.mma_issuers >= 2)) {
    run_issuer(warp == 1 ? 0 : 1);
    __syncwarp();
    // All MMAs of this CTA are issued; what is left is the epilogue of the last tiles.  The next kernel in the stream
    // may become resident as SMs free up (it waits for this grid to finish before it reads anything).  Releasing it
    // earlier only parks its waiting CTAs beside this one, where they compete for issue slots.
    grid_launch_dependents();
  } else if (warp >= kFirstEpilogueWarp) {
    // ------------------------------ epilogue ------------------------------
    // The 16 warps form G (1, 2 or 4, at most the number of accumulator buffers) groups; group g drains the CTA's tiles
    // g, g + G, ...  Within a group the warps of a TMEM lane quarter split the column chunks.  More groups mean fewer
    // hand-offs per warp (good for many small tiles); one group means the shortest tail (good for few large tiles).
    const int quarter = warp & 3;                         // TMEM lanes 32*quarter .. +31 belong to this warp
    const int ew = warp - kFirstEpilogueWarp;
    const int ngroups = 1 << p.epi_groups_log2;
    const int group = (ew >> 2) & (ngroups - 1);
    const int slice = (ew >> 2) >> p.epi_groups_log2;
    const int slices = kEpilogueSlices >> p.epi_groups_log2;
    const int row = quarter * 32 + lane;
    grid_dependency_wait();   // range states, scales and tables may come from earlier kernels in the stream
    // Everything the tables need is requested before the first use of any of it (a warp stalls at the first use of a
    // pending load, and the loads behind it would only start then): one trip to memory instead of three.
    const int et0 = (int)threadIdx.x - kFirstEpilogueWarp * 32;
    constexpr int kCorrAhead = 4;
    int32_t corr_ahead[kCorrAhead];
#pragma unroll
    for (int k = 0; k < kCorrAhead; ++k) {
      const int i = et0 + k * kEpilogueWarps * 32;
      corr_ahead[k] = (p.zc_in_smem && p.corr != nullptr && i < p.zc_elems) ? p.corr[i] : 0;
    }
    const uint8_t rowcls_ahead = (p.cls_in_smem && et0 < p.TH) ? p.rowcls[et0] : (uint8_t)0;
    const uint8_t colcls_ahead = (p.cls_in_smem && et0 < p.TW) ? p.colcls[et0] : (uint8_t)0;
    QParams q;
    {
      const float s_x = p.xq->scale;
      const float s_w = *p.w_scale;
      q.s_acc = __fmul_rn(s_x, s_w);
      q.zx = p.xq->zero_point;
      q.inv_scale = (kOut == kOutInt8) ? p.yq->inv_scale : 1.0f;
      q.zp = (kOut == kOutInt8) ? p.yq->zero_point : 0;
      qparams_finish(q);
      qparams_bound(q, p.acc_bound);
      if (kOut == kOutInt8) qparams_output_mode(q, p.yq->rounding, p.yq->seed, p.yq->step);
    }
    if (blockIdx.x == 0 && ew == 0 && lane == 0) p.yq->acc_scale = q.s_acc;
    // The epilogue's tables are filled here, by the epilogue warps alone, while the first operand tiles are in flight:
    // zx * (sum of in-image weights) per border class and output channel, and the border classes of rows and columns.
    {
      const int et = (int)threadIdx.x - kFirstEpilogueWarp * 32;
      constexpr int kEpiThreads = kEpilogueWarps * 32;
      if (p.zc_in_smem) {
#pragma unroll
        for (int k = 0; k < kCorrAhead; ++k)
          if (et + k * kEpiThreads < p.zc_elems) zc_s[et + k * kEpiThreads] = q.zx * corr_ahead[k];
        if (p.corr != nullptr)
          for (int i = et + kCorrAhead * kEpiThreads; i < p.zc_elems; i += kEpiThreads) zc_s[i] = q.zx * p.corr[i];
      }
      if (p.cls_in_smem) {   // TH, TW <= 512 = the number of epilogue threads
        if (et < p.TH) cls_s[et] = rowcls_ahead;
        if (et < p.TW) cls_s[512 + et] = colcls_ahead;
      }
      asm volatile("bar.sync 1, %0;" ::"r"(kEpiThreads) : "memory");
    }
    int mn = INT32_MAX, mx = INT32_MIN;
    int sat_below = 0, sat_above = 0;
    const int rn = row / (p.Ht * p.Wt);
    const int rh = (row / p.Wt) % p.Ht;
    const int rw = row % p.Wt;
    const int nchunks = p.BN / 16;                      // BN is a multiple of 16
    const int c_begin = (slice * nchunks) / slices;
    const int c_end = ((slice + 1) * nchunks) / slices;
    const bool has_corr = p.corr != nullptr;
    // per-layer part of the condition for the straight-line pass (see below)
    const bool lean_layer = kOut == kOutInt8 && kiters > 0 && out_vec >= 16 && q.fast && p.bias == nullptr && p.row_term == nullptr &&
                            p.zc_in_smem && has_corr && !q.count_sat;
    // The tile loop is instantiated once per epilogue variant (kLean >= 0: the straight-line int8 pass with that rounding
    // for every tile whose columns all lie inside the layer; -1: the general pass only), so that the loop a warp runs holds
    // one variant's code: fewer instruction-cache misses and branches in the hot loop.
    auto run_tiles = [&](auto lean_tag) {
    constexpr int kLean = decltype(lean_tag)::value;
    const QPacked qk = qpacked(q);
    for (int local_tile = group; ; local_tile += ngroups) {
      const int tile = own_tile(local_tile);
      if (tile < 0) break;
      int n0, h0, w0, col0;
      decode(tile, n0, h0, w0, col0);
      int n, i, j;
      bool row_valid;
      if (halo) {
        const int o = h0 + row;
        n = n0;
        i = fdiv(o, p.fd_P);
        j = o - i * p.P;
        row_valid = (o < p.L) && (j < p.TW) && (n < p.n_img);
      } else {
        n = n0 + rn;
        i = h0 + rh;
        j = w0 + rw;
        row_valid = (n < p.n_img) && (i < p.TH) && (j < p.TW);
      }
      const int64_t pix = ((int64_t)n * p.out_H + (i * p.os_h + p.oa_h)) * p.out_W + (j * p.os_w + p.oa_w);
      // correction row of this pixel's border class (row 0 for pixels of tile padding, whose results are dropped)
      int zoff = col0;
      if (has_corr && row_valid) {
        const int rc = p.cls_in_smem ? cls_s[i] : (p.rowcls ? p.rowcls[i] : 0);
        const int cc = p.cls_in_smem ? cls_s[512 + j] : (p.colcls ? p.colcls[j] : 0);
        zoff += (rc * p.ncolcls + cc) * p.corr_ld;
      }
      const int32_t* corr_row = nullptr;
      const int32_t* zrow_s = nullptr;
      if (has_corr && q.zx != 0 && row_valid) {
        if (p.zc_in_smem) zrow_s = zc_s + zoff;   // shared copy, already multiplied by zx
        else corr_row = p.corr + zoff;
      }
      const int buf = local_tile & (nbuf - 1);
      const uint32_t tph = (uint32_t)(local_tile >> nbuf_log2) & 1u;
      if (kiters > 0) {
        int w = 1;
        if (lane == 0) w = mbar_wait(tfull_bar(buf), tph, abort_flag, p.status, kAsyncEpilogueTmemFullWait, 2000u) ? 1 : 0;
        w = __shfl_sync(0xffffffffu, w, 0);
        if (!w) break;
        tc_fence_after();
      }
      const uint32_t taddr = tmem_base + buf * p.tmem_buf_stride + ((uint32_t)(quarter * 32) << 16);
      constexpr int CW = 16;   // columns per pass: 16 accumulators per thread keep the warp's register count low
      // one pass over CW columns held in v: correction, statistics, requantization, store
      auto process = [&](int c0, int (&v)[CW]) {
        int nvalid = p.Nout - (col0 + c0);
        nvalid = nvalid < 0 ? 0 : (nvalid > CW ? CW : nvalid);
        if (!row_valid) nvalid = 0;
        if (zrow_s != nullptr) {   // the tables are padded to whole column tiles
#pragma unroll
          for (int e = 0; e < CW; e += 4) {
            const int4 cr = *reinterpret_cast<const int4*>(zrow_s + c0 + e);
            v[e + 0] -= cr.x;
            v[e + 1] -= cr.y;
            v[e + 2] -= cr.z;
            v[e + 3] -= cr.w;
          }
        } else if (corr_row != nullptr) {
#pragma unroll
          for (int e = 0; e < CW; e += 4) {
            const int4 cr = *reinterpret_cast<const int4*>(corr_row + c0 + e);
            v[e + 0] -= q.zx * cr.x;
            v[e + 1] -= q.zx * cr.y;
            v[e + 2] -= q.zx * cr.z;
            v[e + 3] -= q.zx * cr.w;
          }
        }
        if (p.bias != nullptr) {
#pragma unroll
          for (int e = 0; e < CW; ++e)
            if (e < nvalid) v[e] += p.bias[col0 + c0 + e];
        }
        if (p.row_term != nullptr && row_valid) {   // one number per output pixel
          if (p.rt_fold == 1) {
            const int rt = p.row_term[pix];
#pragma unroll
            for (int e = 0; e < CW; ++e) v[e] -= rt;
          } else {   // the GEMM row holds rt_fold pixels side by side
#pragma unroll
            for (int e = 0; e < CW; ++e)
              if (e < nvalid) v[e] -= p.row_term[pix * p.rt_fold + (col0 + c0 + e) / p.rt_cols];
          }
        }
        if (nvalid == CW) {   // two independent chains, then merged: short dependency depth
          int lo[2], hi[2];
#pragma unroll
          for (int g = 0; g < 2; ++g) {
            const int* x = v + 8 * g;
            lo[g] = min(__vimin3_s32(__vimin3_s32(x[0], x[1], x[2]), x[3], x[4]), __vimin3_s32(x[5], x[6], x[7]));
            hi[g] = max(__vimax3_s32(__vimax3_s32(x[0], x[1], x[2]), x[3], x[4]), __vimax3_s32(x[5], x[6], x[7]));
          }
          mn = __vimin3_s32(mn, lo[0], lo[1]);
          mx = __vimax3_s32(mx, hi[0], hi[1]);
        } else {
#pragma unroll
          for (int e = 0; e < CW; ++e) {
            if (e < nvalid) {
              mn = min(mn, v[e]);
              mx = max(mx, v[e]);
            }
          }
        }
        if (nvalid > 0) {
          if constexpr (kOut == kOutInt8) {
            uint32_t w[CW / 4];
            int r[CW];   // rounded grid coordinate + zero point, before saturation
            if (q.sr) {   // stochastic rounding, one draw per element (shapes that miss the straight-line pass)
              const int64_t e0 = pix * p.ldY + p.out_col0 + col0 + c0;
              if (nvalid == CW && (e0 & 7) == 0) {   // two aligned blocks of eight elements: one generator call each
#pragma unroll
                for (int b = 0; b < 2; ++b) {
                  uint32_t h[8];
                  sr_draws8(q, ((uint64_t)e0 >> 3) + b, h);
#pragma unroll
                  for (int e = 0; e < 8; ++e)
                    r[8 * b + e] = q.fast ? requant_acc_sr<true>(v[8 * b + e], h[e], q) : requant_acc_sr<false>(v[8 * b + e], h[e], q);
                }
              } else {
#pragma unroll
                for (int e = 0; e < CW; ++e)
                  r[e] = e < nvalid
                             ? (q.fast ? requant_acc_sr<true>(v[e], sr_draw1(q, e0 + e), q) : requant_acc_sr<false>(v[e], sr_draw1(q, e0 + e), q))
                             : 0;
              }
            } else if (q.fast) {
#pragma unroll
              for (int e = 0; e < CW; ++e) r[e] = requant_acc<true>(v[e], q);
            } else {
#pragma unroll
              for (int e = 0; e < CW; ++e) r[e] = requant_acc<false>(v[e], q);
            }
            if (q.count_sat) {
#pragma unroll
              for (int e = 0; e < CW; ++e)
                if (e < nvalid) count_clipped(r[e], sat_below, sat_above);
            }
#pragma unroll
            for (int e = 0; e < CW / 4; ++e) w[e] = pack_sat4(r[4 * e + 0], r[4 * e + 1], r[4 * e + 2], r[4 * e + 3]);
            int8_t* dst = reinterpret_cast<int8_t*>(p.out) + pix * p.ldY + col0 + c0;
            if (out_vec >= 16) store_bytes16<16>(dst, w, nvalid);
            else if (out_vec == 8) store_bytes16<8>(dst, w, nvalid);
            else if (out_vec == 4) store_bytes16<4>(dst, w, nvalid);
            else store_bytes16<1>(dst, w, nvalid);
          } else {
            uint32_t* dst = reinterpret_cast<uint32_t*>(p.out) + pix * p.ldY + col0 + c0;
            if (out_vec >= 16 && nvalid == CW) {
              uint32_t w[CW];
#pragma unroll
              for (int e = 0; e < CW; ++e) w[e] = (kOut == kOutF32) ? __float_as_uint(__fmul_rn(__int2float_rn(v[e]), q.s_acc)) : (uint32_t)v[e];
              if (out_vec == 32 && ((col0 + c0) & 7) == 0) {   // whole 32-byte sectors per thread: half the store instructions
                st_global_v8(dst, w);
                st_global_v8(dst + 8, w + 8);
              } else {
#pragma unroll
                for (int e = 0; e < CW / 4; ++e) *reinterpret_cast<uint4*>(dst + 4 * e) = make_uint4(w[4 * e], w[4 * e + 1], w[4 * e + 2], w[4 * e + 3]);
              }
            } else {
#pragma unroll
              for (int e = 0; e < CW; ++e)
                if (e < nvalid) dst[e] = (kOut == kOutF32) ? __float_as_uint(__fmul_rn(__int2float_rn(v[e]), q.s_acc)) : (uint32_t)v[e];
            }
          }
        }
      };
      // Warp-uniform conditions under which a pass is straight-line code: int8 output with 16-byte stores, finite
      // parameters, no bias, every column of the pass inside the layer, correction table in shared memory (it holds
      // zeros when the input zero point is 0).  Rows outside the image (tile padding) are computed like the others
      // and only kept out of the statistics and the store.
      const bool lean = kLean >= 0 && col0 + c_end * CW <= p.Nout;
      if (lean) {
        const int32_t* zrow = zc_s + zoff;
        int8_t* dst_row = reinterpret_cast<int8_t*>(p.out) + pix * p.ldY + col0;
        const int64_t elem_row = pix * p.ldY + p.out_col0 + col0;   // linear index in the output tensor of this row's first column
        int tmn = INT32_MAX, tmx = INT32_MIN;
        // eight columns at a time, two register sets: the load of the next eight is in flight while these are processed
        auto half = [&](int (&x)[8], int c, uint32_t& w0, uint32_t& w1) {
          if constexpr (kLean >= 0) lean_half8m<kLean>(x, zrow + c, tmn, tmx, q, qk, elem_row + c, w0, w1);
        };
        int va[8], vb[8];
        tmem_ld8(taddr + c_begin * CW, va);
        auto pass16 = [&](int ch, uint32_t* w) {   // sixteen columns -> four words of codes
          const int c0 = ch * CW;
          tmem_ld_wait8(va);
          tmem_ld8(taddr + c0 + 8, vb);
          half(va, c0, w[0], w[1]);
          tmem_ld_wait8(vb);
          if (ch + 1 < c_end) tmem_ld8(taddr + c0 + CW, va);
          half(vb, c0 + 8, w[2], w[3]);
        };
        if (out_vec == 32 && ((c_begin | c_end) & 1) == 0 && (col0 & 31) == 0) {
          // 32 columns per store: every thread writes whole 32-byte sectors, in half as many store instructions
          for (int ch = c_begin; ch < c_end; ch += 2) {
            uint32_t w[8];
            pass16(ch, w);
            pass16(ch + 1, w + 4);
            if (row_valid) st_global_v8(reinterpret_cast<uint32_t*>(dst_row + ch * CW), w);
          }
        } else {
          for (int ch = c_begin; ch < c_end; ++ch) {
            uint32_t w[4];
            pass16(ch, w);
            if (row_valid) *reinterpret_cast<uint4*>(dst_row + ch * CW) = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
        if (row_valid) {
          mn = min(mn, tmn);
          mx = max(mx, tmx);
        }
      } else if (kiters > 0) {
        for (int ch = c_begin; ch < c_end; ++ch) {
          int v[CW];
          tmem_ld16(taddr + ch * CW, v);
          tmem_ld_wait();
          process(ch * CW, v);
        }
      } else if (kOut == kOutInt8 && out_vec >= 16 && q.fast && p.bias == nullptr && !has_corr && col0 + c_end * CW <= p.Nout) {
        // no taps (a parity class of a strided backward pass that no filter position reaches): every accumulator is 0,
        // so every code is the zero point, whatever the rounding
        const uint32_t code = (uint32_t)(uint8_t)(int8_t)max(-128, min(127, q.zp)) * 0x01010101u;
        if (row_valid) {
          int8_t* dst_row = reinterpret_cast<int8_t*>(p.out) + pix * p.ldY + col0;
          for (int ch = c_begin; ch < c_end; ++ch) *reinterpret_cast<uint4*>(dst_row + ch * CW) = make_uint4(code, code, code, code);
          mn = min(mn, 0);
          mx = max(mx, 0);
        }
      } else {
        for (int ch = c_begin; ch < c_end; ++ch) {
          int v[CW];
#pragma unroll
          for (int e = 0; e < CW; ++e) v[e] = 0;
          process(ch * CW, v);
        }
      }
      if (kiters > 0) {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if constexpr (kPairK) mbar_arrive_remote(tempty_lead(buf));
          else mbar_arrive(tempty_bar(buf));
        }
      }
    }
    };
    if (!lean_layer) run_tiles(std::integral_constant<int, -1>{});
    else if (q.sr) run_tiles(std::integral_constant<int, kLeanSr>{});
    else if (q.noclamp) run_tiles(std::integral_constant<int, kLeanNoClamp>{});
    else run_tiles(std::integral_constant<int, kLeanClamp>{});
    // statistics: registers -> warp -> CTA -> one atomic pair per CTA
    mn = __reduce_min_sync(0xffffffffu, mn);
    mx = __reduce_max_sync(0xffffffffu, mx);
    if (q.count_sat) {
      sat_below = __reduce_add_sync(0xffffffffu, sat_below);
      sat_above = __reduce_add_sync(0xffffffffu, sat_above);
    }
    if (lane == 0) {
      red_min[ew] = mn;
      red_max[ew] = mx;
      red_below[ew] = sat_below;
      red_above[ew] = sat_above;
    }
    asm volatile("bar.sync 1, %0;" ::"r"(kEpilogueWarps * 32) : "memory");
    if (ew == 0 && lane == 0) {
      for (int e = 1; e < kEpilogueWarps; ++e) {
        mn = min(mn, red_min[e]);
        mx = max(mx, red_max[e]);
        sat_below += red_below[e];
        sat_above += red_above[e];
      }
      if (mn <= mx) {
        atomicMin(&p.yq->acc_min, mn);
        atomicMax(&p.yq->acc_max, mx);
      }
      if (q.count_sat) {
        if (sat_below) atomicAdd(&p.yq->sat_below, (uint32_t)sat_below);
        if (sat_above) atomicAdd(&p.yq->sat_above, (uint32_t)sat_above);
      }
    }
  }

  tc_fence_before();
  if constexpr (kPairK) cluster_sync_all();   // neither CTA leaves while the other may still read its operands or arrive on its barriers
  else __syncthreads();
  if constexpr (!kPairK) {
    // A CTA that gave up does not leave with bulk copies into its shared memory in flight: the threads that issued them wait,
    // again bounded, for the stages they armed last.  (A pair's "full" barriers live in rank 0, which rank 1 cannot poll:
    // pairs rely on the cluster barrier above.)
    if (abort_flag_s != 0) {   // the same for every thread: read after the barrier
      if (kiters > 0 && lane == 0) {
        if (warp == 0) {
          if (two_producers && fin2_s[0] > fin_passed) {   // the other producer got further: drain from where it stood (a stage
            fin_stage = fin2_s[1];                         // the slower one never armed in that lap costs one bounded wait)
            fin_phase = (uint32_t)fin2_s[2];
          }
          ring_drain(a_full, p.stages_a, fin_stage, fin_phase);
        }
        if (warp == 2 && my_tiles > 0) {
          if (p.b_resident) mbar_drain(b_full(0), 0u);
          else if (halo) ring_drain(b_full, p.stages_b, fin_stage, fin_phase);
        }
      }
      __syncthreads();
    }
  }
  if (warp == 1) {
    tc_fence_after();
    if constexpr (kPairK) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(p.tmem_cols) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(p.tmem_cols) : "memory");
  }
}


// ---- measurement: what the tensor cores sustain on kind::i8 with nothing else in the way ---------------------------
// One CTA (or CTA pair) per SM issues the same 128 x BN x 32 (pair: 256 x BN x 32) MMA on operand tiles that sit in
// shared memory for the whole kernel: no loads, no epilogue.  MMAs go out in chunks of kProbeChunk, each chunk followed
// by a commit; the issuer waits for the chunk before the previous one, so one to two chunks are always in flight.
// Operand bytes are pseudo-random (the data pattern moves power and thus clocks).  Gives the denominator "int8 MMA peak
// as measured on this GPU" for the tensor roofline of the layer kernels.
constexpr int kProbeChunk = 32;
template <bool kPairK>
__global__ void __launch_bounds__(128, 1) mma_peak_kernel(int bn, int chunks, uint32_t idesc, int32_t* status) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[2];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag_s;
  volatile int* abort_flag = &abort_flag_s;
  const int warp = threadIdx.x >> 5;
  const uint32_t tile_a = (smem_u32(smem_raw) + 1023u) & ~1023u;   // 128 rows x 128 bytes, 128-byte swizzle
  const uint32_t tile_b = tile_a + 128u * 128u;                     // bn (pair: bn / 2) rows x 128 bytes
  const uint32_t bar0 = smem_u32(bars);
  uint32_t crank = 0u;
  if constexpr (kPairK) crank = cluster_cta_rank();
  {
    uint32_t* w = reinterpret_cast<uint32_t*>(smem_raw + (tile_a - smem_u32(smem_raw)));
    const int words = (128 * 128 + (kPairK ? bn / 2 : bn) * 128) / 4;
    for (int i = threadIdx.x; i < words; i += blockDim.x) {
      uint32_t h = (uint32_t)i * 2654435761u + blockIdx.x * 40503u;
      h ^= h >> 15; h *= 2246822519u; h ^= h >> 13;
      w[i] = h;
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    mbar_init(bar0, 1);
    mbar_init(bar0 + 8u, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  const uint32_t cols = 512;
  if (warp == 0) {
    if constexpr (kPairK) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(cols) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(cols) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  if constexpr (kPairK) cluster_sync_all();
  else __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  if (warp == 1) {   // in a pair rank 0 issues for both tensor cores; the peer follows the same barriers (its copies of the arrivals)
    const uint64_t adesc = make_smem_desc(tile_a, false), bdesc = make_smem_desc(tile_b, false);
    const uint32_t buf_stride = bn <= 256 ? 256u : 512u;
    bool ok = true;
    for (int c = 0; c < chunks && ok; ++c) {
      if (c >= 2) ok = warp_wait(bar0 + 8u * (c & 1), (uint32_t)((c >> 1) - 1) & 1u, abort_flag, status, kAsyncMmaTmemEmptyWait, 200u);
      if (!ok) break;
      tc_fence_after();
      const uint32_t d_tmem = tmem_base + (uint32_t)(c & 1) * buf_stride;
      if (crank == 0 && elect_one()) {
#pragma unroll
        for (int i = 0; i < kProbeChunk / 4; ++i)
#pragma unroll
          for (int k = 0; k < 4; ++k) mma_any<kPairK>(d_tmem, adesc + 2u * k, bdesc + 2u * k, idesc, (i | k) ? 1u : 0u);
        commit_any<kPairK>(bar0 + 8u * (c & 1));   // arrives (in both CTAs of a pair) once every MMA issued so far has finished
      }
      __syncwarp();
    }
    // drain: the last two chunks
    for (int c = (chunks >= 2 ? chunks - 2 : 0); c < chunks && ok; ++c)
      ok = warp_wait(bar0 + 8u * (c & 1), (uint32_t)(c >> 1) & 1u, abort_flag, status, kAsyncMmaTmemEmptyWait, 200u);
  }
  tc_fence_before();
  if constexpr (kPairK) cluster_sync_all();
  else __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    if constexpr (kPairK) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(cols) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(cols) : "memory");
  }
}

}  // namespace

template <int kOut, bool kPairK>
cudaError_t set_smem_attr_one(uint32_t smem_bytes) {
  return cudaFuncSetAttribute(hq_gemm_kernel<kOut, kPairK>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
}
cudaError_t gemm_set_smem_attr(uint32_t smem_bytes) {
  cudaError_t e;
  if ((e = set_smem_attr_one<kOutInt8, false>(smem_bytes)) != cudaSuccess) return e;
  if ((e = set_smem_attr_one<kOutF32, false>(smem_bytes)) != cudaSuccess) return e;
  if ((e = set_smem_attr_one<kOutAcc, false>(smem_bytes)) != cudaSuccess) return e;
  if ((e = set_smem_attr_one<kOutInt8, true>(smem_bytes)) != cudaSuccess) return e;
  if ((e = set_smem_attr_one<kOutF32, true>(smem_bytes)) != cudaSuccess) return e;
  return set_smem_attr_one<kOutAcc, true>(smem_bytes);
}

cudaError_t launch_gemm(const GemmParams& p, const CUtensorMap& ta, const CUtensorMap& tb, int out_mode, int grid, uint32_t smem_bytes,
                        cudaStream_t s, bool overlap) {
  // widest aligned store the output rows allow (bytes; 32: every row starts on a 32-byte boundary, so a thread can write whole sectors)
  int out_vec;
  const uintptr_t addr = reinterpret_cast<uintptr_t>(p.out);
  if (out_mode == kOutInt8) {
    if (p.ldY % 32 == 0 && addr % 32 == 0) out_vec = 32;
    else if (p.ldY % 16 == 0 && addr % 16 == 0) out_vec = 16;
    else if (p.ldY % 8 == 0 && addr % 8 == 0) out_vec = 8;
    else if (p.ldY % 4 == 0 && addr % 4 == 0) out_vec = 4;
    else out_vec = 1;
  } else {
    out_vec = (p.ldY % 8 == 0 && addr % 32 == 0) ? 32 : ((p.ldY % 4 == 0 && addr % 16 == 0) ? 16 : 4);
  }
  if (p.pair) {   // grid is an even number of CTAs: clusters of two
    switch (out_mode) {
      case kOutInt8: return launch_overlapped_cluster(hq_gemm_kernel<kOutInt8, true>, grid, kGemmThreads, smem_bytes, s, overlap, 2u, p, ta, tb, out_vec);
      case kOutF32: return launch_overlapped_cluster(hq_gemm_kernel<kOutF32, true>, grid, kGemmThreads, smem_bytes, s, overlap, 2u, p, ta, tb, out_vec);
      default: return launch_overlapped_cluster(hq_gemm_kernel<kOutAcc, true>, grid, kGemmThreads, smem_bytes, s, overlap, 2u, p, ta, tb, out_vec);
    }
  }
  switch (out_mode) {
    case kOutInt8: return launch_overlapped(hq_gemm_kernel<kOutInt8, false>, grid, kGemmThreads, smem_bytes, s, overlap, p, ta, tb, out_vec);
    case kOutF32: return launch_overlapped(hq_gemm_kernel<kOutF32, false>, grid, kGemmThreads, smem_bytes, s, overlap, p, ta, tb, out_vec);
    default: return launch_overlapped(hq_gemm_kernel<kOutAcc, false>, grid, kGemmThreads, smem_bytes, s, overlap, p, ta, tb, out_vec);
  }
}

}  // namespace hq

namespace hq {
cudaError_t launch_mma_peak(int pair, int bn, int chunks, int num_sms, int32_t* status, cudaStream_t s, uint64_t* ops) {
  // instruction descriptor as for the layer kernel: D = s32, A = B = signed 8-bit, K-major, N = bn, M = 128 (256 across a pair)
  const int m = pair ? 256 : 128;
  const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
  const uint32_t smem = 1024u + 128u * 128u + (uint32_t)(pair ? bn / 2 : bn) * 128u;
  const int grid = pair ? (num_sms / 2) * 2 : num_sms;
  cudaError_t e;
  if (pair) {
    e = cudaFuncSetAttribute(mma_peak_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    e = launch_overlapped_cluster(mma_peak_kernel<true>, grid, 128, smem, s, false, 2u, bn, chunks, idesc, status);
  } else {
    e = cudaFuncSetAttribute(mma_peak_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    e = launch_overlapped(mma_peak_kernel<false>, grid, 128, smem, s, false, bn, chunks, idesc, status);
  }
  if (ops) *ops = 2ull * (uint64_t)m * (uint64_t)bn * 32ull * (uint64_t)kProbeChunk * (uint64_t)chunks * (uint64_t)(pair ? grid / 2 : grid);
  return e;
}
}  // namespace hq
