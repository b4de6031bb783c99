// 3x3 stride-1 depthwise convolution on CUDA cores, three multiply-accumulates per dp4a (arxiv 2105.04246, Sec. 3.2:
// the accumulator is requantized with a range known in advance, statistics taken on the way out).
//
// The activations are NHWC, so a 32-bit word holds four CHANNELS of one pixel, while a depthwise filter row wants three
// neighbouring PIXELS of one channel.  Each thread owns one channel word (4 channels) and a column of output tiles
// 4 pixels wide and kRows high.  Per input row it reads 6 pixel words from the patch in shared memory, transposes them
// in registers (byte permutes) into per-channel words of 4 consecutive pixels, and feeds each of those to dp4a with the
// filter row in bytes 0..2 (or 1..3): 3 dp4a per output instead of 9, and every input row is transposed once and used
// for the three output rows it touches (their accumulators are live side by side).  The patch arrives by one TMA box
// per tile, double buffered; image padding arrives as zeros and the accumulators start at minus the zero-point
// correction of the pixel's border class, so what is left at the end is statistics, requantization and the store.
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "hq_device.cuh"
#include "hq_internal.h"
#include "hq_quant.cuh"

namespace hq {
namespace {

constexpr int kRows = kDwColRows;   // output rows per tile; the patch has kRows + 2
constexpr int kGeneral = -1;        // epilogue variant: any rounding, saturation counts (else a LeanMode)

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) { return __byte_perm(a, b, sel); }

template <int kOut>
__global__ void __launch_bounds__(kDwColMaxThreads) depthwise3x3_col_kernel(const DwParams p, const __grid_constant__ CUtensorMap tmap) {
  extern __shared__ uint8_t dsm_raw[];
  __shared__ __align__(8) uint64_t full_bar[2];
  __shared__ int abort_s;
  __shared__ int red_min[kDwColMaxThreads / 32], red_max[kDwColMaxThreads / 32];
  const uint32_t patch0 = (smem_u32(dsm_raw) + 127u) & ~127u;
  uint8_t* gen = dsm_raw + (patch0 - smem_u32(dsm_raw));
  int32_t* nzc_s = reinterpret_cast<int32_t*>(gen + 2u * p.patch_stride);   // minus (input zero point x in-image weight sum), [class][C]
  uint8_t* rcls_s = reinterpret_cast<uint8_t*>(nzc_s + p.ncls * p.C);
  uint8_t* ccls_s = rcls_s + p.Ho;
  volatile int* abort_flag = &abort_s;
  const int CW = p.C / 4;
  const int cw = threadIdx.x % CW, g = threadIdx.x / CW;   // channel word, group of 4 output columns
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
    tma_load_4d(patch0 + buf * p.patch_stride, &tmap, 0, tw * p.TWt - p.pad_w, th * kRows - p.pad_h, n, bar0 + 8u * buf);
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
  qparams_bound(q, 9.0f * 255.0f * 128.0f);
  if (kOut == kOutInt8) qparams_output_mode(q, p.yq->rounding, p.yq->seed, p.yq->step);
  if (blockIdx.x == 0 && threadIdx.x == 0) p.yq->acc_scale = q.s_acc;
  for (int i = threadIdx.x; i < p.ncls * p.C; i += blockDim.x) nzc_s[i] = -(q.zx * p.corr[i]);
  for (int i = threadIdx.x; i < p.Ho; i += blockDim.x) rcls_s[i] = p.rowcls[i];
  for (int i = threadIdx.x; i < p.Wo; i += blockDim.x) ccls_s[i] = p.colcls[i];
  // filter row f of channel k in bytes 0..2 (wa) and 1..3 (wb) of a word: the two placements of a 3-pixel window
  // inside a word of 4 pixels
  uint32_t wa[3][4], wb[3][4];
  {
    uint32_t t[9];
#pragma unroll
    for (int i = 0; i < 9; ++i) t[i] = *reinterpret_cast<const uint32_t*>(p.w + (int64_t)i * p.C + cw * 4);
#pragma unroll
    for (int f = 0; f < 3; ++f)
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const uint32_t b0 = (t[3 * f + 0] >> (8 * k)) & 0xffu, b1 = (t[3 * f + 1] >> (8 * k)) & 0xffu, b2 = (t[3 * f + 2] >> (8 * k)) & 0xffu;
        wa[f][k] = b0 | (b1 << 8) | (b2 << 16);
        wb[f][k] = wa[f][k] << 8;
      }
  }
  __syncthreads();   // tables complete

  int mn = INT32_MAX, mx = INT32_MIN;
  int sat_below = 0, sat_above = 0;
  const int box_w = p.TWt + 2;
  const int row_bytes = box_w * p.C;
  const QPacked qk = qpacked(q);

  auto run_tiles = [&](auto mode_tag) {
    [[maybe_unused]] constexpr int kMode = decltype(mode_tag)::value;
    int it = 0;
    for (int tile = blockIdx.x; tile < total; tile += gridDim.x, ++it) {
      const int buf = it & 1;
      bool ok = mbar_wait(bar0 + 8u * buf, (uint32_t)(it >> 1) & 1u, abort_flag, p.status, kAsyncDepthwiseFullWait, 1000u);
      ok = __syncthreads_and(ok) != 0;   // one decision for the whole CTA
      if (!ok) break;
      const int tw = tile % p.tiles_w;
      const int th = (tile / p.tiles_w) % p.tiles_h;
      const int n = tile / (p.tiles_w * p.tiles_h);
      const int wo0 = tw * p.TWt + 4 * g;
      const int ho0 = th * kRows;
      if (wo0 < p.Wo) {
        const uint8_t* px = gen + buf * p.patch_stride + (4 * g) * p.C + cw * 4;   // patch row 0, first of this thread's 6 columns
        int ctab[4];   // offset of this thread's corrections for each of its 4 columns, without the row class
#pragma unroll
        for (int j = 0; j < 4; ++j) ctab[j] = ccls_s[min(wo0 + j, p.Wo - 1)] * p.C + cw * 4;
        int acc[3][4][4];   // [output row mod 3][pixel][channel]
#pragma unroll
        for (int i = 0; i < kRows + 2; ++i) {
          if (i < kRows) {   // output row i starts with this input row
            const int rcoff = rcls_s[min(ho0 + i, p.Ho - 1)] * p.ncolcls * p.C;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const int4 z = *reinterpret_cast<const int4*>(nzc_s + rcoff + ctab[j]);
              acc[i % 3][j][0] = z.x;
              acc[i % 3][j][1] = z.y;
              acc[i % 3][j][2] = z.z;
              acc[i % 3][j][3] = z.w;
            }
          }
          // six pixels x four channels -> per channel: pixels 0..3 in ta[k], pixels 2..5 in tw4[k]
          uint32_t r[6];
#pragma unroll
          for (int j = 0; j < 6; ++j) r[j] = *reinterpret_cast<const uint32_t*>(px + i * row_bytes + j * p.C);
          const uint32_t u0 = prmt(r[0], r[1], 0x5140), u1 = prmt(r[2], r[3], 0x5140);   // channels 0,1 of pixel pairs
          const uint32_t u2 = prmt(r[0], r[1], 0x7362), u3 = prmt(r[2], r[3], 0x7362);   // channels 2,3
          const uint32_t v0 = prmt(r[4], r[5], 0x5140), v2 = prmt(r[4], r[5], 0x7362);
          uint32_t ta[4], tw4[4];
          ta[0] = prmt(u0, u1, 0x5410);
          ta[1] = prmt(u0, u1, 0x7632);
          ta[2] = prmt(u2, u3, 0x5410);
          ta[3] = prmt(u2, u3, 0x7632);
          tw4[0] = prmt(ta[0], v0, 0x5432);
          tw4[1] = prmt(ta[1], v0, 0x7632);
          tw4[2] = prmt(ta[2], v2, 0x5432);
          tw4[3] = prmt(ta[3], v2, 0x7632);
#pragma unroll
          for (int f = 0; f < 3; ++f) {
            const int orow = i - f;   // the output row this input row reaches through filter row f
            if (orow >= 0 && orow < kRows) {
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                acc[orow % 3][0][k] = __dp4a((int)ta[k], (int)wa[f][k], acc[orow % 3][0][k]);
                acc[orow % 3][1][k] = __dp4a((int)ta[k], (int)wb[f][k], acc[orow % 3][1][k]);
                acc[orow % 3][2][k] = __dp4a((int)tw4[k], (int)wa[f][k], acc[orow % 3][2][k]);
                acc[orow % 3][3][k] = __dp4a((int)tw4[k], (int)wb[f][k], acc[orow % 3][3][k]);
              }
            }
          }
          if (i >= 2) {   // output row i - 2 is complete
            const int ho = ho0 + i - 2;
            if (ho < p.Ho) {
              int(&a)[4][4] = acc[(i - 2) % 3];
              const int64_t o0 = (((int64_t)n * p.Ho + ho) * p.Wo + wo0) * p.C + cw * 4;
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                if (wo0 + j < p.Wo) {
                  mn = min(__vimin3_s32(mn, a[j][0], a[j][1]), min(a[j][2], a[j][3]));
                  mx = max(__vimax3_s32(mx, a[j][0], a[j][1]), max(a[j][2], a[j][3]));
                  const int64_t o = o0 + (int64_t)j * p.C;
                  if constexpr (kOut == kOutInt8) {
                    uint32_t w;
                    if constexpr (kMode == kLeanNoClamp) w = requant_pack4<false>(a[j][0], a[j][1], a[j][2], a[j][3], q, qk);
                    else if constexpr (kMode == kLeanClamp) w = requant_pack4<true>(a[j][0], a[j][1], a[j][2], a[j][3], q, qk);
                    else w = quant4_acc(a[j][0], a[j][1], a[j][2], a[j][3], o, q, sat_below, sat_above);
                    *reinterpret_cast<uint32_t*>(reinterpret_cast<int8_t*>(p.out) + o) = w;
                  } else {
                    uint32_t w[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                      w[k] = (kOut == kOutF32) ? __float_as_uint(__fmul_rn(__int2float_rn(a[j][k]), q.s_acc)) : (uint32_t)a[j][k];
                    *reinterpret_cast<uint4*>(reinterpret_cast<uint32_t*>(p.out) + o) = make_uint4(w[0], w[1], w[2], w[3]);
                  }
                }
              }
            }
          }
        }
      }
      __syncthreads();   // every thread is done with this buffer
      if (threadIdx.x == 0 && tile + 2 * (int)gridDim.x < total) issue(tile + 2 * gridDim.x, buf);
    }
  };
  if (kOut != kOutInt8 || !q.fast || q.sr || q.count_sat) run_tiles(std::integral_constant<int, kGeneral>{});
  else if (q.noclamp) run_tiles(std::integral_constant<int, kLeanNoClamp>{});
  else run_tiles(std::integral_constant<int, kLeanClamp>{});

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

uint32_t depthwise_col_smem_bytes(const DwParams& p) {
  return 2u * p.patch_stride + (uint32_t)p.ncls * p.C * 4u + (uint32_t)p.Ho + (uint32_t)p.Wo + 256u;
}
cudaError_t depthwise_col_set_smem_attr(uint32_t smem_bytes) {
  cudaError_t e = cudaFuncSetAttribute(depthwise3x3_col_kernel<kOutInt8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(depthwise3x3_col_kernel<kOutF32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(depthwise3x3_col_kernel<kOutAcc>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
}

// threads: (C / 4) channel words x (TWt / 4) column groups; ctas_per_sm: how many CTAs of this size fit one SM
cudaError_t launch_depthwise_col(const DwParams& p, const CUtensorMap& tmap, int out_mode, int num_sms, int ctas_per_sm, cudaStream_t s,
                                 bool overlap) {
  const int threads = (p.C / 4) * (p.TWt / 4);
  const uint32_t smem = depthwise_col_smem_bytes(p);
  const int64_t total = (int64_t)p.N * p.tiles_h * p.tiles_w;
  const int grid = (int)std::max<int64_t>(1, std::min<int64_t>(total, (int64_t)num_sms * ctas_per_sm));
  switch (out_mode) {
    case kOutInt8: return launch_overlapped(depthwise3x3_col_kernel<kOutInt8>, grid, threads, smem, s, overlap, p, tmap);
    case kOutF32: return launch_overlapped(depthwise3x3_col_kernel<kOutF32>, grid, threads, smem, s, overlap, p, tmap);
    default: return launch_overlapped(depthwise3x3_col_kernel<kOutAcc>, grid, threads, smem, s, overlap, p, tmap);
  }
}

}  // namespace hq
