// Weight gradient of a 3x3 stride-1 depthwise layer with padding 1 (arxiv 2105.04246, Sec. 3.1: the backward pass forms the
// weight gradient from the quantized output gradient and the quantized layer input and keeps it in FP32):
//   g[c][r][s] = sum over output pixels (n,h,w) whose tap (h+r-1, w+s-1) lies inside the image of (dy - z_dy)(x - z_x).
// The sum of raw products runs on dp4a with FOUR PIXELS of one channel per word: both tensors are NHWC (a word = four
// channels of a pixel), so each thread transposes 4x4 byte blocks in registers, as the forward kernel of hq_dw3x3.cu does.
// A thread owns one channel word and a column of tiles 4 pixels wide and kWgRows high; per input row of the staged patch
// it forms the three horizontally shifted 4-pixel words of each channel and multiplies them with the transposed dY words
// of the three output rows that row pairs with: 36 dp4a per input row, every one of them four useful products.
// Padding and ragged tile edges arrive as zeros from the copy engine and contribute nothing to the raw sums; both zero
// points are taken out afterwards (dw_wgrad_finish_kernel) from per-channel totals, first/last row and column sums and
// corner pixels of both tensors, which the same kernel gathers over the pixels it owns:
//   sum_valid x  for tap (r,s) = total - (row the tap never reaches) - (column it never reaches) + (their corner).
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "hq_device.cuh"
#include "hq_internal.h"

namespace hq {
namespace {

constexpr int kWgRows = kDwColRows;   // output rows per tile; the input patch has kWgRows + 2

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) { return __byte_perm(a, b, sel); }

// four pixel words (4 channels each) -> four channel words (4 pixels each)
__device__ __forceinline__ void transpose4(const uint32_t (&r)[4], uint32_t (&t)[4]) {
  const uint32_t u0 = prmt(r[0], r[1], 0x5140), u1 = prmt(r[2], r[3], 0x5140);
  const uint32_t u2 = prmt(r[0], r[1], 0x7362), u3 = prmt(r[2], r[3], 0x7362);
  t[0] = prmt(u0, u1, 0x5410);
  t[1] = prmt(u0, u1, 0x7632);
  t[2] = prmt(u2, u3, 0x5410);
  t[3] = prmt(u2, u3, 0x7632);
}

// Layout of the per-channel sums in `out` (and in shared memory): kWgSlots rows of C ints.
//   0..8   raw products of tap r*3+s          9 total of x        10 total of dy
//   11..18 x:  first row, last row, first column, last column, corners (0,0) (0,W-1) (H-1,0) (H-1,W-1)
//   19..26 dy: the same
__global__ void __launch_bounds__(kDwColMaxThreads) dw_wgrad3x3_kernel(const DwWgradParams p, const __grid_constant__ CUtensorMap tmap_x,
                                                                       const __grid_constant__ CUtensorMap tmap_dy) {
  extern __shared__ uint8_t wsm_raw[];
  __shared__ __align__(8) uint64_t full_bar[2];
  __shared__ int abort_s;
  const uint32_t base0 = (smem_u32(wsm_raw) + 127u) & ~127u;
  uint8_t* gen = wsm_raw + (base0 - smem_u32(wsm_raw));
  // per buffer: the x patch, then the dy tile; after both buffers the sums
  int32_t* sum_s = reinterpret_cast<int32_t*>(gen + 2u * p.buf_stride);
  volatile int* abort_flag = &abort_s;
  const int CW = p.C / 4;
  const int cw = threadIdx.x % CW, g = threadIdx.x / CW;
  const uint32_t bar0 = smem_u32(full_bar);
  if (threadIdx.x == 0) {
    abort_s = 0;
    mbar_init(bar0, 1);
    mbar_init(bar0 + 8u, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&tmap_x) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&tmap_dy) : "memory");
  }
  for (int i = threadIdx.x; i < kDwWgSlots * p.C; i += blockDim.x) sum_s[i] = 0;
  __syncthreads();

  const int total = p.N * p.tiles_h * p.tiles_w;
  int armed[2] = {0, 0};
  auto issue = [&](int tile, int buf) {   // one thread: the x patch and the dy tile of `tile` into buffer `buf`
    const int tw = tile % p.tiles_w;
    const int th = (tile / p.tiles_w) % p.tiles_h;
    const int n = tile / (p.tiles_w * p.tiles_h);
    ++armed[buf];
    mbar_expect_tx(bar0 + 8u * buf, p.x_bytes + p.dy_bytes);
    tma_load_4d(base0 + buf * p.buf_stride, &tmap_x, 0, tw * p.TWt - 1, th * kWgRows - 1, n, bar0 + 8u * buf);
    tma_load_4d(base0 + buf * p.buf_stride + p.dy_offset, &tmap_dy, 0, tw * p.TWt, th * kWgRows, n, bar0 + 8u * buf);
  };
  if (threadIdx.x == 0) {
    if ((int)blockIdx.x < total) issue(blockIdx.x, 0);
    if ((int)(blockIdx.x + gridDim.x) < total) issue(blockIdx.x + gridDim.x, 1);
  }

  int acc[3][3][4];   // [filter row][filter column][channel]
  int tx[4] = {0, 0, 0, 0}, ty[4] = {0, 0, 0, 0};
#pragma unroll
  for (int r = 0; r < 3; ++r)
#pragma unroll
    for (int s = 0; s < 3; ++s)
#pragma unroll
      for (int k = 0; k < 4; ++k) acc[r][s][k] = 0;
  const int xrow_bytes = (p.TWt + 2) * p.C, dyrow_bytes = p.TWt * p.C;
  // Border sums.  Columns: a thread's four pixels lie in the same columns for every tile of its tile column, so the first /
  // last column sums are masked dot products into registers (mask 0 for threads that own neither).  Rows and corners
  // concern two image rows in H: the threads that meet them add to shared memory directly.
  int cfx[4] = {0, 0, 0, 0}, clx[4] = {0, 0, 0, 0}, cfy[4] = {0, 0, 0, 0}, cly[4] = {0, 0, 0, 0};
  auto border_rows = [&](int slot0, const uint32_t (&t)[4], int h, int m_fc, int m_lc) {
    const bool first_row = h == 0, last_row = h == p.H - 1;
    if (!(first_row || last_row)) return;
    int32_t* b = sum_s + slot0 * p.C + cw * 4;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int all = __dp4a((int)t[k], 0x01010101, 0), fc = __dp4a((int)t[k], m_fc, 0), lcv = __dp4a((int)t[k], m_lc, 0);
      atomicAdd(b + (first_row ? 0 : 1) * p.C + k, all);
      if (m_fc) atomicAdd(b + (first_row ? 4 : 6) * p.C + k, fc);
      if (m_lc) atomicAdd(b + (first_row ? 5 : 7) * p.C + k, lcv);
      if (first_row && last_row) {   // H == 1 is excluded by the host; kept for completeness of the definition
        atomicAdd(b + 1 * p.C + k, all);
        if (m_fc) atomicAdd(b + 6 * p.C + k, fc);
        if (m_lc) atomicAdd(b + 7 * p.C + k, lcv);
      }
    }
  };

  int it = 0;
  for (int tile = blockIdx.x; tile < total; tile += gridDim.x, ++it) {
    const int buf = it & 1;
    bool ok = mbar_wait(bar0 + 8u * buf, (uint32_t)(it >> 1) & 1u, abort_flag, p.status, kAsyncDepthwiseFullWait, 1000u);
    ok = __syncthreads_and(ok) != 0;
    if (!ok) break;
    const int tw = tile % p.tiles_w;
    const int th = (tile / p.tiles_w) % p.tiles_h;
    const int w0 = tw * p.TWt + 4 * g, h0 = th * kWgRows;
    if (w0 < p.W) {
      const int lc = p.W - 1 - w0;   // which of the thread's four pixels is the last column, if any
      const int m_fc = w0 == 0 ? 1 : 0, m_lc = (lc >= 0 && lc < 4) ? (1 << (8 * lc)) : 0;
      const uint8_t* px = gen + buf * p.buf_stride + (4 * g) * p.C + cw * 4;                  // x patch row 0, this thread's 6 columns
      const uint8_t* py = gen + buf * p.buf_stride + p.dy_offset + (4 * g) * p.C + cw * 4;    // dy tile row 0, this thread's 4 columns
      uint32_t dyt[3][4];   // transposed dy words of the last three output rows, [row mod 3][channel]
#pragma unroll
      for (int i = 0; i < kWgRows + 2; ++i) {
        if (i < kWgRows) {   // output row i: its dy words, their totals and border sums
          uint32_t r4[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) r4[j] = *reinterpret_cast<const uint32_t*>(py + i * dyrow_bytes + j * p.C);
          transpose4(r4, dyt[i % 3]);
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            ty[k] = __dp4a((int)dyt[i % 3][k], 0x01010101, ty[k]);
            cfy[k] = __dp4a((int)dyt[i % 3][k], m_fc, cfy[k]);
            cly[k] = __dp4a((int)dyt[i % 3][k], m_lc, cly[k]);
          }
          border_rows(19, dyt[i % 3], h0 + i, m_fc, m_lc);
        }
        // input row i of the patch: six pixels -> per channel pixels 0..3, 1..4, 2..5
        uint32_t r[6];
#pragma unroll
        for (int j = 0; j < 6; ++j) r[j] = *reinterpret_cast<const uint32_t*>(px + i * xrow_bytes + j * p.C);
        uint32_t xs[3][4];
        {
          const uint32_t ra[4] = {r[0], r[1], r[2], r[3]};
          transpose4(ra, xs[0]);
          const uint32_t v0 = prmt(r[4], r[5], 0x5140), v2 = prmt(r[4], r[5], 0x7362);
          xs[2][0] = prmt(xs[0][0], v0, 0x5432);
          xs[2][1] = prmt(xs[0][1], v0, 0x7632);
          xs[2][2] = prmt(xs[0][2], v2, 0x5432);
          xs[2][3] = prmt(xs[0][3], v2, 0x7632);
#pragma unroll
          for (int k = 0; k < 4; ++k) xs[1][k] = prmt(xs[0][k], xs[2][k], 0x6321);   // pixels 1, 2, 3 of the first and 4 (= byte 2 of pixels 2..5)
        }
        if (i >= 1 && i <= kWgRows) {   // the patch row that holds this thread's own pixels of image row h0 + i - 1
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            tx[k] = __dp4a((int)xs[1][k], 0x01010101, tx[k]);
            cfx[k] = __dp4a((int)xs[1][k], m_fc, cfx[k]);
            clx[k] = __dp4a((int)xs[1][k], m_lc, clx[k]);
          }
          border_rows(11, xs[1], h0 + i - 1, m_fc, m_lc);
        }
#pragma unroll
        for (int fr = 0; fr < 3; ++fr) {
          const int o = i - fr;   // the output row this input row pairs with through filter row fr
          if (o >= 0 && o < kWgRows) {
#pragma unroll
            for (int s = 0; s < 3; ++s)
#pragma unroll
              for (int k = 0; k < 4; ++k) acc[fr][s][k] = __dp4a((int)dyt[o % 3][k], (int)xs[s][k], acc[fr][s][k]);
          }
        }
      }
    }
    __syncthreads();   // every thread is done with this buffer
    if (threadIdx.x == 0 && tile + 2 * (int)gridDim.x < total) issue(tile + 2 * gridDim.x, buf);
  }
  if (*abort_flag != 0 && threadIdx.x == 0) {   // gave up: wait, bounded, for the copies still on their way
    for (int b = 0; b < 2; ++b)
      if (armed[b] > 0) mbar_drain(bar0 + 8u * b, (uint32_t)(armed[b] - 1) & 1u);
  }
  // registers -> CTA (shared memory) -> one atomic per sum and CTA
#pragma unroll
  for (int k = 0; k < 4; ++k) {
#pragma unroll
    for (int fr = 0; fr < 3; ++fr)
#pragma unroll
      for (int s = 0; s < 3; ++s)
        if (acc[fr][s][k] != 0) atomicAdd(sum_s + (fr * 3 + s) * p.C + cw * 4 + k, acc[fr][s][k]);
    if (tx[k] != 0) atomicAdd(sum_s + 9 * p.C + cw * 4 + k, tx[k]);
    if (ty[k] != 0) atomicAdd(sum_s + 10 * p.C + cw * 4 + k, ty[k]);
    if (cfx[k] != 0) atomicAdd(sum_s + 13 * p.C + cw * 4 + k, cfx[k]);
    if (clx[k] != 0) atomicAdd(sum_s + 14 * p.C + cw * 4 + k, clx[k]);
    if (cfy[k] != 0) atomicAdd(sum_s + 21 * p.C + cw * 4 + k, cfy[k]);
    if (cly[k] != 0) atomicAdd(sum_s + 22 * p.C + cw * 4 + k, cly[k]);
  }
  __syncthreads();
  for (int i = threadIdx.x; i < kDwWgSlots * p.C; i += blockDim.x)
    if (sum_s[i] != 0) atomicAdd(p.sums + i, sum_s[i]);
}

// Takes both zero points out of the raw sums and converts: for tap (r,s), with sums over the output pixels whose tap lies
// inside the image, g = raw - z_dy * sum x - z_x * sum dy + z_dy * z_x * count; GW is [C][3][3].
__global__ void dw_wgrad_finish_kernel(const int32_t* __restrict__ sums, int C, int N, int H, int W, const hq_range_state* __restrict__ dyq,
                                       const hq_range_state* __restrict__ xq, float* __restrict__ G) {
  const float sc = __fmul_rn(dyq->scale, xq->scale);
  const int zdy = dyq->zero_point, zx = xq->zero_point;
  for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < C * 9; idx += gridDim.x * blockDim.x) {
    const int c = idx / 9, t = idx - c * 9, r = t / 3, s = t - r * 3;
    auto at = [&](int slot) { return (uint32_t)sums[slot * C + c]; };
    // x: filter row 0 never reaches the last image row, filter row 2 never the first (columns alike);
    // dy: filter row 0 has no input for the first output row, filter row 2 none for the last
    const int xb = 11, yb = 19;
    uint32_t sx = at(9), sy = at(10);
    if (r == 0) { sx -= at(xb + 1); sy -= at(yb + 0); }
    if (r == 2) { sx -= at(xb + 0); sy -= at(yb + 1); }
    if (s == 0) { sx -= at(xb + 3); sy -= at(yb + 2); }
    if (s == 2) { sx -= at(xb + 2); sy -= at(yb + 3); }
    if (r == 0 && s == 0) { sx += at(xb + 7); sy += at(yb + 4); }
    if (r == 0 && s == 2) { sx += at(xb + 6); sy += at(yb + 5); }
    if (r == 2 && s == 0) { sx += at(xb + 5); sy += at(yb + 6); }
    if (r == 2 && s == 2) { sx += at(xb + 4); sy += at(yb + 7); }
    const uint32_t count = (uint32_t)N * (uint32_t)(H - (r != 1 ? 1 : 0)) * (uint32_t)(W - (s != 1 ? 1 : 0));
    uint32_t gsum = at(t);
    gsum -= (uint32_t)zdy * sx;
    gsum -= (uint32_t)zx * (sy - (uint32_t)zdy * count);
    G[idx] = __fmul_rn(__int2float_rn((int)gsum), sc);
  }
}

}  // namespace

uint32_t dw_wgrad3x3_smem_bytes(const DwWgradParams& p) { return 2u * p.buf_stride + (uint32_t)kDwWgSlots * p.C * 4u + 256u; }
cudaError_t dw_wgrad3x3_set_smem_attr(uint32_t smem_bytes) {
  return cudaFuncSetAttribute(dw_wgrad3x3_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
}
cudaError_t launch_dw_wgrad3x3(const DwWgradParams& p, const CUtensorMap& tmap_x, const CUtensorMap& tmap_dy, int num_sms,
                               const hq_range_state* dyq, const hq_range_state* xq, float* G, cudaStream_t s) {
  const int threads = (p.C / 4) * (p.TWt / 4);
  const int64_t total = (int64_t)p.N * p.tiles_h * p.tiles_w;
  const int grid = (int)std::max<int64_t>(1, std::min<int64_t>(total, num_sms));
  dw_wgrad3x3_kernel<<<grid, threads, dw_wgrad3x3_smem_bytes(p), s>>>(p, tmap_x, tmap_dy);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  dw_wgrad_finish_kernel<<<std::max(1, std::min(64, (p.C * 9 + 255) / 256)), 256, 0, s>>>(p.sums, p.C, p.N, p.H, p.W, dyq, xq, G);
  return cudaGetLastError();
}

}  // namespace hq
