// Internal declarations shared by the translation units of libhq (host side + kernel params).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <initializer_list>
#include <string>
#include <utility>
#include <vector>

#include "hq.h"

namespace hq {

constexpr int kMaxTaps = 49;          // 7x7
constexpr int kTileM = 128;           // rows of one accumulator tile = TMEM lanes
constexpr int kEpilogueSlices = 4;    // epilogue warps per TMEM lane quarter; they split the columns
constexpr int kEpilogueWarps = 4 * kEpilogueSlices;
constexpr int kFirstEpilogueWarp = 4; // warps 0..3: A producer, MMA issuer, B producer, spare
constexpr int kGemmThreads = 32 * (kFirstEpilogueWarp + kEpilogueWarps);
constexpr int kMaxStagesA = 12;
constexpr int kMaxStagesB = 32;
constexpr uint32_t kSmemBudget = 212 * 1024;              // operand rings + correction table; barriers sit in static shared memory
constexpr uint32_t kMaxZcBytes = 20 * 1024;               // largest correction table kept in shared memory
constexpr long long kWaitLimitCycles = 4000000000ll;      // bound of every device-side wait, in SM cycles (2 to 4 seconds)

// status-word codes written by kernels when a bounded wait expires
enum AsyncCode : int32_t {
  kAsyncOk = 0,
  kAsyncProducerEmptyWait = 1,
  kAsyncMmaFullWait = 2,
  kAsyncMmaTmemEmptyWait = 3,
  kAsyncEpilogueTmemFullWait = 4,
  kAsyncProducerBEmptyWait = 5,
  kAsyncMmaBFullWait = 6,
  kAsyncDepthwiseFullWait = 7,
};

// Fixed-capacity list for the planner's small tables (tap offsets, border-class masks): planning a layer call makes no
// host heap allocation, so the calls that promise to allocate nothing may plan too.
template <typename T, int kCap>
struct SmallVec {
  T v[kCap];
  int n = 0;
  SmallVec() = default;
  SmallVec(std::initializer_list<T> il) { for (const T& x : il) push_back(x); }
  void push_back(const T& x) { if (n < kCap) v[n++] = x; }
  void clear() { n = 0; }
  void assign(int count, const T& x) { n = 0; for (int i = 0; i < count; ++i) push_back(x); }
  size_t size() const { return (size_t)n; }
  bool empty() const { return n == 0; }
  T& operator[](size_t i) { return v[i]; }
  const T& operator[](size_t i) const { return v[i]; }
  T* begin() { return v; }
  T* end() { return v + n; }
  const T* begin() const { return v; }
  const T* end() const { return v + n; }
  T* data() { return v; }
  const T* data() const { return v; }
};
using TapVec = SmallVec<int, 8>;          // tap offsets of one axis (filters up to 7 wide)
using MaskVec = SmallVec<uint32_t, 64>;   // border-class masks of one axis (more than 16 are refused)

struct FastDiv {                      // n / d == (umulhi(m, n) + n) >> l for 0 <= n < 2^31
  uint32_t m, l;
};

enum OutMode : int { kOutInt8 = 0, kOutF32 = 1, kOutAcc = 2 };
enum GemmMode : int { kModeTap = 0, kModeHalo = 1 };

// One launch of the tensor-core kernel: an implicit GEMM over a "tile space" of output pixels.
//   tile-space pixel (n, i, j), i in [0,TH), j in [0,TW)
//   output pixel     (n, i*os_h + oa_h, j*os_w + oa_w) in an out_H x out_W image of ldY elements per pixel
//   operand A, tap t (n, i*in_mul_h + tap_dh[t], j*in_mul_w + tap_dw[t], c); out-of-image coordinates read as zero
//   operand B        weight matrix [Nout][ntaps][Cpad], K-major
//
// kModeTap : every (tap, channel chunk) is one ring stage = one TMA box of A (128 pixels x BK bytes) and one of B.
// kModeHalo: stride-1 tile spaces only.  The output pixels of an image are numbered o = i*P + j with
//            P = TW + (max tap_dw - min tap_dw) (j >= TW are dead columns); a tile is 128 consecutive o.  One TMA
//            box per channel chunk brings the NR padded input rows the tile touches into shared memory once, and
//            tap (dr, ds) reads them through a matrix descriptor whose start is shifted by (dr*P + ds) pixels.
//            Only the weights stream through the B ring (or stay resident when they fit).
struct GemmParams {
  int32_t mode;
  int32_t n_img, TH, TW;
  int32_t Nt, Ht, Wt;                 // kModeTap: Nt*Ht*Wt == kTileM
  int32_t tiles_n, tiles_h, tiles_w, tiles_col, num_tiles;
  int32_t in_mul_h, in_mul_w;
  int32_t ntaps, chunks_per_tap, BK, Cpad;
  int8_t tap_dh[kMaxTaps], tap_dw[kMaxTaps];
  // kModeHalo
  int32_t P, L, NR, tiles_per_img, dh_min, dw_min;
  uint32_t patch_chunk_stride;        // bytes between channel chunks of one patch (1024-aligned)
  uint32_t patch_box_bytes;           // bytes one patch TMA delivers
  int32_t b_resident;
  int32_t out_col0;                   // column of the output tensor that column 0 of this launch writes (channel slices)
  int32_t weights_early;              // the weight producer may start before the previous kernel in the stream has finished
  // common
  int32_t Nout, BN;
  int32_t out_H, out_W, os_h, os_w, oa_h, oa_w;
  int64_t ldY;
  const int32_t* corr;                // [ncls][corr_ld]: sum of the weights of the taps valid in that border class
  int32_t corr_ld, ncolcls;
  const uint8_t* rowcls;              // [TH] or null (single class)
  const uint8_t* colcls;              // [TW] or null
  int32_t cls_in_smem;                // both tables are non-null and fit the kernel's shared copy (TH, TW <= 512)
  const int32_t* bias;                // [Nout] or null
  int32_t b_slice;                    // kModeTap, streamed weights: image n of the tile space reads operand B at reduction offset n * b_slice
  // kModeTap, streamed operand B shared by groups of column tiles (weight gradient of a stride-1 convolution): column tile ct
  // reads rows (ct % b_group_tiles) * BN at reduction offset + b_k_base + (ct / b_group_tiles) * b_k_step; 0 = off
  int32_t b_group_tiles, b_k_base, b_k_step;
                                      // (the reduction of one GEMM cut into slices that run as "images"; 0 otherwise)
  const int32_t* row_term;            // [output pixels] or null: subtracted from every accumulator of the pixel (weight zero point times
                                      // the pixel's input sum; the weight gradient's input-zero-point term)
  int32_t rt_fold, rt_cols;           // a GEMM row holds rt_fold pixels of rt_cols columns each (folded 1x1 layers; else 1, Nout)
  float acc_bound;                    // upper bound of |accumulator| before the bias: reduction length x 255 x 128
  const hq_range_state* xq;
  const float* w_scale;
  hq_range_state* yq;
  void* out;
  int32_t* status;
  uint32_t idesc;
  uint32_t tmem_cols, tmem_buf_stride;
  int32_t mma_issuers;                // 1, 2 or 3 warps issuing MMAs (tiles in turn)
  int32_t a_producers;                // kModeTap with resident weights: 1, or 2 = the weight producer's warp copies operand A for every second tile
  int32_t pair;                       // 1: launched as clusters of two CTAs that share 256-row tiles (tcgen05 cta_group::2);
                                      //    stage_bytes_b and the B tensor map's box then cover BN/2 rows
  int32_t num_pair_tiles;             // pair tiles (two row tiles x one column tile)
  int32_t tmem_bufs, tmem_bufs_log2;   // accumulator buffers in TMEM (2, 4 or 8)
  int32_t epi_groups_log2;             // epilogue warp groups: 1, 2 or 4 (<= buffers)
  int32_t stages_a, stages_b;
  uint32_t stage_bytes_a, stage_bytes_b;   // kModeTap: A and B part of one stage; kModeHalo: patch stage, B stage
  int32_t swizzle64;                  // 1: 64-byte swizzle (BK = 64), 0: 128-byte swizzle (BK = 128)
  int32_t producer_lanes;             // kModeTap: lanes of the producer warp that issue copies
  FastDiv fd_tiles_col, fd_tiles_per_img, fd_tiles_w, fd_tiles_h, fd_P;
  int32_t zc_in_smem, zc_elems;       // zero-point correction table copied (pre-multiplied) into shared memory
  uint32_t zc_offset;                 // its byte offset from the ring base
};

struct DwParams {                     // depthwise (CUDA cores)
  int32_t N, H, W, C, Ho, Wo, R, S, stride_h, stride_w, pad_h, pad_w;
  const int8_t* x;
  const int8_t* w;                    // [R*S][C] tap-major
  const int32_t* corr;                // [ncls][C]
  const uint8_t* rowcls;
  const uint8_t* colcls;
  int32_t ncolcls;
  const hq_range_state* xq;
  const float* w_scale;
  hq_range_state* yq;
  void* out;
  int32_t w_zp;                       // weight zero point; non-zero layers run the generic kernel with (x - z_x) * (w - z_w) formed directly
  // tiled 3x3 kernel: output tile of TR rows x TWt columns, input patch of (TR + 2) x (TWt + 2) pixels in shared memory
  int32_t TR, TWt, tiles_h, tiles_w, slots, ncls;
  uint32_t patch_bytes;               // bytes one TMA box delivers
  uint32_t patch_stride;              // patch_bytes rounded up to 128: distance of the two buffers (TMA destinations are 128-byte aligned)
  int32_t* status;                    // device status word (expired waits)
};

// Fused forward convolution over few input channels (hq_gather.cu): raw input rows by TMA, im2col rows gathered in shared memory
struct GatherParams {
  int32_t N, H, W, C, Ho, Wo, R, S, stride_h, stride_w, pad_h, pad_w;
  int32_t BN;                          // output channels (a multiple of 16, at most 256): one column tile
  int32_t tiles_w, num_tiles;          // tiles of up to 128 output pixels per output row; N * Ho * tiles_w
  int32_t span, tiles_img, box_rows;   // span = 1 (output rows shorter than a tile): a tile is 128 consecutive pixels of one image in
                                       // row-major order (tiles_img per image, num_tiles = N * tiles_img) and its raw box holds the
                                       // box_rows input rows under every output row it touches; span = 0: box_rows = R
  uint32_t raw_pitch;                  // bytes of one raw row in shared memory = width of the TMA box (a multiple of 16, at most 1024)
  uint32_t raw_box_bytes, raw_stage_stride;   // raw_pitch * box_rows, and that rounded up to 128
  uint32_t a_stage_bytes;              // 128 * Kp
  int32_t stages_raw, stages_a;
  uint32_t off_w, off_zc, off_raw, off_a;   // byte offsets from the 1024-aligned base of dynamic shared memory
  const int32_t* corr;                 // [ncls][corr_ld]
  int32_t zc_elems, corr_ld, ncolcls;
  const uint8_t* rowcls;               // [Ho]
  const uint8_t* colcls;               // [Wo]
  int32_t cls_in_smem;
  const int8_t* wmat;                  // [BN][Kp]: the filter in its own (r, s, c) order, rows zero padded to Kp
  const hq_range_state* xq;
  const float* w_scale;
  hq_range_state* yq;
  void* out;
  int32_t* status;
  uint32_t idesc, tmem_cols, tmem_buf_stride;
  int32_t tmem_bufs, epi_groups;       // powers of two
  int32_t tmem_bufs_log2, epi_groups_log2;
  FastDiv fd_tiles_w, fd_Ho, fd_Wo, fd_tiles_img;
  int32_t weights_early;
  float acc_bound;
};
struct ClassMasksG {
  uint32_t row[16], col[16];
};
bool gather_conv_supported(int R, int SC);
cudaError_t launch_gather_conv(const GatherParams& p, const CUtensorMap& tm, int out_mode, int grid, uint32_t smem, cudaStream_t s, bool overlap);
cudaError_t launch_gather_corr(const int8_t* W, int32_t* corr, int K, int R, int S, int C, const uint32_t* rowmasks, int nrowcls,
                               const uint32_t* colmasks, int ncolcls, int corr_ld, cudaStream_t s);

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Launch that lets the kernel become resident while its predecessor in the stream is still draining (programmatic
// stream serialization).  Kernels launched this way run their set-up (barrier initialisation, TMEM allocation,
// descriptor prefetch) early and execute grid_dependency_wait() before they touch any memory a predecessor may
// have written; they also release their own successor at once, which then waits the same way, so the order of
// memory effects in the stream is unchanged.  overlap = false is an ordinary launch (the two device calls are
// no-ops then).
template <typename... KArgs, typename... Args>
cudaError_t launch_overlapped(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, bool overlap, Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = overlap ? 1u : 0u;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}
// the same, as thread-block clusters of `cluster` consecutive CTAs (grid.x a multiple of it)
template <typename... KArgs, typename... Args>
cudaError_t launch_overlapped_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, bool overlap, unsigned cluster,
                                      Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cluster;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = overlap ? 2u : 1u;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}
#ifdef __CUDACC__
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
#endif

// kernel launchers (defined in the .cu files); `overlap` as in launch_overlapped
cudaError_t launch_gemm(const GemmParams& p, const CUtensorMap& ta, const CUtensorMap& tb, int out_mode, int grid, uint32_t smem_bytes,
                        cudaStream_t s, bool overlap);
cudaError_t gemm_set_smem_attr(uint32_t smem_bytes);
cudaError_t launch_depthwise(const DwParams& p, int out_mode, int num_sms, cudaStream_t s, bool overlap);
// 3x3 stride-1 depthwise with the input patch staged by TMA (p.TR ... p.status filled in); tmap covers the NHWC input
cudaError_t launch_depthwise_tiled(const DwParams& p, const CUtensorMap& tmap, int out_mode, int num_sms, cudaStream_t s);
// 3x3 stride-1 depthwise, columns of tiles of kDwColRows x 4 pixels per thread (hq_dw3x3.cu): TR = kDwColRows, TWt a multiple of 4
constexpr int kDwColRows = 7;
constexpr int kDwColMaxThreads = 448;
// weight gradient of a 3x3 stride-1 pad-1 depthwise layer (hq_dw_wgrad.cu)
constexpr int kDwWgSlots = 27;          // rows of C ints in the sum buffer: 9 taps, 2 totals, 8 border sums per tensor
struct DwWgradParams {
  int32_t N, H, W, C;                   // H == Ho, W == Wo
  int32_t TWt, tiles_h, tiles_w;        // tiles of kDwColRows rows x TWt columns (a multiple of 4)
  uint32_t x_bytes, dy_bytes;           // bytes the two TMA boxes of a tile deliver
  uint32_t dy_offset, buf_stride;       // dy tile behind the x patch; distance of the two buffers (multiples of 128)
  int32_t* sums;                        // [kDwWgSlots][C], zeroed by the caller
  int32_t* status;
};
cudaError_t launch_dw_wgrad3x3(const DwWgradParams& p, const CUtensorMap& tmap_x, const CUtensorMap& tmap_dy, int num_sms,
                               const hq_range_state* dyq, const hq_range_state* xq, float* G, cudaStream_t s);
cudaError_t dw_wgrad3x3_set_smem_attr(uint32_t smem_bytes);
uint32_t dw_wgrad3x3_smem_bytes(const DwWgradParams& p);
cudaError_t launch_depthwise_col(const DwParams& p, const CUtensorMap& tmap, int out_mode, int num_sms, int ctas_per_sm, cudaStream_t s, bool overlap);
cudaError_t depthwise_col_set_smem_attr(uint32_t smem_bytes);
uint32_t depthwise_col_smem_bytes(const DwParams& p);
cudaError_t depthwise_tiled_set_smem_attr(uint32_t smem_bytes);
uint32_t depthwise_tiled_smem_bytes(const DwParams& p);
cudaError_t launch_range_update(hq_range_state* st, int count, float eta, cudaStream_t s, bool overlap);
cudaError_t launch_dynamic_derive(hq_range_state* st, cudaStream_t s, bool overlap);
cudaError_t launch_stats_pack(const hq_range_state* st, int count, int32_t* buf, cudaStream_t s);
cudaError_t launch_stats_unpack(hq_range_state* st, int count, const int32_t* buf, cudaStream_t s);
// MMA-only throughput probe (measurement): one CTA or CTA pair per SM, `chunks` x 32 MMAs of 128 (pair: 256) x bn x 32 each
cudaError_t launch_mma_peak(int pair, int bn, int chunks, int num_sms, int32_t* status, cudaStream_t s, uint64_t* ops);
cudaError_t launch_quantize_pass(const float* y, int8_t* out, int64_t count, hq_range_state* st, int num_sms, cudaStream_t s,
                                 bool overlap);
cudaError_t launch_prep_weights(const int8_t* W, int8_t* Wmat, int Nout, int ntaps, int Cpad, int Ksrc, int R, int S, int Csrc,
                                const int8_t* tap_r, const int8_t* tap_s, int transposed, int blockdiag_g, cudaStream_t s);
cudaError_t launch_corr(const int8_t* Wmat, int32_t* corr, int Nout, int ntaps, int Cpad, int nrowtaps, int ncoltaps, const uint32_t* rowmasks,
                        int nrowcls, const uint32_t* colmasks, int ncolcls, int corr_ld, cudaStream_t s);
cudaError_t launch_patch_matrix(const int8_t* x, int8_t* A, const hq_range_state* xq, int N, int H, int W, int C, int Ho, int Wo, int R, int S,
                                int stride_h, int stride_w, int pad_h, int pad_w, int Kp, int RP, cudaStream_t s);
cudaError_t launch_row_window(const int8_t* x, int8_t* X2, const hq_range_state* xq, int N, int H, int W, int C, int Hg, int Wo, int S, int sh,
                              int stride_w, int pad_w, int SB, cudaStream_t s);
cudaError_t launch_prep_window_weights(const int8_t* W, int8_t* Wmat, int K, int R, int SC, int sh, int SB, int ntaps, int dh_min, int pad_h,
                                       cudaStream_t s);
cudaError_t launch_prep_patch_weights(const int8_t* W, int8_t* Wmat, int K, int R, int SC, int RP, int ld, cudaStream_t s);
cudaError_t launch_pad_rows(const int8_t* src, int8_t* dst, int rows, int K, int Kp, cudaStream_t s);
cudaError_t launch_transpose_rows(const int8_t* in, int8_t* out, int R, int C, int Rp, int ones_row, cudaStream_t s);
cudaError_t launch_im2col_t(const int8_t* X, int8_t* Bt, const hq_range_state* xq, const hq_conv_desc& d, int Ho, int Wo, int64_t Mp, int32_t* colsum,
                            FastDiv fd_wo, FastDiv fd_ho, cudaStream_t s);
// depthwise weight gradient, 3x3 or 5x5 filters, C a multiple of 4 and at most 1024; acc: C*R*S zeroed int32
cudaError_t launch_dw_wgrad(const int8_t* dY, const int8_t* X, const hq_range_state* dyq, const hq_range_state* xq, const hq_conv_desc& d, int Ho,
                            int Wo, int num_sms, FastDiv fd_wo, FastDiv fd_ho, int32_t* acc, float* G, cudaStream_t s);
// Weight gradient of a stride-1 convolution: packs a [N][Hs][Ws][Cs] tensor into channel-major rows over a padded pixel
// index ((n * Hp + row_off + h) * P + w) in horizontally shifted views; sums per (filter row, filter column, channel) go to
// `sums` (see the kernel)
struct PackRanges {
  int32_t nr, ns;                      // filter rows, filter columns
  int16_t row_lo[8], row_hi[8];        // source rows that filter row r pairs with a row inside the other tensor
};
struct TapCounts {
  int32_t v[kMaxTaps + 15];
};
cudaError_t launch_wgrad_pack(const int8_t* src, int8_t* dst, int N, int Hs, int Ws, int Cs, int Hp, int P, int row_off, int sign, int pad, int limit,
                              int64_t pitch, const PackRanges& rg, int32_t* sums, cudaStream_t s);
cudaError_t launch_zero_tail(int8_t* base, int rows, int64_t pitch, int64_t from, cudaStream_t s);
cudaError_t launch_wgrad_reduce_taps(const int32_t* slabs, int nslabs, int rows, int slab_rows, int cols, int C, const int32_t* colsum,
                                     const int32_t* rowsum, const TapCounts& mvalid, const hq_range_state* dyq, const hq_range_state* xq, float* G,
                                     cudaStream_t s);
cudaError_t launch_wgrad_reduce(const int32_t* slabs, int nslabs, int rows, int cols, const int32_t* colsum, const int32_t* rowsum, int M,
                                const hq_range_state* dyq, const hq_range_state* xq, float* G, cudaStream_t s);
cudaError_t launch_wgrad_row_terms(const int8_t* dYt, int M, int Mp, int N, const hq_range_state* dyq, const hq_range_state* xq, int32_t* terms,
                                   cudaStream_t s);
// sum over the in-image taps and the channels of (a - z_a), times zw, per output pixel of the layer (forward: over the
// input windows; backward data: over the output-gradient pixels that reach the input pixel): the weight-zero-point term
cudaError_t launch_rowsum(const int8_t* a, const hq_range_state* aq, const hq_conv_desc& d, int Ho, int Wo, int bwd, int zw, int32_t* out,
                          cudaStream_t s);
// backward data of a depthwise layer with any stride, direct arithmetic (one input pixel x 16 channels per thread)
cudaError_t launch_depthwise_bwd(const DwParams& p, int out_mode, int num_sms, cudaStream_t s);
cudaError_t launch_dw_dense(const int8_t* W, int8_t* Wd, int taps, int c0, int cw, cudaStream_t s);
cudaError_t launch_dw_prep(const int8_t* W, int8_t* Wt, int32_t* corr, int C, int R, int S, const uint32_t* rowmasks, int nrowcls,
                           const uint32_t* colmasks, int ncolcls, int flip, cudaStream_t s);

}  // namespace hq

struct hq_ctx {
  int device = 0;
  int num_sms = 0;
  int32_t* d_status = nullptr;
  int32_t* d_scratch = nullptr;       // column sums of linear weights
  size_t scratch_elems = 0;
  int8_t* d_pad = nullptr;            // zero-padded operand copies for linear layers whose K is not a multiple of 16
  size_t pad_bytes = 0;
  uint8_t* d_wgrad = nullptr;         // weight gradient: transposed operands, int32 accumulators, one range state
  size_t wgrad_bytes = 0;
  hq::EncodeTiledFn encode = nullptr;
  uint64_t launches = 0;
  uint64_t pair_launches = 0;         // of those, layer kernels launched as CTA pairs
  int force_mode = -1;                // -1: choose per layer; else hq::GemmMode where the layer allows it
  int force_dw_tiled = -1;            // depthwise 3x3 stride 1 on CUDA cores: -1 choose, 0 direct loads, 1 patches staged by TMA
  int force_depthwise = -1;           // depthwise layers: -1 choose, 0 CUDA-core kernel, 1 dense expansion on the tensor cores
  int a_producers = -1;               // warps copying operand A in 1x1 layers with resident weights: -1 choose, 1, 2 where the layer allows
  int gather_span = 1;                // few-channel fused kernel: 1 = tiles may run across the ends of short output rows, 0 = one output row per tile
  int force_repack = -1;              // small-C spatial filters: -1 choose, 0 patch rows, 1 window rows where possible
  int force_epi_groups = -1;          // log2 of the epilogue warp groups: -1 chosen per layer, else min(value, log2 of the accumulator buffers)
  int force_cols = -1;                // column tiles: -1 chosen by estimated duration, 0 as wide as the MMA allows, n > 0 at least n
  int force_pair = -1;                // CTA pairs on 256-row tiles: -1 choose per layer, 0 never, 1 wherever the layer allows
  int wgrad_windows = -1;             // dense weight gradient: -1 choose, 0 packed tensors wherever the shape allows, 1 always filter-window copies
  int max_issuers = 3;                // upper limit of the warps that issue MMAs in one CTA (1, 2 or 3)
  cudaStream_t side[3] = {nullptr, nullptr, nullptr};   // independent launches of one call run side by side (see run_conv)
  cudaEvent_t ev_fork = nullptr, ev_join[3] = {nullptr, nullptr, nullptr};
  bool parallel_subs = true;
  bool overlap = true;                // launch the hot-path kernels with programmatic stream serialization
  char err[512] = {0};               // HOST text of the last rejected call (fixed storage: rejecting a call allocates nothing)
};

struct hq_sub_problem {               // one kernel launch of a prepared convolution
  hq::GemmParams p{};                 // everything except per-call pointers
  CUtensorMap tmap_b{};
  int8_t* wmat = nullptr;
  int32_t* corr = nullptr;
  uint8_t* rowcls = nullptr;
  uint8_t* colcls = nullptr;
  uint32_t smem_bytes = 0;
  int a_stride_h = 1, a_stride_w = 1; // traversal strides of the A tensor map
  int a_flat = 0;                     // 1: A is viewed as [pixels][C] (1x1 stride-1 layers and linear)
  int gfold = 1;                      // pixels folded into one GEMM row (channel counts that are not multiples of 16)
  int8_t* patch_matrix = nullptr;     // [pixels][patch_K]: filter windows gathered by a pre-pass (C not a multiple of 16)
  int patch_K = 0;
  int patch_RP = 0;                   // bytes per filter-row slot in a patch-matrix row
  int8_t* window = nullptr;           // [N][Hg][Wo][win_sh * win_SB]: horizontal filter windows of win_sh input rows per pixel
  int win_sh = 0, win_SB = 0, win_Hg = 0;
  int chan0 = 0, chans = 0;           // depthwise on the tensor cores: this launch covers channels [chan0, chan0 + chans)
};

struct hq_prepared_weights {
  hq_conv_desc desc{};
  hq_direction dir = HQ_DIR_FWD;
  bool depthwise = false;
  bool dw_bwd_direct = false;         // depthwise backward data that runs the direct kernel (strided layers, non-zero weight zero point)
  int8_t* dw_w_plain = nullptr;       // its weights, tap-major [R*S][C], not turned
  int32_t w_zp = 0;                   // weight zero point (asymmetric weights); 0: symmetric
  int32_t* row_term = nullptr;        // w_zp != 0: scratch for w_zp * (input sum of every output pixel), written by each call
  size_t row_term_elems = 0;
  // few-channel spatial filter run by the fused gather kernel (hq_gather.cu)
  bool gather = false;
  hq::GatherParams gp{};
  uint32_t gather_smem = 0;
  // prepared weights of a linear layer (hq_linear_prepare)
  bool linear = false;
  int lin_N = 0, lin_K = 0, lin_Kp = 0, lin_maxM = 0;
  int8_t* lin_w = nullptr;            // [N][Kp], zero padded to a multiple of 16 columns
  int32_t* lin_corr = nullptr;        // column sums of the weights (zero padded), for the input zero point
  int8_t* lin_xpad = nullptr;         // Kp != K: room for the padded copy of the input, lin_maxM rows
  hq_conv_desc dw_run{};              // geometry the depthwise kernel runs: desc itself (forward) or, for backward data of a stride-1
                                      // layer, the forward layer over the output gradient with the turned filter
  mutable bool used = false;          // set by the first layer call: later calls know that the tables were complete long before
  std::vector<hq_sub_problem> subs;
  // depthwise tables
  int8_t* dw_w = nullptr;
  int32_t* dw_corr = nullptr;
  uint8_t* dw_rowcls = nullptr;
  uint8_t* dw_colcls = nullptr;
  int dw_ncolcls = 1;
  int dw_ncls = 1;                    // border classes (rows x columns) of the depthwise correction table
  std::vector<void*> allocs;          // everything to cudaFree on release
};
