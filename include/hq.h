/* hq.h -- C ABI of the in-hindsight int8 quantized-layer library for NVIDIA B200 (sm_100a).
 *
 * Method: "In-Hindsight Quantization Range Estimation for Quantized Training",
 * arxiv 2105.04246.  Section/equation numbers below refer to that paper.
 *
 * What the calls compute, in the paper's terms:
 *   - a layer call is the MAC of 8-bit operands into 32-bit accumulators (Sec. 3.1) whose
 *     output is quantized "directly", with a range known in advance (static quantization,
 *     Sec. 3.2) -- here the range estimated on earlier iterations (Sec. 4, step 1) -- while
 *     min/max of the unquantized output are taken at the accumulator (Sec. 4, step 2);
 *   - hq_range_update applies the moving average of Eq. 2-3 (Sec. 4.1) once the whole
 *     output tensor exists, giving the range of the next iteration;
 *   - hq_dynamic_quant is the comparison path of Sec. 3.2 / Eq. 1 / Eq. 5: the 32-bit
 *     output goes to memory, the range is taken from the current tensor, the output is
 *     read back and quantized.
 *
 * General rules of the boundary
 *   - Plain C: no C++ types, no exceptions.  Every call returns an hq_status.
 *   - Unless marked HOST, every pointer argument is a DEVICE pointer owned by the caller.
 *     The library never allocates, frees or keeps caller tensors; it owns only the
 *     context, prepared weights and their internal tables.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Layer,
 *     update and dynamic calls only enqueue work: they do not synchronise and read every
 *     quantization parameter from device memory.  The exceptions are spelled out at the calls
 *     concerned: a call that first meets a shape needing more context-owned scratch than the
 *     context holds grows it with cudaFree + cudaMalloc (which synchronise the device), so make
 *     the first call of each such shape outside stream capture and timed regions.
 *   - The context's device must be the current device for every call that launches work
 *     (HQ_ERR_INVALID_ARG otherwise).
 *   - Context-owned scratch is shared by the calls of one context: the column sums of
 *     hq_linear_fwd / hq_dynamic_quant(linear), the padded copies for K % 16 != 0, and the
 *     weight-gradient scratch.  Calls of ONE context that use the same scratch must not overlap
 *     on the GPU (different streams); use one context per stream for that.
 *   - Arguments are validated before anything is launched; a rejected call launches
 *     nothing and hq_last_error() holds a HOST string describing the reason.
 *   - Every device-side wait is bounded.  If one expires the kernel records a code in the
 *     context's device status word and ends normally; hq_get_async_error() reads it.
 *   - Tensors are dense int8: activations and gradients NHWC, linear operands row-major
 *     [rows][K], convolution weights [K_out][R][S][C_in] (depthwise: [C][R][S]).
 *     Base pointers must be 16-byte aligned.
 */
#ifndef HQ_H_
#define HQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  HQ_OK = 0,
  HQ_ERR_INVALID_ARG = 1,     /* null pointer, non-positive size, inconsistent descriptor      */
  HQ_ERR_UNSUPPORTED = 2,     /* a shape this build has no kernel for                          */
  HQ_ERR_ALIGNMENT = 3,       /* pointer or leading dimension breaks a 16-byte rule            */
  HQ_ERR_CUDA = 4,            /* a CUDA runtime/driver call failed (see hq_last_error)         */
  HQ_ERR_NOT_INITIALIZED = 5, /* library built without / running without its device code       */
  HQ_ERR_TIMEOUT = 6          /* a bounded device-side wait expired (hq_get_async_error)       */
} hq_status;

/* Per-tensor quantizer state, device resident, 64 bytes, 16-byte aligned, plain data:
 * a checkpoint of the method's whole state is a copy of the array of these.
 *   acc_min/acc_max  statistics slot (Sec. 4 step 2): min and max of the zero-point-corrected
 *                    int32 accumulator of the tensor, merged by the layer kernels with atomics.
 *                    Empty slot = {INT32_MAX, INT32_MIN}.
 *   acc_scale        real value of one accumulator unit, fl(s_x * s_w), written by the layer call.
 *   step             number of range updates applied so far; 0 = no range yet (t = 0, Sec. 4.1).
 *   q_min/q_max      running range of Eq. 2-3.
 *   scale, inv_scale, zero_point   the 2^8-level grid derived from the running range:
 *                    lo = min(q_min,0), hi = max(q_max,0), scale = (hi-lo)/255 (1 if not > 0),
 *                    inv_scale = 1/scale, zero_point = clamp(-128 - rint(lo/scale), -128, 127).
 *   rounding, seed   how a layer call that WRITES this tensor rounds: HQ_ROUND_NEAREST_EVEN (0), or
 *                    HQ_ROUND_STOCHASTIC (1) -- the paper's choice for gradients: code =
 *                    sat8(floor(fl(u + r)) + zero_point) with u as for nearest-even and r = h / 65536,
 *                    h the 16-bit draw of Philox4x32-10 (Salmon et al., SC'11) with key (seed, 0) and
 *                    counter (e >> 3 as two words, step, 0) for the element with linear index e in the
 *                    output tensor: half number (e & 7) of the call's four words, low half first.
 *                    `step` is the value at the time of the call, so every iteration draws anew.
 *   dynamic_eta      read by hq_dynamic_quant only: 0 (default) = current min-max (Eq. 1); eta in (0,1) =
 *                    running min-max (Sec. 4.1): the range that quantizes the tensor is
 *                    (1-eta) * its own min/max + eta * the previous range (first tensor: its min/max).
 *   sat_below, sat_above   the saturation statistic of Sec. 4 ("the proportion of values that lie outside the
 *                    quantization grid"), as counts: a layer call that writes this tensor with HQ_COUNT_SATURATION set in
 *                    `rounding` adds the number of outputs whose grid coordinate u = fl(fl(float(acc) * s_acc) * inv_scale)
 *                    lies below the lowest grid point (u < -128 - zero_point) or above the highest (u > 127 - zero_point),
 *                    taken before rounding, so the counts do not depend on the rounding mode.  Dividing by the tensor's
 *                    element count gives the ratio.
 *   last_sat_below, last_sat_above   hq_range_update / hq_dynamic_quant move the counts here and clear the running pair.
 * For a layer INPUT only scale and zero_point are read.                                      */
#define HQ_ROUND_NEAREST_EVEN 0u
#define HQ_ROUND_STOCHASTIC 1u
#define HQ_ROUND_MODE_MASK 0xFFu     /* low byte of `rounding`: the rounding mode */
#define HQ_COUNT_SATURATION 0x100u   /* flag in `rounding`: count the outputs that lie outside the grid */
typedef struct {
  int32_t acc_min, acc_max;
  float acc_scale;
  uint32_t step;
  float q_min, q_max;
  float scale, inv_scale;
  int32_t zero_point;
  uint32_t rounding;
  uint32_t seed;
  float dynamic_eta;
  uint32_t sat_below, sat_above;
  uint32_t last_sat_below, last_sat_above;
} hq_range_state;

/* Forward-convolution geometry.  Input N x H x W x C, output N x Ho x Wo x K with
 * Ho = (H + 2*pad_h - R)/stride_h + 1 (Wo alike).  groups is 1, or C (== K) for depthwise. */
typedef struct {
  int32_t N, H, W, C;
  int32_t K;
  int32_t R, S;
  int32_t stride_h, stride_w;
  int32_t pad_h, pad_w;
  int32_t groups;
} hq_conv_desc;

typedef enum { HQ_DIR_FWD = 0, HQ_DIR_BWD_DATA = 1 } hq_direction;
typedef enum { HQ_OP_LINEAR = 0, HQ_OP_CONV_FWD = 1, HQ_OP_CONV_BWD_DATA = 2 } hq_op_kind;

typedef struct hq_ctx hq_ctx;                           /* HOST handle */
typedef struct hq_prepared_weights hq_prepared_weights; /* HOST handle to device-side tables */

/* Operation descriptor for hq_dynamic_quant and hq_debug_accumulate: the operands of the layer
 * call it mirrors.  kind = HQ_OP_LINEAR uses M, N, K, w, bias; the conv kinds use conv, pw. */
typedef struct {
  int32_t kind;                  /* hq_op_kind */
  int32_t M, N, K;               /* linear only */
  const hq_conv_desc* conv;      /* HOST; conv kinds only */
  const int8_t* x;               /* input (linear X, conv X, or dY for backward data) */
  const hq_range_state* xq;      /* its scale / zero_point */
  const int8_t* w;               /* linear only: W[N][K] */
  const int32_t* bias;           /* linear only, may be NULL */
  const hq_prepared_weights* pw; /* conv kinds; linear: NULL, or a handle from hq_linear_prepare (N, K, w then ignored) */
  const float* w_scale;          /* one float: the weights' scale s_w (zero point 0) */
} hq_op_desc;

/* ---- context ------------------------------------------------------------------------------ */

/* Creates a context on CUDA device `device` (HOST out-pointer).  Allocates a small device
 * status word and scratch for weight column sums.  HQ_ERR_CUDA if the device cannot be used,
 * HQ_ERR_UNSUPPORTED if it is not compute capability 10.0. */
hq_status hq_create(hq_ctx** ctx, int device);
hq_status hq_destroy(hq_ctx* ctx);
const char* hq_status_string(hq_status s);       /* HOST string, static storage */
const char* hq_last_error(const hq_ctx* ctx);    /* HOST string of the last rejected call */
/* Synchronises `stream`, copies the device status word to *code (HOST) and clears it.
 * Returns HQ_ERR_TIMEOUT if a bounded wait expired since the last call, else HQ_OK. */
hq_status hq_get_async_error(hq_ctx* ctx, void* stream, int32_t* code);
/* Number of kernel launches this context has enqueued so far (HOST counter). */
uint64_t hq_launch_count(const hq_ctx* ctx);
/* Of those, the layer-kernel launches that ran as pairs of CTAs on 256-row tiles (option "pair"). */
uint64_t hq_pair_launch_count(const hq_ctx* ctx);
/* Tuning knob (HOST key string), for tests and experiments; results are identical for every value.
 *   "staging": how convolutions prepared AFTER this call bring their input to the MAC array (the
 *              paper's "loaded into the MAC array", Sec. 3.1): -1 = chosen per layer (default),
 *              0 = one copy per filter tap, 1 = input rows kept resident wherever the layer allows.
 *   "depthwise": how depthwise layers prepared AFTER this call run: -1 = library's choice (default; the
 *              CUDA-core kernel), 0 = CUDA-core kernel, 1 = on the tensor cores as dense layers with
 *              diagonal filters, one per 64-channel slice.
 *   "side_by_side": 1 (default) = the independent launches of one call (parity classes of a strided
 *              backward pass) run concurrently on shares of the SMs, forked from and joined into the
 *              caller's stream; 0 = one after the other.
 *   "depthwise_staging": CUDA-core depthwise 3x3 stride-1 layers (read at every call): -1 = library's
 *              choice (default), 0 = direct global loads, 1 = input patches staged in shared memory by TMA
 *              where the shape allows, one multiply-accumulate per 4-way dot-product instruction, 2 = the same
 *              staging with the patch transposed in registers so that one such instruction covers a filter row.
 *   "repack":  how spatial filters over a channel count that is not a multiple of 16 (the RGB stem),
 *              prepared AFTER this call, are brought to the tensor cores: -1 = chosen per layer
 *              (default), 0 = whole filter patches per output pixel gathered into a library-owned matrix,
 *              1 = horizontal filter windows per input row gathered into a library-owned tensor where the
 *              shape allows, 2 = the fused kernel that gathers the filter windows in shared memory (nothing
 *              repacked in global memory) where the shape allows, else as -1.
 *   "gather_span": the fused few-channel kernel of layers prepared AFTER this call, for output rows shorter than a
 *              128-pixel tile: 1 (default) = a tile is 128 consecutive pixels of one image in row-major order, across
 *              row ends (no unused tile rows), 0 = one output row per tile.
 *   "epilogue_groups": layers prepared AFTER this call: -1 = chosen per layer (default); g = 0, 1, 2: the sixteen
 *              epilogue warps form 2^g groups that drain alternate tiles (at most one group per accumulator buffer).
 *   "col_tiles": into how many column tiles (each a multiple of 16 columns, at most 256) the output channels of
 *              layers prepared AFTER this call are split: -1 = chosen per layer by estimated duration (default),
 *              0 = as few as possible, n > 0 = at least n.
 *   "pair":    layers prepared AFTER this call whose weights stream through shared memory: -1 = chosen per layer
 *              (default), 0 = every CTA works on its own 128-row tile, 1 = pairs of CTAs on neighbouring SMs share
 *              256-row tiles (one tensor-core instruction for both, each CTA holding half of the weight rows)
 *              wherever the layer allows.
 *   "wgrad_windows": weight gradients of convolutions (read at every call; 1 also selects the general depthwise form
 *              instead of the transposing one for 3x3 stride-1 pad-1 depthwise layers): -1 = library's choice (default),
 *              0 = stride-1 layers pack both tensors channel-major over a padded pixel index (one copy of dY, one
 *              copy of X per horizontal filter offset) wherever the shape allows, 1 = always the general form
 *              (one transposed copy of X per filter tap).
 *   "issuers": upper limit (1, 2 or 3; default 3) of the warps of a CTA that issue tensor-core instructions,
 *              each for every n-th tile, in layers prepared AFTER this call.
 *   "a_producers": layers prepared AFTER this call that take one copy of the input per filter tap and keep their weights
 *              in shared memory (1x1 layers): -1 = chosen per layer (default), 1 = one warp copies the input tiles,
 *              2 = two warps copy them for alternate tiles (with at most two issuing warps) wherever the layer allows.
 *   "overlap_launches": 1 (default) = the layer and range-update kernels are launched so that their
 *              set-up may run while the previous kernel in the stream drains; each waits for that
 *              kernel to finish before it reads memory, so stream order is unchanged.  0 = ordinary
 *              launches. */
hq_status hq_set_option(hq_ctx* ctx, const char* key, int32_t value);

/* ---- weights ------------------------------------------------------------------------------ */

/* Once per weight update (Sec. 3.1: the weights are quantized before they are loaded into the
 * MAC array; their range can be pre-computed, Sec. 3.1 last paragraph).  Copies W (int8,
 * [K][R][S][C], depthwise [C][R][S]) into library-owned device memory in the operand order the
 * direction needs (backward data: the transposed, spatially reversed filter, split by output
 * parity for strided layers) and builds the integer tables that remove the input zero point
 * at padded borders.  W may be released after the call's work on `stream` completes.
 * The handle is valid for this geometry (including N, H, W) only. */
hq_status hq_weights_prepare(hq_ctx* ctx, void* stream, const hq_conv_desc* desc, hq_direction dir,
                             const int8_t* W, hq_prepared_weights** out);
/* The same for asymmetric weights (Sec. 5.2: the weights are quantized with the current min-max method; with an
 * asymmetric grid they carry a zero point): W holds codes whose real value is s_w * (code - w_zero_point), and every layer
 * call with the handle forms sum (x - z_x) * (w - z_w).  How: sum (x - z_x)(w - z_w) = [sum (x - z_x) w] - z_w * sum (x - z_x);
 * the bracket is what the layer kernels compute for symmetric weights, the second term is one number per output pixel
 * (the sum of the pixel's in-image input window), written by a small kernel at the head of every layer call into scratch
 * the handle owns, and subtracted in the epilogue before statistics and requantization.  w_zero_point in -128..127;
 * 0 gives exactly hq_weights_prepare.  Depthwise layers with a zero point run a direct CUDA-core kernel. */
hq_status hq_weights_prepare_zp(hq_ctx* ctx, void* stream, const hq_conv_desc* desc, hq_direction dir,
                                const int8_t* W, int32_t w_zero_point, hq_prepared_weights** out);
/* Prepared weights of a LINEAR layer, once per weight update: copies W[N][K] (zero-padding K to a multiple of 16) and caches
 * the column sums that remove the input zero point, so that hq_linear_fwd_prepared launches the layer kernel alone and
 * never touches context scratch.  w_zero_point as for hq_weights_prepare_zp.  max_M: the largest row count the handle
 * will be used with; needed (> 0) when K is not a multiple of 16 (room for the padded copy of X) or w_zero_point != 0
 * (room for the per-row term), ignored otherwise.  Release with hq_weights_release. */
hq_status hq_linear_prepare(hq_ctx* ctx, void* stream, int32_t N, int32_t K, const int8_t* W, int32_t w_zero_point,
                            int32_t max_M, hq_prepared_weights** out);
hq_status hq_weights_release(hq_ctx* ctx, hq_prepared_weights* pw);

/* ---- the hot path --------------------------------------------------------------------------- */

/* Y[M][N] = Q_Y( sum_k (X[m][k] - z_x) * W[n][k] + bias[n] ), Sec. 3.1 + Sec. 4 step 1, with
 * z_x = xq->zero_point, s_acc = xq->scale * *w_scale, and (inv_scale, zero_point) taken from *yq
 * as left by the previous hq_range_update / hq_dynamic_quant.  Per element:
 *   y = float(acc) * s_acc;  q = clamp(rint(y * inv_scale) + zero_point, -128, 127)
 * (round half to even, one binary32 rounding per operation).  Merges min/max of acc into
 * yq->acc_min/acc_max (Sec. 4 step 2) and writes yq->acc_scale.  bias may be NULL.
 * K that is not a multiple of 16 is served through zero-padded copies of X and W in context-owned scratch
 * (grown with cudaMalloc when a larger layer is first seen).  Backward data of a linear layer is this call
 * with W transposed. */
hq_status hq_linear_fwd(hq_ctx* ctx, void* stream, int32_t M, int32_t N, int32_t K,
                        const int8_t* X, const hq_range_state* xq,
                        const int8_t* W, const float* w_scale, const int32_t* bias,
                        int8_t* Y, hq_range_state* yq);

/* hq_linear_fwd with weights from hq_linear_prepare: same arithmetic (with the handle's weight zero point), no per-call
 * column sums, no context scratch, nothing allocated.  Two calls with different handles may overlap on the GPU; two calls
 * with the SAME handle may not when the handle owns scratch (K not a multiple of 16, or a weight zero point). */
hq_status hq_linear_fwd_prepared(hq_ctx* ctx, void* stream, int32_t M, const int8_t* X, const hq_range_state* xq,
                                 const hq_prepared_weights* pw, const float* w_scale, const int32_t* bias,
                                 int8_t* Y, hq_range_state* yq);

/* Forward convolution as an implicit GEMM (Sec. 3.1), same epilogue as hq_linear_fwd.
 * Padding is zero in the real domain.  pw must come from hq_weights_prepare(.., HQ_DIR_FWD, ..)
 * with the same descriptor.  groups == C selects the depthwise kernel.  Spatial filters over a channel
 * count that is not a multiple of 16 (an RGB stem) run a fused kernel that gathers the filter windows in shared
 * memory when W * C is a multiple of 16, K a multiple of 16 of at most 256 and the filter is one of the built sizes
 * (7x7x3, 5x5x3, 5x5x4, 3x3x3, 3x3x4, 3x3x5); other such shapes run a gather pre-pass into a library-owned tensor
 * that the handle allocates at preparation time. */
hq_status hq_conv_fwd(hq_ctx* ctx, void* stream, const hq_conv_desc* desc,
                      const int8_t* X, const hq_range_state* xq,
                      const hq_prepared_weights* pw, const float* w_scale,
                      int8_t* Y, hq_range_state* yq);

/* Input gradient of the convolution described by desc (Sec. 3.1, backward pass: G_X from the
 * quantized output gradient and the weights, always quantized by Q_G):
 *   dX[n][hi][wi][c] = Q_G( sum over (r,s,k) with ho*stride_h - pad_h + r == hi (wo alike)
 *                           of (dY[n][ho][wo][k] - z_dy) * W[k][r][s][c] ).
 * dY is N x Ho x Wo x K, dX is N x H x W x C.  pw from hq_weights_prepare(.., HQ_DIR_BWD_DATA, ..).
 * Depthwise layers (groups == C): the sum runs over (r,s) alone with k == c; stride-1 layers run the forward depthwise
 * kernels over the output gradient with the filter turned by 180 degrees, strided layers a direct kernel. */
hq_status hq_conv_bwd_data(hq_ctx* ctx, void* stream, const hq_conv_desc* desc,
                           const int8_t* dY, const hq_range_state* dyq,
                           const hq_prepared_weights* pw, const float* w_scale,
                           int8_t* dX, hq_range_state* dxq);

/* Weight gradient of a linear layer (Sec. 3.1, backward pass: the quantized output gradient and the quantized layer
 * input give G_W, which the paper keeps in FP32):
 *   GW[n][k] = fl( float( sum_m (dY[m][n] - z_dy) * (X[m][k] - z_x) ) * fl(s_dy * s_x) ),  one binary32 rounding per step,
 * with (s_dy, z_dy) = scale / zero_point of *dyq and (s_x, z_x) of *xq.  dY is [M][N], X is [M][K], GW is [N][K] binary32,
 * laid out like the weights.  The sum is formed modulo 2^32, so it is exact whenever the true sum fits in int32 (partial
 * sums may leave that range); M may not exceed 2^24.  The reduction runs over the rows, so the
 * call first transposes both operands into context-owned scratch (grown with cudaMalloc when a larger layer is first
 * seen; calls on one context must not overlap) and runs the tensor-core layer kernel on them with a binary32
 * epilogue.  Nothing is quantized and no range state is written. */
hq_status hq_linear_wgrad(hq_ctx* ctx, void* stream, int32_t M, int32_t N, int32_t K,
                          const int8_t* dY, const hq_range_state* dyq,
                          const int8_t* X, const hq_range_state* xq, float* GW);

/* Weight gradient of a dense convolution (Sec. 3.1, backward pass; kept in FP32 like the paper's):
 *   GW[k][r][s][c] = fl( float( sum over n,ho,wo of (dY[n][ho][wo][k] - z_dy) * (X[n][hi][wi][c] - z_x) ) * fl(s_dy * s_x) ),
 * hi = ho*stride_h - pad_h + r (wi alike), output pixels whose (hi,wi) lies outside the image contributing nothing (padding
 * is zero in the real domain).  dY is N x Ho x Wo x K, X is N x H x W x C, GW has the layout of the weights, binary32.
 * The sum is formed modulo 2^32: exact whenever the true sum fits in int32.  At most 2^24 output pixels.  Depthwise layers
 * (groups == C == K; 3x3 or 5x5 filters, C a multiple of 4, at most 1024): GW is [C][R][S], the sum runs with k == c, on
 * CUDA-core kernels (3x3, stride 1, padding 1, C a multiple of 16 of at most 256: four pixels per 4-way dot product on
 * words transposed in registers, the zero points taken out from per-channel totals and border sums; else one product at
 * a time with integer atomics).
 * How dense layers run: both tensors are written pixels-innermost into context-owned scratch (grown with cudaMalloc when a
 * larger layer is first seen; calls on one context must not overlap) -- stride-1 layers: dY once and X once per horizontal
 * filter offset over a padded pixel index in which a vertical filter offset is a shift of the reduction coordinate
 * (scratch about (S + 1) times the size of X); any other layer: one transposed copy of X per filter tap (R*S times X).
 * The reduction over the pixels is cut into slices that the tensor-core layer kernel multiplies side by side, and a last
 * pass sums the slices, removes both zero points and converts.  No range state is written.  (Option "wgrad_windows".) */
hq_status hq_conv_wgrad(hq_ctx* ctx, void* stream, const hq_conv_desc* desc,
                        const int8_t* dY, const hq_range_state* dyq,
                        const int8_t* X, const hq_range_state* xq, float* GW);

/* Eq. 2-3 for `count` consecutive states, to be enqueued after the layer calls of the iteration:
 *   m_lo = float(acc_min) * acc_scale, m_hi alike;
 *   step == 0:  q_min = m_lo, q_max = m_hi                      (initialisation, Sec. 4.1)
 *   else:       q_min = (1-eta)*m_lo + eta*q_min, q_max alike    (Eq. 2-3)
 * then derives scale / inv_scale / zero_point, increments step, empties the statistics slot and moves the saturation
 * counts to last_sat_below / last_sat_above.  A state whose slot is empty is left untouched. */
hq_status hq_range_update(hq_ctx* ctx, void* stream, hq_range_state* states, int32_t count, float eta);

/* Batch-sharded data parallelism (each GPU runs the layer calls on its slice of the batch with the same weights and
 * the same range states): Sec. 4.1 takes min/max over the WHOLE tensor, so the statistics slots are merged over the
 * ranks before hq_range_update.  hq_stats_pack writes acc_min of the `count` states to buf[0 .. count) and the bitwise
 * complement of acc_max to buf[count .. 2*count) (DEVICE, int32); one element-wise MIN all-reduce of buf over the ranks
 * (NCCL, on the same stream) then merges both columns, the complement turning max into min without overflow and an
 * empty slot being the identity; hq_stats_unpack writes the merged pair back.  Every rank then applies Eq. 2-3 to the
 * same numbers, so the replicated states stay bit-identical.  Both calls only enqueue one small kernel. */
hq_status hq_stats_pack(hq_ctx* ctx, void* stream, const hq_range_state* states, int32_t count, int32_t* buf);
hq_status hq_stats_unpack(hq_ctx* ctx, void* stream, hq_range_state* states, int32_t count, const int32_t* buf);

/* Dynamic quantization of the same layer (Sec. 3.2, Eq. 1; traffic of Eq. 5): kernel 1 runs the
 * layer's MAC loop and writes y = float(acc) * s_acc as binary32 to `workspace` (caller-owned,
 * one float per output element) while reducing min/max; kernel 2 sets q_min/q_max of *yq to the
 * CURRENT tensor's extremes, derives the grid, increments step and empties the slot; kernel 3
 * reads the workspace back and writes the int8 output.  Also serves as iteration 0 of the
 * in-hindsight scheme (q^0 = min/max of the first tensor, Sec. 4.1). */
hq_status hq_dynamic_quant(hq_ctx* ctx, void* stream, const hq_op_desc* op,
                           float* workspace, int8_t* Y, hq_range_state* yq);

/* Largest output, in elements, that hq_dynamic_quant_static accepts (16 MiB of binary32). */
#define HQ_STATIC_WORKSPACE_ELEMS (4 * 1024 * 1024)

/* hq_dynamic_quant for callers that cannot allocate.  (The paper has no counterpart: this is a
 * property of the boundary, not of the method.)  Who needs it: code that runs where cudaMalloc is
 * not allowed or not wanted -- inside an allocator or profiler callback, in a latency-critical loop
 * that must never enter the allocator (cudaMalloc and cudaFree synchronise the device), or in a
 * process whose device memory was handed out in full at start-up -- and that therefore cannot
 * provide the one-float-per-output workspace of hq_dynamic_quant.  Here the workspace is a fixed device array that is part of the library image:
 * every GPU that loads the library sets aside HQ_STATIC_WORKSPACE_ELEMS floats (16 MiB) for it until
 * the process exits.  The call itself allocates and frees nothing: no device memory, through CUDA or any other
 * library, and no host memory either (its launch planning uses fixed-size tables, and a rejected call writes its
 * reason into a fixed buffer of the context).
 *   - Same operands, results and status codes as hq_dynamic_quant; Y and *yq are still the caller's.
 *   - Outputs of more than HQ_STATIC_WORKSPACE_ELEMS elements are rejected with HQ_ERR_UNSUPPORTED
 *     before anything is launched.  So is a linear layer that needs more context scratch than the context
 *     holds at the time of the call: column sums for more than 4096 output columns (unless an earlier
 *     hq_linear_fwd / hq_dynamic_quant on this context already grew that scratch), or K that is not a multiple
 *     of 16 (padded operand copies, unless an earlier call already made room for this size).
 *   - The context's device must be the current device.  The first call on a device looks up the
 *     array's device address (a host-side query, no launch); make that first call before starting
 *     any stream capture.
 *   - All calls on a device share the one array, and it keeps the previous call's contents.  Nothing
 *     in it has to start at zero (the first kernel writes every element the last one reads), but two
 *     calls that overlap on the GPU -- different streams, or different contexts on the same device --
 *     race on it.  Serialise them. */
hq_status hq_dynamic_quant_static(hq_ctx* ctx, void* stream, const hq_op_desc* op, int8_t* Y, hq_range_state* yq);

/* Measurement hook (the paper has no counterpart): enqueues one kernel in which every SM -- pair = 0: one CTA per SM,
 * 128 x bn x 32 per instruction; pair = 1: one CTA pair per two SMs, 256 x bn x 32 -- issues `chunks` x 32 int8
 * tensor-core instructions (the MAC of Sec. 3.1 and nothing else) on operand tiles that stay in shared memory: no loads,
 * no epilogue.  *ops (HOST, may be NULL) receives the 2 x MAC count of the launch; the caller times the launch with
 * events.  This is the "int8 MMA peak as measured on this GPU" that the layer kernels' tensor roofline is quoted against.
 * bn: a multiple of 32, at most 256. */
hq_status hq_mma_peak_probe(hq_ctx* ctx, void* stream, int32_t pair, int32_t bn, int32_t chunks, uint64_t* ops);

/* Test hook: writes the zero-point-corrected int32 accumulator (+bias) of the layer to `acc`
 * (one int32 per output element) and merges its min/max into *yq.  The hot path never
 * materialises this tensor. */
hq_status hq_debug_accumulate(hq_ctx* ctx, void* stream, const hq_op_desc* op, int32_t* acc, hq_range_state* yq);

#ifdef __cplusplus
}
#endif
#endif /* HQ_H_ */
