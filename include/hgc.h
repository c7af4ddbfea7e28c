/*
 * hgc.h - C ABI of the B200 (sm_100a) FP16 convolution-forward library.
 *
 * The library implements the hot path of a forward-only FP16 inference engine in the
 * style of HG-Caffe: the convolution layer forward with the semantics the paper inherits
 * from BVLC Caffe (Section 2.2), FP16 tensors end to end with no float<->half conversion
 * inside the engine (Section 3.3), scalars kept in host types and handed over at the call
 * boundary (Section 3.2), a wide accumulator because FP16 accumulation overflows and loses
 * small terms (Section 3.1), and no third-party compute library on the path (Section 2).
 *
 * General rules
 *   - Every function returns an hgc_status (int); 0 is HGC_OK.  Nothing throws, aborts or
 *     prints.  hgc_status_string() names a code.
 *   - "device pointer" = CUDA global memory of the current device; "host pointer" = ordinary
 *     (preferably pinned) host memory.  Each argument says which.
 *   - Tensors are dense IEEE binary16: x[N][C][H][W], w[K][C/group][R][S], bias[K],
 *     y[N][K][P][Q].  Device tensor pointers must be 16-byte aligned (HGC_BAD_ALIGNMENT) and
 *     must not overlap.  The library borrows them until the work queued on `stream` is done.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - hgc_conv_forward and the layout/repack calls only enqueue kernels on `stream`: they do
 *     not allocate, free or synchronise.  Scratch memory is provided by the caller through
 *     hgc_conv_set_workspace and stays caller-owned.
 *   - A descriptor is not thread-safe; distinct descriptors are independent.
 *   - All element offsets are computed in 64-bit integers.
 */
#ifndef HGC_H_
#define HGC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum hgc_status {
  HGC_OK = 0,
  HGC_INVALID_ARG = 1,    /* NULL where a pointer is required, or an impossible layer */
  HGC_UNSUPPORTED = 2,    /* a valid request this build has no kernel for */
  HGC_BAD_ALIGNMENT = 3,  /* a device tensor pointer is not 16-byte aligned */
  HGC_NO_WORKSPACE = 4,   /* the chosen path needs scratch memory and none (or too little) is set */
  HGC_CUDA_ERROR = 5,     /* a CUDA runtime/driver call or a kernel launch failed */
  HGC_DEVICE_TIMEOUT = 6  /* a bounded device-side wait expired; the output is not valid */
} hgc_status;

/* Which kernel the planner chose for a descriptor (hgc_conv_path). */
typedef enum hgc_path {
  HGC_PATH_DIRECT = 0,     /* direct convolution on CUDA cores, any valid layer */
  HGC_PATH_DEPTHWISE = 1,  /* 3x3 depthwise (group == C == K) stencil on CUDA cores */
  HGC_PATH_IGEMM = 2       /* implicit GEMM on tcgen05 tensor cores with TMEM accumulators */
} hgc_path;

/* Layer description.  Scalars are plain host integers (Section 3.2: scalars stay in host
   types; only tensors are half). */
typedef struct hgc_conv_params {
  int32_t n, c, h, w;        /* input  x[N][C][H][W]                      */
  int32_t k, r, s;           /* weights w[K][C/group][R][S]               */
  int32_t pad_h, pad_w;      /* zero padding, same amount on both sides   */
  int32_t stride_h, stride_w;
  int32_t dil_h, dil_w;      /* dilation: tap r reads row p*stride - pad + r*dil */
  int32_t group;             /* C % group == 0 and K % group == 0         */
  int32_t flags;             /* HGC_FLAG_* bits; 0 = planner's choice     */
} hgc_conv_params;

#define HGC_FLAG_FORCE_DIRECT 1  /* always use HGC_PATH_DIRECT (testing / comparison) */
/*
 * Layout flags for stacks of layers that keep their activations channels-last between layers
 * (the paper's rule "convert only at the input and the output", Section 3.3, applied to the
 * layout): with HGC_FLAG_X_NHWC the input is x[N][H][W][C] and the layout pass is skipped; with
 * HGC_FLAG_Y_NHWC the output is written as y[N][P][Q][K].  Both are taken by the tensor-core path
 * (HGC_FLAG_X_NHWC also needs C, and C/group for grouped layers, to be multiples of 8) and, when
 * given together, by 3x3 depthwise layers of C % 8 == 0 channels (stride 1 or 2, dilation 1);
 * hgc_conv_desc_create returns HGC_UNSUPPORTED otherwise.  Weights and bias are as always.
 * Channels-last output is staged in shared memory and written by TMA when K/group is a multiple
 * of 32 (as fast as the NCHW epilogue); other channel counts are written with plain 2-byte stores.
 */
#define HGC_FLAG_X_NHWC 2
#define HGC_FLAG_Y_NHWC 4
/*
 * Scheduling choices of the tensor-core path (the result is the same layer within the tolerance;
 * the summation order over the input channels changes).
 * HGC_FLAG_CTA_PAIRS (off unless set): layers with more than 128 output channels per group may be
 * launched as CTA pairs (clusters of two SMs that share tiles of 256 output channels through
 * tcgen05 cta_group::2: each CTA fetches its own 128 weight rows and half of the activation
 * tile).  Measured on the VGG-16 layers: within a few per cent of the single-CTA kernel either
 * way, so the planner does not choose it by itself.
 * HGC_FLAG_SHARED_TILES: the ring stages of all tiles are dealt out in equal contiguous ranges,
 * so that every CTA (or pair) gets the same amount of work; a tile that straddles a boundary is
 * reduced by several CTAs inside the one launch (fp32 hand-over through the workspace, added in
 * a fixed order: deterministic).  Such a launch is cooperative.  Without the flag the planner
 * takes this schedule only where its cost model expects a gain (long tiles, at least 2.5 per
 * CTA, a last wave that is mostly empty: VGG-16's 256-channel layers on 56x56 planes at batch
 * 16, 61 -> 56 us); with it, wherever the tiles do not fill whole waves.
 * HGC_FLAG_WHOLE_TILES: never (smaller workspace; ordinary launch).  Wins over the flag above.
 */
#define HGC_FLAG_CTA_PAIRS 8
#define HGC_FLAG_SHARED_TILES 16
#define HGC_FLAG_WHOLE_TILES 64
/*
 * HGC_FLAG_FUSED_LAYOUT (off by default): layers whose input needs the NCHW->NHWC copy and whose
 * output rows are whole 16-byte vectors (3x3 layers on 224, 112, 56 wide planes ...) make that
 * copy inside the tensor-core kernel: eight extra warps of every CTA convert x while the MMAs of
 * earlier tiles run, and a tile starts when the rows it reads are complete (a cooperative
 * launch).  Measured on the VGG-16 layers: no faster than the copy as a kernel of its own (the
 * step runs under the board's power cap, where work that overlaps costs what it costs alone).
 */
#define HGC_FLAG_FUSED_LAYOUT 32
/*
 * 1x1, stride-1, unpadded layers read x (NCHW) as it is when a channel's plane is a multiple of 8
 * pixels (the copy engine fetches pixel-major tiles); other planes take the NHWC copy of x first.
 * HGC_FLAG_GATHER_X (off by default): planes of a multiple of 4 pixels and at most 256 (14x14),
 * with C a multiple of 64, start on 8-byte boundaries only, which no tensor map can describe;
 * with this flag eight extra warps of the tensor-core kernel gather the pixel-major tile
 * themselves with 8-byte asynchronous copies (plan [10] = 4) and no copy of x is made.  Measured
 * (B200, against the layout pass plus the plain kernel): 64 x 1024 -> 256 on 14x14 19.1 us against
 * 20.3; 256 -> 1024 21.8 against 18.4; 32 x 512 -> 512 12.5 against 12.3: it pays only where x is
 * large and the output small, so it is not the planner's choice.
 */
#define HGC_FLAG_GATHER_X 128

typedef struct hgc_conv_desc hgc_conv_desc; /* opaque; owned by the caller via create/destroy */

/*
 * Shape inference and planning (host only, no device work).  Implements the Caffe
 * convolution output size (the layer semantics of Section 2.2):
 *     P = floor((H + 2*pad_h - dil_h*(R-1) - 1) / stride_h) + 1,   Q likewise.
 * HGC_INVALID_ARG if out or p is NULL, any of n,c,h,w,k,r,s,group,stride,dil < 1, pad < 0,
 * C % group != 0, K % group != 0, or P < 1 or Q < 1.  On failure *out is left NULL.
 */
int hgc_conv_desc_create(hgc_conv_desc** out, const hgc_conv_params* p);

/* Frees the descriptor (host memory only).  NULL is accepted.  The caller must make sure
   that no queued work still uses it. */
int hgc_conv_desc_destroy(hgc_conv_desc* d);

/*
 * The layer forward (Sections 2.2, 3.1, 3.3):
 *   y[n,k,p,q] = fp16_rn( act( bias[k] + sum_{c',r,s} X(n, grp(k)*C/g + c',
 *                   p*stride_h - pad_h + r*dil_h, q*stride_w - pad_w + s*dil_w) * w[k,c',r,s] ) )
 * with X zero outside the image, grp(k) = k / (K/group), fp32 accumulation, bias added in
 * fp32 before the activation, act = max(.,0) if relu != 0 else identity, and one
 * round-to-nearest-even conversion to binary16 at the end.
 * x, w, y: device pointers (required).  bias: device pointer or NULL (no bias).
 * Enqueues on `stream` and returns; results are ready when the stream reaches that point.
 * Errors: HGC_INVALID_ARG (NULL d/x/w/y), HGC_BAD_ALIGNMENT, HGC_NO_WORKSPACE,
 * HGC_CUDA_ERROR.  A device-side timeout is reported by hgc_conv_last_device_status.
 */
int hgc_conv_forward(hgc_conv_desc* d, const void* x, const void* w, const void* bias,
                     void* y, int relu, void* stream);

/*
 * Same layer with HOST tensors: copies x, w, bias host->device into the workspace, runs
 * hgc_conv_forward, copies y device->host, all queued on `stream` (asynchronous if the host
 * memory is pinned; the caller synchronises the stream before reading y).  Needs a workspace
 * of at least hgc_conv_host_workspace_bytes.  x, w, bias, y: host pointers.
 */
int hgc_conv_forward_host(hgc_conv_desc* d, const void* x, const void* w, const void* bias,
                          void* y, int relu, void* stream);

/*
 * The same layer for callers that cannot allocate device memory.  (The paper has no counterpart
 * to this entry point; it exists for deployment.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside a host process whose
 * memory pool is owned and fully reserved by another framework, in a plug-in that is forbidden
 * to grow the process's device footprint after start-up, or between the begin and end of a
 * region that must not call the allocator.  Such a caller has tensors to read and write but no
 * way to obtain the scratch buffer that hgc_conv_set_workspace wants.
 *
 * What it does: runs the tensor-core path (HGC_PATH_IGEMM) of hgc_conv_forward with its scratch
 * (status word, re-laid-out weights, NHWC copy of x, fp32 partial sums of a split reduction) in a
 * 32 MiB array that is part of the library image: every device that loads the library holds
 * those 32 MiB until the process exits.  It takes the layer description directly; no descriptor
 * object, no workspace, no weight registration (the weights are re-laid-out on every call).
 * p->flags must be 0 or scheduling flags only (those are ignored): NCHW tensors.  x, w, y: device
 * pointers (required), bias: device pointer or NULL, all 16-byte aligned; everything is queued on
 * `stream`.
 *
 * It calls no cudaMalloc, cudaFree or other allocating routine.  The first call on each device
 * looks up the array's device address (cudaGetSymbolAddress, with that device current); make
 * that first call outside any stream capture.  With the CUDA runtime's default lazy module
 * loading the array itself is only backed by device memory when that first call loads the
 * module, so a caller that may not grow the device footprint later makes one warm-up call per
 * device at start-up (any small layer), or runs with CUDA_MODULE_LOADING=EAGER; on a device with
 * less than 32 MiB free that first call fails with HGC_CUDA_ERROR.  The looked-up address is
 * kept per device ordinal for the life of the process: after cudaDeviceReset it is stale, and
 * this entry point must not be used again in that process.
 *
 * Limits and errors: HGC_UNSUPPORTED if the layer is not one the tensor-core path takes (fewer
 * than 9 channels per group unless it is an image stem, very wide rows ...: use hgc_conv_forward)
 * or if p->flags asks for channels-last tensors or the direct path; HGC_NO_WORKSPACE if the layer
 * needs more than the 32 MiB (1 KiB + K*R*S*c_w*2 + N*H*W*c_pad*2 bytes, channels rounded up,
 * + slices*N*K*P*Q*4 for the few layers whose reduction is split into 2, 4 or 8 slices: inner
 * products, tiny planes); HGC_INVALID_ARG / HGC_BAD_ALIGNMENT as for hgc_conv_forward;
 * HGC_CUDA_ERROR.  A device-side timeout cannot be read back through this entry point.
 *
 * All calls on a device share the one array, and it keeps the previous call's contents (the
 * call clears the part that must start at zero).  Two calls whose GPU work overlaps - different
 * streams, or different host threads - race on it: serialise them on one stream.
 */
int hgc_conv_forward_static(const hgc_conv_params* p, const void* x, const void* w, const void* bias,
                            void* y, int relu, void* stream);

/* Output shape N, K, P, Q of the descriptor (any output pointer may be NULL). */
int hgc_conv_output_dims(const hgc_conv_desc* d, int32_t* n, int32_t* k, int32_t* p, int32_t* q);

/* The kernel path the planner chose (an hgc_path value). */
int hgc_conv_path(const hgc_conv_desc* d, int32_t* path);

/*
 * Tiling the planner chose, for inspection and tests.  Writes up to `count` int32 values:
 * [0] path, then for HGC_PATH_IGEMM: [1] channels per reduction block, [2] 1 if the taps of a
 * kernel row share one activation tile (stride 1), [3] images per pixel tile, [4] rows per pixel
 * tile, [5] accumulator columns per output row, [6] MMA N, [7] number of tiles, [8] depth of the
 * shared-memory ring, [9] weight tiles (taps) per ring stage, [10] where the kernel's activation
 * tiles come from: 0 = an NHWC copy of x made by the layout pass, 1 = x itself (1x1 layers read
 * as pixel-major tiles; channels-last x, which includes every input with a 1x1 plane), 2 = a
 * zero-bordered 8-channel NHWC copy read through
 * overlapping windows (few input channels), 3 = an expanded copy holding, per output pixel, the
 * values under the kernel (few input channels, strided), 4 = x itself, gathered by extra warps of
 * the kernel (1x1 layers on small planes, see HGC_FLAG_GATHER_X), [11] the number of CTAs that share
 * the reduction of one tile (1, or 2 / 4 / 8 for layers with very few tiles, e.g. inner products:
 * each CTA writes fp32 partial sums and a second kernel adds them in a fixed order), [12] the
 * number of CTAs of the launch when the ring stages of all tiles are dealt out as contiguous
 * ranges (0 with reduction slices), [13] 1 if those ranges are equal, so that a tile straddling a
 * boundary is reduced by several CTAs inside the one launch (the CTA holding the tile's first
 * stage adds the others' fp32 accumulators in a fixed order), 0 if every CTA takes whole tiles,
 * [14] 1 if the launch consists of CTA pairs (clusters of two that share tiles of 256 output
 * channels; [3], [4] then describe one CTA's pixel sub-tile, [6] the MMA N of the pair, [7] the
 * number of pair tiles, [12] the number of pairs), [15] 1 if the NCHW->NHWC copy of x ([10] = 0)
 * is made by extra warps of the tensor-core kernel itself instead of a kernel of its own, [16] 1
 * if a layer of 64 output channels runs as row pairs: accumulator lanes 64..127 of the 128-row MMA
 * hold the odd output rows ([4] then counts row pairs per tile, [7] tiles of two output rows, [9]
 * and the kernel's taps are those of a kernel with one more row), [17] the number of copies of the
 * layer's weight rows in a weight tile (2 for epilogue-bound layers of 64 output channels: lane
 * quarters 2 and 3 then hold the same channels as 0 and 1 and take other pixels; else 1), [18] how
 * the epilogue writes y: 1 = staged tiles sent by the copy engine (tensor map over y), 2 = tiles of
 * whole planes of a 1x1 layer, one bulk copy per block of 32 channels (contiguous in y), 0 = plain
 * stores from a staging tile; zeros for the other paths.  info: host pointer; at most 19 values
 * are written.
 */
int hgc_conv_plan_info(const hgc_conv_desc* d, int32_t* info, int32_t count);

/* Scratch bytes hgc_conv_forward needs for this descriptor (0 if none). */
int hgc_conv_workspace_bytes(const hgc_conv_desc* d, size_t* bytes);

/* Scratch bytes hgc_conv_forward_host needs: the above plus device staging for x, w, bias, y. */
int hgc_conv_host_workspace_bytes(const hgc_conv_desc* d, size_t* bytes);

/* Hands the descriptor a caller-owned device buffer (256-byte aligned) used as scratch by
   later forwards.  It must stay valid until those forwards have completed.  Passing
   (NULL, 0) detaches it.  Setting a workspace forgets registered weights. */
int hgc_conv_set_workspace(hgc_conv_desc* d, void* dev_ptr, size_t bytes);

/*
 * Optional: registers a weight tensor (device pointer) and runs the one-off weight
 * re-layout for it on `stream` (Section 3.3: weights are prepared once when loaded, not
 * converted on every use).  Later hgc_conv_forward calls given the same `w` pointer skip
 * that step; a different pointer is re-laid-out on the fly each call.  Needs the workspace
 * to be set if hgc_conv_workspace_bytes is non-zero.  No effect on paths that read w as is.
 */
int hgc_conv_set_weights(hgc_conv_desc* d, const void* w, void* stream);

/* Reads the device status word of the descriptor's last forward (synchronises `stream`
   work that was queued by this descriptor).  *status is HGC_OK or HGC_DEVICE_TIMEOUT.
   Reading a raised word clears it.  Until then every forward of the tensor-core path on this
   descriptor returns at once without touching y (its CTAs find the word raised): after a
   timeout, read the status before using the descriptor again.
   Channels-last depthwise layers share one status word per process (set by any of them,
   cleared when read). */
int hgc_conv_last_device_status(hgc_conv_desc* d, int32_t* status);

/*
 * Layout transforms (the engine keeps tensors in FP16 and only re-arranges them; no value is
 * changed, Section 3.3).  src, dst: device pointers, 16-byte aligned, non-overlapping.
 *   nchw_to_nhwc: dst[n][h][w][c_pad] = src[n][c][h][w] for c < C, 0 for C <= c < c_pad
 *   nhwc_to_nchw: dst[n][c][h][w]     = src[n][h][w][c] for c < C  (padding dropped)
 * c_pad >= c and c_pad % 8 == 0 (one pixel is a whole number of 16-byte vectors).
 */
int hgc_layout_nchw_to_nhwc(const void* src, void* dst, int32_t n, int32_t c, int32_t h,
                            int32_t w, int32_t c_pad, void* stream);
int hgc_layout_nhwc_to_nchw(const void* src, void* dst, int32_t n, int32_t c, int32_t h,
                            int32_t w, int32_t c_pad, void* stream);

/*
 * Weight re-layout for the implicit-GEMM path:
 *   dst[g][K/group][R][S][c_pad] = src[g*(K/group)+k'][c'][r][s] for c' < C/group, else 0.
 * src, dst: device pointers, 16-byte aligned.  c_pad >= C/group, c_pad % 8 == 0.
 */
int hgc_weights_repack(const void* src, void* dst, int32_t k, int32_t c_per_group, int32_t r,
                       int32_t s, int32_t group, int32_t c_pad, void* stream);

/*
 * Inner-product (fully connected) layer, the other layer the paper names as overflowing in FP16
 * because of its long sums (Section 3.1):  y[n][k] = relu?( bias[k] + sum_c x[n][c] * w[k][c] ),
 * FP16 storage, FP32 accumulation, one rounding.  It is the convolution of this library on a 1x1
 * plane with a 1x1 kernel: this call creates exactly that descriptor (x: [n][c], w: [k][c],
 * y: [n][k], all dense FP16), to be used with hgc_conv_forward and the other descriptor calls.
 * n, c, k >= 1.  Errors as hgc_conv_desc_create.
 */
int hgc_inner_product_desc_create(hgc_conv_desc** out, int32_t n, int32_t c, int32_t k);

/*
 * FP32 -> FP16 cast, the arithmetic of a weight-file converter (Section 3.4: models are stored
 * in FP32 and converted once to an FP16 copy): dst[i] = the binary16 value nearest to src[i],
 * ties to even; magnitudes >= 65520 become infinities, NaNs stay NaNs.
 * src: `count` floats, dst: `count` binary16 values, device pointers, 16-byte aligned, not
 * overlapping.  overflow_count: device pointer to a 64-bit counter or NULL; the kernel ADDS the
 * number of finite inputs that became infinite (zero it first; read it after the stream has
 * finished).  Queued on `stream`; nothing is allocated.  count == 0 is a no-op.
 * Errors: HGC_INVALID_ARG (NULL src/dst, count < 0), HGC_BAD_ALIGNMENT, HGC_CUDA_ERROR.
 */
int hgc_cast_f32_to_f16(const void* src, void* dst, int64_t count, uint64_t* overflow_count, void* stream);

/*
 * Batch norm forward (Section 3.1), x and y [n][c][hw] dense FP16 (hw = H*W):
 *     y = (x - mean_c) / sqrt(var_c + eps),   one rounding to FP16,
 * mean_c and var_c (the biased variance) taken per channel over its n*hw values.  The statistics
 * are computed the way the section describes: the values of a channel are partitioned into groups
 * (one image, at most 2048 consecutive pixels), the mean of each group is taken, then the mean
 * of the group means weighted by the group sizes; the centred values are multiplied by
 * 2^shift_log2 before they are squared (the section's 1/32 for large data is -5, its 32 for
 * small data is 5, 0 is no shift) and the variance is shifted back.  All sums are FP32, so the
 * result does not depend on shift_log2 (|shift_log2| <= 8).
 * use_stored == 0: mean and var (device, `c` floats each) are WRITTEN; `workspace` must hold
 * hgc_batchnorm_workspace_bytes(n, c, hw) bytes of device memory (16-byte aligned; contents
 * irrelevant before, undefined after).  use_stored != 0: mean and var are READ (stored
 * statistics, e.g. a trained model's), workspace may be NULL.  No scale/shift parameters: Caffe
 * keeps them in a separate layer (see hgc_bn_fold for inference).
 * x, y: device pointers, 16-byte aligned, not overlapping.  Queued on `stream` (three kernels, or
 * one with stored statistics); nothing is allocated, nothing synchronises.
 * Errors: HGC_INVALID_ARG (NULL pointers, n/c/hw < 1, eps < 0, shift out of range),
 * HGC_UNSUPPORTED (c > 65535 or more than 2^31-1 groups), HGC_BAD_ALIGNMENT, HGC_NO_WORKSPACE
 * (workspace NULL when statistics are to be computed), HGC_CUDA_ERROR.
 */
size_t hgc_batchnorm_workspace_bytes(int32_t n, int32_t c, int64_t hw);
int hgc_batchnorm_forward(const void* x, void* y, int32_t n, int32_t c, int64_t hw, float eps, int32_t shift_log2,
                          int32_t use_stored, float* mean, float* var, void* workspace, void* stream);

/*
 * Inference-time folding of a batch norm with stored statistics (and an optional per-channel
 * scale gamma and shift beta) into the convolution in front of it:
 *     a_k = gamma_k / sqrt(var_k + eps),  w_out[k][j] = w[k][j] * a_k,
 *     b_out[k] = (bias[k] - mean_k) * a_k + beta_k,
 * computed in FP32, rounded once to FP16.  conv(x, w_out) + b_out then equals
 * gamma * (conv(x, w) + bias - mean) / sqrt(var + eps) + beta up to the rounding of w_out and
 * b_out, so the normalisation costs nothing at run time (it rides in the conv epilogue's bias).
 * w, w_out: [k][per_k] FP16 (per_k = (C/group)*R*S); bias: [k] FP16 or NULL (zeros); mean, var:
 * [k] floats; gamma, beta: [k] floats or NULL (ones / zeros); b_out: [k] FP16.  Device pointers;
 * w_out may equal w.  Errors: HGC_INVALID_ARG (NULL required pointer, k or per_k < 1, eps < 0),
 * HGC_CUDA_ERROR.
 */
int hgc_bn_fold(const void* w, const void* bias, const float* mean, const float* var, const float* gamma,
                const float* beta, float eps, int32_t k, int64_t per_k, void* w_out, void* b_out, void* stream);

/*
 * A depthwise-separable block as one kernel (Section 3.3: nothing is converted or stored between
 * layers that the engine itself chains): the 3x3 depthwise layer (group = C, pad 1, stride 1 or
 * 2, + bias, optional ReLU, rounded once to binary16 as the layer's output would be) followed by
 * the 1x1 pointwise layer C -> K (+ bias, optional ReLU).  The depthwise result is never written
 * to memory: extra warps of the tensor-core kernel compute it tile by tile straight into the
 * shared-memory stages that the MMAs of the pointwise layer read.
 *   x: [N][H][W][C] channels-last (C a multiple of 8, at least 16); w_dw: [C][1][3][3];
 *   w_pw: [K][C][1][1]; y: [N][K][P][Q], or [N][P][Q][K] with HGC_FLAG_Y_NHWC in p->flags
 *   (P, Q: the depthwise layer's output plane; hgc_conv_output_dims reports N, K, P, Q).
 * The descriptor is used with hgc_conv_workspace_bytes / hgc_conv_set_workspace /
 * hgc_conv_last_device_status / hgc_conv_desc_destroy like a layer descriptor, and with
 * hgc_dwpw_set_weights (optional: prepares both weight tensors once) and hgc_dwpw_forward
 * (device pointers, 16-byte aligned, bias pointers may be NULL; queued on `stream`).
 * Errors: HGC_INVALID_ARG (NULL, sizes < 1, stride other than 1 or 2, other flags, a layer
 * descriptor passed to hgc_dwpw_* or a block descriptor to hgc_conv_forward), HGC_UNSUPPORTED
 * (C not a multiple of 8 or below 16), HGC_BAD_ALIGNMENT, HGC_NO_WORKSPACE, HGC_CUDA_ERROR.
 */
typedef struct hgc_dwpw_params {
  int32_t n, c, h, w;   /* input, channels-last */
  int32_t k;            /* output channels of the pointwise layer */
  int32_t stride;       /* of the depthwise layer: 1 or 2 */
  int32_t flags;        /* 0 or HGC_FLAG_Y_NHWC */
} hgc_dwpw_params;
int hgc_dwpw_desc_create(hgc_conv_desc** out, const hgc_dwpw_params* p);
int hgc_dwpw_set_weights(hgc_conv_desc* d, const void* w_dw, const void* w_pw, void* stream);
int hgc_dwpw_forward(hgc_conv_desc* d, const void* x, const void* w_dw, const void* bias_dw, const void* w_pw,
                     const void* bias_pw, void* y, int relu_dw, int relu_pw, void* stream);

/*
 * Test hooks for the failure-detection path (Section 3.2 of the paper keeps scalars and control on
 * the host; a device-side wait that cannot be interrupted from the host therefore has to end by
 * itself).  Every wait of the TMA-fed kernels (tensor-core path, channels-last depthwise) on a
 * barrier, a copy or another CTA is bounded by wall-clock time: 2 s by default.  When one runs
 * out, the CTA stops taking work, lets its outstanding copies land, frees its tensor memory and
 * raises the descriptor's status word (hgc_conv_last_device_status reports HGC_DEVICE_TIMEOUT);
 * CTAs and launches that find the word raised return at once, so every later forward on that
 * descriptor is skipped until the status has been read (which clears it).
 * hgc_debug_set_wait_limit_ns: the limit in nanoseconds for all later launches in this process
 * (0 restores the default); synchronous (it writes a device variable of the current device).
 * hgc_debug_drop_copies: index >= 0: in later launches the first CTA announces its index-th
 * copy (tensor-core path: ring stage; depthwise: tile) but never issues it, so the wait for it
 * runs out; -1 switches the hook off.  Nothing faults or traps: the kernel returns through the
 * path described above.  Errors: HGC_CUDA_ERROR.  Host-side state, not thread-safe.
 */
int hgc_debug_set_wait_limit_ns(uint64_t ns);
int hgc_debug_drop_copies(int32_t index);

/*
 * Checked build.  The library can be built with -DHGC_DEBUG (libhgc_debug.so beside libhgc.so,
 * `python -m paper_1901_00858_b200.build` builds both).  In that build every global-memory access
 * that a kernel addresses by hand (the layout, depthwise and direct kernels; the copy and
 * channels-last epilogues, bias loads, partial sums and hand-overs of the tensor-core kernel)
 * is tested against the byte ranges of the call in progress: x, w, bias, y and the workspace, as
 * the descriptor's shapes give them (the copy engine's accesses are clipped to their tensor maps
 * by the hardware).  An access outside is recorded and SKIPPED: nothing faults.
 * hgc_debug_checked_build: 1 in the checked build, else 0.
 * hgc_debug_violations: synchronises the device, then writes the number of accesses outside every
 * range since the last call (0 in the ordinary build) and, of the first one, the source line of
 * its test, its address and size (host pointers; all but count may be NULL); clears the record.
 * hgc_debug_shrink_ranges: test hook: the ranges registered by later calls end `bytes` early, so
 * that the last accesses of correct kernels count as violations (and are skipped) although the
 * memory is there; 0 switches it off.  Errors: HGC_INVALID_ARG, HGC_CUDA_ERROR.
 */
int hgc_debug_checked_build(void);
int hgc_debug_violations(int32_t* count, int32_t* line, uint64_t* addr, uint64_t* bytes);
int hgc_debug_shrink_ranges(int64_t bytes);

/*
 * Launch overlap.  The persistent tensor-core kernels are always launched with the programmatic
 * stream serialization attribute: such a kernel may be scheduled while the previous kernel of
 * the stream is still draining, and waits, before it touches global memory, until that kernel
 * has completed; so its set-up overlaps the tail of the kernel before it, and where one
 * tensor-core kernel follows another its CTAs start as the previous kernel's leave.  Results are
 * the same either way.  Measured on B200, steps replayed as CUDA graphs: ResNet-50 channels-last
 * 1.065 -> 1.018 ms, MobileNet channels-last 0.332 -> 0.321 ms, NCHW steps unchanged.
 * With enabled != 0 EVERY kernel of the library is launched that way (off by default): with
 * eager launches the gap between dependent kernels shrinks (a VGG-16 step 0.776 -> 0.757 ms,
 * ResNet-50 1.76 -> 1.69 ms), but a step replayed as a CUDA graph gets slower when layout passes
 * sit between the tensor-core kernels (NCHW VGG-16 layers: 0.605 -> 0.696 ms), which is why it
 * is off unless asked for (`python bench.py --launch-overlap` repeats the measurement).
 * Applies to all later launches of this process.
 * Always returns HGC_OK.
 */
int hgc_set_launch_overlap(int enabled);

/* Number of kernels this library has launched in this process so far. */
int hgc_kernel_launch_count(uint64_t* count);

/* Static, never-NULL description of a status code. */
const char* hgc_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* HGC_H_ */
