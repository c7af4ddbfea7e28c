// Internal declarations shared by the translation units of libhgc (host planner + kernels).
#pragma once
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "hgc.h"

namespace hgc {

// Geometry of one layer as the kernels see it (all plain integers, passed by value).
struct ConvGeom {
  int32_t n, c, h, w;
  int32_t k, r, s;
  int32_t pad_h, pad_w, stride_h, stride_w, dil_h, dil_w;
  int32_t group;
  int32_t p, q;    // output plane
  int32_t cg, kg;  // channels per group: C/group, K/group
  int32_t x_nhwc, y_nhwc;  // channels-last input / output (tensor-core path only)
  int32_t no_split;        // 1: never let several CTAs share the reduction of a tile (no scratch for it); 0: wherever possible; 2: where the cost model expects a gain
  int32_t no_pair;         // 1: never pair CTAs on 256-channel tiles
  int32_t no_fuse;         // 1: the layout pass stays a kernel of its own
  int32_t no_gather;       // 1: 1x1 layers on small planes keep the separate layout pass (never gathered by the kernel's own warps)
  int32_t dw_stride;       // > 0: the pointwise layer of a depthwise + pointwise block; the depthwise layer's stride
  int32_t rowpair;         // planner-internal: this is the re-stated form of a 64-channel layer (IgemmPlan::rowpair)
};

// First bytes of the tensor-core path's workspace: the device status word (int at byte 0) and,
// from byte 256 on, one hand-over flag per CTA for tiles whose reduction several CTAs share.
constexpr size_t kWsHeaderBytes = 1024;
constexpr size_t kWsFlagsOff = 256;
constexpr int kMaxGrid = 192;

void count_launch();  // bumps the process-wide kernel launch counter

// Test hooks (hgc_debug_*): the limit of the device-side waits, and the index of a copy that the
// first CTA of the next TMA-fed launches announces but never issues (-1: none).
int debug_drop_copies();
cudaError_t igemm_set_wait_limit_ns(uint64_t ns);
cudaError_t depthwise_nhwc_tma_set_wait_limit_ns(uint64_t ns);

// Programmatic dependent launch: a kernel launched with this helper may be scheduled while the
// kernel before it in the stream is still draining; every kernel of this library therefore
// executes grid_dependency_wait() before its first access to global memory (it returns when the
// preceding kernel has completed and its writes are visible; a no-op for a kernel launched
// without the attribute), so only launch latency and on-chip set-up overlap.  Off by default
// (hgc_set_launch_overlap): it helps eager launches by a few per cent and slows a step replayed
// as a CUDA graph down.
bool launch_overlap_enabled();
void set_launch_overlap(bool on);

template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel_attr(bool overlap, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                      cudaStream_t stream, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = overlap ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                 Args... args) {
  return launch_kernel_attr(launch_overlap_enabled(), kernel, grid, block, smem, stream, args...);
}
// The persistent tensor-core kernel is always launched with the attribute: its set-up (barriers,
// tensor memory) then overlaps the tail of the kernel before it, and where one tensor-core kernel
// follows another (channels-last chains, 1x1 layers that read x in place) its CTAs start as the
// previous kernel's CTAs leave.  Measured, steps replayed as CUDA graphs: ResNet-50 channels-last
// 1.065 -> 1.018 ms, MobileNet channels-last 0.332 -> 0.321 ms, NCHW steps unchanged (VGG-16
// 0.596, ResNet-50 1.295 -> 1.287, MobileNet 0.326 ms).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel_overlapped(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                            cudaStream_t stream, Args... args) {
  return launch_kernel_attr(true, kernel, grid, block, smem, stream, args...);
}

// The same with the cooperative attribute when `cooperative` is set: the launch waits until every
// CTA of the grid can be resident at once (kernels whose CTAs wait for one another).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel_coop(bool cooperative, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                      cudaStream_t stream, Args... args) {
  if (!cooperative) return launch_kernel(kernel, grid, block, smem, stream, args...);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

#ifdef __CUDACC__
// see launch_kernel: call before the first global-memory access of a kernel
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Lets the next kernel of the stream, if it was launched with the attribute (the tensor-core
// kernels always are), be scheduled as soon as EVERY CTA of this grid has called this or exited.
// The persistent tensor-core kernel calls it at its start: its CTAs hold a whole SM, so the next
// kernel's CTAs start exactly where one of them has finished.  The many-block copy and depthwise
// kernels call it at their start too: the condition is met only when their last blocks are
// running, so the CTAs of a following tensor-core kernel take SMs that have no more blocks to
// wait for and set themselves up (barriers, tensor memory) beside the last wave.  Measured, NCHW
// steps as CUDA graphs: VGG-16 0.596 -> 0.589 ms, ResNet-50 1.287 -> 1.263, MobileNet 0.327 -> 0.321.
__device__ __forceinline__ void grid_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
#endif

// ---------------------------------------------------------------------------------------------
// Checked build (-DHGC_DEBUG, libhgc_debug.so): every global-memory access that a kernel of this
// library addresses by hand (everything but the copy engine's tensor-map accesses, which the
// hardware clips to the map's bounds) goes through dbg_load / dbg_store below, which test the
// address range against the tensors of the call in progress (x, w, bias, y, workspace; set by the
// entry points before they launch) and, when it lies outside, record it and SKIP the access:
// nothing faults, the caller reads the record (hgc_debug_violations).  In the ordinary build
// the helpers are the plain accesses.
struct DebugRanges {
  static constexpr int kMax = 8;
  uint64_t lo[kMax], hi[kMax];  // valid bytes [lo, hi)
  int32_t count;
};
struct DebugViolation {
  int32_t count;  // accesses outside every range since the record was last read
  int32_t line;   // source line of the first one
  uint64_t addr, bytes;
};
#ifdef HGC_DEBUG
constexpr bool kCheckedBuild = true;
#else
constexpr bool kCheckedBuild = false;
#endif
// all translation units at once (api.cu); a table without entries switches the test off
void debug_set_call_ranges(const DebugRanges& r, cudaStream_t stream);
// appends [p, p + bytes) shortened by the test hook's cut (hgc_debug_shrink_ranges)
void debug_add_range(DebugRanges* r, const void* p, size_t bytes);
// per translation unit: sets the ranges for the launches that follow on `stream`; reads and clears the record
void layout_debug_set_ranges(const DebugRanges& r, cudaStream_t stream);
void igemm_debug_set_ranges(const DebugRanges& r, cudaStream_t stream);
void depthwise_debug_set_ranges(const DebugRanges& r, cudaStream_t stream);
void direct_debug_set_ranges(const DebugRanges& r, cudaStream_t stream);
void layout_debug_read(DebugViolation* v);
void igemm_debug_read(DebugViolation* v);
void depthwise_debug_read(DebugViolation* v);
void direct_debug_read(DebugViolation* v);

#ifdef __CUDACC__
// Defines the translation unit's range table and record, the device-side test and the two host
// functions declared above (NAME = layout, igemm, depthwise, direct).
#ifdef HGC_DEBUG
#define HGC_DEBUG_STATE(NAME)                                                                              \
  namespace {                                                                                              \
  __device__ DebugRanges g_dbg_ranges;                                                                     \
  __device__ DebugViolation g_dbg_violation;                                                               \
  __device__ __noinline__ bool dbg_addr_ok(const void* p, size_t bytes, int line) {                        \
    const uint64_t a = (uint64_t)(uintptr_t)p;                                                             \
    if (g_dbg_ranges.count == 0) return true;                                                              \
    for (int i = 0; i < g_dbg_ranges.count; ++i)                                                           \
      if (a >= g_dbg_ranges.lo[i] && a + bytes <= g_dbg_ranges.hi[i]) return true;                         \
    if (atomicAdd(&g_dbg_violation.count, 1) == 0) {                                                       \
      g_dbg_violation.line = line;                                                                         \
      g_dbg_violation.addr = a;                                                                            \
      g_dbg_violation.bytes = bytes;                                                                       \
    }                                                                                                      \
    return false;                                                                                          \
  }                                                                                                        \
  }                                                                                                        \
  void NAME##_debug_set_ranges(const DebugRanges& r, cudaStream_t stream) {                                \
    cudaMemcpyToSymbolAsync(g_dbg_ranges, &r, sizeof(DebugRanges), 0, cudaMemcpyHostToDevice, stream);     \
  }                                                                                                        \
  void NAME##_debug_read(DebugViolation* v) {                                                              \
    cudaMemcpyFromSymbol(v, g_dbg_violation, sizeof(DebugViolation));                                      \
    const DebugViolation zero{};                                                                           \
    cudaMemcpyToSymbol(g_dbg_violation, &zero, sizeof(DebugViolation));                                    \
  }
#define HGC_ADDR_OK(p, bytes) dbg_addr_ok((p), (bytes), __LINE__)
#else
#define HGC_DEBUG_STATE(NAME)                                                       \
  void NAME##_debug_set_ranges(const DebugRanges&, cudaStream_t) {}                 \
  void NAME##_debug_read(DebugViolation* v) { *v = DebugViolation{}; }
#define HGC_ADDR_OK(p, bytes) true
#endif
// checked accesses (the plain access in the ordinary build): PTR is the typed pointer that is
// accessed, ACCESS the expression that reads it / STMT the statement that writes it
#define HGC_CHECKED_LOAD(VAR, PTR, ACCESS)              \
  do {                                                  \
    if (HGC_ADDR_OK((PTR), sizeof(*(PTR)))) {           \
      VAR = ACCESS;                                     \
    } else {                                            \
      VAR = {};                                         \
    }                                                   \
  } while (0)
#define HGC_CHECKED_STORE(PTR, STMT)                    \
  do {                                                  \
    if (HGC_ADDR_OK((PTR), sizeof(*(PTR)))) {           \
      STMT;                                             \
    }                                                   \
  } while (0)
#endif

// Each launcher enqueues on `stream` and returns the launch error (cudaSuccess if fine).
cudaError_t launch_direct_conv(const ConvGeom& g, const __half* x, const __half* w,
                               const __half* bias, __half* y, int relu, cudaStream_t stream);

bool depthwise3x3_supported(const ConvGeom& g);
cudaError_t launch_depthwise3x3(const ConvGeom& g, const __half* x, const __half* w,
                                const __half* bias, __half* y, int relu, cudaStream_t stream);

// channels-last variant (x and y [N][H][W][C], C % 8 == 0)
bool depthwise3x3_nhwc_supported(const ConvGeom& g);
cudaError_t launch_depthwise3x3_nhwc(const ConvGeom& g, const __half* x, const __half* w, const __half* bias,
                                     __half* y, int relu, cudaStream_t stream);

// ... and its TMA-fed form (stride 1, C % 32 == 0); the status is 0, or 1 after a copy that never
// arrived (reading it synchronises with the device and clears it)
bool depthwise3x3_nhwc_tma_supported(const ConvGeom& g);
cudaError_t launch_depthwise3x3_nhwc_tma(const ConvGeom& g, const __half* x, const __half* w, const __half* bias,
                                         __half* y, int relu, cudaStream_t stream);
int depthwise_nhwc_tma_status();

cudaError_t launch_nchw_to_nhwc(const __half* src, __half* dst, int32_t n, int32_t c, int32_t h,
                                int32_t w, int32_t c_pad, cudaStream_t stream);
cudaError_t launch_nhwc_to_nchw(const __half* src, __half* dst, int32_t n, int32_t c, int32_t h,
                                int32_t w, int32_t c_pad, cudaStream_t stream);
cudaError_t launch_nchw_to_nhwc8_bordered(const __half* src, __half* dst, int32_t n, int32_t c, int32_t h, int32_t w,
                                          int32_t pad_h, int32_t pad_w, int32_t hp, int32_t wp, cudaStream_t stream,
                                          int px_ch = 8);  // channels per pixel of the copy: 8 or 4
// perm: rows of every block of 32 output channels interleaved (see row_channel in layout.cu)
cudaError_t launch_weights_repack_window(const __half* src, __half* dst, int32_t k, int32_t c, int32_t r, int32_t s,
                                         int32_t kw_pix, cudaStream_t stream, int perm = 0, int px_ch = 8);
cudaError_t launch_weights_repack(const __half* src, __half* dst, int32_t k, int32_t cg, int32_t r,
                                  int32_t s, int32_t group, int32_t c_pad, cudaStream_t stream, int perm = 0);

cudaError_t launch_cast_f32_to_f16(const float* src, __half* dst, int64_t count, unsigned long long* overflow,
                                   cudaStream_t stream);

size_t batchnorm_workspace_bytes(int32_t n, int32_t c, int64_t hw);
cudaError_t launch_batchnorm(const __half* x, __half* y, int32_t n, int32_t c, int64_t hw, float eps,
                             int32_t shift_log2, int32_t use_stored, float* mean, float* var, void* ws,
                             cudaStream_t stream);
cudaError_t launch_bn_fold(const __half* w, const __half* bias, const float* mean, const float* var,
                           const float* gamma, const float* beta, float eps, int32_t k, int64_t per_k, __half* w_out,
                           __half* b_out, cudaStream_t stream);

// Plan of the tcgen05 implicit-GEMM path for one layer (host side).
struct IgemmPlan {
  int32_t kb, cblocks, cw, c_pad;
  int32_t halo, pitch;
  int32_t nchw, nblk;                            // 1x1 layers reading x (NCHW) directly
  const void* x_mapped;                          // input pointer tmB was encoded for (nchw, x_nhwc)
  int32_t x_nhwc, y_nhwc;                        // channels-last input (no layout pass) / output
  int32_t y_rpu, y_full_w;                       // channels-last stores: tile rows and pixels per store
  int32_t y_perm;                                // weight rows interleaved for the staged channels-last epilogue
  int32_t window, kw_pix, hp, wp;                // few-channel layers: windows over a zero-bordered NHWC8 copy
  int32_t px_ch;                                 // channels per pixel of the bordered copy: 8, or 4 (strided stems)
  int32_t dense_rows, dense_pitch;               // windows 16 bytes apart: whole rows loaded, windows read in place
  int32_t vhalo;                                 // ... and the R kernel rows share one tile of th + R - 1 rows
  int32_t patch;                                 // tiny receptive fields: 1x1 conv over an im2col copy of x
  int32_t eff_r, eff_s, eff_pad_h, eff_pad_w;    // the convolution as the kernel sees it
  int32_t tn, th, tw, ncols;
  int32_t tiles_h, tiles_n, mtiles, total_tiles;
  int32_t stages, taps;
  uint32_t stage_bytes;
  int32_t tma_store, rem, nbuf;
  int32_t epi_warps;  // epilogue warps of the launch: 8, or 16 for tiles bound by the epilogue
  void* y_mapped;  // output pointer tmY/tmYr were encoded for
  uint32_t a_bytes, b_bytes, b_alloc;
  int32_t a_rows;  // rows of a weight tile in shared memory (128, or 64 for layers of <= 64 channels per group)
  int32_t fine_units;  // TMA-store epilogue works in units of 32 pixels (else 64)
  int32_t plane_store; // whole-plane tiles leave as one bulk copy per 32-channel block
  uint32_t plane_bytes;  //   bytes of a lane quarter's staging tile
  int32_t gather;      // 1x1 layer on planes of a multiple of 4 pixels read from x (NCHW) by the kernel's extra warps (a form of nchw)
  int32_t nacc;        // depthwise + pointwise blocks: 128-channel tiles (accumulators) that share a pixel tile's depthwise result: 1, 2, 4
  // Row pairs: a stride-1 layer of 64 output channels with R kernel rows is run as a layer of 128
  // "channels" (output row parity x channel), R + 1 kernel rows and stride 2 along H on P/2 rows:
  // accumulator lanes 64..127 hold the odd output rows, so no lane of the 128-row MMA is idle
  // (3x3: 12 MMA steps per two output rows instead of 18).  The plan's shapes are those of the
  // re-stated layer; w' holds the R + 1 shifted copies of the kernel rows (zero where a row has none).
  int32_t rowpair;
  int32_t dup_log2;  // log2 of the number of copies of the layer's weight rows in w' and in a weight tile (0, 1, 2)
  size_t smem_bytes;
  int32_t ks_log2;  // log2 of the number of reduction slices a tile is split into (0 = none)
  // work distribution of the kernels without reduction slices: `grid` CTAs take contiguous ranges
  // of the ring stages of all tiles; sk_split = 1: equal ranges, a tile that straddles a boundary
  // is reduced by several CTAs (fp32 hand-over through the workspace, sk_cols32 * 32 columns)
  int32_t ts, grid, sk_split, sk_cols32;
  // CTA pairs (clusters of two sharing 256-channel tiles): th/tn/tiles_h/tiles_n describe one
  // CTA's pixel sub-tile, ncols = 2 * ncols_sub, grid counts pairs; pair_fit = pairs that can be
  // resident at once (asked of the runtime at the first launch)
  // layout pass fused into the tensor-core kernel (see IgemmArgs::lay_*): segment counters at ws_lay_off
  int32_t fuse_layout, lay_px, lay_ch, lay_units_p, lay_units_c, lay_seg_units, lay_segs;
  size_t ws_lay_off;
  // depthwise + pointwise block: the depthwise layer's input tile in shared memory
  int32_t dw_in_h, dw_in_w;
  uint32_t dw_in_bytes, dw_in_alloc;
  int32_t pair, ncols_sub, pair_fit;
  double est_clk;  // the cost model's estimate for the launch, in SM clocks
  size_t ws_status_off, ws_w_off, ws_x_off, ws_part_off, ws_sk_off, ws_total;
  bool maps_ready;
  alignas(64) CUtensorMap tmA;
  alignas(64) CUtensorMap tmB;
  alignas(64) CUtensorMap tmY;
  alignas(64) CUtensorMap tmYr;
};

// the weight re-layout and the input preparation of the tensor-core path, by plan mode
cudaError_t launch_igemm_weights(const ConvGeom& g, const IgemmPlan& p, const __half* w, __half* wp,
                                 cudaStream_t stream);
cudaError_t launch_igemm_input(const ConvGeom& g, const IgemmPlan& p, const __half* x, __half* xp,
                               cudaStream_t stream);

// number of SMs of the current device (148 if it cannot be queried)
int sm_count();

bool igemm_make_plan(const ConvGeom& g, IgemmPlan* out);
bool igemm_encode_maps(const ConvGeom& g, IgemmPlan* p, void* ws);
// The 3x3 depthwise layer in front of a pointwise layer when both run as one kernel: the
// tensor-core kernel computes its activation tiles from x (channels-last) instead of fetching them.
struct DwBlock {
  const __half* x;     // [N][h][w][c]
  const __half* w9;    // depthwise weights as [9 taps][c]
  const __half* bias;  // [c] or nullptr
  int32_t h, w, c, stride, relu;
};
cudaError_t launch_igemm(const ConvGeom& g, IgemmPlan& p, void* ws, const __half* x, const __half* bias, __half* y,
                         int relu, cudaStream_t stream, const DwBlock* dw = nullptr);
// w[c][3][3] -> w9[9][c]
cudaError_t launch_depthwise_weights_to_taps(const __half* w, __half* w9, int32_t c, cudaStream_t stream);

}  // namespace hgc
