// Host side of libhgc: parameter validation, shape inference, path choice, workspace
// bookkeeping and the extern "C" entry points declared in hgc.h.
#include <atomic>
#include <new>

#include "hgc_internal.h"

namespace hgc {
static std::atomic<uint64_t> g_launches{0};
void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }
static std::atomic<int> g_debug_drop{-1};
int debug_drop_copies() { return g_debug_drop.load(std::memory_order_relaxed); }
static std::atomic<bool> g_launch_overlap{false};
static std::atomic<long long> g_debug_shrink{0};
void debug_add_range(DebugRanges* r, const void* p, size_t bytes) {
  if (p == nullptr || bytes == 0 || r->count >= DebugRanges::kMax) return;
  const uint64_t cut = (uint64_t)g_debug_shrink.load(std::memory_order_relaxed);
  r->lo[r->count] = (uint64_t)(uintptr_t)p;
  r->hi[r->count] = r->lo[r->count] + (bytes > cut ? bytes - cut : 0);
  ++r->count;
}
void debug_set_call_ranges(const DebugRanges& r, cudaStream_t stream) {
  if (!kCheckedBuild) return;
  layout_debug_set_ranges(r, stream);
  igemm_debug_set_ranges(r, stream);
  depthwise_debug_set_ranges(r, stream);
  direct_debug_set_ranges(r, stream);
}
bool launch_overlap_enabled() { return g_launch_overlap.load(std::memory_order_relaxed); }
void set_launch_overlap(bool on) { g_launch_overlap.store(on, std::memory_order_relaxed); }
}  // namespace hgc

struct hgc_conv_desc {
  hgc_conv_params params;
  hgc::ConvGeom geom;
  int32_t path;
  size_t ws_needed;       // bytes the chosen path needs
  void* ws;               // caller-owned device scratch
  size_t ws_bytes;
  const void* registered_w;
  hgc::IgemmPlan igemm;
  // depthwise + pointwise block (hgc_dwpw_desc_create): geom / igemm describe the pointwise layer
  // on the depthwise layer's output plane; the depthwise layer itself:
  bool is_dwpw;
  int32_t dw_h, dw_w, dw_stride;
  size_t ws_dw_off;             // depthwise weights as [9][C] in the workspace
  const void* registered_w_dw;
};

namespace {

inline int64_t floor_div_pos(int64_t a, int64_t b) {  // b > 0
  int64_t q = a / b;
  if ((a % b) != 0 && a < 0) --q;
  return q;
}

inline int64_t out_extent(int64_t in, int64_t kernel, int64_t pad, int64_t stride, int64_t dil) {
  return floor_div_pos(in + 2 * pad - dil * (kernel - 1) - 1, stride) + 1;
}

inline bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct HostStaging {
  size_t x_off, w_off, b_off, y_off, total;
  size_t x_bytes, w_bytes, b_bytes, y_bytes;
};

HostStaging host_staging(const hgc_conv_desc* d) {
  const hgc::ConvGeom& g = d->geom;
  HostStaging s;
  s.x_bytes = (size_t)g.n * g.c * g.h * g.w * 2;
  s.w_bytes = (size_t)g.k * g.cg * g.r * g.s * 2;
  s.b_bytes = (size_t)g.k * 2;
  s.y_bytes = (size_t)g.n * g.k * g.p * g.q * 2;
  s.x_off = round_up(d->ws_needed, 256);
  s.w_off = s.x_off + round_up(s.x_bytes, 256);
  s.b_off = s.w_off + round_up(s.w_bytes, 256);
  s.y_off = s.b_off + round_up(s.b_bytes, 256);
  s.total = s.y_off + round_up(s.y_bytes, 256);
  return s;
}

// Checked build: the byte ranges that the kernels of one forward call may touch.
void debug_register_ranges(const hgc::ConvGeom& g, const void* x, const void* w, const void* bias, const void* y,
                           const void* ws, size_t ws_bytes, cudaStream_t stream) {
  if (!hgc::kCheckedBuild) return;
  hgc::DebugRanges r{};
  hgc::debug_add_range(&r, x, (size_t)g.n * g.c * g.h * g.w * 2);
  hgc::debug_add_range(&r, w, (size_t)g.k * g.cg * g.r * g.s * 2);
  hgc::debug_add_range(&r, bias, (size_t)g.k * 2);
  hgc::debug_add_range(&r, y, (size_t)g.n * g.k * g.p * g.q * 2);
  hgc::debug_add_range(&r, ws, ws_bytes);
  hgc::debug_set_call_ranges(r, stream);
}

int forward_impl(hgc_conv_desc* d, const void* x, const void* w, const void* bias, void* y,
                 int relu, cudaStream_t stream) {
  const hgc::ConvGeom& g = d->geom;
  debug_register_ranges(g, x, w, bias, y, d->ws, d->ws_needed, stream);
  const __half* xh = static_cast<const __half*>(x);
  const __half* wh = static_cast<const __half*>(w);
  const __half* bh = static_cast<const __half*>(bias);
  __half* yh = static_cast<__half*>(y);
  cudaError_t err;
  switch (d->path) {
    case HGC_PATH_IGEMM: {
      char* ws = static_cast<char*>(d->ws);
      hgc::IgemmPlan& ip = d->igemm;
      __half* wp = reinterpret_cast<__half*>(ws + ip.ws_w_off);
      __half* xp = reinterpret_cast<__half*>(ws + ip.ws_x_off);
      if (d->registered_w != w) {  // weights not prepared in advance: re-lay them out now
        err = hgc::launch_igemm_weights(g, ip, wh, wp, stream);
        if (err != cudaSuccess) break;
      }
      err = hgc::launch_igemm_input(g, ip, xh, xp, stream);
      if (err != cudaSuccess) break;
      err = hgc::launch_igemm(g, ip, ws, xh, bh, yh, relu, stream);
      break;
    }
    case HGC_PATH_DEPTHWISE:
      err = g.x_nhwc ? (hgc::depthwise3x3_nhwc_tma_supported(g)
                            ? hgc::launch_depthwise3x3_nhwc_tma(g, xh, wh, bh, yh, relu, stream)
                            : hgc::launch_depthwise3x3_nhwc(g, xh, wh, bh, yh, relu, stream))
                     : hgc::launch_depthwise3x3(g, xh, wh, bh, yh, relu, stream);
      break;
    case HGC_PATH_DIRECT:
    default:
      err = hgc::launch_direct_conv(g, xh, wh, bh, yh, relu, stream);
      break;
  }
  if (err == cudaErrorInvalidConfiguration) return HGC_UNSUPPORTED;
  return err == cudaSuccess ? HGC_OK : HGC_CUDA_ERROR;
}

}  // namespace

extern "C" {

int hgc_conv_desc_create(hgc_conv_desc** out, const hgc_conv_params* p) {
  if (out == nullptr) return HGC_INVALID_ARG;
  *out = nullptr;
  if (p == nullptr) return HGC_INVALID_ARG;
  if (p->n < 1 || p->c < 1 || p->h < 1 || p->w < 1 || p->k < 1 || p->r < 1 || p->s < 1)
    return HGC_INVALID_ARG;
  if (p->group < 1 || p->stride_h < 1 || p->stride_w < 1 || p->dil_h < 1 || p->dil_w < 1)
    return HGC_INVALID_ARG;
  if (p->pad_h < 0 || p->pad_w < 0) return HGC_INVALID_ARG;
  if (p->c % p->group != 0 || p->k % p->group != 0) return HGC_INVALID_ARG;
  const int64_t P = out_extent(p->h, p->r, p->pad_h, p->stride_h, p->dil_h);
  const int64_t Q = out_extent(p->w, p->s, p->pad_w, p->stride_w, p->dil_w);
  if (P < 1 || Q < 1) return HGC_INVALID_ARG;
  if (P > 0x7fffffffLL || Q > 0x7fffffffLL) return HGC_UNSUPPORTED;

  hgc_conv_desc* d = new (std::nothrow) hgc_conv_desc();
  if (d == nullptr) return HGC_CUDA_ERROR;
  d->params = *p;
  hgc::ConvGeom& g = d->geom;
  g.n = p->n; g.c = p->c; g.h = p->h; g.w = p->w;
  g.k = p->k; g.r = p->r; g.s = p->s;
  g.pad_h = p->pad_h; g.pad_w = p->pad_w;
  g.stride_h = p->stride_h; g.stride_w = p->stride_w;
  g.dil_h = p->dil_h; g.dil_w = p->dil_w;
  g.group = p->group;
  g.p = (int32_t)P; g.q = (int32_t)Q;
  g.cg = p->c / p->group; g.kg = p->k / p->group;
  g.x_nhwc = (p->flags & HGC_FLAG_X_NHWC) ? 1 : 0;
  g.y_nhwc = (p->flags & HGC_FLAG_Y_NHWC) ? 1 : 0;
  g.no_pair = (p->flags & HGC_FLAG_CTA_PAIRS) ? 0 : 1;
  g.no_split = (p->flags & HGC_FLAG_WHOLE_TILES) ? 1 : ((p->flags & HGC_FLAG_SHARED_TILES) ? 0 : 2);  // 2: the planner's cost model decides
  g.no_fuse = (p->flags & HGC_FLAG_FUSED_LAYOUT) ? 0 : 1;
  g.no_gather = (p->flags & HGC_FLAG_GATHER_X) ? 0 : 1;
  const bool channels_last = g.x_nhwc || g.y_nhwc;

  d->path = HGC_PATH_DIRECT;
  d->ws_needed = 0;
  if (!(p->flags & HGC_FLAG_FORCE_DIRECT)) {
    if (!channels_last && hgc::depthwise3x3_supported(g)) {
      d->path = HGC_PATH_DEPTHWISE;
    } else if (g.x_nhwc && g.y_nhwc && hgc::depthwise3x3_nhwc_supported(g)) {
      d->path = HGC_PATH_DEPTHWISE;  // channels-last on both sides: its own kernel
    } else if (hgc::igemm_make_plan(g, &d->igemm)) {
      d->path = HGC_PATH_IGEMM;
      d->ws_needed = d->igemm.ws_total;
    }
  }
  // channels-last tensors: the tensor-core path, or a depthwise layer with both sides channels-last
  if (channels_last && d->path != HGC_PATH_IGEMM && !(d->path == HGC_PATH_DEPTHWISE && g.x_nhwc && g.y_nhwc)) {
    delete d;
    return HGC_UNSUPPORTED;
  }
  d->ws = nullptr;
  d->ws_bytes = 0;
  d->registered_w = nullptr;
  *out = d;
  return HGC_OK;
}

int hgc_conv_desc_destroy(hgc_conv_desc* d) {
  delete d;
  return HGC_OK;
}

int hgc_conv_forward(hgc_conv_desc* d, const void* x, const void* w, const void* bias, void* y,
                     int relu, void* stream) {
  if (d == nullptr || x == nullptr || w == nullptr || y == nullptr) return HGC_INVALID_ARG;
  if (d->is_dwpw) return HGC_INVALID_ARG;  // a block descriptor: hgc_dwpw_forward
  if (misaligned(x) || misaligned(w) || misaligned(y) || (bias != nullptr && misaligned(bias)))
    return HGC_BAD_ALIGNMENT;
  if (d->ws_needed > 0 && (d->ws == nullptr || d->ws_bytes < d->ws_needed)) return HGC_NO_WORKSPACE;
  return forward_impl(d, x, w, bias, y, relu, static_cast<cudaStream_t>(stream));
}

int hgc_conv_forward_host(hgc_conv_desc* d, const void* x, const void* w, const void* bias, void* y,
                          int relu, void* stream) {
  if (d == nullptr || x == nullptr || w == nullptr || y == nullptr) return HGC_INVALID_ARG;
  if (d->is_dwpw) return HGC_INVALID_ARG;
  const HostStaging s = host_staging(d);
  if (d->ws == nullptr || d->ws_bytes < s.total) return HGC_NO_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* base = static_cast<char*>(d->ws);
  if (cudaMemcpyAsync(base + s.x_off, x, s.x_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess)
    return HGC_CUDA_ERROR;
  if (cudaMemcpyAsync(base + s.w_off, w, s.w_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess)
    return HGC_CUDA_ERROR;
  if (bias != nullptr &&
      cudaMemcpyAsync(base + s.b_off, bias, s.b_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess)
    return HGC_CUDA_ERROR;
  // host weights arrive anew on every call: never treat them as registered
  d->registered_w = nullptr;
  const int rc = forward_impl(d, base + s.x_off, base + s.w_off, bias ? base + s.b_off : nullptr,
                              base + s.y_off, relu, st);
  if (rc != HGC_OK) return rc;
  if (cudaMemcpyAsync(y, base + s.y_off, s.y_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return HGC_CUDA_ERROR;
  return HGC_OK;
}

int hgc_conv_output_dims(const hgc_conv_desc* d, int32_t* n, int32_t* k, int32_t* p, int32_t* q) {
  if (d == nullptr) return HGC_INVALID_ARG;
  if (n) *n = d->geom.n;
  if (k) *k = d->geom.k;
  if (p) *p = d->geom.p;
  if (q) *q = d->geom.q;
  return HGC_OK;
}

int hgc_conv_path(const hgc_conv_desc* d, int32_t* path) {
  if (d == nullptr || path == nullptr) return HGC_INVALID_ARG;
  *path = d->path;
  return HGC_OK;
}

int hgc_conv_plan_info(const hgc_conv_desc* d, int32_t* info, int32_t count) {
  if (d == nullptr || info == nullptr || count < 1) return HGC_INVALID_ARG;
  int32_t v[19] = {d->path, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0};
  if (d->path == HGC_PATH_IGEMM) {
    const hgc::IgemmPlan& p = d->igemm;
    v[1] = p.kb; v[2] = p.halo; v[3] = p.tn; v[4] = p.th; v[5] = p.pitch; v[6] = p.ncols;
    v[7] = p.total_tiles; v[8] = p.stages; v[9] = p.taps;
    v[10] = p.gather ? 4 : ((p.nchw || p.x_nhwc) ? 1 : (p.window ? 2 : (p.patch ? 3 : 0)));
    v[11] = 1 << p.ks_log2;
    v[12] = p.ks_log2 > 0 ? 0 : ((p.pair && p.pair_fit > 0 && p.pair_fit < p.grid) ? p.pair_fit : p.grid);
    v[13] = p.sk_split;
    v[14] = p.pair;
    v[15] = p.fuse_layout;
    v[16] = p.rowpair;
    v[17] = 1 << p.dup_log2;
    v[18] = p.plane_store ? 2 : (p.tma_store ? 1 : 0);
  }
  for (int i = 0; i < count && i < 19; ++i) info[i] = v[i];
  return HGC_OK;
}

int hgc_conv_workspace_bytes(const hgc_conv_desc* d, size_t* bytes) {
  if (d == nullptr || bytes == nullptr) return HGC_INVALID_ARG;
  *bytes = d->ws_needed;
  return HGC_OK;
}

int hgc_conv_host_workspace_bytes(const hgc_conv_desc* d, size_t* bytes) {
  if (d == nullptr || bytes == nullptr) return HGC_INVALID_ARG;
  *bytes = host_staging(d).total;
  return HGC_OK;
}

int hgc_conv_set_workspace(hgc_conv_desc* d, void* dev_ptr, size_t bytes) {
  if (d == nullptr) return HGC_INVALID_ARG;
  if (dev_ptr == nullptr && bytes != 0) return HGC_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(dev_ptr) & 255u) != 0) return HGC_BAD_ALIGNMENT;
  d->ws = dev_ptr;
  d->ws_bytes = dev_ptr ? bytes : 0;
  d->registered_w = nullptr;
  d->registered_w_dw = nullptr;
  d->igemm.maps_ready = false;
  d->igemm.y_mapped = nullptr;
  d->igemm.x_mapped = nullptr;
  if (d->path == HGC_PATH_IGEMM && dev_ptr != nullptr && bytes >= d->ws_needed) {
    // the TMA descriptors point into the workspace: encode them now; clear the status word
    if (!hgc::igemm_encode_maps(d->geom, &d->igemm, dev_ptr)) return HGC_CUDA_ERROR;
    if (cudaMemset(static_cast<char*>(dev_ptr) + d->igemm.ws_status_off, 0, hgc::kWsHeaderBytes) != cudaSuccess)
      return HGC_CUDA_ERROR;
    if (d->igemm.fuse_layout &&
        cudaMemset(static_cast<char*>(dev_ptr) + d->igemm.ws_lay_off, 0,
                   ((size_t)d->geom.n * d->igemm.lay_segs + 1) * sizeof(int)) != cudaSuccess)
      return HGC_CUDA_ERROR;
  }
  return HGC_OK;
}

int hgc_conv_set_weights(hgc_conv_desc* d, const void* w, void* stream) {
  if (d == nullptr || w == nullptr) return HGC_INVALID_ARG;
  if (d->is_dwpw) return HGC_INVALID_ARG;  // hgc_dwpw_set_weights
  if (misaligned(w)) return HGC_BAD_ALIGNMENT;
  if (d->ws_needed > 0 && (d->ws == nullptr || d->ws_bytes < d->ws_needed)) return HGC_NO_WORKSPACE;
  if (d->path == HGC_PATH_IGEMM) {
    const hgc::ConvGeom& g = d->geom;
    __half* wp = reinterpret_cast<__half*>(static_cast<char*>(d->ws) + d->igemm.ws_w_off);
    const cudaError_t err = hgc::launch_igemm_weights(g, d->igemm, static_cast<const __half*>(w), wp,
                                                      static_cast<cudaStream_t>(stream));
    if (err != cudaSuccess) return HGC_CUDA_ERROR;
  }
  d->registered_w = w;
  return HGC_OK;
}

int hgc_conv_last_device_status(hgc_conv_desc* d, int32_t* status) {
  if (d == nullptr || status == nullptr) return HGC_INVALID_ARG;
  *status = HGC_OK;
  if (d->path == HGC_PATH_IGEMM && d->ws != nullptr && d->ws_bytes >= d->ws_needed) {
    int32_t word = 0;
    char* sp = static_cast<char*>(d->ws) + d->igemm.ws_status_off;
    if (cudaMemcpy(&word, sp, sizeof(word), cudaMemcpyDeviceToHost) != cudaSuccess) return HGC_CUDA_ERROR;
    if (word != 0) {
      *status = word;
      // the launch that gave up may have left hand-over flags raised: clear the whole header
      if (cudaMemset(sp, 0, hgc::kWsHeaderBytes) != cudaSuccess) return HGC_CUDA_ERROR;
      if (d->igemm.fuse_layout &&
          cudaMemset(static_cast<char*>(d->ws) + d->igemm.ws_lay_off, 0,
                     ((size_t)d->geom.n * d->igemm.lay_segs + 1) * sizeof(int)) != cudaSuccess)
        return HGC_CUDA_ERROR;
    }
  }
  // the TMA-fed channels-last depthwise kernel keeps one status word per process
  if (d->path == HGC_PATH_DEPTHWISE && d->geom.x_nhwc && hgc::depthwise3x3_nhwc_tma_supported(d->geom)) {
    const int v = hgc::depthwise_nhwc_tma_status();
    if (v < 0) return HGC_CUDA_ERROR;
    if (v != 0) *status = HGC_DEVICE_TIMEOUT;
  }
  return HGC_OK;
}

int hgc_layout_nchw_to_nhwc(const void* src, void* dst, int32_t n, int32_t c, int32_t h, int32_t w,
                            int32_t c_pad, void* stream) {
  if (src == nullptr || dst == nullptr || n < 1 || c < 1 || h < 1 || w < 1 || c_pad < c || (c_pad % 8) != 0)
    return HGC_INVALID_ARG;
  if (misaligned(src) || misaligned(dst)) return HGC_BAD_ALIGNMENT;
  cudaError_t err = hgc::launch_nchw_to_nhwc(static_cast<const __half*>(src), static_cast<__half*>(dst), n,
                                            c, h, w, c_pad, static_cast<cudaStream_t>(stream));
  if (err == cudaErrorInvalidConfiguration) return HGC_UNSUPPORTED;
  return err == cudaSuccess ? HGC_OK : HGC_CUDA_ERROR;
}

int hgc_layout_nhwc_to_nchw(const void* src, void* dst, int32_t n, int32_t c, int32_t h, int32_t w,
                            int32_t c_pad, void* stream) {
  if (src == nullptr || dst == nullptr || n < 1 || c < 1 || h < 1 || w < 1 || c_pad < c || (c_pad % 8) != 0)
    return HGC_INVALID_ARG;
  if (misaligned(src) || misaligned(dst)) return HGC_BAD_ALIGNMENT;
  cudaError_t err = hgc::launch_nhwc_to_nchw(static_cast<const __half*>(src), static_cast<__half*>(dst), n,
                                            c, h, w, c_pad, static_cast<cudaStream_t>(stream));
  if (err == cudaErrorInvalidConfiguration) return HGC_UNSUPPORTED;
  return err == cudaSuccess ? HGC_OK : HGC_CUDA_ERROR;
}

int hgc_weights_repack(const void* src, void* dst, int32_t k, int32_t c_per_group, int32_t r, int32_t s,
                       int32_t group, int32_t c_pad, void* stream) {
  if (src == nullptr || dst == nullptr || k < 1 || c_per_group < 1 || r < 1 || s < 1 || group < 1 ||
      (k % group) != 0 || c_pad < c_per_group || (c_pad % 8) != 0)
    return HGC_INVALID_ARG;
  if (misaligned(src) || misaligned(dst)) return HGC_BAD_ALIGNMENT;
  cudaError_t err = hgc::launch_weights_repack(static_cast<const __half*>(src), static_cast<__half*>(dst), k,
                                              c_per_group, r, s, group, c_pad,
                                              static_cast<cudaStream_t>(stream));
  return err == cudaSuccess ? HGC_OK : HGC_CUDA_ERROR;
}

int hgc_dwpw_desc_create(hgc_conv_desc** out, const hgc_dwpw_params* p) {
  if (out == nullptr) return HGC_INVALID_ARG;
  *out = nullptr;
  if (p == nullptr) return HGC_INVALID_ARG;
  if (p->n < 1 || p->c < 1 || p->h < 1 || p->w < 1 || p->k < 1) return HGC_INVALID_ARG;
  if (p->stride != 1 && p->stride != 2) return HGC_INVALID_ARG;
  if (p->flags & ~HGC_FLAG_Y_NHWC) return HGC_INVALID_ARG;
  // the depthwise layer: 3x3, pad 1; its output plane is the pointwise layer's plane
  const int64_t P = out_extent(p->h, 3, 1, p->stride, 1);
  const int64_t Q = out_extent(p->w, 3, 1, p->stride, 1);
  if (P < 1 || Q < 1) return HGC_INVALID_ARG;
  hgc_conv_desc* d = new (std::nothrow) hgc_conv_desc();
  if (d == nullptr) return HGC_CUDA_ERROR;
  hgc_conv_params& cp = d->params;
  cp.n = p->n; cp.c = p->c; cp.h = (int32_t)P; cp.w = (int32_t)Q; cp.k = p->k; cp.r = 1; cp.s = 1;
  cp.pad_h = 0; cp.pad_w = 0; cp.stride_h = 1; cp.stride_w = 1; cp.dil_h = 1; cp.dil_w = 1; cp.group = 1;
  cp.flags = HGC_FLAG_X_NHWC | (p->flags & HGC_FLAG_Y_NHWC);
  hgc::ConvGeom& g = d->geom;
  g.n = p->n; g.c = p->c; g.h = (int32_t)P; g.w = (int32_t)Q; g.k = p->k; g.r = 1; g.s = 1;
  g.pad_h = 0; g.pad_w = 0; g.stride_h = 1; g.stride_w = 1; g.dil_h = 1; g.dil_w = 1; g.group = 1;
  g.p = (int32_t)P; g.q = (int32_t)Q; g.cg = p->c; g.kg = p->k;
  g.x_nhwc = 1;
  g.y_nhwc = (p->flags & HGC_FLAG_Y_NHWC) ? 1 : 0;
  g.no_pair = 1; g.no_split = 1; g.no_fuse = 1; g.no_gather = 1;
  g.dw_stride = p->stride;
  // the tensor-core plan of the pointwise layer over a channels-last input that is never stored:
  // whole 8-channel chunks, 32- or 64-channel stages, whole tiles on single CTAs
  if ((p->c % 8) != 0 || !hgc::igemm_make_plan(g, &d->igemm) || d->igemm.kb < 32 || d->igemm.ks_log2 > 0 ||
      !d->igemm.x_nhwc || d->igemm.dw_in_bytes == 0) {
    delete d;
    return HGC_UNSUPPORTED;
  }
  d->path = HGC_PATH_IGEMM;
  d->is_dwpw = true;
  d->dw_h = p->h; d->dw_w = p->w; d->dw_stride = p->stride;
  d->ws_dw_off = round_up(d->igemm.ws_total, 256);
  d->ws_needed = d->ws_dw_off + round_up((size_t)9 * p->c * 2, 256);
  d->ws = nullptr;
  d->ws_bytes = 0;
  d->registered_w = nullptr;
  d->registered_w_dw = nullptr;
  *out = d;
  return HGC_OK;
}

int hgc_dwpw_set_weights(hgc_conv_desc* d, const void* w_dw, const void* w_pw, void* stream) {
  if (d == nullptr || w_dw == nullptr || w_pw == nullptr || !d->is_dwpw) return HGC_INVALID_ARG;
  if (misaligned(w_dw) || misaligned(w_pw)) return HGC_BAD_ALIGNMENT;
  if (d->ws == nullptr || d->ws_bytes < d->ws_needed) return HGC_NO_WORKSPACE;
  char* ws = static_cast<char*>(d->ws);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (hgc::launch_igemm_weights(d->geom, d->igemm, static_cast<const __half*>(w_pw),
                                reinterpret_cast<__half*>(ws + d->igemm.ws_w_off), st) != cudaSuccess)
    return HGC_CUDA_ERROR;
  if (hgc::launch_depthwise_weights_to_taps(static_cast<const __half*>(w_dw), reinterpret_cast<__half*>(ws + d->ws_dw_off),
                                            d->geom.c, st) != cudaSuccess)
    return HGC_CUDA_ERROR;
  d->registered_w = w_pw;
  d->registered_w_dw = w_dw;
  return HGC_OK;
}

int hgc_dwpw_forward(hgc_conv_desc* d, const void* x, const void* w_dw, const void* bias_dw, const void* w_pw,
                     const void* bias_pw, void* y, int relu_dw, int relu_pw, void* stream) {
  if (d == nullptr || x == nullptr || w_dw == nullptr || w_pw == nullptr || y == nullptr || !d->is_dwpw)
    return HGC_INVALID_ARG;
  if (misaligned(x) || misaligned(w_dw) || misaligned(w_pw) || misaligned(y) || (bias_dw != nullptr && misaligned(bias_dw)) ||
      (bias_pw != nullptr && misaligned(bias_pw)))
    return HGC_BAD_ALIGNMENT;
  if (d->ws == nullptr || d->ws_bytes < d->ws_needed) return HGC_NO_WORKSPACE;
  char* ws = static_cast<char*>(d->ws);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (hgc::kCheckedBuild) {
    const hgc::ConvGeom& g = d->geom;  // the pointwise layer on the depthwise layer's output plane
    hgc::DebugRanges r{};
    hgc::debug_add_range(&r, x, (size_t)g.n * g.c * d->dw_h * d->dw_w * 2);
    hgc::debug_add_range(&r, w_dw, (size_t)g.c * 9 * 2);
    hgc::debug_add_range(&r, bias_dw, (size_t)g.c * 2);
    hgc::debug_add_range(&r, w_pw, (size_t)g.k * g.c * 2);
    hgc::debug_add_range(&r, bias_pw, (size_t)g.k * 2);
    hgc::debug_add_range(&r, y, (size_t)g.n * g.k * g.p * g.q * 2);
    hgc::debug_add_range(&r, ws, d->ws_needed);
    hgc::debug_set_call_ranges(r, st);
  }
  if (d->registered_w != w_pw || d->registered_w_dw != w_dw) {  // weights not prepared in advance: re-lay them out now
    if (hgc::launch_igemm_weights(d->geom, d->igemm, static_cast<const __half*>(w_pw),
                                  reinterpret_cast<__half*>(ws + d->igemm.ws_w_off), st) != cudaSuccess)
      return HGC_CUDA_ERROR;
    if (hgc::launch_depthwise_weights_to_taps(static_cast<const __half*>(w_dw), reinterpret_cast<__half*>(ws + d->ws_dw_off),
                                              d->geom.c, st) != cudaSuccess)
      return HGC_CUDA_ERROR;
  }
  hgc::DwBlock dw{};
  dw.x = static_cast<const __half*>(x);
  dw.w9 = reinterpret_cast<const __half*>(ws + d->ws_dw_off);
  dw.bias = static_cast<const __half*>(bias_dw);
  dw.h = d->dw_h; dw.w = d->dw_w; dw.c = d->geom.c; dw.stride = d->dw_stride; dw.relu = relu_dw ? 1 : 0;
  const cudaError_t err = hgc::launch_igemm(d->geom, d->igemm, ws, static_cast<const __half*>(x),
                                            static_cast<const __half*>(bias_pw), static_cast<__half*>(y), relu_pw, st, &dw);
  if (err == cudaErrorInvalidConfiguration || err == cudaErrorInvalidValue) return HGC_UNSUPPORTED;
  return err == cudaSuccess ? HGC_OK : HGC_CUDA_ERROR;
}

int hgc_inner_product_desc_create(hgc_conv_desc** out, int32_t n, int32_t c, int32_t k) {
  hgc_conv_params p{};
  p.n = n; p.c = c; p.h = 1; p.w = 1; p.k = k; p.r = 1; p.s = 1;
  p.pad_h = 0; p.pad_w = 0; p.stride_h = 1; p.stride_w = 1; p.dil_h = 1; p.dil_w = 1; p.group = 1; p.flags = 0;
  return hgc_conv_desc_create(out, &p);
}

int hgc_cast_f32_to_f16(const void* src, void* dst, int64_t count, uint64_t* overflow_count, void* stream) {
  if (count < 0 || (count > 0 && (src == nullptr || dst == nullptr))) return HGC_INVALID_ARG;
  if (count == 0) return HGC_OK;
  if (misaligned(src) || misaligned(dst) || (reinterpret_cast<uintptr_t>(overflow_count) & 7u) != 0)
    return HGC_BAD_ALIGNMENT;
  const cudaError_t err =
      hgc::launch_cast_f32_to_f16(static_cast<const float*>(src), static_cast<__half*>(dst), count,
                                  reinterpret_cast<unsigned long long*>(overflow_count),
                                  static_cast<cudaStream_t>(stream));
  return err == cudaSuccess ? HGC_OK : HGC_CUDA_ERROR;
}

size_t hgc_batchnorm_workspace_bytes(int32_t n, int32_t c, int64_t hw) {
  if (n < 1 || c < 1 || hw < 1) return 0;
  return hgc::batchnorm_workspace_bytes(n, c, hw);
}

int hgc_batchnorm_forward(const void* x, void* y, int32_t n, int32_t c, int64_t hw, float eps, int32_t shift_log2,
                          int32_t use_stored, float* mean, float* var, void* workspace, void* stream) {
  if (x == nullptr || y == nullptr || mean == nullptr || var == nullptr) return HGC_INVALID_ARG;
  if (n < 1 || c < 1 || hw < 1 || !(eps >= 0.f) || shift_log2 < -8 || shift_log2 > 8) return HGC_INVALID_ARG;
  const int64_t chunks = (hw + 2047) / 2048;
  if (c > 65535 || (int64_t)n * chunks > 0x7fffffffLL) return HGC_UNSUPPORTED;
  if (misaligned(x) || misaligned(y) || (workspace != nullptr && misaligned(workspace))) return HGC_BAD_ALIGNMENT;
  if ((reinterpret_cast<uintptr_t>(mean) & 3u) != 0 || (reinterpret_cast<uintptr_t>(var) & 3u) != 0)
    return HGC_BAD_ALIGNMENT;
  if (!use_stored && workspace == nullptr) return HGC_NO_WORKSPACE;
  const cudaError_t err =
      hgc::launch_batchnorm(static_cast<const __half*>(x), static_cast<__half*>(y), n, c, hw, eps, shift_log2,
                            use_stored != 0, mean, var, workspace, static_cast<cudaStream_t>(stream));
  return err == cudaSuccess ? HGC_OK : HGC_CUDA_ERROR;
}

int hgc_bn_fold(const void* w, const void* bias, const float* mean, const float* var, const float* gamma,
                const float* beta, float eps, int32_t k, int64_t per_k, void* w_out, void* b_out, void* stream) {
  if (w == nullptr || mean == nullptr || var == nullptr || w_out == nullptr || b_out == nullptr) return HGC_INVALID_ARG;
  if (k < 1 || per_k < 1 || !(eps >= 0.f)) return HGC_INVALID_ARG;
  const cudaError_t err = hgc::launch_bn_fold(static_cast<const __half*>(w), static_cast<const __half*>(bias), mean,
                                              var, gamma, beta, eps, k, per_k, static_cast<__half*>(w_out),
                                              static_cast<__half*>(b_out), static_cast<cudaStream_t>(stream));
  return err == cudaSuccess ? HGC_OK : HGC_CUDA_ERROR;
}

int hgc_debug_set_wait_limit_ns(uint64_t ns) {
  if (hgc::igemm_set_wait_limit_ns(ns) != cudaSuccess) return HGC_CUDA_ERROR;
  if (hgc::depthwise_nhwc_tma_set_wait_limit_ns(ns) != cudaSuccess) return HGC_CUDA_ERROR;
  return HGC_OK;
}

int hgc_debug_drop_copies(int32_t index) {
  hgc::g_debug_drop.store(index < 0 ? -1 : index, std::memory_order_relaxed);
  return HGC_OK;
}

int hgc_debug_checked_build(void) { return hgc::kCheckedBuild ? 1 : 0; }

int hgc_debug_violations(int32_t* count, int32_t* line, uint64_t* addr, uint64_t* bytes) {
  if (count == nullptr) return HGC_INVALID_ARG;
  if (cudaDeviceSynchronize() != cudaSuccess) return HGC_CUDA_ERROR;
  hgc::DebugViolation v[4];
  hgc::layout_debug_read(&v[0]);
  hgc::igemm_debug_read(&v[1]);
  hgc::depthwise_debug_read(&v[2]);
  hgc::direct_debug_read(&v[3]);
  int32_t total = 0;
  const hgc::DebugViolation* first = nullptr;
  for (const hgc::DebugViolation& e : v) {
    total += e.count;
    if (e.count > 0 && first == nullptr) first = &e;
  }
  *count = total;
  if (line != nullptr) *line = first != nullptr ? first->line : 0;
  if (addr != nullptr) *addr = first != nullptr ? first->addr : 0;
  if (bytes != nullptr) *bytes = first != nullptr ? first->bytes : 0;
  return HGC_OK;
}

int hgc_debug_shrink_ranges(int64_t bytes) {
  if (bytes < 0) return HGC_INVALID_ARG;
  hgc::g_debug_shrink.store(bytes, std::memory_order_relaxed);
  return HGC_OK;
}

int hgc_set_launch_overlap(int enabled) {
  hgc::set_launch_overlap(enabled != 0);
  return HGC_OK;
}

int hgc_kernel_launch_count(uint64_t* count) {
  if (count == nullptr) return HGC_INVALID_ARG;
  *count = hgc::g_launches.load(std::memory_order_relaxed);
  return HGC_OK;
}

const char* hgc_status_string(int status) {
  switch (status) {
    case HGC_OK: return "ok";
    case HGC_INVALID_ARG: return "invalid argument";
    case HGC_UNSUPPORTED: return "unsupported";
    case HGC_BAD_ALIGNMENT: return "device pointer not 16-byte aligned";
    case HGC_NO_WORKSPACE: return "workspace missing or too small";
    case HGC_CUDA_ERROR: return "CUDA error";
    case HGC_DEVICE_TIMEOUT: return "device-side wait timed out";
    default: return "unknown status";
  }
}

}  // extern "C"
