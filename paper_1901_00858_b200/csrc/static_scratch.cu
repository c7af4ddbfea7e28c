// hgc_conv_forward_static: the tensor-core convolution for callers that cannot allocate device
// memory.  Everything the implicit-GEMM path normally keeps in a caller-provided workspace (the
// device status word, the re-laid-out weights and the NHWC copy of the input) lives in one
// file-scope device array of fixed size instead.  The array belongs to this translation unit;
// host code never uses its name as an address: the device address is looked up once per device
// with cudaGetSymbolAddress and handed to the kernels as an ordinary pointer.
#include <mutex>

#include "hgc_internal.h"

namespace {

constexpr size_t kStaticScratchBytes = 32u << 20;  // 32 MiB, held by every device that loads the library
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::mutex g_setup_mutex;
void* g_scratch_ptr[kMaxDevices] = {};  // device address of g_static_scratch, per device ordinal

// Device address of the scratch array on the current device (nullptr on failure).
void* scratch_for_current_device() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_scratch_ptr[dev] == nullptr) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) return nullptr;
    g_scratch_ptr[dev] = ptr;
  }
  return g_scratch_ptr[dev];
}

inline int64_t floor_div_pos(int64_t a, int64_t b) {
  int64_t q = a / b;
  if ((a % b) != 0 && a < 0) --q;
  return q;
}

// Same validation and shape inference as descriptor creation, into a caller-provided struct.
int make_geom(const hgc_conv_params* p, hgc::ConvGeom* g) {
  if (p == nullptr) return HGC_INVALID_ARG;
  if (p->n < 1 || p->c < 1 || p->h < 1 || p->w < 1 || p->k < 1 || p->r < 1 || p->s < 1) return HGC_INVALID_ARG;
  if (p->group < 1 || p->stride_h < 1 || p->stride_w < 1 || p->dil_h < 1 || p->dil_w < 1) return HGC_INVALID_ARG;
  if (p->pad_h < 0 || p->pad_w < 0) return HGC_INVALID_ARG;
  if (p->c % p->group != 0 || p->k % p->group != 0) return HGC_INVALID_ARG;
  const int64_t P = floor_div_pos((int64_t)p->h + 2 * p->pad_h - (int64_t)p->dil_h * (p->r - 1) - 1, p->stride_h) + 1;
  const int64_t Q = floor_div_pos((int64_t)p->w + 2 * p->pad_w - (int64_t)p->dil_w * (p->s - 1) - 1, p->stride_w) + 1;
  if (P < 1 || Q < 1) return HGC_INVALID_ARG;
  if (P > 0x7fffffffLL || Q > 0x7fffffffLL) return HGC_UNSUPPORTED;
  // NCHW tensors and the planner's tensor-core path only: a caller that sets a layout flag would
  // otherwise get a tensor in the wrong layout back with HGC_OK
  if (p->flags & (HGC_FLAG_X_NHWC | HGC_FLAG_Y_NHWC | HGC_FLAG_FORCE_DIRECT)) return HGC_UNSUPPORTED;
  g->n = p->n; g->c = p->c; g->h = p->h; g->w = p->w;
  g->k = p->k; g->r = p->r; g->s = p->s;
  g->pad_h = p->pad_h; g->pad_w = p->pad_w;
  g->stride_h = p->stride_h; g->stride_w = p->stride_w;
  g->dil_h = p->dil_h; g->dil_w = p->dil_w;
  g->group = p->group;
  g->p = (int32_t)P; g->q = (int32_t)Q;
  g->cg = p->c / p->group; g->kg = p->k / p->group;
  g->x_nhwc = 0; g->y_nhwc = 0;  // this entry point takes NCHW tensors only
  // the scheduling flags are ignored: whole tiles on single CTAs (no hand-over slots in the fixed array)
  g->no_split = 1;
  g->no_pair = 1;
  g->no_fuse = 1;
  g->no_gather = 1;
  return HGC_OK;
}

inline bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

}  // namespace

extern "C" int hgc_conv_forward_static(const hgc_conv_params* p, const void* x, const void* w, const void* bias,
                                       void* y, int relu, void* stream) {
  if (x == nullptr || w == nullptr || y == nullptr) return HGC_INVALID_ARG;
  hgc::ConvGeom g{};  // (fields this entry point never sets, the block and row-pair markers, must be zero)
  const int rc = make_geom(p, &g);
  if (rc != HGC_OK) return rc;
  if (misaligned(x) || misaligned(w) || misaligned(y) || (bias != nullptr && misaligned(bias))) return HGC_BAD_ALIGNMENT;
  hgc::IgemmPlan plan{};  // on the stack: no host heap either
  if (!hgc::igemm_make_plan(g, &plan)) return HGC_UNSUPPORTED;  // only the tensor-core path has this variant
  if (plan.ws_total > kStaticScratchBytes) return HGC_NO_WORKSPACE;  // layer needs more than the fixed 32 MiB
  char* ws = static_cast<char*>(scratch_for_current_device());
  if (ws == nullptr) return HGC_CUDA_ERROR;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the array keeps whatever the previous call left: the header (status word, hand-over flags)
  // must start at zero; the re-layout kernels rewrite every byte of the weight and input copies
  // that the tensor-core kernel reads, padding included, and a reduction slice writes every
  // partial sum before the second pass reads it
  if (hgc::kCheckedBuild) {
    hgc::DebugRanges r{};
    hgc::debug_add_range(&r, x, (size_t)g.n * g.c * g.h * g.w * 2);
    hgc::debug_add_range(&r, w, (size_t)g.k * g.cg * g.r * g.s * 2);
    hgc::debug_add_range(&r, bias, (size_t)g.k * 2);
    hgc::debug_add_range(&r, y, (size_t)g.n * g.k * g.p * g.q * 2);
    hgc::debug_add_range(&r, ws, plan.ws_total);
    hgc::debug_set_call_ranges(r, st);
  }
  if (cudaMemsetAsync(ws + plan.ws_status_off, 0, hgc::kWsHeaderBytes, st) != cudaSuccess) return HGC_CUDA_ERROR;
  if (!hgc::igemm_encode_maps(g, &plan, ws)) return HGC_CUDA_ERROR;
  const __half* xh = static_cast<const __half*>(x);
  const __half* wh = static_cast<const __half*>(w);
  __half* wp = reinterpret_cast<__half*>(ws + plan.ws_w_off);
  __half* xp = reinterpret_cast<__half*>(ws + plan.ws_x_off);
  if (hgc::launch_igemm_weights(g, plan, wh, wp, st) != cudaSuccess) return HGC_CUDA_ERROR;
  if (hgc::launch_igemm_input(g, plan, xh, xp, st) != cudaSuccess) return HGC_CUDA_ERROR;
  if (hgc::launch_igemm(g, plan, ws, xh, static_cast<const __half*>(bias), static_cast<__half*>(y), relu, st) !=
      cudaSuccess)
    return HGC_CUDA_ERROR;
  return HGC_OK;
}
