// Direct convolution on CUDA cores: the path for any valid layer (and the fallback of the
// planner for shapes the specialised kernels do not take).  NCHW in, NCHW out, fp32
// accumulation, fused bias + ReLU + one round-to-nearest-even conversion to binary16.
//
// Work split: one thread per output pixel, KT output channels of one group per CTA row, so a
// loaded input value feeds KT FMAs.  The CTA's KT weight rows are staged in shared memory in
// chunks of the flattened (c', r, s) tap index; every thread walks the chunk with running
// (c', r, s) counters.
#include "hgc_internal.h"

namespace hgc {
HGC_DEBUG_STATE(direct)
namespace {

constexpr int kThreads = 128;
constexpr int kChunk = 512;  // taps staged per pass

template <int KT>
__global__ void __launch_bounds__(kThreads)
direct_conv_kernel(ConvGeom g, const __half* __restrict__ x, const __half* __restrict__ w,
                   const __half* __restrict__ bias, __half* __restrict__ y, int relu) {
  grid_dependency_wait();
  __shared__ float ws[KT][kChunk];

  // blockIdx.x = (n * ktiles + ktile) * px_tiles + px_tile
  const int ktiles_per_group = (g.kg + KT - 1) / KT;
  const int ktiles = g.group * ktiles_per_group;
  const int64_t pq = (int64_t)g.p * g.q;
  const unsigned px_tiles = (unsigned)((pq + kThreads - 1) / kThreads);
  const unsigned px_tile = blockIdx.x % px_tiles;
  const unsigned nk = blockIdx.x / px_tiles;
  const int ktile = (int)(nk % (unsigned)ktiles);
  const int n = (int)(nk / (unsigned)ktiles);
  const int grp = ktile / ktiles_per_group;
  const int k_in_grp0 = (ktile % ktiles_per_group) * KT;
  const int64_t pix = (int64_t)px_tile * kThreads + threadIdx.x;
  const bool live = pix < pq;
  const int op = live ? (int)(pix / g.q) : 0;
  const int oq = live ? (int)(pix % g.q) : 0;
  const int ih0 = op * g.stride_h - g.pad_h;
  const int iw0 = oq * g.stride_w - g.pad_w;
  const int rs = g.r * g.s;
  const int64_t taps = (int64_t)g.cg * rs;
  const int64_t plane = (int64_t)g.h * g.w;
  const __half* xg = x + ((int64_t)n * g.c + (int64_t)grp * g.cg) * plane;

  float acc[KT];
#pragma unroll
  for (int i = 0; i < KT; ++i) acc[i] = 0.f;

  for (int64_t t0 = 0; t0 < taps; t0 += kChunk) {
    const int len = (int)((taps - t0) < kChunk ? (taps - t0) : kChunk);
    __syncthreads();
    for (int i = threadIdx.x; i < KT * len; i += kThreads) {
      const int kk = i / len, t = i % len;
      const int kin = k_in_grp0 + kk;
      float v = 0.f;
      if (kin < g.kg) v = __half2float(w[((int64_t)grp * g.kg + kin) * taps + t0 + t]);
      ws[kk][t] = v;
    }
    __syncthreads();
    if (live) {
      int cc = (int)(t0 / rs);
      int rem = (int)(t0 % rs);
      int r = rem / g.s, s = rem % g.s;
      for (int t = 0; t < len; ++t) {
        const int ih = ih0 + r * g.dil_h;
        const int iw = iw0 + s * g.dil_w;
        if (ih >= 0 && ih < g.h && iw >= 0 && iw < g.w) {
          float xv = 0.f;
          if (HGC_ADDR_OK(xg + (int64_t)cc * plane + (int64_t)ih * g.w + iw, sizeof(__half)))
            xv = __half2float(__ldg(xg + (int64_t)cc * plane + (int64_t)ih * g.w + iw));
#pragma unroll
          for (int i = 0; i < KT; ++i) acc[i] = fmaf(xv, ws[i][t], acc[i]);
        }
        if (++s == g.s) {
          s = 0;
          if (++r == g.r) {
            r = 0;
            ++cc;
          }
        }
      }
    }
  }

  if (live) {
#pragma unroll
    for (int i = 0; i < KT; ++i) {
      const int kin = k_in_grp0 + i;
      if (kin < g.kg) {
        const int k = grp * g.kg + kin;
        float v = acc[i];
        if (bias != nullptr) v += __half2float(bias[k]);
        if (relu) v = fmaxf(v, 0.f);
        if (HGC_ADDR_OK(y + ((int64_t)n * g.k + k) * pq + pix, sizeof(__half))) y[((int64_t)n * g.k + k) * pq + pix] = __float2half_rn(v);
      }
    }
  }
}

}  // namespace

cudaError_t launch_direct_conv(const ConvGeom& g, const __half* x, const __half* w,
                               const __half* bias, __half* y, int relu, cudaStream_t stream) {
  const int64_t pq = (int64_t)g.p * g.q;
  const int64_t px_tiles = (pq + kThreads - 1) / kThreads;
  const int kt = g.kg >= 4 ? 8 : 1;
  const int64_t ktiles = (int64_t)g.group * ((g.kg + kt - 1) / kt);
  const double total = (double)px_tiles * (double)ktiles * (double)g.n;
  if (total > 2147483647.0) return cudaErrorInvalidConfiguration;
  dim3 grid((unsigned)(px_tiles * ktiles * g.n));
  if (kt == 8)
    launch_kernel(direct_conv_kernel<8>, dim3(grid), dim3(kThreads), 0, stream, g, x, w, bias, y, relu);
  else
    launch_kernel(direct_conv_kernel<1>, dim3(grid), dim3(kThreads), 0, stream, g, x, w, bias, y, relu);
  count_launch();
  return cudaGetLastError();
}

}  // namespace hgc
