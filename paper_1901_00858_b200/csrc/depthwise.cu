// 3x3 depthwise convolution (group == C == K, dilation 1, stride 1 or 2) on CUDA cores.
// It is a 9-tap stencil per channel plane, not a dense contraction: the bound is HBM
// bandwidth (4 bytes per output at stride 1, 10 at stride 2), so the kernel is organised
// around 16-byte aligned global accesses for ANY plane size and works on NCHW directly.
//
// A CTA owns a contiguous piece of the tensor: either several whole (n,c) planes (small
// planes: 7x7, 14x14, 28x28 ...) or a band of output rows of one plane.  Its input span and
// its output span are contiguous in global memory, so both are moved as 16-byte vectors that
// are aligned to the GLOBAL address (the span's first and last vector may be partial; the
// first is over-read inside the tensor, the tail is guarded).  In between, each thread
// slides a 3-row register window down two adjacent output columns, accumulating in fp32, and
// leaves fp16 results in a shared staging span.
#include "hgc_internal.h"

namespace hgc {
HGC_DEBUG_STATE(depthwise)
namespace {

constexpr int kThreads = 256;
constexpr int kInBudget = 16384;   // elements of input a CTA may stage
constexpr int kOutBudget = 12288;  // elements of output a CTA may stage

struct DwPlan {
  int32_t c, h, w, p, q, pad_h, pad_w;
  int32_t th;              // output rows per thread unit
  int32_t planes_per_cta;  // >= 1; > 1 only with bands_per_plane == 1
  int32_t bands_per_plane; // row bands a plane is split into
  int32_t band_rows;       // output rows per band
  int64_t planes;          // N * C
  int64_t x_elems, y_elems;
  int32_t smem_in, smem_out;  // staged elements incl. alignment slack (multiples of 8)
};

template <int S>
__global__ void __launch_bounds__(kThreads)
depthwise3x3_kernel(DwPlan a, const uint16_t* __restrict__ x, const __half* __restrict__ w,
                    const __half* __restrict__ bias, uint16_t* __restrict__ y, int relu) {
  grid_dependency_wait();
  grid_launch_dependents();  // a tensor-core kernel that follows may set itself up beside this one
  extern __shared__ __align__(16) uint16_t smem[];
  uint16_t* sin = smem;
  uint16_t* sout = smem + a.smem_in;
  constexpr int NCOL = S + 3;

  const int64_t hw = (int64_t)a.h * a.w, pq = (int64_t)a.p * a.q;
  int64_t pl0;
  int np, p0, p1;
  if (a.bands_per_plane == 1) {
    pl0 = (int64_t)blockIdx.x * a.planes_per_cta;
    np = (int)((a.planes - pl0) < a.planes_per_cta ? (a.planes - pl0) : a.planes_per_cta);
    p0 = 0;
    p1 = a.p;
  } else {
    pl0 = blockIdx.x / a.bands_per_plane;
    np = 1;
    p0 = (blockIdx.x % a.bands_per_plane) * a.band_rows;
    p1 = p0 + a.band_rows < a.p ? p0 + a.band_rows : a.p;
  }
  // input rows the band touches (whole planes when the CTA owns planes)
  int ih_lo = p0 * S - a.pad_h;
  int ih_hi = (p1 - 1) * S - a.pad_h + 3;
  if (a.bands_per_plane == 1) {
    ih_lo = 0;
    ih_hi = a.h;
  }
  if (ih_lo < 0) ih_lo = 0;
  if (ih_hi > a.h) ih_hi = a.h;
  if (ih_hi < ih_lo) ih_hi = ih_lo;
  const int64_t g_in0 = pl0 * hw + (int64_t)ih_lo * a.w;
  const int64_t in_len = (int64_t)(np - 1) * hw + (int64_t)(ih_hi - ih_lo) * a.w;
  const int mis_in = (int)(g_in0 & 7);
  const int64_t g_out0 = pl0 * pq + (int64_t)p0 * a.q;
  const int64_t out_len = (int64_t)(np - 1) * pq + (int64_t)(p1 - p0) * a.q;
  const int mis_out = (int)(g_out0 & 7);

  // ---- stage the input span: aligned 16-byte vectors --------------------------------
  {
    const int nvec = (int)((mis_in + in_len + 7) >> 3);
    const int64_t gbase = g_in0 - mis_in;
    for (int v = threadIdx.x; v < nvec; v += kThreads) {
      const int64_t ge = gbase + (int64_t)v * 8;
      uint4 val;
      if (ge + 8 <= a.x_elems) {
        HGC_CHECKED_LOAD(val, reinterpret_cast<const uint4*>(x + ge), __ldg(reinterpret_cast<const uint4*>(x + ge)));
      } else {
        uint32_t o[4] = {0, 0, 0, 0};
        for (int j = 0; j < 8; ++j)
          if (ge + j < a.x_elems) o[j >> 1] |= (uint32_t)x[ge + j] << ((j & 1) * 16);
        val = make_uint4(o[0], o[1], o[2], o[3]);
      }
      *reinterpret_cast<uint4*>(sin + v * 8) = val;
    }
  }
  __syncthreads();

  // ---- compute: thread = (unit, column pair) ------------------------------------------
  const int cols2 = (a.q + 1) >> 1;
  const int rows = p1 - p0;
  const int units_per_plane = (rows + a.th - 1) / a.th;
  const int units = np * units_per_plane;
  const int lanes = units * cols2;
  for (int t = threadIdx.x; t < lanes; t += kThreads) {
    const int u = t / cols2, cp = t % cols2;
    const int pl = u / units_per_plane;
    const int r0 = p0 + (u % units_per_plane) * a.th;
    const int r1 = r0 + a.th < p1 ? r0 + a.th : p1;
    const int ch = (int)((pl0 + pl) % a.c);
    // weights and window stay binary16; products and sums use the mixed-precision FMA
    // (f16 x f16 + f32 -> f32), so nothing is converted on the way in
    uint16_t wv[9];
#pragma unroll
    for (int i = 0; i < 9; ++i) wv[i] = __half_as_ushort(__ldg(w + (int64_t)ch * 9 + i));
    const float bv = bias != nullptr ? __half2float(__ldg(bias + ch)) : 0.f;

    const int q0 = cp * 2;
    const int iw0 = q0 * S - a.pad_w;
    bool cvalid[NCOL];
#pragma unroll
    for (int j = 0; j < NCOL; ++j) cvalid[j] = (iw0 + j >= 0) && (iw0 + j < a.w);
    const bool second = (q0 + 1) < a.q;
    // smem index of (plane pl, row ih, col iw0)
    const int in_base = mis_in + pl * (int)hw - ih_lo * a.w + iw0;
    const int out_base = mis_out + pl * (int)pq - p0 * a.q + q0;

    uint16_t win[3][NCOL];
    auto load_row = [&](uint16_t (&dst)[NCOL], int ih) {
      const bool rv = (ih >= 0) && (ih < a.h);
      const uint16_t* src = sin + in_base + ih * a.w;
#pragma unroll
      for (int j = 0; j < NCOL; ++j) {
        uint16_t bits = 0;
        if (rv && cvalid[j]) bits = src[j];
        dst[j] = bits;
      }
    };
    int ih = r0 * S - a.pad_h;
    if (S == 1) {
      load_row(win[0], ih);
      load_row(win[1], ih + 1);
    } else {
      load_row(win[0], ih);
    }
    for (int p = r0; p < r1; ++p, ih += S) {
      if (S == 1) {
        load_row(win[2], ih + 2);
      } else {
        load_row(win[1], ih + 1);
        load_row(win[2], ih + 2);
      }
      float o0 = bv, o1 = bv;
#pragma unroll
      for (int r = 0; r < 3; ++r)
#pragma unroll
        for (int s = 0; s < 3; ++s) {
          asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(o0) : "h"(win[r][s]), "h"(wv[r * 3 + s]));
          asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(o1) : "h"(win[r][s + S]), "h"(wv[r * 3 + s]));
        }
      if (relu) {
        o0 = fmaxf(o0, 0.f);
        o1 = fmaxf(o1, 0.f);
      }
      uint16_t* dst = sout + out_base + p * a.q;
      dst[0] = __half_as_ushort(__float2half_rn(o0));
      if (second) dst[1] = __half_as_ushort(__float2half_rn(o1));
#pragma unroll
      for (int j = 0; j < NCOL; ++j) {
        if (S == 1) {
          win[0][j] = win[1][j];
          win[1][j] = win[2][j];
        } else {
          win[0][j] = win[2][j];
        }
      }
    }
  }
  __syncthreads();

  // ---- write the output span: aligned 16-byte vectors, partial ones element-wise ----
  {
    const int nvec = (int)((mis_out + out_len + 7) >> 3);
    const int64_t gbase = g_out0 - mis_out;
    const int lo = mis_out, hi = mis_out + (int)out_len;  // valid staged range
    for (int v = threadIdx.x; v < nvec; v += kThreads) {
      const int e = v * 8;
      if (e >= lo && e + 8 <= hi) {
        HGC_CHECKED_STORE(reinterpret_cast<uint4*>(y + gbase + e), *reinterpret_cast<uint4*>(y + gbase + e) = *reinterpret_cast<const uint4*>(sout + e));
      } else {
        for (int j = 0; j < 8; ++j)
          if (e + j >= lo && e + j < hi) HGC_CHECKED_STORE(y + gbase + e + j, y[gbase + e + j] = sout[e + j]);
      }
    }
  }
}


// ---- row-vector kernel: planes whose rows are whole 16-byte vectors (W % 8 == 0) -----------------
//
// No shared memory and no block-wide synchronisation: a thread owns one 16-byte vector column (8
// output pixels) of a strip of TH output rows.  It reads each input row it needs as one (stride 1)
// or two (stride 2) aligned 16-byte vectors straight from global memory (consecutive lanes read
// consecutive vectors), fetches the single halo pixel on its left (and right, at stride 1) from
// the neighbouring lanes with warp shuffles, keeps a sliding window of three converted rows in
// registers and writes one aligned 16-byte vector per output row.  Rows shared between strips are
// re-read through L2.
template <int S, int TH>
__global__ void __launch_bounds__(256, 4)
depthwise3x3_rowvec_kernel(const uint16_t* __restrict__ x, const __half* __restrict__ w,
                           const __half* __restrict__ bias, uint16_t* __restrict__ y, int c, int h, int wd,
                           int p, int q, int relu, int64_t total_items, int vec_per_row, int strips) {
  grid_dependency_wait();
  grid_launch_dependents();  // a tensor-core kernel that follows may set itself up beside this one
  // item = (plane, strip, vector); the vectors of a row are consecutive lanes.  32-bit index
  // arithmetic (the launcher checks that the item count fits).
  const uint32_t item = blockIdx.x * blockDim.x + threadIdx.x;
  const bool live = item < (uint32_t)total_items;
  const uint32_t it = live ? item : (uint32_t)total_items - 1u;
  const int v = (int)(it % (uint32_t)vec_per_row);
  const uint32_t t = it / (uint32_t)vec_per_row;
  const int strip = (int)(t % (uint32_t)strips);
  const int64_t plane = (int64_t)(t / (uint32_t)strips);
  const int ch = (int)((uint32_t)(t / (uint32_t)strips) % (uint32_t)c);
  const int lane = threadIdx.x & 31;

  // weights stay binary16: the stencil uses the mixed-precision FMA of sm_100 (f16 x f16 + f32),
  // so no input value is ever converted (the half->float converts run at a quarter of the FMA rate
  // and were the bottleneck of this kernel)
  uint16_t wv[9];
#pragma unroll
  for (int i = 0; i < 9; ++i) wv[i] = __half_as_ushort(__ldg(w + (int64_t)ch * 9 + i));
  const float bv = bias != nullptr ? __half2float(__ldg(bias + ch)) : 0.f;

  const uint16_t* xp = x + plane * (int64_t)h * wd;
  uint16_t* yp = y + plane * (int64_t)p * q;
  const int p_lo = strip * TH;
  // neighbours inside the same row of vectors? (lanes of a warp run over consecutive items)
  const bool has_left = v > 0 && lane > 0;
  const bool has_right = v + 1 < vec_per_row && lane < 31;

  // All input rows of the strip are requested up front (TH*S + 2 rows, one or two 16-byte vectors
  // each): with only a few warps per SM the kernel lives on memory-level parallelism.
  constexpr int NR = TH * S + 2 - (S - 1);  // stride 1: TH + 2 rows; stride 2: 2*TH + 1 rows
  constexpr int NE = 8 * S + 2;             // converted row: elements [-1 .. 8*S] around the 8 outputs
  uint4 ra[NR], rb[S == 2 ? NR : 1];
  uint32_t left[NR], right[NR];
  const int ih0 = p_lo * S - 1;  // pad == 1 (required by the launcher)
#pragma unroll
  for (int i = 0; i < NR; ++i) {
    const int ih = ih0 + i;
    const bool rv = ih >= 0 && ih < h;
    ra[i] = make_uint4(0, 0, 0, 0);
    if (S == 2) rb[i] = make_uint4(0, 0, 0, 0);
    if (rv) {
      const uint4* src = reinterpret_cast<const uint4*>(xp + (int64_t)ih * wd) + (int64_t)v * S;
      HGC_CHECKED_LOAD(ra[i], src, __ldg(src));
      if (S == 2 && (v * 2 + 1) * 8 < wd) HGC_CHECKED_LOAD(rb[i], src + 1, __ldg(src + 1));  // the row may end after the first vector
    }
    // halo pixels that no neighbouring lane holds (warp boundary inside a row)
    left[i] = 0;
    right[i] = 0;
    if (rv && !has_left && v > 0) left[i] = xp[(int64_t)ih * wd + (int64_t)v * 8 * S - 1];
    if (S == 1 && rv && !has_right && v + 1 < vec_per_row) right[i] = xp[(int64_t)ih * wd + (int64_t)(v + 1) * 8];
  }
  // halo from the neighbouring lanes: last element of the left vector(s), first of the right one
#pragma unroll
  for (int i = 0; i < NR; ++i) {
    const uint32_t my_last = (S == 2 ? rb[i].w : ra[i].w) >> 16;
    const uint32_t my_first = ra[i].x & 0xffffu;
    const uint32_t l = __shfl_up_sync(0xffffffffu, my_last, 1);
    const uint32_t r = __shfl_down_sync(0xffffffffu, my_first, 1);
    if (has_left) left[i] = l;
    if (S == 1 && has_right) right[i] = r;
  }

  // one input row as 16-bit lanes: elements [-1 .. 8*S] around the 8 outputs
  auto unpack_row = [&](uint16_t (&dst)[NE], int i) {
    dst[0] = (uint16_t)left[i];
    const uint32_t wa[4] = {ra[i].x, ra[i].y, ra[i].z, ra[i].w};
#pragma unroll
    for (int e = 0; e < 4; ++e)
      asm("mov.b32 {%0, %1}, %2;" : "=h"(dst[1 + 2 * e]), "=h"(dst[2 + 2 * e]) : "r"(wa[e]));
    if (S == 2) {
      const uint32_t wb[4] = {rb[i].x, rb[i].y, rb[i].z, rb[i].w};
#pragma unroll
      for (int e = 0; e < 4; ++e)
        asm("mov.b32 {%0, %1}, %2;" : "=h"(dst[9 + 2 * e]), "=h"(dst[10 + 2 * e]) : "r"(wb[e]));
      dst[NE - 1] = 0;
    } else {
      dst[9] = (uint16_t)right[i];
    }
  };

  uint16_t win[3][NE];
#pragma unroll
  for (int r = 0; r < TH; ++r) {
    const int pr = p_lo + r;
#pragma unroll
    for (int rr = 0; rr < 3; ++rr) unpack_row(win[rr], r * S + rr);  // rows r*S .. r*S+2 of the strip
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float f[2];
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int col = (2 * j + e) * S;  // window index of the tap s = 0
        float acc = bv;
#pragma unroll
        for (int rr = 0; rr < 3; ++rr)
#pragma unroll
          for (int ss = 0; ss < 3; ++ss)
            asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(acc) : "h"(win[rr][col + ss]), "h"(wv[rr * 3 + ss]));
        f[e] = acc;
      }
      // two results -> one packed pair, ReLU folded into the convert
      if (relu)
        asm("cvt.rn.relu.f16x2.f32 %0, %1, %2;" : "=r"(o[j]) : "f"(f[1]), "f"(f[0]));
      else
        asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(o[j]) : "f"(f[1]), "f"(f[0]));
    }
    if (live && pr < p) {
      uint16_t* dst = yp + (int64_t)pr * q + (int64_t)v * 8;
      if ((q & 7) == 0) {
        HGC_CHECKED_STORE(reinterpret_cast<uint4*>(dst), *reinterpret_cast<uint4*>(dst) = make_uint4(o[0], o[1], o[2], o[3]));
      } else {  // q % 8 == 4: rows are 8-byte aligned and the last vector of a row is half full
        reinterpret_cast<uint2*>(dst)[0] = make_uint2(o[0], o[1]);
        if (v * 8 + 8 <= q) reinterpret_cast<uint2*>(dst)[1] = make_uint2(o[2], o[3]);
      }
    }
  }
}

// Small planes (W = 28, 14, 7; pad 1): rows are shorter than a 16-byte vector pattern can use, so
// a thread owns one whole output row of one plane.  It reads its three input rows straight from
// global memory (4-byte words when W is even, else 2-byte elements; consecutive lanes read
// consecutive rows, so a warp's loads cover one contiguous span, and the rows shared with the
// neighbouring lanes come from L1), keeps them in registers with a zero halo on both sides,
// accumulates with the mixed-precision FMA and writes its output row the same way.  No shared
// memory, no synchronisation (staging the span in shared memory first was measured slower).
template <int W, int S>
__global__ void __launch_bounds__(256)
depthwise3x3_smallrow_kernel(const uint16_t* __restrict__ x, const __half* __restrict__ w,
                             const __half* __restrict__ bias, uint16_t* __restrict__ y, int c, int h, int p, int relu,
                             int64_t total_rows) {
  grid_dependency_wait();
  grid_launch_dependents();  // a tensor-core kernel that follows may set itself up beside this one
  constexpr int Q = (W - 1) / S + 1;  // kernel 3, pad 1
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total_rows) return;
  const int64_t plane = idx / p;
  const int pr = (int)(idx - plane * p);
  const int ch = (int)(plane % c);
  uint16_t wv[9];
#pragma unroll
  for (int i = 0; i < 9; ++i) wv[i] = __half_as_ushort(__ldg(w + (int64_t)ch * 9 + i));
  const float bv = bias != nullptr ? __half2float(__ldg(bias + ch)) : 0.f;

  uint16_t in[3][W + 2];  // element e of a row at [e + 1]; [0] and [W + 1] are the zero padding
#pragma unroll
  for (int rr = 0; rr < 3; ++rr) {
    const int ih = pr * S - 1 + rr;
    const bool rv = ih >= 0 && ih < h;
    const uint16_t* xr = x + (plane * h + (rv ? ih : 0)) * W;
    in[rr][0] = 0;
    in[rr][W + 1] = 0;
    if constexpr ((W & 1) == 0) {
#pragma unroll
      for (int e = 0; e < W / 2; ++e) {
        uint32_t v = 0u;
        if (rv) HGC_CHECKED_LOAD(v, reinterpret_cast<const uint32_t*>(xr) + e, __ldg(reinterpret_cast<const uint32_t*>(xr) + e));
        asm("mov.b32 {%0, %1}, %2;" : "=h"(in[rr][1 + 2 * e]), "=h"(in[rr][2 + 2 * e]) : "r"(v));
      }
    } else {
#pragma unroll
      for (int e = 0; e < W; ++e) {
        uint16_t v = 0;
        if (rv) HGC_CHECKED_LOAD(v, xr + e, __ldg(xr + e));
        in[rr][1 + e] = v;
      }
    }
  }
  float f[Q + 1];
#pragma unroll
  for (int j = 0; j < Q; ++j) {
    float acc = bv;
#pragma unroll
    for (int rr = 0; rr < 3; ++rr)
#pragma unroll
      for (int ss = 0; ss < 3; ++ss)
        asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(acc) : "h"(in[rr][j * S + ss]), "h"(wv[rr * 3 + ss]));
    f[j] = acc;
  }
  f[Q] = 0.f;
  uint16_t* yr = y + (plane * p + pr) * Q;
#pragma unroll
  for (int j = 0; j < Q; j += 2) {
    uint32_t o;
    if (relu)
      asm("cvt.rn.relu.f16x2.f32 %0, %1, %2;" : "=r"(o) : "f"(f[j + 1]), "f"(f[j]));
    else
      asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(o) : "f"(f[j + 1]), "f"(f[j]));
    if constexpr ((Q & 1) == 0) {
      reinterpret_cast<uint32_t*>(yr)[j >> 1] = o;
    } else {
      HGC_CHECKED_STORE(yr + j, yr[j] = (uint16_t)(o & 0xffffu));
      if (j + 1 < Q) HGC_CHECKED_STORE(yr + j + 1, yr[j + 1] = (uint16_t)(o >> 16));
    }
  }
}

// Channels-last depthwise 3x3 (x[N][H][W][C], y[N][P][Q][C], C % 8 == 0; any padding, stride 1
// or 2): a thread owns 8 consecutive channels (one 16-byte vector per pixel) and TQ consecutive
// output pixels of one output row.  It issues all its input vectors (3 rows x (TQ-1)*S+3 columns)
// before using the first, keeps its 72 weights in registers, accumulates with the mixed-precision
// FMA and writes one 16-byte vector per output pixel.  Consecutive lanes take consecutive channel
// octets, so a warp's loads and stores are contiguous runs of channels (and of pixels, when a
// pixel has fewer than 32 octets).  Neighbouring threads share input columns through L1.
template <int S, int TQ>
__global__ void __launch_bounds__(256)
depthwise3x3_nhwc_kernel(const uint16_t* __restrict__ x, const uint16_t* __restrict__ w,
                         const uint16_t* __restrict__ bias, uint16_t* __restrict__ y, int c, int h, int wd, int p,
                         int q, int pad_h, int pad_w, int relu, int strips, int64_t items) {
  grid_dependency_wait();
  grid_launch_dependents();  // a tensor-core kernel that follows may set itself up beside this one
  constexpr int COLS = (TQ - 1) * S + 3;
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= items) return;
  const int octets = c >> 3;
  const int oc = (int)(idx % octets);
  int64_t t = idx / octets;
  const int strip = (int)(t % strips);
  t /= strips;
  const int pr = (int)(t % p);
  const int64_t img = t / p;
  const int q0 = strip * TQ;

  // input window: rows pr*S - pad_h .. +2, columns q0*S - pad_w .. + COLS-1; zero outside the image
  uint4 in[3][COLS];
  const int ih0 = pr * S - pad_h, iw0 = q0 * S - pad_w;
#pragma unroll
  for (int rr = 0; rr < 3; ++rr) {
    const int ih = ih0 + rr;
    const bool rv = ih >= 0 && ih < h;
#pragma unroll
    for (int cc = 0; cc < COLS; ++cc) {
      const int iw = iw0 + cc;
      const bool v = rv && iw >= 0 && iw < wd;
      in[rr][cc] = make_uint4(0u, 0u, 0u, 0u);
      if (v) HGC_CHECKED_LOAD(in[rr][cc], reinterpret_cast<const uint4*>(x + ((img * h + ih) * wd + iw) * c) + oc,
                              __ldg(reinterpret_cast<const uint4*>(x + ((img * h + ih) * wd + iw) * c) + oc));
    }
  }
  // weights w[ch][9] of the 8 channels: 144 contiguous bytes, element ch*9 + tap
  uint16_t wv[72];
  {
    const uint4* wp = reinterpret_cast<const uint4*>(w + (int64_t)oc * 72);
#pragma unroll
    for (int i = 0; i < 9; ++i) {
      const uint4 v = __ldg(wp + i);
      const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) asm("mov.b32 {%0, %1}, %2;" : "=h"(wv[8 * i + 2 * j]), "=h"(wv[8 * i + 2 * j + 1]) : "r"(u[j]));
    }
  }
  float bv[8];
  if (bias != nullptr) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(bias) + oc);
    const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      bv[2 * j] = __half2float(__ushort_as_half((uint16_t)(u[j] & 0xffffu)));
      bv[2 * j + 1] = __half2float(__ushort_as_half((uint16_t)(u[j] >> 16)));
    }
  } else {
#pragma unroll
    for (int j = 0; j < 8; ++j) bv[j] = 0.f;
  }
#pragma unroll
  for (int o = 0; o < TQ; ++o) {
    if (q0 + o >= q) break;
    float acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = bv[e];
#pragma unroll
    for (int rr = 0; rr < 3; ++rr)
#pragma unroll
      for (int ss = 0; ss < 3; ++ss) {
        const uint4 v = in[rr][o * S + ss];
        const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          uint16_t lo, hi;
          asm("mov.b32 {%0, %1}, %2;" : "=h"(lo), "=h"(hi) : "r"(u[j]));
          asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(acc[2 * j]) : "h"(lo), "h"(wv[(2 * j) * 9 + rr * 3 + ss]));
          asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(acc[2 * j + 1]) : "h"(hi), "h"(wv[(2 * j + 1) * 9 + rr * 3 + ss]));
        }
      }
    uint32_t ov[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (relu)
        asm("cvt.rn.relu.f16x2.f32 %0, %1, %2;" : "=r"(ov[j]) : "f"(acc[2 * j + 1]), "f"(acc[2 * j]));
      else
        asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(ov[j]) : "f"(acc[2 * j + 1]), "f"(acc[2 * j]));
    }
    HGC_CHECKED_STORE(reinterpret_cast<uint4*>(y + ((img * p + pr) * q + q0 + o) * c) + oc,
                      reinterpret_cast<uint4*>(y + ((img * p + pr) * q + q0 + o) * c)[oc] = make_uint4(ov[0], ov[1], ov[2], ov[3]));
  }
}

// 28x28 and 14x14 planes (pad 1, stride 1 or 2): a lane owns one 4-byte column word (two pixels) of
// one plane and walks down its rows; 32 / (W/2) planes share a warp, so every load and store
// instruction of a warp covers whole contiguous rows (the one-row-per-thread form above reads with
// a stride of one row between lanes, which costs an L1 wavefront per lane or two).  All H words of
// the column are loaded up front; the pixel left of the word and the pixel right of it come from
// the neighbouring lanes by shuffle (zero at the plane's edge).
template <int W, int S>
__global__ void __launch_bounds__(256)
depthwise3x3_colword_kernel(const uint16_t* __restrict__ x, const __half* __restrict__ w,
                            const __half* __restrict__ bias, uint16_t* __restrict__ y, int c, int relu,
                            int64_t planes) {
  grid_dependency_wait();
  grid_launch_dependents();  // a tensor-core kernel that follows may set itself up beside this one
  constexpr int WORDS = W / 2;         // column words per row
  constexpr int PPW = 32 / WORDS;      // planes per warp
  constexpr int H = W;
  const int lane = (int)(threadIdx.x & 31u);
  const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int pl = lane / WORDS, e = lane - pl * WORDS;
  const int64_t plane = warp * PPW + pl;
  const bool live = pl < PPW && plane < planes;
  const int ch = live ? (int)(plane % c) : 0;
  uint16_t wv[9];
#pragma unroll
  for (int i = 0; i < 9; ++i) wv[i] = __half_as_ushort(__ldg(w + (int64_t)ch * 9 + i));
  const float bv = bias != nullptr ? __half2float(__ldg(bias + ch)) : 0.f;
  const uint32_t* xp = reinterpret_cast<const uint32_t*>(x) + (live ? plane : 0) * (H * WORDS) + e;
  uint32_t v[H];
#pragma unroll
  for (int r = 0; r < H; ++r) {
    v[r] = 0u;
    if (live) HGC_CHECKED_LOAD(v[r], xp + r * WORDS, __ldg(xp + r * WORDS));
  }
  // per row: (pixel left of the word, pixel right of it)
  uint32_t lr[H];
#pragma unroll
  for (int r = 0; r < H; ++r) {
    const uint32_t up = __shfl_up_sync(0xffffffffu, v[r], 1);
    const uint32_t dn = __shfl_down_sync(0xffffffffu, v[r], 1);
    const uint32_t left = e > 0 ? (up >> 16) : 0u;
    const uint32_t right = e < WORDS - 1 ? (dn & 0xffffu) : 0u;
    lr[r] = left | (right << 16);
  }
  if constexpr (S == 2) {
    // stride 2: the lane's word holds input columns 2e and 2e+1, so it owns output column e
    // (columns 2e-1, 2e, 2e+1) of output rows p (input rows 2p-1, 2p, 2p+1); 2-byte stores
    constexpr int Q = W / 2;
    uint16_t* yh = y + (live ? plane : 0) * (Q * Q) + e;
#pragma unroll
    for (int p = 0; p < Q; ++p) {
      float a0 = bv;
#pragma unroll
      for (int rr = 0; rr < 3; ++rr) {
        const int r = 2 * p - 1 + rr;
        if (r < 0 || r >= H) continue;
        uint16_t lo, hi, lf, rt;
        asm("mov.b32 {%0, %1}, %2;" : "=h"(lo), "=h"(hi) : "r"(v[r]));
        asm("mov.b32 {%0, %1}, %2;" : "=h"(lf), "=h"(rt) : "r"(lr[r]));
        asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(a0) : "h"(lf), "h"(wv[rr * 3 + 0]));
        asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(a0) : "h"(lo), "h"(wv[rr * 3 + 1]));
        asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(a0) : "h"(hi), "h"(wv[rr * 3 + 2]));
      }
      if (relu) a0 = fmaxf(a0, 0.f);
      if (live) yh[p * Q] = __half_as_ushort(__float2half_rn(a0));
    }
    return;
  }
  uint32_t* yp = reinterpret_cast<uint32_t*>(y) + (live ? plane : 0) * (H * WORDS) + e;
#pragma unroll
  for (int p = 0; p < H; ++p) {
    float a0 = bv, a1 = bv;
#pragma unroll
    for (int rr = 0; rr < 3; ++rr) {
      const int r = p - 1 + rr;
      if (r < 0 || r >= H) continue;
      uint16_t lo, hi, lf, rt;
      asm("mov.b32 {%0, %1}, %2;" : "=h"(lo), "=h"(hi) : "r"(v[r]));
      asm("mov.b32 {%0, %1}, %2;" : "=h"(lf), "=h"(rt) : "r"(lr[r]));
      asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(a0) : "h"(lf), "h"(wv[rr * 3 + 0]));
      asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(a0) : "h"(lo), "h"(wv[rr * 3 + 1]));
      asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(a0) : "h"(hi), "h"(wv[rr * 3 + 2]));
      asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(a1) : "h"(lo), "h"(wv[rr * 3 + 0]));
      asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(a1) : "h"(hi), "h"(wv[rr * 3 + 1]));
      asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(a1) : "h"(rt), "h"(wv[rr * 3 + 2]));
    }
    uint32_t o;
    if (relu)
      asm("cvt.rn.relu.f16x2.f32 %0, %1, %2;" : "=r"(o) : "f"(a1), "f"(a0));
    else
      asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(o) : "f"(a1), "f"(a0));
    if (live) HGC_CHECKED_STORE(yp + p * WORDS, yp[p * WORDS] = o);
  }
}

// shapes the small-row kernel takes
bool smallrow_ok(const ConvGeom& g) {
  if (g.pad_h != 1 || g.pad_w != 1) return false;
  if (g.w != 28 && g.w != 14 && g.w != 7) return false;
  if (g.stride_h != g.stride_w) return false;
  return g.q == (g.w - 1) / g.stride_w + 1;
}

// shapes the row-vector kernel takes: pad 1, W % 8 == 0, whole output vectors per row
bool rowvec_ok(const ConvGeom& g) {
  if (g.pad_h != 1 || g.pad_w != 1) return false;
  if ((g.w & 7) != 0) return false;
  const int S = g.stride_h;
  if (g.q * S != g.w) return false;               // stride 1: Q == W; stride 2: Q == W/2
  if ((g.q & 7) != 0 && (g.q & 7) != 4) return false;  // output rows: whole 16-byte or 8-byte vectors
  return true;
}

bool make_plan(const ConvGeom& g, DwPlan* plan) {
  if (g.r != 3 || g.s != 3 || g.dil_h != 1 || g.dil_w != 1) return false;
  if (g.group != g.c || g.k != g.c) return false;
  if (g.stride_h != g.stride_w || (g.stride_h != 1 && g.stride_h != 2)) return false;
  const int S = g.stride_h;
  DwPlan a{};
  a.c = g.c; a.h = g.h; a.w = g.w; a.p = g.p; a.q = g.q; a.pad_h = g.pad_h; a.pad_w = g.pad_w;
  a.planes = (int64_t)g.n * g.c;
  a.x_elems = a.planes * g.h * g.w;
  a.y_elems = a.planes * g.p * g.q;
  a.th = (g.p % 7 == 0) ? 7 : 8;
  const int64_t hw = (int64_t)g.h * g.w, pq = (int64_t)g.p * g.q;
  const int cols2 = (g.q + 1) / 2;
  if (cols2 > kThreads) return false;
  if (hw <= kInBudget && pq <= kOutBudget) {
    a.bands_per_plane = 1;
    a.band_rows = g.p;
    const int units_per_plane = (g.p + a.th - 1) / a.th;
    int64_t ppc = kThreads / ((int64_t)cols2 * units_per_plane);
    if (ppc < 1) ppc = 1;
    if (ppc > kInBudget / hw) ppc = kInBudget / hw;
    if (ppc > kOutBudget / pq) ppc = kOutBudget / pq;
    if (ppc > a.planes) ppc = a.planes;
    a.planes_per_cta = (int32_t)ppc;
    a.smem_in = (int32_t)(((ppc * hw + 8 + 7) / 8) * 8);
    a.smem_out = (int32_t)(((ppc * pq + 8 + 7) / 8) * 8);
  } else {
    a.planes_per_cta = 1;
    // largest multiple of th whose input rows and output rows fit the budgets
    int tb = 0;
    for (int cand = a.th; cand <= g.p + a.th; cand += a.th) {
      const int64_t in_rows = (int64_t)(cand - 1) * S + 3;
      if (in_rows * g.w > kInBudget || (int64_t)cand * g.q > kOutBudget) break;
      tb = cand;
      if ((int64_t)(cand / a.th) * cols2 >= kThreads) break;  // one pass of the CTA is full
    }
    if (tb == 0) return false;
    a.band_rows = tb;
    a.bands_per_plane = (g.p + tb - 1) / tb;
    const int64_t in_rows = (int64_t)(tb - 1) * S + 3;
    a.smem_in = (int32_t)(((in_rows * g.w + 8 + 7) / 8) * 8);
    a.smem_out = (int32_t)((((int64_t)tb * g.q + 8 + 7) / 8) * 8);
  }
  const int64_t ctas = a.bands_per_plane == 1 ? (a.planes + a.planes_per_cta - 1) / a.planes_per_cta
                                               : a.planes * a.bands_per_plane;
  if (ctas > 0x7fffffffLL) return false;
  // staged indices are 32-bit
  if ((int64_t)a.planes_per_cta * hw > (1 << 24)) return false;
  *plan = a;
  return true;
}

}  // namespace

bool depthwise3x3_nhwc_supported(const ConvGeom& g) {
  if (g.r != 3 || g.s != 3 || g.dil_h != 1 || g.dil_w != 1) return false;
  if (g.group != g.c || g.k != g.c || (g.c & 7) != 0) return false;
  if (g.stride_h != g.stride_w || (g.stride_h != 1 && g.stride_h != 2)) return false;
  const int tq = g.stride_h == 1 ? 4 : 2;
  const int64_t items = (int64_t)g.n * g.p * ((g.q + tq - 1) / tq) * (g.c / 8);
  return (items + 255) / 256 < 0x7fffffffLL;
}

cudaError_t launch_depthwise3x3_nhwc(const ConvGeom& g, const __half* x, const __half* w, const __half* bias,
                                     __half* y, int relu, cudaStream_t stream) {
  if (!depthwise3x3_nhwc_supported(g)) return cudaErrorInvalidConfiguration;
  const int tq = g.stride_h == 1 ? 4 : 2;
  const int strips = (g.q + tq - 1) / tq;
  const int64_t items = (int64_t)g.n * g.p * strips * (g.c / 8);
  const unsigned blocks = (unsigned)((items + 255) / 256);
  const uint16_t* xs = reinterpret_cast<const uint16_t*>(x);
  const uint16_t* ws = reinterpret_cast<const uint16_t*>(w);
  const uint16_t* bs = reinterpret_cast<const uint16_t*>(bias);
  uint16_t* ys = reinterpret_cast<uint16_t*>(y);
  cudaError_t err;
  if (g.stride_h == 1)
    err = launch_kernel(depthwise3x3_nhwc_kernel<1, 4>, dim3(blocks), dim3(256), 0, stream, xs, ws, bs, ys, g.c, g.h, g.w,
                        g.p, g.q, g.pad_h, g.pad_w, relu, strips, items);
  else
    err = launch_kernel(depthwise3x3_nhwc_kernel<2, 2>, dim3(blocks), dim3(256), 0, stream, xs, ws, bs, ys, g.c, g.h, g.w,
                        g.p, g.q, g.pad_h, g.pad_w, relu, strips, items);
  if (err != cudaSuccess) return err;
  count_launch();
  return cudaGetLastError();
}

bool depthwise3x3_supported(const ConvGeom& g) {
  DwPlan a;
  return make_plan(g, &a);
}

cudaError_t launch_depthwise3x3(const ConvGeom& g, const __half* x, const __half* w,
                                const __half* bias, __half* y, int relu, cudaStream_t stream) {
  DwPlan a;
  if (!make_plan(g, &a)) return cudaErrorInvalidConfiguration;
  if (rowvec_ok(g)) {
    const int TH = g.stride_h == 1 ? 4 : 2;  // output rows per thread (bounded by registers: all input rows are prefetched)
    const int vec_per_row = (g.q + 7) / 8;
    const int strips = (g.p + TH - 1) / TH;
    const int64_t items = (int64_t)g.n * g.c * strips * vec_per_row;
    const int64_t blocks = (items + 255) / 256;
    if (items < 0x7fffffffLL) {
      const uint16_t* xs0 = reinterpret_cast<const uint16_t*>(x);
      uint16_t* ys0 = reinterpret_cast<uint16_t*>(y);
      if (g.stride_h == 1)
        launch_kernel(depthwise3x3_rowvec_kernel<1, 4>, dim3((unsigned)blocks), dim3(256), 0, stream, xs0, w, bias, ys0, g.c, g.h, g.w, g.p,
                                                                               g.q, relu, items, vec_per_row, strips);
      else
        launch_kernel(depthwise3x3_rowvec_kernel<2, 2>, dim3((unsigned)blocks), dim3(256), 0, stream, xs0, w, bias, ys0, g.c, g.h, g.w, g.p,
                                                                               g.q, relu, items, vec_per_row, strips);
      count_launch();
      return cudaGetLastError();
    }
  }
  if (smallrow_ok(g) && (g.w == 28 || g.w == 14) && g.h == g.w) {
    const int64_t planes = (int64_t)g.n * g.c;
    const int ppw = g.w == 28 ? 2 : 4;
    const int64_t warps = (planes + ppw - 1) / ppw;
    const int64_t blocks = (warps + 7) / 8;
    if (blocks < 0x7fffffffLL) {
      const uint16_t* xs0 = reinterpret_cast<const uint16_t*>(x);
      uint16_t* ys0 = reinterpret_cast<uint16_t*>(y);
#define HGC_DW_COLWORD(WV, SV)                                                                                   \
  launch_kernel(depthwise3x3_colword_kernel<WV, SV>, dim3((unsigned)blocks), dim3(256), 0, stream, xs0, w, bias, ys0, \
                g.c, relu, planes)
      if (g.w == 28 && g.stride_h == 1) HGC_DW_COLWORD(28, 1);
      else if (g.w == 28) HGC_DW_COLWORD(28, 2);
      else if (g.stride_h == 1) HGC_DW_COLWORD(14, 1);
      else HGC_DW_COLWORD(14, 2);
#undef HGC_DW_COLWORD
      count_launch();
      return cudaGetLastError();
    }
  }
  if (smallrow_ok(g)) {
    const int64_t rows = (int64_t)g.n * g.c * g.p;
    const int64_t blocks = (rows + 255) / 256;
    if (blocks < 0x7fffffffLL) {
      const uint16_t* xs0 = reinterpret_cast<const uint16_t*>(x);
      uint16_t* ys0 = reinterpret_cast<uint16_t*>(y);
      const unsigned gb = (unsigned)blocks;
#define HGC_DW_SMALLROW(WV, SV) \
  launch_kernel(depthwise3x3_smallrow_kernel<WV, SV>, dim3(gb), dim3(256), 0, stream, xs0, w, bias, ys0, g.c, g.h, g.p, relu, rows)
      if (g.w == 28 && g.stride_h == 1) HGC_DW_SMALLROW(28, 1);
      else if (g.w == 28) HGC_DW_SMALLROW(28, 2);
      else if (g.w == 14 && g.stride_h == 1) HGC_DW_SMALLROW(14, 1);
      else if (g.w == 14) HGC_DW_SMALLROW(14, 2);
      else if (g.stride_h == 1) HGC_DW_SMALLROW(7, 1);
      else HGC_DW_SMALLROW(7, 2);
#undef HGC_DW_SMALLROW
      count_launch();
      return cudaGetLastError();
    }
  }
  const int64_t ctas = a.bands_per_plane == 1 ? (a.planes + a.planes_per_cta - 1) / a.planes_per_cta
                                               : a.planes * a.bands_per_plane;
  const size_t smem = (size_t)(a.smem_in + a.smem_out) * sizeof(uint16_t);
  const uint16_t* xs = reinterpret_cast<const uint16_t*>(x);
  uint16_t* ys = reinterpret_cast<uint16_t*>(y);
  cudaError_t err;
  if (g.stride_h == 1) {
    err = cudaFuncSetAttribute(depthwise3x3_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    launch_kernel(depthwise3x3_kernel<1>, dim3((unsigned)ctas), dim3(kThreads), smem, stream, a, xs, w, bias, ys, relu);
  } else {
    err = cudaFuncSetAttribute(depthwise3x3_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    launch_kernel(depthwise3x3_kernel<2>, dim3((unsigned)ctas), dim3(kThreads), smem, stream, a, xs, w, bias, ys, relu);
  }
  count_launch();
  return cudaGetLastError();
}

}  // namespace hgc
