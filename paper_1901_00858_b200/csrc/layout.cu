// Data-movement kernels: NCHW <-> NHWC (channels padded to a multiple of 8 so that a pixel is
// a whole number of 16-byte vectors) and the weight re-layout for the implicit-GEMM path.
// Pure permutations of binary16 bit patterns; bound by HBM bandwidth.
//
// Transposes go through a shared-memory tile of kTileC channels x kTileP pixels.  Global
// accesses are 16-byte vectors wherever the address allows it: always on the NHWC side
// (c_pad % 8 == 0), and on the NCHW side when the plane size is a multiple of 8 elements (so
// every channel row of every tile starts on a 16-byte boundary); other planes (7x7, 14x14,
// 27x27 ...) take 2-byte accesses on the NCHW side.
#include <type_traits>

#include "hgc_internal.h"

namespace hgc {
HGC_DEBUG_STATE(layout)
namespace {

constexpr int kTileC = 64;
constexpr int kTileP = 64;
constexpr int kRow = kTileP + 8;  // shared-memory row pitch in elements (16-byte multiple)
constexpr int kThreads = 256;

// x[n][c][hw] -> x'[n][hw][c_pad]
__global__ void __launch_bounds__(kThreads)
nchw_to_nhwc_kernel(const uint16_t* __restrict__ src, uint16_t* __restrict__ dst, int c, int64_t hw,
                    int c_pad, int vec_ok) {
  grid_dependency_wait();
  grid_launch_dependents();  // a tensor-core kernel that follows may set itself up beside this one
  __shared__ __align__(16) uint16_t tile[kTileC][kRow];
  const int64_t n = blockIdx.z;
  const int c0 = blockIdx.y * kTileC;
  const int64_t p0 = (int64_t)blockIdx.x * kTileP;
  const uint16_t* s = src + n * c * hw;
  uint16_t* d = dst + n * hw * c_pad;

  if (vec_ok) {
    // 64 rows x 8 vectors
    for (int i = threadIdx.x; i < kTileC * (kTileP / 8); i += kThreads) {
      const int row = i / (kTileP / 8), v = i % (kTileP / 8);
      const int ch = c0 + row;
      const int64_t p = p0 + v * 8;
      uint4 val = make_uint4(0, 0, 0, 0);
      if (ch < c && p < hw) {  // hw % 8 == 0
        const uint4* sp = reinterpret_cast<const uint4*>(s + (int64_t)ch * hw + p);
        HGC_CHECKED_LOAD(val, sp, *sp);
      }
      *reinterpret_cast<uint4*>(&tile[row][v * 8]) = val;
    }
  } else {
    for (int i = threadIdx.x; i < kTileC * kTileP; i += kThreads) {
      const int row = i / kTileP, col = i % kTileP;
      const int ch = c0 + row;
      const int64_t p = p0 + col;
      uint16_t e = 0;
      if (ch < c && p < hw) HGC_CHECKED_LOAD(e, s + (int64_t)ch * hw + p, s[(int64_t)ch * hw + p]);
      tile[row][col] = e;
    }
  }
  __syncthreads();
  // 64 pixels x 8 channel-vectors; a warp takes 32 consecutive pixels of one channel-vector
  for (int i = threadIdx.x; i < kTileP * (kTileC / 8); i += kThreads) {
    const int cv = i / kTileP, px = i % kTileP;
    const int ch = c0 + cv * 8;
    const int64_t p = p0 + px;
    if (ch < c_pad && p < hw) {
      uint32_t o[4];
#pragma unroll
      for (int j = 0; j < 4; ++j)
        o[j] = (uint32_t)tile[cv * 8 + 2 * j][px] | ((uint32_t)tile[cv * 8 + 2 * j + 1][px] << 16);
      HGC_CHECKED_STORE(reinterpret_cast<uint4*>(d + p * c_pad + ch),
                        *reinterpret_cast<uint4*>(d + p * c_pad + ch) = make_uint4(o[0], o[1], o[2], o[3]));
    }
  }
}

// x[n][c][hw] -> x'[n][hw][c_pad] for planes of a multiple of PX (8 or 4) pixels, without shared
// memory.  A thread owns 8 channels x PX consecutive pixels: eight 16- or 8-byte loads (one per
// channel), a transpose of the binary16 values in registers (byte permutes), PX 16-byte stores
// (one per pixel).  In a warp, lane % CH picks the 8-channel chunk and lane / CH the pixel
// group, so that a store instruction writes CH*16 contiguous bytes per pixel (whole 32-byte
// sectors) and a load instruction reads (32/CH)*PX*2 contiguous bytes per channel.  A warp's
// unit of work is CH*8 channels x (32/CH)*PX pixels of one image.
template <int CH, int PX>
__global__ void __launch_bounds__(kThreads)
nchw_to_nhwc_regs_kernel(const uint16_t* __restrict__ src, uint16_t* __restrict__ dst, int c, int64_t hw,
                         int c_pad, int64_t units_p, int units_c, int64_t total_units) {
  grid_dependency_wait();
  grid_launch_dependents();  // a tensor-core kernel that follows may set itself up beside this one
  constexpr int PG = 32 / CH;
  constexpr int W32 = PX / 2;  // 32-bit words per channel
  const int lane = threadIdx.x & 31;
  const int c8 = lane % CH, pg = lane / CH;
  const int64_t warp0 = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * kThreads) >> 5;
  for (int64_t u = warp0; u < total_units; u += nwarps) {
    // pixel blocks innermost: neighbouring warps read neighbouring pieces of the same channel rows
    const int64_t up = u % units_p;
    const int64_t t = u / units_p;
    const int uc = (int)(t % units_c);
    const int64_t n = t / units_c;
    const int ch = (uc * CH + c8) * 8;
    const int64_t p = (up * PG + pg) * PX;
    if (ch >= c_pad || p >= hw) continue;
    const uint16_t* s = src + (n * c + ch) * hw + p;
    uint32_t v[8][W32];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      if (ch + i < c) {
        if constexpr (PX == 8) {
          uint4 q;
          HGC_CHECKED_LOAD(q, reinterpret_cast<const uint4*>(s + (int64_t)i * hw), __ldcs(reinterpret_cast<const uint4*>(s + (int64_t)i * hw)));
          v[i][0] = q.x; v[i][1] = q.y; v[i][2] = q.z; v[i][3] = q.w;
        } else {
          uint2 q;
          HGC_CHECKED_LOAD(q, reinterpret_cast<const uint2*>(s + (int64_t)i * hw), __ldcs(reinterpret_cast<const uint2*>(s + (int64_t)i * hw)));
          v[i][0] = q.x; v[i][1] = q.y;
        }
      } else {
#pragma unroll
        for (int w = 0; w < W32; ++w) v[i][w] = 0u;
      }
    }
    uint16_t* d = dst + (n * hw + p) * c_pad + ch;
#pragma unroll
    for (int q = 0; q < PX; ++q) {
      const uint32_t sel = (q & 1) ? 0x7632u : 0x5410u;
      uint32_t o[4];
#pragma unroll
      for (int m = 0; m < 4; ++m) o[m] = __byte_perm(v[2 * m][q >> 1], v[2 * m + 1][q >> 1], sel);
      HGC_CHECKED_STORE(reinterpret_cast<uint4*>(d + (int64_t)q * c_pad),
                        *reinterpret_cast<uint4*>(d + (int64_t)q * c_pad) = make_uint4(o[0], o[1], o[2], o[3]));
    }
  }
}

// x[n][c][hw] -> x'[n][hw][c_pad] for SMALL planes whose size is not a multiple of 8 (7x7, 14x14,
// 13x13 ...): the rows of such planes are not 16-byte aligned, but 64 consecutive channel planes
// of one image are one contiguous, 16-byte aligned span (when C*hw % 8 == 0).  A CTA copies that
// span into shared memory with 16-byte vectors and writes whole-pixel 16-byte vectors out.
__global__ void __launch_bounds__(kThreads)
nchw_to_nhwc_smallplane_kernel(const uint16_t* __restrict__ src, uint16_t* __restrict__ dst, int c, int hw,
                               int c_pad) {
  grid_dependency_wait();
  grid_launch_dependents();  // a tensor-core kernel that follows may set itself up beside this one
  extern __shared__ __align__(16) uint16_t flat[];  // [kTileC][hw]
  const int64_t n = blockIdx.y;
  const int c0 = blockIdx.x * kTileC;
  const int nch = c - c0 < kTileC ? c - c0 : kTileC;   // real channels in this tile (may be <= 0)
  const int span = nch > 0 ? nch * hw : 0;             // elements to copy
  const uint16_t* s = src + (n * c + c0) * (int64_t)hw;
  const int nvec = span >> 3;
  for (int v = threadIdx.x; v < nvec; v += kThreads)
  {
      uint4 q;
      HGC_CHECKED_LOAD(q, reinterpret_cast<const uint4*>(s) + v, __ldg(reinterpret_cast<const uint4*>(s) + v));
      reinterpret_cast<uint4*>(flat)[v] = q;
    }
  for (int e = (nvec << 3) + threadIdx.x; e < span; e += kThreads) {
    uint16_t q;
    HGC_CHECKED_LOAD(q, s + e, s[e]);
    flat[e] = q;
  }
  __syncthreads();
  uint16_t* d = dst + n * (int64_t)hw * c_pad;
  const int cvecs = (c_pad - c0 < kTileC ? c_pad - c0 : kTileC) >> 3;  // 16-byte vectors per pixel in this tile
  for (int i = threadIdx.x; i < hw * cvecs; i += kThreads) {
    const int cv = i % cvecs, px = i / cvecs;
    uint32_t o[4] = {0, 0, 0, 0};
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int ch = cv * 8 + j;
      if (ch < nch) o[j >> 1] |= (uint32_t)flat[ch * hw + px] << ((j & 1) * 16);
    }
    HGC_CHECKED_STORE(reinterpret_cast<uint4*>(d + (int64_t)px * c_pad + c0 + cv * 8),
                      *reinterpret_cast<uint4*>(d + (int64_t)px * c_pad + c0 + cv * 8) = make_uint4(o[0], o[1], o[2], o[3]));
  }
}

// x'[n][hw][c_pad] -> x[n][c][hw]
__global__ void __launch_bounds__(kThreads)
nhwc_to_nchw_kernel(const uint16_t* __restrict__ src, uint16_t* __restrict__ dst, int c, int64_t hw,
                    int c_pad, int vec_ok) {
  grid_dependency_wait();
  grid_launch_dependents();  // a tensor-core kernel that follows may set itself up beside this one
  __shared__ __align__(16) uint16_t tile[kTileC][kRow];
  const int64_t n = blockIdx.z;
  const int c0 = blockIdx.y * kTileC;
  const int64_t p0 = (int64_t)blockIdx.x * kTileP;
  const uint16_t* s = src + n * hw * c_pad;
  uint16_t* d = dst + n * c * hw;

  for (int i = threadIdx.x; i < kTileP * (kTileC / 8); i += kThreads) {
    const int px = i / (kTileC / 8), cv = i % (kTileC / 8);
    const int ch = c0 + cv * 8;
    const int64_t p = p0 + px;
    uint4 val = make_uint4(0, 0, 0, 0);
    if (ch < c_pad && p < hw) val = *reinterpret_cast<const uint4*>(s + p * c_pad + ch);
    const uint32_t o[4] = {val.x, val.y, val.z, val.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      tile[cv * 8 + 2 * j][px] = (uint16_t)(o[j] & 0xffffu);
      tile[cv * 8 + 2 * j + 1][px] = (uint16_t)(o[j] >> 16);
    }
  }
  __syncthreads();
  if (vec_ok) {
    for (int i = threadIdx.x; i < kTileC * (kTileP / 8); i += kThreads) {
      const int row = i / (kTileP / 8), v = i % (kTileP / 8);
      const int ch = c0 + row;
      const int64_t p = p0 + v * 8;
      if (ch < c && p < hw)
        HGC_CHECKED_STORE(reinterpret_cast<uint4*>(d + (int64_t)ch * hw + p),
                          *reinterpret_cast<uint4*>(d + (int64_t)ch * hw + p) = *reinterpret_cast<const uint4*>(&tile[row][v * 8]));
    }
  } else {
    for (int i = threadIdx.x; i < kTileC * kTileP; i += kThreads) {
      const int row = i / kTileP, col = i % kTileP;
      const int ch = c0 + row;
      const int64_t p = p0 + col;
      if (ch < c && p < hw) HGC_CHECKED_STORE(d + (int64_t)ch * hw + p, d[(int64_t)ch * hw + p] = tile[row][col]);
    }
  }
}

// Output channel held by row `row` of the re-laid-out weights.  Normally the row itself; with
// `perm` (layers that write y channels-last through the staged epilogue) the rows of every block
// of 32 are interleaved, row 4*b + a holding channel 8*a + b of the block: the accumulator lanes
// of an epilogue warp then hold the channels in the order in which a transposing matrix store
// writes eight consecutive channels of one pixel as one 16-byte row.
__device__ __forceinline__ int64_t row_channel(int64_t row, int perm) {
  if (!perm) return row;
  const int64_t in = row & 31;
  return (row & ~(int64_t)31) + 8 * (in & 3) + (in >> 2);
}

// w[g*kg + k'][c'][r][s] -> w'[g][k'][r][s][c_pad]; one thread per 8 output channels-of-input
__global__ void weights_repack_kernel(const uint16_t* __restrict__ src, uint16_t* __restrict__ dst,
                                      int64_t k, int cg, int rs, int c_pad, int perm) {
  grid_dependency_wait();
  grid_launch_dependents();  // a tensor-core kernel that follows may set itself up beside this one
  const int64_t vecs_per_k = (int64_t)rs * (c_pad / 8);
  const int64_t total = k * vecs_per_k;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total;
       i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t kk = i / vecs_per_k;
    const int64_t rem = i % vecs_per_k;
    const int t = (int)(rem / (c_pad / 8));
    const int cv = (int)(rem % (c_pad / 8));
    uint32_t o[4] = {0, 0, 0, 0};
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int ch = cv * 8 + j;
      uint32_t v = 0;
      if (ch < cg) {
        uint16_t e;
        HGC_CHECKED_LOAD(e, src + (row_channel(kk, perm) * cg + ch) * rs + t, src[(row_channel(kk, perm) * cg + ch) * rs + t]);
        v = e;
      }
      o[j >> 1] |= v << ((j & 1) * 16);
    }
    HGC_CHECKED_STORE(reinterpret_cast<uint4*>(dst + (kk * rs + t) * c_pad + cv * 8),
                      *reinterpret_cast<uint4*>(dst + (kk * rs + t) * c_pad + cv * 8) = make_uint4(o[0], o[1], o[2], o[3]));
  }
}

// x[n][c][h][w] (c <= 8) -> x'[n][hp][wp][8]: pixel (h, w) lands at (h + pad_h, w + pad_w); the
// border, the extra columns and channels c..7 are zero.  One thread per output pixel (16 bytes).
template <int PC>  // channels per pixel of the copy: 8 (16 bytes) or 4 (8 bytes)
__global__ void __launch_bounds__(256)
nchw_to_nhwc8_bordered_kernel(const uint16_t* __restrict__ src, uint16_t* __restrict__ dst, int c, int h, int w,
                              int pad_h, int pad_w, int hp, int wp, int64_t total) {
  grid_dependency_wait();
  grid_launch_dependents();  // a tensor-core kernel that follows may set itself up beside this one
  const int64_t hw = (int64_t)h * w;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int ow = (int)(i % wp);
    const int64_t t = i / wp;
    const int oh = (int)(t % hp);
    const int64_t n = t / hp;
    const int ih = oh - pad_h, iw = ow - pad_w;
    uint32_t o[4] = {0, 0, 0, 0};
    if (ih >= 0 && ih < h && iw >= 0 && iw < w) {
      const uint16_t* s = src + n * c * hw + (int64_t)ih * w + iw;
#pragma unroll
      for (int ch = 0; ch < PC; ++ch)
        if (ch < c) o[ch >> 1] |= (uint32_t)s[ch * hw] << ((ch & 1) * 16);
    }
    if (PC == 8) HGC_CHECKED_STORE(reinterpret_cast<uint4*>(dst + i * 8), *reinterpret_cast<uint4*>(dst + i * 8) = make_uint4(o[0], o[1], o[2], o[3]));
    else HGC_CHECKED_STORE(reinterpret_cast<uint2*>(dst + i * 4), *reinterpret_cast<uint2*>(dst + i * 4) = make_uint2(o[0], o[1]));
  }
}

// The same copy for rows that are whole 16-byte vectors (w % 8 == 0): a thread takes 8 consecutive
// pixels of one input row, one 16-byte load per channel, and transposes them in registers.  The 8
// pixels (PC * 2 bytes each, contiguous in x') go through shared memory, so that the lanes of a
// warp then write consecutive vectors: 8 lanes per slot, whole 128-byte (64-byte) runs per slot
// instead of 32 scattered 16-byte pieces per store instruction (VGG conv1_1 38.9 -> 36.8 us per layer,
// ResNet-50 stem 87.9 -> 80.0).  The last slot of every output row writes the zero columns left and right of the
// image itself; slots of rows above and below the image write zeros like any other.
template <int PC>
__global__ void __launch_bounds__(256)
nchw_to_nhwc8_bordered_vec_kernel(const uint16_t* __restrict__ src, uint16_t* __restrict__ dst, int c, int h, int w,
                                  int pad_h, int pad_w, int hp, int wp, int64_t items) {
  using Vec = typename std::conditional<PC == 8, uint4, uint2>::type;  // one pixel of x'
  __shared__ Vec stage[256 * 8];
  __shared__ uint16_t* slot_dst[256];
  grid_dependency_wait();
  grid_launch_dependents();  // a tensor-core kernel that follows may set itself up beside this one
  const int slots = w / 8 + 1;
  const int tid = threadIdx.x;
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + tid;
  uint16_t* my_dst = nullptr;
  if (i < items) {
    const int slot = (int)(i % slots);
    const int64_t t = i / slots;
    const int oh = (int)(t % hp);
    const int64_t n = t / hp;
    uint16_t* drow = dst + (n * hp + oh) * (int64_t)wp * PC;
    if (slot == slots - 1) {  // the zero columns of this row
      const Vec zero{};
      for (int ow = 0; ow < pad_w; ++ow) HGC_CHECKED_STORE(reinterpret_cast<Vec*>(drow) + ow, reinterpret_cast<Vec*>(drow)[ow] = zero);
      for (int ow = pad_w + w; ow < wp; ++ow) HGC_CHECKED_STORE(reinterpret_cast<Vec*>(drow) + ow, reinterpret_cast<Vec*>(drow)[ow] = zero);
    } else {
      const int ih = oh - pad_h;
      my_dst = drow + (int64_t)(pad_w + slot * 8) * PC;
      uint4 v[PC];
#pragma unroll
      for (int ch = 0; ch < PC; ++ch) {
        v[ch] = make_uint4(0u, 0u, 0u, 0u);
        if (ch < c && ih >= 0 && ih < h) {
          const uint4* sp = reinterpret_cast<const uint4*>(src + ((n * c + ch) * h + ih) * (int64_t)w) + slot;
          HGC_CHECKED_LOAD(v[ch], sp, __ldcs(sp));
        }
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        uint32_t o[4] = {0u, 0u, 0u, 0u};
#pragma unroll
        for (int k = 0; k < PC / 2; ++k) {
          const uint4 a4 = v[2 * k], b4 = v[2 * k + 1];
          const uint32_t a = (j >> 1) == 0 ? a4.x : ((j >> 1) == 1 ? a4.y : ((j >> 1) == 2 ? a4.z : a4.w));
          const uint32_t b = (j >> 1) == 0 ? b4.x : ((j >> 1) == 1 ? b4.y : ((j >> 1) == 2 ? b4.z : b4.w));
          o[k] = __byte_perm(a, b, (j & 1) ? 0x7632 : 0x5410);
        }
        // (pieces of a slot rotated by the slot number: the transposed reads below hit all banks)
        Vec px;
        if constexpr (PC == 8) px = make_uint4(o[0], o[1], o[2], o[3]);
        else px = make_uint2(o[0], o[1]);
        stage[tid * 8 + (j ^ (tid & 7))] = px;
      }
    }
  }
  slot_dst[tid] = my_dst;
  __syncthreads();
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const int v = tid + 256 * k;
    const int sl = v >> 3, piece = v & 7;
    uint16_t* d = slot_dst[sl];
    if (d != nullptr)
      HGC_CHECKED_STORE(reinterpret_cast<Vec*>(d) + piece, reinterpret_cast<Vec*>(d)[piece] = stage[sl * 8 + (piece ^ (sl & 7))]);
  }
}

// w[k][c][r][s] (c <= 8) -> w'[k][r][kw_pix][8]: tap s, channel ch at [s][ch]; zeros elsewhere.
template <int PC>  // channels per pixel of the window: 8 or 4
__global__ void weights_repack_window_kernel(const uint16_t* __restrict__ src, uint16_t* __restrict__ dst,
                                             int64_t k, int c, int r, int s, int kw_pix, int perm) {
  grid_dependency_wait();
  grid_launch_dependents();  // a tensor-core kernel that follows may set itself up beside this one
  const int64_t total = k * r * kw_pix;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int sp = (int)(i % kw_pix);
    const int64_t t = i / kw_pix;
    const int rr = (int)(t % r);
    const int64_t kk = t / r;
    uint32_t o[4] = {0, 0, 0, 0};
    if (sp < s) {
#pragma unroll
      for (int ch = 0; ch < PC; ++ch)
        if (ch < c)
          o[ch >> 1] |= (uint32_t)src[((row_channel(kk, perm) * c + ch) * r + rr) * s + sp] << ((ch & 1) * 16);
    }
    if (PC == 8) HGC_CHECKED_STORE(reinterpret_cast<uint4*>(dst + i * 8), *reinterpret_cast<uint4*>(dst + i * 8) = make_uint4(o[0], o[1], o[2], o[3]));
    else HGC_CHECKED_STORE(reinterpret_cast<uint2*>(dst + i * 4), *reinterpret_cast<uint2*>(dst + i * 4) = make_uint2(o[0], o[1]));
  }
}

// Patch mode (layers whose whole receptive field R*S*C is at most 64 elements: image stems).
// x[n][c][h][w] -> x''[n][p][q][kelems]: for every OUTPUT pixel the R*S*C input values under the
// kernel, element (r*S + s)*C + ch, zero where the tap falls into the padding and from R*S*C up
// to kelems.  The convolution then is a 1x1 convolution over x'' with kelems channels.
// One thread per output pixel; the specialised form has every index known at compile time.
template <int R, int S, int C>
__global__ void __launch_bounds__(256)
patch_im2col_kernel(const uint16_t* __restrict__ src, uint16_t* __restrict__ dst, int h, int w, int p, int q,
                    int pad_h, int pad_w, int stride_h, int stride_w, int dil_h, int dil_w, int kelems,
                    int64_t total) {
  grid_dependency_wait();
  grid_launch_dependents();  // a tensor-core kernel that follows may set itself up beside this one
  constexpr int E = R * S * C;
  constexpr int EW = (E + 1) / 2;  // 32-bit words that hold real elements
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  const int oq = (int)(i % q);
  const int64_t t = i / q;
  const int op = (int)(t % p);
  const int64_t n = t / p;
  const int64_t hw = (int64_t)h * w;
  const uint16_t* xn = src + n * C * hw;
  uint32_t o[EW];
#pragma unroll
  for (int e = 0; e < EW; ++e) o[e] = 0u;
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const int ih = op * stride_h - pad_h + r * dil_h;
#pragma unroll
    for (int sx = 0; sx < S; ++sx) {
      const int iw = oq * stride_w - pad_w + sx * dil_w;
      const bool ok = ih >= 0 && ih < h && iw >= 0 && iw < w;
#pragma unroll
      for (int ch = 0; ch < C; ++ch) {
        const int e = (r * S + sx) * C + ch;
        const uint32_t v = ok ? (uint32_t)__ldg(xn + ch * hw + (int64_t)ih * w + iw) : 0u;
        o[e >> 1] |= v << ((e & 1) * 16);
      }
    }
  }
  uint4* d = reinterpret_cast<uint4*>(dst + i * kelems);
  const int vecs = kelems >> 3;
#pragma unroll
  for (int v = 0; v < 8; ++v) {
    if (v < vecs) {
      uint32_t a[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) a[j] = (4 * v + j) < EW ? o[(4 * v + j) < EW ? 4 * v + j : 0] : 0u;
      HGC_CHECKED_STORE(d + v, d[v] = make_uint4(a[0], a[1], a[2], a[3]));
    }
  }
}

// The same for 3x3 kernels with stride 2 and padding 1 along W on rows of an even number of pixels
// (the stems of MobileNet-like networks): output pixel oq reads input pixels 2oq-1, 2oq, 2oq+1 of
// three rows.  A warp owns 32 consecutive output pixels of ONE output row; a lane loads the aligned
// 4-byte word (2oq, 2oq+1) per row and channel and takes pixel 2oq-1 from its left neighbour's word
// by shuffle: 9 loads per thread instead of 27 two-byte ones (the MobileNet stem, 32x3x224x224: 36.5 -> 33.8 us with its tensor-core kernel).
template <int C>
__global__ void __launch_bounds__(256)
patch_im2col_s2_kernel(const uint16_t* __restrict__ src, uint16_t* __restrict__ dst, int h, int w, int p, int q,
                       int pad_h, int stride_h, int kelems, int warps_per_row, int64_t total_warps) {
  grid_dependency_wait();
  grid_launch_dependents();  // a tensor-core kernel that follows may set itself up beside this one
  constexpr int E = 9 * C;
  constexpr int EW = (E + 1) / 2;
  const int lane = threadIdx.x & 31;
  const int64_t gw = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (gw >= total_warps) return;
  const int wr = (int)(gw % warps_per_row);
  const int64_t row = gw / warps_per_row;  // (image, output row)
  const int op = (int)(row % p);
  const int64_t n = row / p;
  const int oq = wr * 32 + lane;
  const bool live = oq < q;
  const int64_t hw = (int64_t)h * w;
  const uint16_t* xn = src + n * C * hw;
  uint32_t o[EW];
#pragma unroll
  for (int e = 0; e < EW; ++e) o[e] = 0u;
#pragma unroll
  for (int r = 0; r < 3; ++r) {
    const int ih = op * stride_h - pad_h + r;
    const bool rv = ih >= 0 && ih < h;  // (the same for the whole warp)
#pragma unroll
    for (int ch = 0; ch < C; ++ch) {
      const uint16_t* xr = xn + ch * hw + (int64_t)ih * w;
      uint32_t word = 0u;
      if (rv && live) HGC_CHECKED_LOAD(word, reinterpret_cast<const uint32_t*>(xr + 2 * oq), __ldg(reinterpret_cast<const uint32_t*>(xr + 2 * oq)));
      uint32_t left = __shfl_up_sync(0xffffffffu, word, 1) >> 16;
      if (lane == 0) {
        left = 0u;
        if (rv && live && oq > 0) {
          uint16_t e;
          HGC_CHECKED_LOAD(e, xr + 2 * oq - 1, __ldg(xr + 2 * oq - 1));
          left = e;
        }
      }
      const uint32_t px[3] = {left, word & 0xffffu, word >> 16};
#pragma unroll
      for (int sx = 0; sx < 3; ++sx) {
        const int e = (r * 3 + sx) * C + ch;
        o[e >> 1] |= px[sx] << ((e & 1) * 16);
      }
    }
  }
  if (!live) return;
  uint4* d = reinterpret_cast<uint4*>(dst + ((row * q) + oq) * kelems);
  const int vecs = kelems >> 3;
#pragma unroll
  for (int v = 0; v < 8; ++v) {
    if (v < vecs) {
      uint32_t a[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) a[j] = (4 * v + j) < EW ? o[(4 * v + j) < EW ? 4 * v + j : 0] : 0u;
      HGC_CHECKED_STORE(d + v, d[v] = make_uint4(a[0], a[1], a[2], a[3]));
    }
  }
}

// any R, S, C with R*S*C <= 64: one thread per 8-element chunk of an output pixel's patch
__global__ void __launch_bounds__(256)
patch_im2col_generic_kernel(const uint16_t* __restrict__ src, uint16_t* __restrict__ dst, int c, int h, int w,
                            int p, int q, int r, int s, int pad_h, int pad_w, int stride_h, int stride_w,
                            int dil_h, int dil_w, int kelems, int64_t total_chunks) {
  grid_dependency_wait();
  grid_launch_dependents();  // a tensor-core kernel that follows may set itself up beside this one
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total_chunks) return;
  const int vecs = kelems >> 3;
  const int v = (int)(i % vecs);
  const int64_t pix = i / vecs;
  const int oq = (int)(pix % q);
  const int64_t t = pix / q;
  const int op = (int)(t % p);
  const int64_t n = t / p;
  const int64_t hw = (int64_t)h * w;
  const uint16_t* xn = src + n * c * hw;
  const int rsc = r * s * c;
  uint32_t o[4] = {0, 0, 0, 0};
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int e = v * 8 + j;
    if (e < rsc) {
      const int ch = e % c;
      const int tap = e / c;
      const int sx = tap % s, rr = tap / s;
      const int ih = op * stride_h - pad_h + rr * dil_h;
      const int iw = oq * stride_w - pad_w + sx * dil_w;
      if (ih >= 0 && ih < h && iw >= 0 && iw < w)
        o[j >> 1] |= (uint32_t)__ldg(xn + ch * hw + (int64_t)ih * w + iw) << ((j & 1) * 16);
    }
  }
  HGC_CHECKED_STORE(reinterpret_cast<uint4*>(dst + i * 8), *reinterpret_cast<uint4*>(dst + i * 8) = make_uint4(o[0], o[1], o[2], o[3]));
}

// w[k][c][r][s] -> w'[k][kelems], element (r*S + s)*C + ch; zeros from R*S*C on
__global__ void weights_repack_patch_kernel(const uint16_t* __restrict__ src, uint16_t* __restrict__ dst, int64_t k,
                                            int c, int r, int s, int kelems, int perm) {
  grid_dependency_wait();
  grid_launch_dependents();  // a tensor-core kernel that follows may set itself up beside this one
  const int64_t total = k * kelems;
  const int rsc = r * s * c;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int e = (int)(i % kelems);
    const int64_t kk = i / kelems;
    uint16_t v = 0;
    if (e < rsc) {
      const int ch = e % c;
      const int tap = e / c;
      v = src[(row_channel(kk, perm) * c + ch) * (r * s) + tap];
    }
    HGC_CHECKED_STORE(dst + i, dst[i] = v);
  }
}

}  // namespace

cudaError_t launch_nchw_to_nhwc8_bordered(const __half* src, __half* dst, int32_t n, int32_t c, int32_t h, int32_t w,
                                          int32_t pad_h, int32_t pad_w, int32_t hp, int32_t wp, cudaStream_t stream,
                                          int px_ch) {
  const int64_t total = (int64_t)n * hp * wp;
  if ((w % 8) == 0) {
    const int64_t items = (int64_t)n * hp * (w / 8 + 1);
    const int64_t vblocks = (items + 255) / 256;
    if (vblocks <= 0x7fffffffLL) {
      const uint16_t* s16 = reinterpret_cast<const uint16_t*>(src);
      uint16_t* d16 = reinterpret_cast<uint16_t*>(dst);
      if (px_ch == 4)
        launch_kernel(nchw_to_nhwc8_bordered_vec_kernel<4>, dim3((unsigned)vblocks), dim3(256), 0, stream, s16, d16, c,
                      h, w, pad_h, pad_w, hp, wp, items);
      else
        launch_kernel(nchw_to_nhwc8_bordered_vec_kernel<8>, dim3((unsigned)vblocks), dim3(256), 0, stream, s16, d16, c,
                      h, w, pad_h, pad_w, hp, wp, items);
      count_launch();
      return cudaGetLastError();
    }
  }
  int64_t blocks = (total + 255) / 256;
  if (blocks > 148 * 32) blocks = 148 * 32;
  if (px_ch == 4)
    launch_kernel(nchw_to_nhwc8_bordered_kernel<4>, dim3((unsigned)blocks), dim3(256), 0, stream,
        reinterpret_cast<const uint16_t*>(src), reinterpret_cast<uint16_t*>(dst), c, h, w, pad_h, pad_w, hp, wp, total);
  else
  launch_kernel(nchw_to_nhwc8_bordered_kernel<8>, dim3((unsigned)blocks), dim3(256), 0, stream, 
      reinterpret_cast<const uint16_t*>(src), reinterpret_cast<uint16_t*>(dst), c, h, w, pad_h, pad_w, hp, wp, total);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_weights_repack_window(const __half* src, __half* dst, int32_t k, int32_t c, int32_t r, int32_t s,
                                         int32_t kw_pix, cudaStream_t stream, int perm, int px_ch) {
  const int64_t total = (int64_t)k * r * kw_pix;
  int64_t blocks = (total + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (px_ch == 4)
    launch_kernel(weights_repack_window_kernel<4>, dim3((unsigned)blocks), dim3(256), 0, stream,
        reinterpret_cast<const uint16_t*>(src), reinterpret_cast<uint16_t*>(dst), k, c, r, s, kw_pix, perm);
  else
  launch_kernel(weights_repack_window_kernel<8>, dim3((unsigned)blocks), dim3(256), 0, stream, 
      reinterpret_cast<const uint16_t*>(src), reinterpret_cast<uint16_t*>(dst), k, c, r, s, kw_pix, perm);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_nchw_to_nhwc(const __half* src, __half* dst, int32_t n, int32_t c, int32_t h,
                                int32_t w, int32_t c_pad, cudaStream_t stream) {
  const int64_t hw = (int64_t)h * w;
  const int64_t px_tiles = (hw + kTileP - 1) / kTileP;
  const int c_tiles = (c_pad + kTileC - 1) / kTileC;
  if (px_tiles > 0x7fffffffLL || c_tiles > 65535 || n > 65535) return cudaErrorInvalidConfiguration;
  if ((hw % 4) == 0) {
    // planes of a multiple of 8 (or 4) pixels: every channel row starts on a 16- (8-) byte
    // boundary: register transpose, 8 or 4 channel chunks per pixel per warp
    const int px = (hw % 8) == 0 ? 8 : 4;
    const int ch_per = c_pad >= 64 ? 8 : 4;
    const int64_t units_p = (hw / px + (32 / ch_per) - 1) / (32 / ch_per);
    const int units_c = (c_pad / 8 + ch_per - 1) / ch_per;
    const int64_t total_units = units_p * units_c * n;
    int64_t blocks = (total_units + (kThreads / 32) - 1) / (kThreads / 32);
    const int64_t cap = (int64_t)sm_count() * 8 * 4;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    const uint16_t* s16 = reinterpret_cast<const uint16_t*>(src);
    uint16_t* d16 = reinterpret_cast<uint16_t*>(dst);
    const unsigned gb = (unsigned)blocks;
    if (px == 8 && ch_per == 8)
      launch_kernel(nchw_to_nhwc_regs_kernel<8, 8>, dim3(gb), dim3(kThreads), 0, stream, s16, d16, c, hw, c_pad, units_p, units_c, total_units);
    else if (px == 8)
      launch_kernel(nchw_to_nhwc_regs_kernel<4, 8>, dim3(gb), dim3(kThreads), 0, stream, s16, d16, c, hw, c_pad, units_p, units_c, total_units);
    else if (ch_per == 8)
      launch_kernel(nchw_to_nhwc_regs_kernel<8, 4>, dim3(gb), dim3(kThreads), 0, stream, s16, d16, c, hw, c_pad, units_p, units_c, total_units);
    else
      launch_kernel(nchw_to_nhwc_regs_kernel<4, 4>, dim3(gb), dim3(kThreads), 0, stream, s16, d16, c, hw, c_pad, units_p, units_c, total_units);
    count_launch();
    return cudaGetLastError();
  }
  if ((hw % 8) != 0 && hw <= 640 && ((int64_t)c * hw) % 8 == 0 && (kTileC * hw) % 8 == 0) {
    // small odd plane: contiguous 64-channel spans (at most 80 KB of shared memory)
    const size_t smem = (size_t)kTileC * hw * sizeof(uint16_t);
    cudaError_t err = cudaFuncSetAttribute(nchw_to_nhwc_smallplane_kernel,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    dim3 grid2((unsigned)c_tiles, (unsigned)n);
    launch_kernel(nchw_to_nhwc_smallplane_kernel, dim3(grid2), dim3(kThreads), smem, stream, reinterpret_cast<const uint16_t*>(src),
                                                                      reinterpret_cast<uint16_t*>(dst), c, (int)hw, c_pad);
    count_launch();
    return cudaGetLastError();
  }
  dim3 grid((unsigned)px_tiles, (unsigned)c_tiles, (unsigned)n);
  launch_kernel(nchw_to_nhwc_kernel, dim3(grid), dim3(kThreads), 0, stream, reinterpret_cast<const uint16_t*>(src),
                                                     reinterpret_cast<uint16_t*>(dst), c, hw, c_pad,
                                                     (hw % 8) == 0);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_nhwc_to_nchw(const __half* src, __half* dst, int32_t n, int32_t c, int32_t h,
                                int32_t w, int32_t c_pad, cudaStream_t stream) {
  const int64_t hw = (int64_t)h * w;
  const int64_t px_tiles = (hw + kTileP - 1) / kTileP;
  const int c_tiles = (c + kTileC - 1) / kTileC;
  if (px_tiles > 0x7fffffffLL || c_tiles > 65535 || n > 65535) return cudaErrorInvalidConfiguration;
  dim3 grid((unsigned)px_tiles, (unsigned)c_tiles, (unsigned)n);
  launch_kernel(nhwc_to_nchw_kernel, dim3(grid), dim3(kThreads), 0, stream, reinterpret_cast<const uint16_t*>(src),
                                                     reinterpret_cast<uint16_t*>(dst), c, hw, c_pad,
                                                     (hw % 8) == 0);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_weights_repack(const __half* src, __half* dst, int32_t k, int32_t cg, int32_t r,
                                  int32_t s, int32_t group, int32_t c_pad, cudaStream_t stream, int perm) {
  (void)group;  // groups are contiguous blocks of output channels: the permutation is per k
  const int64_t total = (int64_t)k * r * s * (c_pad / 8);
  int64_t blocks = (total + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (blocks < 1) blocks = 1;
  launch_kernel(weights_repack_kernel, dim3((unsigned)blocks), dim3(256), 0, stream, 
      reinterpret_cast<const uint16_t*>(src), reinterpret_cast<uint16_t*>(dst), k, cg, r * s, c_pad, perm);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_patch_im2col(const ConvGeom& g, const __half* src, __half* dst, int32_t kelems,
                                cudaStream_t stream) {
  const uint16_t* s16 = reinterpret_cast<const uint16_t*>(src);
  uint16_t* d16 = reinterpret_cast<uint16_t*>(dst);
  const int64_t pixels = (int64_t)g.n * g.p * g.q;
  if (g.r == 3 && g.s == 3 && (g.c == 3 || g.c == 1 || g.c == 4) && g.stride_w == 2 && g.pad_w == 1 && g.dil_h == 1 &&
      g.dil_w == 1 && (g.w % 2) == 0 && g.q == g.w / 2) {
    // (even rows: every row of x starts on a 4-byte boundary)
    const int wpr = (g.q + 31) / 32;
    const int64_t warps = (int64_t)g.n * g.p * wpr;
    const int64_t blocks = (warps + 7) / 8;
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
#define HGC_PATCH_S2(CV)                                                                                        \
  launch_kernel(patch_im2col_s2_kernel<CV>, dim3((unsigned)blocks), dim3(256), 0, stream, s16, d16, g.h, g.w, g.p, g.q, \
                g.pad_h, g.stride_h, kelems, wpr, warps)
    if (g.c == 3) HGC_PATCH_S2(3);
    else if (g.c == 1) HGC_PATCH_S2(1);
    else HGC_PATCH_S2(4);
#undef HGC_PATCH_S2
  } else if (g.r == 3 && g.s == 3 && (g.c == 3 || g.c == 1 || g.c == 4)) {
    const int64_t blocks = (pixels + 255) / 256;
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
#define HGC_PATCH(CV)                                                                                         \
  launch_kernel(patch_im2col_kernel<3, 3, CV>, dim3((unsigned)blocks), dim3(256), 0, stream, s16, d16, g.h, g.w, g.p, g.q, g.pad_h, \
                                                                      g.pad_w, g.stride_h, g.stride_w, g.dil_h, \
                                                                      g.dil_w, kelems, pixels)
    if (g.c == 3) HGC_PATCH(3);
    else if (g.c == 1) HGC_PATCH(1);
    else HGC_PATCH(4);
#undef HGC_PATCH
  } else {
    const int64_t chunks = pixels * (kelems / 8);
    const int64_t blocks = (chunks + 255) / 256;
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    launch_kernel(patch_im2col_generic_kernel, dim3((unsigned)blocks), dim3(256), 0, stream, s16, d16, g.c, g.h, g.w, g.p, g.q, g.r, g.s,
                                                                      g.pad_h, g.pad_w, g.stride_h, g.stride_w,
                                                                      g.dil_h, g.dil_w, kelems, chunks);
  }
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_weights_repack_patch(const __half* src, __half* dst, int32_t k, int32_t c, int32_t r, int32_t s,
                                        int32_t kelems, cudaStream_t stream, int perm) {
  const int64_t total = (int64_t)k * kelems;
  int64_t blocks = (total + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (blocks < 1) blocks = 1;
  launch_kernel(weights_repack_patch_kernel, dim3((unsigned)blocks), dim3(256), 0, stream, 
      reinterpret_cast<const uint16_t*>(src), reinterpret_cast<uint16_t*>(dst), k, c, r, s, kelems, perm);
  count_launch();
  return cudaGetLastError();
}

// Row pairs (IgemmPlan::rowpair): w[k][c][r][s] (k < 64) -> w'[half * 64 + k][r'][s][c_pad] with
// r' = r + half, r' in [0, R]; rows r' that a half does not have are zero.  One thread per 8 channels.
__global__ void weights_repack_rowpair_kernel(const uint16_t* __restrict__ src, uint16_t* __restrict__ dst, int cg, int r,
                                              int s, int c_pad) {
  grid_dependency_wait();
  grid_launch_dependents();  // a tensor-core kernel that follows may set itself up beside this one
  const int64_t vecs_per_k = (int64_t)(r + 1) * s * (c_pad / 8);
  const int64_t total = 128 * vecs_per_k;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int kk = (int)(i / vecs_per_k);
    const int64_t rem = i % vecs_per_k;
    const int t = (int)(rem / (c_pad / 8));  // tap r' * s + column
    const int cv = (int)(rem % (c_pad / 8));
    const int half = kk >> 6, k = kk & 63;
    const int rr = t / s - half, ss = t % s;
    uint32_t o[4] = {0, 0, 0, 0};
    if (rr >= 0 && rr < r) {
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int ch = cv * 8 + j;
        uint32_t v = 0;
        if (ch < cg) v = src[(((int64_t)k * cg + ch) * r + rr) * s + ss];
        o[j >> 1] |= v << ((j & 1) * 16);
      }
    }
    HGC_CHECKED_STORE(reinterpret_cast<uint4*>(dst + ((int64_t)kk * (r + 1) * s + t) * c_pad + cv * 8),
                      *reinterpret_cast<uint4*>(dst + ((int64_t)kk * (r + 1) * s + t) * c_pad + cv * 8) = make_uint4(o[0], o[1], o[2], o[3]));
  }
}

// The two preparation steps of the tensor-core path, dispatched on the plan's mode.
cudaError_t launch_igemm_weights(const ConvGeom& g, const IgemmPlan& p, const __half* w, __half* wp,
                                 cudaStream_t stream) {
  if (p.rowpair) {
    const int64_t total = (int64_t)128 * (g.r + 1) * g.s * (p.cw / 8);
    launch_kernel(weights_repack_rowpair_kernel, dim3((unsigned)((total + 255) / 256)), dim3(256), 0, stream,
                  reinterpret_cast<const uint16_t*>(w), reinterpret_cast<uint16_t*>(wp), g.cg, g.r, g.s, p.cw);
    count_launch();
    return cudaGetLastError();
  }
  // (replicated rows: the whole re-laid-out tensor once per replica, one copy after the other)
  const size_t copy_elems = (size_t)g.k * p.eff_r * p.eff_s * p.cw;
  for (int i = 0; i < (1 << p.dup_log2); ++i) {
    __half* dst = wp + (size_t)i * copy_elems;
    cudaError_t e;
    if (p.patch) e = launch_weights_repack_patch(w, dst, g.k, g.c, g.r, g.s, p.cw, stream, p.y_perm);
    else if (p.window) e = launch_weights_repack_window(w, dst, g.k, g.c, g.r, g.s, p.kw_pix, stream, p.y_perm, p.px_ch);
    else e = launch_weights_repack(w, dst, g.k, g.cg, g.r, g.s, g.group, p.cw, stream, p.y_perm);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

__global__ void __launch_bounds__(256)
depthwise_weights_to_taps_kernel(const uint16_t* __restrict__ w, uint16_t* __restrict__ w9, int c) {
  grid_dependency_wait();
  grid_launch_dependents();  // a tensor-core kernel that follows may set itself up beside this one
  const int i = blockIdx.x * blockDim.x + threadIdx.x;  // index into w9: tap * c + channel
  if (i < 9 * c) HGC_CHECKED_STORE(w9 + i, w9[i] = w[(i % c) * 9 + i / c]);
}

cudaError_t launch_depthwise_weights_to_taps(const __half* w, __half* w9, int32_t c, cudaStream_t stream) {
  launch_kernel(depthwise_weights_to_taps_kernel, dim3((unsigned)((9 * c + 255) / 256)), dim3(256), 0, stream,
                reinterpret_cast<const uint16_t*>(w), reinterpret_cast<uint16_t*>(w9), (int)c);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_igemm_input(const ConvGeom& g, const IgemmPlan& p, const __half* x, __half* xp,
                               cudaStream_t stream) {
  if (p.nchw || p.x_nhwc) return cudaSuccess;  // the kernel reads x itself
  if (p.fuse_layout) return cudaSuccess;       // the tensor-core kernel converts x itself
  if (p.patch) return launch_patch_im2col(g, x, xp, p.cw, stream);
  if (p.window) return launch_nchw_to_nhwc8_bordered(x, xp, g.n, g.c, g.h, g.w, g.pad_h, g.pad_w, p.hp, p.wp, stream, p.px_ch);
  return launch_nchw_to_nhwc(x, xp, g.n, g.c, g.h, g.w, p.c_pad, stream);
}

}  // namespace hgc
