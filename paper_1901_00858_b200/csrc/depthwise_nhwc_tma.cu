// Channels-last 3x3 depthwise, stride 1, for C % 32 == 0: the input tile of a block is fetched by
// TMA (x[N][H][W][C] seen as a 4-D tensor; the zero padding is the copy's out-of-bounds fill) into
// one of two shared-memory buffers while the previous tile is being used, so the threads never
// wait on global loads: they read 16-byte vectors (8 channels of a pixel) from shared memory,
// accumulate with the mixed-precision FMA and store 16-byte vectors straight to y.
//
// Block = 256 threads, persistent over the tiles of the layer.  A tile is CB channels (64, or 32)
// x tw output columns x th output rows (tw * th = 256 or 512, the shape that loads least per plane).  A lane owns a channel octet and one of 4 (8)
// adjacent columns, a warp one column group and a strip of 8 output rows: every shared-memory
// read and every global store of a warp covers 512 contiguous bytes.  A thread walks down the 10
// input rows of its strip once and keeps its 8 x 8 accumulators and its 72 weights in registers.
//
// Every wait on a copy is bounded; on expiry the block raises a status word, skips its remaining
// work and returns (the host reads and clears the word through depthwise_nhwc_tma_status()).
#include <cudaTypedefs.h>

#include "hgc_internal.h"

namespace hgc {
namespace {

constexpr int kRowsPerThread = 8;

__device__ int g_dw_tma_status = 0;
// limit of a wait for a copy, in ns of %globaltimer (hgc_debug_set_wait_limit_ns shortens it)
constexpr uint64_t kDwWaitLimitNs = 2000000000ull;
__device__ uint64_t g_dw_wait_limit_ns = kDwWaitLimitNs;

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void bar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void bar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool bar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// two seconds at most (try_wait itself suspends for a while per attempt)
__device__ __noinline__ bool bar_wait_bounded(uint32_t bar, uint32_t parity) {
  uint64_t t0 = 0;
  for (uint32_t i = 0;; ++i) {
    if (bar_try_wait(bar, parity)) return true;
    if (i > 64) __nanosleep(256);
    if ((i & 63u) == 63u) {
      uint64_t t;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
      if (t0 == 0) t0 = t;
      else if (t - t0 > g_dw_wait_limit_ns) return false;
    }
  }
}
__device__ __forceinline__ void tma_load_tile(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int w0,
                                              int h0, int n) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], "
      "[%2];" ::"r"(dst),
      "l"(tm), "r"(bar), "r"(c0), "r"(w0), "r"(h0), "r"(n)
      : "memory");
}

struct DwTmaArgs {
  int32_t n, c, h, w, p, q, pad_h, pad_w;
  int32_t cblocks, row_tiles, col_tiles, th, tw;  // th x tw = output rows x columns per tile
  int64_t tiles;
  uint32_t tile_bytes;
  int32_t dbg_drop;  // test hook: the first block announces its dbg_drop-th copy but never issues it (-1: none)
};

template <int CB>
__global__ void __launch_bounds__(256, 2)
depthwise3x3_nhwc_tma_kernel(const __grid_constant__ CUtensorMap tmX, DwTmaArgs a, const uint16_t* __restrict__ w,
                             const uint16_t* __restrict__ bias, uint16_t* __restrict__ y, int relu) {
  grid_dependency_wait();
  constexpr int OCT = CB / 8;         // channel octets per pixel of the tile
  constexpr int CPW = 32 / OCT;       // adjacent columns per warp
  const int CGROUPS = a.tw / CPW;     // column groups per tile
  const int kIW = a.tw + 2;           // input columns per tile
  extern __shared__ __align__(128) unsigned char dw_smem[];
  __shared__ uint64_t full[2];
  const uint32_t buf0 = (smem_addr(dw_smem) + 127u) & ~127u;
  const int lane = (int)(threadIdx.x & 31u), warp = (int)(threadIdx.x >> 5);
  const int o = lane % OCT, cq = lane / OCT;
  const int col = (warp % CGROUPS) * CPW + cq;            // output column within the tile
  const int row0 = (warp / CGROUPS) * kRowsPerThread;     // first output row of this thread's strip
  if (threadIdx.x == 0) {
    bar_init(smem_addr(&full[0]), 1);
    bar_init(smem_addr(&full[1]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __shared__ int copy_ok;
  __syncthreads();

  // tile t -> (channel block, image, row tile, column tile); channel block slowest
  auto decode = [&](int64_t t, int& cb, int& n, int& rt, int& ct) {
    ct = (int)(t % a.col_tiles);
    t /= a.col_tiles;
    rt = (int)(t % a.row_tiles);
    t /= a.row_tiles;
    n = (int)(t % a.n);
    cb = (int)(t / a.n);
  };
  uint32_t issued = 0;  // (thread 0's count of announced copies)
  auto issue = [&](int64_t t, uint32_t slot) {
    int cb, n, rt, ct;
    decode(t, cb, n, rt, ct);
    const uint32_t bar = smem_addr(&full[slot]);
    bar_expect_tx(bar, a.tile_bytes);
    // test hook: announced but never issued, so that the wait for it runs out
    if (a.dbg_drop >= 0 && blockIdx.x == 0 && issued++ == (uint32_t)a.dbg_drop) return;
    tma_load_tile(buf0 + slot * a.tile_bytes, &tmX, bar, cb * CB, ct * a.tw - a.pad_w, rt * a.th - a.pad_h, n);
  };

  int64_t t = blockIdx.x;
  if (t >= a.tiles) return;
  if (threadIdx.x == 0) issue(t, 0);
  uint16_t wv[72];
  float bv[8];
  int cb_loaded = -1;
  uint32_t it = 0;
  for (; t < a.tiles; t += gridDim.x, ++it) {
    const uint32_t slot = it & 1u;
    // the other buffer was released by the __syncthreads that ended the previous tile
    if (threadIdx.x == 0 && t + gridDim.x < a.tiles) issue(t + gridDim.x, slot ^ 1u);
    int cb, n, rt, ct;
    decode(t, cb, n, rt, ct);
    if (cb != cb_loaded) {
      cb_loaded = cb;
      const int ch0 = cb * CB + o * 8;
      const uint4* wp = reinterpret_cast<const uint4*>(w + (int64_t)ch0 * 9);  // 8 channels x 9 taps: 144 bytes
#pragma unroll
      for (int i = 0; i < 9; ++i) {
        const uint4 v = __ldg(wp + i);
        const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j)
          asm("mov.b32 {%0, %1}, %2;" : "=h"(wv[8 * i + 2 * j]), "=h"(wv[8 * i + 2 * j + 1]) : "r"(u[j]));
      }
      if (bias != nullptr) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(bias + ch0));
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
    }
    // one thread waits (bounded) and tells the block, so that the block leaves the loop as one
    if (threadIdx.x == 0) {
      copy_ok = bar_wait_bounded(smem_addr(&full[slot]), (it >> 1) & 1u) ? 1 : 0;
      if (!copy_ok) g_dw_tma_status = 1;
    }
    __syncthreads();
    if (!copy_ok) {
      // give a copy that is still in flight into the other buffer the same time to land
      if (threadIdx.x == 0 && t + gridDim.x < a.tiles)
        (void)bar_wait_bounded(smem_addr(&full[slot ^ 1u]), ((it + 1) >> 1) & 1u);
      break;
    }
    (void)bar_try_wait(smem_addr(&full[slot]), (it >> 1) & 1u);  // completed phase: every thread observes it itself
    const uint32_t tile = buf0 + slot * a.tile_bytes;
    float acc[kRowsPerThread][8];
#pragma unroll
    for (int r = 0; r < kRowsPerThread; ++r)
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[r][e] = bv[e];
    // input row ir of the strip feeds output rows ir - 2 .. ir (kernel rows 2 .. 0)
#pragma unroll
    for (int ir = 0; ir < kRowsPerThread + 2; ++ir) {
      uint4 xin[3];
#pragma unroll
      for (int ss = 0; ss < 3; ++ss) {
        const uint32_t addr = tile + (uint32_t)(((row0 + ir) * kIW + col + ss) * (CB * 2) + o * 16);
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(xin[ss].x), "=r"(xin[ss].y), "=r"(xin[ss].z), "=r"(xin[ss].w)
                     : "r"(addr));
      }
#pragma unroll
      for (int rr = 0; rr < 3; ++rr) {
        const int orow = ir - rr;
        if (orow < 0 || orow >= kRowsPerThread) continue;
#pragma unroll
        for (int ss = 0; ss < 3; ++ss) {
          const uint32_t u[4] = {xin[ss].x, xin[ss].y, xin[ss].z, xin[ss].w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            uint16_t lo, hi;
            asm("mov.b32 {%0, %1}, %2;" : "=h"(lo), "=h"(hi) : "r"(u[j]));
            asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(acc[orow][2 * j]) : "h"(lo), "h"(wv[(2 * j) * 9 + rr * 3 + ss]));
            asm("fma.rn.f32.f16 %0, %1, %2, %0;"
                : "+f"(acc[orow][2 * j + 1])
                : "h"(hi), "h"(wv[(2 * j + 1) * 9 + rr * 3 + ss]));
          }
        }
      }
    }
    const int q = ct * a.tw + col;
    if (q < a.q) {
#pragma unroll
      for (int r = 0; r < kRowsPerThread; ++r) {
        const int p = rt * a.th + row0 + r;
        if (p >= a.p) break;
        uint32_t ov[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (relu)
            asm("cvt.rn.relu.f16x2.f32 %0, %1, %2;" : "=r"(ov[j]) : "f"(acc[r][2 * j + 1]), "f"(acc[r][2 * j]));
          else
            asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(ov[j]) : "f"(acc[r][2 * j + 1]), "f"(acc[r][2 * j]));
        }
        *reinterpret_cast<uint4*>(y + (((int64_t)n * a.p + p) * a.q + q) * a.c + cb * CB + o * 8) =
            make_uint4(ov[0], ov[1], ov[2], ov[3]);
      }
    }
    __syncthreads();  // every thread is done with this buffer: the copy after next may overwrite it
  }
}

PFN_cuTensorMapEncodeTiled_v12000 dw_encode_fn() {
  static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(p);
  }
  return fn;
}

}  // namespace

bool depthwise3x3_nhwc_tma_supported(const ConvGeom& g) {
  if (!depthwise3x3_nhwc_supported(g)) return false;
  if (g.stride_h != 1 || (g.c % 32) != 0) return false;
  if (g.p < 12 || g.q < 12) return false;  // tiles of at least 8 rows: tiny planes would be mostly padding
  if (g.w > 65535 || g.h > 65535) return false;
  return true;
}

cudaError_t depthwise_nhwc_tma_set_wait_limit_ns(uint64_t ns) {
  const uint64_t v = ns == 0 ? kDwWaitLimitNs : ns;
  return cudaMemcpyToSymbol(g_dw_wait_limit_ns, &v, sizeof(v));
}

int depthwise_nhwc_tma_status() {
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, g_dw_tma_status, sizeof(int)) != cudaSuccess) return -1;
  if (v != 0) {
    const int zero = 0;
    (void)cudaMemcpyToSymbol(g_dw_tma_status, &zero, sizeof(int));
  }
  return v;
}

cudaError_t launch_depthwise3x3_nhwc_tma(const ConvGeom& g, const __half* x, const __half* w, const __half* bias,
                                         __half* y, int relu, cudaStream_t stream) {
  PFN_cuTensorMapEncodeTiled_v12000 enc = dw_encode_fn();
  if (enc == nullptr) return cudaErrorInvalidConfiguration;
  const int cb = (g.c % 64) == 0 ? 64 : 32;
  const int cpw = 32 / (cb / 8);
  DwTmaArgs a{};
  a.n = g.n; a.c = g.c; a.h = g.h; a.w = g.w; a.p = g.p; a.q = g.q; a.pad_h = g.pad_h; a.pad_w = g.pad_w;
  // tile shape: column groups x row strips = 8 warps; the shape that loads the fewest input pixels
  // per plane (padding of the plane to whole tiles and the one-pixel halo around each tile)
  int64_t best = -1;
  for (int cgroups = 1; cgroups <= 8; cgroups *= 2) {
    const int tw = cgroups * cpw, th = (8 / cgroups) * kRowsPerThread;
    const int64_t area = (int64_t)((g.q + tw - 1) / tw) * ((g.p + th - 1) / th) * (tw + 2) * (th + 2);
    if (best < 0 || area < best) {
      best = area;
      a.tw = tw;
      a.th = th;
    }
  }
  a.cblocks = g.c / cb;
  a.row_tiles = (g.p + a.th - 1) / a.th;
  a.col_tiles = (g.q + a.tw - 1) / a.tw;
  a.tiles = (int64_t)a.cblocks * g.n * a.row_tiles * a.col_tiles;
  const int ih = a.th + 2, kIW = a.tw + 2;
  a.tile_bytes = (uint32_t)(ih * kIW * cb * 2);
  a.dbg_drop = debug_drop_copies();
  CUtensorMap tm;
  cuuint64_t dims[4] = {(cuuint64_t)g.c, (cuuint64_t)g.w, (cuuint64_t)g.h, (cuuint64_t)g.n};
  cuuint64_t strides[3] = {(cuuint64_t)g.c * 2, (cuuint64_t)g.c * 2 * g.w, (cuuint64_t)g.c * 2 * g.w * g.h};
  cuuint32_t box[4] = {(cuuint32_t)cb, (cuuint32_t)kIW, (cuuint32_t)ih, 1};
  cuuint32_t es[4] = {1, 1, 1, 1};
  if (enc(&tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, const_cast<__half*>(x), dims, strides, box, es,
          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return cudaErrorInvalidConfiguration;
  const size_t smem = 2 * (size_t)a.tile_bytes + 128;
  int64_t blocks = a.tiles;
  const int64_t cap = (int64_t)sm_count() * 2;
  if (blocks > cap) blocks = cap;
  const uint16_t* ws = reinterpret_cast<const uint16_t*>(w);
  const uint16_t* bs = reinterpret_cast<const uint16_t*>(bias);
  uint16_t* ys = reinterpret_cast<uint16_t*>(y);
  cudaError_t err;
  if (cb == 64) {
    err = cudaFuncSetAttribute(depthwise3x3_nhwc_tma_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    err = launch_kernel(depthwise3x3_nhwc_tma_kernel<64>, dim3((unsigned)blocks), dim3(256), smem, stream, tm, a, ws, bs,
                        ys, relu);
  } else {
    err = cudaFuncSetAttribute(depthwise3x3_nhwc_tma_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    err = launch_kernel(depthwise3x3_nhwc_tma_kernel<32>, dim3((unsigned)blocks), dim3(256), smem, stream, tm, a, ws, bs,
                        ys, relu);
  }
  if (err != cudaSuccess) return err;
  count_launch();
  return cudaGetLastError();
}

}  // namespace hgc
