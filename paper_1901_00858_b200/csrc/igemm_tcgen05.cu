// Implicit-GEMM convolution on the 5th-generation tensor cores (tcgen05) of sm_100a.
//
// GEMM view, per group:   D[k][pixel] = sum_{r,s,c} W'[k][(r,s,c)] * X'[pixel @ tap (r,s)][c]
//   M (TMEM lanes)   = 128 output channels of the group
//   N (TMEM columns) = a tile of output pixels: tn images x th rows x the full output width
//   K (reduction)    = taps (r,s) x channel blocks of kb = 64 / 32 / 16 channels
// Both operands are K-major in shared memory (channels innermost):
//   A = re-laid-out weights  w'[g][K/g][R][S][cw]        (TMA, 3-D map, box kb x 128 x 1)
//   B = NHWC copy of the input x'[N][H][W][c_pad]        (TMA, 5-D map (c, g, w, h, n),
//       box kb x 1 x tw*stride x th*stride x tn with element strides = conv stride; the
//       start coordinate (q0*stride - pad + s*dil, p0*stride - pad + r*dil) may lie outside the
//       image: TMA zero-fills, which IS the zero padding)
// TMA writes the 128/64/32-byte swizzled layout the UMMA shared-memory descriptors name.
//
// One CTA computes one 128 x N tile:  warp 0 = TMA producer, warp 1 = TMEM allocator and MMA
// issuer (one elected lane issues tcgen05.mma; tcgen05.commit releases smem stages through
// mbarriers), warps 2..5 = epilogue: tcgen05.ld of the fp32 accumulators (lane = output
// channel, so a thread owns a run of consecutive pixels of one NCHW channel plane), + bias,
// ReLU, cvt.rn.f16, 16-byte stores straight into y (no NHWC->NCHW pass for the output).
//
// Every wait on an mbarrier is bounded by wall-clock time; on expiry the CTA raises a status
// word, lets its outstanding copies land, frees its TMEM and returns.
#include <cuda.h>
#include <cudaTypedefs.h>

#include "hgc_internal.h"

namespace hgc {
namespace {

constexpr int kIgemmThreads = 192;
constexpr uint64_t kWaitLimitNs = 2000000000ull;  // 2 s per wait

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}

__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait: false if the limit expired or another role already gave up.
__device__ __noinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  uint64_t t0 = 0;
  for (uint32_t i = 0;; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 63u) == 63u) {
      if (*abort_flag) return false;
      const uint64_t t = global_timer_ns();
      if (t0 == 0) {
        t0 = t;
      } else if (t - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        return false;
      }
    }
  }
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1,
                                            int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1,
                                            int c2, int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
      ::"r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                         uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
      "}\n" ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}

__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr)
      : "memory");
}

struct IgemmArgs {
  int32_t N, K, P, Q;
  int32_t kg, group;
  int32_t R, S, pad_h, pad_w, stride_h, stride_w, dil_h, dil_w;
  int32_t kb;        // channels per reduction block (64 / 32 / 16)
  int32_t cblocks;   // blocks per tap
  int32_t cw;        // channels per tap in w' (cblocks * kb)
  int32_t tn, th, tw;  // pixel tile: images x rows x full width (tw == Q)
  int32_t ncols;     // MMA N: tn*th*tw rounded up to 16
  int32_t tiles_h;   // row tiles per plane
  int32_t mtiles;    // 128-channel tiles per group
  int32_t stages;
  int32_t tmem_cols; // power of two >= ncols
  uint32_t a_bytes, b_bytes, b_alloc;  // TMA bytes of A and B per stage, smem reserved for B
  uint32_t idesc;
  uint64_t desc_hi;  // shared-memory descriptor bits other than the start address
  int32_t relu;
};

__global__ void __launch_bounds__(kIgemmThreads, 1)
igemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
             const IgemmArgs a, const __half* __restrict__ bias, __half* __restrict__ y, int* status) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[8];
  __shared__ __align__(8) uint64_t empty_bar[8];
  __shared__ __align__(8) uint64_t acc_bar;
  __shared__ uint32_t tmem_slot;
  __shared__ volatile int abort_flag;

  // a CTA of an earlier wave gave up: do not start new work on a path that is not progressing
  if (status != nullptr && *reinterpret_cast<volatile int*>(status) != 0) return;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t stage_bytes = a.a_bytes + a.b_alloc;

  // tile coordinates
  const int tile_n = blockIdx.x / a.tiles_h;
  const int tile_h = blockIdx.x % a.tiles_h;
  const int n0 = tile_n * a.tn;
  const int p0 = tile_h * a.th;
  const int grp = blockIdx.y / a.mtiles;
  const int m0 = (blockIdx.y % a.mtiles) * 128;
  const int niter = a.R * a.S * a.cblocks;

  if (threadIdx.x == 0) {
    for (int s = 0; s < a.stages; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), 1);
    }
    mbar_init(smem_u32(&acc_bar), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                 "r"((uint32_t)a.tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = tmem_slot;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      int issued = 0;
      int r = 0, s = 0, cb = 0;
      for (int it = 0; it < niter; ++it) {
        const int st = it % a.stages;
        const uint32_t ph = (uint32_t)(it / a.stages) & 1u;
        if (!mbar_wait(smem_u32(&empty_bar[st]), ph ^ 1u, &abort_flag)) break;
        const uint32_t fb = smem_u32(&full_bar[st]);
        mbar_expect_tx(fb, a.a_bytes + a.b_bytes);
        const uint32_t sa = tiles_base + (uint32_t)st * stage_bytes;
        tma_load_3d(sa, &tmA, fb, (r * a.S + s) * a.cw + cb * a.kb, m0, grp);
        tma_load_5d(sa + a.a_bytes, &tmB, fb, cb * a.kb, grp, s * a.dil_w - a.pad_w,
                    p0 * a.stride_h - a.pad_h + r * a.dil_h, n0);
        issued = it + 1;
        if (++cb == a.cblocks) {
          cb = 0;
          if (++s == a.S) {
            s = 0;
            ++r;
          }
        }
      }
      if (abort_flag) {
        // let the copies that were issued land before the CTA's shared memory goes away
        const int first = issued > a.stages ? issued - a.stages : 0;
        for (int it = first; it < issued; ++it) {
          uint64_t t0 = global_timer_ns();
          while (!mbar_try_wait(smem_u32(&full_bar[it % a.stages]), (uint32_t)(it / a.stages) & 1u)) {
            if (global_timer_ns() - t0 > kWaitLimitNs) break;
          }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      bool ok = true;
      const int ksteps = a.kb / 16;
      for (int it = 0; it < niter; ++it) {
        const int st = it % a.stages;
        const uint32_t ph = (uint32_t)(it / a.stages) & 1u;
        if (!mbar_wait(smem_u32(&full_bar[st]), ph, &abort_flag)) {
          ok = false;
          break;
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t sa = tiles_base + (uint32_t)st * stage_bytes;
        const uint32_t sb = sa + a.a_bytes;
        const uint64_t adesc = a.desc_hi | (uint64_t)((sa & 0x3FFFFu) >> 4);
        const uint64_t bdesc = a.desc_hi | (uint64_t)((sb & 0x3FFFFu) >> 4);
        for (int k = 0; k < ksteps; ++k) {
          // 16 channels = 32 bytes further along the swizzled row: +2 in the address field
          umma_f16(tmem_base, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), a.idesc,
                   (it > 0 || k > 0) ? 1u : 0u);
        }
        umma_commit(smem_u32(&empty_bar[st]));  // frees the stage when these MMAs have read it
      }
      if (ok) umma_commit(smem_u32(&acc_bar));  // accumulator complete
    }
    __syncwarp();
  } else {
    // ---------------- epilogue (warps 2..5) ----------------
    const int quarter = warp & 3;  // the TMEM lane quarter this warp may read
    const int row = quarter * 32 + lane;
    const int kin = m0 + row;
    const bool kvalid = kin < a.kg;
    const int k = grp * a.kg + (kvalid ? kin : 0);
    const float bv = (bias != nullptr && kvalid) ? __half2float(__ldg(bias + k)) : 0.f;
    const bool ok = mbar_wait(smem_u32(&acc_bar), 0, &abort_flag);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (ok) {
      const int64_t pq = (int64_t)a.P * a.Q;
      const int plane_tile = a.th * a.tw;
      const int ntile = a.tn * plane_tile;
      const int64_t plane_off0 = (int64_t)p0 * a.Q;
      uint16_t* yb = reinterpret_cast<uint16_t*>(y);
      for (int col0 = 0; col0 < a.ncols; col0 += 16) {
        uint32_t v[16];
        tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)col0, v);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int h8 = 0; h8 < 2; ++h8) {
          const int j = col0 + h8 * 8;
          if (j >= ntile || !kvalid) continue;
          uint32_t o[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            float f0 = __uint_as_float(v[h8 * 8 + 2 * e]) + bv;
            float f1 = __uint_as_float(v[h8 * 8 + 2 * e + 1]) + bv;
            if (a.relu) {
              f0 = fmaxf(f0, 0.f);
              f1 = fmaxf(f1, 0.f);
            }
            o[e] = (uint32_t)__half_as_ushort(__float2half_rn(f0)) |
                   ((uint32_t)__half_as_ushort(__float2half_rn(f1)) << 16);
          }
          const int in = j / plane_tile;
          const int rem = j - in * plane_tile;
          const int n = n0 + in;
          const int64_t off = plane_off0 + rem;
          uint16_t* dst = yb + ((int64_t)n * a.K + k) * pq + off;
          if (rem + 7 < plane_tile && n < a.N && off + 7 < pq && (reinterpret_cast<uintptr_t>(dst) & 15u) == 0) {
            *reinterpret_cast<uint4*>(dst) = make_uint4(o[0], o[1], o[2], o[3]);
          } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const int jj = j + e;
              if (jj < ntile) {
                const int in2 = jj / plane_tile;
                const int rem2 = jj - in2 * plane_tile;
                const int n2 = n0 + in2;
                const int64_t off2 = plane_off0 + rem2;
                if (n2 < a.N && off2 < pq)
                  yb[((int64_t)n2 * a.K + k) * pq + off2] = (uint16_t)((o[e >> 1] >> ((e & 1) * 16)) & 0xffffu);
              }
            }
          }
        }
        __syncwarp();  // tcgen05.ld is warp-collective: reconverge before the next one
      }
    }
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)a.tmem_cols)
                 : "memory");
  }
  if (threadIdx.x == 0 && abort_flag && status != nullptr) atomicExch(status, (int)HGC_DEVICE_TIMEOUT);
}

// ---- host side ----------------------------------------------------------------------------------

PFN_cuTensorMapEncodeTiled_v12000 encode_fn() {
  static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(p);
  }
  return fn;
}

inline size_t round_up_sz(size_t v, size_t a) { return (v + a - 1) / a * a; }

}  // namespace

bool igemm_make_plan(const ConvGeom& g, IgemmPlan* out) {
  IgemmPlan p{};
  if (g.cg < 9) return false;                         // too few channels per tap for a K=16 MMA step
  if (g.group > 1 && (g.cg % 8) != 0) return false;  // group stride of x' must be 16-byte aligned
  p.kb = g.cg > 32 ? 64 : (g.cg > 16 ? 32 : 16);
  p.cblocks = (g.cg + p.kb - 1) / p.kb;
  p.cw = p.cblocks * p.kb;
  p.c_pad = (g.c + 7) / 8 * 8;
  // pixel tile: full output width, as many rows (then images) as fit 256 columns
  if (g.q > 256 || (int64_t)g.q * g.stride_w > 256) return false;
  p.tw = g.q;
  const int th_max = 256 / g.q;
  if (th_max >= g.p) {
    p.th = g.p;
    p.tiles_h = 1;
    int tn_max = 256 / (g.p * g.q);
    if (tn_max > g.n) tn_max = g.n;
    const int nt = (g.n + tn_max - 1) / tn_max;
    p.tn = (g.n + nt - 1) / nt;
  } else {
    p.tiles_h = (g.p + th_max - 1) / th_max;
    p.th = (g.p + p.tiles_h - 1) / p.tiles_h;
    p.tn = 1;
  }
  if ((int64_t)p.th * g.stride_h > 256) return false;
  p.tiles_n = (g.n + p.tn - 1) / p.tn;
  p.ncols = (p.tn * p.th * p.tw + 15) / 16 * 16;
  p.mtiles = (g.kg + 127) / 128;
  if ((int64_t)p.tiles_n * p.tiles_h > 0x7fffffffLL || (int64_t)p.mtiles * g.group > 65535) return false;
  p.a_bytes = 128u * p.kb * 2u;
  p.b_bytes = (uint32_t)(p.tn * p.th * p.tw) * p.kb * 2u;
  p.b_alloc = (uint32_t)round_up_sz((size_t)p.ncols * p.kb * 2u, 1024);
  const size_t stage = p.a_bytes + p.b_alloc;
  int stages = (int)((220u * 1024u) / stage);
  if (stages > 8) stages = 8;
  if (stages < 2) return false;
  p.stages = stages;
  p.smem_bytes = stage * stages + 1024;
  p.tmem_cols = p.ncols <= 32 ? 32 : p.ncols <= 64 ? 64 : p.ncols <= 128 ? 128 : 256;
  // workspace: status word, re-laid-out weights, NHWC input
  p.ws_status_off = 0;
  p.ws_w_off = 256;
  p.ws_x_off = p.ws_w_off + round_up_sz((size_t)g.k * g.r * g.s * p.cw * 2, 256);
  p.ws_total = p.ws_x_off + round_up_sz((size_t)g.n * g.h * g.w * p.c_pad * 2, 256);
  *out = p;
  return true;
}

// Encodes the two tensor maps over the workspace tensors.  Returns false on failure.
bool igemm_encode_maps(const ConvGeom& g, IgemmPlan* p, void* ws) {
  PFN_cuTensorMapEncodeTiled_v12000 enc = encode_fn();
  if (enc == nullptr) return false;
  char* base = static_cast<char*>(ws);
  const CUtensorMapSwizzle sw = p->kb == 64 ? CU_TENSOR_MAP_SWIZZLE_128B
                               : p->kb == 32 ? CU_TENSOR_MAP_SWIZZLE_64B
                                             : CU_TENSOR_MAP_SWIZZLE_32B;
  {
    const cuuint64_t kred = (cuuint64_t)g.r * g.s * p->cw;
    cuuint64_t dims[3] = {kred, (cuuint64_t)g.kg, (cuuint64_t)g.group};
    cuuint64_t strides[2] = {kred * 2, kred * 2 * (cuuint64_t)g.kg};
    cuuint32_t box[3] = {(cuuint32_t)p->kb, 128, 1};
    cuuint32_t es[3] = {1, 1, 1};
    if (enc(&p->tmA, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, base + p->ws_w_off, dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return false;
  }
  {
    const cuuint64_t cdim = g.group > 1 ? (cuuint64_t)g.cg : (cuuint64_t)p->c_pad;
    const cuuint64_t pix = (cuuint64_t)p->c_pad * 2;
    cuuint64_t dims[5] = {cdim, (cuuint64_t)g.group, (cuuint64_t)g.w, (cuuint64_t)g.h, (cuuint64_t)g.n};
    cuuint64_t strides[4] = {g.group > 1 ? (cuuint64_t)g.cg * 2 : pix, pix, pix * g.w, pix * g.w * g.h};
    cuuint32_t box[5] = {(cuuint32_t)p->kb, 1, (cuuint32_t)(p->tw * g.stride_w), (cuuint32_t)(p->th * g.stride_h),
                         (cuuint32_t)p->tn};
    cuuint32_t es[5] = {1, 1, (cuuint32_t)g.stride_w, (cuuint32_t)g.stride_h, 1};
    if (enc(&p->tmB, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 5, base + p->ws_x_off, dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return false;
  }
  p->maps_ready = true;
  return true;
}

cudaError_t launch_igemm(const ConvGeom& g, const IgemmPlan& p, void* ws, const __half* bias, __half* y,
                         int relu, cudaStream_t stream) {
  if (!p.maps_ready) return cudaErrorInvalidValue;
  IgemmArgs a{};
  a.N = g.n; a.K = g.k; a.P = g.p; a.Q = g.q;
  a.kg = g.kg; a.group = g.group;
  a.R = g.r; a.S = g.s; a.pad_h = g.pad_h; a.pad_w = g.pad_w;
  a.stride_h = g.stride_h; a.stride_w = g.stride_w; a.dil_h = g.dil_h; a.dil_w = g.dil_w;
  a.kb = p.kb; a.cblocks = p.cblocks; a.cw = p.cw;
  a.tn = p.tn; a.th = p.th; a.tw = p.tw; a.ncols = p.ncols;
  a.tiles_h = p.tiles_h; a.mtiles = p.mtiles; a.stages = p.stages; a.tmem_cols = p.tmem_cols;
  a.a_bytes = p.a_bytes; a.b_bytes = p.b_bytes; a.b_alloc = p.b_alloc;
  // instruction descriptor: D = f32, A = B = f16, both K-major, N >> 3 at bit 17, M >> 4 at bit 24
  a.idesc = (1u << 4) | ((uint32_t)(p.ncols >> 3) << 17) | ((128u >> 4) << 24);
  // shared-memory descriptor: 8-row groups are 8 * row bytes apart; descriptor version 1;
  // swizzle mode 2 = 128 B, 4 = 64 B, 6 = 32 B
  const uint64_t sbo = (uint64_t)(8 * p.kb * 2) >> 4;
  const uint64_t layout = p.kb == 64 ? 2 : (p.kb == 32 ? 4 : 6);
  a.desc_hi = (1ull << 16) | (sbo << 32) | (1ull << 46) | (layout << 61);
  a.relu = relu;
  cudaError_t err = cudaFuncSetAttribute(igemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)p.smem_bytes);
  if (err != cudaSuccess) return err;
  dim3 grid((unsigned)(p.tiles_n * p.tiles_h), (unsigned)(p.mtiles * g.group));
  int* status = reinterpret_cast<int*>(static_cast<char*>(ws) + p.ws_status_off);
  igemm_kernel<<<grid, kIgemmThreads, p.smem_bytes, stream>>>(p.tmA, p.tmB, a, bias, y, status);
  count_launch();
  return cudaGetLastError();
}

}  // namespace hgc
