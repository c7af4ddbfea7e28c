// Implicit-GEMM convolution on the 5th-generation tensor cores (tcgen05) of sm_100a.
//
// GEMM view, per group:   D[k][pixel] = sum_{r,s,c} W'[k][(r,s,c)] * X'[pixel @ tap (r,s)][c]
//   M (TMEM lanes)   = 128 output channels of the group
//   N (TMEM columns) = a tile of output pixels: tn images x th rows x the full output width
//   K (reduction)    = taps (r,s) x channel blocks of kb = 64 / 32 / 16 channels
// Operands in shared memory (written by TMA in the 128/64/32-byte swizzled layouts that the UMMA
// shared-memory descriptors name):
//   A = re-laid-out weights  w'[g][K/g][R][S][cw], K-major   (3-D map, box kb x 128 (or 64) x 1)
//   B = activations, one of
//       - the NHWC copy x'[N][H][W][c_pad], K-major (5-D map (c, g, w, h, n), box kb x 1 x
//         tw*stride x th*stride x tn with element strides = conv stride; the start coordinate
//         (q0*stride - pad + s*dil, p0*stride - pad + r*dil) may lie outside the image: TMA
//         zero-fills, which IS the zero padding).  At stride 1 the S taps of a kernel row share one
//         tile: tap s starts s*dil pixel rows further in (a descriptor start offset);
//       - x itself for 1x1 layers (3-D map (pixel, channel, image), boxes of 64 pixels x kb
//         channels): pixel-major ("MN-major") tiles, no copy of x at all;
//       - for few-channel stems, overlapping windows of a zero-bordered 8-channel copy, or an
//         expanded copy holding the values under the kernel per output pixel.
//
// One persistent CTA per SM walks its tiles:  warp 0 = TMA producer (a ring stage = one
// activation tile + the weight tiles of its taps, one mbarrier), warp 1 = TMEM allocator and MMA
// issuer (one elected lane issues tcgen05.mma; tcgen05.commit releases ring stages and hands
// accumulators over through mbarriers; two 256-column accumulators alternate), warps 2.. =
// epilogue, two (or four) per TMEM lane quarter: tcgen05.ld of the fp32 accumulators (lane =
// output channel), + bias, ReLU, cvt.rn.f16x2, staged as fp16 in shared memory and written to
// NCHW y either by TMA stores or by coalesced plain stores (no NHWC->NCHW pass for the output).
//
// Every wait on an mbarrier is bounded by wall-clock time; on expiry the CTA raises a status
// word, lets its outstanding copies land, frees its TMEM and returns.
#include <cuda.h>
#include <cudaTypedefs.h>


#include "hgc_internal.h"

namespace hgc {
HGC_DEBUG_STATE(igemm)
namespace {

constexpr int kEpilogueWarps = 8;       // two per TMEM lane quarter (the default)
constexpr int kEpilogueWarpsWide = 16;  // four per quarter: layers whose tiles are bound by the epilogue
constexpr int kPassElems = 64;               // output pixels per channel staged per TMA store
// one warp's staging tile: 32 channels x 64 pixels (or 64 pixels x 32 channels, or 32 rows of 32
// floats): 4 KB, 1024-byte aligned
constexpr uint32_t kWarpStageBytes = 4096u;
constexpr uint64_t kWaitLimitNs = 2000000000ull;  // 2 s per wait unless the debug hook shortens it
// the limit of every device-side wait of this file, in ns of %globaltimer (hgc_debug_set_wait_limit_ns)
__device__ uint64_t g_wait_limit_ns = kWaitLimitNs;

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

__device__ __forceinline__ uint32_t mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n"
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

// Bounded wait: false if the limit expired or another role already gave up.  `sleep_ns` > 0
// makes a waiting warp yield its issue slots between polls (the epilogue warps wait for whole
// tiles and must not compete with the single TMA and MMA issuing threads).
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                            uint32_t sleep_ns) {
  uint64_t t0 = 0;
  for (uint32_t i = 0;; ++i) {
    // the suspending form: a waiting warp must not burn issue slots or shared-memory bandwidth
    // that the working warps need
    if (mbar_try_wait(bar, parity)) return true;
    if (sleep_ns) __nanosleep(sleep_ns);
    if ((i & 1023u) == 1023u) {
      if (*abort_flag) return false;
      const uint64_t t = global_timer_ns();
      if (t0 == 0) {
        t0 = t;
      } else if (t - t0 > g_wait_limit_ns) {
        *abort_flag = 1;
        return false;
      }
    }
  }
}

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          uint32_t sleep_ns = 0) {
  if (mbar_test_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, abort_flag, sleep_ns);
}

// One lane of a converged warp.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "elect.sync _|p, 0xffffffff;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(pred));
  return pred != 0;
}

// Position in a ring of mbarrier-guarded stages: index and the phase parity of the current lap.
struct Ring {
  uint32_t idx = 0, phase = 0;
  __device__ __forceinline__ void advance(uint32_t depth) {
    if (++idx == depth) {
      idx = 0;
      phase ^= 1u;
    }
  }
};

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1,
                                            int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1,
                                            int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
      ::"r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1,
                                            int c2, int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
      ::"r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(bar)
      : "memory");
}

// The same copies issued by a CTA of a pair: the data lands in the issuing CTA's shared memory,
// the bytes are counted on a barrier that may live in the other CTA of the pair (`bar` is a
// shared::cluster address).  No multicast: every CTA fetches its own tiles.
__device__ __forceinline__ void tma_load_4d_pair(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1,
                                                 int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
      ::"r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void tma_load_5d_pair(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1,
                                                 int c2, int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
      ::"r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(bar)
      : "memory");
}

// shared::cluster address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t cluster_addr(uint32_t local, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
  return r;
}

__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
}

__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
      "h"((uint16_t)3)
      : "memory");
}

__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}

// 32 consecutive accumulator columns of this warp's 32 lanes in one instruction: a TMEM load
// costs the issuing warp about 100 cycles whatever its width (measured), so wide loads matter
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
        "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
        "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}

__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t* v) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
               : "r"(taddr)
               : "memory");
}

__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
        "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]), "r"(v[17]),
        "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]), "r"(v[24]), "r"(v[25]), "r"(v[26]),
        "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
      : "memory");
}

// One unit of the fused layout pass (see IgemmArgs::lay_*): a thread owns 8 channels x PX
// consecutive pixels: eight 16- or 8-byte loads (one per channel plane), a transpose of the
// binary16 values in registers, PX 16-byte stores (one per pixel).  lane % CH picks the 8-channel
// chunk and lane / CH the pixel group, so a store instruction writes CH*16 contiguous bytes per pixel.
template <int CH, int PX>
struct LayoutUnit {
  static constexpr int PG = 32 / CH;
  static constexpr int W32 = PX / 2;
  uint32_t v[8][W32];
  int64_t out;  // element offset of the thread's first output pixel in x', or -1: nothing to do
  __device__ __forceinline__ void load(const uint16_t* __restrict__ src, int c, int64_t hw, int c_pad, int64_t n, int uc,
                                       int64_t up) {
    const int lane = threadIdx.x & 31;
    const int c8 = lane % CH, pg = lane / CH;
    const int ch = (uc * CH + c8) * 8;
    const int64_t p = (up * PG + pg) * PX;
    out = -1;
    if (ch >= c_pad || p >= hw) return;
    out = (n * hw + p) * c_pad + ch;
    const uint16_t* s = src + (n * c + ch) * hw + p;
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
  }
  __device__ __forceinline__ void store(uint16_t* __restrict__ dst, int c_pad) const {
    if (out < 0) return;
    uint16_t* d = dst + out;
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
};

// The layout warps' loop: global warp `gw` of `nwarps` takes units gw, gw + nwarps, ... of the
// sequence (image, pixel unit, channel unit), channel units fastest, two at a time (all loads of
// both are under way before the first store), and reports each one.
template <int CH, int PX>
__device__ __noinline__ void layout_warp_loop(const uint16_t* __restrict__ src, uint16_t* __restrict__ dst, int c, int hw,
                                              int c_pad, int units_p, int units_c, int seg_units, int segs, int N,
                                              int* flags, int64_t gw, int64_t nwarps) {
  const int64_t total = (int64_t)N * units_p * units_c;
  for (int64_t u = gw; u < total; u += 2 * nwarps) {
    LayoutUnit<CH, PX> a0, a1;
    const int uc0 = (int)(u % units_c);
    const int64_t t0 = u / units_c;
    const int up0 = (int)(t0 % units_p);
    const int64_t n0 = t0 / units_p;
    a0.load(src, c, hw, c_pad, n0, uc0, up0);
    const int64_t u1 = u + nwarps;
    int up1 = 0;
    int64_t n1 = 0;
    if (u1 < total) {
      const int uc1 = (int)(u1 % units_c);
      const int64_t t1 = u1 / units_c;
      up1 = (int)(t1 % units_p);
      n1 = t1 / units_p;
      a1.load(src, c, hw, c_pad, n1, uc1, up1);
    } else {
      a1.out = -1;
    }
    a0.store(dst, c_pad);
    a1.store(dst, c_pad);
    // the stores must be visible to the copy engines of every SM before the units are counted
    asm volatile("fence.proxy.async.global;" ::: "memory");
    __threadfence();
    __syncwarp();
    if ((threadIdx.x & 31) == 0) {
      atomicAdd(flags + n0 * segs + up0 / seg_units, 1);
      if (u1 < total) atomicAdd(flags + n1 * segs + up1 / seg_units, 1);
    }
  }
}

// Waits (bounded) until the pixel segments under input rows [h_lo, h_hi) of images n0 .. n0 + tn - 1
// have been converted.  Whole warp; lane 0 polls.
__device__ __noinline__ bool layout_wait(const int* flags, int N, int plane_h, int plane_w, int seg_px, int seg_units,
                                         int segs, int units_p, int units_c, int n0, int tn, int h_lo, int h_hi,
                                         volatile int* abort_flag) {
  bool ok = true;
  if ((threadIdx.x & 31) == 0) {
    if (h_lo < 0) h_lo = 0;
    if (h_hi > plane_h) h_hi = plane_h;
    if (h_hi > h_lo) {
      const int s_lo = (h_lo * plane_w) / seg_px, s_hi = (h_hi * plane_w - 1) / seg_px;
      for (int img = 0; img < tn && ok; ++img) {
        if (n0 + img >= N) break;
        for (int sgm = s_lo; sgm <= s_hi && ok; ++sgm) {
          const int units_here = units_p - sgm * seg_units < seg_units ? units_p - sgm * seg_units : seg_units;
          const int target = units_here * units_c;
          const int* f = flags + (int64_t)(n0 + img) * segs + sgm;
          uint64_t t0 = 0;
          for (uint32_t spin = 0;; ++spin) {
            int v;
            asm volatile("ld.acquire.gpu.global.b32 %0, [%1];" : "=r"(v) : "l"(f) : "memory");
            if (v >= target) break;
            __nanosleep(64);
            if ((spin & 255u) == 255u) {
              const uint64_t t = global_timer_ns();
              if (t0 == 0) t0 = t;
              if (*abort_flag || t - t0 > g_wait_limit_ns) {
                *abort_flag = 1;
                ok = false;
                break;
              }
            }
          }
        }
      }
    }
    asm volatile("fence.proxy.async.global;" ::: "memory");
  }
  ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
  return ok;
}

// Meeting point of the epilogue warps (one arrival per warp on an mbarrier initialised to their
// number), with a bounded wait: false if it ran out or another role already gave up.  A plain
// named barrier would hang the warps that reach it after others have left on a timeout.
__device__ __forceinline__ bool epi_sync(uint32_t bar, uint32_t& phase, volatile int* abort_flag) {
  __syncwarp();
  if ((threadIdx.x & 31) == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
  const bool ok = mbar_wait(bar, phase, abort_flag, 32);
  phase ^= 1u;
  __syncwarp();
  return ok;
}

// A tile reduced by several CTAs (IgemmArgs::sk_split).  The accumulators travel as fp32 in the
// order [column][128 lanes]: a warp's 32 lanes are 128 contiguous bytes per column.  (Moving them
// with the bulk copy engine through the warp's 4 KB staging tiles was measured slower: two copies
// in flight per warp do not hide their latency.)
// sk_hand_over: this warp's lane quarter of the accumulator -> slot.
__device__ __noinline__ void sk_hand_over(uint32_t t_addr, int quarter, int cols32, float* slot) {
  const int lane = threadIdx.x & 31;
  float* dst = slot + quarter * 32 + lane;
  for (int c = 0; c < cols32; ++c) {
    uint32_t v[32];
    tmem_ld32(t_addr + (uint32_t)(c * 32), v);
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int j = 0; j < 32; ++j) HGC_CHECKED_STORE(dst + (size_t)(c * 32 + j) * 128, __stcg(dst + (size_t)(c * 32 + j) * 128, __uint_as_float(v[j])));
  }
}

// sk_preload: the sum of the slots first_slot, first_slot + slot_step, ... (count of them, in that
// order: the sum does not depend on timing) -> this warp's lane quarter of an accumulator that the
// MMAs of the tile's first part then add to.  A column of a warp is 128 contiguous bytes of a
// slot: one coalesced load per column, 32 in flight.
__device__ __noinline__ void sk_preload(uint32_t t_addr, int quarter, int cols32, const float* slots, size_t slot_elems,
                                        int first_slot, int slot_step, int count) {
  const int lane = threadIdx.x & 31;
  for (int c = 0; c < cols32; ++c) {
    const float* src = slots + (size_t)first_slot * slot_elems + (size_t)c * 32 * 128 + quarter * 32 + lane;
    float v[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) HGC_CHECKED_LOAD(v[j], src + (size_t)j * 128, __ldcg(src + (size_t)j * 128));
    for (int i = 1; i < count; ++i) {
      src += (size_t)slot_step * slot_elems;
      float w[32];
#pragma unroll
      for (int j = 0; j < 32; ++j) HGC_CHECKED_LOAD(w[j], src + (size_t)j * 128, __ldcg(src + (size_t)j * 128));
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] += w[j];
    }
    uint32_t u[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) u[j] = __float_as_uint(v[j]);
    tmem_st32(t_addr + (uint32_t)(c * 32), u);
  }
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

// two fp32 -> packed fp16x2 (round to nearest even), lo = first value; optional ReLU in the convert
template <bool RELU>
__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi) {
  uint32_t d;
  if (RELU)
    asm("cvt.rn.relu.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  else
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}

// `nchunks` (<= 4) chunks of 8 accumulator columns (+ bias, optional ReLU) -> 16-byte fp16 chunks
// at dst0 ^ (chunk << 4) (the swizzled staging row of this lane).  The ReLU choice is a template
// parameter: a run-time test around every convert costs more than the convert.
template <bool RELU>
__device__ __forceinline__ void convert_store(const uint32_t (&v)[32], int nchunks, float bv, uint32_t dst0,
                                              uint32_t chunk0) {
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    if (c < nchunks) {
      uint32_t o[4];
#pragma unroll
      for (int i = 0; i < 4; ++i)
        o[i] = pack_f16x2<RELU>(__uint_as_float(v[8 * c + 2 * i]) + bv, __uint_as_float(v[8 * c + 2 * i + 1]) + bv);
      const uint32_t dst = dst0 ^ ((chunk0 + (uint32_t)c) << 4);
      asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3])
                   : "memory");
    }
  }
}

__device__ __forceinline__ void tma_store_4d(const CUtensorMap* tm, uint32_t src, int c0, int c1, int c2, int c3) {
  asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4, %5}], [%1];" ::"l"(tm),
               "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
               : "memory");
}

// Polls barrier `next_bar` (non-blocking), issues KSTEPS MMAs of one shared-memory stage from one
// elected lane (16 channels per step: +32 bytes = +2 in the descriptors' address field), commits
// them to `a_bar` (and to `b_bar` if release_b), and returns the poll's result.  Warp-collective.
// The poll is issued first and its answer read last, so its latency hides behind the MMA issue.
// PAIR: the MMAs are those of a CTA pair (cta_group::2: 256 output channels, each CTA's tensor
// core reads its own 128 weight rows and both halves of the activation tile) and the commits
// arrive on the barriers at the same offsets in both CTAs.
#define HGC_MMA_FIRST(CG) "@p_mma tcgen05.mma.cta_group::" CG ".kind::f16 [%3], %4, %5, %6, p_acc;\n"
#define HGC_MMA_NEXT(CG)      \
  "add.u64 da, da, 2;\n"      \
  "add.u64 db, db, %12;\n"    \
  "@p_mma tcgen05.mma.cta_group::" CG ".kind::f16 [%3], da, db, %6, p_one;\n"
#define HGC_COMMITS_1                                                                      \
  "@p_el tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%8];\n"    \
  "@p_rel tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%9];\n"
#define HGC_COMMITS_2                                                                                            \
  "@p_el tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%8], cm;\n"   \
  "@p_rel tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%9], cm;\n"
#define HGC_STAGE_HEAD                                                  \
  "{\n"                                                                 \
  ".reg .pred p_next, p_el, p_mma, p_acc, p_one, p_rel;\n"              \
  ".reg .b64 da, db;\n"                                                 \
  ".reg .b16 cm;\n"                                                     \
  "mov.b16 cm, 3;\n"                                                    \
  "mov.b64 da, %4;\n"                                                   \
  "mov.b64 db, %5;\n"                                                   \
  "mbarrier.test_wait.parity.shared::cta.b64 p_next, [%1], %2;\n"       \
  "elect.sync _|p_el, 0xffffffff;\n"                                    \
  "setp.ne.b32 p_mma, %11, 0;\n"                                        \
  "and.pred p_mma, p_mma, p_el;\n"                                      \
  "setp.ne.b32 p_acc, %7, 0;\n"                                         \
  "setp.eq.b32 p_one, 0, 0;\n"                                          \
  "setp.ne.b32 p_rel, %10, 0;\n"                                        \
  "and.pred p_rel, p_rel, p_el;\n"
#define HGC_STAGE_TAIL "selp.u32 %0, 1, 0, p_next;\n}\n"
template <int KSTEPS, bool PAIR>
__device__ __forceinline__ uint32_t issue_stage(uint32_t next_bar, uint32_t next_parity, uint32_t d_tmem,
                                                uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc,
                                                uint32_t a_bar, uint32_t b_bar, uint32_t release_b,
                                                uint32_t do_mma, uint64_t b_step) {
  uint32_t ready;
#define HGC_STAGE_OPERANDS                                                                                   \
  : "=r"(ready)                                                                                              \
  : "r"(next_bar), "r"(next_parity), "r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc), "r"(a_bar), \
    "r"(b_bar), "r"(release_b), "r"(do_mma), "l"(b_step)                                                     \
  : "memory"
  if constexpr (!PAIR) {
    if (KSTEPS == 4) {
      asm volatile(HGC_STAGE_HEAD HGC_MMA_FIRST("1") HGC_MMA_NEXT("1") HGC_MMA_NEXT("1") HGC_MMA_NEXT("1") HGC_COMMITS_1
                       HGC_STAGE_TAIL HGC_STAGE_OPERANDS);
    } else if (KSTEPS == 2) {
      asm volatile(HGC_STAGE_HEAD HGC_MMA_FIRST("1") HGC_MMA_NEXT("1") HGC_COMMITS_1 HGC_STAGE_TAIL HGC_STAGE_OPERANDS);
    } else {
      asm volatile(HGC_STAGE_HEAD HGC_MMA_FIRST("1") HGC_COMMITS_1 HGC_STAGE_TAIL HGC_STAGE_OPERANDS);
    }
  } else {
    if (KSTEPS == 4) {
      asm volatile(HGC_STAGE_HEAD HGC_MMA_FIRST("2") HGC_MMA_NEXT("2") HGC_MMA_NEXT("2") HGC_MMA_NEXT("2") HGC_COMMITS_2
                       HGC_STAGE_TAIL HGC_STAGE_OPERANDS);
    } else if (KSTEPS == 2) {
      asm volatile(HGC_STAGE_HEAD HGC_MMA_FIRST("2") HGC_MMA_NEXT("2") HGC_COMMITS_2 HGC_STAGE_TAIL HGC_STAGE_OPERANDS);
    } else {
      asm volatile(HGC_STAGE_HEAD HGC_MMA_FIRST("2") HGC_COMMITS_2 HGC_STAGE_TAIL HGC_STAGE_OPERANDS);
    }
  }
#undef HGC_STAGE_OPERANDS
  return ready;
}

// KSTEPS MMAs of one weight tile against one activation tile, issued by one elected lane.
#define HGC_MMAS_HEAD                             \
  "{\n"                                           \
  ".reg .pred p_el, p_mma, p_acc, p_one;\n"       \
  ".reg .b64 da, db;\n"                           \
  "mov.b64 da, %1;\n"                             \
  "mov.b64 db, %2;\n"                             \
  "elect.sync _|p_el, 0xffffffff;\n"              \
  "setp.ne.b32 p_mma, %5, 0;\n"                   \
  "and.pred p_mma, p_mma, p_el;\n"                \
  "setp.ne.b32 p_acc, %4, 0;\n"                   \
  "setp.eq.b32 p_one, 0, 0;\n"
#define HGC_MMAS_FIRST(CG) "@p_mma tcgen05.mma.cta_group::" CG ".kind::f16 [%0], %1, %2, %3, p_acc;\n"
#define HGC_MMAS_NEXT(CG)    \
  "add.u64 da, da, 2;\n"     \
  "add.u64 db, db, %6;\n"    \
  "@p_mma tcgen05.mma.cta_group::" CG ".kind::f16 [%0], da, db, %3, p_one;\n"
template <int KSTEPS, bool PAIR>
__device__ __forceinline__ void issue_mmas(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                           uint32_t acc, uint32_t do_mma, uint64_t b_step) {
#define HGC_MMA_OPERANDS ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc), "r"(do_mma), "l"(b_step) : "memory"
  if constexpr (!PAIR) {
    if (KSTEPS == 4) {
      asm volatile(HGC_MMAS_HEAD HGC_MMAS_FIRST("1") HGC_MMAS_NEXT("1") HGC_MMAS_NEXT("1") HGC_MMAS_NEXT("1") "}\n" HGC_MMA_OPERANDS);
    } else if (KSTEPS == 2) {
      asm volatile(HGC_MMAS_HEAD HGC_MMAS_FIRST("1") HGC_MMAS_NEXT("1") "}\n" HGC_MMA_OPERANDS);
    } else {
      asm volatile(HGC_MMAS_HEAD HGC_MMAS_FIRST("1") "}\n" HGC_MMA_OPERANDS);
    }
  } else {
    if (KSTEPS == 4) {
      asm volatile(HGC_MMAS_HEAD HGC_MMAS_FIRST("2") HGC_MMAS_NEXT("2") HGC_MMAS_NEXT("2") HGC_MMAS_NEXT("2") "}\n" HGC_MMA_OPERANDS);
    } else if (KSTEPS == 2) {
      asm volatile(HGC_MMAS_HEAD HGC_MMAS_FIRST("2") HGC_MMAS_NEXT("2") "}\n" HGC_MMA_OPERANDS);
    } else {
      asm volatile(HGC_MMAS_HEAD HGC_MMAS_FIRST("2") "}\n" HGC_MMA_OPERANDS);
    }
  }
#undef HGC_MMA_OPERANDS
}

// Copy epilogue (every shape the TMA-store epilogue does not take: planes whose size is not a
// multiple of 8 pixels, tiles with junk columns between their rows, several images per tile).
// A unit of work is this warp's 32 channels (its TMEM lanes) x up to 64 accumulator columns of
// one image.  The warp converts the unit into its own staging tile in shared memory (32 rows of
// 128 bytes, one per channel, 16-byte chunks XOR-swizzled by the row so that the 16-byte stores
// of 8 lanes fall into 8 different bank groups), then copies it out with the roles turned: a
// lane owns one or two COLUMNS and walks the 32 channel rows, so that every store instruction
// writes consecutive pixels of one channel plane (64 or 128 contiguous bytes).  The two warps
// of a lane quarter take alternate units.  Kept out of line: the hot loops of the kernel should
// stay compact in the instruction cache.
__device__ __noinline__ void epilogue_copy(uint32_t t_addr, uint32_t sbuf, int first_unit, int unit_step, int tn, int th,
                                           int pitch, int N, int K, int P, int Q, int n0, int p0, int k0,
                                           int kvalid_rows, float bv, bool relu, uint16_t* yb) {
  const int lane = threadIdx.x & 31;
  const int64_t pq = (int64_t)P * Q;
  const int rows_valid = (P - p0) < th ? (P - p0) : th;
  const int cols_need = (rows_valid - 1) * pitch + Q;  // columns of one image up to its last real pixel
  const int img_cols = th * pitch;
  // pairs of columns can be copied as 4-byte words when rows (with their junk columns, if any) are
  // an even number of columns long, so that a pair never straddles a row end, and every image's
  // first pixel and every channel plane start on a 4-byte boundary
  const bool words = (Q & 1) == 0 && (pitch & 1) == 0 && (pq & 1) == 0 && ((p0 * Q) & 1) == 0 && (cols_need & 1) == 0;
  const uint32_t row_off = (uint32_t)lane * 128u;
  int unit = 0;
  for (int img = 0; img < tn; ++img) {
    if (n0 + img >= N) break;
    uint16_t* yimg = yb + ((int64_t)(n0 + img) * K + k0) * pq;  // this warp's first channel plane
    for (int c0 = 0; c0 < cols_need; c0 += 64, ++unit) {
      if (unit % unit_step != first_unit) continue;
      const int ncol = cols_need - c0 < 64 ? cols_need - c0 : 64;
      const uint32_t tcol = t_addr + (uint32_t)(img * img_cols + c0);
      // ---- accumulators -> fp16 staging tile (lane = channel) ----
      __syncwarp();  // the previous unit has been copied out
#pragma unroll 1
      for (int g = 0; g < 2; ++g) {
        if (g * 32 >= ncol) break;
        uint32_t v[32];
        if (g * 32 + 32 <= ncol) {
          tmem_ld32(tcol + (uint32_t)(g * 32), v);
        } else {
#pragma unroll
          for (int c = 0; c < 4; ++c)
            if (g * 32 + c * 8 < ncol) tmem_ld8(tcol + (uint32_t)(g * 32 + c * 8), &v[8 * c]);
        }
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        {
          const int nch = (ncol - g * 32 + 7) >> 3;  // chunks with real columns in this batch
          const uint32_t dst0 = sbuf + row_off + (((uint32_t)lane & 7u) << 4);
          if (relu) convert_store<true>(v, nch < 4 ? nch : 4, bv, dst0, (uint32_t)(g * 4));
          else convert_store<false>(v, nch < 4 ? nch : 4, bv, dst0, (uint32_t)(g * 4));
        }
      }
      __syncwarp();
      // ---- staging tile -> y (lane = column) ----
      if (words) {
        const int col = 2 * lane;  // columns col, col + 1 of the unit
        const int cabs = c0 + col;
        const int hr = cabs / pitch;
        const int wc = cabs - hr * pitch;
        if (col < ncol && wc < Q) {  // ncol is even here; junk columns come in pairs too
          uint16_t* dst = yimg + (int64_t)(p0 + hr) * Q + wc;
          const uint32_t chunk = (uint32_t)col >> 3, within = ((uint32_t)col & 7u) * 2u;
#pragma unroll 4
          for (int r = 0; r < kvalid_rows; ++r) {
            uint32_t w;
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(w) : "r"(sbuf + (uint32_t)r * 128u + ((chunk ^ ((uint32_t)r & 7u)) << 4) + within));
            HGC_CHECKED_STORE(reinterpret_cast<uint32_t*>(dst + (int64_t)r * pq), *reinterpret_cast<uint32_t*>(dst + (int64_t)r * pq) = w);
          }
        }
      } else {
#pragma unroll
        for (int hcol = 0; hcol < 2; ++hcol) {
          const int col = lane + 32 * hcol;
          const int cabs = c0 + col;
          const int hr = cabs / pitch;
          const int wc = cabs - hr * pitch;
          if (col < ncol && wc < Q) {
            uint16_t* dst = yimg + (int64_t)(p0 + hr) * Q + wc;
            const uint32_t chunk = (uint32_t)col >> 3, within = ((uint32_t)col & 7u) * 2u;
#pragma unroll 4
            for (int r = 0; r < kvalid_rows; ++r) {
              uint16_t w;
              asm volatile("ld.shared.b16 %0, [%1];" : "=h"(w) : "r"(sbuf + (uint32_t)r * 128u + ((chunk ^ ((uint32_t)r & 7u)) << 4) + within));
              HGC_CHECKED_STORE(dst + (int64_t)r * pq, dst[(int64_t)r * pq] = w);
            }
          }
        }
      }
    }
  }
  __syncwarp();
}

// Epilogue of the inner-product layer (1x1 output plane: a column is an image).  y[n][k] has the
// channels of one image contiguous, so the lanes (channels) of a warp write 64 contiguous bytes
// per column straight from registers.
__device__ __noinline__ void epilogue_columns(uint32_t t_addr, int first_unit, int unit_step, int nimg, int K, int n0,
                                              int k0, int kvalid_rows, float bv, bool relu, uint16_t* yb) {
  const int lane = threadIdx.x & 31;
  for (int c0 = first_unit * 32; c0 < nimg; c0 += unit_step * 32) {
    uint32_t v[32];
    tmem_ld32(t_addr + (uint32_t)c0, v);  // columns past the tile's last image are read and dropped
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
    if (lane < kvalid_rows) {
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        if (c0 + j < nimg) {
          float f = __uint_as_float(v[j]) + bv;
          if (relu) f = fmaxf(f, 0.f);
          HGC_CHECKED_STORE(yb + (int64_t)(n0 + c0 + j) * K + k0 + lane, yb[(int64_t)(n0 + c0 + j) * K + k0 + lane] = __half_as_ushort(__float2half_rn(f)));
        }
      }
    }
  }
  __syncwarp();
}

// Epilogue of a reduction slice: the fp32 accumulators go, unrounded, to this slice's copy of
// the output (same [n][k][p][q] order as y).  Same two-phase scheme as epilogue_copy with 4-byte
// elements: a unit is 32 channels x 32 columns; lane = channel stages its row of 32 floats
// (128 bytes, swizzled), then lane = column walks the 32 rows, so a store instruction writes 32
// consecutive floats of one channel plane.  On a 1x1 plane (inner product) a column is an image
// and the lanes' channels are contiguous: straight from registers.
__device__ __noinline__ void epilogue_partial(uint32_t t_addr, uint32_t sbuf, int first_unit, int unit_step, int tn,
                                              int th, int pitch, int N, int K, int P, int Q, int n0, int p0, int k0,
                                              int kvalid_rows, float* part) {
  const int lane = threadIdx.x & 31;
  const int64_t pq = (int64_t)P * Q;
  if (pq == 1) {
    const int nimg = N - n0 < tn ? N - n0 : tn;
    for (int c0 = first_unit * 32; c0 < nimg; c0 += unit_step * 32) {
      uint32_t v[32];
      tmem_ld32(t_addr + (uint32_t)c0, v);  // columns past the tile's last image are read and dropped
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      if (lane < kvalid_rows) {
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (c0 + j < nimg) HGC_CHECKED_STORE(part + (int64_t)(n0 + c0 + j) * K + k0 + lane, part[(int64_t)(n0 + c0 + j) * K + k0 + lane] = __uint_as_float(v[j]));
      }
    }
    __syncwarp();
    return;
  }
  const int rows_valid = (P - p0) < th ? (P - p0) : th;
  const int cols_need = (rows_valid - 1) * pitch + Q;
  const int img_cols = th * pitch;
  const uint32_t row_off = (uint32_t)lane * 128u;
  int unit = 0;
  for (int img = 0; img < tn; ++img) {
    if (n0 + img >= N) break;
    float* pimg = part + ((int64_t)(n0 + img) * K + k0) * pq;
    for (int c0 = 0; c0 < cols_need; c0 += 32, ++unit) {
      if (unit % unit_step != first_unit) continue;
      const int ncol = cols_need - c0 < 32 ? cols_need - c0 : 32;
      const uint32_t tcol = t_addr + (uint32_t)(img * img_cols + c0);
      __syncwarp();  // the previous unit has been copied out
      uint32_t v[32];
      if (ncol == 32) {
        tmem_ld32(tcol, v);
      } else {
#pragma unroll
        for (int c = 0; c < 4; ++c)
          if (c * 8 < ncol) tmem_ld8(tcol + (uint32_t)(c * 8), &v[8 * c]);
      }
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        if (c * 4 < ncol) {
          const uint32_t dst = sbuf + row_off + ((uint32_t)(c ^ (lane & 7)) << 4);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(v[4 * c]), "r"(v[4 * c + 1]),
                       "r"(v[4 * c + 2]), "r"(v[4 * c + 3])
                       : "memory");
        }
      }
      __syncwarp();
      const int cabs = c0 + lane;
      const int hr = cabs / pitch;
      const int wc = cabs - hr * pitch;
      if (lane < ncol && wc < Q) {
        float* dst = pimg + (int64_t)(p0 + hr) * Q + wc;
        const uint32_t chunk = (uint32_t)lane >> 2, within = ((uint32_t)lane & 3u) * 4u;
#pragma unroll 4
        for (int r = 0; r < kvalid_rows; ++r) {
          uint32_t w;
          asm volatile("ld.shared.b32 %0, [%1];" : "=r"(w) : "r"(sbuf + (uint32_t)r * 128u + ((chunk ^ ((uint32_t)r & 7u)) << 4) + within));
          HGC_CHECKED_STORE(dst + (int64_t)r * pq, dst[(int64_t)r * pq] = __uint_as_float(w));
        }
      }
    }
  }
  __syncwarp();
}

// y = round( relu?( bias[k] + partial[0] + partial[1] + ... ) ): the slices are added in a fixed
// order, so the result does not depend on which CTA finished first
__global__ void __launch_bounds__(256)
splitk_finish_kernel(const float* __restrict__ part, int slices, int64_t stride, const __half* __restrict__ bias,
                     uint16_t* __restrict__ y, int K, int64_t pq, int64_t total, int relu) {
  grid_dependency_wait();
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    float acc = bias != nullptr ? __half2float(__ldg(bias + (int)((i / pq) % K))) : 0.f;
    for (int sidx = 0; sidx < slices; ++sidx) {
      float pv;
      HGC_CHECKED_LOAD(pv, part + sidx * stride + i, __ldcs(part + sidx * stride + i));
      acc += pv;
    }
    if (relu) acc = fmaxf(acc, 0.f);
    HGC_CHECKED_STORE(y + i, y[i] = __half_as_ushort(__float2half_rn(acc)));
  }
}

// Channels-last epilogue (y[N][P][Q][K]): a lane owns a channel, so for every output pixel the 32
// lanes of a warp write 32 consecutive channels (64 contiguous bytes) straight from registers.
// A unit of work is one tile row x up to 32 pixels; the warps of a lane quarter take units in turn.
__device__ __noinline__ void epilogue_nhwc(uint32_t t_addr, int first_unit, int unit_step, int tn, int th, int pitch,
                                           int N, int K, int P, int Q, int n0, int p0, int k, bool kvalid, float bv,
                                           bool relu, uint16_t* yb) {
  const int rows_valid = (P - p0) < th ? (P - p0) : th;
  int unit = 0;
  for (int img = 0; img < tn; ++img) {
    if (n0 + img >= N) break;
    for (int hr = 0; hr < rows_valid; ++hr) {
      for (int wc0 = 0; wc0 < Q; wc0 += 32, ++unit) {
        if (unit % unit_step != first_unit) continue;
        const int ncol = Q - wc0 < 32 ? Q - wc0 : 32;
        const uint32_t tcol = t_addr + (uint32_t)((img * th + hr) * pitch + wc0);
        uint32_t v[32];
        if (ncol == 32) {
          tmem_ld32(tcol, v);
        } else {
#pragma unroll
          for (int c = 0; c < 4; ++c)
            if (c * 8 < ncol) tmem_ld8(tcol + (uint32_t)(c * 8), &v[8 * c]);
        }
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        uint16_t* dst = yb + (((int64_t)(n0 + img) * P + (p0 + hr)) * Q + wc0) * K + k;
#pragma unroll
        for (int j = 0; j < 32; j += 2) {
          if (j < ncol) {
            const float f0 = __uint_as_float(v[j]) + bv, f1 = __uint_as_float(v[j + 1]) + bv;
            const uint32_t o = relu ? pack_f16x2<true>(f0, f1) : pack_f16x2<false>(f0, f1);
            if (kvalid) {
              HGC_CHECKED_STORE(dst + (int64_t)j * K, dst[(int64_t)j * K] = (uint16_t)(o & 0xffffu));
              if (j + 1 < ncol) HGC_CHECKED_STORE(dst + (int64_t)(j + 1) * K, dst[(int64_t)(j + 1) * K] = (uint16_t)(o >> 16));
            }
          }
        }
      }
    }
  }
  __syncwarp();
}

// Channels-last staging: up to 32 accumulator columns (pixels) of this lane's channel -> fp16
// pairs -> a dense [pixel][32 channels] tile in shared memory (64 bytes per pixel).  Each group of
// 8 pixels is four 8x8 matrices (one per pixel pair) spread over the warp's registers; a
// transposing matrix store writes them as 16-byte rows of eight channels of one pixel.  That needs
// the lanes to hold the channels interleaved (lane 4*b + a = channel 8*a + b of the warp's 32),
// which the weight re-layout arranges.  `dst` is this lane's row address for the first 8 pixels:
// lane T addresses pixel 2*(T/8) + T%2, channels 8*((T%8)/2)...
template <bool RELU>
__device__ __forceinline__ void convert_store_pixels(const uint32_t (&v)[32], int npix, float bv, uint32_t dst) {
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    if (c * 8 < npix) {
      const uint32_t o0 = pack_f16x2<RELU>(__uint_as_float(v[8 * c + 0]) + bv, __uint_as_float(v[8 * c + 1]) + bv);
      const uint32_t o1 = pack_f16x2<RELU>(__uint_as_float(v[8 * c + 2]) + bv, __uint_as_float(v[8 * c + 3]) + bv);
      const uint32_t o2 = pack_f16x2<RELU>(__uint_as_float(v[8 * c + 4]) + bv, __uint_as_float(v[8 * c + 5]) + bv);
      const uint32_t o3 = pack_f16x2<RELU>(__uint_as_float(v[8 * c + 6]) + bv, __uint_as_float(v[8 * c + 7]) + bv);
      asm volatile("stmatrix.sync.aligned.m8n8.x4.trans.shared.b16 [%0], {%1, %2, %3, %4};" ::"r"(dst + (uint32_t)c * 512u),
                   "r"(o0), "r"(o1), "r"(o2), "r"(o3)
                   : "memory");
    }
  }
}

struct IgemmArgs {
  int32_t N, K, P, Q;
  int32_t kg, group;
  int32_t R, S, pad_h, pad_w, stride_h, stride_w, dil_h, dil_w;
  int32_t kb;        // channels per reduction block (64 / 32 / 16)
  int32_t cblocks;   // blocks per tap
  int32_t cw;        // channels per tap in w' (cblocks * kb)
  int32_t halo;      // 1: one B load per kernel row r serves its S taps (stride 1); 0: one B load per tap
  int32_t tn, th;    // pixel tile: images x rows (full output width)
  int32_t pitch;     // accumulator columns per output row (Q + (S-1)*dil in halo mode, else Q)
  int32_t ncols;     // MMA N
  int32_t tiles_h;   // row tiles per plane
  int32_t tiles_px;  // pixel tiles in total
  int32_t mtiles;    // 128-channel tiles per group
  int32_t total_tiles;
  int32_t stages;    // ring depth
  int32_t taps;      // weight tiles per stage: S in halo mode, else 1
  uint32_t stage_bytes;
  uint32_t a_bytes, b_bytes, b_alloc;  // TMA bytes of A and B per load, smem reserved per B stage
  uint32_t idesc;
  uint64_t desc_hi;    // shared-memory descriptor bits other than the start address (weights; activations too unless nchw)
  uint64_t desc_hi_b;  // the same for the activation operand
  uint64_t b_kstep;    // address-field increment of the activation descriptor per 16-channel MMA step
  int32_t nchw;        // 1: 1x1 layer reading x as it is (NCHW): pixel-major activation tiles of 64-pixel blocks
  int32_t nblk;        // 64-pixel blocks per activation tile (nchw)
  int32_t cg;          // channels per group (nchw: channel coordinate of the tile)
  int32_t relu;
  int32_t tma_store;  // 1: the epilogue stages fp16 tiles in shared memory and stores them with TMA
  int32_t plane_store;  // 1, 2: whole-plane tiles leave as one bulk copy per 32-channel block (epilogue_planes: its mode)
  uint32_t plane_bytes; //    bytes of a lane quarter's staging tile
  int32_t rem;        // (th*Q) % 64: width of the last staged pass of a full tile (0 = none)
  int32_t nbuf;       // staging tiles per epilogue warp (1 or 2)
  int32_t dup_log2;   // log2 of the number of copies of the layer's rows in a weight tile (0, 1, 2)
  int32_t fine_units; // TMA-store epilogue: units of 32 pixels instead of 64
  int32_t rowpair;    // lanes 64..127 hold the odd output rows of the layer's 64 channels (IgemmPlan::rowpair)
  int32_t nacc;       // depthwise + pointwise blocks: channel tiles (accumulators) per pixel tile: 1, 2 or 4
  // 1x1 layers on planes that start on 8-byte boundaries only: the extra warps gather the
  // pixel-major activation tile from x (NCHW) themselves
  int32_t gather, g_hw, g_c;
  const uint16_t* g_x;
  int32_t mshift;     // log2 of the channel tiles that one work item covers (pairs: 1; nacc: 0, 1, 2)
  int32_t acc_stride; // accumulator columns between the channel tiles of an item (nacc > 1: 512 / nacc)
  // split reduction (its own kernel instantiation): the channel blocks of a tile are dealt out to
  // 2^ks_log2 CTAs, each of which writes its fp32 partial sums to its own slice of `partials`; a
  // second kernel adds the slices in a fixed order (+ bias, ReLU, rounding)
  int32_t ks_log2;
  int64_t part_stride;  // elements between two slices: N * K * P * Q
  int32_t y_tma;        // channels-last output staged for TMA stores (else plain stores)
  int32_t y_full_w;     // pixels of a full channels-last store
  int32_t y_rpu;        // tile rows per channels-last store (rows of at most 32 pixels are batched)
  // Work distribution (kernels without a split reduction): the ring stages of all tiles form one
  // sequence (tile, channel block, kernel row, tap group); CTA i takes a contiguous range of it.
  // sk_split = 0: ranges end on tile boundaries (whole tiles, at most one tile apart between CTAs).
  // sk_split = 1: equal ranges; a tile that straddles a boundary is reduced by two or more CTAs:
  // the CTA that holds the tile's first stage finishes it, the others hand over their fp32
  // accumulators through `sk_part` (one slot per CTA, [column][128 lanes]) and raise `sk_flags`.
  // Layout pass fused into the kernel (its own instantiations): extra warps of every CTA turn
  // x[N][C][HW] into x'[N][HW][c_pad] in global memory, unit by unit in the order the tiles need
  // them (a unit = 32 or 64 channels x 16 to 64 pixels of one image, channel chunks fastest), and
  // count finished units per (image, pixel segment) in lay_flags; a tile's copies start when the
  // segments under its input rows are complete.
  const uint16_t* lay_x;
  uint16_t* lay_xp;
  int* lay_flags;        // [N][lay_segs] counters, then one counter of CTAs that have finished
  int32_t lay_c, lay_cpad, lay_ch, lay_px;  // channels, padded channels, 8-channel chunks per unit (8 / 4), pixels per thread (8 / 4)
  int32_t lay_hw, lay_w;                    // plane size and row width in pixels
  int32_t lay_units_p, lay_units_c;         // units per image along the pixels / along the channels
  int32_t lay_seg_units, lay_segs;          // pixel units per segment, segments per image
  // Depthwise + pointwise block in one kernel (its own instantiations): the layer the kernel sees
  // is the 1x1 convolution; its activation tiles are not fetched but COMPUTED: eight extra warps
  // apply the 3x3 depthwise layer (stride dw_stride, pad 1, + bias, optional ReLU, one rounding to
  // binary16) to the channels-last input dw_x[N][dw_h][dw_w][dw_c] and write the results straight
  // into the ring stages in the swizzled K-major layout the MMA reads.
  const uint16_t* dw_x;
  const uint16_t* dw_w9;   // depthwise weights re-laid-out as [9 taps][dw_c]
  const uint16_t* dw_b;    // depthwise bias [dw_c] or nullptr
  int32_t dw_h, dw_wd, dw_c, dw_stride, dw_relu;
  // its input tiles ([tn][dw_in_h][dw_in_w][KB], fetched by TMA with the zero padding as
  // out-of-bounds fill) alternate between two buffers behind the epilogue's staging tiles
  int32_t dw_in_h, dw_in_w;
  uint32_t dw_in_bytes, dw_in_alloc;
  int32_t dbg_drop;     // test hook: stage of the first CTA whose copies are left out (-1: none)
  int32_t ts;           // ring stages per tile: cblocks * R * (S / taps)
  // CTA pairs (clusters of two, tcgen05 cta_group::2): a tile is 256 output channels x two pixel
  // sub-tiles of tn x th; CTA r of the pair fetches weight rows r*128.. and pixel sub-tile r, its
  // tensor memory receives output channels r*128.. of BOTH sub-tiles (sub-tile j at column
  // j * ncols_sub).  tiles_h / tiles_px then count sub-tiles, total_tiles counts pair tiles.
  int32_t pair;         // 0 / 1 (also the shift between CTA index and work-unit index)
  int32_t ncols_sub;    // accumulator columns of one sub-tile (MMA N = 2 * ncols_sub)
  int32_t sk_split;
  int32_t sk_cols32;    // accumulator columns handed over, in units of 32
  float* sk_part;
  int* sk_flags;
};

// The tiles of one CTA: blockIdx.x, blockIdx.x + gridDim.x, ...  Tile t = (pixel tile px, channel
// tile mg) with mg fastest, px = (image tile, row tile).  The decomposition is kept up to date
// by additions (a handful of divisions once per kernel instead of five per tile and role).
template <bool SPLIT>
struct TileIter {
  int tile, mg, pt, ph;  // current tile, its channel tile, image tile and row tile
  int stride, d_mg, d_pt, d_ph;
  // with a split reduction the slices of a tile are the fastest index
  __device__ __forceinline__ int ks(const IgemmArgs& a) const { return SPLIT ? a.ks_log2 : 0; }
  __device__ __forceinline__ void init(const IgemmArgs& a) {
    const int mgn = (a.mtiles * a.group) << ks(a);
    tile = blockIdx.x;
    const int px = tile / mgn;
    mg = tile - px * mgn;
    pt = px / a.tiles_h;
    ph = px - pt * a.tiles_h;
    stride = gridDim.x;
    const int d_px = stride / mgn;
    d_mg = stride - d_px * mgn;
    d_pt = d_px / a.tiles_h;
    d_ph = d_px - d_pt * a.tiles_h;
  }
  __device__ __forceinline__ bool valid(const IgemmArgs& a) const { return tile < (a.total_tiles << ks(a)); }
  __device__ __forceinline__ void next(const IgemmArgs& a) {
    const int mgn = (a.mtiles * a.group) << ks(a);
    tile += stride;
    mg += d_mg;
    ph += d_ph;
    pt += d_pt;
    if (mg >= mgn) {
      mg -= mgn;
      ++ph;
    }
    if (ph >= a.tiles_h) {
      ph -= a.tiles_h;
      ++pt;
    }
  }
  // group and first output channel (within the group) of the channel tile
  __device__ __forceinline__ void channel_tile(const IgemmArgs& a, int& grp, int& m0) const {
    const int mgc = mg >> ks(a);
    if (a.group == 1) {
      grp = 0;
      m0 = mgc * 128;
    } else {
      grp = mgc / a.mtiles;
      m0 = (mgc - grp * a.mtiles) * 128;
    }
  }
  // reduction slice of this unit and its range of channel blocks
  __device__ __forceinline__ int slice(const IgemmArgs& a) const { return SPLIT ? (mg & ((1 << a.ks_log2) - 1)) : 0; }
  __device__ __forceinline__ void block_range(const IgemmArgs& a, int& cb0, int& cb1) const {
    if (SPLIT) {
      const int sl = slice(a);
      cb0 = (sl * a.cblocks) >> a.ks_log2;
      cb1 = ((sl + 1) * a.cblocks) >> a.ks_log2;
    } else {
      cb0 = 0;
      cb1 = a.cblocks;
    }
  }
  // the same as a range of ring stages of the tile
  __device__ __forceinline__ void stage_range(const IgemmArgs& a, int& s0, int& s1) const {
    int cb0, cb1;
    block_range(a, cb0, cb1);
    const int per_block = a.ts / a.cblocks;
    s0 = cb0 * per_block;
    s1 = cb1 * per_block;
  }
  __device__ __forceinline__ int kind(const IgemmArgs&) const { return 0; }
  __device__ __forceinline__ bool sub_tile(const IgemmArgs&, int, int&, int&) const { return true; }  // (no CTA pairs here)
};

// The work items of one CTA when the stages of all tiles are dealt out as contiguous ranges (see
// IgemmArgs::sk_split): item = (tile, stages [s0, s1) of it).  Only the first item of a CTA can
// start inside a tile and only the last one can end inside a tile.
template <bool SHARED>
struct SegIter {
  int tile, mg, px, pt, ph;  // px: pixel tile (pair of sub-tiles for CTA pairs); pt, ph: its image and row tile (single CTAs)
  int s0, s1;
  int64_t g, g_end;  // shared tiles: position in the global stage sequence, end of this unit's range
  int stride, d_mg, d_px, d_pt, d_ph;  // whole tiles: step between this unit's tiles and its decomposition
  // work units: CTAs, or CTA pairs
  __device__ __forceinline__ static int unit(const IgemmArgs& a) { return (int)blockIdx.x >> a.pair; }
  __device__ __forceinline__ static int units(const IgemmArgs& a) { return (int)gridDim.x >> a.pair; }
  __device__ __forceinline__ static int64_t range_start(const IgemmArgs& a, int u) {
    return (int64_t)a.total_tiles * a.ts * u / units(a);
  }
  // Whole tiles (sk_split = 0): unit u takes tiles u, u + units, ...  Tiles that run at the same
  // time are then neighbours in x and y, which is what the memory system likes (contiguous ranges
  // per CTA measured 10 to 50 % slower on the memory-bound layers).  Shared tiles (sk_split = 1):
  // a contiguous range of the stage sequence, which may begin and end inside a tile.
  __device__ __forceinline__ void init(const IgemmArgs& a) {
    const int mgn = a.mtiles * a.group;
    if constexpr (SHARED) {
      g = range_start(a, unit(a));
      g_end = range_start(a, unit(a) + 1);
      tile = (int)(g / a.ts);
      s0 = (int)(g - (int64_t)tile * a.ts);
      const int64_t left = g_end - g;
      s1 = left < (int64_t)(a.ts - s0) ? s0 + (int)left : a.ts;
      stride = 1;
    } else {
      tile = unit(a);
      stride = units(a);
      s0 = 0;
      s1 = a.ts;
      g = 0;
      g_end = 0;
    }
    px = tile / mgn;
    mg = tile - px * mgn;
    pt = px / a.tiles_h;
    ph = px - pt * a.tiles_h;
    d_px = stride / mgn;
    d_mg = stride - d_px * mgn;
    d_pt = d_px / a.tiles_h;
    d_ph = d_px - d_pt * a.tiles_h;
  }
  __device__ __forceinline__ bool valid(const IgemmArgs& a) const { return SHARED ? g < g_end : tile < a.total_tiles; }
  __device__ __forceinline__ void next(const IgemmArgs& a) {
    if constexpr (SHARED) {
      g += s1 - s0;
      s0 = 0;
      const int64_t left = g_end - g;
      s1 = left < (int64_t)a.ts ? (int)left : a.ts;
    }
    tile += stride;
    mg += d_mg;
    px += d_px;
    ph += d_ph;
    pt += d_pt;
    if (mg >= a.mtiles * a.group) {
      mg -= a.mtiles * a.group;
      ++px;
      ++ph;
    }
    if (ph >= a.tiles_h) {
      ph -= a.tiles_h;
      ++pt;
    }
  }
  // group and first output channel (within the group) of the channel tile (of the pair's 256)
  __device__ __forceinline__ void channel_tile(const IgemmArgs& a, int& grp, int& m0) const {
    if (a.group == 1) {
      grp = 0;
      m0 = (mg * 128) << a.mshift;
    } else {
      grp = mg / a.mtiles;
      m0 = ((mg - grp * a.mtiles) * 128) << a.mshift;
    }
  }
  // first image and output row of pixel sub-tile j of the current pair tile; a pair tile past the
  // last sub-tile gets an image index past the batch (its loads are zero-filled, nothing is stored)
  __device__ __forceinline__ bool sub_tile(const IgemmArgs& a, int j, int& n0, int& p0) const {
    const int sub = 2 * px + j;
    const int spt = sub / a.tiles_h;
    n0 = spt * a.tn;
    p0 = (sub - spt * a.tiles_h) * a.th;
    if (sub < a.tiles_px) return true;
    n0 = a.N;
    p0 = 0;
    return false;
  }
  __device__ __forceinline__ void stage_range(const IgemmArgs& a, int& a0, int& a1) const {
    a0 = SHARED ? s0 : 0;
    a1 = SHARED ? s1 : a.ts;
  }
  // 0: the whole tile; 1: a later part of a tile another CTA finishes (hand the accumulators
  // over); 2: the first part of a tile whose later parts other CTAs computed (add theirs, finish)
  __device__ __forceinline__ int kind(const IgemmArgs& a) const {
    return SHARED ? (s0 > 0 ? 1 : (s1 < a.ts ? 2 : 0)) : 0;
  }
};

template <bool SPLIT, bool SHARED>
struct WorkIterOf { using type = SegIter<SHARED>; };
template <bool SHARED>
struct WorkIterOf<true, SHARED> { using type = TileIter<true>; };

constexpr int kMaxStages = 8;

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// Persistent kernel: each CTA walks tiles blockIdx.x, blockIdx.x + gridDim.x, ...; the two TMEM
// accumulators alternate so that the epilogue of one tile overlaps the MMAs of the next.
// EPI: 0 = TMA-store epilogue, 1 = copy epilogue (NCHW, any shape), 2 = channels-last output,
// 3 = whole-plane tiles sent as bulk copies (NCHW; epilogue_planes)
// Depthwise + pointwise blocks: two horizontally adjacent outputs of the 3x3 depthwise layer
// (stride SD) for 8 channels, from an input tile in shared memory: 3 rows x (SD + 3) columns of
// 16 bytes, `row_bytes` between rows and `px_bytes` between columns; fp32 accumulation.
template <int SD>
__device__ __forceinline__ void dw_pair(uint32_t src0, uint32_t row_bytes, uint32_t px_bytes, const uint32_t (&wv)[9][4],
                                        float (&acc)[2][8]) {
#pragma unroll
  for (int r = 0; r < 3; ++r) {
#pragma unroll
    for (int col = 0; col < SD + 3; ++col) {
      uint32_t u[4];
      asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                   : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3])
                   : "r"(src0 + (uint32_t)r * row_bytes + (uint32_t)col * px_bytes));
      uint16_t xl[4], xh[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) asm("mov.b32 {%0, %1}, %2;" : "=h"(xl[j]), "=h"(xh[j]) : "r"(u[j]));
      if (col < 3) {  // tap (r, col) of the first output
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          uint16_t wl, wh;
          asm("mov.b32 {%0, %1}, %2;" : "=h"(wl), "=h"(wh) : "r"(wv[r * 3 + col][j]));
          asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(acc[0][2 * j]) : "h"(xl[j]), "h"(wl));
          asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(acc[0][2 * j + 1]) : "h"(xh[j]), "h"(wh));
        }
      }
      if (col >= SD) {  // tap (r, col - SD) of the second output
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          uint16_t wl, wh;
          asm("mov.b32 {%0, %1}, %2;" : "=h"(wl), "=h"(wh) : "r"(wv[r * 3 + col - SD][j]));
          asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(acc[1][2 * j]) : "h"(xl[j]), "h"(wl));
          asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(acc[1][2 * j + 1]) : "h"(xh[j]), "h"(wh));
        }
      }
    }
  }
}

// Whole-plane epilogue: tiles that hold whole output planes (of one or several images) of a 1x1
// or strided layer (accumulator columns are the planes' pixels) whose 32-channel blocks are runs of
// 32 * P*Q contiguous, 16-byte aligned halves in y (K % 32 == 0).  The block is built in a staging
// tile that is its memory image ([32 channels][P*Q], a lane writes its channel's row: 8-byte
// stores when P*Q % 4 == 0, which are conflict-free within a half warp, else 2-byte stores) and
// leaves with a single bulk copy.  One image per tile (mode 1): the two warps of a lane quarter
// convert alternate groups of 32 columns into one tile, meet, and one lane sends it.  Several images per tile (mode 2): the warps take alternate images, each with a
// staging tile of its own, and need not meet.  (The copy epilogue's stores, 128 bytes per
// instruction and channel row, cost a 14x14 layer of 1024 output channels 8.9 of its 22.7 us:
// measured with the stores left out.)
// The meetings are on an mbarrier of the quarter with a bounded wait (a named barrier would hang a
// warp whose partner has left on a timeout); returns the barrier's next phase, or ~0 after giving up.
__device__ __noinline__ uint32_t epilogue_planes(uint32_t t_addr, uint32_t qstage, int half, int mode, int tn, int N, int K, int pq,
                                                 int n0, int k0, float bv, bool relu, uint16_t* yb, uint32_t qbar, uint32_t phase,
                                                 volatile int* abort_flag) {
  const int lane = threadIdx.x & 31;
  const bool shared_tile = mode == 1;
  const uint32_t tile_bytes = (uint32_t)(((32 * pq * 2) + 127) & ~127);
  const uint32_t tile = shared_tile ? qstage : qstage + (uint32_t)half * tile_bytes;
  const uint32_t row = tile + (uint32_t)lane * (uint32_t)(pq * 2);
  const bool wide = (pq & 3) == 0;
  const bool sender = lane == 0 && (half == 0 || !shared_tile);
  for (int img = shared_tile ? 0 : half; img < tn; img += shared_tile ? 1 : 2) {
    if (n0 + img >= N) break;
    // the staging tile's previous copy must have read it
    if (sender) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
    if (shared_tile) {
      if (!epi_sync(qbar, phase, abort_flag)) return ~0u;
    } else {
      __syncwarp();
    }
    for (int c0 = shared_tile ? half * 32 : 0; c0 < pq; c0 += shared_tile ? 64 : 32) {
      const int ncol = pq - c0 < 32 ? pq - c0 : 32;
      const uint32_t tcol = t_addr + (uint32_t)(img * pq + c0);
      uint32_t v[32];
      if (ncol == 32) {
        tmem_ld32(tcol, v);
      } else {
#pragma unroll
        for (int c = 0; c < 4; ++c)
          if (c * 8 < ncol) tmem_ld8(tcol + (uint32_t)(c * 8), &v[8 * c]);
      }
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      if (wide) {  // (ncol is a multiple of 4)
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (4 * j < ncol) {
            const float f0 = __uint_as_float(v[4 * j]) + bv, f1 = __uint_as_float(v[4 * j + 1]) + bv;
            const float f2 = __uint_as_float(v[4 * j + 2]) + bv, f3 = __uint_as_float(v[4 * j + 3]) + bv;
            const uint32_t o0 = relu ? pack_f16x2<true>(f0, f1) : pack_f16x2<false>(f0, f1);
            const uint32_t o1 = relu ? pack_f16x2<true>(f2, f3) : pack_f16x2<false>(f2, f3);
            asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(row + (uint32_t)((c0 + 4 * j) * 2)), "r"(o0), "r"(o1) : "memory");
          }
        }
      } else {  // rows of the tile start on 2-byte boundaries (7x7 planes: 98 bytes)
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          if (2 * j < ncol) {
            const float f0 = __uint_as_float(v[2 * j]) + bv, f1 = __uint_as_float(v[2 * j + 1]) + bv;
            const uint32_t o = relu ? pack_f16x2<true>(f0, f1) : pack_f16x2<false>(f0, f1);
            asm volatile("st.shared.b16 [%0], %1;" ::"r"(row + (uint32_t)((c0 + 2 * j) * 2)), "h"((uint16_t)(o & 0xffffu)) : "memory");
            if (2 * j + 1 < ncol)
              asm volatile("st.shared.b16 [%0], %1;" ::"r"(row + (uint32_t)((c0 + 2 * j + 1) * 2)), "h"((uint16_t)(o >> 16)) : "memory");
          }
        }
      }
    }
    // the copy engine reads the tile through the async proxy
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (shared_tile) {
      if (!epi_sync(qbar, phase, abort_flag)) return ~0u;
    } else {
      __syncwarp();
    }
    if (sender) {
      uint16_t* dst = yb + ((int64_t)(n0 + img) * K + k0) * pq;
      const uint32_t bytes = (uint32_t)(32 * pq * 2);
      if (HGC_ADDR_OK(dst, bytes)) {
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(tile), "r"(bytes) : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
      }
    }
  }
  return phase;
}

constexpr int kLayoutWarps = 8;  // extra warps of the instantiations with the fused layout pass
constexpr int kDwWarps = 8;      // extra warps of the depthwise + pointwise instantiations

template <int KB, bool HALO, int EW, int EPI, bool SPLIT, bool PAIR = false, bool SHARED = false, bool FUSEL = false,
          bool DWPW = false>
__global__ void __launch_bounds__(64 + 32 * EW + (FUSEL ? 32 * kLayoutWarps : 0) + (DWPW ? 32 * kDwWarps : 0), 1)
igemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
             const __grid_constant__ CUtensorMap tmY, const __grid_constant__ CUtensorMap tmYr,
             const IgemmArgs a, const __half* __restrict__ bias, __half* __restrict__ y, float* __restrict__ partials,
             int* status) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[kMaxStages], empty_bar[kMaxStages];
  __shared__ __align__(8) uint64_t acc_full[2], acc_empty[2];
  __shared__ uint32_t tmem_slot;
  __shared__ volatile int abort_flag;
  __shared__ __align__(8) uint64_t sk_bar;    // shared tiles: the partial sums of the unit's last tile are in its accumulator
  __shared__ __align__(8) uint64_t meet_bar;  // shared tiles: meeting point of all epilogue warps,
  __shared__ __align__(8) uint64_t ho_bar;    //   of the warps that hand accumulators over (the first of each lane quarter),
  __shared__ __align__(8) uint64_t pl_bar;    //   of the warps that fetch partial sums (the second of each lane quarter)
  __shared__ __align__(8) uint64_t in_full[2], in_empty[2];  // depthwise input tiles (depthwise + pointwise blocks)
  __shared__ __align__(8) uint64_t q_bar[4];  // whole-plane epilogue: meeting point of the two warps of a lane quarter

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  // ring of stages; a stage holds one activation tile followed by `taps` weight tiles
  const uint32_t ring_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  // CTA pairs: rank 0 issues the MMAs of both and owns the barriers the two producers and the two
  // epilogues report to
  uint32_t rank = 0;
  if constexpr (PAIR) asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));

  if (threadIdx.x == 0) {
    for (int s = 0; s < a.stages; ++s) {
      // (the weight copy + one arrival per depthwise / gathering warp)
      mbar_init(smem_u32(&full_bar[s]), DWPW ? 1 + kDwWarps : 1);
      mbar_init(smem_u32(&empty_bar[s]), 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(smem_u32(&acc_full[s]), 1);
      mbar_init(smem_u32(&acc_empty[s]), PAIR ? 2 * EW : EW);  // one arrival per epilogue warp (of both CTAs)
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&in_full[b]), 1);
      mbar_init(smem_u32(&in_empty[b]), kDwWarps);
    }
    mbar_init(smem_u32(&sk_bar), PAIR ? EW : EW / 2);  // one arrival per fetching warp (of both CTAs)
    for (int q = 0; q < 4; ++q) mbar_init(smem_u32(&q_bar[q]), EW / 4);
    mbar_init(smem_u32(&meet_bar), EW);
    mbar_init(smem_u32(&ho_bar), EW / 2);
    mbar_init(smem_u32(&pl_bar), EW / 2);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    // the whole TMEM (512 columns): the kernel's shared-memory request keeps it alone on the SM
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                 "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  if constexpr (PAIR) cluster_sync_all();  // the partner's barriers must exist before anything arrives on them
  else __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = tmem_slot;

  // everything above touched only this CTA's shared and tensor memory and may overlap the tail of
  // the previous kernel in the stream; from here on global memory is read and written
  grid_dependency_wait();
  grid_launch_dependents();
  // an earlier CTA gave up: do not start new work on a path that is not progressing
  const bool skip = status != nullptr && *reinterpret_cast<volatile int*>(status) != 0;

  if (skip) {
    // fall through to the release of the tensor memory
  } else if (warp == 0) {
    // ---------------- TMA producer ----------------
    // The whole warp walks the loop (warp-uniform control flow keeps addresses, coordinates and
    // barrier operands in uniform registers); one elected lane issues the copies.  A stage is
    // the activation tile of one kernel row (or one tap when taps cannot share it) plus the
    // weight tiles of its `taps` taps, all completing on one barrier: the MMA warp then pays the
    // barrier handshake once per taps*KB/16 MMAs.
    Ring ring;
    uint32_t issued = 0;
    bool ok = true;
    const uint32_t depth = (uint32_t)a.stages;
    const int groups_per_row = a.S / a.taps;  // 1 in halo mode (taps == S), S otherwise (taps == 1)
    typename WorkIterOf<SPLIT, SHARED>::type it;
    const int stages_per_block = a.R * groups_per_row;
    for (it.init(a); it.valid(a) && ok; it.next(a)) {
      int grp, m0;
      it.channel_tile(a, grp, m0);
      int n0 = it.pt * a.tn;
      int p0 = it.ph * a.th;
      if constexpr (PAIR) {  // this CTA's half of the pair tile: weight rows and pixel sub-tile `rank`
        m0 += (int)rank * 128;
        it.sub_tile(a, (int)rank, n0, p0);
      }
      const int h_base = p0 * a.stride_h - a.pad_h;
      int s0, s1;
      it.stage_range(a, s0, s1);
      if constexpr (FUSEL) {
        // the tile reads input rows h_base .. h_base + (th-1)*stride + (R-1)*dil of tn images
        if (!layout_wait(a.lay_flags, a.N, a.lay_hw / a.lay_w, a.lay_w, a.lay_seg_units * (32 / a.lay_ch) * a.lay_px,
                         a.lay_seg_units, a.lay_segs, a.lay_units_p, a.lay_units_c, n0, a.tn, h_base,
                         h_base + (a.th - 1) * a.stride_h + (a.R - 1) * a.dil_h + 1, &abort_flag)) {
          ok = false;
          break;
        }
      }
      // stage s of a tile = (channel block cb, kernel row r, tap group sg), sg fastest
      int cb = 0, r = 0, sg = 0;
      if (SHARED || SPLIT) {  // (whole tiles start at stage 0)
        cb = s0 / stages_per_block;
        r = (s0 - cb * stages_per_block) / groups_per_row;
        sg = s0 - cb * stages_per_block - r * groups_per_row;
      }
      int tap0 = (r * groups_per_row + sg) * a.taps;  // first tap (r*S + s) of the stage
      for (int st = s0; st < s1; ++st) {
        if (!mbar_wait(smem_u32(&empty_bar[ring.idx]), ring.phase ^ 1u, &abort_flag, 64)) {
          ok = false;
          break;
        }
        const uint32_t sbase = ring_base + ring.idx * a.stage_bytes;
        // test hook: the first CTA announces the bytes of its `dbg_drop`-th stage but never fetches
        // them, so that the wait for that stage runs out (hgc_debug_drop_copies)
        const bool drop = a.dbg_drop >= 0 && blockIdx.x == 0 && issued == (uint32_t)a.dbg_drop;
        if (drop) {
          if (lane == 0) mbar_expect_tx(smem_u32(&full_bar[ring.idx]), (PAIR ? 2u : 1u) * (a.b_bytes + (uint32_t)((DWPW ? a.nacc : 1) * a.taps) * a.a_bytes));
        } else if constexpr (DWPW) {
          // the activation tile of the stage is computed by the depthwise warps from an input tile
          // (with its one-pixel border) that is fetched here, beside the pointwise weights
          const uint32_t fb = smem_u32(&full_bar[ring.idx]);
          // the weight tiles of the item's channel tiles (one per accumulator), behind one another
          if (lane == 0) mbar_expect_tx(fb, (uint32_t)(a.nacc * a.taps) * a.a_bytes);
          __syncwarp();
          if (lane < a.nacc)
            tma_load_4d(sbase + a.b_alloc + (uint32_t)(lane * a.taps) * a.a_bytes, &tmA, fb, cb * KB, m0 + lane * 128, tap0, grp);
          const uint32_t ib = issued & 1u;
          if (!a.gather && !mbar_wait(smem_u32(&in_empty[ib]), ((issued >> 1) & 1u) ^ 1u, &abort_flag, 64)) {
            ok = false;
            break;
          }
          if (lane == 0 && !a.gather) {
            const uint32_t in_base = ring_base + (uint32_t)a.stages * a.stage_bytes + (uint32_t)(EW * a.nbuf) * kWarpStageBytes;
            mbar_expect_tx(smem_u32(&in_full[ib]), a.dw_in_bytes);
            tma_load_5d(in_base + ib * a.dw_in_alloc, &tmB, smem_u32(&in_full[ib]), cb * KB, 0, -1, p0 * a.dw_stride - 1, n0);
          }
        } else if constexpr (PAIR) {
          // both CTAs' copies are counted on the first CTA's barrier, which expects the bytes of both
          const uint32_t fb = cluster_addr(smem_u32(&full_bar[ring.idx]), 0);
          if (lane == 0 && rank == 0)
            mbar_expect_tx(smem_u32(&full_bar[ring.idx]), 2u * (a.b_bytes + (uint32_t)a.taps * a.a_bytes));
          if (lane == 0)
            tma_load_5d_pair(sbase, &tmB, fb, cb * KB, grp, (HALO ? 0 : sg * a.dil_w) - a.pad_w, h_base + r * a.dil_h, n0);
          if (lane == 8) tma_load_4d_pair(sbase + a.b_alloc, &tmA, fb, cb * KB, m0, tap0, grp);
        } else {
        const uint32_t fb = smem_u32(&full_bar[ring.idx]);
        // A thread gets a bulk-tensor copy under way only every few hundred clocks, whatever its
        // size (measured), so a stage is few, large copies issued by different lanes at once:
        // lane 0 announces the bytes and fetches the activation tile, lane 8 fetches the weight
        // tiles of all taps of the stage as one box (the 1x1 mode's 64-pixel blocks: one lane each).
        if (lane == 0) mbar_expect_tx(fb, a.b_bytes + (uint32_t)a.taps * a.a_bytes);
        if (a.nchw) {
          // x itself, (pixel, channel, image): blocks of 64 pixels x KB channels, pixels contiguous
          if (lane < a.nblk)
            tma_load_3d(sbase + (uint32_t)lane * (uint32_t)(KB * 128), &tmB, fb, p0 * a.Q + 64 * lane,
                        grp * a.cg + cb * KB, n0);
        } else if (lane == 0) {
          tma_load_5d(sbase, &tmB, fb, cb * KB, grp, (HALO ? 0 : sg * a.dil_w) - a.pad_w, h_base + r * a.dil_h, n0);
        }
        if (lane == 8) tma_load_4d(sbase + a.b_alloc, &tmA, fb, cb * KB, m0, tap0, grp);
        }
        __syncwarp();
        tap0 += a.taps;
        if (++sg == groups_per_row) {
          sg = 0;
          if (++r == a.R) {
            r = 0;
            ++cb;
            tap0 = 0;
          }
        }
        ring.advance(depth);
        ++issued;
      }
    }
    if (PAIR && rank != 0) {
      // (its copies are counted on the partner's barriers: after giving up it just waits a while)
      if (abort_flag && lane == 0) {
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 2000000ull) __nanosleep(1000);
      }
    } else if (abort_flag && lane == 0) {
      // let the copies that were issued land before the CTA's shared memory goes away
      const uint32_t first = issued > depth ? issued - depth : 0;
      for (uint32_t it = first; it < issued; ++it) {
        const uint32_t bar = smem_u32(&full_bar[it % depth]);
        const uint64_t t0 = global_timer_ns();
        while (!mbar_try_wait(bar, (it / depth) & 1u)) {
          if (global_timer_ns() - t0 > g_wait_limit_ns) break;
        }
      }
    }
    __syncwarp();
  } else if (warp == 1 && (!PAIR || rank == 0)) {
    // ---------------- MMA issuer (of a pair: the first CTA's, for both) ----------------
    // Warp-uniform loop; one elected lane issues tcgen05.mma and tcgen05.commit (always the same
    // lane: a commit tracks the MMAs of the thread that executes it).
    Ring ring;
    uint32_t lt = 0;
    bool ok = true;
    constexpr int ksteps = KB / 16;
    constexpr uint32_t row_bytes = (uint32_t)KB * 2u;
    const uint32_t depth = (uint32_t)a.stages;
    const uint32_t tap_step = (uint32_t)a.dil_w * row_bytes;  // halo mode: tap s starts s*dil pixels in
    const uint64_t desc_hi = a.desc_hi;
    const uint32_t idesc = a.idesc;
    const uint32_t do_mma = 1u;
    uint32_t ready = mbar_test_wait(smem_u32(&full_bar[0]), 0u);
    typename WorkIterOf<SPLIT, SHARED>::type it;
    for (it.init(a); it.valid(a) && ok; it.next(a), ++lt) {  // only the number of stages of an item matters here
      int s0, s1;
      it.stage_range(a, s0, s1);
      const int groups_per_tile = s1 - s0;
      // two accumulators take turns; a block kernel with several channel tiles per pixel tile has
      // one set of them, which the epilogue must have drained before the next tile starts
      const bool one_set = DWPW && a.nacc > 1;
      const uint32_t buf = one_set ? 0u : (lt & 1u);
      // the epilogue must have drained this accumulator (two tiles ago)
      if (!mbar_wait(smem_u32(&acc_empty[buf]), ((one_set ? lt : (lt >> 1)) & 1u) ^ 1u, &abort_flag, 64)) {
        ok = false;
        break;
      }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t d_tmem = tmem_base + buf * 256u;
      uint32_t acc = 0;
      if constexpr (!SPLIT && SHARED) {
        if (it.kind(a) == 2) {
          // the first part of a tile whose later parts other units computed: the epilogue warps
          // have put the sum of those parts into the accumulator (see there); add to it
          if (!mbar_wait(smem_u32(&sk_bar), 0u, &abort_flag, 64)) {
            ok = false;
            break;
          }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          acc = 1;
        }
      }
      for (int gi = 0; gi < groups_per_tile; ++gi) {
        if (!ready && !mbar_wait(smem_u32(&full_bar[ring.idx]), ring.phase, &abort_flag)) {
          ok = false;
          break;
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t sbase = ring_base + ring.idx * a.stage_bytes;
        const uint32_t e_bar = smem_u32(&empty_bar[ring.idx]);
        uint64_t bdesc = a.desc_hi_b | (uint64_t)((sbase & 0x3FFFFu) >> 4);
        uint64_t adesc = desc_hi | (uint64_t)(((sbase + a.b_alloc) & 0x3FFFFu) >> 4);
        ring.advance(depth);
        if constexpr (DWPW) {
          // further channel tiles of the item: the same activation tile against their weight tiles
          for (int ci = 0; ci + 1 < a.nacc; ++ci) {
            issue_mmas<ksteps, PAIR>(d_tmem + (uint32_t)(ci * a.acc_stride), adesc, bdesc, idesc, acc, do_mma, a.b_kstep);
            adesc += (uint64_t)(((uint32_t)a.taps * a.a_bytes) >> 4);
          }
        }
        const uint32_t d_last = DWPW ? d_tmem + (uint32_t)((a.nacc - 1) * a.acc_stride) : d_tmem;
        // all taps but the last: MMAs only
        for (int t = 0; t + 1 < a.taps; ++t) {
          issue_mmas<ksteps, PAIR>(d_last, adesc, bdesc, idesc, acc, do_mma, a.b_kstep);
          acc = 1;
          adesc += (uint64_t)(a.a_bytes >> 4);
          bdesc += (uint64_t)(tap_step >> 4);
        }
        // last tap: poll the NEXT stage's barrier first and read the answer after the MMAs and the
        // commit have been issued, so that the poll's latency hides behind them
        ready = issue_stage<ksteps, PAIR>(smem_u32(&full_bar[ring.idx]), ring.phase, d_last, adesc, bdesc, idesc, acc, e_bar,
                                    e_bar, 0u, do_mma, a.b_kstep);
        acc = 1;
      }
      if (ok) {
        if (elect_one()) {  // accumulator complete
          if constexpr (PAIR) umma_commit_pair(smem_u32(&acc_full[buf]));
          else umma_commit(smem_u32(&acc_full[buf]));
        }
        __syncwarp();
      }
    }
  } else if (DWPW && warp >= 2 + EW) {
    // ---------------- depthwise warps: compute the activation tiles of the 1x1 layer ----------------
    // A stage holds [pixel of the tile][KB channels], 16-byte chunks of 8 channels swizzled by the
    // pixel row as the copy engine would have written them.  The input tile of the stage lies in
    // shared memory as [image][row][column][KB] with a zero border.  Thread dt owns chunk
    // dt % (KB/8) of every (256 / (KB/8))-th pair of horizontally adjacent output pixels: the pair
    // shares its input columns (3 rows x 4 or 5 columns of 16 bytes for two outputs), and the
    // threads of a warp read consecutive chunks: no bank conflicts.
    constexpr int CPR = KB / 8;                     // chunks per pixel
    constexpr int PASS = kDwWarps * 32 / CPR;       // pairs per pass of the 256 threads
    const int dt = (warp - 2 - EW) * 32 + lane;
    const int chunk = dt % CPR;
    const int slot = dt / CPR;
    Ring ring;
    uint32_t produced = 0;
    bool ok = true;
    const uint32_t depth = (uint32_t)a.stages;
    const int pairs_per_row = (a.Q + 1) >> 1;
    const int pairs_total = a.tn * a.th * pairs_per_row;
    const int sd = a.dw_stride;
    const uint32_t in_base = ring_base + (uint32_t)a.stages * a.stage_bytes + (uint32_t)(EW * a.nbuf) * kWarpStageBytes;
    typename WorkIterOf<SPLIT, SHARED>::type it;
    if (a.gather) {
      // ---- 1x1 layer on NCHW planes of a multiple of 4 pixels: the stage is the pixel-major tile
      // [64-pixel block][KB channel rows of 128 bytes], 128-byte swizzle, as the copy engine writes
      // it for planes it can address.  The KB planes of a stage follow one another in x, so the
      // stage is one contiguous run of 8-byte pieces (4 pixels of a channel); a thread copies every
      // 256th of them with cp.async.  Where a piece goes does not depend on the stage: the offsets
      // are computed once.  Up to three stages' copies are in flight; the oldest is waited for,
      // made visible to the tensor core's proxy and reported on its barrier.
      constexpr int kMaxPieces = 16;                      // per thread: KB * 64 pieces at most (planes of <= 256 pixels)
      const int pieces_pc = a.g_hw >> 2;                 // pieces per channel
      const int pieces = KB * pieces_pc;                  // per stage
      uint32_t doff[kMaxPieces];
#pragma unroll
      for (int i = 0; i < kMaxPieces; ++i) {
        const int pc = dt + i * (kDwWarps * 32);
        const int cl = pc / pieces_pc, px = (pc - cl * pieces_pc) << 2;  // channel row, first pixel of the piece
        doff[i] = (uint32_t)(px >> 6) * (uint32_t)(KB * 128) + (uint32_t)cl * 128u +
                  (((uint32_t)((px & 63) >> 3) ^ ((uint32_t)cl & 7u)) << 4) + (uint32_t)(px & 4) * 2u;
      }
      // stages whose copies are in flight, oldest first (at most depth - 1, and at most 3)
      const int max_fly = (int)depth - 1 < 3 ? (int)depth - 1 : 3;
      int fly_idx[3] = {0, 0, 0};
      int fly = 0;
      auto retire_oldest = [&]() {  // wait for the oldest stage's copies, publish it, report it
        if (fly == 3) asm volatile("cp.async.wait_group 2;" ::: "memory");
        else if (fly == 2) asm volatile("cp.async.wait_group 1;" ::: "memory");
        else asm volatile("cp.async.wait_group 0;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&full_bar[fly_idx[0]]));
        fly_idx[0] = fly_idx[1];
        fly_idx[1] = fly_idx[2];
        --fly;
      };
      for (it.init(a); it.valid(a) && ok; it.next(a)) {
        const int n0 = it.pt * a.tn;
        for (int cb = 0; cb < a.cblocks && ok; ++cb) {
          if (fly == max_fly) retire_oldest();
          if (!mbar_wait(smem_u32(&empty_bar[ring.idx]), ring.phase ^ 1u, &abort_flag, 32)) {
            ok = false;
            break;
          }
          const uint32_t sbase = ring_base + ring.idx * a.stage_bytes;
          const uint16_t* src = a.g_x + ((int64_t)n0 * a.g_c + (int64_t)cb * KB) * a.g_hw + (int64_t)dt * 4;
#pragma unroll
          for (int i = 0; i < kMaxPieces; ++i) {
            if (dt + i * (kDwWarps * 32) < pieces) {
              const uint16_t* sp = src + (int64_t)i * (kDwWarps * 32 * 4);
              if (HGC_ADDR_OK(sp, 8))
                asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(sbase + doff[i]), "l"(sp) : "memory");
            }
          }
          asm volatile("cp.async.commit_group;" ::: "memory");
          fly_idx[fly++] = (int)ring.idx;
          ring.advance(depth);
        }
      }
      if (ok) {
        while (fly > 0) retire_oldest();
      } else {
        asm volatile("cp.async.wait_group 0;" ::: "memory");
      }
    } else
    for (it.init(a); it.valid(a) && ok; it.next(a)) {
      for (int cb = 0; cb < a.cblocks && ok; ++cb, ++produced) {
        const int c0 = cb * KB + chunk * 8;
        const bool cvalid = c0 < a.dw_c;            // (dw_c is a multiple of 8)
        // this thread's 8 channels: the nine taps' weights (packed pairs) and the bias
        uint32_t wv[9][4];
        float bv[8];
#pragma unroll
        for (int t = 0; t < 9; ++t) {
          const uint4 q = cvalid ? __ldg(reinterpret_cast<const uint4*>(a.dw_w9 + (int64_t)t * a.dw_c + c0)) : make_uint4(0, 0, 0, 0);
          wv[t][0] = q.x; wv[t][1] = q.y; wv[t][2] = q.z; wv[t][3] = q.w;
        }
        {
          const uint4 q = (cvalid && a.dw_b != nullptr) ? __ldg(reinterpret_cast<const uint4*>(a.dw_b + c0)) : make_uint4(0, 0, 0, 0);
          const uint32_t u[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            bv[2 * j] = __half2float(__ushort_as_half((uint16_t)(u[j] & 0xffffu)));
            bv[2 * j + 1] = __half2float(__ushort_as_half((uint16_t)(u[j] >> 16)));
          }
        }
        const uint32_t ib = produced & 1u;
        if (!mbar_wait(smem_u32(&in_full[ib]), (produced >> 1) & 1u, &abort_flag, 32) ||
            !mbar_wait(smem_u32(&empty_bar[ring.idx]), ring.phase ^ 1u, &abort_flag, 32)) {
          ok = false;
          break;
        }
        const uint32_t sbase = ring_base + ring.idx * a.stage_bytes;
        const uint32_t tile_in = in_base + ib * a.dw_in_alloc + (uint32_t)chunk * 16u;
        for (int pr = slot; pr < pairs_total; pr += PASS) {
          const int rowi = pr / pairs_per_row;               // (image, output row) of the tile
          const int wc = (pr - rowi * pairs_per_row) * 2;    // first output column of the pair
          const int img = rowi / a.th, hr = rowi - img * a.th;
          float acc[2][8];
#pragma unroll
          for (int j = 0; j < 8; ++j) acc[0][j] = acc[1][j] = bv[j];
          const uint32_t src0 = tile_in + (uint32_t)(((img * a.dw_in_h + hr * sd) * a.dw_in_w + wc * sd) * (KB * 2));
          if (sd == 1) dw_pair<1>(src0, (uint32_t)(a.dw_in_w * KB * 2), (uint32_t)(KB * 2), wv, acc);
          else dw_pair<2>(src0, (uint32_t)(a.dw_in_w * KB * 2), (uint32_t)(KB * 2), wv, acc);
          const int row = rowi * a.Q + wc;                   // row of the stage = accumulator column
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            if (wc + e < a.Q) {
              uint32_t o[4];
#pragma unroll
              for (int j = 0; j < 4; ++j)
                o[j] = a.dw_relu ? pack_f16x2<true>(acc[e][2 * j], acc[e][2 * j + 1]) : pack_f16x2<false>(acc[e][2 * j], acc[e][2 * j + 1]);
              // row of KB*2 bytes; the swizzle of the copy engine XORs the 16-byte chunk index with
              // address bits 7..9 (128-byte rows: the row index; 64-byte rows: the row index / 2)
              const uint32_t rr = (uint32_t)(row + e);
              const uint32_t sw = KB == 64 ? (rr & 7u) : ((rr >> 1) & 3u);
              const uint32_t dst = sbase + rr * (uint32_t)(KB * 2) + (((uint32_t)chunk ^ sw) << 4);
              asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3])
                           : "memory");
            }
          }
        }
        // the tensor core reads the stage through the async proxy
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(smem_u32(&full_bar[ring.idx]));
          mbar_arrive(smem_u32(&in_empty[ib]));   // (this warp has read its part of the input tile)
        }
        ring.advance(depth);
      }
    }
  } else if (FUSEL && warp >= 2 + EW) {
    // ---------------- fused layout pass (warps past the epilogue's) ----------------
    const int64_t gw = (int64_t)blockIdx.x * kLayoutWarps + (warp - 2 - EW);
    const int64_t nw = (int64_t)gridDim.x * kLayoutWarps;
    if (a.lay_ch == 8 && a.lay_px == 8)
      layout_warp_loop<8, 8>(a.lay_x, a.lay_xp, a.lay_c, a.lay_hw, a.lay_cpad, a.lay_units_p, a.lay_units_c, a.lay_seg_units,
                             a.lay_segs, a.N, a.lay_flags, gw, nw);
    else if (a.lay_px == 8)
      layout_warp_loop<4, 8>(a.lay_x, a.lay_xp, a.lay_c, a.lay_hw, a.lay_cpad, a.lay_units_p, a.lay_units_c, a.lay_seg_units,
                             a.lay_segs, a.N, a.lay_flags, gw, nw);
    else if (a.lay_ch == 8)
      layout_warp_loop<8, 4>(a.lay_x, a.lay_xp, a.lay_c, a.lay_hw, a.lay_cpad, a.lay_units_p, a.lay_units_c, a.lay_seg_units,
                             a.lay_segs, a.N, a.lay_flags, gw, nw);
    else
      layout_warp_loop<4, 4>(a.lay_x, a.lay_xp, a.lay_c, a.lay_hw, a.lay_cpad, a.lay_units_p, a.lay_units_c, a.lay_seg_units,
                             a.lay_segs, a.N, a.lay_flags, gw, nw);
  } else if (warp >= 2 && warp < 2 + EW) {
    // ---------------- epilogue (warps 2..9) ----------------
    // Warp w may read TMEM lanes 32*(w%4)..+31; the EW/4 warps of a lane quarter take the units of
    // a tile in turn.
    constexpr int kPerQuarter = EW / 4;
    const int ew = warp - 2;
    const int quarter = warp & 3;
    const int half = ew >> 2;  // which of the quarter's warps this is
    // accumulator lane = output channel within the tile (interleaved within the warp's 32 when the
    // staged channels-last epilogue runs: see convert_store_pixels)
    // Replicated weight rows (layers of 64 or 32 output channels, TMA-store epilogue): lane
    // quarters 2 and 3 (1, 2 and 3) hold the same channels as quarter 0 and 1 (0), because the
    // weight tile holds the layer's rows two (four) times; the replicas take different pixels, so
    // that every epilogue warp has work although the layer fills only part of the MMA's 128 rows.
    // Row pairs: quarters 2 and 3 hold the same channels too, but of the odd output rows; the
    // two halves do not share pixels, they store to rows 2 * p0 and 2 * p0 + 1.
    const int rep_q = EPI == 0 ? (a.rowpair ? 2 : (4 >> a.dup_log2)) : 4;  // lane quarters per replica
    const int cq = quarter & (rep_q - 1);                                  // the quarter's place among the channels
    const bool split_px = EPI == 0 && !a.rowpair;
    const int half_eff = split_px ? (quarter / rep_q) * kPerQuarter + half : half;  // which of the warps that share the pixels
    const int per_eff = split_px ? (kPerQuarter << a.dup_log2) : kPerQuarter;
    const int odd_row = (EPI == 0 && a.rowpair) ? (quarter >> 1) : 0;
    const int row = cq * 32 + ((EPI == 2 && a.y_tma) ? ((lane & 3) << 3) + (lane >> 2) : lane);
    uint16_t* yb = reinterpret_cast<uint16_t*>(y);
    const uint32_t stage_base = ring_base + (uint32_t)a.stages * a.stage_bytes;
    const bool relu = a.relu != 0;
    // this warp's own staging tiles: 32 channel rows of 128 bytes each, 128-byte swizzled
    const uint32_t my_stage = stage_base + (uint32_t)ew * (uint32_t)a.nbuf * kWarpStageBytes;
    const uint32_t row_off = (uint32_t)lane * 128u + (((uint32_t)lane & 7u) << 4);
    uint32_t unit_ctr = 0, stage_sel = 0;
    uint32_t lt = 0;
    uint32_t meet_phase = 0, ho_phase = 0, pl_phase = 0, q_phase = 0;
    bool gave_up = false;  // (a meeting of the whole-plane epilogue ran out of time)
    float bv = 0.f;
    int bias_k = -1;
    // Shared tiles: when this unit's range ends inside a tile whose first stage it holds, it
    // finishes that tile (its last item), and the following units computed the tile's later parts
    // first of all.  The sum of their partial accumulators is put into the tile's accumulator
    // BEFORE its MMAs start (which then add to it), while the MMAs of the items before run: by the
    // second warp of every lane quarter, at the top of the item before the last (of the first item
    // when there are at most two: that accumulator has not been used yet).  Handing over (the
    // unit's first item, when its range begins inside a tile) is the first warps' work, so that a
    // unit's hand-over never waits for its own fetch: no chain of waits through the units.
    int fin_item = -1, fin_tile = 0;
    if constexpr (!SPLIT && SHARED) {
      const int u = SegIter<SHARED>::unit(a);
      const int64_t g_beg = SegIter<SHARED>::range_start(a, u), g_end = SegIter<SHARED>::range_start(a, u + 1);
      fin_tile = (int)(g_end / a.ts);
      if (g_end > g_beg && g_end % a.ts != 0 && (int64_t)fin_tile * a.ts >= g_beg) fin_item = fin_tile - (int)(g_beg / a.ts);
    }
    typename WorkIterOf<SPLIT, SHARED>::type it;
    for (it.init(a); it.valid(a); it.next(a), ++lt) {
      if constexpr (!SPLIT && SHARED) {
        if (fin_item >= 0 && (int)lt == (fin_item >= 2 ? fin_item - 1 : 0)) {
          // every warp has drained the accumulator's previous tile, two items back
          if (fin_item >= 2 && !epi_sync(smem_u32(&meet_bar), meet_phase, &abort_flag)) break;
          if (half == 1) {
            const int unit = SegIter<SHARED>::unit(a);
            const size_t slot_elems = (size_t)a.sk_cols32 * 32 * 128;
            const int64_t tile_end = (int64_t)(fin_tile + 1) * a.ts;
            int count = 0;
            while (unit + 1 + count < SegIter<SHARED>::units(a) && SegIter<SHARED>::range_start(a, unit + 1 + count) < tile_end) ++count;
            const int first_slot = ((unit + 1) << a.pair) + (int)rank;
            const int slot_step = 1 << a.pair;
            int good = 1;
            if (lane == 0) {
              for (int i = 0; i < count && good; ++i) {
                const int* f = a.sk_flags + first_slot + i * slot_step;
                const uint64_t t0 = global_timer_ns();
                for (uint32_t spin = 0;; ++spin) {
                  int v;
                  asm volatile("ld.acquire.gpu.global.b32 %0, [%1];" : "=r"(v) : "l"(f) : "memory");
                  if (v != 0) break;
                  if ((spin & 255u) == 255u && (abort_flag || global_timer_ns() - t0 > g_wait_limit_ns)) {
                    abort_flag = 1;
                    good = 0;
                    break;
                  }
                  __nanosleep(128);
                }
              }
            }
            good = __shfl_sync(0xffffffffu, good, 0);
            if (!good) break;
            const int mgn = a.mtiles * a.group;
            const int mg_f = fin_tile % mgn;
            const int m0_f = (((a.group == 1 ? mg_f : mg_f % a.mtiles) * 128) << a.pair) + (PAIR ? (int)rank * 128 : 0);
            if (m0_f + quarter * 32 < a.kg)
              sk_preload(tmem_base + (uint32_t)(fin_item & 1) * 256u + ((uint32_t)(quarter * 32) << 16), quarter, a.sk_cols32,
                         a.sk_part, slot_elems, first_slot, slot_step, count);
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
              if constexpr (PAIR) mbar_arrive_cluster(cluster_addr(smem_u32(&sk_bar), 0));
              else mbar_arrive(smem_u32(&sk_bar));
            }
            // every part has been read by the four warps: lower the flags for the next launch
            if (!epi_sync(smem_u32(&pl_bar), pl_phase, &abort_flag)) break;
            if (quarter == 0)
              for (int i = lane; i < count; i += 32) a.sk_flags[first_slot + i * slot_step] = 0;
          }
        }
      }
      int grp, m0_item;
      it.channel_tile(a, grp, m0_item);
      if constexpr (PAIR) m0_item += (int)rank * 128;  // this CTA's tensor memory holds its own 128 channels
      // (block kernels with several channel tiles per pixel tile come back here for each of them)
      int ci = 0;
    [[maybe_unused]] next_channel_tile:
      const int m0 = m0_item + ci * 128;
      const int kin = m0 + row;
      const bool kvalid = kin < (a.rowpair ? 64 : a.kg);
      const int k = grp * a.kg + (kvalid ? kin : 0);
      // (fetched again only when the channel changes: a load from global memory at the head of
      //  every tile's epilogue costs several hundred clocks, a third of a short tile's epilogue)
      const int bias_key = kvalid ? k : -2;
      if (bias_key != bias_k) {
        bv = 0.f;
        if (bias != nullptr && kvalid) {
          if (HGC_ADDR_OK(bias + k, sizeof(__half))) bv = __half2float(__ldg(bias + k));
        }
        bias_k = bias_key;
      }
      const bool one_set = DWPW && a.nacc > 1;  // (see the MMA issuer)
      const uint32_t buf = one_set ? 0u : (lt & 1u);
      if (ci == 0) {
        if (!mbar_wait(smem_u32(&acc_full[buf]), (one_set ? lt : (lt >> 1)) & 1u, &abort_flag, 256)) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      }
      const uint32_t t_tile = tmem_base + buf * 256u + (uint32_t)(DWPW ? ci * a.acc_stride : 0) + ((uint32_t)(quarter * 32) << 16);
      const bool quarter_live = m0 + cq * 32 < (a.rowpair ? 64 : a.kg);  // any real output channel in this warp's lanes?
      // the barrier the accumulator is handed back on (of a pair: the first CTA's)
      const uint32_t acc_empty_bar = PAIR ? cluster_addr(smem_u32(&acc_empty[buf]), 0) : smem_u32(&acc_empty[buf]);

      if constexpr (!SPLIT && SHARED) {
        const int kind = it.kind(a);
        const size_t slot_elems = (size_t)a.sk_cols32 * 32 * 128;
        // slots and flags are per CTA; the parts of a tile come from the following work units
        // (the CTA of the same rank in the following pairs)
        if (kind == 1) {
          // a later part of a tile that another CTA finishes: hand the accumulators over
          if (half == 0) {
            if (quarter_live) sk_hand_over(t_tile, quarter, a.sk_cols32, a.sk_part + (size_t)blockIdx.x * slot_elems);
            __threadfence();
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            if (!epi_sync(smem_u32(&ho_bar), ho_phase, &abort_flag)) break;
            if (ew == 0 && lane == 0) {
              __threadfence();
              asm volatile("st.release.gpu.global.b32 [%0], %1;" ::"l"(a.sk_flags + blockIdx.x), "r"(1) : "memory");
            }
          }
          __syncwarp();
          if (lane == 0) {
            if constexpr (PAIR) mbar_arrive_cluster(acc_empty_bar);
            else mbar_arrive(acc_empty_bar);
          }
          continue;
        }
      }

      // the pixel sub-tiles of the tile: one, or the two of a CTA pair (side by side in the accumulator)
#pragma unroll 1
      for (int sub = 0; sub < (PAIR ? 2 : 1); ++sub) {
      int n0 = it.pt * a.tn;
      int p0 = it.ph * a.th;
      if constexpr (PAIR) {
        if (!it.sub_tile(a, sub, n0, p0)) break;  // (only the last pair tile can lack its second sub-tile)
      }
      const uint32_t t_addr = t_tile + (uint32_t)(sub * a.ncols_sub);
      if constexpr (EPI == 0) {
        // ---- staged epilogue: TMEM -> registers -> swizzled fp16 tile in smem -> TMA store ----
        // (taken when Q % 8 == 0, hence P*Q % 8 == 0, and a tile holds one image: every staged run
        //  of pixels then starts on a 16-byte boundary of y).  A unit of work is 32 channels (this
        //  warp's TMEM lanes) x 64 consecutive output pixels; the two warps of a lane quarter take
        //  alternate units.  Each warp owns its staging tiles and issues its own stores, so the
        //  epilogue warps never wait for one another.
        if (quarter_live) {
          const int rows_valid = (a.P - p0) < a.th ? (a.P - p0) : a.th;
          const int e_valid = rows_valid * a.Q;  // output pixels of one channel in this tile
          const bool last_row_tile = p0 + a.th >= a.P;
          // (row, column) of the unit's first pixel, kept up to date without divisions
          const bool linear = a.pitch == a.Q;  // no junk columns: accumulator columns are consecutive pixels
          // pixels per unit: 64, or 32 where the replicas would otherwise leave warps without a unit
          const int upx = a.fine_units ? 32 : kPassElems;
          int hr = 0, wc = half_eff * upx;
          while (!linear && wc >= a.Q) { wc -= a.Q; ++hr; }
          for (int e_lo = half_eff * upx; e_lo < e_valid; e_lo += per_eff * upx, ++unit_ctr) {
            const int e_hi = e_lo + upx < e_valid ? e_lo + upx : e_valid;
            const uint32_t sbuf = my_stage + stage_sel * kWarpStageBytes;
            stage_sel = a.nbuf == 2 ? stage_sel ^ 1u : 0u;
            int uh = hr, uw = wc;  // walks through this unit
#pragma unroll 1
            for (int g = 0; g < 2; ++g) {
              const int e0 = e_lo + g * 32;
              if (e0 >= e_hi) break;
              const int nchunks = (e_hi - e0) >= 32 ? 4 : (e_hi - e0) >> 3;
              uint32_t v[32];
              // 32 pixels: one wide accumulator load when they are 32 consecutive columns (always
              // when columns are pixels; else when the row does not end inside them)
              if (nchunks == 4 && (linear || uw + 32 <= a.Q)) {
                tmem_ld32(t_addr + (uint32_t)(linear ? e0 : uh * a.pitch + uw), v);
                if (!linear) {
                  uw += 32;
                  if (uw == a.Q) { uw = 0; ++uh; }
                }
              } else {
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                  uint32_t col;
                  if (linear) {
                    col = (uint32_t)(e0 + 8 * c);  // columns are pixels
                  } else {
                    col = (uint32_t)(uh * a.pitch + uw);
                    uw += 8;
                    if (uw == a.Q) { uw = 0; ++uh; }  // next output row: the junk columns of the pitch are skipped
                  }
                  if (c < nchunks) tmem_ld8(t_addr + col, &v[8 * c]);
                }
              }
              if (g == 0) {
                // this buffer's previous store must have been read out of shared memory
                if (lane == 0) {
                  if (a.nbuf == 1) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                  else asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                }
                __syncwarp();
              }
              asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
              if (relu) convert_store<true>(v, nchunks, bv, sbuf + row_off, (uint32_t)(g * 4));
              else convert_store<false>(v, nchunks, bv, sbuf + row_off, (uint32_t)(g * 4));
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
              // past P*Q the store is clipped (row pairs: the next row of y belongs to other warps)
              const bool full_box = !a.fine_units && ((e_hi - e_lo == kPassElems) || (last_row_tile && !a.rowpair));
              tma_store_4d(full_box ? &tmY : &tmYr, sbuf, (a.rowpair ? 2 * p0 + odd_row : p0) * a.Q + e_lo, m0 + cq * 32, grp, n0);
              asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            }
            // first pixel of this warp's next unit
            wc += per_eff * upx;
            while (!linear && wc >= a.Q) { wc -= a.Q; ++hr; }
          }
        }
      } else {
        // ---- direct epilogue: each thread stores runs of its own channel plane ----
        {
          // the warps of a lane quarter take alternate units
          if constexpr (EPI == 2) {
            if (quarter_live && a.y_tma) {
              // staged channels-last epilogue (output channels per group a multiple of 8: every
              // pixel's run of channels starts on a 16-byte boundary of y).  A unit of work is this
              // warp's 32 channels x up to 64 consecutive output pixels: a piece of a tile row, or
              // several whole rows when rows are at most 32 pixels wide; one TMA store per unit,
              // clipped at the last channel of the group and at the end of the image.
              const uint32_t lane_off = (2u * ((uint32_t)lane >> 3) + ((uint32_t)lane & 1u)) * 64u +
                                        (((uint32_t)lane & 7u) >> 1) * 16u;
              const int rows_valid = (a.P - p0) < a.th ? (a.P - p0) : a.th;
              const int cpu = a.Q > kPassElems ? kPassElems : a.Q;  // columns per unit
              int unit = 0;
              for (int img = 0; img < a.tn; ++img) {
                if (n0 + img >= a.N) break;
                for (int hr0 = 0; hr0 < rows_valid; hr0 += a.y_rpu) {
                  for (int wc0 = 0; wc0 < a.Q; wc0 += cpu, ++unit) {
                    if (unit % kPerQuarter != half) continue;
                    const int nrows = rows_valid - hr0 < a.y_rpu ? rows_valid - hr0 : a.y_rpu;
                    const int ncol = a.Q - wc0 < cpu ? a.Q - wc0 : cpu;
                    const uint32_t sbuf = my_stage + stage_sel * kWarpStageBytes;
                    stage_sel = a.nbuf == 2 ? stage_sel ^ 1u : 0u;
                    bool first = true;
#pragma unroll 1
                    for (int r = 0; r < nrows; ++r) {
#pragma unroll 1
                      for (int g = 0; g < 2; ++g) {
                        const int rem = ncol - g * 32;
                        if (rem <= 0) break;
                        const uint32_t tcol = t_addr + (uint32_t)((img * a.th + hr0 + r) * a.pitch + wc0 + g * 32);
                        uint32_t v[32];
                        if (rem >= 32) {
                          tmem_ld32(tcol, v);
                        } else {
#pragma unroll
                          for (int c = 0; c < 4; ++c)
                            if (c * 8 < rem) tmem_ld8(tcol + (uint32_t)(c * 8), &v[8 * c]);
                        }
                        if (first) {
                          // this buffer's previous store must have been read out of shared memory
                          if (lane == 0) {
                            if (a.nbuf == 1) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                            else asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                          }
                          __syncwarp();
                          first = false;
                        }
                        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                        const uint32_t dst = sbuf + (uint32_t)(r * ncol + g * 32) * 64u + lane_off;
                        if (relu) convert_store_pixels<true>(v, rem, bv, dst);
                        else convert_store_pixels<false>(v, rem, bv, dst);
                      }
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) {
                      // a short unit at the end of the image takes the full box: the rest is clipped
                      const bool image_end = p0 + hr0 + nrows == a.P && wc0 + ncol == a.Q;
                      tma_store_4d((nrows * ncol == a.y_full_w || image_end) ? &tmY : &tmYr, sbuf, m0 + quarter * 32, grp,
                                   (p0 + hr0) * a.Q + wc0, n0 + img);
                      asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    }
                  }
                }
              }
            }
            else if (EW == 8 && quarter_live)  // (16 epilogue warps only ever run the staged form)
              epilogue_nhwc(t_addr, half, kPerQuarter, a.tn, a.th, a.pitch, a.N, a.K, a.P, a.Q, n0, p0, k, kvalid, bv,
                            relu, yb);
          } else if constexpr (SPLIT) {
            if (quarter_live) {
              const int kleft = a.kg - (m0 + quarter * 32);
              epilogue_partial(t_addr, my_stage, half, kPerQuarter, a.tn, a.th, a.pitch, a.N, a.K, a.P, a.Q, n0, p0,
                               grp * a.kg + m0 + quarter * 32, kleft < 32 ? kleft : 32,
                               partials + (int64_t)it.slice(a) * a.part_stride);
            }
          } else {
            if (quarter_live && a.P * a.Q == 1) {
              const int kleft = a.kg - (m0 + quarter * 32);
              const int nimg = a.N - n0 < a.tn ? a.N - n0 : a.tn;
              epilogue_columns(t_addr, half, kPerQuarter, nimg, a.K, n0, grp * a.kg + m0 + quarter * 32,
                               kleft < 32 ? kleft : 32, bv, relu, yb);
            } else if constexpr (EPI == 3) {
              // whole-plane tiles (instantiations of their own: the other kernels' code stays as it is)
              if (quarter_live) {
                q_phase = epilogue_planes(t_addr, stage_base + (uint32_t)quarter * a.plane_bytes, half, a.plane_store, a.tn, a.N, a.K,
                                          a.P * a.Q, n0, grp * a.kg + m0 + quarter * 32, bv, relu, yb, smem_u32(&q_bar[quarter]),
                                          q_phase, &abort_flag);
                if (q_phase == ~0u) gave_up = true;
              }
            } else if (quarter_live) {
              const int kleft = a.kg - (m0 + quarter * 32);
              epilogue_copy(t_addr, my_stage, half, kPerQuarter, a.tn, a.th, a.pitch, a.N, a.K, a.P, a.Q, n0, p0,
                            grp * a.kg + m0 + quarter * 32, kleft < 32 ? kleft : 32, bv, relu, yb);
            }
          }
        }
      }
      }  // sub-tiles
      if (gave_up) break;
      if constexpr (DWPW) {
        if (++ci < a.nacc) goto next_channel_tile;
      }
      // this warp has read its lanes of the accumulator: hand the buffer back to the MMA issuer
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) {
        if constexpr (PAIR) mbar_arrive_cluster(acc_empty_bar);
        else mbar_arrive(acc_empty_bar);
      }
    }
    // the shared-memory tiles of outstanding stores must stay intact until they have been read,
    // and the stores themselves must be complete before the kernel ends
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  // (a pair leaves together: the first CTA's MMAs read the partner's shared memory and write its tensor memory)
  if constexpr (PAIR) cluster_sync_all();
  else __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
  if (threadIdx.x == 0 && abort_flag && status != nullptr) atomicExch(status, (int)HGC_DEVICE_TIMEOUT);
  if constexpr (FUSEL) {
    // the CTA that finishes last lowers the segment counters for the next launch
    __shared__ int last_cta;
    const int nflags = a.N * a.lay_segs;
    if (threadIdx.x == 0) {
      __threadfence();
      last_cta = atomicAdd(a.lay_flags + nflags, 1) == (int)gridDim.x - 1;
    }
    __syncthreads();
    if (last_cta) {
      for (int i = threadIdx.x; i <= nflags; i += blockDim.x) a.lay_flags[i] = 0;
    }
  }
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

// Launches a kernel of CTA pairs (clusters of two).  p.grid pairs are wanted, but never more than
// can be resident at once: a persistent kernel must not leave a pair waiting for a second round.
template <typename... KArgs, typename... Args>
cudaError_t launch_pair(void (*kernel)(KArgs...), IgemmPlan& p, int sms, bool cooperative, dim3 block,
                        cudaStream_t stream, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = p.smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeCooperative;
  attr[1].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = cooperative ? 2 : 1;
  if (p.pair_fit == 0) {
    int n = 0;
    cfg.gridDim = dim3((unsigned)(2 * (sms / 2)));
    p.pair_fit = (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) == cudaSuccess && n > 0) ? n : sms / 2;
    (void)cudaGetLastError();
  }
  const int fit = p.pair_fit < p.grid ? p.pair_fit : p.grid;
  cfg.gridDim = dim3((unsigned)(2 * fit));
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

}  // namespace

cudaError_t igemm_set_wait_limit_ns(uint64_t ns) {
  const uint64_t v = ns == 0 ? kWaitLimitNs : ns;
  return cudaMemcpyToSymbol(g_wait_limit_ns, &v, sizeof(v));
}

int sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0)
      n = v;
    else
      return 148;  // B200; not cached so that a later call can still query the device
  }
  return n;
}

namespace {
bool make_plan_impl(const ConvGeom& g, IgemmPlan* out, bool want_pair, int kb_max, bool wide_stages);
}

// The plan of a layer: the single-CTA form, or CTA pairs where they were asked for and the layer
// has more than 128 output channels per group.
// The layer that a row-pair plan (IgemmPlan::rowpair) runs in place of layer g: 128 "channels"
// (parity of the output row x the 64 channels), R + 1 kernel rows, stride 2 along H, P/2 rows.
static ConvGeom rowpair_geom(const ConvGeom& g) {
  ConvGeom r = g;
  r.k = r.kg = 128;
  r.r = g.r + 1;
  r.stride_h = 2;
  r.p = g.p / 2;
  r.rowpair = 1;
  return r;
}
static inline ConvGeom effective_geom(const ConvGeom& g, const IgemmPlan& p) { return p.rowpair ? rowpair_geom(g) : g; }

bool igemm_make_plan(const ConvGeom& g, IgemmPlan* out) {
  // Row pairs: stride-1 layers of exactly 64 output channels with at least two kernel rows and a
  // wide, even output plane, NCHW output through the TMA-store epilogue (VGG-16 conv1_2: the
  // kernel 77 -> ... us).  Narrow planes would need several row pairs per tile, whose rows of
  // one parity are not contiguous in y: not built.
  if (!g.rowpair && g.group == 1 && g.kg == 64 && g.cg >= 16 && g.r >= 2 && g.stride_h == 1 && g.stride_w == 1 &&
      g.dil_h == 1 && g.dil_w == 1 && !g.y_nhwc && g.dw_stride == 0 && (g.p % 2) == 0 && (g.q % 8) == 0 && g.q >= 112 &&
      g.q + (g.s - 1) <= 256) {
    ConvGeom g2 = rowpair_geom(g);
    g2.no_pair = 1;
    g2.no_split = 1;
    IgemmPlan rp{};
    if (make_plan_impl(g2, &rp, false, 64, false) && rp.th == 1 && rp.tn == 1 && rp.tma_store && rp.halo && !rp.nchw &&
        rp.ks_log2 == 0 && !rp.fuse_layout) {
      rp.rowpair = 1;
      *out = rp;
      return true;
    }
  }
  ConvGeom gs = g;
  gs.no_pair = 1;
  IgemmPlan single{};
  bool ok_single = make_plan_impl(gs, &single, false, 64, false);
  if (ok_single && single.kb == 32 && g.cg > 32) {
    // the layer was given 32-channel stages for the sake of a deeper ring: where three 64-channel
    // stages fit as well (small pixel tiles: 14x14 and 7x7 planes) they are faster, because the
    // copies then move 128-byte rows (measured: VGG conv5 27.7 -> 22.9 us)
    IgemmPlan wide{};
    if (make_plan_impl(gs, &wide, false, 64, true) && wide.kb == 64 && wide.stages >= 3) single = wide;
  }
  if (!g.no_pair && g.kg > 128) {
    IgemmPlan pair{};
    bool ok_pair = make_plan_impl(g, &pair, true, 64, true);
    if (ok_pair && pair.kb == 64 && pair.stages < 3) ok_pair = make_plan_impl(g, &pair, true, 32, true);
    if (ok_pair) {  // asked for (HGC_FLAG_CTA_PAIRS) and possible
      *out = pair;
      return true;
    }
  }
  if (ok_single) *out = single;
  return ok_single;
}

namespace {
bool make_plan_impl(const ConvGeom& g, IgemmPlan* out, bool want_pair, int kb_max, bool wide_stages) {
  IgemmPlan p{};
  if (g.group > 1 && (g.cg % 8) != 0) return false;  // group stride of x' must be 16-byte aligned
  p.x_nhwc = g.x_nhwc;
  p.y_nhwc = g.y_nhwc;
  // channels-last input: x is used as x' (a pixel must be a whole number of 16-byte vectors)
  if (p.x_nhwc && ((g.c % 8) != 0 || g.cg < 9)) return false;
  // a 1x1 input plane (inner products) is channels-last as it stands: no layout pass
  if (g.h == 1 && g.w == 1 && (g.c % 8) == 0 && g.cg >= 9) p.x_nhwc = 1;
  // Few input channels (image stems, C <= 8): a tap alone is too short for a K=16 MMA step.
  // The input is copied to a zero-bordered NHWC buffer with 8 channels per pixel; the S taps of
  // a kernel row are then S*8 CONTIGUOUS elements, read as one "window" per output pixel through
  // a tensor map whose pixel stride (stride_w pixels) is smaller than the window.  The kernel
  // sees a convolution with R taps (one per kernel row), no padding and kw_pix*8 channels.
  // Tiny receptive fields (R*S*C <= 64, one group: 3x3 stems): "patch mode".  The input is
  // expanded to x''[N][P][Q][kelems] (per output pixel the R*S*C values under the kernel, zero
  // padded to 16/32/64 elements) and the kernel sees a 1x1, stride-1, unpadded convolution with
  // kelems channels on the OUTPUT plane: one pipeline stage and one dense activation tile per
  // pixel tile instead of one overlapping-window load per kernel row.  Taken for strided layers
  // (measured: 3x3 stride-2 stem 50.6 us against 56.8 us in window mode; at stride 1 the window
  // mode wins, 74.7 us against 82.5 us, because the expansion pass writes 64 bytes per pixel).
  const int64_t rsc = (int64_t)g.r * g.s * g.cg;
  p.patch = (!p.x_nhwc && g.group == 1 && rsc <= 64 && (g.stride_h > 1 || g.stride_w > 1) && g.cg <= 8) ? 1 : 0;
  p.window = (!p.x_nhwc && !p.patch && g.cg <= 8 && g.group == 1 && g.dil_w == 1) ? 1 : 0;
  if (!p.window && !p.patch && g.cg < 9) return false;
  if (p.patch) {
    const int kelems = rsc <= 16 ? 16 : (rsc <= 32 ? 32 : 64);
    p.kb = kelems;
    p.cblocks = 1;
    p.cw = kelems;
    p.c_pad = kelems;
    p.eff_r = 1; p.eff_s = 1; p.eff_pad_h = 0; p.eff_pad_w = 0;
    p.halo = 0;
  } else if (p.window) {
    // Pixels of the bordered copy hold 8 channels (16 bytes), or 4 (8 bytes) for layers of at most
    // 4 channels with stride 2 along W: consecutive windows then start 2 pixels = 16 bytes apart,
    // which lets them take the dense form below too, at half the reduction length.
    p.px_ch = (g.cg <= 4 && g.stride_w == 2 && g.s * 4 <= 64) ? 4 : 8;
    for (;;) {
      const int elems = g.s * p.px_ch;
      const int kelems = elems <= 16 ? 16 : elems <= 32 ? 32 : (elems + 63) / 64 * 64;
      p.kw_pix = kelems / p.px_ch;
      p.kb = kelems >= 64 ? 64 : kelems;
      p.cblocks = kelems / p.kb;
      p.cw = kelems;
      p.c_pad = p.px_ch;
      p.hp = g.h + 2 * g.pad_h;
      p.wp = g.w + 2 * g.pad_w;
      if (p.wp < (g.q - 1) * g.stride_w + p.kw_pix) p.wp = (g.q - 1) * g.stride_w + p.kw_pix;
      // Windows that start 16 bytes apart (stride 1 with 8-channel pixels, stride 2 with 4-channel
      // pixels) are not fetched one by one: whole rows of the bordered copy (a multiple of 128 bytes
      // wide) are loaded densely, 128 bytes per TMA request, and the MMA reads the overlapping
      // windows straight out of them: an unswizzled K-major operand whose rows (windows) are 16
      // bytes apart and whose 16-byte K chunks are also 16 bytes apart.  The accumulator then has
      // one column per 16 bytes of the padded row (junk columns at the end of each tile row).
      const int per128 = 64 / p.px_ch;  // pixels per 128 bytes
      const int wp_dense = (p.wp + per128 - 1) / per128 * per128;
      const int pitch_dense = wp_dense * p.px_ch / 8;
      p.dense_rows = (g.stride_w * p.px_ch == 8 && p.cblocks == 1 && pitch_dense <= 256) ? 1 : 0;
      if (p.dense_rows) {
        p.wp = wp_dense;
        p.dense_pitch = pitch_dense;
      }
      if (p.px_ch == 4 && !p.dense_rows) {  // 4-channel pixels only pay in the dense form
        p.px_ch = 8;
        continue;
      }
      break;
    }
    p.eff_r = g.r; p.eff_s = 1; p.eff_pad_h = 0; p.eff_pad_w = 0;
    p.halo = 0;
    // ... and with stride 1 along H too, the R kernel rows share one tile of th + R - 1 dense rows
    // (the mechanism of the shared taps of a kernel row, turned by 90 degrees: tap r starts r
    // image rows = r * wp pixels further in shared memory): one pipeline stage per tile
    // (with a stride along H the tile is one output row: rows of a taller tile would be
    // stride_h image rows apart, more accumulator columns than there are)
    if (p.dense_rows && g.dil_h == 1) {
      p.vhalo = 1;
      p.halo = 1;
      p.eff_r = 1;
      p.eff_s = g.r;
    }
  } else {
    p.kb = g.cg > 32 ? 64 : (g.cg > 16 ? 32 : 16);
    // stride-1 layers with three or more taps per kernel row and at least two 64-channel blocks:
    // 32-channel stages halve a stage (one activation tile + S weight tiles) so that the ring
    // is four or five deep instead of two; measured 3-5 % faster on 3x3 layers of 128-512 channels.
    // (`wide_stages` keeps 64, for CTA pairs and for tiles small enough for three such stages: a
    // copy engine handles about one row of a box per clock whatever the row's width (measured),
    // and with 64-byte rows the rows of a stage take as long as its MMAs.)
    if (!wide_stages && p.kb == 64 && g.stride_h == 1 && g.stride_w == 1 && g.s >= 3 && g.cg >= 128) p.kb = 32;
    if (p.kb > kb_max) p.kb = kb_max;
    p.cblocks = (g.cg + p.kb - 1) / p.kb;
    p.cw = p.cblocks * p.kb;
    p.c_pad = (g.c + 7) / 8 * 8;
    p.eff_r = g.r; p.eff_s = g.s; p.eff_pad_h = g.pad_h; p.eff_pad_w = g.pad_w;
    // stride 1: the S taps of a kernel row read one shared tile, shifted by s*dil pixels
    p.halo = ((g.stride_h == 1 || g.rowpair) && g.stride_w == 1) ? 1 : 0;  // (row pairs: one row of columns per tile)
  }
  // 1x1, stride 1, unpadded layers on planes of a multiple of 8 pixels read x as it is (no NHWC
  // copy): the activation operand is then pixel-major ("MN-major") in shared memory
  p.nchw = (!p.x_nhwc && !p.window && !p.patch && g.r == 1 && g.s == 1 && g.stride_h == 1 && g.stride_w == 1 && g.pad_h == 0 &&
            g.pad_w == 0 && g.group == 1 && ((int64_t)g.h * g.w) % 8 == 0)
               ? 1
               : 0;
  // The same layers on small planes of a multiple of 4 pixels (14x14), on request
  // (HGC_FLAG_GATHER_X): a channel's plane starts on an 8-byte boundary only, which no tensor map
  // can describe, so extra warps of the kernel gather the pixel-major tile themselves with 8-byte
  // asynchronous copies (the kernel of the depthwise + pointwise blocks, whose extra warps produce
  // the activation tile too).  A tile is one whole plane; whole 64-channel blocks only (nothing
  // fills channels past the last one).  Measured against the layout pass + plain kernel: 64 x 1024
  // -> 256 on 14x14 19.1 us against 20.3, 256 -> 1024 21.8 against 18.4 (with the copies left out
  // 13.6 and 25.8 before the whole-plane epilogue): a gain only where x is large and y small, hence opt-in.
  p.gather = 0;
  if (!p.nchw && !p.x_nhwc && !p.window && !p.patch && g.r == 1 && g.s == 1 && g.stride_h == 1 && g.stride_w == 1 &&
      g.pad_h == 0 && g.pad_w == 0 && g.group == 1 && g.dw_stride == 0 && !g.rowpair && !want_pair && p.kb == 64 &&
      (g.c % 64) == 0 && ((int64_t)g.h * g.w) % 4 == 0 && (int64_t)g.h * g.w <= 256 && !g.no_gather) {
    p.nchw = 1;
    p.gather = 1;
  }
  p.pitch = p.dense_rows ? p.dense_pitch : (p.halo ? g.q + (g.s - 1) * g.dil_w : g.q);
  p.tw = g.q;
  const int box_w = (p.halo && !p.vhalo) ? p.pitch : ((p.window || p.patch) ? g.q : g.q * g.stride_w);
  if (p.pitch > 256 || box_w > 256) return false;
  p.mtiles = (g.kg + 127) / 128;
  const int64_t mg = (int64_t)p.mtiles * g.group;
  // pixel tile = tn images x th rows; accumulator columns = tn*th*pitch (<= 256).  Among the
  // feasible shapes pick the one with the least estimated time: waves over the SMs x the
  // estimated clocks of one tile.
  const int sms = sm_count();
  const int junk = p.pitch - g.q;
  // An MMA step (128 channels x ncols pixels x 16 reduction elements) is bounded by
  //   the tensor pipe:     ncols / 2 clocks,
  //   L2 -> shared memory  (about 30 bytes per clock and SM, measured): its 4 KB slice of the
  //                        weights plus its share of the activation tile, which the taps and
  //                        16-channel steps of a stage share,
  //   the issuing thread:  about 45 clocks per MMA plus about 400 per barrier hand-shake;
  // the epilogue of the previous tile runs beside the main loop and bounds short main loops.
  const int taps_est = p.halo ? p.eff_s : 1;
  const double mps = (double)taps_est * (p.kb / 16.0);                       // MMAs per stage
  const double mpt = (double)p.cblocks * p.eff_r * p.eff_s * (p.kb / 16.0);  // MMAs per tile
  const double a_bytes_mma = 32.0 * (g.kg < 128 ? g.kg : 128);
  // ks: log2 of the number of CTAs that share the reduction of a tile (each then writes fp32
  // partial sums, added by a second kernel): main loop / 2^ks, an epilogue of twice the bytes
  // clocks of one MMA step in the main loop of a tile of `cols` accumulator columns
  auto mma_clk = [&](int64_t brow, int64_t cols) {
    const double ncols = (double)((cols + 15) / 16 * 16);
    const double brows = p.nchw ? (double)((cols + 63) / 64 * 64) : (double)brow;
    const double t_l2 = (a_bytes_mma + brows * p.kb * 2.0 / mps) / 30.0;
    // the tensor pipe needs N/2 clocks for a step of N columns, but never less than about 86
    // (measured: back-to-back steps of 64 to 170 columns all take 86 clocks)
    const double t_tensor = ncols / 2.0 > 86.0 ? ncols / 2.0 : 86.0;
    const double t_issue = 45.0 + 400.0 / mps;
    double t = t_tensor > t_l2 ? t_tensor : t_l2;
    if (t_issue > t) t = t_issue;
    return t;
  };
  auto epilogue_clk = [&](int64_t cols) { return 600.0 + 10.0 * (double)((cols + 15) / 16 * 16); };
  auto tile_clk = [&](int64_t brow, int64_t cols, int ks) {
    const double main_loop = mpt / (double)(1 << ks) * mma_clk(brow, cols);
    const double epilogue = epilogue_clk(cols) * (ks > 0 ? 2.0 : 1.0);
    return (main_loop > epilogue ? main_loop : epilogue) + 300.0;
  };
  // Contiguous ranges of ring stages per CTA (kernels without reduction slices).  Whole tiles per
  // CTA when that balances; otherwise equal ranges, with the tiles that straddle a boundary
  // reduced by several CTAs (a hand-over of fp32 accumulators through the workspace).
  const int ts_est = p.cblocks * p.eff_r * (p.halo ? 1 : p.eff_s);  // ring stages per tile
  auto shared_plan = [&](int64_t tiles, double t_mma, int64_t cols, int units, int* grid_out, double* cost_out) {
    const double stage_clk = mps * t_mma;
    const int64_t total = tiles * ts_est;
    // a range is at least 4 stages and 24 MMA steps long, and a tile is shared by at most 4 CTAs
    int64_t min_stages = (int64_t)(24.0 / mps + 0.999);
    if (min_stages < 4) min_stages = 4;
    int64_t grid = total / min_stages;
    if (grid > units) grid = units;
    if (grid > 4 * tiles) grid = 4 * tiles;
    if (grid < 1) grid = 1;
    const double per_cta = (double)((total + grid - 1) / grid);
    const double tiles_per_cta = (double)tiles / (double)grid;
    const double main_loop = per_cta * stage_clk;
    const double epi = tiles_per_cta * epilogue_clk(cols);
    // a hand-over: the accumulators of a part go to the workspace (beside the next tile's MMAs) and
    // from there into the finishing CTA's idle operand ring by bulk copy, 16 KB per 32 columns
    const double parts = tiles >= grid ? 1.0 : (double)grid / (double)tiles;  // accumulators added per shared tile
    const double hand_over = 5000.0 + parts * (1500.0 + 15.0 * (double)cols);  // (measured: 3 to 4 us for 240 columns)
    *grid_out = (int)grid;
    *cost_out = (main_loop > epi ? main_loop : epi) + 300.0 * (tiles_per_cta > 1.0 ? tiles_per_cta : 1.0) + hand_over;
  };
  // the second kernel of a split reduction: a launch plus reading the slices and writing y
  auto finish_clk = [&](int ks) {
    if (ks == 0) return 0.0;
    const double elems = (double)g.n * g.k * g.p * g.q;
    return 8000.0 + elems * (4.0 * (1 << ks) + 2.0) / 3000.0;
  };
  // the split kernel exists for 64-channel stages of stride-1 layers without the direct-x mode
  const bool can_split = p.kb == 64 && p.halo && !p.nchw && !p.y_nhwc;
  double best = 1e300;
  int best_th = 0, best_tn = 0, best_ks = 0, best_shared = 0, best_grid = 0;
  // shared tiles: asked for (no_split == 0: taken wherever tiles do not fill whole waves), or left
  // to this cost model (no_split == 2)
  const bool can_share = g.no_split != 1 && sms <= kMaxGrid && p.kb >= 32 && !p.gather;
  const bool force_share = g.no_split == 0;
  for (int th = 1; th <= g.p; ++th) {
    if ((int64_t)th * p.pitch - junk > 256 || (int64_t)th * (p.patch ? 1 : g.stride_h) > 256) break;
    if (p.vhalo && g.stride_h > 1 && th > 1) break;
    if (g.rowpair && th > 1) break;
    if (p.nchw && th != g.p && ((int64_t)th * g.q) % 8 != 0) continue;  // tiles must start on 16-byte boundaries of x
    if (p.gather && th != g.p) continue;
    const int tn_hi = (th == g.p && !p.nchw && !p.vhalo) ? g.n : 1;  // several images only when a tile holds whole planes
    for (int tn = 1; tn <= tn_hi; ++tn) {
      const int64_t cols = (int64_t)tn * th * p.pitch - junk;
      // several images per tile: image boundaries need not fall on multiples of 8 columns, and an
      // 8-column accumulator read that starts in the tile must end inside the 256-column buffer
      if (cols > (tn > 1 ? 248 : 256) || tn > 256) break;
      if (g.dw_stride > 0) {
        // depthwise + pointwise block: the depthwise layer's input tile (one-pixel border) of a
        // 64- / 32-channel block, twice, must fit beside the ring: at most 48 KB each
        const int64_t in_h = (int64_t)(th - 1) * g.dw_stride + 3, in_w = (int64_t)(g.q - 1) * g.dw_stride + 3;
        if (in_h > 256 || in_w > 256 || tn * in_h * in_w * p.kb * 2 > 48 * 1024) break;
      }
      const int64_t tiles = (int64_t)((g.n + tn - 1) / tn) * ((g.p + th - 1) / th) * mg;
      for (int ks = 0; ks <= 3; ++ks) {
        // a slice keeps at least two channel blocks and a main loop of 24 MMAs; only layers whose
        // tiles leave three quarters of the SMs idle are split (inner products, tiny planes): on
        // a 14x14 layer of 128 tiles the second pass costs what the split gains (measured)
        if (ks > 0 && (!can_split || (p.cblocks >> ks) < 2 || mpt / (1 << ks) < 24.0 || 4 * tiles > sms)) break;
        const int64_t units = tiles << ks;
        const int64_t waves = (units + sms - 1) / sms;
        double cost = (double)waves * tile_clk((int64_t)tn * th * p.pitch, cols, ks) + finish_clk(ks) +
                      1e-3 * (double)units;
        if (force_share && can_share && tiles % sms != 0) cost *= 1e3;  // shared tiles were asked for (HGC_FLAG_SHARED_TILES)
        if (cost < best - 1e-9 ||
            (cost < best + 1e-9 && ks == best_ks && !best_shared && (int64_t)tn * th > (int64_t)best_tn * best_th)) {
          best = cost;
          best_th = th;
          best_tn = tn;
          best_ks = ks;
          best_shared = 0;
          best_grid = (int)(tiles < sms ? tiles : sms);
        }
      }
      if (can_share && tiles % sms != 0) {
        int grid_s = 0;
        double cost_s = 0.0;
        shared_plan(tiles, mma_clk((int64_t)tn * th * p.pitch, cols), cols, sms, &grid_s, &cost_s);
        if (!force_share) {
          // Measured (VGG-16, batch 16): a unit hands its first partial tile over and fetches the
          // partial sums of its last one beside the MMAs of the tiles between them, which takes
          // whole tiles in between (at least 2.5 tiles per unit); the contiguous ranges cost some
          // locality in L2 and the hand-overs some time, together about 10k clocks per launch
          // (conv3_2: 3.03 waves of 11 us tiles, 61.3 -> 55.6 us; conv2_2, conv4_x: slower).
          cost_s = (double)tiles / (double)sms * tile_clk((int64_t)tn * th * p.pitch, cols, 0) + 10000.0;
          if (2 * tiles < 5 * (int64_t)sms || grid_s != sms || ts_est < 16) grid_s = 0;
        }
        if (grid_s > 1 && cost_s < best - 1e-9) {
          best = cost_s;
          best_th = th;
          best_tn = tn;
          best_ks = 0;
          best_shared = 1;
          best_grid = grid_s;
        }
      }
    }
  }
  if (best_th == 0) return false;
  p.est_clk = best;
  // CTA pairs (tcgen05 cta_group::2) for layers with more than 128 output channels per group: a
  // tile is 256 channels x two pixel sub-tiles of at most 128 accumulator columns each.  Every
  // CTA then reads 128 weight rows and HALF of the activation tile from its own shared memory per
  // MMA step (and fetches only those): the single-CTA kernel is bound by shared-memory traffic
  // (operand reads of the tensor core + ring refills: about 150 clocks per 240-column step
  // against 120 of tensor time, measured), the pair is not.
  p.pair = 0;
  p.ncols_sub = 0;
  const int pairs = sms / 2;
  if (want_pair && (p.nchw || p.window || p.patch || pairs < 1)) return false;
  if (want_pair) {
    const int64_t mgp = (int64_t)((g.kg + 255) / 256) * g.group;
    double best_pair = 1e300;
    int pth = 0, ptn = 0, pshared = 0, pgrid = 0;
    for (int th = 1; th <= g.p; ++th) {
      if ((int64_t)th * p.pitch - junk > 128 || (int64_t)th * g.stride_h > 256) break;
      const int tn_hi = th == g.p ? g.n : 1;
      for (int tn = 1; tn <= tn_hi; ++tn) {
        const int64_t cols = (int64_t)tn * th * p.pitch - junk;
        if (cols > (tn > 1 ? 120 : 128)) break;
        const int64_t subs = (int64_t)((g.n + tn - 1) / tn) * ((g.p + th - 1) / th);
        const int64_t tiles = (subs + 1) / 2 * mgp;
        const double ncols = (double)(2 * ((cols + 7) / 8 * 8));
        double t = ncols / 2.0 > 86.0 ? ncols / 2.0 : 86.0;
        const double t_issue = 45.0 + 400.0 / mps;
        if (t_issue > t) t = t_issue;
        const double main_loop = mpt * t * 1.03;
        const double epi = 600.0 + 10.0 * ncols;
        const int64_t waves = (tiles + pairs - 1) / pairs;
        double cost = (double)waves * ((main_loop > epi ? main_loop : epi) + 300.0) + 1e-3 * (double)tiles;
        if (can_share && tiles % pairs != 0) cost *= 1e3;
        if (cost < best_pair - 1e-9 || (cost < best_pair + 1e-9 && !pshared && (int64_t)tn * th > (int64_t)ptn * pth)) {
          best_pair = cost;
          pth = th;
          ptn = tn;
          pshared = 0;
          pgrid = (int)(tiles < pairs ? tiles : pairs);
        }
        if (can_share && tiles % pairs != 0) {
          int grid_s = 0;
          double cost_s = 0.0;
          shared_plan(tiles, t * 1.03, (int64_t)ncols, pairs, &grid_s, &cost_s);
          if (grid_s > 1 && cost_s < best_pair - 1e-9) {
            best_pair = cost_s;
            pth = th;
            ptn = tn;
            pshared = 1;
            pgrid = grid_s;
          }
        }
      }
    }
    if (pth == 0) return false;
    p.pair = 1;
    p.est_clk = best_pair;
    best_th = pth;
    best_tn = ptn;
    best_shared = pshared;
    best_grid = pgrid;
    best_ks = 0;
  }
  // Depthwise + pointwise blocks: the depthwise warps, not the MMAs, bound a stage (about 33 clocks
  // per pixel of a 64-channel block, measured), and every 128-channel tile of the pointwise layer
  // that is computed from its own pass repeats that work.  So a work item covers up to four
  // channel tiles (accumulators of 512 / nacc columns, one set: the epilogue is not overlapped)
  // that share the depthwise result, and the pixel tile is chosen together with their number.
  p.nacc = 1;
  if (g.dw_stride > 0) {
    double best_blk = 1e300;
    int bth = 0, btn = 0, bna = 1;
    for (int th = 1; th <= g.p; ++th) {
      const int64_t in_h = (int64_t)(th - 1) * g.dw_stride + 3, in_w = (int64_t)(g.q - 1) * g.dw_stride + 3;
      if ((int64_t)th * g.q > 256 || in_h > 256 || in_w > 256) break;
      const int tn_hi = th == g.p ? g.n : 1;
      for (int tn = 1; tn <= tn_hi; ++tn) {
        const int64_t px = (int64_t)tn * th * g.q;
        if (px > (tn > 1 ? 248 : 256) || tn * in_h * in_w * p.kb * 2 > 48 * 1024) break;
        for (int na = 1; na <= 4; na *= 2) {
          if (na > 1 && (px > 512 / na || (int64_t)(na / 2) * 128 >= g.kg)) break;
          {
            // two ring stages (activation tile + na weight tiles), both input tiles and the
            // epilogue's staging tiles must fit into shared memory
            const size_t stage = round_up_sz((size_t)((px + 15) / 16 * 16) * p.kb * 2, 1024) + (size_t)na * 128 * p.kb * 2;
            const size_t in_tile = round_up_sz((size_t)tn * in_h * in_w * p.kb * 2 + 2u * p.kb * 2u, 1024);
            if (2 * stage + 2 * in_tile + (size_t)kEpilogueWarps * kWarpStageBytes > 232448u - 1024u - 512u) break;
          }
          const int64_t tiles = (int64_t)((g.n + tn - 1) / tn) * ((g.p + th - 1) / th) * ((p.mtiles + na - 1) / na);
          const double waves = (double)((tiles + sms - 1) / sms);
          const double t_dw = 33.0 * (double)px * (p.kb / 64.0);
          const double t_mma = (double)na * (p.kb / 16.0) * ((double)px / 2.0 > 58.0 ? (double)px / 2.0 : 58.0);
          const double units = (double)((px + 63) / 64);
          const double t_epi = 2000.0 * units * (na > 1 ? 2.0 * na : 1.0);  // (one set of accumulators: not hidden)
          const double cost = waves * ((double)p.cblocks * (t_dw > t_mma ? t_dw : t_mma) + t_epi + 4000.0);
          if (cost < best_blk) {
            best_blk = cost;
            bth = th; btn = tn; bna = na;
          }
        }
      }
    }
    if (bth == 0) return false;
    best_th = bth;
    best_tn = btn;
    best_ks = 0;
    best_shared = 0;
    p.nacc = bna;
    const int64_t tiles = (int64_t)((g.n + btn - 1) / btn) * ((g.p + bth - 1) / bth) * ((p.mtiles + bna - 1) / bna);
    best_grid = (int)(tiles < sms ? tiles : sms);
  }
  p.th = best_th;
  p.tn = best_tn;
  p.tiles_h = (g.p + p.th - 1) / p.th;
  p.tiles_n = (g.n + p.tn - 1) / p.tn;
  p.ncols = (p.tn * p.th * p.pitch - junk + 15) / 16 * 16;
  int64_t total = (int64_t)p.tiles_n * p.tiles_h * mg;
  if (p.nacc > 1) {  // (blocks: one group, so mg == mtiles)
    p.mtiles = (p.mtiles + p.nacc - 1) / p.nacc;
    total = (int64_t)p.tiles_n * p.tiles_h * p.mtiles * g.group;
  }
  if (p.pair) {
    p.ncols_sub = (p.tn * p.th * p.pitch - junk + 7) / 8 * 8;
    p.ncols = 2 * p.ncols_sub;
    p.mtiles = (g.kg + 255) / 256;
    total = ((int64_t)p.tiles_n * p.tiles_h + 1) / 2 * p.mtiles * g.group;
  }
  if (total > 0x7fffffffLL) return false;
  p.total_tiles = (int32_t)total;
  // weight tile rows: 128, or 64 when the layer has at most 64 output channels per group (the MMA
  // still reads 128 rows: the upper 64 come from whatever follows in shared memory and land in
  // accumulator lanes that no epilogue warp reads; half the tile bytes, one more ring stage)
  p.a_rows = g.kg <= 64 ? 64 : 128;
  p.dup_log2 = 0;
  p.fine_units = 0;
  const uint32_t box_rows = (uint32_t)(p.tn * p.th * p.pitch);
  p.b_bytes = box_rows * p.kb * 2u;
  // rows the MMA may touch: the last tap starts (S-1)*dil rows in and reads ncols rows
  uint32_t rows = (uint32_t)(p.halo ? (g.s - 1) * g.dil_w : 0) + (uint32_t)(p.pair ? p.ncols_sub : p.ncols);
  if (rows < box_rows) rows = box_rows;
  p.b_alloc = (uint32_t)round_up_sz((size_t)rows * p.kb * 2u, 1024);
  // the epilogue stages fp16 tiles for TMA stores when every staged run of pixels starts on a
  // 16-byte boundary of y: Q % 8 == 0 (so P*Q % 8 == 0 too) and one image per tile
  // (or, when the tile has no junk columns, plane and tile sizes are multiples of 8 pixels)
  p.tma_store = (p.tn == 1 && ((g.q % 8) == 0 || (p.pitch == g.q && ((int64_t)g.p * g.q) % 8 == 0 &&
                                                  ((int64_t)p.th * g.q) % 8 == 0)))
                    ? 1
                    : 0;
  p.rem = (p.th * g.q) % kPassElems;
  // epilogue warps: 16 when the main loop of a tile is shorter than its epilogue (1x1 layers of
  // few input channels, stems) and the layer takes the TMA-store epilogue, else 8
  p.epi_warps = kEpilogueWarps;
  if (p.tma_store && mpt * 130.0 < 600.0 + 10.0 * p.ncols && (p.th * g.q) > 2 * kPassElems)
    p.epi_warps = kEpilogueWarpsWide;
  if (p.y_nhwc) {
    // channels-last output: up to 64 pixels x 32 channels staged for TMA stores when the groups
    // have whole blocks of 32 output channels (the weight rows are then interleaved for the
    // transposing staging stores), else plain stores (any shape)
    p.tma_store = (g.kg % 32) == 0 ? 1 : 0;
    p.y_perm = p.tma_store;
    p.y_rpu = g.q > 32 ? 1 : (kPassElems / g.q < p.th ? kPassElems / g.q : p.th);
    p.y_full_w = g.q > kPassElems ? kPassElems : p.y_rpu * g.q;
    p.rem = g.q > kPassElems ? g.q % kPassElems : (p.th % p.y_rpu) * g.q;
    p.epi_warps = kEpilogueWarps;
    if (p.tma_store && mpt * 130.0 < 600.0 + 10.0 * p.ncols && p.tn * p.th * ((g.q + kPassElems - 1) / kPassElems) > 2)
      p.epi_warps = kEpilogueWarpsWide;
  }
  p.sk_split = best_shared;
  p.grid = best_grid;
  // Layers of exactly 64 output channels and a short reduction whose tiles are bound by the
  // epilogue (the wide epilogue was chosen): the weight tensor is laid out twice, one copy after the
  // other, the weight tile is 128 rows again, and all lane quarters hold real channels (see the kernel).
  if (p.epi_warps == kEpilogueWarpsWide && !p.y_nhwc && p.tma_store && g.group == 1 && best_ks == 0 && !best_shared &&
      !want_pair && g.dw_stride == 0 && g.kg == 64 && mpt <= 8.0) {
    // (measured: VGG conv1_1 47.5 -> 41.1 us, 1x1 layers 32 -> 64 and 64 -> 64 channels 7 % faster;
    //  with a longer reduction the doubled weight traffic costs more than the epilogue gains, and
    //  four copies of a 32-channel layer were slower than one)
    p.dup_log2 = 1;
    p.a_rows = 128;
    // a tile's units of 64 pixels x 32 channels are fewer than the warps that can now take them:
    // units of 32 pixels (stored through the remainder map, whose box is then 32 pixels)
    const int px = p.th * g.q;
    if (px % 32 == 0 && ((px + 63) / 64) * (g.kg / 32) < p.epi_warps) p.fine_units = 1;
  }
  p.a_bytes = (uint32_t)p.a_rows * p.kb * 2u;
  p.sk_cols32 = (p.ncols + 31) / 32;
  if (p.pair || p.sk_split || g.dw_stride > 0 || p.gather) p.epi_warps = kEpilogueWarps;
  // split reduction (chosen with the tile shape above): fp32 partials, copy-style epilogue
  p.ks_log2 = best_ks;
  if (p.ks_log2 > 0) {
    p.epi_warps = kEpilogueWarps;
    p.tma_store = 0;
  }
  // Whole-plane tiles whose 32-channel blocks are contiguous, 16-byte aligned runs in y: one bulk
  // copy per block (epilogue_planes)
  p.plane_store = 0;
  p.plane_bytes = 0;
  {
    const int64_t pq = (int64_t)g.p * g.q;
    // (1x1 layers: no junk columns between the rows of a tile.  With them, 3x3 layers on 14x14, the
    //  row-by-row accumulator loads made this form slower than the copy epilogue: 22.1 against 20.7 us.)
    //  Strided layers never share a tile between taps, so their columns are pixels as well.
    const bool linear_cols = (g.r == 1 && g.s == 1) || !p.halo;
    if (!p.tma_store && !p.y_nhwc && p.ks_log2 == 0 && !p.pair && !p.sk_split && g.group == 1 && g.dw_stride == 0 && linear_cols &&
        p.th == g.p && !p.patch && !p.window && pq > 1 && pq <= 256 && (g.k % 32) == 0 && p.epi_warps == kEpilogueWarps) {
      // one image per tile: the two warps of a lane quarter share a staging tile; several: one each
      p.plane_store = p.tn == 1 ? 1 : 2;
      p.plane_bytes = (uint32_t)round_up_sz((size_t)(32 * pq * 2), 128) * (uint32_t)p.plane_store;
    }
  }
  const size_t stage_buf_bytes = p.plane_store ? (size_t)4 * p.plane_bytes : (size_t)p.epi_warps * kWarpStageBytes;
  // rings: B two or three deep, A with what is left (each A stage feeds kb/16 MMAs).  227 KB per
  // CTA minus alignment slack, static barriers and the two epilogue staging buffers.
  size_t budget_all = 232448u - 1024u - 512u;
  p.dw_in_h = p.dw_in_w = 0;
  p.dw_in_bytes = p.dw_in_alloc = 0;
  if (g.dw_stride > 0) {
    p.dw_in_h = (p.th - 1) * g.dw_stride + 3;
    p.dw_in_w = (g.q - 1) * g.dw_stride + 3;
    p.dw_in_bytes = (uint32_t)((size_t)p.tn * p.dw_in_h * p.dw_in_w * p.kb * 2);
    // (a pair of outputs at the end of a row reads up to two pixels past the tile)
    p.dw_in_alloc = (uint32_t)round_up_sz((size_t)p.dw_in_bytes + 2u * p.kb * 2u, 1024);
    budget_all -= 2u * p.dw_in_alloc;
  }
  const size_t budget = budget_all - stage_buf_bytes;
  // ring of stages: one activation tile + `taps` weight tiles each, at least two deep; if the
  // S taps of a kernel row do not fit twice, fall back to one tap (and its own tile) per stage
  for (;;) {
    p.taps = p.halo ? p.eff_s : 1;
    p.pitch = p.dense_rows ? p.dense_pitch : (p.halo ? g.q + (g.s - 1) * g.dil_w : g.q);
    const uint32_t box_rows2 = (uint32_t)(p.tn * (p.vhalo ? (p.th - 1) * g.stride_h + g.r : p.th) * p.pitch);
    p.b_bytes = box_rows2 * p.kb * 2u;
    uint32_t rows2 = (uint32_t)(p.halo ? (g.s - 1) * g.dil_w : 0) + (uint32_t)(p.pair ? p.ncols_sub : p.ncols);
    if (rows2 < box_rows2) rows2 = box_rows2;
    p.b_alloc = (uint32_t)round_up_sz((size_t)rows2 * p.kb * 2u, 1024);
    if (p.dense_rows) {
      // 16 bytes per pixel of the tile's rows; the last window read starts at column ncols - 1
      p.b_bytes = box_rows2 * 16u;
      const size_t reach = ((size_t)(p.vhalo ? (g.r - 1) * p.pitch : 0) + p.ncols + p.cw / 8) * 16u;
      p.b_alloc = (uint32_t)round_up_sz(reach > p.b_bytes ? reach : (size_t)p.b_bytes, 1024);
    }
    if (p.nchw) {
      p.nblk = (p.ncols + 63) / 64;
      p.b_bytes = (uint32_t)p.nblk * (uint32_t)p.kb * 128u;
      p.b_alloc = p.b_bytes;
    }
    p.stage_bytes = p.b_alloc + (uint32_t)(p.nacc > 1 ? p.nacc : 1) * (uint32_t)p.taps * p.a_bytes;
    p.stages = (int)(budget / p.stage_bytes);
    if (p.stages > 8) p.stages = 8;
    if (p.stages >= 2) break;
    if (!p.halo) return false;
    // without sharing, the accumulator pitch is Q again: the tile found above still fits
    p.halo = 0;
    if (p.vhalo) {  // dense rows: the kernel rows take a stage each again, same columns
      p.vhalo = 0;
      p.eff_r = g.r;
      p.eff_s = 1;
    } else if (p.pair) {
      p.ncols_sub = (p.tn * p.th * g.q + 7) / 8 * 8;
      p.ncols = 2 * p.ncols_sub;
    } else {
      p.ncols = (p.tn * p.th * g.q + 15) / 16 * 16;
    }
  }
  // a second staging tile per epilogue warp (its store overlaps the next unit) if memory is left
  p.nbuf = (!p.plane_store && (size_t)p.stages * p.stage_bytes + 2u * stage_buf_bytes <= budget_all) ? 2 : 1;
  p.smem_bytes = (size_t)p.stages * p.stage_bytes + (size_t)p.nbuf * stage_buf_bytes + 2u * p.dw_in_alloc + 1024;
  // more than half of an SM's shared memory: at most one CTA per SM, so that the kernel can take
  // all 512 TMEM columns without ever waiting for another CTA to free them
  if (p.smem_bytes < 120u * 1024u) p.smem_bytes = 120u * 1024u;
  // ring stages per tile as the kernel walks them; equal ranges need the stage count the cost
  // model assumed (the ring fitted with the taps of a kernel row sharing a stage)
  p.ts = p.cblocks * p.eff_r * (p.eff_s / p.taps);
  if (p.sk_split && p.ts != ts_est) {
    p.sk_split = 0;
    const int units = p.pair ? sms / 2 : sms;
    p.grid = (int)(p.total_tiles < units ? p.total_tiles : units);
  }
  // workspace: header (status word, hand-over flags), re-laid-out weights, NHWC input
  p.ws_status_off = 0;
  p.ws_w_off = kWsHeaderBytes;
  p.ws_x_off = p.ws_w_off + round_up_sz(((size_t)g.k << p.dup_log2) * p.eff_r * p.eff_s * p.cw * 2, 256);
  p.ws_part_off = 0;
  p.ws_total = p.ws_x_off + ((p.nchw || p.x_nhwc) ? 0
                                    : round_up_sz(p.patch    ? (size_t)g.n * g.p * g.q * p.cw * 2
                                                  : p.window ? (size_t)g.n * p.hp * p.wp * p.px_ch * 2 + 256
                                                           : (size_t)g.n * g.h * g.w * p.c_pad * 2, 256));
  if (p.ks_log2 > 0) {
    p.ws_part_off = p.ws_total;
    p.ws_total += round_up_sz(((size_t)g.n * g.k * g.p * g.q * 4) << p.ks_log2, 256);
  }
  // Layout pass inside the tensor-core kernel (extra warps convert x while the MMAs run; a tile
  // waits for the segments it reads): layers that take the plain NHWC copy of x, planes of a
  // multiple of 4 pixels, whole 8-channel chunks, 8 epilogue warps, NCHW output.
  p.fuse_layout = 0;
  p.ws_lay_off = 0;
  // On request (HGC_FLAG_FUSED_LAYOUT), with the TMA-store epilogue (planes whose rows are whole
  // 16-byte vectors: the large ones, where the copy is worth hiding).  Measured: the VGG-16 layers
  // take as long as with the separate pass (conv1_2 116 us against 112, conv3_2 65 against 61):
  // they run under the power cap, and on small inputs the first tiles wait for their rows.
  if (!g.no_fuse && !p.nchw && !p.x_nhwc && !p.window && !p.patch && !p.pair && !p.sk_split && p.ks_log2 == 0 &&
      !p.y_nhwc && p.tma_store && p.kb >= 32 && p.epi_warps == kEpilogueWarps && ((int64_t)g.h * g.w) % 4 == 0 &&
      (g.c % 8) == 0 && (int64_t)g.h * g.w <= 0x7fffffffLL / 4 && sms <= kMaxGrid) {
    p.fuse_layout = 1;
    const int hw = g.h * g.w;
    p.lay_px = (hw % 8) == 0 ? 8 : 4;
    p.lay_ch = p.c_pad >= 64 ? 8 : 4;
    const int unit_px = (32 / p.lay_ch) * p.lay_px;
    p.lay_units_p = (hw + unit_px - 1) / unit_px;
    p.lay_units_c = (p.c_pad / 8 + p.lay_ch - 1) / p.lay_ch;
    // segments of about 512 pixels (at least one unit)
    p.lay_seg_units = 512 / unit_px > 0 ? 512 / unit_px : 1;
    p.lay_segs = (p.lay_units_p + p.lay_seg_units - 1) / p.lay_seg_units;
    p.ws_lay_off = p.ws_total;
    p.ws_total += round_up_sz(((size_t)g.n * p.lay_segs + 1) * sizeof(int), 256);
  }
  p.ws_sk_off = 0;
  if (p.sk_split) {  // one hand-over slot per CTA: [sk_cols32 * 32 columns][128 lanes] fp32
    p.ws_sk_off = p.ws_total;
    p.ws_total += (size_t)(p.grid << p.pair) * p.sk_cols32 * 32 * 128 * 4;
  }
  *out = p;
  return true;
}
}  // namespace

// The 5-D map (channel in group, group, W, H, N) over a channels-last activation tensor at `base`:
// the NHWC copy in the workspace, or the caller's x itself when it is channels-last already.
bool encode_nhwc_map(const ConvGeom& g, IgemmPlan* p, void* base) {
  PFN_cuTensorMapEncodeTiled_v12000 enc = encode_fn();
  if (enc == nullptr) return false;
  const CUtensorMapSwizzle sw = p->kb == 64 ? CU_TENSOR_MAP_SWIZZLE_128B
                               : p->kb == 32 ? CU_TENSOR_MAP_SWIZZLE_64B
                                             : CU_TENSOR_MAP_SWIZZLE_32B;
  const cuuint64_t cdim = g.group > 1 ? (cuuint64_t)g.cg : (cuuint64_t)p->c_pad;
  const cuuint64_t pix = (cuuint64_t)p->c_pad * 2;
  cuuint64_t dims[5] = {cdim, (cuuint64_t)g.group, (cuuint64_t)g.w, (cuuint64_t)g.h, (cuuint64_t)g.n};
  cuuint64_t strides[4] = {g.group > 1 ? (cuuint64_t)g.cg * 2 : pix, pix, pix * g.w, pix * g.w * g.h};
  const cuuint32_t box_w = p->halo ? (cuuint32_t)p->pitch : (cuuint32_t)(p->tw * g.stride_w);
  cuuint32_t box[5] = {(cuuint32_t)p->kb, 1, box_w, (cuuint32_t)(p->th * g.stride_h), (cuuint32_t)p->tn};
  cuuint32_t es[5] = {1, 1, (cuuint32_t)g.stride_w, (cuuint32_t)g.stride_h, 1};
  return enc(&p->tmB, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 5, base, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
             sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Depthwise + pointwise block: the 5-D map (channel, -, W, H, N) over the block's channels-last
// input; a box is the input tile of one pixel tile and channel block with its one-pixel border
// (zero padding = out-of-bounds fill), dense in shared memory.
bool encode_dw_input_map(const DwBlock& dw, int n, IgemmPlan* p) {
  PFN_cuTensorMapEncodeTiled_v12000 enc = encode_fn();
  if (enc == nullptr) return false;
  const cuuint64_t pix = (cuuint64_t)dw.c * 2;
  cuuint64_t dims[5] = {(cuuint64_t)dw.c, 1, (cuuint64_t)dw.w, (cuuint64_t)dw.h, (cuuint64_t)n};
  cuuint64_t strides[4] = {pix, pix, pix * dw.w, pix * dw.w * dw.h};
  cuuint32_t box[5] = {(cuuint32_t)p->kb, 1, (cuuint32_t)p->dw_in_w, (cuuint32_t)p->dw_in_h, (cuuint32_t)p->tn};
  cuuint32_t es[5] = {1, 1, 1, 1, 1};
  return enc(&p->tmB, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 5, const_cast<__half*>(dw.x), dims, strides, box, es,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Encodes the two tensor maps over the workspace tensors.  Returns false on failure.
bool igemm_encode_maps(const ConvGeom& g_layer, IgemmPlan* p, void* ws) {
  const ConvGeom g = effective_geom(g_layer, *p);
  PFN_cuTensorMapEncodeTiled_v12000 enc = encode_fn();
  if (enc == nullptr) return false;
  char* base = static_cast<char*>(ws);
  const CUtensorMapSwizzle sw = p->kb == 64 ? CU_TENSOR_MAP_SWIZZLE_128B
                               : p->kb == 32 ? CU_TENSOR_MAP_SWIZZLE_64B
                                             : CU_TENSOR_MAP_SWIZZLE_32B;
  {
    // w'[group][K/g][tap][cw] as (channel of the tap, output channel, tap, group): one box holds
    // the kb-channel slices of `taps` consecutive taps for 128 (64) output channels, tap-major in
    // shared memory, i.e. one K-major weight tile per tap
    const cuuint64_t ntaps = (cuuint64_t)p->eff_r * p->eff_s;
    const cuuint64_t kred = ntaps * p->cw;
    cuuint64_t dims[4] = {(cuuint64_t)p->cw, (cuuint64_t)g.kg << p->dup_log2, ntaps, (cuuint64_t)g.group};  // (replicas: group == 1)
    cuuint64_t strides[3] = {kred * 2, (cuuint64_t)p->cw * 2, kred * 2 * (cuuint64_t)g.kg};
    cuuint32_t box[4] = {(cuuint32_t)p->kb, (cuuint32_t)p->a_rows, (cuuint32_t)p->taps, 1};
    cuuint32_t es[4] = {1, 1, 1, 1};
    if (enc(&p->tmA, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, base + p->ws_w_off, dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return false;
  }
  if (p->nchw) {
    // the activation map is over the caller's x and is encoded when x is known (igemm_encode_x_map)
  } else if (p->patch) {
    // x''[N][P][Q][kelems] as (element, -, output column, output row, image)
    const cuuint64_t pix = (cuuint64_t)p->cw * 2;
    cuuint64_t dims[5] = {(cuuint64_t)p->cw, 1, (cuuint64_t)g.q, (cuuint64_t)g.p, (cuuint64_t)g.n};
    cuuint64_t strides[4] = {pix, pix, pix * (cuuint64_t)g.q, pix * (cuuint64_t)g.q * (cuuint64_t)g.p};
    cuuint32_t box[5] = {(cuuint32_t)p->kb, 1, (cuuint32_t)p->tw, (cuuint32_t)p->th, (cuuint32_t)p->tn};
    cuuint32_t es[5] = {1, 1, 1, 1, 1};
    if (enc(&p->tmB, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 5, base + p->ws_x_off, dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return false;
  } else if (p->window && p->dense_rows) {
    // (8 pixels x 8 channels = 128 bytes, block of 8 pixels, -, padded input row, image): whole
    // rows of the bordered copy, dense in shared memory
    const cuuint64_t row_bytes = (cuuint64_t)p->wp * p->px_ch * 2;
    const cuuint32_t blocks = (cuuint32_t)(row_bytes / 128);
    cuuint64_t dims[5] = {64, blocks, 1, (cuuint64_t)p->hp, (cuuint64_t)g.n};
    cuuint64_t strides[4] = {128, row_bytes, row_bytes, row_bytes * (cuuint64_t)p->hp};
    cuuint32_t box[5] = {64, blocks, 1,
                         (cuuint32_t)(p->vhalo ? (p->th - 1) * g.stride_h + g.r : p->th * g.stride_h),
                         (cuuint32_t)p->tn};
    cuuint32_t es[5] = {1, 1, 1, (cuuint32_t)(p->vhalo ? 1 : g.stride_h), 1};
    if (enc(&p->tmB, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 5, base + p->ws_x_off, dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return false;
  } else if (p->window) {
    // (window element, -, output column, padded input row, image): the column stride is stride_w
    // pixels of 16 bytes, i.e. consecutive windows overlap
    const cuuint64_t pix = 16;
    cuuint64_t dims[5] = {(cuuint64_t)p->cw, 1, (cuuint64_t)g.q, (cuuint64_t)p->hp, (cuuint64_t)g.n};
    cuuint64_t strides[4] = {pix, pix * (cuuint64_t)g.stride_w, pix * (cuuint64_t)p->wp,
                             pix * (cuuint64_t)p->wp * (cuuint64_t)p->hp};
    cuuint32_t box[5] = {(cuuint32_t)p->kb, 1, (cuuint32_t)p->tw, (cuuint32_t)(p->th * g.stride_h), (cuuint32_t)p->tn};
    cuuint32_t es[5] = {1, 1, 1, (cuuint32_t)g.stride_h, 1};
    if (enc(&p->tmB, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 5, base + p->ws_x_off, dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return false;
  } else if (p->x_nhwc) {
    // the activation map is over the caller's x (channels-last) and is encoded when x is known
  } else if (!encode_nhwc_map(g, p, base + p->ws_x_off)) {
    return false;
  }
  p->maps_ready = true;
  return true;
}

// 1x1 layers that read x directly: x[N][C][H*W] seen as (pixel, channel, image), 64 pixels x kb
// channels per box, 128-byte swizzle (pixel-major operand tiles).
bool igemm_encode_x_map(const ConvGeom& g, IgemmPlan* p, const void* x) {
  PFN_cuTensorMapEncodeTiled_v12000 enc = encode_fn();
  if (enc == nullptr) return false;
  const cuuint64_t hw = (cuuint64_t)g.h * g.w;
  cuuint64_t dims[3] = {hw, (cuuint64_t)g.c, (cuuint64_t)g.n};
  cuuint64_t strides[2] = {hw * 2, hw * 2 * (cuuint64_t)g.c};
  cuuint32_t box[3] = {64, (cuuint32_t)p->kb, 1};
  cuuint32_t es[3] = {1, 1, 1};
  if (enc(&p->tmB, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void*>(x), dims, strides, box, es,
          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  p->x_mapped = x;
  return true;
}

// Tensor maps of the output y[N][K][P*Q] seen as (pixels, channels of a group, groups, images):
// one with a 64-pixel box and one with the narrower box of a tile's last staged pass.
bool igemm_encode_y_maps(const ConvGeom& g, IgemmPlan* p, void* y) {
  PFN_cuTensorMapEncodeTiled_v12000 enc = encode_fn();
  if (enc == nullptr) return false;
  const cuuint64_t pq = (cuuint64_t)g.p * g.q;
  if (p->y_nhwc) {
    // y[N][P*Q][group][kg]: a store is up to 64 pixels of one row x 32 channels, dense in smem
    cuuint64_t dims[4] = {(cuuint64_t)g.kg, (cuuint64_t)g.group, pq, (cuuint64_t)g.n};
    cuuint64_t strides[3] = {(cuuint64_t)g.kg * 2, (cuuint64_t)g.k * 2, pq * 2 * (cuuint64_t)g.k};
    cuuint32_t es[4] = {1, 1, 1, 1};
    const cuuint32_t full_w = (cuuint32_t)p->y_full_w;
    for (int i = 0; i < 2; ++i) {
      cuuint32_t box[4] = {32, 1, (i == 0 || p->rem == 0) ? full_w : (cuuint32_t)p->rem, 1};
      if (enc(i == 0 ? &p->tmY : &p->tmYr, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, y, dims, strides, box, es,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    }
    p->y_mapped = y;
    return true;
  }
  cuuint64_t dims[4] = {pq, (cuuint64_t)g.kg, (cuuint64_t)g.group, (cuuint64_t)g.n};
  cuuint64_t strides[3] = {pq * 2, pq * 2 * (cuuint64_t)g.kg, pq * 2 * (cuuint64_t)g.k};
  cuuint32_t es[4] = {1, 1, 1, 1};
  for (int i = 0; i < 2; ++i) {
    cuuint32_t box[4] = {(cuuint32_t)(i == 0 ? kPassElems : (p->fine_units ? 32 : (p->rem == 0 ? kPassElems : p->rem))), 32, 1, 1};
    if (enc(i == 0 ? &p->tmY : &p->tmYr, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, y, dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return false;
  }
  p->y_mapped = y;
  return true;
}

cudaError_t launch_igemm(const ConvGeom& g_layer, IgemmPlan& p, void* ws, const __half* x, const __half* bias, __half* y,
                         int relu, cudaStream_t stream, const DwBlock* dw) {
  const ConvGeom g = effective_geom(g_layer, p);
  if (!p.maps_ready) return cudaErrorInvalidValue;
  if (dw != nullptr && (!p.x_nhwc || p.pair || p.sk_split || p.ks_log2 > 0 || p.fuse_layout || p.kb < 32))
    return cudaErrorInvalidValue;
  if (p.nchw && !p.gather && p.x_mapped != x && !igemm_encode_x_map(g, &p, x)) return cudaErrorInvalidValue;
  if (dw != nullptr && p.x_mapped != x) {  // the block's input tiles come from x (channels-last) with their border
    if (p.dw_in_bytes == 0 || !encode_dw_input_map(*dw, g.n, &p)) return cudaErrorInvalidValue;
    p.x_mapped = x;
  }
  if (dw == nullptr && p.x_nhwc && p.x_mapped != x) {
    if (!encode_nhwc_map(g, &p, const_cast<__half*>(x))) return cudaErrorInvalidValue;
    p.x_mapped = x;
  }
  if (p.tma_store && p.y_mapped != y && !igemm_encode_y_maps(g_layer, &p, y)) return cudaErrorInvalidValue;  // (y is the layer's)
  IgemmArgs a{};
  a.N = g.n; a.K = g.k; a.P = g.p; a.Q = g.q;
  a.kg = g.kg; a.group = g.group;
  a.R = p.eff_r; a.S = p.eff_s; a.pad_h = p.eff_pad_h; a.pad_w = p.eff_pad_w;
  a.stride_h = g.stride_h; a.stride_w = g.stride_w; a.dil_h = g.dil_h; a.dil_w = g.dil_w;
  if (p.patch) { a.stride_h = a.stride_w = a.dil_h = a.dil_w = 1; }  // 1x1 over the expanded input
  a.kb = p.kb; a.cblocks = p.cblocks; a.cw = p.cw;
  a.halo = p.halo; a.tn = p.tn; a.th = p.th; a.pitch = p.pitch; a.ncols = p.ncols;
  a.tiles_h = p.tiles_h; a.tiles_px = p.tiles_h * p.tiles_n; a.mtiles = p.mtiles;
  a.total_tiles = p.total_tiles; a.stages = p.stages; a.taps = p.taps; a.stage_bytes = p.stage_bytes;
  a.a_bytes = p.a_bytes; a.b_bytes = p.b_bytes; a.b_alloc = p.b_alloc;
  // instruction descriptor: D = f32, A = B = f16, both K-major, N >> 3 at bit 17, M >> 4 at bit 24
  a.idesc = (1u << 4) | ((uint32_t)(p.ncols >> 3) << 17) | (((p.pair ? 256u : 128u) >> 4) << 24);
  if (p.nchw) a.idesc |= 1u << 16;  // activation operand is pixel-major (MN-major)
  // shared-memory descriptor: 8-row groups are 8 * row bytes apart; descriptor version 1;
  // swizzle mode 2 = 128 B, 4 = 64 B, 6 = 32 B
  const uint64_t sbo = (uint64_t)(8 * p.kb * 2) >> 4;
  const uint64_t layout = p.kb == 64 ? 2 : (p.kb == 32 ? 4 : 6);
  a.desc_hi = (1ull << 16) | (sbo << 32) | (1ull << 46) | (layout << 61);
  a.desc_hi_b = a.desc_hi;
  a.b_kstep = 2;  // 16 channels = 32 bytes along a swizzled K-major row
  a.nchw = p.nchw; a.nblk = p.nblk; a.cg = g.cg;
  if (p.nchw) {
    // pixel-major tile: 64-pixel blocks of kb channel rows (128 bytes each, 128-byte swizzle):
    // leading offset = one block, stride offset = 8 channel rows; 16 channels = 2048 bytes
    const uint64_t lbo = (uint64_t)(p.kb * 128) >> 4;
    a.desc_hi_b = (lbo << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
    a.b_kstep = 2048 >> 4;
  }
  if (p.dense_rows) {
    // unswizzled K-major tile of overlapping windows: a row (pixel) every 16 bytes, the next 16-byte
    // K chunk (the next pixel of the window) 16 bytes on, the next 8 rows 128 bytes on
    a.desc_hi_b = (1ull << 16) | (8ull << 32) | (1ull << 46);
    a.b_kstep = 2;  // 16 window elements = two pixels
    // shared kernel rows: the kernel advances the activation descriptor by dil_w rows of kb
    // elements per tap; one image row is wp pixels of 8 elements
    if (p.vhalo) a.dil_w = p.pitch * 8 / p.kb;
  }
  a.relu = relu;
  a.tma_store = p.tma_store;
  a.plane_store = p.plane_store;
  a.plane_bytes = p.plane_bytes;
  a.rem = p.rem;
  a.nbuf = p.nbuf;
  a.dup_log2 = p.dup_log2;
  a.fine_units = p.fine_units;
  a.rowpair = p.rowpair;
  a.nacc = p.nacc > 0 ? p.nacc : 1;
  a.acc_stride = a.nacc > 1 ? 512 / a.nacc : 0;
  a.mshift = p.pair + (a.nacc == 4 ? 2 : (a.nacc == 2 ? 1 : 0));
  a.ks_log2 = p.ks_log2;
  a.part_stride = (int64_t)g.n * g.k * g.p * g.q;
  a.y_tma = (p.y_nhwc && p.tma_store) ? 1 : 0;
  a.y_full_w = p.y_full_w;
  a.y_rpu = p.y_rpu > 0 ? p.y_rpu : 1;
  a.dbg_drop = debug_drop_copies();
  if (dw != nullptr) {
    a.dw_x = reinterpret_cast<const uint16_t*>(dw->x);
    a.dw_w9 = reinterpret_cast<const uint16_t*>(dw->w9);
    a.dw_b = reinterpret_cast<const uint16_t*>(dw->bias);
    a.dw_h = dw->h; a.dw_wd = dw->w; a.dw_c = dw->c; a.dw_stride = dw->stride; a.dw_relu = dw->relu;
    a.dw_in_h = p.dw_in_h; a.dw_in_w = p.dw_in_w; a.dw_in_bytes = p.dw_in_bytes; a.dw_in_alloc = p.dw_in_alloc;
  }
  a.gather = p.gather;
  a.g_x = reinterpret_cast<const uint16_t*>(x);
  a.g_hw = g.h * g.w;
  a.g_c = g.c;
  a.lay_x = reinterpret_cast<const uint16_t*>(x);
  a.lay_xp = reinterpret_cast<uint16_t*>(static_cast<char*>(ws) + p.ws_x_off);
  a.lay_flags = reinterpret_cast<int*>(static_cast<char*>(ws) + p.ws_lay_off);
  a.lay_c = g.c; a.lay_cpad = p.c_pad; a.lay_ch = p.lay_ch; a.lay_px = p.lay_px;
  a.lay_hw = g.h * g.w; a.lay_w = g.w;
  a.lay_units_p = p.lay_units_p; a.lay_units_c = p.lay_units_c;
  a.lay_seg_units = p.lay_seg_units; a.lay_segs = p.lay_segs;
  a.ts = p.ts;
  a.pair = p.pair;
  a.ncols_sub = p.ncols_sub;
  a.sk_split = p.sk_split;
  a.sk_cols32 = p.sk_cols32;
  a.sk_part = p.sk_split ? reinterpret_cast<float*>(static_cast<char*>(ws) + p.ws_sk_off) : nullptr;
  a.sk_flags = reinterpret_cast<int*>(static_cast<char*>(ws) + p.ws_status_off + kWsFlagsOff);
  float* partials = p.ks_log2 > 0 ? reinterpret_cast<float*>(static_cast<char*>(ws) + p.ws_part_off) : nullptr;
  const int sms = sm_count();
  const int64_t units = (int64_t)p.total_tiles << p.ks_log2;
  dim3 grid((unsigned)(p.ks_log2 > 0 ? (units < sms ? units : sms) : p.grid));
  // CTAs that share a tile wait for one another: all of them must be resident together
  const bool cooperative = p.sk_split != 0;
  int* status = reinterpret_cast<int*>(static_cast<char*>(ws) + p.ws_status_off);
  cudaError_t err = cudaSuccess;
  // four instantiations per (kb, halo): TMA-store epilogue with 8 or 16 epilogue warps, copy
  // epilogue and channels-last epilogue with 8 (each kernel carries only the epilogue it runs: the hot loops are sensitive to
  // the size of the code around them)
#define HGC_LAUNCH_IGEMM_EW(KBV, HALOV, EWV, EPIV, SPLITV)                                                 \
  do {                                                                                                     \
    err = cudaFuncSetAttribute(igemm_kernel<KBV, HALOV, EWV, EPIV, SPLITV>,                                \
                               cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem_bytes);            \
    if (err == cudaSuccess)                                                                                \
      err = launch_kernel_overlapped(igemm_kernel<KBV, HALOV, EWV, EPIV, SPLITV>, grid, dim3(64 + 32 * EWV), \
                          p.smem_bytes, stream, p.tmA, p.tmB, p.tmY, p.tmYr, a, bias, y, partials, status); \
  } while (0)
  // depthwise + pointwise block: its own instantiations (8 epilogue + 8 depthwise warps)
#define HGC_LAUNCH_DWPW_EPI(KBV, EPIV)                                                                     \
  do {                                                                                                     \
    err = cudaFuncSetAttribute(igemm_kernel<KBV, true, 8, EPIV, false, false, false, false, true>,         \
                               cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem_bytes);            \
    if (err == cudaSuccess)                                                                                \
      err = launch_kernel_overlapped(igemm_kernel<KBV, true, 8, EPIV, false, false, false, false, true>, grid, \
                          dim3(64 + 32 * 8 + 32 * kDwWarps), p.smem_bytes, stream, p.tmA, p.tmB, p.tmY,    \
                          p.tmYr, a, bias, y, partials, status);                                           \
  } while (0)
#define HGC_LAUNCH_DWPW(KBV)                                   \
  do {                                                         \
    if (p.y_nhwc) HGC_LAUNCH_DWPW_EPI(KBV, 2);                 \
    else if (p.plane_store) HGC_LAUNCH_DWPW_EPI(KBV, 3);       \
    else if (!p.tma_store) HGC_LAUNCH_DWPW_EPI(KBV, 1);        \
    else HGC_LAUNCH_DWPW_EPI(KBV, 0);                          \
  } while (0)
  // fused layout pass: its own instantiations (8 epilogue + 4 layout warps), launched cooperatively
  // (a tile waits for segments that other CTAs' layout warps convert)
#define HGC_LAUNCH_FUSED_EPI(KBV, HALOV, EPIV)                                                             \
  do {                                                                                                     \
    err = cudaFuncSetAttribute(igemm_kernel<KBV, HALOV, 8, EPIV, false, false, false, true>,               \
                               cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem_bytes);            \
    if (err == cudaSuccess)                                                                                \
      err = launch_kernel_coop(true, igemm_kernel<KBV, HALOV, 8, EPIV, false, false, false, true>, grid,   \
                               dim3(64 + 32 * 8 + 32 * kLayoutWarps), p.smem_bytes, stream, p.tmA, p.tmB,  \
                               p.tmY, p.tmYr, a, bias, y, partials, status);                               \
  } while (0)
#define HGC_LAUNCH_FUSED(KBV, HALOV) HGC_LAUNCH_FUSED_EPI(KBV, HALOV, 0)
  // tiles shared between CTAs: their own instantiations (8 epilogue warps), launched cooperatively
#define HGC_LAUNCH_SHARED_EPI(KBV, HALOV, EPIV)                                                            \
  do {                                                                                                     \
    err = cudaFuncSetAttribute(igemm_kernel<KBV, HALOV, 8, EPIV, false, false, true>,                      \
                               cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem_bytes);            \
    if (err == cudaSuccess)                                                                                \
      err = launch_kernel_coop(true, igemm_kernel<KBV, HALOV, 8, EPIV, false, false, true>, grid,          \
                               dim3(64 + 32 * 8), p.smem_bytes, stream, p.tmA, p.tmB, p.tmY, p.tmYr, a,    \
                               bias, y, partials, status);                                                 \
  } while (0)
#define HGC_LAUNCH_SHARED(KBV, HALOV)                                \
  do {                                                               \
    if (p.y_nhwc) HGC_LAUNCH_SHARED_EPI(KBV, HALOV, 2);              \
    else if (!p.tma_store) HGC_LAUNCH_SHARED_EPI(KBV, HALOV, 1);     \
    else HGC_LAUNCH_SHARED_EPI(KBV, HALOV, 0);                       \
  } while (0)
#define HGC_LAUNCH_IGEMM(KBV, HALOV)                                                              \
  do {                                                                                            \
    if (p.y_nhwc && p.epi_warps == kEpilogueWarpsWide) HGC_LAUNCH_IGEMM_EW(KBV, HALOV, 16, 2, false); \
    else if (p.y_nhwc) HGC_LAUNCH_IGEMM_EW(KBV, HALOV, 8, 2, false);                              \
    else if (p.plane_store) HGC_LAUNCH_IGEMM_EW(KBV, HALOV, 8, 3, false);                         \
    else if (!p.tma_store) HGC_LAUNCH_IGEMM_EW(KBV, HALOV, 8, 1, false);                          \
    else if (p.epi_warps == kEpilogueWarpsWide) HGC_LAUNCH_IGEMM_EW(KBV, HALOV, 16, 0, false);    \
    else HGC_LAUNCH_IGEMM_EW(KBV, HALOV, 8, 0, false);                                            \
  } while (0)
  // CTA pairs: launched as clusters of two, 8 epilogue warps, the three epilogue kinds
#define HGC_LAUNCH_PAIR_EPI(KBV, HALOV, EPIV)                                                                  \
  do {                                                                                                       \
    if (cooperative) {                                                                                       \
      err = cudaFuncSetAttribute(igemm_kernel<KBV, HALOV, 8, EPIV, false, true, true>,                       \
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem_bytes);            \
      if (err == cudaSuccess)                                                                                \
        err = launch_pair(igemm_kernel<KBV, HALOV, 8, EPIV, false, true, true>, p, sms, true,                \
                          dim3(64 + 32 * 8), stream, p.tmA, p.tmB, p.tmY, p.tmYr, a, bias, y, partials, status); \
    } else {                                                                                                 \
      err = cudaFuncSetAttribute(igemm_kernel<KBV, HALOV, 8, EPIV, false, true, false>,                      \
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem_bytes);            \
      if (err == cudaSuccess)                                                                                \
        err = launch_pair(igemm_kernel<KBV, HALOV, 8, EPIV, false, true, false>, p, sms, false,              \
                          dim3(64 + 32 * 8), stream, p.tmA, p.tmB, p.tmY, p.tmYr, a, bias, y, partials, status); \
    }                                                                                                        \
  } while (0)
#define HGC_LAUNCH_PAIR(KBV, HALOV)                                \
  do {                                                             \
    if (p.y_nhwc) HGC_LAUNCH_PAIR_EPI(KBV, HALOV, 2);              \
    else if (!p.tma_store) HGC_LAUNCH_PAIR_EPI(KBV, HALOV, 1);     \
    else HGC_LAUNCH_PAIR_EPI(KBV, HALOV, 0);                       \
  } while (0)
  if (dw != nullptr || p.gather) {
    if (p.kb == 64) HGC_LAUNCH_DWPW(64); else HGC_LAUNCH_DWPW(32);
  } else if (p.pair) {
    if (p.kb == 64) {
      if (p.halo) HGC_LAUNCH_PAIR(64, true); else HGC_LAUNCH_PAIR(64, false);
    } else if (p.kb == 32) {
      if (p.halo) HGC_LAUNCH_PAIR(32, true); else HGC_LAUNCH_PAIR(32, false);
    } else {
      err = cudaErrorInvalidValue;  // (the planner pairs CTAs only with 32- or 64-channel stages)
    }
  } else if (p.fuse_layout) {
    if (p.kb == 64) {
      if (p.halo) HGC_LAUNCH_FUSED(64, true); else HGC_LAUNCH_FUSED(64, false);
    } else if (p.kb == 32) {
      if (p.halo) HGC_LAUNCH_FUSED(32, true); else HGC_LAUNCH_FUSED(32, false);
    } else {
      err = cudaErrorInvalidValue;
    }
  } else if (p.sk_split) {
    if (p.kb == 64) {
      if (p.halo) HGC_LAUNCH_SHARED(64, true); else HGC_LAUNCH_SHARED(64, false);
    } else if (p.kb == 32) {
      if (p.halo) HGC_LAUNCH_SHARED(32, true); else HGC_LAUNCH_SHARED(32, false);
    } else {
      err = cudaErrorInvalidValue;  // (the planner shares tiles only with 32- or 64-channel stages)
    }
  } else
  if (p.ks_log2 > 0) {
    HGC_LAUNCH_IGEMM_EW(64, true, 8, 1, true);  // the one instantiation with a split reduction
  } else
  if (p.kb == 64) {
    if (p.halo) HGC_LAUNCH_IGEMM(64, true); else HGC_LAUNCH_IGEMM(64, false);
  } else if (p.kb == 32) {
    if (p.halo) HGC_LAUNCH_IGEMM(32, true); else HGC_LAUNCH_IGEMM(32, false);
  } else {
    if (p.halo) HGC_LAUNCH_IGEMM(16, true); else HGC_LAUNCH_IGEMM(16, false);
  }
#undef HGC_LAUNCH_IGEMM_EW
#undef HGC_LAUNCH_IGEMM
#undef HGC_LAUNCH_PAIR_EPI
#undef HGC_LAUNCH_PAIR
#undef HGC_LAUNCH_SHARED_EPI
#undef HGC_LAUNCH_SHARED
#undef HGC_LAUNCH_FUSED_EPI
#undef HGC_LAUNCH_FUSED
#undef HGC_LAUNCH_DWPW_EPI
#undef HGC_LAUNCH_DWPW
  if (err != cudaSuccess) return err;
  count_launch();
  if (p.ks_log2 > 0) {
    const int64_t total = a.part_stride;
    int64_t blocks = (total + 255) / 256;
    if (blocks > (int64_t)sms * 16) blocks = (int64_t)sms * 16;
    err = launch_kernel(splitk_finish_kernel, dim3((unsigned)blocks), dim3(256), 0, stream, (const float*)partials,
                        1 << p.ks_log2, a.part_stride, bias, reinterpret_cast<uint16_t*>(y), g.k,
                        (int64_t)g.p * g.q, total, relu);
    if (err != cudaSuccess) return err;
    count_launch();
  }
  return cudaGetLastError();
}

}  // namespace hgc
