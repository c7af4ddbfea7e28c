// FP32 -> FP16 cast: the arithmetic core of a weight-file converter (Section 3.4 of the paper:
// models are stored in FP32 and converted once to an FP16 copy).  Round to nearest even
// (cvt.rn), values of magnitude >= 65520 become infinities as IEEE prescribes; the number of
// FINITE inputs that no finite binary16 can hold is reported so that a converter can warn.
// Bound by HBM bandwidth: 4 bytes read and 2 written per element.
#include "hgc_internal.h"

namespace hgc {
namespace {

__device__ __forceinline__ uint32_t cvt2(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}

// finite, but rounds to an infinity
__device__ __forceinline__ int overflows(float v) { return fabsf(v) >= 65520.f && fabsf(v) < __int_as_float(0x7f800000); }

// a thread converts 8 consecutive elements (two 16-byte loads, one 16-byte store); the elements
// after the last whole group of 8 are converted one by one by the first threads of block 0
__global__ void __launch_bounds__(256)
cast_f32_to_f16_kernel(const float* __restrict__ src, uint16_t* __restrict__ dst, int64_t count,
                       unsigned long long* __restrict__ overflow) {
  grid_dependency_wait();
  const int64_t groups = count >> 3;
  int over = 0;
  for (int64_t gidx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; gidx < groups;
       gidx += (int64_t)gridDim.x * blockDim.x) {
    const float4 a = __ldcs(reinterpret_cast<const float4*>(src) + 2 * gidx);
    const float4 b = __ldcs(reinterpret_cast<const float4*>(src) + 2 * gidx + 1);
    over += overflows(a.x) + overflows(a.y) + overflows(a.z) + overflows(a.w) + overflows(b.x) + overflows(b.y) +
            overflows(b.z) + overflows(b.w);
    reinterpret_cast<uint4*>(dst)[gidx] = make_uint4(cvt2(a.x, a.y), cvt2(a.z, a.w), cvt2(b.x, b.y), cvt2(b.z, b.w));
  }
  if (blockIdx.x == 0) {
    const int64_t i = (groups << 3) + threadIdx.x;
    if (threadIdx.x < 8 && i < count) {
      const float v = src[i];
      over += overflows(v);
      dst[i] = (uint16_t)(cvt2(v, 0.f) & 0xffffu);
    }
  }
  if (overflow != nullptr) {
    // one atomic per warp that saw any
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) over += __shfl_xor_sync(0xffffffffu, over, off);
    if ((threadIdx.x & 31) == 0 && over > 0) atomicAdd(overflow, (unsigned long long)over);
  }
}

}  // namespace

cudaError_t launch_cast_f32_to_f16(const float* src, __half* dst, int64_t count, unsigned long long* overflow,
                                   cudaStream_t stream) {
  if (count <= 0) return cudaSuccess;
  int64_t blocks = ((count >> 3) + 255) / 256;
  const int64_t cap = (int64_t)sm_count() * 16;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  launch_kernel(cast_f32_to_f16_kernel, dim3((unsigned)blocks), dim3(256), 0, stream, src, reinterpret_cast<uint16_t*>(dst), count, overflow);
  count_launch();
  return cudaGetLastError();
}

}  // namespace hgc
