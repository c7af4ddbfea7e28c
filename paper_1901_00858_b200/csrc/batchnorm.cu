// Batch norm forward in the form Section 3.1 of the paper describes for narrow arithmetic:
//   * grouped mean: the N*H*W values of a channel are partitioned into groups (one image, one run
//     of at most 2048 consecutive pixels), the mean of every group is taken separately, then the
//     mean of those means (weighted by the group sizes, which only differ for the last run of a
//     plane);
//   * shifting before squaring: the centred value is multiplied by a power of two (1/32 for data
//     with large values, 32 for data with small values, 1 for neither) before it is squared, and
//     the variance is shifted back by the square of that factor afterwards.
// On this GPU every sum is carried in FP32, so neither step is needed to stay in range: they are
// kept because they cost nothing (a grouped mean is how a parallel reduction is organised anyway,
// and scaling by a power of two is exact), and the result is independent of the shift.
//
//   y = (x - mean_c) / sqrt(var_c + eps),  var_c the biased variance, one rounding to FP16.
//
// Three passes over x (group means, group mean squares, normalise), all bound by HBM bandwidth
// (or L2 for tensors that fit): 8 bytes per element.  With stored statistics only the third runs.
// Every reduction has a fixed order: results are deterministic and every block of a channel
// derives bit-identical statistics from the per-group values.
#include "hgc_internal.h"

namespace hgc {
namespace {

constexpr int kBnThreads = 256;
constexpr int kBnWarps = kBnThreads / 32;
constexpr int kBnGroup = 2048;  // elements per group: 64 per lane, eight 16-byte loads

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
  return v;
}

__device__ __forceinline__ float h_lo(uint32_t w) { return __half2float(__ushort_as_half((uint16_t)(w & 0xffffu))); }
__device__ __forceinline__ float h_hi(uint32_t w) { return __half2float(__ushort_as_half((uint16_t)(w >> 16))); }

// Sum over one group of x (SQ == false) or of ((x - mean) * shift)^2 (SQ == true); warp-collective,
// every lane returns the total.  `vec`: the group starts on a 16-byte boundary.
template <bool SQ>
__device__ __forceinline__ float group_sum(const uint16_t* __restrict__ p, int count, bool vec, float mean,
                                           float shift) {
  const int lane = (int)(threadIdx.x & 31u);
  float acc = 0.f;
  int done = 0;
  auto add = [&](const uint4& q) {
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float a = h_lo(w[j]), b = h_hi(w[j]);
      if (SQ) {
        a = (a - mean) * shift;
        b = (b - mean) * shift;
        acc += a * a + b * b;
      } else {
        acc += a + b;
      }
    }
  };
  if (vec) {
    const uint4* pv = reinterpret_cast<const uint4*>(p);
    if (count == kBnGroup) {
      // a full group: the lane's eight loads are issued before the first is used
      uint4 q[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) q[j] = __ldg(pv + lane + 32 * j);
#pragma unroll
      for (int j = 0; j < 8; ++j) add(q[j]);
      return warp_sum(acc);
    }
    const int nvec = count >> 3;
    for (int i = lane; i < nvec; i += 32) add(__ldg(pv + i));
    done = nvec << 3;
  }
  for (int i = done + lane; i < count; i += 32) {
    float a = __half2float(__ushort_as_half(__ldg(p + i)));
    if (SQ) {
      a = (a - mean) * shift;
      acc += a * a;
    } else {
      acc += a;
    }
  }
  return warp_sum(acc);
}

// Weighted mean of the G per-group values of channel c (weights = group sizes), computed by the
// whole block in a fixed order; every thread returns the result.  `red` holds kBnWarps floats.
__device__ __forceinline__ float channel_mean_of_groups(const float* __restrict__ vals, int n_img, int chunks,
                                                        int64_t hw, float* red) {
  const int G = n_img * chunks;
  const int last = (int)(hw - (int64_t)(chunks - 1) * kBnGroup);  // size of the last group of a plane
  float acc = 0.f;
  for (int g = (int)threadIdx.x; g < G; g += kBnThreads) {
    const int cnt = (g % chunks) == chunks - 1 ? last : kBnGroup;
    acc += vals[g] * (float)cnt;
  }
  acc = warp_sum(acc);
  __syncthreads();  // red may still be read from a previous call
  if ((threadIdx.x & 31u) == 0) red[threadIdx.x >> 5] = acc;
  __syncthreads();
  float total = 0.f;
#pragma unroll
  for (int w = 0; w < kBnWarps; ++w) total += red[w];
  return total / ((float)n_img * (float)hw);
}

// pass 1 (SQ == false): vals_out[c][g] = mean of group g.
// pass 2 (SQ == true):  vals_out[c][g] = mean over group g of ((x - mean_c) * shift)^2, mean_c
//                       from the group means of pass 1 (vals_in).
template <bool SQ>
__global__ void __launch_bounds__(kBnThreads)
bn_group_kernel(const uint16_t* __restrict__ x, const float* __restrict__ vals_in, float* __restrict__ vals_out,
                int n_img, int C, int64_t hw, int chunks, float shift) {
  grid_dependency_wait();
  __shared__ float red[kBnWarps];
  const int c = (int)blockIdx.y;
  const int G = n_img * chunks;
  float mean = 0.f;
  if (SQ) mean = channel_mean_of_groups(vals_in + (int64_t)c * G, n_img, chunks, hw, red);
  const bool vec = (hw % 8) == 0;
  const int warp = (int)(threadIdx.x >> 5);
  for (int g = (int)blockIdx.x * kBnWarps + warp; g < G; g += (int)gridDim.x * kBnWarps) {
    const int img = g / chunks, ch = g % chunks;
    const int64_t start = (int64_t)ch * kBnGroup;
    const int count = (int)(hw - start < kBnGroup ? hw - start : kBnGroup);
    const float s = group_sum<SQ>(x + ((int64_t)img * C + c) * hw + start, count, vec, mean, shift);
    if ((threadIdx.x & 31u) == 0) vals_out[(int64_t)c * G + g] = s / (float)count;
  }
}

// pass 3: statistics from the per-group values (or the stored ones), then y.
__global__ void __launch_bounds__(kBnThreads)
bn_apply_kernel(const uint16_t* __restrict__ x, uint16_t* __restrict__ y, const float* __restrict__ group_means,
                const float* __restrict__ group_sq, float* __restrict__ mean_io, float* __restrict__ var_io,
                int use_stored, int n_img, int C, int64_t hw, int chunks, float eps, float inv_shift_sq) {
  grid_dependency_wait();
  __shared__ float red[kBnWarps];
  const int c = (int)blockIdx.y;
  const int G = n_img * chunks;
  float mean, var;
  if (use_stored) {
    mean = mean_io[c];
    var = var_io[c];
  } else {
    mean = channel_mean_of_groups(group_means + (int64_t)c * G, n_img, chunks, hw, red);
    var = channel_mean_of_groups(group_sq + (int64_t)c * G, n_img, chunks, hw, red) * inv_shift_sq;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
      mean_io[c] = mean;
      var_io[c] = var;
    }
  }
  const float inv = 1.0f / sqrtf(var + eps);
  const bool vec = (hw % 8) == 0;
  const int warp = (int)(threadIdx.x >> 5), lane = (int)(threadIdx.x & 31u);
  for (int g = (int)blockIdx.x * kBnWarps + warp; g < G; g += (int)gridDim.x * kBnWarps) {
    const int img = g / chunks, ch = g % chunks;
    const int64_t start = (int64_t)ch * kBnGroup;
    const int count = (int)(hw - start < kBnGroup ? hw - start : kBnGroup);
    const int64_t base = ((int64_t)img * C + c) * hw + start;
    int done = 0;
    if (vec) {
      const uint4* pv = reinterpret_cast<const uint4*>(x + base);
      uint4* py = reinterpret_cast<uint4*>(y + base);
      auto norm = [&](const uint4& q) {
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
        uint32_t o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const __half2 h = __floats2half2_rn((h_lo(w[j]) - mean) * inv, (h_hi(w[j]) - mean) * inv);
          o[j] = *reinterpret_cast<const uint32_t*>(&h);
        }
        return make_uint4(o[0], o[1], o[2], o[3]);
      };
      if (count == kBnGroup) {
        uint4 q[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) q[j] = __ldcs(pv + lane + 32 * j);
#pragma unroll
        for (int j = 0; j < 8; ++j) py[lane + 32 * j] = norm(q[j]);
        continue;
      }
      const int nvec = count >> 3;
      for (int i = lane; i < nvec; i += 32) py[i] = norm(__ldcs(pv + i));
      done = nvec << 3;
    }
    for (int i = done + lane; i < count; i += 32) {
      const float v = (__half2float(__ushort_as_half(x[base + i])) - mean) * inv;
      y[base + i] = __half_as_ushort(__float2half_rn(v));
    }
  }
}

// Folding stored statistics and an optional scale/shift into the convolution before the batch
// norm: a_k = gamma_k / sqrt(var_k + eps); w'[k][j] = w[k][j] * a_k; b'[k] = (b[k] - mean_k) * a_k
// + beta_k.  One block per output channel.
__global__ void __launch_bounds__(256)
bn_fold_kernel(const uint16_t* __restrict__ w, const uint16_t* __restrict__ bias, const float* __restrict__ mean,
               const float* __restrict__ var, const float* __restrict__ gamma, const float* __restrict__ beta,
               float eps, int64_t per_k, uint16_t* __restrict__ w_out, uint16_t* __restrict__ b_out) {
  grid_dependency_wait();
  const int64_t k = blockIdx.x;
  const float a = (gamma != nullptr ? gamma[k] : 1.0f) / sqrtf(var[k] + eps);
  for (int64_t j = threadIdx.x; j < per_k; j += blockDim.x)
    w_out[k * per_k + j] = __half_as_ushort(__float2half_rn(__half2float(__ushort_as_half(w[k * per_k + j])) * a));
  if (threadIdx.x == 0) {
    const float b = bias != nullptr ? __half2float(__ushort_as_half(bias[k])) : 0.f;
    b_out[k] = __half_as_ushort(__float2half_rn(fmaf(b - mean[k], a, beta != nullptr ? beta[k] : 0.f)));
  }
}

int bn_chunks(int64_t hw) { return (int)((hw + kBnGroup - 1) / kBnGroup); }

}  // namespace

size_t batchnorm_workspace_bytes(int32_t n, int32_t c, int64_t hw) {
  return (size_t)2 * (size_t)c * (size_t)n * (size_t)bn_chunks(hw) * sizeof(float);
}

cudaError_t launch_batchnorm(const __half* x, __half* y, int32_t n, int32_t c, int64_t hw, float eps,
                             int32_t shift_log2, int32_t use_stored, float* mean, float* var, void* ws,
                             cudaStream_t stream) {
  const int chunks = bn_chunks(hw);
  const int64_t G = (int64_t)n * chunks;
  // blocks per channel: one group per warp unless that would be far more blocks than the GPU can
  // hold several times over
  int64_t bx = (G + kBnWarps - 1) / kBnWarps;
  const int64_t cap = ((int64_t)sm_count() * 64 + c - 1) / c;
  if (bx > cap) bx = cap;
  if (bx < 1) bx = 1;
  const dim3 grid((unsigned)bx, (unsigned)c);
  const uint16_t* x16 = reinterpret_cast<const uint16_t*>(x);
  float* gm = static_cast<float*>(ws);
  float* gs = gm != nullptr ? gm + (int64_t)c * G : nullptr;
  const float shift = ldexpf(1.0f, shift_log2);
  cudaError_t err;
  if (!use_stored) {
    err = launch_kernel(bn_group_kernel<false>, grid, dim3(kBnThreads), 0, stream, x16, (const float*)nullptr, gm,
                        (int)n, (int)c, hw, chunks, 1.0f);
    if (err != cudaSuccess) return err;
    count_launch();
    err = launch_kernel(bn_group_kernel<true>, grid, dim3(kBnThreads), 0, stream, x16, (const float*)gm, gs, (int)n,
                        (int)c, hw, chunks, shift);
    if (err != cudaSuccess) return err;
    count_launch();
  }
  err = launch_kernel(bn_apply_kernel, grid, dim3(kBnThreads), 0, stream, x16, reinterpret_cast<uint16_t*>(y),
                      (const float*)gm, (const float*)gs, mean, var, (int)use_stored, (int)n, (int)c, hw, chunks, eps,
                      1.0f / (shift * shift));
  if (err != cudaSuccess) return err;
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_bn_fold(const __half* w, const __half* bias, const float* mean, const float* var,
                           const float* gamma, const float* beta, float eps, int32_t k, int64_t per_k, __half* w_out,
                           __half* b_out, cudaStream_t stream) {
  const cudaError_t err =
      launch_kernel(bn_fold_kernel, dim3((unsigned)k), dim3(256), 0, stream, reinterpret_cast<const uint16_t*>(w),
                    reinterpret_cast<const uint16_t*>(bias), mean, var, gamma, beta, eps, per_k,
                    reinterpret_cast<uint16_t*>(w_out), reinterpret_cast<uint16_t*>(b_out));
  if (err != cudaSuccess) return err;
  count_launch();
  return cudaGetLastError();
}

}  // namespace hgc
