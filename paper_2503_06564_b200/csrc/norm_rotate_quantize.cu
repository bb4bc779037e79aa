// LayerNorm and adaLN modulation folded in front of the online transform (Sec. 3.2 Eq. 10 G_t; Sec. 3.1 Eq. 1-2):
//   h[m,k] = (x[m,k] - mean_m) / sqrt(var_m + eps) * (1 + scale[s,k]) + shift[s,k],  s = m / rows_per_sample
//   v = ((h o vec) . BlockDiag(H_128)),  codes = rne(v * fl(127 / amax)),  scale = amax / 127.
// The quantized linears of a transformer block read exactly this tensor; computing it here removes its round trip
// through memory (one bf16 write and one read of [M, K]) and keeps it in fp32 instead of rounding it to bf16.
//
// Layout and arithmetic of the rotation and the quantizer are those of the activation kernel for narrow rows
// (rotate_quantize.cu): four lanes own one 128-block of one row, 32 values each as fp32 pairs, packed fp32x2
// instructions, a CTA owns whole rows.  Row statistics: every lane group forms the mean and the sum of squared
// deviations of its own 128 values, the groups of a row exchange them through shared memory, and every group combines
// them in the same fixed order (mean = average of the block means, M2 = sum of the block M2 + 128 sum (mean_b - mean)^2),
// so the result does not depend on scheduling: the same input always gives the same codes.  One extra barrier per tile;
// the shared statistics alternate between two copies so that none is needed before they are reused.
#include <cuda_bf16.h>

#include <algorithm>

#include "internal.h"
#include "lane_group.cuh"
#include "ptx.cuh"

namespace trdq {
namespace {

__device__ __forceinline__ float group4_sum(float s) {
  s = __fadd_rn(s, __shfl_xor_sync(0xffffffffu, s, 1));
  s = __fadd_rn(s, __shfl_xor_sync(0xffffffffu, s, 2));
  return s;
}

__device__ __forceinline__ float2 bf16x2_to_float2(uint32_t w) {
  return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u));  // exact widening
}

// blockDim.x = rows_per_tile * (K / 128) * 4 rounded up to a warp (at most 320);
// dynamic shared memory: K floats (fused vector) + 2 copies x 2 arrays x rows_per_tile * (K / 128) floats.
template <int MIN_CTAS>
__global__ void __launch_bounds__(320, MIN_CTAS)
norm_rotate_quantize_rows_kernel(const uint16_t* __restrict__ x, int64_t ldx, int32_t M, int32_t K, const float* __restrict__ vec,
                                 const uint16_t* __restrict__ shift, const uint16_t* __restrict__ scale, int32_t rows_per_sample, float eps,
                                 int8_t* __restrict__ codes, float* __restrict__ scales, int32_t rows_per_tile, float zero) {
  extern __shared__ float smem_f[];
  __shared__ unsigned int row_max[3][32];
  float* svec = smem_f;
  float* stats = smem_f + K;
  const int nb = K / TRDQ_BLOCK;
  const int items = rows_per_tile * nb;
  const int lane4 = threadIdx.x & (kFastLanes - 1);
  const int item = threadIdx.x / kFastLanes;
  const bool active = item < items;
  const int r = active ? item / nb : 0;
  const int b = active ? item % nb : 0;
  const float inv_nb = __fdiv_rn(1.0f, static_cast<float>(nb));
  const float inv_k = __fdiv_rn(1.0f, static_cast<float>(K));

  for (int i = threadIdx.x; i < K / 4; i += blockDim.x) reinterpret_cast<float4*>(svec)[i] = __ldg(reinterpret_cast<const float4*>(vec) + i);
  if (threadIdx.x < 32) row_max[0][threadIdx.x] = 0u;
  __syncthreads();
  griddep_launch_dependents();
  griddep_wait();  // x and the modulation rows may be written, and the code buffer still read, by the kernel before

  const int num_tiles = (M + rows_per_tile - 1) / rows_per_tile;
  const int col0 = b * TRDQ_BLOCK + lane4 * 8;  // first element of chunk 0 of this lane; chunk c is 32 further
  const float2* sv = reinterpret_cast<const float2*>(svec + col0);

  uint4 raw[4];
  auto fetch = [&](int tile) {
    const int64_t row = static_cast<int64_t>(tile) * rows_per_tile + r;
    if (active && tile < num_tiles && row < M) {
      const uint4* src = reinterpret_cast<const uint4*>(x + row * ldx + col0);
#pragma unroll
      for (int c = 0; c < 4; ++c) raw[c] = __ldg(src + 4 * c);
    } else {
#pragma unroll
      for (int c = 0; c < 4; ++c) raw[c] = make_uint4(0u, 0u, 0u, 0u);
    }
  };
  fetch(blockIdx.x);

  int it = 0;
  for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++it) {
    const int buf = it % 3;
    if (threadIdx.x < 32) row_max[(it + 1) % 3][threadIdx.x] = 0u;
    const int row = tile * rows_per_tile + r;
    const bool valid = active && row < M;
    float* mean_b = stats + (it & 1) * 2 * items;
    float* m2_b = mean_b + items;

    // v[4c + j] = elements (2j, 2j+1) of chunk c
    float2 v[16];
    widen_chunks_lanes4(raw, v);
    fetch(tile + gridDim.x);  // next tile's rows are in flight while this one is reduced and transformed

    // statistics of this group's 128 values: mean, then the sum of squared deviations from it
    float2 s2 = make_float2(0.0f, 0.0f);
#pragma unroll
    for (int p = 0; p < 16; ++p) s2 = __fadd2_rn(s2, v[p]);
    const float gmean = __fmul_rn(group4_sum(__fadd_rn(s2.x, s2.y)), 0.0078125f);
    const float2 ngm = make_float2(-gmean, -gmean);
    float2 q2 = make_float2(0.0f, 0.0f);
#pragma unroll
    for (int p = 0; p < 16; ++p) {
      const float2 d = __fadd2_rn(v[p], ngm);
      q2 = __ffma2_rn(d, d, q2);
    }
    const float gm2 = group4_sum(__fadd_rn(q2.x, q2.y));
    if (active && lane4 == 0) {
      mean_b[item] = gmean;
      m2_b[item] = gm2;
    }
    __syncthreads();
    // combine the row's blocks in a fixed order: lane l takes blocks l, l + 4, ..., then the shuffle tree
    float sm = 0.0f;
    for (int bb = lane4; bb < nb; bb += 4) sm = __fadd_rn(sm, mean_b[r * nb + bb]);
    const float mean = __fmul_rn(group4_sum(sm), inv_nb);
    float dev = 0.0f, m2 = 0.0f;
    for (int bb = lane4; bb < nb; bb += 4) {
      const float dm = __fsub_rn(mean_b[r * nb + bb], mean);
      dev = __fmaf_rn(dm, dm, dev);
      m2 = __fadd_rn(m2, m2_b[r * nb + bb]);
    }
    const float var = __fmul_rn(__fmaf_rn(128.0f, group4_sum(dev), group4_sum(m2)), inv_k);
    const float rstd = __fdiv_rn(1.0f, __fsqrt_rn(__fadd_rn(var, eps)));

    if (valid) {
      // h = (x - mean) * rstd * (1 + scale) + shift, then the fused vector of the rotation
      const int64_t sidx = static_cast<int64_t>(row / rows_per_sample) * K + col0;
      const float2 nmean = make_float2(-mean, -mean), rstd2 = make_float2(rstd, rstd), one2 = make_float2(1.0f, 1.0f);
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const uint4 sc_raw = scale ? __ldg(reinterpret_cast<const uint4*>(scale + sidx) + 4 * c) : make_uint4(0u, 0u, 0u, 0u);
        const uint4 sh_raw = shift ? __ldg(reinterpret_cast<const uint4*>(shift + sidx) + 4 * c) : make_uint4(0u, 0u, 0u, 0u);
        const uint32_t scw[4] = {sc_raw.x, sc_raw.y, sc_raw.z, sc_raw.w};
        const uint32_t shw[4] = {sh_raw.x, sh_raw.y, sh_raw.z, sh_raw.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float2 n = __fmul2_rn(__fadd2_rn(v[4 * c + j], nmean), rstd2);
          const float2 h = __ffma2_rn(n, __fadd2_rn(one2, bf16x2_to_float2(scw[j])), bf16x2_to_float2(shw[j]));
          v[4 * c + j] = __fmul2_rn(h, sv[16 * c + j]);
        }
      }
    } else {
#pragma unroll
      for (int p = 0; p < 16; ++p) v[p] = make_float2(0.0f, 0.0f);
    }

    wht128_lanes4(v, lane4);

    const float m = absmax_lanes4(v);
    if (valid && lane4 == 0) atomicMax(&row_max[buf][r], __float_as_uint(m));
    __syncthreads();

    if (valid) {
      const float amax = __uint_as_float(row_max[buf][r]);
      quantize_store_lanes4(v, amax, zero, codes + static_cast<int64_t>(row) * K + col0);
      if (b == 0 && lane4 == 0) scales[row] = __fdiv_rn(amax, 127.0f);
    }
  }
}

}  // namespace

cudaError_t launch_norm_rotate_quantize(const void* x_bf16, int64_t ldx, int32_t M, int32_t K, const float* vec, const void* shift_bf16,
                                        const void* scale_bf16, int32_t rows_per_sample, float eps, int8_t* codes, float* scales,
                                        cudaStream_t stream) {
  const int nb = K / TRDQ_BLOCK;
  if (nb > 64) return cudaErrorInvalidValue;  // one row must fit a CTA: K <= 8192
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int rows = rows_per_tile_by_rounds(M, std::max(1, std::min(32, 72 / nb)), sms);  // at most about 72 lane groups (288 threads) per CTA
  const int threads = (rows * nb * kFastLanes + 31) / 32 * 32;
  const size_t smem = (static_cast<size_t>(K) + 4u * rows * nb) * sizeof(float);
  const int num_tiles = (M + rows - 1) / rows;
  const int grid = std::min(num_tiles, sms * 2);
  return launch_overlapped(norm_rotate_quantize_rows_kernel<2>, dim3(grid), dim3(threads), smem, stream,
                           static_cast<const uint16_t*>(x_bf16), ldx, M, K, vec, static_cast<const uint16_t*>(shift_bf16),
                           static_cast<const uint16_t*>(scale_bf16), rows_per_sample, eps, codes, scales, rows, 0.0f);
}

}  // namespace trdq
