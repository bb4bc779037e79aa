// Fused online transform + dynamic quantizer (Sec. 3.2 Eq. 10, G_t; Sec. 3.1 Eq. 1-2):
// scale by the group's fused vector, rotate every 128-block with a Walsh-Hadamard butterfly
// held in registers, take the absmax of the row (or of the block for 4-bit weights), and
// emit integer codes.  One read of the input, one write of the codes; the rotated values
// never leave the register file.
//
// Work decomposition.  A group of 8 consecutive lanes owns one 128-block of one row: lane l
// holds elements 16*l .. 16*l+15 (two 16-byte loads).  Butterfly stages h = 1, 2, 4, 8 pair
// registers of one thread; stages h = 16, 32, 64 pair lanes l ^ 1, l ^ 2, l ^ 4 by warp
// shuffle.  All additions are separately rounded fp32 operations in this fixed order.
// A CTA owns `rows` consecutive rows at a time (rows * K/128 groups); the row absmax is
// combined through a shared-memory atomic max on the (non-negative) float bit patterns.
#include <cuda_bf16.h>

#include <algorithm>
#include <cstdio>

#include "internal.h"
#include "lane_group.cuh"
#include "ptx.cuh"

namespace trdq {
namespace {

// MODE 0: int8 per row.  MODE 1: int4 per 128-block, packed.
// P = blocks handled by one lane group per tile (P > 1 only for very wide rows).
template <int MODE, int P>
__global__ void __launch_bounds__(1024) rotate_quantize_kernel(const __nv_bfloat16* __restrict__ x, int64_t ldx, int32_t M, int32_t K,
                                                               const float* __restrict__ vec, int8_t* __restrict__ codes,
                                                               uint8_t* __restrict__ packed, float* __restrict__ scales,
                                                               int32_t rows_per_tile, int32_t groups) {
  __shared__ unsigned int row_max[3][32];
  const int nb = K / TRDQ_BLOCK;
  const int lane8 = threadIdx.x & (kLanesPerBlock - 1);
  const int group = threadIdx.x / kLanesPerBlock;
  const int items = rows_per_tile * nb;

  if (MODE == 0) {
    if (threadIdx.x < 32) row_max[0][threadIdx.x] = 0u;
    __syncthreads();
  }

  // per-item placement inside a tile (fixed over the tile loop)
  int r_of[P], b_of[P];
  bool active[P];
  float vreg[P][16];
#pragma unroll
  for (int p = 0; p < P; ++p) {
    const int item = group + p * groups;
    active[p] = (group < groups) && (item < items);
    r_of[p] = active[p] ? item / nb : 0;
    b_of[p] = active[p] ? item % nb : 0;
    const float4* vp = reinterpret_cast<const float4*>(vec + b_of[p] * TRDQ_BLOCK + lane8 * kElemsPerLane);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float4 f = __ldg(vp + j);
      vreg[p][4 * j] = f.x;
      vreg[p][4 * j + 1] = f.y;
      vreg[p][4 * j + 2] = f.z;
      vreg[p][4 * j + 3] = f.w;
    }
  }

  const int num_tiles = (M + rows_per_tile - 1) / rows_per_tile;
  int it = 0;
  for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++it) {
    const int buf = it % 3;
    if (MODE == 0 && threadIdx.x < 32) row_max[(it + 1) % 3][threadIdx.x] = 0u;

    float u[P][16];
    float gmax[P];
    bool valid[P];
#pragma unroll
    for (int p = 0; p < P; ++p) {
      const int64_t row = static_cast<int64_t>(tile) * rows_per_tile + r_of[p];
      valid[p] = active[p] && row < M;
      if (valid[p]) {
        const uint4* src = reinterpret_cast<const uint4*>(x + row * ldx + b_of[p] * TRDQ_BLOCK + lane8 * kElemsPerLane);
        load_scaled16(src, vreg[p], u[p]);
      } else {
#pragma unroll
        for (int i = 0; i < 16; ++i) u[p][i] = 0.0f;
      }
    }
#pragma unroll
    for (int p = 0; p < P; ++p) {
      wht128(u[p], lane8);
      gmax[p] = group_max(absmax16(u[p]));
      if (MODE == 0 && valid[p] && lane8 == 0) atomicMax(&row_max[buf][r_of[p]], __float_as_uint(gmax[p]));
    }
    if (MODE == 0) __syncthreads();

#pragma unroll
    for (int p = 0; p < P; ++p) {
      if (!valid[p]) continue;
      const int64_t row = static_cast<int64_t>(tile) * rows_per_tile + r_of[p];
      const int64_t elem = row * K + b_of[p] * TRDQ_BLOCK + lane8 * kElemsPerLane;
      if (MODE == 0) {
        const float amax = __uint_as_float(row_max[buf][r_of[p]]);
        const float inv = amax > 0.0f ? __fdiv_rn(127.0f, amax) : 0.0f;
        uint32_t out[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          uint32_t word = 0;
#pragma unroll
          for (int b = 0; b < 4; ++b) {
            int q = quantize_one(u[p][4 * j + b], inv);
            q = max(-127, min(127, q));
            word |= (static_cast<uint32_t>(q) & 0xFFu) << (8 * b);
          }
          out[j] = word;
        }
        *reinterpret_cast<uint4*>(codes + elem) = make_uint4(out[0], out[1], out[2], out[3]);
        if (b_of[p] == 0 && lane8 == 0) scales[row] = __fdiv_rn(amax, 127.0f);
      } else {
        const float amax = gmax[p];
        const float inv = amax > 0.0f ? __fdiv_rn(7.0f, amax) : 0.0f;
        uint32_t out[2] = {0u, 0u};
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          int q = quantize_one(u[p][i], inv);
          q = max(-7, min(7, q));
          out[i / 8] |= (static_cast<uint32_t>(q) & 0xFu) << (4 * (i % 8));  // even k -> low nibble of its byte
        }
        *reinterpret_cast<uint2*>(packed + elem / 2) = make_uint2(out[0], out[1]);
        if (lane8 == 0) scales[row * nb + b_of[p]] = __fdiv_rn(amax, 7.0f);
      }
    }
  }
}


// ---------------------------------------------------------------------------------------------
// Full balancing transform of Eq. 9 / Eq. 10:  (x o vec1) . R1-blocks, zigzag permutation, scale by vec2,
// second block rotation, then the quantizer.  Same lane-group layout as the kernel above (8 lanes per
// 128-block).  Between the two rotations the rotated row is parked in shared memory as fp32 so that every
// lane group can gather its 128 permuted channels from anywhere in the row:
//     v2[j] = fl32(v1[perm[j]] * vec2[j]).
// MODE 0: int8 per row.  MODE 1: int4 per 128-block, packed.
// ---------------------------------------------------------------------------------------------
template <int MODE>
__global__ void __launch_bounds__(1024) rotate2_quantize_kernel(const __nv_bfloat16* __restrict__ x, int64_t ldx, int32_t M, int32_t K,
                                                                const float* __restrict__ vec1, const int32_t* __restrict__ perm,
                                                                const float* __restrict__ vec2, int8_t* __restrict__ codes,
                                                                uint8_t* __restrict__ packed, float* __restrict__ scales,
                                                                int32_t rows_per_tile) {
  extern __shared__ float row_buf[];  // [rows_per_tile][K]
  __shared__ unsigned int row_max[3][32];
  const int nb = K / TRDQ_BLOCK;
  const int lane8 = threadIdx.x & (kLanesPerBlock - 1);
  const int group = threadIdx.x / kLanesPerBlock;
  const bool active = group < rows_per_tile * nb;
  const int r = active ? group / nb : 0;
  const int b = active ? group % nb : 0;
  const int col0 = b * TRDQ_BLOCK + lane8 * kElemsPerLane;

  if (threadIdx.x < 32) row_max[0][threadIdx.x] = 0u;
  float v1reg[16], v2reg[16];
  int src[16];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float4 f = __ldg(reinterpret_cast<const float4*>(vec1 + col0) + j);
    const float4 g2 = __ldg(reinterpret_cast<const float4*>(vec2 + col0) + j);
    const int4 pi = __ldg(reinterpret_cast<const int4*>(perm + col0) + j);
    v1reg[4 * j] = f.x, v1reg[4 * j + 1] = f.y, v1reg[4 * j + 2] = f.z, v1reg[4 * j + 3] = f.w;
    v2reg[4 * j] = g2.x, v2reg[4 * j + 1] = g2.y, v2reg[4 * j + 2] = g2.z, v2reg[4 * j + 3] = g2.w;
    src[4 * j] = pi.x, src[4 * j + 1] = pi.y, src[4 * j + 2] = pi.z, src[4 * j + 3] = pi.w;
  }
  __syncthreads();

  const int num_tiles = (M + rows_per_tile - 1) / rows_per_tile;
  int it = 0;
  for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++it) {
    const int buf = it % 3;
    if (threadIdx.x < 32) row_max[(it + 1) % 3][threadIdx.x] = 0u;
    const int64_t row = static_cast<int64_t>(tile) * rows_per_tile + r;
    const bool valid = active && row < M;

    float u[16];
    if (valid) {
      load_scaled16(reinterpret_cast<const uint4*>(x + row * ldx + col0), v1reg, u);
    } else {
#pragma unroll
      for (int i = 0; i < 16; ++i) u[i] = 0.0f;
    }
    wht128(u, lane8);  // first rotation
    if (active) {
      float4* dst = reinterpret_cast<float4*>(row_buf + static_cast<size_t>(r) * K + col0);
#pragma unroll
      for (int j = 0; j < 4; ++j) dst[j] = make_float4(u[4 * j], u[4 * j + 1], u[4 * j + 2], u[4 * j + 3]);
    }
    __syncthreads();
    // permutation (a gather over the whole row) and the second rotation's scaling
#pragma unroll
    for (int i = 0; i < 16; ++i) u[i] = __fmul_rn(row_buf[static_cast<size_t>(r) * K + src[i]], v2reg[i]);
    wht128(u, lane8);  // second rotation
    const float gmax = group_max(absmax16(u));
    if (MODE == 0 && valid && lane8 == 0) atomicMax(&row_max[buf][r], __float_as_uint(gmax));
    __syncthreads();  // row maxima complete; every gather of this tile is done, the row buffer may be overwritten

    if (!valid) continue;
    const int64_t elem = row * K + col0;
    if (MODE == 0) {
      const float amax = __uint_as_float(row_max[buf][r]);
      const float inv = amax > 0.0f ? __fdiv_rn(127.0f, amax) : 0.0f;
      uint32_t out[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        uint32_t word = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          int q = quantize_one(u[4 * j + e], inv);
          q = max(-127, min(127, q));
          word |= (static_cast<uint32_t>(q) & 0xFFu) << (8 * e);
        }
        out[j] = word;
      }
      *reinterpret_cast<uint4*>(codes + elem) = make_uint4(out[0], out[1], out[2], out[3]);
      if (b == 0 && lane8 == 0) scales[row] = __fdiv_rn(amax, 127.0f);
    } else {
      const float inv = gmax > 0.0f ? __fdiv_rn(7.0f, gmax) : 0.0f;
      uint32_t out[2] = {0u, 0u};
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        int q = quantize_one(u[i], inv);
        q = max(-7, min(7, q));
        out[i / 8] |= (static_cast<uint32_t>(q) & 0xFu) << (4 * (i % 8));
      }
      *reinterpret_cast<uint2*>(packed + elem / 2) = make_uint2(out[0], out[1]);
      if (lane8 == 0) scales[row * nb + b] = __fdiv_rn(gmax, 7.0f);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Fast path for per-row int8 codes (the online activation kernel).
//
// Four lanes own one 128-block of one row, 32 elements each, as four 16-byte chunks interleaved
// across the lanes: lane l holds chunks l, l+4, l+8, l+12 (chunk = 8 consecutive elements), so a
// warp-wide 16-byte load covers whole 32-byte sectors.  With element index bits i0..i6: i0..i2 lie
// inside a chunk, i3 i4 select the lane, i5 i6 the chunk of a lane.  Stages h = 1, 2, 4, 32, 64 pair
// registers of a thread, h = 8, 16 pair lanes by shuffle; the stage order h = 1 .. 64 is kept.
// Values are held as fp32 pairs (i0 = 0, 1) and processed with the packed fp32x2 add / mul / fma
// instructions of sm_100, each lane of which rounds exactly like the scalar instruction.
// Rounding to the integer code uses the exact identity rne(y) = (y + 1.5 * 2^23) - 1.5 * 2^23 for
// |y| < 2^22: after the addition the low byte of the fp32 pattern is the two's-complement code.
// ---------------------------------------------------------------------------------------------
template <int MIN_CTAS>
__global__ void __launch_bounds__(320, MIN_CTAS)
rotate_quantize_rows_kernel(const __nv_bfloat16* __restrict__ x, int64_t ldx, int32_t M, int32_t K, const float* __restrict__ vec,
                            int8_t* __restrict__ codes, float* __restrict__ scales, int32_t rows_per_tile, float zero) {
  extern __shared__ float svec[];  // the group's fused vector, K floats
  __shared__ unsigned int row_max[3][32];
  const int nb = K / TRDQ_BLOCK;
  const int lane4 = threadIdx.x & (kFastLanes - 1);
  const int item = threadIdx.x / kFastLanes;
  const bool active = item < rows_per_tile * nb;
  const int r = active ? item / nb : 0;
  const int b = active ? item % nb : 0;

  for (int i = threadIdx.x; i < K / 4; i += blockDim.x) reinterpret_cast<float4*>(svec)[i] = __ldg(reinterpret_cast<const float4*>(vec) + i);
  if (threadIdx.x < 32) row_max[0][threadIdx.x] = 0u;
  __syncthreads();
  griddep_launch_dependents();
  griddep_wait();  // x may be written, and the code buffer still read, by the kernel before (the group vector is constant)

  const int num_tiles = (M + rows_per_tile - 1) / rows_per_tile;
  const int col0 = b * TRDQ_BLOCK + lane4 * 8;  // first element of chunk 0 of this lane; chunk c is 32 further
  const float2* sv = reinterpret_cast<const float2*>(svec + col0);

  uint4 raw[4];
  auto fetch = [&](int tile) {
    const int64_t row = static_cast<int64_t>(tile) * rows_per_tile + r;
    if (active && tile < num_tiles && row < M) {
      const uint4* src = reinterpret_cast<const uint4*>(x + row * ldx + col0);
#pragma unroll
      for (int c = 0; c < 4; ++c) raw[c] = __ldg(src + 4 * c);  // +32 elements = +4 uint4
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
    const int64_t row = static_cast<int64_t>(tile) * rows_per_tile + r;
    const bool valid = active && row < M;

    // v[4c + j] = elements (2j, 2j+1) of chunk c, scaled by the fused vector
    float2 v[16];
    scale_chunks_lanes4(raw, sv, v);
    fetch(tile + gridDim.x);  // next tile's rows are in flight while this one is transformed

    wht128_lanes4(v, lane4);

    const float m = absmax_lanes4(v);
    if (valid && lane4 == 0) atomicMax(&row_max[buf][r], __float_as_uint(m));
    __syncthreads();

    if (valid) {
      const float amax = __uint_as_float(row_max[buf][r]);
      quantize_store_lanes4(v, amax, zero, codes + row * K + col0);
      if (b == 0 && lane4 == 0) scales[row] = __fdiv_rn(amax, 127.0f);
    }
  }
}

// Full transform (Eq. 9) in the four-lanes-per-block layout, per-row int8 codes: first rotation as above, the
// rotated row parked in shared memory as fp32, gather by the permutation with the second scaling
// (v2[j] = fl32(v1[perm[j]] * vec2[j])), second rotation, quantizer.  The permutation indices of a thread's
// 32 columns do not change from tile to tile and are kept packed two per register (K <= 16384).
template <int MIN_CTAS>
__global__ void __launch_bounds__(320, MIN_CTAS)
rotate2_quantize_rows_kernel(const __nv_bfloat16* __restrict__ x, int64_t ldx, int32_t M, int32_t K, const float* __restrict__ vec1,
                             const int32_t* __restrict__ perm, const float* __restrict__ vec2, int8_t* __restrict__ codes,
                             float* __restrict__ scales, int32_t rows_per_tile, float zero) {
  extern __shared__ float smem_f[];  // svec[K], then row_buf[rows_per_tile][K]
  __shared__ unsigned int row_max[3][32];
  float* svec = smem_f;
  float* row_buf = smem_f + K;
  const int nb = K / TRDQ_BLOCK;
  const int lane4 = threadIdx.x & (kFastLanes - 1);
  const int item = threadIdx.x / kFastLanes;
  const bool active = item < rows_per_tile * nb;
  const int r = active ? item / nb : 0;
  const int b = active ? item % nb : 0;
  const int col0 = b * TRDQ_BLOCK + lane4 * 8;

  for (int i = threadIdx.x; i < K / 4; i += blockDim.x) reinterpret_cast<float4*>(svec)[i] = __ldg(reinterpret_cast<const float4*>(vec1) + i);
  if (threadIdx.x < 32) row_max[0][threadIdx.x] = 0u;
  uint32_t pidx[16];  // perm of columns col0 + 32c + 2j (low half) and + 1 (high half)
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    const int4 p0 = __ldg(reinterpret_cast<const int4*>(perm + col0 + 32 * c));
    const int4 p1 = __ldg(reinterpret_cast<const int4*>(perm + col0 + 32 * c) + 1);
    pidx[4 * c] = static_cast<uint32_t>(p0.x) | (static_cast<uint32_t>(p0.y) << 16);
    pidx[4 * c + 1] = static_cast<uint32_t>(p0.z) | (static_cast<uint32_t>(p0.w) << 16);
    pidx[4 * c + 2] = static_cast<uint32_t>(p1.x) | (static_cast<uint32_t>(p1.y) << 16);
    pidx[4 * c + 3] = static_cast<uint32_t>(p1.z) | (static_cast<uint32_t>(p1.w) << 16);
  }
  __syncthreads();
  griddep_launch_dependents();
  griddep_wait();

  const int num_tiles = (M + rows_per_tile - 1) / rows_per_tile;
  const float2* sv = reinterpret_cast<const float2*>(svec + col0);
  const float2* v2p = reinterpret_cast<const float2*>(vec2 + col0);
  float* my_row = row_buf + static_cast<size_t>(r) * K;

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
    const int64_t row = static_cast<int64_t>(tile) * rows_per_tile + r;
    const bool valid = active && row < M;

    float2 v[16];
    scale_chunks_lanes4(raw, sv, v);
    fetch(tile + gridDim.x);
    wht128_lanes4(v, lane4);  // first rotation
    if (active) {
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        float4* dst = reinterpret_cast<float4*>(my_row + col0 + 32 * c);
        dst[0] = make_float4(v[4 * c].x, v[4 * c].y, v[4 * c + 1].x, v[4 * c + 1].y);
        dst[1] = make_float4(v[4 * c + 2].x, v[4 * c + 2].y, v[4 * c + 3].x, v[4 * c + 3].y);
      }
    }
    __syncthreads();
    // zigzag permutation (a gather over the row) and the scaling of the second rotation
#pragma unroll
    for (int c = 0; c < 4; ++c) {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint32_t pp = pidx[4 * c + j];
        const float2 g2 = make_float2(my_row[pp & 0xFFFFu], my_row[pp >> 16]);
        v[4 * c + j] = __fmul2_rn(g2, __ldg(v2p + 16 * c + j));
      }
    }
    wht128_lanes4(v, lane4);  // second rotation

    const float m = absmax_lanes4(v);
    if (valid && lane4 == 0) atomicMax(&row_max[buf][r], __float_as_uint(m));
    __syncthreads();  // row maxima complete; all gathers done, the row buffer may be overwritten

    if (valid) {
      const float amax = __uint_as_float(row_max[buf][r]);
      quantize_store_lanes4(v, amax, zero, codes + row * K + col0);
      if (b == 0 && lane4 == 0) scales[row] = __fdiv_rn(amax, 127.0f);
    }
  }
}

// Literal asymmetric quantizer of Eq. 1-3 after the block rotation: per row min and max,
//   s = (max - min) / 255,  z = -rne(min * fl(255 / (max - min))),  code = min(rne(v * fl(255 / (max - min))) + z, 255)
// (the lower clamp of Eq. 1 can never bind: rounding is monotone and z cancels the minimum's own code).
// Same four-lanes-per-block layout and butterfly as rotate_quantize_rows_kernel; the row minimum and maximum
// are combined through shared-memory atomics on an order-preserving integer image of the floats.
__device__ __forceinline__ unsigned int float_order_key(float f) {
  const unsigned int b = __float_as_uint(f);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float float_from_order_key(unsigned int k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}

template <int MIN_CTAS>
__global__ void __launch_bounds__(320, MIN_CTAS)
rotate_quantize_rows_asym_kernel(const __nv_bfloat16* __restrict__ x, int64_t ldx, int32_t M, int32_t K, const float* __restrict__ vec,
                                 uint8_t* __restrict__ codes, float* __restrict__ scales, int32_t* __restrict__ zero_points,
                                 int32_t rows_per_tile) {
  extern __shared__ float svec[];
  __shared__ unsigned int row_hi[3][32], row_lo[3][32];
  const int nb = K / TRDQ_BLOCK;
  const int lane4 = threadIdx.x & (kFastLanes - 1);
  const int item = threadIdx.x / kFastLanes;
  const bool active = item < rows_per_tile * nb;
  const int r = active ? item / nb : 0;
  const int b = active ? item % nb : 0;

  for (int i = threadIdx.x; i < K / 4; i += blockDim.x) reinterpret_cast<float4*>(svec)[i] = __ldg(reinterpret_cast<const float4*>(vec) + i);
  if (threadIdx.x < 32) {
    row_hi[0][threadIdx.x] = 0u;
    row_lo[0][threadIdx.x] = 0xFFFFFFFFu;
  }
  __syncthreads();
  griddep_launch_dependents();
  griddep_wait();

  const int num_tiles = (M + rows_per_tile - 1) / rows_per_tile;
  const int col0 = b * TRDQ_BLOCK + lane4 * 8;
  const float2* sv = reinterpret_cast<const float2*>(svec + col0);
  int it = 0;
  for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++it) {
    const int buf = it % 3;
    if (threadIdx.x < 32) {
      row_hi[(it + 1) % 3][threadIdx.x] = 0u;
      row_lo[(it + 1) % 3][threadIdx.x] = 0xFFFFFFFFu;
    }
    const int64_t row = static_cast<int64_t>(tile) * rows_per_tile + r;
    const bool valid = active && row < M;
    float2 v[16];
    if (valid) {
      const uint4* src = reinterpret_cast<const uint4*>(x + row * ldx + col0);
      uint4 raw[4];
#pragma unroll
      for (int c = 0; c < 4; ++c) raw[c] = __ldg(src + 4 * c);
      scale_chunks_lanes4(raw, sv, v);
    } else {
#pragma unroll
      for (int p = 0; p < 16; ++p) v[p] = make_float2(0.0f, 0.0f);
    }
    wht128_lanes4(v, lane4);
    float hi = v[0].x, lo = v[0].x;
#pragma unroll
    for (int p = 0; p < 16; ++p) {
      hi = fmaxf(fmaxf(hi, v[p].x), v[p].y);
      lo = fminf(fminf(lo, v[p].x), v[p].y);
    }
#pragma unroll
    for (int mask = 1; mask <= 2; mask <<= 1) {
      hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, mask));
      lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, mask));
    }
    if (valid && lane4 == 0) {
      atomicMax(&row_hi[buf][r], float_order_key(hi));
      atomicMin(&row_lo[buf][r], float_order_key(lo));
    }
    __syncthreads();
    if (!valid) continue;
    const float vmax = float_from_order_key(row_hi[buf][r]);
    const float vmin = float_from_order_key(row_lo[buf][r]);
    const float range = __fsub_rn(vmax, vmin);
    const float inv = range > 0.0f ? __fdiv_rn(255.0f, range) : 0.0f;
    const int z = -__float2int_rn(__fmul_rn(vmin, inv));
    uint8_t* dst = codes + row * K + col0;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      uint32_t wd[2] = {0u, 0u};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int q0 = min(__float2int_rn(__fmul_rn(v[4 * c + j].x, inv)) + z, 255);
        const int q1 = min(__float2int_rn(__fmul_rn(v[4 * c + j].y, inv)) + z, 255);
        wd[j / 2] |= (static_cast<uint32_t>(q0) | (static_cast<uint32_t>(q1) << 8)) << (16 * (j & 1));
      }
      *reinterpret_cast<uint2*>(dst + 32 * c) = make_uint2(wd[0], wd[1]);
    }
    if (b == 0 && lane4 == 0) {
      scales[row] = __fdiv_rn(range, 255.0f);
      zero_points[row] = z;
    }
  }
}

cudaError_t launch_rows_fast(const void* x, int64_t ldx, int32_t M, int32_t K, const float* vec, void* codes, float* scales,
                             cudaStream_t stream) {
  const int nb = K / TRDQ_BLOCK;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  int rows_max = 72 / nb;  // about 72 lane groups (288 threads) per CTA
  if (rows_max < 1) rows_max = 1;
  if (rows_max > 32) rows_max = 32;
  const int rows = rows_per_tile_by_rounds(M, rows_max, sms);
  int threads = rows * nb * kFastLanes;
  threads = (threads + 31) / 32 * 32;
  const int num_tiles = (M + rows - 1) / rows;
  const int grid = min(num_tiles, sms * 2);
  const size_t smem = static_cast<size_t>(K) * sizeof(float);
  return launch_overlapped(rotate_quantize_rows_kernel<2>, dim3(grid), dim3(threads), smem, stream, static_cast<const __nv_bfloat16*>(x),
                           ldx, M, K, vec, static_cast<int8_t*>(codes), scales, rows, 0.0f);
}

template <int MODE, int P>
cudaError_t launch(const void* x, int64_t ldx, int32_t M, int32_t K, const float* vec, void* codes, float* scales,
                   int rows_per_tile, int groups, cudaStream_t stream) {
  int threads = groups * kLanesPerBlock;
  threads = (threads + 31) / 32 * 32;
  const int num_tiles = (M + rows_per_tile - 1) / rows_per_tile;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int ctas_per_sm = max(1, 2048 / threads);
  const int grid = min(num_tiles, sms * ctas_per_sm);
  rotate_quantize_kernel<MODE, P><<<grid, threads, 0, stream>>>(
      static_cast<const __nv_bfloat16*>(x), ldx, M, K, vec, static_cast<int8_t*>(codes), static_cast<uint8_t*>(codes), scales,
      rows_per_tile, groups);
  return cudaGetLastError();
}

template <int MODE>
cudaError_t dispatch(const void* x, int64_t ldx, int32_t M, int32_t K, const float* vec, void* codes, float* scales,
                     cudaStream_t stream) {
  const int nb = K / TRDQ_BLOCK;
  if (nb <= 128) {
    // about 32 lane groups (256 threads) per CTA, whole rows only, at most 32 rows per tile
    int rows = 32 / nb;
    if (rows < 1) rows = 1;
    if (rows > 32) rows = 32;
    return launch<MODE, 1>(x, ldx, M, K, vec, codes, scales, rows, rows * nb, stream);
  }
  const int p = (nb + 127) / 128;  // nb <= 1024 -> p <= 8
  if (p <= 2) return launch<MODE, 2>(x, ldx, M, K, vec, codes, scales, 1, (nb + 1) / 2, stream);
  if (p <= 4) return launch<MODE, 4>(x, ldx, M, K, vec, codes, scales, 1, (nb + 3) / 4, stream);
  return launch<MODE, 8>(x, ldx, M, K, vec, codes, scales, 1, (nb + 7) / 8, stream);
}

}  // namespace

// Asymmetric per-row quantizer (Eq. 1-3).  Rows of up to 80 blocks (K <= 10240); cudaErrorInvalidValue beyond that.
cudaError_t launch_rotate_quantize_asym(const void* x_bf16, int64_t ldx, int32_t M, int32_t K, const float* vec, uint8_t* codes,
                                        float* scales, int32_t* zero_points, cudaStream_t stream) {
  if (M == 0) return cudaSuccess;
  const int nb = K / TRDQ_BLOCK;
  if (nb > 80) return cudaErrorInvalidValue;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int rows = rows_per_tile_by_rounds(M, std::max(1, std::min(32, 72 / nb)), sms);
  int threads = rows * nb * kFastLanes;
  threads = (threads + 31) / 32 * 32;
  const int num_tiles = (M + rows - 1) / rows;
  return launch_overlapped(rotate_quantize_rows_asym_kernel<2>, dim3(min(num_tiles, sms * 2)), dim3(threads),
                           static_cast<size_t>(K) * sizeof(float), stream, static_cast<const __nv_bfloat16*>(x_bf16), ldx, M, K, vec, codes,
                           scales, zero_points, rows);
}

// Full transform.  Rows of up to 128 blocks (K <= 16384); cudaErrorInvalidValue beyond that.
cudaError_t launch_rotate2_quantize(const void* x_bf16, int64_t ldx, int32_t M, int32_t K, const float* vec1, const int32_t* perm,
                                    const float* vec2, int mode, void* codes, float* scales, cudaStream_t stream) {
  if (M == 0) return cudaSuccess;
  const int nb = K / TRDQ_BLOCK;
  if (nb > 128) return cudaErrorInvalidValue;
  if (mode == 0 && nb <= 72) {
    // four lanes per block, packed arithmetic: about 72 lane groups per CTA, two CTAs per SM
    int rows2 = 72 / nb;
    if (rows2 > 32) rows2 = 32;
    int threads2 = rows2 * nb * kFastLanes;
    threads2 = (threads2 + 31) / 32 * 32;
    const size_t smem2 = (static_cast<size_t>(K) + static_cast<size_t>(rows2) * K) * sizeof(float);
    int dev2 = 0, sms2 = 148;
    cudaGetDevice(&dev2);
    cudaDeviceGetAttribute(&sms2, cudaDevAttrMultiProcessorCount, dev2);
    static PerDeviceFlag configured2;
    if (!configured2.get(dev2)) {
      const cudaError_t e = cudaFuncSetAttribute(rotate2_quantize_rows_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
      if (e != cudaSuccess) return e;
      configured2.set(dev2, true);
    }
    const int tiles2 = (M + rows2 - 1) / rows2;
    return launch_overlapped(rotate2_quantize_rows_kernel<2>, dim3(min(tiles2, sms2 * 2)), dim3(threads2), smem2, stream,
                             static_cast<const __nv_bfloat16*>(x_bf16), ldx, M, K, vec1, perm, vec2, static_cast<int8_t*>(codes), scales,
                             rows2, 0.0f);
  }
  int rows = 32 / nb;
  if (rows < 1) rows = 1;
  int threads = rows * nb * kLanesPerBlock;
  threads = (threads + 31) / 32 * 32;
  const size_t smem = static_cast<size_t>(rows) * K * sizeof(float);
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  static PerDeviceFlag configured;
  if (!configured.get(dev)) {
    cudaError_t e = cudaFuncSetAttribute(rotate2_quantize_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(rotate2_quantize_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
    if (e != cudaSuccess) return e;
    configured.set(dev, true);
  }
  const int num_tiles = (M + rows - 1) / rows;
  const int ctas_per_sm = max(1, min(2048 / threads, static_cast<int>((200 * 1024) / (smem + 1024))));
  const int grid = min(num_tiles, sms * ctas_per_sm);
  if (mode == 0)
    rotate2_quantize_kernel<0><<<grid, threads, smem, stream>>>(static_cast<const __nv_bfloat16*>(x_bf16), ldx, M, K, vec1, perm, vec2,
                                                                static_cast<int8_t*>(codes), static_cast<uint8_t*>(codes), scales, rows);
  else
    rotate2_quantize_kernel<1><<<grid, threads, smem, stream>>>(static_cast<const __nv_bfloat16*>(x_bf16), ldx, M, K, vec1, perm, vec2,
                                                                static_cast<int8_t*>(codes), static_cast<uint8_t*>(codes), scales, rows);
  return cudaGetLastError();
}

// Name of the kernel trdq_rotate_quantize runs for M rows of K channels (single rotation, symmetric codes).
void describe_rotate_quantize_kernel(int32_t M, int32_t K, char* name, size_t cap) {
  if (rotate_quantize_prefers_team(M, K))
    snprintf(name, cap, "rotate_quantize_team_kernel");
  else if (K / TRDQ_BLOCK <= 80 && static_cast<size_t>(K) * sizeof(float) <= 40 * 1024)
    snprintf(name, cap, "rotate_quantize_rows_kernel");
  else
    snprintf(name, cap, "rotate_quantize_kernel");
}

cudaError_t launch_rotate_quantize(const void* x_bf16, int64_t ldx, int32_t M, int32_t K, const float* vec, int mode,
                                   void* codes, float* scales, cudaStream_t stream) {
  if (M == 0) return cudaSuccess;
  if (mode == 0) {
    // fast path: the whole tile of a CTA fits 320 threads and the vector fits the default shared memory
    if (K / TRDQ_BLOCK <= 80 && static_cast<size_t>(K) * sizeof(float) <= 40 * 1024)
      return launch_rows_fast(x_bf16, ldx, M, K, vec, codes, scales, stream);
    return dispatch<0>(x_bf16, ldx, M, K, vec, codes, scales, stream);
  }
  return dispatch<1>(x_bf16, ldx, M, K, vec, codes, scales, stream);
}

}  // namespace trdq
