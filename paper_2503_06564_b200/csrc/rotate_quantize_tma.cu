// Fused online transform + per-token quantizer (Sec. 3.2 Eq. 10 G_t; Sec. 3.1 Eq. 1-2), the
// variant for rows of at most 36 blocks: TMA-staged input, ONE THREAD PER 128-BLOCK.
//
// Why this shape.  The butterfly kernel that spreads a block over several lanes spends most of the
// load/store data path on warp shuffles (two per element) and on re-reading the group vector.
// Here a thread holds a whole block (128 fp32 values in registers), so all seven butterfly stages
// are register-to-register, and the memory system is decoupled from the arithmetic:
//   * a producer warp streams tiles of R rows x K columns into a two-stage shared-memory ring with
//     TMA (boxes of 64 columns x R rows, 128-byte swizzle), so loads never wait on registers;
//   * compute threads read their 256 bytes with conflict-free 16-byte shared loads (eight consecutive
//     threads = eight consecutive rows of one block column, which the swizzle spreads over all
//     banks), release the stage at once, transform, exchange the row absmax through shared memory,
//     quantize, and write the codes into a swizzled staging tile that TMA stores to global memory.
// The arithmetic (one fp32 multiply by the fused vector, stages h = 1 .. 64 in this order with
// separately rounded additions, rne via the 1.5 * 2^23 addition) is the same as in the other kernels
// of rotate_quantize.cu and bit-identical to a scalar evaluation.  Every wait is bounded.
#include <cuda_bf16.h>

#include "internal.h"
#include "ptx.cuh"

namespace trdq {
namespace {

constexpr int kMaxComputeThreads = 288;
constexpr float kRoundMagic = 12582912.0f;  // 1.5 * 2^23

struct alignas(64) RqParams {
  // Both maps view a row as K/64 (K/128) column boxes: dims (column in box, row, box), so that ONE copy
  // moves a whole R-row tile and lays it out box after box, each box R rows of 128 bytes, 128-byte swizzle.
  CUtensorMap tmap_x;      // bf16: (64, M, K/64), box 64 x R x K/64
  CUtensorMap tmap_codes;  // int8: (128, M, K/128), box 128 x R x K/128
  const float* vec;        // fused vector of the group, K floats
  float* scales;           // [M]
  int32_t M, K, R;         // R rows per tile, a multiple of 8
  int32_t compute_threads; // R * K/128 rounded up to a warp multiple
  float zero;              // 0.0f, see the quantizer below
  uint32_t* status;
};

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}

__device__ __forceinline__ uint32_t pack4(float2 a, float2 b) {
  const uint32_t lo = __byte_perm(__float_as_uint(a.x), __float_as_uint(a.y), 0x0040);
  const uint32_t hi = __byte_perm(__float_as_uint(b.x), __float_as_uint(b.y), 0x0040);
  return __byte_perm(lo, hi, 0x5410);
}

// MAXT compute threads per CTA, MINB CTAs per SM: narrow rows run two smaller CTAs per SM so that one
// transforms while the other waits at its row-max barrier or moves data.
template <int MAXT, int MINB>
__global__ void __launch_bounds__(MAXT + 32, MINB) rotate_quantize_tma_kernel(const __grid_constant__ RqParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
  const int nb = p.K / TRDQ_BLOCK;
  const int R = p.R;
  const uint32_t box_in_bytes = R * 128;              // 64 bf16 columns x R rows
  const uint32_t stage_bytes = 2 * nb * box_in_bytes; // R x K bf16
  const uint32_t out_bytes = nb * box_in_bytes;       // R x K int8
  const uint32_t out_base = smem_base + 2 * stage_bytes;
  float* svec = reinterpret_cast<float*>(smem + 2 * stage_bytes + out_bytes);
  unsigned int* row_max = reinterpret_cast<unsigned int*>(svec + p.K);  // [3][R]
  uint64_t* bars = reinterpret_cast<uint64_t*>(row_max + 3 * R);        // 8-byte aligned: K and R are multiples of 8
  const uint32_t bar_full = smem_u32(bars);        // [2]
  const uint32_t bar_empty = bar_full + 16;        // [2]

  const int tid = threadIdx.x;
  const int warp = tid >> 5, lane = tid & 31;
  const int compute_warps = p.compute_threads / 32;
  const int num_tiles = (p.M + R - 1) / R;

  if (tid == 0) {
    for (int s = 0; s < 2; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, compute_warps);
    }
    fence_mbar_init();
  }
  for (int i = tid; i < p.K / 4; i += blockDim.x) reinterpret_cast<float4*>(svec)[i] = __ldg(reinterpret_cast<const float4*>(p.vec) + i);
  for (int i = tid; i < 3 * R; i += blockDim.x) row_max[i] = 0u;
  __syncthreads();
  griddep_launch_dependents();
  griddep_wait();  // X may be written, and the code buffer still read, by the kernel before (the group vector is constant)

  if (warp == compute_warps) {
    // ------------------------------------------------------------ TMA producer
    if (elect_one()) {
      prefetch_tensormap(&p.tmap_x);
      prefetch_tensormap(&p.tmap_codes);
      BoundedWaiter w(p.status, kStatusTimeoutProducer);
      int stage = 0;
      uint32_t phase = 0;
      for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
        w.wait(bar_empty + 8 * stage, phase ^ 1);
        mbar_arrive_expect_tx(bar_full + 8 * stage, stage_bytes);
        const uint32_t dst = smem_base + stage * stage_bytes;
        tma_load_3d(dst, &p.tmap_x, 0, tile * R, 0, bar_full + 8 * stage);  // all 2 * nb column boxes in one copy
        if (++stage == 2) {
          stage = 0;
          phase ^= 1;
        }
      }
      w.settle();
    }
    return;
  }

  // ------------------------------------------------------------------ compute
  // eight consecutive threads = eight consecutive rows of one block column
  const bool active = tid < R * nb;
  const int quarter = active ? tid >> 3 : 0;
  const int r8 = tid & 7;
  const int groups_of_8 = R >> 3;
  const int b = quarter / groups_of_8;
  const int r = (quarter - b * groups_of_8) * 8 + r8;
  const float4* sv4 = reinterpret_cast<const float4*>(svec + b * TRDQ_BLOCK);
  const float2 neg1 = make_float2(-1.0f, -1.0f);

  BoundedWaiter w(p.status, kStatusTimeoutEpilogue);
  int stage = 0;
  uint32_t phase = 0;
  int it = 0;
  for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++it) {
    const int buf = it % 3;
    if (tid < R) row_max[((it + 1) % 3) * R + tid] = 0u;

    w.wait(bar_full + 8 * stage, phase);
    __syncwarp();
    // v[32h + 4j + i] = elements (2i, 2i+1) of 16-byte chunk j of half h, times the fused vector
    float2 v[64];
    const uint32_t in_row = smem_base + stage * stage_bytes + (2 * b) * box_in_bytes + r * 128;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const uint4 raw = lds128(in_row + h * box_in_bytes + ((j ^ r8) << 4));
        const float4 s0 = sv4[h * 16 + j * 2], s1 = sv4[h * 16 + j * 2 + 1];
        const uint32_t wd[4] = {raw.x, raw.y, raw.z, raw.w};
        const float2 sc[4] = {make_float2(s0.x, s0.y), make_float2(s0.z, s0.w), make_float2(s1.x, s1.y), make_float2(s1.z, s1.w)};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          // bf16 -> fp32 is exact: the 16 bits become the high half of the fp32 pattern
          const float2 xv = make_float2(__uint_as_float(wd[i] << 16), __uint_as_float(wd[i] & 0xFFFF0000u));
          v[h * 32 + j * 4 + i] = __fmul2_rn(xv, sc[i]);
        }
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(bar_empty + 8 * stage);  // the stage can be refilled while this tile is transformed
    if (++stage == 2) {
      stage = 0;
      phase ^= 1;
    }

    // h = 1: inside a pair; h = 2 .. 64: pair index bits 0 .. 5
#pragma unroll
    for (int q = 0; q < 64; ++q) v[q] = make_float2(__fadd_rn(v[q].x, v[q].y), __fsub_rn(v[q].x, v[q].y));
#pragma unroll
    for (int hb = 1; hb < 64; hb <<= 1) {
#pragma unroll
      for (int q = 0; q < 64; ++q) {
        if ((q & hb) == 0) {
          const float2 a = v[q], c = v[q + hb];
          v[q] = __fadd2_rn(a, c);
          v[q + hb] = __ffma2_rn(c, neg1, a);  // a - c, one rounding
        }
      }
    }
    float m = 0.0f;
#pragma unroll
    for (int q = 0; q < 64; ++q) m = fmaxf(fmaxf(m, fabsf(v[q].x)), fabsf(v[q].y));
    if (active) atomicMax(&row_max[buf * R + r], __float_as_uint(m));
    if (tid == 0) bulk_wait_group_read<0>();  // the previous tile's stores have finished reading the staging tile
    asm volatile("bar.sync 1, %0;" ::"r"(p.compute_threads) : "memory");

    const float amax = __uint_as_float(row_max[buf * R + r]);
    const float inv = amax > 0.0f ? __fdiv_rn(127.0f, amax) : 0.0f;
    const float2 inv2 = make_float2(inv, inv);
    const float2 magic2 = make_float2(kRoundMagic, kRoundMagic);
    // The product must be rounded to fp32 before the magic addition rounds it to an integer.  A packed
    // multiply feeding a packed add is contracted into one fused operation by the assembler, so the
    // product is written as fma(v, inv, zero) with `zero` a kernel argument equal to 0.0f.
    const float2 zero2 = make_float2(p.zero, p.zero);
    if (active) {
      const uint32_t out_row = out_base + b * box_in_bytes + r * 128;
#pragma unroll
      for (int c = 0; c < 8; ++c) {  // 16 codes = 8 pairs per 16-byte chunk
        float2 q[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) q[i] = __fadd2_rn(__ffma2_rn(v[c * 8 + i], inv2, zero2), magic2);
        st_shared_v4(out_row + ((c ^ r8) << 4), pack4(q[0], q[1]), pack4(q[2], q[3]), pack4(q[4], q[5]), pack4(q[6], q[7]));
      }
      const int64_t row = static_cast<int64_t>(tile) * R + r;
      if (b == 0 && row < p.M) p.scales[row] = __fdiv_rn(amax, 127.0f);
    }
    fence_proxy_async_smem();
    asm volatile("bar.sync 2, %0;" ::"r"(p.compute_threads) : "memory");
    if (tid == 0) {
      tma_store_3d(&p.tmap_codes, 0, tile * R, 0, out_base);  // all nb column boxes; rows >= M are clipped
      bulk_commit_group();
    }
  }
  if (tid == 0) bulk_wait_group_read<0>();  // the staging tile has been read; the stores complete before the grid does
  w.settle();
}

}  // namespace

constexpr int kSmallComputeThreads = 144;

// Rows per tile for this kernel, or 0 if the row is too wide for it.
int rotate_quantize_tma_rows(int32_t K) {
  const int nb = K / TRDQ_BLOCK;
  const int budget = kMaxComputeThreads;
  int rows = (budget / nb) / 8 * 8;
  if (rows > 256) rows = 256;  // TMA box limit
  return rows >= 8 ? rows : 0;
}

// The one-thread-per-block kernel keeps a whole tile of R rows in the registers of one CTA (one CTA per SM), so its
// time comes in rounds of one tile per SM, plus the fill of its ring; the lane-group kernel spreads the same rows over
// twice as many smaller CTAs with finer tiles.  Measured crossover (K = 1024 .. 4608): with fewer than about six
// rounds the lane-group kernel finishes sooner (by 6 - 14 % at 2.6 - 5.2 rounds), from 6.9 rounds on this one wins
// (by 5 - 23 %).
bool rotate_quantize_prefers_tma(int32_t M, int32_t K) {
  const int R = rotate_quantize_tma_rows(K);
  if (R == 0) return false;
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  return (static_cast<int64_t>(M) + R - 1) / R >= 6ll * sms;
}

trdq_status launch_rotate_quantize_tma(const void* x_bf16, int64_t ldx, int32_t M, int32_t K, const float* vec, int8_t* codes,
                                       float* scales, cudaStream_t stream) {
  const int R = rotate_quantize_tma_rows(K);
  if (R == 0) return TRDQ_ERR_SHAPE;
  const int nb = K / TRDQ_BLOCK;
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) != cudaSuccess) return TRDQ_ERR_CUDA;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  RqParams p;
  trdq_status st = encode_tmap_boxes(&p.tmap_x, x_bf16, 2, 64, static_cast<uint64_t>(M), static_cast<uint64_t>(ldx) * 2,
                                     static_cast<uint32_t>(2 * nb), static_cast<uint32_t>(R));
  if (st != TRDQ_OK) return st;
  st = encode_tmap_boxes(&p.tmap_codes, codes, 1, 128, static_cast<uint64_t>(M), static_cast<uint64_t>(K), static_cast<uint32_t>(nb),
                         static_cast<uint32_t>(R));
  if (st != TRDQ_OK) return st;
  p.vec = vec;
  p.scales = scales;
  p.M = M;
  p.K = K;
  p.R = R;
  p.compute_threads = (R * nb + 31) / 32 * 32;
  p.zero = 0.0f;
  p.status = device_status_word();
  if (!p.status) return TRDQ_ERR_CUDA;
  const size_t smem = 1024 + 2 * static_cast<size_t>(R) * K * 2 + static_cast<size_t>(R) * K + static_cast<size_t>(K) * 4 +
                      3 * static_cast<size_t>(R) * 4 + 64;
  static PerDeviceFlag configured;
  if (!configured.get(dev)) {
    if (cudaFuncSetAttribute(rotate_quantize_tma_kernel<kMaxComputeThreads, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             227 * 1024) != cudaSuccess ||
        cudaFuncSetAttribute(rotate_quantize_tma_kernel<kSmallComputeThreads, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             113 * 1024) != cudaSuccess)
      return TRDQ_ERR_CUDA;
    configured.set(dev, true);
  }
  const bool small = false;  // two smaller CTAs per SM measured slower on 9- and 18-block rows, as did twelve compute warps with a one-stage ring
  if (smem > (small ? 113u : 227u) * 1024) return TRDQ_ERR_SHAPE;
  const int num_tiles = (M + R - 1) / R;
  const int slots = small ? 2 * sms : sms;
  const int grid = num_tiles < slots ? num_tiles : slots;
  const cudaError_t e =
      small ? launch_overlapped(rotate_quantize_tma_kernel<kSmallComputeThreads, 2>, dim3(grid), dim3(p.compute_threads + 32), smem, stream, p)
            : launch_overlapped(rotate_quantize_tma_kernel<kMaxComputeThreads, 1>, dim3(grid), dim3(p.compute_threads + 32), smem, stream, p);
  return e == cudaSuccess ? TRDQ_OK : TRDQ_ERR_CUDA;
}

}  // namespace trdq
