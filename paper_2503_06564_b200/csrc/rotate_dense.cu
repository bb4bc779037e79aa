// Dense block rotations (Sec. 3.2, Eq. 6-8) applied online on the tensor cores, then the per-token
// quantizer (Sec. 3.1, Eq. 1-2 in its symmetric 8-bit form).
//
// Eq. 8 makes the rotation block diagonal with dense 2^n x 2^n blocks (here 128 x 128), each the greedy
// product of Eq. 6-7.  With a dense block the online transform v = (x o Delta) R is a real contraction:
// per token row and block, a 1 x 128 by 128 x 128 product.  The smoothing vector is folded into the rows
// of the block and the result is held in bf16, S_b[i][j] = bf16(Delta[128 b + i] R_b[i][j]); the
// activations are bf16 already, so one tcgen05.mma (kind::f16, fp32 accumulation in tensor memory)
// per 16 input channels computes v exactly up to the accumulation order.
//
// The per-token scale needs the maximum of |v| over the WHOLE row before any code can be formed, and a
// tile of 128 tokens x K channels of fp32 does not fit in tensor memory (512 columns).  So X is read twice:
//   pass 0 (amax)      a CTA owns token tiles and walks across the K/128 blocks; X tile and S_b arrive together
//                      through a three-stage ring (S comes from L2, X from HBM); the drain warps keep a running
//                      per-row maximum of |v| in registers and write amax[m] once per row.
//   pass 1 (quantize)  a CTA owns ONE block column b (S_b stays in shared memory, so matrix traffic is paid once)
//                      and walks down the token tiles in the opposite order of pass 0, so that what was read
//                      last is still in L2; the product is formed again (bit-identical: same instructions on
//                      the same operands), codes = rne(v * fl(127 / amax)), written through TMA stores.
// Both passes are warp specialised: warp 0 issues TMA loads, warp 1 the MMAs into one of four 128-column
// accumulators, warp 2 owns tensor memory, warps 4.. drain.  Every wait is bounded.
#include <cuda_bf16.h>

#include <algorithm>

#include "internal.h"
#include "ptx.cuh"

namespace trdq {
namespace {

constexpr int kRows = 128;                          // token rows per tile = M of the MMA
constexpr int kTileBytes = kRows * TRDQ_BLOCK * 2;  // 128 x 128 bf16: two swizzle atoms of 128 rows x 64 columns
constexpr int kAtomBytes = kTileBytes / 2;
constexpr int kAccSlots = 4;
constexpr int kAccCols = TRDQ_BLOCK;
constexpr int kTmemCols = 512;
constexpr int kThreads = 384;                       // warp 0 TMA, warp 1 MMA, warp 2 tensor-memory owner, warps 4-11 drain
constexpr int kBarrierBytes = 256;
// pass 0: ring of (X tile, S_b) pairs
constexpr int kStages0 = 3;
constexpr int kSmemBytes0 = 1024 + kStages0 * 2 * kTileBytes + kBarrierBytes;
// pass 1: resident S_b, ring of X tiles, one staging tile per drain warp
constexpr int kStages1 = 4;
constexpr int kDrainWarps1 = 8;
constexpr int kOutStageBytes = kDrainWarps1 * 4096;  // per drain warp one staging tile of 32 rows x 128 codes
constexpr int kSmemBytes1 = 1024 + kTileBytes + kStages1 * kTileBytes + kOutStageBytes + kBarrierBytes;
constexpr float kRoundMagic = 12582912.0f;          // 1.5 * 2^23: adding it leaves rne(u) in the low mantissa bits

struct alignas(64) DenseParams {
  CUtensorMap tmap_x;      // bf16 [M, K] (row stride ldx), box 64 columns x 128 rows, 128-byte swizzle
  CUtensorMap tmap_s;      // bf16 [G * K/128 * 128, 128]: S_b transposed (row j = output channel), same box
  CUtensorMap tmap_codes;  // int8 [M, K], box 128 x 32, 128-byte swizzle
  float* amax;             // [splits][M]: max of |v| over the row's blocks of each split
  float* scales;           // [M]
  int32_t M, K;
  int32_t tile_begin, tile_end;      // token tiles of this launch
  int32_t splits, blocks_per_split;  // pass 0 cuts the K/128 blocks into `splits` ranges when there are few token tiles
  int32_t s_row0;          // first row of this group's matrices in tmap_s
  uint32_t* status;
};
constexpr int kMaxSplits = 8;

// kind::f16 instruction descriptor: bf16 A and B, both K-major, fp32 D, M = 128, N = 128.
constexpr uint32_t kIdescBf16 = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(TRDQ_BLOCK >> 3) << 17) |
                                (static_cast<uint32_t>(kRows >> 4) << 24);

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t accumulate) {
  asm volatile(
      "{\n\t"
      ".reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t"
      "}\n" ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(kIdescBf16), "r"(accumulate)
      : "memory");
}

// One 128 x 128 x 128 product: X tile (two atoms) times S_b (two atoms) into the accumulator at d_tmem.
__device__ __forceinline__ void mma_tile(uint32_t d_tmem, uint32_t x_addr, uint32_t s_addr) {
#pragma unroll
  for (int a = 0; a < 2; ++a) {
    const uint64_t a_desc = umma_desc_k_sw128(x_addr + a * kAtomBytes);
    const uint64_t b_desc = umma_desc_k_sw128(s_addr + a * kAtomBytes);
#pragma unroll
    for (int k = 0; k < 4; ++k)  // 16 input channels = 32 bytes along K = +2 in the 16-byte address field
      umma_bf16(d_tmem, a_desc + 2 * k, b_desc + 2 * k, (a | k) != 0 ? 1u : 0u);
  }
}

struct Pipe {
  int idx = 0;
  uint32_t phase = 0;
  __device__ __forceinline__ void advance(int n) {
    if (++idx == n) {
      idx = 0;
      phase ^= 1;
    }
  }
};

// ------------------------------------------------------------------------------ pass 0 ----
__global__ void __launch_bounds__(kThreads, 1) rotate_dense_amax_kernel(const __grid_constant__ DenseParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages0 * 2 * kTileBytes);
  const uint32_t bar_full = smem_u32(bars);             // [kStages0]
  const uint32_t bar_empty = bar_full + 8 * kStages0;   // [kStages0]
  const uint32_t bar_tfull = bar_empty + 8 * kStages0;  // [kAccSlots]
  const uint32_t bar_tempty = bar_tfull + 8 * kAccSlots;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStages0 + 2 * kAccSlots);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int b_begin = blockIdx.y * p.blocks_per_split;
  const int b_end = min(p.K / TRDQ_BLOCK, b_begin + p.blocks_per_split);
  const int tile_first = p.tile_begin + blockIdx.x;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages0; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int a = 0; a < kAccSlots; ++a) {
      mbar_init(bar_tfull + 8 * a, 1);
      mbar_init(bar_tempty + 8 * a, 4);  // one drain warp per lane quarter
    }
    fence_mbar_init();
  }
  if (warp == 2) {
    tmem_alloc(smem_u32(tmem_slot), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  if (threadIdx.x == 0) {
    prefetch_tensormap(&p.tmap_x);
    prefetch_tensormap(&p.tmap_s);
  }
  griddep_launch_dependents();
  griddep_wait();  // X comes from the kernel before; amax may still be read by it

  if (warp == 0) {
    if (elect_one()) {
      BoundedWaiter w(p.status, kStatusTimeoutProducer);
      Pipe st;
      for (int tile = tile_first; tile < p.tile_end; tile += gridDim.x)
        for (int b = b_begin; b < b_end; ++b) {
          w.wait(bar_empty + 8 * st.idx, st.phase ^ 1);
          const uint32_t dst = smem_base + st.idx * 2 * kTileBytes;
          const uint32_t bar = bar_full + 8 * st.idx;
          mbar_arrive_expect_tx(bar, 2 * kTileBytes);
          tma_load_2d(dst, &p.tmap_x, b * TRDQ_BLOCK, tile * kRows, bar);  // rows >= M read as zero
          tma_load_2d(dst + kAtomBytes, &p.tmap_x, b * TRDQ_BLOCK + 64, tile * kRows, bar);
          tma_load_2d(dst + kTileBytes, &p.tmap_s, 0, p.s_row0 + b * TRDQ_BLOCK, bar);
          tma_load_2d(dst + kTileBytes + kAtomBytes, &p.tmap_s, 64, p.s_row0 + b * TRDQ_BLOCK, bar);
          st.advance(kStages0);
        }
      w.settle();
    }
  } else if (warp == 1) {
    if (elect_one()) {
      BoundedWaiter w(p.status, kStatusTimeoutMma);
      Pipe st, acc;
      for (int tile = tile_first; tile < p.tile_end; tile += gridDim.x)
        for (int b = b_begin; b < b_end; ++b) {
          w.wait(bar_tempty + 8 * acc.idx, acc.phase ^ 1);
          w.wait(bar_full + 8 * st.idx, st.phase);
          tc_fence_after();
          const uint32_t x_addr = smem_base + st.idx * 2 * kTileBytes;
          mma_tile(tmem_base + acc.idx * kAccCols, x_addr, x_addr + kTileBytes);
          umma_commit(bar_empty + 8 * st.idx);
          umma_commit(bar_tfull + 8 * acc.idx);
          st.advance(kStages0);
          acc.advance(kAccSlots);
        }
      w.settle();
    }
  } else if (warp >= 4 && warp < 8) {
    const int q = warp & 3;  // the lane quarter of tensor memory this warp may read
    BoundedWaiter w(p.status, kStatusTimeoutEpilogue);
    Pipe acc;
    for (int tile = tile_first; tile < p.tile_end; tile += gridDim.x) {
      const int row = tile * kRows + q * 32 + lane;
      float mx = 0.0f;
      for (int b = b_begin; b < b_end; ++b) {
        w.wait(bar_tfull + 8 * acc.idx, acc.phase);
        __syncwarp();
        tc_fence_after();
        const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc.idx * kAccCols;
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          uint32_t r[32];
          tmem_ld_32x32(t_row + c * 32, r);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; ++j) mx = fmaxf(mx, fabsf(__uint_as_float(r[j])));
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_tempty + 8 * acc.idx);
        acc.advance(kAccSlots);
      }
      if (row < p.M) p.amax[static_cast<size_t>(blockIdx.y) * p.M + row] = mx;
    }
    w.settle();
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 2) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ------------------------------------------------------------------------------ pass 1 ----
__global__ void __launch_bounds__(kThreads, 1) rotate_dense_quantize_kernel(const __grid_constant__ DenseParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t s_tile = smem_base;                            // S_b, resident
  const uint32_t x_ring = smem_base + kTileBytes;
  const uint32_t out_stage_base = x_ring + kStages1 * kTileBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kTileBytes + kStages1 * kTileBytes + kOutStageBytes);
  const uint32_t bar_full = smem_u32(bars);             // [kStages1]
  const uint32_t bar_empty = bar_full + 8 * kStages1;   // [kStages1]
  const uint32_t bar_tfull = bar_empty + 8 * kStages1;  // [kAccSlots]
  const uint32_t bar_tempty = bar_tfull + 8 * kAccSlots;
  const uint32_t bar_s = bar_tempty + 8 * kAccSlots;    // S_b has landed
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStages1 + 2 * kAccSlots + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int b = blockIdx.y;  // block column of this CTA

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages1; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int a = 0; a < kAccSlots; ++a) {
      mbar_init(bar_tfull + 8 * a, 1);
      mbar_init(bar_tempty + 8 * a, kDrainWarps1 / 2);  // the four warps that drain this tile
    }
    mbar_init(bar_s, 1);
    fence_mbar_init();
  }
  if (warp == 2) {
    tmem_alloc(smem_u32(tmem_slot), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  if (threadIdx.x == 0) {
    prefetch_tensormap(&p.tmap_x);
    prefetch_tensormap(&p.tmap_s);
    prefetch_tensormap(&p.tmap_codes);
    // the matrices are constants of the rotation object: they may be fetched while the kernel before still runs
    mbar_arrive_expect_tx(bar_s, kTileBytes);
    tma_load_2d(s_tile, &p.tmap_s, 0, p.s_row0 + b * TRDQ_BLOCK, bar_s);
    tma_load_2d(s_tile + kAtomBytes, &p.tmap_s, 64, p.s_row0 + b * TRDQ_BLOCK, bar_s);
  }
  griddep_launch_dependents();
  griddep_wait();  // X and the row maxima come from the kernels before; the code buffer may still be read by them

  // This CTA's tiles, from the last token tile of the launch backwards.
  const int tiles = p.tile_end - p.tile_begin;
  const int my_tiles = static_cast<int>(blockIdx.x) < tiles ? (tiles - 1 - static_cast<int>(blockIdx.x)) / static_cast<int>(gridDim.x) + 1 : 0;
  auto tile_row0 = [&](int it) { return (p.tile_end - 1 - (static_cast<int>(blockIdx.x) + it * static_cast<int>(gridDim.x))) * kRows; };

  if (warp == 0) {
    if (elect_one()) {
      BoundedWaiter w(p.status, kStatusTimeoutProducer);
      Pipe st;
      for (int it = 0; it < my_tiles; ++it) {
        const int row0 = tile_row0(it);
        w.wait(bar_empty + 8 * st.idx, st.phase ^ 1);
        const uint32_t dst = x_ring + st.idx * kTileBytes;
        mbar_arrive_expect_tx(bar_full + 8 * st.idx, kTileBytes);
        tma_load_2d(dst, &p.tmap_x, b * TRDQ_BLOCK, row0, bar_full + 8 * st.idx);
        tma_load_2d(dst + kAtomBytes, &p.tmap_x, b * TRDQ_BLOCK + 64, row0, bar_full + 8 * st.idx);
        st.advance(kStages1);
      }
      w.settle();
    }
  } else if (warp == 1) {
    if (elect_one()) {
      BoundedWaiter w(p.status, kStatusTimeoutMma);
      w.wait(bar_s, 0);
      Pipe st, acc;
      for (int it = 0; it < my_tiles; ++it) {
        w.wait(bar_tempty + 8 * acc.idx, acc.phase ^ 1);
        w.wait(bar_full + 8 * st.idx, st.phase);
        tc_fence_after();
        mma_tile(tmem_base + acc.idx * kAccCols, x_ring + st.idx * kTileBytes, s_tile);
        umma_commit(bar_empty + 8 * st.idx);
        umma_commit(bar_tfull + 8 * acc.idx);
        st.advance(kStages1);
        acc.advance(kAccSlots);
      }
      w.settle();
    }
  } else if (warp >= 4) {
    const int ew = warp - 4;
    const int q = ew & 3;        // = warp % 4: the lane quarter of tensor memory this warp may read
    const int parity = ew >> 2;  // warps 4-7 drain this CTA's even tiles, warps 8-11 the odd ones: 32 rows x all 128 columns each,
                                 // so that a store writes whole 128-byte lines of the code matrix
    const uint32_t tile_smem = out_stage_base + ew * 4096;
    BoundedWaiter w(p.status, kStatusTimeoutEpilogue);
    // the row maxima of this warp's next tile are fetched while the current one is drained (raw values are kept in
    // registers and only combined one iteration later, so that the loads never stall this warp)
    float part[kMaxSplits];
    auto fetch = [&](int it) {
      const int row = tile_row0(it) + q * 32 + lane;
#pragma unroll
      for (int s = 0; s < kMaxSplits; ++s) part[s] = (s < p.splits && row < p.M) ? __ldg(p.amax + static_cast<size_t>(s) * p.M + row) : 0.0f;
    };
    if (parity < my_tiles) fetch(parity);
    for (int it = parity; it < my_tiles; it += 2) {
      const int acc_idx = it & (kAccSlots - 1);
      const uint32_t acc_phase = (it / kAccSlots) & 1;
      const int row0 = tile_row0(it);
      const int row = row0 + q * 32 + lane;
      float amax = part[0];
#pragma unroll
      for (int s = 1; s < kMaxSplits; ++s) amax = fmaxf(amax, part[s]);
      if (it + 2 < my_tiles) fetch(it + 2);
      if (row < p.M && b == 0) p.scales[row] = __fdiv_rn(amax, 127.0f);
      const float inv = amax > 0.0f ? __fdiv_rn(127.0f, amax) : 0.0f;
      w.wait(bar_tfull + 8 * acc_idx, acc_phase);
      __syncwarp();
      tc_fence_after();
      const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc_idx * kAccCols;
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        uint32_t r[32];
        tmem_ld_32x32(t_row + c * 32, r);
        tmem_wait_ld();
        uint32_t wds[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          uint32_t by[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) by[e] = __float_as_uint(__fadd_rn(__fmul_rn(__uint_as_float(r[4 * j + e]), inv), kRoundMagic));
          wds[j] = __byte_perm(__byte_perm(by[0], by[1], 0x0040), __byte_perm(by[2], by[3], 0x0040), 0x5410);
        }
        if (c == 0) {
          if (lane == 0) bulk_wait_group_read<0>();  // this warp's previous store has finished reading the buffer
          __syncwarp();
        }
        // staging tile: row = lane, 128 bytes per row, 16-byte chunk v stored at v ^ (lane & 7)
        st_shared_v4(tile_smem + lane * 128 + (((2 * c) ^ (lane & 7)) << 4), wds[0], wds[1], wds[2], wds[3]);
        st_shared_v4(tile_smem + lane * 128 + (((2 * c + 1) ^ (lane & 7)) << 4), wds[4], wds[5], wds[6], wds[7]);
      }
      tc_fence_before();
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(bar_tempty + 8 * acc_idx);
        tma_store_2d(&p.tmap_codes, b * TRDQ_BLOCK, row0 + q * 32, tile_smem);  // rows >= M are clipped
        bulk_commit_group();
      }
    }
    if (lane == 0) bulk_wait_group_read<0>();
    w.settle();
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 2) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ------------------------------------------------------------------ weight side (offline) ----
// H_t(W) with dense blocks: the activations were multiplied by S_b, so the weights take its inverse,
//   wr[n, 128 b + j] = fl32( sum_i inv_b[j][i] * W[n, 128 b + i] )          ((X S)(S^-1 W^T) = X W^T, Eq. 9 / Eq. 10)
// with products and sums in fp64, each rounded separately, i ascending.  inv_t[b][i][j] = inv_b[j][i], so that
// consecutive threads (j) read consecutive addresses.  One CTA: one block, kWRows weight rows; thread j keeps
// kWRows running sums so that every matrix element is read once per kWRows rows.
constexpr int kWRows = 16;

__global__ void __launch_bounds__(TRDQ_BLOCK) dense_weight_rotate_kernel(const __nv_bfloat16* __restrict__ W, int N, int K,
                                                                         const double* __restrict__ inv_t, float* __restrict__ wr) {
  __shared__ double wrow[kWRows][TRDQ_BLOCK];
  const int b = blockIdx.x;
  const int n0 = blockIdx.y * kWRows;
  const int j = threadIdx.x;
  for (int r = 0; r < kWRows; ++r) {
    const int n = n0 + r;
    wrow[r][j] = n < N ? static_cast<double>(__bfloat162float(W[static_cast<size_t>(n) * K + b * TRDQ_BLOCK + j])) : 0.0;
  }
  __syncthreads();
  double s[kWRows];
#pragma unroll
  for (int r = 0; r < kWRows; ++r) s[r] = 0.0;
  const double* m = inv_t + static_cast<size_t>(b) * TRDQ_BLOCK * TRDQ_BLOCK + j;
  for (int i = 0; i < TRDQ_BLOCK; ++i) {
    const double mij = m[static_cast<size_t>(i) * TRDQ_BLOCK];
#pragma unroll
    for (int r = 0; r < kWRows; ++r) s[r] = __dadd_rn(s[r], __dmul_rn(mij, wrow[r][i]));
  }
  for (int r = 0; r < kWRows; ++r) {
    const int n = n0 + r;
    if (n < N) wr[static_cast<size_t>(n) * K + b * TRDQ_BLOCK + j] = static_cast<float>(s[r]);
  }
}

__device__ __forceinline__ float block_max_256(float v, float* scratch) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
  __syncthreads();
  float r = scratch[0];
#pragma unroll
  for (int w = 1; w < 8; ++w) r = fmaxf(r, scratch[w]);
  __syncthreads();
  return r;
}

// Per-output-channel symmetric 8-bit quantizer on fp32 rows (Sec. 3.1: per-channel for weights): one CTA per row.
__global__ void __launch_bounds__(256) quantize_rows_w8_kernel(const float* __restrict__ wr, int K, int8_t* __restrict__ codes,
                                                               float* __restrict__ scales) {
  __shared__ float scratch[8];
  const float* row = wr + static_cast<size_t>(blockIdx.x) * K;
  float mx = 0.0f;
  for (int k = threadIdx.x; k < K; k += 256) mx = fmaxf(mx, fabsf(row[k]));
  const float amax = block_max_256(mx, scratch);
  const float inv = amax > 0.0f ? __fdiv_rn(127.0f, amax) : 0.0f;
  if (threadIdx.x == 0) scales[blockIdx.x] = __fdiv_rn(amax, 127.0f);
  for (int k = threadIdx.x; k < K; k += 256) {
    const int q = __float2int_rn(__fmul_rn(row[k], inv));
    codes[static_cast<size_t>(blockIdx.x) * K + k] = static_cast<int8_t>(max(-127, min(127, q)));
  }
}

// 4-bit weights: one scale per (output channel, 128 consecutive k), codes in [-7, 7], two per byte with the even
// k in the low nibble.  One warp per group, four consecutive k per lane.
__global__ void __launch_bounds__(256) quantize_rows_w4_kernel(const float* __restrict__ wr, int64_t groups_total,
                                                               uint8_t* __restrict__ packed, float* __restrict__ scales) {
  const int64_t grp = static_cast<int64_t>(blockIdx.x) * 8 + (threadIdx.x >> 5);
  if (grp >= groups_total) return;
  const int lane = threadIdx.x & 31;
  const float4 v = *reinterpret_cast<const float4*>(wr + grp * TRDQ_BLOCK + 4 * lane);
  float mx = fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w)));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  const float inv = mx > 0.0f ? __fdiv_rn(7.0f, mx) : 0.0f;
  if (lane == 0) scales[grp] = __fdiv_rn(mx, 7.0f);
  const float e[4] = {v.x, v.y, v.z, v.w};
  uint32_t nib[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) nib[i] = static_cast<uint32_t>(max(-7, min(7, __float2int_rn(__fmul_rn(e[i], inv))))) & 0xFu;
  const uint16_t two = static_cast<uint16_t>(nib[0] | (nib[1] << 4) | (nib[2] << 8) | (nib[3] << 12));
  *reinterpret_cast<uint16_t*>(packed + grp * (TRDQ_BLOCK / 2) + 2 * lane) = two;
}

template <typename Kernel>
cudaError_t launch_pass(Kernel kernel, int smem_bytes, PerDeviceFlag& configured, const DenseParams& p, dim3 grid, cudaStream_t stream) {
  int dev = 0;
  cudaGetDevice(&dev);
  if (!configured.get(dev)) {
    const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
    if (e != cudaSuccess) return e;
    configured.set(dev, true);
  }
  return launch_overlapped(kernel, grid, dim3(kThreads), smem_bytes, stream, p);
}

}  // namespace

uint64_t rotate_dense_workspace_bytes(int32_t M, int32_t K) {
  (void)K;
  return static_cast<uint64_t>(kMaxSplits) * static_cast<uint64_t>(M) * sizeof(float);
}

trdq_status launch_rotate_dense_quantize(const trdq_rotation* rot, int g, const void* x_bf16, int64_t ldx, int32_t M, int8_t* codes,
                                         float* scales, float* workspace, cudaStream_t stream) {
  const int K = rot->K, nb = K / TRDQ_BLOCK;
  DenseParams p;
  trdq_status st = encode_tmap_2d(&p.tmap_x, x_bf16, 2, K, M, static_cast<uint64_t>(ldx) * 2, 64, kRows, 128);
  if (st != TRDQ_OK) return st;
  p.tmap_s = rot->tmap_dense;
  st = encode_tmap_2d(&p.tmap_codes, codes, 1, K, M, K, 128, 32, 128);
  if (st != TRDQ_OK) return st;
  p.amax = workspace;
  p.scales = scales;
  p.M = M;
  p.K = K;
  p.s_row0 = g * nb * TRDQ_BLOCK;
  p.status = device_status_word();
  if (!p.status) return TRDQ_ERR_CUDA;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return TRDQ_ERR_CUDA;
  static PerDeviceFlag configured0, configured1;
  // Both passes cover all token tiles in one launch each.  (Cutting the rows into L2-sized chunks, each with its own
  // pair of launches, was measured: the second read then hits L2, but the extra launches cost what the hits save.)
  const int tiles = (M + kRows - 1) / kRows;
  p.tile_begin = 0;
  p.tile_end = tiles;
  // pass 0: CTAs over the token tiles; with few tiles the blocks are cut into ranges so that the SMs are filled
  p.splits = std::max(1, std::min({kMaxSplits, nb, sms / tiles}));
  p.blocks_per_split = (nb + p.splits - 1) / p.splits;
  p.splits = (nb + p.blocks_per_split - 1) / p.blocks_per_split;
  if (launch_pass(rotate_dense_amax_kernel, kSmemBytes0, configured0, p, dim3(std::min(tiles, sms), p.splits), stream) != cudaSuccess)
    return TRDQ_ERR_CUDA;
  // pass 1: every block column gets the same number of CTAs, each walking its share of the token tiles
  const int per_column = std::max(1, std::min(tiles, sms / nb));
  if (launch_pass(rotate_dense_quantize_kernel, kSmemBytes1, configured1, p, dim3(per_column, nb), stream) != cudaSuccess)
    return TRDQ_ERR_CUDA;
  return TRDQ_OK;
}

cudaError_t launch_dense_prepare(const void* w_bf16, int32_t N, int32_t K, const double* inv_t, int wbits, float* wr_scratch,
                                 void* codes, float* scales, cudaStream_t stream) {
  const int nb = K / TRDQ_BLOCK;
  dense_weight_rotate_kernel<<<dim3(nb, (N + kWRows - 1) / kWRows), TRDQ_BLOCK, 0, stream>>>(
      static_cast<const __nv_bfloat16*>(w_bf16), N, K, inv_t, wr_scratch);
  if (wbits == 8) {
    quantize_rows_w8_kernel<<<N, 256, 0, stream>>>(wr_scratch, K, static_cast<int8_t*>(codes), scales);
  } else {
    const int64_t groups_total = static_cast<int64_t>(N) * nb;
    quantize_rows_w4_kernel<<<static_cast<unsigned>((groups_total + 7) / 8), 256, 0, stream>>>(wr_scratch, groups_total,
                                                                                                static_cast<uint8_t*>(codes), scales);
  }
  return cudaGetLastError();
}

}  // namespace trdq
