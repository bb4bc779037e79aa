// Fused online transform + per-token quantizer (Sec. 3.2 Eq. 10 G_t; Sec. 3.1 Eq. 1-2): TMA-staged input, ONE THREAD
// PER 128-BLOCK, and the CTA split into small TEAMS that each run their own pipeline.
//
// A thread holds a whole block (128 fp32 values in registers), so all seven butterfly stages are register-to-register
// packed fp32x2 operations.  That costs ~160 registers per thread, i.e. at most twelve warps per SM, so latency cannot be
// hidden by occupancy.  It is hidden by letting the warps run out of phase instead: a team is the smallest group of warps
// that holds whole rows (K = 1152: one warp = 3 rows of 9 blocks, 27 of 32 lanes; K = 4608: five warps = 4 rows of 36
// blocks, 144 of 160 lanes), and every team has its own two-stage TMA ring, its own row-maximum exchange, its own code
// staging tile and its own named barrier.  Nothing synchronises two teams, so while one waits for data or for its row
// maximum the others transform; there is no producer warp (lane 0 of a team refills the stage its team has just read).
//
// The arithmetic (one fp32 multiply by the fused vector, stages h = 1 .. 64 in this order with separately rounded
// additions, rne via the 1.5 * 2^23 addition) is the same as in the other kernels of rotate_quantize.cu and
// bit-identical to a scalar evaluation.  Every wait is bounded.
#include <cuda_bf16.h>

#include "internal.h"
#include "lane_group.cuh"
#include "ptx.cuh"

namespace trdq {
namespace {

constexpr int kMaxWarps = 12;        // 12 x 32 threads x <= 168 registers fill the register file
constexpr int kVecPadFloats = 4;     // the fused vector of block b starts at float b * (128 + 4): see the staging loop

struct alignas(64) TeamParams {
  // Both maps view a row as K/64 (K/128) column boxes: dims (column in box, row, box), so that ONE copy moves a tile of R
  // whole rows and lays it out box after box, each box R rows of 128 bytes, 128-byte swizzle.
  CUtensorMap tmap_x;      // bf16: (64, M, K/64), box 64 x R x K/64
  CUtensorMap tmap_codes;  // int8: (128, M, K/128), box 128 x R x K/128
  const float* vec;        // fused vector of the group, K floats
  float* scales;           // [M]
  int32_t M, K;
  int32_t R;               // rows per team tile
  int32_t team_warps;      // warps per team (R * K/128 <= 32 * team_warps)
  int32_t teams;           // teams per CTA
  float zero;              // 0.0f, see the quantizer below
  uint32_t* status;
};

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}

// max(|a|, |b|, |c|) in one instruction
__device__ __forceinline__ float max3_abs(float a, float b, float c) {
  float r;
  asm("max.abs.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

__device__ __forceinline__ void team_barrier(int team, int team_threads) {
  if (team_threads == 32)
    __syncwarp();
  else
    asm volatile("bar.sync %0, %1;" ::"r"(team + 1), "r"(team_threads) : "memory");
}

__global__ void __launch_bounds__(kMaxWarps * 32, 1) rotate_quantize_team_kernel(const __grid_constant__ TeamParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 127u) & ~127u;  // TMA destinations need 128 bytes; the swizzle is a function of the address
  uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
  const int nb = p.K / TRDQ_BLOCK;
  const int R = p.R;
  const uint32_t box_bytes = R * 128;             // one column box: R rows of 128 bytes
  const uint32_t in_bytes = 2 * nb * box_bytes;   // R x K bf16
  const uint32_t out_bytes = nb * box_bytes;      // R x K int8
  const uint32_t team_bytes = 2 * in_bytes + out_bytes;
  float* svec = reinterpret_cast<float*>(smem + p.teams * team_bytes);
  unsigned int* row_max_all = reinterpret_cast<unsigned int*>(svec + nb * (TRDQ_BLOCK + kVecPadFloats));  // [teams][3][R]
  uint64_t* bars = reinterpret_cast<uint64_t*>(row_max_all + ((p.teams * 3 * R + 1) & ~1));                  // [teams][2]

  const int tid = threadIdx.x;
  const int team_threads = p.team_warps * 32;
  const int team = tid / team_threads;
  const int tt = tid - team * team_threads;
  const uint32_t team_base = smem_base + team * team_bytes;
  const uint32_t out_base = team_base + 2 * in_bytes;
  unsigned int* row_max = row_max_all + team * 3 * R;
  const uint32_t bar_full = smem_u32(bars + 2 * team);  // [2]

  if (tt == 0) {
    mbar_init(bar_full, 1);
    mbar_init(bar_full + 8, 1);
    fence_mbar_init();
  }
  // The fused vector, block b at float b * 132: lanes of a quarter warp that hold different blocks then read different
  // bank groups with their 16-byte loads (same block: same address, a broadcast).
  for (int i = tid; i < p.K / 4; i += blockDim.x) {
    const int b = i >> 5;
    reinterpret_cast<float4*>(svec + b * (TRDQ_BLOCK + kVecPadFloats))[i & 31] = __ldg(reinterpret_cast<const float4*>(p.vec) + i);
  }
  for (int i = tid; i < p.teams * 3 * R; i += blockDim.x) row_max_all[i] = 0u;
  if (tid == 0) {
    prefetch_tensormap(&p.tmap_x);
    prefetch_tensormap(&p.tmap_codes);
  }
  __syncthreads();
  griddep_launch_dependents();
  griddep_wait();  // X may be written, and the code buffer still read, by the kernel before (the group vector is constant)

  // Tiles of R rows are dealt to the teams of the whole grid, SM after SM, so that the teams with one tile more than
  // the others are spread over all SMs.
  const int num_tiles = (p.M + R - 1) / R;
  const int stride = gridDim.x * p.teams;
  const int first = team * gridDim.x + blockIdx.x;
  // Only the FIRST tile of every team is requested here; the second one follows when the first has landed (below).  All
  // teams of all CTAs start together, so asking for both at once doubles the burst every first tile has to wait behind.
  if (tt == 0 && first < num_tiles) {
    mbar_arrive_expect_tx(bar_full, in_bytes);
    tma_load_3d(team_base, &p.tmap_x, 0, first * R, 0, bar_full);  // all 2 * nb column boxes in one copy
  }

  // consecutive threads = consecutive rows of one block column
  const bool active = tt < R * nb;
  const int b = active ? tt / R : 0;
  const int r = active ? tt - b * R : 0;
  const float4* sv4 = reinterpret_cast<const float4*>(svec + b * (TRDQ_BLOCK + kVecPadFloats));
  const float2 neg1 = make_float2(-1.0f, -1.0f);

  BoundedWaiter w(p.status, kStatusTimeoutEpilogue);
  int it = 0;
  for (int tile = first; tile < num_tiles; tile += stride, ++it) {
    const int s = it & 1;
    const uint32_t phase = (it >> 1) & 1;
    const int buf = it % 3;
    if (tt < R) row_max[((it + 1) % 3) * R + tt] = 0u;

    w.wait(bar_full + 8 * s, phase);
    if (it == 0 && tt == 0 && tile + stride < num_tiles) {  // the team's second tile, into the other stage
      mbar_arrive_expect_tx(bar_full + 8, in_bytes);
      tma_load_3d(team_base + in_bytes, &p.tmap_x, 0, (tile + stride) * R, 0, bar_full + 8);
    }
    // v[32h + 4j + i] = elements (2i, 2i+1) of 16-byte chunk j of half h, times the fused vector
    float2 v[64];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const uint32_t in_row = team_base + s * in_bytes + (2 * b + h) * box_bytes + r * 128;
      const uint32_t swz = (in_row >> 7) & 7u;  // 128-byte swizzle: chunk index xor address bits 7..9
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const uint4 raw = lds128(in_row + ((j ^ swz) << 4));
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
    for (int q = 0; q < 64; ++q) m = max3_abs(m, v[q].x, v[q].y);
    if (active) atomicMax(&row_max[buf * R + r], __float_as_uint(m));
    if (tt == 0) bulk_wait_group_read<0>();  // the previous tile's store has finished reading the staging tile
    team_barrier(team, team_threads);        // row maxima complete; every thread of the team has read stage s

    if (tt == 0) {
      const int next = tile + 2 * stride;
      if (next < num_tiles) {
        mbar_arrive_expect_tx(bar_full + 8 * s, in_bytes);
        tma_load_3d(team_base + s * in_bytes, &p.tmap_x, 0, next * R, 0, bar_full + 8 * s);
      }
    }

    const float amax = __uint_as_float(row_max[buf * R + r]);
    const float inv = amax > 0.0f ? __fdiv_rn(127.0f, amax) : 0.0f;
    const float2 inv2 = make_float2(inv, inv);
    const float2 magic2 = make_float2(kRoundMagic, kRoundMagic);
    // The product must be rounded to fp32 before the magic addition rounds it to an integer.  A packed multiply feeding
    // a packed add is contracted into one fused operation by the assembler, so the product is written as
    // fma(v, inv, zero) with `zero` a kernel argument equal to 0.0f.
    const float2 zero2 = make_float2(p.zero, p.zero);
    if (active) {
      const uint32_t out_row = out_base + b * box_bytes + r * 128;
      const uint32_t oswz = (out_row >> 7) & 7u;
#pragma unroll
      for (int c = 0; c < 8; ++c) {  // 16 codes = 8 pairs per 16-byte chunk
        float2 q[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) q[i] = __fadd2_rn(__ffma2_rn(v[c * 8 + i], inv2, zero2), magic2);
        st_shared_v4(out_row + ((c ^ oswz) << 4), pack4(q[0], q[1]), pack4(q[2], q[3]), pack4(q[4], q[5]), pack4(q[6], q[7]));
      }
      const int64_t row = static_cast<int64_t>(tile) * R + r;
      if (b == 0 && row < p.M) p.scales[row] = __fdiv_rn(amax, 127.0f);
    }
    fence_proxy_async_smem();
    team_barrier(team, team_threads);
    if (tt == 0) {
      tma_store_3d(&p.tmap_codes, 0, tile * R, 0, out_base);  // all nb column boxes; rows >= M are clipped
      bulk_commit_group();
    }
  }
  if (tt == 0) bulk_wait_group_read<0>();  // the staging tile has been read; the stores complete before the grid does
  w.settle();
}

struct TeamShape {
  int R, team_warps, teams;
  size_t smem;
  double use;  // fraction of the twelve warps' lanes that hold a block
};

size_t team_smem_bytes(int K, int R, int teams) {
  const int nb = K / TRDQ_BLOCK;
  return 128 + static_cast<size_t>(teams) * 5 * R * K + static_cast<size_t>(nb) * (TRDQ_BLOCK + kVecPadFloats) * 4 +
         (static_cast<size_t>(teams) * 3 * R + 2) * 4 + static_cast<size_t>(teams) * 16 + 16;
}

// The team of `tw` warps for rows of K channels: as many whole rows as its lanes hold, as many teams as registers
// (twelve warps) and shared memory (two input stages and a code tile per team) allow.  At least two teams, so that one
// can transform while another waits.
bool team_shape_for(int K, int tw, TeamShape* out) {
  const int nb = K / TRDQ_BLOCK;
  int rows = tw * 32 / nb;
  if (rows < 1) return false;
  if (rows > 32) rows = 32;
  int teams = kMaxWarps / tw;
  while (teams > 0 && team_smem_bytes(K, rows, teams) > 227u * 1024u) --teams;
  if (teams < 2) return false;
  *out = TeamShape{rows, tw, teams, team_smem_bytes(K, rows, teams),
                   static_cast<double>(rows) * nb / (tw * 32) * (static_cast<double>(teams * tw) / kMaxWarps)};
  return true;
}

// Team size by lane use (K = 1152: one warp, 3 rows, 27 of 32 lanes, twelve teams; K = 4608: four warps, 3 rows, 108 of
// 128 lanes, three teams).  With fewer than about one tile per team the next larger team is taken when the best one
// is a single warp: fewer, fatter tiles finish sooner when nothing is left to overlap (K = 1152, M = 4096: 6.2 against
// 6.7 us, measured).
bool choose_team_shape(int M, int K, int sms, TeamShape* out) {
  TeamShape best = {0, 0, 0, 0, 0.0};
  for (int tw = 1; tw <= kMaxWarps / 2; ++tw) {
    TeamShape s;
    if (team_shape_for(K, tw, &s) && s.use > best.use + 1e-9) best = s;
  }
  if (best.teams == 0) return false;
  const int64_t tiles = (static_cast<int64_t>(M) + best.R - 1) / best.R;
  TeamShape wider;
  if (best.team_warps == 1 && 4 * tiles < 5ll * best.teams * sms && team_shape_for(K, 2, &wider)) best = wider;
  *out = best;
  return true;
}

int device_sm_count(int* dev_out) {
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) != cudaSuccess) return -1;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (dev_out) *dev_out = dev;
  return sms;
}

}  // namespace

// The team kernel serves rows for which at least two teams fit in shared memory, once there is at least a tile per SM; below
// that the lane-group kernel, whose CTAs are smaller and start sooner, finishes first (M = 256, K = 1024: 2.3 against 3.3 us).
bool rotate_quantize_prefers_team(int32_t M, int32_t K) {
  const int sms = device_sm_count(nullptr);
  TeamShape s;
  if (sms <= 0 || !choose_team_shape(M, K, sms, &s)) return false;
  return (static_cast<int64_t>(M) + s.R - 1) / s.R >= sms;
}

trdq_status launch_rotate_quantize_team(const void* x_bf16, int64_t ldx, int32_t M, int32_t K, const float* vec, int8_t* codes,
                                        float* scales, cudaStream_t stream) {
  int dev = 0;
  const int sms = device_sm_count(&dev);
  if (sms <= 0) return TRDQ_ERR_CUDA;
  TeamShape shape;
  if (!choose_team_shape(M, K, sms, &shape)) return TRDQ_ERR_SHAPE;
  const int nb = K / TRDQ_BLOCK;
  TeamParams p;
  trdq_status st = encode_tmap_boxes(&p.tmap_x, x_bf16, 2, 64, static_cast<uint64_t>(M), static_cast<uint64_t>(ldx) * 2,
                                     static_cast<uint32_t>(2 * nb), static_cast<uint32_t>(shape.R));
  if (st != TRDQ_OK) return st;
  st = encode_tmap_boxes(&p.tmap_codes, codes, 1, 128, static_cast<uint64_t>(M), static_cast<uint64_t>(K), static_cast<uint32_t>(nb),
                         static_cast<uint32_t>(shape.R));
  if (st != TRDQ_OK) return st;
  p.vec = vec;
  p.scales = scales;
  p.M = M;
  p.K = K;
  p.R = shape.R;
  p.team_warps = shape.team_warps;
  p.teams = shape.teams;
  p.zero = 0.0f;
  p.status = device_status_word();
  if (!p.status) return TRDQ_ERR_CUDA;
  static PerDeviceFlag configured;
  if (!configured.get(dev)) {
    if (cudaFuncSetAttribute(rotate_quantize_team_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
      return TRDQ_ERR_CUDA;
    configured.set(dev, true);
  }
  const int num_tiles = (M + shape.R - 1) / shape.R;
  const int grid = num_tiles < sms ? num_tiles : sms;  // few tiles: spread them over the SMs, fewer busy teams on each
  const cudaError_t e = launch_overlapped(rotate_quantize_team_kernel, dim3(grid), dim3(shape.teams * shape.team_warps * 32), shape.smem,
                                          stream, p);
  return e == cudaSuccess ? TRDQ_OK : TRDQ_ERR_CUDA;
}

}  // namespace trdq
