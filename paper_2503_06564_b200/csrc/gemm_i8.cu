// INT8 x INT8 -> INT32 GEMM of Eq. 10 (G_t(X) . H_t(W) on the integer codes) with the
// dequantizing epilogue  y = acc * sx[m] * sw[n] + bias[n]  ->  bf16.
//
// Persistent, warp-specialised kernel for sm_100a, one CTA per SM:
//   warp 0      TMA producer: 128 x 128-byte tiles of the activation codes (A) and BN x 128-byte
//               tiles of the weight codes (B), 128-byte swizzle, into a ring of shared-memory stages
//   warp 1      MMA issuer: one thread issues tcgen05.mma kind::i8 (128 x BN x 32 per instruction,
//               four per stage); accumulators live in tensor memory, two stages of BN columns
//   warp 2      allocates / frees tensor memory
//   warps 4-11  epilogue: tcgen05.ld of the finished accumulator (a warp reads the tensor-memory
//               lanes 32*(warp%4) .. +31, one output row per thread; warps 4-7 take the left half of
//               the columns, warps 8-11 the right half), fp32 dequantization, bf16 pack into a
//               swizzled 32 x 32 staging tile in shared memory, one TMA store per tile of 32 columns
//               (row-scattered 16-byte stores from registers turned out to bound the whole kernel)
// The epilogue of tile i overlaps the main loop of tile i+1 through the second accumulator.
// Tiles are visited column-block major so that concurrently running CTAs share one weight
// tile; both CFG row segments are part of the same tile list, so a weight tile is fetched
// once for both.  Every wait is bounded (see BoundedWaiter).
#include <cuda_bf16.h>

#include <cstdio>
#include <cstdlib>

#include "epilogue.cuh"
#include "internal.h"
#include "ptx.cuh"

namespace trdq {
namespace {

constexpr int kTileM = 128;
constexpr int kTileKBytes = 128;  // one swizzle atom: 128 int8 along K per stage
constexpr int kUmmaK = 32;        // K of one kind::i8 instruction
constexpr int kThreads = 384;
constexpr int kEpilogueThreads = 256;
constexpr int kAccStride = 256;   // tensor-memory columns between the two accumulator stages
constexpr int kTmemCols = 512;
constexpr int kSmemBudget = 227 * 1024;

template <int BN>
struct Cfg {
  static constexpr int kABytes = kTileM * kTileKBytes;
  static constexpr int kBBytes = BN * kTileKBytes;
  static constexpr int kStageBytes = kABytes + kBBytes;
  // parameters staged for the epilogue: (sw, bias) and the cancellation threshold per column, one
  // buffer per accumulator stage
  static constexpr int kParamBytes = 2 * BN * 16;  // (sw, bias), threshold and (asymmetric mode) weight column sums
  static constexpr int kBarrierBytes = 256;
  // output staging: one 32-row x 32-column bf16 tile (2 KB, 64-byte swizzle) per epilogue warp
  static constexpr int kOutStageBytes = (kEpilogueThreads / 32) * 2048;
  static constexpr int kStages = (kSmemBudget - 1024 - kOutStageBytes - kParamBytes - kBarrierBytes) / kStageBytes;
  static constexpr int kSmemBytes = 1024 + kStages * kStageBytes + kOutStageBytes + kParamBytes + kBarrierBytes;
  static_assert(kStages >= 3, "pipeline too shallow");
  static_assert(kStages <= 12, "barrier area too small");
};

struct alignas(64) GemmParams {
  CUtensorMap tmap_a[2];
  CUtensorMap tmap_b;
  CUtensorMap tmap_out[2];  // bf16 output of each segment, box 32 x 32, 64-byte swizzle
  const float* sx[2];
  void* out[2];
  int64_t ld[2];
  int32_t M[2];
  int32_t tiles_m[2];
  const float* sw;
  const __nv_bfloat16* bias;
  // asymmetric activation codes (mode 2): per-row zero points of each segment and per-channel sums of the weight codes
  const int32_t* zp[2];
  const int32_t* colsum;
  int32_t N, K, tiles_n;
  // split-K (raw-accumulator mode only): the k-blocks are cut into `splits` ranges of `kb_per_split`; split s
  // writes its partial sums at out + s * split_stride (elements).  splits = 1 is the ordinary GEMM.
  int32_t splits, kb_per_split;
  int64_t split_stride;
  uint32_t* status;
};

struct TileCoord {
  int seg, m0, n0, split;
};
__device__ __forceinline__ TileCoord tile_coord(const GemmParams& p, int tile, int bn) {
  const int tiles_m = p.tiles_m[0] + p.tiles_m[1];
  const int per_split = tiles_m * p.tiles_n;
  TileCoord c;
  c.split = tile / per_split;
  tile -= c.split * per_split;
  const int nt = tile / tiles_m;
  int mt = tile - nt * tiles_m;
  c.seg = mt >= p.tiles_m[0] ? 1 : 0;
  if (c.seg) mt -= p.tiles_m[0];
  c.m0 = mt * kTileM;
  c.n0 = nt * bn;
  return c;
}

// MODE 0: bf16 dequantizing epilogue.  MODE 1: raw int32 accumulators.
// MODE 2: unsigned activation codes with zero points (Eq. 1-3): acc - z[m] * colsum[n], then the epilogue of mode 0.
// MODE 3: mode 0 with GELU (tanh form) applied to the dequantized value before the bf16 rounding.
template <int BN, int MODE>
__global__ void __launch_bounds__(kThreads, 1) gemm_w8a8_kernel(const __grid_constant__ GemmParams p) {
  using C = Cfg<BN>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t out_stage_base = smem_base + C::kStages * C::kStageBytes;
  float2* param_buf = reinterpret_cast<float2*>(smem + C::kStages * C::kStageBytes + C::kOutStageBytes);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::kStages * C::kStageBytes + C::kOutStageBytes + C::kParamBytes);
  // barrier layout: full[S], empty[S], tmem_full[2], tmem_empty[2], then the tensor-memory base address
  const uint32_t bar_full = smem_u32(bars);
  const uint32_t bar_empty = bar_full + 8 * C::kStages;
  const uint32_t bar_tfull = bar_empty + 8 * C::kStages;
  const uint32_t bar_tempty = bar_tfull + 16;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * C::kStages + 4);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int total_tiles = (p.tiles_m[0] + p.tiles_m[1]) * p.tiles_n * p.splits;
  const int num_kb_all = p.K / kTileKBytes;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_tfull + 8 * a, 1);
      mbar_init(bar_tempty + 8 * a, kEpilogueThreads / 32);
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
  if (threadIdx.x == 0) {  // descriptors are kernel arguments: fetch them while the previous kernel may still be running
    prefetch_tensormap(&p.tmap_a[0]);
    prefetch_tensormap(&p.tmap_a[1]);
    prefetch_tensormap(&p.tmap_b);
    prefetch_tensormap(&p.tmap_out[0]);
    prefetch_tensormap(&p.tmap_out[1]);
  }
  griddep_launch_dependents();
  // The weights are constants of the prepared object: the weight tiles of the first tile's first stages are requested
  // before waiting for the kernel before (which produced the activation codes), so their latency overlaps its tail.
  // RULE this relies on: griddepcontrol.wait orders this kernel only against its immediate predecessor in the stream, so
  // the weight codes must be complete before that predecessor can start.  trdq_prepare_weights guarantees it: the last
  // kernel it enqueues per group (column sums / 4-bit multipliers, or a stream synchronisation for dense rotations) is
  // launched the ordinary way, i.e. with a full dependency on the kernels that wrote the codes, and never triggers its
  // dependents early.
  int prefetched = 0;
  if (static_cast<int>(blockIdx.x) < total_tiles) {
    const TileCoord tc0 = tile_coord(p, blockIdx.x, BN);
    const int kb0 = tc0.split * p.kb_per_split;
    prefetched = min(C::kStages, min(kb0 + p.kb_per_split, num_kb_all) - kb0);
    if (threadIdx.x == 0) {
      for (int i = 0; i < prefetched; ++i) {
        mbar_arrive_expect_tx(bar_full + 8 * i, C::kStageBytes);  // the whole stage; the activation tile follows below
        tma_load_2d(smem_base + i * C::kStageBytes + C::kABytes, &p.tmap_b, (kb0 + i) * kTileKBytes, tc0.n0, bar_full + 8 * i);
      }
    }
  }
  griddep_wait();  // codes and scales may come from the kernel before; Y may still be read by it

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (elect_one()) {
      BoundedWaiter w(p.status, kStatusTimeoutProducer);
      int stage = 0;
      uint32_t phase = 0;
      for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
        const TileCoord tc = tile_coord(p, tile, BN);
        const int kb0 = tc.split * p.kb_per_split;
        const int kb1 = min(kb0 + p.kb_per_split, num_kb_all);
        for (int kb = kb0; kb < kb1; ++kb) {
          w.wait(bar_empty + 8 * stage, phase ^ 1);
          const uint32_t a_dst = smem_base + stage * C::kStageBytes;
          const uint32_t b_dst = a_dst + C::kABytes;
          const bool b_in_flight = tile == static_cast<int>(blockIdx.x) && kb - kb0 < prefetched;
          if (!b_in_flight) mbar_arrive_expect_tx(bar_full + 8 * stage, C::kStageBytes);
          tma_load_2d(a_dst, &p.tmap_a[tc.seg], kb * kTileKBytes, tc.m0, bar_full + 8 * stage);
          if (!b_in_flight) tma_load_2d(b_dst, &p.tmap_b, kb * kTileKBytes, tc.n0, bar_full + 8 * stage);
          if (++stage == C::kStages) {
            stage = 0;
            phase ^= 1;
          }
        }
      }
      w.settle();
    }
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    if (elect_one()) {
      BoundedWaiter w(p.status, kStatusTimeoutMma);
      constexpr uint32_t idesc = MODE == 2 ? umma_idesc_u8s8(BN) : umma_idesc_s8(BN);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
        w.wait(bar_tempty + 8 * acc, acc_phase ^ 1);
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * kAccStride;
        const int num_kb = min(p.kb_per_split, num_kb_all - (tile / ((p.tiles_m[0] + p.tiles_m[1]) * p.tiles_n)) * p.kb_per_split);
        for (int kb = 0; kb < num_kb; ++kb) {
          w.wait(bar_full + 8 * stage, phase);
          tc_fence_after();
          const uint32_t a_addr = smem_base + stage * C::kStageBytes;
          const uint64_t a_desc = umma_desc_k_sw128(a_addr);
          const uint64_t b_desc = umma_desc_k_sw128(a_addr + C::kABytes);
#pragma unroll
          for (int k = 0; k < kTileKBytes / kUmmaK; ++k) {
            // +32 bytes along K inside the swizzle atom = +2 in the 16-byte address field
            umma_i8(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit(bar_empty + 8 * stage);  // frees the stage once these MMAs have read it
          if (++stage == C::kStages) {
            stage = 0;
            phase ^= 1;
          }
        }
        umma_commit(bar_tfull + 8 * acc);  // accumulator complete
        if (++acc == 2) {
          acc = 0;
          acc_phase ^= 1;
        }
      }
      w.settle();
    }
  } else if (warp >= 4) {
    // ---------------------------------------------------------------- epilogue
    const int ew = warp - 4;                // 0..7
    const int q = ew & 3;                   // = warp % 4: the lane quarter of tensor memory this warp may read
    const int half = ew >> 2;               // which half of the tile's columns
    const int et = threadIdx.x - 4 * 32;    // 0..255
    constexpr int kChunksPerWarp = BN / 64; // 32-column chunks per warp
    const uint32_t my_stage = out_stage_base + ew * 2048;
    BoundedWaiter w(p.status, kStatusTimeoutEpilogue);
    int acc = 0;
    uint32_t acc_phase = 0;
    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
      const TileCoord tc = tile_coord(p, tile, BN);
      float2* pb = param_buf + acc * BN;                                           // (sw, bias)
      float* thr = reinterpret_cast<float*>(param_buf + 2 * BN) + acc * BN;        // 2^-10 * |bias|
      int32_t* csum = reinterpret_cast<int32_t*>(reinterpret_cast<float*>(param_buf + 2 * BN) + 2 * BN) + acc * BN;
      if (MODE != 1) {
        stage_column_params(pb, thr, p.sw, p.bias, tc.n0, p.N, BN, et, kEpilogueThreads);
        if (MODE == 2)
          for (int c = et; c < BN; c += kEpilogueThreads) csum[c] = tc.n0 + c < p.N ? __ldg(p.colsum + tc.n0 + c) : 0;
        asm volatile("bar.sync 1, %0;" ::"n"(kEpilogueThreads) : "memory");
      }
      const int row = tc.m0 + q * 32 + lane;
      const bool row_ok = row < p.M[tc.seg];
      const float sxm = (MODE != 1 && row_ok) ? __ldg(p.sx[tc.seg] + row) : 0.0f;
      const int32_t zrow = (MODE == 2 && row_ok) ? __ldg(p.zp[tc.seg] + row) : 0;

      w.wait(bar_tfull + 8 * acc, acc_phase);
      __syncwarp();
      tc_fence_after();
      const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * kAccStride;
#pragma unroll 1
      for (int cc = 0; cc < kChunksPerWarp; ++cc) {
        const int c = half * kChunksPerWarp + cc;
        uint32_t r[32];
        tmem_ld_32x32(t_row + c * 32, r);
        tmem_wait_ld();
        const int n_base = tc.n0 + c * 32;
        if (MODE == 2) {
          // sum_k (q - z) * qw = sum_k q * qw - z * sum_k qw
#pragma unroll
          for (int j = 0; j < 32; ++j) r[j] = static_cast<uint32_t>(static_cast<int32_t>(r[j]) - zrow * csum[c * 32 + j]);
        }
        if (MODE != 1) {
          const float4* pb4 = reinterpret_cast<const float4*>(pb + c * 32);
          const float4* thr4 = reinterpret_cast<const float4*>(thr + c * 32);
          uint32_t packed[16];
          dequant_row32<MODE == 3>(r, sxm, pb4, thr4, packed);
          // staging tile: row = lane, 64 bytes per row, 16-byte chunk j stored at j ^ ((lane >> 1) & 3)
          if (lane == 0) bulk_wait_group_read<0>();  // the previous store has finished reading the tile
          __syncwarp();
#pragma unroll
          for (int v = 0; v < 4; ++v)
            st_shared_v4(my_stage + lane * 64 + ((v ^ ((lane >> 1) & 3)) << 4), packed[4 * v], packed[4 * v + 1], packed[4 * v + 2],
                         packed[4 * v + 3]);
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) {
            tma_store_2d(&p.tmap_out[tc.seg], n_base, tc.m0 + q * 32, my_stage);  // rows >= M and columns >= N are clipped
            bulk_commit_group();
          }
        } else if (row_ok) {
          int32_t* out = static_cast<int32_t*>(p.out[tc.seg]) + tc.split * p.split_stride + static_cast<int64_t>(row) * p.ld[tc.seg] + n_base;
#pragma unroll
          for (int v = 0; v < 8; ++v) {
            if (n_base + 4 * v < p.N)
              *reinterpret_cast<uint4*>(out + 4 * v) = make_uint4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_tempty + 8 * acc);
      if (++acc == 2) {
        acc = 0;
        acc_phase ^= 1;
      }
    }
    if (MODE != 1 && lane == 0) bulk_wait_group_read<0>();  // the staging tiles have been read; the stores complete before the grid does
    w.settle();
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 2) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

template <int BN, int MODE>
cudaError_t launch_one(const GemmParams& p, int grid, cudaStream_t stream) {
  using C = Cfg<BN>;
  static PerDeviceFlag configured;
  int dev = 0;
  cudaGetDevice(&dev);
  if (!configured.get(dev)) {
    cudaError_t e = cudaFuncSetAttribute(gemm_w8a8_kernel<BN, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
    if (e != cudaSuccess) return e;
    configured.set(dev, true);
  }
  return launch_overlapped(gemm_w8a8_kernel<BN, MODE>, dim3(grid), dim3(kThreads), C::kSmemBytes, stream, p);
}

// Cost model for the tile width: waves of CTAs times the time of one tile (main loop grows
// with BN; the 128-row operand and the fixed per-tile overhead do not).
int choose_tile_n(int64_t tiles_m, int N, int sms) {
  int best = 0;
  double best_cost = 1e300;
  for (int i = 0; i < kNumTileN; ++i) {
    const int bn = kTileN[i];
    const int64_t tiles = tiles_m * ((N + bn - 1) / bn);
    const int64_t waves = (tiles + sms - 1) / sms;
    const double cost = static_cast<double>(waves) * (bn + 24.0);
    if (cost < best_cost) {
      best_cost = cost;
      best = i;
    }
  }
  return best;
}

}  // namespace

// Row count from which the CTA-pair kernel is used (two SMs per 256-row tile, a third less operand traffic per SM).
static int pair_min_rows() {
  static const int rows = [] {
    const char* e = getenv("TRDQ_PAIR_MIN_M");
    return e ? atoi(e) : 2048;
  }();
  return rows;
}

// Name of the kernel trdq_linear runs for M rows against [N, K] weights of `wbits` bits (one row segment).
void describe_gemm_kernel(int32_t M, int32_t K, int32_t N, int32_t wbits, char* name, size_t cap) {
  (void)K;
  if (wbits == 4) {
    snprintf(name, cap, "gemm_w4a8_kernel");
    return;
  }
  if (M >= pair_min_rows()) {
    const int bn = gemm_w8_pair_tile_width((static_cast<int64_t>(M) + 2 * kTileM - 1) / (2 * kTileM), N);
    if (bn > 0) {
      snprintf(name, cap, "gemm_w8a8_pair_kernel<%d>", bn);
      return;
    }
  }
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  snprintf(name, cap, "gemm_w8a8_kernel<%d>", kTileN[choose_tile_n((static_cast<int64_t>(M) + kTileM - 1) / kTileM, N, sms)]);
}

static trdq_status launch_gemm_w8_mode(const trdq_weights* w, int g, const GemmSegment seg[2], const void* bias_bf16, int mode,
                                       const int32_t* const zp[2], cudaStream_t stream, int act = 0) {
  const bool raw_i32 = mode == 1;
  if (mode == 0 && static_cast<int64_t>(seg[0].M) + seg[1].M >= pair_min_rows()) {
    const trdq_status st = launch_gemm_w8_pair(w, g, seg, bias_bf16, stream, act);
    if (st != TRDQ_ERR_SHAPE) return st;
  }
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) != cudaSuccess) return TRDQ_ERR_CUDA;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);

  GemmParams p;
  int64_t tiles_m = 0;
  for (int s = 0; s < 2; ++s) {
    p.sx[s] = seg[s].sx;
    p.out[s] = seg[s].out;
    p.ld[s] = seg[s].ld;
    p.M[s] = seg[s].M;
    p.tiles_m[s] = (seg[s].M + kTileM - 1) / kTileM;
    tiles_m += p.tiles_m[s];
  }
  if (tiles_m == 0) return TRDQ_OK;
  const int ti = choose_tile_n(tiles_m, w->N, sms);
  const int bn = kTileN[ti];
  for (int s = 0; s < 2; ++s) {
    // an empty segment still needs a valid descriptor object; reuse the other segment's
    const GemmSegment& src = seg[s].M > 0 ? seg[s] : seg[1 - s];
    trdq_status st = encode_tmap_u8_sw128(&p.tmap_a[s], src.codes, static_cast<uint64_t>(w->K), static_cast<uint64_t>(src.M),
                                          static_cast<uint64_t>(w->K), kTileKBytes, kTileM);
    if (st != TRDQ_OK) return st;
  }
  for (int s = 0; s < 2 && !raw_i32; ++s) {
    const GemmSegment& src = seg[s].M > 0 ? seg[s] : seg[1 - s];
    trdq_status st = encode_tmap_2d(&p.tmap_out[s], src.out, 2, static_cast<uint64_t>(w->N), static_cast<uint64_t>(src.M),
                                    static_cast<uint64_t>(src.ld) * 2, 32, 32, 64);
    if (st != TRDQ_OK) return st;
  }
  if (raw_i32) p.tmap_out[0] = p.tmap_out[1] = p.tmap_a[0];  // unused by the raw-accumulator mode
  p.tmap_b = w->groups[g].tmap_b[ti];
  p.sw = w->groups[g].scales;
  p.bias = static_cast<const __nv_bfloat16*>(bias_bf16);
  p.N = w->N;
  p.K = w->K;
  p.tiles_n = (w->N + bn - 1) / bn;
  p.splits = 1;
  p.kb_per_split = w->K / kTileKBytes;
  p.split_stride = 0;
  p.zp[0] = zp ? zp[0] : nullptr;
  p.zp[1] = zp ? zp[1] : nullptr;
  p.colsum = w->groups[g].colsum;
  p.status = device_status_word();
  if (!p.status) return TRDQ_ERR_CUDA;
  const int64_t total = tiles_m * p.tiles_n;
  const int grid = static_cast<int>(total < sms ? total : sms);

  cudaError_t e;
  if (raw_i32) {
    e = bn == 128 ? launch_one<128, 1>(p, grid, stream) : bn == 192 ? launch_one<192, 1>(p, grid, stream) : launch_one<256, 1>(p, grid, stream);
  } else if (mode == 2) {
    e = bn == 128 ? launch_one<128, 2>(p, grid, stream) : bn == 192 ? launch_one<192, 2>(p, grid, stream) : launch_one<256, 2>(p, grid, stream);
  } else if (act) {
    e = bn == 128 ? launch_one<128, 3>(p, grid, stream) : bn == 192 ? launch_one<192, 3>(p, grid, stream) : launch_one<256, 3>(p, grid, stream);
  } else {
    e = bn == 128 ? launch_one<128, 0>(p, grid, stream) : bn == 192 ? launch_one<192, 0>(p, grid, stream) : launch_one<256, 0>(p, grid, stream);
  }
  return e == cudaSuccess ? TRDQ_OK : TRDQ_ERR_CUDA;
}

trdq_status launch_gemm_w8(const trdq_weights* w, int g, const GemmSegment seg[2], const void* bias_bf16, bool raw_i32,
                           cudaStream_t stream, int act) {
  return launch_gemm_w8_mode(w, g, seg, bias_bf16, raw_i32 ? 1 : 0, nullptr, stream, act);
}

// Unsigned activation codes with per-row zero points (Eq. 1-3); `w` must carry the column sums of its codes.
trdq_status launch_gemm_w8_asym(const trdq_weights* w, int g, const GemmSegment seg[2], const int32_t* const zp[2],
                                const void* bias_bf16, cudaStream_t stream) {
  if (!w->groups[g].colsum) return TRDQ_ERR_WBITS;
  return launch_gemm_w8_mode(w, g, seg, bias_bf16, 2, zp, stream);
}

// Row sums of the int8 weight codes, one warp per output channel.
namespace {
__global__ void weight_colsum_kernel(const int8_t* __restrict__ codes, int32_t N, int32_t K, int32_t* __restrict__ colsum) {
  const int n = blockIdx.x * (blockDim.x / 32) + (threadIdx.x >> 5);
  if (n >= N) return;
  const int lane = threadIdx.x & 31;
  const int4* row = reinterpret_cast<const int4*>(codes + static_cast<int64_t>(n) * K);
  int32_t s = 0;
  for (int i = lane; i < K / 16; i += 32) {
    const int4 v = row[i];
    const int32_t wd[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) s = __dp4a(wd[j], 0x01010101, s);  // four signed bytes times 1
  }
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if (lane == 0) colsum[n] = s;
}
}  // namespace

cudaError_t launch_weight_colsum(const int8_t* codes, int32_t N, int32_t K, int32_t* colsum, cudaStream_t stream) {
  weight_colsum_kernel<<<(N + 7) / 8, 256, 0, stream>>>(codes, N, K, colsum);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Split-K for problems with too few output tiles to fill the GPU (few rows, long K): the k-blocks
// are divided among `splits` CTAs per output tile, each writes exact int32 partial sums to a
// workspace, and a second kernel adds them (integer addition: the result does not depend on the
// order) and applies the same dequantizing arithmetic as the fused epilogue.
// ---------------------------------------------------------------------------------------------
namespace {

__global__ void __launch_bounds__(256) splitk_reduce_epilogue_kernel(const int32_t* __restrict__ part, int splits, int64_t split_stride, int M,
                                                                     int N, const float* __restrict__ sx, const float* __restrict__ sw,
                                                                     const __nv_bfloat16* __restrict__ bias, __nv_bfloat16* __restrict__ y,
                                                                     int64_t ldy) {
  griddep_launch_dependents();
  griddep_wait();
  const int vec_per_row = N / 8;  // N is a multiple of 16
  const int64_t total = static_cast<int64_t>(M) * vec_per_row;
  for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < total; i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const int m = static_cast<int>(i / vec_per_row);
    const int n = static_cast<int>(i - static_cast<int64_t>(m) * vec_per_row) * 8;
    int32_t acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    for (int s = 0; s < splits; ++s) {
      const int4* src = reinterpret_cast<const int4*>(part + s * split_stride + static_cast<int64_t>(m) * N + n);
      const int4 a = src[0], b = src[1];
      acc[0] += a.x; acc[1] += a.y; acc[2] += a.z; acc[3] += a.w;
      acc[4] += b.x; acc[5] += b.y; acc[6] += b.z; acc[7] += b.w;
    }
    const float sxm = __ldg(sx + m);
    uint32_t packed[4];
#pragma unroll
    for (int e = 0; e < 8; e += 2) {
      float v2[2];
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const float swn = __ldg(sw + n + e + u);
        const float bn = bias ? __bfloat162float(bias[n + e + u]) : 0.0f;
        v2[u] = dequant_one(acc[e + u], sxm, swn, bn, fabsf(bn) * 0.0009765625f);
      }
      const __nv_bfloat162 h = __floats2bfloat162_rn(v2[0], v2[1]);
      packed[e / 2] = *reinterpret_cast<const uint32_t*>(&h);
    }
    *reinterpret_cast<uint4*>(y + static_cast<int64_t>(m) * ldy + n) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
  }
}

}  // namespace

// Number of k-ranges worth using for an M-row problem on the current device (1 = split-K does not pay).
int splitk_choose(const trdq_weights* w, int32_t M) {
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int64_t tiles = static_cast<int64_t>((M + kTileM - 1) / kTileM) * ((w->N + 127) / 128);
  const int num_kb = w->K / kTileKBytes;
  // Measured on B200: the second kernel and its launch cost about as much as 40 k-blocks of main loop, so
  // splitting only pays when the reduction is long (K >= 8192) and the tiles fill less than half the SMs.
  if (w->wbits != 8 || tiles <= 0 || tiles * 2 > sms || num_kb < 64) return 1;
  int splits = static_cast<int>(sms / tiles);
  if (splits > 8) splits = 8;
  while (splits > 1 && num_kb / splits < 4) --splits;  // at least four k-blocks per range
  if (splits < 1) splits = 1;
  const int per = (num_kb + splits - 1) / splits;
  return (num_kb + per - 1) / per;  // no empty range
}

trdq_status launch_gemm_w8_splitk(const trdq_weights* w, int g, const GemmSegment& seg, const void* bias_bf16, int splits,
                                  int32_t* workspace, cudaStream_t stream) {
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) != cudaSuccess) return TRDQ_ERR_CUDA;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  GemmParams p;
  p.sx[0] = p.sx[1] = nullptr;
  p.out[0] = p.out[1] = workspace;
  p.ld[0] = p.ld[1] = w->N;
  p.M[0] = seg.M;
  p.M[1] = 0;
  p.tiles_m[0] = (seg.M + kTileM - 1) / kTileM;
  p.tiles_m[1] = 0;
  trdq_status st = encode_tmap_u8_sw128(&p.tmap_a[0], seg.codes, static_cast<uint64_t>(w->K), static_cast<uint64_t>(seg.M),
                                        static_cast<uint64_t>(w->K), kTileKBytes, kTileM);
  if (st != TRDQ_OK) return st;
  p.tmap_a[1] = p.tmap_a[0];
  p.tmap_out[0] = p.tmap_out[1] = p.tmap_a[0];  // unused in the raw-accumulator mode
  p.tmap_b = w->groups[g].tmap_b[0];             // 128-column tiles
  p.sw = nullptr;
  p.bias = nullptr;
  p.zp[0] = p.zp[1] = nullptr;
  p.colsum = nullptr;
  p.N = w->N;
  p.K = w->K;
  p.tiles_n = (w->N + 127) / 128;
  const int num_kb = w->K / kTileKBytes;
  p.kb_per_split = (num_kb + splits - 1) / splits;
  p.splits = (num_kb + p.kb_per_split - 1) / p.kb_per_split;
  p.split_stride = static_cast<int64_t>(seg.M) * w->N;
  p.status = device_status_word();
  if (!p.status) return TRDQ_ERR_CUDA;
  const int64_t total = static_cast<int64_t>(p.tiles_m[0]) * p.tiles_n * p.splits;
  const int grid = static_cast<int>(total < sms ? total : sms);
  if (launch_one<128, 1>(p, grid, stream) != cudaSuccess) return TRDQ_ERR_CUDA;
  const int64_t vecs = static_cast<int64_t>(seg.M) * (w->N / 8);
  int64_t rgrid = (vecs + 255) / 256;
  if (rgrid > static_cast<int64_t>(sms) * 8) rgrid = static_cast<int64_t>(sms) * 8;
  const cudaError_t e = launch_overlapped(splitk_reduce_epilogue_kernel, dim3(static_cast<unsigned>(rgrid)), dim3(256), 0, stream,
                                          static_cast<const int32_t*>(workspace), p.splits, p.split_stride, seg.M, w->N, seg.sx,
                                          static_cast<const float*>(w->groups[g].scales), static_cast<const __nv_bfloat16*>(bias_bf16),
                                          static_cast<__nv_bfloat16*>(seg.out), seg.ld);
  return e == cudaSuccess ? TRDQ_OK : TRDQ_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------------
// Split-K without any allocation: the partial sums live in a fixed array that is part of the
// library image.  Every device that loads the library carries these 8 MiB until the process exits.
// ---------------------------------------------------------------------------------------------
static __device__ __align__(256) int32_t g_static_splitk_scratch[TRDQ_STATIC_SCRATCH_ELEMS];

// Device address of the array on the CURRENT device.  In host code the array's name is only a handle
// for the runtime, not an address a kernel could use, so the address is asked for once per device
// (with that device current) and remembered.
static int32_t* static_scratch_address() {
  static PerDevice<int32_t*> cached;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  int32_t* ptr = cached.get(dev);
  if (!ptr) {
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_static_splitk_scratch) != cudaSuccess || !ptr) {
      cudaGetLastError();
      return nullptr;
    }
    cached.set(dev, ptr);
  }
  return ptr;
}

trdq_status launch_gemm_w8_splitk_static(const trdq_weights* w, int g, const GemmSegment& seg, const void* bias_bf16, int splits,
                                         cudaStream_t stream) {
  if (static_cast<uint64_t>(splits) * static_cast<uint64_t>(seg.M) * static_cast<uint64_t>(w->N) > TRDQ_STATIC_SCRATCH_ELEMS)
    return TRDQ_ERR_SCRATCH;
  int32_t* scratch = static_scratch_address();
  if (!scratch) return TRDQ_ERR_CUDA;
  // Nothing has to be cleared: the first kernel writes every partial sum (all ranges, all rows < M, all
  // columns < N) that the second kernel reads, so what an earlier call left behind is never seen.
  return launch_gemm_w8_splitk(w, g, seg, bias_bf16, splits, scratch, stream);
}

}  // namespace trdq
