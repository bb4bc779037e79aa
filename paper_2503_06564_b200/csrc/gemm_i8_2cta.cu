// INT8 GEMM + dequantizing epilogue, CTA-PAIR variant (tcgen05 cta_group::2).
//
// Two CTAs of a cluster (two SMs) compute one 256 x BN tile of Y.  Each CTA loads its own 128 rows of
// the activation codes and HALF of the weight tile (BN/2 rows); one thread of the leader CTA issues
// tcgen05.mma cta_group::2 (256 x BN x 32), which reads A and B from both CTAs' shared memory and
// writes each CTA's 128 rows of the accumulator into that CTA's tensor memory.  Per multiply-add the
// pair pulls 2/3 (BN = 256) of the operand bytes the single-CTA kernel pulls from L2, which is what
// bounded that kernel (measured with operand loads removed: 2.7 -> 4.0 PTOPS at K = N = 4608).
//
// Synchronisation (all mbarriers; every wait bounded):
//   full[s]    in the LEADER: both producers arrive with their byte counts; both CTAs' TMA copies
//              complete on it (the copies carry .cta_group::2 so that they may signal the peer CTA)
//   empty[s]   in each CTA: tcgen05.commit multicast to both CTAs when the MMAs reading stage s are done
//   tfull[a]   in each CTA: tcgen05.commit multicast when accumulator a is complete
//   tempty[a]  in the LEADER: the epilogue warps of both CTAs arrive (16 arrivals)
// The epilogue is the single-CTA kernel's (one row per thread, eight warps per CTA), but stores two 32-column chunks
// at a time (a 32 x 64 bf16 tile per TMA store: whole 128-byte lines).  No TMA multicast is used.
#include <cuda_bf16.h>

#include "epilogue.cuh"
#include "internal.h"
#include "ptx.cuh"

namespace trdq {
namespace {

constexpr int kTileM = 128;       // rows per CTA; the pair covers 256
constexpr int kTileKBytes = 128;
constexpr int kUmmaK = 32;
constexpr int kThreads = 384;
constexpr int kEpilogueThreads = 256;
constexpr int kAccStride = 256;
constexpr int kTmemCols = 512;
constexpr int kSmemBudget = 227 * 1024;

template <int BN>
struct Cfg2 {
  static constexpr int kABytes = kTileM * kTileKBytes;
  static constexpr int kBBytes = (BN / 2) * kTileKBytes;  // this CTA's half of the weight tile
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kParamBytes = 2 * BN * 12;
  static constexpr int kBarrierBytes = 256;
  static constexpr int kOutStageBytes = (kEpilogueThreads / 32) * 4096;  // one 32 x 64 bf16 tile per warp
  static constexpr int kStages = (kSmemBudget - 1024 - kOutStageBytes - kParamBytes - kBarrierBytes) / kStageBytes;
  static constexpr int kSmemBytes = 1024 + kStages * kStageBytes + kOutStageBytes + kParamBytes + kBarrierBytes;
  static_assert(kStages >= 3 && kStages <= 10, "stage count out of range");
  static_assert(kStageBytes % 1024 == 0, "stage tiles must stay 1024-byte aligned");
};

struct alignas(64) Gemm2Params {
  CUtensorMap tmap_a[2];    // codes of each segment, box 128 B x 128 rows
  CUtensorMap tmap_b;       // weights, box 128 B x BN/2 rows
  CUtensorMap tmap_out[2];     // bf16 output, box 64 x 32, 128-byte swizzle: two 32-column chunks per store
  CUtensorMap tmap_out32[2];   // box 32 x 32, 64-byte swizzle: the odd chunk of BN = 192
  const float* sx[2];
  int32_t M[2];
  int32_t pair_tiles_m[2];  // 256-row tiles per segment
  const float* sw;
  const __nv_bfloat16* bias;
  int32_t N, K, tiles_n;
  int32_t band;  // row tiles per band of the tile order; 0: column-block major over all row tiles
  uint32_t* status;
};

struct TileCoord {
  int seg, m0, n0;
};
__device__ __forceinline__ TileCoord pair_tile_coord(const Gemm2Params& p, int tile, int bn) {
  // Order of the tiles.  The clusters that run at the same time take consecutive tiles, so the order decides what they
  // share in L2: within a band of `band` row tiles the tiles go column block by column block, i.e. a wave of clusters
  // covers a band-high, many-columns-wide rectangle and re-reads few distinct panels of either operand.
  const int tiles_m = p.pair_tiles_m[0] + p.pair_tiles_m[1];
  int nt, mt;
  if (p.band <= 0) {
    nt = tile / tiles_m;
    mt = tile - nt * tiles_m;
  } else {
    const int per_band = p.band * p.tiles_n;
    const int b = tile / per_band;
    const int r = tile - b * per_band;
    const int rows = min(p.band, tiles_m - b * p.band);
    nt = r / rows;
    mt = b * p.band + (r - nt * rows);
  }
  TileCoord c;
  c.seg = mt >= p.pair_tiles_m[0] ? 1 : 0;
  if (c.seg) mt -= p.pair_tiles_m[0];
  c.m0 = mt * 2 * kTileM;
  c.n0 = nt * bn;
  return c;
}

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_remote_arrive(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void mbar_remote_arrive_expect_tx(uint32_t cluster_addr, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%0], %1;" ::"r"(cluster_addr), "r"(bytes) : "memory");
}
// TMA load into THIS CTA's shared memory whose completion is counted on a barrier that may live in the peer CTA.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst_smem, const void* tmap, int32_t x, int32_t y, uint32_t bar_cluster_addr) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst_smem), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(bar_cluster_addr), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_i8_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t"
      ".reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t"
      "}\n" ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrives on the barrier at this shared-memory offset in BOTH CTAs once the MMAs issued so far are done.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
               "h"(static_cast<uint16_t>(3))
               : "memory");
}
// kind::i8 instruction descriptor for the pair: M = 256.
__host__ __device__ constexpr uint32_t umma_idesc_s8_pair(int n) {
  return (2u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(256 >> 4) << 24);
}

// ACT: GELU (tanh form) on the dequantized value before the bf16 rounding.
template <int BN, bool ACT>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1) gemm_w8a8_pair_kernel(const __grid_constant__ Gemm2Params p) {
  using C = Cfg2<BN>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t out_stage_base = smem_base + C::kStages * C::kStageBytes;
  float2* param_buf = reinterpret_cast<float2*>(smem + C::kStages * C::kStageBytes + C::kOutStageBytes);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::kStages * C::kStageBytes + C::kOutStageBytes + C::kParamBytes);
  const uint32_t bar_full = smem_u32(bars);                  // [S]   used in the leader
  const uint32_t bar_empty = bar_full + 8 * C::kStages;      // [S]   each CTA's own
  const uint32_t bar_tfull = bar_empty + 8 * C::kStages;     // [2]   each CTA's own
  const uint32_t bar_tempty = bar_tfull + 16;                // [2]   used in the leader
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * C::kStages + 4);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  const int cluster_id = blockIdx.x >> 1;
  const int num_clusters = gridDim.x >> 1;
  const int total_tiles = (p.pair_tiles_m[0] + p.pair_tiles_m[1]) * p.tiles_n;
  const int num_kb = p.K / kTileKBytes;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(bar_full + 8 * s, 2);   // one arrive.expect_tx from each CTA's producer
      mbar_init(bar_empty + 8 * s, 1);  // one multicast commit
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_tfull + 8 * a, 1);
      mbar_init(bar_tempty + 8 * a, 2 * (kEpilogueThreads / 32));  // epilogue warps of both CTAs
    }
    fence_mbar_init();
  }
  if (warp == 2) {
    tmem_alloc_pair(smem_u32(tmem_slot), kTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // the peer's barriers are initialised and its tensor memory allocated before anything is signalled
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  if (threadIdx.x == 0) {  // descriptors are kernel arguments: fetch them while the previous kernel may still be running
    prefetch_tensormap(&p.tmap_a[0]);
    prefetch_tensormap(&p.tmap_a[1]);
    prefetch_tensormap(&p.tmap_b);
    prefetch_tensormap(&p.tmap_out[0]);
    prefetch_tensormap(&p.tmap_out[1]);
    if ((BN / 64) % 2) {
      prefetch_tensormap(&p.tmap_out32[0]);
      prefetch_tensormap(&p.tmap_out32[1]);
    }
  }
  griddep_launch_dependents();
  // The weights are constants of the prepared object, so the weight halves of the first tile's first stages are requested
  // before waiting for the kernel before (which produced the activation codes): their latency overlaps its tail.
  // RULE this relies on: griddepcontrol.wait orders this kernel only against its immediate predecessor in the stream, so
  // the weight codes must be complete before that predecessor can start.  trdq_prepare_weights guarantees it: the last
  // kernel it enqueues per group (column sums / 4-bit multipliers, or a stream synchronisation for dense rotations) is
  // launched the ordinary way, i.e. with a full dependency on the kernels that wrote the codes, and never triggers its
  // dependents early.
  const int prefetched = cluster_id < total_tiles ? min(C::kStages, num_kb) : 0;
  if (threadIdx.x == 0) {
    const uint32_t leader_full0 = map_to_cta(bar_full, 0);
    const TileCoord tc0 = pair_tile_coord(p, cluster_id < total_tiles ? cluster_id : 0, BN);
    for (int kb = 0; kb < prefetched; ++kb) {
      const uint32_t full_s = leader_full0 + 8 * kb;
      mbar_remote_arrive_expect_tx(full_s, C::kStageBytes);  // this CTA's whole stage; the activation half follows below
      tma_load_2d_pair(smem_base + kb * C::kStageBytes + C::kABytes, &p.tmap_b, kb * kTileKBytes, tc0.n0 + rank * (BN / 2), full_s);
    }
  }
  griddep_wait();

  if (warp == 0) {
    // ---------------------------------------------------- TMA producer (both CTAs)
    if (elect_one()) {
      BoundedWaiter w(p.status, kStatusTimeoutProducer);
      const uint32_t leader_full = map_to_cta(bar_full, 0);
      int stage = 0;
      uint32_t phase = 0;
      for (int tile = cluster_id; tile < total_tiles; tile += num_clusters) {
        const TileCoord tc = pair_tile_coord(p, tile, BN);
        for (int kb = 0; kb < num_kb; ++kb) {
          w.wait(bar_empty + 8 * stage, phase ^ 1);
          const uint32_t a_dst = smem_base + stage * C::kStageBytes;
          const uint32_t b_dst = a_dst + C::kABytes;
          const uint32_t full_s = leader_full + 8 * stage;
          const bool b_in_flight = tile == cluster_id && kb < prefetched;
          if (!b_in_flight) mbar_remote_arrive_expect_tx(full_s, C::kStageBytes);
          tma_load_2d_pair(a_dst, &p.tmap_a[tc.seg], kb * kTileKBytes, tc.m0 + rank * kTileM, full_s);
          if (!b_in_flight) tma_load_2d_pair(b_dst, &p.tmap_b, kb * kTileKBytes, tc.n0 + rank * (BN / 2), full_s);
          if (++stage == C::kStages) {
            stage = 0;
            phase ^= 1;
          }
        }
      }
      w.settle();
    }
  } else if (warp == 1) {
    // ---------------------------------------------------- MMA issuer (leader only)
    if (leader && elect_one()) {
      BoundedWaiter w(p.status, kStatusTimeoutMma);
      constexpr uint32_t idesc = umma_idesc_s8_pair(BN);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      for (int tile = cluster_id; tile < total_tiles; tile += num_clusters) {
        w.wait(bar_tempty + 8 * acc, acc_phase ^ 1);
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * kAccStride;
        for (int kb = 0; kb < num_kb; ++kb) {
          w.wait(bar_full + 8 * stage, phase);
          tc_fence_after();
          const uint32_t a_addr = smem_base + stage * C::kStageBytes;
          const uint64_t a_desc = umma_desc_k_sw128(a_addr);
          const uint64_t b_desc = umma_desc_k_sw128(a_addr + C::kABytes);
#pragma unroll
          for (int k = 0; k < kTileKBytes / kUmmaK; ++k) umma_i8_pair(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
          umma_commit_pair(bar_empty + 8 * stage);
          if (++stage == C::kStages) {
            stage = 0;
            phase ^= 1;
          }
        }
        umma_commit_pair(bar_tfull + 8 * acc);
        if (++acc == 2) {
          acc = 0;
          acc_phase ^= 1;
        }
      }
      w.settle();
    }
  } else if (warp >= 4) {
    // ---------------------------------------------------- epilogue (both CTAs, own 128 rows)
    const int ew = warp - 4;
    const int q = ew & 3;
    const int half = ew >> 2;
    const int et = threadIdx.x - 4 * 32;
    constexpr int kChunksPerWarp = BN / 64;
    const uint32_t my_stage = out_stage_base + ew * 4096;
    const uint32_t leader_tempty = map_to_cta(bar_tempty, 0);
    BoundedWaiter w(p.status, kStatusTimeoutEpilogue);
    int acc = 0;
    uint32_t acc_phase = 0;
    for (int tile = cluster_id; tile < total_tiles; tile += num_clusters) {
      const TileCoord tc = pair_tile_coord(p, tile, BN);
      const int m0 = tc.m0 + rank * kTileM;
      float2* pb = param_buf + acc * BN;
      float* thr = reinterpret_cast<float*>(param_buf + 2 * BN) + acc * BN;
      stage_column_params(pb, thr, p.sw, p.bias, tc.n0, p.N, BN, et, kEpilogueThreads);
      asm volatile("bar.sync 1, %0;" ::"n"(kEpilogueThreads) : "memory");
      const int row = m0 + q * 32 + lane;
      const float sxm = row < p.M[tc.seg] ? __ldg(p.sx[tc.seg] + row) : 0.0f;

      w.wait(bar_tfull + 8 * acc, acc_phase);
      __syncwarp();
      tc_fence_after();
      const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * kAccStride;
      // two 32-column chunks per store: a 32 x 64 bf16 tile (128-byte rows, 128-byte swizzle), full lines on the way out
#pragma unroll 1
      for (int cc = 0; cc + 1 < kChunksPerWarp; cc += 2) {
        const int c = half * kChunksPerWarp + cc;
#pragma unroll
        for (int h2 = 0; h2 < 2; ++h2) {
          uint32_t r[32];
          tmem_ld_32x32(t_row + (c + h2) * 32, r);
          tmem_wait_ld();
          uint32_t packed[16];
          dequant_row32<ACT>(r, sxm, reinterpret_cast<const float4*>(pb + (c + h2) * 32), reinterpret_cast<const float4*>(thr + (c + h2) * 32),
                             packed);
          if (h2 == 0) {
            if (lane == 0) bulk_wait_group_read<0>();  // the previous store has finished reading the tile
            __syncwarp();
          }
#pragma unroll
          for (int v = 0; v < 4; ++v)
            st_shared_v4(my_stage + lane * 128 + (((4 * h2 + v) ^ (lane & 7)) << 4), packed[4 * v], packed[4 * v + 1], packed[4 * v + 2],
                         packed[4 * v + 3]);
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          tma_store_2d(&p.tmap_out[tc.seg], tc.n0 + c * 32, m0 + q * 32, my_stage);  // rows >= M and columns >= N are clipped
          bulk_commit_group();
        }
      }
      if (kChunksPerWarp % 2) {
        // the odd chunk (BN = 192): a 32 x 32 tile, 64-byte rows, chunk v stored at v ^ ((lane >> 1) & 3)
        const int c = half * kChunksPerWarp + kChunksPerWarp - 1;
        uint32_t r[32];
        tmem_ld_32x32(t_row + c * 32, r);
        tmem_wait_ld();
        uint32_t packed[16];
        dequant_row32<ACT>(r, sxm, reinterpret_cast<const float4*>(pb + c * 32), reinterpret_cast<const float4*>(thr + c * 32), packed);
        if (lane == 0) bulk_wait_group_read<0>();
        __syncwarp();
#pragma unroll
        for (int v = 0; v < 4; ++v)
          st_shared_v4(my_stage + lane * 64 + ((v ^ ((lane >> 1) & 3)) << 4), packed[4 * v], packed[4 * v + 1], packed[4 * v + 2],
                       packed[4 * v + 3]);
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          tma_store_2d(&p.tmap_out32[tc.seg], tc.n0 + c * 32, m0 + q * 32, my_stage);
          bulk_commit_group();
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_remote_arrive(leader_tempty + 8 * acc);
      if (++acc == 2) {
        acc = 0;
        acc_phase ^= 1;
      }
    }
    if (lane == 0) bulk_wait_group_read<0>();  // the staging tiles have been read; the stores complete before the grid does
    w.settle();
  }

  // Neither CTA may release its shared or tensor memory while the other's MMAs or copies can still touch it.
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 2) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

template <int BN, bool ACT>
cudaError_t launch_pair(const Gemm2Params& p, int clusters, cudaStream_t stream) {
  using C = Cfg2<BN>;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * clusters);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = C::kSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, gemm_w8a8_pair_kernel<BN, ACT>, p);
}

// Clusters of two CTAs that can be resident at once (at most SMs / 2; fewer if a GPC has an odd SM count).
template <int BN>
int max_clusters(int dev) {
  static PerDevice<int> cached;
  if (dev < 0 || dev >= kMaxDevices) return 0;
  int known = cached.get(dev);
  if (known == 0) {
    using C = Cfg2<BN>;
    if (cudaFuncSetAttribute(gemm_w8a8_pair_kernel<BN, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes) != cudaSuccess ||
        cudaFuncSetAttribute(gemm_w8a8_pair_kernel<BN, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes) != cudaSuccess) {
      cudaGetLastError();
      cached.set(dev, -1);
      return 0;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = C::kSmemBytes;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, gemm_w8a8_pair_kernel<BN, false>, &cfg) != cudaSuccess || n <= 0) {
      cudaGetLastError();
      cached.set(dev, -1);
      return 0;
    }
    known = n;
    cached.set(dev, n);
  }
  return known > 0 ? known : 0;
}

// Tile width: waves of resident clusters times the time of one tile.  The kernel is bound by operand delivery from L2,
// so a tile costs what it loads, (256 + BN) panel rows of K bytes; wider tiles load less per multiply-add.  Checked
// against a sweep of all three widths over the layer shapes at M = 4096 ... 32768 with the banded tile order: the model
// picks the fastest width or one within 2 % of it (the earlier model, waves x (BN + 24), left 4 - 15 % on the table at
// M >= 16384; without the ragged-tile factor N = 1152 got width 256 where 192 is 2 - 3 % faster).
// Returns the index into kTileN (and the resident clusters of that width), or -1 if the kernel cannot run here.
int pair_tile_choice(int64_t tiles_m, int N, int dev, int* clusters_out) {
  int best = -1;
  double best_cost = 1e300;
  int clusters_of[kNumTileN];
  for (int i = 0; i < kNumTileN; ++i) {
    const int bn = kTileN[i];
    clusters_of[i] = bn == 128 ? max_clusters<128>(dev) : bn == 192 ? max_clusters<192>(dev) : max_clusters<256>(dev);
    if (clusters_of[i] <= 0) continue;
    const int64_t tiles_n = (N + bn - 1) / bn;
    const int64_t tiles = tiles_m * tiles_n;
    // whole waves while there are few of them; with four or more the persistent clusters even a partial wave out
    const double waves = tiles >= 4ll * clusters_of[i] ? static_cast<double>(tiles) / clusters_of[i]
                                                       : static_cast<double>((tiles + clusters_of[i] - 1) / clusters_of[i]);
    // a ragged last column tile loads and multiplies columns that do not exist (N = 1152 in tiles of 256: 11 %)
    const double cost = waves * (256.0 + bn) * (static_cast<double>(tiles_n * bn) / N);
    if (cost < best_cost) {
      best_cost = cost;
      best = i;
    }
  }
  if (best >= 0 && clusters_out) *clusters_out = clusters_of[best];
  return best;
}

// ---------------------------------------------------------------------------------------------
// Measurement aid: the tensor pipe by itself.  Every CTA pair issues `mmas` tcgen05.mma (256 x 256 x 32, int8) on
// operands that already sit in shared memory, so there is no load and no epilogue: the rate this kernel reaches is the
// ceiling any GEMM built on the instruction can approach on the device at its current clocks.
// ---------------------------------------------------------------------------------------------
constexpr int kCeilingThreads = 128;
constexpr int kCeilingSmemBytes = 1024 + 2 * kTileM * kTileKBytes + 64;

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kCeilingThreads, 1) mma_ceiling_kernel(int mmas, uint32_t* status) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + 2 * kTileM * kTileKBytes);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2);
  const uint32_t bar_done = smem_u32(bars);
  const int warp = threadIdx.x >> 5;
  const bool leader = cluster_ctarank() == 0;
  // operands: 128 rows of A and this CTA's 128 rows of B, all ones (the layout does not matter for constant data)
  for (int i = threadIdx.x; i < 2 * kTileM * kTileKBytes / 16; i += blockDim.x)
    reinterpret_cast<uint4*>(smem)[i] = make_uint4(0x01010101u, 0x01010101u, 0x01010101u, 0x01010101u);
  if (threadIdx.x == 0) {
    mbar_init(bar_done, 1);
    fence_mbar_init();
  }
  fence_proxy_async_smem();
  if (warp == 2) {
    tmem_alloc_pair(smem_u32(tmem_slot), kTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  BoundedWaiter w(status, kStatusTimeoutMma);
  if (warp == 1 && leader && elect_one()) {
    constexpr uint32_t idesc = umma_idesc_s8_pair(256);
    const uint64_t a_desc = umma_desc_k_sw128(smem_base);
    const uint64_t b_desc = umma_desc_k_sw128(smem_base + kTileM * kTileKBytes);
    for (int i = 0; i < mmas; ++i) {
      const int k = i & 3;
      umma_i8_pair(tmem_base + ((i >> 2) & 1) * kAccStride, a_desc + 2 * k, b_desc + 2 * k, idesc, i >= 8 ? 1u : 0u);
    }
    umma_commit_pair(bar_done);
  }
  if (warp == 0) {
    w.wait(bar_done, 0);  // arrives in both CTAs once every MMA has completed
    w.settle();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 2) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

}  // namespace

int gemm_w8_pair_tile_width(int64_t tiles_m, int N) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  const int i = pair_tile_choice(tiles_m, N, dev, nullptr);
  return i < 0 ? 0 : kTileN[i];
}

trdq_status launch_mma_ceiling(int32_t mmas_per_cluster, int32_t* clusters_out, cudaStream_t stream) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return TRDQ_ERR_CUDA;
  static PerDevice<int> cached;
  int clusters = cached.get(dev);
  if (clusters == 0) {
    if (cudaFuncSetAttribute(mma_ceiling_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kCeilingSmemBytes) != cudaSuccess) return TRDQ_ERR_CUDA;
    cudaLaunchConfig_t q = {};
    q.gridDim = dim3(2);
    q.blockDim = dim3(kCeilingThreads);
    q.dynamicSmemBytes = kCeilingSmemBytes;
    // one CTA per SM, as in the GEMM (a CTA holds all 512 tensor-memory columns): never more clusters than SM pairs
    int sms = 0;
    if (cudaOccupancyMaxActiveClusters(&clusters, mma_ceiling_kernel, &q) != cudaSuccess || clusters <= 0 ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
      cudaGetLastError();
      return TRDQ_ERR_CUDA;
    }
    if (clusters > sms / 2) clusters = sms / 2;
    cached.set(dev, clusters);
  }
  uint32_t* status = device_status_word();
  if (!status) return TRDQ_ERR_CUDA;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * clusters);
  cfg.blockDim = dim3(kCeilingThreads);
  cfg.dynamicSmemBytes = kCeilingSmemBytes;
  cfg.stream = stream;
  if (cudaLaunchKernelEx(&cfg, mma_ceiling_kernel, static_cast<int>(mmas_per_cluster), status) != cudaSuccess) return TRDQ_ERR_CUDA;
  if (clusters_out) *clusters_out = clusters;
  return TRDQ_OK;
}

// Returns TRDQ_ERR_SHAPE when the pair kernel does not apply (caller falls back to the single-CTA kernel).
trdq_status launch_gemm_w8_pair(const trdq_weights* w, int g, const GemmSegment seg[2], const void* bias_bf16, cudaStream_t stream,
                                int act) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return TRDQ_ERR_CUDA;
  Gemm2Params p;
  int64_t tiles_m = 0;
  for (int s = 0; s < 2; ++s) {
    p.sx[s] = seg[s].sx;
    p.M[s] = seg[s].M;
    p.pair_tiles_m[s] = (seg[s].M + 2 * kTileM - 1) / (2 * kTileM);
    tiles_m += p.pair_tiles_m[s];
  }
  if (tiles_m == 0) return TRDQ_OK;
  int resident = 0;
  const int best = pair_tile_choice(tiles_m, w->N, dev, &resident);
  if (best < 0) return TRDQ_ERR_SHAPE;
  const int bn = kTileN[best];
  for (int s = 0; s < 2; ++s) {
    const GemmSegment& src = seg[s].M > 0 ? seg[s] : seg[1 - s];
    trdq_status st = encode_tmap_u8_sw128(&p.tmap_a[s], src.codes, static_cast<uint64_t>(w->K), static_cast<uint64_t>(src.M),
                                          static_cast<uint64_t>(w->K), kTileKBytes, kTileM);
    if (st != TRDQ_OK) return st;
    st = encode_tmap_2d(&p.tmap_out[s], src.out, 2, static_cast<uint64_t>(w->N), static_cast<uint64_t>(src.M),
                        static_cast<uint64_t>(src.ld) * 2, 64, 32, 128);
    if (st != TRDQ_OK) return st;
    st = encode_tmap_2d(&p.tmap_out32[s], src.out, 2, static_cast<uint64_t>(w->N), static_cast<uint64_t>(src.M),
                        static_cast<uint64_t>(src.ld) * 2, 32, 32, 64);
    if (st != TRDQ_OK) return st;
  }
  p.tmap_b = w->groups[g].tmap_b_half[best];
  p.sw = w->groups[g].scales;
  p.bias = static_cast<const __nv_bfloat16*>(bias_bf16);
  p.N = w->N;
  p.K = w->K;
  p.tiles_n = (w->N + bn - 1) / bn;
  // Bands of four row tiles from 32 row tiles on (measured at M = 32768: +5 % on the K = 1152 layers, +22 % on
  // 4608 -> 1152, any band height from 2 to 8 alike; at M = 4096 the plain column-block-major order is 1 % ahead).
  p.band = tiles_m >= 32 ? 4 : 0;
  p.status = device_status_word();
  if (!p.status) return TRDQ_ERR_CUDA;
  const int64_t total = tiles_m * p.tiles_n;
  const int clusters = static_cast<int>(total < resident ? total : resident);
  cudaError_t e;
  if (act)
    e = bn == 128 ? launch_pair<128, true>(p, clusters, stream) : bn == 192 ? launch_pair<192, true>(p, clusters, stream) : launch_pair<256, true>(p, clusters, stream);
  else
    e = bn == 128 ? launch_pair<128, false>(p, clusters, stream) : bn == 192 ? launch_pair<192, false>(p, clusters, stream) : launch_pair<256, false>(p, clusters, stream);
  return e == cudaSuccess ? TRDQ_OK : TRDQ_ERR_CUDA;
}

}  // namespace trdq
