// W4A8 variant of the integer GEMM: int8 activation codes against int4 weight codes that carry one
// fp32 scale per (output channel, 128 consecutive k):
//     y[m, n] = sx[m] * sum_kg sw4[n, kg] * ( sum_{k in kg} q[m, k] * q4[n, k] ) + bias[n]
//
// The k-block of the pipeline is exactly one scale group.  Per k-block:
//   warp 0       TMA: 128 x 128-byte tile of activation codes and 128 x 64-byte tile of packed nibbles
//   warps 2-3    unpack in registers: 16 bytes of nibbles -> 32 int8 (nibble << 4, i.e. 16 * q4, which is
//                sign-correct without any sign extension) written in the 128-byte-swizzled K-major
//                layout the tensor core reads
//   warp 1       four tcgen05.mma kind::i8 (128 x 128 x 32) into a FRESH tensor-memory accumulator
//                (four accumulators of 128 columns rotate)
//   warps 4-11   drain that accumulator: acc64[n] += acc32[n] * mult[kg][n] with 64-bit integer
//                multiply-adds.  mult are the group scales of a channel on a common power-of-two grid
//                (sw4[n,kg] = mult[kg][n] * base[n]), so the sum over groups is EXACT integer arithmetic
//                and no cancellation between groups can lose bits.
// At the end of a tile the 64-bit sums are converted once: y = fma(float(S), sx * base[n], bias[n]),
// with the same cancellation check against the bias as the 8-bit kernel, staged in shared memory and
// written by TMA stores.  Every wait is bounded.
#include <cuda_bf16.h>

#include "epilogue.cuh"
#include "internal.h"
#include "ptx.cuh"

namespace trdq {
namespace {

constexpr int kTileM = 128;
constexpr int kTileNW4 = 128;
constexpr int kTileK = 128;
constexpr int kThreads = 384;
constexpr int kEpilogueThreads = 256;
constexpr int kUnpackThreads = 64;
constexpr int kAccStages = 4;
constexpr int kTmemCols = 512;
constexpr int kABytes = kTileM * kTileK;       // 16 KB int8
constexpr int kBPackedBytes = kTileNW4 * 64;     // 8 KB nibbles
constexpr int kB8Bytes = kTileNW4 * kTileK;      // 16 KB int8 after unpacking
constexpr int kStageBytes = kABytes + kB8Bytes + kBPackedBytes;  // A and B8 first: both need 1024-byte alignment
constexpr int kStages = 4;
constexpr int kOutStageBytes = (kEpilogueThreads / 32) * 2048;
constexpr int kParamBytes = kTileNW4 * 12;
constexpr int kBarrierBytes = 256;
constexpr int kFixedSmemBytes = 1024 + kStages * kStageBytes + kOutStageBytes + kParamBytes + kBarrierBytes;
// The tile's multipliers ([K/128][128] int32) are staged in shared memory when they fit.
constexpr int kMaxSmemGroups = (227 * 1024 - kFixedSmemBytes) / (kTileNW4 * 4);

struct alignas(64) W4Params {
  CUtensorMap tmap_a[2];
  CUtensorMap tmap_b;
  CUtensorMap tmap_out[2];
  const float* sx[2];
  int32_t M[2];
  int32_t tiles_m[2];
  const int32_t* mult_t;  // [K/128][n_pad]
  const float* base;      // [n_pad]
  const __nv_bfloat16* bias;
  int32_t N, K, tiles_n, n_pad;
  int32_t mult_in_smem;  // 1: all K/128 multiplier rows of a tile fit the shared-memory table
  uint32_t* status;
};

struct TileCoord {
  int seg, m0, n0;
};
__device__ __forceinline__ TileCoord tile_coord(const W4Params& p, int tile) {
  const int tiles_m = p.tiles_m[0] + p.tiles_m[1];
  const int nt = tile / tiles_m;
  int mt = tile - nt * tiles_m;
  TileCoord c;
  c.seg = mt >= p.tiles_m[0] ? 1 : 0;
  if (c.seg) mt -= p.tiles_m[0];
  c.m0 = mt * kTileM;
  c.n0 = nt * kTileNW4;
  return c;
}

// ACT: GELU (tanh form) on the dequantized value before the bf16 rounding.
template <bool ACT>
__global__ void __launch_bounds__(kThreads, 1) gemm_w4a8_kernel(const __grid_constant__ W4Params p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t out_stage_base = smem_base + kStages * kStageBytes;
  float2* param_buf = reinterpret_cast<float2*>(smem + kStages * kStageBytes + kOutStageBytes);  // (base, bias)[128]
  float* thr_buf = reinterpret_cast<float*>(param_buf + kTileNW4);                                 // 2^-10 |bias|
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes + kOutStageBytes + kParamBytes);
  // barriers: raw[S] (TMA landed), b8[S] (unpacked), empty[S], tfull[4], tempty[4]
  const uint32_t bar_raw = smem_u32(bars);
  const uint32_t bar_b8 = bar_raw + 8 * kStages;
  const uint32_t bar_empty = bar_b8 + 8 * kStages;
  const uint32_t bar_tfull = bar_empty + 8 * kStages;
  const uint32_t bar_tempty = bar_tfull + 8 * kAccStages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 3 * kStages + 2 * kAccStages);
  int32_t* mult_smem = reinterpret_cast<int32_t*>(smem + kStages * kStageBytes + kOutStageBytes + kParamBytes + kBarrierBytes);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int total_tiles = (p.tiles_m[0] + p.tiles_m[1]) * p.tiles_n;
  const int num_kb = p.K / kTileK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(bar_raw + 8 * s, 1);
      mbar_init(bar_b8 + 8 * s, kUnpackThreads / 32);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int a = 0; a < kAccStages; ++a) {
      mbar_init(bar_tfull + 8 * a, 1);
      mbar_init(bar_tempty + 8 * a, kEpilogueThreads / 32);
    }
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  griddep_launch_dependents();
  griddep_wait();  // codes, scales and weights may come from the kernel before; Y may still be read by it

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (elect_one()) {
      prefetch_tensormap(&p.tmap_a[0]);
      prefetch_tensormap(&p.tmap_a[1]);
      prefetch_tensormap(&p.tmap_b);
      prefetch_tensormap(&p.tmap_out[0]);
      prefetch_tensormap(&p.tmap_out[1]);
      BoundedWaiter w(p.status, kStatusTimeoutProducer);
      int stage = 0;
      uint32_t phase = 0;
      for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
        const TileCoord tc = tile_coord(p, tile);
        for (int kb = 0; kb < num_kb; ++kb) {
          w.wait(bar_empty + 8 * stage, phase ^ 1);
          const uint32_t a_dst = smem_base + stage * kStageBytes;
          const uint32_t bp_dst = a_dst + kABytes + kB8Bytes;
          mbar_arrive_expect_tx(bar_raw + 8 * stage, kABytes + kBPackedBytes);
          tma_load_2d(a_dst, &p.tmap_a[tc.seg], kb * kTileK, tc.m0, bar_raw + 8 * stage);
          tma_load_2d(bp_dst, &p.tmap_b, kb * (kTileK / 2), tc.n0, bar_raw + 8 * stage);
          if (++stage == kStages) {
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
      constexpr uint32_t idesc = umma_idesc_s8(kTileNW4);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
        for (int kb = 0; kb < num_kb; ++kb) {
          w.wait(bar_tempty + 8 * acc, acc_phase ^ 1);  // accumulator drained
          w.wait(bar_b8 + 8 * stage, phase);            // A landed and B unpacked
          tc_fence_after();
          const uint32_t a_addr = smem_base + stage * kStageBytes;
          const uint64_t a_desc = umma_desc_k_sw128(a_addr);
          const uint64_t b_desc = umma_desc_k_sw128(a_addr + kABytes);
          const uint32_t d_tmem = tmem_base + acc * kTileNW4;
#pragma unroll
          for (int k = 0; k < kTileK / 32; ++k) umma_i8(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, k != 0 ? 1u : 0u);
          umma_commit(bar_empty + 8 * stage);
          umma_commit(bar_tfull + 8 * acc);
          if (++stage == kStages) {
            stage = 0;
            phase ^= 1;
          }
          if (++acc == kAccStages) {
            acc = 0;
            acc_phase ^= 1;
          }
        }
      }
      w.settle();
    }
  } else if (warp == 2 || warp == 3) {
    // ------------------------------------------------- unpack nibbles -> int8
    const int ut = threadIdx.x - 64;  // 0..63
    BoundedWaiter w(p.status, kStatusTimeoutUnpack);
    int stage = 0;
    uint32_t phase = 0;
    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
      for (int kb = 0; kb < num_kb; ++kb) {
        w.wait(bar_raw + 8 * stage, phase);
        __syncwarp();
        const uint8_t* bp = smem + stage * kStageBytes + kABytes + kB8Bytes;
        const uint32_t b8 = smem_base + stage * kStageBytes + kABytes;
#pragma unroll
        for (int i = 0; i < (kTileNW4 * 4) / kUnpackThreads; ++i) {
          const int id = ut + kUnpackThreads * i;  // 16-byte source chunk: row = id / 4, chunk = id % 4
          const int row = id >> 2, sc = id & 3;
          const uint4 src = *reinterpret_cast<const uint4*>(bp + row * 64 + sc * 16);
          const uint32_t wsrc[4] = {src.x, src.y, src.z, src.w};
          uint32_t o[8];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint32_t even = (wsrc[j] << 4) & 0xF0F0F0F0u;  // k even: low nibble moved to the high half
            const uint32_t odd = wsrc[j] & 0xF0F0F0F0u;          // k odd: already in the high half
            o[2 * j] = __byte_perm(even, odd, 0x5140);
            o[2 * j + 1] = __byte_perm(even, odd, 0x7362);
          }
          const uint32_t dst_row = b8 + row * 128;
          st_shared_v4(dst_row + (((2 * sc) ^ (row & 7)) << 4), o[0], o[1], o[2], o[3]);
          st_shared_v4(dst_row + (((2 * sc + 1) ^ (row & 7)) << 4), o[4], o[5], o[6], o[7]);
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_b8 + 8 * stage);
        if (++stage == kStages) {
          stage = 0;
          phase ^= 1;
        }
      }
    }
    w.settle();
  } else {
    // ---------------------------------------------------------------- epilogue
    const int ew = warp - 4;
    const int q = ew & 3;
    const int half = ew >> 2;
    const int et = threadIdx.x - 4 * 32;
    const uint32_t my_stage = out_stage_base + ew * 2048;
    BoundedWaiter w(p.status, kStatusTimeoutEpilogue);
    int acc = 0;
    uint32_t acc_phase = 0;
    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
      const TileCoord tc = tile_coord(p, tile);
      // all epilogue threads are past the previous tile's parameter reads before these writes
      asm volatile("bar.sync 1, %0;" ::"n"(kEpilogueThreads) : "memory");
      for (int c = et; c < kTileNW4; c += kEpilogueThreads) {
        const int n = tc.n0 + c;
        float2 v = make_float2(0.0f, 0.0f);
        if (n < p.N) {
          v.x = __ldg(p.base + n);
          v.y = p.bias ? __bfloat162float(p.bias[n]) : 0.0f;
        }
        param_buf[c] = v;
        thr_buf[c] = fabsf(v.y) * 0.0009765625f;
      }
      if (p.mult_in_smem) {
        // this tile's multipliers for every scale group: [num_kb][128] int32
        const int4* src = reinterpret_cast<const int4*>(p.mult_t + tc.n0);
        for (int i = et; i < num_kb * (kTileNW4 / 4); i += kEpilogueThreads) {
          const int kb = i / (kTileNW4 / 4), c4 = i % (kTileNW4 / 4);
          reinterpret_cast<int4*>(mult_smem)[i] = __ldg(src + static_cast<int64_t>(kb) * (p.n_pad / 4) + c4);
        }
      }
      asm volatile("bar.sync 1, %0;" ::"n"(kEpilogueThreads) : "memory");
      const int row = tc.m0 + q * 32 + lane;
      const bool row_ok = row < p.M[tc.seg];
      const float sxm = row_ok ? __ldg(p.sx[tc.seg] + row) : 0.0f;

      long long sum[64];
#pragma unroll
      for (int j = 0; j < 64; ++j) sum[j] = 0;
      const int col0 = half * 64;
      for (int kb = 0; kb < num_kb; ++kb) {
        const int4* mrow = p.mult_in_smem ? reinterpret_cast<const int4*>(mult_smem + kb * kTileNW4 + col0)
                                          : reinterpret_cast<const int4*>(p.mult_t + static_cast<int64_t>(kb) * p.n_pad + tc.n0 + col0);
        w.wait(bar_tfull + 8 * acc, acc_phase);
        __syncwarp();
        tc_fence_after();
        const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * kTileNW4 + col0;
        // two register buffers: the load of chunk ch + 1 is in flight while chunk ch is accumulated
        uint32_t r[2][16];
        tmem_ld_32x16(t_row, r[0]);
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
          tmem_wait_ld();
          if (ch < 3) tmem_ld_32x16(t_row + (ch + 1) * 16, r[(ch + 1) & 1]);
#pragma unroll
          for (int j4 = 0; j4 < 4; ++j4) {
            const int4 m = mrow[ch * 4 + j4];
            const int mv[4] = {m.x, m.y, m.z, m.w};
#pragma unroll
            for (int e = 0; e < 4; ++e)
              sum[ch * 16 + j4 * 4 + e] +=
                  static_cast<long long>(static_cast<int32_t>(r[ch & 1][j4 * 4 + e])) * static_cast<long long>(mv[e]);
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_tempty + 8 * acc);
        if (++acc == kAccStages) {
          acc = 0;
          acc_phase ^= 1;
        }
      }

      // final conversion: y = float(S) * (sx * base) + bias   (base is a power of two: the product is exact)
#pragma unroll
      for (int c2 = 0; c2 < 2; ++c2) {
        uint32_t packed[16];
#pragma unroll
        for (int j = 0; j < 32; j += 2) {
          float y[2];
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int col = col0 + c2 * 32 + j + e;
            const float2 pb = param_buf[col];
            const long long S = sum[c2 * 32 + j + e];
            const float sf = __ll2float_rn(S);
            const float cm = __fmul_rn(sxm, pb.x);
            float v = __fmaf_rn(sf, cm, pb.y);
            if (fabsf(v) < thr_buf[col]) v = __fmaf_rn(__ll2float_rn(S - __float2ll_rz(sf)), cm, v);  // the part fp32 dropped
            y[e] = ACT ? gelu_tanh(v) : v;
          }
          const __nv_bfloat162 h = __floats2bfloat162_rn(y[0], y[1]);
          packed[j / 2] = *reinterpret_cast<const uint32_t*>(&h);
        }
        if (lane == 0) bulk_wait_group_read<0>();
        __syncwarp();
#pragma unroll
        for (int v = 0; v < 4; ++v)
          st_shared_v4(my_stage + lane * 64 + ((v ^ ((lane >> 1) & 3)) << 4), packed[4 * v], packed[4 * v + 1], packed[4 * v + 2],
                       packed[4 * v + 3]);
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          tma_store_2d(&p.tmap_out[tc.seg], tc.n0 + col0 + c2 * 32, tc.m0 + q * 32, my_stage);
          bulk_commit_group();
        }
      }
    }
    if (lane == 0) bulk_wait_group_read<0>();  // the staging tiles have been read; the stores complete before the grid does
    w.settle();
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// One thread per output channel: put the channel's group scales on a common power-of-two grid.
__global__ void w4_multipliers_kernel(const float* __restrict__ scales, int32_t N, int32_t groups, int32_t n_pad,
                                      int32_t* __restrict__ mult_t, float* __restrict__ base) {
  const int n = blockIdx.x * blockDim.x + threadIdx.x;
  if (n >= n_pad) return;
  if (n >= N) {
    for (int g = 0; g < groups; ++g) mult_t[static_cast<int64_t>(g) * n_pad + n] = 0;
    base[n] = 0.0f;
    return;
  }
  float smax = 0.0f;
  for (int g = 0; g < groups; ++g) smax = fmaxf(smax, scales[static_cast<int64_t>(n) * groups + g]);
  int e_max = 0;
  frexpf(smax, &e_max);  // smax = f * 2^e_max, f in [0.5, 1); smax == 0 gives e_max = 0
  if (e_max < -90) e_max = -90;  // keeps base a normal number; such channels are numerically zero anyway
  for (int g = 0; g < groups; ++g) {
    const float s = scales[static_cast<int64_t>(n) * groups + g];
    mult_t[static_cast<int64_t>(g) * n_pad + n] = __float2int_rn(ldexpf(s, 30 - e_max));  // < 2^30, exact if the exponents span < 7 bits
  }
  // the tensor core sees 16 * q4 (the nibble sits in the high half of the byte): fold the 1/16 here
  base[n] = ldexpf(1.0f, e_max - 30 - 4);
}

}  // namespace

cudaError_t launch_w4_multipliers(const float* scales, int32_t N, int32_t groups, int32_t n_pad, int32_t* mult_t, float* base,
                                  cudaStream_t stream) {
  w4_multipliers_kernel<<<(n_pad + 127) / 128, 128, 0, stream>>>(scales, N, groups, n_pad, mult_t, base);
  return cudaGetLastError();
}

trdq_status launch_gemm_w4(const trdq_weights* w, int g, const GemmSegment seg[2], const void* bias_bf16, cudaStream_t stream, int act) {
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) != cudaSuccess) return TRDQ_ERR_CUDA;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  W4Params p;
  int64_t tiles_m = 0;
  for (int s = 0; s < 2; ++s) {
    p.sx[s] = seg[s].sx;
    p.M[s] = seg[s].M;
    p.tiles_m[s] = (seg[s].M + kTileM - 1) / kTileM;
    tiles_m += p.tiles_m[s];
  }
  if (tiles_m == 0) return TRDQ_OK;
  for (int s = 0; s < 2; ++s) {
    const GemmSegment& src = seg[s].M > 0 ? seg[s] : seg[1 - s];
    trdq_status st = encode_tmap_u8_sw128(&p.tmap_a[s], src.codes, static_cast<uint64_t>(w->K), static_cast<uint64_t>(src.M),
                                          static_cast<uint64_t>(w->K), kTileK, kTileM);
    if (st != TRDQ_OK) return st;
    st = encode_tmap_2d(&p.tmap_out[s], src.out, 2, static_cast<uint64_t>(w->N), static_cast<uint64_t>(src.M),
                        static_cast<uint64_t>(src.ld) * 2, 32, 32, 64);
    if (st != TRDQ_OK) return st;
  }
  p.tmap_b = w->groups[g].tmap_b[0];
  p.mult_t = w->groups[g].mult_t;
  p.base = w->groups[g].base;
  p.bias = static_cast<const __nv_bfloat16*>(bias_bf16);
  p.N = w->N;
  p.K = w->K;
  p.tiles_n = (w->N + kTileNW4 - 1) / kTileNW4;
  p.n_pad = p.tiles_n * kTileNW4;
  p.status = device_status_word();
  if (!p.status) return TRDQ_ERR_CUDA;
  const int groups = w->K / kTileK;
  p.mult_in_smem = groups <= kMaxSmemGroups ? 1 : 0;
  const int smem_bytes = kFixedSmemBytes + (p.mult_in_smem ? groups * kTileNW4 * 4 : 0);
  const int64_t total = tiles_m * p.tiles_n;
  const int grid = static_cast<int>(total < sms ? total : sms);
  static PerDeviceFlag configured;
  if (!configured.get(dev)) {
    const int max_smem = kFixedSmemBytes + kMaxSmemGroups * kTileNW4 * 4;
    if (cudaFuncSetAttribute(gemm_w4a8_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem) != cudaSuccess ||
        cudaFuncSetAttribute(gemm_w4a8_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem) != cudaSuccess)
      return TRDQ_ERR_CUDA;
    configured.set(dev, true);
  }
  const cudaError_t e = act ? launch_overlapped(gemm_w4a8_kernel<true>, dim3(grid), dim3(kThreads), smem_bytes, stream, p)
                            : launch_overlapped(gemm_w4a8_kernel<false>, dim3(grid), dim3(kThreads), smem_bytes, stream, p);
  return e == cudaSuccess ? TRDQ_OK : TRDQ_ERR_CUDA;
}

}  // namespace trdq
