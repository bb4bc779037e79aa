// Internal declarations shared by the translation units of the library (not installed).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <vector>

#include "../../include/trdq.h"

struct trdq_rotation {
  int32_t K = 0;
  int32_t num_groups = 0;
  int device = 0;
  std::vector<int32_t> t_bounds;  // host [G+1]
  float* act_vec = nullptr;       // dev [G][K]: d * Delta * 2^-3.5
  float* weight_vec = nullptr;    // dev [G][K]: d / Delta * 2^-3.5
  // full balancing transform (Eq. 9) only; perm == nullptr means the single-rotation path
  int32_t* perm = nullptr;        // dev [G][K]: (v P)[j] = v[perm[j]]
  float* vec2 = nullptr;          // dev [G][K]: d2 * 2^-3.5, scaling before the second rotation
  // dense block rotations (Eq. 6-8) only; dense == nullptr means a Hadamard path
  uint16_t* dense = nullptr;      // dev bf16 [G][K/128][128 j][128 i]: S_b[i][j] = bf16(Delta_i R_b[i][j]), stored transposed
  double* dense_inv_t = nullptr;  // dev [G][K/128][128 i][128 j] = (S_b^-1)[j][i], for the weight side
  CUtensorMap tmap_dense;         // `dense` as a [G * K/128 * 128, 128] bf16 matrix, box 64 x 128, 128-byte swizzle
};

namespace trdq {

// Candidate accumulator tile widths of the GEMM (columns of Y per CTA tile).
constexpr int kNumTileN = 3;
constexpr int kTileN[kNumTileN] = {128, 192, 256};

struct GroupWeights {
  void* codes = nullptr;                // dev int8 [N,K] or packed uint8 [N,K/2]
  float* scales = nullptr;              // dev fp32 [N] or [N,K/128]
  CUtensorMap tmap_b[kNumTileN];        // TMA descriptors of `codes`, one per tile width (4-bit: only [0], 128 rows x 64 bytes)
  CUtensorMap tmap_b_half[kNumTileN];   // 8-bit only: boxes of half a tile width (64 / 96 / 128 rows) for the CTA-pair kernel
  // 4-bit weights only: the scales of an output channel as integers on a common power-of-two grid,
  //   scales[n][kg] = mult_t[kg][n] * base[n]   (exact whenever the exponents of a channel span < 7 bits)
  int32_t* colsum = nullptr;            // 8-bit only: dev int32 [N], sum over k of the codes (for asymmetric activations)
  int32_t* mult_t = nullptr;            // dev int32 [K/128][n_pad], n_pad = N rounded up to 128
  float* base = nullptr;                // dev fp32 [n_pad], a power of two (already divided by 16, see gemm_w4a8.cu)
};

}  // namespace trdq

struct trdq_weights {
  int32_t N = 0, K = 0, wbits = 8, num_groups = 0;
  int device = 0;
  std::vector<int32_t> t_bounds;
  std::vector<trdq::GroupWeights> groups;
};

namespace trdq {

// Per-device memo for set-up done by the first call on a device (kernel attributes, symbol addresses, occupancy
// queries).  Several host threads may make that first call at once: repeating the set-up is harmless, a torn
// read of the memo is not, hence the atomics.  A zero value means "not done yet".
constexpr int kMaxDevices = 64;
template <typename T>
struct PerDevice {
  std::atomic<T> slot[kMaxDevices];
  T get(int dev) const { return dev >= 0 && dev < kMaxDevices ? slot[dev].load(std::memory_order_acquire) : T(); }
  void set(int dev, T v) {
    if (dev >= 0 && dev < kMaxDevices) slot[dev].store(v, std::memory_order_release);
  }
};
using PerDeviceFlag = PerDevice<bool>;

// TRDQ_DEBUG=1: waits for the call's own work and turns a device error or an expired wait into the call's return code.
trdq_status finish(trdq_status st, void* stream);

uint32_t* device_status_word();  // device address of the status word of the current device (nullptr on failure)

// rotate_quantize.cu
// mode 0: per-row int8 codes + fp32 scale per row; mode 1: per-128-block int4 codes packed + scale per block
cudaError_t launch_rotate_quantize(const void* x_bf16, int64_t ldx, int32_t M, int32_t K, const float* vec, int mode,
                                   void* codes, float* scales, cudaStream_t stream);

cudaError_t launch_rotate2_quantize(const void* x_bf16, int64_t ldx, int32_t M, int32_t K, const float* vec1, const int32_t* perm,
                                    const float* vec2, int mode, void* codes, float* scales, cudaStream_t stream);

// rotate_quantize_team.cu: per-row int8 path, TMA-staged, one thread per block, independent teams of warps per CTA
bool rotate_quantize_prefers_team(int32_t M, int32_t K);
trdq_status launch_rotate_quantize_team(const void* x_bf16, int64_t ldx, int32_t M, int32_t K, const float* vec, int8_t* codes,
                                        float* scales, cudaStream_t stream);

// norm_rotate_quantize.cu: LayerNorm + per-sample modulation in front of the rotation (K <= 8192)
cudaError_t launch_norm_rotate_quantize(const void* x_bf16, int64_t ldx, int32_t M, int32_t K, const float* vec, const void* shift_bf16,
                                        const void* scale_bf16, int32_t rows_per_sample, float eps, int8_t* codes, float* scales,
                                        cudaStream_t stream);

// rotate_dense.cu: dense block rotation on the tensor cores + per-token quantizer (two passes over X)
uint64_t rotate_dense_workspace_bytes(int32_t M, int32_t K);
trdq_status launch_rotate_dense_quantize(const trdq_rotation* rot, int g, const void* x_bf16, int64_t ldx, int32_t M, int8_t* codes,
                                         float* scales, float* workspace, cudaStream_t stream);
// weight side: wr = W S^-1 (fp64 sums, one fp32 rounding) into wr_scratch [N,K], then the 8- or 4-bit quantizer
cudaError_t launch_dense_prepare(const void* w_bf16, int32_t N, int32_t K, const double* inv_t, int wbits, float* wr_scratch,
                                 void* codes, float* scales, cudaStream_t stream);

// gemm_i8.cu
struct GemmSegment {
  const int8_t* codes;  // dev [M,K]
  const float* sx;      // dev [M]
  void* out;            // dev bf16 [M,ld] (or int32 [M,ld] for the raw mode)
  int64_t ld;
  int32_t M;
};
// act: 0 = none, 1 = GELU (tanh form) applied to the dequantized value before the bf16 rounding
trdq_status launch_gemm_w8(const trdq_weights* w, int g, const GemmSegment seg[2], const void* bias_bf16, bool raw_i32,
                           cudaStream_t stream, int act = 0);
trdq_status launch_gemm_w4(const trdq_weights* w, int g, const GemmSegment seg[2], const void* bias_bf16,
                           cudaStream_t stream, int act = 0);
trdq_status launch_gemm_w8_asym(const trdq_weights* w, int g, const GemmSegment seg[2], const int32_t* const zp[2],
                                const void* bias_bf16, cudaStream_t stream);
cudaError_t launch_weight_colsum(const int8_t* codes, int32_t N, int32_t K, int32_t* colsum, cudaStream_t stream);
cudaError_t launch_rotate_quantize_asym(const void* x_bf16, int64_t ldx, int32_t M, int32_t K, const float* vec, uint8_t* codes,
                                        float* scales, int32_t* zero_points, cudaStream_t stream);
// split-K (8-bit weights, one segment): partial int32 sums in `workspace` (splits * M * N), then reduce + epilogue
int splitk_choose(const trdq_weights* w, int32_t M);
trdq_status launch_gemm_w8_splitk(const trdq_weights* w, int g, const GemmSegment& seg, const void* bias_bf16, int splits,
                                  int32_t* workspace, cudaStream_t stream);
trdq_status launch_gemm_w8_splitk_static(const trdq_weights* w, int g, const GemmSegment& seg, const void* bias_bf16, int splits,
                                         cudaStream_t stream);
// which kernel a call would run (for reports; the launchers use the same functions)
void describe_rotate_quantize_kernel(int32_t M, int32_t K, char* name, size_t cap);
void describe_gemm_kernel(int32_t M, int32_t K, int32_t N, int32_t wbits, char* name, size_t cap);
int gemm_w8_pair_tile_width(int64_t pair_tiles_m, int N);  // 0: the pair kernel cannot run on this device
// measurement aid: `mmas_per_cluster` back-to-back 256 x 256 x 32 int8 MMAs per CTA pair on resident operands
trdq_status launch_mma_ceiling(int32_t mmas_per_cluster, int32_t* clusters_out, cudaStream_t stream);
// gemm_i8_2cta.cu: CTA-pair kernel; TRDQ_ERR_SHAPE means "not applicable here, use the single-CTA kernel"
trdq_status launch_gemm_w8_pair(const trdq_weights* w, int g, const GemmSegment seg[2], const void* bias_bf16,
                                cudaStream_t stream, int act = 0);
cudaError_t launch_w4_multipliers(const float* scales, int32_t N, int32_t groups, int32_t n_pad, int32_t* mult_t, float* base,
                                  cudaStream_t stream);

// tensor maps (driver entry point fetched through the runtime; no link-time libcuda dependency)
// 2-D uint8 row-major [rows, row_bytes-wide], box = 128 bytes x box_rows, 128-byte swizzle.
trdq_status encode_tmap_u8_sw128(CUtensorMap* out, const void* base, uint64_t row_bytes, uint64_t rows,
                                 uint64_t row_stride_bytes, uint32_t box_bytes, uint32_t box_rows);
// General 2-D row-major map: `cols` elements of `elem_bytes` (1, 2 or 4) per row, box = box_cols x box_rows,
// swizzle_bytes in {0, 32, 64, 128}.
trdq_status encode_tmap_2d(CUtensorMap* out, const void* base, uint32_t elem_bytes, uint64_t cols, uint64_t rows,
                           uint64_t row_stride_bytes, uint32_t box_cols, uint32_t box_rows, uint32_t swizzle_bytes);

// A row-major [rows, boxes * box_cols] matrix viewed as (column in box, row, box): one copy of
// box_cols x box_rows x boxes moves a tile of box_rows full rows and stores it box after box, each box
// being box_rows rows of box_cols elements (128 bytes), 128-byte swizzle.
trdq_status encode_tmap_boxes(CUtensorMap* out, const void* base, uint32_t elem_bytes, uint32_t box_cols, uint64_t rows,
                              uint64_t row_stride_bytes, uint32_t boxes, uint32_t box_rows);

// Tile height for the row kernels that run two CTAs per SM over tiles of whole rows: the CTAs work through the tiles
// in rounds, a round costs about (rows + 2) row-times, and slightly smaller tiles can fill the last round
// (M = 4096, K = 1152: 7 rows give 586 tiles = 1.98 rounds of 296 CTAs, 8 rows give 1.73 rounds that cost 2).
inline int rows_per_tile_by_rounds(int32_t M, int rows_max, int sms) {
  int rows = rows_max;
  long best_cost = -1;
  for (int cand = rows_max; cand >= (rows_max + 1) / 2; --cand) {
    const long tiles = (M + cand - 1) / cand;
    const long rounds = (tiles + 2 * sms - 1) / (2 * sms);
    const long cost = rounds * (cand + 2);
    if (best_cost < 0 || cost < best_cost) {
      best_cost = cost;
      rows = cand;
    }
  }
  return rows;
}

// Launches `kernel` so that its prologue may overlap the tail of the previous kernel in the stream
// (the kernel itself orders its memory accesses with griddep_wait()).
template <typename... KArgs, typename... Args>
cudaError_t launch_overlapped(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

}  // namespace trdq
