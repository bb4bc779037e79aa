// Host side of the C ABI: argument validation, the time-step -> group table, object
// lifetime, tensor-map encoding and the device status word.  No arithmetic of the method
// happens here except the fused per-channel vectors, which are formed once per group.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>

#include "internal.h"
#include "ptx.cuh"

namespace trdq {

// One status word per device, written by kernels whose bounded waits expire.
__device__ uint32_t g_status_word;

uint32_t* device_status_word() {
  static PerDevice<uint32_t*> cached;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  uint32_t* addr = cached.get(dev);
  if (!addr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_status_word) != cudaSuccess) return nullptr;
    addr = static_cast<uint32_t*>(p);
    cached.set(dev, addr);
  }
  return addr;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static const EncodeTiledFn fn = [] {   // initialised once, also under concurrent first calls
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess) p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// Encoded tensor maps are remembered by their full description: a caller that issues the same layer step after
// step without a CUDA graph re-describes the same buffers every call (two maps per rotate + quantize, four to six per
// GEMM), and an encode costs about a microsecond of host time.  Direct-mapped, 512 entries, one mutex; a map is a pure
// function of its key, so a stale entry cannot exist: a freed and reused address with the same shape gives the same map.
struct TmapKey {
  const void* base;
  uint64_t dims[3];
  uint64_t strides[2];
  uint32_t box[3];
  uint32_t rank, dtype, swizzle;
};
struct TmapEntry {
  bool valid = false;
  TmapKey key;
  CUtensorMap map;
};
static std::mutex g_tmap_mutex;
static TmapEntry g_tmap_cache[512];

static trdq_status encode_cached(CUtensorMap* out, CUtensorMapDataType dt, uint32_t rank, const void* base, const cuuint64_t* dims,
                                 const cuuint64_t* strides, const cuuint32_t* box, CUtensorMapSwizzle sw) {
  TmapKey key;
  std::memset(&key, 0, sizeof key);
  key.base = base;
  key.rank = rank;
  key.dtype = static_cast<uint32_t>(dt);
  key.swizzle = static_cast<uint32_t>(sw);
  for (uint32_t i = 0; i < rank; ++i) {
    key.dims[i] = dims[i];
    key.box[i] = box[i];
    if (i + 1 < rank) key.strides[i] = strides[i];
  }
  uint64_t h = 1469598103934665603ull;
  const unsigned char* kb = reinterpret_cast<const unsigned char*>(&key);
  for (size_t i = 0; i < sizeof key; ++i) h = (h ^ kb[i]) * 1099511628211ull;
  TmapEntry& slot = g_tmap_cache[h & 511u];
  {
    std::lock_guard<std::mutex> lock(g_tmap_mutex);
    if (slot.valid && std::memcmp(&slot.key, &key, sizeof key) == 0) {
      *out = slot.map;
      return TRDQ_OK;
    }
  }
  EncodeTiledFn fn = encode_fn();
  if (!fn) return TRDQ_ERR_CUDA;
  const cuuint32_t elem_strides[3] = {1, 1, 1};
  const CUresult r = fn(out, dt, rank, const_cast<void*>(base), dims, strides, box, elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return TRDQ_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_tmap_mutex);
  slot.key = key;
  slot.map = *out;
  slot.valid = true;
  return TRDQ_OK;
}

trdq_status encode_tmap_u8_sw128(CUtensorMap* out, const void* base, uint64_t row_bytes, uint64_t rows,
                                 uint64_t row_stride_bytes, uint32_t box_bytes, uint32_t box_rows) {
  const cuuint64_t dims[2] = {row_bytes, rows};
  const cuuint64_t strides[1] = {row_stride_bytes};
  const cuuint32_t box[2] = {box_bytes, box_rows};
  return encode_cached(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, base, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B);
}

trdq_status encode_tmap_2d(CUtensorMap* out, const void* base, uint32_t elem_bytes, uint64_t cols, uint64_t rows,
                           uint64_t row_stride_bytes, uint32_t box_cols, uint32_t box_rows, uint32_t swizzle_bytes) {
  const CUtensorMapDataType dt = elem_bytes == 1   ? CU_TENSOR_MAP_DATA_TYPE_UINT8
                                 : elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_UINT16
                                                   : CU_TENSOR_MAP_DATA_TYPE_UINT32;
  const CUtensorMapSwizzle sw = swizzle_bytes == 128  ? CU_TENSOR_MAP_SWIZZLE_128B
                                : swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                : swizzle_bytes == 32 ? CU_TENSOR_MAP_SWIZZLE_32B
                                                      : CU_TENSOR_MAP_SWIZZLE_NONE;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {row_stride_bytes};
  const cuuint32_t box[2] = {box_cols, box_rows};
  return encode_cached(out, dt, 2, base, dims, strides, box, sw);
}

trdq_status encode_tmap_boxes(CUtensorMap* out, const void* base, uint32_t elem_bytes, uint32_t box_cols, uint64_t rows,
                              uint64_t row_stride_bytes, uint32_t boxes, uint32_t box_rows) {
  const CUtensorMapDataType dt = elem_bytes == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_UINT16;
  const cuuint64_t dims[3] = {box_cols, rows, boxes};
  const cuuint64_t strides[2] = {row_stride_bytes, static_cast<cuuint64_t>(box_cols) * elem_bytes};
  const cuuint32_t box[3] = {box_cols, box_rows, boxes};
  return encode_cached(out, dt, 3, base, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B);
}

// TRDQ_DEBUG=1 (read once per process): every online call waits for its own work and reports what the device did with it:
// a CUDA error becomes TRDQ_ERR_CUDA at the call that caused it, an expired bounded wait TRDQ_ERR_TIMEOUT (the status word
// is read and cleared).  The stand-in for a sanitizer run: the kernels clip every access by construction (TMA boxes, row and
// column guards), so what a debug run adds is WHERE something went wrong.  Not usable while a stream is being captured.
static bool debug_mode() {
  static const bool on = [] {
    const char* e = getenv("TRDQ_DEBUG");
    return e && e[0] != '\0' && e[0] != '0';
  }();
  return on;
}
trdq_status finish(trdq_status st, void* stream) {
  if (st != TRDQ_OK || !debug_mode()) return st;
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess || cudaGetLastError() != cudaSuccess) return TRDQ_ERR_CUDA;
  return trdq_device_status(nullptr);
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static bool aligned_to(const void* p, uintptr_t bytes) { return (reinterpret_cast<uintptr_t>(p) & (bytes - 1)) == 0; }

// Objects hold device memory and tensor maps of the device they were created on; a call made with another device
// current would launch there with pointers of the first one.
static bool on_current_device(int device) {
  int cur = -1;
  return cudaGetDevice(&cur) == cudaSuccess && cur == device;
}

// Pointer, stride and alignment rules of ONE row segment of a linear call.  Every linear entry point goes through
// this function, so a bad argument is reported on the host and never reaches a kernel (which would read sx[m] as
// a float, bias[n] as bf16 and store 16-byte pieces of Y).  `raw`: int32 accumulators out, no scales.
static trdq_status check_linear_segment(const trdq_weights* w, const void* codes, const float* scales, const void* out, int64_t ld,
                                        bool raw) {
  if (!codes || !out || (!raw && !scales)) return TRDQ_ERR_NULL;
  if (ld < w->N) return TRDQ_ERR_SHAPE;
  if (ld % (raw ? 4 : 8) != 0 || !aligned16(codes) || !aligned16(out) || (!raw && !aligned_to(scales, 4))) return TRDQ_ERR_ALIGN;
  return TRDQ_OK;
}

static trdq_status check_bias(const void* bias_bf16) { return bias_bf16 && !aligned_to(bias_bf16, 2) ? TRDQ_ERR_ALIGN : TRDQ_OK; }

static int find_group(const std::vector<int32_t>& bounds, int32_t t) {
  const int G = static_cast<int>(bounds.size()) - 1;
  for (int g = 0; g < G; ++g)
    if (bounds[g] <= t && t < bounds[g + 1]) return g;
  return -1;
}

// Self-test of the bounded wait: one warp waits on a barrier that nothing ever signals.  The wait gives up
// after 20 ms, records its bit in the status word and the kernel returns normally.
__global__ void selftest_wait_expiry_kernel(uint32_t* status) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    fence_mbar_init();
  }
  __syncthreads();
  BoundedWaiter w(status, kStatusTimeoutSelfTest, 20000000ull);
  w.wait(smem_u32(&bar), 0);
}

}  // namespace trdq

using namespace trdq;

extern "C" {

const char* trdq_status_string(trdq_status s) {
  switch (s) {
    case TRDQ_OK: return "ok";
    case TRDQ_ERR_NULL: return "null pointer";
    case TRDQ_ERR_SHAPE: return "unsupported shape";
    case TRDQ_ERR_ALIGN: return "pointer or stride not 16-byte aligned";
    case TRDQ_ERR_TIMESTEP: return "time-step outside the covered range";
    case TRDQ_ERR_GROUP: return "invalid group specification";
    case TRDQ_ERR_WBITS: return "unsupported weight bit-width";
    case TRDQ_ERR_CUDA: return "CUDA call failed";
    case TRDQ_ERR_NOMEM: return "out of memory";
    case TRDQ_ERR_TIMEOUT: return "bounded device-side wait expired";
    case TRDQ_ERR_MISMATCH: return "objects do not belong together";
    case TRDQ_ERR_SCRATCH: return "problem exceeds the built-in scratch area";
  }
  return "unknown status";
}

int32_t trdq_version(void) { return 100; }

trdq_status trdq_rotation_create(const trdq_rotation_spec* spec, trdq_rotation** out) {
  if (!spec || !out || !spec->t_bounds || !spec->signs) return TRDQ_ERR_NULL;
  if (spec->block != TRDQ_BLOCK || spec->K <= 0 || spec->K % TRDQ_BLOCK != 0 || spec->K > TRDQ_MAX_K) return TRDQ_ERR_SHAPE;
  if (spec->num_groups < 1) return TRDQ_ERR_GROUP;
  const int G = spec->num_groups, K = spec->K;
  for (int g = 0; g < G; ++g)
    if (spec->t_bounds[g] >= spec->t_bounds[g + 1]) return TRDQ_ERR_GROUP;
  const size_t n = static_cast<size_t>(G) * K;
  for (size_t i = 0; i < n; ++i) {
    if (spec->signs[i] != 1 && spec->signs[i] != -1) return TRDQ_ERR_GROUP;
    if (spec->smooth && !(spec->smooth[i] > 0.0f && std::isfinite(spec->smooth[i]))) return TRDQ_ERR_GROUP;
  }

  trdq_rotation* rot = new (std::nothrow) trdq_rotation;
  if (!rot) return TRDQ_ERR_NOMEM;
  rot->K = K;
  rot->num_groups = G;
  rot->t_bounds.assign(spec->t_bounds, spec->t_bounds + G + 1);

  // d * Delta / sqrt(128) and d / (Delta * sqrt(128)), in double, rounded once to fp32
  const double norm = 0x1.6a09e667f3bcdp-4;  // 2^-3.5 = sqrt(2)/16, correctly rounded
  std::vector<float> act(n), wv(n);
  for (size_t i = 0; i < n; ++i) {
    const double d = static_cast<double>(spec->signs[i]);
    const double delta = spec->smooth ? static_cast<double>(spec->smooth[i]) : 1.0;
    act[i] = static_cast<float>(d * delta * norm);
    wv[i] = static_cast<float>(d / delta * norm);
  }
  if (cudaGetDevice(&rot->device) != cudaSuccess) {
    delete rot;
    return TRDQ_ERR_CUDA;
  }
  if (cudaMalloc(&rot->act_vec, n * sizeof(float)) != cudaSuccess || cudaMalloc(&rot->weight_vec, n * sizeof(float)) != cudaSuccess) {
    cudaGetLastError();
    trdq_rotation_destroy(rot);
    return TRDQ_ERR_NOMEM;
  }
  if (cudaMemcpy(rot->act_vec, act.data(), n * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(rot->weight_vec, wv.data(), n * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess) {
    trdq_rotation_destroy(rot);
    return TRDQ_ERR_CUDA;
  }
  *out = rot;
  return TRDQ_OK;
}

trdq_status trdq_rotation_create_full(const trdq_rotation_spec* spec, const int32_t* perm, const int8_t* signs2, trdq_rotation** out) {
  if (!spec || !perm || !out) return TRDQ_ERR_NULL;
  if (spec->K <= 0 || spec->K % TRDQ_BLOCK != 0 || spec->K > 16384) return TRDQ_ERR_SHAPE;
  if (spec->num_groups < 1) return TRDQ_ERR_GROUP;
  const int G = spec->num_groups, K = spec->K;
  const size_t n = static_cast<size_t>(G) * K;
  std::vector<char> seen(K);
  for (int g = 0; g < G; ++g) {
    std::fill(seen.begin(), seen.end(), 0);
    for (int j = 0; j < K; ++j) {
      const int32_t s = perm[static_cast<size_t>(g) * K + j];
      if (s < 0 || s >= K || seen[s]) return TRDQ_ERR_GROUP;
      seen[s] = 1;
    }
  }
  if (signs2)
    for (size_t i = 0; i < n; ++i)
      if (signs2[i] != 1 && signs2[i] != -1) return TRDQ_ERR_GROUP;
  trdq_rotation* rot = nullptr;
  const trdq_status st = trdq_rotation_create(spec, &rot);
  if (st != TRDQ_OK) return st;
  const double norm = 0x1.6a09e667f3bcdp-4;  // 2^-3.5
  std::vector<float> v2(n);
  for (size_t i = 0; i < n; ++i) v2[i] = static_cast<float>((signs2 ? static_cast<double>(signs2[i]) : 1.0) * norm);
  if (cudaMalloc(&rot->perm, n * sizeof(int32_t)) != cudaSuccess || cudaMalloc(&rot->vec2, n * sizeof(float)) != cudaSuccess) {
    cudaGetLastError();
    trdq_rotation_destroy(rot);
    return TRDQ_ERR_NOMEM;
  }
  if (cudaMemcpy(rot->perm, perm, n * sizeof(int32_t), cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(rot->vec2, v2.data(), n * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess) {
    trdq_rotation_destroy(rot);
    return TRDQ_ERR_CUDA;
  }
  *out = rot;
  return TRDQ_OK;
}

trdq_status trdq_zigzag_permutation(const float* magnitude, int32_t K, int32_t* perm) {
  if (!magnitude || !perm) return TRDQ_ERR_NULL;
  if (K <= 0 || K % TRDQ_BLOCK != 0) return TRDQ_ERR_SHAPE;
  const int blocks = K / TRDQ_BLOCK;
  std::vector<int32_t> order(K);
  for (int j = 0; j < K; ++j) order[j] = j;
  std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return magnitude[a] > magnitude[b]; });
  for (int round = 0; round < TRDQ_BLOCK; ++round)
    for (int i = 0; i < blocks; ++i) {
      const int block = (round & 1) ? blocks - 1 - i : i;
      perm[block * TRDQ_BLOCK + round] = order[static_cast<size_t>(round) * blocks + i];
    }
  return TRDQ_OK;
}

trdq_status trdq_rotation_destroy(trdq_rotation* rot) {
  if (!rot) return TRDQ_OK;
  if (rot->act_vec) cudaFree(rot->act_vec);
  if (rot->weight_vec) cudaFree(rot->weight_vec);
  if (rot->perm) cudaFree(rot->perm);
  if (rot->vec2) cudaFree(rot->vec2);
  if (rot->dense) cudaFree(rot->dense);
  if (rot->dense_inv_t) cudaFree(rot->dense_inv_t);
  delete rot;
  return TRDQ_OK;
}

trdq_status trdq_find_group(const int32_t* t_bounds, int32_t num_groups, int32_t t, int32_t* g) {
  if (!t_bounds || !g) return TRDQ_ERR_NULL;
  if (num_groups < 1) return TRDQ_ERR_GROUP;
  for (int i = 0; i < num_groups; ++i)
    if (t_bounds[i] >= t_bounds[i + 1]) return TRDQ_ERR_GROUP;
  for (int i = 0; i < num_groups; ++i)
    if (t_bounds[i] <= t && t < t_bounds[i + 1]) {
      *g = i;
      return TRDQ_OK;
    }
  return TRDQ_ERR_TIMESTEP;
}

trdq_status trdq_group_of(const trdq_rotation* rot, int32_t t, int32_t* g) {
  if (!rot || !g) return TRDQ_ERR_NULL;
  const int r = find_group(rot->t_bounds, t);
  if (r < 0) return TRDQ_ERR_TIMESTEP;
  *g = r;
  return TRDQ_OK;
}

trdq_status trdq_prepare_weights(const trdq_rotation* rot, const void* W_bf16, int32_t N, int32_t wbits, trdq_weights** out,
                                 void* stream) {
  if (!rot || !W_bf16 || !out) return TRDQ_ERR_NULL;
  if (wbits != 8 && wbits != 4) return TRDQ_ERR_WBITS;
  if (N <= 0 || N % 16 != 0) return TRDQ_ERR_SHAPE;
  if (!aligned16(W_bf16)) return TRDQ_ERR_ALIGN;
  if (!on_current_device(rot->device)) return TRDQ_ERR_MISMATCH;
  const int K = rot->K, G = rot->num_groups;

  trdq_weights* w = new (std::nothrow) trdq_weights;
  if (!w) return TRDQ_ERR_NOMEM;
  w->N = N;
  w->K = K;
  w->wbits = wbits;
  w->num_groups = G;
  w->t_bounds = rot->t_bounds;
  w->groups.resize(G);
  if (cudaGetDevice(&w->device) != cudaSuccess) {
    delete w;
    return TRDQ_ERR_CUDA;
  }
  const size_t code_bytes = wbits == 8 ? static_cast<size_t>(N) * K : static_cast<size_t>(N) * K / 2;
  const size_t scale_count = wbits == 8 ? static_cast<size_t>(N) : static_cast<size_t>(N) * (K / TRDQ_BLOCK);
  const uint64_t row_bytes = wbits == 8 ? K : K / 2;
  const uint32_t box_bytes = wbits == 8 ? 128 : 64;
  for (int g = 0; g < G; ++g) {
    GroupWeights& gw = w->groups[g];
    if (cudaMalloc(&gw.codes, code_bytes) != cudaSuccess || cudaMalloc(&gw.scales, scale_count * sizeof(float)) != cudaSuccess) {
      cudaGetLastError();
      trdq_weights_destroy(w);
      return TRDQ_ERR_NOMEM;
    }
    if (rot->dense) {
      // dense blocks (Eq. 6-8): W S^-1 into an fp32 scratch, then the quantizer
      float* wr = nullptr;
      if (cudaMalloc(&wr, static_cast<size_t>(N) * K * sizeof(float)) != cudaSuccess) {
        cudaGetLastError();
        trdq_weights_destroy(w);
        return TRDQ_ERR_NOMEM;
      }
      const size_t per_group = static_cast<size_t>(K / TRDQ_BLOCK) * TRDQ_BLOCK * TRDQ_BLOCK;
      const cudaError_t ed = launch_dense_prepare(W_bf16, N, K, rot->dense_inv_t + static_cast<size_t>(g) * per_group, wbits, wr, gw.codes,
                                                  gw.scales, static_cast<cudaStream_t>(stream));
      const cudaError_t es = ed == cudaSuccess ? cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) : ed;  // the scratch is freed next
      cudaFree(wr);
      if (es != cudaSuccess) {
        trdq_weights_destroy(w);
        return TRDQ_ERR_CUDA;
      }
    }
    const cudaError_t e =
        rot->dense ? cudaSuccess :
        rot->perm ? launch_rotate2_quantize(W_bf16, K, N, K, rot->weight_vec + static_cast<size_t>(g) * K, rot->perm + static_cast<size_t>(g) * K,
                                            rot->vec2 + static_cast<size_t>(g) * K, wbits == 8 ? 0 : 1, gw.codes, gw.scales,
                                            static_cast<cudaStream_t>(stream))
                  : launch_rotate_quantize(W_bf16, K, N, K, rot->weight_vec + static_cast<size_t>(g) * K, wbits == 8 ? 0 : 1, gw.codes,
                                           gw.scales, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) {
      trdq_weights_destroy(w);
      return TRDQ_ERR_CUDA;
    }
    for (int i = 0; i < kNumTileN; ++i) {
      const trdq_status st = wbits == 8
                                 ? encode_tmap_u8_sw128(&gw.tmap_b[i], gw.codes, row_bytes, N, row_bytes, box_bytes, kTileN[i])
                                 : encode_tmap_2d(&gw.tmap_b[i], gw.codes, 1, row_bytes, N, row_bytes, box_bytes, 128, 0);
      if (st != TRDQ_OK) {
        trdq_weights_destroy(w);
        return st;
      }
      if (wbits == 8 && encode_tmap_u8_sw128(&gw.tmap_b_half[i], gw.codes, row_bytes, N, row_bytes, box_bytes, kTileN[i] / 2) != TRDQ_OK) {
        trdq_weights_destroy(w);
        return TRDQ_ERR_CUDA;
      }
    }
    // The kernels below end the group's preparation and MUST stay ordinary launches (full stream dependency, no early
    // trigger of dependents): the GEMM kernels request weight tiles before their dependent-launch wait, which orders
    // them only against the kernel directly before them, so the codes have to be complete before that kernel starts.
    if (wbits == 8) {
      if (cudaMalloc(&gw.colsum, static_cast<size_t>(N) * sizeof(int32_t)) != cudaSuccess) {
        cudaGetLastError();
        trdq_weights_destroy(w);
        return TRDQ_ERR_NOMEM;
      }
      if (launch_weight_colsum(static_cast<const int8_t*>(gw.codes), N, K, gw.colsum, static_cast<cudaStream_t>(stream)) != cudaSuccess) {
        trdq_weights_destroy(w);
        return TRDQ_ERR_CUDA;
      }
    }
    if (wbits == 4) {
      const int n_pad = (N + 127) / 128 * 128;
      const int groups = K / TRDQ_BLOCK;
      if (cudaMalloc(&gw.mult_t, static_cast<size_t>(groups) * n_pad * sizeof(int32_t)) != cudaSuccess ||
          cudaMalloc(&gw.base, static_cast<size_t>(n_pad) * sizeof(float)) != cudaSuccess) {
        cudaGetLastError();
        trdq_weights_destroy(w);
        return TRDQ_ERR_NOMEM;
      }
      if (launch_w4_multipliers(gw.scales, N, groups, n_pad, gw.mult_t, gw.base, static_cast<cudaStream_t>(stream)) != cudaSuccess) {
        trdq_weights_destroy(w);
        return TRDQ_ERR_CUDA;
      }
    }
  }
  *out = w;
  return TRDQ_OK;
}

trdq_status trdq_weights_destroy(trdq_weights* w) {
  if (!w) return TRDQ_OK;
  for (auto& gw : w->groups) {
    if (gw.codes) cudaFree(gw.codes);
    if (gw.scales) cudaFree(gw.scales);
    if (gw.colsum) cudaFree(gw.colsum);
    if (gw.mult_t) cudaFree(gw.mult_t);
    if (gw.base) cudaFree(gw.base);
  }
  delete w;
  return TRDQ_OK;
}

trdq_status trdq_weights_info(const trdq_weights* w, int32_t* N, int32_t* K, int32_t* wbits, int32_t* num_groups) {
  if (!w) return TRDQ_ERR_NULL;
  if (N) *N = w->N;
  if (K) *K = w->K;
  if (wbits) *wbits = w->wbits;
  if (num_groups) *num_groups = w->num_groups;
  return TRDQ_OK;
}

trdq_status trdq_weights_view(const trdq_weights* w, int32_t g, const void** Wq, const float** scales) {
  if (!w) return TRDQ_ERR_NULL;
  if (g < 0 || g >= w->num_groups) return TRDQ_ERR_GROUP;
  if (Wq) *Wq = w->groups[g].codes;
  if (scales) *scales = w->groups[g].scales;
  return TRDQ_OK;
}

trdq_status trdq_weights_export(const trdq_weights* w, int32_t g, void* codes_out, float* scales_out, void* stream) {
  if (!w) return TRDQ_ERR_NULL;
  if (g < 0 || g >= w->num_groups) return TRDQ_ERR_GROUP;
  const size_t code_bytes = w->wbits == 8 ? static_cast<size_t>(w->N) * w->K : static_cast<size_t>(w->N) * w->K / 2;
  const size_t scale_count = w->wbits == 8 ? static_cast<size_t>(w->N) : static_cast<size_t>(w->N) * (w->K / TRDQ_BLOCK);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (codes_out && cudaMemcpyAsync(codes_out, w->groups[g].codes, code_bytes, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return TRDQ_ERR_CUDA;
  if (scales_out &&
      cudaMemcpyAsync(scales_out, w->groups[g].scales, scale_count * sizeof(float), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return TRDQ_ERR_CUDA;
  return TRDQ_OK;
}

trdq_status trdq_rotate_quantize(const trdq_rotation* rot, int32_t t, const void* X_bf16, int64_t ldx, int32_t M, int8_t* codes,
                                 float* scales, void* stream) {
  if (!rot) return TRDQ_ERR_NULL;
  if (rot->dense) return TRDQ_ERR_MISMATCH;  // dense blocks need the workspace of trdq_rotate_dense_quantize
  if (M < 0) return TRDQ_ERR_SHAPE;
  const int g = find_group(rot->t_bounds, t);
  if (g < 0) return TRDQ_ERR_TIMESTEP;
  if (M == 0) return TRDQ_OK;
  if (!X_bf16 || !codes || !scales) return TRDQ_ERR_NULL;
  if (ldx < rot->K) return TRDQ_ERR_SHAPE;
  if (ldx % 8 != 0 || !aligned16(X_bf16) || !aligned16(codes) || (reinterpret_cast<uintptr_t>(scales) & 3u)) return TRDQ_ERR_ALIGN;
  if (!on_current_device(rot->device)) return TRDQ_ERR_MISMATCH;
  const float* vec = rot->act_vec + static_cast<size_t>(g) * rot->K;
  if (rot->perm) {
    const cudaError_t e2 = launch_rotate2_quantize(X_bf16, ldx, M, rot->K, vec, rot->perm + static_cast<size_t>(g) * rot->K,
                                                   rot->vec2 + static_cast<size_t>(g) * rot->K, 0, codes, scales,
                                                   static_cast<cudaStream_t>(stream));
    return finish(e2 == cudaSuccess ? TRDQ_OK : TRDQ_ERR_CUDA, stream);
  }
  if (rotate_quantize_prefers_team(M, rot->K))
    return finish(launch_rotate_quantize_team(X_bf16, ldx, M, rot->K, vec, codes, scales, static_cast<cudaStream_t>(stream)), stream);
  const cudaError_t e = launch_rotate_quantize(X_bf16, ldx, M, rot->K, vec, 0, codes, scales, static_cast<cudaStream_t>(stream));
  return finish(e == cudaSuccess ? TRDQ_OK : TRDQ_ERR_CUDA, stream);
}

trdq_status trdq_norm_rotate_quantize(const trdq_rotation* rot, int32_t t, const void* X_bf16, int64_t ldx, int32_t M,
                                      const void* shift_bf16, const void* scale_bf16, int32_t rows_per_sample, float eps, int8_t* codes,
                                      float* scales, void* stream) {
  if (!rot) return TRDQ_ERR_NULL;
  if (rot->dense || rot->perm) return TRDQ_ERR_MISMATCH;
  if (M < 0 || rot->K > 8192 || rows_per_sample <= 0 || !(eps >= 0.0f) || !std::isfinite(eps)) return TRDQ_ERR_SHAPE;
  const int g = find_group(rot->t_bounds, t);
  if (g < 0) return TRDQ_ERR_TIMESTEP;
  if (M == 0) return TRDQ_OK;
  if (!X_bf16 || !codes || !scales) return TRDQ_ERR_NULL;
  if (ldx < rot->K) return TRDQ_ERR_SHAPE;
  if (ldx % 8 != 0 || !aligned16(X_bf16) || !aligned16(codes) || (reinterpret_cast<uintptr_t>(scales) & 3u) ||
      (shift_bf16 && !aligned16(shift_bf16)) || (scale_bf16 && !aligned16(scale_bf16)))
    return TRDQ_ERR_ALIGN;
  if (!on_current_device(rot->device)) return TRDQ_ERR_MISMATCH;
  const cudaError_t e = launch_norm_rotate_quantize(X_bf16, ldx, M, rot->K, rot->act_vec + static_cast<size_t>(g) * rot->K, shift_bf16,
                                                    scale_bf16, rows_per_sample, eps, codes, scales, static_cast<cudaStream_t>(stream));
  return finish(e == cudaSuccess ? TRDQ_OK : TRDQ_ERR_CUDA, stream);
}

static trdq_status linear_common(const trdq_weights* w, int32_t t, const int8_t* const codes[2], const float* const scales[2],
                                 const int32_t M[2], const void* bias, void* const Y[2], const int64_t ld[2], bool raw,
                                 void* stream, int act = 0) {
  if (!w || !codes || !M || !Y || !ld || (!raw && !scales)) return TRDQ_ERR_NULL;
  if (M[0] < 0 || M[1] < 0) return TRDQ_ERR_SHAPE;
  const int g = find_group(w->t_bounds, t);
  if (g < 0) return TRDQ_ERR_TIMESTEP;
  if (raw && w->wbits != 8) return TRDQ_ERR_WBITS;
  GemmSegment seg[2];
  for (int s = 0; s < 2; ++s) {
    seg[s] = GemmSegment{codes[s], raw ? nullptr : scales[s], Y[s], ld[s], M[s]};
    if (M[s] == 0) continue;
    const trdq_status st = check_linear_segment(w, codes[s], raw ? nullptr : scales[s], Y[s], ld[s], raw);
    if (st != TRDQ_OK) return st;
  }
  if (M[0] == 0 && M[1] == 0) return TRDQ_OK;
  if (check_bias(bias) != TRDQ_OK) return TRDQ_ERR_ALIGN;
  if (!on_current_device(w->device)) return TRDQ_ERR_MISMATCH;
  if (w->wbits == 8) return finish(launch_gemm_w8(w, g, seg, bias, raw, static_cast<cudaStream_t>(stream), act), stream);
  return finish(launch_gemm_w4(w, g, seg, bias, static_cast<cudaStream_t>(stream), act), stream);
}

trdq_status trdq_linear(const trdq_weights* w, int32_t t, const int8_t* codes, const float* scales, int32_t M, const void* bias_bf16,
                        void* Y_bf16, int64_t ldy, void* stream) {
  const int8_t* c[2] = {codes, nullptr};
  const float* s[2] = {scales, nullptr};
  const int32_t m[2] = {M, 0};
  void* y[2] = {Y_bf16, nullptr};
  const int64_t l[2] = {ldy, ldy};
  return linear_common(w, t, c, s, m, bias_bf16, y, l, false, stream);
}

trdq_status trdq_linear_act(const trdq_weights* w, int32_t t, const int8_t* codes, const float* scales, int32_t M, const void* bias_bf16,
                            void* Y_bf16, int64_t ldy, int32_t act, void* stream) {
  if (act != TRDQ_ACT_NONE && act != TRDQ_ACT_GELU_TANH) return TRDQ_ERR_SHAPE;
  const int8_t* c[2] = {codes, nullptr};
  const float* s[2] = {scales, nullptr};
  const int32_t m[2] = {M, 0};
  void* y[2] = {Y_bf16, nullptr};
  const int64_t l[2] = {ldy, ldy};
  return linear_common(w, t, c, s, m, bias_bf16, y, l, false, stream, act);
}

trdq_status trdq_linear_cfg(const trdq_weights* w, int32_t t, const int8_t* const codes[2], const float* const scales[2],
                            const int32_t M[2], const void* bias_bf16, void* const Y_bf16[2], const int64_t ldy[2], void* stream) {
  return linear_common(w, t, codes, scales, M, bias_bf16, Y_bf16, ldy, false, stream);
}

trdq_status trdq_linear_splitk_workspace(const trdq_weights* w, int32_t M, int32_t* splits, uint64_t* bytes) {
  if (!w) return TRDQ_ERR_NULL;
  if (M < 0) return TRDQ_ERR_SHAPE;
  const int s = M > 0 ? splitk_choose(w, M) : 1;
  if (splits) *splits = s;
  if (bytes) *bytes = s > 1 ? static_cast<uint64_t>(s) * static_cast<uint64_t>(M) * static_cast<uint64_t>(w->N) * 4u : 0u;
  return TRDQ_OK;
}

trdq_status trdq_linear_splitk(const trdq_weights* w, int32_t t, const int8_t* codes, const float* scales, int32_t M,
                               const void* bias_bf16, void* Y_bf16, int64_t ldy, void* workspace, uint64_t workspace_bytes,
                               void* stream) {
  if (!w) return TRDQ_ERR_NULL;
  if (M < 0) return TRDQ_ERR_SHAPE;
  const int splits = M > 0 ? splitk_choose(w, M) : 1;
  if (splits <= 1) return trdq_linear(w, t, codes, scales, M, bias_bf16, Y_bf16, ldy, stream);
  const int g = find_group(w->t_bounds, t);
  if (g < 0) return TRDQ_ERR_TIMESTEP;
  if (!workspace) return TRDQ_ERR_NULL;
  const trdq_status chk = check_linear_segment(w, codes, scales, Y_bf16, ldy, false);
  if (chk != TRDQ_OK) return chk;
  if (!aligned16(workspace) || check_bias(bias_bf16) != TRDQ_OK) return TRDQ_ERR_ALIGN;
  if (!on_current_device(w->device)) return TRDQ_ERR_MISMATCH;
  if (workspace_bytes < static_cast<uint64_t>(splits) * static_cast<uint64_t>(M) * static_cast<uint64_t>(w->N) * 4u) return TRDQ_ERR_NOMEM;
  const GemmSegment seg{codes, scales, Y_bf16, ldy, M};
  return finish(launch_gemm_w8_splitk(w, g, seg, bias_bf16, splits, static_cast<int32_t*>(workspace), static_cast<cudaStream_t>(stream)), stream);
}

trdq_status trdq_linear_splitk_static(const trdq_weights* w, int32_t t, const int8_t* codes, const float* scales, int32_t M,
                                      const void* bias_bf16, void* Y_bf16, int64_t ldy, void* stream) {
  if (!w) return TRDQ_ERR_NULL;
  if (M < 0) return TRDQ_ERR_SHAPE;
  const int splits = M > 0 ? splitk_choose(w, M) : 1;
  if (splits <= 1) return trdq_linear(w, t, codes, scales, M, bias_bf16, Y_bf16, ldy, stream);
  const int g = find_group(w->t_bounds, t);
  if (g < 0) return TRDQ_ERR_TIMESTEP;
  const trdq_status chk = check_linear_segment(w, codes, scales, Y_bf16, ldy, false);
  if (chk != TRDQ_OK) return chk;
  if (check_bias(bias_bf16) != TRDQ_OK) return TRDQ_ERR_ALIGN;
  if (!on_current_device(w->device)) return TRDQ_ERR_MISMATCH;
  const GemmSegment seg{codes, scales, Y_bf16, ldy, M};
  return finish(launch_gemm_w8_splitk_static(w, g, seg, bias_bf16, splits, static_cast<cudaStream_t>(stream)), stream);
}

trdq_status trdq_rotate_quantize_asym(const trdq_rotation* rot, int32_t t, const void* X_bf16, int64_t ldx, int32_t M, uint8_t* codes,
                                      float* scales, int32_t* zero_points, void* stream) {
  if (!rot) return TRDQ_ERR_NULL;
  if (rot->dense) return TRDQ_ERR_MISMATCH;
  if (M < 0 || rot->K > 10240 || rot->perm) return TRDQ_ERR_SHAPE;
  const int g = find_group(rot->t_bounds, t);
  if (g < 0) return TRDQ_ERR_TIMESTEP;
  if (M == 0) return TRDQ_OK;
  if (!X_bf16 || !codes || !scales || !zero_points) return TRDQ_ERR_NULL;
  if (ldx < rot->K) return TRDQ_ERR_SHAPE;
  if (ldx % 8 != 0 || !aligned16(X_bf16) || !aligned16(codes) || (reinterpret_cast<uintptr_t>(scales) & 3u) ||
      (reinterpret_cast<uintptr_t>(zero_points) & 3u))
    return TRDQ_ERR_ALIGN;
  if (!on_current_device(rot->device)) return TRDQ_ERR_MISMATCH;
  const cudaError_t e = launch_rotate_quantize_asym(X_bf16, ldx, M, rot->K, rot->act_vec + static_cast<size_t>(g) * rot->K, codes, scales,
                                                    zero_points, static_cast<cudaStream_t>(stream));
  return finish(e == cudaSuccess ? TRDQ_OK : TRDQ_ERR_CUDA, stream);
}

trdq_status trdq_linear_asym(const trdq_weights* w, int32_t t, const uint8_t* codes, const float* scales, const int32_t* zero_points,
                             int32_t M, const void* bias_bf16, void* Y_bf16, int64_t ldy, void* stream) {
  if (!w) return TRDQ_ERR_NULL;
  if (w->wbits != 8) return TRDQ_ERR_WBITS;
  if (M < 0 || w->K > 32768) return TRDQ_ERR_SHAPE;
  const int g = find_group(w->t_bounds, t);
  if (g < 0) return TRDQ_ERR_TIMESTEP;
  if (M == 0) return TRDQ_OK;
  if (!zero_points) return TRDQ_ERR_NULL;
  const trdq_status chk = check_linear_segment(w, codes, scales, Y_bf16, ldy, false);
  if (chk != TRDQ_OK) return chk;
  if (!aligned_to(zero_points, 4) || check_bias(bias_bf16) != TRDQ_OK) return TRDQ_ERR_ALIGN;
  if (!on_current_device(w->device)) return TRDQ_ERR_MISMATCH;
  GemmSegment seg[2] = {GemmSegment{reinterpret_cast<const int8_t*>(codes), scales, Y_bf16, ldy, M}, GemmSegment{nullptr, nullptr, nullptr, ldy, 0}};
  const int32_t* zp[2] = {zero_points, nullptr};
  return finish(launch_gemm_w8_asym(w, g, seg, zp, bias_bf16, static_cast<cudaStream_t>(stream)), stream);
}

trdq_status trdq_gemm_i32(const trdq_weights* w, int32_t t, const int8_t* codes, int32_t M, int32_t* acc, int64_t ldacc, void* stream) {
  const int8_t* c[2] = {codes, nullptr};
  const int32_t m[2] = {M, 0};
  void* y[2] = {acc, nullptr};
  const int64_t l[2] = {ldacc, ldacc};
  return linear_common(w, t, c, nullptr, m, nullptr, y, l, true, stream);
}

trdq_status trdq_run_layers(const trdq_layer_op* ops, int32_t count, int32_t t, void* stream) {
  if (count < 0) return TRDQ_ERR_SHAPE;
  if (count == 0) return TRDQ_OK;
  if (!ops) return TRDQ_ERR_NULL;
  for (int i = 0; i < count; ++i) {
    const trdq_layer_op& op = ops[i];
    if (!op.rot || !op.w) return TRDQ_ERR_NULL;
    if (op.rot->K != op.w->K || op.rot->t_bounds != op.w->t_bounds || op.rot->device != op.w->device) return TRDQ_ERR_MISMATCH;
    if (op.rot->dense && op.M > 0) {
      if (!op.workspace) return TRDQ_ERR_NULL;
      if (op.workspace_bytes < rotate_dense_workspace_bytes(op.M, op.rot->K)) return TRDQ_ERR_NOMEM;
    }
    if (find_group(op.rot->t_bounds, t) < 0) return TRDQ_ERR_TIMESTEP;
    if (op.M < 0 || op.ldx < op.rot->K || op.ldy < op.w->N) return TRDQ_ERR_SHAPE;
    if (op.M > 0 && (!op.X_bf16 || !op.codes || !op.scales || !op.Y_bf16)) return TRDQ_ERR_NULL;
    if (op.ldx % 8 != 0 || op.ldy % 8 != 0 || !aligned16(op.X_bf16) || !aligned16(op.codes) || !aligned16(op.Y_bf16) ||
        !aligned_to(op.scales, 4) || check_bias(op.bias_bf16) != TRDQ_OK)
      return TRDQ_ERR_ALIGN;
    if (op.act != TRDQ_ACT_NONE && op.act != TRDQ_ACT_GELU_TANH) return TRDQ_ERR_SHAPE;
  }
  for (int i = 0; i < count; ++i) {
    const trdq_layer_op& op = ops[i];
    trdq_status st = op.rot->dense ? trdq_rotate_dense_quantize(op.rot, t, op.X_bf16, op.ldx, op.M, op.codes, op.scales, op.workspace,
                                                                op.workspace_bytes, stream)
                                   : trdq_rotate_quantize(op.rot, t, op.X_bf16, op.ldx, op.M, op.codes, op.scales, stream);
    if (st != TRDQ_OK) return st;
    st = trdq_linear_act(op.w, t, op.codes, op.scales, op.M, op.bias_bf16, op.Y_bf16, op.ldy, op.act, stream);
    if (st != TRDQ_OK) return st;
  }
  return TRDQ_OK;
}

trdq_status trdq_kernel_choice(int32_t stage, int32_t M, int32_t K, int32_t N, int32_t wbits, char* name, int32_t name_bytes) {
  if (!name) return TRDQ_ERR_NULL;
  if (name_bytes < 48 || M <= 0 || K <= 0 || K % TRDQ_BLOCK != 0) return TRDQ_ERR_SHAPE;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return TRDQ_ERR_CUDA;  // the choice depends on the device (SM count, resident clusters)
  if (stage == 0) {
    describe_rotate_quantize_kernel(M, K, name, static_cast<size_t>(name_bytes));
    return TRDQ_OK;
  }
  if (stage != 1 || N <= 0) return TRDQ_ERR_SHAPE;
  if (wbits != 8 && wbits != 4) return TRDQ_ERR_WBITS;
  describe_gemm_kernel(M, K, N, wbits, name, static_cast<size_t>(name_bytes));
  return TRDQ_OK;
}

trdq_status trdq_measure_mma_ceiling(int32_t mmas_per_cluster, int32_t* clusters, void* stream) {
  if (!clusters) return TRDQ_ERR_NULL;
  if (mmas_per_cluster < 8 || mmas_per_cluster > (1 << 22)) return TRDQ_ERR_SHAPE;
  return launch_mma_ceiling(mmas_per_cluster, clusters, static_cast<cudaStream_t>(stream));
}

trdq_status trdq_selftest_wait_expiry(void* stream) {
  uint32_t* status = device_status_word();
  if (!status) return TRDQ_ERR_CUDA;
  selftest_wait_expiry_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(status);
  return finish(cudaGetLastError() == cudaSuccess ? TRDQ_OK : TRDQ_ERR_CUDA, stream);
}

trdq_status trdq_device_status(uint32_t* word) {
  uint32_t v = 0, zero = 0;
  if (cudaDeviceSynchronize() != cudaSuccess) return TRDQ_ERR_CUDA;
  if (cudaMemcpyFromSymbol(&v, g_status_word, sizeof v) != cudaSuccess) return TRDQ_ERR_CUDA;
  if (v != 0 && cudaMemcpyToSymbol(g_status_word, &zero, sizeof zero) != cudaSuccess) return TRDQ_ERR_CUDA;
  if (word) *word = v;
  return v == 0 ? TRDQ_OK : TRDQ_ERR_TIMEOUT;
}

}  // extern "C"
