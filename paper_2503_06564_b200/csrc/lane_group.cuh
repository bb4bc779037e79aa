// Pieces shared by the kernels that give one 128-block of a row to a group of 8 consecutive lanes (lane l holds
// elements 16 l .. 16 l + 15): the scaled load, the 128-point Walsh-Hadamard butterfly of Eq. 8's blocks with its fixed
// order of separately rounded fp32 additions (stages h = 1, 2, 4, 8 inside a thread, h = 16, 32, 64 across lanes l ^ 1,
// l ^ 2, l ^ 4 by warp shuffle), the group maximum and the quantizer step of Eq. 1.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace trdq {

constexpr int kLanesPerBlock = 8;
constexpr int kElemsPerLane = 16;

__device__ __forceinline__ void load_scaled16(const uint4* src, const float (&vec)[16], float (&u)[16]) {
  const uint4 a = __ldg(src);
  const uint4 b = __ldg(src + 1);
  const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    // bf16 -> fp32 is exact: the 16 bits become the high half of the fp32 pattern
    const float lo = __uint_as_float(w[i] << 16);
    const float hi = __uint_as_float(w[i] & 0xFFFF0000u);
    u[2 * i] = __fmul_rn(lo, vec[2 * i]);
    u[2 * i + 1] = __fmul_rn(hi, vec[2 * i + 1]);
  }
}

// 128-point unnormalised Walsh-Hadamard transform across the 8 lanes of a group, natural
// (Sylvester) order: stage h maps (a, b) = (u[i], u[i+h]) to (a + b, a - b).
__device__ __forceinline__ void wht128(float (&u)[16], int lane8) {
#pragma unroll
  for (int h = 1; h < 16; h <<= 1) {
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      if ((i & h) == 0) {
        const float a = u[i];
        const float b = u[i + h];
        u[i] = __fadd_rn(a, b);
        u[i + h] = __fsub_rn(a, b);
      }
    }
  }
#pragma unroll
  for (int mask = 1; mask < 8; mask <<= 1) {
    const bool upper = (lane8 & mask) != 0;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const float other = __shfl_xor_sync(0xffffffffu, u[i], mask);
      // lower lane: a + b with a = own; upper lane: a - b with a = other, b = own
      u[i] = __fadd_rn(other, upper ? -u[i] : u[i]);
    }
  }
}

__device__ __forceinline__ float absmax16(const float (&u)[16]) {
  float m = 0.0f;
#pragma unroll
  for (int i = 0; i < 16; ++i) m = fmaxf(m, fabsf(u[i]));
  return m;
}

__device__ __forceinline__ float group_max(float m) {
  m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
  m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
  m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 4));
  return m;
}

// Symmetric quantizer of Eq. 1 with z = 0: q = rne(v * fl(qmax / amax)).
__device__ __forceinline__ int quantize_one(float v, float inv) { return __float2int_rn(__fmul_rn(v, inv)); }

// ---- four lanes per 128-block, fp32 pairs (see the layout description in rotate_quantize.cu) ----
constexpr int kFastLanes = 4;
constexpr float kRoundMagic = 12582912.0f;  // 1.5 * 2^23

__device__ __forceinline__ float2 shfl_xor2(float2 v, int mask) {
  return make_float2(__shfl_xor_sync(0xffffffffu, v.x, mask), __shfl_xor_sync(0xffffffffu, v.y, mask));
}

__device__ __forceinline__ uint32_t pack4(float2 a, float2 b) {
  const uint32_t lo = __byte_perm(__float_as_uint(a.x), __float_as_uint(a.y), 0x0040);
  const uint32_t hi = __byte_perm(__float_as_uint(b.x), __float_as_uint(b.y), 0x0040);
  return __byte_perm(lo, hi, 0x5410);
}

// The lane's four 16-byte chunks of bf16 values widened to fp32 pairs (exact: the 16 bits become the high half of the
// fp32 pattern): v[4c + j] = elements (2j, 2j+1) of chunk c.
__device__ __forceinline__ void widen_chunks_lanes4(const uint4 (&raw)[4], float2 (&v)[16]) {
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    const uint32_t w[4] = {raw[c].x, raw[c].y, raw[c].z, raw[c].w};
#pragma unroll
    for (int j = 0; j < 4; ++j) v[4 * c + j] = make_float2(__uint_as_float(w[j] << 16), __uint_as_float(w[j] & 0xFFFF0000u));
  }
}

// The same, times the fused vector (sv points at the lane's first column; chunk c is 32 columns = 16 pairs further).
__device__ __forceinline__ void scale_chunks_lanes4(const uint4 (&raw)[4], const float2* sv, float2 (&v)[16]) {
  widen_chunks_lanes4(raw, v);
#pragma unroll
  for (int c = 0; c < 4; ++c) {
#pragma unroll
    for (int j = 0; j < 4; ++j) v[4 * c + j] = __fmul2_rn(v[4 * c + j], sv[16 * c + j]);
  }
}

// Largest magnitude of the block: the lane's 32 values, then the four lanes of the group.
__device__ __forceinline__ float absmax_lanes4(const float2 (&v)[16]) {
  float m = 0.0f;
#pragma unroll
  for (int p = 0; p < 16; ++p) m = fmaxf(fmaxf(m, fabsf(v[p].x)), fabsf(v[p].y));
  m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
  return fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
}

// Symmetric int8 codes of the lane's 32 values to dst (+ 32 c per chunk): q = rne(fl(v * inv)) with inv = fl(127 / amax).
// The product must be rounded to fp32 before the magic addition rounds it to an integer.  A packed multiply feeding a
// packed add gets contracted into one fused operation (a single rounding) by the assembler, so the product is written
// as fma(v, inv, zero) with `zero` a kernel argument equal to 0.0f: one rounding of v * inv, nothing left to contract.
__device__ __forceinline__ void quantize_store_lanes4(const float2 (&v)[16], float amax, float zero, int8_t* dst) {
  const float inv = amax > 0.0f ? __fdiv_rn(127.0f, amax) : 0.0f;
  const float2 inv2 = make_float2(inv, inv);
  const float2 magic2 = make_float2(kRoundMagic, kRoundMagic);
  const float2 zero2 = make_float2(zero, zero);
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    float2 q[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) q[j] = __fadd2_rn(__ffma2_rn(v[4 * c + j], inv2, zero2), magic2);
    *reinterpret_cast<uint2*>(dst + 32 * c) = make_uint2(pack4(q[0], q[1]), pack4(q[2], q[3]));
  }
}

// 128-point transform of one block spread over four lanes (16 fp32 pairs per lane, layout as described above).
__device__ __forceinline__ void wht128_lanes4(float2 (&v)[16], int lane4) {
  // h = 1: inside a pair
#pragma unroll
  for (int p = 0; p < 16; ++p) v[p] = make_float2(__fadd_rn(v[p].x, v[p].y), __fsub_rn(v[p].x, v[p].y));
  // h = 2, 4: pair index bits 0, 1
#pragma unroll
  for (int hb = 1; hb <= 2; hb <<= 1) {
#pragma unroll
    for (int p = 0; p < 16; ++p) {
      if ((p & hb) == 0) {
        const float2 a = v[p], c2 = v[p + hb];
        v[p] = __fadd2_rn(a, c2);
        v[p + hb] = __ffma2_rn(c2, make_float2(-1.0f, -1.0f), a);  // a - c, one rounding
      }
    }
  }
  // h = 8, 16: lanes l ^ 1, l ^ 2; upper lane computes other - own, lower lane own + other
#pragma unroll
  for (int mask = 1; mask <= 2; mask <<= 1) {
    const float sgn = (lane4 & mask) ? -1.0f : 1.0f;
    const float2 s2 = make_float2(sgn, sgn);
#pragma unroll
    for (int p = 0; p < 16; ++p) v[p] = __ffma2_rn(v[p], s2, shfl_xor2(v[p], mask));
  }
  // h = 32, 64: pair index bits 2, 3 (the chunk of the lane)
#pragma unroll
  for (int hb = 4; hb <= 8; hb <<= 1) {
#pragma unroll
    for (int p = 0; p < 16; ++p) {
      if ((p & hb) == 0) {
        const float2 a = v[p], c2 = v[p + hb];
        v[p] = __fadd2_rn(a, c2);
        v[p + hb] = __ffma2_rn(c2, make_float2(-1.0f, -1.0f), a);  // a - c, one rounding
      }
    }
  }

}

}  // namespace trdq
