// Dequantizing epilogue arithmetic shared by the 8-bit GEMM kernels (Eq. 10 on the codes, then the
// per-token and per-channel scales of Sec. 3.1 and the bias).
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace trdq {

// One output: y = acc * sx * sw + bias in fp32.  fp32 is accurate to 2^-23 of the product; only when
// product and bias cancel below `thr` = 2^-10 |bias| can that exceed a bf16 rounding step of the result;
// then the scale product is carried as an exact two-term sum and the part of the accumulator that
// fp32 could not hold is added back.
__device__ __forceinline__ float dequant_one(int32_t a, float sxm, float swn, float biasn, float thr) {
  const float af = static_cast<float>(a);
  const float s_hi = __fmul_rn(sxm, swn);
  float v = __fmaf_rn(af, s_hi, biasn);
  if (fabsf(v) < thr) {
    const float s_lo = __fmaf_rn(sxm, swn, -s_hi);
    v = __fmaf_rn(af, s_lo, v);
    v = __fmaf_rn(static_cast<float>(a - __float2int_rz(af)), s_hi, v);
  }
  return v;
}

// GELU in its tanh form, the activation between the two MLP linears of a DiT block:
//   gelu(x) = 0.5 x (1 + tanh(u)) = x / (1 + exp(-2u)) = x exp(2u) / (1 + exp(2u)),   u = sqrt(2/pi) (x + 0.044715 x^3).
// With e = exp(-|2u|) in (0, 1] the denominator 1 + e stays in [1, 2] on both sides, so nothing overflows and the
// fast division is in its defined range.  exp through ex2.approx: relative error near 1e-6, far inside a bf16
// rounding step; results below about 1e-37 in magnitude (x < -10) flush to zero.
__device__ __forceinline__ float gelu_tanh(float x) {
  const float k = 1.5957691216057308f;  // 2 sqrt(2/pi)
  const float t = __fmul_rn(x, __fmaf_rn(__fmul_rn(x, x), 0.044715f * k, k));  // 2u, same sign as x
  const float e = __expf(-fabsf(t));
  const float num = t >= 0.0f ? x : __fmul_rn(x, e);
  return __fdividef(num, __fadd_rn(1.0f, e));
}

// 32 consecutive columns of one output row: y = acc * sx * sw[n] + bias[n] (then GELU if ACT), packed to bf16 pairs.
// pb4: (sw, bias) of the 32 columns as 16 float4; thr4: 2^-10 * |bias| as 8 float4.
template <bool ACT = false>
__device__ __forceinline__ void dequant_row32(const uint32_t (&r)[32], float sxm, const float4* pb4, const float4* thr4,
                                              uint32_t (&packed)[16]) {
#pragma unroll
  for (int j = 0; j < 32; j += 4) {
    const float4 p01 = pb4[j / 2], p23 = pb4[j / 2 + 1], th = thr4[j / 4];
    const float swv[4] = {p01.x, p01.z, p23.x, p23.z};
    const float bv[4] = {p01.y, p01.w, p23.y, p23.w};
    const float tv[4] = {th.x, th.y, th.z, th.w};
    float y[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) y[e] = dequant_one(static_cast<int32_t>(r[j + e]), sxm, swv[e], bv[e], tv[e]);
    if (ACT) {
#pragma unroll
      for (int e = 0; e < 4; ++e) y[e] = gelu_tanh(y[e]);
    }
    const __nv_bfloat162 h0 = __floats2bfloat162_rn(y[0], y[1]);
    const __nv_bfloat162 h1 = __floats2bfloat162_rn(y[2], y[3]);
    packed[j / 2] = *reinterpret_cast<const uint32_t*>(&h0);
    packed[j / 2 + 1] = *reinterpret_cast<const uint32_t*>(&h1);
  }
}

// Stages the epilogue parameters of `count` columns starting at n0: (sw, bias) and the cancellation threshold.
__device__ __forceinline__ void stage_column_params(float2* pb, float* thr, const float* sw, const __nv_bfloat16* bias, int n0, int N,
                                                    int count, int tid, int nthreads) {
  for (int c = tid; c < count; c += nthreads) {
    const int n = n0 + c;
    float2 v = make_float2(0.0f, 0.0f);
    if (n < N) {
      v.x = __ldg(sw + n);
      v.y = bias ? __bfloat162float(bias[n]) : 0.0f;
    }
    pb[c] = v;
    thr[c] = fabsf(v.y) * 0.0009765625f;
  }
}

}  // namespace trdq
