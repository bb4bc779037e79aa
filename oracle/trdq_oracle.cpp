// CPU oracle for the time-rotated quantized linear layer (TR-DQ).
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of what the
// hot path computes, written from the paper's definitions.  It shares no code,
// header, table or helper with the CUDA library, and the library never calls it.
// Only the tests, the smoke check and the benchmark's cpu-baseline leg use it.
//
// What is followed, step by step (names as in the paper):
//   * Sec. 3.1, Eq. 1-2: uniform integer quantizer with nearest rounding, used in
//     its symmetric signed 8-bit form (zero-point 0, scale = absmax / 127);
//     per-token scales for activations and per-output-channel scales for weights
//     (the granularity paragraph of Sec. 3.1).
//   * Sec. 3.1, Eq. 4: channel scaling vector Delta.  Following Eq. 10 the online
//     side MULTIPLIES X by Delta_t and the offline side multiplies W by 1/Delta_t.
//   * Sec. 3.2, Eq. 8: block-diagonal orthogonal rotation, blocks of 2^n x 2^n;
//     here n = 7 and every block is diag(d) * H_128 / sqrt(128) with H_128 the
//     Sylvester-Walsh-Hadamard matrix and d a +-1 vector per time-step group.
//   * Sec. 3.2, Eq. 10: F_t(X, W) = G_t(X) . H_t(W) with the parameter set chosen
//     by the current time-step; the activation scales are computed online from each
//     token's own rotated values (Sec. 3.2, paragraph after Eq. 9).
//
// Parity notes.  The quantizer, the integer GEMM and the dequantising epilogue are
// pinned by the tests against closed forms and brute force.  Two things are
// conventions of this implementation that the paper does not fix ("parity unpinned" by the
// paper): the order of the fp32 additions inside the butterfly (h = 1, 2, ..., 64,
// natural output order) and the 4-bit weight storage format (two's complement
// nibbles, even k in the low nibble, one fp32 scale per 128 consecutive k).
//
// The full balancing transform of Eq. 9 (second block rotation after a zigzag permutation) is restated at
// the end of this file; its permutation convention and the Hadamard form of the second rotation are, like
// the first rotation's, conventions the paper leaves open ("parity unpinned" by the paper).
//
// Build: g++ -O2 -ffp-contract=off -fopenmp -shared -fPIC (no fast-math).
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

constexpr int kBlock = 128;
// 2^-3.5 = 1/sqrt(128): the normalisation that makes H_128/sqrt(128) orthogonal.
constexpr double kHadamardNorm = 0.08838834764831845;

inline float bf16_to_float(uint16_t b) {
  uint32_t u = static_cast<uint32_t>(b) << 16;
  float f;
  std::memcpy(&f, &u, sizeof f);
  return f;
}

// In-place Walsh-Hadamard butterfly on 128 fp32 values, unnormalised.
// Stage h pairs index i with i+h (bit h of i clear): (a, b) -> (a + b, a - b).
// Natural (Sylvester) order: out[i] = sum_j (-1)^popcount(i & j) in[j].
void butterfly128(float* u) {
  for (int h = 1; h < kBlock; h <<= 1) {
    for (int i = 0; i < kBlock; ++i) {
      if ((i & h) == 0) {
        const float a = u[i];
        const float b = u[i + h];
        u[i] = a + b;
        u[i + h] = a - b;
      }
    }
  }
}

// Scale one row by the fused vector and rotate every 128-block (Eq. 10, G_t / H_t).
void rotate_row(const uint16_t* row_bf16, const float* vec, int K, float* out) {
  for (int c = 0; c < K; c += kBlock) {
    float u[kBlock];
    for (int i = 0; i < kBlock; ++i) u[i] = bf16_to_float(row_bf16[c + i]) * vec[c + i];
    butterfly128(u);
    for (int i = 0; i < kBlock; ++i) out[c + i] = u[i];
  }
}

// Symmetric signed quantizer over `n` values with `qmax` levels each side (Eq. 1-2, z = 0).
// Returns the scale; writes integer codes.
float quantize_span(const float* v, int n, float qmax, int8_t* q) {
  float amax = 0.0f;
  for (int i = 0; i < n; ++i) amax = std::fmax(amax, std::fabs(v[i]));
  const float scale = amax / qmax;
  const float inv = amax > 0.0f ? qmax / amax : 0.0f;
  const int lim = static_cast<int>(qmax);
  for (int i = 0; i < n; ++i) {
    const float scaled = v[i] * inv;
    int r = static_cast<int>(std::nearbyintf(scaled));  // default mode: ties to even
    if (r > lim) r = lim;
    if (r < -lim) r = -lim;
    q[i] = static_cast<int8_t>(r);
  }
  return scale;
}


// ---- full balancing transform (Sec. 3.2, Eq. 9 / Eq. 10):  G_t(X) = (X Delta) R1 P R2 ------------
// R1 and R2 are block rotations of the same form, diag(d) . BlockDiag(H_128) / sqrt(128), with their own
// +-1 vectors d1, d2; P is the zigzag channel permutation, held as an index vector:
//     (v P)[j] = v[perm[j]]            (column j of P has its single 1 in row perm[j]).
// Row by row:  u = x o vec1;  v1 = blockWHT(u);  v2[j] = fl32(v1[perm[j]] * vec2[j]);  v3 = blockWHT(v2),
// with vec1 = d1 * Delta * 2^-3.5 (or d1 / Delta * 2^-3.5 on the weight side) and vec2 = d2 * 2^-3.5.
void rotate2_row(const uint16_t* row_bf16, const float* vec1, const int32_t* perm, const float* vec2, int K, float* out) {
  std::vector<float> v1(K);
  rotate_row(row_bf16, vec1, K, v1.data());
  for (int c = 0; c < K; c += kBlock) {
    float u[kBlock];
    for (int i = 0; i < kBlock; ++i) u[i] = v1[perm[c + i]] * vec2[c + i];
    butterfly128(u);
    for (int i = 0; i < kBlock; ++i) out[c + i] = u[i];
  }
}


// Asymmetric 8-bit quantizer of Eq. 1-3 over `n` values, literally:  X_int = clamp(round(X / s) + z, 0, 255),
// s = (max - min) / 255, with the zero point taken as z = -round(min / s) (Eq. 3 prints +round(min / s), which
// with Eq. 1's "+ z" would map the minimum to 2 * min / s instead of 0; the sign is read as a typo).
// As in the symmetric form, X / s is evaluated as X * fl(255 / (max - min)).  z is not clamped; codes are.
// Returns the scale, writes the zero point and unsigned codes.  A constant span (max == min) has scale 0, z = 0, codes 0.
float quantize_span_asym(const float* v, int n, uint8_t* q, int32_t* zero_point) {
  float vmin = v[0], vmax = v[0];
  for (int i = 1; i < n; ++i) {
    vmin = std::fmin(vmin, v[i]);
    vmax = std::fmax(vmax, v[i]);
  }
  const float range = vmax - vmin;
  const float scale = range / 255.0f;
  const float inv = range > 0.0f ? 255.0f / range : 0.0f;
  const int z = -static_cast<int>(std::nearbyintf(vmin * inv));
  for (int i = 0; i < n; ++i) {
    int r = static_cast<int>(std::nearbyintf(v[i] * inv)) + z;
    if (r > 255) r = 255;
    if (r < 0) r = 0;
    q[i] = static_cast<uint8_t>(r);
  }
  *zero_point = z;
  return scale;
}

// GELU in its tanh form (the activation between the two MLP linears of a DiT block), in double:
//   gelu(x) = 0.5 x (1 + tanh(u)),  u = sqrt(2/pi) (x + 0.044715 x^3).
// Written through the identity 0.5 (1 + tanh(u)) = 1 / (1 + exp(-2u)): the printed form loses all digits to the
// cancellation in 1 + tanh(u) once u < -18 (x < -7) even in double, this one is accurate on both tails.
// The paper does not discuss activations; this backs the fused-epilogue variant of the linear layer.
inline double gelu_tanh(double x) {
  const double c = 0.7978845608028654;  // sqrt(2/pi)
  const double u = c * (x + 0.044715 * x * x * x);
  return x / (1.0 + std::exp(-2.0 * u));
}

}  // namespace

extern "C" {

// Time-step -> group (Sec. 3.2: the parameter set is selected by the current
// time-step).  Returns g with bounds[g] <= t < bounds[g+1], or -1.
int oracle_group_of(const int32_t* bounds, int num_groups, int t) {
  for (int g = 0; g < num_groups; ++g)
    if (bounds[g] <= t && t < bounds[g + 1]) return g;
  return -1;
}

// Fused per-channel vectors of one group, computed in double and rounded once:
//   act[j]    = fl32(d[j] * Delta[j] * 2^-3.5)   (applied to X, Eq. 10 G_t)
//   weight[j] = fl32(d[j] / Delta[j] * 2^-3.5)   (applied to W, Eq. 10 H_t)
// smooth == nullptr means Delta = 1.
void oracle_fused_vectors(const int8_t* signs, const float* smooth, int K, float* act, float* weight) {
  for (int j = 0; j < K; ++j) {
    const double d = static_cast<double>(signs[j]);
    const double delta = smooth ? static_cast<double>(smooth[j]) : 1.0;
    act[j] = static_cast<float>(d * delta * kHadamardNorm);
    weight[j] = static_cast<float>(d / delta * kHadamardNorm);
  }
}

// Rotated rows in fp32 (no quantisation): v = (x o vec) . BlockDiag(H_128).
void oracle_rotate(const uint16_t* x_bf16, int64_t ldx, int M, int K, const float* vec, float* v) {
#pragma omp parallel for schedule(static)
  for (int m = 0; m < M; ++m) rotate_row(x_bf16 + static_cast<int64_t>(m) * ldx, vec, K, v + static_cast<int64_t>(m) * K);
}

// Per-row symmetric int8 quantiser on already-rotated fp32 rows.
void oracle_quantize_rows(const float* v, int M, int K, int8_t* codes, float* scales) {
#pragma omp parallel for schedule(static)
  for (int m = 0; m < M; ++m)
    scales[m] = quantize_span(v + static_cast<int64_t>(m) * K, K, 127.0f, codes + static_cast<int64_t>(m) * K);
}

// Online activation path: rotate then quantise per token.
void oracle_rotate_quantize(const uint16_t* x_bf16, int64_t ldx, int M, int K, const float* act_vec,
                            int8_t* codes, float* scales) {
#pragma omp parallel for schedule(static)
  for (int m = 0; m < M; ++m) {
    std::vector<float> v(K);
    rotate_row(x_bf16 + static_cast<int64_t>(m) * ldx, act_vec, K, v.data());
    scales[m] = quantize_span(v.data(), K, 127.0f, codes + static_cast<int64_t>(m) * K);
  }
}

// Offline weight path, 8-bit: rotate each output channel's row with the weight
// vector, quantise per output channel.
void oracle_prepare_w8(const uint16_t* w_bf16, int N, int K, const float* weight_vec, int8_t* codes, float* scales) {
  oracle_rotate_quantize(w_bf16, K, N, K, weight_vec, codes, scales);
}

// Offline weight path, 4-bit: one scale per (output channel, 128 consecutive k),
// codes in [-7, 7], two per byte (even k in the low nibble, two's complement).
void oracle_prepare_w4(const uint16_t* w_bf16, int N, int K, const float* weight_vec, uint8_t* packed, float* scales) {
  const int groups = K / kBlock;
#pragma omp parallel for schedule(static)
  for (int n = 0; n < N; ++n) {
    std::vector<float> v(K);
    rotate_row(w_bf16 + static_cast<int64_t>(n) * K, weight_vec, K, v.data());
    for (int kg = 0; kg < groups; ++kg) {
      int8_t q[kBlock];
      scales[static_cast<int64_t>(n) * groups + kg] = quantize_span(v.data() + kg * kBlock, kBlock, 7.0f, q);
      for (int i = 0; i < kBlock; i += 2) {
        const uint8_t lo = static_cast<uint8_t>(q[i]) & 0xF;
        const uint8_t hi = static_cast<uint8_t>(q[i + 1]) & 0xF;
        packed[(static_cast<int64_t>(n) * K + kg * kBlock + i) / 2] = static_cast<uint8_t>(lo | (hi << 4));
      }
    }
  }
}

// Sign-extending unpack of the 4-bit storage format back to int8 codes [N, K].
void oracle_unpack_w4(const uint8_t* packed, int64_t count, int8_t* codes) {
  for (int64_t i = 0; i < count; ++i) {
    const uint8_t byte = packed[i / 2];
    const int nib = (i & 1) ? (byte >> 4) : (byte & 0xF);
    codes[i] = static_cast<int8_t>(nib >= 8 ? nib - 16 : nib);
  }
}

// Integer GEMM (Eq. 10: G_t(X) . H_t(W) on the integer codes): exact int32 sums.
void oracle_gemm_i32(const int8_t* q, const int8_t* qw, int M, int N, int K, int32_t* acc) {
#pragma omp parallel for schedule(static)
  for (int m = 0; m < M; ++m)
    for (int n = 0; n < N; ++n) {
      int32_t s = 0;
      for (int k = 0; k < K; ++k)
        s += static_cast<int32_t>(q[static_cast<int64_t>(m) * K + k]) * static_cast<int32_t>(qw[static_cast<int64_t>(n) * K + k]);
      acc[static_cast<int64_t>(m) * N + n] = s;
    }
}

// Dequantising epilogue: y = acc * sx[m] * sw[n] + bias[n], evaluated in double and
// rounded once to fp32.  bias may be null.
void oracle_epilogue(const int32_t* acc, const float* sx, const float* sw, const uint16_t* bias_bf16, int M, int N, float* y) {
#pragma omp parallel for schedule(static)
  for (int m = 0; m < M; ++m)
    for (int n = 0; n < N; ++n) {
      double r = static_cast<double>(acc[static_cast<int64_t>(m) * N + n]) * static_cast<double>(sx[m]) * static_cast<double>(sw[n]);
      if (bias_bf16) r += static_cast<double>(bf16_to_float(bias_bf16[n]));
      y[static_cast<int64_t>(m) * N + n] = static_cast<float>(r);
    }
}

// W8A8 linear on a row subset: rows[i] selects the token; y is [num_rows, N].
// act: 0 = none, 1 = GELU (tanh form) applied to the double value before the single rounding to fp32.
void oracle_linear_w8_rows_act(const int8_t* q, const float* sx, const int8_t* qw, const float* sw, const uint16_t* bias_bf16,
                               const int64_t* rows, int num_rows, int N, int K, int act, float* y) {
#pragma omp parallel for schedule(static)
  for (int i = 0; i < num_rows; ++i) {
    const int64_t m = rows[i];
    for (int n = 0; n < N; ++n) {
      int32_t s = 0;
      for (int k = 0; k < K; ++k)
        s += static_cast<int32_t>(q[m * K + k]) * static_cast<int32_t>(qw[static_cast<int64_t>(n) * K + k]);
      double r = static_cast<double>(s) * static_cast<double>(sx[m]) * static_cast<double>(sw[n]);
      if (bias_bf16) r += static_cast<double>(bf16_to_float(bias_bf16[n]));
      if (act == 1) r = gelu_tanh(r);
      y[static_cast<int64_t>(i) * N + n] = static_cast<float>(r);
    }
  }
}
void oracle_linear_w8_rows(const int8_t* q, const float* sx, const int8_t* qw, const float* sw, const uint16_t* bias_bf16,
                           const int64_t* rows, int num_rows, int N, int K, float* y) {
  oracle_linear_w8_rows_act(q, sx, qw, sw, bias_bf16, rows, num_rows, N, K, 0, y);
}

// W4A8 linear on a row subset.  Every 128-wide k group has its own exact int32
// partial sum, scaled by that group's weight scale:
//   y = sx[m] * sum_kg (acc_kg * sw4[n, kg]) + bias[n]     (double, rounded once)
void oracle_linear_w4_rows_act(const int8_t* q, const float* sx, const uint8_t* packed, const float* sw4, const uint16_t* bias_bf16,
                               const int64_t* rows, int num_rows, int N, int K, int act, float* y) {
  const int groups = K / kBlock;
#pragma omp parallel for schedule(static)
  for (int i = 0; i < num_rows; ++i) {
    const int64_t m = rows[i];
    for (int n = 0; n < N; ++n) {
      double total = 0.0;
      for (int kg = 0; kg < groups; ++kg) {
        int32_t s = 0;
        for (int k = kg * kBlock; k < (kg + 1) * kBlock; ++k) {
          const uint8_t byte = packed[(static_cast<int64_t>(n) * K + k) / 2];
          const int nib = (k & 1) ? (byte >> 4) : (byte & 0xF);
          const int wq = nib >= 8 ? nib - 16 : nib;
          s += static_cast<int32_t>(q[m * K + k]) * wq;
        }
        total += static_cast<double>(s) * static_cast<double>(sw4[static_cast<int64_t>(n) * groups + kg]);
      }
      double r = static_cast<double>(sx[m]) * total;
      if (bias_bf16) r += static_cast<double>(bf16_to_float(bias_bf16[n]));
      if (act == 1) r = gelu_tanh(r);
      y[static_cast<int64_t>(i) * N + n] = static_cast<float>(r);
    }
  }
}
void oracle_linear_w4_rows(const int8_t* q, const float* sx, const uint8_t* packed, const float* sw4, const uint16_t* bias_bf16,
                           const int64_t* rows, int num_rows, int N, int K, float* y) {
  oracle_linear_w4_rows_act(q, sx, packed, sw4, bias_bf16, rows, num_rows, N, K, 0, y);
}

// ---- fp64 cross-check path (structurally different from the butterfly) -------
// Dense K x K rotation of one group, R = diag(d) . BlockDiag(H_128) / sqrt(128),
// with H built by the Sylvester recursion H_2n = [[H, H], [H, -H]].
void oracle_dense_rotation(const int8_t* signs, int K, double* R) {
  std::vector<double> H(kBlock * kBlock, 0.0);
  H[0] = 1.0;
  for (int n = 1; n < kBlock; n <<= 1)
    for (int i = 0; i < n; ++i)
      for (int j = 0; j < n; ++j) {
        const double h = H[i * kBlock + j];
        H[i * kBlock + (j + n)] = h;
        H[(i + n) * kBlock + j] = h;
        H[(i + n) * kBlock + (j + n)] = -h;
      }
  const double norm = 1.0 / std::sqrt(static_cast<double>(kBlock));
  for (int64_t i = 0; i < static_cast<int64_t>(K) * K; ++i) R[i] = 0.0;
  for (int c = 0; c < K; c += kBlock)
    for (int i = 0; i < kBlock; ++i)
      for (int j = 0; j < kBlock; ++j)
        R[static_cast<int64_t>(c + i) * K + (c + j)] = static_cast<double>(signs[c + i]) * H[i * kBlock + j] * norm;
}

// C[M,N] = A[M,K] . B[K,N], plain triple loop in double.
void oracle_matmul_f64(const double* A, const double* B, int M, int K, int N, double* C) {
#pragma omp parallel for schedule(static)
  for (int m = 0; m < M; ++m)
    for (int n = 0; n < N; ++n) {
      double s = 0.0;
      for (int k = 0; k < K; ++k) s += A[static_cast<int64_t>(m) * K + k] * B[static_cast<int64_t>(k) * N + n];
      C[static_cast<int64_t>(m) * N + n] = s;
    }
}

// Second-stage vector of one group: vec2[j] = fl32(d2[j] * 2^-3.5)  (d2 == nullptr means all +1).
void oracle_second_vector(const int8_t* signs2, int K, float* vec2) {
  for (int j = 0; j < K; ++j) vec2[j] = static_cast<float>((signs2 ? static_cast<double>(signs2[j]) : 1.0) * kHadamardNorm);
}

// Zigzag permutation (Sec. 3.2): channels sorted by magnitude, largest first, are dealt to the blocks in
// serpentine order -- round 0 fills slot 0 of blocks 0, 1, ..., B-1, round 1 fills slot 1 of blocks B-1, ..., 0,
// and so on -- so that no block collects only the largest or only the smallest channels.  Ties keep the
// lower channel index first.  perm[block * 128 + slot] = source channel.
void oracle_zigzag_permutation(const float* magnitude, int K, int32_t* perm) {
  const int blocks = K / kBlock;
  std::vector<int32_t> order(K);
  for (int j = 0; j < K; ++j) order[j] = j;
  // stable insertion-style ordering written out plainly (K is at most a few thousand)
  for (int i = 1; i < K; ++i) {
    const int32_t c = order[i];
    int j = i - 1;
    while (j >= 0 && magnitude[order[j]] < magnitude[c]) {
      order[j + 1] = order[j];
      --j;
    }
    order[j + 1] = c;
  }
  for (int round = 0; round < kBlock; ++round)
    for (int i = 0; i < blocks; ++i) {
      const int block = (round % 2 == 0) ? i : blocks - 1 - i;
      perm[block * kBlock + round] = order[round * blocks + i];
    }
}

// Rotated rows of the full transform in fp32 (no quantisation).
void oracle_rotate2(const uint16_t* x_bf16, int64_t ldx, int M, int K, const float* vec1, const int32_t* perm, const float* vec2,
                    float* v) {
#pragma omp parallel for schedule(static)
  for (int m = 0; m < M; ++m) rotate2_row(x_bf16 + static_cast<int64_t>(m) * ldx, vec1, perm, vec2, K, v + static_cast<int64_t>(m) * K);
}

// Full transform followed by the per-row symmetric int8 quantiser (activations, or 8-bit weights per output channel).
void oracle_rotate2_quantize(const uint16_t* x_bf16, int64_t ldx, int M, int K, const float* vec1, const int32_t* perm,
                             const float* vec2, int8_t* codes, float* scales) {
#pragma omp parallel for schedule(static)
  for (int m = 0; m < M; ++m) {
    std::vector<float> v(K);
    rotate2_row(x_bf16 + static_cast<int64_t>(m) * ldx, vec1, perm, vec2, K, v.data());
    scales[m] = quantize_span(v.data(), K, 127.0f, codes + static_cast<int64_t>(m) * K);
  }
}

// Full transform of the weight rows followed by the 4-bit quantiser (one scale per 128 consecutive k).
void oracle_prepare2_w4(const uint16_t* w_bf16, int N, int K, const float* vec1, const int32_t* perm, const float* vec2,
                        uint8_t* packed, float* scales) {
  const int groups = K / kBlock;
#pragma omp parallel for schedule(static)
  for (int n = 0; n < N; ++n) {
    std::vector<float> v(K);
    rotate2_row(w_bf16 + static_cast<int64_t>(n) * K, vec1, perm, vec2, K, v.data());
    for (int kg = 0; kg < groups; ++kg) {
      int8_t q[kBlock];
      scales[static_cast<int64_t>(n) * groups + kg] = quantize_span(v.data() + kg * kBlock, kBlock, 7.0f, q);
      for (int i = 0; i < kBlock; i += 2) {
        const uint8_t lo = static_cast<uint8_t>(q[i]) & 0xF;
        const uint8_t hi = static_cast<uint8_t>(q[i + 1]) & 0xF;
        packed[(static_cast<int64_t>(n) * K + kg * kBlock + i) / 2] = static_cast<uint8_t>(lo | (hi << 4));
      }
    }
  }
}

// Dense K x K permutation matrix of an index vector, P[perm[j]][j] = 1 (fp64 cross-check path).
void oracle_dense_permutation(const int32_t* perm, int K, double* P) {
  for (int64_t i = 0; i < static_cast<int64_t>(K) * K; ++i) P[i] = 0.0;
  for (int j = 0; j < K; ++j) P[static_cast<int64_t>(perm[j]) * K + j] = 1.0;
}

// ---- literal asymmetric activations (Eq. 1-3) ------------------------------------------------------------
// Per-row asymmetric quantiser on already-rotated fp32 rows.
void oracle_quantize_rows_asym(const float* v, int M, int K, uint8_t* codes, float* scales, int32_t* zero_points) {
#pragma omp parallel for schedule(static)
  for (int m = 0; m < M; ++m)
    scales[m] = quantize_span_asym(v + static_cast<int64_t>(m) * K, K, codes + static_cast<int64_t>(m) * K, zero_points + m);
}

// Rotate (single block rotation, as oracle_rotate_quantize) then quantise each token with its own min / max.
void oracle_rotate_quantize_asym(const uint16_t* x_bf16, int64_t ldx, int M, int K, const float* act_vec, uint8_t* codes,
                                 float* scales, int32_t* zero_points) {
#pragma omp parallel for schedule(static)
  for (int m = 0; m < M; ++m) {
    std::vector<float> v(K);
    rotate_row(x_bf16 + static_cast<int64_t>(m) * ldx, act_vec, K, v.data());
    scales[m] = quantize_span_asym(v.data(), K, codes + static_cast<int64_t>(m) * K, zero_points + m);
  }
}

// Linear layer on asymmetric activation codes and symmetric per-channel weights, row subset:
//   y = sx[m] * sw[n] * sum_k (q[m,k] - z[m]) * qw[n,k] + bias[n]      (integer sum exact; the rest in double, rounded once)
void oracle_linear_asym_rows(const uint8_t* q, const float* sx, const int32_t* z, const int8_t* qw, const float* sw,
                             const uint16_t* bias_bf16, const int64_t* rows, int num_rows, int N, int K, float* y) {
#pragma omp parallel for schedule(static)
  for (int i = 0; i < num_rows; ++i) {
    const int64_t m = rows[i];
    for (int n = 0; n < N; ++n) {
      int64_t s = 0;
      for (int k = 0; k < K; ++k)
        s += (static_cast<int64_t>(q[m * K + k]) - z[m]) * static_cast<int64_t>(qw[static_cast<int64_t>(n) * K + k]);
      double r = static_cast<double>(s) * static_cast<double>(sx[m]) * static_cast<double>(sw[n]);
      if (bias_bf16) r += static_cast<double>(bf16_to_float(bias_bf16[n]));
      y[static_cast<int64_t>(i) * N + n] = static_cast<float>(r);
    }
  }
}

// ---- dense block rotations (Sec. 3.2, Eq. 6-8) -----------------------------------------------------------
// Eq. 8: R = BlockDiag(R_b1 .. R_bK), every block a dense 128 x 128 orthogonal matrix (a greedy product of
// Eq. 6 factors, built offline).  Online side of Eq. 10 with such blocks: v = (x o Delta) . R per block.
// The smoothing vector is folded into the rows of each block and the result is STORED IN BF16 (the format
// the matrix is applied in):  S_b[i][j] = bf16_rne(Delta[128 b + i] * R_b[i][j]).  Because S is what is
// applied to the activations, the weight side uses the exact inverse of S (not R^T Delta^-1), so the
// identity (X S)(S^-1 W) = X W of Eq. 9 holds whatever the rounding did.  The storage precision is a
// convention of this implementation ("parity unpinned" by the paper, which does not say how R is held).

// Round a double to the nearest bf16 (8 significand bits), ties to even; returns the bf16 bit pattern.
static uint16_t double_to_bf16_bits(double p) {
  if (p == 0.0) return 0;
  int e = 0;
  const double m = std::frexp(p, &e);                  // |m| in [0.5, 1)
  const double r = std::nearbyint(std::ldexp(m, 8));    // |r| in [128, 256], integer, ties to even
  const float f = static_cast<float>(std::ldexp(r, e - 8));  // exact: r has at most 9 bits
  uint32_t u;
  std::memcpy(&u, &f, sizeof u);
  return static_cast<uint16_t>(u >> 16);
}

// stored[b][i][j] = bf16(Delta[128 b + i] * blocks[b][i][j]); smooth == nullptr means Delta = 1.
void oracle_dense_stored_blocks(const float* blocks, const float* smooth, int K, uint16_t* stored) {
  const int nb = K / kBlock;
  for (int b = 0; b < nb; ++b)
    for (int i = 0; i < kBlock; ++i) {
      const double delta = smooth ? static_cast<double>(smooth[b * kBlock + i]) : 1.0;
      for (int j = 0; j < kBlock; ++j) {
        const int64_t at = (static_cast<int64_t>(b) * kBlock + i) * kBlock + j;
        stored[at] = double_to_bf16_bits(delta * static_cast<double>(blocks[at]));  // product of two floats: exact in double
      }
    }
}

// v[m, 128 b + j] = fl32( sum_i x[m, 128 b + i] * S_b[i][j] ), the sum taken in double in index order
// (every product of two bf16 values is exact).
void oracle_rotate_dense(const uint16_t* x_bf16, int64_t ldx, int M, int K, const uint16_t* stored, float* v) {
  const int nb = K / kBlock;
#pragma omp parallel for schedule(static)
  for (int m = 0; m < M; ++m)
    for (int b = 0; b < nb; ++b)
      for (int j = 0; j < kBlock; ++j) {
        double s = 0.0;
        for (int i = 0; i < kBlock; ++i)
          s += static_cast<double>(bf16_to_float(x_bf16[m * ldx + b * kBlock + i])) *
               static_cast<double>(bf16_to_float(stored[(static_cast<int64_t>(b) * kBlock + i) * kBlock + j]));
        v[static_cast<int64_t>(m) * K + b * kBlock + j] = static_cast<float>(s);
      }
}

// inv[b] = S_b^-1 in double: Gauss-Jordan elimination with partial pivoting on [S | I].
// Returns 0, or 1 + the index of the first singular block.
int oracle_invert_blocks(const uint16_t* stored, int nb, double* inv) {
  const int n = kBlock;
  for (int b = 0; b < nb; ++b) {
    std::vector<double> a(static_cast<size_t>(n) * n);
    double* x = inv + static_cast<int64_t>(b) * n * n;
    for (int i = 0; i < n; ++i)
      for (int j = 0; j < n; ++j) {
        a[i * n + j] = static_cast<double>(bf16_to_float(stored[(static_cast<int64_t>(b) * n + i) * n + j]));
        x[i * n + j] = i == j ? 1.0 : 0.0;
      }
    for (int c = 0; c < n; ++c) {
      int piv = c;
      for (int r = c + 1; r < n; ++r)
        if (std::fabs(a[r * n + c]) > std::fabs(a[piv * n + c])) piv = r;
      if (a[piv * n + c] == 0.0) return b + 1;
      if (piv != c)
        for (int j = 0; j < n; ++j) {
          std::swap(a[c * n + j], a[piv * n + j]);
          std::swap(x[c * n + j], x[piv * n + j]);
        }
      const double d = a[c * n + c];
      for (int j = 0; j < n; ++j) {
        a[c * n + j] /= d;
        x[c * n + j] /= d;
      }
      for (int r = 0; r < n; ++r) {
        if (r == c) continue;
        const double f = a[r * n + c];
        if (f == 0.0) continue;
        for (int j = 0; j < n; ++j) {
          a[r * n + j] -= f * a[c * n + j];
          x[r * n + j] -= f * x[c * n + j];
        }
      }
    }
  }
  return 0;
}

// Weight side of Eq. 10 with dense blocks: wr[n, 128 b + j] = fl32( sum_i inv_b[j][i] * W[n, 128 b + i] ),
// i.e. the column vector S_b^-1 w; products and sums in double, in index order, each rounded separately.
void oracle_prepare_dense_rotate(const uint16_t* w_bf16, int N, int K, const double* inv, float* wr) {
  const int nb = K / kBlock;
#pragma omp parallel for schedule(static)
  for (int n = 0; n < N; ++n)
    for (int b = 0; b < nb; ++b)
      for (int j = 0; j < kBlock; ++j) {
        double s = 0.0;
        for (int i = 0; i < kBlock; ++i)
          s += inv[(static_cast<int64_t>(b) * kBlock + j) * kBlock + i] *
               static_cast<double>(bf16_to_float(w_bf16[static_cast<int64_t>(n) * K + b * kBlock + i]));
        wr[static_cast<int64_t>(n) * K + b * kBlock + j] = static_cast<float>(s);
      }
}

// 4-bit quantiser on already-rotated fp32 weight rows (same format as oracle_prepare_w4).
void oracle_quantize_w4_rows(const float* wr, int N, int K, uint8_t* packed, float* scales) {
  const int groups = K / kBlock;
#pragma omp parallel for schedule(static)
  for (int n = 0; n < N; ++n)
    for (int kg = 0; kg < groups; ++kg) {
      int8_t q[kBlock];
      scales[static_cast<int64_t>(n) * groups + kg] = quantize_span(wr + static_cast<int64_t>(n) * K + kg * kBlock, kBlock, 7.0f, q);
      for (int i = 0; i < kBlock; i += 2) {
        const uint8_t lo = static_cast<uint8_t>(q[i]) & 0xF;
        const uint8_t hi = static_cast<uint8_t>(q[i + 1]) & 0xF;
        packed[(static_cast<int64_t>(n) * K + kg * kBlock + i) / 2] = static_cast<uint8_t>(lo | (hi << 4));
      }
    }
}

// ---- greedy construction of one block (Sec. 3.2, Eq. 6-7) ------------------------------------------------
// Eq. 6: R^k = C1 Q C2.  C1 swaps the first column with the column holding the largest-magnitude entry of the
// current activations; Q is a random orthogonal matrix whose first row is uniform (every entry 1/sqrt(128)),
// so the outlier now sitting in position 0 is spread evenly over all outputs; C2 swaps the two columns back.
// The random part of Q is an input: a Gaussian draw G per step.  Row 0 of Q is the uniform row, rows 1..127
// are G's rows 1..127 made orthonormal to all earlier rows by modified Gram-Schmidt.
static void uniform_first_row_orthogonal(const double* G, double* Q) {
  const int n = kBlock;
  for (int j = 0; j < n; ++j) Q[j] = 1.0 / std::sqrt(static_cast<double>(n));
  for (int r = 1; r < n; ++r) {
    double* q = Q + r * n;
    for (int j = 0; j < n; ++j) q[j] = G[r * n + j];
    for (int s = 0; s < r; ++s) {
      double dot = 0.0;
      for (int j = 0; j < n; ++j) dot += q[j] * Q[s * n + j];
      for (int j = 0; j < n; ++j) q[j] -= dot * Q[s * n + j];
    }
    double nrm = 0.0;
    for (int j = 0; j < n; ++j) nrm += q[j] * q[j];
    nrm = std::sqrt(nrm);
    for (int j = 0; j < n; ++j) q[j] /= nrm;
  }
}

// Eq. 7: R = R^1 R^2 ... R^n with n = argmin_k max_ij |(X R^1 ... R^k)_ij| over k = 1..steps (the first k
// reaching the minimum).  Xc: calibration activations of this block [Mc, 128]; gauss: [steps][128][128].
// Outputs the product R [128][128], the per-step maxima trace[steps], and returns n.
int oracle_greedy_block(const double* Xc, int Mc, int steps, const double* gauss, double* R, double* trace) {
  const int n = kBlock;
  std::vector<double> Y(Xc, Xc + static_cast<size_t>(Mc) * n), Yn(static_cast<size_t>(Mc) * n);
  std::vector<double> P(static_cast<size_t>(n) * n, 0.0), Pn(static_cast<size_t>(n) * n), Q(static_cast<size_t>(n) * n), Rk(static_cast<size_t>(n) * n);
  for (int i = 0; i < n; ++i) P[i * n + i] = 1.0;
  int best_k = 0;
  double best = 0.0;
  for (int k = 1; k <= steps; ++k) {
    int d = 0;
    double mx = -1.0;
    for (int m = 0; m < Mc; ++m)
      for (int j = 0; j < n; ++j)
        if (std::fabs(Y[static_cast<size_t>(m) * n + j]) > mx) {
          mx = std::fabs(Y[static_cast<size_t>(m) * n + j]);
          d = j;
        }
    uniform_first_row_orthogonal(gauss + static_cast<size_t>(k - 1) * n * n, Q.data());
    // (C1 Q C2)[i][j] = Q[s(i)][s(j)] with s the transposition of 0 and d
    for (int i = 0; i < n; ++i) {
      const int si = i == 0 ? d : (i == d ? 0 : i);
      for (int j = 0; j < n; ++j) {
        const int sj = j == 0 ? d : (j == d ? 0 : j);
        Rk[i * n + j] = Q[si * n + sj];
      }
    }
    for (int m = 0; m < Mc; ++m)
      for (int j = 0; j < n; ++j) {
        double s = 0.0;
        for (int i = 0; i < n; ++i) s += Y[static_cast<size_t>(m) * n + i] * Rk[i * n + j];
        Yn[static_cast<size_t>(m) * n + j] = s;
      }
    Y.swap(Yn);
    for (int a = 0; a < n; ++a)
      for (int j = 0; j < n; ++j) {
        double s = 0.0;
        for (int i = 0; i < n; ++i) s += P[a * n + i] * Rk[i * n + j];
        Pn[a * n + j] = s;
      }
    P.swap(Pn);
    double now = 0.0;
    for (size_t i = 0; i < Y.size(); ++i) now = std::fmax(now, std::fabs(Y[i]));
    trace[k - 1] = now;
    if (best_k == 0 || now < best) {
      best = now;
      best_k = k;
      std::memcpy(R, P.data(), sizeof(double) * n * n);
    }
  }
  return best_k;
}

// ---- normalisation and modulation folded in front of the rotation ------------------------------------------
// The quantized linears of a DiT block read a LayerNorm output modulated per sample (adaLN):
//   h[m, k] = (x[m, k] - mean_m) / sqrt(var_m + eps) * (1 + scale[s, k]) + shift[s, k],   s = m / rows_per_sample,
// mean and (biased) variance over the row's K channels.  Evaluated in double and rounded once to fp32; h then takes the
// place of the bf16 input of the rotation (oracle_rotate_f32).  scale / shift may be null (zero).  The paper does not
// discuss normalisation; this backs the fused variant of the online call.
void oracle_norm_modulate(const uint16_t* x_bf16, int64_t ldx, int M, int K, const uint16_t* shift_bf16, const uint16_t* scale_bf16,
                          int rows_per_sample, double eps, float* h) {
#pragma omp parallel for schedule(static)
  for (int m = 0; m < M; ++m) {
    const uint16_t* row = x_bf16 + static_cast<int64_t>(m) * ldx;
    double mean = 0.0;
    for (int k = 0; k < K; ++k) mean += static_cast<double>(bf16_to_float(row[k]));
    mean /= K;
    double var = 0.0;
    for (int k = 0; k < K; ++k) {
      const double d = static_cast<double>(bf16_to_float(row[k])) - mean;
      var += d * d;
    }
    var /= K;
    const double rstd = 1.0 / std::sqrt(var + eps);
    const int64_t s = m / rows_per_sample;
    for (int k = 0; k < K; ++k) {
      const double sc = scale_bf16 ? static_cast<double>(bf16_to_float(scale_bf16[s * K + k])) : 0.0;
      const double sh = shift_bf16 ? static_cast<double>(bf16_to_float(shift_bf16[s * K + k])) : 0.0;
      h[static_cast<int64_t>(m) * K + k] = static_cast<float>((static_cast<double>(bf16_to_float(row[k])) - mean) * rstd * (1.0 + sc) + sh);
    }
  }
}

// The block rotation of oracle_rotate on fp32 rows: u = fl32(h * vec), then the butterfly.
void oracle_rotate_f32(const float* h, int M, int K, const float* vec, float* v) {
#pragma omp parallel for schedule(static)
  for (int m = 0; m < M; ++m)
    for (int c = 0; c < K; c += kBlock) {
      float u[kBlock];
      for (int i = 0; i < kBlock; ++i) u[i] = h[static_cast<int64_t>(m) * K + c + i] * vec[c + i];
      butterfly128(u);
      for (int i = 0; i < kBlock; ++i) v[static_cast<int64_t>(m) * K + c + i] = u[i];
    }
}

int oracle_num_threads() {
  int n = 1;
#ifdef _OPENMP
#pragma omp parallel
  {
#pragma omp single
    n = omp_get_num_threads();
  }
#endif
  return n;
}

}  // extern "C"
