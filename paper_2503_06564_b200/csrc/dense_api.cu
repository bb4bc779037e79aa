// Host side of the dense block rotations (Sec. 3.2, Eq. 6-8): storing the blocks in the format they are
// applied in, inverting them for the weight side, the greedy construction of a block from calibration
// activations, and the entry points of the online call.
#include <cmath>
#include <cstring>
#include <new>
#include <vector>

#include "internal.h"

namespace {

constexpr int kB = TRDQ_BLOCK;

// Nearest bf16 (8 significand bits, ties to even) of a double, by integer arithmetic on its bit pattern.
// Returns false for a non-finite value or one beyond the bf16 range; magnitudes below 2^-126 become zero.
bool round_to_bf16(double v, uint16_t* out) {
  uint64_t u;
  std::memcpy(&u, &v, sizeof u);
  const uint16_t sign = static_cast<uint16_t>((u >> 63) << 15);
  const int e = static_cast<int>((u >> 52) & 0x7FF);
  const uint64_t frac = u & ((1ull << 52) - 1);
  if (e == 0x7FF) return false;
  if (e == 0) {
    *out = sign;
    return true;
  }
  int e32 = e - 1023 + 127;
  uint64_t keep = frac >> 45;  // the 7 stored fraction bits
  const uint64_t rest = frac & ((1ull << 45) - 1), half = 1ull << 44;
  if (rest > half || (rest == half && (keep & 1))) ++keep;
  if (keep == 128) {
    keep = 0;
    ++e32;
  }
  if (e32 >= 255) return false;
  if (e32 <= 0) {
    *out = sign;
    return true;
  }
  *out = static_cast<uint16_t>(sign | (e32 << 7) | keep);
  return true;
}

double bf16_value(uint16_t b) {
  const uint32_t u = static_cast<uint32_t>(b) << 16;
  float f;
  std::memcpy(&f, &u, sizeof f);
  return static_cast<double>(f);
}

// Inverse of one 128 x 128 matrix (row-major) by elimination on the augmented rows [A | I] with row pivoting.
bool invert_block(const double* A, double* inv) {
  const int n = kB, w = 2 * kB;
  std::vector<double> aug(static_cast<size_t>(n) * w, 0.0);
  for (int r = 0; r < n; ++r) {
    std::memcpy(&aug[static_cast<size_t>(r) * w], A + static_cast<size_t>(r) * n, sizeof(double) * n);
    aug[static_cast<size_t>(r) * w + n + r] = 1.0;
  }
  for (int col = 0; col < n; ++col) {
    int best = col;
    for (int r = col + 1; r < n; ++r)
      if (std::fabs(aug[static_cast<size_t>(r) * w + col]) > std::fabs(aug[static_cast<size_t>(best) * w + col])) best = r;
    if (aug[static_cast<size_t>(best) * w + col] == 0.0) return false;
    if (best != col)
      for (int j = 0; j < w; ++j) std::swap(aug[static_cast<size_t>(best) * w + j], aug[static_cast<size_t>(col) * w + j]);
    double* prow = &aug[static_cast<size_t>(col) * w];
    const double pivot = prow[col];
    for (int j = 0; j < w; ++j) prow[j] /= pivot;
    for (int r = 0; r < n; ++r) {
      if (r == col) continue;
      double* row = &aug[static_cast<size_t>(r) * w];
      const double f = row[col];
      if (f == 0.0) continue;
      for (int j = 0; j < w; ++j) row[j] -= f * prow[j];
    }
  }
  for (int r = 0; r < n; ++r) std::memcpy(inv + static_cast<size_t>(r) * n, &aug[static_cast<size_t>(r) * w + n], sizeof(double) * n);
  return true;
}

}  // namespace

using namespace trdq;

extern "C" {

trdq_status trdq_rotation_create_dense(int32_t K, int32_t num_groups, const int32_t* t_bounds, const float* blocks, const float* smooth,
                                       trdq_rotation** out) {
  if (!t_bounds || !blocks || !out) return TRDQ_ERR_NULL;
  if (K <= 0 || K % kB != 0 || K > TRDQ_MAX_K) return TRDQ_ERR_SHAPE;
  if (num_groups < 1) return TRDQ_ERR_GROUP;
  for (int g = 0; g < num_groups; ++g)
    if (t_bounds[g] >= t_bounds[g + 1]) return TRDQ_ERR_GROUP;
  const int nb = K / kB;
  const size_t per_group = static_cast<size_t>(nb) * kB * kB;
  const size_t total = per_group * num_groups;
  if (smooth)
    for (size_t i = 0; i < static_cast<size_t>(num_groups) * K; ++i)
      if (!(smooth[i] > 0.0f && std::isfinite(smooth[i]))) return TRDQ_ERR_GROUP;

  // S_b[i][j] = bf16(Delta[128 b + i] * R_b[i][j]) (the product of two floats is exact in double), kept transposed;
  // inv_t[i][j] = (S_b^-1)[j][i]
  std::vector<uint16_t> stored_t(total);
  std::vector<double> inv_t(total), S(static_cast<size_t>(kB) * kB), inv(static_cast<size_t>(kB) * kB);
  for (int g = 0; g < num_groups; ++g)
    for (int b = 0; b < nb; ++b) {
      const size_t base = static_cast<size_t>(g) * per_group + static_cast<size_t>(b) * kB * kB;
      for (int i = 0; i < kB; ++i) {
        const double delta = smooth ? static_cast<double>(smooth[static_cast<size_t>(g) * K + b * kB + i]) : 1.0;
        for (int j = 0; j < kB; ++j) {
          uint16_t bits;
          if (!round_to_bf16(delta * static_cast<double>(blocks[base + static_cast<size_t>(i) * kB + j]), &bits)) return TRDQ_ERR_GROUP;
          stored_t[base + static_cast<size_t>(j) * kB + i] = bits;
          S[static_cast<size_t>(i) * kB + j] = bf16_value(bits);
        }
      }
      if (!invert_block(S.data(), inv.data())) return TRDQ_ERR_GROUP;  // singular block
      for (int i = 0; i < kB; ++i)
        for (int j = 0; j < kB; ++j) inv_t[base + static_cast<size_t>(i) * kB + j] = inv[static_cast<size_t>(j) * kB + i];
    }

  trdq_rotation* rot = new (std::nothrow) trdq_rotation;
  if (!rot) return TRDQ_ERR_NOMEM;
  rot->K = K;
  rot->num_groups = num_groups;
  rot->t_bounds.assign(t_bounds, t_bounds + num_groups + 1);
  if (cudaGetDevice(&rot->device) != cudaSuccess) {
    delete rot;
    return TRDQ_ERR_CUDA;
  }
  if (cudaMalloc(&rot->dense, total * sizeof(uint16_t)) != cudaSuccess || cudaMalloc(&rot->dense_inv_t, total * sizeof(double)) != cudaSuccess) {
    cudaGetLastError();
    trdq_rotation_destroy(rot);
    return TRDQ_ERR_NOMEM;
  }
  if (cudaMemcpy(rot->dense, stored_t.data(), total * sizeof(uint16_t), cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(rot->dense_inv_t, inv_t.data(), total * sizeof(double), cudaMemcpyHostToDevice) != cudaSuccess) {
    trdq_rotation_destroy(rot);
    return TRDQ_ERR_CUDA;
  }
  const trdq_status st = encode_tmap_2d(&rot->tmap_dense, rot->dense, 2, kB, static_cast<uint64_t>(num_groups) * nb * kB, kB * 2, 64, 128, 128);
  if (st != TRDQ_OK) {
    trdq_rotation_destroy(rot);
    return st;
  }
  *out = rot;
  return TRDQ_OK;
}

trdq_status trdq_rotate_dense_workspace(const trdq_rotation* rot, int32_t M, uint64_t* bytes) {
  if (!rot || !bytes) return TRDQ_ERR_NULL;
  if (!rot->dense) return TRDQ_ERR_MISMATCH;
  if (M < 0) return TRDQ_ERR_SHAPE;
  *bytes = rotate_dense_workspace_bytes(M, rot->K);
  return TRDQ_OK;
}

trdq_status trdq_rotate_dense_quantize(const trdq_rotation* rot, int32_t t, const void* X_bf16, int64_t ldx, int32_t M, int8_t* codes,
                                       float* scales, void* workspace, uint64_t workspace_bytes, void* stream) {
  if (!rot) return TRDQ_ERR_NULL;
  if (!rot->dense) return TRDQ_ERR_MISMATCH;
  if (M < 0) return TRDQ_ERR_SHAPE;
  int32_t g = -1;
  const trdq_status sg = trdq_group_of(rot, t, &g);
  if (sg != TRDQ_OK) return sg;
  if (M == 0) return TRDQ_OK;
  if (!X_bf16 || !codes || !scales || !workspace) return TRDQ_ERR_NULL;
  if (ldx < rot->K) return TRDQ_ERR_SHAPE;
  const auto misaligned = [](const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) != 0; };
  if (ldx % 8 != 0 || misaligned(X_bf16, 16) || misaligned(codes, 16) || misaligned(scales, 4) || misaligned(workspace, 4)) return TRDQ_ERR_ALIGN;
  if (workspace_bytes < rotate_dense_workspace_bytes(M, rot->K)) return TRDQ_ERR_NOMEM;
  return trdq::finish(launch_rotate_dense_quantize(rot, g, X_bf16, ldx, M, codes, scales, static_cast<float*>(workspace), static_cast<cudaStream_t>(stream)),
                      stream);
}

// Eq. 6-7 for one block, on the host in double.  Step k: d = column of the largest |Y| (Y = X R^1 .. R^(k-1), first
// such column in row-major order); Q_k = the orthogonal matrix whose first row is uniform (1/sqrt(128)) and whose
// other rows are the Gaussian rows made orthonormal one after the other; R^k = C Q_k C with C the swap of columns 0
// and d.  The product up to the step with the smallest max |Y| is returned.
trdq_status trdq_greedy_rotation_block(const float* x_calib, int32_t rows, int32_t steps, const double* gauss, float* R_out, int32_t* n_used) {
  if (!x_calib || !gauss || !R_out) return TRDQ_ERR_NULL;
  if (rows <= 0 || steps <= 0) return TRDQ_ERR_SHAPE;
  const int n = kB;
  const size_t nn = static_cast<size_t>(n) * n;
  std::vector<double> Y(static_cast<size_t>(rows) * n), Ynext(Y.size()), prod(nn, 0.0), prod_next(nn), Q(nn), best_prod(nn);
  for (size_t i = 0; i < Y.size(); ++i) {
    if (!std::isfinite(x_calib[i])) return TRDQ_ERR_GROUP;
    Y[i] = static_cast<double>(x_calib[i]);
  }
  for (int i = 0; i < n; ++i) prod[static_cast<size_t>(i) * n + i] = 1.0;
  const double uniform = 1.0 / std::sqrt(static_cast<double>(n));
  std::vector<int> swap_of(n);
  double best_max = 0.0;
  int best_step = 0;
  for (int step = 1; step <= steps; ++step) {
    // column of the outlier
    int d = 0;
    double seen = -1.0;
    for (int m = 0; m < rows; ++m)
      for (int j = 0; j < n; ++j) {
        const double a = std::fabs(Y[static_cast<size_t>(m) * n + j]);
        if (a > seen) {
          seen = a;
          d = j;
        }
      }
    // Q: uniform first row, then Gram-Schmidt (each row against all rows before it, one at a time)
    const double* G = gauss + static_cast<size_t>(step - 1) * nn;
    for (int j = 0; j < n; ++j) Q[j] = uniform;
    for (int r = 1; r < n; ++r) {
      double* q = &Q[static_cast<size_t>(r) * n];
      for (int j = 0; j < n; ++j) q[j] = G[static_cast<size_t>(r) * n + j];
      for (int s = 0; s < r; ++s) {
        const double* e = &Q[static_cast<size_t>(s) * n];
        double dot = 0.0;
        for (int j = 0; j < n; ++j) dot += q[j] * e[j];
        for (int j = 0; j < n; ++j) q[j] -= dot * e[j];
      }
      double len = 0.0;
      for (int j = 0; j < n; ++j) len += q[j] * q[j];
      len = std::sqrt(len);
      if (!(len > 0.0) || !std::isfinite(len)) return TRDQ_ERR_GROUP;
      for (int j = 0; j < n; ++j) q[j] /= len;
    }
    // (C Q C)[i][j] = Q[swap(i)][swap(j)]
    for (int i = 0; i < n; ++i) swap_of[i] = i;
    swap_of[0] = d;
    swap_of[d] = 0;
    for (int m = 0; m < rows; ++m)
      for (int j = 0; j < n; ++j) {
        double s = 0.0;
        for (int i = 0; i < n; ++i) s += Y[static_cast<size_t>(m) * n + i] * Q[static_cast<size_t>(swap_of[i]) * n + swap_of[j]];
        Ynext[static_cast<size_t>(m) * n + j] = s;
      }
    Y.swap(Ynext);
    for (int a = 0; a < n; ++a)
      for (int j = 0; j < n; ++j) {
        double s = 0.0;
        for (int i = 0; i < n; ++i) s += prod[static_cast<size_t>(a) * n + i] * Q[static_cast<size_t>(swap_of[i]) * n + swap_of[j]];
        prod_next[static_cast<size_t>(a) * n + j] = s;
      }
    prod.swap(prod_next);
    double now = 0.0;
    for (size_t i = 0; i < Y.size(); ++i) now = std::fmax(now, std::fabs(Y[i]));
    if (best_step == 0 || now < best_max) {
      best_max = now;
      best_step = step;
      best_prod = prod;
    }
  }
  for (size_t i = 0; i < nn; ++i) R_out[i] = static_cast<float>(best_prod[i]);
  if (n_used) *n_used = best_step;
  return TRDQ_OK;
}

}  // extern "C"
