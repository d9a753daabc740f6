// Ridge penalty per expert by marginal likelihood (App. Calibration Details): for every candidate
// lambda the evidence of the centred ridge model needs log det(G_c + lambda I) and the quadratic form
// q_c^T (G_c + lambda I)^-1 q_c. Both come out of one Cholesky factorisation G_c + lambda I = L L^T:
// log det = 2 sum log L_ii, and with w = L^-1 q_c the quadratic form is |w|^2. (The paper takes one
// eigendecomposition per expert and evaluates all penalties from it; a factorisation per penalty gives
// the same numbers, is exact for repeated and zero eigenvalues, and needs no eigen-solver on the
// device.) One CTA per expert, fp64 throughout, the matrix in a global scratch square of d x d
// doubles per expert. Included by calib.cu.
#pragma once

namespace base {

namespace {

constexpr int kEvThreads = 512;
constexpr int kEvNb = 32;      // panel width
constexpr int kEvTile = 64;    // trailing-update tile

struct LambdaGrid {
  double v[kCalibMaxLambdas];
  int n;
  int default_index;   // for experts with fewer than two pairs
};

// Cholesky of the 32 x 32 diagonal block held in shared memory (row stride 33), by one warp; lane = row.
// Returns the sum of log L_jj over the block through *logsum (lane 0) and clears *ok on a pivot <= 0.
__device__ __forceinline__ void ev_factor_diag(double (*D)[kEvNb + 1], int lane, double* logsum, int* ok) {
  double ls = 0.0;
  for (int j = 0; j < kEvNb; ++j) {
    double djj = D[j][j];
    if (!(djj > 0.0)) {
      if (lane == 0) *ok = 0;
      djj = 1.0;
    }
    djj = sqrt(djj);
    ls += log(djj);
    __syncwarp();
    double lij = 0.0;
    if (lane == j) D[j][j] = djj;
    if (lane > j) {
      lij = D[lane][j] / djj;
      D[lane][j] = lij;
    }
    __syncwarp();
    if (lane > j)
      for (int c = j + 1; c <= lane; ++c) D[lane][c] -= lij * D[c][j];
    __syncwarp();
  }
  if (lane == 0) *logsum += ls;
}

__global__ void __launch_bounds__(kEvThreads) calib_evidence_kernel(CalibState st, double* __restrict__ chol, int d,
                                                                    LambdaGrid grid) {
  extern __shared__ double s_ev[];
  double* m = s_ev;                 // [d] mean of the inputs
  double* qc = m + d;               // [d] centred cross-moment
  double* w = qc + d;               // [d] running right-hand side of the forward solve
  double* At = w + d;               // [kEvNb][kEvTile] panel rows of the tile's row block, transposed
  double* Bt = At + kEvNb * kEvTile;   // [kEvNb][2 * kEvTile] ... of its column block (128 columns)
  __shared__ double D[kEvNb][kEvNb + 1];
  __shared__ double s_logsum;
  __shared__ int s_pd, s_best;
  const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const double n = st.n[u];
  double* ev_out = st.evidence + size_t(u) * kCalibMaxLambdas;
  if (n < 2.0) {
    // nothing to judge by, and nothing to fit: a = 0, b = the one target (0 without a pair)
    if (tid == 0) {
      st.lambda_index[u] = grid.default_index;
      st.lambda[u] = grid.v[grid.default_index];
      st.coef_b[u] = n >= 1.0 ? st.sum_y[u] / n : 0.0;
      st.iters[u] = 0;
    }
    for (int i = tid; i < kCalibMaxLambdas; i += kEvThreads) ev_out[i] = 0.0;
    for (int j = tid; j < d; j += kEvThreads) st.coef_a[size_t(u) * d + j] = 0.0;
    return;
  }
  const double sy = st.sum_y[u];
  for (int j = tid; j < d; j += kEvThreads) {
    const double mj = st.sum_z[size_t(u) * d + j] / n;
    m[j] = mj;
    qc[j] = st.sum_yz[size_t(u) * d + j] - sy * mj;
  }
  __syncthreads();
  const double yy = st.sum_yy[u] - sy * sy / n;
  const double r_floor = 1e-12 * yy + 1e-300;
  const float* G = st.gram + size_t(u) * d * d;
  double* A = chol + size_t(u) * d * d;
  double best = 0.0;
  int best_i = -1;

  // passes 0 .. n-1: the evidence of every candidate; pass n: the chosen candidate once more, this time
  // keeping the factor, for the ridge solution a = L^-T (L^-1 q_c)
  for (int pass = 0; pass <= grid.n; ++pass) {
    const bool last = pass == grid.n;
    const int li = last ? s_best : pass;
    const double lam = grid.v[li];
    // ---- A (lower triangle) = G - n m m^T + lambda I
    for (int i = warp; i < d; i += kEvThreads / 32) {
      const double nmi = n * m[i];
      for (int j = lane; j <= i; j += 32)
        A[size_t(i) * d + j] = double(G[size_t(i) * d + j]) - nmi * m[j] + (i == j ? lam : 0.0);
    }
    for (int j = tid; j < d; j += kEvThreads) w[j] = qc[j];
    if (tid == 0) {
      s_logsum = 0.0;
      s_pd = 1;
    }
    __syncthreads();
    double wnorm2 = 0.0;   // accumulated by warp 0 / lane 0 only

    for (int k0 = 0; k0 < d; k0 += kEvNb) {
      // ---- diagonal block: factor, then the block's part of w = L^-1 q
      for (int idx = tid; idx < kEvNb * kEvNb; idx += kEvThreads) {
        const int i = idx >> 5, j = idx & 31;
        D[i][j] = j <= i ? A[size_t(k0 + i) * d + k0 + j] : 0.0;
      }
      __syncthreads();
      if (warp == 0) {
        ev_factor_diag(D, lane, &s_logsum, &s_pd);
        for (int j = 0; j < kEvNb; ++j) {
          const double wj = w[k0 + j] / D[j][j];
          __syncwarp();
          if (lane == j) w[k0 + j] = wj;
          if (lane > j) w[k0 + lane] -= D[lane][j] * wj;
          __syncwarp();
        }
        const double wl = w[k0 + lane];
        double s2 = wl * wl;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s2 += __shfl_down_sync(0xffffffffu, s2, o);
        wnorm2 += s2;
      }
      __syncthreads();
      if (last) {   // the back substitution reads the factor from the scratch matrix
        for (int idx = tid; idx < kEvNb * kEvNb; idx += kEvThreads) {
          const int i = idx >> 5, j = idx & 31;
          if (j <= i) A[size_t(k0 + i) * d + k0 + j] = D[i][j];
        }
      }
      const int r0 = k0 + kEvNb;
      const int mrows = d - r0;
      if (mrows <= 0) break;
      // ---- panel: X = A21 L11^-T, row by row (one thread per row), and w_rest -= X w_k
      // (the block is read through a volatile pointer: hoisting its 528 loads ahead of the substitution
      // would spill the row)
      const volatile double (*Dv)[kEvNb + 1] = D;
      for (int i = r0 + tid; i < d; i += kEvThreads) {
        double x[kEvNb];
        double* row = A + size_t(i) * d + k0;
#pragma unroll
        for (int j = 0; j < kEvNb; ++j) x[j] = row[j];
        double dot = 0.0;
#pragma unroll
        for (int j = 0; j < kEvNb; ++j) {
          double v = x[j];
#pragma unroll
          for (int c = 0; c < j; ++c) v -= x[c] * Dv[j][c];
          v /= Dv[j][j];
          x[j] = v;
          dot += v * w[k0 + j];
        }
#pragma unroll
        for (int j = 0; j < kEvNb; ++j) row[j] = x[j];
        w[i] -= dot;
      }
      __syncthreads();
      // ---- trailing update of the lower triangle: C -= X_bi X_bj^T in tiles of 64 rows x 128 columns
      const int mt = (mrows + kEvTile - 1) / kEvTile;
      // a warp owns 4 rows of the tile, a lane the columns {2 tx, 2 tx + 1} and {64 + 2 tx, 64 + 2 tx + 1}
      const int ty = tid >> 5, tx = tid & 31;
      for (int bi = 0; bi < mt; ++bi) {
        // the row block of the panel is staged once per tile row, transposed: At[k][row]
        {
          const int i = tid & 63, kg = tid >> 6;   // 64 rows x 8 groups of 4 columns
          const int ga = r0 + bi * kEvTile + i;
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const int kk = kg * 4 + k;
            At[kk * kEvTile + i] = ga < d ? A[size_t(ga) * d + k0 + kk] : 0.0;
          }
        }
        for (int bj = 0; bj * 2 <= bi; ++bj) {
          const int c0 = r0 + bj * 2 * kEvTile;
          // the tile of C is requested first, so that its latency hides behind the staging and the products
          double cval[4][4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int gi = r0 + bi * kEvTile + ty * 4 + i;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const int gj = c0 + (j >> 1) * kEvTile + tx * 2 + (j & 1);
              cval[i][j] = (gi < d && gj <= gi) ? A[size_t(gi) * d + gj] : 0.0;
            }
          }
          {
            const int i = tid & 127, kg = tid >> 7;   // 128 rows x 4 groups of 8 columns
            const int gb = c0 + i;
            const bool in = gb < d && gb <= r0 + bi * kEvTile + kEvTile - 1;   // rows past the diagonal block are not needed
#pragma unroll
            for (int k = 0; k < 8; ++k) {
              const int kk = kg * 8 + k;
              Bt[kk * 2 * kEvTile + i] = in ? A[size_t(gb) * d + k0 + kk] : 0.0;
            }
          }
          __syncthreads();
          double acc[4][4] = {};
#pragma unroll 8
          for (int k = 0; k < kEvNb; ++k) {
            const double2 a01 = *reinterpret_cast<const double2*>(At + k * kEvTile + ty * 4);
            const double2 a23 = *reinterpret_cast<const double2*>(At + k * kEvTile + ty * 4 + 2);
            const double2 b01 = *reinterpret_cast<const double2*>(Bt + k * 2 * kEvTile + tx * 2);
            const double2 b23 = *reinterpret_cast<const double2*>(Bt + k * 2 * kEvTile + kEvTile + tx * 2);
            const double a[4] = {a01.x, a01.y, a23.x, a23.y}, b[4] = {b01.x, b01.y, b23.x, b23.y};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
              for (int j = 0; j < 4; ++j) acc[i][j] = fma(a[i], b[j], acc[i][j]);
          }
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int gi = r0 + bi * kEvTile + ty * 4 + i;
            if (gi >= d) continue;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const int gj = c0 + (j >> 1) * kEvTile + tx * 2 + (j & 1);
              if (gj <= gi) A[size_t(gi) * d + gj] = cval[i][j] - acc[i][j];
            }
          }
          __syncthreads();
        }
      }
    }
    if (last) break;
    // ---- evidence of this penalty
    if (tid == 0) {
      double ev;
      if (s_pd) {
        const double r = fmax(yy - wnorm2, r_floor);
        ev = -0.5 * (n - 1.0) * log(r) - 0.5 * (2.0 * s_logsum - double(d) * log(lam));
      } else {
        ev = -INFINITY;   // rounding of the stored Gram matrix made G_c + lambda I indefinite: not a candidate
      }
      ev_out[li] = ev;
      if (best_i < 0 || ev > best) {
        best = ev;
        best_i = li;
      }
      s_best = best_i;
    }
    __syncthreads();
  }
  if (tid == 0) {
    for (int i = grid.n; i < kCalibMaxLambdas; ++i) ev_out[i] = 0.0;
    st.lambda_index[u] = best_i;
    st.lambda[u] = grid.v[best_i];
    st.iters[u] = 0;
  }
  // ---- back substitution L^T a = w, block rows from the bottom up; a overwrites w in place
  __syncthreads();
  double* colsum = At;   // [warps][32] partial column sums
  for (int k0 = d - kEvNb; k0 >= 0; k0 -= kEvNb) {
    const int r0 = k0 + kEvNb;
    // s_j = sum over the rows below of L[i][k0 + j] a[i]
    double part[kEvNb];
#pragma unroll
    for (int j = 0; j < kEvNb; ++j) part[j] = 0.0;
    for (int i = r0 + tid; i < d; i += kEvThreads) {
      const double ai = w[i];
      const double* row = A + size_t(i) * d + k0;
#pragma unroll
      for (int j = 0; j < kEvNb; ++j) part[j] = fma(row[j], ai, part[j]);
    }
#pragma unroll
    for (int j = 0; j < kEvNb; ++j) {
      double v = part[j];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
      if (lane == 0) colsum[warp * kEvNb + j] = v;
    }
    for (int idx = tid; idx < kEvNb * kEvNb; idx += kEvThreads) {
      const int i = idx >> 5, j = idx & 31;
      D[i][j] = j <= i ? A[size_t(k0 + i) * d + k0 + j] : 0.0;
    }
    __syncthreads();
    if (warp == 0) {
      double sj = 0.0;
      for (int wp = 0; wp < kEvThreads / 32; ++wp) sj += colsum[wp * kEvNb + lane];   // fixed order
      double rhs = w[k0 + lane] - sj;
      // upper-triangular solve with L11^T: lane = unknown, from the last one up
      for (int j = kEvNb - 1; j >= 0; --j) {
        const double aj = __shfl_sync(0xffffffffu, rhs, j) / D[j][j];
        if (lane == j) w[k0 + j] = aj;
        if (lane < j) rhs -= D[j][lane] * aj;
      }
    }
    __syncthreads();
  }
  double dot = 0.0;
  for (int j = tid; j < d; j += kEvThreads) {
    const double aj = w[j];
    st.coef_a[size_t(u) * d + j] = aj;
    dot += aj * m[j];
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) dot += __shfl_down_sync(0xffffffffu, dot, o);
  __syncthreads();
  if (lane == 0) colsum[warp] = dot;
  __syncthreads();
  if (tid == 0) {
    double t = 0.0;
    for (int wp = 0; wp < kEvThreads / 32; ++wp) t += colsum[wp];
    st.coef_b[u] = sy / n - t;
  }
}

}  // namespace

size_t calib_evidence_scratch_bytes(const base_layer_shape& s) { return size_t(s.E) * s.d * s.d * sizeof(double); }

cudaError_t launch_calib_evidence(const base_layer_shape& s, const CalibState& st, void* scratch, const double* lambdas,
                                  int n_lambda, int default_index, cudaStream_t stream) {
  LambdaGrid g{};
  g.n = n_lambda;
  g.default_index = default_index;
  for (int i = 0; i < n_lambda; ++i) g.v[i] = lambdas[i];
  const size_t smem = (size_t(3) * s.d + 3 * kEvNb * kEvTile) * sizeof(double);
  static size_t set_for = 0;
  if (smem > set_for) {
    cudaError_t a = cudaFuncSetAttribute(calib_evidence_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    if (a != cudaSuccess) return a;
    set_for = smem;
  }
  calib_evidence_kernel<<<s.E, kEvThreads, smem, stream>>>(st, static_cast<double*>(scratch), s.d, g);
  return cudaGetLastError();
}

}  // namespace base
