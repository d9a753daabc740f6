// Selection-quality diagnostics on the device: true removal costs of routed pairs
// (Eq. individual_expert_damage) from the per-pair expert outputs that the layer leaves in its
// workspace, the exact error of an active set with its individual and cross parts
// (Eq. error_decomposition), and the retained-energy ratio (Eq. energy_retained).
#include "common.cuh"

namespace base {

// One CTA per token: the token's row of the dense cost matrix is cleared, then one warp per route
// squares and sums its output row (summing the partial copies of a split down pass first, in copy
// order). All sums have a fixed order, so the result does not depend on scheduling.
__global__ void __launch_bounds__(256) pair_energy_kernel(const float* __restrict__ ypair, int n_split,
                                                          size_t split_stride,
                                                          const int32_t* __restrict__ exec_ids,
                                                          const float* __restrict__ exec_gates,
                                                          const int32_t* __restrict__ token_slot,
                                                          float* __restrict__ true_costs,
                                                          float* __restrict__ pair_energy, int E, int K, int d) {
  const int t = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  pdl_launch_dependents();
  pdl_wait();
  for (int e = threadIdx.x; e < E; e += blockDim.x) true_costs[size_t(t) * E + e] = 0.f;
  __syncthreads();
  for (int k = warp; k < K; k += int(blockDim.x >> 5)) {
    const int e = exec_ids[t * K + k];
    const int slot = token_slot[t * K + k];
    float en = 0.f;
    if (e >= 0 && slot >= 0) {
      float acc = 0.f;
      for (int c = lane * 4; c < d; c += 128) {
        float4 v = *reinterpret_cast<const float4*>(ypair + size_t(slot) * d + c);
        for (int s = 1; s < n_split; ++s) {
          const float4 w = *reinterpret_cast<const float4*>(ypair + size_t(s) * split_stride + size_t(slot) * d + c);
          v.x += w.x;
          v.y += w.y;
          v.z += w.z;
          v.w += w.w;
        }
        acc = fmaf(v.x, v.x, acc);
        acc = fmaf(v.y, v.y, acc);
        acc = fmaf(v.z, v.z, acc);
        acc = fmaf(v.w, v.w, acc);
      }
      en = warp_sum(acc);
    }
    if (lane == 0) {
      if (pair_energy) pair_energy[t * K + k] = en;
      if (e >= 0) {
        const float g = exec_gates[t * K + k];
        true_costs[size_t(t) * E + e] = g * g * en;
      }
    }
  }
}

cudaError_t launch_pair_energy(const Workspace& ws, int n_split, float* true_costs, float* pair_energy, int T, int E,
                               int K, int d, cudaStream_t st) {
  return launch_pdl(pair_energy_kernel, dim3(T), dim3(256), 0, st, 1, static_cast<const float*>(ws.ypair), n_split,
                    ws.ypair_stride, static_cast<const int32_t*>(ws.exec_ids),
                    static_cast<const float*>(ws.exec_gates), static_cast<const int32_t*>(ws.token_slot), true_costs,
                    pair_energy, E, K, d);
}

// Exact error of serving the batch with active set A and no replacement (Eq. error_decomposition):
// per token the omitted contributions a_{t,u} = w_{t,u} E_u(z_t), u in R_t \ A, are added and squared,
// E(A) = sum_t || sum_u a_{t,u} ||^2, next to the individual part sum_t sum_u ||a_{t,u}||^2; the cross
// terms are their difference. One CTA per token writes its two numbers; a second kernel adds them in
// token order.
__global__ void __launch_bounds__(256) exact_error_token_kernel(const float* __restrict__ ypair, int n_split,
                                                                size_t split_stride,
                                                                const int32_t* __restrict__ exec_ids,
                                                                const float* __restrict__ exec_gates,
                                                                const int32_t* __restrict__ token_slot,
                                                                const uint8_t* __restrict__ mask, int K, int d,
                                                                float* __restrict__ per_token) {
  __shared__ int s_slot[kMaxK];
  __shared__ float s_gate[kMaxK];
  __shared__ float s_tot[8], s_ind[8];
  const int t = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  pdl_launch_dependents();
  pdl_wait();
  if (threadIdx.x < kMaxK) {
    int slot = -1;
    float g = 0.f;
    if (int(threadIdx.x) < K) {
      const int e = exec_ids[t * K + threadIdx.x];
      if (e >= 0 && !mask[e]) {   // an omitted route
        slot = token_slot[t * K + threadIdx.x];
        g = exec_gates[t * K + threadIdx.x];
      }
    }
    s_slot[threadIdx.x] = slot;
    s_gate[threadIdx.x] = g;
  }
  __syncthreads();
  float tot = 0.f, ind = 0.f;
  for (int c = threadIdx.x; c < d; c += 256) {
    float v = 0.f;
    for (int k = 0; k < K; ++k) {
      const int slot = s_slot[k];
      if (slot < 0) continue;
      float y = ypair[size_t(slot) * d + c];
      for (int s = 1; s < n_split; ++s) y += ypair[size_t(s) * split_stride + size_t(slot) * d + c];
      const float a = s_gate[k] * y;
      v += a;
      ind = fmaf(a, a, ind);
    }
    tot = fmaf(v, v, tot);
  }
  tot = warp_sum(tot);
  ind = warp_sum(ind);
  if (lane == 0) {
    s_tot[warp] = tot;
    s_ind[warp] = ind;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    float a = 0.f, b = 0.f;
    for (int w = 0; w < 8; ++w) {
      a += s_tot[w];
      b += s_ind[w];
    }
    per_token[2 * t] = a;
    per_token[2 * t + 1] = b;
  }
}

__global__ void exact_error_sum_kernel(const float* __restrict__ per_token, int T, float* __restrict__ out) {
  pdl_launch_dependents();
  pdl_wait();
  if (threadIdx.x != 0) return;
  double tot = 0.0, ind = 0.0;
  for (int t = 0; t < T; ++t) {
    tot += double(per_token[2 * t]);
    ind += double(per_token[2 * t + 1]);
  }
  out[0] = float(tot);
  out[1] = float(ind);
  out[2] = float(tot - ind);
}

cudaError_t launch_exact_error(const Workspace& ws, int n_split, const uint8_t* mask, float* per_token, float* out, int T,
                               int K, int d, cudaStream_t st) {
  cudaError_t e = launch_pdl(exact_error_token_kernel, dim3(T), dim3(256), 0, st, 1, static_cast<const float*>(ws.ypair),
                             n_split, ws.ypair_stride, static_cast<const int32_t*>(ws.exec_ids),
                             static_cast<const float*>(ws.exec_gates), static_cast<const int32_t*>(ws.token_slot), mask, K,
                             d, per_token);
  if (e != cudaSuccess) return e;
  return launch_pdl(exact_error_sum_kernel, dim3(1), dim3(32), 0, st, 1, static_cast<const float*>(per_token), T, out);
}

// Retained energy of an active set: one CTA. An expert belongs to the oracle set A* when fewer than
// `budget` experts come before it (score descending, ties to the lower id). Both sums run over the
// experts in id order (per-thread strips, then a fixed tree).
constexpr int kErThreads = 256;

__global__ void __launch_bounds__(kErThreads) energy_retained_kernel(const float* __restrict__ scores,
                                                                    const uint8_t* __restrict__ mask, int E,
                                                                    int budget, float* __restrict__ out) {
  __shared__ float s_sc[1024];
  __shared__ float s_num[kErThreads], s_den[kErThreads];
  pdl_launch_dependents();
  pdl_wait();
  for (int e = threadIdx.x; e < E; e += kErThreads) s_sc[e] = scores[e];
  __syncthreads();
  // contiguous strip of experts per thread keeps the summation in id order
  const int per = (E + kErThreads - 1) / kErThreads;
  float num = 0.f, den = 0.f;
  for (int i = 0; i < per; ++i) {
    const int e = threadIdx.x * per + i;
    if (e >= E) break;
    const float se = s_sc[e];
    int r = 0;
    for (int j = 0; j < E; ++j) {
      const float sj = s_sc[j];
      r += (sj > se) || (sj == se && j < e);
    }
    if (r < budget) den += se;
    if (mask[e]) num += se;
  }
  s_num[threadIdx.x] = num;
  s_den[threadIdx.x] = den;
  __syncthreads();
  for (int o = kErThreads / 2; o > 0; o >>= 1) {
    if (int(threadIdx.x) < o) {
      s_num[threadIdx.x] += s_num[threadIdx.x + o];
      s_den[threadIdx.x] += s_den[threadIdx.x + o];
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) out[0] = s_den[0] > 0.f ? s_num[0] / s_den[0] : 1.f;
}

cudaError_t launch_energy_retained(const float* scores, const uint8_t* mask, int E, int budget, float* out,
                                   cudaStream_t st) {
  return launch_pdl(energy_retained_kernel, dim3(1), dim3(kErThreads), 0, st, 1, scores, mask, E, budget, out);
}

}  // namespace base
