// Offline calibration of the log-energy predictor on the device (App. Calibration Details):
// streaming sufficient statistics per expert -- sample count, first moments, Gram matrix (fp32),
// input-target cross-moment and scalar sums (fp64) -- over batches of calibration tokens, a
// closed-form centred ridge solve per expert, and the retransformation correction of the intercept.
//
// One accumulate call runs the layer with every original route executed, takes the true output
// energy of every routed pair from the per-pair expert outputs, and adds the pair to the statistics
// of its expert. The Gram update G_u += sum_t zbar_t zbar_t^T is the one dense contraction of the
// method; it runs on tcgen05 tensor cores from a transposed copy of the normalised inputs, split
// into a bf16 head and a bf16 remainder (three products per tile keep about 16 bits of the inputs).
#include <cuda.h>

#include <algorithm>

#include "calib.cuh"
#include "ffn_tc.cuh"
#include "tc_ptx.cuh"

namespace base {

namespace {

constexpr float kEnergyEps = 1e-12f;   // target: log(energy + eps) (Sec. 3.4)

// ------------------------------------------------------------------------------------------------
// k-block offsets of the experts' padded token segments: every dispatched expert owns whole k-blocks
// of 64 columns of the transposed operand, so that a tensor-core tile never mixes two experts.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(512) calib_offsets_kernel(const int32_t* __restrict__ expert_count, int E,
                                                            int32_t* __restrict__ koff) {
  __shared__ int s_w[16];
  pdl_launch_dependents();
  pdl_wait();
  const int e = threadIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int nkb = e < E ? (expert_count[e] + 63) >> 6 : 0;
  int incl = nkb;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int x = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += x;
  }
  if (lane == 31) s_w[warp] = incl;
  __syncthreads();
  int before = 0;
  for (int w = 0; w < warp; ++w) before += s_w[w];
  if (e < E) koff[e] = before + incl - nkb;
  if (e == E - 1) koff[E] = before + incl;
}

// Energy of every sorted row: ||E_u(z_t)||^2 from the per-pair outputs (partial copies of a split
// down pass are added first, in copy order). One warp per row, fixed summation order.
__global__ void __launch_bounds__(256) calib_row_energy_kernel(const float* __restrict__ ypair, int n_split,
                                                               size_t split_stride,
                                                               const int32_t* __restrict__ counters, int d,
                                                               float* __restrict__ row_energy) {
  pdl_launch_dependents();
  pdl_wait();
  const int n_rows = counters[kCtrSlots];
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= n_rows) return;
  float acc = 0.f;
  for (int c = lane * 4; c < d; c += 128) {
    float4 v = *reinterpret_cast<const float4*>(ypair + size_t(row) * d + c);
    for (int s = 1; s < n_split; ++s) {
      const float4 w = *reinterpret_cast<const float4*>(ypair + size_t(s) * split_stride + size_t(row) * d + c);
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
  acc = warp_sum(acc);
  if (lane == 0) row_energy[row] = acc;
}

// Expert that owns k-block kb of the padded columns: last u with koff[u] <= kb.
__device__ __forceinline__ int expert_of_kblock(const int32_t* koff, int E, int kb) {
  int lo = 0, hi = E - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (koff[mid] <= kb) lo = mid;
    else hi = mid - 1;
  }
  return lo;
}

__device__ __forceinline__ float inv_norm_of(const float* znorm2, int t) {
  return 1.0f / fmaxf(sqrtf(znorm2[t]), 1e-30f);
}
__device__ __forceinline__ float bf16_to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }

// ------------------------------------------------------------------------------------------------
// Transposed, split operand of the Gram update: zt_hi[j][col] + zt_lo[j][col] ~ zbar_t[j] for the
// token t in padded column col of its expert's segment (zero in the padding). One CTA moves a tile
// of 64 columns (one k-block, one expert) x 64 features through shared memory so that both the reads
// (along d) and the writes (along the columns) are coalesced.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) calib_transpose_kernel(const __nv_bfloat16* __restrict__ hidden,
                                                              const float* __restrict__ znorm2,
                                                              const int32_t* __restrict__ slot_token,
                                                              const int32_t* __restrict__ expert_offset,
                                                              const int32_t* __restrict__ expert_count,
                                                              const int32_t* __restrict__ koff, int E, int d,
                                                              size_t ld_cols, __nv_bfloat16* __restrict__ zt_hi,
                                                              __nv_bfloat16* __restrict__ zt_lo) {
  __shared__ float s_tile[64][65];
  __shared__ int s_tok[64];
  __shared__ float s_inv[64];
  pdl_launch_dependents();
  pdl_wait();
  const int kb = blockIdx.x;
  if (kb >= koff[E]) return;
  const int u = expert_of_kblock(koff, E, kb);
  const int pos0 = (kb - koff[u]) * 64, cnt = expert_count[u], off = expert_offset[u];
  if (threadIdx.x < 64) {
    const int pos = pos0 + threadIdx.x;
    const int t = pos < cnt ? slot_token[off + pos] : -1;
    s_tok[threadIdx.x] = t;
    s_inv[threadIdx.x] = t >= 0 ? inv_norm_of(znorm2, t) : 0.f;
  }
  __syncthreads();
  const int j0 = blockIdx.y * 64;
  for (int i = threadIdx.x; i < 64 * 64; i += 256) {
    const int c = i >> 6, j = i & 63;
    const int t = s_tok[c];
    s_tile[c][j] = t >= 0 ? bf16_to_f32(hidden[size_t(t) * d + j0 + j]) * s_inv[c] : 0.f;
  }
  __syncthreads();
  for (int i = threadIdx.x; i < 64 * 64; i += 256) {
    const int j = i >> 6, c = i & 63;
    const float v = s_tile[c][j];
    const __nv_bfloat16 h = __float2bfloat16_rn(v);
    const __nv_bfloat16 l = __float2bfloat16_rn(v - __bfloat162float(h));
    const size_t o = size_t(j0 + j) * ld_cols + size_t(kb) * 64 + c;
    zt_hi[o] = h;
    zt_lo[o] = l;
  }
}

// ------------------------------------------------------------------------------------------------
// Vector and scalar statistics in fp64, in two levels so that a popular expert (thousands of pairs
// under a skewed router) does not serialise the pass: one CTA per (k-block of 64 pairs, 256
// features) sums its pairs in row order into a partial; one CTA per (expert, 256 features) then adds
// the expert's partials in k-block order to the state. Every sum has a fixed order.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) calib_vector_partials_kernel(const __nv_bfloat16* __restrict__ hidden,
                                                                    const float* __restrict__ znorm2,
                                                                    const int32_t* __restrict__ slot_token,
                                                                    const int32_t* __restrict__ expert_offset,
                                                                    const int32_t* __restrict__ expert_count,
                                                                    const int32_t* __restrict__ koff,
                                                                    const float* __restrict__ row_energy, int E, int d,
                                                                    double* __restrict__ part_z,
                                                                    double* __restrict__ part_yz,
                                                                    double* __restrict__ part_s) {
  __shared__ int s_tok[64];
  __shared__ float s_inv[64];
  __shared__ double s_y[64];
  pdl_launch_dependents();
  pdl_wait();
  const int kb = blockIdx.x;
  if (kb >= koff[E]) return;
  const int u = expert_of_kblock(koff, E, kb);
  const int pos0 = (kb - koff[u]) * 64, off = expert_offset[u];
  const int np = min(64, expert_count[u] - pos0);
  if (threadIdx.x < 64) {
    const bool in = int(threadIdx.x) < np;
    const int t = in ? slot_token[off + pos0 + threadIdx.x] : 0;
    s_tok[threadIdx.x] = t;
    s_inv[threadIdx.x] = in ? inv_norm_of(znorm2, t) : 0.f;
    s_y[threadIdx.x] = in ? log(double(row_energy[off + pos0 + threadIdx.x]) + double(kEnergyEps)) : 0.0;
  }
  __syncthreads();
  const int j = blockIdx.y * 256 + threadIdx.x;
  if (j < d) {
    double sz = 0.0, syz = 0.0;
    for (int p = 0; p < np; ++p) {
      const double zb = double(bf16_to_f32(hidden[size_t(s_tok[p]) * d + j]) * s_inv[p]);
      sz += zb;
      syz += s_y[p] * zb;
    }
    part_z[size_t(kb) * d + j] = sz;
    part_yz[size_t(kb) * d + j] = syz;
  }
  if (blockIdx.y == 0 && threadIdx.x == 0) {
    double sy = 0.0, syy = 0.0, se = 0.0;
    for (int p = 0; p < np; ++p) {
      sy += s_y[p];
      syy += s_y[p] * s_y[p];
      se += double(row_energy[off + pos0 + p]);
    }
    part_s[size_t(kb) * 4 + 0] = sy;
    part_s[size_t(kb) * 4 + 1] = syy;
    part_s[size_t(kb) * 4 + 2] = se;
  }
}

__global__ void __launch_bounds__(256) calib_vector_reduce_kernel(const int32_t* __restrict__ expert_count,
                                                                  const int32_t* __restrict__ koff, int d,
                                                                  const double* __restrict__ part_z,
                                                                  const double* __restrict__ part_yz,
                                                                  const double* __restrict__ part_s, CalibState st) {
  pdl_launch_dependents();
  pdl_wait();
  const int u = blockIdx.x, j = blockIdx.y * 256 + threadIdx.x;
  const int cnt = expert_count[u];
  if (cnt == 0) return;
  const int kb0 = koff[u], kb1 = koff[u + 1];
  if (j < d) {
    double sz = 0.0, syz = 0.0;
    for (int kb = kb0; kb < kb1; ++kb) {
      sz += part_z[size_t(kb) * d + j];
      syz += part_yz[size_t(kb) * d + j];
    }
    st.sum_z[size_t(u) * d + j] += sz;
    st.sum_yz[size_t(u) * d + j] += syz;
  }
  if (blockIdx.y == 0 && threadIdx.x == 0) {
    double sy = 0.0, syy = 0.0, se = 0.0;
    for (int kb = kb0; kb < kb1; ++kb) {
      sy += part_s[size_t(kb) * 4 + 0];
      syy += part_s[size_t(kb) * 4 + 1];
      se += part_s[size_t(kb) * 4 + 2];
    }
    st.n[u] += double(cnt);
    st.sum_y[u] += sy;
    st.sum_yy[u] += syy;
    st.sum_e[u] += se;
  }
}

}  // namespace

}  // namespace base

#include "calib_gram.cuh"
#include "calib_solve.cuh"
#include "calib_evidence.cuh"
