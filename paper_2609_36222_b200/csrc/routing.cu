// Routing side of the decode layer: router/predictor GEMV, predicted removal costs, batch
// aggregation, top-M selection, restricted routing with backfill, and the expert-sorted
// dispatch lists. Everything between the GEMV and the expert FFN runs in one CTA with no host
// round trip.
#include <limits.h>
#include <math.h>

#include "common.cuh"

namespace base {

// ------------------------------------------------------------------------------------------------
// Stand-alone scoring kernel (Eq. log_energy_predictor): one CTA per token, one warp per routed
// expert, 128-bit loads of the predictor row and the token.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) predict_costs_kernel(const __nv_bfloat16* __restrict__ hidden,
                                                            const int32_t* __restrict__ ids,
                                                            const float* __restrict__ w,
                                                            const __nv_bfloat16* __restrict__ A,
                                                            const float* __restrict__ b, float* __restrict__ costs,
                                                            int d, int E, int K) {
  const int t = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
  const __nv_bfloat16* z = hidden + size_t(t) * d;
  __shared__ float s_part[8];
  __shared__ float s_inv;
  // ||z||^2 over the block
  float zz = 0.f;
  for (int j = threadIdx.x * 8; j < d; j += blockDim.x * 8) {
    float f[8];
    unpack8(ldg16(z + j), f);
#pragma unroll
    for (int i = 0; i < 8; ++i) zz = fmaf(f[i], f[i], zz);
  }
  zz = warp_sum(zz);
  if (lane == 0) s_part[warp] = zz;
  for (int e = threadIdx.x; e < E; e += blockDim.x) costs[size_t(t) * E + e] = 0.f;
  __syncthreads();
  if (threadIdx.x == 0) {
    float s = 0.f;
    for (int i = 0; i < nwarp; ++i) s += s_part[i];
    s_inv = 1.0f / fmaxf(sqrtf(s), 1e-30f);
  }
  __syncthreads();
  const float inv = s_inv;
  for (int k = warp; k < K; k += nwarp) {
    const int u = ids[size_t(t) * K + k];
    if (u < 0 || u >= E) continue;
    const __nv_bfloat16* a = A + size_t(u) * d;
    float acc = 0.f;
    for (int j = lane * 8; j < d; j += 256) {
      float fz[8], fa[8];
      unpack8(ldg16(z + j), fz);
      unpack8(ldg16(a + j), fa);
#pragma unroll
      for (int i = 0; i < 8; ++i) acc = fmaf(fz[i], fa[i], acc);
    }
    acc = warp_sum(acc);
    if (lane == 0) {
      const float wk = w[size_t(t) * K + k];
      costs[size_t(t) * E + u] = wk * wk * expf(acc * inv + b[u]);
    }
  }
}

cudaError_t launch_predict_costs(const void* hidden, const int32_t* ids, const float* w, const void* A,
                                 const float* b, float* costs, int T, int d, int E, int K, cudaStream_t st) {
  predict_costs_kernel<<<T, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(hidden), ids, w,
                                          static_cast<const __nv_bfloat16*>(A), b, costs, d, E, K);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Shared pieces of aggregation and selection.
// Column sum in a fixed order: lane l adds tokens l, l+32, ... in ascending order, then an xor tree.
// Both the stand-alone and the fused path use this order, so their scores are bit-identical.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ float sortable(float s, int* nonfinite) {
  if (!isfinite(s)) *nonfinite = 1;
  return isnan(s) ? -INFINITY : s;
}

// rank of expert e among s[0..E): number of experts that come before it (score desc, id asc).
__device__ __forceinline__ int rank_of(const float* s, int E, int e) {
  const float se = s[e];
  int r = 0;
  for (int j = 0; j < E; ++j) {
    const float sj = s[j];
    r += (sj > se) || (sj == se && j < e);
  }
  return r;
}

__global__ void __launch_bounds__(1024) aggregate_select_kernel(const float* __restrict__ costs, int T, int E, int M,
                                                                float* __restrict__ scores,
                                                                int32_t* __restrict__ selected,
                                                                uint8_t* __restrict__ mask) {
  __shared__ float s_sc[1024];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
  for (int e = warp; e < E; e += nwarp) {
    float acc = 0.f;
    for (int t = lane; t < T; t += 32) acc += costs[size_t(t) * E + e];
    acc = warp_sum(acc);
    if (lane == 0) {
      scores[e] = acc;
      int nf = 0;
      s_sc[e] = sortable(acc, &nf);
    }
  }
  __syncthreads();
  for (int e = threadIdx.x; e < E; e += blockDim.x) {
    const int r = rank_of(s_sc, E, e);
    mask[e] = r < M;
    if (r < M) selected[r] = e;
  }
}

cudaError_t launch_aggregate_select(const float* costs, int T, int E, int M, float* scores, int32_t* sel,
                                    uint8_t* mask, cudaStream_t st) {
  aggregate_select_kernel<<<1, 1024, 0, st>>>(costs, T, E, M, scores, sel, mask);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Router + predictor GEMV for every (token, expert) pair: logits[t,e] = z_t . W_r[e] + bias[e] and
// shat[t,e] = a_e . z_t / ||z_t|| + b_e. grid = (E, token chunks); the two weight rows sit in shared
// memory, each warp streams its tokens with 128-bit loads. Computing shat for all pairs (not only
// the routed ones) removes the dependency on the top-K result; it costs one more 2*E*d-byte read.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) route_scores_kernel(const __nv_bfloat16* __restrict__ hidden,
                                                           const __nv_bfloat16* __restrict__ router_w,
                                                           const float* __restrict__ router_bias,
                                                           const __nv_bfloat16* __restrict__ pred_A,
                                                           const float* __restrict__ pred_b,
                                                           float* __restrict__ logits, float* __restrict__ shat,
                                                           int T, int d, int E, int tokens_per_cta) {
  extern __shared__ uint4 s_rows[];  // [2][d/8]
  const int e = blockIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
  const int dv = d >> 3;
  const bool do_logits = logits != nullptr;
  for (int j = threadIdx.x; j < dv; j += blockDim.x) {
    s_rows[j] = do_logits ? ldg16(router_w + size_t(e) * d + j * 8) : make_uint4(0, 0, 0, 0);
    s_rows[dv + j] = ldg16(pred_A + size_t(e) * d + j * 8);
  }
  __syncthreads();
  const int t0 = blockIdx.y * tokens_per_cta;
  const int t1 = min(T, t0 + tokens_per_cta);
  for (int t = t0 + warp; t < t1; t += nwarp) {
    const __nv_bfloat16* z = hidden + size_t(t) * d;
    float accL = 0.f, accA = 0.f, accZ = 0.f;
    for (int j = lane; j < dv; j += 32) {
      float fz[8], fr[8], fa[8];
      unpack8(ldg16(z + j * 8), fz);
      unpack8(s_rows[j], fr);
      unpack8(s_rows[dv + j], fa);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        accL = fmaf(fz[i], fr[i], accL);
        accA = fmaf(fz[i], fa[i], accA);
        accZ = fmaf(fz[i], fz[i], accZ);
      }
    }
    accL = warp_sum(accL);
    accA = warp_sum(accA);
    accZ = warp_sum(accZ);
    if (lane == 0) {
      if (do_logits) logits[size_t(t) * E + e] = accL + (router_bias ? router_bias[e] : 0.f);
      shat[size_t(t) * E + e] = accA / fmaxf(sqrtf(accZ), 1e-30f) + pred_b[e];
    }
  }
}

cudaError_t launch_route_scores(const void* hidden, const void* router_w, const float* router_bias,
                                const void* pred_A, const float* pred_b, float* logits_out, float* shat,
                                int T, int d, int E, cudaStream_t st) {
  int chunks = (2 * 148 + E - 1) / E;               // aim at >= 2 CTAs per SM
  chunks = max(1, min(chunks, (T + 7) / 8));        // at least one token per warp
  const int tpc = (T + chunks - 1) / chunks;
  dim3 grid(E, (T + tpc - 1) / tpc);
  route_scores_kernel<<<grid, 256, size_t(d) * 4, st>>>(
      static_cast<const __nv_bfloat16*>(hidden), static_cast<const __nv_bfloat16*>(router_w), router_bias,
      static_cast<const __nv_bfloat16*>(pred_A), pred_b, logits_out, shat, T, d, E, tpc);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// The routing kernel: one CTA.
//   A  per token: top-K of the logits (value desc, id asc), q = exp(l - max), S = sum over R_t,
//      w = q/S, predicted cost c = w^2 exp(shat)                                (Sec. 3.1, 3.4)
//   B  D[u] = sum_t c[t,u]                                                      (Sec. 3.4)
//   C  active set = top-M of D by rank counting                                 (Sec. 3.5)
//   D  per token: K highest-ranked experts inside the active set, gate = q / S  (Sec. 3.5)
//   E  expert-sorted dispatch: counts, offsets, row of every executed pair, work segments
// ------------------------------------------------------------------------------------------------
constexpr int kNone = INT_MAX;

__device__ __forceinline__ void warp_argbest(float& v, int& idx) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, v, o);
    const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
    if (oi != kNone && (idx == kNone || ov > v || (ov == v && oi < idx))) {
      v = ov;
      idx = oi;
    }
  }
}

// Pick the best available entry of this warp's logit row and mark it taken. All lanes return it.
__device__ __forceinline__ void take_best(const float (&v)[kMaxVals], uint32_t& avail, int lane, float& bv, int& bi) {
  bv = -INFINITY;
  bi = kNone;
#pragma unroll
  for (int i = 0; i < kMaxVals; ++i) {
    if ((avail >> i) & 1u) {
      if (bi == kNone || v[i] > bv) {
        bv = v[i];
        bi = lane + 32 * i;
      }
    }
  }
  warp_argbest(bv, bi);
  if (bi != kNone && (bi & 31) == lane) avail &= ~(1u << (bi >> 5));
}

__global__ void __launch_bounds__(1024) routing_kernel(RoutingArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int T = a.T, E = a.E, K = a.K, S = T * K;
  int32_t* s_ids = reinterpret_cast<int32_t*>(smem_raw);      // [S] original routes
  float* s_cost = reinterpret_cast<float*>(s_ids + S);        // [S] predicted costs, later positions
  int32_t* s_eids = reinterpret_cast<int32_t*>(s_cost + S);   // [S] executed routes
  float* s_m = reinterpret_cast<float*>(s_eids + S);          // [T]
  float* s_S = s_m + T;                                       // [T]
  float* s_sc = s_S + T;                                      // [E]
  int32_t* s_cnt = reinterpret_cast<int32_t*>(s_sc + E);      // [E]
  int32_t* s_off = s_cnt + E;                                 // [E+1]
  uint8_t* s_mask = reinterpret_cast<uint8_t*>(s_off + E + 1);  // [E]
  __shared__ int s_status;

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
  const int nv = (E + 31) >> 5;
  if (threadIdx.x == 0) s_status = 0;
  __syncthreads();

  // ---- A: original routes and predicted costs
  for (int t = warp; t < T; t += nwarp) {
    float v[kMaxVals];
    uint32_t avail = 0;
#pragma unroll
    for (int i = 0; i < kMaxVals; ++i) {
      const int e = lane + 32 * i;
      v[i] = -INFINITY;
      if (i < nv && e < E) {
        const float l = a.logits[size_t(t) * E + e];
        v[i] = isnan(l) ? -INFINITY : l;
        avail |= 1u << i;
        a.ws.costs[size_t(t) * E + e] = 0.f;
      }
    }
    float m = -INFINITY;
#pragma unroll
    for (int i = 0; i < kMaxVals; ++i) m = fmaxf(m, v[i]);
    m = warp_max(m);
    if (!(m > -INFINITY)) m = 0.f;
    float S_t = 0.f, myq = 0.f;
    int myid = kNone;
    for (int k = 0; k < K; ++k) {
      float bv;
      int bi;
      take_best(v, avail, lane, bv, bi);
      const float q = (bi == kNone) ? 0.f : expf(bv - m);
      S_t += q;
      if (lane == k) {
        myq = q;
        myid = bi;
      }
    }
    __syncwarp();
    if (lane < K) {
      const bool ok = myid != kNone;
      const float w = (ok && S_t > 0.f) ? myq / S_t : 0.f;
      float c = 0.f;
      if (ok) {
        c = w * w * expf(a.shat[size_t(t) * E + myid]);
        a.ws.costs[size_t(t) * E + myid] = c;
      }
      const int idx = t * K + lane;
      s_ids[idx] = ok ? myid : -1;
      s_cost[idx] = c;
      a.ws.topk_ids[idx] = ok ? myid : -1;
      a.ws.topk_w[idx] = w;
      if (a.dbg.topk_ids) a.dbg.topk_ids[idx] = ok ? myid : -1;
      if (a.dbg.topk_w) a.dbg.topk_w[idx] = w;
    }
    if (lane == 0) {
      s_m[t] = m;
      s_S[t] = S_t;
    }
  }
  __syncthreads();
  if (a.dbg.costs) {
    for (int i = threadIdx.x; i < T * E; i += blockDim.x) a.dbg.costs[i] = a.ws.costs[i];
  }
  if (a.dbg.logits) {
    for (int i = threadIdx.x; i < T * E; i += blockDim.x) a.dbg.logits[i] = a.logits[i];
  }

  // ---- B: batch aggregation, fixed order (see aggregate_select_kernel)
  for (int e = warp; e < E; e += nwarp) {
    float acc = 0.f;
    for (int t = lane; t < T; t += 32) {
      float c = 0.f;
      for (int k = 0; k < K; ++k)
        if (s_ids[t * K + k] == e) c = s_cost[t * K + k];
      acc += c;
    }
    acc = warp_sum(acc);
    if (lane == 0) {
      int nf = 0;
      s_sc[e] = sortable(acc, &nf);
      if (nf) atomicOr(&s_status, BASE_DEV_NONFINITE_SCORE);
      a.ws.scores[e] = acc;
      if (a.dbg.scores) a.dbg.scores[e] = acc;
    }
  }
  __syncthreads();

  // ---- C: top-M by rank counting
  const int M = min(a.M, E);
  for (int e = threadIdx.x; e < E; e += blockDim.x) {
    const int r = rank_of(s_sc, E, e);
    const uint8_t in = r < M;
    a.ws.mask[e] = in;
    if (in) a.ws.selected[r] = e;
    if (a.dbg.active_mask) a.dbg.active_mask[e] = in;
    if (in && a.dbg.selected_ids) a.dbg.selected_ids[r] = e;
    s_mask[e] = a.forced_mask ? (a.forced_mask[e] != 0) : in;
    s_cnt[e] = 0;
  }
  __syncthreads();

  // ---- D: restricted routes and gates
  for (int t = warp; t < T; t += nwarp) {
    float v[kMaxVals];
    uint32_t avail = 0;
#pragma unroll
    for (int i = 0; i < kMaxVals; ++i) {
      const int e = lane + 32 * i;
      v[i] = -INFINITY;
      if (i < nv && e < E) {
        const float l = a.logits[size_t(t) * E + e];
        v[i] = isnan(l) ? -INFINITY : l;
        bool ok = s_mask[e] != 0;
        if (ok && a.fill_rule == BASE_FILL_DROP) {
          ok = false;
          for (int k = 0; k < K; ++k) ok |= (s_ids[t * K + k] == e);
        }
        if (ok) avail |= 1u << i;
      }
    }
    const float m = s_m[t];
    float sumq = 0.f, myq = 0.f;
    int myid = kNone;
    for (int k = 0; k < K; ++k) {
      float bv;
      int bi;
      take_best(v, avail, lane, bv, bi);
      const float q = (bi == kNone) ? 0.f : expf(bv - m);
      sumq += q;
      if (lane == k) {
        myq = q;
        myid = bi;
      }
    }
    if (lane < K) {
      const float den = (a.gate_rule == BASE_GATE_RENORM) ? sumq : s_S[t];
      const bool ok = myid != kNone;
      const float g = (ok && den > 0.f) ? myq / den : 0.f;
      const int idx = t * K + lane;
      s_eids[idx] = ok ? myid : -1;
      a.ws.exec_ids[idx] = ok ? myid : -1;
      a.ws.exec_gates[idx] = g;
      if (a.dbg.exec_ids) a.dbg.exec_ids[idx] = ok ? myid : -1;
      if (a.dbg.exec_gates) a.dbg.exec_gates[idx] = g;
    }
  }
  __syncthreads();

  // ---- E: dispatch lists. Position of a pair inside its expert = number of lower-numbered tokens
  // routed to that expert, so each expert's rows are in token order.
  int32_t* s_pos = reinterpret_cast<int32_t*>(s_cost);
  for (int e = warp; e < E; e += nwarp) {
    int base_cnt = 0;
    for (int t0 = 0; t0 < T; t0 += 32) {
      const int t = t0 + lane;
      int kk = -1;
      if (t < T) {
        for (int k = 0; k < K; ++k)
          if (s_eids[t * K + k] == e) kk = k;
      }
      const uint32_t bal = __ballot_sync(0xffffffffu, kk >= 0);
      if (kk >= 0) s_pos[t * K + kk] = base_cnt + __popc(bal & ((1u << lane) - 1u));
      base_cnt += __popc(bal);
    }
    if (lane == 0) s_cnt[e] = base_cnt;
  }
  __syncthreads();
  if (warp == 0) {
    // exclusive scan of the counts, the compact list of dispatched experts, and the work segments
    int run = 0, nseg = 0, ndisp = 0;
    for (int e0 = 0; e0 < E; e0 += 32) {
      const int e = e0 + lane;
      const int c = (e < E) ? s_cnt[e] : 0;
      const int segs = (c + kSegTokens - 1) / kSegTokens;
      int incl = c, sincl = segs;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int x = __shfl_up_sync(0xffffffffu, incl, o);
        const int y = __shfl_up_sync(0xffffffffu, sincl, o);
        if (lane >= o) {
          incl += x;
          sincl += y;
        }
      }
      const int off = run + incl - c;
      if (e < E) {
        s_off[e] = off;
        a.ws.expert_offset[e] = off;
        a.ws.expert_count[e] = c;
        if (a.dbg.expert_counts) a.dbg.expert_counts[e] = c;
        for (int s = 0; s < segs; ++s) {
          const int si = nseg + sincl - segs + s;
          a.ws.seg_expert[si] = e;
          a.ws.seg_offset[si] = off + s * kSegTokens;
          a.ws.seg_count[si] = min(kSegTokens, c - s * kSegTokens);
        }
      }
      ndisp += __popc(__ballot_sync(0xffffffffu, c > 0));
      run += __shfl_sync(0xffffffffu, incl, 31);
      nseg += __shfl_sync(0xffffffffu, sincl, 31);
    }
    if (lane == 0) {
      s_off[E] = run;
      a.ws.expert_offset[E] = run;
      a.ws.counters[kCtrDispatched] = ndisp;
      a.ws.counters[kCtrSegments] = nseg;
      a.ws.counters[kCtrSlots] = run;
      if (a.dbg.n_dispatched) a.dbg.n_dispatched[0] = ndisp;
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < S; i += blockDim.x) {
    const int e = s_eids[i];
    int slot = -1;
    if (e >= 0) {
      slot = s_off[e] + s_pos[i];
      a.ws.slot_token[slot] = i / K;
    }
    a.ws.token_slot[i] = slot;
  }
  for (int e = threadIdx.x; e < E; e += blockDim.x) a.ws.counters[kCtrReady + e] = 0;
  if (threadIdx.x == 0) {
    a.ws.counters[kCtrStatus] = s_status;
    a.ws.counters[kCtrTicket] = 0;
    if (a.dbg.status) a.dbg.status[0] = s_status;
  }
}

size_t routing_smem_bytes(int T, int E, int K) {
  const size_t S = size_t(T) * K;
  return 3 * S * 4 + 2 * size_t(T) * 4 + size_t(E) * 4 + size_t(E) * 4 + size_t(E + 1) * 4 + size_t(E) + 16;
}

cudaError_t launch_routing(const RoutingArgs& a, cudaStream_t st) {
  const size_t smem = routing_smem_bytes(a.T, a.E, a.K);
  static thread_local size_t configured = 0;
  if (smem > 48 * 1024 && smem > configured) {
    cudaError_t e = cudaFuncSetAttribute(routing_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    if (e != cudaSuccess) return e;
    configured = smem;
  }
  int threads = 32 * max(4, min(32, max(a.T, (a.E + 31) / 32)));
  routing_kernel<<<1, threads, smem, st>>>(a);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Gather the token inputs into expert-sorted order: x_sorted[slot] = hidden[slot_token[slot]].
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) gather_kernel(const __nv_bfloat16* __restrict__ hidden,
                                                     const int32_t* __restrict__ slot_token,
                                                     const int32_t* __restrict__ counters,
                                                     __nv_bfloat16* __restrict__ x_sorted, int d) {
  const int slot = blockIdx.x;
  if (slot >= counters[kCtrSlots]) return;
  const int t = slot_token[slot];
  const uint4* src = reinterpret_cast<const uint4*>(hidden + size_t(t) * d);
  uint4* dst = reinterpret_cast<uint4*>(x_sorted + size_t(slot) * d);
  for (int j = threadIdx.x; j < (d >> 3); j += blockDim.x) dst[j] = __ldg(src + j);
}

cudaError_t launch_gather(const void* hidden, const Workspace& ws, int T, int K, int d, cudaStream_t st) {
  gather_kernel<<<T * K, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(hidden), ws.slot_token, ws.counters,
                                       ws.x_sorted, d);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Combine: y[t] = sum_k gate[t,k] * ypair[row(t,k)] in slot order k = 0..K-1 (deterministic).
// With x_next != nullptr also writes rmsnorm(hidden[t] + y[t]) (no gain) as bf16: the wiring
// between consecutive layers of the stack workload.
// ------------------------------------------------------------------------------------------------
constexpr int kCombineIters = 8;  // d <= 256 threads * 4 * 8 = 8192

__global__ void __launch_bounds__(256) combine_kernel(const float* __restrict__ ypair,
                                                      const int32_t* __restrict__ token_slot,
                                                      const float* __restrict__ gates,
                                                      const __nv_bfloat16* __restrict__ hidden, void* __restrict__ out,
                                                      int out_is_fp32, __nv_bfloat16* __restrict__ x_next, int K,
                                                      int d) {
  const int t = blockIdx.x;
  __shared__ int s_slot[kMaxK];
  __shared__ float s_gate[kMaxK];
  __shared__ float s_red[8];
  if (threadIdx.x < K) {
    s_slot[threadIdx.x] = token_slot[t * K + threadIdx.x];
    s_gate[threadIdx.x] = gates[t * K + threadIdx.x];
  }
  __syncthreads();
  float4 keep[kCombineIters];
  float ss = 0.f;
#pragma unroll
  for (int it = 0; it < kCombineIters; ++it) {
    const int c = (it * 256 + threadIdx.x) * 4;
    if (c >= d) break;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int k = 0; k < K; ++k) {
      const int slot = s_slot[k];
      if (slot < 0) continue;
      const float g = s_gate[k];
      const float4 v = *reinterpret_cast<const float4*>(ypair + size_t(slot) * d + c);
      acc.x = fmaf(g, v.x, acc.x);
      acc.y = fmaf(g, v.y, acc.y);
      acc.z = fmaf(g, v.z, acc.z);
      acc.w = fmaf(g, v.w, acc.w);
    }
    if (out) {
      if (out_is_fp32) {
        *reinterpret_cast<float4*>(static_cast<float*>(out) + size_t(t) * d + c) = acc;
      } else {
        __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
        uint2 p;
        p.x = *reinterpret_cast<uint32_t*>(&lo);
        p.y = *reinterpret_cast<uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(out) + size_t(t) * d + c) = p;
      }
    }
    if (x_next) {
      const uint2 hx = *reinterpret_cast<const uint2*>(hidden + size_t(t) * d + c);
      acc.x += __uint_as_float(hx.x << 16);
      acc.y += __uint_as_float(hx.x & 0xffff0000u);
      acc.z += __uint_as_float(hx.y << 16);
      acc.w += __uint_as_float(hx.y & 0xffff0000u);
      ss += acc.x * acc.x + acc.y * acc.y + acc.z * acc.z + acc.w * acc.w;
      keep[it] = acc;
    }
  }
  if (!x_next) return;
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) tot += s_red[i];
  const float r = rsqrtf(tot / float(d));
#pragma unroll
  for (int it = 0; it < kCombineIters; ++it) {
    const int c = (it * 256 + threadIdx.x) * 4;
    if (c >= d) break;
    const float4 v = keep[it];
    __nv_bfloat162 lo = __floats2bfloat162_rn(v.x * r, v.y * r), hi = __floats2bfloat162_rn(v.z * r, v.w * r);
    uint2 p;
    p.x = *reinterpret_cast<uint32_t*>(&lo);
    p.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(x_next + size_t(t) * d + c) = p;
  }
}

cudaError_t launch_combine(const Workspace& ws, const void* hidden, void* out, int out_is_fp32, void* x_next,
                           int T, int K, int d, cudaStream_t st) {
  combine_kernel<<<T, 256, 0, st>>>(ws.ypair, ws.token_slot, ws.exec_gates,
                                    static_cast<const __nv_bfloat16*>(hidden), out, out_is_fp32,
                                    static_cast<__nv_bfloat16*>(x_next), K, d);
  return cudaGetLastError();
}

}  // namespace base
