// Plain CUDA-core grouped SwiGLU FFN over the dispatched experts. This is the simple, easily
// checked implementation (opt->ffn_impl = 1): every warp owns four weight rows and streams them
// with 128-bit loads against eight tokens at a time. The tensor-core streaming kernels are the
// default path; this one exists to cross-check them on the device.
#include "common.cuh"

namespace base {

constexpr int kRowsPerWarp = 4;
constexpr int kTokChunk = 8;
constexpr int kRowsPerCta = 8 * kRowsPerWarp;

// h[row, i] = silu(W_gate[e,i,:] . x_row) * (W_up[e,i,:] . x_row) for the expert's sorted rows.
__global__ void __launch_bounds__(256) ffn1_simple_kernel(const __nv_bfloat16* __restrict__ w_gate,
                                                          const __nv_bfloat16* __restrict__ w_up,
                                                          const __nv_bfloat16* __restrict__ x_sorted,
                                                          const int32_t* __restrict__ expert_count,
                                                          const int32_t* __restrict__ expert_offset,
                                                          __nv_bfloat16* __restrict__ h, int d, int I) {
  const int e = blockIdx.y;
  const int cnt = expert_count[e];
  if (cnt == 0) return;
  const int off = expert_offset[e];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int row0 = blockIdx.x * kRowsPerCta + warp * kRowsPerWarp;
  if (row0 >= I) return;
  const __nv_bfloat16* wg = w_gate + (size_t(e) * I + row0) * d;
  const __nv_bfloat16* wu = w_up + (size_t(e) * I + row0) * d;
  for (int n0 = 0; n0 < cnt; n0 += kTokChunk) {
    float ag[kRowsPerWarp][kTokChunk], au[kRowsPerWarp][kTokChunk];
#pragma unroll
    for (int r = 0; r < kRowsPerWarp; ++r)
#pragma unroll
      for (int n = 0; n < kTokChunk; ++n) ag[r][n] = au[r][n] = 0.f;
    for (int j = lane * 8; j < d; j += 256) {
      float fx[kTokChunk][8];
#pragma unroll
      for (int n = 0; n < kTokChunk; ++n) {
        if (n0 + n < cnt) {
          unpack8(ldg16(x_sorted + size_t(off + n0 + n) * d + j), fx[n]);
        } else {
#pragma unroll
          for (int i = 0; i < 8; ++i) fx[n][i] = 0.f;
        }
      }
#pragma unroll
      for (int r = 0; r < kRowsPerWarp; ++r) {
        float fg[8], fu[8];
        unpack8(ldg16(wg + size_t(r) * d + j), fg);
        unpack8(ldg16(wu + size_t(r) * d + j), fu);
#pragma unroll
        for (int n = 0; n < kTokChunk; ++n)
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            ag[r][n] = fmaf(fg[i], fx[n][i], ag[r][n]);
            au[r][n] = fmaf(fu[i], fx[n][i], au[r][n]);
          }
      }
    }
    float myg = 0.f, myu = 0.f;
#pragma unroll
    for (int r = 0; r < kRowsPerWarp; ++r)
#pragma unroll
      for (int n = 0; n < kTokChunk; ++n) {
        const float g = warp_sum(ag[r][n]);
        const float u = warp_sum(au[r][n]);
        if (lane == r * kTokChunk + n) {
          myg = g;
          myu = u;
        }
      }
    const int r = lane / kTokChunk, n = lane % kTokChunk;
    if (n0 + n < cnt) h[size_t(off + n0 + n) * I + row0 + r] = __float2bfloat16_rn(silu_f(myg) * myu);
  }
}

// ypair[row, c] = W_down[e,c,:] . h[row,:]
__global__ void __launch_bounds__(256) ffn2_simple_kernel(const __nv_bfloat16* __restrict__ w_down,
                                                          const __nv_bfloat16* __restrict__ h,
                                                          const int32_t* __restrict__ expert_count,
                                                          const int32_t* __restrict__ expert_offset,
                                                          float* __restrict__ ypair, int d, int I) {
  const int e = blockIdx.y;
  const int cnt = expert_count[e];
  if (cnt == 0) return;
  const int off = expert_offset[e];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int row0 = blockIdx.x * kRowsPerCta + warp * kRowsPerWarp;
  if (row0 >= d) return;
  const __nv_bfloat16* wd = w_down + (size_t(e) * d + row0) * I;
  for (int n0 = 0; n0 < cnt; n0 += kTokChunk) {
    float acc[kRowsPerWarp][kTokChunk];
#pragma unroll
    for (int r = 0; r < kRowsPerWarp; ++r)
#pragma unroll
      for (int n = 0; n < kTokChunk; ++n) acc[r][n] = 0.f;
    for (int j = lane * 8; j < I; j += 256) {
      float fh[kTokChunk][8];
#pragma unroll
      for (int n = 0; n < kTokChunk; ++n) {
        if (n0 + n < cnt) {
          unpack8(ldg16(h + size_t(off + n0 + n) * I + j), fh[n]);
        } else {
#pragma unroll
          for (int i = 0; i < 8; ++i) fh[n][i] = 0.f;
        }
      }
#pragma unroll
      for (int r = 0; r < kRowsPerWarp; ++r) {
        float fw[8];
        unpack8(ldg16(wd + size_t(r) * I + j), fw);
#pragma unroll
        for (int n = 0; n < kTokChunk; ++n)
#pragma unroll
          for (int i = 0; i < 8; ++i) acc[r][n] = fmaf(fw[i], fh[n][i], acc[r][n]);
      }
    }
    float mine = 0.f;
#pragma unroll
    for (int r = 0; r < kRowsPerWarp; ++r)
#pragma unroll
      for (int n = 0; n < kTokChunk; ++n) {
        const float v = warp_sum(acc[r][n]);
        if (lane == r * kTokChunk + n) mine = v;
      }
    const int r = lane / kTokChunk, n = lane % kTokChunk;
    if (n0 + n < cnt) ypair[size_t(off + n0 + n) * d + row0 + r] = mine;
  }
}

cudaError_t launch_ffn_simple(const base_layer_shape& s, const base_layer_weights& w, const Workspace& ws,
                              cudaStream_t st, int* launches) {
  dim3 g1((s.I + kRowsPerCta - 1) / kRowsPerCta, s.E);
  // h is read before it is fully written only across kernels, never inside one: two launches.
  ffn1_simple_kernel<<<g1, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(w.w_gate),
                                         static_cast<const __nv_bfloat16*>(w.w_up), ws.x_sorted, ws.expert_count,
                                         ws.expert_offset, ws.h, s.d, s.I);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  dim3 g2((s.d + kRowsPerCta - 1) / kRowsPerCta, s.E);
  ffn2_simple_kernel<<<g2, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(w.w_down), ws.h, ws.expert_count,
                                         ws.expert_offset, ws.ypair, s.d, s.I);
  *launches += 2;
  return cudaGetLastError();
}

}  // namespace base
