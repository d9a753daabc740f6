// Grouped SwiGLU expert FFN for sm_100a: TMA-staged weight streaming + tcgen05 MMA with TMEM
// accumulators (Eq. moe_latency: the step is bound by fetching the dispatched experts' weights).
//
// Orientation ("swap-AB"): the weight rows are the MMA M axis (128 rows per tile, K-major, streamed
// once, fully sequential in DRAM), the expert's tokens are the N axis (16..128 per work unit).
//   gate/up pass: A = [64 rows of W_gate ; the same 64 rows of W_up] (two TMA boxes stacked in one
//                 128-row tile), B = the expert's token inputs, D[0:64] = gate, D[64:128] = up;
//                 epilogue: h = silu(gate) * up -> bf16, expert-sorted rows.
//   down pass:    A = 128 rows of W_down, B = the expert's h rows, D -> fp32 output per routed pair.
// One persistent CTA per SM, warp-specialised: warp 0 issues TMA, warp 1 issues MMA and owns the
// TMEM allocation, warps 2-5 drain the accumulators. Shared-memory stages and the two accumulator
// stages are handed over with mbarriers, so the weight stream never waits for an epilogue.
// Every wait is bounded: on expiry the CTA raises an abort flag, all roles leave their loops, TMEM
// is freed and BASE_DEV_WAIT_EXPIRED is OR-ed into the status word.
#include <cuda.h>

#include <mutex>
#include <unordered_map>

#include "ffn_tc.cuh"

namespace base {

namespace {

constexpr int kStages = 5;
constexpr int kBlockK = 64;                 // bf16 per k-block = one 128-byte swizzled row
constexpr int kTileABytes = 128 * 128;      // 128 rows x 128 B
constexpr int kTileBBytes = kSegTokens * 128;
constexpr int kStageBytes = kTileABytes + kTileBBytes;
constexpr int kExBytes = kSegTokens * 64 * 4;  // up-projection exchange buffer [token][row] fp32
constexpr int kThreads = 192;
constexpr int kAccCols = kSegTokens;        // TMEM columns per accumulator stage
constexpr int kTmemCols = 2 * kAccCols;
constexpr int kBoxRowsB = 16;
constexpr uint32_t kSpinLimit = 1u << 22;
constexpr unsigned long long kWaitNs = 2000000000ull;  // 2 s

struct Bars {
  unsigned long long full[kStages];
  unsigned long long empty[kStages];
  unsigned long long acc_full[2];
  unsigned long long acc_empty[2];
  uint32_t tmem_base;
  int abort_flag;
};

constexpr size_t kSmemBytes = 1024 + size_t(kStages) * kStageBytes + kExBytes + sizeof(Bars) + 64;

struct FfnParams {
  const int32_t* seg_expert;
  const int32_t* seg_offset;
  const int32_t* seg_count;
  int32_t* counters;
  __nv_bfloat16* h;   // gate/up pass output
  float* ypair;       // down pass output
  int rows_per_expert;  // I (gate/up) or d (down): rows of one expert in the A tensor map
  int tiles;            // work units per segment
  int kblocks;          // K extent / 64
  int I, d;
};

// ------------------------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait. Returns false when the wait ran out or another role has raised the abort flag.
__device__ __noinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 63u) == 63u) {
      if (*abort_flag) return false;
      if (global_ns() - t0 > kWaitNs) break;
      __nanosleep(64);
    }
  }
  if (mbar_try_wait(bar, parity)) return true;
  *abort_flag = 1;
  return false;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(tm), "r"(x), "r"(y), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void tcgen05_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}

// D[tmem] (+)= A[smem] * B[smem], bf16 inputs, fp32 accumulate, M=128, K=16.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// 16 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// K-major, 128-byte swizzled operand tile: rows of 128 B, 8-row groups 1024 B apart.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr) {
  const uint32_t lo = ((saddr & 0x3FFFFu) >> 4) | (1u << 16);
  const uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);
  return (uint64_t(hi) << 32) | lo;
}
// kind::f16 instruction descriptor: fp32 accumulate, bf16 x bf16, both K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t make_idesc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(n >> 3) << 17) | (uint32_t(128 >> 4) << 24);
}

__device__ __forceinline__ void named_sync(int id, int threads) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory"); }
__device__ __forceinline__ void named_arrive(int id, int threads) { asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(threads) : "memory"); }
// AND-reduction of a predicate over the `threads` threads meeting at barrier `id`.
__device__ __forceinline__ bool named_and(int id, int threads, bool pred) {
  uint32_t out;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.b32 p, %3, 0;\n\t"
      "barrier.cta.red.and.pred q, %1, %2, p;\n\t"
      "selp.u32 %0, 1, 0, q;\n\t}"
      : "=r"(out)
      : "r"(id), "r"(threads), "r"(uint32_t(pred))
      : "memory");
  return out != 0;
}

struct Unit {
  int expert, offset, count, npad, tile;
};

__device__ __forceinline__ Unit decode_unit(const FfnParams& p, int u) {
  Unit r;
  const int seg = u / p.tiles;
  r.tile = u - seg * p.tiles;
  r.expert = p.seg_expert[seg];
  r.offset = p.seg_offset[seg];
  r.count = p.seg_count[seg];
  r.npad = (r.count + 15) & ~15;
  return r;
}

// ------------------------------------------------------------------------------------------- the kernel
template <int kPhase>
__global__ void __launch_bounds__(kThreads, 1)
ffn_tc_kernel(const __grid_constant__ CUtensorMap tm_a0, const __grid_constant__ CUtensorMap tm_a1,
              const __grid_constant__ CUtensorMap tm_b, const FfnParams p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* base_ptr = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* stages = base_ptr;
  float* ex = reinterpret_cast<float*>(base_ptr + size_t(kStages) * kStageBytes);
  Bars* bars = reinterpret_cast<Bars*>(base_ptr + size_t(kStages) * kStageBytes + kExBytes);
  volatile int* abort_flag = &bars->abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_units = p.counters[kCtrSegments] * p.tiles;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&bars->full[s]), 1);
      mbar_init(smem_u32(&bars->empty[s]), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(smem_u32(&bars->acc_full[a]), 1);
      mbar_init(smem_u32(&bars->acc_empty[a]), 128);
    }
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_a0) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_b) : "memory");
    if (kPhase == 1) asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_a1) : "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(&bars->tmem_base), kTmemCols);
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem_base = bars->tmem_base;

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < n_units && ok; u += gridDim.x) {
        const Unit un = decode_unit(p, u);
        const int arow = un.expert * p.rows_per_expert + un.tile * (kPhase == 1 ? 64 : 128);
        for (int kb = 0; kb < p.kblocks; ++kb) {
          if (!mbar_wait(smem_u32(&bars->empty[stage]), phase ^ 1u, abort_flag)) {
            ok = false;
            break;
          }
          const uint32_t full = smem_u32(&bars->full[stage]);
          const uint32_t sa = smem_u32(stages + size_t(stage) * kStageBytes);
          const uint32_t sb = sa + kTileABytes;
          mbar_expect_tx(full, uint32_t(kTileABytes + un.npad * 128));
          if (kPhase == 1) {
            tma_load_2d(sa, &tm_a0, kb * kBlockK, arow, full);
            tma_load_2d(sa + kTileABytes / 2, &tm_a1, kb * kBlockK, arow, full);
          } else {
            tma_load_2d(sa, &tm_a0, kb * kBlockK, arow, full);
          }
          for (int j = 0; j < un.npad; j += kBoxRowsB) tma_load_2d(sb + j * 128, &tm_b, kb * kBlockK, un.offset + j, full);
          if (++stage == kStages) {
            stage = 0;
            phase ^= 1u;
          }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < n_units && ok; u += gridDim.x) {
        const Unit un = decode_unit(p, u);
        if (!mbar_wait(smem_u32(&bars->acc_empty[acc]), acc_phase ^ 1u, abort_flag)) break;
        tcgen05_fence_after();
        const uint32_t d_tmem = tmem_base + uint32_t(acc * kAccCols);
        const uint32_t idesc = make_idesc(un.npad);
        for (int kb = 0; kb < p.kblocks; ++kb) {
          if (!mbar_wait(smem_u32(&bars->full[stage]), phase, abort_flag)) {
            ok = false;
            break;
          }
          tcgen05_fence_after();
          const uint32_t sa = smem_u32(stages + size_t(stage) * kStageBytes);
          const uint64_t adesc = make_smem_desc(sa);
          const uint64_t bdesc = make_smem_desc(sa + kTileABytes);
#pragma unroll
          for (int k4 = 0; k4 < kBlockK / 16; ++k4)
            umma_bf16(d_tmem, adesc + uint64_t(k4 * 2), bdesc + uint64_t(k4 * 2), idesc, uint32_t((kb | k4) != 0));
          umma_commit(smem_u32(&bars->empty[stage]));
          if (++stage == kStages) {
            stage = 0;
            phase ^= 1u;
          }
        }
        if (!ok) break;
        umma_commit(smem_u32(&bars->acc_full[acc]));
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      }
    }
    __syncwarp();
  } else {
    // ---------------------------------------------------------------- epilogue warps (TMEM -> global)
    const int q = warp & 3;  // TMEM lane quarter this warp may read
    int acc = 0;
    uint32_t acc_phase = 0;
    for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
      const Unit un = decode_unit(p, u);
      const bool got = mbar_wait(smem_u32(&bars->acc_full[acc]), acc_phase, abort_flag);
      if (!named_and(1, 128, got)) break;
      tcgen05_fence_after();
      const uint32_t taddr = tmem_base + (uint32_t(q * 32) << 16) + uint32_t(acc * kAccCols);
      if (kPhase == 1) {
        const int r = (q & 1) * 32 + lane;  // row inside the 64-row slice
        if (q >= 2) {
          // up rows: park them in shared memory for the gate warps
          named_sync(3, 128);  // the gate warps have finished reading the previous unit's values
          for (int c0 = 0; c0 < un.npad; c0 += 16) {
            float v[16];
            tmem_ld16(taddr + c0, v);
#pragma unroll
            for (int c = 0; c < 16; ++c) ex[(c0 + c) * 64 + r] = v[c];
          }
          tcgen05_fence_before();
          mbar_arrive(smem_u32(&bars->acc_empty[acc]));
          __threadfence_block();
          named_arrive(2, 128);
        } else {
          named_arrive(3, 128);
          named_sync(2, 128);  // up values are in shared memory
          __nv_bfloat16* hrow = p.h + size_t(un.offset) * p.I + un.tile * 64 + r;
          for (int c0 = 0; c0 < un.npad; c0 += 16) {
            float v[16];
            tmem_ld16(taddr + c0, v);
#pragma unroll
            for (int c = 0; c < 16; ++c) {
              if (c0 + c < un.count) {
                const float up = ex[(c0 + c) * 64 + r];
                hrow[size_t(c0 + c) * p.I] = __float2bfloat16_rn(silu_f(v[c]) * up);
              }
            }
          }
          tcgen05_fence_before();
          mbar_arrive(smem_u32(&bars->acc_empty[acc]));
        }
      } else {
        float* yrow = p.ypair + size_t(un.offset) * p.d + un.tile * 128 + q * 32 + lane;
        for (int c0 = 0; c0 < un.npad; c0 += 16) {
          float v[16];
          tmem_ld16(taddr + c0, v);
#pragma unroll
          for (int c = 0; c < 16; ++c)
            if (c0 + c < un.count) yrow[size_t(c0 + c) * p.d] = v[c];
        }
        tcgen05_fence_before();
        mbar_arrive(smem_u32(&bars->acc_empty[acc]));
      }
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    }
  }

  // ---------------------------------------------------------------- teardown
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
  if (threadIdx.x == 0 && bars->abort_flag) atomicOr(&p.counters[kCtrStatus], BASE_DEV_WAIT_EXPIRED);
}

// ------------------------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      f = nullptr;
    return reinterpret_cast<EncodeTiledFn>(f);
  }();
  return fn;
}

struct MapKey {
  const void* ptr;
  uint64_t rows, cols;
  uint32_t box_rows;
  bool operator==(const MapKey& o) const { return ptr == o.ptr && rows == o.rows && cols == o.cols && box_rows == o.box_rows; }
};
struct MapKeyHash {
  size_t operator()(const MapKey& k) const {
    size_t h = reinterpret_cast<size_t>(k.ptr);
    h ^= k.rows * 0x9E3779B97F4A7C15ull + (h << 6) + (h >> 2);
    h ^= k.cols * 0xBF58476D1CE4E5B9ull + (h << 6) + (h >> 2);
    h ^= k.box_rows * 0x94D049BB133111EBull + (h << 6) + (h >> 2);
    return h;
  }
};

// 2-D bf16 tensor [rows, cols] (cols contiguous), box = [box_rows, 64 cols], 128-byte swizzle. Cached: the
// encoding is a pure function of the key.
bool tensor_map_2d(const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows, CUtensorMap* out) {
  static std::mutex mu;
  static std::unordered_map<MapKey, CUtensorMap, MapKeyHash> cache;
  const MapKey key{ptr, rows, cols, box_rows};
  {
    std::lock_guard<std::mutex> g(mu);
    auto it = cache.find(key);
    if (it != cache.end()) {
      *out = it->second;
      return true;
    }
  }
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * 2};
  const cuuint32_t box[2] = {uint32_t(kBlockK), box_rows};
  const cuuint32_t estr[2] = {1, 1};
  CUtensorMap m;
  CUresult r = fn(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  {
    std::lock_guard<std::mutex> g(mu);
    if (cache.size() > 4096) cache.clear();
    cache.emplace(key, m);
  }
  *out = m;
  return true;
}

int sm_count() {
  static int n = [] {
    int dev = 0, v = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
    return v > 0 ? v : 148;
  }();
  return n;
}

template <int kPhase>
cudaError_t configure() {
  static cudaError_t st = cudaFuncSetAttribute(ffn_tc_kernel<kPhase>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kSmemBytes));
  return st;
}

}  // namespace

cudaError_t launch_ffn_tc(const base_layer_shape& s, const base_layer_weights& w, const Workspace& ws, int T,
                          cudaStream_t st, int* launches) {
  const uint64_t slots = uint64_t(T) * s.K + kRowPad;
  CUtensorMap tm_g, tm_u, tm_x, tm_d, tm_h;
  if (!tensor_map_2d(w.w_gate, uint64_t(s.E) * s.I, s.d, 64, &tm_g) ||
      !tensor_map_2d(w.w_up, uint64_t(s.E) * s.I, s.d, 64, &tm_u) ||
      !tensor_map_2d(ws.x_sorted, slots, s.d, kBoxRowsB, &tm_x) ||
      !tensor_map_2d(w.w_down, uint64_t(s.E) * s.d, s.I, 128, &tm_d) ||
      !tensor_map_2d(ws.h, slots, s.I, kBoxRowsB, &tm_h))
    return cudaErrorInvalidValue;
  cudaError_t e = configure<1>();
  if (e != cudaSuccess) return e;
  e = configure<2>();
  if (e != cudaSuccess) return e;

  const int segs = max_segments(s.E, T, s.K);
  FfnParams p{};
  p.seg_expert = ws.seg_expert;
  p.seg_offset = ws.seg_offset;
  p.seg_count = ws.seg_count;
  p.counters = ws.counters;
  p.h = ws.h;
  p.ypair = ws.ypair;
  p.I = s.I;
  p.d = s.d;

  p.rows_per_expert = s.I;
  p.tiles = s.I / 64;
  p.kblocks = s.d / kBlockK;
  int grid = min(sm_count(), segs * p.tiles);
  ffn_tc_kernel<1><<<grid, kThreads, kSmemBytes, st>>>(tm_g, tm_u, tm_x, p);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;

  p.rows_per_expert = s.d;
  p.tiles = s.d / 128;
  p.kblocks = s.I / kBlockK;
  grid = min(sm_count(), segs * p.tiles);
  ffn_tc_kernel<2><<<grid, kThreads, kSmemBytes, st>>>(tm_d, tm_d, tm_h, p);
  *launches += 2;
  return cudaGetLastError();
}

}  // namespace base
