// Token entropy (paper Sec. 3.1, Eq. 2) from logits that already exist in memory.
// A serving engine that has just run its LM head for sampling holds the [rows, V] logits of the
// step; the entropy then costs one pass over those values instead of a second LM-head GEMM.
// HBM-bound: 16-byte coalesced loads, one running (m, s, t2) per thread (same definition as the
// LM-head kernel's epilogue), warp-shuffle and shared-memory combine, one partial per
// (row, vocabulary split) in the layout the merge kernels read; when the caller wants H itself, the last block
// of a row to finish merges the row's partials, so that entropy from logits is a single launch.
#include "kernels.h"
#include "entropy_merge.cuh"
#include "sm100_ptx.cuh"
#include "../../include/egtp.h"

#include <cuda_bf16.h>

#include <algorithm>

namespace egtp {

namespace {

constexpr int kLogitsThreads = 128;
constexpr int kLogitsBlocksPerSm = 8;   // 64 registers per thread at most: 32 warps per SM
constexpr float kLog2e = 1.4426950408889634f;

// Eight consecutive logits as they come out of memory.  bf16 values stay packed until they are consumed: the
// maximum of the eight is taken on the packed pairs (exact: the maximum of bf16 numbers is one of them), and
// a value is widened to fp32 (a shift or a mask) only where the exponential needs it.
template <typename T>
struct Vec8;
template <>
struct Vec8<__nv_bfloat16> {
  uint4 q;
  __device__ __forceinline__ void load(const __nv_bfloat16* p) { q = __ldcs(reinterpret_cast<const uint4*>(p)); }   // streamed once
  __device__ __forceinline__ float vmax() const {
    const __nv_bfloat162 a = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&q.x), *reinterpret_cast<const __nv_bfloat162*>(&q.y));
    const __nv_bfloat162 b = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&q.z), *reinterpret_cast<const __nv_bfloat162*>(&q.w));
    const __nv_bfloat162 c = __hmax2(a, b);
    const uint32_t w = *reinterpret_cast<const uint32_t*>(&c);
    return fmaxf(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u));
  }
  __device__ __forceinline__ void get(float (&v)[8]) const {
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
};
template <>
struct Vec8<float> {
  float4 a, b;
  __device__ __forceinline__ void load(const float* p) {
    a = __ldcs(reinterpret_cast<const float4*>(p));
    b = __ldcs(reinterpret_cast<const float4*>(p) + 1);
  }
  __device__ __forceinline__ float vmax() const {
    return fmaxf(fmaxf(fmaxf(a.x, a.y), fmaxf(a.z, a.w)), fmaxf(fmaxf(b.x, b.y), fmaxf(b.z, b.w)));
  }
  __device__ __forceinline__ void get(float (&v)[8]) const {
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
    v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
  }
};

// vectors of eight logits a thread has in flight while it folds the previous ones: 64 bytes either way
template <typename T>
constexpr int kVecPerBatch = sizeof(T) == 2 ? 4 : 2;

// Running state of one thread: max m and four independent (s, t2) accumulators kept as two packed pairs, so that
// the three fp32 operations per logit besides the exponential (y = x log2 e - m log2 e, s += e, t2 += e y) are
// issued two logits at a time (fma / add on f32x2).
struct ThreadState {
  float m;
  uint64_t s[2];
  uint64_t t[2];
  __device__ __forceinline__ void init() {
    m = kNegBig;
    s[0] = s[1] = t[0] = t[1] = pack_f32x2(0.f, 0.f);
  }
  __device__ __forceinline__ void raise_max(float cmax) {
    if (cmax > m) {
      // new running max: s <- s r, t2 <- r (t2 + dm s) with dm = (m - cmax) log2 e, r = 2^dm
      const float dm = (m - cmax) * kLog2e;
      const float r = ex2_approx(dm);
      const uint64_t r2 = pack_f32x2(r, r), dm2 = pack_f32x2(dm, dm);
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        t[i] = mul_f32x2(r2, fma_f32x2(dm2, s[i], t[i]));
        s[i] = mul_f32x2(s[i], r2);
      }
      m = cmax;
    }
  }
  // kN vectors of eight values at once: one running-max update, then 8 kN independent exponentials
  template <typename T, int kN>
  __device__ __forceinline__ void fold(const Vec8<T> (&x)[kN]) {
    float cmax = x[0].vmax();
#pragma unroll
    for (int u = 1; u < kN; ++u) cmax = fmaxf(cmax, x[u].vmax());
    raise_max(cmax);
    const float neg_m_l2 = -m * kLog2e;
    const uint64_t l2 = pack_f32x2(kLog2e, kLog2e), nm2 = pack_f32x2(neg_m_l2, neg_m_l2);
#pragma unroll
    for (int u = 0; u < kN; ++u) {
      float v[8];
      x[u].get(v);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint64_t y2 = fma_f32x2(pack_f32x2(v[2 * j], v[2 * j + 1]), l2, nm2);
        float y0, y1;
        unpack_f32x2(y2, y0, y1);
        const uint64_t e2 = pack_f32x2(ex2_approx(y0), ex2_approx(y1));
        s[j & 1] = add_f32x2(s[j & 1], e2);
        t[j & 1] = fma_f32x2(e2, y2, t[j & 1]);
      }
    }
  }
  __device__ __forceinline__ EntropyPartial total() const {
    float s0, s1, s2, s3, t0, t1, t2, t3;
    unpack_f32x2(s[0], s0, s1); unpack_f32x2(s[1], s2, s3);
    unpack_f32x2(t[0], t0, t1); unpack_f32x2(t[1], t2, t3);
    return {m, (s0 + s1) + (s2 + s3), (t0 + t1) + (t2 + t3)};
  }
};

template <typename T>
__device__ __forceinline__ float to_float(T v);
template <>
__device__ __forceinline__ float to_float<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_float<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// block (split, row): columns [split * cols_per_split, ...) of one row.  The loads of the next batch of vectors are
// issued before the current batch is folded, so that every warp keeps memory requests in flight while it computes
// (one ex2 and about five other instructions per logit: the arithmetic alone takes most of the time the memory
// system needs to deliver the row).
template <typename T>
__global__ void __launch_bounds__(kLogitsThreads, kLogitsBlocksPerSm)
logits_entropy_kernel(const T* __restrict__ logits, int64_t ldl, int V, int cols_per_split, int splits,
                      float* __restrict__ partials, float* __restrict__ H_out, int32_t* __restrict__ arrivals,
                      const int32_t* __restrict__ status) {
  if (*status != 0) return;
  __shared__ EntropyPartial red[kLogitsThreads / 32];
  __shared__ int is_last;
  const int64_t row = blockIdx.x / splits;
  const int split = static_cast<int>(blockIdx.x - row * splits);
  const int c0 = split * cols_per_split;
  const int c1 = min(V, c0 + cols_per_split);
  const T* base = logits + row * ldl + c0;
  ThreadState ts;
  ts.init();
  const int n_vec = max(0, c1 - c0) >> 3;                       // cols_per_split is a multiple of 8
  constexpr int kN = kVecPerBatch<T>;
  constexpr int kBatch = kN * kLogitsThreads;                    // vectors per block and batch
  const int n_batches = n_vec / kBatch;
  const T* p = base + 8 * threadIdx.x;
  Vec8<T> cur[kN], nxt[kN];
  if (n_batches > 0) {
#pragma unroll
    for (int u = 0; u < kN; ++u) cur[u].load(p + 8 * u * kLogitsThreads);
  }
  for (int b = 0; b < n_batches; ++b) {
    p += 8 * kBatch;
    if (b + 1 < n_batches) {
#pragma unroll
      for (int u = 0; u < kN; ++u) nxt[u].load(p + 8 * u * kLogitsThreads);
    }
    ts.fold<T, kN>(cur);
#pragma unroll
    for (int u = 0; u < kN; ++u) cur[u] = nxt[u];
  }
  for (int v = n_batches * kBatch + threadIdx.x; v < n_vec; v += kLogitsThreads) {
    Vec8<T> one[1];
    one[0].load(base + 8 * v);
    ts.fold<T, 1>(one);
  }
  EntropyPartial st = ts.total();
  // ragged tail of the row (fewer than 8 columns), handled by one thread
  if (threadIdx.x == 0) {
    for (int c = c0 + 8 * n_vec; c < c1; ++c) {
      const EntropyPartial one = {to_float<T>(logits[row * ldl + c]), 1.f, 0.f};
      st = combine_partials(st, one);
    }
  }
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  st = warp_combine_partials(st);
  if (lane == 0) red[wid] = st;
  __syncthreads();
  if (threadIdx.x == 0) {
    EntropyPartial acc = red[0];
    for (int w = 1; w < kLogitsThreads / 32; ++w) acc = combine_partials(acc, red[w]);
    float* dst = partials + (row * splits + split) * 3;
    dst[0] = acc.m; dst[1] = acc.s; dst[2] = acc.t2;
    if (H_out != nullptr) {
      // the block that finds all other partials of its row already written merges them (slot order, so the result
      // does not depend on which block that is) and leaves the row's arrival counter at zero for the next call
      __threadfence();
      is_last = atomicAdd(arrivals + row, 1) == splits - 1 ? 1 : 0;
    }
  }
  if (H_out == nullptr) return;
  __syncthreads();
  if (is_last == 0 || wid != 0) return;
  __threadfence();
  const float h = merge_partials_warp(partials + row * splits * 3, splits, 3, lane);
  if (lane == 0) {
    H_out[row] = h;
    arrivals[row] = 0;
  }
}

}  // namespace

int logits_entropy_pick_splits(int64_t rows, int V, int num_sms) {
  // One wave of blocks: seven 128-thread blocks per SM fit at once (kLogitsBlocksPerSm), and every thread should see a few
  // hundred logits so that the per-block combine is amortised; never less than 2K columns per block.
  int64_t splits = std::max<int64_t>(1, (static_cast<int64_t>(kLogitsBlocksPerSm) * num_sms) / std::max<int64_t>(rows, 1));
  splits = std::min<int64_t>(splits, std::max(1, V / 2048));
  return static_cast<int>(std::max<int64_t>(1, std::min<int64_t>(splits, 128)));
}

cudaError_t launch_logits_entropy(const void* logits, int64_t ldl, bool bf16, int64_t rows, int V, int splits,
                                  float* partials, float* H_out, int32_t* arrivals, const int32_t* status,
                                  cudaStream_t stream) {
  int cols_per_split = (V + splits - 1) / splits;
  cols_per_split = (cols_per_split + 7) / 8 * 8;
  if (rows * splits >= (int64_t{1} << 31) || (H_out != nullptr && arrivals == nullptr)) return cudaErrorInvalidValue;
  const unsigned grid = static_cast<unsigned>(rows * splits);      // block = (row, split), splits of a row adjacent
  if (bf16) {
    logits_entropy_kernel<__nv_bfloat16><<<grid, kLogitsThreads, 0, stream>>>(
        static_cast<const __nv_bfloat16*>(logits), ldl, V, cols_per_split, splits, partials, H_out, arrivals, status);
  } else {
    logits_entropy_kernel<float><<<grid, kLogitsThreads, 0, stream>>>(static_cast<const float*>(logits), ldl, V,
                                                                     cols_per_split, splits, partials, H_out, arrivals,
                                                                     status);
  }
  return cudaGetLastError();
}

}  // namespace egtp
