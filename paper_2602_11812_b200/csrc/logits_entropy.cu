// Token entropy (paper Sec. 3.1, Eq. 2) from logits that already exist in memory.
// A serving engine that has just run its LM head for sampling holds the [rows, V] logits of the
// step; the entropy then costs one pass over those values instead of a second LM-head GEMM.
// HBM-bound: 16-byte coalesced loads, one running (m, s, t2) per thread (same definition as the
// LM-head kernel's epilogue), warp-shuffle and shared-memory combine, one partial per
// (row, vocabulary split) in the layout the merge kernels read.
#include "kernels.h"
#include "entropy_merge.cuh"
#include "sm100_ptx.cuh"
#include "../../include/egtp.h"

#include <cuda_bf16.h>

#include <algorithm>

namespace egtp {

namespace {

constexpr int kLogitsThreads = 128;
constexpr float kLog2e = 1.4426950408889634f;

// Running state of one thread: max m and four independent (s, t2) accumulators (short dependency chains).
struct ThreadState {
  float m;
  float s[4];
  float t[4];
  __device__ __forceinline__ void init() {
    m = kNegBig;
#pragma unroll
    for (int i = 0; i < 4; ++i) { s[i] = 0.f; t[i] = 0.f; }
  }
  __device__ __forceinline__ void fold8(const float (&x)[8]) {
    const float cmax = fmaxf(fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3])), fmaxf(fmaxf(x[4], x[5]), fmaxf(x[6], x[7])));
    if (cmax > m) {
      const float dm = (m - cmax) * kLog2e;
      const float r = ex2_approx(dm);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        t[i] = r * fmaf(dm, s[i], t[i]);
        s[i] *= r;
      }
      m = cmax;
    }
    const float neg_m_l2 = -m * kLog2e;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float y = fmaf(x[j], kLog2e, neg_m_l2);
      const float e = ex2_approx(y);
      s[j & 3] += e;
      t[j & 3] = fmaf(e, y, t[j & 3]);
    }
  }
  // 32 values at once: one running-max update, then 32 independent exponentials (more work in flight)
  __device__ __forceinline__ void fold32(const float (&a)[8], const float (&b)[8], const float (&c)[8],
                                         const float (&d)[8]) {
    float ma = a[0], mb = b[0], mc = c[0], md = d[0];
#pragma unroll
    for (int j = 1; j < 8; ++j) {
      ma = fmaxf(ma, a[j]); mb = fmaxf(mb, b[j]); mc = fmaxf(mc, c[j]); md = fmaxf(md, d[j]);
    }
    const float cmax = fmaxf(fmaxf(ma, mb), fmaxf(mc, md));
    if (cmax > m) {
      const float dm = (m - cmax) * kLog2e;
      const float r = ex2_approx(dm);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        t[i] = r * fmaf(dm, s[i], t[i]);
        s[i] *= r;
      }
      m = cmax;
    }
    const float neg_m_l2 = -m * kLog2e;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float ya = fmaf(a[j], kLog2e, neg_m_l2), yb = fmaf(b[j], kLog2e, neg_m_l2);
      const float yc = fmaf(c[j], kLog2e, neg_m_l2), yd = fmaf(d[j], kLog2e, neg_m_l2);
      const float ea = ex2_approx(ya), eb = ex2_approx(yb), ec = ex2_approx(yc), ed = ex2_approx(yd);
      s[0] += ea; s[1] += eb; s[2] += ec; s[3] += ed;
      t[0] = fmaf(ea, ya, t[0]); t[1] = fmaf(eb, yb, t[1]); t[2] = fmaf(ec, yc, t[2]); t[3] = fmaf(ed, yd, t[3]);
    }
  }
  __device__ __forceinline__ EntropyPartial total() const {
    return {m, (s[0] + s[1]) + (s[2] + s[3]), (t[0] + t[1]) + (t[2] + t[3])};
  }
};

template <typename T>
__device__ __forceinline__ void load8_logits(const T* p, float (&v)[8]);
template <>
__device__ __forceinline__ void load8_logits<__nv_bfloat16>(const __nv_bfloat16* p, float (&v)[8]) {
  const uint4 q = __ldcs(reinterpret_cast<const uint4*>(p));   // streamed once: do not keep in cache
  const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}
template <>
__device__ __forceinline__ void load8_logits<float>(const float* p, float (&v)[8]) {
  const float4 a = __ldcs(reinterpret_cast<const float4*>(p));
  const float4 b = __ldcs(reinterpret_cast<const float4*>(p) + 1);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
  v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
template <typename T>
__device__ __forceinline__ float to_float(T v);
template <>
__device__ __forceinline__ float to_float<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_float<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// block (split, row): columns [split * cols_per_split, ...) of one row
template <typename T>
__global__ void __launch_bounds__(kLogitsThreads)
logits_entropy_kernel(const T* __restrict__ logits, int64_t ldl, int V, int cols_per_split, int splits,
                      float* __restrict__ partials, const int32_t* __restrict__ status) {
  if (*status != 0) return;
  __shared__ EntropyPartial red[kLogitsThreads / 32];
  const int split = blockIdx.x;
  const int64_t row = blockIdx.y;
  const int c0 = split * cols_per_split;
  const int c1 = min(V, c0 + cols_per_split);
  const T* base = logits + row * ldl;
  ThreadState ts;
  ts.init();
  const int n_vec = max(0, c1 - c0) >> 3;                       // cols_per_split is a multiple of 8
  int v = threadIdx.x;
  for (; v + 3 * kLogitsThreads < n_vec; v += 4 * kLogitsThreads) {   // four 16-byte loads in flight
    float x0[8], x1[8], x2[8], x3[8];
    load8_logits<T>(base + c0 + 8 * v, x0);
    load8_logits<T>(base + c0 + 8 * (v + kLogitsThreads), x1);
    load8_logits<T>(base + c0 + 8 * (v + 2 * kLogitsThreads), x2);
    load8_logits<T>(base + c0 + 8 * (v + 3 * kLogitsThreads), x3);
    ts.fold32(x0, x1, x2, x3);
  }
  for (; v < n_vec; v += kLogitsThreads) {
    float x0[8];
    load8_logits<T>(base + c0 + 8 * v, x0);
    ts.fold8(x0);
  }
  EntropyPartial st = ts.total();
  // ragged tail of the row (fewer than 8 columns), handled by one thread
  if (threadIdx.x == 0) {
    for (int c = c0 + 8 * n_vec; c < c1; ++c) {
      const EntropyPartial one = {to_float<T>(base[c]), 1.f, 0.f};
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
  }
}

}  // namespace

int logits_entropy_pick_splits(int64_t rows, int V, int num_sms) {
  // One wave of blocks: about seven 128-thread blocks per SM fit at once, and every thread should see a few
  // hundred logits so that the per-block combine is amortised; never less than 2K columns per block.
  int64_t splits = std::max<int64_t>(1, (7ll * num_sms) / std::max<int64_t>(rows, 1));
  splits = std::min<int64_t>(splits, std::max(1, V / 2048));
  return static_cast<int>(std::max<int64_t>(1, std::min<int64_t>(splits, 128)));
}

cudaError_t launch_logits_entropy(const void* logits, int64_t ldl, bool bf16, int64_t rows, int V, int splits,
                                  float* partials, const int32_t* status, cudaStream_t stream) {
  int cols_per_split = (V + splits - 1) / splits;
  cols_per_split = (cols_per_split + 7) / 8 * 8;
  dim3 grid(splits, static_cast<unsigned>(rows));
  if (bf16) {
    logits_entropy_kernel<__nv_bfloat16><<<grid, kLogitsThreads, 0, stream>>>(
        static_cast<const __nv_bfloat16*>(logits), ldl, V, cols_per_split, splits, partials, status);
  } else {
    logits_entropy_kernel<float><<<grid, kLogitsThreads, 0, stream>>>(static_cast<const float*>(logits), ldl, V,
                                                                     cols_per_split, splits, partials, status);
  }
  return cudaGetLastError();
}

}  // namespace egtp
