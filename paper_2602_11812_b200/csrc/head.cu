// Prediction head (paper Sec. 3.2, Eq. 6): u = ReLU(W1 z + b1), o = W2 u + b2, then either the
// scalar o[0] or the expectation of softmax(o) over the bin centres.
// Layer 1 has two forms.  With bf16 weights it runs on the tensor cores: split_hi_lo_kernel writes every fp32
// input row as two bf16 halves and the LM-head kernel multiplies them against W1 (a launch over the head
// columns alone, K split over the SMs).  head_hidden_kernel is the CUDA-core form (fp32 weights, and the entry
// point that works without a context): plain fp32 FMA, register-tiled, split along d so that small batches
// still fill the GPU.  Either way the split partials are added in a fixed order by head_out_kernel.
#include "kernels.h"
#include "head_out.cuh"
#include "../../include/egtp.h"

#include <cuda_bf16.h>

#include <algorithm>

namespace egtp {

namespace {

constexpr int kHT = 64;        // rows and hidden units per block tile
constexpr int kHK = 32;        // k extent per shared-memory stage
constexpr int kHThreads = 128; // 16 x 8 threads, 8 x 4 outputs each
constexpr int kHOutThreads = 256;

template <typename TW>
__device__ __forceinline__ void load8w(const TW* p, float (&v)[8]);
template <>
__device__ __forceinline__ void load8w<float>(const float* p, float (&v)[8]) {
  const float4 a = __ldg(reinterpret_cast<const float4*>(p));
  const float4 b = __ldg(reinterpret_cast<const float4*>(p) + 1);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
  v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
template <>
__device__ __forceinline__ void load8w<__nv_bfloat16>(const __nv_bfloat16* p, float (&v)[8]) {
  const uint4 q = __ldg(reinterpret_cast<const uint4*>(p));
  const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}

// partial[split][row][j] = sum_{k in split} z[row][k] * W1[j][k]
// 64 x 64 outputs per block, 8 x 4 per thread; the global loads of k-block i+1 are in flight while
// k-block i is multiplied out of shared memory (two buffers, one barrier per k-block).
template <typename TW>
__global__ void __launch_bounds__(kHThreads)
head_hidden_kernel(const float* __restrict__ z, int64_t ldz, const TW* __restrict__ W1, int rows, int d, int m_h,
                   int k_per_split, float* __restrict__ partial, const int32_t* __restrict__ status) {
  if (*status != 0) return;
  __shared__ float zs[2][kHK][kHT + 4];
  __shared__ float ws[2][kHK][kHT + 4];
  const int j0 = blockIdx.x * kHT, r0 = blockIdx.y * kHT, split = blockIdx.z;
  const int k_begin = split * k_per_split;
  const int k_end = min(d, k_begin + k_per_split);
  const int tid = threadIdx.x;
  const int lrow = tid >> 1, lk = (tid & 1) * 16;  // loader: 64 rows x 2 groups of 16 k
  const int tx = tid & 15, ty = tid >> 4;          // compute: outputs rows ty*8.., units tx*4..
  const bool z_ok = r0 + lrow < rows, w_ok = j0 + lrow < m_h;
  const float* zp = z + static_cast<int64_t>(r0 + lrow) * ldz + lk;
  const TW* wp = W1 + static_cast<int64_t>(j0 + lrow) * d + lk;
  float acc[8][4];
#pragma unroll
  for (int a = 0; a < 8; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;

  float zv[16], wv[16];
  auto fetch = [&](int k0) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const bool k_in = k0 + lk + 8 * h < k_end;   // d is a multiple of 16: a group of 8 is wholly inside or outside
      float tz[8], tw[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) { tz[i] = 0.f; tw[i] = 0.f; }
      if (z_ok && k_in) load8w<float>(zp + k0 + 8 * h, tz);
      if (w_ok && k_in) load8w<TW>(wp + k0 + 8 * h, tw);
#pragma unroll
      for (int i = 0; i < 8; ++i) { zv[8 * h + i] = tz[i]; wv[8 * h + i] = tw[i]; }
    }
  };
  if (k_begin < k_end) fetch(k_begin);
  int buf = 0;
  for (int k0 = k_begin; k0 < k_end; k0 += kHK) {
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      zs[buf][lk + i][lrow] = zv[i];
      ws[buf][lk + i][lrow] = wv[i];
    }
    __syncthreads();
    if (k0 + kHK < k_end) fetch(k0 + kHK);
#pragma unroll
    for (int k = 0; k < kHK; ++k) {
      const float4 a0 = *reinterpret_cast<const float4*>(&zs[buf][k][ty * 8]);
      const float4 a1 = *reinterpret_cast<const float4*>(&zs[buf][k][ty * 8 + 4]);
      const float4 b = *reinterpret_cast<const float4*>(&ws[buf][k][tx * 4]);
      const float av[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
      const float bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    buf ^= 1;   // the other buffer was last read two k-blocks ago: the barrier above already fenced it
  }
  float* out = partial + static_cast<int64_t>(split) * rows * m_h;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int r = r0 + ty * 8 + i;
    if (r >= rows) continue;
    const int jj = j0 + tx * 4;
    float* o = out + static_cast<int64_t>(r) * m_h + jj;
    if (jj + 3 < m_h && (m_h & 3) == 0) {
      *reinterpret_cast<float4*>(o) = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (jj + j < m_h) o[j] = acc[i][j];
    }
  }
}

// One block per row: u = ReLU(sum of split partials + b1) into shared memory, o_c = W2[c] . u + b2[c]
// (one warp per output, lanes stride the hidden units), then the output mode.
template <typename TW>
__global__ void __launch_bounds__(kHOutThreads)
head_out_kernel(const float* __restrict__ partial, int64_t split_stride, int64_t row_stride, int splits, int m_h, int d_out,
                const float* __restrict__ b1, const TW* __restrict__ W2, const float* __restrict__ b2,
                const float* __restrict__ centres, int mode, float* __restrict__ y, float* __restrict__ phat,
                const int32_t* __restrict__ status) {
  if (*status != 0) return;
  extern __shared__ float smem[];
  float* u = smem;            // [m_h]
  float* o = smem + m_h;      // [d_out]
  const int r = blockIdx.x, tid = threadIdx.x;
  for (int j = tid; j < m_h; j += blockDim.x) {
    const float* pj = partial + static_cast<int64_t>(r) * row_stride + j;
    const int64_t stride = split_stride;
    float v = 0.f;
    int s = 0;
    for (; s + 4 <= splits; s += 4) {     // four loads in flight; the additions keep split order
      const float p0 = __ldg(pj + s * stride), p1 = __ldg(pj + (s + 1) * stride), p2 = __ldg(pj + (s + 2) * stride),
                  p3 = __ldg(pj + (s + 3) * stride);
      v = (((v + p0) + p1) + p2) + p3;
    }
    for (; s < splits; ++s) v += __ldg(pj + s * stride);
    u[j] = fmaxf(0.f, v + b1[j]);
  }
  head_output_stage<TW>(u, o, m_h, d_out, W2, b2, centres, mode, y, phat, r);
}

// out[r][j] = sum over splits of partial[split][r][j], added in split order: the projection W1 x of rows x
// that are not pooled vectors (the running sums of a PLP state bound to a head).
__global__ void __launch_bounds__(256)
head_partial_sum_kernel(const float* __restrict__ partial, int64_t split_stride, int64_t row_stride, int rows,
                        int splits, int m_h, float* __restrict__ out, int64_t ld_out,
                        const int32_t* __restrict__ status) {
  if (*status != 0) return;
  const int64_t n = static_cast<int64_t>(rows) * m_h;
  for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < n;
       i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const int64_t r = i / m_h;
    const int64_t j = i - r * m_h;
    const float* pj = partial + r * row_stride + j;
    float v = 0.f;
    for (int s = 0; s < splits; ++s) v += __ldg(pj + s * split_stride);
    out[r * ld_out + j] = v;
  }
}

// xcat[r][0..d) = bf16(x[r]), xcat[r][d..2d) = bf16(x[r] - bf16(x[r])); 8 elements per thread
__global__ void __launch_bounds__(256)
split_hi_lo_kernel(const float* __restrict__ x, int64_t ldx, int rows, int d, __nv_bfloat16* __restrict__ xcat,
                   const int32_t* __restrict__ status) {
  if (*status != 0) return;
  const int per_row = d / 8;
  const int64_t n = static_cast<int64_t>(rows) * per_row;
  for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < n;
       i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const int64_t r = i / per_row;
    const int col = static_cast<int>(i - r * per_row) * 8;
    float v[8];
    load8w<float>(x + r * ldx + col, v);
    __align__(16) __nv_bfloat16 hi[8], lo[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      hi[k] = __float2bfloat16_rn(v[k]);
      lo[k] = __float2bfloat16_rn(v[k] - __bfloat162float(hi[k]));
    }
    __nv_bfloat16* dst = xcat + r * (2 * static_cast<int64_t>(d)) + col;
    *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(hi);
    *reinterpret_cast<uint4*>(dst + d) = *reinterpret_cast<const uint4*>(lo);
  }
}

}  // namespace

int head_pick_splits(int rows, int d, int m_h, int num_sms, int64_t partial_capacity_floats) {
  const int64_t tiles = static_cast<int64_t>((rows + kHT - 1) / kHT) * ((m_h + kHT - 1) / kHT);
  int splits = static_cast<int>(std::max<int64_t>(1, (2ll * num_sms + tiles - 1) / tiles));
  splits = std::min(splits, std::max(1, d / 256));
  const int64_t per_split = static_cast<int64_t>(rows) * m_h;
  while (splits > 1 && per_split * splits > partial_capacity_floats) --splits;
  if (per_split * splits > partial_capacity_floats) return 0;
  return splits;
}

cudaError_t launch_head_hidden(const HeadArgs& h, const float* z, int64_t ldz, int rows, int splits,
                               float* partial, const int32_t* status, cudaStream_t stream) {
  int k_per_split = (h.d + splits - 1) / splits;
  k_per_split = (k_per_split + kHK - 1) / kHK * kHK;
  dim3 grid((h.m_h + kHT - 1) / kHT, (rows + kHT - 1) / kHT, splits);
  if (h.bf16) {
    head_hidden_kernel<__nv_bfloat16><<<grid, kHThreads, 0, stream>>>(
        z, ldz, static_cast<const __nv_bfloat16*>(h.W1), rows, h.d, h.m_h, k_per_split, partial, status);
  } else {
    head_hidden_kernel<float><<<grid, kHThreads, 0, stream>>>(z, ldz, static_cast<const float*>(h.W1), rows, h.d,
                                                              h.m_h, k_per_split, partial, status);
  }
  return cudaGetLastError();
}

cudaError_t launch_head_out(const HeadArgs& h, const float* partial, int rows, int splits, float* y, float* phat,
                            const int32_t* status, cudaStream_t stream, int64_t split_stride, int64_t row_stride) {
  const size_t smem = static_cast<size_t>(h.m_h + h.d_out) * sizeof(float);
  if (row_stride == 0) row_stride = h.m_h;
  if (split_stride == 0) split_stride = static_cast<int64_t>(rows) * h.m_h;
  if (h.bf16) {
    head_out_kernel<__nv_bfloat16><<<rows, kHOutThreads, smem, stream>>>(partial, split_stride, row_stride, splits, h.m_h, h.d_out, h.b1,
                                                               static_cast<const __nv_bfloat16*>(h.W2), h.b2,
                                                               h.centres, h.mode, y, phat, status);
  } else {
    head_out_kernel<float><<<rows, kHOutThreads, smem, stream>>>(partial, split_stride, row_stride, splits, h.m_h, h.d_out, h.b1,
                                                       static_cast<const float*>(h.W2), h.b2, h.centres, h.mode, y,
                                                       phat, status);
  }
  return cudaGetLastError();
}

cudaError_t launch_head_partial_sum(const float* partial, int rows, int splits, int m_h, float* out, int64_t ld_out,
                                    const int32_t* status, cudaStream_t stream, int64_t split_stride,
                                    int64_t row_stride) {
  if (row_stride == 0) row_stride = m_h;
  if (split_stride == 0) split_stride = static_cast<int64_t>(rows) * m_h;
  const int64_t n = static_cast<int64_t>(rows) * m_h;
  const int blocks = static_cast<int>(std::min<int64_t>(1184, (n + 255) / 256));
  head_partial_sum_kernel<<<std::max(1, blocks), 256, 0, stream>>>(partial, split_stride, row_stride, rows, splits, m_h, out,
                                                                  ld_out, status);
  return cudaGetLastError();
}

cudaError_t launch_split_hi_lo(const float* x, int64_t ldx, int rows, int d, void* xcat, const int32_t* status,
                               cudaStream_t stream) {
  const int64_t n = static_cast<int64_t>(rows) * (d / 8);
  const int blocks = static_cast<int>(std::max<int64_t>(1, std::min<int64_t>(1184, (n + 255) / 256)));
  split_hi_lo_kernel<<<blocks, 256, 0, stream>>>(x, ldx, rows, d, static_cast<__nv_bfloat16*>(xcat), status);
  return cudaGetLastError();
}

}  // namespace egtp
