// Offsets check, entropy merge (Eq. 2), per-prompt softmax weights (Eq. 3) and the
// entropy-weighted ragged pooling (Eq. 4).  HBM-bound work: plain coalesced 16-byte loads,
// fp32 accumulation, warp-shuffle / block reductions, no floating-point atomics.
#include "kernels.h"
#include "entropy_merge.cuh"
#include "../../include/egtp.h"

#include <cuda_bf16.h>

namespace egtp {

namespace {

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Largest b in [0, B] with offsets[b] <= t (offsets non-decreasing, offsets[0] <= t assumed).
__device__ __forceinline__ int upper_segment(const int32_t* __restrict__ off, int B, int64_t t) {
  int lo = 0, hi = B;   // invariant: off[lo] <= t
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (static_cast<int64_t>(off[mid]) <= t) lo = mid; else hi = mid - 1;
  }
  return lo;
}

// --------------------------------------------------------------------------- offsets check
__global__ void validate_offsets_kernel(const int32_t* __restrict__ off, int B, int64_t T, int32_t* status) {
  bool bad = false;
  for (int b = threadIdx.x; b <= B; b += blockDim.x) {
    const int64_t v = off[b];
    if (v < 0 || v > T) bad = true;
    if (b < B && static_cast<int64_t>(off[b + 1]) < v) bad = true;
  }
  if (__syncthreads_or(bad ? 1 : 0)) {
    if (threadIdx.x == 0) atomicCAS(status, 0, EGTP_ERR_BAD_OFFSETS);
  }
}

// --------------------------------------------------------------------------- Eq. 2: merge
// One warp per token: lanes stride over the token's (m, s, t2) partials (contiguous in memory),
// fold them in a fixed order, then combine across lanes: H = ln S - ln2 * T2 / S.
// Also writes the token's prompt index and clears its weight.
__global__ void entropy_merge_kernel(const float* __restrict__ partials, int slots, int64_t row_stride,
                                     int64_t slot_stride, int64_t T, int64_t row0, float* __restrict__ H, const int32_t* __restrict__ off, int B,
                                     int32_t* __restrict__ seg_id, float* __restrict__ weights,
                                     const int32_t* __restrict__ status) {
  if (*status != 0) return;
  const int lane = threadIdx.x & 31;
  const int64_t i = static_cast<int64_t>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (i >= T) return;
  const float h = merge_partials_warp(partials + i * row_stride, slots, slot_stride, lane);
  if (lane == 0) {
    const int64_t g = row0 + i;      // token index in the whole batch (the partials may cover one piece of it)
    H[g] = h;
    if (weights != nullptr) weights[g] = 0.f;
    if (seg_id != nullptr) {
      int sid = -1;
      if (B > 0 && g >= off[0] && g < off[B]) sid = upper_segment(off, B, g);
      seg_id[g] = sid;
    }
  }
}

// One warp per row: folds the row's per-chunk partials into a single (m, s, t2) triple, the unit that
// GPUs holding different vocabulary shards exchange.
__global__ void partials_reduce_kernel(const float* __restrict__ partials, int slots, int64_t rows,
                                       float* __restrict__ out, const int32_t* __restrict__ status) {
  if (*status != 0) return;
  const int lane = threadIdx.x & 31;
  const int64_t i = static_cast<int64_t>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (i >= rows) return;
  const EntropyPartial p = merge_partials_warp_raw(partials + i * slots * 3, slots, 3, lane);
  if (lane == 0) {
    out[3 * i] = p.m;
    out[3 * i + 1] = p.s;
    out[3 * i + 2] = p.t2;
  }
}

// --------------------------------------------------------------------------- Eq. 3: weights
// One block per prompt: M = max_i H_i/alpha, Z = sum_i exp(H_i/alpha - M), w_i = exp(.)/Z.
__global__ void segment_weights_kernel(const float* __restrict__ H, const int32_t* __restrict__ off, int B,
                                       float inv_alpha, float* __restrict__ weights, float* __restrict__ seg_m,
                                       float* __restrict__ seg_s, const int32_t* __restrict__ status) {
  if (*status != 0) return;
  __shared__ float red[32];
  __shared__ float bcast;
  const int b = blockIdx.x;
  const int s0 = off[b], s1 = off[b + 1];
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, nw = blockDim.x >> 5;
  if (s1 <= s0) {
    if (tid == 0) {
      if (seg_m) seg_m[b] = -INFINITY;
      if (seg_s) seg_s[b] = 0.f;
    }
    return;
  }
  float mx = -INFINITY;
  for (int i = s0 + tid; i < s1; i += blockDim.x) mx = fmaxf(mx, H[i] * inv_alpha);
  mx = warp_max(mx);
  if (lane == 0) red[wid] = mx;
  __syncthreads();
  if (wid == 0) {
    float v = lane < nw ? red[lane] : -INFINITY;
    v = warp_max(v);
    if (lane == 0) bcast = v;
  }
  __syncthreads();
  const float M = bcast;
  float sum = 0.f;
  for (int i = s0 + tid; i < s1; i += blockDim.x) sum += expf(H[i] * inv_alpha - M);
  sum = warp_sum(sum);
  __syncthreads();
  if (lane == 0) red[wid] = sum;
  __syncthreads();
  if (wid == 0) {
    float v = lane < nw ? red[lane] : 0.f;
    v = warp_sum(v);
    if (lane == 0) bcast = v;
  }
  __syncthreads();
  const float Z = bcast;
  const float invZ = 1.f / Z;
  for (int i = s0 + tid; i < s1; i += blockDim.x) weights[i] = expf(H[i] * inv_alpha - M) * invZ;
  if (tid == 0) {
    if (seg_m) seg_m[b] = M;
    if (seg_s) seg_s[b] = Z;
  }
}

// Weights of the pooling alternatives in the paper's ablation (Table 3) that are weighted sums:
// average pooling (w = 1/n) and last-token pooling (w = 1 on the prompt's last token).
__global__ void baseline_weights_kernel(const int32_t* __restrict__ off, int B, int mode, float* __restrict__ weights,
                                        const int32_t* __restrict__ status) {
  if (*status != 0) return;
  const int b = blockIdx.x;
  const int s0 = off[b], s1 = off[b + 1];
  if (s1 <= s0) return;
  const float inv_n = 1.f / static_cast<float>(s1 - s0);
  for (int i = s0 + threadIdx.x; i < s1; i += blockDim.x)
    weights[i] = mode == EGTP_POOL_MEAN ? inv_n : (i == s1 - 1 ? 1.f : 0.f);
}

// --------------------------------------------------------------------------- Eq. 4: pooling
template <typename T>
struct Row8;
template <>
struct Row8<__nv_bfloat16> {
  static __device__ __forceinline__ void load(const __nv_bfloat16* p, float (&v)[8]) {
    const uint4 q = __ldg(reinterpret_cast<const uint4*>(p));
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
};
template <>
struct Row8<float> {
  static __device__ __forceinline__ void load(const float* p, float (&v)[8]) {
    const float4 a = __ldg(reinterpret_cast<const float4*>(p));
    const float4 b = __ldg(reinterpret_cast<const float4*>(p) + 1);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
    v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
  }
};

__device__ __forceinline__ void store8(float* p, const float (&v)[8]) {
  reinterpret_cast<float4*>(p)[0] = make_float4(v[0], v[1], v[2], v[3]);
  reinterpret_cast<float4*>(p)[1] = make_float4(v[4], v[5], v[6], v[7]);
}

// Block (c, y): tokens [c*64, (c+1)*64) clipped to [offsets[0], offsets[B]), channels
// [(y*128 + tid)*8, +8).  A prompt that lies wholly inside the chunk is finished here; a prompt
// that crosses chunk borders leaves one piece per chunk: piece_a[c] if it entered from the
// left, piece_b[c] if it starts here and leaves to the right.  The combine kernel adds the
// pieces of each prompt in chunk order.
// With kMax the weights are ignored and the channel-wise maximum is taken instead of the weighted sum
// (max pooling, Table 3); pieces of a prompt that spans chunks are then combined with max.
template <typename T, bool kMax>
__global__ void __launch_bounds__(kPoolThreads)
pool_kernel(const T* __restrict__ hidden, int64_t ldh, const float* __restrict__ weights,
            const int32_t* __restrict__ off, int B, int d, float* __restrict__ pooled,
            float* __restrict__ piece_a, float* __restrict__ piece_b, const int32_t* __restrict__ status) {
  if (*status != 0) return;
  const int64_t c = blockIdx.x;
  const int col = (blockIdx.y * kPoolThreads + threadIdx.x) * 8;
  const int64_t c_lo = c * kPoolChunkTokens, c_hi = c_lo + kPoolChunkTokens;
  int64_t t0 = max(c_lo, static_cast<int64_t>(off[0]));
  const int64_t t1 = min(c_hi, static_cast<int64_t>(off[B]));
  if (t0 >= t1 || col >= d) return;
  int b = upper_segment(off, B, t0);
  while (t0 < t1) {
    const int64_t seg_begin = off[b], seg_end = off[b + 1];
    if (seg_end <= t0) { ++b; continue; }       // empty prompts own no token
    const int64_t run_end = min(seg_end, t1);
    float acc[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) acc[k] = kMax ? -INFINITY : 0.f;
    const T* rowp = hidden + t0 * ldh + col;
    int64_t t = t0;
    for (; t + 4 <= run_end; t += 4) {           // four rows in flight per thread
      float w0 = 0.f, w1 = 0.f, w2 = 0.f, w3 = 0.f;
      if constexpr (!kMax) {
        w0 = __ldg(weights + t); w1 = __ldg(weights + t + 1); w2 = __ldg(weights + t + 2); w3 = __ldg(weights + t + 3);
        // rows that carry no weight (last-token pooling: all but one) are not read at all
        if (w0 == 0.f && w1 == 0.f && w2 == 0.f && w3 == 0.f) { rowp += 4 * ldh; continue; }
      }
      float v0[8], v1[8], v2[8], v3[8];
      Row8<T>::load(rowp, v0);
      Row8<T>::load(rowp + ldh, v1);
      Row8<T>::load(rowp + 2 * ldh, v2);
      Row8<T>::load(rowp + 3 * ldh, v3);
      if constexpr (kMax) {
#pragma unroll
        for (int k = 0; k < 8; ++k) acc[k] = fmaxf(fmaxf(acc[k], fmaxf(v0[k], v1[k])), fmaxf(v2[k], v3[k]));
      } else {
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          acc[k] = fmaf(w0, v0[k], acc[k]);
          acc[k] = fmaf(w1, v1[k], acc[k]);
          acc[k] = fmaf(w2, v2[k], acc[k]);
          acc[k] = fmaf(w3, v3[k], acc[k]);
        }
      }
      rowp += 4 * ldh;
    }
    for (; t < run_end; ++t) {
      float v0[8];
      Row8<T>::load(rowp, v0);
      if constexpr (kMax) {
#pragma unroll
        for (int k = 0; k < 8; ++k) acc[k] = fmaxf(acc[k], v0[k]);
      } else {
        const float w0 = __ldg(weights + t);
#pragma unroll
        for (int k = 0; k < 8; ++k) acc[k] = fmaf(w0, v0[k], acc[k]);
      }
      rowp += ldh;
    }
    float* dst;
    if (seg_begin >= c_lo && seg_end <= c_hi) dst = pooled + static_cast<int64_t>(b) * d + col;
    else if (seg_begin < c_lo) dst = piece_a + c * d + col;
    else dst = piece_b + c * d + col;
    store8(dst, acc);
    t0 = run_end;
    ++b;
  }
}

// One block per prompt (x) and 1024-channel slab (y): zero for an empty prompt, nothing for a
// prompt finished by the first stage, else piece_b[c0] + piece_a[c0+1] + ... + piece_a[c1].
template <bool kMax>
__global__ void __launch_bounds__(kPoolThreads)
pool_combine_kernel(const int32_t* __restrict__ off, int B, int d, const float* __restrict__ piece_a,
                    const float* __restrict__ piece_b, float* __restrict__ pooled,
                    const int32_t* __restrict__ status) {
  if (*status != 0) return;
  const int b = blockIdx.x;
  const int col = (blockIdx.y * kPoolThreads + threadIdx.x) * 8;
  if (col >= d) return;
  const int64_t s0 = off[b], s1 = off[b + 1];
  float acc[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) acc[k] = 0.f;
  float* dst = pooled + static_cast<int64_t>(b) * d + col;
  if (s1 <= s0) { store8(dst, acc); return; }
  const int64_t c0 = s0 / kPoolChunkTokens, c1 = (s1 - 1) / kPoolChunkTokens;
  if (c0 == c1) return;
  {
    const float4* p = reinterpret_cast<const float4*>(piece_b + c0 * d + col);
    const float4 a = p[0], bq = p[1];
    acc[0] = a.x; acc[1] = a.y; acc[2] = a.z; acc[3] = a.w;
    acc[4] = bq.x; acc[5] = bq.y; acc[6] = bq.z; acc[7] = bq.w;
  }
  for (int64_t c = c0 + 1; c <= c1; ++c) {
    const float4* p = reinterpret_cast<const float4*>(piece_a + c * d + col);
    const float4 a = p[0], bq = p[1];
    const float pv[8] = {a.x, a.y, a.z, a.w, bq.x, bq.y, bq.z, bq.w};
#pragma unroll
    for (int k = 0; k < 8; ++k) acc[k] = kMax ? fmaxf(acc[k], pv[k]) : acc[k] + pv[k];
  }
  store8(dst, acc);
}

}  // namespace

cudaError_t launch_validate_offsets(const int32_t* offsets, int B, int64_t T, int32_t* status, cudaStream_t stream) {
  validate_offsets_kernel<<<1, 256, 0, stream>>>(offsets, B, T, status);
  return cudaGetLastError();
}

cudaError_t launch_entropy_merge(const float* partials, int slots, int64_t row_stride, int64_t slot_stride, int64_t T,
                                 int64_t row0, float* H, const int32_t* offsets, int B, int32_t* seg_id_out, float* weights_zero,
                                 const int32_t* status, cudaStream_t stream) {
  const int threads = 256, rows_per_block = threads / 32;
  const unsigned blocks = static_cast<unsigned>((T + rows_per_block - 1) / rows_per_block);
  entropy_merge_kernel<<<blocks, threads, 0, stream>>>(partials, slots, row_stride, slot_stride, T, row0, H, offsets, B,
                                                       seg_id_out, weights_zero, status);
  return cudaGetLastError();
}

cudaError_t launch_partials_reduce(const float* partials, int slots, int64_t rows, float* out, const int32_t* status,
                                   cudaStream_t stream) {
  const int threads = 256, rows_per_block = threads / 32;
  const unsigned blocks = static_cast<unsigned>((rows + rows_per_block - 1) / rows_per_block);
  partials_reduce_kernel<<<blocks, threads, 0, stream>>>(partials, slots, rows, out, status);
  return cudaGetLastError();
}

cudaError_t launch_segment_weights(const float* H, const int32_t* offsets, int B, float inv_alpha, float* weights,
                                   float* seg_m, float* seg_s, const int32_t* status, cudaStream_t stream) {
  segment_weights_kernel<<<B, 256, 0, stream>>>(H, offsets, B, inv_alpha, weights, seg_m, seg_s, status);
  return cudaGetLastError();
}

cudaError_t launch_baseline_weights(const int32_t* offsets, int B, int mode, float* weights, const int32_t* status,
                                    cudaStream_t stream) {
  baseline_weights_kernel<<<B, 256, 0, stream>>>(offsets, B, mode, weights, status);
  return cudaGetLastError();
}

cudaError_t launch_pool(const void* hidden, int64_t ldh, bool bf16, bool take_max, const float* weights,
                        const int32_t* offsets, int B, int64_t T, int d, float* pooled, float* piece_a,
                        float* piece_b, const int32_t* status, cudaStream_t stream) {
  const unsigned chunks = static_cast<unsigned>((T + kPoolChunkTokens - 1) / kPoolChunkTokens);
  const unsigned slabs = static_cast<unsigned>((d + kPoolThreads * 8 - 1) / (kPoolThreads * 8));
  dim3 grid(chunks, slabs);
  const __nv_bfloat16* hb = static_cast<const __nv_bfloat16*>(hidden);
  const float* hf = static_cast<const float*>(hidden);
  if (bf16 && take_max)
    pool_kernel<__nv_bfloat16, true><<<grid, kPoolThreads, 0, stream>>>(hb, ldh, weights, offsets, B, d, pooled, piece_a, piece_b, status);
  else if (bf16)
    pool_kernel<__nv_bfloat16, false><<<grid, kPoolThreads, 0, stream>>>(hb, ldh, weights, offsets, B, d, pooled, piece_a, piece_b, status);
  else if (take_max)
    pool_kernel<float, true><<<grid, kPoolThreads, 0, stream>>>(hf, ldh, weights, offsets, B, d, pooled, piece_a, piece_b, status);
  else
    pool_kernel<float, false><<<grid, kPoolThreads, 0, stream>>>(hf, ldh, weights, offsets, B, d, pooled, piece_a, piece_b, status);
  return cudaGetLastError();
}

cudaError_t launch_pool_combine(const int32_t* offsets, int B, int d, bool take_max, const float* piece_a,
                                const float* piece_b, float* pooled, const int32_t* status, cudaStream_t stream) {
  const unsigned slabs = static_cast<unsigned>((d + kPoolThreads * 8 - 1) / (kPoolThreads * 8));
  dim3 grid(B, slabs);
  if (take_max)
    pool_combine_kernel<true><<<grid, kPoolThreads, 0, stream>>>(offsets, B, d, piece_a, piece_b, pooled, status);
  else
    pool_combine_kernel<false><<<grid, kPoolThreads, 0, stream>>>(offsets, B, d, piece_a, piece_b, pooled, status);
  return cudaGetLastError();
}

namespace {

// dst [dst_rows][row_bytes] <- src rows (src_rows of them, ld_bytes apart), remaining rows zero; 16 bytes per thread
__global__ void __launch_bounds__(256)
pad_rows_kernel(const uint8_t* __restrict__ src, int64_t ld_bytes, int src_rows, int64_t row_bytes,
                uint8_t* __restrict__ dst, int dst_rows, const int32_t* __restrict__ status) {
  if (*status != 0) return;
  const int64_t per_row = row_bytes / 16;
  const int64_t n = per_row * dst_rows;
  for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < n;
       i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const int64_t r = i / per_row, c = (i - r * per_row) * 16;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (r < src_rows) v = *reinterpret_cast<const uint4*>(src + r * ld_bytes + c);
    *reinterpret_cast<uint4*>(dst + r * row_bytes + c) = v;
  }
}

}  // namespace

cudaError_t launch_pad_rows(const void* src, int64_t ld_bytes, int src_rows, int64_t row_bytes, void* dst,
                            int dst_rows, const int32_t* status, cudaStream_t stream) {
  const int64_t n = row_bytes / 16 * dst_rows;
  const int blocks = static_cast<int>(std::max<int64_t>(1, std::min<int64_t>(296, (n + 255) / 256)));
  pad_rows_kernel<<<blocks, 256, 0, stream>>>(static_cast<const uint8_t*>(src), ld_bytes, src_rows, row_bytes,
                                              static_cast<uint8_t*>(dst), dst_rows, status);
  return cudaGetLastError();
}

}  // namespace egtp
