// Offsets check, entropy merge (Eq. 2) and the entropy-weighted ragged pooling with its softmax over each
// prompt's entropies folded in (Eq. 3-4).  HBM-bound work: plain coalesced 16-byte loads,
// fp32 accumulation, warp-shuffle / block reductions, no floating-point atomics.
#include "kernels.h"
#include "entropy_merge.cuh"
#include "../../include/egtp.h"

#include <cuda_bf16.h>

namespace egtp {

namespace {

constexpr int kMergeThreads = 256;   // four lanes for each token of a 64-token pooling chunk

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
__device__ __forceinline__ bool offsets_bad(const int32_t* __restrict__ off, int B, int64_t T) {
  bool bad = false;
  for (int b = threadIdx.x; b <= B; b += blockDim.x) {
    const int64_t v = off[b];
    if (v < 0 || v > T) bad = true;
    if (b < B && static_cast<int64_t>(off[b + 1]) < v) bad = true;
  }
  return bad;
}

__global__ void validate_offsets_kernel(const int32_t* __restrict__ off, int B, int64_t T, int32_t* status) {
  if (__syncthreads_or(offsets_bad(off, B, T) ? 1 : 0)) {
    if (threadIdx.x == 0) atomicCAS(status, 0, EGTP_ERR_BAD_OFFSETS);
  }
}

// --------------------------------------------------------------------------- Eq. 2: merge (and the first half of Eq. 3)
// One block per pooling chunk of 64 tokens, four lanes per token: the lanes stride over the token's (m, s, t2)
// partials (contiguous in memory), fold them in a fixed order, then combine across lanes: H = ln S - ln2 * T2 / S.
// Also writes the token's prompt index.  With T_check >= 0, block 0 first checks the offsets against that token
// count (the kernels that index tokens through the offsets come later in the stream and see the status).
// With `weights` given, the block then prepares the pooling of its chunk: for every run of tokens of one prompt inside
// the chunk, m = max H_i/alpha over the run, the unnormalised weights w_i = exp(H_i/alpha - m) (Eq. 3 up to the
// normaliser) and (m, sum w) of the run, stored where the pooling kernels expect them: seg_m / seg_s for a prompt
// that lies wholly inside the chunk, else ms_a[c] (run entered from the left) or ms_b[c] (run leaves to the right).
__global__ void __launch_bounds__(kMergeThreads)
entropy_merge_kernel(const float* __restrict__ partials, int slots, int64_t row_stride, int64_t slot_stride, int64_t T,
                     int64_t row0, float* __restrict__ H, const int32_t* __restrict__ off, int B,
                     int32_t* __restrict__ seg_id, int64_t T_check, float inv_alpha, float* __restrict__ weights,
                     float2* __restrict__ ms_a, float2* __restrict__ ms_b, float* __restrict__ seg_m,
                     float* __restrict__ seg_s, int32_t* __restrict__ status) {
  if (*status != 0) return;
  if (T_check >= 0 && blockIdx.x == 0) {
    if (__syncthreads_or(offsets_bad(off, B, T_check) ? 1 : 0)) {
      if (threadIdx.x == 0) atomicCAS(status, 0, EGTP_ERR_BAD_OFFSETS);
    }
  }
  __shared__ float a_s[kPoolChunkTokens];
  __shared__ int sid_s[kPoolChunkTokens];
  // four lanes per token, eight tokens per warp at once: thread 4 idx + q works on token idx of the chunk
  static_assert(kMergeThreads == 4 * kPoolChunkTokens, "four lanes per token of the chunk");
  const int idx = threadIdx.x >> 2, q = threadIdx.x & 3;
  const int64_t i0 = static_cast<int64_t>(blockIdx.x) * kPoolChunkTokens;      // first token of the chunk in this piece
  const int64_t i = i0 + idx;
  const bool in_range = i < T;
  // (rows past the end take part with zero slots: the group shuffles need every lane of the warp)
  const EntropyPartial ep = merge_partials_group_raw<4>(partials + (in_range ? i : 0) * row_stride, in_range ? slots : 0,
                                                        slot_stride, q);
  if (q == 0) {
    if (!in_range) {
      sid_s[idx] = -1;
    } else {
      const float h = entropy_of(ep);
      const int64_t g = row0 + i;      // token index in the whole batch (the partials may cover one piece of it)
      H[g] = h;
      int sid = -1;
      if (off != nullptr && B > 0 && g >= off[0] && g < off[B]) sid = upper_segment(off, B, g);
      if (seg_id != nullptr) seg_id[g] = sid;
      a_s[idx] = h * inv_alpha;
      sid_s[idx] = sid;
    }
  }
  if (weights == nullptr) return;
  __syncthreads();
  const int t = threadIdx.x;
  if (t >= kPoolChunkTokens || i0 + t >= T) return;
  const int64_t g = row0 + i0 + t;
  const int sid = sid_s[t];
  if (sid < 0) { weights[g] = 0.f; return; }
  int lo = t, hi = t + 1;                                   // the run of this prompt inside the chunk: [lo, hi)
  while (lo > 0 && sid_s[lo - 1] == sid) --lo;
  while (hi < kPoolChunkTokens && sid_s[hi] == sid) ++hi;
  float m = a_s[lo];
  for (int j = lo + 1; j < hi; ++j) m = fmaxf(m, a_s[j]);
  weights[g] = expf(a_s[t] - m);
  if (t == lo) {
    float wsum = 0.f;
    for (int j = lo; j < hi; ++j) wsum += expf(a_s[j] - m);
    const int64_t c = (row0 + i0) / kPoolChunkTokens;       // chunk index in the whole batch
    const int64_t c_lo = c * kPoolChunkTokens, c_hi = c_lo + kPoolChunkTokens;
    const int64_t seg_begin = off[sid], seg_end = off[sid + 1];
    if (seg_begin >= c_lo && seg_end <= c_hi) {
      if (seg_m) seg_m[sid] = m;
      if (seg_s) seg_s[sid] = wsum;
    } else if (seg_begin < c_lo) {
      ms_a[c] = make_float2(m, wsum);
    } else {
      ms_b[c] = make_float2(m, wsum);
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

// --------------------------------------------------------------------------- Eq. 3: weights as an output
// The pooling kernels below never materialise the normalised weights; a caller that wants them gets
// w_i = exp(H_i/alpha - M_b) / Z_b from the per-prompt state (M_b, Z_b) the pooling left behind (0 outside prompts).
__global__ void token_weights_kernel(const float* __restrict__ H, const int32_t* __restrict__ off, int B, int64_t T,
                                     float inv_alpha, const float* __restrict__ seg_m, const float* __restrict__ seg_s,
                                     float* __restrict__ weights, const int32_t* __restrict__ status) {
  if (*status != 0) return;
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= T) return;
  float w = 0.f;
  if (B > 0 && i >= off[0] && i < off[B]) {
    const int b = upper_segment(off, B, i);
    w = expf(H[i] * inv_alpha - seg_m[b]) / seg_s[b];
  }
  weights[i] = w;
}

// --------------------------------------------------------------------------- Eq. 3 + Eq. 4: pooling
// Eight consecutive channels of one row: loaded as they are (16 bytes of bf16, or 32 bytes of fp32) and widened
// only where they are consumed, so that four rows in flight cost a thread 16 registers in the bf16 case.
template <typename T>
struct Row8;
template <>
struct Row8<__nv_bfloat16> {
  uint4 q;
  __device__ __forceinline__ void load(const __nv_bfloat16* p) { q = __ldg(reinterpret_cast<const uint4*>(p)); }
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
struct Row8<float> {
  float4 a, b;
  __device__ __forceinline__ void load(const float* p) {
    a = __ldg(reinterpret_cast<const float4*>(p));
    b = __ldg(reinterpret_cast<const float4*>(p) + 1);
  }
  __device__ __forceinline__ void get(float (&v)[8]) const {
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
    v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
  }
};
// acc += w * row, or acc = max(acc, row)
template <typename T, bool kMax>
__device__ __forceinline__ void fold_row(float (&acc)[8], const Row8<T>& row, float w) {
  float v[8];
  row.get(v);
#pragma unroll
  for (int k = 0; k < 8; ++k) acc[k] = kMax ? fmaxf(acc[k], v[k]) : fmaf(w, v[k], acc[k]);
}

__device__ __forceinline__ void store8(float* p, const float (&v)[8]) {
  reinterpret_cast<float4*>(p)[0] = make_float4(v[0], v[1], v[2], v[3]);
  reinterpret_cast<float4*>(p)[1] = make_float4(v[4], v[5], v[6], v[7]);
}
__device__ __forceinline__ void load8f(const float* p, float (&v)[8]) {
  const float4 a = reinterpret_cast<const float4*>(p)[0], b = reinterpret_cast<const float4*>(p)[1];
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
  v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}

// [hi | lo] halves of a row of fp32 values: hi = bf16(x), lo = bf16(x - hi); the input format of the head's
// tensor-core layer 1
__device__ __forceinline__ void store8_hi_lo(__nv_bfloat16* row, int d, int col, const float (&v)[8]) {
  __align__(16) __nv_bfloat16 hi[8], lo[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    hi[k] = __float2bfloat16_rn(v[k]);
    lo[k] = __float2bfloat16_rn(v[k] - __bfloat162float(hi[k]));
  }
  *reinterpret_cast<uint4*>(row + col) = *reinterpret_cast<const uint4*>(hi);
  *reinterpret_cast<uint4*>(row + d + col) = *reinterpret_cast<const uint4*>(lo);
}

// Pooling modes: the paper's entropy-weighted pooling (Eq. 3-4) and the alternatives of its ablation (Table 3).
// All but the maximum are weighted sums sum_i w_i h_i / sum_i w_i with unnormalised weights
//   entropy: w_i = exp(H_i/alpha - m), m = the largest H_i/alpha among the tokens summed together
//   mean:    w_i = 1                    last: w_i = 1 for the prompt's last token, else 0
// so one kernel serves them: a block sums a run of tokens with weights relative to the run's own m, which leaves
// (m, sum w, sum w h) per run (in entropy mode the weights and the two scalars come prepared from the merge
// kernel); runs of one prompt are merged later by rescaling to the common maximum (the same recurrence as the PLP
// state, Eq. 8).  The normalised weights of Eq. 3 are never stored.
enum : int { kPoolEntropy = 0, kPoolMean = 1, kPoolMax = 2, kPoolLast = 3 };

// Block (c, y): tokens [c*64, (c+1)*64) clipped to [offsets[0], offsets[B]), channels [(y*128 + tid)*8, +8).
// A prompt that lies wholly inside the chunk is finished here (pooled row, and its (M, Z) by the y = 0 block); a
// prompt that crosses chunk borders leaves one piece per chunk: piece_a[c] if it entered from the left, piece_b[c]
// if it starts here and leaves to the right, each with its (m, sum w) in piece_ms.  The combine kernel merges the
// pieces of each prompt in chunk order.
template <typename T, int kMode>
__global__ void __launch_bounds__(kPoolThreads, sizeof(T) == 2 ? (kMode == kPoolEntropy ? 16 : 12) : 8)   // bf16: 32 (40) registers, an SM full of warps keeps the row loads in flight
pool_kernel(const T* __restrict__ hidden, int64_t ldh, const float* __restrict__ weights,
            const int32_t* __restrict__ off, int B, int d, float* __restrict__ pooled,
            float* __restrict__ piece_a, float* __restrict__ piece_b, float2* __restrict__ ms_a,
            float2* __restrict__ ms_b, float* __restrict__ seg_m, float* __restrict__ seg_s,
            const int32_t* __restrict__ status) {
  if (*status != 0) return;
  const int64_t c = blockIdx.x;
  const int col = (blockIdx.y * kPoolThreads + threadIdx.x) * 8;
  const int64_t c_lo = c * kPoolChunkTokens, c_hi = c_lo + kPoolChunkTokens;
  int64_t t0 = max(c_lo, static_cast<int64_t>(off[0]));
  const int64_t t1 = min(c_hi, static_cast<int64_t>(off[B]));
  if (t0 >= t1 || col >= d) return;
  const bool scribe = blockIdx.y == 0 && threadIdx.x == 0;      // writes the per-run scalars
  int b = upper_segment(off, B, t0);
  while (t0 < t1) {
    const int64_t seg_begin = off[b], seg_end = off[b + 1];
    if (seg_end <= t0) { ++b; continue; }       // empty prompts own no token
    const int64_t run_end = min(seg_end, t1);
    float acc[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) acc[k] = kMode == kPoolMax ? -INFINITY : 0.f;
    float wsum = 0.f;
    if constexpr (kMode == kPoolLast) {
      if (run_end == seg_end) {                   // the prompt's last token is in this run: read that row only
        Row8<T> r;
        r.load(hidden + (seg_end - 1) * ldh + col);
        r.get(acc);
        wsum = 1.f;
      }
    } else {
      constexpr bool kIsMax = kMode == kPoolMax;
      const T* rowp = hidden + t0 * ldh + col;
      int64_t t = t0;
      for (; t + 4 <= run_end; t += 4) {           // four rows in flight per thread
        Row8<T> r0, r1, r2, r3;
        r0.load(rowp);
        r1.load(rowp + ldh);
        r2.load(rowp + 2 * ldh);
        r3.load(rowp + 3 * ldh);
        float w0 = 1.f, w1 = 1.f, w2 = 1.f, w3 = 1.f;
        if constexpr (kMode == kPoolEntropy) {
          w0 = __ldg(weights + t); w1 = __ldg(weights + t + 1); w2 = __ldg(weights + t + 2); w3 = __ldg(weights + t + 3);
        }
        fold_row<T, kIsMax>(acc, r0, w0);
        fold_row<T, kIsMax>(acc, r1, w1);
        fold_row<T, kIsMax>(acc, r2, w2);
        fold_row<T, kIsMax>(acc, r3, w3);
        rowp += 4 * ldh;
      }
      for (; t < run_end; ++t) {
        Row8<T> r0;
        r0.load(rowp);
        fold_row<T, kIsMax>(acc, r0, kMode == kPoolEntropy ? __ldg(weights + t) : 1.f);
        rowp += ldh;
      }
      if constexpr (kMode == kPoolMean) wsum = static_cast<float>(run_end - t0);
    }
    // entropy mode: (m, sum w) of every run were left by the merge kernel; the other modes have m = 0 and count here
    if (seg_begin >= c_lo && seg_end <= c_hi) {       // the whole prompt: normalise and finish
      if constexpr (kMode != kPoolMax) {
        const float inv = 1.f / (kMode == kPoolEntropy ? seg_s[b] : wsum);
#pragma unroll
        for (int k = 0; k < 8; ++k) acc[k] *= inv;
      }
      store8(pooled + static_cast<int64_t>(b) * d + col, acc);
      if (kMode != kPoolEntropy && scribe) {
        if (seg_m) seg_m[b] = 0.f;
        if (seg_s) seg_s[b] = wsum;
      }
    } else if (seg_begin < c_lo) {
      store8(piece_a + c * d + col, acc);
      if (kMode != kPoolEntropy && scribe) ms_a[c] = make_float2(0.f, wsum);
    } else {
      store8(piece_b + c * d + col, acc);
      if (kMode != kPoolEntropy && scribe) ms_b[c] = make_float2(0.f, wsum);
    }
    t0 = run_end;
    ++b;
  }
}

// One block per prompt (x) and 256-channel slab (y): zero for an empty prompt; a prompt finished by the first stage
// is left as it is; else the pieces piece_b[c0], piece_a[c0+1], ..., piece_a[c1] are rescaled to the largest m, summed
// and normalised (maximum: channel-wise max).  The block's four warps take every fourth piece each (two in flight per
// thread) and their sums are added in warp order, so the result does not depend on timing.  Also leaves the prompt's
// (M, Z) and, if zcat is given, the pooled row once more as [hi | lo] bf16 halves (input of the head's tensor-core layer 1).
constexpr int kCombineLanes = 4;                         // warps of a block = pieces worked on at once
constexpr int kCombineChannels = 32 * 8;                 // channels per block: one warp, 8 per thread
template <int kMode>
__global__ void __launch_bounds__(32 * kCombineLanes)
pool_combine_kernel(const int32_t* __restrict__ off, int B, int d, const float* __restrict__ piece_a,
                    const float* __restrict__ piece_b, const float2* __restrict__ ms_a,
                    const float2* __restrict__ ms_b, float* __restrict__ pooled, float* __restrict__ seg_m,
                    float* __restrict__ seg_s, __nv_bfloat16* __restrict__ zcat, const int32_t* __restrict__ status) {
  if (*status != 0) return;
  __shared__ float part[kCombineLanes][32][9];            // per warp and thread: 8 channel sums and the weight sum
  const int b = blockIdx.x;
  const int pl = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int col = blockIdx.y * kCombineChannels + lane * 8;
  const bool in_d = col < d;
  const bool scribe = blockIdx.y == 0 && threadIdx.x == 0;
  const int64_t s0 = off[b], s1 = off[b + 1];
  float acc[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) acc[k] = 0.f;
  float* dst = pooled + static_cast<int64_t>(b) * d + col;
  __nv_bfloat16* zrow = zcat ? zcat + static_cast<int64_t>(b) * (2 * static_cast<int64_t>(d)) : nullptr;
  if (s1 <= s0) {
    if (pl == 0 && in_d) {
      store8(dst, acc);
      if (zrow) store8_hi_lo(zrow, d, col, acc);
    }
    if (scribe) {
      if (seg_m) seg_m[b] = -INFINITY;
      if (seg_s) seg_s[b] = 0.f;
    }
    return;
  }
  const int64_t c0 = s0 / kPoolChunkTokens, c1 = (s1 - 1) / kPoolChunkTokens;
  if (c0 == c1) {
    if (zrow && pl == 0 && in_d) {
      load8f(dst, acc);
      store8_hi_lo(zrow, d, col, acc);
    }
    return;
  }
  // pieces in order: index 0 = piece_b[c0], index j >= 1 = piece_a[c0 + j]; warp pl takes j = pl, pl + 4, ...
  const int64_t n_pieces = c1 - c0 + 1;
  float M = 0.f;
  if constexpr (kMode != kPoolMax) {
    M = ms_b[c0].x;
    for (int64_t c = c0 + 1; c <= c1; ++c) M = fmaxf(M, ms_a[c].x);
  } else {
#pragma unroll
    for (int k = 0; k < 8; ++k) acc[k] = -INFINITY;
  }
  float Z = 0.f;
  auto piece_ptr = [&](int64_t j) { return (j == 0 ? piece_b : piece_a) + (c0 + j) * d + col; };
  auto piece_ms = [&](int64_t j) { return j == 0 ? ms_b[c0] : ms_a[c0 + j]; };
  auto fold = [&](const float (&pv)[8], float2 ms) {
    if constexpr (kMode == kPoolMax) {
#pragma unroll
      for (int k = 0; k < 8; ++k) acc[k] = fmaxf(acc[k], pv[k]);
    } else {
      const float r = expf(ms.x - M);
      Z = fmaf(ms.y, r, Z);
#pragma unroll
      for (int k = 0; k < 8; ++k) acc[k] = fmaf(pv[k], r, acc[k]);
    }
  };
  if (in_d) {
    int64_t j = pl;
    for (; j + kCombineLanes < n_pieces; j += 2 * kCombineLanes) {     // two pieces in flight per thread
      float p0[8], p1[8];
      const float2 m0 = kMode == kPoolMax ? make_float2(0.f, 0.f) : piece_ms(j);
      const float2 m1 = kMode == kPoolMax ? make_float2(0.f, 0.f) : piece_ms(j + kCombineLanes);
      load8f(piece_ptr(j), p0);
      load8f(piece_ptr(j + kCombineLanes), p1);
      fold(p0, m0);
      fold(p1, m1);
    }
    if (j < n_pieces) {
      float p0[8];
      const float2 m0 = kMode == kPoolMax ? make_float2(0.f, 0.f) : piece_ms(j);
      load8f(piece_ptr(j), p0);
      fold(p0, m0);
    }
  }
#pragma unroll
  for (int k = 0; k < 8; ++k) part[pl][lane][k] = acc[k];
  part[pl][lane][8] = Z;
  __syncthreads();
  if (pl != 0) return;
#pragma unroll
  for (int w = 1; w < kCombineLanes; ++w) {
#pragma unroll
    for (int k = 0; k < 8; ++k) acc[k] = kMode == kPoolMax ? fmaxf(acc[k], part[w][lane][k]) : acc[k] + part[w][lane][k];
    Z += part[w][lane][8];
  }
  if constexpr (kMode != kPoolMax) {
    const float inv = 1.f / Z;
#pragma unroll
    for (int k = 0; k < 8; ++k) acc[k] *= inv;
    if (scribe) {
      if (seg_m) seg_m[b] = M;
      if (seg_s) seg_s[b] = Z;
    }
  }
  if (in_d) {
    store8(dst, acc);
    if (zrow) store8_hi_lo(zrow, d, col, acc);
  }
}

}  // namespace

cudaError_t launch_validate_offsets(const int32_t* offsets, int B, int64_t T, int32_t* status, cudaStream_t stream) {
  validate_offsets_kernel<<<1, 256, 0, stream>>>(offsets, B, T, status);
  return cudaGetLastError();
}

cudaError_t launch_entropy_merge(const float* partials, int slots, int64_t row_stride, int64_t slot_stride, int64_t T,
                                 int64_t row0, float* H, const int32_t* offsets, int B, int32_t* seg_id_out,
                                 int64_t T_check, int32_t* status, cudaStream_t stream, const PoolPrep* prep) {
  if (prep != nullptr && (row0 % kPoolChunkTokens != 0 || offsets == nullptr)) return cudaErrorInvalidValue;
  const unsigned blocks = static_cast<unsigned>((T + kPoolChunkTokens - 1) / kPoolChunkTokens);
  float2* ms_a = prep ? reinterpret_cast<float2*>(prep->piece_ms) : nullptr;
  float2* ms_b = prep ? ms_a + prep->chunks : nullptr;
  entropy_merge_kernel<<<blocks, kMergeThreads, 0, stream>>>(partials, slots, row_stride, slot_stride, T, row0, H, offsets, B,
                                                             seg_id_out, T_check, prep ? prep->inv_alpha : 1.f,
                                                             prep ? prep->weights : nullptr, ms_a, ms_b,
                                                             prep ? prep->seg_m : nullptr, prep ? prep->seg_s : nullptr, status);
  return cudaGetLastError();
}

cudaError_t launch_partials_reduce(const float* partials, int slots, int64_t rows, float* out, const int32_t* status,
                                   cudaStream_t stream) {
  const int threads = 256, rows_per_block = threads / 32;
  const unsigned blocks = static_cast<unsigned>((rows + rows_per_block - 1) / rows_per_block);
  partials_reduce_kernel<<<blocks, threads, 0, stream>>>(partials, slots, rows, out, status);
  return cudaGetLastError();
}

cudaError_t launch_token_weights(const float* H, const int32_t* offsets, int B, int64_t T, float inv_alpha,
                                 const float* seg_m, const float* seg_s, float* weights, const int32_t* status,
                                 cudaStream_t stream) {
  const unsigned blocks = static_cast<unsigned>((T + 255) / 256);
  token_weights_kernel<<<blocks, 256, 0, stream>>>(H, offsets, B, T, inv_alpha, seg_m, seg_s, weights, status);
  return cudaGetLastError();
}

namespace {

template <typename T>
void launch_pool_typed(int mode, dim3 grid, cudaStream_t stream, const T* hidden, int64_t ldh, const float* weights,
                       const int32_t* off, int B, int d, float* pooled, float* piece_a, float* piece_b,
                       float2* ms_a, float2* ms_b, float* seg_m, float* seg_s, const int32_t* status) {
  switch (mode) {
    case kPoolEntropy:
      pool_kernel<T, kPoolEntropy><<<grid, kPoolThreads, 0, stream>>>(hidden, ldh, weights, off, B, d, pooled, piece_a, piece_b, ms_a, ms_b, seg_m, seg_s, status);
      break;
    case kPoolMean:
      pool_kernel<T, kPoolMean><<<grid, kPoolThreads, 0, stream>>>(hidden, ldh, weights, off, B, d, pooled, piece_a, piece_b, ms_a, ms_b, seg_m, seg_s, status);
      break;
    case kPoolMax:
      pool_kernel<T, kPoolMax><<<grid, kPoolThreads, 0, stream>>>(hidden, ldh, weights, off, B, d, pooled, piece_a, piece_b, ms_a, ms_b, seg_m, seg_s, status);
      break;
    default:
      pool_kernel<T, kPoolLast><<<grid, kPoolThreads, 0, stream>>>(hidden, ldh, weights, off, B, d, pooled, piece_a, piece_b, ms_a, ms_b, seg_m, seg_s, status);
      break;
  }
}

}  // namespace

static_assert(static_cast<int>(kPoolMean) == static_cast<int>(EGTP_POOL_MEAN) && static_cast<int>(kPoolMax) == static_cast<int>(EGTP_POOL_MAX) &&
                  static_cast<int>(kPoolLast) == static_cast<int>(EGTP_POOL_LAST), "pooling mode codes");

cudaError_t launch_pool(const void* hidden, int64_t ldh, bool bf16, int mode, const float* weights,
                        const int32_t* offsets, int B, int64_t T, int d, float* pooled, float* piece_a,
                        float* piece_b, float* piece_ms, float* seg_m, float* seg_s, const int32_t* status,
                        cudaStream_t stream) {
  const unsigned chunks = static_cast<unsigned>((T + kPoolChunkTokens - 1) / kPoolChunkTokens);
  const unsigned slabs = static_cast<unsigned>((d + kPoolThreads * 8 - 1) / (kPoolThreads * 8));
  dim3 grid(chunks, slabs);
  float2* ms_a = reinterpret_cast<float2*>(piece_ms);
  float2* ms_b = ms_a + chunks;
  if (bf16)
    launch_pool_typed<__nv_bfloat16>(mode, grid, stream, static_cast<const __nv_bfloat16*>(hidden), ldh, weights, offsets, B, d,
                                     pooled, piece_a, piece_b, ms_a, ms_b, seg_m, seg_s, status);
  else
    launch_pool_typed<float>(mode, grid, stream, static_cast<const float*>(hidden), ldh, weights, offsets, B, d, pooled,
                             piece_a, piece_b, ms_a, ms_b, seg_m, seg_s, status);
  return cudaGetLastError();
}

cudaError_t launch_pool_combine(const int32_t* offsets, int B, int64_t T, int d, int mode, const float* piece_a,
                                const float* piece_b, const float* piece_ms, float* pooled, float* seg_m, float* seg_s,
                                void* zcat, const int32_t* status, cudaStream_t stream) {
  const unsigned chunks = static_cast<unsigned>((T + kPoolChunkTokens - 1) / kPoolChunkTokens);
  const unsigned slabs = static_cast<unsigned>((d + kCombineChannels - 1) / kCombineChannels);
  dim3 grid(B, slabs);
  const float2* ms_a = reinterpret_cast<const float2*>(piece_ms);
  const float2* ms_b = ms_a + chunks;
  __nv_bfloat16* zc = static_cast<__nv_bfloat16*>(zcat);
  constexpr int kThreads = 32 * kCombineLanes;
  if (mode == kPoolMax)
    pool_combine_kernel<kPoolMax><<<grid, kThreads, 0, stream>>>(offsets, B, d, piece_a, piece_b, ms_a, ms_b, pooled, seg_m, seg_s, zc, status);
  else
    pool_combine_kernel<kPoolEntropy><<<grid, kThreads, 0, stream>>>(offsets, B, d, piece_a, piece_b, ms_a, ms_b, pooled, seg_m, seg_s, zc, status);
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
