// Second layer and output mode of the prediction head (paper Sec. 3.2, Eq. 6), shared by the head
// kernel and by the PLP update of a state that is bound to a head.
#pragma once

#include "kernels.h"
#include "../../include/egtp.h"

#include <cuda_bf16.h>

namespace egtp {

template <typename TW>
__device__ __forceinline__ float to_f32(TW v);
template <>
__device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// Called by every thread of a block once the row's hidden activations u[m_h] = ReLU(W1 z + b1) have been
// written to shared memory (the barrier that publishes them is taken here).  o[d_out] is shared scratch.
// o_c = W2[c] . u + b2[c] (one warp per output, lanes stride the hidden units), then
//   scalar mode: y[r] = o[0];  bins mode: p = softmax(o), y[r] = sum_c p_c centres[c]  (Eq. 6).
template <typename TW>
__device__ __forceinline__ void head_output_stage(const float* u, float* o, int m_h, int d_out,
                                                  const TW* __restrict__ W2, const float* __restrict__ b2,
                                                  const float* __restrict__ centres, int mode, float* __restrict__ y,
                                                  float* __restrict__ phat, int r) {
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  __syncthreads();
  for (int c = wid; c < d_out; c += (blockDim.x >> 5)) {
    float v = 0.f;
    for (int j = lane; j < m_h; j += 32) v = fmaf(to_f32<TW>(W2[static_cast<int64_t>(c) * m_h + j]), u[j], v);
#pragma unroll
    for (int of = 16; of > 0; of >>= 1) v += __shfl_xor_sync(0xffffffffu, v, of);
    if (lane == 0) o[c] = v + b2[c];
  }
  __syncthreads();
  if (tid == 0) {
    if (mode == EGTP_HEAD_SCALAR) {
      if (y) y[r] = o[0];
    } else {
      float mx = o[0];
      for (int c = 1; c < d_out; ++c) mx = fmaxf(mx, o[c]);
      float den = 0.f;
      for (int c = 0; c < d_out; ++c) den += expf(o[c] - mx);
      float ev = 0.f;
      for (int c = 0; c < d_out; ++c) {
        const float pc = expf(o[c] - mx) / den;
        ev = fmaf(pc, centres[c], ev);
        if (phat) phat[static_cast<int64_t>(r) * d_out + c] = pc;
      }
      if (y) y[r] = ev;
    }
  }
}

}  // namespace egtp
