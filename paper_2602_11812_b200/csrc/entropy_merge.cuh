// Merge of the LM-head kernel's per-slot entropy partials (paper Eq. 2).
// A partial is (m, s, t2) over a range of the vocabulary: m = max logit, s = sum 2^y,
// t2 = sum 2^y * y with y = (x - m) log2 e.  Two partials combine by rescaling both to the
// larger m; the token's entropy is H = ln S - ln2 * T2 / S (both terms are >= 0).
#pragma once

#include "kernels.h"

namespace egtp {

struct EntropyPartial {
  float m, s, t2;
};

__device__ __forceinline__ EntropyPartial combine_partials(const EntropyPartial& a, const EntropyPartial& b) {
  constexpr float kLog2e = 1.4426950408889634f;
  EntropyPartial r;
  r.m = fmaxf(a.m, b.m);
  const float da = (a.m - r.m) * kLog2e, db = (b.m - r.m) * kLog2e;
  const float ra = exp2f(da), rb = exp2f(db);
  r.s = fmaf(a.s, ra, b.s * rb);
  r.t2 = ra * fmaf(da, a.s, a.t2) + rb * fmaf(db, b.s, b.t2);
  return r;
}

// Combines the 32 lanes' partials: every lane returns the same (m, s, t2).  The warp maximum is found
// first, then each lane rescales once and the sums go through an xor butterfly (commutative pairs, so
// all lanes hold bitwise the same result and the result does not depend on scheduling).
__device__ __forceinline__ EntropyPartial warp_combine_partials(EntropyPartial p) {
  constexpr float kLog2e = 1.4426950408889634f;
  float M = p.m;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
  const float dm = (p.m - M) * kLog2e;
  const float r = exp2f(dm);
  float s = p.s * r;
  float t2 = r * fmaf(dm, p.s, p.t2);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    s += __shfl_xor_sync(0xffffffffu, s, o);
    t2 += __shfl_xor_sync(0xffffffffu, t2, o);
  }
  return {M, s, t2};
}

// All 32 lanes of a warp call this with the same row pointer ([slots][3] floats); every lane
// returns H.  The order of operations is fixed, so the result is bitwise reproducible.
// slot j of the row lives at row + j * slot_stride (floats): 3 for the LM-head kernel's [row][slot][3]
// layout, rows * 3 for partials gathered rank-major from several GPUs ([rank][row][3]).
__device__ __forceinline__ EntropyPartial merge_partials_warp_raw(const float* __restrict__ row, int slots,
                                                                  int64_t slot_stride, int lane) {
  EntropyPartial acc = {kNegBig, 0.f, 0.f};
  for (int j = lane; j < slots; j += 32) {
    const float* pj = row + j * slot_stride;
    const EntropyPartial q = {pj[0], pj[1], pj[2]};
    acc = combine_partials(acc, q);
  }
  return warp_combine_partials(acc);
}

// The same merge by a group of kLanes consecutive lanes (kLanes a power of two): 32 / kLanes rows per warp at
// once.  Every lane of the group returns the row's (m, s, t2).
template <int kLanes>
__device__ __forceinline__ EntropyPartial merge_partials_group_raw(const float* __restrict__ row, int slots,
                                                                   int64_t slot_stride, int lane_in_group) {
  constexpr float kLog2e = 1.4426950408889634f;
  EntropyPartial acc = {kNegBig, 0.f, 0.f};
  for (int j = lane_in_group; j < slots; j += kLanes) {
    const float* pj = row + j * slot_stride;
    const EntropyPartial q = {pj[0], pj[1], pj[2]};
    acc = combine_partials(acc, q);
  }
  float M = acc.m;
#pragma unroll
  for (int o = kLanes / 2; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
  const float dm = (acc.m - M) * kLog2e;
  const float r = exp2f(dm);
  float s = acc.s * r;
  float t2 = r * fmaf(dm, acc.s, acc.t2);
#pragma unroll
  for (int o = kLanes / 2; o > 0; o >>= 1) {
    s += __shfl_xor_sync(0xffffffffu, s, o);
    t2 += __shfl_xor_sync(0xffffffffu, t2, o);
  }
  return {M, s, t2};
}

__device__ __forceinline__ float entropy_of(const EntropyPartial& p) {
  constexpr float kLn2 = 0.6931471805599453f;
  return logf(p.s) - kLn2 * p.t2 / p.s;
}

__device__ __forceinline__ float merge_partials_warp(const float* __restrict__ row, int slots, int64_t slot_stride,
                                                     int lane) {
  return entropy_of(merge_partials_warp_raw(row, slots, slot_stride, lane));
}

}  // namespace egtp
