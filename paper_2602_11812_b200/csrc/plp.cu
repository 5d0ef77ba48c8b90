// Progressive Length Prediction, running-state update (paper Sec. 3.3, Eq. 8).
// z_t is the entropy-weighted pool (Eq. 3-4) over a sequence's prompt tokens followed by its
// generated tokens 1..t.  Per slot the library keeps the online-softmax triple
//   m = max_i H_i/alpha,  s = sum_i exp(H_i/alpha - m),  acc = sum_i exp(H_i/alpha - m) h_i,
// which one new token (entropy H', hidden h') updates to
//   m' = max(m, H'/alpha), s' = s e^(m-m') + e^(H'/alpha-m'), acc' = acc e^(m-m') + e^(H'/alpha-m') h',
// and z = acc'/s'.  H' is merged here from the LM-head kernel's partials (no separate launch).
// HBM-bound (acc read + write, hidden read, z write): one block per live row.
#include "kernels.h"
#include "entropy_merge.cuh"
#include "head_out.cuh"
#include "sm100_ptx.cuh"
#include "../../include/egtp.h"

#include <cuda_bf16.h>

#include <algorithm>

namespace egtp {

namespace {

template <typename T>
__device__ __forceinline__ void load8(const T* p, float (&v)[8]);
template <>
__device__ __forceinline__ void load8<__nv_bfloat16>(const __nv_bfloat16* p, float (&v)[8]) {
  const uint4 q = __ldg(reinterpret_cast<const uint4*>(p));
  const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}
template <>
__device__ __forceinline__ void load8<float>(const float* p, float (&v)[8]) {
  const float4 a = __ldg(reinterpret_cast<const float4*>(p));
  const float4 b = __ldg(reinterpret_cast<const float4*>(p) + 1);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
  v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}

constexpr int kPlpMaxThreads = 1024;

// Two live rows of one step must not name the same slot (they would race on its state).  Every step of a state has
// a stamp (epoch[0]); a block claims its slot by swapping the stamp into the slot's owner word and finds the stamp
// already there if another row of the same step was first.  The last block of a launch to leave (epoch[1] counts them)
// moves the stamp on, so every block of a launch sees the same stamp whatever the order they run in, and a step that is
// replayed from a CUDA graph gets a fresh stamp each time.
__device__ __forceinline__ bool claim_slot(int32_t* owner, int slot, int stamp) {
  return atomicExch(owner + slot, stamp) != stamp;
}
__device__ __forceinline__ void leave_step(int32_t* epoch, int stamp) {
  __threadfence();
  if (atomicAdd(epoch + 1, 1) == static_cast<int>(gridDim.x) - 1) {
    epoch[1] = 0;
    __threadfence();
    *reinterpret_cast<volatile int32_t*>(epoch) = stamp == 0x7fffffff ? 1 : stamp + 1;
  }
}

template <typename T>
__global__ void __launch_bounds__(kPlpMaxThreads)
plp_update_kernel(const T* __restrict__ hidden_step, int64_t ldh, const float* __restrict__ partials, int slots,
                  int64_t row_stride, int64_t slot_stride, float* __restrict__ Hstep_out, const int32_t* __restrict__ slot_ids,
                  const int32_t* __restrict__ reset_src, const float* __restrict__ src_m,
                  const float* __restrict__ src_s, const float* __restrict__ src_pooled, int n_src, int d,
                  int num_slots, float inv_alpha, float* __restrict__ st_m, float* __restrict__ st_s,
                  float* __restrict__ st_acc, float* __restrict__ z, int64_t ldz, __nv_bfloat16* __restrict__ zcat,
                  int32_t* __restrict__ owner, int32_t* __restrict__ epoch, int32_t* status) {
  __shared__ int refused;
  const int stamp = *reinterpret_cast<volatile int32_t*>(epoch);
  const int i = blockIdx.x;
  const int slot = slot_ids ? slot_ids[i] : i;
  const int rs = reset_src ? reset_src[i] : PLP_RESET_KEEP;
  if (threadIdx.x == 0) {
    int r = *status != 0 ? 1 : 0;
    if (r == 0 && (slot < 0 || slot >= num_slots || rs < PLP_RESET_KEEP || rs >= n_src || !claim_slot(owner, slot, stamp))) {
      atomicCAS(status, 0, EGTP_ERR_BAD_SLOT);      // out of range, or a second row of this step on the same slot
      r = 1;
    }
    refused = r;
  }
  __syncthreads();
  if (refused != 0) {
    if (threadIdx.x == 0) leave_step(epoch, stamp);
    return;
  }
  // state before this token
  float m_old, s_old;
  const float* acc_src;   // nullptr = zeros
  float acc_scale_in;     // factor that turns *acc_src into acc (src_pooled rows are normalised pools)
  if (rs == PLP_RESET_KEEP) {
    m_old = st_m[slot]; s_old = st_s[slot];
    acc_src = st_acc + static_cast<int64_t>(slot) * d; acc_scale_in = 1.f;
  } else if (rs == PLP_RESET_EMPTY) {
    m_old = -INFINITY; s_old = 0.f; acc_src = nullptr; acc_scale_in = 0.f;
  } else {
    m_old = src_m[rs]; s_old = src_s[rs];
    acc_src = src_pooled + static_cast<int64_t>(rs) * d; acc_scale_in = s_old;
  }
  if (!(s_old > 0.f)) acc_src = nullptr;    // an empty sequence carries nothing over
  float* acc_dst = st_acc + static_cast<int64_t>(slot) * d;
  const T* hrow = hidden_step + static_cast<int64_t>(i) * ldh;
  float* zrow = z ? z + static_cast<int64_t>(i) * ldz : nullptr;
  // zcat (optional): z as two bf16 halves [hi | lo] per row, the operand of the head's tensor-core layer 1
  __nv_bfloat16* zc = zcat ? zcat + static_cast<int64_t>(i) * (2 * static_cast<int64_t>(d)) : nullptr;

  // first pass of loads is issued before the entropy merge so that both latencies overlap
  int col = threadIdx.x * 8;
  float h[8], acc[8];
  const bool first = col < d;
  if (first) {
    load8<T>(hrow + col, h);
    if (acc_src != nullptr) load8<float>(acc_src + col, acc);
  }
  // Eq. 2 for this row: every warp merges the row's partials (same value in all of them)
  const float H_new = merge_partials_warp(partials + static_cast<int64_t>(i) * row_stride, slots, slot_stride, threadIdx.x & 31);
  if (threadIdx.x == 0 && Hstep_out != nullptr) Hstep_out[i] = H_new;
  const float a = H_new * inv_alpha;
  const float m_new = fmaxf(m_old, a);
  const float carry = (s_old > 0.f) ? expf(m_old - m_new) : 0.f;
  const float e = expf(a - m_new);
  const float s_new = fmaf(s_old, carry, e);
  const float inv_s = 1.f / s_new;
  const float acc_factor = carry * acc_scale_in;
  __syncthreads();   // every thread has read the old state before anyone overwrites it
  for (; col < d; col += blockDim.x * 8) {
    if (col != static_cast<int>(threadIdx.x) * 8) {
      load8<T>(hrow + col, h);
      if (acc_src != nullptr) load8<float>(acc_src + col, acc);
    }
    if (acc_src != nullptr) {
#pragma unroll
      for (int k = 0; k < 8; ++k) acc[k] = fmaf(acc[k], acc_factor, e * h[k]);
    } else {
#pragma unroll
      for (int k = 0; k < 8; ++k) acc[k] = e * h[k];
    }
    reinterpret_cast<float4*>(acc_dst + col)[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
    reinterpret_cast<float4*>(acc_dst + col)[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
    if (zrow != nullptr) {
      reinterpret_cast<float4*>(zrow + col)[0] = make_float4(acc[0] * inv_s, acc[1] * inv_s, acc[2] * inv_s, acc[3] * inv_s);
      reinterpret_cast<float4*>(zrow + col)[1] = make_float4(acc[4] * inv_s, acc[5] * inv_s, acc[6] * inv_s, acc[7] * inv_s);
    }
    if (zc != nullptr) {
      __align__(16) __nv_bfloat16 hi[8], lo[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const float zv = acc[k] * inv_s;
        hi[k] = __float2bfloat16_rn(zv);
        lo[k] = __float2bfloat16_rn(zv - __bfloat162float(hi[k]));
      }
      *reinterpret_cast<uint4*>(zc + col) = *reinterpret_cast<const uint4*>(hi);
      *reinterpret_cast<uint4*>(zc + d + col) = *reinterpret_cast<const uint4*>(lo);
    }
  }
  if (threadIdx.x == 0) {
    st_m[slot] = m_new;
    st_s[slot] = s_new;
    leave_step(epoch, stamp);
  }
}

// The same update for a state that is bound to a prediction head (Sec. 3.2-3.3).  Layer 1 of the head is linear
// before its ReLU, W1 z = (W1 acc) / s, so next to acc the slot keeps P = W1 acc [m_h] and advances it with the
// same recurrence, P' = P e^(m-m') + e^(H'/alpha-m') (W1 h'), where g = W1 h' was produced by the LM-head kernel
// as extra output columns (or by a launch of that kernel over the head columns alone, K split over g_splits
// slices that are added here in order).  The block then finishes the head for its row: u = ReLU(P'/s' + b1), o = W2 u + b2,
// output mode (Eq. 6).  A row that restarts from EGTP row r takes P from src_proj[r] = W1 src_pooled[r].
// z is written only when the caller asked for it.
template <typename T, typename TW>
__global__ void __launch_bounds__(kPlpMaxThreads)
plp_update_bound_kernel(const T* __restrict__ hidden_step, int64_t ldh, const float* __restrict__ partials, int slots,
                        int64_t row_stride, int64_t slot_stride, float* __restrict__ Hstep_out,
                        const int32_t* __restrict__ slot_ids, const int32_t* __restrict__ reset_src,
                        const float* __restrict__ src_m, const float* __restrict__ src_s,
                        const float* __restrict__ src_pooled, const float* __restrict__ src_proj, int n_src, int d,
                        int num_slots, float inv_alpha, float* __restrict__ st_m, float* __restrict__ st_s,
                        float* __restrict__ st_acc, float* __restrict__ st_proj, float* __restrict__ z, int64_t ldz,
                        const float* __restrict__ g, int64_t ldg, int g_splits, int64_t g_split_stride, int m_h,
                        int d_out, const float* __restrict__ b1,
                        const TW* __restrict__ W2, const float* __restrict__ b2, const float* __restrict__ centres,
                        int mode, float* __restrict__ y, int32_t* __restrict__ owner, int32_t* __restrict__ epoch,
                        int32_t* status) {
  // Launched with programmatic stream serialization: this block may start while the LM-head kernel is still
  // running.  Its inputs and the state rows (last written by an earlier, completed kernel) are read ahead;
  // the status word, the entropy partials and g come after pdl_wait().
  extern __shared__ float smem[];
  float* u = smem;            // [m_h]
  float* o = smem + m_h;      // [d_out]
  // the next step's LM-head kernel may set its blocks up as this grid drains (it waits for this grid's end before
  // it reads or writes anything in global memory)
  pdl_launch_dependents();
  __shared__ int refused;
  const int i = blockIdx.x;
  const int slot_in = slot_ids ? slot_ids[i] : i;
  const int rs_in = reset_src ? reset_src[i] : PLP_RESET_KEEP;
  // a row with a slot or reset source out of range reads ahead as if it were row 0 of an untouched state and is
  // refused after the wait below (every block has to take part in the step's bookkeeping there)
  const bool in_range = slot_in >= 0 && slot_in < num_slots && rs_in >= PLP_RESET_KEEP && rs_in < n_src;
  const int slot = in_range ? slot_in : 0;
  const int rs = in_range ? rs_in : PLP_RESET_KEEP;
  float m_old, s_old;
  const float* acc_src;    // nullptr = zeros
  const float* proj_src;   // W1 times the vector acc_src points at
  float acc_scale_in;
  if (rs == PLP_RESET_KEEP) {
    m_old = st_m[slot]; s_old = st_s[slot];
    acc_src = st_acc + static_cast<int64_t>(slot) * d; proj_src = st_proj + static_cast<int64_t>(slot) * m_h;
    acc_scale_in = 1.f;
  } else if (rs == PLP_RESET_EMPTY) {
    m_old = -INFINITY; s_old = 0.f; acc_src = nullptr; proj_src = nullptr; acc_scale_in = 0.f;
  } else {
    m_old = src_m[rs]; s_old = src_s[rs];
    acc_src = src_pooled + static_cast<int64_t>(rs) * d; proj_src = src_proj + static_cast<int64_t>(rs) * m_h;
    acc_scale_in = s_old;
  }
  if (!(s_old > 0.f)) { acc_src = nullptr; proj_src = nullptr; }
  float* acc_dst = st_acc + static_cast<int64_t>(slot) * d;
  const T* hrow = hidden_step + static_cast<int64_t>(i) * ldh;
  float* zrow = z ? z + static_cast<int64_t>(i) * ldz : nullptr;

  int col = threadIdx.x * 8;
  float h[8], acc[8];
  const bool first = col < d;
  if (first) {
    load8<T>(hrow + col, h);
    if (acc_src != nullptr) load8<float>(acc_src + col, acc);
  }
  pdl_wait();
  // Thread 0 looks at the status word and claims the slot while all warps already merge the row's entropy (reads
  // only); nothing is written before the block knows that it may go ahead.
  const int stamp = *reinterpret_cast<volatile int32_t*>(epoch);
  if (threadIdx.x == 0) {
    int r = *status != 0 ? 1 : 0;
    if (r == 0 && (!in_range || !claim_slot(owner, slot, stamp))) {
      atomicCAS(status, 0, EGTP_ERR_BAD_SLOT);      // out of range, or a second row of this step on the same slot
      r = 1;
    }
    refused = r;
  }
  const float H_new = merge_partials_warp(partials + static_cast<int64_t>(i) * row_stride, slots, slot_stride, threadIdx.x & 31);
  const float a = H_new * inv_alpha;
  const float m_new = fmaxf(m_old, a);
  const float carry = (s_old > 0.f) ? expf(m_old - m_new) : 0.f;
  const float e = expf(a - m_new);
  const float s_new = fmaf(s_old, carry, e);
  const float inv_s = 1.f / s_new;
  const float acc_factor = carry * acc_scale_in;
  __syncthreads();
  if (refused != 0) {
    if (threadIdx.x == 0) leave_step(epoch, stamp);
    return;
  }
  if (threadIdx.x == 0 && Hstep_out != nullptr) Hstep_out[i] = H_new;
  // the projected state and the head's hidden layer
  const float* grow = g + static_cast<int64_t>(i) * ldg;
  float* proj_dst = st_proj + static_cast<int64_t>(slot) * m_h;
  for (int j = threadIdx.x; j < m_h; j += blockDim.x) {
    float gj = grow[j];
    for (int sp = 1; sp < g_splits; ++sp) gj += grow[sp * g_split_stride + j];   // K splits, added in order
    const float pj = (proj_src != nullptr) ? fmaf(proj_src[j], acc_factor, e * gj) : e * gj;
    u[j] = fmaxf(0.f, fmaf(pj, inv_s, b1[j]));
    proj_dst[j] = pj;      // element j is read and written by this thread only
  }
  __syncthreads();   // every thread has read the old state before anyone overwrites it
  for (; col < d; col += blockDim.x * 8) {
    if (col != static_cast<int>(threadIdx.x) * 8) {
      load8<T>(hrow + col, h);
      if (acc_src != nullptr) load8<float>(acc_src + col, acc);
    }
    if (acc_src != nullptr) {
#pragma unroll
      for (int k = 0; k < 8; ++k) acc[k] = fmaf(acc[k], acc_factor, e * h[k]);
    } else {
#pragma unroll
      for (int k = 0; k < 8; ++k) acc[k] = e * h[k];
    }
    reinterpret_cast<float4*>(acc_dst + col)[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
    reinterpret_cast<float4*>(acc_dst + col)[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
    if (zrow != nullptr) {
      reinterpret_cast<float4*>(zrow + col)[0] = make_float4(acc[0] * inv_s, acc[1] * inv_s, acc[2] * inv_s, acc[3] * inv_s);
      reinterpret_cast<float4*>(zrow + col)[1] = make_float4(acc[4] * inv_s, acc[5] * inv_s, acc[6] * inv_s, acc[7] * inv_s);
    }
  }
  if (threadIdx.x == 0) {
    st_m[slot] = m_new;
    st_s[slot] = s_new;
    leave_step(epoch, stamp);
  }
  head_output_stage<TW>(u, o, m_h, d_out, W2, b2, centres, mode, y, nullptr, i);
}

}  // namespace

// One block per row, eight channels per thread and pass.  A row is a chain of dependent round trips (partials ->
// entropy -> update), so the kernel wants every block resident at once: with more rows than fit at d / 8 threads
// per block, blocks shrink (down to 128 threads, several passes over the row) until one wave holds them all.
int update_threads(int rows, int d, int min_threads) {
  int threads = std::min(kPlpMaxThreads, std::max(min_threads, (d / 8 + 31) / 32 * 32));
  int device = 0, sms = 0;
  if (cudaGetDevice(&device) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sms <= 0)
    return threads;
  while (threads > 128 && static_cast<int64_t>(rows) > static_cast<int64_t>(sms) * (2048 / threads))
    threads = std::max(128, (threads / 2 + 31) / 32 * 32);
  return threads;
}

cudaError_t launch_plp_update_bound(const void* hidden_step, int64_t ldh, const float* partials, int slots,
                                    int64_t row_stride, int64_t slot_stride, float* Hstep_out, const int32_t* slot_ids,
                                    const int32_t* reset_src, const float* src_m, const float* src_s,
                                    const float* src_pooled, const float* src_proj, int n_src, int rows, int d,
                                    int num_slots, float inv_alpha, float* st_m, float* st_s, float* st_acc,
                                    float* st_proj, float* z, int64_t ldz, const float* g, int64_t ldg, int g_splits,
                                    int64_t g_split_stride, const HeadArgs& h, float* y, int32_t* owner, int32_t* epoch,
                                    int32_t* status, cudaStream_t stream, bool overlap_previous) {
  const int threads = update_threads(rows, d, 64);
  const size_t smem = static_cast<size_t>(h.m_h + h.d_out) * sizeof(float);
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(rows);
  cfg.blockDim = dim3(threads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr{};
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = overlap_previous ? 1 : 0;
  const __nv_bfloat16* hs = static_cast<const __nv_bfloat16*>(hidden_step);
  const __nv_bfloat16* W2 = static_cast<const __nv_bfloat16*>(h.W2);
  return cudaLaunchKernelEx(&cfg, plp_update_bound_kernel<__nv_bfloat16, __nv_bfloat16>, hs, ldh, partials, slots,
                            row_stride, slot_stride, Hstep_out, slot_ids, reset_src, src_m, src_s, src_pooled, src_proj,
                            n_src, d, num_slots, inv_alpha, st_m, st_s, st_acc, st_proj, z, ldz, g, ldg, g_splits, g_split_stride,
                            h.m_h, h.d_out,
                            h.b1, W2, h.b2, h.centres, h.mode, y, owner, epoch, status);
}

cudaError_t launch_plp_update(const void* hidden_step, int64_t ldh, bool bf16, const float* partials, int slots,
                              int64_t row_stride, int64_t slot_stride, float* Hstep_out, const int32_t* slot_ids, const int32_t* reset_src, const float* src_m,
                              const float* src_s, const float* src_pooled, int n_src, int rows, int d, int num_slots,
                              float inv_alpha, float* st_m, float* st_s, float* st_acc, float* z, int64_t ldz,
                              int32_t* owner, int32_t* epoch, int32_t* status, cudaStream_t stream, void* zcat) {
  const int threads = update_threads(rows, d, 32);
  if (bf16) {
    plp_update_kernel<__nv_bfloat16><<<rows, threads, 0, stream>>>(
        static_cast<const __nv_bfloat16*>(hidden_step), ldh, partials, slots, row_stride, slot_stride, Hstep_out, slot_ids, reset_src, src_m, src_s, src_pooled,
        n_src, d, num_slots, inv_alpha, st_m, st_s, st_acc, z, ldz, static_cast<__nv_bfloat16*>(zcat), owner, epoch, status);
  } else {
    plp_update_kernel<float><<<rows, threads, 0, stream>>>(static_cast<const float*>(hidden_step), ldh, partials, slots, row_stride, slot_stride, Hstep_out, slot_ids,
                                                       reset_src, src_m, src_s, src_pooled, n_src, d, num_slots,
                                                       inv_alpha, st_m, st_s, st_acc, z, ldz, static_cast<__nv_bfloat16*>(zcat), owner, epoch, status);
  }
  return cudaGetLastError();
}

}  // namespace egtp
