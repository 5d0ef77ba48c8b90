// C ABI of the library (see include/egtp.h): argument checks, workspace, TMA tensor maps,
// kernel sequencing, per-kernel event timing.  No arithmetic of the method lives here.
#include "../../include/egtp.h"
#include "kernels.h"

#include <cuda.h>
#include <cuda_runtime.h>
#include <cudaTypedefs.h>

#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>
#include <vector>

using namespace egtp;

namespace {

struct EventPair {
  cudaEvent_t start, stop;
  int kernel;
};

}  // namespace

struct egtp_ctx {
  int device = 0;
  int num_sms = 0;
  int pair_workers = 0;           // CTA pairs of the pair kernels this device holds at once
  int64_t max_tokens = 0;
  int32_t max_batch = 0, max_d = 0, max_V = 0;
  PFN_cuTensorMapEncodeTiled_v12000 encode = nullptr;

  // workspace (device)
  float* partials = nullptr;      int64_t slot_row_capacity = 0;   // rows x slots the partial buffer holds
  float* H = nullptr;             // [max(max_tokens, max_batch)]
  int32_t* arrivals = nullptr;    // [max(max_tokens, max_batch)], zero between calls: per-row block counters
  float* weights = nullptr;       // [max_tokens]: unnormalised Eq. 3 weights, chunk-local reference
  float* seg_m = nullptr;         // [max_batch]
  float* seg_s = nullptr;         // [max_batch]
  float* pooled = nullptr;        // [max_batch][max_d]  (also z of a PLP step)
  float* piece_a = nullptr;       // [chunks][max_d]
  float* piece_b = nullptr;       // [chunks][max_d]
  float* piece_ms = nullptr;      // [2 * chunks][2]: (m, sum of weights) of every piece
  float* head_partial = nullptr;  int64_t head_partial_floats = 0;
  void* small_rows = nullptr;     // [kMinLmheadRows][max_d] in the widest dtype: tiny batches, zero-padded
  void* zcat = nullptr;           // [max_batch][2 * max_d] bf16: head inputs as [hi | lo] halves (tensor-core layer 1)
  float* yhat = nullptr;          // [max_batch]
  int32_t* status = nullptr;      // [1]
  // staging for the *_host entry points (device)
  void* hidden_stage = nullptr;   // [max_tokens][max_d] in the widest supported dtype; NULL without host staging
  bool host_staging = true;
  int32_t* offsets_stage = nullptr;  // [max_batch + 1]
  int32_t* reset_stage = nullptr;    // [2][max_batch]
  int64_t stage_bytes = 0;           // bytes of hidden_stage
  cudaEvent_t host_in_ready[2] = {}, host_stage_free[2] = {};   // pipelined host steps: two halves of the staging buffers
  int host_parity = 0;
  int64_t bytes = 0;

  // bookkeeping
  int lmhead_mode = EGTP_LMHEAD_AUTO;
  int lmhead_chunks = 0;          // 0 = chosen by the planner
  bool launch_overlap = true;     // programmatic dependent launch of the LM-head and bound-update kernels
  // host-buffer entry points: copies run on their own stream, one event per piece of the batch
  static constexpr int kMaxPieces = 4;
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t piece_ready[kMaxPieces] = {};
  cudaEvent_t stage_free = nullptr;
  cudaEvent_t fork_ev = nullptr, join_ev = nullptr;   // side work that runs next to the main stream inside one call
  int64_t launches = 0;
  bool profiling = false;
  std::vector<EventPair> pending;
  std::vector<EventPair> free_events;
  double ms_acc[EGTP_NUM_KERNELS] = {};
  int64_t n_acc[EGTP_NUM_KERNELS] = {};
};

struct plp_state {
  egtp_ctx* ctx = nullptr;
  int device = 0;               // the context's device (kept here: the state may outlive the context object)
  int32_t num_slots = 0, d = 0;
  float* m = nullptr;
  float* s = nullptr;
  float* acc = nullptr;
  int32_t* owner = nullptr;     // [num_slots]: stamp of the last step that touched the slot (duplicate slot ids)
  int32_t* epoch = nullptr;     // [2]: stamp of the next step, blocks of the running step that have left
  // binding to one prediction head (plp_state_bind_head)
  bool bound = false;
  egtp_head bound_head{};
  float* proj = nullptr;        // [num_slots][m_h]: W1 acc
  bool proj_valid = false;      // false: acc was changed without proj (import, a step through another route)
  float* src_proj = nullptr;    // [ctx->max_batch][m_h]: W1 src_pooled of the current step
  float* head_g = nullptr;      // [g_rows][ldg_max]: W1 h' of the current step, written by the LM-head kernel
  int64_t g_rows = 0, ldg_max = 0;
  int g_max_splits = 1;         // K splits head_g has room for (projection launches without an LM head)
};

namespace {

const char* const kKernelNames[EGTP_NUM_KERNELS] = {
    "validate_offsets", "lmhead_entropy", "entropy_merge", "token_weights", "pool",
    "pool_combine",     "head_hidden",    "head_out",      "plp_update",    "logits_entropy",
    "stage_rows"};

template <typename T>
cudaError_t dev_alloc(egtp_ctx* c, T** p, int64_t count) {
  const size_t bytes = static_cast<size_t>(std::max<int64_t>(count, 1)) * sizeof(T);
  cudaError_t e = cudaMalloc(reinterpret_cast<void**>(p), bytes);
  if (e == cudaSuccess) c->bytes += static_cast<int64_t>(bytes);
  return e;
}

void free_ctx_memory(egtp_ctx* c) {
  cudaFree(c->partials); cudaFree(c->H); cudaFree(c->arrivals); cudaFree(c->weights); cudaFree(c->seg_m); cudaFree(c->seg_s);
  cudaFree(c->pooled); cudaFree(c->piece_a); cudaFree(c->piece_b); cudaFree(c->piece_ms); cudaFree(c->head_partial); cudaFree(c->zcat); cudaFree(c->small_rows); cudaFree(c->yhat);
  cudaFree(c->status); cudaFree(c->hidden_stage); cudaFree(c->offsets_stage); cudaFree(c->reset_stage);
  if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
  for (auto& e : c->piece_ready) if (e) cudaEventDestroy(e);
  if (c->stage_free) cudaEventDestroy(c->stage_free);
  for (auto& e : c->host_in_ready) if (e) cudaEventDestroy(e);
  for (auto& e : c->host_stage_free) if (e) cudaEventDestroy(e);
  if (c->fork_ev) cudaEventDestroy(c->fork_ev);
  if (c->join_ev) cudaEventDestroy(c->join_ev);
  for (auto& e : c->pending) { cudaEventDestroy(e.start); cudaEventDestroy(e.stop); }
  for (auto& e : c->free_events) { cudaEventDestroy(e.start); cudaEventDestroy(e.stop); }
}

// Brackets one kernel launch with events when profiling is on; counts launches always.
struct LaunchScope {
  egtp_ctx* c;
  cudaStream_t stream;
  EventPair ev{};
  bool timed = false;
  LaunchScope(egtp_ctx* ctx, int kernel, cudaStream_t s) : c(ctx), stream(s) {
    c->launches += 1;
    if (!c->profiling) return;
    if (!c->free_events.empty()) {
      ev = c->free_events.back();
      c->free_events.pop_back();
    } else {
      if (cudaEventCreate(&ev.start) != cudaSuccess) return;
      if (cudaEventCreate(&ev.stop) != cudaSuccess) { cudaEventDestroy(ev.start); return; }
    }
    ev.kernel = kernel;
    timed = true;
    cudaEventRecord(ev.start, stream);
  }
  ~LaunchScope() {
    if (!timed) return;
    cudaEventRecord(ev.stop, stream);
    c->pending.push_back(ev);
  }
};

int elem_bytes(int dtype) { return dtype == EGTP_BF16 ? 2 : 4; }

// 2-D K-major tensor map: inner dimension = d elements, outer = rows; box = 128 bytes x box_rows,
// 128-byte swizzle, out-of-range elements read as zero.
int make_tensor_map(egtp_ctx* c, CUtensorMap* map, const void* base, int dtype, int64_t rows, int d, int64_t ld,
                    int box_rows) {
  const int eb = elem_bytes(dtype);
  cuuint64_t gdim[2] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(rows)};
  cuuint64_t gstride[1] = {static_cast<cuuint64_t>(ld) * eb};
  cuuint32_t box[2] = {static_cast<cuuint32_t>(kRowBytes / eb), static_cast<cuuint32_t>(box_rows)};
  cuuint32_t estr[2] = {1, 1};
  const CUtensorMapDataType dt = dtype == EGTP_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
  // 256-byte L2 promotion: a 128-byte row segment brings its neighbour (the next k block of the same row)
  // into L2 with it; measured 10 % faster than no promotion when W streams from HBM
  CUresult r = c->encode(map, dt, 2, const_cast<void*>(base), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? EGTP_OK : EGTP_ERR_CUDA;
}

int check_lm(const egtp_ctx* c, const egtp_lm_head* lm, const void* hidden, int64_t ldh) {
  if (!lm || !lm->W || !hidden) return EGTP_ERR_INVALID_ARG;
  if (lm->d <= 0 || lm->V <= 0 || lm->ldw < lm->d || ldh < lm->d) return EGTP_ERR_INVALID_ARG;
  if (lm->dtype != EGTP_F32 && lm->dtype != EGTP_BF16) return EGTP_ERR_UNSUPPORTED;
  const int eb = elem_bytes(lm->dtype);
  if (lm->d % 16 != 0) return EGTP_ERR_UNSUPPORTED;
  if ((lm->ldw * eb) % 16 != 0 || (ldh * eb) % 16 != 0) return EGTP_ERR_UNSUPPORTED;
  if (reinterpret_cast<uintptr_t>(lm->W) % 16 != 0 || reinterpret_cast<uintptr_t>(hidden) % 16 != 0)
    return EGTP_ERR_UNSUPPORTED;
  if (lm->d > c->max_d || lm->V > c->max_V) return EGTP_ERR_CAPACITY;
  return EGTP_OK;
}

int check_head(const egtp_ctx* c, const egtp_head* h, int d) {
  (void)c;
  if (!h->W1 || !h->b1 || !h->W2 || !h->b2) return EGTP_ERR_INVALID_ARG;
  if (h->d != d || h->m_h <= 0 || h->d_out <= 0) return EGTP_ERR_INVALID_ARG;
  if (h->wdtype != EGTP_F32 && h->wdtype != EGTP_BF16) return EGTP_ERR_UNSUPPORTED;
  if (h->m_h > 8192 || h->d_out > 256) return EGTP_ERR_UNSUPPORTED;
  if (h->mode == EGTP_HEAD_SCALAR) {
    if (h->d_out != 1) return EGTP_ERR_INVALID_ARG;
  } else if (h->mode == EGTP_HEAD_BINS) {
    if (!h->centres) return EGTP_ERR_INVALID_ARG;
  } else {
    return EGTP_ERR_INVALID_ARG;
  }
  if (reinterpret_cast<uintptr_t>(h->W1) % 16 != 0) return EGTP_ERR_UNSUPPORTED;
  return EGTP_OK;
}

HeadArgs head_args(const egtp_head* h) {
  HeadArgs a{};
  a.W1 = h->W1; a.b1 = h->b1; a.W2 = h->W2; a.b2 = h->b2; a.centres = h->centres;
  a.d = h->d; a.m_h = h->m_h; a.d_out = h->d_out; a.bf16 = h->wdtype == EGTP_BF16; a.mode = h->mode;
  return a;
}

#define EGTP_CUDA_TRY(expr)                       \
  do {                                            \
    if ((expr) != cudaSuccess) return EGTP_ERR_CUDA; \
  } while (0)

// Eq. 2 for `rows` rows, first part: the LM-head kernel leaves per-slot partials in the workspace.
// Fewer hidden rows than this are first copied into a zero-padded buffer of this many rows.  Every SM reads the
// same few hidden rows for every k block; with fewer than 16 rows (of 8 KB) those reads fall on too few L2 slices
// at a time: measured at d = 4096, V = 151936, 1 to 12 rows took 227-258 us per step against 206 us for 16 to 128
// rows, and the same 1 to 8 rows padded to 16 with zeros take 206 us.
constexpr int kMinLmheadRows = 16;

// With fuse_W1 != NULL (bf16 only) the m_h rows of that matrix ride along as extra output columns and
// head_g [plan.rows_pad][plan.head_cols_pad] receives W1 hidden[i] for every row.
// head_g must then have room for g_rows x g_ld floats: a plan that needs more is refused before anything is launched.
int run_lmhead(egtp_ctx* c, const egtp_lm_head* lm, const void* hidden, int64_t ldh, int64_t rows, int32_t* status,
               cudaStream_t stream, LmheadPlan* plan_out, const void* fuse_W1 = nullptr, int fuse_m_h = 0,
               float* head_g = nullptr, int64_t g_rows = 0, int64_t g_ld = 0) {
  const bool fuse = fuse_W1 != nullptr;
  if (rows < kMinLmheadRows) {
    const int64_t row_bytes = static_cast<int64_t>(lm->d) * elem_bytes(lm->dtype);
    {
      LaunchScope ls(c, EGTP_K_STAGE_ROWS, stream);
      EGTP_CUDA_TRY(launch_pad_rows(hidden, ldh * elem_bytes(lm->dtype), static_cast<int>(rows), row_bytes, c->small_rows,
                                    kMinLmheadRows, status, stream));
    }
    hidden = c->small_rows;
    ldh = lm->d;
    rows = kMinLmheadRows;      // the padding rows get entropies too (ln V); nothing downstream reads them
  }
  const LmheadPlan plan = make_lmhead_plan(rows, lm->d, lm->V, elem_bytes(lm->dtype), c->num_sms, c->slot_row_capacity,
                                           c->lmhead_mode, fuse ? fuse_m_h : 0, c->lmhead_chunks, c->pair_workers);
  if (plan.rows_pad * plan.slots > c->slot_row_capacity) return EGTP_ERR_CAPACITY;
  if (fuse && (plan.rows_pad > g_rows || plan.head_cols_pad > g_ld)) return EGTP_ERR_CAPACITY;
  CUtensorMap map_a, map_b, map_b_tile, map_c, map_c_tile;
  LmheadMaps maps;
  int rc = make_tensor_map(c, &map_a, hidden, lm->dtype, rows, lm->d, ldh, plan.a_box_rows);
  if (rc != EGTP_OK) return rc;
  rc = make_tensor_map(c, &map_b, lm->W, lm->dtype, lm->V, lm->d, lm->ldw, plan.b_box_rows);
  if (rc != EGTP_OK) return rc;
  maps.hidden = &map_a;
  maps.w = maps.w_tile = &map_b;
  const bool pair = plan.variant >= 4;
  if (!pair && plan.b_box_rows != plan.tile_cols) {
    rc = make_tensor_map(c, &map_b_tile, lm->W, lm->dtype, lm->V, lm->d, lm->ldw, plan.tile_cols);
    if (rc != EGTP_OK) return rc;
    maps.w_tile = &map_b_tile;
  }
  if (fuse) {
    rc = make_tensor_map(c, &map_c, fuse_W1, lm->dtype, fuse_m_h, lm->d, lm->d, plan.b_box_rows);
    if (rc != EGTP_OK) return rc;
    maps.w1 = maps.w1_tile = &map_c;
    if (!pair && plan.b_box_rows != plan.tile_cols) {
      rc = make_tensor_map(c, &map_c_tile, fuse_W1, lm->dtype, fuse_m_h, lm->d, lm->d, plan.tile_cols);
      if (rc != EGTP_OK) return rc;
      maps.w1_tile = &map_c_tile;
    }
  }
  LaunchScope ls(c, EGTP_K_LMHEAD_ENTROPY, stream);
  // (per-kernel event timing would charge an overlapped start to the kernel before)
  EGTP_CUDA_TRY(launch_lmhead_entropy(plan, lm->dtype == EGTP_F32, maps, rows, lm->V, c->partials, status, stream,
                                      head_g, /*overlap_previous=*/c->launch_overlap && !c->profiling));
  *plan_out = plan;
  return EGTP_OK;
}

// Layer 1 of the head on the tensor cores: possible when the weights are bf16 and the rows fit the context's
// [hi | lo] staging buffer.  The fp32 input rows are split into two bf16 halves (16 significant bits together),
// the LM-head kernel multiplies [x_hi | x_lo] against W1 twice over (head columns only, K split over the SMs) and
// head_out adds the slices up.
bool head_on_tensor_cores(const egtp_ctx* c, const egtp_head* head, int rows) {
  return head->wdtype == EGTP_BF16 && head->d % 64 == 0 && head->d <= c->max_d && rows <= c->max_batch &&
         reinterpret_cast<uintptr_t>(head->W1) % 16 == 0;
}

// W1 x for rows already staged in c->zcat as [hi | lo] halves: slices [plan.k_splits][rows_pad][head_cols_pad] in
// c->head_partial
int run_projection_staged(egtp_ctx* c, const egtp_head* head, int rows, int32_t* status, cudaStream_t stream,
                          LmheadPlan* plan_out) {
  const HeadArgs ha = head_args(head);
  const int64_t rows_pad = (static_cast<int64_t>(rows) + kTileM - 1) / kTileM * kTileM;
  const int64_t cols_pad = (static_cast<int64_t>(ha.m_h) + 255) / 256 * 256;
  const int max_splits = static_cast<int>(std::min<int64_t>(8, c->head_partial_floats / (rows_pad * cols_pad)));
  if (max_splits < 1) return EGTP_ERR_CAPACITY;
  const LmheadPlan plan = make_headproj_plan(rows, ha.d, ha.m_h, 2, c->num_sms, max_splits, /*a_repeats=*/2);
  CUtensorMap map_a, map_c;
  int rc = make_tensor_map(c, &map_a, c->zcat, EGTP_BF16, rows, 2 * ha.d, 2 * static_cast<int64_t>(ha.d), plan.a_box_rows);
  if (rc != EGTP_OK) return rc;
  rc = make_tensor_map(c, &map_c, ha.W1, EGTP_BF16, ha.m_h, ha.d, ha.d, plan.b_box_rows);
  if (rc != EGTP_OK) return rc;
  LmheadMaps maps;
  maps.hidden = &map_a;
  maps.w = maps.w_tile = maps.w1 = maps.w1_tile = &map_c;
  LaunchScope ls(c, EGTP_K_HEAD_HIDDEN, stream);
  EGTP_CUDA_TRY(launch_lmhead_entropy(plan, false, maps, rows, 0, nullptr, status, stream, c->head_partial));
  *plan_out = plan;
  return EGTP_OK;
}

// y = head(x) for rows already staged in c->zcat
int run_head_staged(egtp_ctx* c, const egtp_head* head, int rows, float* y, float* phat, int32_t* status,
                    cudaStream_t stream) {
  LmheadPlan plan;
  int rc = run_projection_staged(c, head, rows, status, stream, &plan);
  if (rc != EGTP_OK) return rc;
  LaunchScope ls(c, EGTP_K_HEAD_OUT, stream);
  EGTP_CUDA_TRY(launch_head_out(head_args(head), c->head_partial, rows, plan.k_splits, y, phat, status, stream,
                                plan.rows_pad * static_cast<int64_t>(plan.head_cols_pad), plan.head_cols_pad));
  return EGTP_OK;
}

int run_head(egtp_ctx* c, const egtp_head* head, const float* z, int64_t ldz, int rows, float* y, float* phat,
             int32_t* status, cudaStream_t stream) {
  if (head_on_tensor_cores(c, head, rows) && ldz % 4 == 0 && reinterpret_cast<uintptr_t>(z) % 16 == 0) {
    {
      LaunchScope ls(c, EGTP_K_HEAD_HIDDEN, stream);
      EGTP_CUDA_TRY(launch_split_hi_lo(z, ldz, rows, head->d, c->zcat, status, stream));
    }
    return run_head_staged(c, head, rows, y, phat, status, stream);
  }
  // fp32 weights or odd sizes: layer 1 on the CUDA cores
  const HeadArgs ha = head_args(head);
  const int splits = head_pick_splits(rows, ha.d, ha.m_h, c->num_sms, c->head_partial_floats);
  if (splits <= 0) return EGTP_ERR_CAPACITY;
  {
    LaunchScope ls(c, EGTP_K_HEAD_HIDDEN, stream);
    EGTP_CUDA_TRY(launch_head_hidden(ha, z, ldz, rows, splits, c->head_partial, status, stream));
  }
  {
    LaunchScope ls(c, EGTP_K_HEAD_OUT, stream);
    EGTP_CUDA_TRY(launch_head_out(ha, c->head_partial, rows, splits, y, phat, status, stream));
  }
  return EGTP_OK;
}

// Eq. 2 from logits in memory: per-(row, split) partials into the workspace.
// H_out != NULL: the same launch also merges them into H_out[rows].
int run_logits_entropy(egtp_ctx* c, const void* logits, int64_t ldl, int dtype, int64_t rows, int V, int32_t* status,
                       cudaStream_t stream, int* slots_out, float* H_out = nullptr) {
  if (!logits || V <= 0 || ldl < V) return EGTP_ERR_INVALID_ARG;
  if (dtype != EGTP_F32 && dtype != EGTP_BF16) return EGTP_ERR_UNSUPPORTED;
  if ((ldl * elem_bytes(dtype)) % 16 != 0 || reinterpret_cast<uintptr_t>(logits) % 16 != 0) return EGTP_ERR_UNSUPPORTED;
  if (rows > std::max<int64_t>(c->max_tokens, c->max_batch)) return EGTP_ERR_CAPACITY;
  int splits = logits_entropy_pick_splits(rows, V, c->num_sms);
  while (splits > 1 && rows * splits > c->slot_row_capacity) --splits;
  if (rows * splits > c->slot_row_capacity) return EGTP_ERR_CAPACITY;
  LaunchScope ls(c, EGTP_K_LOGITS_ENTROPY, stream);
  EGTP_CUDA_TRY(launch_logits_entropy(logits, ldl, dtype == EGTP_BF16, rows, V, splits, c->partials, H_out, c->arrivals,
                                      status, stream));
  *slots_out = splits;
  return EGTP_OK;
}

int check_plp_common(const egtp_ctx* c, const plp_state* st, const egtp_head* head, const float* src_m,
                     const float* src_s, const float* src_pooled, int n_src, int B_live, float alpha,
                     const float* yrem_out) {
  if (B_live < 0 || n_src < 0 || !(alpha > 0.f) || !std::isfinite(alpha)) return EGTP_ERR_INVALID_ARG;
  if (n_src > 0 && (!src_m || !src_s || !src_pooled)) return EGTP_ERR_INVALID_ARG;
  if (!head && yrem_out) return EGTP_ERR_INVALID_ARG;
  if (B_live > c->max_batch || B_live > st->num_slots || st->d > c->max_d) return EGTP_ERR_CAPACITY;
  return EGTP_OK;
}

// out[r] = W1 x[r] for rows of fp32 vectors x (layer 1 of the head without bias and ReLU), in row chunks that fit
// the split-K workspace.
int project_rows(egtp_ctx* c, const egtp_head* head, const float* x, int64_t ldx, int rows, float* out, int64_t ld_out,
                 int32_t* status, cudaStream_t stream) {
  const HeadArgs ha = head_args(head);
  if (head_on_tensor_cores(c, head, 1) && ldx % 4 == 0 && reinterpret_cast<uintptr_t>(x) % 16 == 0) {
    // tensor cores, max_batch rows at a time through the [hi | lo] staging buffer
    for (int r0 = 0; r0 < rows; r0 += c->max_batch) {
      const int n = std::min<int>(c->max_batch, rows - r0);
      {
        LaunchScope ls(c, EGTP_K_HEAD_HIDDEN, stream);
        EGTP_CUDA_TRY(launch_split_hi_lo(x + static_cast<int64_t>(r0) * ldx, ldx, n, ha.d, c->zcat, status, stream));
      }
      LmheadPlan plan;
      int rc = run_projection_staged(c, head, n, status, stream, &plan);
      if (rc != EGTP_OK) return rc;
      LaunchScope ls(c, EGTP_K_HEAD_OUT, stream);
      EGTP_CUDA_TRY(launch_head_partial_sum(c->head_partial, n, plan.k_splits, ha.m_h, out + static_cast<int64_t>(r0) * ld_out,
                                            ld_out, status, stream,
                                            plan.rows_pad * static_cast<int64_t>(plan.head_cols_pad), plan.head_cols_pad));
    }
    return EGTP_OK;
  }
  const int chunk = static_cast<int>(std::max<int64_t>(1, std::min<int64_t>(rows, c->head_partial_floats / ha.m_h)));
  for (int r0 = 0; r0 < rows; r0 += chunk) {
    const int n = std::min(chunk, rows - r0);
    const int splits = head_pick_splits(n, ha.d, ha.m_h, c->num_sms, c->head_partial_floats);
    if (splits <= 0) return EGTP_ERR_CAPACITY;
    {
      LaunchScope ls(c, EGTP_K_HEAD_HIDDEN, stream);
      EGTP_CUDA_TRY(launch_head_hidden(ha, x + static_cast<int64_t>(r0) * ldx, ldx, n, splits, c->head_partial, status, stream));
    }
    {
      LaunchScope ls(c, EGTP_K_HEAD_OUT, stream);
      EGTP_CUDA_TRY(launch_head_partial_sum(c->head_partial, n, splits, ha.m_h, out + static_cast<int64_t>(r0) * ld_out, ld_out, status, stream));
    }
  }
  return EGTP_OK;
}

// True when this step can take the route of a state bound to `head`: the LM-head kernel also produces W1 h'.
bool plp_fused_route(const egtp_ctx* c, const plp_state* st, int hidden_dtype, const egtp_head* head,
                     int B_live, int n_src, const float* yrem_out) {
  if (!st->bound || !head || !yrem_out) return false;
  const egtp_head& b = st->bound_head;
  if (head->W1 != b.W1 || head->m_h != b.m_h || head->d != b.d || head->wdtype != b.wdtype) return false;
  if (hidden_dtype != EGTP_BF16 || head->wdtype != EGTP_BF16) return false;
  if (n_src > c->max_batch) return false;
  const int64_t rows_pad = B_live <= 2 * kTileM ? (B_live <= kTileM ? kTileM : 2 * kTileM)
                                                : (static_cast<int64_t>(B_live) + kTileM - 1) / kTileM * kTileM;
  return rows_pad <= st->g_rows;
}

// --- steps on a state bound to its head whose entropies do not come from an LM-head launch -----------------------
bool plp_bound_tail_route(const egtp_ctx* c, const plp_state* st, int hidden_dtype, const egtp_head* head, int B_live,
                          int n_src, const float* yrem_out, const void* hidden_step, int64_t ldh) {
  return plp_fused_route(c, st, hidden_dtype, head, B_live, n_src, yrem_out) &&
         reinterpret_cast<uintptr_t>(hidden_step) % 16 == 0 && (ldh * 2) % 16 == 0;
}

// P = W1 acc if it is stale, and W1 src_pooled for rows that restart from EGTP rows
int plp_bound_prepare(egtp_ctx* c, plp_state* st, const egtp_head* head, const int32_t* reset_src,
                      const float* src_pooled, int n_src, int32_t* status, cudaStream_t stream) {
  if (!st->proj_valid) {
    int rc = project_rows(c, head, st->acc, st->d, st->num_slots, st->proj, head->m_h, status, stream);
    if (rc != EGTP_OK) return rc;
    st->proj_valid = true;
  }
  if (reset_src && n_src > 0) {
    int rc = project_rows(c, head, src_pooled, st->d, n_src, st->src_proj, head->m_h, status, stream);
    if (rc != EGTP_OK) return rc;
  }
  return EGTP_OK;
}

// W1 h' for the step's rows: the LM-head kernel over the head columns alone, K split over the SMs, into the
// slices of st->head_g.  Independent of the step's entropies, so it may run on another stream next to them.
int plp_bound_project(egtp_ctx* c, plp_state* st, const egtp_head* head, const void* hidden_step, int64_t ldh,
                      int B_live, int32_t* status, cudaStream_t stream, LmheadPlan* plan_out) {
  const LmheadPlan plan = make_headproj_plan(B_live, st->d, head->m_h, 2, c->num_sms, st->g_max_splits);
  if (plan.rows_pad > st->g_rows || plan.head_cols_pad > st->ldg_max) return EGTP_ERR_CAPACITY;
  CUtensorMap map_a, map_c;
  int rc = make_tensor_map(c, &map_a, hidden_step, EGTP_BF16, B_live, st->d, ldh, plan.a_box_rows);
  if (rc != EGTP_OK) return rc;
  rc = make_tensor_map(c, &map_c, head->W1, EGTP_BF16, head->m_h, st->d, st->d, plan.b_box_rows);
  if (rc != EGTP_OK) return rc;
  LmheadMaps maps;
  maps.hidden = &map_a;
  maps.w = maps.w_tile = maps.w1 = maps.w1_tile = &map_c;
  LaunchScope ls(c, EGTP_K_HEAD_HIDDEN, stream);
  EGTP_CUDA_TRY(launch_lmhead_entropy(plan, false, maps, B_live, 0, nullptr, status, stream, st->head_g));
  *plan_out = plan;
  return EGTP_OK;
}

// Second half of a PLP step: merge the entropy partials, update the slots (Eq. 8), run the head.
// projected != NULL: the caller has already taken the bound route's first two steps (plp_bound_prepare,
// plp_bound_project with this plan) and ordered them before `stream`'s next work.
int plp_update_and_head(egtp_ctx* c, plp_state* st, const egtp_head* head, const void* hidden_step, int64_t ldh,
                        int hidden_dtype, const float* partials, int slots, int64_t row_stride, int64_t slot_stride,
                        const int32_t* slot_ids, const int32_t* reset_src,
                        const float* src_m, const float* src_s, const float* src_pooled, int n_src, int B_live,
                        float alpha, float* Hstep_out, float* z_out, float* yrem_out, int32_t* status,
                        cudaStream_t stream, const LmheadPlan* projected = nullptr) {
  if (projected != nullptr || plp_bound_tail_route(c, st, hidden_dtype, head, B_live, n_src, yrem_out, hidden_step, ldh)) {
    LmheadPlan plan;
    if (projected != nullptr) {
      plan = *projected;
    } else {
      int rc = plp_bound_prepare(c, st, head, reset_src, src_pooled, n_src, status, stream);
      if (rc != EGTP_OK) return rc;
      rc = plp_bound_project(c, st, head, hidden_step, ldh, B_live, status, stream, &plan);
      if (rc != EGTP_OK) return rc;
    }
    LaunchScope ls(c, EGTP_K_PLP_UPDATE, stream);
    EGTP_CUDA_TRY(launch_plp_update_bound(hidden_step, ldh, partials, slots, row_stride, slot_stride, Hstep_out, slot_ids,
                                          reset_src, src_m, src_s, src_pooled, st->src_proj, n_src, B_live, st->d,
                                          st->num_slots, 1.f / alpha, st->m, st->s, st->acc, st->proj, z_out, st->d,
                                          st->head_g, plan.head_cols_pad, plan.k_splits,
                                          plan.rows_pad * static_cast<int64_t>(plan.head_cols_pad), head_args(head),
                                          yrem_out, st->owner, st->epoch, status, stream, /*overlap_previous=*/false));
    return EGTP_OK;
  }
  st->proj_valid = false;   // acc moves on without the projection a bound state keeps
  const bool want_head = head && yrem_out;
  // with the head's first layer on the tensor cores the update writes z straight into the [hi | lo] staging
  // buffer (and as fp32 only if the caller asked for z)
  const bool staged = want_head && head_on_tensor_cores(c, head, B_live);
  float* z = z_out ? z_out : (staged ? nullptr : c->pooled);
  {
    LaunchScope ls(c, EGTP_K_PLP_UPDATE, stream);
    EGTP_CUDA_TRY(launch_plp_update(hidden_step, ldh, hidden_dtype == EGTP_BF16, partials, slots, row_stride, slot_stride, Hstep_out,
                                    slot_ids,
                                    reset_src, src_m, src_s, src_pooled, n_src, B_live, st->d, st->num_slots,
                                    1.f / alpha, st->m, st->s, st->acc, z, st->d, st->owner, st->epoch, status, stream,
                                    staged ? c->zcat : nullptr));
  }
  if (staged) return run_head_staged(c, head, B_live, yrem_out, nullptr, status, stream);
  if (want_head) return run_head(c, head, z, st->d, B_live, yrem_out, nullptr, status, stream);
  return EGTP_OK;
}

// The whole EGTP chain.  With pieces > 1 the LM-head phase runs over the row ranges [piece_begin[p], piece_begin[p+1])
// of the batch one after the other (boundaries on multiples of 256 rows), each waiting for its own event (the host
// entry point records one when that range's copy has landed), so that the copy of range i+1 overlaps the GEMM of range i.
int predict_impl(egtp_ctx* c, const egtp_lm_head* lm, const egtp_head* head, const void* hidden, int64_t ldh,
                 const int32_t* offsets, int32_t B, int64_t T_total, float alpha, float* H_out, float* weights_out,
                 int32_t* seg_id_out, float* pooled_out, float* state_m_out, float* state_s_out, float* yhat_out,
                 float* phat_out, int32_t* status_dev, void* stream_v, int pieces, const int64_t* piece_begin,
                 const cudaEvent_t* piece_ready) {
  if (!c) return EGTP_ERR_INVALID_ARG;
  if (B < 0 || T_total < 0 || !(alpha > 0.f) || !std::isfinite(alpha)) return EGTP_ERR_INVALID_ARG;
  if (B == 0 && T_total == 0) return EGTP_OK;
  if (!offsets && B > 0) return EGTP_ERR_INVALID_ARG;
  if (!head && (yhat_out || phat_out)) return EGTP_ERR_INVALID_ARG;
  if (T_total > c->max_tokens || B > c->max_batch) return EGTP_ERR_CAPACITY;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  int32_t* status = status_dev ? status_dev : c->status;
  if (T_total > 0) {
    int rc = check_lm(c, lm, hidden, ldh);
    if (rc != EGTP_OK) return rc;
  } else if (!lm || lm->d <= 0 || lm->d > c->max_d) {
    return EGTP_ERR_INVALID_ARG;
  }
  if (head) {
    int rc = check_head(c, head, lm->d);
    if (rc != EGTP_OK) return rc;
  }
  if (cudaSetDevice(c->device) != cudaSuccess) return EGTP_ERR_CUDA;
  if (!status_dev) EGTP_CUDA_TRY(cudaMemsetAsync(c->status, 0, sizeof(int32_t), stream));

  const int d = lm->d;
  float* H = H_out ? H_out : c->H;
  float* pooled = pooled_out ? pooled_out : c->pooled;
  float* seg_m = state_m_out ? state_m_out : c->seg_m;
  float* seg_s = state_s_out ? state_s_out : c->seg_s;
  const bool want_head = head && (yhat_out || phat_out);
  // bf16 head weights: layer 1 runs on the tensor cores and the pooling writes its [hi | lo] input directly
  const bool staged = want_head && head_on_tensor_cores(c, head, B);

  if (B > 0 && T_total == 0) {      // only empty prompts can be valid; no merge launch will check the offsets
    LaunchScope ls(c, EGTP_K_VALIDATE, stream);
    EGTP_CUDA_TRY(launch_validate_offsets(offsets, B, T_total, status, stream));
  }
  for (int p = 0; p < pieces && T_total > 0; ++p) {
    const int64_t r0 = piece_begin ? piece_begin[p] : 0;
    const int64_t rows = (piece_begin ? piece_begin[p + 1] : T_total) - r0;
    if (rows <= 0) continue;
    if (piece_ready) EGTP_CUDA_TRY(cudaStreamWaitEvent(stream, piece_ready[p], 0));
    const char* piece_ptr = static_cast<const char*>(hidden) + r0 * ldh * elem_bytes(lm->dtype);
    LmheadPlan plan;
    int rc = run_lmhead(c, lm, piece_ptr, ldh, rows, status, stream, &plan);
    if (rc != EGTP_OK) return rc;
    // the first merge launch also checks the offsets (everything that indexes tokens through them comes later);
    // every merge launch prepares the pooling of its tokens (unnormalised Eq. 3 weights per 64-token chunk)
    const PoolPrep prep{1.f / alpha, c->weights, c->piece_ms,
                        (T_total + kPoolChunkTokens - 1) / kPoolChunkTokens, seg_m, seg_s};
    LaunchScope ls(c, EGTP_K_ENTROPY_MERGE, stream);
    EGTP_CUDA_TRY(launch_entropy_merge(c->partials, plan.slots, plan.slots * 3, 3, rows, r0, H, offsets, B, seg_id_out,
                                       (p == 0 && B > 0) ? T_total : -1, status, stream, B > 0 ? &prep : nullptr));
  }
  if (B == 0) return EGTP_OK;
  if (T_total > 0) {
    LaunchScope ls(c, EGTP_K_POOL, stream);
    EGTP_CUDA_TRY(launch_pool(hidden, ldh, lm->dtype == EGTP_BF16, 0, c->weights, offsets, B, T_total, d, pooled,
                              c->piece_a, c->piece_b, c->piece_ms, seg_m, seg_s, status, stream));
  }
  {
    LaunchScope ls(c, EGTP_K_POOL_COMBINE, stream);
    EGTP_CUDA_TRY(launch_pool_combine(offsets, B, T_total, d, 0, c->piece_a, c->piece_b, c->piece_ms, pooled, seg_m, seg_s,
                                      staged ? c->zcat : nullptr, status, stream));
  }
  if (weights_out) {
    LaunchScope ls(c, EGTP_K_TOKEN_WEIGHTS, stream);
    EGTP_CUDA_TRY(launch_token_weights(H, offsets, B, T_total, 1.f / alpha, seg_m, seg_s, weights_out, status, stream));
  }
  if (staged) return run_head_staged(c, head, B, yhat_out, phat_out, status, stream);
  if (want_head) return run_head(c, head, pooled, d, B, yhat_out, phat_out, status, stream);
  return EGTP_OK;
}


}  // namespace

extern "C" {

const char* egtp_status_string(int status) {
  switch (status) {
    case EGTP_OK: return "ok";
    case EGTP_ERR_INVALID_ARG: return "invalid argument";
    case EGTP_ERR_UNSUPPORTED: return "unsupported dtype, alignment or layout";
    case EGTP_ERR_CAPACITY: return "exceeds the capacity the context or state was created with";
    case EGTP_ERR_CUDA: return "CUDA call failed";
    case EGTP_ERR_BAD_OFFSETS: return "offsets are not non-decreasing within [0, T_total]";
    case EGTP_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel ran out";
    case EGTP_ERR_BAD_SLOT: return "slot id or reset source out of range";
    default: return "unknown status";
  }
}

const char* egtp_kernel_name(int kernel_id) {
  if (kernel_id < 0 || kernel_id >= EGTP_NUM_KERNELS) return "unknown";
  return kKernelNames[kernel_id];
}

int egtp_create(egtp_ctx** out, int device, int64_t max_tokens, int32_t max_batch, int32_t max_d, int32_t max_V) {
  return egtp_create_ex(out, device, max_tokens, max_batch, max_d, max_V, 0);
}

int egtp_create_ex(egtp_ctx** out, int device, int64_t max_tokens, int32_t max_batch, int32_t max_d, int32_t max_V,
                   int32_t flags) {
  if (!out || max_tokens <= 0 || max_batch <= 0 || max_d <= 0 || max_V <= 0) return EGTP_ERR_INVALID_ARG;
  if ((flags & ~EGTP_CREATE_NO_HOST_STAGING) != 0) return EGTP_ERR_INVALID_ARG;
  if (max_tokens >= (1ll << 31)) return EGTP_ERR_UNSUPPORTED;   // offsets are int32 token indices
  if (cudaSetDevice(device) != cudaSuccess) return EGTP_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return EGTP_ERR_CUDA;
  if (prop.major != 10) return EGTP_ERR_UNSUPPORTED;
  egtp_ctx* c = new (std::nothrow) egtp_ctx();
  if (!c) return EGTP_ERR_CUDA;
  c->device = device;
  c->num_sms = prop.multiProcessorCount;
  c->max_tokens = max_tokens; c->max_batch = max_batch; c->max_d = max_d; c->max_V = max_V;

  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || fn == nullptr) {
    delete c;
    return EGTP_ERR_CUDA;
  }
  c->encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
  if (lmhead_prepare_device(&c->pair_workers) != cudaSuccess) { delete c; return EGTP_ERR_CUDA; }

  const int64_t rows_cap = std::max<int64_t>(max_tokens, max_batch);
  const int64_t rows_pad = (rows_cap + kTileM - 1) / kTileM * kTileM;
  // room for 24 vocabulary chunks (two partial slots each) at the largest token count, for one chunk per SM
  // on decode-sized batches, and never less than 2 M slot rows (24 MB): batches of a few dozen row blocks need
  // 30 to 60 chunks before (row blocks x chunks) fills whole rounds of the SMs
  c->slot_row_capacity = std::max<int64_t>(
      std::max<int64_t>(rows_pad * 24 * kEpiSplit, static_cast<int64_t>(2 * kTileM) * c->num_sms * kEpiSplit),
      int64_t{1} << 21);
  const int64_t pool_chunks = (max_tokens + kPoolChunkTokens - 1) / kPoolChunkTokens + 1;
  c->head_partial_floats = std::max<int64_t>(8ll << 20, static_cast<int64_t>(max_batch) * 8192);

  bool ok = true;
  ok = ok && dev_alloc(c, &c->partials, c->slot_row_capacity * 3) == cudaSuccess;
  ok = ok && dev_alloc(c, &c->H, rows_cap) == cudaSuccess;
  ok = ok && dev_alloc(c, &c->arrivals, rows_cap) == cudaSuccess;
  ok = ok && cudaMemset(c->arrivals, 0, sizeof(int32_t) * static_cast<size_t>(rows_cap)) == cudaSuccess;
  ok = ok && dev_alloc(c, &c->weights, max_tokens) == cudaSuccess;
  ok = ok && dev_alloc(c, &c->seg_m, max_batch) == cudaSuccess;
  ok = ok && dev_alloc(c, &c->seg_s, max_batch) == cudaSuccess;
  ok = ok && dev_alloc(c, &c->pooled, static_cast<int64_t>(max_batch) * max_d) == cudaSuccess;
  ok = ok && dev_alloc(c, &c->piece_a, pool_chunks * max_d) == cudaSuccess;
  ok = ok && dev_alloc(c, &c->piece_b, pool_chunks * max_d) == cudaSuccess;
  ok = ok && dev_alloc(c, &c->piece_ms, pool_chunks * 4) == cudaSuccess;
  ok = ok && dev_alloc(c, &c->head_partial, c->head_partial_floats) == cudaSuccess;
  ok = ok && dev_alloc(c, reinterpret_cast<float**>(&c->small_rows), static_cast<int64_t>(kMinLmheadRows) * max_d) == cudaSuccess;
  ok = ok && dev_alloc(c, reinterpret_cast<float**>(&c->zcat), static_cast<int64_t>(max_batch) * max_d) == cudaSuccess;
  ok = ok && dev_alloc(c, &c->yhat, max_batch) == cudaSuccess;
  ok = ok && dev_alloc(c, &c->status, 1) == cudaSuccess;
  // staging for the hidden states of the *_host entry points: the largest single buffer of the context
  // (rows x max_d x 4 bytes), left out on request
  c->host_staging = (flags & EGTP_CREATE_NO_HOST_STAGING) == 0;
  if (c->host_staging)
    ok = ok && dev_alloc(c, reinterpret_cast<float**>(&c->hidden_stage), rows_cap * max_d) == cudaSuccess;
  ok = ok && dev_alloc(c, &c->offsets_stage, static_cast<int64_t>(max_batch) + 1) == cudaSuccess;
  ok = ok && dev_alloc(c, &c->reset_stage, 2 * static_cast<int64_t>(max_batch)) == cudaSuccess;
  c->stage_bytes = c->host_staging ? rows_cap * static_cast<int64_t>(max_d) * 4 : 0;
  ok = ok && cudaMemset(c->status, 0, sizeof(int32_t)) == cudaSuccess;
  ok = ok && cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking) == cudaSuccess;
  for (auto& e : c->piece_ready) ok = ok && cudaEventCreateWithFlags(&e, cudaEventDisableTiming) == cudaSuccess;
  ok = ok && cudaEventCreateWithFlags(&c->stage_free, cudaEventDisableTiming) == cudaSuccess;
  for (auto& e : c->host_in_ready) ok = ok && cudaEventCreateWithFlags(&e, cudaEventDisableTiming) == cudaSuccess;
  for (auto& e : c->host_stage_free) ok = ok && cudaEventCreateWithFlags(&e, cudaEventDisableTiming) == cudaSuccess;
  ok = ok && cudaEventCreateWithFlags(&c->fork_ev, cudaEventDisableTiming) == cudaSuccess;
  ok = ok && cudaEventCreateWithFlags(&c->join_ev, cudaEventDisableTiming) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    free_ctx_memory(c);
    delete c;
    return EGTP_ERR_CUDA;
  }
  *out = c;
  return EGTP_OK;
}

int egtp_destroy(egtp_ctx* c) {
  if (!c) return EGTP_ERR_INVALID_ARG;
  cudaSetDevice(c->device);
  free_ctx_memory(c);
  delete c;
  return EGTP_OK;
}

int64_t egtp_workspace_bytes(const egtp_ctx* c) { return c ? c->bytes : 0; }
int64_t egtp_launch_count(const egtp_ctx* c) { return c ? c->launches : 0; }

int egtp_lmhead_plan(const egtp_ctx* c, int64_t T, int32_t d, int32_t V, int32_t dtype, int32_t info[8]) {
  if (!c || !info || T <= 0 || d <= 0 || V <= 0) return EGTP_ERR_INVALID_ARG;
  const LmheadPlan p = make_lmhead_plan(T, d, V, elem_bytes(dtype), c->num_sms, c->slot_row_capacity, c->lmhead_mode, 0, c->lmhead_chunks, c->pair_workers);
  info[0] = p.grid; info[1] = p.row_blocks; info[2] = p.rows_per_block; info[3] = p.chunks;
  info[4] = p.slots; info[5] = p.tile_cols; info[6] = p.k_blocks; info[7] = p.smem_bytes;
  return EGTP_OK;
}

int egtp_lmhead_plan_for(int32_t num_sms, int32_t pair_workers, int64_t T, int32_t d, int32_t V, int32_t dtype,
                         int32_t mode, int32_t head_cols, int32_t info[12]) {
  if (!info || num_sms <= 0 || pair_workers < 0 || T <= 0 || d <= 0 || V <= 0 || head_cols < 0) return EGTP_ERR_INVALID_ARG;
  if (dtype != EGTP_F32 && dtype != EGTP_BF16) return EGTP_ERR_UNSUPPORTED;
  if (mode < EGTP_LMHEAD_AUTO || mode > EGTP_LMHEAD_CTA_PAIRS_WIDE) return EGTP_ERR_INVALID_ARG;
  // the workspace rule of egtp_create for a context sized for exactly T rows
  const int64_t rows_pad = (T + kTileM - 1) / kTileM * kTileM;
  const int64_t capacity = std::max<int64_t>(
      std::max<int64_t>(rows_pad * 24 * kEpiSplit, static_cast<int64_t>(2 * kTileM) * num_sms * kEpiSplit), int64_t{1} << 21);
  const LmheadPlan p = make_lmhead_plan(T, d, V, elem_bytes(dtype), num_sms, capacity, mode, head_cols, 0, pair_workers);
  info[0] = p.grid; info[1] = p.row_blocks; info[2] = p.rows_per_block; info[3] = p.chunks;
  info[4] = p.slots; info[5] = p.tile_cols; info[6] = p.k_blocks; info[7] = p.smem_bytes;
  info[8] = p.variant; info[9] = p.group_rb; info[10] = p.col_gran; info[11] = p.n_groups;
  return EGTP_OK;
}

int egtp_set_lmhead_mode(egtp_ctx* c, int mode) {
  if (!c || mode < EGTP_LMHEAD_AUTO || mode > EGTP_LMHEAD_CTA_PAIRS_WIDE)
    return EGTP_ERR_INVALID_ARG;
  c->lmhead_mode = mode;
  return EGTP_OK;
}

int egtp_set_lmhead_chunks(egtp_ctx* c, int32_t chunks) {
  if (!c || chunks < 0) return EGTP_ERR_INVALID_ARG;
  c->lmhead_chunks = chunks;
  return EGTP_OK;
}

int egtp_set_launch_overlap(egtp_ctx* c, int on) {
  if (!c) return EGTP_ERR_INVALID_ARG;
  c->launch_overlap = on != 0;
  return EGTP_OK;
}

int egtp_selftest_wait_timeout(egtp_ctx* c, int32_t limit_ms, int32_t* status_dev, void* stream_v) {
  if (!c || !status_dev || limit_ms <= 0 || limit_ms > 1000) return EGTP_ERR_INVALID_ARG;
  if (cudaSetDevice(c->device) != cudaSuccess) return EGTP_ERR_CUDA;
  c->launches += 1;
  EGTP_CUDA_TRY(launch_wait_timeout_selftest(static_cast<uint64_t>(limit_ms) * 1000000ull, status_dev,
                                             static_cast<cudaStream_t>(stream_v)));
  return EGTP_OK;
}

int egtp_profile_enable(egtp_ctx* c, int on) {
  if (!c) return EGTP_ERR_INVALID_ARG;
  c->profiling = on != 0;
  return EGTP_OK;
}

int egtp_profile_read(egtp_ctx* c, double* ms_by_kernel, int64_t* launches_by_kernel) {
  if (!c) return EGTP_ERR_INVALID_ARG;
  if (cudaSetDevice(c->device) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) return EGTP_ERR_CUDA;
  for (auto& e : c->pending) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, e.start, e.stop) == cudaSuccess) {
      c->ms_acc[e.kernel] += ms;
      c->n_acc[e.kernel] += 1;
    }
    c->free_events.push_back(e);
  }
  c->pending.clear();
  for (int k = 0; k < EGTP_NUM_KERNELS; ++k) {
    if (ms_by_kernel) ms_by_kernel[k] = c->ms_acc[k];
    if (launches_by_kernel) launches_by_kernel[k] = c->n_acc[k];
    c->ms_acc[k] = 0.0;
    c->n_acc[k] = 0;
  }
  return EGTP_OK;
}

int egtp_predict(egtp_ctx* c, const egtp_lm_head* lm, const egtp_head* head, const void* hidden, int64_t ldh,
                 const int32_t* offsets, int32_t B, int64_t T_total, float alpha, float* H_out, float* weights_out,
                 int32_t* seg_id_out, float* pooled_out, float* state_m_out, float* state_s_out, float* yhat_out,
                 float* phat_out, int32_t* status_dev, void* stream_v) {
  return predict_impl(c, lm, head, hidden, ldh, offsets, B, T_total, alpha, H_out, weights_out, seg_id_out, pooled_out,
                      state_m_out, state_s_out, yhat_out, phat_out, status_dev, stream_v, 1, nullptr, nullptr);
}

int egtp_pool_baseline(egtp_ctx* c, const egtp_head* head, const void* hidden, int64_t ldh, int32_t dtype, int32_t d,
                       const int32_t* offsets, int32_t B, int64_t T_total, int32_t mode, float* pooled_out,
                       float* yhat_out, int32_t* status_dev, void* stream_v) {
  if (!c || !hidden || !offsets || B < 0 || T_total < 0 || d <= 0 || ldh < d) return EGTP_ERR_INVALID_ARG;
  if (mode != EGTP_POOL_MEAN && mode != EGTP_POOL_MAX && mode != EGTP_POOL_LAST) return EGTP_ERR_INVALID_ARG;
  if (!head && yhat_out) return EGTP_ERR_INVALID_ARG;
  if (dtype != EGTP_F32 && dtype != EGTP_BF16) return EGTP_ERR_UNSUPPORTED;
  if (d % 16 != 0 || (ldh * elem_bytes(dtype)) % 16 != 0 || reinterpret_cast<uintptr_t>(hidden) % 16 != 0)
    return EGTP_ERR_UNSUPPORTED;
  if (T_total > c->max_tokens || B > c->max_batch || d > c->max_d) return EGTP_ERR_CAPACITY;
  if (B == 0) return EGTP_OK;
  if (head) {
    int rc = check_head(c, head, d);
    if (rc != EGTP_OK) return rc;
  }
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  if (cudaSetDevice(c->device) != cudaSuccess) return EGTP_ERR_CUDA;
  int32_t* status = status_dev ? status_dev : c->status;
  if (!status_dev) EGTP_CUDA_TRY(cudaMemsetAsync(c->status, 0, sizeof(int32_t), stream));
  float* pooled = pooled_out ? pooled_out : c->pooled;
  const bool want_head = head && yhat_out;
  const bool staged = want_head && head_on_tensor_cores(c, head, B);
  {
    LaunchScope ls(c, EGTP_K_VALIDATE, stream);
    EGTP_CUDA_TRY(launch_validate_offsets(offsets, B, T_total, status, stream));
  }
  if (T_total > 0) {
    LaunchScope ls(c, EGTP_K_POOL, stream);
    EGTP_CUDA_TRY(launch_pool(hidden, ldh, dtype == EGTP_BF16, mode, nullptr, offsets, B, T_total, d, pooled,
                              c->piece_a, c->piece_b, c->piece_ms, nullptr, nullptr, status, stream));
  }
  {
    LaunchScope ls(c, EGTP_K_POOL_COMBINE, stream);
    EGTP_CUDA_TRY(launch_pool_combine(offsets, B, T_total, d, mode, c->piece_a, c->piece_b, c->piece_ms, pooled, nullptr,
                                      nullptr, staged ? c->zcat : nullptr, status, stream));
  }
  if (staged) return run_head_staged(c, head, B, yhat_out, nullptr, status, stream);
  if (want_head) return run_head(c, head, pooled, d, B, yhat_out, nullptr, status, stream);
  return EGTP_OK;
}

int egtp_predict_host(egtp_ctx* c, const egtp_lm_head* lm, const egtp_head* head, const void* hidden_host,
                      const int32_t* offsets_host, int32_t B, int64_t T_total, float alpha, float* yhat_host,
                      float* pooled_host, int32_t* status_host, void* stream_v) {
  if (!c || !lm || !head || !hidden_host || !offsets_host || !yhat_host || !status_host) return EGTP_ERR_INVALID_ARG;
  if (B <= 0 || T_total <= 0) return EGTP_ERR_INVALID_ARG;
  if (!c->host_staging) return EGTP_ERR_UNSUPPORTED;
  if (T_total > c->max_tokens || B > c->max_batch || lm->d > c->max_d) return EGTP_ERR_CAPACITY;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  if (cudaSetDevice(c->device) != cudaSuccess) return EGTP_ERR_CUDA;
  // The hidden states travel in up to four row ranges on the context's copy stream; the LM-head kernel of range i
  // starts when its copy has landed, while range i+1 is still on the bus.  A row is copied several times faster than
  // it is multiplied against the vocabulary, so the ranges grow fourfold from a small first one (512 rows: the only
  // copy nothing hides) and the last takes the rest: most rows run in one large, efficient launch.
  const int eb = elem_bytes(lm->dtype);
  int64_t piece_begin[egtp_ctx::kMaxPieces + 1] = {0};
  int pieces = 0;
  if (T_total < 4096) {
    piece_begin[++pieces] = T_total;
  } else {
    int64_t next = 512;
    while (pieces < egtp_ctx::kMaxPieces - 1 && piece_begin[pieces] + next + 1024 <= T_total) {
      piece_begin[pieces + 1] = piece_begin[pieces] + next;
      ++pieces;
      next *= 4;
    }
    piece_begin[++pieces] = T_total;
  }
  // the staging buffer may still be read by earlier work on `stream`
  EGTP_CUDA_TRY(cudaEventRecord(c->stage_free, stream));
  EGTP_CUDA_TRY(cudaStreamWaitEvent(c->copy_stream, c->stage_free, 0));
  for (int p = 0; p < pieces; ++p) {
    const int64_t r0 = piece_begin[p];
    const int64_t rows = piece_begin[p + 1] - r0;
    const size_t off_bytes = static_cast<size_t>(r0) * lm->d * eb;
    EGTP_CUDA_TRY(cudaMemcpyAsync(static_cast<char*>(c->hidden_stage) + off_bytes,
                                  static_cast<const char*>(hidden_host) + off_bytes,
                                  static_cast<size_t>(rows) * lm->d * eb, cudaMemcpyHostToDevice, c->copy_stream));
    EGTP_CUDA_TRY(cudaEventRecord(c->piece_ready[p], c->copy_stream));
  }
  EGTP_CUDA_TRY(cudaMemcpyAsync(c->offsets_stage, offsets_host, sizeof(int32_t) * (static_cast<size_t>(B) + 1),
                                cudaMemcpyHostToDevice, stream));
  int rc = predict_impl(c, lm, head, c->hidden_stage, lm->d, c->offsets_stage, B, T_total, alpha, nullptr, nullptr,
                        nullptr, nullptr, nullptr, nullptr, c->yhat, nullptr, nullptr, stream, pieces, piece_begin,
                        c->piece_ready);
  if (rc != EGTP_OK) {
    cudaStreamSynchronize(c->copy_stream);
    return rc;
  }
  EGTP_CUDA_TRY(cudaMemcpyAsync(yhat_host, c->yhat, sizeof(float) * B, cudaMemcpyDeviceToHost, stream));
  if (pooled_host)
    EGTP_CUDA_TRY(cudaMemcpyAsync(pooled_host, c->pooled, sizeof(float) * static_cast<size_t>(B) * lm->d,
                                  cudaMemcpyDeviceToHost, stream));
  EGTP_CUDA_TRY(cudaMemcpyAsync(status_host, c->status, sizeof(int32_t), cudaMemcpyDeviceToHost, stream));
  EGTP_CUDA_TRY(cudaStreamSynchronize(stream));
  return EGTP_OK;
}

int plp_state_create(egtp_ctx* c, plp_state** out, int32_t num_slots, int32_t d) {
  if (!c || !out || num_slots <= 0 || d <= 0) return EGTP_ERR_INVALID_ARG;
  if (d % 16 != 0) return EGTP_ERR_UNSUPPORTED;
  if (cudaSetDevice(c->device) != cudaSuccess) return EGTP_ERR_CUDA;
  plp_state* st = new (std::nothrow) plp_state();
  if (!st) return EGTP_ERR_CUDA;
  st->ctx = c; st->device = c->device; st->num_slots = num_slots; st->d = d;
  bool ok = cudaMalloc(reinterpret_cast<void**>(&st->m), sizeof(float) * num_slots) == cudaSuccess;
  ok = ok && cudaMalloc(reinterpret_cast<void**>(&st->s), sizeof(float) * num_slots) == cudaSuccess;
  ok = ok && cudaMalloc(reinterpret_cast<void**>(&st->acc), sizeof(float) * static_cast<size_t>(num_slots) * d) == cudaSuccess;
  ok = ok && cudaMalloc(reinterpret_cast<void**>(&st->owner), sizeof(int32_t) * num_slots) == cudaSuccess;
  ok = ok && cudaMalloc(reinterpret_cast<void**>(&st->epoch), sizeof(int32_t) * 2) == cudaSuccess;
  if (ok) {
    const int32_t epoch0[2] = {1, 0};
    ok = cudaMemset(st->owner, 0, sizeof(int32_t) * num_slots) == cudaSuccess &&
         cudaMemcpy(st->epoch, epoch0, sizeof(epoch0), cudaMemcpyHostToDevice) == cudaSuccess;
  }
  if (ok) {
    std::vector<float> neg(num_slots, -INFINITY);
    ok = cudaMemcpy(st->m, neg.data(), sizeof(float) * num_slots, cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && cudaMemset(st->s, 0, sizeof(float) * num_slots) == cudaSuccess;
    ok = ok && cudaMemset(st->acc, 0, sizeof(float) * static_cast<size_t>(num_slots) * d) == cudaSuccess;
  }
  if (!ok) {
    cudaGetLastError();
    cudaFree(st->m); cudaFree(st->s); cudaFree(st->acc); cudaFree(st->owner); cudaFree(st->epoch);
    delete st;
    return EGTP_ERR_CUDA;
  }
  *out = st;
  return EGTP_OK;
}

int plp_state_destroy(plp_state* st) {
  if (!st) return EGTP_ERR_INVALID_ARG;
  cudaSetDevice(st->device);
  cudaFree(st->m); cudaFree(st->s); cudaFree(st->acc); cudaFree(st->owner); cudaFree(st->epoch);
  cudaFree(st->proj); cudaFree(st->src_proj); cudaFree(st->head_g);
  delete st;
  return EGTP_OK;
}

int plp_state_export(plp_state* st, float* m, float* s, float* acc, void* stream_v) {
  if (!st || !m || !s || !acc) return EGTP_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  if (cudaSetDevice(st->device) != cudaSuccess) return EGTP_ERR_CUDA;
  EGTP_CUDA_TRY(cudaMemcpyAsync(m, st->m, sizeof(float) * st->num_slots, cudaMemcpyDeviceToDevice, stream));
  EGTP_CUDA_TRY(cudaMemcpyAsync(s, st->s, sizeof(float) * st->num_slots, cudaMemcpyDeviceToDevice, stream));
  EGTP_CUDA_TRY(cudaMemcpyAsync(acc, st->acc, sizeof(float) * static_cast<size_t>(st->num_slots) * st->d,
                                cudaMemcpyDeviceToDevice, stream));
  return EGTP_OK;
}

int plp_state_import(plp_state* st, const float* m, const float* s, const float* acc, void* stream_v) {
  if (!st || !m || !s || !acc) return EGTP_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  if (cudaSetDevice(st->device) != cudaSuccess) return EGTP_ERR_CUDA;
  EGTP_CUDA_TRY(cudaMemcpyAsync(st->m, m, sizeof(float) * st->num_slots, cudaMemcpyDeviceToDevice, stream));
  EGTP_CUDA_TRY(cudaMemcpyAsync(st->s, s, sizeof(float) * st->num_slots, cudaMemcpyDeviceToDevice, stream));
  EGTP_CUDA_TRY(cudaMemcpyAsync(st->acc, acc, sizeof(float) * static_cast<size_t>(st->num_slots) * st->d,
                                cudaMemcpyDeviceToDevice, stream));
  st->proj_valid = false;
  return EGTP_OK;
}

int plp_step(egtp_ctx* c, plp_state* st, const egtp_lm_head* lm, const egtp_head* head, const void* hidden_step,
             int64_t ldh, const int32_t* slot_ids, const int32_t* reset_src, const float* src_m, const float* src_s,
             const float* src_pooled, int32_t n_src, int32_t B_live, float alpha, float* Hstep_out, float* z_out,
             float* yrem_out, int32_t* status_dev, void* stream_v) {
  if (!c || !st || st->ctx != c) return EGTP_ERR_INVALID_ARG;
  if (B_live == 0) return EGTP_OK;
  int rc = check_plp_common(c, st, head, src_m, src_s, src_pooled, n_src, B_live, alpha, yrem_out);
  if (rc != EGTP_OK) return rc;
  rc = check_lm(c, lm, hidden_step, ldh);
  if (rc != EGTP_OK) return rc;
  if (lm->d != st->d) return EGTP_ERR_INVALID_ARG;
  if (head) {
    rc = check_head(c, head, lm->d);
    if (rc != EGTP_OK) return rc;
  }
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  if (cudaSetDevice(c->device) != cudaSuccess) return EGTP_ERR_CUDA;
  int32_t* status = status_dev ? status_dev : c->status;
  if (!status_dev) EGTP_CUDA_TRY(cudaMemsetAsync(c->status, 0, sizeof(int32_t), stream));
  LmheadPlan plan;
  if (plp_fused_route(c, st, lm->dtype, head, B_live, n_src, yrem_out)) {
    // bound state: W1 h' comes out of the LM-head kernel, one kernel finishes the step
    if (!st->proj_valid) {
      rc = project_rows(c, head, st->acc, st->d, st->num_slots, st->proj, head->m_h, status, stream);
      if (rc != EGTP_OK) return rc;
      st->proj_valid = true;
    }
    if (reset_src && n_src > 0) {
      rc = project_rows(c, head, src_pooled, st->d, n_src, st->src_proj, head->m_h, status, stream);
      if (rc != EGTP_OK) return rc;
    }
    rc = run_lmhead(c, lm, hidden_step, ldh, B_live, status, stream, &plan, head->W1, head->m_h, st->head_g, st->g_rows,
                    st->ldg_max);
    if (rc != EGTP_OK) return rc;
    LaunchScope ls(c, EGTP_K_PLP_UPDATE, stream);
    EGTP_CUDA_TRY(launch_plp_update_bound(hidden_step, ldh, c->partials, plan.slots, plan.slots * 3, 3, Hstep_out, slot_ids,
                                          reset_src, src_m, src_s, src_pooled, st->src_proj, n_src, B_live, st->d,
                                          st->num_slots, 1.f / alpha, st->m, st->s, st->acc, st->proj, z_out, st->d,
                                          st->head_g, plan.head_cols_pad, 1, 0, head_args(head), yrem_out, st->owner, st->epoch, status, stream,
                                          /*overlap_previous=*/c->launch_overlap && !c->profiling));
    return EGTP_OK;
  }
  rc = run_lmhead(c, lm, hidden_step, ldh, B_live, status, stream, &plan);
  if (rc != EGTP_OK) return rc;
  return plp_update_and_head(c, st, head, hidden_step, ldh, lm->dtype, c->partials, plan.slots, plan.slots * 3, 3, slot_ids, reset_src, src_m, src_s,
                             src_pooled, n_src, B_live, alpha, Hstep_out, z_out, yrem_out, status, stream);
}

int plp_state_bind_head(plp_state* st, const egtp_head* head) {
  if (!st || !head) return EGTP_ERR_INVALID_ARG;
  egtp_ctx* c = st->ctx;
  int rc = check_head(c, head, st->d);
  if (rc != EGTP_OK) return rc;
  if (head->wdtype != EGTP_BF16) return EGTP_ERR_UNSUPPORTED;
  if (cudaSetDevice(c->device) != cudaSuccess) return EGTP_ERR_CUDA;
  if (cudaDeviceSynchronize() != cudaSuccess) return EGTP_ERR_CUDA;   // buffers of an earlier binding may be in use
  cudaFree(st->proj); cudaFree(st->src_proj); cudaFree(st->head_g);
  st->proj = st->src_proj = st->head_g = nullptr;
  st->bound = false;
  // head_g: one row per padded LM-head row (decode shapes pad to 128 / 256 rows, larger batches to 128),
  // columns padded to the coarsest column granularity of the LM-head shapes (256)
  const int64_t cap = std::min<int64_t>(c->max_batch, st->num_slots);
  st->g_rows = std::max<int64_t>(2 * kTileM, (cap + kTileM - 1) / kTileM * kTileM);
  st->ldg_max = (static_cast<int64_t>(head->m_h) + 255) / 256 * 256;   // covers every shape's column granularity
  bool ok = cudaMalloc(reinterpret_cast<void**>(&st->proj), sizeof(float) * static_cast<size_t>(st->num_slots) * head->m_h) == cudaSuccess;
  ok = ok && cudaMalloc(reinterpret_cast<void**>(&st->src_proj), sizeof(float) * static_cast<size_t>(c->max_batch) * head->m_h) == cudaSuccess;
  // room for up to 16 K-split slices (steps whose entropies do not come from an LM-head launch), at most 64 MB
  const int64_t slice_bytes = static_cast<int64_t>(sizeof(float)) * st->g_rows * st->ldg_max;
  st->g_max_splits = static_cast<int>(std::max<int64_t>(1, std::min<int64_t>(16, (64ll << 20) / slice_bytes)));
  ok = ok && cudaMalloc(reinterpret_cast<void**>(&st->head_g), static_cast<size_t>(slice_bytes) * st->g_max_splits) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    cudaFree(st->proj); cudaFree(st->src_proj); cudaFree(st->head_g);
    st->proj = st->src_proj = st->head_g = nullptr;
    return EGTP_ERR_CUDA;
  }
  st->bound_head = *head;
  st->bound = true;
  st->proj_valid = false;   // the first step through the bound route projects the current acc
  return EGTP_OK;
}

int egtp_entropy_from_logits(egtp_ctx* c, const void* logits, int64_t ldl, int32_t logits_dtype, int64_t rows,
                             int32_t V, float* H_out, int32_t* status_dev, void* stream_v) {
  if (!c || !H_out || rows < 0) return EGTP_ERR_INVALID_ARG;
  if (rows == 0) return EGTP_OK;
  int slots = 0;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  if (cudaSetDevice(c->device) != cudaSuccess) return EGTP_ERR_CUDA;
  int32_t* status = status_dev ? status_dev : c->status;
  if (!status_dev) EGTP_CUDA_TRY(cudaMemsetAsync(c->status, 0, sizeof(int32_t), stream));
  return run_logits_entropy(c, logits, ldl, logits_dtype, rows, V, status, stream, &slots, H_out);
}

int plp_step_from_logits(egtp_ctx* c, plp_state* st, const void* logits, int64_t ldl, int32_t logits_dtype, int32_t V,
                         const egtp_head* head, const void* hidden_step, int64_t ldh, int32_t hidden_dtype,
                         const int32_t* slot_ids, const int32_t* reset_src, const float* src_m, const float* src_s,
                         const float* src_pooled, int32_t n_src, int32_t B_live, float alpha, float* Hstep_out,
                         float* z_out, float* yrem_out, int32_t* status_dev, void* stream_v) {
  if (!c || !st || st->ctx != c) return EGTP_ERR_INVALID_ARG;
  if (B_live == 0) return EGTP_OK;
  int rc = check_plp_common(c, st, head, src_m, src_s, src_pooled, n_src, B_live, alpha, yrem_out);
  if (rc != EGTP_OK) return rc;
  if (!hidden_step || ldh < st->d) return EGTP_ERR_INVALID_ARG;
  if (hidden_dtype != EGTP_F32 && hidden_dtype != EGTP_BF16) return EGTP_ERR_UNSUPPORTED;
  if ((ldh * elem_bytes(hidden_dtype)) % 16 != 0 || reinterpret_cast<uintptr_t>(hidden_step) % 16 != 0)
    return EGTP_ERR_UNSUPPORTED;
  if (head) {
    rc = check_head(c, head, st->d);
    if (rc != EGTP_OK) return rc;
  }
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  if (cudaSetDevice(c->device) != cudaSuccess) return EGTP_ERR_CUDA;
  int32_t* status = status_dev ? status_dev : c->status;
  if (!status_dev) EGTP_CUDA_TRY(cudaMemsetAsync(c->status, 0, sizeof(int32_t), stream));
  // State bound to this head: W1 h' does not depend on the logits, so its launch goes to the context's side stream
  // and runs next to the pass over the logits; the update waits for both.
  LmheadPlan proj_plan;
  const bool bound = plp_bound_tail_route(c, st, hidden_dtype, head, B_live, n_src, yrem_out, hidden_step, ldh);
  if (bound) {
    rc = plp_bound_prepare(c, st, head, reset_src, src_pooled, n_src, status, stream);
    if (rc != EGTP_OK) return rc;
    EGTP_CUDA_TRY(cudaEventRecord(c->fork_ev, stream));
    EGTP_CUDA_TRY(cudaStreamWaitEvent(c->copy_stream, c->fork_ev, 0));
    rc = plp_bound_project(c, st, head, hidden_step, ldh, B_live, status, c->copy_stream, &proj_plan);
    if (cudaEventRecord(c->join_ev, c->copy_stream) != cudaSuccess) return EGTP_ERR_CUDA;
  }
  int slots = 0;
  const int rc_entropy = run_logits_entropy(c, logits, ldl, logits_dtype, B_live, V, status, stream, &slots);
  // the side stream always rejoins, whatever failed (a stream capture in progress must not be left forked)
  if (bound && cudaStreamWaitEvent(stream, c->join_ev, 0) != cudaSuccess) return EGTP_ERR_CUDA;
  if (rc != EGTP_OK) return rc;
  if (rc_entropy != EGTP_OK) return rc_entropy;
  return plp_update_and_head(c, st, head, hidden_step, ldh, hidden_dtype, c->partials, slots, slots * 3, 3, slot_ids, reset_src, src_m, src_s,
                             src_pooled, n_src, B_live, alpha, Hstep_out, z_out, yrem_out, status, stream,
                             bound ? &proj_plan : nullptr);
}

int egtp_entropy_partials(egtp_ctx* c, const egtp_lm_head* lm_shard, const void* hidden, int64_t ldh, int64_t rows,
                          float* partial_out, int32_t* status_dev, void* stream_v) {
  if (!c || !partial_out || rows < 0) return EGTP_ERR_INVALID_ARG;
  if (rows == 0) return EGTP_OK;
  if (rows > std::max<int64_t>(c->max_tokens, c->max_batch)) return EGTP_ERR_CAPACITY;
  int rc = check_lm(c, lm_shard, hidden, ldh);
  if (rc != EGTP_OK) return rc;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  if (cudaSetDevice(c->device) != cudaSuccess) return EGTP_ERR_CUDA;
  int32_t* status = status_dev ? status_dev : c->status;
  if (!status_dev) EGTP_CUDA_TRY(cudaMemsetAsync(c->status, 0, sizeof(int32_t), stream));
  LmheadPlan plan;
  rc = run_lmhead(c, lm_shard, hidden, ldh, rows, status, stream, &plan);
  if (rc != EGTP_OK) return rc;
  LaunchScope ls(c, EGTP_K_ENTROPY_MERGE, stream);
  EGTP_CUDA_TRY(launch_partials_reduce(c->partials, plan.slots, rows, partial_out, status, stream));
  return EGTP_OK;
}

int egtp_entropy_from_partials(egtp_ctx* c, const float* gathered, int32_t num_shards, int64_t rows, float* H_out,
                               int32_t* status_dev, void* stream_v) {
  if (!c || !gathered || !H_out || num_shards <= 0 || rows < 0) return EGTP_ERR_INVALID_ARG;
  if (rows == 0) return EGTP_OK;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  if (cudaSetDevice(c->device) != cudaSuccess) return EGTP_ERR_CUDA;
  int32_t* status = status_dev ? status_dev : c->status;
  if (!status_dev) EGTP_CUDA_TRY(cudaMemsetAsync(c->status, 0, sizeof(int32_t), stream));
  LaunchScope ls(c, EGTP_K_ENTROPY_MERGE, stream);
  EGTP_CUDA_TRY(launch_entropy_merge(gathered, num_shards, 3, rows * 3, rows, 0, H_out, nullptr, 0, nullptr, -1, status,
                                     stream));
  return EGTP_OK;
}

int plp_step_from_partials(egtp_ctx* c, plp_state* st, const float* gathered, int32_t num_shards,
                           const egtp_head* head, const void* hidden_step, int64_t ldh, int32_t hidden_dtype,
                           const int32_t* slot_ids, const int32_t* reset_src, const float* src_m, const float* src_s,
                           const float* src_pooled, int32_t n_src, int32_t B_live, float alpha, float* Hstep_out,
                           float* z_out, float* yrem_out, int32_t* status_dev, void* stream_v) {
  if (!c || !st || st->ctx != c || !gathered || num_shards <= 0) return EGTP_ERR_INVALID_ARG;
  if (B_live == 0) return EGTP_OK;
  int rc = check_plp_common(c, st, head, src_m, src_s, src_pooled, n_src, B_live, alpha, yrem_out);
  if (rc != EGTP_OK) return rc;
  if (!hidden_step || ldh < st->d) return EGTP_ERR_INVALID_ARG;
  if (hidden_dtype != EGTP_F32 && hidden_dtype != EGTP_BF16) return EGTP_ERR_UNSUPPORTED;
  if ((ldh * elem_bytes(hidden_dtype)) % 16 != 0 || reinterpret_cast<uintptr_t>(hidden_step) % 16 != 0)
    return EGTP_ERR_UNSUPPORTED;
  if (head) {
    rc = check_head(c, head, st->d);
    if (rc != EGTP_OK) return rc;
  }
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  if (cudaSetDevice(c->device) != cudaSuccess) return EGTP_ERR_CUDA;
  int32_t* status = status_dev ? status_dev : c->status;
  if (!status_dev) EGTP_CUDA_TRY(cudaMemsetAsync(c->status, 0, sizeof(int32_t), stream));
  return plp_update_and_head(c, st, head, hidden_step, ldh, hidden_dtype, gathered, num_shards, 3,
                             static_cast<int64_t>(B_live) * 3, slot_ids, reset_src, src_m, src_s, src_pooled, n_src,
                             B_live, alpha, Hstep_out, z_out, yrem_out, status, stream);
}

int plp_step_host(egtp_ctx* c, plp_state* st, const egtp_lm_head* lm, const egtp_head* head,
                  const void* hidden_step_host, const int32_t* reset_src_host, const float* src_m, const float* src_s,
                  const float* src_pooled, int32_t n_src, int32_t B_live, float alpha, float* yrem_host,
                  int32_t* status_host, void* stream_v) {
  if (!c || !st || !lm || !head || !hidden_step_host || !yrem_host || !status_host) return EGTP_ERR_INVALID_ARG;
  if (B_live <= 0) return EGTP_ERR_INVALID_ARG;
  if (!c->host_staging) return EGTP_ERR_UNSUPPORTED;
  if (B_live > c->max_batch || lm->d > c->max_d) return EGTP_ERR_CAPACITY;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  if (cudaSetDevice(c->device) != cudaSuccess) return EGTP_ERR_CUDA;
  const size_t hbytes = static_cast<size_t>(B_live) * lm->d * elem_bytes(lm->dtype);
  EGTP_CUDA_TRY(cudaMemcpyAsync(c->hidden_stage, hidden_step_host, hbytes, cudaMemcpyHostToDevice, stream));
  if (reset_src_host)
    EGTP_CUDA_TRY(cudaMemcpyAsync(c->reset_stage, reset_src_host, sizeof(int32_t) * B_live, cudaMemcpyHostToDevice,
                                  stream));
  int rc = plp_step(c, st, lm, head, c->hidden_stage, lm->d, nullptr, reset_src_host ? c->reset_stage : nullptr,
                    src_m, src_s, src_pooled, n_src, B_live, alpha, nullptr, nullptr, c->yhat, nullptr, stream);
  if (rc != EGTP_OK) return rc;
  EGTP_CUDA_TRY(cudaMemcpyAsync(yrem_host, c->yhat, sizeof(float) * B_live, cudaMemcpyDeviceToHost, stream));
  EGTP_CUDA_TRY(cudaMemcpyAsync(status_host, c->status, sizeof(int32_t), cudaMemcpyDeviceToHost, stream));
  EGTP_CUDA_TRY(cudaStreamSynchronize(stream));
  return EGTP_OK;
}

int plp_step_host_async(egtp_ctx* c, plp_state* st, const egtp_lm_head* lm, const egtp_head* head,
                        const void* hidden_step_host, const int32_t* reset_src_host, const float* src_m, const float* src_s,
                        const float* src_pooled, int32_t n_src, int32_t B_live, float alpha, float* yrem_host,
                        int32_t* status_host, void* stream_v) {
  if (!c || !st || !lm || !head || !hidden_step_host || !yrem_host || !status_host) return EGTP_ERR_INVALID_ARG;
  if (B_live <= 0) return EGTP_ERR_INVALID_ARG;
  if (!c->host_staging) return EGTP_ERR_UNSUPPORTED;
  if (lm->dtype != EGTP_F32 && lm->dtype != EGTP_BF16) return EGTP_ERR_UNSUPPORTED;
  if (B_live > c->max_batch || lm->d > c->max_d) return EGTP_ERR_CAPACITY;
  const size_t hbytes = static_cast<size_t>(B_live) * lm->d * elem_bytes(lm->dtype);
  const size_t half = static_cast<size_t>(c->stage_bytes / 2) / 256 * 256;
  if (hbytes > half) return EGTP_ERR_CAPACITY;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  if (cudaSetDevice(c->device) != cudaSuccess) return EGTP_ERR_CUDA;
  // Calls alternate between the two halves of the staging buffers.  The copy of this call's rows runs on the
  // context's copy stream, behind the step that read this half two calls ago and next to the previous call's kernels.
  const int p = c->host_parity;
  char* hidden_dev = static_cast<char*>(c->hidden_stage) + p * half;
  int32_t* reset_dev = c->reset_stage + static_cast<int64_t>(p) * c->max_batch;
  EGTP_CUDA_TRY(cudaStreamWaitEvent(c->copy_stream, c->host_stage_free[p], 0));
  EGTP_CUDA_TRY(cudaMemcpyAsync(hidden_dev, hidden_step_host, hbytes, cudaMemcpyHostToDevice, c->copy_stream));
  if (reset_src_host)
    EGTP_CUDA_TRY(cudaMemcpyAsync(reset_dev, reset_src_host, sizeof(int32_t) * B_live, cudaMemcpyHostToDevice, c->copy_stream));
  EGTP_CUDA_TRY(cudaEventRecord(c->host_in_ready[p], c->copy_stream));
  EGTP_CUDA_TRY(cudaStreamWaitEvent(stream, c->host_in_ready[p], 0));
  int rc = plp_step(c, st, lm, head, hidden_dev, lm->d, nullptr, reset_src_host ? reset_dev : nullptr, src_m, src_s,
                    src_pooled, n_src, B_live, alpha, nullptr, nullptr, c->yhat, nullptr, stream);
  // whatever happened, the half counts as used by `stream` up to here
  if (cudaEventRecord(c->host_stage_free[p], stream) != cudaSuccess) return EGTP_ERR_CUDA;
  c->host_parity ^= 1;
  if (rc != EGTP_OK) return rc;
  EGTP_CUDA_TRY(cudaMemcpyAsync(yrem_host, c->yhat, sizeof(float) * B_live, cudaMemcpyDeviceToHost, stream));
  EGTP_CUDA_TRY(cudaMemcpyAsync(status_host, c->status, sizeof(int32_t), cudaMemcpyDeviceToHost, stream));
  return EGTP_OK;
}

}  // extern "C"
