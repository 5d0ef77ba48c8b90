// Internal launcher interface between the C ABI (api.cu) and the kernels. Not installed.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace egtp {

// Finite stand-in for "no logit seen yet" / "masked column": keeps every product finite.
constexpr float kNegBig = -1.0e30f;

// ---- K1: LM-head GEMM with online entropy epilogue ---------------------------------------
constexpr int kTileM = 128;        // token rows per tile (UMMA M, one TMEM lane per row)
constexpr int kRowBytes = 128;     // K extent of one pipeline stage in bytes (one swizzle row)
constexpr int kEpiSplit = 2;       // epilogue warps per TMEM lane quadrant (column halves)
constexpr int kLmheadThreads = (2 + 4 * kEpiSplit) * 32;

struct LmheadPlan {
  int variant;        // 0 prompt shape, 1 decode <= 128 rows, 2 decode <= 256 rows, 4 / 5 CTA-pair prompt / decode
  int a_box_rows;     // rows of one TMA box of the hidden states
  int grid;           // persistent CTAs
  int row_blocks;     // ceil(T / rows_per_block)
  int rows_per_block; // 128 or 256: rows a CTA (or CTA pair) multiplies against each W tile
  int tile_cols;      // vocabulary columns per tile
  int b_box_rows;     // rows of one TMA box of W
  int col_gran;       // vocabulary chunks start at multiples of this many columns
  int n_groups;       // ceil(V / col_gran) + head_cols_pad / col_gran
  int v_pad;          // V rounded up to col_gran: column index of the first fused head column
  int head_cols_pad;  // fused head columns (rows of the head's W1) rounded up to col_gran; 0 = none
  int chunks;         // vocabulary chunks S; a work unit is (row block, chunk)
  int slots;          // partial slots per row
  int group_rb;       // row blocks that sweep the vocabulary together (L2 reuse of W tiles)
  int k_blocks;       // ceil(d * elem / 128)
  int b_k_blocks;     // > 0: W1 has this many k blocks and is read again from its start for every further segment of A
  int k_splits;       // > 1: K is split over that many units per (row block, chunk); head projection launches only
  int smem_bytes;     // dynamic shared memory
  int64_t rows_pad;   // row_blocks * rows_per_block: rows of the partial buffer
};

// Picks chunks / grouping for T rows; slot_limit bounds chunks * kEpiSplit * rows_pad by the
// partial buffer's capacity (in rows x slots).
// pair_workers states how many CTA pairs the device can co-schedule (lmhead_prepare_device measures it; 0 = none).  force_chunks > 0 overrides the number of vocabulary chunks of prompt batches (clamped to the workspace).
// head_cols > 0: that many rows of a second matrix (the head's W1) are appended to the vocabulary as
// extra columns whose raw products the kernel writes out (bf16, one-CTA shapes only).
LmheadPlan make_lmhead_plan(int64_t T, int d, int V, int elem_bytes, int num_sms, int64_t slot_row_capacity,
                            int mode, int head_cols, int force_chunks, int pair_workers);

// Launch shape for W1 hidden[i] alone (no vocabulary): the head columns of the prompt shape with K split over
// up to max_splits units, each writing its own slice head_g[split][rows_pad][head_cols_pad].
// a_repeats > 1: the rows of A are a_repeats segments of d elements (d * elem_bytes a multiple of 128) that are all
// multiplied against the same W1 and summed, e.g. the high and low bf16 halves of fp32 vectors.
LmheadPlan make_headproj_plan(int64_t T, int d, int m_h, int elem_bytes, int num_sms, int max_splits,
                              int a_repeats = 1);

// Opts the kernels into their dynamic shared-memory size on the current device and reports how many CTA pairs of
// the pair kernels that device can hold at once.
cudaError_t lmhead_prepare_device(int* pair_workers_out);

// partials layout: [rows_pad][slots][3] floats: (m, s, t2) with m the running max logit,
// s = sum 2^((x-m) log2 e), t2 = sum 2^(...) * (x-m) log2 e over the slot's vocabulary range.
// Tensor maps of one launch (K-major, 128-byte rows, 128-byte swizzle).  w / w1: boxes of plan.b_box_rows rows;
// w_tile / w1_tile: boxes of plan.tile_cols rows (one copy per full tile; may equal w / w1 when the two box
// heights are the same, must be NULL for the CTA-pair variants that do not use them).  w1 and w1_tile describe
// the head's W1 [m_h][d] and are needed only with plan.head_cols_pad > 0; head_g [plan.rows_pad][plan.head_cols_pad]
// then receives head_g[i][j] = W1[j] . hidden[i].
struct LmheadMaps {
  const CUtensorMap* hidden = nullptr;
  const CUtensorMap* w = nullptr;
  const CUtensorMap* w_tile = nullptr;
  const CUtensorMap* w1 = nullptr;
  const CUtensorMap* w1_tile = nullptr;
};
// overlap_previous: launch with programmatic stream serialization: the blocks set themselves up while the kernel
// before this one in the stream is still finishing and wait for its end before they touch global memory.
cudaError_t launch_lmhead_entropy(const LmheadPlan& plan, bool tf32, const LmheadMaps& maps, int64_t T, int V,
                                  float* partials, int32_t* status, cudaStream_t stream, float* head_g = nullptr,
                                  bool overlap_previous = false);

// ---- K2: entropy merge, Eq. 3-4 pooling -------------------------------------
constexpr int kPoolChunkTokens = 64;   // tokens per first-stage pooling chunk
constexpr int kPoolThreads = 128;      // each thread owns 8 consecutive channels

cudaError_t launch_validate_offsets(const int32_t* offsets, int B, int64_t T, int32_t* status, cudaStream_t stream);

// slot j of row i is read at partials + i * row_stride + j * slot_stride (floats); row i is token row0 + i of
// the batch (H, weights and segment ids are indexed by the batch-wide token index)
cudaError_t launch_partials_reduce(const float* partials, int slots, int64_t rows, float* out, const int32_t* status,
                                   cudaStream_t stream);
// What the merge kernel leaves for the entropy-weighted pooling of the same tokens (Eq. 3 up to its normaliser): per
// token the unnormalised weight exp(H/alpha - m) relative to the maximum m of its prompt's run inside its 64-token
// chunk, and (m, sum of weights) per run: in seg_m / seg_s for prompts inside one chunk, else in piece_ms
// ([2 * chunks][2], chunks = ceil(T_total / kPoolChunkTokens) of the whole batch).
struct PoolPrep {
  float inv_alpha;
  float* weights;      // [T_total]
  float* piece_ms;
  int64_t chunks;
  float* seg_m;        // [B]
  float* seg_s;        // [B]
};
// T_check >= 0: the launch also checks the offsets against that token count (EGTP_ERR_BAD_OFFSETS in *status).
// prep != NULL needs offsets and row0 a multiple of kPoolChunkTokens.
cudaError_t launch_entropy_merge(const float* partials, int slots, int64_t row_stride, int64_t slot_stride, int64_t T,
                                 int64_t row0, float* H, const int32_t* offsets, int B, int32_t* seg_id_out,
                                 int64_t T_check, int32_t* status, cudaStream_t stream, const PoolPrep* prep = nullptr);

// Eq. 3 weights as an output: w_i = exp(H_i/alpha - M_b) / Z_b from the per-prompt state the pooling left (0 outside prompts)
cudaError_t launch_token_weights(const float* H, const int32_t* offsets, int B, int64_t T, float inv_alpha,
                                 const float* seg_m, const float* seg_s, float* weights, const int32_t* status,
                                 cudaStream_t stream);

// Pooling over the prompts' token spans.  mode 0: entropy-weighted (Eq. 3-4) with the unnormalised weights, seg_s and
// piece_ms a merge launch with a PoolPrep left; EGTP_POOL_MEAN / _MAX / _LAST: the alternatives of the paper's
// ablation (weights unused; the kernel fills seg_m / seg_s / piece_ms itself).  piece_a / piece_b [chunks][d] and
// piece_ms [2 * chunks][2] (chunks = ceil(T / kPoolChunkTokens)) hold the pieces of prompts that span several chunks.
cudaError_t launch_pool(const void* hidden, int64_t ldh, bool bf16, int mode, const float* weights,
                        const int32_t* offsets, int B, int64_t T, int d, float* pooled, float* piece_a,
                        float* piece_b, float* piece_ms, float* seg_m, float* seg_s, const int32_t* status,
                        cudaStream_t stream);

// Merges the pieces (same T and mode as the launch_pool before it), zero-fills empty prompts, completes seg_m / seg_s and,
// with zcat != NULL, also writes every pooled row as [hi | lo] bf16 halves: zcat [B][2 d]
cudaError_t launch_pool_combine(const int32_t* offsets, int B, int64_t T, int d, int mode, const float* piece_a,
                                const float* piece_b, const float* piece_ms, float* pooled, float* seg_m, float* seg_s,
                                void* zcat, const int32_t* status, cudaStream_t stream);

// dst [dst_rows][row_bytes] <- the first src_rows rows of src (ld_bytes apart), the other rows zero.
// row_bytes and ld_bytes are multiples of 16, both pointers 16-byte aligned.
cudaError_t launch_pad_rows(const void* src, int64_t ld_bytes, int src_rows, int64_t row_bytes, void* dst,
                            int dst_rows, const int32_t* status, cudaStream_t stream);

// ---- Eq. 2 from logits already in memory -------------------------------------------------------
int logits_entropy_pick_splits(int64_t rows, int V, int num_sms);
// partials [rows][splits][3] in the layout of the LM-head kernel's partials.  H_out != NULL: the kernel also merges
// each row's partials into H_out[row] (the last block of the row to finish does it); arrivals [rows] int32 must
// then be zero on entry and is zero again on exit.
cudaError_t launch_logits_entropy(const void* logits, int64_t ldl, bool bf16, int64_t rows, int V, int splits,
                                  float* partials, float* H_out, int32_t* arrivals, const int32_t* status,
                                  cudaStream_t stream);

// ---- K3: head ------------------------------------------------------------------------------
struct HeadArgs {
  const void* W1;
  const float* b1;
  const void* W2;
  const float* b2;
  const float* centres;
  int d, m_h, d_out;
  bool bf16;
  int mode;
};
int head_pick_splits(int rows, int d, int m_h, int num_sms, int64_t partial_capacity_floats);

cudaError_t launch_head_hidden(const HeadArgs& h, const float* z, int64_t ldz, int rows, int splits,
                               float* partial, const int32_t* status, cudaStream_t stream);

// partial[s * split_stride + r * row_stride + j]; strides 0 = the dense [splits][rows][m_h] layout
cudaError_t launch_head_out(const HeadArgs& h, const float* partial, int rows, int splits, float* y, float* phat,
                            const int32_t* status, cudaStream_t stream, int64_t split_stride = 0,
                            int64_t row_stride = 0);

// xcat[r] = [bf16(x[r]) | bf16(x[r] - bf16(x[r]))]: fp32 rows as two bf16 halves (16 significant bits together)
cudaError_t launch_split_hi_lo(const float* x, int64_t ldx, int rows, int d, void* xcat, const int32_t* status,
                               cudaStream_t stream);

// out[r][j] = sum_s partial[s][r][j] (split order): W1 x for rows x that are not pooled vectors
// (strides as in launch_head_out)
cudaError_t launch_head_partial_sum(const float* partial, int rows, int splits, int m_h, float* out, int64_t ld_out,
                                    const int32_t* status, cudaStream_t stream, int64_t split_stride = 0,
                                    int64_t row_stride = 0);

// ---- self-test of the bounded wait (a wait on a barrier nobody signals must end with an error status)
cudaError_t launch_wait_timeout_selftest(uint64_t limit_ns, int32_t* status, cudaStream_t stream);

// ---- K4: PLP running-state update ---------------------------------------------------------
// Merges the row's entropy partials itself (Eq. 2), optionally writes H' to Hstep_out, then updates the slot.
// owner [num_slots] (zero-initialised) and epoch [2] (initialised to {1, 0}) belong to the state: with them the kernels
// refuse a second row of one step on the same slot (EGTP_ERR_BAD_SLOT).
cudaError_t launch_plp_update(const void* hidden_step, int64_t ldh, bool bf16, const float* partials, int slots,
                              int64_t row_stride, int64_t slot_stride, float* Hstep_out,
                              const int32_t* slot_ids, const int32_t* reset_src, const float* src_m,
                              const float* src_s, const float* src_pooled, int n_src, int rows, int d, int num_slots,
                              float inv_alpha, float* st_m, float* st_s, float* st_acc, float* z, int64_t ldz,
                              int32_t* owner, int32_t* epoch, int32_t* status, cudaStream_t stream, void* zcat = nullptr);

// The update for a state bound to a head (bf16 hidden states and head weights): also advances the slot's
// projection st_proj = W1 acc with g = W1 h' from the LM-head kernel and finishes the head for the row.
// src_proj [n_src][m_h] = W1 src_pooled; z may be NULL; g is the sum of g_splits slices g_split_stride floats apart.  overlap_previous: launch with programmatic stream
// serialization, so that blocks are staged (and read their state rows) while the LM-head kernel before it in the
// stream is still running; the kernel waits for that kernel's end before it reads its results.
cudaError_t launch_plp_update_bound(const void* hidden_step, int64_t ldh, const float* partials, int slots,
                                    int64_t row_stride, int64_t slot_stride, float* Hstep_out, const int32_t* slot_ids,
                                    const int32_t* reset_src, const float* src_m, const float* src_s,
                                    const float* src_pooled, const float* src_proj, int n_src, int rows, int d,
                                    int num_slots, float inv_alpha, float* st_m, float* st_s, float* st_acc,
                                    float* st_proj, float* z, int64_t ldz, const float* g, int64_t ldg, int g_splits,
                                    int64_t g_split_stride, const HeadArgs& h, float* y, int32_t* owner, int32_t* epoch,
                                    int32_t* status, cudaStream_t stream, bool overlap_previous);

}  // namespace egtp
