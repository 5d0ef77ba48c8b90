/*
 * egtp.h - C ABI of the B200 (sm_100a) hot path of the entropy-guided length predictor:
 * Entropy-Guided Token Pooling (EGTP, paper Sec. 3.1, Eq. 2-4), the prediction head's forward
 * pass (Sec. 3.2, Eq. 6) and Progressive Length Prediction (PLP, Sec. 3.3, Eq. 8).
 *
 * Conventions that hold for every entry point
 *   - Plain C types only.  "device" pointers are CUDA device addresses on the context's GPU,
 *     "host" pointers are ordinary (ideally pinned) host addresses.  Each argument says which.
 *   - The caller owns every buffer it passes in.  The library owns only egtp_ctx / plp_state
 *     and keeps no caller pointer beyond the work a call enqueues on its stream.
 *   - Every function returns an egtp_status (0 = success, negative = error).  Problems the
 *     host can see (NULL pointers, sizes beyond the context's capacity, unsupported layouts)
 *     are returned at once and nothing is launched.  Problems only the device can see
 *     (malformed offsets, an out-of-range slot, a bounded wait that ran out) are written to
 *     the device status word: the first error wins, later kernels of the call do nothing,
 *     nothing traps and the CUDA context stays usable.
 *   - Device-pointer entry points are asynchronous: they enqueue on `stream` (a cudaStream_t
 *     passed as void*, NULL = the default stream) and return.  They never allocate device
 *     memory and never synchronise; all workspace is created by egtp_create /
 *     plp_state_create.  The *_host entry points copy their inputs host->device, run, copy
 *     the result back and synchronise the stream before returning.
 *   - Calls that use the same context must not overlap on the GPU (they share workspace).
 *   - Same inputs give bitwise identical outputs (no floating-point atomics anywhere).
 *   - Matrices are row-major.  The LM head is W[V][d] (row v = vocabulary entry v), so the
 *     logit of token i for entry v is sum_k hidden[i][k] * W[v][k]; no bias, norm or
 *     temperature is applied (the caller passes the tensor that feeds its LM head).
 *   - Supported layouts: hidden and W in the same dtype (EGTP_F32 or EGTP_BF16); rows start
 *     on 16-byte boundaries (d * element size and both leading dimensions are multiples of
 *     16 bytes); d is a multiple of 16.  Anything else is EGTP_ERR_UNSUPPORTED; there is no
 *     CPU fallback.
 */
#ifndef EGTP_H_
#define EGTP_H_

#include <stdint.h>

#if defined(__GNUC__)
#define EGTP_API __attribute__((visibility("default")))
#else
#define EGTP_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct egtp_ctx egtp_ctx;     /* device workspace, tensor-map encoder, SM count */
typedef struct plp_state plp_state;   /* per-slot running state (m, s, acc[d]) in device memory */

enum {
  EGTP_OK = 0,
  EGTP_ERR_INVALID_ARG = -1,      /* NULL where data is required, negative size, alpha <= 0 ... */
  EGTP_ERR_UNSUPPORTED = -2,      /* dtype / alignment / layout the kernels do not handle */
  EGTP_ERR_CAPACITY = -3,         /* larger than what egtp_create / plp_state_create was sized for */
  EGTP_ERR_CUDA = -4,             /* a CUDA runtime or driver call failed */
  EGTP_ERR_BAD_OFFSETS = -5,      /* (device) offsets not non-decreasing inside [0, T_total] */
  EGTP_ERR_DEVICE_TIMEOUT = -6,   /* (device) a bounded wait inside a kernel ran out */
  EGTP_ERR_BAD_SLOT = -7          /* (device) slot id or reset source out of range */
};

enum { EGTP_F32 = 0, EGTP_BF16 = 1 };                 /* element type of hidden, W and head weights */
enum { EGTP_HEAD_SCALAR = 0, EGTP_HEAD_BINS = 1 };    /* head output mode */
enum { PLP_RESET_KEEP = -2, PLP_RESET_EMPTY = -1 };   /* values of reset_src besides row ids >= 0 */

/* LM head (Sec. 3.1: the next-token distribution over the vocabulary V). Device memory, read-only. */
typedef struct {
  const void* W;      /* device; [V][ldw] elements, first d of each row used */
  int64_t ldw;        /* leading dimension in elements, >= d, ldw * element size % 16 == 0 */
  int32_t d;          /* hidden size */
  int32_t V;          /* vocabulary size */
  int32_t dtype;      /* EGTP_F32 or EGTP_BF16; must equal the dtype of the hidden states */
  int32_t reserved;
} egtp_lm_head;

/* Prediction head (Sec. 3.2): u = ReLU(W1 z + b1), o = W2 u + b2.
 * EGTP_HEAD_SCALAR (d_out == 1): y = o[0].
 * EGTP_HEAD_BINS   (d_out == K): p = softmax(o), y = sum_k p[k] * centres[k]   (Eq. 6).
 * Device memory, read-only. */
typedef struct {
  const void* W1;        /* device; [m_h][d] in `wdtype` */
  const float* b1;       /* device; [m_h] */
  const void* W2;        /* device; [d_out][m_h] in `wdtype` */
  const float* b2;       /* device; [d_out] */
  const float* centres;  /* device; [d_out] bin centres c_k, NULL in scalar mode */
  int32_t d, m_h, d_out; /* m_h <= 8192, d_out <= 256 */
  int32_t wdtype;        /* EGTP_F32 or EGTP_BF16 */
  int32_t mode;          /* EGTP_HEAD_SCALAR or EGTP_HEAD_BINS */
  int32_t reserved;
} egtp_head;

/* Creates a context on CUDA device `device` and allocates all workspace once, sized for at
 * most max_tokens packed tokens per call, max_batch prompts (or live sequences), hidden
 * size max_d and vocabulary max_V.  *out is set only on success.  The device must be an
 * sm_100 GPU (EGTP_ERR_UNSUPPORTED otherwise; EGTP_ERR_CUDA if allocation fails). */
EGTP_API int egtp_create(egtp_ctx** out, int device, int64_t max_tokens, int32_t max_batch,
                int32_t max_d, int32_t max_V);

/* egtp_create with options.  EGTP_CREATE_NO_HOST_STAGING leaves out the device copy of the hidden states that
 * only the *_host entry points use (max(max_tokens, max_batch) * max_d * 4 bytes, the largest buffer of a context
 * sized for long prompt batches); egtp_predict_host and plp_step_host then return EGTP_ERR_UNSUPPORTED.
 * flags == 0 is egtp_create.  Unknown flag bits: EGTP_ERR_INVALID_ARG. */
enum { EGTP_CREATE_NO_HOST_STAGING = 1 };
EGTP_API int egtp_create_ex(egtp_ctx** out, int device, int64_t max_tokens, int32_t max_batch,
                int32_t max_d, int32_t max_V, int32_t flags);

/* Frees the context's device memory. Outstanding work on its streams must have finished. */
EGTP_API int egtp_destroy(egtp_ctx* ctx);

/* Static description of a status code (never NULL). */
EGTP_API const char* egtp_status_string(int status);

/* Bytes of device memory the context holds. */
EGTP_API int64_t egtp_workspace_bytes(const egtp_ctx* ctx);

/* EGTP over a packed ragged batch of prompts (Sec. 3.1 Eq. 2-4, then the head of Sec. 3.2).
 *   Eq. 2: H[i] = -sum_v p_v ln p_v with p = softmax(W hidden[i]) (natural log), for every
 *          token row i in [0, T_total); the T x V logits are never written to memory.
 *   Eq. 3: within prompt b (tokens offsets[b] <= i < offsets[b+1]):
 *          w_i = exp(H_i/alpha) / sum_j exp(H_j/alpha); alpha = 1 is the equation as printed.
 *   Eq. 4: pooled[b] = sum_i w_i hidden[i].
 *   Eq. 6: yhat[b] = head(pooled[b]).
 * An empty prompt gives pooled = 0, state (m, s) = (-inf, 0) and yhat = head(0).  Tokens
 * before offsets[0] or at/after offsets[B] get an entropy but join no prompt (seg_id -1,
 * weight 0).
 * Arguments (all pointers device unless stated):
 *   lm, head      host structs holding device pointers; head may be NULL (then yhat_out and
 *                 phat_out must be NULL and the head is skipped)
 *   hidden        [T_total][ldh] rows in lm->dtype, read-only
 *   offsets       int32 [B+1], token units, must satisfy 0 <= offsets[0] <= ... <= offsets[B]
 *                 <= T_total (checked on the device: EGTP_ERR_BAD_OFFSETS in the status word)
 *   alpha         temperature dividing the entropies in Eq. 3, > 0
 *   H_out         [T_total] or NULL      token entropies (nats)
 *   weights_out   [T_total] or NULL      w_i of Eq. 3 (0 for tokens in no prompt); the pooling itself never stores
 *                 normalised weights, so asking for them costs one more small launch
 *   seg_id_out    int32 [T_total] or NULL  prompt index of each token, -1 if none
 *   pooled_out    [B][d] or NULL         Eq. 4
 *   state_m_out, state_s_out  [B] each or NULL: max_i H_i/alpha and sum_i exp(H_i/alpha - max),
 *                 the softmax normaliser that lets plp_step continue from this prompt
 *   yhat_out      [B] or NULL            predicted length
 *   phat_out      [B][d_out] or NULL     bin probabilities (bins mode only)
 *   status_dev    int32 [1] or NULL: device status word (caller zeroes it before the call; a
 *                 non-zero word on entry turns the whole call into a no-op). NULL = a word the
 *                 context owns, zeroed at the start of the call.
 *   stream        cudaStream_t
 * Returns EGTP_OK once the work is enqueued. B = 0 or T_total = 0 enqueue nothing. */
EGTP_API int egtp_predict(egtp_ctx* ctx, const egtp_lm_head* lm, const egtp_head* head,
                 const void* hidden, int64_t ldh, const int32_t* offsets,
                 int32_t B, int64_t T_total, float alpha,
                 float* H_out, float* weights_out, int32_t* seg_id_out,
                 float* pooled_out, float* state_m_out, float* state_s_out,
                 float* yhat_out, float* phat_out,
                 int32_t* status_dev, void* stream);

/* Same computation with the per-call data in HOST memory: hidden_host [T_total][d] (dense,
 * lm->dtype), offsets_host int32 [B+1], yhat_host float [B] (output), pooled_host [B][d] or NULL
 * (output), status_host int32 [1] (output: final device status word).  lm and head still
 * point at device-resident parameters.  Copies in, runs, copies out, synchronises `stream`.
 * For batches of 4096 tokens or more the hidden states are copied in up to four row ranges on a stream the
 * context owns (512 rows first, then ranges four times as long, the last one taking the rest), and the LM-head
 * kernel of one range runs while the next range is still being copied. */
EGTP_API int egtp_predict_host(egtp_ctx* ctx, const egtp_lm_head* lm, const egtp_head* head,
                      const void* hidden_host, const int32_t* offsets_host,
                      int32_t B, int64_t T_total, float alpha,
                      float* yhat_host, float* pooled_host, int32_t* status_host, void* stream);

/* Running PLP state for num_slots decode slots of hidden size d (Sec. 3.3): per slot the
 * online-softmax triple (m, s, acc[d]) of Eq. 3-4 over the tokens the sequence has
 * contributed so far; all slots start empty.  Allocates num_slots * (d + 2) floats. */
EGTP_API int plp_state_create(egtp_ctx* ctx, plp_state** out, int32_t num_slots, int32_t d);
EGTP_API int plp_state_destroy(plp_state* st);

/* Checkpoint / restore of the running state: m [num_slots], s [num_slots], acc [num_slots][d],
 * all device pointers, copied on `stream`. */
EGTP_API int plp_state_export(plp_state* st, float* m, float* s, float* acc, void* stream);
EGTP_API int plp_state_import(plp_state* st, const float* m, const float* s, const float* acc, void* stream);

/* One PLP decode step over B_live live sequences, one new token each (Sec. 3.3, Eq. 8).
 * Aggregate(h, {h'_1..h'_t}) is read as token-axis concatenation followed by EGTP: z_t is the
 * entropy-weighted pool (one joint softmax, Eq. 3-4) over the prompt's tokens and generated
 * tokens 1..t, kept incrementally in the slot's (m, s, acc); the head then gives the
 * remaining length.  For row i (slot = slot_ids[i]):
 *   reset_src[i] == PLP_RESET_KEEP : continue the slot's sequence;
 *   reset_src[i] == PLP_RESET_EMPTY: start a new sequence with no prompt;
 *   reset_src[i] == r >= 0         : start a new sequence from EGTP row r, i.e. from
 *                                    (src_m[r], src_s[r], src_pooled[r]) as egtp_predict wrote them;
 *   then the new token's entropy H' (Eq. 2) enters the softmax and hidden_step[i] the pool.
 * Arguments (device unless stated):
 *   hidden_step   [B_live][ldh] rows in lm->dtype
 *   slot_ids      int32 [B_live], distinct, each in [0, num_slots); NULL = identity (row i -> slot i).  A slot out of
 *                 range, or named by two rows of one step (they would race on its state), is refused on the device:
 *                 EGTP_ERR_BAD_SLOT in the status word, the refused rows change nothing
 *   reset_src     int32 [B_live] or NULL (all keep)
 *   src_m, src_s  [n_src]; src_pooled [n_src][d]; may be NULL when n_src == 0
 *   Hstep_out     [B_live] or NULL   entropy of each new token
 *   z_out         [B_live][d] or NULL  Eq. 8
 *   yrem_out      [B_live] or NULL   predicted remaining length (needs head)
 *   status_dev, stream as in egtp_predict. */
EGTP_API int plp_step(egtp_ctx* ctx, plp_state* st, const egtp_lm_head* lm, const egtp_head* head,
             const void* hidden_step, int64_t ldh,
             const int32_t* slot_ids, const int32_t* reset_src,
             const float* src_m, const float* src_s, const float* src_pooled, int32_t n_src,
             int32_t B_live, float alpha,
             float* Hstep_out, float* z_out, float* yrem_out,
             int32_t* status_dev, void* stream);

/* Binds a PLP state to one prediction head so that a decode step needs no separate layer-1 GEMM
 * (Sec. 3.2 head on the Sec. 3.3 aggregate).  Layer 1 of the head is linear before its ReLU and z = acc / s,
 * so W1 z = (W1 acc) / s.  A bound state keeps P = W1 acc [num_slots][m_h] next to acc and advances it with
 * the recurrence of the pool itself, P' = P e^(m-m') + e^(H'/alpha-m') (W1 h').  W1 h' for all live rows is
 * produced by the LM-head kernel: the m_h rows of W1 are appended to the vocabulary as extra output columns
 * whose products are written out instead of entering the entropy (0.2 % more GEMM work at m_h = 256).  One
 * kernel then merges the entropy partials, updates (m, s, acc, P) and finishes the head for its row.  The
 * result equals the unbound plp_step up to floating-point summation order.
 *   head   host struct with device pointers; wdtype must be EGTP_BF16 (EGTP_ERR_UNSUPPORTED otherwise).  The
 *          struct is copied; the weights it points at must stay in place and unchanged while bound.
 * Allocates num_slots * m_h + max_batch * m_h floats and up to 16 slices (64 MB at most) of (padded rows) x (padded
 * m_h) floats, and synchronises the device (a create-time call, not for the decode loop).  Binding again replaces the previous binding.
 * plp_step, plp_step_from_logits and plp_step_from_partials take the bound route when they are given the same
 * head (same W1 pointer, m_h, d, dtype) with yrem_out != NULL, bf16 hidden states (and LM head), and n_src <= the
 * context's max_batch; the two that run no LM-head GEMM get W1 h' from a launch of the LM-head kernel over the
 * head columns alone.  Every other call (another head, no head, plp_state_import) takes the ordinary route or
 * changes acc directly, and the next bound step first recomputes P = W1 acc for all slots (one layer-1 pass
 * over num_slots rows).  A bound step that restarts rows from EGTP rows (reset_src != NULL and n_src > 0)
 * first projects the n_src source rows (W1 src_pooled), so pass reset_src = NULL on steps without restarts
 * or keep n_src small.  All calls on one state must be ordered on the GPU (one stream, or events). */
EGTP_API int plp_state_bind_head(plp_state* st, const egtp_head* head);

/* plp_step with the step's data in HOST memory: hidden_step_host [B_live][d] dense,
 * reset_src_host int32 [B_live] or NULL, yrem_host float [B_live] (output), status_host int32 [1]
 * (output).  Rows map to slots 0..B_live-1.  The EGTP source table stays on the device. */
EGTP_API int plp_step_host(egtp_ctx* ctx, plp_state* st, const egtp_lm_head* lm, const egtp_head* head,
                  const void* hidden_step_host, const int32_t* reset_src_host,
                  const float* src_m, const float* src_s, const float* src_pooled, int32_t n_src,
                  int32_t B_live, float alpha, float* yrem_host, int32_t* status_host, void* stream);

/* plp_step_host without the wait at its end, for a decode loop that hands over step t + 1 while step t is still
 * running: the call enqueues the copy of hidden_step_host (on a stream the context owns, into one of two halves of
 * its staging buffer), the step and the copies of yrem_host and status_host (on `stream`), and returns.  The copy
 * of one call therefore overlaps the kernels of the call before it.  yrem_host and status_host hold the step's
 * results once `stream` has reached the end of the call's work (synchronise the stream or an event recorded behind
 * the call); all four host buffers must be pinned and stay untouched until then.  Any number of calls may be in
 * flight; B_live * d elements must fit half of the staging buffer (EGTP_ERR_CAPACITY otherwise).  Do not mix with
 * the blocking host entry points while calls are in flight. */
EGTP_API int plp_step_host_async(egtp_ctx* ctx, plp_state* st, const egtp_lm_head* lm, const egtp_head* head,
                  const void* hidden_step_host, const int32_t* reset_src_host,
                  const float* src_m, const float* src_s, const float* src_pooled, int32_t n_src,
                  int32_t B_live, float alpha, float* yrem_host, int32_t* status_host, void* stream);

/* Prediction head alone, for callers that cannot allocate device memory.  (The paper has no
 * counterpart of this entry point; it exists for deployment reasons only.)
 * Who needs it: code that runs inside a host which owns all GPU memory and rules out cudaMalloc
 * while it serves - an inference engine whose pool was carved up at start-up, a plugin inside
 * another runtime, a process with a fixed memory budget.  Such callers cannot use egtp_create,
 * which allocates its workspace.  This call needs no context and calls neither cudaMalloc nor
 * cudaFree nor any allocating library routine: the scratch for the first layer's split-K partial
 * sums is a fixed 4 MiB (+256 B) array inside the library image, held by every GPU that has
 * loaded the library's device code until the process exits (CUDA loads that code lazily: on a device
 * that has not run anything of this library yet, the first call is what places the array, and it can
 * fail with EGTP_ERR_CUDA if the device's memory is exhausted at that moment, so make one warm-up call
 * at start-up).
 * Computes y_out[r] = head(z[r]) for r < rows exactly as egtp_predict / plp_step do for their
 * pooled vectors (Eq. 6 in bins mode), on the CURRENT device.
 *   head      host struct with device pointers, as above
 *   z         device, float [rows][ldz], ldz >= d, ldz % 4 == 0, 16-byte aligned
 *   rows      rows * head->m_h must not exceed 1048576 (2^20) floats of scratch;
 *             beyond that the call returns EGTP_ERR_CAPACITY and launches nothing
 *   y_out     device, float [rows]
 *   phat_out  device, float [rows][d_out] or NULL (bins mode)
 *   stream    cudaStream_t
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress) and
 * the SM count; make that first call outside any stream capture.  Every call on a device uses
 * the same array: two calls whose kernels may overlap on the GPU (different streams without an
 * ordering between them) race on it, so order them.  The array keeps the previous call's
 * contents; the call clears the one word that must start at zero itself. */
EGTP_API int egtp_head_forward_static(const egtp_head* head, const float* z, int64_t ldz, int32_t rows,
                                      float* y_out, float* phat_out, void* stream);

/* Eq. 2 from logits that already exist in device memory (Sec. 3.1; the paper reuses the
 * activations the model has produced anyway): H_out[i] = entropy of softmax(logits[i][0..V)) in nats.
 * For a serving engine that has just run its own LM head for sampling, this replaces a second
 * LM-head GEMM by one streaming pass over the logits.
 *   logits  device, [rows][ldl] in logits_dtype (EGTP_F32 or EGTP_BF16), ldl >= V, rows start on
 *           16-byte boundaries; rows <= max(max_tokens, max_batch) of the context
 *   H_out   device, float [rows]
 * status_dev and stream as in egtp_predict. */
EGTP_API int egtp_entropy_from_logits(egtp_ctx* ctx, const void* logits, int64_t ldl, int32_t logits_dtype,
                                      int64_t rows, int32_t V, float* H_out, int32_t* status_dev, void* stream);

/* plp_step (Sec. 3.3, Eq. 8) with the new tokens' entropies taken from logits in memory instead
 * of an LM-head GEMM: logits [B_live][ldl] as above; hidden_step [B_live][ldh] in hidden_dtype with
 * d = the state's hidden size.  Everything else (slots, resets, EGTP source table, outputs, status,
 * stream) is as in plp_step. */
EGTP_API int plp_step_from_logits(egtp_ctx* ctx, plp_state* st, const void* logits, int64_t ldl,
                                  int32_t logits_dtype, int32_t V, const egtp_head* head,
                                  const void* hidden_step, int64_t ldh, int32_t hidden_dtype,
                                  const int32_t* slot_ids, const int32_t* reset_src,
                                  const float* src_m, const float* src_s, const float* src_pooled, int32_t n_src,
                                  int32_t B_live, float alpha,
                                  float* Hstep_out, float* z_out, float* yrem_out,
                                  int32_t* status_dev, void* stream);

/* Vocabulary-parallel form of Eq. 2 for LM heads that are sharded over several GPUs (tensor-parallel
 * serving): each GPU holds the rows [v0, v1) of W and can only see its part of every token's
 * distribution.  A shard reduces its part to one triple per token,
 *   m = max_v x_v,  s = sum_v 2^((x_v - m) log2 e),  t2 = sum_v 2^(..) * (x_v - m) log2 e,
 * the ranks exchange the triples (one all-gather of rows * 3 floats per rank: the path's only
 * collective, done by the caller, e.g. with NCCL), and every rank merges them: triples of disjoint
 * vocabulary ranges combine exactly like the per-chunk partials inside one GPU.
 *
 * egtp_entropy_partials: partial_out (device, float [rows][3]) for this GPU's shard `lm_shard`
 *   (W pointing at the shard's first row, V = rows of the shard), hidden [rows][ldh] as in egtp_predict.
 * egtp_entropy_from_partials: gathered (device, float [num_shards][rows][3], rank-major as an
 *   all-gather leaves it) -> H_out (device, float [rows]).
 * plp_step_from_partials: plp_step with the step's entropies taken from such gathered triples
 *   (gathered [num_shards][B_live][3]); all other arguments as in plp_step_from_logits. */
EGTP_API int egtp_entropy_partials(egtp_ctx* ctx, const egtp_lm_head* lm_shard, const void* hidden, int64_t ldh,
                                   int64_t rows, float* partial_out, int32_t* status_dev, void* stream);
EGTP_API int egtp_entropy_from_partials(egtp_ctx* ctx, const float* gathered, int32_t num_shards, int64_t rows,
                                        float* H_out, int32_t* status_dev, void* stream);
EGTP_API int plp_step_from_partials(egtp_ctx* ctx, plp_state* st, const float* gathered, int32_t num_shards,
                                    const egtp_head* head, const void* hidden_step, int64_t ldh, int32_t hidden_dtype,
                                    const int32_t* slot_ids, const int32_t* reset_src,
                                    const float* src_m, const float* src_s, const float* src_pooled, int32_t n_src,
                                    int32_t B_live, float alpha,
                                    float* Hstep_out, float* z_out, float* yrem_out,
                                    int32_t* status_dev, void* stream);

/* The pooling alternatives the paper compares EGTP against (ablation, Table 3): average pooling,
 * max pooling and last-token pooling over the same ragged batch, followed by the same head.  No LM
 * head and no entropy are involved.  An empty prompt pools to zero.
 *   hidden      device, [T_total][ldh] rows in `dtype` (EGTP_F32 / EGTP_BF16), d a multiple of 16
 *   offsets     device, int32 [B+1], as in egtp_predict (checked on the device)
 *   mode        EGTP_POOL_MEAN, EGTP_POOL_MAX or EGTP_POOL_LAST
 *   pooled_out  device, float [B][d] or NULL;  yhat_out device, float [B] or NULL (needs head)
 * status_dev and stream as in egtp_predict. */
enum { EGTP_POOL_MEAN = 1, EGTP_POOL_MAX = 2, EGTP_POOL_LAST = 3 };
EGTP_API int egtp_pool_baseline(egtp_ctx* ctx, const egtp_head* head, const void* hidden, int64_t ldh,
                                int32_t dtype, int32_t d, const int32_t* offsets, int32_t B, int64_t T_total,
                                int32_t mode, float* pooled_out, float* yhat_out,
                                int32_t* status_dev, void* stream);

/* Tile shape of the LM-head kernel (Sec. 3.1, Eq. 2).
 *   EGTP_LMHEAD_AUTO (default): one CTA per SM on 128 x 256 tiles for prompt batches and for up to 128 rows;
 *     batches of 129..256 rows (decode steps) run as clusters of two CTAs on 256 x 512 tiles with
 *     tcgen05.mma.cta_group::2: every SM then loads half of the hidden rows per 512 instead of 256 vocabulary
 *     columns, a quarter less operand traffic per flop where the step is bound by streaming W (measured
 *     4 % faster per decode step than the one-CTA form, in short bursts and sustained).
 *   EGTP_LMHEAD_CTA_PAIRS: CTA pairs for prompt batches too (256 x 256 tiles).  On a power-capped B200 this
 *     measured equal or slower than AUTO for prompts, so it is an option.
 *   EGTP_LMHEAD_SINGLE_CTA: never use CTA pairs (129..256 rows then run both row tiles in one CTA).
 *   fp32 inputs always run one CTA per SM, whatever the mode: each operand is split into two tf32 parts in shared
 *   memory and every k step issues three MMAs (hi.hi + hi.lo + lo.hi), so that the logits keep fp32-level accuracy.
 *   EGTP_LMHEAD_CTA_PAIRS_WIDE: CTA pairs on 256 x 512 tiles for prompt batches too (the decode tile shape): half
 *     the operand bytes an SM pulls in per flop, one accumulator set (the epilogue of a tile does not overlap the next
 *     tile's MMAs).
 * All modes give the same entropies up to summation order. */
enum { EGTP_LMHEAD_AUTO = 0, EGTP_LMHEAD_CTA_PAIRS = 1, EGTP_LMHEAD_SINGLE_CTA = 2, EGTP_LMHEAD_CTA_PAIRS_WIDE = 3 };
EGTP_API int egtp_set_lmhead_mode(egtp_ctx* ctx, int mode);

/* Tuning knob for prompt batches (more than 256 rows): the LM-head kernel cuts the vocabulary into `chunks`
 * ranges and deals (row block, range) units to the SMs round-robin; every range costs one partial (m, s, t2) per
 * row and column half (Eq. 2 is merged from them).  0 (default) lets the library choose the smallest count whose
 * rounds x tiles-per-range product is close to the best reachable (within 0.5 % for rows of up to 4 KB, 2 % for
 * longer rows); a positive value forces that count (clamped to what the workspace holds).  Results do not depend
 * on it beyond summation order. */
EGTP_API int egtp_set_lmhead_chunks(egtp_ctx* ctx, int32_t chunks);

/* Launch overlap (on by default).  The LM-head kernel and the kernel that finishes a PLP step on a state bound to
 * its head are launched with programmatic stream serialization: their blocks are set up (barriers, tensor memory,
 * state rows read ahead) while the kernel before them in the stream is still finishing, and each waits for that
 * kernel's end before it reads anything the stream wrote earlier or writes anything the stream may still read.
 * Results are identical either way; on = 0 launches them plainly (per-kernel event timing does the same while it
 * is enabled, because an overlapped start would be charged to the kernel before). */
EGTP_API int egtp_set_launch_overlap(egtp_ctx* ctx, int on);

/* Failure-detection self-test.  Every wait inside the pipeline kernels (on an mbarrier fed by TMA, by the
 * tensor core or by another warp) is bounded: when its limit runs out the kernel writes
 * EGTP_ERR_DEVICE_TIMEOUT to the status word, releases its tensor memory and returns, so a protocol
 * fault becomes an error code instead of a hung GPU.  This call runs the same wait primitive on a
 * barrier that nothing ever signals, with a limit of limit_ms (1..1000) milliseconds: afterwards
 * *status_dev (device, int32, zeroed by the caller) holds EGTP_ERR_DEVICE_TIMEOUT and the context
 * is usable as before. */
EGTP_API int egtp_selftest_wait_timeout(egtp_ctx* ctx, int32_t limit_ms, int32_t* status_dev, void* stream);

/* Per-kernel timing. With profiling on, every kernel launch of this context is bracketed by
 * CUDA events on its own stream.  egtp_profile_read synchronises the device, adds up the
 * elapsed milliseconds and launch counts per kernel since the last read and clears them.
 * Kernel ids index the two output arrays (host pointers, EGTP_NUM_KERNELS entries each). */
enum {
  EGTP_K_VALIDATE = 0,      /* offsets check as a kernel of its own (normally part of the merge) */
  EGTP_K_LMHEAD_ENTROPY,    /* tcgen05 LM-head GEMM with the online entropy epilogue */
  EGTP_K_ENTROPY_MERGE,     /* merge of per-vocabulary-chunk partials into H, offsets check, unnormalised Eq. 3 weights */
  EGTP_K_TOKEN_WEIGHTS,     /* normalised Eq. 3 weights, only when the caller asks for them */
  EGTP_K_POOL,              /* Eq. 4, first stage */
  EGTP_K_POOL_COMBINE,      /* Eq. 3-4, deterministic combine of prompts that span chunks, (M, Z), head input */
  EGTP_K_HEAD_HIDDEN,       /* head layer 1 */
  EGTP_K_HEAD_OUT,          /* head layer 2 + output mode */
  EGTP_K_PLP_UPDATE,        /* PLP running-state update */
  EGTP_K_LOGITS_ENTROPY,    /* Eq. 2 from logits already in memory */
  EGTP_K_STAGE_ROWS,        /* batches of fewer than 16 rows copied into a zero-padded 16-row buffer */
  EGTP_NUM_KERNELS
};
EGTP_API int egtp_profile_enable(egtp_ctx* ctx, int on);
EGTP_API int egtp_profile_read(egtp_ctx* ctx, double* ms_by_kernel, int64_t* launches_by_kernel);
EGTP_API const char* egtp_kernel_name(int kernel_id);

/* Total number of kernels this context has launched since it was created. */
EGTP_API int64_t egtp_launch_count(const egtp_ctx* ctx);

/* Launch shape the LM-head kernel uses for T rows of hidden size d against V vocabulary rows:
 * info[0] = grid (CTAs), [1] = row blocks, [2] = rows per block (128 or 256), [3] = vocabulary
 * chunks, [4] = partial slots per row, [5] = vocabulary columns per tile, [6] = k blocks,
 * [7] = dynamic shared memory bytes.  Host pointer; nothing is launched. */
EGTP_API int egtp_lmhead_plan(const egtp_ctx* ctx, int64_t T, int32_t d, int32_t V, int32_t dtype, int32_t info[8]);

/* The same plan without a context or a GPU: for a device with num_sms SMs that can co-schedule pair_workers
 * clusters of two CTAs (0 = none; a B200 has 148 SMs and 74 pairs), a context sized for exactly T rows, and
 * head_cols head columns riding along (0 = none; the m_h of a bound state, Sec. 3.2-3.3).  info[0..7] as above,
 * [8] = kernel form (0 prompt shape, 1 / 2 one-CTA decode shapes for <= 128 / <= 256 rows, 4 / 5 CTA pairs for
 * prompts / decode), [9] = row blocks that sweep the vocabulary together, [10] = column granularity of the
 * vocabulary split, [11] = number of such column groups (head columns included).  Pure host arithmetic. */
EGTP_API int egtp_lmhead_plan_for(int32_t num_sms, int32_t pair_workers, int64_t T, int32_t d, int32_t V, int32_t dtype,
                                  int32_t mode, int32_t head_cols, int32_t info[12]);

#ifdef __cplusplus
}
#endif
#endif /* EGTP_H_ */
