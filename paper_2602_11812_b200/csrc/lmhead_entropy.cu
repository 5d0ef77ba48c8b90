// LM-head GEMM with an online entropy epilogue (paper Sec. 3.1, Eq. 2).
//
// For every token row i the kernel needs H_i = -sum_v p_v ln p_v with p = softmax(W h_i).
// Logit tiles (128 rows x 256 vocabulary entries, fp32) are produced by tcgen05.mma into
// tensor memory and consumed there: the epilogue folds each tile into a per-row running
// (m, s, t2) = (max logit, sum 2^y, sum 2^y * y) with y = (x - m) log2 e, so the T x V logits
// never reach shared or global memory.  H = ln s - ln2 * t2 / s is formed by the merge kernel
// from the per-vocabulary-chunk partials written here.
//
// One persistent CTA per SM, warp-specialised:
//   warp 0      TMA producer: streams hidden tiles and W tiles (rows of 128 bytes, 128-byte swizzle,
//               K-major) through a 4-stage shared-memory ring
//   warp 1      MMA issuer (one thread) and owner of the TMEM allocation (512 columns = two
//               256-column fp32 accumulator sets, so the epilogue of tile j overlaps the MMAs of j+1)
//   warps 2..9  epilogue: TMEM lane quadrant = warp % 4, accumulator column half = (warp - 2) / 4;
//               one row per thread, 128 columns per tile, tcgen05.ld in 32-column pieces
// A work unit is (row block, vocabulary chunk); units are ordered so that CTAs running at the
// same time share W tiles (same chunk, neighbouring row blocks) and hidden tiles stay in L2.
// One-CTA tile shapes: prompts (128 rows x 256 columns per tile, tensor-bound), and two decode shapes
// for <= 128 and <= 256 rows, where the step is bound by streaming W from HBM once: every SM
// gets its own vocabulary range (equal to within 32 columns) and, for 129..256 rows, multiplies
// both row tiles against each W tile it loads.  The CTA-pair kernel further down (tcgen05.mma.cta_group::2)
// is the default for 129..256 rows (256 x 512 tiles) and an option for prompts (256 x 256 or 256 x 512 tiles).
// fp32 inputs (prompt shape and the <= 128-row decode shape only): every operand is split in shared memory into two
// tf32 parts and each k step issues three MMAs, which keeps the logits at fp32-level accuracy.
// Both kernels are launched with programmatic stream serialization: what comes before griddepcontrol.wait touches
// only the block's own shared and tensor memory.
//
// Two more uses of the same machinery (prediction head, Sec. 3.2; PLP, Sec. 3.3): with kFuse the column space
// continues past the vocabulary with the rows of the head's W1, whose products are written out instead of
// entering the entropy; and a launch over those head columns alone, with K split over the SMs, is layer 1 of
// the head for any batch of input rows (bf16 rows, or fp32 rows given as two bf16 halves along K).
#include "kernels.h"
#include "sm100_ptx.cuh"
#include "../../include/egtp.h"

#include <algorithm>
#include <type_traits>


namespace egtp {

namespace {

constexpr int kBarrierBytes = 256;
constexpr uint32_t kTmemCols = 512;
constexpr float kLog2e = 1.4426950408889634f;
constexpr int kMaxStages = 8;

struct UnitCoord {
  int row_block;
  int chunk;
  int col_begin;
  int col_end;
  int kb_begin, kb_end;   // k blocks of this unit (all of them unless the launch splits K)
  int k_split;
};

struct KParams {
  int row_blocks, chunks, group_rb, k_blocks;
  int n_groups, col_gran;      // the vocabulary is split at multiples of col_gran columns
  int total_units;
  int V;
  int slots;
  float* partials;
  int32_t* status;
  // head columns appended to the vocabulary (fused form only): column v_pad + j is row j of the head's W1
  int v_pad;          // first head column: V rounded up to col_gran
  int ldg;            // floats per row of head_g (head columns rounded up to col_gran)
  float* head_g;      // [k_splits][rows_pad][ldg]: sum over splits of head_g[s][i][j] = W1[j] . hidden[i]
  // K split (one-CTA kernel with head columns only; 1 = none): unit u covers k blocks
  // [(u % k_splits) * kb_per_split, ...) of the unit u / k_splits and writes its own slice of head_g
  int k_splits, kb_per_split;
  int64_t g_split_stride;
  // > 0: the matrices behind map_b / map_c have only this many k blocks and are read again from their start
  // after that (A = [x_hi | x_lo], two bf16 halves of fp32 rows, multiplied against the same W1 twice)
  int b_k_blocks;
};

__device__ __forceinline__ UnitCoord unit_coord(int u_in, const KParams& p) {
  UnitCoord c;
  int u = u_in;
  if (p.k_splits > 1) {
    u = u_in / p.k_splits;
    c.k_split = u_in - u * p.k_splits;
    c.kb_begin = c.k_split * p.kb_per_split;
    c.kb_end = min(p.k_blocks, c.kb_begin + p.kb_per_split);
  } else {
    c.k_split = 0;
    c.kb_begin = 0;
    c.kb_end = p.k_blocks;
  }
  const int per_group = p.group_rb * p.chunks;
  const int g = u / per_group;
  const int r = u - g * per_group;
  const int gm = min(p.group_rb, p.row_blocks - g * p.group_rb);
  c.chunk = r / gm;
  c.row_block = g * p.group_rb + (r - c.chunk * gm);
  c.col_begin = static_cast<int>((static_cast<int64_t>(c.chunk) * p.n_groups) / p.chunks) * p.col_gran;
  c.col_end = static_cast<int>((static_cast<int64_t>(c.chunk + 1) * p.n_groups) / p.chunks) * p.col_gran;
  return c;
}

// Running per-row entropy state over the columns seen so far, in base-2 exponent units.
struct RowState {
  float m;
  float s[4];
  float t[4];
  __device__ __forceinline__ void init() {
    m = kNegBig;
#pragma unroll
    for (int i = 0; i < 4; ++i) { s[i] = 0.f; t[i] = 0.f; }
  }
  // Folds 32 logits in. With kMasked, only the first `valid` (>= 1) columns exist (the piece
  // straddles the end of the vocabulary or of the tile); the rest are ignored.
  template <bool kMasked>
  __device__ __forceinline__ void fold(const uint32_t (&raw)[32], int valid) {
    float x[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) x[j] = (!kMasked || j < valid) ? __uint_as_float(raw[j]) : kNegBig;
    float cmax = x[0];
#pragma unroll
    for (int j = 1; j < 32; ++j) cmax = fmaxf(cmax, x[j]);
    if (cmax > m) {
      // new running max: s <- s r, t2 <- r (t2 + dm s) with dm = (m - cmax) log2 e, r = 2^dm
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
    for (int j = 0; j < 32; ++j) {
      const float y = fmaf(x[j], kLog2e, neg_m_l2);
      const float e = ex2_approx(y);
      s[j & 3] += e;
      t[j & 3] = fmaf(e, y, t[j & 3]);
    }
  }
  __device__ __forceinline__ void fold_n(const uint32_t (&raw)[32], int valid) {
    if (valid >= 32) fold<false>(raw, 32); else fold<true>(raw, valid);
  }
};

// One piece of an accumulator row: 32 columns starting at column c0 of the (extended) column space, of which the
// first `produced` were computed and belong to this warp's span.  Without kFuse they are vocabulary columns (the
// caller has already cut `produced` at V).  With kFuse, columns from p.v_pad on are rows of the prediction head's
// W1 (Sec. 3.2) and are written to p.head_g as they are; columns between V and v_pad are padding.
template <bool kFuse>
__device__ __forceinline__ void consume_piece(RowState& st, const uint32_t (&buf)[32], int c0, int produced,
                                              const KParams& p, int64_t row, int k_split = 0) {
  if constexpr (kFuse) {
    if (c0 >= p.v_pad) {
      float4* dst = reinterpret_cast<float4*>(p.head_g + k_split * p.g_split_stride + row * p.ldg + (c0 - p.v_pad));
#pragma unroll
      for (int q = 0; q < 8; ++q)
        dst[q] = make_float4(__uint_as_float(buf[4 * q]), __uint_as_float(buf[4 * q + 1]),
                             __uint_as_float(buf[4 * q + 2]), __uint_as_float(buf[4 * q + 3]));
    } else {
      const int valid = min(produced, p.V - c0);
      if (valid > 0) st.fold_n(buf, valid);
    }
  } else {
    st.fold_n(buf, produced);
  }
}

// kMT   row tiles (of 128 rows) a CTA multiplies against every W tile it loads: 1 for prompt
//       batches, 2 for decode batches of 129..256 rows (each W byte is then fetched once per GPU)
// kBN   vocabulary columns per tile; kMT * kBN TMEM columns per accumulator set (256: two sets, 512: one)
// kBBox rows of one TMA box of W (kBN for the tensor-bound shape; 32 for decode shapes, whose
//       vocabulary ranges end on 32-column boundaries so that all SMs get equal shares)
// kFuse the column space continues past the vocabulary with the rows of a second matrix (map_c: the
//       prediction head's W1, Sec. 3.2); the accumulators of those columns are written to p.head_g as they
//       are instead of entering the entropy.  Layer 1 of the head is linear before its ReLU, so W1 h' for
//       the step's new tokens is all a PLP step needs to advance W1 acc (Sec. 3.3) without a second GEMM.
template <bool kTf32, int kMT, int kBN, int kBBox, int kNumStages, bool kFuse>
__global__ void __launch_bounds__(kLmheadThreads, 1)
lmhead_entropy_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                      const __grid_constant__ CUtensorMap map_b_tile, const __grid_constant__ CUtensorMap map_c,
                      const __grid_constant__ CUtensorMap map_c_tile, const KParams p) {
  // map_b / map_c: boxes of kBBox rows of W / W1; map_b_tile / map_c_tile: boxes of kBN rows (a whole tile in
  // one copy; the same maps when kBBox == kBN)
  constexpr int kABytes = kMT * kTileM * kRowBytes;
  constexpr int kBBytes = kBN * kRowBytes;
  // fp32 operands: a stage holds the tiles twice, as loaded (turned into their high parts in place) and their low parts
  constexpr int kStageBytes = (kTf32 ? 2 : 1) * (kABytes + kBBytes);
  constexpr int kAccCols = kMT * kBN;                 // TMEM columns of one accumulator set
  constexpr int kNumAcc = kTmemCols / kAccCols;       // 2: epilogue of tile j overlaps MMAs of tile j+1; 1 for 256 x 256 tiles
  constexpr int kSpan = kAccCols / kEpiSplit;         // TMEM columns one epilogue warp reads per tile
  static_assert((kAccCols == 256 || kAccCols == 512) && kBN <= 256, "accumulator sets of 256 or 512 TMEM columns");
  static_assert(kNumStages <= kMaxStages && kBN % kBBox == 0 && kBBox % 8 == 0, "bad tile configuration");
  static_assert(kStageBytes % 1024 == 0 && kABytes % 1024 == 0, "stages must keep 1024-byte alignment");

  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bar_base = smem_base + kNumStages * kStageBytes;
  // barrier layout (8 bytes each): full[kMaxStages], empty[kMaxStages], acc_full[2], acc_empty[2]
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kMaxStages + s); };
  auto acc_full_bar = [&](int a) { return bar_base + 8u * (2 * kMaxStages + a); };
  auto acc_empty_bar = [&](int a) { return bar_base + 8u * (2 * kMaxStages + 2 + a); };
  volatile uint32_t* tmem_slot =
      reinterpret_cast<volatile uint32_t*>(smem_gen + kNumStages * kStageBytes + 8 * (2 * kMaxStages + 4));
  volatile uint32_t* abort_flag = tmem_slot + 1;
  volatile uint32_t* skip_flag = tmem_slot + 2;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  // This kernel may have been started (programmatic dependent launch) while the kernel before it in the stream is
  // still finishing: everything up to pdl_wait() below touches only this block's shared and tensor memory and the
  // kernel's own parameters.

  if (threadIdx.x == 0) {
    for (int s = 0; s < kNumStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < kNumAcc; ++a) {
      mbar_init(acc_full_bar(a), 1);
      mbar_init(acc_empty_bar(a), 4 * kEpiSplit);
    }
    *abort_flag = 0u;
    mbar_fence_init();
    tma_prefetch_descriptor(&map_a);
    tma_prefetch_descriptor(&map_b);
    if (kBBox < kBN) tma_prefetch_descriptor(&map_b_tile);
    if (kFuse) tma_prefetch_descriptor(&map_c);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  // From here on the kernel reads what earlier work in the stream wrote (hidden rows, the status word) and writes
  // what that work may still be reading (the partials).
  pdl_wait();
  // Only now may the kernel after this one be staged on SMs this grid has left (it waits for this grid's end before it
  // reads anything written here, but it reads its own state rows ahead: those must be final, which they are once
  // the work before this kernel has completed).
  pdl_launch_dependents();
  // An earlier step of this call failed: do nothing.  One thread reads the word so that the
  // whole block takes the same decision.
  if (threadIdx.x == 0) *skip_flag = (*p.status != 0) ? 1u : 0u;
  __syncthreads();
  const bool skip = *skip_flag != 0u;

  constexpr int kElemsPerStage = kTf32 ? kRowBytes / 4 : kRowBytes / 2;   // K elements per stage
  constexpr int kMmaPerStage = 4;                                         // 32 bytes of K per MMA
  constexpr uint32_t kIdescNoN = umma_idesc(kTf32 ? 2u : 1u, kTileM, 0);  // N is filled in per tile

  if (skip) {
    // nothing to do
  } else if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < p.total_units && ok; u += gridDim.x) {
        const UnitCoord uc = unit_coord(u, p);
        for (int n0 = uc.col_begin; n0 < uc.col_end && ok; n0 += kBN) {
          const int ncols = min(kBN, uc.col_end - n0);
          // A full tile that lies wholly in W or wholly in W1 is fetched with one copy, a ragged tile (the end of
          // an SM's column range, or a tile that straddles v_pad) box by box, each box from the matrix its rows
          // belong to.  Every source gets a copy loop of its own: a tensor-map address picked per copy at run
          // time made the copy instruction issue twice and cost a quarter of the decode step.
          const bool in_w1 = kFuse && n0 >= p.v_pad;
          const bool whole = kBBox < kBN && ncols == kBN && (!kFuse || in_w1 || n0 + kBN <= p.v_pad);
          const int b_loads = whole ? kBN / kBBox : (ncols + kBBox - 1) / kBBox;
          const int b_loads_w = kFuse ? max(0, min(b_loads, (p.v_pad - n0) / kBBox)) : b_loads;   // boxes from W
          const uint32_t tx_bytes = kABytes + b_loads * kBBox * kRowBytes;
          // kSource 0: whole tile of W, 1: whole tile of W1, 2: boxes
          auto stream_tile = [&](auto source) {
            constexpr int kSource = decltype(source)::value;
            for (int kb = uc.kb_begin; kb < uc.kb_end; ++kb) {
              if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
              const uint32_t a_dst = smem_base + stage * kStageBytes;
              const uint32_t b_dst = a_dst + kABytes;
              const int kx = kb * kElemsPerStage;
              const int kxb = (kFuse && p.b_k_blocks > 0) ? (kb % p.b_k_blocks) * kElemsPerStage : kx;
              mbar_arrive_expect_tx(full_bar(stage), tx_bytes);
              tma_load_2d(a_dst, &map_a, kx, uc.row_block * (kMT * kTileM), full_bar(stage));
              if constexpr (kSource == 0) {
                tma_load_2d(b_dst, &map_b_tile, kxb, n0, full_bar(stage));
              } else if constexpr (kSource == 1) {
                tma_load_2d(b_dst, &map_c_tile, kxb, n0 - p.v_pad, full_bar(stage));
              } else {
                for (int i = 0; i < b_loads_w; ++i)
                  tma_load_2d(b_dst + i * (kBBox * kRowBytes), &map_b, kxb, n0 + i * kBBox, full_bar(stage));
                if constexpr (kFuse) {
                  for (int i = b_loads_w; i < b_loads; ++i)
                    tma_load_2d(b_dst + i * (kBBox * kRowBytes), &map_c, kxb, n0 + i * kBBox - p.v_pad, full_bar(stage));
                }
              }
              if (++stage == kNumStages) { stage = 0; phase ^= 1u; }
            }
          };
          if (whole && !in_w1) stream_tile(std::integral_constant<int, 0>{});
          else if (kFuse && whole) stream_tile(std::integral_constant<int, 1>{});
          else stream_tile(std::integral_constant<int, 2>{});
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if constexpr (kTf32) {
      // fp32 operands.  kind::tf32 keeps 10 mantissa bits of each operand, which alone would cost the entropy
      // its 1e-3 tolerance once the logits are a few units large.  So every operand x is taken apart as
      // x = hi + lo, hi = x with its 13 low mantissa bits cleared (exact in tf32), lo = x - hi (exact in fp32, then
      // cut to tf32 as well), and each k step issues three MMAs: hi.hi + hi.lo + lo.hi (the dropped lo.lo term is
      // 2^-22 of the product).  The whole warp splits a stage in shared memory once its copy has landed: the high
      // parts replace the loaded values in place, the low parts go to the second half of the stage, same swizzled
      // layout, so the same descriptors (plus an offset) address them.  Conversion of stage s+1 overlaps the MMAs of
      // stage s; this path serves the small fp32 configuration, not the throughput workloads (those are bf16).
      constexpr int kHalfBytes = kABytes + kBBytes;
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < p.total_units && ok; u += gridDim.x) {
        const UnitCoord uc = unit_coord(u, p);
        for (int n0 = uc.col_begin; n0 < uc.col_end && ok; n0 += kBN) {
          const int ncols = min(kBN, uc.col_end - n0);
          const uint32_t idesc = kIdescNoN | (static_cast<uint32_t>(ncols >> 3) << 17);
          ok = __all_sync(0xffffffffu, mbar_wait(acc_empty_bar(acc), acc_phase ^ 1u, abort_flag));
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * kAccCols);
          for (int kb = uc.kb_begin; kb < uc.kb_end; ++kb) {
            ok = __all_sync(0xffffffffu, mbar_wait(full_bar(stage), phase, abort_flag));
            if (!ok) break;
            uint4* hi_p = reinterpret_cast<uint4*>(smem_gen + stage * kStageBytes);
            uint4* lo_p = reinterpret_cast<uint4*>(smem_gen + stage * kStageBytes + kHalfBytes);
            for (int i = lane; i < kHalfBytes / 16; i += 32) {
              const uint4 v = hi_p[i];
              const uint32_t x[4] = {v.x, v.y, v.z, v.w};
              uint32_t h[4], l[4];
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                h[q] = x[q] & 0xFFFFE000u;
                l[q] = __float_as_uint(__uint_as_float(x[q]) - __uint_as_float(h[q])) & 0xFFFFE000u;
              }
              hi_p[i] = make_uint4(h[0], h[1], h[2], h[3]);
              lo_p[i] = make_uint4(l[0], l[1], l[2], l[3]);
            }
            fence_proxy_async_shared();      // the MMAs read shared memory through the async proxy
            __syncwarp();
            if (lane == 0) {
              tc_fence_after_sync();
              const uint32_t a_src = smem_base + stage * kStageBytes;
              const uint64_t b_hi = umma_desc_k_major_sw128(a_src + kABytes);
              const uint64_t b_lo = umma_desc_k_major_sw128(a_src + kHalfBytes + kABytes);
#pragma unroll
              for (int mt = 0; mt < kMT; ++mt) {
                const uint64_t a_hi = umma_desc_k_major_sw128(a_src + mt * (kTileM * kRowBytes));
                const uint64_t a_lo = umma_desc_k_major_sw128(a_src + kHalfBytes + mt * (kTileM * kRowBytes));
#pragma unroll
                for (int k = 0; k < kMmaPerStage; ++k) {
                  umma_ss<true>(d_tmem + mt * kBN, a_lo + 2u * k, b_hi + 2u * k, idesc, (kb != uc.kb_begin || k != 0) ? 1u : 0u);
                  umma_ss<true>(d_tmem + mt * kBN, a_hi + 2u * k, b_lo + 2u * k, idesc, 1u);
                  umma_ss<true>(d_tmem + mt * kBN, a_hi + 2u * k, b_hi + 2u * k, idesc, 1u);
                }
              }
              umma_commit(empty_bar(stage));
            }
            __syncwarp();
            if (++stage == kNumStages) { stage = 0; phase ^= 1u; }
          }
          if (ok && lane == 0) umma_commit(acc_full_bar(acc));
          __syncwarp();
          if (++acc == kNumAcc) { acc = 0; acc_phase ^= 1u; }
        }
      }
    } else if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < p.total_units && ok; u += gridDim.x) {
        const UnitCoord uc = unit_coord(u, p);
        for (int n0 = uc.col_begin; n0 < uc.col_end && ok; n0 += kBN) {
          const int ncols = min(kBN, uc.col_end - n0);
          const uint32_t idesc = kIdescNoN | (static_cast<uint32_t>(ncols >> 3) << 17);
          if (!mbar_wait(acc_empty_bar(acc), acc_phase ^ 1u, abort_flag)) { ok = false; break; }
          tc_fence_after_sync();
          const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * kAccCols);
          for (int kb = uc.kb_begin; kb < uc.kb_end; ++kb) {
            if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t a_src = smem_base + stage * kStageBytes;
            const uint64_t b_desc = umma_desc_k_major_sw128(a_src + kABytes);
#pragma unroll
            for (int mt = 0; mt < kMT; ++mt) {
              const uint64_t a_desc = umma_desc_k_major_sw128(a_src + mt * (kTileM * kRowBytes));
#pragma unroll
              for (int k = 0; k < kMmaPerStage; ++k) {
                // advancing K by 32 bytes inside the swizzled row = +2 in the (address >> 4) field
                umma_ss<kTf32>(d_tmem + mt * kBN, a_desc + 2u * k, b_desc + 2u * k, idesc,
                               (kb != uc.kb_begin || k != 0) ? 1u : 0u);
              }
            }
            umma_commit(empty_bar(stage));          // stage reusable once these MMAs have read it
            if (++stage == kNumStages) { stage = 0; phase ^= 1u; }
          }
          if (ok) umma_commit(acc_full_bar(acc));   // accumulator complete
          if (++acc == kNumAcc) { acc = 0; acc_phase ^= 1u; }
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    // Warp (quad, half) reads TMEM lanes 32*quad.. and accumulator columns [half*kSpan, (half+1)*kSpan):
    // with kMT == 1 that is one half of the tile's 256 vocabulary columns, with kMT == 2 the whole
    // tile of row tile `half`.
    const int quad = warp & 3;
    const int half = (warp - 2) >> 2;
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int u = blockIdx.x; u < p.total_units && ok; u += gridDim.x) {
      const UnitCoord uc = unit_coord(u, p);
      const int64_t row = (static_cast<int64_t>(uc.row_block) * kMT + (kMT == 1 ? 0 : half)) * kTileM + quad * 32 + lane;
      RowState st;
      st.init();
      for (int n0 = uc.col_begin; n0 < uc.col_end; n0 += kBN) {
        ok = __all_sync(0xffffffffu, mbar_wait(acc_full_bar(acc), acc_phase, abort_flag));
        if (!ok) break;
        tc_fence_after_sync();
        // tile columns this warp has to look at: all that were computed in the fused form (head columns
        // lie beyond V), otherwise only those that exist in the vocabulary
        const int tile_cols = min(kBN, uc.col_end - n0);
        const int ncols = kFuse ? tile_cols : min(tile_cols, p.V - n0);
        const int cols_valid = (kMT == 1) ? min(kSpan, ncols - half * kSpan) : ncols;   // of this warp's span
        const int npieces = cols_valid > 0 ? (cols_valid + 31) >> 5 : 0;
        const int c_base = n0 + (kMT == 1 ? half * kSpan : 0);                          // first column of the span
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) +
                               static_cast<uint32_t>(acc * kAccCols + half * kSpan);
        auto release = [&]() {
          // every read of the accumulator by this warp has completed: hand it back to the MMA warp
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(acc_empty_bar(acc));
        };
        // piece pc = 32 accumulator columns starting at vocabulary / head column c_base + 32 pc
        auto consume = [&](const uint32_t (&buf)[32], int pc) {
          consume_piece<kFuse>(st, buf, c_base + pc * 32, cols_valid - pc * 32, p, row, uc.k_split);
        };
        uint32_t bufA[32], bufB[32];
        if (npieces == 0) {
          release();
        } else {
          // software pipeline: the load of piece i+1 is in flight while piece i is folded
          tmem_ld_32(taddr, bufA);
          tmem_ld_wait(bufA);
          for (int pc = 0; pc < npieces; pc += 2) {
            const bool has1 = pc + 1 < npieces;
            if (has1) tmem_ld_32(taddr + (pc + 1) * 32, bufB); else release();
            consume(bufA, pc);
            if (has1) {
              tmem_ld_wait(bufB);
              const bool has2 = pc + 2 < npieces;
              if (has2) tmem_ld_32(taddr + (pc + 2) * 32, bufA); else release();
              consume(bufB, pc + 1);
              if (has2) tmem_ld_wait(bufA);
            }
          }
        }
        if (++acc == kNumAcc) { acc = 0; acc_phase ^= 1u; }
      }
      if (ok && p.partials != nullptr) {     // no partials: a launch that only projects onto head columns
        const int slot = (kMT == 1) ? uc.chunk * kEpiSplit + half : uc.chunk;
        float* dst = p.partials + (row * p.slots + slot) * 3;
        dst[0] = st.m;
        dst[1] = (st.s[0] + st.s[1]) + (st.s[2] + st.s[3]);
        dst[2] = (st.t[0] + st.t[1]) + (st.t[2] + st.t[3]);
      }
    }
  }

  // ---------------------------------------------------------------------- teardown
  __syncthreads();
  if (*abort_flag != 0u) {
    if (threadIdx.x == 0) atomicCAS(p.status, 0, EGTP_ERR_DEVICE_TIMEOUT);
    // give copies and MMAs still in flight time to land before shared and tensor memory go away
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 2000000ull) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 1) {
    __syncwarp();
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ---------------------------------------------------------------------------------------------
// CTA-pair form: a cluster of two CTAs (two SMs) works on one 256-row x 256-column tile with
// tcgen05.mma.cta_group::2.  Each CTA loads only its own 128 rows of the hidden states and its own
// half of the W tile, so the bytes an SM has to pull in per flop are halved against the one-CTA
// form (which is limited by the SM's L2 read port, not by the tensor pipe), and each CTA's TMEM
// still holds two 128 x 256 accumulators, so the epilogue keeps overlapping the next tile's MMAs.
//   both CTAs, warp 0   TMA producer for the CTA's own operand halves; completion bytes are counted
//                       on the leader CTA's "full" barrier
//   leader, warp 1      one thread issues the MMAs for both CTAs and commits to the "empty" and
//                       "accumulator full" barriers of both CTAs
//   both CTAs, warp 1   TMEM allocation / release (collective over the pair)
//   both CTAs, 2..9     epilogue on the CTA's own 128 rows; arrivals go to the leader's
//                       "accumulator empty" barrier
// No load in this kernel is multicast; the only multicast is the arrival of tcgen05.commit.
// kNT  256-column subtiles per tile: 1 = 256 x 256 tiles, two accumulator sets; 2 = 256 x 512 tiles (two MMAs of
//      N = 256 per k step into the two halves of one 512-column accumulator set): every 128 rows of hidden states
//      an SM loads then meet 512 instead of 256 vocabulary columns, a quarter less operand traffic per flop, at
//      the price of an epilogue that no longer overlaps the next tile's MMAs
// kFuse as in the one-CTA kernel: the column space continues past the vocabulary with the rows of W1 (map_c)
template <bool kTf32, int kBBox, int kNumStages, int kNT, bool kFuse>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kLmheadThreads, 1)
lmhead_entropy_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                           const __grid_constant__ CUtensorMap map_c, const KParams p) {
  constexpr int kSubN = 256;                      // columns of one MMA over the pair
  constexpr int kBN = kSubN * kNT;                // tile columns over the pair
  constexpr int kABytes = kTileM * kRowBytes;     // this CTA's 128 rows
  constexpr int kSubBBytes = (kSubN / 2) * kRowBytes;   // this CTA's half of one subtile of W
  constexpr int kBBytes = kNT * kSubBBytes;
  constexpr int kStageBytes = kABytes + kBBytes;
  constexpr int kAccCols = kBN;
  constexpr int kNumAcc = kTmemCols / kAccCols;
  static_assert(kNumStages <= kMaxStages && (kSubN / 2) % kBBox == 0 && kBBox % 8 == 0, "bad tile configuration");
  static_assert((kNT == 1 && kNumAcc == 2) || (kNT == 2 && kNumAcc == 1), "two 256-column accumulators or one of 512 columns");

  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bar_base = smem_base + kNumStages * kStageBytes;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kMaxStages + s); };
  auto acc_full_bar = [&](int a) { return bar_base + 8u * (2 * kMaxStages + a); };
  auto acc_empty_bar = [&](int a) { return bar_base + 8u * (2 * kMaxStages + 2 + a); };
  volatile uint32_t* tmem_slot =
      reinterpret_cast<volatile uint32_t*>(smem_gen + kNumStages * kStageBytes + 8 * (2 * kMaxStages + 4));
  volatile uint32_t* abort_flag = tmem_slot + 1;
  volatile uint32_t* skip_flag = tmem_slot + 2;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();        // 0 = leader
  const bool leader = rank == 0;
  const int pair = blockIdx.x >> 1;
  const int num_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kNumStages; ++s) {
      mbar_init(full_bar(s), 1);            // leader: its own arrive.expect_tx (bytes of both CTAs)
      mbar_init(empty_bar(s), 1);           // one commit arrival, delivered to both CTAs
    }
    // 256 x 256 tiles: two accumulator sets, each with its "full" and "empty" barrier.  256 x 512 tiles: one set, one
    // "full" barrier, but an "empty" barrier per 256-column subtile, so that the next tile's MMAs into the first
    // subtile can start while the epilogue is still reading the second
    for (int a = 0; a < 2; ++a) {
      mbar_init(acc_full_bar(a), 1);                    // commit arrival, delivered to both CTAs
      mbar_init(acc_empty_bar(a), 2 * 4 * kEpiSplit);   // leader: the epilogue warps of both CTAs
    }
    *abort_flag = 0u;
    mbar_fence_init();
    tma_prefetch_descriptor(&map_a);
    tma_prefetch_descriptor(&map_b);
    if (kFuse) tma_prefetch_descriptor(&map_c);
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before_sync();
  __syncthreads();
  pdl_wait();                   // see the one-CTA kernel: nothing before this line touched global memory
  pdl_launch_dependents();
  if (threadIdx.x == 0) *skip_flag = (*p.status != 0) ? 1u : 0u;            // an earlier step of this call failed
  cluster_sync_all();           // barriers of both CTAs are initialised before anyone signals across
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  // both CTAs follow the leader's reading of the status word
  const bool skip = ld_shared_cluster_u32(map_to_cta(smem_u32(const_cast<uint32_t*>(skip_flag)), 0)) != 0u;

  constexpr int kElemsPerStage = kTf32 ? kRowBytes / 4 : kRowBytes / 2;
  constexpr int kMmaPerStage = 4;
  constexpr uint32_t kIdescNoN = umma_idesc(kTf32 ? 2u : 1u, 2 * kTileM, 0);   // M = 256 over the pair

  if (skip) {
    // nothing to do
  } else if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int u = pair; u < p.total_units && ok; u += num_pairs) {
        const UnitCoord uc = unit_coord(u, p);
        for (int n0 = uc.col_begin; n0 < uc.col_end && ok; n0 += kBN) {
          const int ncols = min(kBN, uc.col_end - n0);
          // per subtile t: its columns, the W rows this CTA supplies (one half), and the boxes that takes
          int half_cols[kNT], b_loads[kNT];
          uint32_t b_bytes = 0;
#pragma unroll
          for (int t = 0; t < kNT; ++t) {
            const int nc = max(0, min(kSubN, ncols - t * kSubN));
            half_cols[t] = nc >> 1;
            b_loads[t] = (half_cols[t] + kBBox - 1) / kBBox;
            b_bytes += b_loads[t] * kBBox * kRowBytes;
          }
          const uint32_t tx_bytes = 2u * (kABytes + b_bytes);   // both CTAs
          for (int kb = 0; kb < p.k_blocks; ++kb) {
            if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
            const uint32_t a_dst = smem_base + stage * kStageBytes;
            const uint32_t b_dst = a_dst + kABytes;
            const uint32_t full_leader = map_to_cta(full_bar(stage), 0);
            if (leader) mbar_arrive_expect_tx(full_bar(stage), tx_bytes);
            tma_load_2d_pair(a_dst, &map_a, kb * kElemsPerStage, uc.row_block * (2 * kTileM) + rank * kTileM,
                             full_leader);
#pragma unroll
            for (int t = 0; t < kNT; ++t) {
              // this CTA's rows of subtile t start at r0; boxes below v_pad come from W, the others from W1
              // (a loop per matrix: a tensor-map address picked per copy at run time makes the copy issue twice)
              const int r0 = n0 + t * kSubN + rank * half_cols[t];
              const int from_w = kFuse ? max(0, min(b_loads[t], (p.v_pad - r0) / kBBox)) : b_loads[t];
              for (int i = 0; i < from_w; ++i)
                tma_load_2d_pair(b_dst + t * kSubBBytes + i * (kBBox * kRowBytes), &map_b, kb * kElemsPerStage,
                                 r0 + i * kBBox, full_leader);
              if constexpr (kFuse) {
                for (int i = from_w; i < b_loads[t]; ++i)
                  tma_load_2d_pair(b_dst + t * kSubBBytes + i * (kBBox * kRowBytes), &map_c, kb * kElemsPerStage,
                                   r0 + i * kBBox - p.v_pad, full_leader);
              }
            }
            if (++stage == kNumStages) { stage = 0; phase ^= 1u; }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader only)
    if (leader && lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      // MMAs of k block `stg` of the current tile into subtile t
      auto issue = [&](int stg, int t, const uint32_t (&idesc)[kNT], uint32_t d_tmem, bool first_kb) {
        const uint32_t a_src = smem_base + stg * kStageBytes;
        const uint64_t a_desc = umma_desc_k_major_sw128(a_src);
        const uint64_t b_desc = umma_desc_k_major_sw128(a_src + kABytes + t * kSubBBytes);
#pragma unroll
        for (int k = 0; k < kMmaPerStage; ++k)
          umma_ss_pair<kTf32>(d_tmem + t * kSubN, a_desc + 2u * k, b_desc + 2u * k, idesc[t], (!first_kb || k != 0) ? 1u : 0u);
      };
      for (int u = pair; u < p.total_units && ok; u += num_pairs) {
        const UnitCoord uc = unit_coord(u, p);
        for (int n0 = uc.col_begin; n0 < uc.col_end && ok; n0 += kBN) {
          const int ncols = min(kBN, uc.col_end - n0);
          uint32_t idesc[kNT];
#pragma unroll
          for (int t = 0; t < kNT; ++t)
            idesc[t] = kIdescNoN | (static_cast<uint32_t>(max(0, min(kSubN, ncols - t * kSubN)) >> 3) << 17);
          if constexpr (kNT == 1) {
            if (!mbar_wait(acc_empty_bar(acc), acc_phase ^ 1u, abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * kAccCols);
            for (int kb = 0; kb < p.k_blocks; ++kb) {
              if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
              tc_fence_after_sync();
              issue(stage, 0, idesc, d_tmem, kb == 0);
              umma_commit_pair(empty_bar(stage), 0x3);        // frees the stage in both CTAs
              if (++stage == kNumStages) { stage = 0; phase ^= 1u; }
            }
            if (ok) umma_commit_pair(acc_full_bar(acc), 0x3); // accumulator complete in both CTAs
            if (++acc == kNumAcc) { acc = 0; acc_phase ^= 1u; }
          } else {
            // One 512-column accumulator set.  The epilogue hands back the first subtile when it is half way through,
            // so the first kLag k blocks are multiplied into the first subtile alone (their stages stay held), then,
            // once the second subtile is free as well, into the second; from there on both per k block.
            constexpr int kLag = kNumStages - 1;
            const bool two = ncols > kSubN;                     // ragged tiles may have no second subtile
            const int lag = min(kLag, p.k_blocks);
            if (!mbar_wait(acc_empty_bar(0), acc_phase ^ 1u, abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            int held = stage;                                   // first of the stages held back
            for (int kb = 0; kb < lag && ok; ++kb) {
              if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
              tc_fence_after_sync();
              issue(stage, 0, idesc, tmem_base, kb == 0);
              if (++stage == kNumStages) { stage = 0; phase ^= 1u; }
            }
            if (!ok) break;
            if (!mbar_wait(acc_empty_bar(1), acc_phase ^ 1u, abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            for (int kb = 0; kb < lag; ++kb) {
              if (two) issue(held, 1, idesc, tmem_base, kb == 0);
              umma_commit_pair(empty_bar(held), 0x3);
              if (++held == kNumStages) held = 0;
            }
            for (int kb = lag; kb < p.k_blocks; ++kb) {
              if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
              tc_fence_after_sync();
              issue(stage, 0, idesc, tmem_base, kb == 0);
              if (two) issue(stage, 1, idesc, tmem_base, kb == 0);
              umma_commit_pair(empty_bar(stage), 0x3);
              if (++stage == kNumStages) { stage = 0; phase ^= 1u; }
            }
            if (ok) umma_commit_pair(acc_full_bar(0), 0x3);
            acc_phase ^= 1u;
          }
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (both CTAs, own rows)
    const int quad = warp & 3;
    const int half = (warp - 2) >> 2;
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int u = pair; u < p.total_units && ok; u += num_pairs) {
      const UnitCoord uc = unit_coord(u, p);
      const int64_t row = static_cast<int64_t>(uc.row_block) * (2 * kTileM) + rank * kTileM + quad * 32 + lane;
      RowState st;
      st.init();
      for (int n0 = uc.col_begin; n0 < uc.col_end; n0 += kBN) {
        ok = __all_sync(0xffffffffu, mbar_wait(acc_full_bar(acc), acc_phase, abort_flag));
        if (!ok) break;
        tc_fence_after_sync();
        const int tile_cols = min(kBN, uc.col_end - n0);
        const int ncols = kFuse ? tile_cols : min(tile_cols, p.V - n0);
        // This warp reads 128 columns of every 256-column subtile (column half `half`) and hands each subtile back
        // as soon as it has read it: with 256 x 512 tiles the first subtile is free again when the epilogue is half way.
        constexpr int kSubSpan = kSubN / kEpiSplit;
#pragma unroll
        for (int sub = 0; sub < kNT; ++sub) {
          const int co = sub * kSubN + half * kSubSpan;             // first column of the span inside the tile
          const int cols_valid = min(kSubSpan, ncols - co);
          const int npieces = cols_valid > 0 ? (cols_valid + 31) >> 5 : 0;
          const int c_base = n0 + co;
          const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) +
                                 static_cast<uint32_t>(acc * kAccCols + co);
          const uint32_t acc_empty_leader = map_to_cta(acc_empty_bar(kNT == 1 ? acc : sub), 0);
          auto release = [&]() {
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(acc_empty_leader);
          };
          auto consume = [&](const uint32_t (&buf)[32], int pc) {
            consume_piece<kFuse>(st, buf, c_base + pc * 32, cols_valid - pc * 32, p, row);
          };
          uint32_t bufA[32], bufB[32];
          if (npieces == 0) {
            release();
          } else {
            tmem_ld_32(taddr, bufA);
            tmem_ld_wait(bufA);
            for (int pc = 0; pc < npieces; pc += 2) {
              const bool has1 = pc + 1 < npieces;
              if (has1) tmem_ld_32(taddr + (pc + 1) * 32, bufB); else release();
              consume(bufA, pc);
              if (has1) {
                tmem_ld_wait(bufB);
                const bool has2 = pc + 2 < npieces;
                if (has2) tmem_ld_32(taddr + (pc + 2) * 32, bufA); else release();
                consume(bufB, pc + 1);
                if (has2) tmem_ld_wait(bufA);
              }
            }
          }
        }
        if (++acc == kNumAcc) { acc = 0; acc_phase ^= 1u; }
      }
      if (ok) {
        const int slot = uc.chunk * kEpiSplit + half;
        float* dst = p.partials + (row * p.slots + slot) * 3;
        dst[0] = st.m;
        dst[1] = (st.s[0] + st.s[1]) + (st.s[2] + st.s[3]);
        dst[2] = (st.t[0] + st.t[1]) + (st.t[2] + st.t[3]);
      }
    }
  }

  // ---------------------------------------------------------------------- teardown
  __syncthreads();
  if (*abort_flag != 0u) {
    if (threadIdx.x == 0) atomicCAS(p.status, 0, EGTP_ERR_DEVICE_TIMEOUT);
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 2000000ull) __nanosleep(1000);
    __syncthreads();
  }
  // neither CTA may leave (and give up its shared and tensor memory) while its partner can still signal it
  tc_fence_before_sync();
  cluster_sync_all();
  tc_fence_after_sync();
  if (warp == 1) {
    __syncwarp();
    tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

// fp32 operands: two stages, each holding its tiles twice (high and low parts)
constexpr int kF32Stages = 2;
constexpr int smem_bytes_for(int mt, int bn, int stages, bool f32 = false) {
  return (f32 ? 2 * kF32Stages : stages) * (mt * kTileM * kRowBytes + bn * kRowBytes) + kBarrierBytes + 1024;   // + slack for alignment
}

// The three shapes the host chooses from.
struct Shape { int mt, bn, bbox, stages, col_gran; };   // mt = 128-row tiles per row block (2 in pair forms too)
constexpr Shape kShapePrompt = {1, 256, 256, 4, 256};   // tensor-bound: many row tiles
constexpr Shape kShapeDecode1 = {1, 256, 32, 4, 32};    // <= 128 rows: W streamed once, 32-column balance
constexpr Shape kShapeDecode2 = {2, 256, 32, 3, 32};    // 129..256 rows: both row tiles share each W tile

constexpr Shape kShapePairPrompt = {2, 256, 128, 6, 256};  // CTA pairs, 256 x 256 tiles
constexpr Shape kShapePairDecode = {2, 512, 32, 4, 64};    // CTA pairs, 256 x 512 tiles, one vocabulary range per pair
constexpr Shape kShapePairWide = {2, 512, 32, 4, 512};     // CTA pairs, 256 x 512 tiles, prompt batches
constexpr int kPairStages = 6;         // 256 x 256 tiles: 6 x 32 KB
constexpr int kPairWideStages = 4;     // 256 x 512 tiles: 4 x 48 KB
constexpr int kPairSmemBytes = kPairStages * (kTileM * kRowBytes + 128 * kRowBytes) + kBarrierBytes + 1024;
static_assert(kPairWideStages * (kTileM * kRowBytes + 2 * 128 * kRowBytes) + kBarrierBytes + 1024 == kPairSmemBytes, "both pair forms use the same shared memory");

const Shape& shape_of(int variant) {
  if (variant == 4) return kShapePairPrompt;
  if (variant == 5) return kShapePairDecode;
  if (variant == 6) return kShapePairWide;
  return variant == 1 ? kShapeDecode1 : (variant == 2 ? kShapeDecode2 : kShapePrompt);
}

// overlap: launch with programmatic stream serialization, so that the blocks may be set up (barriers, tensor memory)
// while the kernel before this one in the stream is still finishing; the kernel waits for that kernel's end before
// it touches global memory
struct LaunchConfig {
  cudaLaunchConfig_t cfg{};
  cudaLaunchAttribute attr{};
  LaunchConfig(int grid, int smem_bytes, cudaStream_t stream, bool overlap) {
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kLmheadThreads);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = stream;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = overlap ? 1 : 0;
  }
};

template <bool kTf32, int kMT, int kBN, int kBBox, int kNumStages, bool kFuse = false>
cudaError_t launch_shape(const LmheadPlan& plan, const LmheadMaps& m, const KParams& p, cudaStream_t stream, bool overlap) {
  auto kernel = lmhead_entropy_kernel<kTf32, kMT, kBN, kBBox, kNumStages, kFuse>;
  const CUtensorMap* c = kFuse ? m.w1 : m.w;
  const CUtensorMap* c_tile = kFuse ? m.w1_tile : m.w_tile;
  LaunchConfig lc(plan.grid, smem_bytes_for(kMT, kBN, kNumStages, kTf32), stream, overlap);
  return cudaLaunchKernelEx(&lc.cfg, kernel, *m.hidden, *m.w, *m.w_tile, *c, *c_tile, p);
}

template <bool kTf32, int kMT, int kBN, int kBBox, int kNumStages, bool kFuse = false>
cudaError_t prepare_shape() {
  auto kernel = lmhead_entropy_kernel<kTf32, kMT, kBN, kBBox, kNumStages, kFuse>;
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              smem_bytes_for(kMT, kBN, kNumStages, kTf32));
}

// kBBox 128: 256 x 256 tiles (prompt batches); 32: 256 x 512 tiles (decode batches), optionally with head columns
template <bool kTf32, int kBBox, bool kFuse = false>
cudaError_t launch_pair(const LmheadPlan& plan, const LmheadMaps& m, const KParams& p, cudaStream_t stream, bool overlap) {
  auto kernel = kBBox == 32 ? lmhead_entropy_pair_kernel<kTf32, kBBox, kPairWideStages, 2, kFuse>
                            : lmhead_entropy_pair_kernel<kTf32, kBBox, kPairStages, 1, kFuse>;
  LaunchConfig lc(plan.grid, kPairSmemBytes, stream, overlap);
  return cudaLaunchKernelEx(&lc.cfg, kernel, *m.hidden, *m.w, kFuse ? *m.w1 : *m.w, p);
}

// *pair_workers receives the smaller of its value and the CTA pairs of this kernel that can be resident at once
template <bool kTf32, int kBBox, bool kFuse = false>
cudaError_t prepare_pair(int num_sms, int* pair_workers) {
  auto kernel = kBBox == 32 ? lmhead_entropy_pair_kernel<kTf32, kBBox, kPairWideStages, 2, kFuse>
                            : lmhead_entropy_pair_kernel<kTf32, kBBox, kPairStages, 1, kFuse>;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPairSmemBytes);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(num_sms / 2 * 2);
  cfg.blockDim = dim3(kLmheadThreads);
  cfg.dynamicSmemBytes = kPairSmemBytes;
  cudaLaunchAttribute attr{};
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  int clusters = 0;
  e = cudaOccupancyMaxActiveClusters(&clusters, kernel, &cfg);
  if (e != cudaSuccess) return e;
  *pair_workers = std::min(*pair_workers, clusters);
  return cudaSuccess;
}

// One entry per Shape above (template arguments must be literals).
#define EGTP_SHAPE_PROMPT 1, 256, 256, 4
#define EGTP_SHAPE_DECODE1 1, 256, 32, 4
#define EGTP_SHAPE_DECODE2 2, 256, 32, 3
#define EGTP_SHAPE_PROMPT_F32 1, 256, 256, kF32Stages
#define EGTP_SHAPE_DECODE1_F32 1, 256, 32, kF32Stages
static_assert(kShapePrompt.mt == 1 && kShapePrompt.bn == 256 && kShapePrompt.bbox == 256 && kShapePrompt.stages == 4, "");
static_assert(kShapeDecode1.mt == 1 && kShapeDecode1.bn == 256 && kShapeDecode1.bbox == 32 && kShapeDecode1.stages == 4, "");
static_assert(kShapeDecode2.mt == 2 && kShapeDecode2.bn == 256 && kShapeDecode2.bbox == 32 && kShapeDecode2.stages == 3, "");

}  // namespace

LmheadPlan make_lmhead_plan(int64_t T, int d, int V, int elem_bytes, int num_sms, int64_t slot_row_capacity,
                            int mode, int head_cols, int force_chunks, int pair_workers) {
  // CTA pairs the device can co-schedule (what lmhead_prepare_device found on the context's device, or a number
  // the caller states when planning for a device that is not present)
  const int pair_cap = pair_workers;
  LmheadPlan pl{};
  // decode batches of 129..256 rows run as CTA pairs on 256 x 512 tiles unless single CTAs are asked for or the
  // device cannot co-schedule the pairs; prompt batches run as pairs only on request (and never with head columns)
  // fp32 rows (three tf32 MMAs per k step on operands split in shared memory) have the prompt shape and the
  // one-row-tile decode shape only, always one CTA per SM
  const bool f32 = elem_bytes == 4;
  pl.variant = T <= kTileM ? 1 : ((T <= 2 * kTileM && !f32) ? 2 : 0);
  const bool pairs_ok = pair_cap > 0 && mode != EGTP_LMHEAD_SINGLE_CTA && !f32;
  if (pl.variant == 2 && pairs_ok) pl.variant = 5;
  if (pl.variant == 0 && pairs_ok && mode == EGTP_LMHEAD_CTA_PAIRS && head_cols == 0) pl.variant = 4;
  if (pl.variant == 0 && pairs_ok && mode == EGTP_LMHEAD_CTA_PAIRS_WIDE && head_cols == 0) pl.variant = 6;
  const bool pair = pl.variant >= 4;
  const bool one_block = pl.variant == 1 || pl.variant == 2 || pl.variant == 5;
  const Shape& sh = shape_of(pl.variant);
  pl.rows_per_block = sh.mt * kTileM;
  pl.a_box_rows = pair ? kTileM : pl.rows_per_block;
  pl.tile_cols = sh.bn;
  pl.b_box_rows = sh.bbox;
  pl.col_gran = sh.col_gran;
  pl.row_blocks = static_cast<int>((T + pl.rows_per_block - 1) / pl.rows_per_block);
  pl.n_groups = (V + sh.col_gran - 1) / sh.col_gran;
  pl.v_pad = pl.n_groups * sh.col_gran;
  pl.head_cols_pad = (head_cols + sh.col_gran - 1) / sh.col_gran * sh.col_gran;
  pl.n_groups += pl.head_cols_pad / sh.col_gran;     // head columns follow the (padded) vocabulary
  pl.rows_pad = static_cast<int64_t>(pl.row_blocks) * pl.rows_per_block;
  pl.k_blocks = static_cast<int>((static_cast<int64_t>(d) * elem_bytes + kRowBytes - 1) / kRowBytes);
  pl.smem_bytes = pair ? kPairSmemBytes : smem_bytes_for(sh.mt, sh.bn, sh.stages, f32);
  // partial slots a row gets per vocabulary chunk: its tile columns are split over two epilogue
  // warps unless the two warps serve two different row tiles
  const int slots_per_chunk = pl.variant == 2 ? 1 : kEpiSplit;
  // CTAs, or CTA pairs that fit on the device at once
  const int workers_max = pair ? std::max(1, pair_cap > 0 ? std::min(pair_cap, num_sms / 2) : num_sms / 2)
                               : num_sms;
  const int64_t s_cap = std::max<int64_t>(1, slot_row_capacity / (pl.rows_pad * slots_per_chunk));
  const int s_max = static_cast<int>(std::min<int64_t>(pl.n_groups, s_cap));
  int workers;
  if (!one_block) {
    workers = static_cast<int>(std::min<int64_t>(workers_max, static_cast<int64_t>(pl.row_blocks) * pl.n_groups));
    // Units are dealt round-robin to the workers, so the step takes ceil(units / workers) rounds of
    // ceil(n_tiles / S) tiles.  Take the smallest S whose makespan is close to the best reachable one (fewer
    // chunks = fewer partials to write and merge).  How close, measured with interleaved runs on B200:
    // rows of up to 4 KB sweep the vocabulary as one group, W tiles are shared by all row blocks whatever S is,
    // and the product alone decides (T = 9555, d = 2048: S = 33 at 4.22 ms against 4.31 ms with S = 17), so 0.5 %;
    // with longer rows only a few row blocks sweep together and every extra chunk leaves fewer groups in step on
    // the same W tiles (T = 25629, d = 4096: S = 8 at 23.7 ms, S = 11 at 24.3 ms, S = 22 at 25.7 ms although
    // the product falls), so 2 %.
    auto makespan = [&](int S) {
      const int64_t units = static_cast<int64_t>(pl.row_blocks) * S;
      const int64_t rounds = (units + workers - 1) / workers;
      return rounds * ((pl.n_groups + S - 1) / S);
    };
    const bool one_group = static_cast<int64_t>(d) * elem_bytes <= 4096;
    const int64_t tol_num = one_group ? 201 : 102, tol_den = one_group ? 200 : 100;
    const int s_lim = std::min(s_max, 64);     // more chunks only add partials to write and merge
    int64_t best = makespan(1);
    for (int S = 2; S <= s_lim; ++S) best = std::min(best, makespan(S));
    int pick = 1;
    for (int S = 1; S <= s_lim; ++S) {
      if (makespan(S) * tol_den <= best * tol_num) { pick = S; break; }
    }
    // With long rows (row blocks sweep in small groups) a batch of few row blocks is better off in ONE round, every row block in step on the same W tiles (W then
    // streams from HBM once), than in several rounds of shorter units: 8 row blocks of 10 KB rows as 3 rounds of
    // 8 x 55 units measured 1.33 ms against 1.09 ms for one round of 8 x 18, although the product says 33 : 34.
    if (!one_group && pl.row_blocks <= workers) {
      const int s_one = std::max(1, std::min(s_lim, workers / pl.row_blocks));
      if (makespan(s_one) * 100 <= best * 106) pick = s_one;
    }
    pl.chunks = force_chunks > 0 ? std::min(force_chunks, s_max) : pick;
  } else {
    // One row block: one vocabulary range per worker, ranges differ by at most col_gran columns.
    pl.chunks = std::max(1, std::min(s_max, workers_max));
    workers = pl.chunks;
  }
  pl.grid = pair ? 2 * workers : workers;
  pl.slots = pl.chunks * slots_per_chunk;
  // Row blocks that sweep the vocabulary together (the rest of the batch waits for the next sweep).
  // A larger group re-reads W from HBM fewer times but keeps more hidden tiles circulating in L2 while W
  // streams through it.  Measured on B200 (interleaved A/B runs): with rows of up to 4 KB (d = 2048 bf16)
  // the whole batch in one group is fastest even at 94 MB of hidden states; with 8 KB and 10 KB rows
  // (d = 4096, 5120) about 4 MB per group is fastest and one 70 MB group is 17 % slower.
  const int64_t a_tile_bytes = static_cast<int64_t>(pl.rows_per_block) * d * elem_bytes;
  const int64_t group_bytes = static_cast<int64_t>(d) * elem_bytes <= 4096 ? (128ll << 20) : (4ll << 20);
  int gm = static_cast<int>(std::max<int64_t>(1, group_bytes / std::max<int64_t>(1, a_tile_bytes)));
  gm = std::min(gm, pl.row_blocks);
  gm = std::min(gm, std::max(1, workers));
  pl.group_rb = gm;
  return pl;
}

LmheadPlan make_headproj_plan(int64_t T, int d, int m_h, int elem_bytes, int num_sms, int max_splits, int a_repeats) {
  // The prompt shape (128-row blocks, 256-column tiles) over the head columns alone, K split so that the grid
  // fills the GPU while every split still streams several k blocks.
  LmheadPlan pl{};
  const Shape& sh = kShapePrompt;
  pl.variant = 0;
  pl.rows_per_block = kTileM;
  pl.a_box_rows = kTileM;
  pl.tile_cols = sh.bn;
  pl.b_box_rows = sh.bbox;
  pl.col_gran = sh.col_gran;
  pl.row_blocks = static_cast<int>((T + kTileM - 1) / kTileM);
  pl.v_pad = 0;
  pl.head_cols_pad = (m_h + sh.col_gran - 1) / sh.col_gran * sh.col_gran;
  pl.n_groups = pl.head_cols_pad / sh.col_gran;
  pl.rows_pad = static_cast<int64_t>(pl.row_blocks) * kTileM;
  pl.k_blocks = static_cast<int>((static_cast<int64_t>(d) * elem_bytes + kRowBytes - 1) / kRowBytes);
  if (a_repeats > 1) {               // A rows are a_repeats segments of d elements, each against the same W1
    pl.b_k_blocks = pl.k_blocks;
    pl.k_blocks *= a_repeats;
  }
  pl.smem_bytes = smem_bytes_for(sh.mt, sh.bn, sh.stages);
  pl.chunks = pl.n_groups;           // one 256-column tile per unit
  pl.slots = pl.chunks * kEpiSplit;  // unused: no entropy partials are written
  pl.group_rb = pl.row_blocks;
  const int base_units = pl.row_blocks * pl.chunks;
  int splits = std::max(1, num_sms / std::max(1, base_units));
  splits = std::min(splits, std::max(1, pl.k_blocks / 4));
  splits = std::max(1, std::min(splits, max_splits));
  const int kb_per = (pl.k_blocks + splits - 1) / splits;
  pl.k_splits = (pl.k_blocks + kb_per - 1) / kb_per;      // every split owns at least one k block
  pl.grid = std::min(num_sms, base_units * pl.k_splits);
  return pl;
}

cudaError_t lmhead_prepare_device(int* pair_workers_out) {
  cudaError_t e;
  if ((e = prepare_shape<false, EGTP_SHAPE_PROMPT>()) != cudaSuccess) return e;
  if ((e = prepare_shape<false, EGTP_SHAPE_DECODE1>()) != cudaSuccess) return e;
  if ((e = prepare_shape<false, EGTP_SHAPE_DECODE2>()) != cudaSuccess) return e;
  if ((e = prepare_shape<true, EGTP_SHAPE_PROMPT_F32>()) != cudaSuccess) return e;
  if ((e = prepare_shape<true, EGTP_SHAPE_DECODE1_F32>()) != cudaSuccess) return e;
  if ((e = prepare_shape<false, EGTP_SHAPE_PROMPT, true>()) != cudaSuccess) return e;
  if ((e = prepare_shape<false, EGTP_SHAPE_DECODE1, true>()) != cudaSuccess) return e;
  if ((e = prepare_shape<false, EGTP_SHAPE_DECODE2, true>()) != cudaSuccess) return e;
  int device = 0, num_sms = 0;
  if ((e = cudaGetDevice(&device)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, device)) != cudaSuccess) return e;
  int pairs = num_sms / 2;
  if ((e = prepare_pair<false, 128>(num_sms, &pairs)) != cudaSuccess) return e;
  if ((e = prepare_pair<false, 32>(num_sms, &pairs)) != cudaSuccess) return e;
  if ((e = prepare_pair<false, 32, true>(num_sms, &pairs)) != cudaSuccess) return e;
  *pair_workers_out = pairs;
  return cudaSuccess;
}

cudaError_t launch_lmhead_entropy(const LmheadPlan& plan, bool tf32, const LmheadMaps& maps, int64_t T, int V,
                                  float* partials, int32_t* status, cudaStream_t stream, float* head_g,
                                  bool overlap_previous) {
  (void)T;
  KParams p{};
  p.row_blocks = plan.row_blocks;
  p.chunks = plan.chunks;
  p.group_rb = plan.group_rb;
  p.k_blocks = plan.k_blocks;
  p.n_groups = plan.n_groups;
  p.col_gran = plan.col_gran;
  p.k_splits = std::max(1, plan.k_splits);
  p.kb_per_split = (plan.k_blocks + p.k_splits - 1) / p.k_splits;
  p.g_split_stride = plan.rows_pad * static_cast<int64_t>(plan.head_cols_pad);
  p.b_k_blocks = plan.b_k_blocks;
  p.total_units = plan.row_blocks * plan.chunks * p.k_splits;
  p.V = V;
  p.slots = plan.slots;
  p.partials = partials;
  p.status = status;
  p.v_pad = plan.v_pad;
  p.ldg = plan.head_cols_pad;
  p.head_g = head_g;
  if (maps.hidden == nullptr || maps.w == nullptr || (plan.variant < 4 && maps.w_tile == nullptr)) return cudaErrorInvalidValue;
  if (p.k_splits > 1 && (plan.head_cols_pad == 0 || plan.variant != 0)) return cudaErrorInvalidValue;
  if (plan.head_cols_pad > 0) {
    // fused head columns: bf16, one CTA per SM only
    if (tf32 || maps.w1 == nullptr || (plan.variant < 4 && maps.w1_tile == nullptr) || head_g == nullptr) return cudaErrorInvalidValue;
    switch (plan.variant) {
      case 0: return launch_shape<false, EGTP_SHAPE_PROMPT, true>(plan, maps, p, stream, overlap_previous);
      case 1: return launch_shape<false, EGTP_SHAPE_DECODE1, true>(plan, maps, p, stream, overlap_previous);
      case 2: return launch_shape<false, EGTP_SHAPE_DECODE2, true>(plan, maps, p, stream, overlap_previous);
      case 5: return launch_pair<false, 32, true>(plan, maps, p, stream, overlap_previous);
      default: return cudaErrorInvalidValue;
    }
  }
  if (tf32) {
    switch (plan.variant) {
      case 0: return launch_shape<true, EGTP_SHAPE_PROMPT_F32>(plan, maps, p, stream, overlap_previous);
      case 1: return launch_shape<true, EGTP_SHAPE_DECODE1_F32>(plan, maps, p, stream, overlap_previous);
      default: return cudaErrorInvalidValue;     // the planner gives fp32 rows no other shape
    }
  }
  switch (plan.variant) {
    case 1: return launch_shape<false, EGTP_SHAPE_DECODE1>(plan, maps, p, stream, overlap_previous);
    case 2: return launch_shape<false, EGTP_SHAPE_DECODE2>(plan, maps, p, stream, overlap_previous);
    case 4: return launch_pair<false, 128>(plan, maps, p, stream, overlap_previous);
    case 5:
    case 6: return launch_pair<false, 32>(plan, maps, p, stream, overlap_previous);
    default: return launch_shape<false, EGTP_SHAPE_PROMPT>(plan, maps, p, stream, overlap_previous);
  }
}

}  // namespace egtp
