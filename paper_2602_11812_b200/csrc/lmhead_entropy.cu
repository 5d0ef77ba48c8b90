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
//   warp 0      TMA producer: streams 128x(128 B) hidden tiles and 256x(128 B) W tiles through a
//               4-stage shared-memory ring (128-byte swizzle, K-major)
//   warp 1      MMA issuer (one thread) and owner of the TMEM allocation (512 columns = two
//               128x256 fp32 accumulators, so the epilogue of tile j overlaps the MMAs of j+1)
//   warps 2..9  epilogue: TMEM lane quadrant = warp % 4, column half = (warp - 2) / 4;
//               one row per thread, 128 columns per tile, tcgen05.ld in 32-column pieces
// A work unit is (row tile, vocabulary chunk); units are ordered so that CTAs running at the
// same time share W tiles (same chunk, neighbouring row tiles) and hidden tiles stay in L2.
#include "kernels.h"
#include "sm100_ptx.cuh"
#include "../../include/egtp.h"

#include <algorithm>

namespace egtp {

namespace {

constexpr int kABytes = kTileM * kRowBytes;            // 16 KB
constexpr int kBBytes = kTileN * kRowBytes;            // 32 KB
constexpr int kStageBytes = kABytes + kBBytes;         // 48 KB
constexpr int kBarrierBytes = 128;
constexpr int kSmemBytes = kStages * kStageBytes + kBarrierBytes + 1024;   // + slack for 1024-B alignment
constexpr uint32_t kTmemCols = 512;
constexpr float kLog2e = 1.4426950408889634f;

struct UnitCoord {
  int m_tile;
  int n_begin;
  int n_end;
  int chunk;
};

struct KParams {
  int m_tiles, n_tiles, chunks, group_m, k_blocks;
  int total_units;
  int V;
  int64_t rows_pad;
  float* partials;
  int32_t* status;
};

__device__ __forceinline__ UnitCoord unit_coord(int u, const KParams& p) {
  const int per_group = p.group_m * p.chunks;
  const int g = u / per_group;
  const int r = u - g * per_group;
  const int gm = min(p.group_m, p.m_tiles - g * p.group_m);
  UnitCoord c;
  c.chunk = r / gm;
  c.m_tile = g * p.group_m + (r - c.chunk * gm);
  c.n_begin = static_cast<int>((static_cast<int64_t>(c.chunk) * p.n_tiles) / p.chunks);
  c.n_end = static_cast<int>((static_cast<int64_t>(c.chunk + 1) * p.n_tiles) / p.chunks);
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
  // straddles the end of the vocabulary); the rest are ignored.
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
};

template <bool kTf32>
__global__ void __launch_bounds__(kLmheadThreads, 1)
lmhead_entropy_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                      const KParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bar_base = smem_base + kStages * kStageBytes;
  // barrier layout (8 bytes each): full[kStages], empty[kStages], acc_full[2], acc_empty[2]
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
  auto acc_full_bar = [&](int a) { return bar_base + 8u * (2 * kStages + a); };
  auto acc_empty_bar = [&](int a) { return bar_base + 8u * (2 * kStages + 2 + a); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + kStages * kStageBytes + 8 * (2 * kStages + 4));
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  // An earlier step of this call failed: do nothing.  One thread reads the word so that the
  // whole block takes the same decision.
  if (threadIdx.x == 0) *abort_flag = (*p.status != 0) ? 1u : 0u;
  __syncthreads();
  if (*abort_flag != 0u) return;
  __syncthreads();

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(acc_full_bar(a), 1);
      mbar_init(acc_empty_bar(a), 4 * kEpiSplit);
    }
    *abort_flag = 0u;
    mbar_fence_init();
    tma_prefetch_descriptor(&map_a);
    tma_prefetch_descriptor(&map_b);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  constexpr int kElemsPerStage = kTf32 ? kRowBytes / 4 : kRowBytes / 2;   // K elements per stage
  constexpr int kMmaPerStage = 4;                                         // 32 bytes of K per MMA
  constexpr uint32_t kIdesc = umma_idesc(kTf32 ? 2u : 1u, kTileM, kTileN);

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < p.total_units && ok; u += gridDim.x) {
        const UnitCoord uc = unit_coord(u, p);
        for (int nt = uc.n_begin; nt < uc.n_end && ok; ++nt) {
          for (int kb = 0; kb < p.k_blocks; ++kb) {
            if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
            const uint32_t a_dst = smem_base + stage * kStageBytes;
            const uint32_t b_dst = a_dst + kABytes;
            mbar_arrive_expect_tx(full_bar(stage), kStageBytes);
            tma_load_2d(a_dst, &map_a, kb * kElemsPerStage, uc.m_tile * kTileM, full_bar(stage));
            tma_load_2d(b_dst, &map_b, kb * kElemsPerStage, nt * kTileN, full_bar(stage));
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < p.total_units && ok; u += gridDim.x) {
        const UnitCoord uc = unit_coord(u, p);
        for (int nt = uc.n_begin; nt < uc.n_end && ok; ++nt) {
          if (!mbar_wait(acc_empty_bar(acc), acc_phase ^ 1u, abort_flag)) { ok = false; break; }
          tc_fence_after_sync();
          const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * kTileN);
          for (int kb = 0; kb < p.k_blocks; ++kb) {
            if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t a_src = smem_base + stage * kStageBytes;
            const uint64_t a_desc = umma_desc_k_major_sw128(a_src);
            const uint64_t b_desc = umma_desc_k_major_sw128(a_src + kABytes);
#pragma unroll
            for (int k = 0; k < kMmaPerStage; ++k) {
              // advancing K by 32 bytes inside the swizzled row = +2 in the (address >> 4) field
              umma_ss<kTf32>(d_tmem, a_desc + 2u * k, b_desc + 2u * k, kIdesc, (kb | k) != 0 ? 1u : 0u);
            }
            umma_commit(empty_bar(stage));          // stage reusable once these MMAs have read it
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
          if (ok) umma_commit(acc_full_bar(acc));   // accumulator complete
          acc ^= 1;
          if (acc == 0) acc_phase ^= 1u;
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const int quad = warp & 3;                 // TMEM lanes 32*quad .. 32*quad+31
    const int half = (warp - 2) >> 2;          // which 128 of the tile's 256 columns
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int u = blockIdx.x; u < p.total_units && ok; u += gridDim.x) {
      const UnitCoord uc = unit_coord(u, p);
      RowState st;
      st.init();
      for (int nt = uc.n_begin; nt < uc.n_end; ++nt) {
        ok = __all_sync(0xffffffffu, mbar_wait(acc_full_bar(acc), acc_phase, abort_flag));
        if (!ok) break;
        tc_fence_after_sync();
        const int col0 = nt * kTileN + half * (kTileN / kEpiSplit);
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) +
                               static_cast<uint32_t>(acc * kTileN + half * (kTileN / kEpiSplit));
        static_assert(kTileN / kEpiSplit == 128, "epilogue is written for 128 columns per warp and tile");
        const int cols_left = p.V - col0;         // columns of this warp's range that exist (may be <= 0)
        uint32_t bufA[32], bufB[32];
        if (cols_left >= 128) {
          // software pipeline: the load of piece c+1 is in flight while piece c is folded
          tmem_ld_32(taddr, bufA);
          tmem_ld_wait(bufA);
          tmem_ld_32(taddr + 32, bufB);
          st.fold<false>(bufA, 32);
          tmem_ld_wait(bufB);
          tmem_ld_32(taddr + 64, bufA);
          st.fold<false>(bufB, 32);
          tmem_ld_wait(bufA);
          tmem_ld_32(taddr + 96, bufB);
          st.fold<false>(bufA, 32);
          tmem_ld_wait(bufB);
          // every read of the accumulator has completed: hand it back before the last fold
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(acc_empty_bar(acc));
          st.fold<false>(bufB, 32);
        } else {
          for (int c = 0; c < 4 && c * 32 < cols_left; ++c) {
            tmem_ld_32(taddr + c * 32, bufA);
            tmem_ld_wait(bufA);
            st.fold<true>(bufA, min(32, cols_left - c * 32));
          }
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(acc_empty_bar(acc));
        }
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      }
      if (ok) {
        const int64_t row = static_cast<int64_t>(uc.m_tile) * kTileM + quad * 32 + lane;
        const int slot = uc.chunk * kEpiSplit + half;
        float* dst = p.partials + static_cast<int64_t>(slot) * 3 * p.rows_pad + row;
        dst[0] = st.m;
        dst[p.rows_pad] = (st.s[0] + st.s[1]) + (st.s[2] + st.s[3]);
        dst[2 * p.rows_pad] = (st.t[0] + st.t[1]) + (st.t[2] + st.t[3]);
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

}  // namespace

LmheadPlan make_lmhead_plan(int64_t T, int d, int V, int elem_bytes, int num_sms, int64_t slot_row_capacity) {
  LmheadPlan pl{};
  pl.m_tiles = static_cast<int>((T + kTileM - 1) / kTileM);
  pl.n_tiles = (V + kTileN - 1) / kTileN;
  pl.rows_pad = static_cast<int64_t>(pl.m_tiles) * kTileM;
  pl.k_blocks = static_cast<int>((static_cast<int64_t>(d) * elem_bytes + kRowBytes - 1) / kRowBytes);
  pl.smem_bytes = kSmemBytes;
  const int64_t tiles = static_cast<int64_t>(pl.m_tiles) * pl.n_tiles;
  pl.grid = static_cast<int>(std::min<int64_t>(num_sms, tiles));
  // Units are dealt round-robin to the CTAs, so the step takes ceil(units / grid) rounds of
  // ceil(n_tiles / S) tiles.  Take the smallest S whose makespan is within 2 % of the best
  // reachable one (fewer chunks = fewer partials to write and merge).
  int64_t s_cap = std::max<int64_t>(1, slot_row_capacity / (pl.rows_pad * kEpiSplit));
  const int s_max = static_cast<int>(std::min<int64_t>(pl.n_tiles, s_cap));
  auto makespan = [&](int S) {
    const int64_t units = static_cast<int64_t>(pl.m_tiles) * S;
    const int64_t rounds = (units + pl.grid - 1) / pl.grid;
    return rounds * ((pl.n_tiles + S - 1) / S);
  };
  int64_t best = makespan(1);
  for (int S = 2; S <= s_max; ++S) best = std::min(best, makespan(S));
  int pick = 1;
  for (int S = 1; S <= s_max; ++S) {
    if (makespan(S) * 100 <= best * 102) { pick = S; break; }
  }
  pl.chunks = pick;
  pl.slots = pick * kEpiSplit;
  // Row tiles that sweep the vocabulary together: enough of them that a W tile fetched from HBM
  // is shared by many CTAs, few enough that their hidden tiles (re-read per vocabulary tile) stay in L2.
  const int64_t a_tile_bytes = static_cast<int64_t>(kTileM) * d * elem_bytes;
  int gm = static_cast<int>(std::max<int64_t>(1, (48ll << 20) / std::max<int64_t>(1, a_tile_bytes)));
  gm = std::min(gm, pl.m_tiles);
  gm = std::min(gm, std::max(1, pl.grid));
  pl.group_m = gm;
  return pl;
}

cudaError_t lmhead_prepare_device() {
  cudaError_t err = cudaFuncSetAttribute(lmhead_entropy_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         kSmemBytes);
  if (err != cudaSuccess) return err;
  return cudaFuncSetAttribute(lmhead_entropy_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
}

cudaError_t launch_lmhead_entropy(const LmheadPlan& plan, bool tf32, const CUtensorMap* map_hidden,
                                  const CUtensorMap* map_w, int64_t T, int V, float* partials,
                                  int32_t* status, cudaStream_t stream) {
  (void)T;
  KParams p{};
  p.m_tiles = plan.m_tiles;
  p.n_tiles = plan.n_tiles;
  p.chunks = plan.chunks;
  p.group_m = plan.group_m;
  p.k_blocks = plan.k_blocks;
  p.total_units = plan.m_tiles * plan.chunks;
  p.V = V;
  p.rows_pad = plan.rows_pad;
  p.partials = partials;
  p.status = status;
  if (tf32) {
    lmhead_entropy_kernel<true><<<plan.grid, kLmheadThreads, kSmemBytes, stream>>>(*map_hidden, *map_w, p);
  } else {
    lmhead_entropy_kernel<false><<<plan.grid, kLmheadThreads, kSmemBytes, stream>>>(*map_hidden, *map_w, p);
  }
  return cudaGetLastError();
}

}  // namespace egtp
