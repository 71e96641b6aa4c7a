// dK / dV side of the fused attention backward with the GProj correction for sm_100a, head dimension 64, 128-wide steps
// (Algorithm 1).
//
// Same arithmetic as bwd_dkv_kernel in attn_bwd.cuh, with a TMEM plan that lets EVERY score product be an N = 128
// instruction (the full 8192 FLOP/clk/SM; an N = 64 instruction costs 48 clk for 32 clk of work):
//
//   columns   0..127  X   S^T of the even steps, then their packed r^T / t^T
//           128..255  Y   dP^T of every step (single-buffered)
//           256..383  Z   S^T of the odd steps, then their packed r^T / t^T
//           384..447  dV accumulator,   448..511  dK accumulator
//
// A step is 128 streamed query rows.  Its arithmetic runs in two phases: phase 1 needs only S^T (p = exp2(..), r = BF16(p),
// p kept in FP32 registers), phase 2 needs dP^T (t = BF16(p (dP - D))).  Because dP^T is consumed quickly and S^T is
// double-buffered, the tensor core computes the scores of step n + 1 while the ALUs work on step n, and the products
// that need only r^T start while t^T is still being computed:
//
//   issuer 1:  S^T(n) -> [X|Z]   when stage n landed and the second-stage products of step n - 2 are done
//              dP^T(n) -> Y       when phase 2 of step n - 1 has read Y
//   ALUs:      phase 1(n) after S^T(n): r^T -> over S^T;   phase 2(n) after dP^T(n): t^T -> over S^T, Y free
//   issuer 2:  [dV | dK] += r^T [dO | Z] after phase 1(n);   dK += t^T Q after phase 2(n);   then [X|Z] of step n is free
//
// All four compute warpgroups work on the same step, warpgroup w on the 32-column slice w (thread <-> (key row, slice)).
// Everything else (persistent tile schedule, TMA staging, epilogue through a swizzled staging buffer, packed-sequence
// descriptors, bounded waits) is as in attn_bwd.cuh.  Measured against the 64-wide kernel at d = 64: 6 % faster on
// workload 2, 9 % on a non-causal problem; the same layout for the dQ side was 5 % SLOWER than its 64-wide kernel (its
// phases also carry the row-mass sums) and is not kept.
#pragma once
#include "attn_bwd.cuh"

namespace gproj {

struct BwdW128 {
  static constexpr int D = 64;
  static constexpr int kTileBytes = 128 * 128;                     // 128 rows x 64 BF16: one 128-byte-row slab
  static constexpr int kStepRows = 128;
  static constexpr int kStages = 3;
  static constexpr int kWG = 4, kCompute = 128 * kWG, kThreads = 96 + kCompute;   // warp 0: stage producer (lane 0) and tile loader (lane 1); warps 1, 2: MMA issuers; 16 compute warps
  static constexpr int kSliceCols = kStepRows / kWG;               // 32 columns per thread and step
  static constexpr uint32_t kColX = 0, kColY = 128, kColZ = 256, kColAcc0 = 384, kColAcc1 = 448;
  static constexpr int kTmemCols = 512;
  // K, V resident, ring of (Q, dO, Z, two 64-row statistic blocks) step tiles, staging (dK, dV)
  static constexpr int kDkvStageBytes = 3 * kTileBytes + 1024;
  static constexpr int kDkvSmemBytes = 2 * kTileBytes + kStages * kDkvStageBytes + 2 * kTileBytes + 1024;
  static_assert(kDkvSmemBytes <= 227 * 1024, "shared memory budget");
};

enum BwdW128WaitCode {
  kWkRes = 0x51, kWkQ = 0x52, kWkQEmpty = 0x53, kWkS = 0x54, kWkDP = 0x55, kWkR = 0x56, kWkT = 0x57, kWkSFree = 0x58, kWkYFree = 0x59,
  kWkAcc = 0x5a, kWkAccFree = 0x5b, kWkResFree = 0x5c
};

// Phase 2 of the dK/dV side for a step that may reach past the statistics that were written (ragged end of a sequence):
// a column with p = 0 gets t = 0 explicitly instead of 0 * (dP - D), because its -D may be arbitrary bits.
__device__ __forceinline__ void dkv_phase2_guarded(uint32_t tS, uint32_t tdP, const float *nd, const float (&p)[32]) {
  uint32_t xp[2][16];
  tmem_ld16(tdP, xp[0]);
#pragma unroll
  for (int c = 0; c < 2; ++c) {
    tmem_wait_ld();
    if (c == 0) tmem_ld16(tdP + 16, xp[1]);
    uint32_t pt[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const ulonglong2 d4 = *reinterpret_cast<const ulonglong2 *>(nd + 16 * c + 4 * i);
      const int col = 16 * c + 4 * i;
      float t[4];
      f32x2_split(mul2(f32x2(p[col], p[col + 1]), add2(f32x2_bits(xp[c][4 * i], xp[c][4 * i + 1]), d4.x)), t[0], t[1]);
      f32x2_split(mul2(f32x2(p[col + 2], p[col + 3]), add2(f32x2_bits(xp[c][4 * i + 2], xp[c][4 * i + 3]), d4.y)), t[2], t[3]);
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if (p[col + e] == 0.f) t[e] = 0.f;
      pt[2 * i] = pack_bf16x2(t[0], t[1]);
      pt[2 * i + 1] = pack_bf16x2(t[2], t[3]);
    }
    tmem_st8(tS + 16 * c + 8, pt);
  }
}

// ============================================================================================
// dK / dV side, d = 64, 128-query steps
// ============================================================================================
template <bool CAUSAL>
__global__ void __launch_bounds__(BwdW128::kThreads, 1)
bwd_dkv_w128_kernel(const __grid_constant__ CUtensorMap tmK,    // box 64 x 128 rows
                    const __grid_constant__ CUtensorMap tmV,    // box 64 x 128 rows
                    const __grid_constant__ CUtensorMap tmQ,    // box 64 x 128 rows
                    const __grid_constant__ CUtensorMap tmdO,   // box 64 x 128 rows
                    const __grid_constant__ CUtensorMap tmZ,    // box 64 x 128 rows
                    const __grid_constant__ CUtensorMap tmdK,   // store, box 64 x 128 rows
                    const __grid_constant__ CUtensorMap tmdV,   // store, box 64 x 128 rows
                    const float *__restrict__ stats,
                    __nv_bfloat16 *__restrict__ dKg, __nv_bfloat16 *__restrict__ dVg,
                    const int4 *__restrict__ plan, int nblk,
                    int N, int Nq, int BH, int Hkv, int G, int total_tiles, const ItemOrder order, float scale_log2, float alpha, unsigned flags, int *status) {
  // BH counts (batch, KV head) pairs.  With grouped queries one work item walks the query steps of all G query heads of
  // its KV head, so that their contributions are summed in the FP32 accumulators (Section 3.1).
  using C = BwdW128;
  constexpr int D = C::D, S = C::kStages;
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t *sK = smem;
  uint8_t *sV = sK + C::kTileBytes;
  uint8_t *sStage = sV + C::kTileBytes;   // stage s: Q, dO, Z step tiles, then two blocks of {64 x -LSE log2 e, 64 x -D}
  uint8_t *sOut = sStage + S * C::kDkvStageBytes;   // staging: dK tile, then dV tile

  __shared__ uint64_t bar_res_full, bar_res_free, bar_q_full[S], bar_q_empty[S];
  __shared__ uint64_t bar_s_full[2], bar_r_ready[2], bar_t_ready[2], bar_s_free[2], bar_dp_full, bar_y_free;
  __shared__ uint64_t bar_acc_done, bar_acc_free, bar_drain[2];
  __shared__ uint32_t tmem_base_smem;
  __shared__ int cta_abort, cta_skip;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) cta_skip = *reinterpret_cast<volatile int *>(status);
  __syncthreads();
  if (cta_skip != 0) return;

  const bool use_z = (flags & kFlagNoKCorrection) == 0;
  const uint32_t stage_tx = (use_z ? 3 : 2) * C::kTileBytes + 1024;

  AbortState ab{status, &cta_abort};
  if (threadIdx.x == 0) {
    cta_abort = 0;
    mbar_init(&bar_res_full, 1);
    mbar_init(&bar_res_free, 1);   // the last score product alone: the epilogue has its own staging buffer and never touches K / V
    for (int s = 0; s < S; ++s) { mbar_init(&bar_q_full[s], 1); mbar_init(&bar_q_empty[s], 1); }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&bar_s_full[b], 1); mbar_init(&bar_s_free[b], 1);
      mbar_init(&bar_r_ready[b], C::kCompute); mbar_init(&bar_t_ready[b], C::kCompute);
    }
    mbar_init(&bar_dp_full, 1);
    mbar_init(&bar_y_free, C::kCompute);
    mbar_init(&bar_acc_done, 1);
    mbar_init(&bar_acc_free, C::kCompute);
    mbar_init(&bar_drain[0], 1);
    mbar_init(&bar_drain[1], 1);
    fence_mbar_init();
  }
  if (warp == 1) { tmem_alloc(&tmem_base_smem, C::kTmemCols); tmem_relinquish(); }
  if (warp == 0 && lane == 0) {
    tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV); tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmdO); tma_prefetch_desc(&tmZ);
    tma_prefetch_desc(&tmdK); tma_prefetch_desc(&tmdV);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = __shfl_sync(0xffffffffu, tmem_base_smem, 0);

  TileSched sched(total_tiles);
  // A step may reach past the end of the sequence: those query columns are zero fill or the next packed sequence's rows,
  // and are masked.
  // N: key rows per head (own operand), Nq: query rows per head.  A key j is seen by the queries i >= j - (L_k - L_q).
  auto tix = [&](int lin) { return order.rank(lin); };
  auto hix = [&](int lin) { return order.head(lin); };
  auto tile_of = [&](int lin) { return tile_info(plan, tix(lin), tix(lin), N, Nq); };
  // First query (inside its sequence, rounded down to a 64-row statistics block) that sees this key tile, and the steps
  // from there to the end of the queries; at least one step, fully masked if no query sees the tile.
  auto q_start_of = [&](const TileInfo &t) {
    const int Lq = t.oseq_end - t.oseq0, off = (t.seq_end - t.seq0) - Lq;
    const int first = CAUSAL ? (max(0, t.row0 - t.seq0 - off) & ~63) : 0;
    return min(first, ((Lq - 1) >> 6) << 6);
  };
  auto steps_of = [&](const TileInfo &t) { return max(1, (t.oseq_end - t.oseq0 - q_start_of(t) + C::kStepRows - 1) / C::kStepRows); };

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer of the streamed (Q, dO, Z, stats) step tiles
    if (lane == 0) {
      // Z and the row statistics come from the dQ-side kernel, which may still be running (programmatic dependent
      // launch); everything this CTA did so far, and the stationary-tile loads of the other loader warp, did not need it.
      griddep_wait();
      int g = 0;
      for (int lin = sched.next(); lin >= 0; lin = sched.next()) {
        const TileInfo tl = tile_of(lin);
        const int bh = hix(lin), T = steps_of(tl), q_start = q_start_of(tl);
        const int q_head0 = (bh / Hkv) * (Hkv * G) + (bh % Hkv) * G;     // first query head of the group (flat index)
        for (int n = 0; n < G * T; ++n, ++g) {
          const int st = g % S;
          if (g >= S) mbar_wait(&bar_q_empty[st], ((g / S) - 1) & 1, ab, kWkQEmpty);
          mbar_expect_tx(&bar_q_full[st], stage_tx);
          uint8_t *dst = sStage + st * C::kDkvStageBytes;
          const int qh = q_head0 + n / T, qrel = q_start + (n % T) * C::kStepRows, qrow = tl.oseq0 + qrel;
          tma_load_3d(dst, &tmQ, &bar_q_full[st], 0, qrow, qh);
          tma_load_3d(dst + C::kTileBytes, &tmdO, &bar_q_full[st], 0, qrow, qh);
          if (use_z) tma_load_3d(dst + 2 * C::kTileBytes, &tmZ, &bar_q_full[st], 0, qrow, qh);
          // two 64-row statistic blocks (the second may lie past the sequence's last block: its columns are masked)
          bulk_load_1d(dst + 3 * C::kTileBytes, stats + (static_cast<size_t>(qh) * nblk + tl.blk0 + (qrel >> 6)) * 128, 1024,
                       &bar_q_full[st]);
        }
      }
      if (cta_abort) {
        for (int q = (g > S ? g - S : 0); q < g; ++q)
          for (int spin = 0; spin < 100000 && !mbar_try_wait(&bar_q_full[q % S], (q / S) & 1); ++spin) {}
      }
    } else if (lane == 1) {
      // -------------------------------------------------------------- TMA loader of the stationary (K, V) tiles (second lane of
      // the producer's warp: the two single-thread roles share a warp, which leaves 608 threads and 104 registers each)
      int ti = 0;
      for (int lin = sched.next(); lin >= 0; lin = sched.next(), ++ti) {
        const int bh = hix(lin), krow0 = tile_of(lin).row0;
        if (ti >= 1) mbar_wait(&bar_res_free, (ti - 1) & 1, ab, kWkResFree);
        mbar_expect_tx(&bar_res_full, 2 * C::kTileBytes);
        tma_load_3d(sK, &tmK, &bar_res_full, 0, krow0, bh);
        tma_load_3d(sV, &tmV, &bar_res_full, 0, krow0, bh);
      }
      if (cta_abort && ti > 0)
        for (int spin = 0; spin < 100000 && !mbar_try_wait(&bar_res_full, (ti - 1) & 1); ++spin) {}
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- tensor-core issuer 1: S^T = K Q^T, dP^T = V dO^T
    constexpr uint32_t idesc_s = idesc_bf16_f32(128, 128, 0, 0);   // [128 keys] x [128 queries], contraction over d
    const SmemDesc dscK = make_smem_desc(smem_u32(sK), 16, 1024), dscV = make_smem_desc(smem_u32(sV), 16, 1024);
    const SmemDesc dscQ0 = make_smem_desc(smem_u32(sStage), 16, 1024);
    int g = 0, ti = 0;
    for (int lin = sched.next(); lin >= 0; lin = sched.next(), ++ti) {
      const int T = G * steps_of(tile_of(lin));
      mbar_wait(&bar_res_full, ti & 1, ab, kWkRes);
      for (int n = 0; n < T; ++n, ++g) {
        const int st = g % S, sb = g & 1;
        mbar_wait(&bar_q_full[st], (g / S) & 1, ab, kWkQ);
        if (g >= 2) mbar_wait(&bar_s_free[sb], ((g >> 1) - 1) & 1, ab, kWkSFree);   // r, t of step g - 2 consumed
        tc_fence_after();
        const SmemDesc dscQ = dscQ0.advanced(st * C::kDkvStageBytes), dscdO = dscQ.advanced(C::kTileBytes);
        const uint32_t tS = tmem_base + (sb ? C::kColZ : C::kColX);
        if (elect_one_sync()) {
#pragma unroll
          for (int k = 0; k < D / 16; ++k) umma_ss(tS, dscK.at(k * 32), dscQ.at(k * 32), idesc_s, k > 0);
          umma_commit(&bar_s_full[sb]);
        }
        __syncwarp();
        if (g >= 1) mbar_wait(&bar_y_free, (g - 1) & 1, ab, kWkYFree);               // phase 2 of step g - 1 has read dP^T
        tc_fence_after();
        if (elect_one_sync()) {
#pragma unroll
          for (int k = 0; k < D / 16; ++k) umma_ss(tmem_base + C::kColY, dscV.at(k * 32), dscdO.at(k * 32), idesc_s, k > 0);
          umma_commit(&bar_dp_full);
          if (n == T - 1) umma_commit(&bar_res_free);   // no MMA reads this K / V tile any more
        }
        __syncwarp();
      }
    }
    drain_mmas_if_aborted(&bar_drain[0], ab);
  } else if (warp == 2) {
    // ---------------------------------------------------------------- tensor-core issuer 2: [dV | dK] += r^T [dO | Z], then dK += t^T Q
    constexpr uint32_t idesc_a = idesc_bf16_f32(128, D, 0, 1);         // [128 keys] x [d], contraction over 128 queries
    constexpr uint32_t idesc_fused = idesc_bf16_f32(128, 128, 0, 1);   // [128 keys] x [dO | Z]
    const SmemDesc dscQ0mn = make_smem_desc(smem_u32(sStage), C::kTileBytes, 1024);        // MN-major view of stage 0
    int g = 0, ti = 0;
    for (int lin = sched.next(); lin >= 0; lin = sched.next(), ++ti) {
      const int T = G * steps_of(tile_of(lin));
      if (ti > 0) mbar_wait(&bar_acc_free, (ti - 1) & 1, ab, kWkAccFree);   // the previous epilogue has read dV, dK
      for (int p = 0; p < T; ++p, ++g) {
        const int st = g % S, sb = g & 1;
        const SmemDesc dscQ = dscQ0mn.advanced(st * C::kDkvStageBytes), dscdO = dscQ.advanced(C::kTileBytes);
        // packed BF16 operands of query slice k (16 queries): r^T over columns 16 k .. 16 k + 7 of the S region, t^T over the next eight
        const uint32_t tR = tmem_base + (sb ? C::kColZ : C::kColX), tT = tR + 8;
        const uint32_t acc = (p > 0) ? 1u : 0u;
        mbar_wait(&bar_r_ready[sb], (g >> 1) & 1, ab, kWkR);
        tc_fence_after();
        if (elect_one_sync()) {
          if (use_z) {
            // the dO and Z step tiles are adjacent 64-column atoms of one MN-major operand and the dV and dK accumulators
            // are adjacent TMEM columns: r^T [dO | -BF16(lambda Q)] is ONE N = 128 product (Algorithm 1 lines 17-18)
#pragma unroll
            for (int k = 0; k < C::kStepRows / 16; ++k)
              umma_ts(tmem_base + C::kColAcc0, tR + 16 * k, dscdO.at(k * 2048), idesc_fused, k > 0 ? 1u : acc);
          } else {
#pragma unroll
            for (int k = 0; k < C::kStepRows / 16; ++k)      // dV += r^T dO
              umma_ts(tmem_base + C::kColAcc0, tR + 16 * k, dscdO.at(k * 2048), idesc_a, k > 0 ? 1u : acc);
          }
        }
        __syncwarp();
        mbar_wait(&bar_t_ready[sb], (g >> 1) & 1, ab, kWkT);
        tc_fence_after();
        if (elect_one_sync()) {
          const uint32_t acc_k = use_z ? 1u : acc;           // with the correction, dK already holds this step's r^T Z
#pragma unroll
          for (int k = 0; k < C::kStepRows / 16; ++k)        // dK += t^T Q
            umma_ts(tmem_base + C::kColAcc1, tT + 16 * k, dscQ.at(k * 2048), idesc_a, k > 0 ? 1u : acc_k);
          umma_commit(&bar_s_free[sb]);
          umma_commit(&bar_q_empty[st]);
          if (p == T - 1) umma_commit(&bar_acc_done);
        }
        __syncwarp();
      }
    }
    drain_mmas_if_aborted(&bar_drain[1], ab);
  } else {
    // ---------------------------------------------------------------- compute: thread <-> (key row, 32-query slice of every step)
    const int wg = (warp - 3) >> 2;
    const int row = 32 * (warp & 3) + lane;                  // key row within the tile
    const uint32_t lane_addr = static_cast<uint32_t>(32 * (warp & 3)) << 16;
    const uint32_t slice_addr = tmem_base + lane_addr + C::kSliceCols * wg;
    int g0 = 0, ti = 0;
    for (int lin = sched.next(); lin >= 0; lin = sched.next(), ++ti) {
      const TileInfo tl = tile_of(lin);
      const int bh = hix(lin), Th = steps_of(tl), T = G * Th, q_start = q_start_of(tl);
      // (Issuing the first TMEM load of a phase early, when its barrier had already completed, and letting warpgroup pairs
      // take turns in phase 1, were both measured slower.)
      for (int n = 0; n < T; ++n) {
        const int g = g0 + n, st = g % S, sb = g & 1;
        const uint32_t tS = slice_addr + (sb ? C::kColZ : C::kColX), tdP = slice_addr + C::kColY;
        // The scores of this step were issued after its stage (and with it the row statistics) had landed in shared
        // memory, so their completion covers both.  Slice w of the 128 columns lies in statistic block w / 2.
        const float *nl = reinterpret_cast<const float *>(sStage + st * C::kDkvStageBytes + 3 * C::kTileBytes) + (wg >> 1) * 128 + (wg & 1) * 32;
        const int nh = n % Th;                                              // step within the current query head
        const int Lq = tl.oseq_end - tl.oseq0, off = (tl.seq_end - tl.seq0) - Lq, krel0 = tl.row0 - tl.seq0;
        const int qs = q_start + nh * C::kStepRows;                         // first query (inside its sequence) of the step
        const int q0 = qs + C::kSliceCols * wg;                             // ... of the slice's column 0
        const bool masked = (CAUSAL && qs < krel0 + 128 - off) || qs + C::kStepRows > Lq;
        float pkeep[32];
        mbar_wait(&bar_s_full[sb], (g >> 1) & 1, ab, kWkS);
        tc_fence_after();
        if (masked) dkv_phase1<true>(tS, nl, scale_log2, CAUSAL ? krel0 + row - off - q0 : 0, Lq - 1 - q0, pkeep);
        else        dkv_phase1<false>(tS, nl, scale_log2, 0, 0, pkeep);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&bar_r_ready[sb]);
        mbar_wait(&bar_dp_full, g & 1, ab, kWkDP);
        tc_fence_after();
        if (masked) dkv_phase2_guarded(tS, tdP, nl + 64, pkeep);
        else        dkv_phase2(tS, tdP, nl + 64, pkeep);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&bar_y_free);                      // dP^T of this step has been read: the next one may be computed
        mbar_arrive(&bar_t_ready[sb]);
      }

      mbar_wait(&bar_acc_done, ti & 1, ab, kWkAcc);
      tc_fence_after();
      uint8_t *stage_dk = sOut, *stage_dv = sOut + C::kTileBytes;
      uint32_t a[16], b[16];
      tmem_ld16(tmem_base + C::kColAcc0 + lane_addr + 16 * wg, a);
      tmem_ld16(tmem_base + C::kColAcc1 + lane_addr + 16 * wg, b);
      tmem_wait_ld();
      tc_fence_before();
      mbar_arrive(&bar_acc_free);          // the accumulators may be overwritten by the next tile
      if (threadIdx.x == 96) bulk_wait_group_read0();   // the previous tile's stores have left the staging buffer
      named_bar_sync(1, C::kCompute);
#pragma unroll
      for (int v = 0; v < 2; ++v) {
        const uint32_t off = swz128_offset(row, 2 * wg + v);
        uint32_t vw[4], kw[4];
#pragma unroll
        for (int w = 0; w < 4; ++w) {
          const int i = 8 * v + 2 * w;
          vw[w] = pack_bf16x2(__uint_as_float(a[i]), __uint_as_float(a[i + 1]));
          kw[w] = pack_bf16x2(__fmul_rn(alpha, __uint_as_float(b[i])), __fmul_rn(alpha, __uint_as_float(b[i + 1])));
        }
        *reinterpret_cast<uint4 *>(stage_dv + off) = make_uint4(vw[0], vw[1], vw[2], vw[3]);
        *reinterpret_cast<uint4 *>(stage_dk + off) = make_uint4(kw[0], kw[1], kw[2], kw[3]);
      }
      fence_proxy_async_smem();
      named_bar_sync(1, C::kCompute);
      if (tile_store_by_tma(tl, N)) {
        if (threadIdx.x == 96) {
          tma_store_3d(&tmdV, stage_dv, 0, tl.row0, bh);
          tma_store_3d(&tmdK, stage_dk, 0, tl.row0, bh);
          bulk_commit_group();
        }
      } else {
        // ragged last tile of a packed sequence that another sequence follows: rows past its end are not ours to write
        if (wg < 2) store_rows_clipped<D>(wg == 0 ? stage_dk : stage_dv, C::kTileBytes,
                                         (wg == 0 ? dKg : dVg) + (static_cast<size_t>(bh) * N + tl.row0) * D, row, tl.seq_end - tl.row0);
        named_bar_sync(1, C::kCompute);
      }
      g0 += T;
    }
    if (threadIdx.x == 96) bulk_wait_group_read0();
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, C::kTmemCols);
}

}  // namespace gproj
