// dK / dV side of the fused attention backward with the GProj correction for sm_100a, head dimension 64, 128-wide steps
// (Algorithm 1).
//
// Same arithmetic as bwd_dkv_kernel in attn_bwd.cuh, with a TMEM plan that lets EVERY score product be an N = 128
// instruction (the full 8192 FLOP/clk/SM; an N = 64 instruction costs 48 clk for 32 clk of work):
//
//   columns   0..127  X   S^T of the even steps, then their packed r^T / t^T
//           128..255  Y   dP^T of every step (single-buffered, consumed into registers at the start of the step)
//           256..383  Z   S^T of the odd steps, then their packed r^T / t^T
//           384..447  dV accumulator,   448..511  dK accumulator
//
// A step is 128 streamed query rows.  Thread <-> (key row, two 16-column chunks of the step: columns 16 w .. 16 w + 15 of
// the first 64 queries, then of the last 64; w = warpgroup).  At the start of a step a thread takes dP^T of both chunks
// into registers and releases the single dP^T buffer at once, so the tensor core writes the next step's dP^T while this
// step is in the ALUs.  Each chunk is then done in one pass (p = exp2(..), r = BF16(p), t = BF16(p (dP - D))) and the two
// halves of the step are handed over separately, so the second-stage products of the first 64 queries run while the
// last 64 are in the ALUs.
//
//   issuer 1:  S^T(n) -> [X|Z]   when stage n landed and the second-stage products of step n - 2 are done
//   issuer 3:  dP^T(n) -> Y       when the ALUs hold dP^T of step n - 1 in registers
//   ALUs:      dP^T(n) -> registers, Y free;  chunk 0: r^T, t^T over S^T, first half ready;  chunk 1: second half ready
//   issuer 2:  per half:  [dV | dK] += r^T [dO | Z],  dK += t^T Q;   after the second half [X|Z] of step n is free
//
// Three issuing warps, because the tensor core takes its work in the order it is issued and holds an issuing thread for
// as long as its products execute: dP^T(n + 1), which the ALUs want the moment they finish step n, must not wait in one
// thread's program order behind S^T(n + 1) (whose buffer frees late) nor behind the second-stage products of step n.
// (Measured on workload 2, against two-phase arithmetic with two issuing warps: 79.3 -> 77.6 us back to back.  Not kept,
// all measured no faster: the two halves of the step on two warpgroup pairs running half a step apart; the next step's
// TMEM loads issued behind the last stores of the current one; dP^T issued by the second-stage warp one step ahead.)
// Everything else (persistent tile schedule, TMA staging, epilogue through a swizzled staging buffer, packed-sequence
// descriptors, bounded waits) is as in attn_bwd.cuh.  Against the 64-wide kernel at d = 64 this kernel is about 8 % faster
// on workload 2; the same layout for the dQ side was 5 % SLOWER than its 64-wide kernel (its arithmetic also carries the
// row-mass sums) and is not kept.
#pragma once
#include "attn_bwd.cuh"

namespace gproj {

struct BwdW128 {
  static constexpr int D = 64;
  static constexpr int kTileBytes = 128 * 128;                     // 128 rows x 64 BF16: one 128-byte-row slab
  static constexpr int kStepRows = 128;
  static constexpr int kStages = 3;
  static constexpr int kWG = 4, kCompute = 128 * kWG, kLoaderWarp = 4 + 4 * kWG, kThreads = 128 + kCompute + 32;  // warp 0: stage producer; warps 1, 2, 3: MMA issuers (S^T; second stage; dP^T); 16 compute warps; last warp: K / V tile loader
  static constexpr uint32_t kColX = 0, kColY = 128, kColZ = 256, kColAcc0 = 384, kColAcc1 = 448;
  static constexpr int kTmemCols = 512;
  // K, V resident, ring of (Q, dO, Z, two 64-row blocks of the row-constant tile) step tiles, staging (dK, dV)
  static constexpr int kExtBytes = 2 * kExtBlockBytes;             // 128 rows x 16 BF16 columns
  static constexpr int kDkvStageBytes = 3 * kTileBytes + kExtBytes;
  static constexpr int kDkvSmemBytes = 2 * kTileBytes + kStages * kDkvStageBytes + 2 * kTileBytes + 1024;
  static_assert(kDkvSmemBytes <= 227 * 1024, "shared memory budget");
};

enum BwdW128WaitCode {
  kWkRes = 0x51, kWkQ = 0x52, kWkQEmpty = 0x53, kWkS = 0x54, kWkDP = 0x55, kWkR = 0x56, kWkT = 0x57, kWkSFree = 0x58, kWkYFree = 0x59,
  kWkAcc = 0x5a, kWkAccFree = 0x5b, kWkResFree = 0x5c
};

// Arithmetic of one 16-column chunk of the dK/dV side (thread <-> key row, columns = queries), Algorithm 1 lines 5-8:
//   p = exp2((x - LSE / alpha) * (alpha log2 e)),  r = BF16(p),  t = BF16(fl32[p * (dP - D)]).
// Both row constants arrive with the products: the score product carries one extra K = 16 slice whose operands are a
// constant matrix of ones (three columns) and the step's row-constant tile, so xs holds x - LSE / alpha and xp holds
// dP - D, accumulated in FP32 by the tensor core (the three BF16 pieces of a constant add up to its FP32 value; the
// subtraction is rounded by the accumulator instead of by an add.rn: a different last bit at most).  Reading the
// constants per column from shared memory instead cost this kernel 14 % (every lane needs every column's value).
// With MASKED, column c is dropped when c < lim (a query before this key) or c > hi (past the sequence's last query);
// a dropped column gets t = 0 explicitly, because its constants may be arbitrary bits.  The packed operands go over the
// chunk's own S^T columns: r the first eight, t the last eight.
template <bool MASKED>
__device__ __forceinline__ void dkv_chunk(uint32_t tS, const uint32_t (&xs)[16], const uint32_t (&xp)[16], float scale_log2, int lim, int hi) {
  const uint64_t scale2 = f32x2(scale_log2, scale_log2);
  uint32_t pr[8], pt[8];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float a[4], p[4], t[4];
    f32x2_split(mul2(f32x2_bits(xs[4 * i], xs[4 * i + 1]), scale2), a[0], a[1]);
    f32x2_split(mul2(f32x2_bits(xs[4 * i + 2], xs[4 * i + 3]), scale2), a[2], a[3]);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      p[e] = fast_exp2(a[e]);
      if (MASKED && (4 * i + e < lim || 4 * i + e > hi)) p[e] = 0.f;
    }
    f32x2_split(mul2(f32x2(p[0], p[1]), f32x2_bits(xp[4 * i], xp[4 * i + 1])), t[0], t[1]);
    f32x2_split(mul2(f32x2(p[2], p[3]), f32x2_bits(xp[4 * i + 2], xp[4 * i + 3])), t[2], t[3]);
    if (MASKED) {
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if (p[e] == 0.f) t[e] = 0.f;
    }
    pr[2 * i] = pack_bf16x2(p[0], p[1]);
    pr[2 * i + 1] = pack_bf16x2(p[2], p[3]);
    pt[2 * i] = pack_bf16x2(t[0], t[1]);
    pt[2 * i + 1] = pack_bf16x2(t[2], t[3]);
  }
  tmem_st8(tS, pr);
  tmem_st8(tS + 8, pt);
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
  uint8_t *sStage = sV + C::kTileBytes;   // stage s: Q, dO, Z step tiles, then the step's row-constant tile (two 64-row blocks)
  uint8_t *sOut = sStage + S * C::kDkvStageBytes;   // staging: dK tile, then dV tile

  __shared__ uint64_t bar_res_full, bar_res_free, bar_q_full[S], bar_q_empty[S];
  __shared__ uint64_t bar_s_full[2], bar_rt_ready[2][2], bar_dp_full, bar_y_free;
  __shared__ uint64_t bar_acc_done, bar_acc_free, bar_drain[3];
  __shared__ uint32_t tmem_base_smem;
  __shared__ int cta_abort, cta_skip;
  // Constant operand of the extra K = 16 slice: three eight-row core matrices (zeros, rows of (1, 1, 1, 0, 0, 0, 0, 0), zeros).
  // S^T reads (ones, zeros): it adds columns 0..2 of the row-constant tile; dP^T reads (zeros, ones): columns 8..10.
  __shared__ __align__(128) uint4 s_ones[24];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) cta_skip = *reinterpret_cast<volatile int *>(status);
  __syncthreads();
  if (cta_skip != 0) return;

  const bool use_z = (flags & kFlagNoKCorrection) == 0;
  const uint32_t stage_tx = (use_z ? 3 : 2) * C::kTileBytes + C::kExtBytes;
  if (threadIdx.x < 24) {
    s_ones[threadIdx.x] = (threadIdx.x >= 8 && threadIdx.x < 16) ? make_uint4(0x3f803f80u, 0x00003f80u, 0u, 0u) : make_uint4(0u, 0u, 0u, 0u);
    fence_proxy_async_smem();
  }

  AbortState ab{status, &cta_abort};
  if (threadIdx.x == 0) {
    cta_abort = 0;
    mbar_init(&bar_res_full, 1);
    mbar_init(&bar_res_free, 2);   // the last S^T product (issuer 1) and the last dP^T product (issuer 2): the epilogue never touches K / V
    for (int s = 0; s < S; ++s) { mbar_init(&bar_q_full[s], 1); mbar_init(&bar_q_empty[s], 1); }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&bar_s_full[b], 1);
      mbar_init(&bar_rt_ready[b][0], C::kCompute); mbar_init(&bar_rt_ready[b][1], C::kCompute);
    }
    mbar_init(&bar_dp_full, 1);
    mbar_init(&bar_y_free, C::kCompute);
    mbar_init(&bar_acc_done, 1);
    mbar_init(&bar_acc_free, C::kCompute);
    mbar_init(&bar_drain[0], 1);
    mbar_init(&bar_drain[1], 1);
    mbar_init(&bar_drain[2], 1);
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
          // two 64-row blocks of the row-constant tile (the second may lie past the sequence's last block: its columns are masked)
          bulk_load_1d(dst + 3 * C::kTileBytes, reinterpret_cast<const uint8_t *>(stats) + (static_cast<size_t>(qh) * nblk + tl.blk0 + (qrel >> 6)) * kExtBlockBytes,
                       C::kExtBytes, &bar_q_full[st]);
        }
      }
      if (cta_abort) {
        for (int q = (g > S ? g - S : 0); q < g; ++q)
          for (int spin = 0; spin < 100000 && !mbar_try_wait(&bar_q_full[q % S], (q / S) & 1); ++spin) {}
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- tensor-core issuer 1: S^T = K Q^T, dP^T = V dO^T
    constexpr uint32_t idesc_s = idesc_bf16_f32(128, 128, 0, 0);   // [128 keys] x [128 queries], contraction over d
    const SmemDesc dscK = make_smem_desc(smem_u32(sK), 16, 1024), dscV = make_smem_desc(smem_u32(sV), 16, 1024);
    const SmemDesc dscQ0 = make_smem_desc(smem_u32(sStage), 16, 1024);
    const SmemDesc dscOnes = make_smem_desc_noswizzle(smem_u32(s_ones) + 128, 128, 0);                 // (ones, zeros), every row group the same
    const SmemDesc dscExt0 = make_smem_desc_noswizzle(smem_u32(sStage + 3 * C::kTileBytes), 128, 256);
    int g = 0, ti = 0;
    for (int lin = sched.next(); lin >= 0; lin = sched.next(), ++ti) {
      const int T = G * steps_of(tile_of(lin));
      mbar_wait(&bar_res_full, ti & 1, ab, kWkRes);
      for (int n = 0; n < T; ++n, ++g) {
        const int st = g % S, sb = g & 1;
        mbar_wait(&bar_q_full[st], (g / S) & 1, ab, kWkQ);
        if (g >= 2) mbar_wait(&bar_q_empty[(g - 2) % S], ((g - 2) / S) & 1, ab, kWkSFree);   // step g - 2 done: its r, t are consumed
        tc_fence_after();
        const SmemDesc dscQ = dscQ0.advanced(st * C::kDkvStageBytes), dscdO = dscQ.advanced(C::kTileBytes);
        const uint32_t tS = tmem_base + (sb ? C::kColZ : C::kColX);
        if (elect_one_sync()) {
#pragma unroll
          for (int k = 0; k < D / 16; ++k) umma_ss(tS, dscK.at(k * 32), dscQ.at(k * 32), idesc_s, k > 0);
          umma_ss(tS, dscOnes.at(0), dscExt0.at(st * C::kDkvStageBytes), idesc_s, 1u);   // - LSE / alpha in every key row
          umma_commit(&bar_s_full[sb]);
        }
        __syncwarp();
        if (n == T - 1) {
          if (elect_one_sync()) umma_commit(&bar_res_free);   // first of two arrivals: no score product reads this K tile any more
          __syncwarp();
        }
      }
    }
    drain_mmas_if_aborted(&bar_drain[0], ab);
  } else if (warp == 3) {
    // ---------------------------------------------------------------- tensor-core issuer 3: dP^T = V dO^T
    // A warp of its own: the tensor core takes its work in the order it is issued and an issuing thread is held for as
    // long as its products execute, so dP^T of step g + 1 -- which the ALUs want the moment they finish step g, and which
    // may be written as soon as they hold dP^T of step g in registers -- must neither wait behind this step's S^T (whose
    // buffer frees late) in one thread's program order nor behind the second-stage products in another's.
    constexpr uint32_t idesc_s = idesc_bf16_f32(128, 128, 0, 0);
    const SmemDesc dscV = make_smem_desc(smem_u32(sV), 16, 1024);
    const SmemDesc dscQ0 = make_smem_desc(smem_u32(sStage), 16, 1024);
    const SmemDesc dscOnes = make_smem_desc_noswizzle(smem_u32(s_ones), 128, 0);                       // (zeros, ones)
    const SmemDesc dscExt0 = make_smem_desc_noswizzle(smem_u32(sStage + 3 * C::kTileBytes), 128, 256);
    int g = 0, ti = 0;
    for (int lin = sched.next(); lin >= 0; lin = sched.next(), ++ti) {
      const int T = G * steps_of(tile_of(lin));
      mbar_wait(&bar_res_full, ti & 1, ab, kWkRes);
      for (int n = 0; n < T; ++n, ++g) {
        const int st = g % S;
        mbar_wait(&bar_q_full[st], (g / S) & 1, ab, kWkQ);
        if (g >= 1) mbar_wait(&bar_y_free, (g - 1) & 1, ab, kWkYFree);               // the ALUs hold dP^T of step g - 1 in registers
        tc_fence_after();
        const SmemDesc dscdO = dscQ0.advanced(st * C::kDkvStageBytes + C::kTileBytes);
        if (elect_one_sync()) {
#pragma unroll
          for (int k = 0; k < D / 16; ++k) umma_ss(tmem_base + C::kColY, dscV.at(k * 32), dscdO.at(k * 32), idesc_s, k > 0);
          umma_ss(tmem_base + C::kColY, dscOnes.at(0), dscExt0.at(st * C::kDkvStageBytes), idesc_s, 1u);   // - D in every key row
          umma_commit(&bar_dp_full);
          if (n == T - 1) umma_commit(&bar_res_free);   // second of two arrivals: no product reads this V tile any more
        }
        __syncwarp();
      }
    }
    drain_mmas_if_aborted(&bar_drain[2], ab);
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
        // Every compute thread finishes the first 64 query columns of the step (k = 0..3) before the last 64, and hands
        // the two halves over separately: the products of the first half run while the second half is in the ALUs.
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          mbar_wait(&bar_rt_ready[sb][h], (g >> 1) & 1, ab, kWkR);
          tc_fence_after();
          if (elect_one_sync()) {
            if (use_z) {
              // the dO and Z step tiles are adjacent 64-column atoms of one MN-major operand and the dV and dK accumulators
              // are adjacent TMEM columns: r^T [dO | -BF16(lambda Q)] is ONE N = 128 product (Algorithm 1 lines 17-18)
#pragma unroll
              for (int k = 4 * h; k < 4 * h + 4; ++k)
                umma_ts(tmem_base + C::kColAcc0, tR + 16 * k, dscdO.at(k * 2048), idesc_fused, k > 0 ? 1u : acc);
            } else {
#pragma unroll
              for (int k = 4 * h; k < 4 * h + 4; ++k)      // dV += r^T dO
                umma_ts(tmem_base + C::kColAcc0, tR + 16 * k, dscdO.at(k * 2048), idesc_a, k > 0 ? 1u : acc);
            }
            const uint32_t acc_k = use_z ? 1u : acc;         // with the correction, dK already holds this step's r^T Z
#pragma unroll
            for (int k = 4 * h; k < 4 * h + 4; ++k)          // dK += t^T Q
              umma_ts(tmem_base + C::kColAcc1, tT + 16 * k, dscQ.at(k * 2048), idesc_a, k > 0 ? 1u : acc_k);
            if (h == 1) {
              umma_commit(&bar_q_empty[st]);               // step done: its stage and its S^T buffer are free
              if (p == T - 1) umma_commit(&bar_acc_done);
            }
          }
          __syncwarp();
        }
      }
    }
    drain_mmas_if_aborted(&bar_drain[1], ab);
  } else if (warp == C::kLoaderWarp) {
    // ---------------------------------------------------------------- TMA loader of the stationary (K, V) tiles.  A warp of its
    // own: as a second lane of the stage producer's warp its loads at a tile boundary waited for the producer's polling loop.
    if (lane == 0) {
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
  } else {
    // ---------------------------------------------------------------- compute: thread <-> (key row, 32-query slice of every step)
    const int wg = (warp - 4) >> 2;
    const int row = 32 * (warp & 3) + lane;                  // key row within the tile
    const uint32_t lane_addr = static_cast<uint32_t>(32 * (warp & 3)) << 16;
    int g0 = 0, ti = 0;
    for (int lin = sched.next(); lin >= 0; lin = sched.next(), ++ti) {
      const TileInfo tl = tile_of(lin);
      const int bh = hix(lin), Th = steps_of(tl), T = G * Th, q_start = q_start_of(tl);
#ifdef GPROJ_TRACE
      const unsigned long long ev_n0 = global_ns(); const long long ev_c0 = clock64(); unsigned long long ev_n1 = 0;
#endif
      for (int n = 0; n < T; ++n) {
        const int g = g0 + n, sb = g & 1;
        // This thread's two 16-column chunks: columns 16 w .. 16 w + 15 of the step's first 64 queries, then of its last 64
        // (operand slices k = w and k = 4 + w).
        const int cb = 16 * wg;
        const uint32_t tS0 = tmem_base + lane_addr + (sb ? C::kColZ : C::kColX) + 16 * wg, tS1 = tS0 + 64;
        const uint32_t tdP0 = tmem_base + lane_addr + C::kColY + 16 * wg, tdP1 = tdP0 + 64;
        constexpr int kChunk1 = 64;
        const int nh = n % Th;                                              // step within the current query head
        const int Lq = tl.oseq_end - tl.oseq0, off = (tl.seq_end - tl.seq0) - Lq, krel0 = tl.row0 - tl.seq0;
        const int qs = q_start + nh * C::kStepRows;                         // first query (inside its sequence) of the step
        const int q0 = qs + cb;                                             // ... of this thread's first chunk
        const bool masked = (CAUSAL && qs < krel0 + 128 - off) || qs + C::kStepRows > Lq;
        const int lim = CAUSAL ? krel0 + row - off - q0 : 0, hi = Lq - 1 - q0;
        // dP^T of both chunks and S^T of the first go to registers at the start of the step; dP^T (single-buffered) is then
        // released to the tensor core.
        mbar_wait(&bar_s_full[sb], (g >> 1) & 1, ab, kWkS);
        mbar_wait(&bar_dp_full, g & 1, ab, kWkDP);
        tc_fence_after();
#ifdef GPROJ_TRACE
        if (n == 0) ev_n1 = global_ns();
#endif
        uint32_t xp[32], xs[16];
        tmem_ld16(tdP0, *reinterpret_cast<uint32_t (*)[16]>(&xp[0]));
        tmem_ld16(tdP1, *reinterpret_cast<uint32_t (*)[16]>(&xp[16]));
        tmem_ld16(tS0, xs);
        tmem_wait_ld();
        tc_fence_before();
        mbar_arrive(&bar_y_free);                   // dP^T is in registers: the tensor core may write the next step's
        if (masked) dkv_chunk<true>(tS0, xs, *reinterpret_cast<const uint32_t (*)[16]>(&xp[0]), scale_log2, lim, hi);
        else        dkv_chunk<false>(tS0, xs, *reinterpret_cast<const uint32_t (*)[16]>(&xp[0]), scale_log2, 0, 0);
        tmem_ld16(tS1, xs);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&bar_rt_ready[sb][0]);
        tmem_wait_ld();
        if (masked) dkv_chunk<true>(tS1, xs, *reinterpret_cast<const uint32_t (*)[16]>(&xp[16]), scale_log2, lim - kChunk1, hi - kChunk1);
        else        dkv_chunk<false>(tS1, xs, *reinterpret_cast<const uint32_t (*)[16]>(&xp[16]), scale_log2, 0, 0);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&bar_rt_ready[sb][1]);
      }

#ifdef GPROJ_TRACE
      const unsigned long long ev_n2 = global_ns();
#endif
      mbar_wait(&bar_acc_done, ti & 1, ab, kWkAcc);
      tc_fence_after();
      uint8_t *stage_dk = sOut, *stage_dv = sOut + C::kTileBytes;
      uint32_t a[16], b[16];
      tmem_ld16(tmem_base + C::kColAcc0 + lane_addr + 16 * wg, a);
      tmem_ld16(tmem_base + C::kColAcc1 + lane_addr + 16 * wg, b);
      tmem_wait_ld();
      tc_fence_before();
      mbar_arrive(&bar_acc_free);          // the accumulators may be overwritten by the next tile
      if (threadIdx.x == 128) bulk_wait_group_read0();   // the previous tile's stores have left the staging buffer
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
        if (threadIdx.x == 128) {
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
#ifdef GPROJ_TRACE
      if ((threadIdx.x & 127) == 0 && wg == 0) tile_event(8, lin, T, ev_n0, ev_n1, ev_n2, global_ns(), ev_c0, clock64());
#endif
      g0 += T;
    }
    if (threadIdx.x == 128) bulk_wait_group_read0();
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, C::kTmemCols);
}

}  // namespace gproj
