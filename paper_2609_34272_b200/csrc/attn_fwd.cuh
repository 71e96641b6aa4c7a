// Fused attention forward for sm_100a: O = softmax(alpha Q K^T) V and the row log-sum-exp.
//
// A persistent CTA (one per SM) walks a static list of work items.  Roles (384 threads):
//   warp 0        TMA producer of the streamed K_j / V_j tiles (separate barriers: S needs only K, P~V only V)
//   warp 1        tensor-core issuer 1: S_t = Q K_j^T (N = 128, FP32 in TMEM); owns TMEM
//   warp 2        tensor-core issuer 2: O_t += P~_t V_j with the BF16 probabilities read straight from TMEM
//   warp 3        TMA loader of the stationary Q tile(s)
//   warps 4..7    softmax warpgroup 0, warps 8..11 softmax warpgroup 1: thread <-> query row (TMEM lane), so every
//                 row statistic is a private register.  While one warpgroup is in the ALUs the tensor core works for
//                 the other one (the tensor-core queue is only 1-2 instructions deep, hence two issuing warps: each
//                 one's barrier polls overlap the other's MMAs).
// Work items (template parameter MODE):
//   pairs (0, 1)  one item = two 128-row query tiles of one (batch, head), warpgroup t <-> tile t, every K / V tile
//                 serves both; with MODE 1 the warpgroups also take turns in the exponential phase.
//   split (2)     one item = one query tile; warpgroup t takes the key tiles j = t (mod 2) with its own running
//                 maximum, normaliser and accumulator, and warpgroup 0 merges the two halves at the end.  Used when
//                 pairs would leave SMs idle and for packed sequences.
// Softmax arithmetic (FMA_SOFTMAX = false, the default): online softmax on the UNSCALED logits with the
// subtract-before-scale rounding of
// Eq. "gproj-forward": z = exp2(fl32[ fl32(x - x_max) * (alpha log2 e) ]); l accumulates the FP32 z, the value
// product uses BF16(z); the running maximum is raised lazily and the accumulator rescaled only then.
// The saved state is BF16 O (staged in the TMA layout over the consumed Q tile, written by a TMA store) and
// FP32 LSE = alpha x_max + ln l  (Algorithm 1, "Input").
// TMEM: S_0, S_1 (128 columns each), O_0, O_1 (d each); at d = 64 the packed P~_t have their own 64 columns, so
// S_t of the next key tile can be issued as soon as the softmax has copied the current one to registers; at d = 128
// TMEM is full and P~_t overwrites the first half of S_t.
#pragma once
#include "attn_bwd.cuh"   // TileSched
#include "sm100_primitives.cuh"

namespace gproj {

// Floor of the running row maximum (see the softmax loop): far below any score, far above -FLT_MAX.
constexpr float kFwdMaxFloor = -1.0e30f;

template <int D>
struct FwdCfg {
  static constexpr int kBlockM = 128;                  // rows of one query tile (two per work item)
  static constexpr int kBlockN = 128;
  static constexpr int kSlabs = D / 64;                // 64-column (128-byte) swizzle slabs per tile
  static constexpr int kSlabBytes = 128 * 128;         // 128 rows x 128 B
  static constexpr int kTileBytes = kSlabs * kSlabBytes;
  static constexpr int kStages = (D == 64) ? 4 : 2;    // ring of (K, V) tile pairs
  static constexpr int kSmemBytes = 2 * kTileBytes + kStages * 2 * kTileBytes + 1024;
  static constexpr int kTmemCols = 512;
  static constexpr bool kSepP = (D == 64);             // P~ in its own TMEM columns
  static constexpr uint32_t kColS = 0, kColO = 256, kColP = 256 + 2 * D;   // S_t at 128 t, O_t at 256 + D t, P_t at kColP + 64 t
  static constexpr int kThreads = 384;
};

enum FwdWaitCode {
  kFwdWaitQ = 0x11, kFwdWaitK = 0x12, kFwdWaitV = 0x13, kFwdWaitKVEmpty = 0x14, kFwdWaitS = 0x15, kFwdWaitP = 0x16,
  kFwdWaitPV = 0x17, kFwdWaitSFree = 0x18, kFwdWaitOFree = 0x19, kFwdWaitQFree = 0x1a, kFwdWaitTurn = 0x1b, kFwdWaitMerge = 0x1c
};


// z = exp2(fl32[(x - x_max) (alpha log2 e)]) for the 128 columns of one row (two columns per packed FP32 instruction:
// the subtraction and the scale keep their separate roundings, add.rn / mul.rn; the fused variant of
// Eq. "historical-fma" is one fma.rn), BF16 pairs stored to TMEM at tP, returns the FP32 row sum of z (four packed
// partial sums).
template <bool FMA_SOFTMAX>
__device__ __forceinline__ float softmax_exp_store(const uint32_t (&xr)[4][32], uint32_t tP, float m_new, float scale_log2, float m_scaled) {
  const uint64_t negm2 = f32x2(-m_new, -m_new), scale2 = f32x2(scale_log2, scale_log2), negms2 = f32x2(-m_scaled, -m_scaled);
  uint64_t rs2[2] = {f32x2(0.f, 0.f), f32x2(0.f, 0.f)};
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    uint32_t pk[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const uint64_t x2 = f32x2_bits(xr[c][2 * i], xr[c][2 * i + 1]);
      const uint64_t a2 = FMA_SOFTMAX ? fma2(x2, scale2, negms2) : mul2(add2(x2, negm2), scale2);
      float a0, a1;
      f32x2_split(a2, a0, a1);
      const float z0 = fast_exp2(a0), z1 = fast_exp2(a1);
      rs2[i & 1] = add2(rs2[i & 1], f32x2(z0, z1));
      pk[i] = pack_bf16x2(z0, z1);
    }
    tmem_st16(tP + 16 * c, pk);
  }
  float r0, r1, r2, r3;
  f32x2_split(rs2[0], r0, r1);
  f32x2_split(rs2[1], r2, r3);
  return (r0 + r1) + (r2 + r3);
}

// MODE: 0 = pairs of query tiles, 1 = pairs whose warpgroups take turns in the exponential phase, 2 = single tiles with
// the key range split between the warpgroups.
template <int D, bool CAUSAL, bool FMA_SOFTMAX, int MODE>
__global__ void __launch_bounds__(384, 1)
attn_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO,
                __nv_bfloat16 *__restrict__ Og, const int4 *__restrict__ plan, float *__restrict__ LSE, int N, int Nk, int BH, int Hq, int G, int tiles_per_item, int total_items, const ItemOrder order, float scale_log2, float alpha,
                int *status) {
  using C = FwdCfg<D>;
  constexpr int S = C::kStages;
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t *sQ = smem;                              // tile 0, then tile 1 (each later reused to stage O_t)
  uint8_t *sKV = sQ + 2 * C::kTileBytes;            // stage s: K tile, then V tile

  __shared__ int s_item[4][2];
  __shared__ uint64_t bar_q_full[2], bar_q_free[2], bar_k_full[S], bar_v_full[S], bar_kv_empty[S];
  __shared__ uint64_t bar_s_full[2], bar_s_free[2], bar_p_ready[2], bar_pv_done[2], bar_o_free[2], bar_turn[2], bar_merge, bar_drain[2];
  __shared__ float s_m1[2][128], s_l1[2][128];   // split mode: running maximum and normaliser of the second warpgroup
  __shared__ uint32_t tmem_base_smem;
  __shared__ int cta_abort, cta_skip;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) cta_skip = *reinterpret_cast<volatile int *>(status);
  __syncthreads();
  if (cta_skip != 0) return;   // an earlier wait gave up: drain the rest of the grid quickly

  const int n_qt = (N + C::kBlockM - 1) / C::kBlockM;   // the last tile may be ragged: rows past N load as zero, stores clip
  const int TPI = tiles_per_item;                  // 2: a pair of query tiles per work item; 1: single tiles, key range split
  constexpr bool split = (MODE == 2);              // one query tile; warpgroup t takes the key tiles j = t (mod 2), merged at the end
  constexpr bool TURNS = (MODE == 1);
  const int n_pairs = (n_qt + TPI - 1) / TPI;
  AbortState ab{status, &cta_abort};
  if (threadIdx.x == 0) {
    cta_abort = 0;
    mbar_init(&bar_merge, 128);
    for (int b = 0; b < 2; ++b) {
      mbar_init(&bar_q_full[b], 1);
      mbar_init(&bar_q_free[b], tiles_per_item);    // one arrival per query tile slot: its O store has left shared memory
    }
    for (int s = 0; s < S; ++s) { mbar_init(&bar_k_full[s], 1); mbar_init(&bar_v_full[s], 1); mbar_init(&bar_kv_empty[s], 1); }
    for (int t = 0; t < 2; ++t) {
      mbar_init(&bar_drain[t], 1);
      mbar_init(&bar_s_full[t], 1); mbar_init(&bar_s_free[t], 128); mbar_init(&bar_p_ready[t], 128); mbar_init(&bar_pv_done[t], 1); mbar_init(&bar_o_free[t], 128); mbar_init(&bar_turn[t], 128);
    }
    fence_mbar_init();
  }
  if (warp == 1) { tmem_alloc(&tmem_base_smem, C::kTmemCols); tmem_relinquish(); }
  if (warp == 0 && lane == 0) { tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV); tma_prefetch_desc(&tmO); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = __shfl_sync(0xffffffffu, tmem_base_smem, 0);   // the shuffle marks it warp-uniform

  // Work items ordered by decreasing work (causal: last pair first).  Item -> (sequence, first query tile, tiles) and head.
  // Dense calls: one sequence [0, N) per head, items are pairs (or single tiles); packed calls: single tiles from the plan.
  // qt0: index of the first query tile inside its sequence; nq: query tiles; n_kt: key tiles walked; kseq0, klen: the keys.
  // Causal support of query i: keys j <= i + off with off = klen - len (the diagonal ends at the last query and last key).
  struct Item { int seq0, len, qt0, nq, n_kt, kseq0, klen, off; };
  auto tix = [&](int lin) { return order.rank(lin); };
  auto hix = [&](int lin) { return order.head(lin); };
  TileSched sched(total_items);
  auto decode_rank = [&](int rank) {       // rank: position of the item's tile (pair) in its head's list, longest first
    Item it;
    if (plan != nullptr) {
      const TileInfo ti = tile_info(plan, rank, 0, N, Nk);
      it.seq0 = ti.seq0; it.len = ti.seq_end - ti.seq0; it.qt0 = (ti.row0 - ti.seq0) / C::kBlockM; it.nq = 1;
      it.kseq0 = ti.oseq0; it.klen = ti.oseq_end - ti.oseq0;
    } else {
      const int pair = CAUSAL ? (n_pairs - 1 - rank) : rank;
      it.seq0 = 0; it.len = N; it.qt0 = TPI * pair; it.nq = min(TPI, n_qt - it.qt0);
      it.kseq0 = 0; it.klen = Nk;
    }
    it.off = it.klen - it.len;
    // key tiles up to the last key the item's last row sees; at least one (fully masked if the item sees no key at all)
    const int kend = CAUSAL ? min(it.klen, (it.qt0 + it.nq) * C::kBlockM + it.off) : it.klen;
    it.n_kt = max(1, (max(kend, 0) + C::kBlockN - 1) / C::kBlockN);
    return it;
  };
  auto decode = [&](int lin) { return decode_rank(tix(lin)); };
  // query tile t of the item takes part in key step j?  (key tile 0 always, so that every tile has a first step)
  auto active = [&](const Item &it, int t, int j) {
    return t < it.nq && (!CAUSAL || j <= max(0, ((it.qt0 + t) * C::kBlockM + C::kBlockM - 1 + it.off) >> 7));
  };

  // Q buffers: a pair item fills both tile slots of the one buffer; single-tile items (split mode) alternate between the
  // two slots, so that the next item's Q is loaded, and its first scores are computed, during this item's epilogue.
  auto q_buf = [&](int ti) { return split ? (ti & 1) : 0; };
  auto q_use = [&](int ti) { return split ? (ti >> 1) : ti; };      // how often the buffer has been used before item ti

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer of K_j, V_j
    if (lane == 0) {
      int g = 0;
      for (int lin = sched.next(); lin >= 0; lin = sched.next()) {
        const Item it = decode(lin);
        const int bh = hix(lin), T = it.n_kt;
        for (int j = 0; j < T; ++j, ++g) {
          const int st = g % S;
          if (g >= S) mbar_wait(&bar_kv_empty[st], ((g / S) - 1) & 1, ab, kFwdWaitKVEmpty);
          uint8_t *dK = sKV + st * 2 * C::kTileBytes, *dV = dK + C::kTileBytes;
          const int kvh = kv_head_of(bh, Hq, G), krow = it.kseq0 + j * C::kBlockN;   // grouped-query: the group's shared K / V head
          mbar_expect_tx(&bar_k_full[st], C::kTileBytes);
          for (int s = 0; s < C::kSlabs; ++s) tma_load_3d(dK + s * C::kSlabBytes, &tmK, &bar_k_full[st], s * 64, krow, kvh);
          mbar_expect_tx(&bar_v_full[st], C::kTileBytes);
          for (int s = 0; s < C::kSlabs; ++s) tma_load_3d(dV + s * C::kSlabBytes, &tmV, &bar_v_full[st], s * 64, krow, kvh);
        }
      }
      // Every load is consumed by an MMA the epilogue waits for, so nothing is in flight at exit unless the
      // CTA aborted; then give the copies a bounded chance to land before shared memory is released.
      if (cta_abort) {
        for (int q = (g > S ? g - S : 0); q < g; ++q) {
          for (int spin = 0; spin < 100000 && !mbar_try_wait(&bar_k_full[q % S], (q / S) & 1); ++spin) {}
          for (int spin = 0; spin < 100000 && !mbar_try_wait(&bar_v_full[q % S], (q / S) & 1); ++spin) {}
        }
      }
    }
  } else if (warp == 3) {
    // ---------------------------------------------------------------- TMA loader of the stationary Q pair
    if (lane == 0) {
      int ti = 0;
      for (int lin = sched.next(); lin >= 0; lin = sched.next(), ++ti) {
        const Item it = decode(lin);
        const int bh = hix(lin), tiles = it.nq;
        const int qb = q_buf(ti), use = q_use(ti);
        if (use >= 1) mbar_wait(&bar_q_free[qb], (use - 1) & 1, ab, kFwdWaitQFree);
        // The softmax warps (168 registers, the kernel's tightest code) take the item's rank and head from here instead
        // of decoding the item number themselves; the barrier's completion publishes the two words.  The loader is at
        // most two items ahead of them, the ring has four entries.
        s_item[ti & 3][0] = tix(lin);
        s_item[ti & 3][1] = bh;
        mbar_expect_tx(&bar_q_full[qb], tiles * C::kTileBytes);
        for (int t = 0; t < tiles; ++t)
          for (int s = 0; s < C::kSlabs; ++s)
            tma_load_3d(sQ + (qb + t) * C::kTileBytes + s * C::kSlabBytes, &tmQ, &bar_q_full[qb], s * 64, it.seq0 + (it.qt0 + t) * C::kBlockM, bh);
      }
      if (cta_abort)
        for (int q = (ti > 2 ? ti - 2 : 0); q < ti; ++q)
          for (int spin = 0; spin < 100000 && !mbar_try_wait(&bar_q_full[q_buf(q)], q_use(q) & 1); ++spin) {}
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- tensor-core issuer 1: S_t = Q_t K_j^T
    // The whole warp runs this loop so that every address stays provably warp-uniform (descriptor operands
    // then live in uniform registers); one elected lane issues the MMAs and commits.
    constexpr uint32_t idesc_s = idesc_bf16_f32(128, 128, 0, 0);   // both operands K-major
    const SmemDesc dscQ0 = make_smem_desc(smem_u32(sQ), 16, 1024);
    const SmemDesc dscK0 = make_smem_desc(smem_u32(sKV), 16, 1024);
    int g = 0, ti = 0, cnt[2] = {0, 0};
    for (int lin = sched.next(); lin >= 0; lin = sched.next(), ++ti) {
      const Item it = decode(lin);
      const int T = it.n_kt;
      const int qb = q_buf(ti);
      mbar_wait(&bar_q_full[qb], q_use(ti) & 1, ab, kFwdWaitQ);
      for (int j = 0; j < T; ++j, ++g) {
        const int st = g % S;
        mbar_wait(&bar_k_full[st], (g / S) & 1, ab, kFwdWaitK);
        const SmemDesc dscK = dscK0.advanced(st * 2 * C::kTileBytes);
#pragma unroll
        for (int t = 0; t < 2; ++t) {
          if (split ? ((j & 1) != t) : !active(it, t, j)) continue;
          // S_t may be overwritten once its previous contents are dead: copied to registers by the softmax (P~ has its
          // own columns), or, when P~ lives in the same columns, consumed by the previous P~V product.
          if (cnt[t] > 0) {
            if (C::kSepP) mbar_wait(&bar_s_free[t], (cnt[t] - 1) & 1, ab, kFwdWaitSFree);
            else          mbar_wait(&bar_pv_done[t], (cnt[t] - 1) & 1, ab, kFwdWaitSFree);
          }
          tc_fence_after();
          const SmemDesc dscQ = dscQ0.advanced((split ? qb : t) * C::kTileBytes);
          if (elect_one_sync()) {
#pragma unroll
            for (int k = 0; k < D / 16; ++k) {
              const uint32_t off = (k / 4) * C::kSlabBytes + (k % 4) * 32;
              umma_ss(tmem_base + C::kColS + 128 * t, dscQ.at(off), dscK.at(off), idesc_s, k > 0);
            }
            umma_commit(&bar_s_full[t]);
          }
          __syncwarp();
          ++cnt[t];
        }
      }
    }
    drain_mmas_if_aborted(&bar_drain[0], ab);
  } else if (warp == 2) {
    // ---------------------------------------------------------------- tensor-core issuer 2: O_t += P~_t V_j
    constexpr uint32_t idesc_o = idesc_bf16_f32(128, D, 0, 1);     // V is MN-major (d contiguous)
    const SmemDesc dscV0 = make_smem_desc(smem_u32(sKV + C::kTileBytes), C::kSlabBytes, 1024);
    int g = 0, ti = 0, cnt[2] = {0, 0};
    for (int lin = sched.next(); lin >= 0; lin = sched.next(), ++ti) {
      const Item it = decode(lin);
      const int T = it.n_kt;
      for (int j = 0; j < T; ++j, ++g) {
        const int st = g % S;
        mbar_wait(&bar_v_full[st], (g / S) & 1, ab, kFwdWaitV);
        const SmemDesc dscV = dscV0.advanced(st * 2 * C::kTileBytes);
#pragma unroll
        for (int t = 0; t < 2; ++t) {
          if (split ? ((j & 1) != t) : !active(it, t, j)) continue;
          const bool first = split ? (j < 2) : (j == 0);     // first product into O_t in this work item
          if (first && ti > 0) mbar_wait(&bar_o_free[t], (ti - 1) & 1, ab, kFwdWaitOFree);   // previous epilogue has read O_t
          mbar_wait(&bar_p_ready[t], cnt[t] & 1, ab, kFwdWaitP);
          tc_fence_after();
          const uint32_t tP = tmem_base + (C::kSepP ? C::kColP + 64 * t : C::kColS + 128 * t);
          const uint32_t acc = first ? 0u : 1u;
          if (elect_one_sync()) {
#pragma unroll
            for (int k = 0; k < C::kBlockN / 16; ++k)
              umma_ts(tmem_base + C::kColO + D * t, tP + 8 * k, dscV.at(k * 2048), idesc_o, k > 0 ? 1u : acc);
            umma_commit(&bar_pv_done[t]);
          }
          __syncwarp();
          ++cnt[t];
        }
        if (elect_one_sync()) umma_commit(&bar_kv_empty[st]);    // every MMA that reads this K / V stage has been issued
        __syncwarp();
      }
    }
    drain_mmas_if_aborted(&bar_drain[1], ab);
  } else {
    // ---------------------------------------------------------------- softmax: warpgroup t <-> query tile t, thread <-> row
    const int t = (warp - 4) >> 2;
    const int row = 32 * (warp & 3) + lane;
    const uint32_t lane_addr = static_cast<uint32_t>(32 * (warp & 3)) << 16;
    const uint32_t tS = tmem_base + C::kColS + 128 * t + lane_addr;
    const uint32_t tO = tmem_base + C::kColO + D * t + lane_addr;
    const uint32_t tP = tmem_base + (C::kSepP ? C::kColP + 64 * t : C::kColS + 128 * t) + lane_addr;
    int ti = 0, cnt = 0, turn = 0;
    for (int lin = sched.next(); lin >= 0; lin = sched.next(), ++ti) {
      const int qb = q_buf(ti);
      mbar_wait(&bar_q_full[qb], q_use(ti) & 1, ab, kFwdWaitQ);   // the item's Q has landed, and with it its description
      const Item it = decode_rank(s_item[ti & 3][0]);
      const int bh = s_item[ti & 3][1], T = it.n_kt;
      const int qt = it.qt0 + (split ? 0 : t);        // this warpgroup's query tile inside the sequence
      // Masking, reduced to two numbers per tile: column c of key tile j is outside the row's support when
      // 128 j + c > rk, with rk the last key the row sees (causal diagonal and end of the keys, whichever comes first);
      // no key tile before jm needs the test for any row of the tile.
      const int rk = CAUSAL ? min(row + qt * C::kBlockM + it.off, it.klen - 1) : it.klen - 1;
      const int jl = CAUSAL ? max(0, (qt * C::kBlockM + C::kBlockM - 1 + it.off) >> 7) : T;   // last key tile of this query tile
      const int jm = CAUSAL ? min((qt * C::kBlockM + it.off + 1) >> 7, it.klen >> 7) : (it.klen >> 7);
      if (!split && t >= it.nq) {
        // Odd number of query tiles: the last pair has no second tile.  This warpgroup is in step with the item (it has
        // waited for its Q above), so it may hand back the slot without any barrier running ahead of its waiters.
        if (row == 0) mbar_arrive(&bar_q_free[0]);
        mbar_arrive(&bar_o_free[t]);
        continue;
      }
      float m_run = -INFINITY, l_run = 0.f;
#ifdef GPROJ_TRACE
      const unsigned long long ev_n0 = global_ns(); const long long ev_c0 = clock64();
#endif
      // Both tiles of the pair exist: the warpgroups alternate in the exponential phase, step by step, tile 0 first.
      const bool take_turns = TURNS && it.nq == 2;
      const int cnt_item0 = cnt;
      for (int j = split ? t : 0; j < T; j += split ? 2 : 1) {
        const bool first = split ? (j < 2) : (j == 0);     // this warpgroup's first key tile of the item
        if (!split && j > jl) {
          // no work in this step (causal: the first tile of the pair ends one key tile earlier): pass the turn on
          if (take_turns) {
            if (t == 1 || turn > 0) mbar_wait(&bar_turn[t], (t == 1 ? turn : turn - 1) & 1, ab, kFwdWaitTurn);
            mbar_arrive(&bar_turn[1 - t]);
            ++turn;
          }
          continue;
        }
        mbar_wait(&bar_s_full[t], cnt & 1, ab, kFwdWaitS);
        tc_fence_after();
        uint32_t xr[4][32];
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_ld32(tS + 32 * c, xr[c]);
        tmem_wait_ld();
        if (C::kSepP) { tc_fence_before(); mbar_arrive(&bar_s_free[t]); }   // the next S_t may be issued while this one is in the ALUs
        // Keys beyond the causal diagonal, and the zero-filled columns past the last key of a ragged tile, get -inf.
        if (j >= jm) {
          const int lim = rk - j * C::kBlockN;
#pragma unroll
          for (int c = 0; c < 4; ++c)
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (32 * c + i > lim) xr[c][i] = 0xff800000u;
        }
        // Row maximum over eight independent chains of three-input maxima (only two softmax warps share a scheduler, so a
        // 128-long dependent chain would be pure latency).
        float mxp[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) mxp[i] = fmaxf(__uint_as_float(xr[0][i]), __uint_as_float(xr[0][8 + i]));
#pragma unroll
        for (int e = 16; e < 128; e += 16)
#pragma unroll
          for (int i = 0; i < 8; ++i)
            mxp[i] = fmax3(mxp[i], __uint_as_float(xr[(e + i) >> 5][(e + i) & 31]), __uint_as_float(xr[(e + 8 + i) >> 5][(e + 8 + i) & 31]));
        // The floor keeps the maximum finite for a row that has seen no key yet (unequal lengths: rows before the causal
        // diagonal reaches key 0), so that such a row gives z = exp2(-inf) = 0 instead of NaN from (-inf) - (-inf).
        const float mx = fmax3(fmax3(mxp[0], mxp[1], mxp[2]), fmax3(mxp[3], mxp[4], mxp[5]), fmax3(mxp[6], mxp[7], kFwdMaxFloor));
        // Lazy maximum: the running maximum is only raised when the tile's maximum exceeds it by more than 8 in the
        // base-two exponent domain; otherwise the stale value stays (z <= 2^8, harmless in FP32 / BF16: O = acc / l and
        // LSE = alpha m + ln l do not depend on which reference m was subtracted) and neither l nor the accumulator
        // needs a rescale.  The first tile always sets it (m_run = -inf).  The fused variant always takes the true
        // running maximum, so that it is the arithmetic of Eq. "historical-fma" and nothing else.
        float m_new = fmaxf(m_run, mx);
#ifndef GPROJ_FWD_EAGER_MAX
        if (!FMA_SOFTMAX && __fmul_rn(__fsub_rn(m_new, m_run), scale_log2) <= 8.0f) m_new = m_run;
#endif
        const float corr = fast_exp2(__fmul_rn(__fsub_rn(m_run, m_new), scale_log2));
        // FMA_SOFTMAX reproduces the native fused form of Eq. "historical-fma": z = exp2(fma(x, a, -fl32(x_max a))),
        // in which x a is not rounded separately, so the largest score need not map to exactly zero.
        const float m_scaled = __fmul_rn(m_new, scale_log2);
        // P~ of the previous key tile must have been consumed (and O_t updated) before either is touched
        if (!first) { mbar_wait(&bar_pv_done[t], (cnt - 1) & 1, ab, kFwdWaitPV); tc_fence_after(); }
        // The exponential phase is the only heavy user of the special-function unit (16 results per clock per SM, the
        // forward's scarcest pipe).  With TURNS the two warpgroups alternate in it, so that one's exponentials run against
        // the other's loads, maxima and barrier work instead of both phases colliding and then both leaving the unit idle
        // (measured: +9 % at d = 128, -4 % at d = 64, so the host enables it for d = 128 with paired tiles only).
        if (take_turns) { if (t == 1 || turn > 0) mbar_wait(&bar_turn[t], (t == 1 ? turn : turn - 1) & 1, ab, kFwdWaitTurn); }
        const float rs = softmax_exp_store<FMA_SOFTMAX>(xr, tP, m_new, scale_log2, m_scaled);
        if (take_turns) { mbar_arrive(&bar_turn[1 - t]); ++turn; }
        l_run = l_run * corr + rs;
        if (!first && __any_sync(0xffffffffu, m_new != m_run)) {
#pragma unroll
          for (int c = 0; c < D / 32; ++c) {
            uint32_t o[32];
            tmem_ld32(tO + 32 * c, o);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * corr);
            tmem_st32(tO + 32 * c, o);
          }
        }
        m_run = m_new;
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&bar_p_ready[t]);
        ++cnt;
      }
#ifdef GPROJ_TRACE
      const unsigned long long ev_n2 = global_ns();
#endif
      // ---- epilogue: O = BF16(acc / l) staged in the TMA layout over this tile's Q, LSE = alpha x_max + ln l
      if (cnt > cnt_item0) { mbar_wait(&bar_pv_done[t], (cnt - 1) & 1, ab, kFwdWaitPV); tc_fence_after(); }
      if (split && t == 1) {
        // hand this half's statistics to warpgroup 0, which merges the two accumulators (l = 0: no key tiles here).
        // With two Q slots this warpgroup could finish a second item before warpgroup 0 has looked at the first one's
        // hand-over, and the merge barrier would be two phases ahead of its waiter; so it first waits until
        // warpgroup 0 has read the previous item's accumulators.
        if (ti > 0) mbar_wait(&bar_o_free[1], (ti - 1) & 1, ab, kFwdWaitOFree);
        s_m1[ti & 1][row] = m_run;
        s_l1[ti & 1][row] = l_run;
        tc_fence_before();
        mbar_arrive(&bar_merge);
#ifdef GPROJ_TRACE
        if (row == 0) tile_event(21, lin, T, ev_n0, ev_n0, ev_n2, global_ns(), ev_c0, clock64());
#endif
        continue;
      }
      // Split mode: O = (O_0 s_0 + O_1 s_1) / (l_0 s_0 + l_1 s_1) with s_t = exp2((m_t - max(m_0, m_1)) alpha log2 e).
      const bool has1 = split && T >= 2;               // the second warpgroup had at least one key tile
      float a0 = (l_run > 0.f) ? 1.0f / l_run : 0.f, a1 = 0.f;   // a row with an empty support has l = 0: O = 0
      if (split) {
        mbar_wait(&bar_merge, ti & 1, ab, kFwdWaitMerge);
        tc_fence_after();
        if (has1) {
          const float m1 = s_m1[ti & 1][row], l1 = s_l1[ti & 1][row];
          const float m = fmaxf(m_run, m1);
          const float s0 = fast_exp2(__fmul_rn(__fsub_rn(m_run, m), scale_log2)), s1 = fast_exp2(__fmul_rn(__fsub_rn(m1, m), scale_log2));
          l_run = fmaf(l_run, s0, l1 * s1);
          m_run = m;
          const float inv = (l_run > 0.f) ? 1.0f / l_run : 0.f;   // neither half has seen a key: O = 0
          a0 = s0 * inv;
          a1 = s1 * inv;
        }
      }
      const float inv_l = has1 ? 1.0f : a0;            // with two halves the weights a_0, a_1 already carry 1 / l
      uint8_t *stage = sQ + (split ? qb : t) * C::kTileBytes;   // no MMA reads this Q tile any more
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t o[32];
        tmem_ld32(tO + 32 * c, o);
        if (has1) {
          uint32_t o1[32];
          tmem_ld32(tO + D + 32 * c, o1);              // O_1 sits D columns after O_0, same lanes
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(fmaf(__uint_as_float(o1[i]), a1, __uint_as_float(o[i]) * a0));
        }
        tmem_wait_ld();
        const uint32_t slab = (c >> 1) * C::kSlabBytes;
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          uint32_t pk[4];
#pragma unroll
          for (int w = 0; w < 4; ++w)
            pk[w] = pack_bf16x2(__uint_as_float(o[8 * v + 2 * w]) * inv_l, __uint_as_float(o[8 * v + 2 * w + 1]) * inv_l);
          *reinterpret_cast<uint4 *>(stage + slab + swz128_offset(row, 4 * (c & 1) + v)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
      }
      tc_fence_before();
      mbar_arrive(&bar_o_free[t]);                     // O_t may be overwritten by the next work item
      if (split) mbar_arrive(&bar_o_free[1]);          // warpgroup 0 has read both accumulators
      const int qrow0 = it.seq0 + qt * C::kBlockM;      // first row of the tile inside the head
      if (qt * C::kBlockM + row < it.len) LSE[static_cast<size_t>(bh) * N + qrow0 + row] = (l_run > 0.f) ? fmaf(m_run, alpha, logf(l_run)) : INFINITY;
      fence_proxy_async_smem();
      named_bar_sync(1 + t, 128);
      const TileInfo tinfo{qrow0, it.seq0, it.seq0 + it.len, 0};
      if (tile_store_by_tma(tinfo, N)) {
        if (row == 0) {
          for (int sl = 0; sl < C::kSlabs; ++sl) tma_store_3d(&tmO, stage + sl * C::kSlabBytes, sl * 64, qrow0, bh);
          bulk_commit_group();
          bulk_wait_group_read0();
          mbar_arrive(&bar_q_free[qb]);                // this tile's slot of the Q buffer may be reloaded
        }
      } else {
        // ragged last tile of a packed sequence that another sequence follows: rows past its end are not ours to write
        store_rows_clipped<D>(stage, C::kSlabBytes, Og + (static_cast<size_t>(bh) * N + qrow0) * D, row, it.len - qt * C::kBlockM);
        named_bar_sync(1 + t, 128);
        if (row == 0) mbar_arrive(&bar_q_free[qb]);
      }
#ifdef GPROJ_TRACE
      if (row == 0) tile_event(20 + t, lin, T, ev_n0, ev_n0, ev_n2, global_ns(), ev_c0, clock64());
#endif
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, C::kTmemCols);
}

}  // namespace gproj
