// Fused attention backward with the GProj correction for sm_100a (Algorithm 1).
//
// The work of Algorithm 1 is organised as two stationary kernels so that every accumulator lives
// in TMEM from its first to its last contribution (no atomics, no BF16 round trip, deterministic):
//
//   bwd_dq_kernel   query tile stationary; streams 64-key steps.  Per step: S = Q K^T, dP = dO V^T
//                   (tensor core -> TMEM), then per row (thread <-> TMEM lane): P = exp(S - LSE),
//                   r = BF16(P), t = BF16(P (dP - D)), rho += sum t, m += sum r (sums of the ROUNDED
//                   operands, Eq. "gproj-row-mass"), and two more contractions A += t K, B += r K with
//                   t, r read from TMEM.  Epilogue: lambda = rho / m (0 if m = 0),
//                   dQ = BF16(alpha (A - lambda B)) (Eq. "gproj-query-implemented"), and the scaled-query
//                   operand of the key correction, stored negated: Z = -BF16(lambda q).
//                   Also produces D = rowsum(dO * O) (Algorithm 1 line 1) and keeps it, with LSE in base
//                   two, for the second kernel.
//   bwd_dkv_kernel  key tile stationary; streams 64-query steps.  Per step: S^T = K Q^T, dP^T = V dO^T,
//                   r^T, t^T as above (thread <-> key row; LSE, D are per-column values from shared
//                   memory), dV += r^T dO, dK += t^T Q + r^T Z  -- the correction lands in the FP32
//                   accumulator before the final cast (Eq. "gproj-key-implemented").
//                   Epilogue: dK = BF16(alpha acc), dV = BF16(acc).
//
// Pipeline.  TMEM holds kNB score buffers (S and dP of one 64-wide step each) next to the two FP32
// accumulators: 3 buffers at d = 64, 2 at d = 128 (512 columns either way).  Four compute warpgroups form two
// groups; a group takes every second step and its two warpgroups split the step's 64 columns (thread <-> (row,
// 32-column slice)).  A buffer is back with the tensor core after half the ALU time one warpgroup per step would
// take -- that time bounds the loop  scores -> ALUs -> second-stage products -> buffer free  each buffer runs
// through -- while the two groups, at different phases, hide each other's TMEM and barrier latencies.
// The packed BF16 operands r / t overwrite the consumed S columns of their own 16-column chunk.
// The dK/dV kernel further splits a step's arithmetic in two phases with their own barriers (r^T from S^T first, then
// t^T from dP^T), so that dV += r^T dO and dK += r^T Z run on the tensor core while t^T is still being computed.  The tensor-core queue is only one or two instructions deep, so an issuing warp is stalled
// for as long as its MMAs execute and anything else it does (barrier polls, commits) would idle the pipe.
// Two warps therefore issue: warp 1 the score products of every step, warp 2 the second-stage products; each
// one's bookkeeping overlaps the other's MMAs.  Reuse of a score buffer is ordered by an explicit barrier
// (second-stage MMAs of step n committed -> scores of step n + kNB may be issued).
//
// Persistence.  One CTA per SM walks a static list of tiles: tiles are ordered by decreasing work and dealt
// to the CTAs in boustrophedon rounds, which balances causal work as well as a greedy scheduler would while
// staying deterministic and needing no counter.  Barrier set-up, the TMEM allocation and the launch latency
// are paid once; the step pipeline (stage ring, score buffers) runs on across tile boundaries, the stationary
// tile of the next work item is fetched by its own warp as soon as the last score product of the current one
// has been issued and completed, and the epilogue of one tile overlaps the first steps of the next.
#pragma once
#include "sm100_primitives.cuh"

namespace gproj {

constexpr unsigned kFlagNoQCorrection = 1u;
constexpr unsigned kFlagNoKCorrection = 2u;

// Bytes of one 64-row block of the row-constant tile (64 rows x 16 BF16 columns).
constexpr int kExtBlockBytes = 2048;

template <int D>
struct BwdCfg {
  static constexpr int kSlabs = D / 64;
  static constexpr int kBigSlabBytes = 128 * 128;                 // 128-row slab (stationary tile)
  static constexpr int kBigTileBytes = kSlabs * kBigSlabBytes;
  static constexpr int kStepRows = 64;                            // rows of a streamed tile
  static constexpr int kStepSlabBytes = kStepRows * 128;
  static constexpr int kStepTileBytes = kSlabs * kStepSlabBytes;
  static constexpr int kNB = (D == 64) ? 3 : 2;                   // score buffers (steps in flight)
  // Compute warpgroups: kGroups groups of kSlices warpgroups.  Group a takes the steps g = a (mod kGroups); inside it
  // warpgroup h takes columns [kSliceCols h, kSliceCols (h + 1)) of the step.  Two groups keep two steps in the ALUs at
  // different phases (one group's TMEM / barrier latencies hide behind the other's arithmetic); two slices halve the
  // time a score buffer stays away from the tensor core.
  static constexpr int kGroups = 2, kSlices = 2;
  static constexpr int kWG = kGroups * kSlices;
  static constexpr int kSliceCols = kStepRows / kSlices;
  static constexpr int kCompute = 128 * kWG;                      // compute threads
  static constexpr int kThreads = 128 + kCompute;                 // stage producer, 2 MMA warps, tile loader; compute warpgroups
  // Output staging for the TMA stores: its own buffer where shared memory allows (d = 64), else over the stationary tile.
  static constexpr bool kSepStaging = (D == 64);
  // TMEM columns: buffer b holds S at 128 b and dP at 128 b + 64; accumulators follow
  static constexpr int kTmemCols = 512;
  static constexpr uint32_t kColAcc0 = 128 * kNB, kColAcc1 = 128 * kNB + D;
  static_assert(kColAcc1 + D <= 512, "TMEM budget");
  // dQ-side kernel: Q, dO resident; ring of (K, V) step tiles
  static constexpr int kDqStages = (D == 64) ? 6 : 4;
  static constexpr int kDqStageBytes = 2 * kStepTileBytes;
  static constexpr int kDqResBufs = (D == 64) ? 2 : 1;             // stationary (Q, dO) buffers
  // d = 64 (two stationary buffers): D = rowsum(dO o O), LSE and the row-constant tile of a tile are prepared by the
  // stationary-tile loader's warp as soon as the tile's dO has landed, i.e. while the tile before it still runs; the
  // compute warps only pick the two values up.  At d = 128 there is one stationary buffer and the compute warps do it at
  // the tile's start.
  static constexpr bool kLoaderStats = (D == 64);
  static constexpr int kDqSmemBytes = kDqResBufs * 2 * kBigTileBytes + kDqStages * kDqStageBytes + (kSepStaging ? 2 * kBigTileBytes : 0) +
                                      1024;
  // dK/dV-side kernel: K, V resident; ring of (Q, dO, Z, stats) step tiles
  static constexpr int kDkvStages = (D == 64) ? 5 : 3;
  static constexpr int kDkvStageBytes = 3 * kStepTileBytes + kExtBlockBytes;   // + the step's 64-row block of the row-constant tile
  static constexpr int kDkvSmemBytes = 2 * kBigTileBytes + kDkvStages * kDkvStageBytes + (kSepStaging ? 2 * kBigTileBytes : 0) + 1024;
  static_assert(kDqStages >= kNB + 1 && kDkvStages >= kNB + 1, "a stage stays busy until its second-stage MMAs finish");
};

// Static persistent schedule: work items are numbered by decreasing work; round r hands item r G + c to CTA c
// on even rounds and item r G + (G - 1 - c) on odd rounds (G = number of CTAs).
struct TileSched {
  int total, G, c, round;
  __device__ __forceinline__ explicit TileSched(int total_tiles)
      : total(total_tiles), G(static_cast<int>(gridDim.x)), c(static_cast<int>(blockIdx.x)), round(0) {}
  __device__ __forceinline__ int next() {
    const int idx = round * G + ((round & 1) ? (G - 1 - c) : c);
    ++round;
    return idx < total ? idx : -1;
  }
  __device__ __forceinline__ int peek() const {     // the item next() would return, without taking it
    const int idx = round * G + ((round & 1) ? (G - 1 - c) : c);
    return idx < total ? idx : -1;
  }
};

// Item number -> (rank of the tile in decreasing work, head).  Items are dealt in groups of `group` consecutive ranks of
// all heads; inside a group the ranks of one head are adjacent, so that CTAs running at the same time work on the same
// head and share the rows they stream (the other operand) in L2 instead of fetching one head each out of HBM.
// group = 1: every head's longest tile first (the exact longest-first order; packed calls, whose plan is already
// sorted); group = tiles per head: head-major (dense non-causal calls, whose tiles are all alike); in between for
// causal calls with many heads, where a few adjacent ranks differ little in work.
// Division of a non-negative 31-bit number by a divisor fixed at launch: quotient = umulhi(x, mul) >> shr (x itself if
// the divisor is 1), with L = ceil(log2 divisor), mul = ceil(2^(31 + L) / divisor) < 2^32 and shr = L - 1, set by the
// host.  Three instructions instead of the forty-odd of a division by a run-time value, which sat on every role's path
// at each tile.
struct FastDiv {
  unsigned div, mul, shr;
#ifdef __CUDACC__
  __device__ __forceinline__ int quot(int x) const {
    return div == 1u ? x : static_cast<int>(__umulhi(static_cast<unsigned>(x), mul) >> shr);
  }
#endif
};
struct ItemOrder {
  int gk, n_full;                   // ranks per group, full groups
  FastDiv per_group, by_gk, by_rem; // items per group (heads x gk); ranks per group; ranks of the short last group
#ifdef __CUDACC__
  __device__ __forceinline__ void decode(int lin, int &rank, int &head) const {
    const int g = per_group.quot(lin), within = lin - g * static_cast<int>(per_group.div);
    const bool full = g < n_full;
    head = full ? by_gk.quot(within) : by_rem.quot(within);
    rank = g * gk + within - head * static_cast<int>(full ? by_gk.div : by_rem.div);
  }
  __device__ __forceinline__ int rank(int lin) const { int r, h; decode(lin, r, h); return r; }
  __device__ __forceinline__ int head(int lin) const { int r, h; decode(lin, r, h); return h; }
#endif
};

// One 128-row tile of one sequence.  Rows are counted inside a head ([heads][rows][d] tensors): dense calls have one
// sequence [0, N) per head; packed (variable-length) calls have several, listed tile by tile in a plan the host
// prepared, two int4 per tile: {row0, seq0, seq_end, blk0} with blk0 the first 64-row block of row statistics of the
// sequence's QUERIES, and {oseq0, oseq_end, -, -}.
// [oseq0, oseq_end) is the range of the OTHER operand's rows the tile works against (keys for a query tile, queries for a
// key tile); it differs from [seq0, seq_end) when query and key lengths are unequal.
struct TileInfo { int row0, seq0, seq_end, blk0, oseq0, oseq_end; };
__device__ __forceinline__ TileInfo tile_info(const int4 *plan, int idx, int dense_tile, int N, int N_other) {
  if (plan != nullptr) {
    const int4 e = __ldg(plan + 2 * idx), o = __ldg(plan + 2 * idx + 1);
    return TileInfo{e.x, e.y, e.z, e.w, o.x, o.y};
  }
  return TileInfo{128 * dense_tile, 0, N, 0, 0, N_other};
}
// Rows [row0, row0 + 128) may be written by a TMA store (which clips at the tensor's end N) unless the tile is the
// ragged tail of a sequence that is followed by another one.
__device__ __forceinline__ bool tile_store_by_tma(const TileInfo &t, int N) { return t.row0 + 128 <= t.seq_end || t.seq_end == N; }
// Plain row-wise copy of a staged [128 x D] BF16 tile (128-byte swizzled slabs) to global memory, rows < rows_valid only.
template <int D>
__device__ __forceinline__ void store_rows_clipped(const uint8_t *stage, int slab_bytes, __nv_bfloat16 *dst_row0, int row, int rows_valid) {
  if (row < rows_valid) {
    uint4 *dst = reinterpret_cast<uint4 *>(dst_row0 + static_cast<size_t>(row) * D);
#pragma unroll
    for (int ch = 0; ch < D / 8; ++ch)
      dst[ch] = *reinterpret_cast<const uint4 *>(stage + (ch >> 3) * slab_bytes + swz128_offset(row, ch & 7));
  }
}

enum BwdWaitCode {
  kDqWaitQ = 0x21, kDqWaitKV = 0x22, kDqWaitKVEmpty = 0x23, kDqWaitSdP = 0x24, kDqWaitTR = 0x25, kDqWaitAcc = 0x26, kDqWaitBuf = 0x27, kDqWaitResFree = 0x28, kDqWaitAccFree = 0x29,
  kDkvWaitKV = 0x31, kDkvWaitQ = 0x32, kDkvWaitQEmpty = 0x33, kDkvWaitSdP = 0x34, kDkvWaitTR = 0x35, kDkvWaitAcc = 0x36, kDkvWaitBuf = 0x37, kDkvWaitResFree = 0x38, kDkvWaitAccFree = 0x39
};

// Arithmetic of one pair of adjacent score columns, shared by both kernels (Algorithm 1 lines 5-8):
//   p = exp2(x * (alpha log2 e) - LSE log2 e),  r = BF16(p),  t = BF16(fl32[p * fl32(dP - D)]).
// x2 / dp2 are the raw TMEM words of the two columns; nl2 = {-LSE log2 e} and nd2 = {-D} per column.
// keep0 / keep1 zero a probability beyond the causal diagonal.
template <bool MASKED>
__device__ __forceinline__ void score_pair(uint32_t x0, uint32_t x1, uint32_t dp0, uint32_t dp1, uint64_t scale2, uint64_t nl2,
                                           uint64_t nd2, bool keep0, bool keep1, uint32_t &r_packed, uint32_t &t_packed) {
  float a0, a1;
  f32x2_split(fma2(f32x2_bits(x0, x1), scale2, nl2), a0, a1);
  float p0 = fast_exp2(a0), p1 = fast_exp2(a1);
  if (MASKED) {
    if (!keep0) p0 = 0.f;
    if (!keep1) p1 = 0.f;
  }
  float t0, t1;
  f32x2_split(mul2(f32x2(p0, p1), add2(f32x2_bits(dp0, dp1), nd2)), t0, t1);
  r_packed = pack_bf16x2(p0, p1);
  t_packed = pack_bf16x2(t0, t1);
}

// One step of the dQ side for one query row and one slice (kSliceCols = 32 keys) of the step's 64 keys, in two 16-column
// chunks: the second chunk's TMEM load is in flight while the first is in the ALUs.  tS / tdP address the slice's S and
// dP columns; `lim` = (row index) - (key index of the slice's column 0): with MASKED, column c is beyond the causal
// diagonal (or past the last key) when c > lim.  The packed BF16 operands overwrite the chunk's OWN score columns (r over
// its first eight, t over its last eight: one K = 16 MMA slice each), so nobody writes over scores yet to be read.
template <bool MASKED>
__device__ __forceinline__ void dq_slice(uint32_t tS, uint32_t tdP, float scale_log2, float neg_lse2, float Dv, int lim,
                                         uint64_t &rho2, uint64_t &msum2) {
  const uint64_t scale2 = f32x2(scale_log2, scale_log2), nl2 = f32x2(neg_lse2, neg_lse2), nd2 = f32x2(-Dv, -Dv);
  uint32_t xs[2][16], xp[2][16];
  tmem_ld16(tS, xs[0]);
  tmem_ld16(tdP, xp[0]);
#pragma unroll
  for (int c = 0; c < 2; ++c) {
    tmem_wait_ld();
    if (c == 0) {
      tmem_ld16(tS + 16, xs[1]);
      tmem_ld16(tdP + 16, xp[1]);
    }
    uint32_t pr[8], pt[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int col = 16 * c + 2 * i;
      score_pair<MASKED>(xs[c][2 * i], xs[c][2 * i + 1], xp[c][2 * i], xp[c][2 * i + 1], scale2, nl2, nd2, col <= lim, col + 1 <= lim,
                         pr[i], pt[i]);
      // row masses of the operands AS ROUNDED (Eq. "gproj-row-mass"): re-expand the BF16 pairs and add in FP32
      msum2 = add2(msum2, f32x2_bits(pr[i] << 16, pr[i] & 0xffff0000u));
      rho2 = add2(rho2, f32x2_bits(pt[i] << 16, pt[i] & 0xffff0000u));
    }
    tmem_st8(tS + 16 * c, pr);
    tmem_st8(tS + 16 * c + 8, pt);
  }
}

// The dK/dV side does the arithmetic of a step in two phases, so that the tensor core can start on the products that need
// only r^T while the ALUs are still busy with t^T (measured: -15 % on that kernel at d = 128; the dQ side did not gain):
//   phase 1 (needs S^T):   p = exp2(x * (alpha log2 e) - LSE log2 e), r = BF16(p); p is kept in FP32 registers
//   phase 2 (needs dP^T):  t = BF16(fl32[p * fl32(dP - D)])
// Each thread owns one key row and one slice (32 query columns) of the step, handled in two 16-column chunks whose TMEM
// loads are software-pipelined; the packed operands overwrite the chunk's own consumed S columns (r the first eight, t
// the last eight).

// Phase 1 of the dK/dV side (thread <-> key row, columns = queries).  `lim` = (key row) - (query index of the slice's
// column 0): with MASKED, column c is a query before this key when c < lim; `hi` = (last query of the sequence) - (query
// index of column 0): a column c > hi belongs to the next packed sequence (or is zero fill).  The scores arrive as
// x - LSE / alpha: the score product carries one extra K = 16 slice (a constant matrix of ones times the step's
// row-constant tile), so no per-column constant has to be read here (every lane would need every column's value:
// broadcast reads from shared memory cost the 64-query kernel at d = 64 14 % when it still had them).
template <bool MASKED>
__device__ __forceinline__ void dkv_phase1(uint32_t tS, float scale_log2, int lim, int hi, float (&p)[32]) {
  const uint64_t scale2 = f32x2(scale_log2, scale_log2);
  uint32_t xs[2][16];
  tmem_ld16(tS, xs[0]);
#pragma unroll
  for (int c = 0; c < 2; ++c) {
    tmem_wait_ld();
    if (c == 0) tmem_ld16(tS + 16, xs[1]);
    uint32_t pr[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int col = 16 * c + 4 * i;
      float a[4];
      f32x2_split(mul2(f32x2_bits(xs[c][4 * i], xs[c][4 * i + 1]), scale2), a[0], a[1]);
      f32x2_split(mul2(f32x2_bits(xs[c][4 * i + 2], xs[c][4 * i + 3]), scale2), a[2], a[3]);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float pe = fast_exp2(a[e]);
        if (MASKED && (col + e < lim || col + e > hi)) pe = 0.f;
        p[col + e] = pe;
      }
      pr[2 * i] = pack_bf16x2(p[col], p[col + 1]);
      pr[2 * i + 1] = pack_bf16x2(p[col + 2], p[col + 3]);
    }
    tmem_st8(tS + 16 * c, pr);
  }
}

// Phase 2 of the dK/dV side.  The products arrive as dP - D (same extra slice as for the scores).
__device__ __forceinline__ void dkv_phase2(uint32_t tS, uint32_t tdP, const float (&p)[32]) {
  uint32_t xp[2][16];
  tmem_ld16(tdP, xp[0]);
#pragma unroll
  for (int c = 0; c < 2; ++c) {
    tmem_wait_ld();
    if (c == 0) tmem_ld16(tdP + 16, xp[1]);
    uint32_t pt[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int col = 16 * c + 4 * i;
      float t0, t1, t2, t3;
      f32x2_split(mul2(f32x2(p[col], p[col + 1]), f32x2_bits(xp[c][4 * i], xp[c][4 * i + 1])), t0, t1);
      f32x2_split(mul2(f32x2(p[col + 2], p[col + 3]), f32x2_bits(xp[c][4 * i + 2], xp[c][4 * i + 3])), t2, t3);
      pt[2 * i] = pack_bf16x2(t0, t1);
      pt[2 * i + 1] = pack_bf16x2(t2, t3);
    }
    tmem_st8(tS + 16 * c + 8, pt);
  }
}

// Row constants of one query row for the dK/dV side, which takes them through its score products instead of reading
// them per column.  Per 64-row block a K-major operand tile of 16 BF16 columns without swizzle (eight-row groups of 256
// bytes: the rows' first eight columns, then their last eight): columns 0..2 hold -LSE / alpha and columns 8..10 hold -D,
// each as three BF16 pieces whose sum is the FP32 value, the other columns zero.  A row with an empty support
// (LSE = +inf) gets a large finite value: its probabilities are zero either way, and an infinity would turn the zero
// entries of the constant operand into NaN.
__device__ __forceinline__ void write_row_constants(float *stats, size_t block, int row_in_block, float neg_lse2, float Dv, float scale_log2) {
  const float c = fmaxf(__fdiv_rn(neg_lse2, scale_log2), -1.0e30f), nd = -Dv;
  const uint32_t c0 = pack_bf16x2(c, 0.f), n0 = pack_bf16x2(nd, 0.f);
  const float c_r1 = c - bf16_lo_to_f32(c0), n_r1 = nd - bf16_lo_to_f32(n0);
  const uint32_t c1 = pack_bf16x2(c_r1, 0.f), n1 = pack_bf16x2(n_r1, 0.f);
  const uint32_t c2 = pack_bf16x2(c_r1 - bf16_lo_to_f32(c1), 0.f), n2 = pack_bf16x2(n_r1 - bf16_lo_to_f32(n1), 0.f);
  uint8_t *blk = reinterpret_cast<uint8_t *>(stats) + block * kExtBlockBytes + (row_in_block >> 3) * 256 + (row_in_block & 7) * 16;
  *reinterpret_cast<uint4 *>(blk) = make_uint4(c0 | (c1 << 16), c2, 0u, 0u);
  *reinterpret_cast<uint4 *>(blk + 128) = make_uint4(n0 | (n1 << 16), n2, 0u, 0u);
}

// ============================================================================================
// dQ side
// ============================================================================================
template <int D, bool CAUSAL>
__global__ void __launch_bounds__(BwdCfg<D>::kThreads, 1)
bwd_dq_kernel(const __grid_constant__ CUtensorMap tmQ,    // box 64 x 128 rows
              const __grid_constant__ CUtensorMap tmdO,   // box 64 x 128 rows
              const __grid_constant__ CUtensorMap tmK,    // box 64 x 64 rows
              const __grid_constant__ CUtensorMap tmV,    // box 64 x 64 rows
              const __grid_constant__ CUtensorMap tmdQ,   // store, box 64 x 128 rows
              const __grid_constant__ CUtensorMap tmZ,    // store, box 64 x 128 rows
              const __nv_bfloat16 *__restrict__ Og, const __nv_bfloat16 *__restrict__ dOg,
              const float *__restrict__ LSE, float *__restrict__ stats,
              __nv_bfloat16 *__restrict__ dQg, __nv_bfloat16 *__restrict__ Zg,   // plain-store targets of clipped tiles
              const int4 *__restrict__ plan, int nblk,                          // packed sequences: tile list; 64-row statistic blocks per head
              int N, int Nk, int BH, int Hq, int G, int total_tiles, const ItemOrder order, float scale_log2, float alpha, unsigned flags, int *status) {
  // N: query rows per head (own operand), Nk: key rows per head.  Causal support of query i: keys j <= i + (L_k - L_q).
  using C = BwdCfg<D>;
  constexpr int NB = C::kNB, R = C::kDqResBufs, S = C::kDqStages;
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t *sRes = smem;                                        // buffer rb: Q tile, then dO tile
  uint8_t *sKV = sRes + R * 2 * C::kBigTileBytes;              // stage s: K step tile, then V step tile
  uint8_t *sOut = sKV + S * C::kDqStageBytes;                  // staging (dQ tile, then Z tile) when separate

  __shared__ uint64_t bar_res_full[R], bar_res_free[R], bar_kv_full[S], bar_kv_empty[S];
  __shared__ uint64_t bar_sdp_full[NB], bar_tr_ready[NB], bar_acc_done, bar_acc_free, bar_drain[2], bar_stats_ready[R];
  __shared__ uint32_t tmem_base_smem;
  __shared__ int cta_abort, cta_skip;
  __shared__ float s_rho[C::kWG - 1][128], s_m[C::kWG - 1][128], s_lam[128], s_D[R][128], s_lse[R][128];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) cta_skip = *reinterpret_cast<volatile int *>(status);
  __syncthreads();
  if (cta_skip != 0) return;   // an earlier wait gave up: drain the rest of the grid quickly

  // Ragged N: tiles and steps round up; rows past N load as zero (TMA fill) and are clipped on store.
  const int n_qt = (N + 127) / 128;
  AbortState ab{status, &cta_abort};
  if (threadIdx.x == 0) {
    cta_abort = 0;
    for (int r = 0; r < R; ++r) { mbar_init(&bar_res_full[r], 1); mbar_init(&bar_res_free[r], 2); mbar_init(&bar_stats_ready[r], 32); }
    for (int s = 0; s < S; ++s) { mbar_init(&bar_kv_full[s], 1); mbar_init(&bar_kv_empty[s], 1); }
    for (int b = 0; b < NB; ++b) { mbar_init(&bar_sdp_full[b], 1); mbar_init(&bar_tr_ready[b], 128 * C::kSlices); }
    mbar_init(&bar_acc_done, 1);
    mbar_init(&bar_acc_free, C::kCompute);
    mbar_init(&bar_drain[0], 1);
    mbar_init(&bar_drain[1], 1);
    fence_mbar_init();
  }
  if (warp == 1) { tmem_alloc(&tmem_base_smem, C::kTmemCols); tmem_relinquish(); }
  if (warp == 0 && lane == 0) {
    tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmdO); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
    tma_prefetch_desc(&tmdQ); tma_prefetch_desc(&tmZ);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = __shfl_sync(0xffffffffu, tmem_base_smem, 0);   // the shuffle marks it warp-uniform

  // The dK/dV-side kernel that follows in the stream may be scheduled on SMs this kernel has left: its set-up and its
  // stationary-tile loads need nothing from here, and it waits (griddep_wait) before it reads the statistics and Z.
  griddep_launch_dependents();

  TileSched sched(total_tiles);
  // tile decode: causal -> longest rows first
  auto tix = [&](int lin) { return order.rank(lin); };
  auto hix = [&](int lin) { return order.head(lin); };
  auto tile_of = [&](int lin) { return tile_info(plan, tix(lin), CAUSAL ? (n_qt - 1 - tix(lin)) : tix(lin), N, Nk); };
  // 64-key steps of a query tile: the keys its last row sees (causal) or all of them; at least one step, fully masked
  // if the tile sees no key at all, so that every tile runs through the same pipeline.
  auto steps_of = [&](const TileInfo &t) {
    const int Lk = t.oseq_end - t.oseq0, off = Lk - (t.seq_end - t.seq0);
    const int kend = CAUSAL ? min(Lk, t.row0 - t.seq0 + 128 + off) : Lk;
    return max(1, (max(kend, 0) + C::kStepRows - 1) / C::kStepRows);
  };

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer of the streamed (K, V) step tiles
    if (lane == 0) {
      int g = 0;
      for (int lin = sched.next(); lin >= 0; lin = sched.next()) {
        const TileInfo tl = tile_of(lin);
        const int bh = hix(lin), T = steps_of(tl);
        for (int n = 0; n < T; ++n, ++g) {
          const int st = g % S;
          if (g >= S) mbar_wait(&bar_kv_empty[st], ((g / S) - 1) & 1, ab, kDqWaitKVEmpty);
          mbar_expect_tx(&bar_kv_full[st], C::kDqStageBytes);
          uint8_t *dst = sKV + st * C::kDqStageBytes;
          const int kvh = kv_head_of(bh, Hq, G), krow = tl.oseq0 + n * C::kStepRows;   // grouped-query: the group's shared K / V head
          for (int s = 0; s < C::kSlabs; ++s) {
            tma_load_3d(dst + s * C::kStepSlabBytes, &tmK, &bar_kv_full[st], s * 64, krow, kvh);
            tma_load_3d(dst + C::kStepTileBytes + s * C::kStepSlabBytes, &tmV, &bar_kv_full[st], s * 64, krow, kvh);
          }
        }
      }
      // Every load is consumed by an MMA the epilogue waits for, so nothing is in flight at exit unless the
      // CTA aborted; then give the copies a bounded chance to land before shared memory is released.
      if (cta_abort) {
        for (int q = (g > S ? g - S : 0); q < g; ++q)
          for (int spin = 0; spin < 100000 && !mbar_try_wait(&bar_kv_full[q % S], (q / S) & 1); ++spin) {}
      }
    }
  } else if (warp == 3) {
    // ---------------------------------------------------------------- TMA loader of the stationary (Q, dO) tiles; with
    // kLoaderStats the whole warp then prepares the tile's row constants (see below)
    int ti = 0;
    for (int lin = sched.next(); lin >= 0; lin = sched.next(), ++ti) {
      const int rb = ti % R, bh = hix(lin);
      const TileInfo tl = tile_of(lin);
      if (lane == 0) {
        if (ti >= R) mbar_wait(&bar_res_free[rb], ((ti / R) - 1) & 1, ab, kDqWaitResFree);
        mbar_expect_tx(&bar_res_full[rb], 2 * C::kBigTileBytes);
        uint8_t *dst = sRes + rb * 2 * C::kBigTileBytes;
        for (int s = 0; s < C::kSlabs; ++s) {
          tma_load_3d(dst + s * C::kBigSlabBytes, &tmQ, &bar_res_full[rb], s * 64, tl.row0, bh);
          tma_load_3d(dst + C::kBigTileBytes + s * C::kBigSlabBytes, &tmdO, &bar_res_full[rb], s * 64, tl.row0, bh);
        }
      }
      __syncwarp();
      if (C::kLoaderStats && ti > 0) {       // the first tile's are computed by the (then idle) compute warps: sixteen warps are faster
        // D_i = sum_c dO_ic O_ic from the saved BF16 output, FP32 (Algorithm 1 line 1), LSE, and the row-constant tile
        // for the dK/dV side, for the four rows lane, lane + 32, ... of the tile: dO from the stationary tile in shared
        // memory, O from global memory.  The sum keeps the order of the d = 128 path (eight elements by sequential FMAs,
        // the eight partial sums by a butterfly).  The buffer pair rb is free: lane 0 has seen its release above.
        mbar_wait(&bar_res_full[rb], (ti / R) & 1, ab, kDqWaitQ);
        const size_t head_row0 = static_cast<size_t>(bh) * N;
        const uint8_t *sdO = sRes + rb * 2 * C::kBigTileBytes + C::kBigTileBytes;
#pragma unroll
        for (int it = 0; it < 4; ++it) {
          const int r = lane + 32 * it, qrow = tl.row0 + r;
          float part[D / 8];
#pragma unroll
          for (int c = 0; c < D / 8; ++c) {
            uint4 a = make_uint4(0u, 0u, 0u, 0u), b = a;
            if (qrow < tl.seq_end) {
              a = __ldg(reinterpret_cast<const uint4 *>(Og + (head_row0 + qrow) * D) + c);
              b = *reinterpret_cast<const uint4 *>(sdO + (c >> 3) * C::kBigSlabBytes + swz128_offset(r, c & 7));
            }
            const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
            float acc = 0.f;
#pragma unroll
            for (int w = 0; w < 4; ++w) {
              acc = fmaf(bf16_lo_to_f32(aw[w]), bf16_lo_to_f32(bw[w]), acc);
              acc = fmaf(bf16_hi_to_f32(aw[w]), bf16_hi_to_f32(bw[w]), acc);
            }
            part[c] = acc;
          }
#pragma unroll
          for (int off = D / 16; off >= 1; off >>= 1)
#pragma unroll
            for (int c = 0; c < off; ++c) part[c] += part[c + off];
          const float Dv = part[0];
          const float lse_row = (qrow < tl.seq_end) ? LSE[head_row0 + qrow] : 0.f;
          s_D[rb][r] = Dv;
          s_lse[rb][r] = lse_row;
          const int rel = qrow - tl.seq0;                  // row inside the sequence
          if (rel < ((tl.seq_end - tl.seq0 + 63) / 64) * 64)
            write_row_constants(stats, (static_cast<size_t>(bh) * nblk + tl.blk0 + (rel >> 6)), rel & 63, -lse_row * 1.4426950408889634f, Dv, scale_log2);
        }
        mbar_arrive(&bar_stats_ready[rb]);
      }
    }
    if (lane == 0 && cta_abort) {
      for (int q = (ti > R ? ti - R : 0); q < ti; ++q)
        for (int spin = 0; spin < 100000 && !mbar_try_wait(&bar_res_full[q % R], (q / R) & 1); ++spin) {}
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- tensor-core issuer 1: scores
    // The whole warp runs this loop so that every address stays provably warp-uniform (descriptor operands
    // then live in uniform registers); one elected lane issues the MMAs and commits.
    constexpr uint32_t idesc_s = idesc_bf16_f32(128, 64, 0, 0);    // [128 queries] x [64 keys], contraction over d
    const SmemDesc dscRes0 = make_smem_desc(smem_u32(sRes), 16, 1024);
    const SmemDesc dscK0 = make_smem_desc(smem_u32(sKV), 16, 1024);                          // K-major view of stage 0
    int g = 0, ti = 0;
    for (int lin = sched.next(); lin >= 0; lin = sched.next(), ++ti) {
      const int T = steps_of(tile_of(lin)), rb = ti % R;
      mbar_wait(&bar_res_full[rb], (ti / R) & 1, ab, kDqWaitQ);
      const SmemDesc dscQ = dscRes0.advanced(rb * 2 * C::kBigTileBytes), dscdO = dscQ.advanced(C::kBigTileBytes);
      for (int n = 0; n < T; ++n, ++g) {
        const int st = g % S, b = g % NB;
        mbar_wait(&bar_kv_full[st], (g / S) & 1, ab, kDqWaitKV);
        // r, t of step g - NB consumed: that step's second-stage products are complete.  One commit per step serves this
        // wait and the stage ring's (every commit costs the tensor pipe some forty cycles in this stream of short products).
        if (g >= NB) mbar_wait(&bar_kv_empty[(g - NB) % S], ((g - NB) / S) & 1, ab, kDqWaitBuf);
        tc_fence_after();
        const SmemDesc dscK = dscK0.advanced(st * C::kDqStageBytes), dscV = dscK.advanced(C::kStepTileBytes);
        const uint32_t tS = tmem_base + 128 * b, tdP = tS + 64;
        if (elect_one_sync()) {
#pragma unroll
          for (int k = 0; k < D / 16; ++k) {
            const uint32_t oa = (k / 4) * C::kBigSlabBytes + (k % 4) * 32, ob = (k / 4) * C::kStepSlabBytes + (k % 4) * 32;
            umma_ss(tS, dscQ.at(oa), dscK.at(ob), idesc_s, k > 0);
          }
#pragma unroll
          for (int k = 0; k < D / 16; ++k) {
            const uint32_t oa = (k / 4) * C::kBigSlabBytes + (k % 4) * 32, ob = (k / 4) * C::kStepSlabBytes + (k % 4) * 32;
            umma_ss(tdP, dscdO.at(oa), dscV.at(ob), idesc_s, k > 0);
          }
          umma_commit(&bar_sdp_full[b]);
          if (n == T - 1) umma_commit(&bar_res_free[rb]);   // no MMA reads this Q / dO buffer any more
        }
        __syncwarp();
      }
    }
    drain_mmas_if_aborted(&bar_drain[0], ab);
  } else if (warp == 2) {
    // ---------------------------------------------------------------- tensor-core issuer 2: A += t K, B += r K
    constexpr uint32_t idesc_a = idesc_bf16_f32(128, D, 0, 1);     // [128 queries] x [d], contraction over 64 keys
    const SmemDesc dscK0mn = make_smem_desc(smem_u32(sKV), C::kStepSlabBytes, 1024);       // MN-major view of stage 0
    int g = 0, ti = 0;
    for (int lin = sched.next(); lin >= 0; lin = sched.next(), ++ti) {
      const int T = steps_of(tile_of(lin));
      if (ti > 0) mbar_wait(&bar_acc_free, (ti - 1) & 1, ab, kDqWaitAccFree);   // the previous epilogue has read A, B
      for (int p = 0; p < T; ++p, ++g) {
        const int st = g % S, b = g % NB;
        mbar_wait(&bar_tr_ready[b], (g / NB) & 1, ab, kDqWaitTR);
        tc_fence_after();
        const SmemDesc dscK = dscK0mn.advanced(st * C::kDqStageBytes);
        // packed BF16 operands of key slice k (16 keys): r over columns 16 k .. 16 k + 7 of the buffer, t over the next eight
        const uint32_t tR = tmem_base + 128 * b, tT = tR + 8;
        const uint32_t acc = (p > 0) ? 1u : 0u;
        if (elect_one_sync()) {
#pragma unroll
          for (int k = 0; k < C::kStepRows / 16; ++k)
            umma_ts(tmem_base + C::kColAcc0, tT + 16 * k, dscK.at(k * 2048), idesc_a, k > 0 ? 1u : acc);
#pragma unroll
          for (int k = 0; k < C::kStepRows / 16; ++k)
            umma_ts(tmem_base + C::kColAcc1, tR + 16 * k, dscK.at(k * 2048), idesc_a, k > 0 ? 1u : acc);
          umma_commit(&bar_kv_empty[st]);                   // step done: its stage and its score buffer are free
          if (p == T - 1) umma_commit(&bar_acc_done);
        }
        __syncwarp();
      }
    }
    drain_mmas_if_aborted(&bar_drain[1], ab);
  } else {
    // ---------------------------------------------------------------- compute: thread <-> (query row, key slice of every kGroups-th step)
    const int wg = (warp - 4) >> 2, grp = wg / C::kSlices, slice = wg % C::kSlices;
    const int row = 32 * (warp & 3) + lane;
    const uint32_t lane_addr = static_cast<uint32_t>(32 * (warp & 3)) << 16;
    const uint32_t slice_addr = tmem_base + lane_addr + C::kSliceCols * slice;
    int g0 = 0, ti = 0;
    constexpr int L = D / 8, RPI = 32 / L;               // D computation: lanes per row, rows per warp-wide load
    const int sub = lane / L, part = lane % L;
    for (int lin = sched.next(); lin >= 0; lin = sched.next(), ++ti) {
      const TileInfo tl = tile_of(lin);
      const int bh = hix(lin), T = steps_of(tl), rb = ti % R;
      const size_t head_row0 = static_cast<size_t>(bh) * N;
      const int qrow = tl.row0 + row;                  // this thread's query row within the head (past seq_end in a ragged tile)
#ifdef GPROJ_TRACE
      const unsigned long long ev_n0 = global_ns(); const long long ev_c0 = clock64(); unsigned long long ev_n1 = 0, ev_n2 = 0;
#endif

      float Dv, lse_row;
      if (C::kLoaderStats && ti > 0) {
        // prepared by the loader's warp while the previous tile ran
        mbar_wait(&bar_res_full[rb], (ti / R) & 1, ab, kDqWaitQ);       // the tile's Q is read in the epilogue
        mbar_wait(&bar_stats_ready[rb], ((ti - 1) / R) & 1, ab, kDqWaitQ);
        Dv = s_D[rb][row];
        lse_row = s_lse[rb][row];
      } else {
        if (C::kLoaderStats) mbar_wait(&bar_res_full[rb], (ti / R) & 1, ab, kDqWaitQ);
        // D_i = sum_c dO_ic O_ic from the saved BF16 output, FP32 (Algorithm 1 line 1): each of the 16 compute warps
        // takes eight rows, 16-byte loads (D/8 lanes share a row) and a shuffle reduction.
#pragma unroll
        for (int it = 0; it < 8 / RPI; ++it) {
          const int r = 8 * (warp - 4) + it * RPI + sub;
          uint4 a = make_uint4(0u, 0u, 0u, 0u), b = a;
          if (tl.row0 + r < tl.seq_end) {
            a = __ldg(reinterpret_cast<const uint4 *>(Og + (head_row0 + tl.row0 + r) * D) + part);
            b = __ldg(reinterpret_cast<const uint4 *>(dOg + (head_row0 + tl.row0 + r) * D) + part);
          }
          const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
          float acc = 0.f;
#pragma unroll
          for (int w = 0; w < 4; ++w) {
            acc = fmaf(bf16_lo_to_f32(aw[w]), bf16_lo_to_f32(bw[w]), acc);
            acc = fmaf(bf16_hi_to_f32(aw[w]), bf16_hi_to_f32(bw[w]), acc);
          }
#pragma unroll
          for (int off = L / 2; off >= 1; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
          if (part == 0) s_D[rb][r] = acc;
        }
        named_bar_sync(2, C::kCompute);
        Dv = s_D[rb][row];
        lse_row = (qrow < tl.seq_end) ? LSE[head_row0 + qrow] : 0.f;
        // Row constants for the dK/dV side, per 64-row block of a sequence (the last one padded with zeros).
        const int rel = qrow - tl.seq0;                  // row inside the sequence
        if (wg == 0 && rel < ((tl.seq_end - tl.seq0 + 63) / 64) * 64)
          write_row_constants(stats, static_cast<size_t>(bh) * nblk + tl.blk0 + (rel >> 6), rel & 63, -lse_row * 1.4426950408889634f, Dv, scale_log2);
      }
      const float neg_lse2 = -lse_row * 1.4426950408889634f;

      uint64_t rho2 = f32x2(0.f, 0.f), msum2 = f32x2(0.f, 0.f);
#ifdef GPROJ_TRACE
      ev_n1 = global_ns();
#endif
      for (int n = (grp - g0 % C::kGroups + C::kGroups) % C::kGroups; n < T; n += C::kGroups) {
        const int g = g0 + n, b = g % NB;
        mbar_wait(&bar_sdp_full[b], (g / NB) & 1, ab, kDqWaitSdP);
        tc_fence_after();
        const uint32_t tS16 = slice_addr + 128 * b, tdP16 = tS16 + 64;
        // Probabilities are zeroed beyond the causal diagonal and, in the ragged last step, for the zero-filled keys
        // past N (which would otherwise enter the row masses).  Rows of a causal tile never reach such keys.
        const int Lk = tl.oseq_end - tl.oseq0, off = Lk - (tl.seq_end - tl.seq0);
        const int krel0 = n * C::kStepRows + C::kSliceCols * slice;          // key (inside its sequence) of the slice's column 0
        const bool masked = (CAUSAL && (n + 1) * C::kStepRows - 1 > tl.row0 - tl.seq0 + off) || (n + 1) * C::kStepRows > Lk;
        if (masked) {
          const int lim_c = CAUSAL ? qrow - tl.seq0 + off - krel0 : (1 << 30);
          dq_slice<true>(tS16, tdP16, scale_log2, neg_lse2, Dv, min(lim_c, Lk - 1 - krel0), rho2, msum2);
        } else {
          dq_slice<false>(tS16, tdP16, scale_log2, neg_lse2, Dv, 0, rho2, msum2);
        }
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&bar_tr_ready[b]);
      }

#ifdef GPROJ_TRACE
      ev_n2 = global_ns();
#endif
      // ---- row statistics of all warpgroups (fixed order), lambda = rho / m with the zero-mass rule (Algorithm 1 line 14)
      float rho_lo, rho_hi, m_lo, m_hi;
      f32x2_split(rho2, rho_lo, rho_hi);
      f32x2_split(msum2, m_lo, m_hi);
      float rho_t = rho_lo + rho_hi, m_t = m_lo + m_hi;
      if (wg > 0) { s_rho[wg - 1][row] = rho_t; s_m[wg - 1][row] = m_t; }
      if (C::kSepStaging && threadIdx.x == 128) bulk_wait_group_read0();   // the previous tile's stores have left the staging buffer
      named_bar_sync(1, C::kCompute);
      if (wg == 0) {
#pragma unroll
        for (int w = 0; w < C::kWG - 1; ++w) { rho_t += s_rho[w][row]; m_t += s_m[w][row]; }
        s_lam[row] = (m_t != 0.f) ? __fdiv_rn(rho_t, m_t) : 0.f;
      }
      named_bar_sync(1, C::kCompute);
      const float lam = s_lam[row];
      const float lam_q = (flags & kFlagNoQCorrection) ? 0.f : lam;
      const float lam_k = (flags & kFlagNoKCorrection) ? 0.f : lam;

      mbar_wait(&bar_acc_done, ti & 1, ab, kDqWaitAcc);
      tc_fence_after();
      // The 16-column chunks of the epilogue are dealt round-robin to the warpgroups.  Results are staged in the
      // TMA (128-byte swizzled) layout and written out by TMA stores: Z = -BF16(lambda q), dQ.
      uint8_t *sQt = sRes + rb * 2 * C::kBigTileBytes, *sdOt = sQt + C::kBigTileBytes;
      uint8_t *stage_dq = C::kSepStaging ? sOut : sdOt, *stage_z = C::kSepStaging ? sOut + C::kBigTileBytes : sQt;
      constexpr int kCh = D / (16 * C::kWG);               // 16-column epilogue chunks per warpgroup
      uint32_t a[kCh][16], b[kCh][16];
#pragma unroll
      for (int nch = 0; nch < kCh; ++nch) {
        const int cc = wg + nch * C::kWG;
        tmem_ld16(tmem_base + C::kColAcc0 + lane_addr + 16 * cc, a[nch]);
        tmem_ld16(tmem_base + C::kColAcc1 + lane_addr + 16 * cc, b[nch]);
      }
      tmem_wait_ld();
      tc_fence_before();
      mbar_arrive(&bar_acc_free);          // the accumulators may be overwritten by the next tile
#pragma unroll
      for (int nch = 0; nch < kCh; ++nch) {
        const int cc = wg + nch * C::kWG;
        const uint32_t slab = (cc >> 2) * C::kBigSlabBytes;
#pragma unroll
        for (int v = 0; v < 2; ++v) {
          const uint32_t off = slab + swz128_offset(row, 2 * (cc & 3) + v);
          const uint4 qv = *reinterpret_cast<const uint4 *>(sQt + off);
          const uint32_t qw[4] = {qv.x, qv.y, qv.z, qv.w};
          uint32_t dqw[4], zw[4];
#pragma unroll
          for (int w = 0; w < 4; ++w) {
            const int i = 8 * v + 2 * w;
            const float g0v = __fmul_rn(alpha, __fsub_rn(__uint_as_float(a[nch][i]), __fmul_rn(lam_q, __uint_as_float(b[nch][i]))));
            const float g1v = __fmul_rn(alpha, __fsub_rn(__uint_as_float(a[nch][i + 1]), __fmul_rn(lam_q, __uint_as_float(b[nch][i + 1]))));
            dqw[w] = pack_bf16x2(g0v, g1v);
            // z = BF16(fl32[lambda q]); the sign flip is exact
            zw[w] = pack_bf16x2(__fmul_rn(lam_k, bf16_lo_to_f32(qw[w])), __fmul_rn(lam_k, bf16_hi_to_f32(qw[w]))) ^ 0x80008000u;
          }
          *reinterpret_cast<uint4 *>(stage_dq + off) = make_uint4(dqw[0], dqw[1], dqw[2], dqw[3]);
          *reinterpret_cast<uint4 *>(stage_z + off) = make_uint4(zw[0], zw[1], zw[2], zw[3]);
        }
      }
      fence_proxy_async_smem();
      named_bar_sync(1, C::kCompute);
      if (tile_store_by_tma(tl, N)) {
        if (threadIdx.x == 128) {
          for (int sl = 0; sl < C::kSlabs; ++sl) {
            tma_store_3d(&tmdQ, stage_dq + sl * C::kBigSlabBytes, sl * 64, tl.row0, bh);
            tma_store_3d(&tmZ, stage_z + sl * C::kBigSlabBytes, sl * 64, tl.row0, bh);
          }
          bulk_commit_group();
          if (!C::kSepStaging) bulk_wait_group_read0();   // staging shares the Q / dO buffer: reads must finish first
          mbar_arrive(&bar_res_free[rb]);                 // second arrival: the epilogue no longer needs this buffer
        }
      } else {
        // ragged last tile of a packed sequence that another sequence follows: rows past its end are not ours to write
        if (wg < 2) store_rows_clipped<D>(wg == 0 ? stage_dq : stage_z, C::kBigSlabBytes,
                                         (wg == 0 ? dQg : Zg) + (head_row0 + tl.row0) * D, row, tl.seq_end - tl.row0);
        named_bar_sync(1, C::kCompute);
        if (threadIdx.x == 128) mbar_arrive(&bar_res_free[rb]);
      }
#ifdef GPROJ_TRACE
      if ((threadIdx.x & 127) == 0) tile_event(1 + wg, lin, T, ev_n0, ev_n1, ev_n2, global_ns(), ev_c0, clock64());
#endif
      g0 += T;
    }
    if (threadIdx.x == 128) bulk_wait_group_read0();
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, C::kTmemCols);
}

// ============================================================================================
// dK / dV side
// ============================================================================================
template <int D, bool CAUSAL>
__global__ void __launch_bounds__(BwdCfg<D>::kThreads, 1)
bwd_dkv_kernel(const __grid_constant__ CUtensorMap tmK,    // box 64 x 128 rows
               const __grid_constant__ CUtensorMap tmV,    // box 64 x 128 rows
               const __grid_constant__ CUtensorMap tmQ,    // box 64 x 64 rows
               const __grid_constant__ CUtensorMap tmdO,   // box 64 x 64 rows
               const __grid_constant__ CUtensorMap tmZ,    // box 64 x 64 rows
               const __grid_constant__ CUtensorMap tmdK,   // store, box 64 x 128 rows
               const __grid_constant__ CUtensorMap tmdV,   // store, box 64 x 128 rows
               const float *__restrict__ stats,
               __nv_bfloat16 *__restrict__ dKg, __nv_bfloat16 *__restrict__ dVg,   // plain-store targets of clipped tiles
               const int4 *__restrict__ plan, int nblk,                           // packed sequences: tile list; statistic blocks per head
               int N, int Nq, int BH, int Hkv, int G, int total_tiles, const ItemOrder order, float scale_log2, float alpha, unsigned flags, int *status) {
  // BH counts (batch, KV head) pairs here.  With grouped queries (G > 1) one work item walks the query steps of all G
  // query heads of its KV head, so their contributions are summed in the FP32 accumulators (Section 3.1: key and value
  // contributions also sum over the query heads that share a KV head).
  using C = BwdCfg<D>;
  constexpr int NB = C::kNB, S = C::kDkvStages;
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t *sK = smem;
  uint8_t *sV = sK + C::kBigTileBytes;
  uint8_t *sStage = sV + C::kBigTileBytes;   // stage s: Q, dO, Z step tiles, then 64 x {-LSE log2 e} and 64 x {-D}
  uint8_t *sOut = sStage + S * C::kDkvStageBytes;   // staging (dK tile, then dV tile) when separate

  __shared__ uint64_t bar_res_full, bar_res_free, bar_q_full[S], bar_q_empty[S];
  __shared__ uint64_t bar_s_full[NB], bar_dp_full[NB], bar_r_ready[NB], bar_t_ready[NB], bar_acc_done, bar_acc_free, bar_drain[2];
  __shared__ uint32_t tmem_base_smem;
  __shared__ int cta_abort, cta_skip;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) cta_skip = *reinterpret_cast<volatile int *>(status);
  __syncthreads();
  if (cta_skip != 0) return;

  const bool use_z = (flags & kFlagNoKCorrection) == 0;
  const uint32_t stage_tx = (use_z ? 3 : 2) * C::kStepTileBytes + kExtBlockBytes;
  // Constant operand of the extra K = 16 slice of the score products: three eight-row core matrices (zeros, rows of
  // (1, 1, 1, 0, 0, 0, 0, 0), zeros).  S^T reads (ones, zeros): it adds columns 0..2 of the row-constant tile, the three
  // BF16 pieces of -LSE / alpha; dP^T reads (zeros, ones): columns 8..10, the pieces of -D.
  __shared__ __align__(128) uint4 s_ones[24];
  if (threadIdx.x < 24) {
    s_ones[threadIdx.x] = (threadIdx.x >= 8 && threadIdx.x < 16) ? make_uint4(0x3f803f80u, 0x00003f80u, 0u, 0u) : make_uint4(0u, 0u, 0u, 0u);
    fence_proxy_async_smem();
  }

  AbortState ab{status, &cta_abort};
  if (threadIdx.x == 0) {
    cta_abort = 0;
    mbar_init(&bar_res_full, 1);
    mbar_init(&bar_res_free, 2);
    for (int s = 0; s < S; ++s) { mbar_init(&bar_q_full[s], 1); mbar_init(&bar_q_empty[s], 1); }
    for (int b = 0; b < NB; ++b) {
      mbar_init(&bar_s_full[b], 1); mbar_init(&bar_dp_full[b], 1);
      mbar_init(&bar_r_ready[b], 128 * C::kSlices); mbar_init(&bar_t_ready[b], 128 * C::kSlices);
    }
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
  // tile decode: causal -> key tile 0 has the most query steps and comes first
  // Ragged N: query steps round up.  A zero-filled query column past N contributes exactly nothing (its dO, Q and Z rows
  // are zero and its padded statistics are zero, so t = 0 and r multiplies zero rows); key rows past N are clipped on store.
  // In a packed layout the query columns past the end of the sequence are the next sequence's rows and are masked.
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
          if (g >= S) mbar_wait(&bar_q_empty[st], ((g / S) - 1) & 1, ab, kDkvWaitQEmpty);
          mbar_expect_tx(&bar_q_full[st], stage_tx);
          uint8_t *dst = sStage + st * C::kDkvStageBytes;
          const int qh = q_head0 + n / T, qrel = q_start + (n % T) * C::kStepRows, qrow = tl.oseq0 + qrel;
          for (int s = 0; s < C::kSlabs; ++s) {
            tma_load_3d(dst + s * C::kStepSlabBytes, &tmQ, &bar_q_full[st], s * 64, qrow, qh);
            tma_load_3d(dst + C::kStepTileBytes + s * C::kStepSlabBytes, &tmdO, &bar_q_full[st], s * 64, qrow, qh);
            if (use_z) tma_load_3d(dst + 2 * C::kStepTileBytes + s * C::kStepSlabBytes, &tmZ, &bar_q_full[st], s * 64, qrow, qh);
          }
          bulk_load_1d(dst + 3 * C::kStepTileBytes, reinterpret_cast<const uint8_t *>(stats) + (static_cast<size_t>(qh) * nblk + tl.blk0 + (qrel >> 6)) * kExtBlockBytes,
                       kExtBlockBytes, &bar_q_full[st]);
        }
      }
      if (cta_abort) {
        for (int q = (g > S ? g - S : 0); q < g; ++q)
          for (int spin = 0; spin < 100000 && !mbar_try_wait(&bar_q_full[q % S], (q / S) & 1); ++spin) {}
      }
    }
  } else if (warp == 3) {
    // ---------------------------------------------------------------- TMA loader of the stationary (K, V) tiles
    if (lane == 0) {
      int ti = 0;
      for (int lin = sched.next(); lin >= 0; lin = sched.next(), ++ti) {
        const int bh = hix(lin), krow0 = tile_of(lin).row0;
        if (ti >= 1) mbar_wait(&bar_res_free, (ti - 1) & 1, ab, kDkvWaitResFree);
        mbar_expect_tx(&bar_res_full, 2 * C::kBigTileBytes);
        for (int s = 0; s < C::kSlabs; ++s) {
          tma_load_3d(sK + s * C::kBigSlabBytes, &tmK, &bar_res_full, s * 64, krow0, bh);
          tma_load_3d(sV + s * C::kBigSlabBytes, &tmV, &bar_res_full, s * 64, krow0, bh);
        }
      }
      if (cta_abort && ti > 0)
        for (int spin = 0; spin < 100000 && !mbar_try_wait(&bar_res_full, (ti - 1) & 1); ++spin) {}
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- tensor-core issuer 1: scores (warp-uniform loop, elected issue)
    constexpr uint32_t idesc_s = idesc_bf16_f32(128, 64, 0, 0);    // [128 keys] x [64 queries], contraction over d
    const SmemDesc dscK = make_smem_desc(smem_u32(sK), 16, 1024), dscV = make_smem_desc(smem_u32(sV), 16, 1024);
    const SmemDesc dscQ0 = make_smem_desc(smem_u32(sStage), 16, 1024);                       // K-major view of stage 0
    const SmemDesc dscOnesS = make_smem_desc_noswizzle(smem_u32(s_ones) + 128, 128, 0);      // (ones, zeros), every row group the same
    const SmemDesc dscOnesP = make_smem_desc_noswizzle(smem_u32(s_ones), 128, 0);            // (zeros, ones)
    const SmemDesc dscExt0 = make_smem_desc_noswizzle(smem_u32(sStage + 3 * C::kStepTileBytes), 128, 256);
    int g = 0, ti = 0;
    for (int lin = sched.next(); lin >= 0; lin = sched.next(), ++ti) {
      const int T = G * steps_of(tile_of(lin));
      mbar_wait(&bar_res_full, ti & 1, ab, kDkvWaitKV);
      for (int n = 0; n < T; ++n, ++g) {
        const int st = g % S, b = g % NB;
        mbar_wait(&bar_q_full[st], (g / S) & 1, ab, kDkvWaitQ);
        if (g >= NB) mbar_wait(&bar_q_empty[(g - NB) % S], ((g - NB) / S) & 1, ab, kDkvWaitBuf);   // step g - NB done: its r, t are consumed
        tc_fence_after();
        const SmemDesc dscQ = dscQ0.advanced(st * C::kDkvStageBytes), dscdO = dscQ.advanced(C::kStepTileBytes);
        const uint32_t tS = tmem_base + 128 * b, tdP = tS + 64;
        if (elect_one_sync()) {
#pragma unroll
          for (int k = 0; k < D / 16; ++k) {
            const uint32_t oa = (k / 4) * C::kBigSlabBytes + (k % 4) * 32, ob = (k / 4) * C::kStepSlabBytes + (k % 4) * 32;
            umma_ss(tS, dscK.at(oa), dscQ.at(ob), idesc_s, k > 0);
          }
          umma_ss(tS, dscOnesS.at(0), dscExt0.at(st * C::kDkvStageBytes), idesc_s, 1u);     // - LSE / alpha in every key row
          umma_commit(&bar_s_full[b]);                      // phase 1 of the ALUs needs only S^T
#pragma unroll
          for (int k = 0; k < D / 16; ++k) {
            const uint32_t oa = (k / 4) * C::kBigSlabBytes + (k % 4) * 32, ob = (k / 4) * C::kStepSlabBytes + (k % 4) * 32;
            umma_ss(tdP, dscV.at(oa), dscdO.at(ob), idesc_s, k > 0);
          }
          umma_ss(tdP, dscOnesP.at(0), dscExt0.at(st * C::kDkvStageBytes), idesc_s, 1u);    // - D in every key row
          umma_commit(&bar_dp_full[b]);
          if (n == T - 1) umma_commit(&bar_res_free);   // no MMA reads this K / V tile any more
        }
        __syncwarp();
      }
    }
    drain_mmas_if_aborted(&bar_drain[0], ab);
  } else if (warp == 2) {
    // ---------------------------------------------------------------- tensor-core issuer 2: dV += r^T dO, dK += t^T Q + r^T Z
    constexpr uint32_t idesc_a = idesc_bf16_f32(128, D, 0, 1);     // [128 keys] x [d], contraction over 64 queries
    constexpr uint32_t idesc_fused = idesc_bf16_f32(128, 128, 0, 1);   // d = 64 only: [128 keys] x [dO | Z]
    const SmemDesc dscQ0mn = make_smem_desc(smem_u32(sStage), C::kStepSlabBytes, 1024);    // MN-major view of stage 0
    int g = 0, ti = 0;
    for (int lin = sched.next(); lin >= 0; lin = sched.next(), ++ti) {
      const int T = G * steps_of(tile_of(lin));
      if (ti > 0) mbar_wait(&bar_acc_free, (ti - 1) & 1, ab, kDkvWaitAccFree);   // the previous epilogue has read dV, dK
      for (int p = 0; p < T; ++p, ++g) {
        const int st = g % S, b = g % NB;
        const SmemDesc dscQ = dscQ0mn.advanced(st * C::kDkvStageBytes), dscdO = dscQ.advanced(C::kStepTileBytes),
                       dscZ = dscdO.advanced(C::kStepTileBytes);
        // packed BF16 operands of query slice k (16 queries): r^T over columns 16 k .. 16 k + 7 of the buffer, t^T over the next eight
        const uint32_t tR = tmem_base + 128 * b, tT = tR + 8;
        const uint32_t acc = (p > 0) ? 1u : 0u;
        mbar_wait(&bar_r_ready[b], (g / NB) & 1, ab, kDkvWaitTR);        // r^T is complete: its products run while t^T is computed
        tc_fence_after();
        if (elect_one_sync()) {
          if (D == 64 && use_z) {
            // d = 64: the dO and Z step tiles are adjacent 64-column atoms of one MN-major operand and the dV and dK
            // accumulators are adjacent TMEM columns, so r^T [dO | Z] is ONE full-rate N = 128 product
            // (an N = 64 instruction costs as much as 0.7 of an N = 128 one).
#pragma unroll
            for (int k = 0; k < C::kStepRows / 16; ++k)    // [dV | dK] += r^T [dO | -BF16(lambda Q)]
              umma_ts(tmem_base + C::kColAcc0, tR + 16 * k, dscdO.at(k * 2048), idesc_fused, k > 0 ? 1u : acc);
          } else {
#pragma unroll
            for (int k = 0; k < C::kStepRows / 16; ++k)      // dV += r^T dO
              umma_ts(tmem_base + C::kColAcc0, tR + 16 * k, dscdO.at(k * 2048), idesc_a, k > 0 ? 1u : acc);
            if (use_z) {
#pragma unroll
              for (int k = 0; k < C::kStepRows / 16; ++k)    // dK += r^T (-BF16(lambda Q))   (Algorithm 1 lines 17-18)
                umma_ts(tmem_base + C::kColAcc1, tR + 16 * k, dscZ.at(k * 2048), idesc_a, k > 0 ? 1u : acc);
            }
          }
        }
        __syncwarp();
        mbar_wait(&bar_t_ready[b], (g / NB) & 1, ab, kDkvWaitTR);
        tc_fence_after();
        if (elect_one_sync()) {
          const uint32_t acc_k = use_z ? 1u : acc;           // with the correction, dK already holds this step's r^T Z
#pragma unroll
          for (int k = 0; k < C::kStepRows / 16; ++k)        // dK += t^T Q
            umma_ts(tmem_base + C::kColAcc1, tT + 16 * k, dscQ.at(k * 2048), idesc_a, k > 0 ? 1u : acc_k);
          umma_commit(&bar_q_empty[st]);                    // step done: its stage and its score buffer are free
          if (p == T - 1) umma_commit(&bar_acc_done);
        }
        __syncwarp();
      }
    }
    drain_mmas_if_aborted(&bar_drain[1], ab);
  } else {
    // ---------------------------------------------------------------- compute: thread <-> (key row, query slice of every kGroups-th step)
    const int wg = (warp - 4) >> 2, grp = wg / C::kSlices, slice = wg % C::kSlices;
    const int row = 32 * (warp & 3) + lane;                  // key row within the tile
    const uint32_t lane_addr = static_cast<uint32_t>(32 * (warp & 3)) << 16;
    const uint32_t slice_addr = tmem_base + lane_addr + C::kSliceCols * slice;
    int g0 = 0, ti = 0;
    for (int lin = sched.next(); lin >= 0; lin = sched.next(), ++ti) {
      const TileInfo tl = tile_of(lin);
      const int bh = hix(lin), Th = steps_of(tl), T = G * Th, q_start = q_start_of(tl);
#ifdef GPROJ_TRACE
      const unsigned long long tile_t0 = global_ns();
#endif
      for (int n = (grp - g0 % C::kGroups + C::kGroups) % C::kGroups; n < T; n += C::kGroups) {
        const int g = g0 + n, b = g % NB;
        mbar_wait(&bar_s_full[b], (g / NB) & 1, ab, kDkvWaitSdP);
        tc_fence_after();
        const uint32_t tS16 = slice_addr + 128 * b, tdP16 = tS16 + 64;
        const int nh = n % Th;                                      // step within the current query head
        const int Lq = tl.oseq_end - tl.oseq0, off = (tl.seq_end - tl.seq0) - Lq, krel0 = tl.row0 - tl.seq0;
        const int qs = q_start + nh * C::kStepRows;                           // first query (inside its sequence) of the step
        const int q0 = qs + C::kSliceCols * slice;                            // ... of the slice's column 0
        float pkeep[32];
        if ((CAUSAL && qs < krel0 + 128 - off) || qs + C::kStepRows > Lq)
          dkv_phase1<true>(tS16, scale_log2, CAUSAL ? krel0 + row - off - q0 : 0, Lq - 1 - q0, pkeep);
        else
          dkv_phase1<false>(tS16, scale_log2, 0, 0, pkeep);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&bar_r_ready[b]);
        mbar_wait(&bar_dp_full[b], (g / NB) & 1, ab, kDkvWaitSdP);
        tc_fence_after();
        dkv_phase2(tS16, tdP16, pkeep);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&bar_t_ready[b]);
      }

      mbar_wait(&bar_acc_done, ti & 1, ab, kDkvWaitAcc);
      tc_fence_after();
      uint8_t *stage_dk = C::kSepStaging ? sOut : sK, *stage_dv = C::kSepStaging ? sOut + C::kBigTileBytes : sV;
      constexpr int kCh = D / (16 * C::kWG);               // 16-column epilogue chunks per warpgroup
      uint32_t a[kCh][16], b[kCh][16];
#pragma unroll
      for (int nch = 0; nch < kCh; ++nch) {
        const int cc = wg + nch * C::kWG;
        tmem_ld16(tmem_base + C::kColAcc0 + lane_addr + 16 * cc, a[nch]);
        tmem_ld16(tmem_base + C::kColAcc1 + lane_addr + 16 * cc, b[nch]);
      }
      tmem_wait_ld();
      tc_fence_before();
      mbar_arrive(&bar_acc_free);          // the accumulators may be overwritten by the next tile
      if (C::kSepStaging) {
        if (threadIdx.x == 128) {
          mbar_arrive(&bar_res_free);      // second arrival: with its own staging buffer the epilogue never touches K / V
          bulk_wait_group_read0();         // the previous tile's stores have left the staging buffer
        }
        named_bar_sync(1, C::kCompute);
      }
      // staged in the TMA (128-byte swizzled) layout, then stored by TMA
#pragma unroll
      for (int nch = 0; nch < kCh; ++nch) {
        const int cc = wg + nch * C::kWG;
        const uint32_t slab = (cc >> 2) * C::kBigSlabBytes;
#pragma unroll
        for (int v = 0; v < 2; ++v) {
          const uint32_t off = slab + swz128_offset(row, 2 * (cc & 3) + v);
          uint32_t vw[4], kw[4];
#pragma unroll
          for (int w = 0; w < 4; ++w) {
            const int i = 8 * v + 2 * w;
            vw[w] = pack_bf16x2(__uint_as_float(a[nch][i]), __uint_as_float(a[nch][i + 1]));
            kw[w] = pack_bf16x2(__fmul_rn(alpha, __uint_as_float(b[nch][i])), __fmul_rn(alpha, __uint_as_float(b[nch][i + 1])));
          }
          *reinterpret_cast<uint4 *>(stage_dv + off) = make_uint4(vw[0], vw[1], vw[2], vw[3]);
          *reinterpret_cast<uint4 *>(stage_dk + off) = make_uint4(kw[0], kw[1], kw[2], kw[3]);
        }
      }
      fence_proxy_async_smem();
      named_bar_sync(1, C::kCompute);
      if (tile_store_by_tma(tl, N)) {
        if (threadIdx.x == 128) {
          for (int sl = 0; sl < C::kSlabs; ++sl) {
            tma_store_3d(&tmdV, stage_dv + sl * C::kBigSlabBytes, sl * 64, tl.row0, bh);
            tma_store_3d(&tmdK, stage_dk + sl * C::kBigSlabBytes, sl * 64, tl.row0, bh);
          }
          bulk_commit_group();
          if (!C::kSepStaging) {           // staging shares the K / V tile: its reads must finish before the next load
            bulk_wait_group_read0();
            mbar_arrive(&bar_res_free);
          }
#ifdef GPROJ_TRACE
          tile_trace(lin, tile_t0, global_ns());
#endif
        }
      } else {
        // ragged last tile of a packed sequence that another sequence follows: rows past its end are not ours to write
        if (wg < 2) store_rows_clipped<D>(wg == 0 ? stage_dk : stage_dv, C::kBigSlabBytes,
                                         (wg == 0 ? dKg : dVg) + (static_cast<size_t>(bh) * N + tl.row0) * D, row, tl.seq_end - tl.row0);
        named_bar_sync(1, C::kCompute);
        if (!C::kSepStaging && threadIdx.x == 128) mbar_arrive(&bar_res_free);
      }
      g0 += T;
    }
    if (threadIdx.x == 128) bulk_wait_group_read0();
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, C::kTmemCols);
}

}  // namespace gproj
