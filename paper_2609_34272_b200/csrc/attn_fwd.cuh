// Fused attention forward for sm_100a: O = softmax(alpha Q K^T) V and the row log-sum-exp.
//
// One CTA owns a tile of 128 query rows of one (batch, head) and walks the key tiles.
// Roles (warp-specialised, 192 threads):
//   warp 0      TMA producer: Q tile once, then K_j / V_j tiles through a ring of stages
//   warp 1      tensor-core issuer: S = Q K_j^T (FP32 in TMEM), then O += P~ V_j with the BF16
//               probabilities read straight from TMEM; owns the TMEM allocation
//   warps 2..5  softmax: thread <-> query row (TMEM lane), so every row statistic is a private
//               register; online softmax on the UNSCALED logits with the subtract-before-scale
//               rounding of Eq. "gproj-forward": z = exp2(fl32[ fl32(x - x_max) * (alpha log2 e) ]);
//               l accumulates the FP32 z, the value product uses BF16(z).
// The saved state is BF16 O and FP32 LSE = alpha x_max + ln l  (Algorithm 1, "Input").
#pragma once
#include "sm100_primitives.cuh"

namespace gproj {

template <int D>
struct FwdCfg {
  static constexpr int kBlockM = 128;
  static constexpr int kBlockN = 128;
  static constexpr int kSlabs = D / 64;               // 64-column (128-byte) swizzle slabs per tile
  static constexpr int kSlabBytes = 128 * 128;         // 128 rows x 128 B
  static constexpr int kTileBytes = kSlabs * kSlabBytes;
  static constexpr int kStages = (D == 64) ? 3 : 2;
  static constexpr int kSmemBytes = kTileBytes * (1 + 2 * kStages) + 1024;
  static constexpr int kTmemCols = 256;                // S: [0,128)  (P~ aliases its first 64)   O: [128,128+D)
  static constexpr int kThreads = 192;
};

enum FwdWaitCode { kFwdWaitQ = 0x11, kFwdWaitKV = 0x12, kFwdWaitKVEmpty = 0x13, kFwdWaitS = 0x14, kFwdWaitP = 0x15, kFwdWaitO = 0x16 };

template <int D, bool CAUSAL>
__global__ void __launch_bounds__(192, 1)
attn_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, __nv_bfloat16 *__restrict__ O, float *__restrict__ LSE,
                int N, int BH, float scale_log2, float alpha, int *status) {
  using C = FwdCfg<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t *sQ = smem;
  uint8_t *sK = sQ + C::kTileBytes;
  uint8_t *sV = sK + C::kStages * C::kTileBytes;

  __shared__ uint64_t bar_q, bar_kv_full[C::kStages], bar_kv_empty[C::kStages], bar_s_full, bar_p_ready, bar_o_done;
  __shared__ uint32_t tmem_base_smem;
  __shared__ int cta_abort, cta_skip;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) cta_skip = *reinterpret_cast<volatile int *>(status);
  __syncthreads();
  if (cta_skip != 0) return;   // an earlier wait gave up: drain the rest of the grid quickly
  const int n_qt = N / C::kBlockM;
  const int lin = blockIdx.x;
  const int qt = CAUSAL ? (n_qt - 1 - lin / BH) : (lin / BH);   // causal: longest rows first
  const int bh = lin % BH;
  const int n_kv = CAUSAL ? qt + 1 : n_qt;
  const int row0 = bh * N + qt * C::kBlockM;                      // first row of this tile in the [BH*N, d] view

  AbortState ab{status, &cta_abort};
  if (threadIdx.x == 0) {
    cta_abort = 0;
    mbar_init(&bar_q, 1);
    for (int s = 0; s < C::kStages; ++s) { mbar_init(&bar_kv_full[s], 1); mbar_init(&bar_kv_empty[s], 1); }
    mbar_init(&bar_s_full, 1);
    mbar_init(&bar_p_ready, 128);
    mbar_init(&bar_o_done, 1);
    fence_mbar_init();
  }
  if (warp == 1) { tmem_alloc(&tmem_base_smem, C::kTmemCols); tmem_relinquish(); }
  if (warp == 0 && lane == 0) { tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = __shfl_sync(0xffffffffu, tmem_base_smem, 0);   // shuffle marks it warp-uniform
  const uint32_t tS = tmem_base, tO = tmem_base + 128;

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      mbar_expect_tx(&bar_q, C::kTileBytes);
      for (int s = 0; s < C::kSlabs; ++s) tma_load_2d(sQ + s * C::kSlabBytes, &tmQ, &bar_q, s * 64, row0);
      for (int j = 0; j < n_kv; ++j) {
        const int st = j % C::kStages;
        if (j >= C::kStages) mbar_wait(&bar_kv_empty[st], ((j / C::kStages) - 1) & 1, ab, kFwdWaitKVEmpty);
        mbar_expect_tx(&bar_kv_full[st], 2 * C::kTileBytes);
        const int krow = bh * N + j * C::kBlockN;
        for (int s = 0; s < C::kSlabs; ++s) {
          tma_load_2d(sK + st * C::kTileBytes + s * C::kSlabBytes, &tmK, &bar_kv_full[st], s * 64, krow);
          tma_load_2d(sV + st * C::kTileBytes + s * C::kSlabBytes, &tmV, &bar_kv_full[st], s * 64, krow);
        }
      }
      // every load above is consumed by an MMA that the epilogue waits for, so nothing is in flight at exit
      // unless the CTA aborted; then give the copies a bounded chance to land before shared memory is released.
      if (cta_abort) {
        for (int j = (n_kv > C::kStages ? n_kv - C::kStages : 0); j < n_kv; ++j) {
          const int st = j % C::kStages;
          for (int spin = 0; spin < 100000 && !mbar_try_wait(&bar_kv_full[st], (j / C::kStages) & 1); ++spin) {}
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- tensor-core issuer
    // The whole warp runs this loop so that every address stays provably warp-uniform (descriptor operands
    // then live in uniform registers); one elected lane issues the MMAs and commits.
    {
      constexpr uint32_t idesc_s = idesc_bf16_f32(128, 128, 0, 0);   // S = Q K^T, both operands K-major
      constexpr uint32_t idesc_o = idesc_bf16_f32(128, D, 0, 1);     // O += P V, V is MN-major (d contiguous)
      const SmemDesc dscQ = make_smem_desc(smem_u32(sQ), 16, 1024);
      const SmemDesc dscK0 = make_smem_desc(smem_u32(sK), 16, 1024);                  // K-major view of K stage 0
      const SmemDesc dscV0 = make_smem_desc(smem_u32(sV), C::kSlabBytes, 1024);       // MN-major view of V stage 0
      mbar_wait(&bar_q, 0, ab, kFwdWaitQ);
      for (int j = 0; j < n_kv; ++j) {
        const int st = j % C::kStages;
        mbar_wait(&bar_kv_full[st], (j / C::kStages) & 1, ab, kFwdWaitKV);
        tc_fence_after();
        const SmemDesc dscK = dscK0.advanced(st * C::kTileBytes), dscV = dscV0.advanced(st * C::kTileBytes);
        if (elect_one_sync()) {
#pragma unroll
          for (int k = 0; k < D / 16; ++k) {
            const uint32_t off = (k / 4) * C::kSlabBytes + (k % 4) * 32;
            umma_ss(tS, dscQ.at(off), dscK.at(off), idesc_s, k > 0);
          }
          umma_commit(&bar_s_full);
        }
        __syncwarp();
        mbar_wait(&bar_p_ready, j & 1, ab, kFwdWaitP);
        tc_fence_after();
        const uint32_t acc = (j > 0) ? 1u : 0u;
        if (elect_one_sync()) {
#pragma unroll
          for (int k = 0; k < C::kBlockN / 16; ++k) umma_ts(tO, tS + 8 * k, dscV.at(k * 2048), idesc_o, k > 0 ? 1u : acc);
          umma_commit(&bar_kv_empty[st]);
        }
        __syncwarp();
      }
      if (elect_one_sync())
      umma_commit(&bar_o_done);
    }
  } else {
    // ---------------------------------------------------------------- softmax: one thread per query row
    const int row = 32 * (warp & 3) + lane;
    const uint32_t lane_addr = static_cast<uint32_t>(32 * (warp & 3)) << 16;
    float m_run = -INFINITY, l_run = 0.f;
    for (int j = 0; j < n_kv; ++j) {
      mbar_wait(&bar_s_full, j & 1, ab, kFwdWaitS);
      tc_fence_after();
      uint32_t xr[4][32];
#pragma unroll
      for (int c = 0; c < 4; ++c) tmem_ld32(tS + lane_addr + 32 * c, xr[c]);
      tmem_wait_ld();
      float mx = -INFINITY;
      if (CAUSAL && j == n_kv - 1) {
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (32 * c + i > row) xr[c][i] = 0xff800000u;   // -inf: key beyond the diagonal
      }
#pragma unroll
      for (int c = 0; c < 4; ++c)
#pragma unroll
        for (int i = 0; i < 32; ++i) mx = fmaxf(mx, __uint_as_float(xr[c][i]));
      const float m_new = fmaxf(m_run, mx);
      const float corr = fast_exp2(__fmul_rn(__fsub_rn(m_run, m_new), scale_log2));
      float rs = 0.f;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t pk[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const float z0 = fast_exp2(__fmul_rn(__fsub_rn(__uint_as_float(xr[c][2 * i]), m_new), scale_log2));
          const float z1 = fast_exp2(__fmul_rn(__fsub_rn(__uint_as_float(xr[c][2 * i + 1]), m_new), scale_log2));
          rs += z0 + z1;
          pk[i] = pack_bf16x2(z0, z1);
        }
        tmem_st16(tS + lane_addr + 16 * c, pk);   // P~ overwrites the S columns already consumed
      }
      l_run = l_run * corr + rs;
      // The accumulator may be rescaled now: bar_s_full also covers the previous P~ V product
      // (a commit tracks every MMA issued before it).
      if (j > 0 && __any_sync(0xffffffffu, m_new != m_run)) {
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          uint32_t o[32];
          tmem_ld32(tO + lane_addr + 32 * c, o);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * corr);
          tmem_st32(tO + lane_addr + 32 * c, o);
        }
      }
      m_run = m_new;
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&bar_p_ready);
    }
    // ---- epilogue: O = BF16(acc / l), LSE = alpha x_max + ln l
    mbar_wait(&bar_o_done, 0, ab, kFwdWaitO);
    tc_fence_after();
    const float inv_l = 1.0f / l_run;
    __nv_bfloat16 *orow = O + static_cast<size_t>(row0 + row) * D;
#pragma unroll
    for (int c = 0; c < D / 32; ++c) {
      uint32_t o[32];
      tmem_ld32(tO + lane_addr + 32 * c, o);
      tmem_wait_ld();
      uint32_t pk[16];
#pragma unroll
      for (int i = 0; i < 16; ++i)
        pk[i] = pack_bf16x2(__uint_as_float(o[2 * i]) * inv_l, __uint_as_float(o[2 * i + 1]) * inv_l);
      uint4 *dst = reinterpret_cast<uint4 *>(orow + 32 * c);
#pragma unroll
      for (int v = 0; v < 4; ++v) dst[v] = make_uint4(pk[4 * v], pk[4 * v + 1], pk[4 * v + 2], pk[4 * v + 3]);
    }
    LSE[row0 + row] = fmaf(m_run, alpha, logf(l_run));
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, C::kTmemCols);
}

}  // namespace gproj
