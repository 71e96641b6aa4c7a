// Fused FP32 attention, forward and backward, in plain SIMT arithmetic: the paper's "fused FP32" comparison arm
// (Appendix "Accuracy and Cost", paragraph "Fused FP32 baseline"; Table "method-definitions", row "FP32 attention").
// It decodes the BF16 inputs, computes every product, the softmax and the gradients with FP32 fused multiply-adds on
// the CUDA cores (no tensor core, no TF32), returns BF16 outputs and gradients, and saves an FP32 output plus three
// FP32 row statistics (log-sum-exp, row maximum, inverse normaliser); nothing of size N^2 is stored.
// It exists to be compared with, not to be fast: 64 x 64 tiles in shared memory, 128 threads, each thread a 4 x 8
// block of scores and a 4 x (d / 8) block of an output tile.
//
//   fp32_attn_fwd_kernel   query tile stationary, online softmax over 64-key tiles (Eq. "row-attention")
//   fp32_attn_dq_kernel    query tile stationary:  D = rowsum(dO * O32), P = exp(s - max) / l, dS = P (dP - D), dQ = alpha dS K
//   fp32_attn_dkv_kernel   key tile stationary:    dV = P^T dO, dK = alpha dS^T Q            (Eq. "row-gradients")
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace gproj {

template <int D>
struct Fp32Cfg {
  static constexpr int kTile = 64, kThreads = 128, kLd = D + 4, kLdP = kTile + 1;
  static constexpr int kFwdSmem = (3 * kTile * kLd + kTile * kLdP) * 4;
  static constexpr int kBwdSmem = (4 * kTile * kLd + 2 * kTile * kLdP) * 4;
};

// rows [row0, row0 + 64) of a [rows_total x D] BF16 matrix -> FP32 shared memory [64][ld]; rows past rows_total are zero
template <int D>
__device__ __forceinline__ void fp32_load_tile(float *dst, int ld, const __nv_bfloat16 *src, int row0, int rows_total) {
  for (int i = threadIdx.x; i < 64 * (D / 8); i += blockDim.x) {
    const int r = i / (D / 8), c8 = i % (D / 8);
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (row0 + r < rows_total) v = *reinterpret_cast<const uint4 *>(src + static_cast<size_t>(row0 + r) * D + 8 * c8);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    float *o = dst + r * ld + 8 * c8;
#pragma unroll
    for (int k = 0; k < 4; ++k) { o[2 * k] = __uint_as_float(w[k] << 16); o[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u); }
  }
}
template <int D>
__device__ __forceinline__ void fp32_load_tile_f32(float *dst, int ld, const float *src, int row0, int rows_total) {
  for (int i = threadIdx.x; i < 64 * (D / 4); i += blockDim.x) {
    const int r = i / (D / 4), c4 = i % (D / 4);
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (row0 + r < rows_total) v = *reinterpret_cast<const float4 *>(src + static_cast<size_t>(row0 + r) * D + 4 * c4);
    *reinterpret_cast<float4 *>(dst + r * ld + 4 * c4) = v;
  }
}
// acc[4][8] = A[4 ty + r][:] . B[8 tx + c][:]   (both [64][ld], contraction over D)
template <int D>
__device__ __forceinline__ void fp32_scores(float (&acc)[4][8], const float *A, const float *B, int ld, int ty, int tx) {
#pragma unroll
  for (int r = 0; r < 4; ++r)
#pragma unroll
    for (int c = 0; c < 8; ++c) acc[r][c] = 0.f;
  for (int k = 0; k < D; k += 4) {
    float4 a[4], b[8];
#pragma unroll
    for (int r = 0; r < 4; ++r) a[r] = *reinterpret_cast<const float4 *>(A + (4 * ty + r) * ld + k);
#pragma unroll
    for (int c = 0; c < 8; ++c) b[c] = *reinterpret_cast<const float4 *>(B + (8 * tx + c) * ld + k);
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        acc[r][c] = fmaf(a[r].x, b[c].x, acc[r][c]);
        acc[r][c] = fmaf(a[r].y, b[c].y, acc[r][c]);
        acc[r][c] = fmaf(a[r].z, b[c].z, acc[r][c]);
        acc[r][c] = fmaf(a[r].w, b[c].w, acc[r][c]);
      }
  }
}
// out[4][D / 8] += sum_j P[4 ty + r][j] X[j][(D / 8) tx + c]      (P [64][ldp], X [64][ld])
template <int D>
__device__ __forceinline__ void fp32_apply(float (&out)[4][D / 8], const float *P, int ldp, const float *X, int ld, int ty, int tx) {
  for (int j = 0; j < 64; ++j) {
    float p[4], x[D / 8];
#pragma unroll
    for (int r = 0; r < 4; ++r) p[r] = P[(4 * ty + r) * ldp + j];
#pragma unroll
    for (int c = 0; c < D / 8; c += 4) *reinterpret_cast<float4 *>(&x[c]) = *reinterpret_cast<const float4 *>(X + j * ld + (D / 8) * tx + c);
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < D / 8; ++c) out[r][c] = fmaf(p[r], x[c], out[r][c]);
  }
}
// out[4][D / 8] += sum_i P[i][4 ty + r] X[i][(D / 8) tx + c]      (the transposed use: rows of `out` are columns of P)
template <int D>
__device__ __forceinline__ void fp32_apply_t(float (&out)[4][D / 8], const float *P, int ldp, const float *X, int ld, int ty, int tx) {
  for (int i = 0; i < 64; ++i) {
    float p[4], x[D / 8];
#pragma unroll
    for (int r = 0; r < 4; ++r) p[r] = P[i * ldp + 4 * ty + r];
#pragma unroll
    for (int c = 0; c < D / 8; c += 4) *reinterpret_cast<float4 *>(&x[c]) = *reinterpret_cast<const float4 *>(X + i * ld + (D / 8) * tx + c);
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < D / 8; ++c) out[r][c] = fmaf(p[r], x[c], out[r][c]);
  }
}
__device__ __forceinline__ float fp32_row_max8(float v) {      // over the eight threads (consecutive lanes) that share a row
  v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 1)); v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 2)); return fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 4));
}
__device__ __forceinline__ float fp32_row_sum8(float v) {
  v += __shfl_xor_sync(0xffffffffu, v, 1); v += __shfl_xor_sync(0xffffffffu, v, 2); return v + __shfl_xor_sync(0xffffffffu, v, 4);
}
template <int D>
__device__ __forceinline__ void fp32_store_bf16(__nv_bfloat16 *dst, int row0, int rows_total, const float (&v)[4][D / 8], float scale, int ty, int tx) {
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int row = row0 + 4 * ty + r;
    if (row < rows_total) {
#pragma unroll
      for (int c = 0; c < D / 8; c += 2)
        *reinterpret_cast<__nv_bfloat162 *>(dst + static_cast<size_t>(row) * D + (D / 8) * tx + c) =
            __floats2bfloat162_rn(v[r][c] * scale, v[r][c + 1] * scale);
    }
  }
}

// saved state per (head, row): O32 [N][D], then lse, row maximum of the scaled scores, inverse normaliser ([N] each)
template <int D, bool CAUSAL>
__global__ void __launch_bounds__(128) fp32_attn_fwd_kernel(const __nv_bfloat16 *__restrict__ Q, const __nv_bfloat16 *__restrict__ K,
                                                           const __nv_bfloat16 *__restrict__ V, __nv_bfloat16 *__restrict__ O,
                                                           float *__restrict__ O32, float *__restrict__ stats, int N, float alpha) {
  using C = Fp32Cfg<D>;
  extern __shared__ float fsm[];
  float *sQ = fsm, *sK = sQ + 64 * C::kLd, *sV = sK + 64 * C::kLd, *sP = sV + 64 * C::kLd;
  const int head = blockIdx.y, q0 = 64 * (gridDim.x - 1 - blockIdx.x);       // longest causal tiles first
  const int ty = threadIdx.x / 8, tx = threadIdx.x % 8;
  const size_t hoff = static_cast<size_t>(head) * N * D;
  fp32_load_tile<D>(sQ, C::kLd, Q + hoff, q0, N);
  float m_run[4], l_run[4], acc[4][D / 8];
#pragma unroll
  for (int r = 0; r < 4; ++r) { m_run[r] = -INFINITY; l_run[r] = 0.f;
#pragma unroll
    for (int c = 0; c < D / 8; ++c) acc[r][c] = 0.f; }
  const int kend = CAUSAL ? min(N, q0 + 64) : N;
  for (int k0 = 0; k0 < kend; k0 += 64) {
    __syncthreads();
    fp32_load_tile<D>(sK, C::kLd, K + hoff, k0, N);
    fp32_load_tile<D>(sV, C::kLd, V + hoff, k0, N);
    __syncthreads();
    float s[4][8];
    fp32_scores<D>(s, sQ, sK, C::kLd, ty, tx);
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int qi = q0 + 4 * ty + r;
      float mx = -INFINITY;
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const int kj = k0 + 8 * tx + c;
        s[r][c] = (kj < N && (!CAUSAL || kj <= qi)) ? s[r][c] * alpha : -INFINITY;
        mx = fmaxf(mx, s[r][c]);
      }
      mx = fp32_row_max8(mx);
      const float m_new = fmaxf(m_run[r], mx), corr = (m_run[r] == -INFINITY) ? 0.f : __expf(m_run[r] - m_new);
      float sum = 0.f;
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const float p = (s[r][c] == -INFINITY) ? 0.f : __expf(s[r][c] - m_new);
        sP[(4 * ty + r) * C::kLdP + 8 * tx + c] = p;
        sum += p;
      }
      sum = fp32_row_sum8(sum);
      l_run[r] = l_run[r] * corr + sum;
      m_run[r] = m_new;
#pragma unroll
      for (int c = 0; c < D / 8; ++c) acc[r][c] *= corr;
    }
    __syncthreads();
    fp32_apply<D>(acc, sP, C::kLdP, sV, C::kLd, ty, tx);
  }
  float *lse = stats + static_cast<size_t>(head) * 3 * N, *rmax = lse + N, *rinv = rmax + N;
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int qi = q0 + 4 * ty + r;
    const float inv = 1.f / l_run[r];
#pragma unroll
    for (int c = 0; c < D / 8; ++c) acc[r][c] *= inv;
    if (qi < N) {
#pragma unroll
      for (int c = 0; c < D / 8; c += 4)
        *reinterpret_cast<float4 *>(O32 + hoff + static_cast<size_t>(qi) * D + (D / 8) * tx + c) = make_float4(acc[r][c], acc[r][c + 1], acc[r][c + 2], acc[r][c + 3]);
      if (tx == 0) { lse[qi] = m_run[r] + __logf(l_run[r]); rmax[qi] = m_run[r]; rinv[qi] = inv; }
    }
  }
  fp32_store_bf16<D>(O + hoff, q0, N, acc, 1.f, ty, tx);
}

// P, dS of one 64 x 64 tile into shared memory: P = exp(alpha s - max) inv,  dS = P (dP - D)
template <int D, bool CAUSAL>
__device__ __forceinline__ void fp32_p_ds_tile(float *sP, float *sdS, int ldp, const float *sQ, const float *sdO, const float *sK, const float *sV,
                                               int ld, int q0, int k0, int N, float alpha, const float *rmax, const float *rinv, const float *Dv,
                                               int ty, int tx) {
  float s[4][8], dp[4][8];
  fp32_scores<D>(s, sQ, sK, ld, ty, tx);
  fp32_scores<D>(dp, sdO, sV, ld, ty, tx);
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int qi = q0 + 4 * ty + r;
    const float mx = qi < N ? rmax[qi] : 0.f, inv = qi < N ? rinv[qi] : 0.f, dd = qi < N ? Dv[4 * ty + r] : 0.f;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      const int kj = k0 + 8 * tx + c;
      const bool keep = qi < N && kj < N && (!CAUSAL || kj <= qi);
      const float p = keep ? __expf(fmaf(s[r][c], alpha, -mx)) * inv : 0.f;
      sP[(4 * ty + r) * ldp + 8 * tx + c] = p;
      sdS[(4 * ty + r) * ldp + 8 * tx + c] = p * (dp[r][c] - dd);
    }
  }
}

template <int D, bool CAUSAL>
__global__ void __launch_bounds__(128) fp32_attn_dq_kernel(const __nv_bfloat16 *__restrict__ Q, const __nv_bfloat16 *__restrict__ K,
                                                          const __nv_bfloat16 *__restrict__ V, const __nv_bfloat16 *__restrict__ dO,
                                                          const float *__restrict__ O32, const float *__restrict__ stats,
                                                          float *__restrict__ Drow, __nv_bfloat16 *__restrict__ dQ, int N, float alpha) {
  using C = Fp32Cfg<D>;
  extern __shared__ float fsm[];
  float *sQ = fsm, *sdO = sQ + 64 * C::kLd, *sK = sdO + 64 * C::kLd, *sV = sK + 64 * C::kLd, *sP = sV + 64 * C::kLd, *sdS = sP + 64 * C::kLdP;
  __shared__ float sD[64];
  const int head = blockIdx.y, q0 = 64 * (gridDim.x - 1 - blockIdx.x);
  const int ty = threadIdx.x / 8, tx = threadIdx.x % 8;
  const size_t hoff = static_cast<size_t>(head) * N * D;
  const float *rmax = stats + static_cast<size_t>(head) * 3 * N + N, *rinv = rmax + N;
  fp32_load_tile<D>(sQ, C::kLd, Q + hoff, q0, N);
  fp32_load_tile<D>(sdO, C::kLd, dO + hoff, q0, N);
  fp32_load_tile_f32<D>(sK, C::kLd, O32 + hoff, q0, N);          // the saved FP32 output, only for D
  __syncthreads();
  if (threadIdx.x < 64) {                                        // D_i = sum_c dO_ic O_ic in FP32 from the FP32 output
    float a = 0.f;
    for (int c = 0; c < D; ++c) a = fmaf(sdO[threadIdx.x * C::kLd + c], sK[threadIdx.x * C::kLd + c], a);
    sD[threadIdx.x] = a;
    if (q0 + threadIdx.x < N) Drow[static_cast<size_t>(head) * N + q0 + threadIdx.x] = a;
  }
  float acc[4][D / 8];
#pragma unroll
  for (int r = 0; r < 4; ++r)
#pragma unroll
    for (int c = 0; c < D / 8; ++c) acc[r][c] = 0.f;
  const int kend = CAUSAL ? min(N, q0 + 64) : N;
  for (int k0 = 0; k0 < kend; k0 += 64) {
    __syncthreads();
    fp32_load_tile<D>(sK, C::kLd, K + hoff, k0, N);
    fp32_load_tile<D>(sV, C::kLd, V + hoff, k0, N);
    __syncthreads();
    fp32_p_ds_tile<D, CAUSAL>(sP, sdS, C::kLdP, sQ, sdO, sK, sV, C::kLd, q0, k0, N, alpha, rmax, rinv, sD, ty, tx);
    __syncthreads();
    fp32_apply<D>(acc, sdS, C::kLdP, sK, C::kLd, ty, tx);        // dQ += dS K
  }
  fp32_store_bf16<D>(dQ + hoff, q0, N, acc, alpha, ty, tx);
}

template <int D, bool CAUSAL>
__global__ void __launch_bounds__(128) fp32_attn_dkv_kernel(const __nv_bfloat16 *__restrict__ Q, const __nv_bfloat16 *__restrict__ K,
                                                           const __nv_bfloat16 *__restrict__ V, const __nv_bfloat16 *__restrict__ dO,
                                                           const float *__restrict__ stats, const float *__restrict__ Drow,
                                                           __nv_bfloat16 *__restrict__ dK, __nv_bfloat16 *__restrict__ dV, int N, float alpha) {
  using C = Fp32Cfg<D>;
  extern __shared__ float fsm[];
  float *sQ = fsm, *sdO = sQ + 64 * C::kLd, *sK = sdO + 64 * C::kLd, *sV = sK + 64 * C::kLd, *sP = sV + 64 * C::kLd, *sdS = sP + 64 * C::kLdP;
  __shared__ float sD[64];
  const int head = blockIdx.y, k0 = 64 * blockIdx.x;             // key tile 0 has the most query tiles (causal) and comes first
  const int ty = threadIdx.x / 8, tx = threadIdx.x % 8;
  const size_t hoff = static_cast<size_t>(head) * N * D;
  const float *rmax = stats + static_cast<size_t>(head) * 3 * N + N, *rinv = rmax + N;
  fp32_load_tile<D>(sK, C::kLd, K + hoff, k0, N);
  fp32_load_tile<D>(sV, C::kLd, V + hoff, k0, N);
  float accK[4][D / 8], accV[4][D / 8];
#pragma unroll
  for (int r = 0; r < 4; ++r)
#pragma unroll
    for (int c = 0; c < D / 8; ++c) { accK[r][c] = 0.f; accV[r][c] = 0.f; }
  for (int q0 = CAUSAL ? k0 : 0; q0 < N; q0 += 64) {
    __syncthreads();
    fp32_load_tile<D>(sQ, C::kLd, Q + hoff, q0, N);
    fp32_load_tile<D>(sdO, C::kLd, dO + hoff, q0, N);
    if (threadIdx.x < 64) sD[threadIdx.x] = (q0 + threadIdx.x < N) ? Drow[static_cast<size_t>(head) * N + q0 + threadIdx.x] : 0.f;
    __syncthreads();
    fp32_p_ds_tile<D, CAUSAL>(sP, sdS, C::kLdP, sQ, sdO, sK, sV, C::kLd, q0, k0, N, alpha, rmax, rinv, sD, ty, tx);
    __syncthreads();
    fp32_apply_t<D>(accV, sP, C::kLdP, sdO, C::kLd, ty, tx);     // dV += P^T dO
    fp32_apply_t<D>(accK, sdS, C::kLdP, sQ, C::kLd, ty, tx);     // dK += dS^T Q
  }
  fp32_store_bf16<D>(dV + hoff, k0, N, accV, 1.f, ty, tx);
  fp32_store_bf16<D>(dK + hoff, k0, N, accK, alpha, ty, tx);
}

}  // namespace gproj
