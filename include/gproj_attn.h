/*
 * gproj_attn.h -- C ABI of the fused BF16 attention forward / backward with the GProj
 * (gauge projection) correction, for NVIDIA B200 (sm_100a).
 *
 * Conventions shared by every entry point
 *   - Tensors Q, K, V, O, dO, dQ, dK, dV are DEVICE pointers to BF16 (16-bit patterns),
 *     layout [B][H][N][d] contiguous with d fastest; base addresses 16-byte aligned.
 *   - LSE is a DEVICE pointer to FP32 [B][H][N]: the natural-log sum-exp of the scaled scores
 *     s_ij = softmax_scale * q_i . k_j over the row's support.
 *   - Supported shapes: d in {64, 128}; any N >= 1 (tiles of 128 rows; a ragged last tile is zero-filled on load,
 *     masked where it would enter a row statistic and clipped on store); B, H >= 1 with B*H*N < 2^31, B*H < 2^20 and
 *     N <= 2^24 (packed calls: fewer than 2^24 query tiles and key tiles); anything else is GPROJ_ERR_SHAPE;
 *     N_q = N_k = N; causal != 0 means row i attends to j <= i.  The *_gqa entry points take separate query / KV head counts, the
 *     *_rect entry points separate query / key lengths.
 *   - The caller owns all memory.  The library never allocates device memory, frees or synchronises; work is
 *     enqueued on `stream` (a cudaStream_t passed as void*; NULL = the default stream).  (The host-buffer entry point
 *     also uses two streams of its own, see there.)
 *     After the first call on a device (one-time attribute set-up), gproj_attn_fwd and gproj_attn_bwd with a
 *     caller-supplied workspace have been captured into a CUDA graph and replayed (that is what is tested).
 *   - Return value: GPROJ_OK (0) or a negative gproj_status.  Nothing throws, aborts or traps.
 *     Inputs are never modified; outputs are fully overwritten; non-finite inputs are undefined
 *     behaviour (the paper's error decomposition assumes finite quantities).
 *   - Every in-kernel wait is bounded.  A wait that gives up makes the launch finish early with
 *     undefined outputs and records a code readable through gproj_last_device_status().
 */
#ifndef GPROJ_ATTN_H
#define GPROJ_ATTN_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum gproj_status {
  GPROJ_OK = 0,
  GPROJ_ERR_NULL = -1,      /* a required pointer is NULL */
  GPROJ_ERR_SHAPE = -2,     /* unsupported d, non-positive dimension, H not a multiple of Hkv, or a size limit
                               (B*H*N >= 2^31, B*H >= 2^20, N > 2^24, 2^24 or more tiles in a packed call) */
  GPROJ_ERR_ALIGN = -3,     /* a tensor base address is not 16-byte aligned */
  GPROJ_ERR_WORKSPACE = -4, /* workspace NULL, misaligned or smaller than gproj_attn_bwd_workspace_bytes() */
  GPROJ_ERR_SCALE = -5,     /* softmax_scale not finite or not > 0 */
  GPROJ_ERR_ARCH = -6,      /* current device is not compute capability 10.x */
  GPROJ_ERR_CUDA = -7,      /* a CUDA runtime / driver call failed (descriptor encode, launch) */
  GPROJ_ERR_TIMEOUT = -8,   /* reported by gproj_last_device_status(): a bounded in-kernel wait gave up */
  GPROJ_ERR_FLAGS = -9      /* unknown bit set in flags, or both ONLY_* bits */
} gproj_status;

/* flags of gproj_attn_bwd (ablations of Section 5.2: "FA3-SBS" = both bits, "GProj-Q" = bit 1 only) */
#define GPROJ_FLAG_NO_Q_CORRECTION 1u /* dQ = BF16(alpha * tK): Algorithm 1 line 14 without the lambda term */
#define GPROJ_FLAG_NO_K_CORRECTION 2u /* dK = BF16(alpha * t^T Q): Algorithm 1 without Pass 2 (lines 15-18) */
/* Profiling aids (no counterpart in the paper): launch one of the two backward kernels only, so that it can be
 * timed by itself.  ONLY_DKV reads the row statistics and the scaled-query operand that an earlier full or
 * ONLY_DQ call with the same inputs left in the same workspace.  The two bits are mutually exclusive. */
#define GPROJ_FLAG_ONLY_DQ_PASS 4u  /* writes dQ (and the workspace); dK, dV untouched */
#define GPROJ_FLAG_ONLY_DKV_PASS 8u /* writes dK, dV; dQ untouched */

/*
 * Forward: O = softmax(softmax_scale * Q K^T [causal]) V and the row log-sum-exp.
 * Follows Eq. "row-attention" (Section 3.1) with the subtract-before-scale softmax of
 * Eq. "gproj-forward" (Appendix "Implemented Arithmetic and Rounding", "Forward and saved state"):
 * the unscaled maximum is subtracted with its own FP32 rounding before the scale and the
 * base-two exponential; the value product uses BF16 probabilities, the normaliser their FP32 values.
 * One deviation from the literal equation: the subtracted value is a LAZY running maximum.  Key tiles are taken in
 * order; the reference m is the true maximum of the first tile and is raised to the running maximum only when a later
 * tile exceeds it by more than 8 in the base-two exponent domain (alpha log2 e (x_max - m) > 8).  So m <= x_max < m +
 * 8 / (alpha log2 e) and z can reach 2^8 instead of at most 1; O = (sum z v) / (sum z) and LSE = alpha m + ln(sum z) do not
 * depend on the reference, and a row with a single key still has z = 1 exactly (o_0 = v_0 bitwise).
 *   in : Q, K, V  (device, BF16)        out: O (device, BF16), LSE (device, FP32)
 */
int gproj_attn_fwd(const void *Q, const void *K, const void *V, void *O, float *LSE,
                   int B, int H, int N, int d, float softmax_scale, int causal, void *stream);

/*
 * Bytes of device scratch gproj_attn_bwd needs for this shape (0 if the shape is unsupported).
 * The paper's resource statement (Appendix "Implemented Arithmetic", "Cost") allows a query-shaped
 * workspace and two row-statistic arrays; this implementation uses one BF16 query-shaped array
 * (the operand BF16(lambda_i q_i) of Algorithm 1 line 17) and the two row constants (LSE, D) in blocks of 64 rows,
 * thirty-two bytes per row: they reach the dK/dV side as a 16-column BF16 operand of its score products (each
 * constant as three BF16 pieces that add up to the FP32 value).
 */
size_t gproj_attn_bwd_workspace_bytes(int B, int H, int N, int d);

/*
 * Backward with the GProj correction: Algorithm 1 (Section 4), rounding points of
 * Eq. "gproj-row-mass", "gproj-query-implemented" and "gproj-key-implemented".
 *   D = rowsum(dO * O) from the saved BF16 O; P = exp(S - LSE); r = BF16(P); t = BF16(P (dP - D));
 *   rho = rowsum(t), m = rowsum(r), lambda = rho / m (0 where m = 0);
 *   dQ = BF16(alpha (tK - lambda rK));  dK = BF16(alpha (t^T Q - r^T BF16(lambda Q)));  dV = BF16(r^T dO).
 *   in : Q, K, V, O, dO (device, BF16), LSE (device, FP32, as written by gproj_attn_fwd)
 *   out: dQ, dK, dV (device, BF16)
 *   workspace: device scratch, 256-byte aligned, at least gproj_attn_bwd_workspace_bytes(); contents
 *              undefined on entry and on exit; must not be shared by calls that overlap on the GPU.
 *   flags: 0 = full GProj; see GPROJ_FLAG_*.
 */
int gproj_attn_bwd(const void *Q, const void *K, const void *V, const void *O, const float *LSE, const void *dO,
                   void *dQ, void *dK, void *dV,
                   int B, int H, int N, int d, float softmax_scale, int causal,
                   void *workspace, size_t workspace_bytes, unsigned flags, void *stream);

/*
 * Grouped-query variants: Q, O, dO, dQ have H query heads ([B][H][N][d], LSE [B][H][N]); K, V, dK, dV have Hkv heads
 * ([B][Hkv][N][d]) with H a multiple of Hkv; query head h reads key / value head h / (H / Hkv).  Key and value
 * gradients sum over the query heads that share a KV head (Section 3.1, text after Eq. "row-gradients"; Appendix
 * "Rounding in the implemented key correction": grouped queries only enlarge the set of contributing query heads); the
 * sum is taken in the FP32 accumulators, before the single final BF16 cast.  Everything else, including the workspace
 * size (gproj_attn_bwd_workspace_bytes(B, H, N, d) with the QUERY head count), is as for the functions above, which are
 * the case Hkv = H.  This is the paper's own layout (16 query / 4 KV heads, d = 64).
 */
int gproj_attn_fwd_gqa(const void *Q, const void *K, const void *V, void *O, float *LSE,
                       int B, int H, int Hkv, int N, int d, float softmax_scale, int causal, void *stream);
int gproj_attn_bwd_gqa(const void *Q, const void *K, const void *V, const void *O, const float *LSE, const void *dO,
                       void *dQ, void *dK, void *dV,
                       int B, int H, int Hkv, int N, int d, float softmax_scale, int causal,
                       void *workspace, size_t workspace_bytes, unsigned flags, void *stream);

/*
 * Forward with options (fwd_flags = 0 is gproj_attn_fwd_gqa).  GPROJ_FWD_FLAG_FMA_SOFTMAX selects the native fused form
 * of the softmax exponent, z = exp2(fma(x, a, -fl32(x_max a))) with a = softmax_scale * log2 e (Eq. "historical-fma",
 * Appendix "The source of the saved-output error"): x a is not rounded on its own, so the largest score of a row need
 * not map to exactly zero and a one-key row can return o_0 != v_0.  With this flag x_max is always the true running
 * maximum (no lazy rule).  It exists to reproduce the paper's "FA3" forward next to the subtract-before-scale one on
 * the same kernels; training code should leave it off.
 */
#define GPROJ_FWD_FLAG_FMA_SOFTMAX 1u
int gproj_attn_fwd_ex(const void *Q, const void *K, const void *V, void *O, float *LSE,
                      int B, int H, int Hkv, int N, int d, float softmax_scale, int causal,
                      unsigned fwd_flags, void *stream);

/*
 * Unequal query and key lengths (Appendix "Synthetic Numerical Suite": unequal lengths, empty causal rows).  Q, O, dO, dQ
 * are [B][H][Nq][d] and LSE [B][H][Nq]; K, V, dK, dV are [B][Hkv][Nk][d]; Nq >= 1, Nk >= 1, otherwise as the grouped-query
 * functions, which are the case Nq = Nk.  Non-causal: every query sees all Nk keys.  Causal: the diagonal ends at the
 * last query and the last key, i.e. the support of query i is the keys j <= i + (Nk - Nq) (the paper does not fix an
 * alignment; this is the one under which appending cached keys in front of a block of new queries stays causal).  For
 * Nq > Nk the first Nq - Nk queries then have an EMPTY support: their O and dQ rows are written as zero and their LSE as
 * +infinity, so that P = exp(S - LSE) = 0 wherever the backward meets them; they add nothing to dK or dV, and they get
 * no correction (Algorithm 1, line 14: lambda = 0 when the rounded row mass is zero).  The backward takes the LSE this
 * forward wrote.  Workspace: gproj_attn_bwd_workspace_bytes(B, H, Nq, d), i.e. sized by the QUERY rows.  Errors as for
 * gproj_attn_fwd_ex / gproj_attn_bwd_gqa, with GPROJ_ERR_SHAPE also for Nk <= 0 or B*Hkv*Nk >= 2^31.
 */
int gproj_attn_fwd_rect(const void *Q, const void *K, const void *V, void *O, float *LSE,
                        int B, int H, int Hkv, int Nq, int Nk, int d, float softmax_scale, int causal,
                        unsigned fwd_flags, void *stream);
int gproj_attn_bwd_rect(const void *Q, const void *K, const void *V, const void *O, const float *LSE, const void *dO,
                        void *dQ, void *dK, void *dV,
                        int B, int H, int Hkv, int Nq, int Nk, int d, float softmax_scale, int causal,
                        void *workspace, size_t workspace_bytes, unsigned flags, void *stream);

/*
 * Packed (variable-length) sequences.  The paper's synthetic suite exercises "packed segments" and "unequal lengths"
 * (Appendix "Synthetic Numerical Suite"); its training layout packs documents into one row axis.  Here the tensors are
 * [H][T][d] (queries, O, dO, dQ) and [Hkv][T][d] (keys, values, dK, dV) with T = cu_seqlens[num_seqs] rows per head; sequence
 * s owns rows cu_seqlens[s] .. cu_seqlens[s+1]-1 of EVERY head, and a query attends only to keys of its own sequence
 * (Eq. "row-attention" with the support L restricted to the sequence; causal: keys at or before it inside the sequence).
 * LSE is [H][T].  Query and key lengths of a sequence are equal, so no row has an empty support.  Empty sequences
 * (two equal offsets) are allowed and skipped.
 *   - cu_seqlens is a HOST array of num_seqs + 1 non-decreasing ints starting at 0 (read during the call, not kept).
 *   - The kernels need a tile list in DEVICE memory.  gproj_attn_varlen_plan() writes it into a HOST buffer of
 *     gproj_attn_varlen_plan_bytes() bytes; the caller copies that buffer to 16-byte aligned device memory (any way it
 *     likes) and passes the device pointer.  The plan depends on cu_seqlens and on `causal` (tiles are ordered by
 *     decreasing work), not on H, d or the data; it can be reused for every layer and step with the same packing.
 *   - Arithmetic, flags, status codes and workspace rules are those of gproj_attn_fwd_ex / gproj_attn_bwd_gqa; the
 *     workspace size comes from gproj_attn_bwd_varlen_workspace_bytes().  Errors: GPROJ_ERR_SHAPE for a malformed
 *     cu_seqlens (or H*T >= 2^31), GPROJ_ERR_NULL / GPROJ_ERR_ALIGN for the plan pointer, GPROJ_ERR_WORKSPACE for a plan
 *     buffer or workspace that is too small.
 */
size_t gproj_attn_varlen_plan_bytes(const int *cu_seqlens, int num_seqs);
int gproj_attn_varlen_plan(const int *cu_seqlens, int num_seqs, int causal, void *plan_host, size_t plan_bytes);
int gproj_attn_fwd_varlen(const void *Q, const void *K, const void *V, void *O, float *LSE, const int *cu_seqlens,
                          int num_seqs, const void *plan_device, int H, int Hkv, int d, float softmax_scale, int causal,
                          unsigned fwd_flags, void *stream);
size_t gproj_attn_bwd_varlen_workspace_bytes(const int *cu_seqlens, int num_seqs, int H, int d);
int gproj_attn_bwd_varlen(const void *Q, const void *K, const void *V, const void *O, const float *LSE, const void *dO,
                          void *dQ, void *dK, void *dV, const int *cu_seqlens, int num_seqs, const void *plan_device,
                          int H, int Hkv, int d, float softmax_scale, int causal, void *workspace, size_t workspace_bytes,
                          unsigned flags, void *stream);

/*
 * Packed sequences whose query and key lengths differ (Appendix "Synthetic Numerical Suite": packed segments, unequal
 * lengths, empty causal rows).  Queries, O, dO, dQ are [H][Tq][d] with Tq = cu_seqlens_q[num_seqs], LSE [H][Tq]; keys,
 * values, dK, dV are [Hkv][Tk][d] with Tk = cu_seqlens_k[num_seqs]; sequence s owns query rows cu_seqlens_q[s] ..
 * cu_seqlens_q[s+1]-1 and key rows cu_seqlens_k[s] .. cu_seqlens_k[s+1]-1.  Inside a sequence the rules are those of the
 * *_rect entry points: causal means query i sees the keys j <= i + (Lk - Lq), a query without visible key gets O = 0,
 * dQ = 0 and LSE = +infinity.  A sequence may have no queries (its dK, dV rows are written as zero), no keys (all its
 * queries are such empty rows), or neither (skipped); Tq and Tk must both be positive.  Plan, workspace
 * (gproj_attn_bwd_varlen_workspace_bytes() of cu_seqlens_q), flags and errors are as for the packed entry points above,
 * which are the case cu_seqlens_k == cu_seqlens_q; a plan built by one pair of plan functions works only with the
 * forward / backward of the same pair and the same offsets.
 */
size_t gproj_attn_varlen_qk_plan_bytes(const int *cu_seqlens_q, const int *cu_seqlens_k, int num_seqs);
int gproj_attn_varlen_qk_plan(const int *cu_seqlens_q, const int *cu_seqlens_k, int num_seqs, int causal, void *plan_host,
                              size_t plan_bytes);
int gproj_attn_fwd_varlen_qk(const void *Q, const void *K, const void *V, void *O, float *LSE, const int *cu_seqlens_q,
                             const int *cu_seqlens_k, int num_seqs, const void *plan_device, int H, int Hkv, int d,
                             float softmax_scale, int causal, unsigned fwd_flags, void *stream);
int gproj_attn_bwd_varlen_qk(const void *Q, const void *K, const void *V, const void *O, const float *LSE, const void *dO,
                             void *dQ, void *dK, void *dV, const int *cu_seqlens_q, const int *cu_seqlens_k, int num_seqs,
                             const void *plan_device, int H, int Hkv, int d, float softmax_scale, int causal, void *workspace,
                             size_t workspace_bytes, unsigned flags, void *stream);

/*
 * Forward and backward in one call from HOST buffers (a convenience around the entry points above; the paper's
 * Algorithm 1 starts from tensors already on the device).  Q, K, V, dO are copied to the device, the forward
 * (Eq. "gproj-forward") and the backward (Algorithm 1) run, and dQ, dK, dV (and O, LSE when those pointers are not NULL)
 * are copied back.  Large problems are cut into up to 16 slabs of whole KV heads (about 2 MiB of Q each) that are pipelined:
 * the kernels run on `stream`, the copies in and out on two internal streams, ordered by events so that nothing of the call
 * starts before the work already queued on `stream` and `stream` reaches the end of the call only after the last copy-out.
 *   - Q, K, V, dO, O, LSE, dQ, dK, dV are HOST pointers with the layouts of gproj_attn_fwd_gqa / gproj_attn_bwd_gqa.  Page-locked
 *     memory makes the call asynchronous; pageable memory works but serialises in the CUDA runtime.  The buffers must stay
 *     valid until the stream has reached the end of the call's work.
 *   - `staging` is DEVICE memory owned by the caller, 256-byte aligned, at least gproj_attn_host_staging_bytes() bytes (copies
 *     of the eight tensors, LSE and the backward workspace); GPROJ_ERR_WORKSPACE otherwise.  No device memory is allocated;
 *     the first pipelined call on a device creates the two streams and 34 events, which live until the process exits.
 *   - flags: those of gproj_attn_bwd without the ONLY_* bits (GPROJ_ERR_FLAGS for those).
 *   - Calls from several host threads on one device are serialised while they enqueue.
 *   - If the call returns an error after it has begun to enqueue work, `stream` has been made to wait for everything
 *     the call queued on its internal streams, so synchronising `stream` is enough before the host buffers are reused.
 */
size_t gproj_attn_host_staging_bytes(int B, int H, int Hkv, int N, int d);
int gproj_attn_fwd_bwd_host(const void *Q, const void *K, const void *V, const void *dO, void *O, float *LSE,
                            void *dQ, void *dK, void *dV, int B, int H, int Hkv, int N, int d, float softmax_scale,
                            int causal, void *staging, size_t staging_bytes, unsigned flags, void *stream);

/*
 * Backward for callers that must not allocate device memory (the paper has no counterpart: this is a
 * convenience of this library).  Some hosts of this code cannot call cudaMalloc at the point where they
 * need a gradient: a plugin running inside another framework's memory pool, a real-time or safety-audited
 * process whose memory is fixed at start-up, or a callback in which the CUDA allocator may not be entered.
 * This entry point takes no workspace: the scratch of gproj_attn_bwd lives in a fixed device array of
 * GPROJ_STATIC_SCRATCH_BYTES that is part of the library image, so every GPU that loads the library holds
 * that much memory until the process exits.
 *   - Same inputs, outputs, flags and arithmetic as gproj_attn_bwd; results are bitwise the same.
 *   - Shapes whose gproj_attn_bwd_workspace_bytes() exceeds GPROJ_STATIC_SCRATCH_BYTES are rejected with
 *     GPROJ_ERR_WORKSPACE (problems up to about 7.5 Mi elements B*H*N*d at d = 64 fit, e.g. B*H = 16, N = 4096); nothing is launched.
 *   - The first call on each device looks up the array's device address (with that device current); make
 *     that first call before any stream capture begins.  No call allocates or frees anything.
 *   - All calls on a device share the one array, and it keeps whatever the last call left there, possibly from
 *     another shape.  Nothing in it has to start at zero: the first kernel writes every word whose value the second
 *     one uses; the few words the second kernel reads beyond those (the spare statistics block behind a sequence
 *     whose length is not a multiple of 128) belong to masked columns and never reach a result.  Two calls that
 *     overlap on the GPU (different streams, no dependency) race on the array: serialise them.
 */
#define GPROJ_STATIC_SCRATCH_BYTES (16u << 20)
int gproj_attn_bwd_static_scratch(const void *Q, const void *K, const void *V, const void *O, const float *LSE,
                                  const void *dO, void *dQ, void *dK, void *dV,
                                  int B, int H, int N, int d, float softmax_scale, int causal,
                                  unsigned flags, void *stream);

/*
 * Fused FP32 attention, the paper's "fused FP32" comparison arm (Appendix "Accuracy and Cost", paragraph "Fused FP32
 * baseline"; Table "method-definitions", row "FP32 attention"): the BF16 inputs are decoded and every product, the
 * softmax (Eq. "row-attention") and the gradients (Eq. "row-gradients") are computed in FP32 fused multiply-adds on the
 * CUDA cores (no tensor core, no TF32); outputs and gradients are returned in BF16.  The forward saves an FP32 output
 * and three FP32 row statistics (log-sum-exp, row maximum of the scaled scores, inverse normaliser); the backward
 * recomputes P = exp(s - max) / l tile by tile and takes D = rowsum(dO * O) from the FP32 output.  Nothing of size N^2 is
 * stored.  A baseline to compare accuracy and cost with, an order of magnitude slower than the tensor-core path.
 *   Q, K, V, dO, O, dQ, dK, dV: DEVICE BF16 [B][H][N][d] (one head count; d in {64, 128}; any N >= 1); causal as above.
 *   saved: DEVICE scratch, 256-byte aligned, gproj_fp32_attn_saved_bytes() bytes, written by the forward and read (its
 *   row-term part also written) by the backward of the same problem; GPROJ_ERR_WORKSPACE if NULL, misaligned or short.
 *   Other errors as for gproj_attn_fwd.  One launch (forward) / two launches (backward) on `stream`.
 */
size_t gproj_fp32_attn_saved_bytes(int B, int H, int N, int d);
int gproj_fp32_attn_fwd(const void *Q, const void *K, const void *V, void *O, void *saved, size_t saved_bytes,
                        int B, int H, int N, int d, float softmax_scale, int causal, void *stream);
int gproj_fp32_attn_bwd(const void *Q, const void *K, const void *V, const void *dO, void *saved, size_t saved_bytes,
                        void *dQ, void *dK, void *dV, int B, int H, int N, int d, float softmax_scale, int causal, void *stream);

/*
 * Key smoothing, the comparison arm of Section 5.1 and of Table "method-definitions" ("FA3 on mean-subtracted keys"):
 * subtract the per-sequence, per-KV-head mean row, Y_j = BF16(fl32(X_j - mean_j X_j)), mean and subtraction in FP32.
 * The arm is built from calls of this library: K~ = gproj_key_smooth(K); the forward on (Q, K~, V) with
 * GPROJ_FWD_FLAG_FMA_SOFTMAX; the backward with both corrections off; dK = gproj_key_smooth(dK~), which is the
 * vector-Jacobian product of the subtraction (dK_j = dK~_j - mean_l dK~_l).  Softmax is unchanged by the shift in exact
 * arithmetic; what the shift removes is the common component of the keys that the leaked row mass multiplies, not
 * the leak itself (Section 2).  The paper's experiments use it only as a baseline; so does this library.
 *   X, Y: DEVICE BF16, [B][Hkv][N][d] (dense) or [Hkv][T][d] with HOST offsets cu_seqlens (packed; the mean is taken
 *   inside each sequence; empty sequences are skipped); Y may be X.  One launch per sequence, on `stream`.
 *   Errors: GPROJ_ERR_NULL, GPROJ_ERR_SHAPE (d not 64 / 128, non-positive sizes, malformed offsets), GPROJ_ERR_ALIGN,
 *   GPROJ_ERR_ARCH, GPROJ_ERR_CUDA.
 */
int gproj_key_smooth(const void *X, void *Y, int B, int Hkv, int N, int d, void *stream);
int gproj_key_smooth_varlen(const void *X, void *Y, const int *cu_seqlens, int num_seqs, int Hkv, int d, void *stream);

/*
 * Synchronises `stream`, then returns GPROJ_OK, GPROJ_ERR_TIMEOUT if any kernel launched by this
 * library on the current device since the last call recorded an abandoned wait, or GPROJ_ERR_CUDA.
 * If `detail` is non-NULL it receives the raw device code (0 when fine) and the code is cleared.
 * (No counterpart in the paper: diagnostics only.)
 */
int gproj_last_device_status(void *stream, int *detail);

/*
 * Failure-detection self-test (no counterpart in the paper): enqueues a one-warp kernel whose only wait can never be
 * satisfied.  The wait gives up after its budget (a fraction of a second), so a following gproj_last_device_status()
 * returns GPROJ_ERR_TIMEOUT with detail 0x7e01, and clears it.  Nothing faults, traps or hangs; the context stays usable.
 * Until the status is read and cleared, kernels launched by this library on the device return early without working.
 */
int gproj_selftest_wait_timeout(void *stream);

/* Static, human-readable name of a status code. */
const char *gproj_status_string(int status);

/* Number of kernels the most recent successful gproj_attn_fwd / gproj_attn_bwd call on this thread launched. */
int gproj_last_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* GPROJ_ATTN_H */
