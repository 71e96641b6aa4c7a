// Host side of the C ABI declared in include/gproj_attn.h: argument checks, TMA descriptors,
// kernel launches.  No allocation, no synchronisation (except gproj_last_device_status).
#include "gproj_attn.h"

#include <cmath>
#include <cstdint>
#include <algorithm>
#include <map>
#include <mutex>
#include <tuple>
#include <vector>

#include "attn_bwd.cuh"
#include "attn_bwd_w128.cuh"
#include "attn_fwd.cuh"
#include "key_smoothing.cuh"
#include "attn_fp32.cuh"

namespace {

using namespace gproj;

// Launch-status word: written by a kernel whose bounded wait gave up, read back on request.
__device__ int g_device_status;

// Self-test of the bounded-wait machinery: one warp waits on an mbarrier that nothing will ever arrive on.  The wait
// gives up after its cycle budget, records its code in the status word and the kernel returns normally.
__global__ void wait_timeout_selftest_kernel(int *status) {
  __shared__ uint64_t bar;
  __shared__ int cta_abort;
  if (threadIdx.x == 0) { cta_abort = 0; mbar_init(&bar, 1); fence_mbar_init(); }
  __syncthreads();
  AbortState ab{status, &cta_abort};
  mbar_wait(&bar, 0, ab, 0x7e);
  __syncthreads();
}

constexpr int kMaxDevices = 64;

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

#ifndef GPROJ_HOST_SLAB_LOG2
#define GPROJ_HOST_SLAB_LOG2 21
#endif
constexpr int kHostSlabLog2 = GPROJ_HOST_SLAB_LOG2;   // log2 of the Q bytes per slab of the host-buffer entry point
constexpr int kMaxSlabs = 16;   // the host-buffer entry point pipelines at most this many slabs of heads

struct DeviceState {
  bool ready = false;
  bool arch_ok = false;
  int *status_ptr = nullptr;
  int sm_count = 0;
  // host-buffer entry point only: copy-in and copy-out streams and the events that order them against the caller's stream
  bool pipe_ready = false;
  cudaStream_t in_stream = nullptr, out_stream = nullptr;
  cudaEvent_t ev_start = nullptr, ev_end = nullptr, ev_in[kMaxSlabs] = {}, ev_done[kMaxSlabs] = {};
};

std::mutex g_mutex;
std::mutex g_pipe_mutex;   // serialises the host-buffer entry point's use of the per-device streams and events
DeviceState g_dev[kMaxDevices];
EncodeTiledFn g_encode = nullptr;
thread_local int tl_launch_count = 0;

template <typename Kernel>
cudaError_t allow_smem(Kernel kernel, int bytes) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
}

// One-time, per-device set-up: capability check, status word address, shared-memory opt-in.
int device_state(DeviceState **out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return GPROJ_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mutex);
  DeviceState &st = g_dev[dev];
  if (!st.ready) {
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return GPROJ_ERR_CUDA;
    st.arch_ok = (major == 10);
    if (cudaDeviceGetAttribute(&st.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || st.sm_count <= 0)
      return GPROJ_ERR_CUDA;
    if (st.arch_ok) {
      if (!g_encode) {
        cudaDriverEntryPointQueryResult q;
        void *fn = nullptr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn)
          return GPROJ_ERR_CUDA;
        g_encode = reinterpret_cast<EncodeTiledFn>(fn);
      }
      if (cudaGetSymbolAddress(reinterpret_cast<void **>(&st.status_ptr), g_device_status) != cudaSuccess)
        return GPROJ_ERR_CUDA;
      bool ok = true;
      ok &= allow_smem(attn_fwd_kernel<64, true, false, 0>, FwdCfg<64>::kSmemBytes) == cudaSuccess;
      ok &= allow_smem(attn_fwd_kernel<64, true, false, 2>, FwdCfg<64>::kSmemBytes) == cudaSuccess;
      ok &= allow_smem(attn_fwd_kernel<64, true, true, 0>, FwdCfg<64>::kSmemBytes) == cudaSuccess;
      ok &= allow_smem(attn_fwd_kernel<64, true, true, 2>, FwdCfg<64>::kSmemBytes) == cudaSuccess;
      ok &= allow_smem(attn_fwd_kernel<64, false, false, 0>, FwdCfg<64>::kSmemBytes) == cudaSuccess;
      ok &= allow_smem(attn_fwd_kernel<64, false, false, 2>, FwdCfg<64>::kSmemBytes) == cudaSuccess;
      ok &= allow_smem(attn_fwd_kernel<64, false, true, 0>, FwdCfg<64>::kSmemBytes) == cudaSuccess;
      ok &= allow_smem(attn_fwd_kernel<64, false, true, 2>, FwdCfg<64>::kSmemBytes) == cudaSuccess;
      ok &= allow_smem(attn_fwd_kernel<128, true, false, 0>, FwdCfg<128>::kSmemBytes) == cudaSuccess;
      ok &= allow_smem(attn_fwd_kernel<128, true, false, 1>, FwdCfg<128>::kSmemBytes) == cudaSuccess;
      ok &= allow_smem(attn_fwd_kernel<128, true, false, 2>, FwdCfg<128>::kSmemBytes) == cudaSuccess;
      ok &= allow_smem(attn_fwd_kernel<128, true, true, 0>, FwdCfg<128>::kSmemBytes) == cudaSuccess;
      ok &= allow_smem(attn_fwd_kernel<128, true, true, 2>, FwdCfg<128>::kSmemBytes) == cudaSuccess;
      ok &= allow_smem(attn_fwd_kernel<128, false, false, 0>, FwdCfg<128>::kSmemBytes) == cudaSuccess;
      ok &= allow_smem(attn_fwd_kernel<128, false, false, 1>, FwdCfg<128>::kSmemBytes) == cudaSuccess;
      ok &= allow_smem(attn_fwd_kernel<128, false, false, 2>, FwdCfg<128>::kSmemBytes) == cudaSuccess;
      ok &= allow_smem(attn_fwd_kernel<128, false, true, 0>, FwdCfg<128>::kSmemBytes) == cudaSuccess;
      ok &= allow_smem(attn_fwd_kernel<128, false, true, 2>, FwdCfg<128>::kSmemBytes) == cudaSuccess;
      ok &= allow_smem(bwd_dkv_w128_kernel<true>, BwdW128::kDkvSmemBytes) == cudaSuccess;
      ok &= allow_smem(bwd_dkv_w128_kernel<false>, BwdW128::kDkvSmemBytes) == cudaSuccess;
      ok &= allow_smem(bwd_dq_kernel<64, true>, BwdCfg<64>::kDqSmemBytes) == cudaSuccess;
      ok &= allow_smem(bwd_dq_kernel<64, false>, BwdCfg<64>::kDqSmemBytes) == cudaSuccess;
      ok &= allow_smem(bwd_dq_kernel<128, true>, BwdCfg<128>::kDqSmemBytes) == cudaSuccess;
      ok &= allow_smem(bwd_dq_kernel<128, false>, BwdCfg<128>::kDqSmemBytes) == cudaSuccess;
      ok &= allow_smem(bwd_dkv_kernel<128, true>, BwdCfg<128>::kDkvSmemBytes) == cudaSuccess;
      ok &= allow_smem(bwd_dkv_kernel<128, false>, BwdCfg<128>::kDkvSmemBytes) == cudaSuccess;
      if (!ok) { (void)cudaGetLastError(); return GPROJ_ERR_CUDA; }
    }
    st.ready = true;
  }
  *out = &st;
  return st.arch_ok ? GPROJ_OK : GPROJ_ERR_ARCH;
}

// [heads x N x d] BF16 row-major view, box = 64 columns (128 B, one swizzle atom) x box_rows of ONE head: a tile never
// crosses into the next head, rows past N read as zero and are skipped by stores.
bool make_map(CUtensorMap *map, const void *base, int heads, int N, int d, int box_rows) {
  cuuint64_t dims[3] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(N), static_cast<cuuint64_t>(heads)};
  cuuint64_t strides[2] = {static_cast<cuuint64_t>(d) * 2, static_cast<cuuint64_t>(N) * d * 2};
  cuuint32_t box[3] = {64, static_cast<cuuint32_t>(box_rows), 1};
  cuuint32_t elem[3] = {1, 1, 1};
  return g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, elem,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_shape(int B, int H, int N, int d) {
  if (B <= 0 || H <= 0 || N <= 0) return GPROJ_ERR_SHAPE;
  if (d != 64 && d != 128) return GPROJ_ERR_SHAPE;
  const long long rows = static_cast<long long>(B) * H * N;
  if (rows >= (1LL << 31) || static_cast<long long>(B) * H >= (1LL << 20) || N > (1 << 24)) return GPROJ_ERR_SHAPE;
  return GPROJ_OK;
}

size_t align256(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }

// Launch `kernel`; with overlap_previous it may be scheduled while the kernel before it in the stream still runs
// (programmatic dependent launch: the kernel itself waits, by griddep_wait, before it reads what that kernel writes).
template <typename... Params, typename... Args>
void launch_after(void (*kernel)(Params...), dim3 grid, int threads, size_t smem, cudaStream_t s, bool overlap_previous,
                  Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(static_cast<unsigned>(threads));
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = overlap_previous ? 1 : 0;
  (void)cudaLaunchKernelEx(&cfg, kernel, static_cast<Params>(args)...);   // the caller reads cudaGetLastError()
}

int launch_fwd(const void *Q, const void *K, const void *V, void *O, float *LSE, int B, int H, int Hkv, int N, int Nk, int d,
               float softmax_scale, int causal, unsigned fwd_flags, const int4 *plan, int n_plan_tiles, void *stream);
int launch_bwd(const void *Q, const void *K, const void *V, const void *O, const float *LSE, const void *dO,
               void *dQ, void *dK, void *dV, int B, int H, int Hkv, int N, int Nk, int d, float softmax_scale, int causal,
               void *workspace, size_t workspace_bytes, unsigned flags, const int4 *plan_q, const int4 *plan_kv,
               int n_plan_q_tiles, int n_plan_kv_tiles, int nblk, void *stream);

// Row constants (-LSE / alpha, -D) for the dK/dV side: per 64 rows one K-major operand tile of 16 BF16 columns (2048 B;
// per head ceil(N / 64) of them, the last one zero-padded), plus one spare block: the 128-wide steps fetch two blocks at
// a time and may reach one past the end.
size_t stats_blocks_bytes(size_t blocks, int) { return align256((blocks + 1) * static_cast<size_t>(gproj::kExtBlockBytes)); }
size_t stats_bytes(int heads, int N, int d) { return stats_blocks_bytes(static_cast<size_t>(heads) * ((N + 63) / 64), d); }

}  // namespace

extern "C" {

int gproj_attn_fwd(const void *Q, const void *K, const void *V, void *O, float *LSE, int B, int H, int N, int d,
                   float softmax_scale, int causal, void *stream) {
  return gproj_attn_fwd_gqa(Q, K, V, O, LSE, B, H, H, N, d, softmax_scale, causal, stream);
}

int gproj_attn_fwd_gqa(const void *Q, const void *K, const void *V, void *O, float *LSE, int B, int H, int Hkv, int N,
                       int d, float softmax_scale, int causal, void *stream) {
  return gproj_attn_fwd_ex(Q, K, V, O, LSE, B, H, Hkv, N, d, softmax_scale, causal, 0u, stream);
}

int gproj_attn_fwd_ex(const void *Q, const void *K, const void *V, void *O, float *LSE, int B, int H, int Hkv, int N,
                      int d, float softmax_scale, int causal, unsigned fwd_flags, void *stream) {
  return launch_fwd(Q, K, V, O, LSE, B, H, Hkv, N, N, d, softmax_scale, causal, fwd_flags, nullptr, 0, stream);
}

}  // extern "C"

namespace {

// The kernels' item order for `heads` heads of n_per_head tiles dealt in groups of `group` ranks (clamped to 1 .. n_per_head).
FastDiv fast_div(unsigned d) {
  FastDiv f;
  f.div = d;
  f.mul = 0;
  f.shr = 0;
  if (d > 1) {
    unsigned lg = 0;
    while ((1ull << lg) < d) ++lg;                       // ceil(log2 d)
    const unsigned p = 31 + lg;
    f.mul = static_cast<unsigned>(((1ull << p) + d - 1) / d);
    f.shr = p - 32;
  }
  return f;
}

ItemOrder item_order(int heads, int n_per_head, int group) {
  ItemOrder o;
  o.gk = std::max(1, std::min(group, n_per_head));
  o.n_full = n_per_head / o.gk;
  o.per_group = fast_div(static_cast<unsigned>(heads) * static_cast<unsigned>(o.gk));
  o.by_gk = fast_div(static_cast<unsigned>(o.gk));
  o.by_rem = fast_div(static_cast<unsigned>(std::max(1, n_per_head - o.n_full * o.gk)));
  return o;
}

// Longest CTA of the static boustrophedon deal (TileSched) of `items` items with the given costs.
template <typename WorkOf>
double deal_makespan(long long items, int sms, WorkOf work_of) {
  const int G = static_cast<int>(std::min<long long>(items, sms));
  std::vector<double> load(static_cast<size_t>(G), 0.0);
  for (long long lin = 0; lin < items; ++lin) {
    const long long r = lin / G, pos = lin % G;
    load[static_cast<size_t>((r & 1) ? G - 1 - pos : pos)] += work_of(lin);
  }
  return *std::max_element(load.begin(), load.end());
}

// How many adjacent tile ranks of one head the kernels deal consecutively (see ItemOrder).  Packed calls: 1 (their plan is
// sorted).  Dense non-causal calls: all of them (head-major; the tiles are all alike).  Dense causal calls: 1 while the
// operand the tiles stream (streamed_bytes over all heads) stays L2-resident or the heads are few; otherwise the largest
// of 16, 8, 4, 2 whose replayed deal stays within 1 % of the longest-first one (an item of rank r costs n_per_head - r
// plus item_cost, the kernel's measured per-item overhead in the same unit), so that CTAs running at the same time
// share a head's stream.
// Measured, causal, 128 heads x 8192 x 128: backward 9.97 -> 8.3 ms; 256 heads x 4096 x 128: 5.48 -> 4.4 ms.
int tile_group_of(bool packed, bool causal, int heads, int n_per_head, size_t streamed_bytes, int sms, double item_cost) {
  if (packed) return 1;
  if (!causal) return 1 << 30;
  if (heads < 32 || n_per_head < 2 || streamed_bytes <= (size_t(64) << 20)) return 1;
  const long long items = static_cast<long long>(heads) * n_per_head;
  if (items > (1 << 16)) return 8;   // hundreds of items per CTA: any small group balances
  // the replay costs a fraction of a millisecond of host time: remember the answer for this shape
  static std::mutex memo_mutex;
  static std::map<std::tuple<int, int, int, int>, int> memo;
  const auto key = std::make_tuple(heads, n_per_head, sms, static_cast<int>(item_cost * 100.0));
  {
    std::lock_guard<std::mutex> lock(memo_mutex);
    const auto hit = memo.find(key);
    if (hit != memo.end()) return hit->second;
  }
  auto makespan = [&](int k) {
    const long long per_group = static_cast<long long>(heads) * k;
    const int n_full = n_per_head / k;
    return deal_makespan(items, sms, [&](long long lin) {
      const long long g = lin / per_group, within = lin - g * per_group;
      const int kk = (g < n_full) ? k : (n_per_head - n_full * k);
      const long long rank = g * k + within % kk;
      return static_cast<double>(n_per_head - rank) + item_cost;
    });
  };
  const double base = makespan(1);
  int best = 1;
  for (int k = 16; k >= 2 && best == 1; k /= 2)
    if (k <= n_per_head && makespan(k) <= 1.01 * base) best = k;
  std::lock_guard<std::mutex> lock(memo_mutex);
  if (memo.size() < 4096) memo[key] = best;
  return best;
}

// Causal forward at d = 64: paired query tiles or single tiles with the key range split between the warpgroups?
// Measured on B200 (in units of one key-tile step of a pair): a pair item costs its key tiles + 2.9 per item, a single
// tile 0.855 x half its key tiles + 2.9 per item (the split steady state is faster, the per-item cost is paid twice as
// often), and the kernel time is the longest CTA's sum under the static boustrophedon deal.  This replays the deal; the
// constants reproduce the measured ratio of the two modes within 4 % for 8 to 128 heads and N from 1024 to 32768.
bool fwd_prefers_single_tiles(int BH, int n_qt, int sms) {
  const long long n_pairs = (n_qt + 1) / 2, items_p = BH * n_pairs, items_s = static_cast<long long>(BH) * n_qt;
  if (items_s > (1 << 16)) return false;   // many items per SM: both deals balance, pairs have the lower per-item cost
  static std::mutex memo_mutex;
  static std::map<std::tuple<int, int, int>, bool> memo;
  const auto key = std::make_tuple(BH, n_qt, sms);
  {
    std::lock_guard<std::mutex> lock(memo_mutex);
    const auto hit = memo.find(key);
    if (hit != memo.end()) return hit->second;
  }
  auto longest = [&](long long items, auto work_of) {
    const int G = static_cast<int>(std::min<long long>(items, sms));
    std::vector<double> load(static_cast<size_t>(G), 0.0);
    for (long long lin = 0; lin < items; ++lin) {
      const long long r = lin / G, pos = lin % G;
      load[static_cast<size_t>((r & 1) ? G - 1 - pos : pos)] += work_of(lin);
    }
    return *std::max_element(load.begin(), load.end());
  };
  const double kItem = 2.9, kSplitStep = 0.855;
  const double t_pairs = longest(items_p, [&](long long lin) {
    const long long p = n_pairs - 1 - lin / BH;                       // longest pairs first, as the kernel orders them
    return static_cast<double>(2 * p + std::min<long long>(2, n_qt - 2 * p)) + kItem;
  });
  const double t_single = longest(items_s, [&](long long lin) {
    const long long t = n_qt - 1 - lin / BH;
    return kSplitStep * 0.5 * static_cast<double>(t + 1) + kItem;
  });
  std::lock_guard<std::mutex> lock(memo_mutex);
  if (memo.size() < 4096) memo[key] = t_single < t_pairs;
  return t_single < t_pairs;
}

// Dense call: plan == nullptr, one sequence [0, N) per head.  Packed call: B = 1, N = total tokens, plan = device tile
// list (query order) with n_plan_tiles entries.
int launch_fwd(const void *Q, const void *K, const void *V, void *O, float *LSE, int B, int H, int Hkv, int N, int Nk, int d,
               float softmax_scale, int causal, unsigned fwd_flags, const int4 *plan, int n_plan_tiles, void *stream) {
  if (!Q || !K || !V || !O || !LSE) return GPROJ_ERR_NULL;
  if (fwd_flags & ~GPROJ_FWD_FLAG_FMA_SOFTMAX) return GPROJ_ERR_FLAGS;
  const bool fma = (fwd_flags & GPROJ_FWD_FLAG_FMA_SOFTMAX) != 0;
  if (int rc = check_shape(B, H, N, d)) return rc;
  if (Hkv <= 0 || H % Hkv != 0 || check_shape(B, Hkv, Nk, d) != GPROJ_OK) return GPROJ_ERR_SHAPE;
  const int G = H / Hkv;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || (reinterpret_cast<uintptr_t>(LSE) & 3u))
    return GPROJ_ERR_ALIGN;
  if (!std::isfinite(softmax_scale) || !(softmax_scale > 0.f)) return GPROJ_ERR_SCALE;
  DeviceState *st = nullptr;
  if (int rc = device_state(&st)) return rc;

  const int BH = B * H;
  const int BHkv = B * Hkv;
  CUtensorMap mQ, mK, mV, mO;
  if (!make_map(&mQ, Q, BH, N, d, 128) || !make_map(&mK, K, BHkv, Nk, d, 128) || !make_map(&mV, V, BHkv, Nk, d, 128) ||
      !make_map(&mO, O, BH, N, d, 128))
    return GPROJ_ERR_CUDA;
  const float scale_log2 = static_cast<float>(static_cast<double>(softmax_scale) * 1.4426950408889634);
  // One work item = a pair of query tiles of one head (two softmax warpgroups ping-pong on the tensor core); when
  // that leaves too few items to balance the SMs, items are single tiles.
  const int n_qt = plan ? n_plan_tiles : (N + 127) / 128;
  int tiles_per_item = (!plan && static_cast<long long>(BH) * ((n_qt + 1) / 2) * 2 >= 3LL * st->sm_count) ? 2 : 1;
  if (tiles_per_item == 2 && d == 64 && causal && N == Nk && fwd_prefers_single_tiles(BH, n_qt, st->sm_count)) tiles_per_item = 1;
  const int total_items = BH * ((n_qt + tiles_per_item - 1) / tiles_per_item);
  if (total_items <= 0) return GPROJ_OK;   // nothing but empty sequences
  const ItemOrder fwd_order = item_order(BH, total_items / BH, tile_group_of(plan != nullptr, causal != 0, BH, total_items / BH, 2 * static_cast<size_t>(BHkv) * Nk * d * 2, st->sm_count,
                                                            tiles_per_item == 2 ? 1.45 : 6.8));
  const dim3 grid(static_cast<unsigned>(total_items < st->sm_count ? total_items : st->sm_count));   // persistent
  cudaStream_t s = static_cast<cudaStream_t>(stream);
#define GPROJ_LAUNCH_FWD(DD, CC, FF, MM)                                                                            \
  attn_fwd_kernel<DD, CC, FF, MM><<<grid, FwdCfg<DD>::kThreads, FwdCfg<DD>::kSmemBytes, s>>>(                         \
      mQ, mK, mV, mO, static_cast<__nv_bfloat16 *>(O), plan, LSE, N, Nk, BH, H, G, tiles_per_item, total_items, fwd_order, scale_log2, \
      softmax_scale, st->status_ptr)
#define GPROJ_LAUNCH_FWD_C(DD, FF, MM)                                                                              \
  do { if (causal) GPROJ_LAUNCH_FWD(DD, true, FF, MM); else GPROJ_LAUNCH_FWD(DD, false, FF, MM); } while (0)
#define GPROJ_LAUNCH_FWD_F(DD, MM)                                                                                  \
  do { if (fma) GPROJ_LAUNCH_FWD_C(DD, true, MM); else GPROJ_LAUNCH_FWD_C(DD, false, MM); } while (0)
  // Single tiles: the two softmax warpgroups split the key range of the tile.  Pairs: one tile each, and at d = 128
  // they alternate in the exponential phase (measured to pay there only).
  const bool split = (tiles_per_item == 1), turns = (d == 128) && !split && !fma;
  if (d == 64) { if (split) GPROJ_LAUNCH_FWD_F(64, 2); else GPROJ_LAUNCH_FWD_F(64, 0); }
  else if (split) GPROJ_LAUNCH_FWD_F(128, 2);
  else if (turns) GPROJ_LAUNCH_FWD_C(128, false, 1);
  else GPROJ_LAUNCH_FWD_F(128, 0);
#undef GPROJ_LAUNCH_FWD_F
#undef GPROJ_LAUNCH_FWD_C
#undef GPROJ_LAUNCH_FWD
  if (cudaGetLastError() != cudaSuccess) return GPROJ_ERR_CUDA;
  tl_launch_count = 1;
  return GPROJ_OK;
}

}  // namespace

extern "C" {

size_t gproj_attn_bwd_workspace_bytes(int B, int H, int N, int d) {
  if (check_shape(B, H, N, d) != GPROJ_OK) return 0;
  return stats_bytes(B * H, N, d) + align256(static_cast<size_t>(B) * H * N * static_cast<size_t>(d) * 2);
}

int gproj_attn_bwd(const void *Q, const void *K, const void *V, const void *O, const float *LSE, const void *dO,
                   void *dQ, void *dK, void *dV, int B, int H, int N, int d, float softmax_scale, int causal,
                   void *workspace, size_t workspace_bytes, unsigned flags, void *stream) {
  return gproj_attn_bwd_gqa(Q, K, V, O, LSE, dO, dQ, dK, dV, B, H, H, N, d, softmax_scale, causal, workspace, workspace_bytes,
                            flags, stream);
}

int gproj_attn_bwd_gqa(const void *Q, const void *K, const void *V, const void *O, const float *LSE, const void *dO,
                       void *dQ, void *dK, void *dV, int B, int H, int Hkv, int N, int d, float softmax_scale, int causal,
                       void *workspace, size_t workspace_bytes, unsigned flags, void *stream) {
  return launch_bwd(Q, K, V, O, LSE, dO, dQ, dK, dV, B, H, Hkv, N, N, d, softmax_scale, causal, workspace, workspace_bytes, flags,
                    nullptr, nullptr, 0, 0, (N + 63) / 64, stream);
}

}  // extern "C"

namespace {

// Dense call: plans == nullptr.  Packed call: B = 1, N / Nk = total query / key rows, plan_q / plan_kv = device tile lists
// in the order of the dQ-side and the dK/dV-side kernel, nblk = 64-row statistic blocks per head.
int launch_bwd(const void *Q, const void *K, const void *V, const void *O, const float *LSE, const void *dO,
               void *dQ, void *dK, void *dV, int B, int H, int Hkv, int N, int Nk, int d, float softmax_scale, int causal,
               void *workspace, size_t workspace_bytes, unsigned flags, const int4 *plan_q, const int4 *plan_kv,
               int n_plan_q_tiles, int n_plan_kv_tiles, int nblk, void *stream) {
  if (!Q || !K || !V || !O || !LSE || !dO || !dQ || !dK || !dV) return GPROJ_ERR_NULL;
  if (int rc = check_shape(B, H, N, d)) return rc;
  if (Hkv <= 0 || H % Hkv != 0 || check_shape(B, Hkv, Nk, d) != GPROJ_OK) return GPROJ_ERR_SHAPE;
  const int G = H / Hkv;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(dO) || !aligned16(dQ) ||
      !aligned16(dK) || !aligned16(dV) || (reinterpret_cast<uintptr_t>(LSE) & 3u))
    return GPROJ_ERR_ALIGN;
  if (!std::isfinite(softmax_scale) || !(softmax_scale > 0.f)) return GPROJ_ERR_SCALE;
  if (flags & ~(GPROJ_FLAG_NO_Q_CORRECTION | GPROJ_FLAG_NO_K_CORRECTION | GPROJ_FLAG_ONLY_DQ_PASS | GPROJ_FLAG_ONLY_DKV_PASS))
    return GPROJ_ERR_FLAGS;
  const bool run_dq = !(flags & GPROJ_FLAG_ONLY_DKV_PASS);
  bool run_dkv = !(flags & GPROJ_FLAG_ONLY_DQ_PASS);
  if (!run_dq && !run_dkv) return GPROJ_ERR_FLAGS;
  const size_t stats_sz = stats_blocks_bytes(static_cast<size_t>(B) * H * nblk, d);
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
      workspace_bytes < stats_sz + align256(static_cast<size_t>(B) * H * N * static_cast<size_t>(d) * 2))
    return GPROJ_ERR_WORKSPACE;
  DeviceState *st = nullptr;
  if (int rc = device_state(&st)) return rc;

  const int BH = B * H, BHkv = B * Hkv;
  float *stats = static_cast<float *>(workspace);   // per 64-row block: the row-constant tile (see stats_blocks_bytes)
  __nv_bfloat16 *Zneg = reinterpret_cast<__nv_bfloat16 *>(static_cast<uint8_t *>(workspace) + stats_sz);

  CUtensorMap mQ128, mdO128, mK64, mV64, mK128, mV128, mQ64, mdO64, mZ64, mdQst, mZst, mdKst, mdVst;
  bool ok = make_map(&mQ128, Q, BH, N, d, 128) && make_map(&mdO128, dO, BH, N, d, 128) && make_map(&mK64, K, BHkv, Nk, d, 64) &&
            make_map(&mV64, V, BHkv, Nk, d, 64) && make_map(&mK128, K, BHkv, Nk, d, 128) && make_map(&mV128, V, BHkv, Nk, d, 128) &&
            make_map(&mQ64, Q, BH, N, d, 64) && make_map(&mdO64, dO, BH, N, d, 64) && make_map(&mZ64, Zneg, BH, N, d, 64) &&
            make_map(&mdQst, dQ, BH, N, d, 128) && make_map(&mZst, Zneg, BH, N, d, 128) && make_map(&mdKst, dK, BHkv, Nk, d, 128) &&
            make_map(&mdVst, dV, BHkv, Nk, d, 128);
  if (!ok) return GPROJ_ERR_CUDA;

  const float scale_log2 = static_cast<float>(static_cast<double>(softmax_scale) * 1.4426950408889634);
  const int n_qt = plan_q ? n_plan_q_tiles : (N + 127) / 128, n_kt = plan_q ? n_plan_kv_tiles : (Nk + 127) / 128;
  const int total_tiles = BH * n_qt, total_kv_tiles = BHkv * n_kt;
  if (total_tiles <= 0) return GPROJ_OK;   // nothing but empty sequences
  if (total_kv_tiles <= 0) run_dkv = false;   // packed call in which no sequence has both queries and keys
  const ItemOrder group_q = item_order(BH, n_qt, tile_group_of(plan_q != nullptr, causal != 0, BH, n_qt, 2 * static_cast<size_t>(BHkv) * Nk * d * 2, st->sm_count, 3.25));    // streams K, V
  const ItemOrder group_kv = item_order(BHkv, std::max(n_kt, 1), tile_group_of(plan_q != nullptr, causal != 0, BHkv, n_kt, 3 * static_cast<size_t>(BH) * N * d * 2, st->sm_count, 2.3));   // streams Q, dO, Z
  const dim3 grid(static_cast<unsigned>(total_tiles < st->sm_count ? total_tiles : st->sm_count));   // persistent: one CTA per SM
  const dim3 grid_kv(static_cast<unsigned>(total_kv_tiles < st->sm_count ? total_kv_tiles : st->sm_count));
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const __nv_bfloat16 *Ob = static_cast<const __nv_bfloat16 *>(O), *dOb = static_cast<const __nv_bfloat16 *>(dO);
#define GPROJ_LAUNCH_BWD(DD, CC)                                                                                        \
  do {                                                                                                                  \
    if (run_dq)                                                                                                         \
      bwd_dq_kernel<DD, CC><<<grid, BwdCfg<DD>::kThreads, BwdCfg<DD>::kDqSmemBytes, s>>>(                               \
          mQ128, mdO128, mK64, mV64, mdQst, mZst, Ob, dOb, LSE, stats, static_cast<__nv_bfloat16 *>(dQ), Zneg, plan_q, nblk,   \
          N, Nk, BH, H, G, total_tiles, group_q, scale_log2, softmax_scale,                                           \
          flags,                                                                                                        \
          st->status_ptr);                                                                                              \
    if (run_dkv)                                                                                                        \
      launch_after(bwd_dkv_kernel<DD, CC>, grid_kv, BwdCfg<DD>::kThreads, BwdCfg<DD>::kDkvSmemBytes, s, run_dq,            \
          mK128, mV128, mQ64, mdO64, mZ64, mdKst, mdVst, stats, static_cast<__nv_bfloat16 *>(dK),                        \
          static_cast<__nv_bfloat16 *>(dV), plan_kv, nblk, Nk, N, BHkv, Hkv, G, total_kv_tiles, group_kv, scale_log2, softmax_scale, \
          flags,                                                                                                        \
          st->status_ptr);                                                                                              \
  } while (0)
  // At d = 64 the dK/dV side runs with 128-wide steps (every score product an N = 128 instruction); it streams 128-row
  // boxes, which the stationary-tile maps of the dQ side already are.
#define GPROJ_LAUNCH_BWD_W128(CC)                                                                                       \
  do {                                                                                                                  \
    if (run_dq)                                                                                                         \
      bwd_dq_kernel<64, CC><<<grid, BwdCfg<64>::kThreads, BwdCfg<64>::kDqSmemBytes, s>>>(                                \
          mQ128, mdO128, mK64, mV64, mdQst, mZst, Ob, dOb, LSE, stats, static_cast<__nv_bfloat16 *>(dQ), Zneg, plan_q,    \
          nblk, N, Nk, BH, H, G, total_tiles, group_q, scale_log2, softmax_scale, flags, st->status_ptr);                 \
    if (run_dkv)                                                                                                        \
      launch_after(bwd_dkv_w128_kernel<CC>, grid_kv, BwdW128::kThreads, BwdW128::kDkvSmemBytes, s, run_dq,               \
          mK128, mV128, mQ128, mdO128, mZst, mdKst, mdVst, stats, static_cast<__nv_bfloat16 *>(dK),                       \
          static_cast<__nv_bfloat16 *>(dV), plan_kv, nblk, Nk, N, BHkv, Hkv, G, total_kv_tiles, group_kv, scale_log2, softmax_scale,\
          flags, st->status_ptr);                                                                                       \
  } while (0)
  if (d == 64) { if (causal) GPROJ_LAUNCH_BWD_W128(true); else GPROJ_LAUNCH_BWD_W128(false); }
  else         { if (causal) GPROJ_LAUNCH_BWD(128, true); else GPROJ_LAUNCH_BWD(128, false); }
#undef GPROJ_LAUNCH_BWD_W128
#undef GPROJ_LAUNCH_BWD
  if (cudaGetLastError() != cudaSuccess) return GPROJ_ERR_CUDA;
  tl_launch_count = (run_dq ? 1 : 0) + (run_dkv ? 1 : 0);
  return GPROJ_OK;
}

}  // namespace

extern "C" {

// ---- unequal query and key lengths ------------------------------------------------------------------
int gproj_attn_fwd_rect(const void *Q, const void *K, const void *V, void *O, float *LSE, int B, int H, int Hkv, int Nq,
                        int Nk, int d, float softmax_scale, int causal, unsigned fwd_flags, void *stream) {
  return launch_fwd(Q, K, V, O, LSE, B, H, Hkv, Nq, Nk, d, softmax_scale, causal, fwd_flags, nullptr, 0, stream);
}

int gproj_attn_bwd_rect(const void *Q, const void *K, const void *V, const void *O, const float *LSE, const void *dO,
                        void *dQ, void *dK, void *dV, int B, int H, int Hkv, int Nq, int Nk, int d, float softmax_scale,
                        int causal, void *workspace, size_t workspace_bytes, unsigned flags, void *stream) {
  return launch_bwd(Q, K, V, O, LSE, dO, dQ, dK, dV, B, H, Hkv, Nq, Nk, d, softmax_scale, causal, workspace, workspace_bytes,
                    flags, nullptr, nullptr, 0, 0, (Nq + 63) / 64, stream);
}

// ---- packed (variable-length) sequences ------------------------------------------------------------
}  // extern "C"

namespace {

// total_q / total_k: rows per head of the query-side / key-side tensors; q_tiles: query tiles of sequences with queries;
// kv_tiles: key tiles of sequences with both queries and keys; nblk: 64-row statistic blocks of the queries.
struct PackedShape { int total_q, total_k, q_tiles, kv_tiles, nblk; };

// cu_q, cu_k: num_seqs + 1 non-decreasing row offsets each, the first one 0 (cu_k == cu_q: equal lengths).  Sequences
// without queries, without keys or without both are allowed.
bool packed_shape(const int *cu_q, const int *cu_k, int num_seqs, PackedShape *out) {
  if (!cu_q || !cu_k || num_seqs <= 0 || cu_q[0] != 0 || cu_k[0] != 0) return false;
  long long q_tiles = 0, kv_tiles = 0, blocks = 0;
  for (int s = 0; s < num_seqs; ++s) {
    const long long lq = static_cast<long long>(cu_q[s + 1]) - cu_q[s], lk = static_cast<long long>(cu_k[s + 1]) - cu_k[s];
    if (lq < 0 || lk < 0) return false;
    q_tiles += (lq + 127) / 128;
    if (lq > 0) kv_tiles += (lk + 127) / 128;
    blocks += (lq + 63) / 64;
  }
  if (cu_q[num_seqs] <= 0 || cu_k[num_seqs] <= 0 || q_tiles >= (1LL << 24) || kv_tiles >= (1LL << 24)) return false;
  out->total_q = cu_q[num_seqs];
  out->total_k = cu_k[num_seqs];
  out->q_tiles = static_cast<int>(q_tiles);
  out->kv_tiles = static_cast<int>(kv_tiles);
  out->nblk = static_cast<int>(blocks);
  return true;
}

size_t plan_bytes_of(const PackedShape &ps) { return 2 * (static_cast<size_t>(ps.q_tiles) + ps.kv_tiles) * sizeof(int4); }

// Tile list of a packing: the query tiles in the order the query-stationary kernels deal them, then the key tiles in the
// order of the key-stationary kernel; two int4 per tile, {row0, seq0, seq_end, first statistics block of the sequence's
// queries} and {other operand's seq0, seq_end, 0, 0}.
int build_plan(const int *cu_q, const int *cu_k, int num_seqs, int causal, void *plan_host, size_t plan_bytes) {
  PackedShape ps;
  if (!packed_shape(cu_q, cu_k, num_seqs, &ps)) return GPROJ_ERR_SHAPE;
  if (!plan_host) return GPROJ_ERR_NULL;
  if (plan_bytes < plan_bytes_of(ps)) return GPROJ_ERR_WORKSPACE;
  struct Entry { int4 e, o; long long work; };
  std::vector<Entry> vq, vk;
  vq.reserve(static_cast<size_t>(ps.q_tiles));
  vk.reserve(static_cast<size_t>(ps.kv_tiles));
  int blk0 = 0;
  for (int s = 0; s < num_seqs; ++s) {
    const int q0 = cu_q[s], q1 = cu_q[s + 1], k0 = cu_k[s], k1 = cu_k[s + 1], lq = q1 - q0, lk = k1 - k0;
    const long long off = static_cast<long long>(lk) - lq;   // causal: query i sees the keys j <= i + off
    for (int t = 0; t * 128 < lq; ++t) {
      const long long last_row = std::min<long long>((t + 1) * 128LL, lq) - 1;
      const long long keys = causal ? std::max<long long>(0, std::min<long long>(lk, last_row + 1 + off)) : lk;
      vq.push_back(Entry{make_int4(q0 + 128 * t, q0, q1, blk0), make_int4(k0, k1, 0, 0), keys});
    }
    for (int t = 0; lq > 0 && t * 128 < lk; ++t) {
      const long long first_q = causal ? std::max<long long>(0, 128LL * t - off) : 0;
      vk.push_back(Entry{make_int4(k0 + 128 * t, k0, k1, blk0), make_int4(q0, q1, 0, 0), std::max<long long>(0, lq - first_q)});
    }
    blk0 += (lq + 63) / 64;
  }
  // the persistent kernels deal tiles in this order: longest first (stable, so equal tiles keep their memory order)
  auto by_work = [](const Entry &a, const Entry &b) { return a.work > b.work; };
  std::stable_sort(vq.begin(), vq.end(), by_work);
  std::stable_sort(vk.begin(), vk.end(), by_work);
  int4 *out = static_cast<int4 *>(plan_host);
  for (const Entry &en : vq) { *out++ = en.e; *out++ = en.o; }
  for (const Entry &en : vk) { *out++ = en.e; *out++ = en.o; }
  return GPROJ_OK;
}

int fwd_packed(const void *Q, const void *K, const void *V, void *O, float *LSE, const int *cu_q, const int *cu_k, int num_seqs,
               const void *plan_device, int H, int Hkv, int d, float softmax_scale, int causal, unsigned fwd_flags, void *stream) {
  PackedShape ps;
  if (!packed_shape(cu_q, cu_k, num_seqs, &ps)) return GPROJ_ERR_SHAPE;
  if (!plan_device) return GPROJ_ERR_NULL;
  if (reinterpret_cast<uintptr_t>(plan_device) & 15u) return GPROJ_ERR_ALIGN;
  return launch_fwd(Q, K, V, O, LSE, 1, H, Hkv, ps.total_q, ps.total_k, d, softmax_scale, causal, fwd_flags,
                    static_cast<const int4 *>(plan_device), ps.q_tiles, stream);
}

int bwd_packed(const void *Q, const void *K, const void *V, const void *O, const float *LSE, const void *dO, void *dQ, void *dK,
               void *dV, const int *cu_q, const int *cu_k, int num_seqs, const void *plan_device, int H, int Hkv, int d,
               float softmax_scale, int causal, void *workspace, size_t workspace_bytes, unsigned flags, void *stream) {
  PackedShape ps;
  if (!packed_shape(cu_q, cu_k, num_seqs, &ps)) return GPROJ_ERR_SHAPE;
  if (!plan_device) return GPROJ_ERR_NULL;
  if (reinterpret_cast<uintptr_t>(plan_device) & 15u) return GPROJ_ERR_ALIGN;
  const int4 *plan = static_cast<const int4 *>(plan_device);
  const int rc = launch_bwd(Q, K, V, O, LSE, dO, dQ, dK, dV, 1, H, Hkv, ps.total_q, ps.total_k, d, softmax_scale, causal, workspace,
                            workspace_bytes, flags, plan, plan + 2 * static_cast<size_t>(ps.q_tiles), ps.q_tiles, ps.kv_tiles,
                            ps.nblk, stream);
  if (rc != GPROJ_OK || (flags & GPROJ_FLAG_ONLY_DQ_PASS)) return rc;
  // Keys of a sequence without queries are in no tile: their gradient rows are zero.
  const int launches = tl_launch_count;
  const size_t row = static_cast<size_t>(d) * 2, pitch = static_cast<size_t>(ps.total_k) * row;
  for (int s = 0; s < num_seqs; ++s) {
    if (cu_q[s + 1] != cu_q[s] || cu_k[s + 1] == cu_k[s]) continue;
    const size_t at = static_cast<size_t>(cu_k[s]) * row, width = static_cast<size_t>(cu_k[s + 1] - cu_k[s]) * row;
    if (cudaMemset2DAsync(static_cast<uint8_t *>(dK) + at, pitch, 0, width, Hkv, static_cast<cudaStream_t>(stream)) != cudaSuccess ||
        cudaMemset2DAsync(static_cast<uint8_t *>(dV) + at, pitch, 0, width, Hkv, static_cast<cudaStream_t>(stream)) != cudaSuccess) {
      (void)cudaGetLastError();
      return GPROJ_ERR_CUDA;
    }
  }
  tl_launch_count = launches;
  return GPROJ_OK;
}

}  // namespace

extern "C" {

size_t gproj_attn_varlen_plan_bytes(const int *cu_seqlens, int num_seqs) {
  return gproj_attn_varlen_qk_plan_bytes(cu_seqlens, cu_seqlens, num_seqs);
}

int gproj_attn_varlen_plan(const int *cu_seqlens, int num_seqs, int causal, void *plan_host, size_t plan_bytes) {
  return build_plan(cu_seqlens, cu_seqlens, num_seqs, causal, plan_host, plan_bytes);
}

int gproj_attn_fwd_varlen(const void *Q, const void *K, const void *V, void *O, float *LSE, const int *cu_seqlens,
                          int num_seqs, const void *plan_device, int H, int Hkv, int d, float softmax_scale, int causal,
                          unsigned fwd_flags, void *stream) {
  return fwd_packed(Q, K, V, O, LSE, cu_seqlens, cu_seqlens, num_seqs, plan_device, H, Hkv, d, softmax_scale, causal, fwd_flags, stream);
}

size_t gproj_attn_bwd_varlen_workspace_bytes(const int *cu_seqlens, int num_seqs, int H, int d) {
  PackedShape ps;
  if (!packed_shape(cu_seqlens, cu_seqlens, num_seqs, &ps) || check_shape(1, H, ps.total_q, d) != GPROJ_OK) return 0;
  return stats_blocks_bytes(static_cast<size_t>(H) * ps.nblk, d) + align256(static_cast<size_t>(H) * ps.total_q * static_cast<size_t>(d) * 2);
}

int gproj_attn_bwd_varlen(const void *Q, const void *K, const void *V, const void *O, const float *LSE, const void *dO,
                          void *dQ, void *dK, void *dV, const int *cu_seqlens, int num_seqs, const void *plan_device, int H,
                          int Hkv, int d, float softmax_scale, int causal, void *workspace, size_t workspace_bytes,
                          unsigned flags, void *stream) {
  return bwd_packed(Q, K, V, O, LSE, dO, dQ, dK, dV, cu_seqlens, cu_seqlens, num_seqs, plan_device, H, Hkv, d, softmax_scale, causal,
                    workspace, workspace_bytes, flags, stream);
}

// packed sequences whose query and key lengths differ
size_t gproj_attn_varlen_qk_plan_bytes(const int *cu_seqlens_q, const int *cu_seqlens_k, int num_seqs) {
  PackedShape ps;
  if (!packed_shape(cu_seqlens_q, cu_seqlens_k, num_seqs, &ps)) return 0;
  return plan_bytes_of(ps);
}

int gproj_attn_varlen_qk_plan(const int *cu_seqlens_q, const int *cu_seqlens_k, int num_seqs, int causal, void *plan_host,
                              size_t plan_bytes) {
  return build_plan(cu_seqlens_q, cu_seqlens_k, num_seqs, causal, plan_host, plan_bytes);
}

int gproj_attn_fwd_varlen_qk(const void *Q, const void *K, const void *V, void *O, float *LSE, const int *cu_seqlens_q,
                             const int *cu_seqlens_k, int num_seqs, const void *plan_device, int H, int Hkv, int d,
                             float softmax_scale, int causal, unsigned fwd_flags, void *stream) {
  return fwd_packed(Q, K, V, O, LSE, cu_seqlens_q, cu_seqlens_k, num_seqs, plan_device, H, Hkv, d, softmax_scale, causal, fwd_flags,
                    stream);
}

int gproj_attn_bwd_varlen_qk(const void *Q, const void *K, const void *V, const void *O, const float *LSE, const void *dO,
                             void *dQ, void *dK, void *dV, const int *cu_seqlens_q, const int *cu_seqlens_k, int num_seqs,
                             const void *plan_device, int H, int Hkv, int d, float softmax_scale, int causal, void *workspace,
                             size_t workspace_bytes, unsigned flags, void *stream) {
  return bwd_packed(Q, K, V, O, LSE, dO, dQ, dK, dV, cu_seqlens_q, cu_seqlens_k, num_seqs, plan_device, H, Hkv, d, softmax_scale,
                    causal, workspace, workspace_bytes, flags, stream);
}

// ---- forward + backward from host buffers ----------------------------------------------------------
size_t gproj_attn_host_staging_bytes(int B, int H, int Hkv, int N, int d) {
  if (check_shape(B, H, N, d) != GPROJ_OK || Hkv <= 0 || H % Hkv != 0) return 0;
  const size_t q = align256(static_cast<size_t>(B) * H * N * d * 2), kv = align256(static_cast<size_t>(B) * Hkv * N * d * 2);
  return 4 * q + 4 * kv + align256(static_cast<size_t>(B) * H * N * sizeof(float)) + gproj_attn_bwd_workspace_bytes(B, H, N, d);
}

int gproj_attn_fwd_bwd_host(const void *Q, const void *K, const void *V, const void *dO, void *O, float *LSE, void *dQ,
                            void *dK, void *dV, int B, int H, int Hkv, int N, int d, float softmax_scale, int causal,
                            void *staging, size_t staging_bytes, unsigned flags, void *stream) {
  if (!Q || !K || !V || !dO || !dQ || !dK || !dV) return GPROJ_ERR_NULL;
  const size_t need = gproj_attn_host_staging_bytes(B, H, Hkv, N, d);
  if (need == 0) return GPROJ_ERR_SHAPE;
  if (!staging || (reinterpret_cast<uintptr_t>(staging) & 255u) || staging_bytes < need) return GPROJ_ERR_WORKSPACE;
  if (flags & (GPROJ_FLAG_ONLY_DQ_PASS | GPROJ_FLAG_ONLY_DKV_PASS)) return GPROJ_ERR_FLAGS;
  const size_t qb = static_cast<size_t>(B) * H * N * d * 2, kvb = static_cast<size_t>(B) * Hkv * N * d * 2;
  const size_t lb = static_cast<size_t>(B) * H * N * sizeof(float);
  uint8_t *p = static_cast<uint8_t *>(staging);
  auto take = [&](size_t bytes) { uint8_t *r = p; p += align256(bytes); return r; };
  uint8_t *dQin = take(qb), *dOin = take(qb), *dOout = take(qb), *dQout = take(qb);
  uint8_t *dKin = take(kvb), *dVin = take(kvb), *dKout = take(kvb), *dVout = take(kvb);
  uint8_t *dLSE = take(lb);
  uint8_t *ws = p;
  const size_t ws_bytes = gproj_attn_bwd_workspace_bytes(B, H, N, d);
  DeviceState *st = nullptr;
  if (int rc = device_state(&st)) return rc;

  // The (batch, KV head) axis is cut into slabs of whole KV heads with their query heads (contiguous in every tensor), and
  // the slabs are pipelined: copy-in of slab c + 1 and copy-out of slab c - 1 run on two internal streams while the
  // caller's stream computes slab c.  About 2 MiB of Q and at least 128 key tiles per slab: smaller slabs leave the
  // persistent kernels too few tiles (measured: slower than no pipeline at all), larger ones leave the copies exposed.
  const int kv_heads = B * Hkv, G = H / Hkv;
  int slabs = static_cast<int>((qb + (size_t(1) << (kHostSlabLog2 - 1))) >> kHostSlabLog2);
  const long long kv_tiles = static_cast<long long>(kv_heads) * ((N + 127) / 128);
  slabs = std::min(slabs, static_cast<int>(std::min<long long>(kv_tiles / 128, kMaxSlabs)));   // >= 128 key tiles per slab
  slabs = std::max(1, std::min(slabs, kv_heads));
  cudaStream_t s = static_cast<cudaStream_t>(stream);

  std::lock_guard<std::mutex> lock(g_pipe_mutex);   // the internal streams and events are shared by all callers of the device
  if (slabs > 1 && !st->pipe_ready) {
    bool ok = cudaStreamCreateWithFlags(&st->in_stream, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&st->out_stream, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&st->ev_start, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&st->ev_end, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; ok && i < kMaxSlabs; ++i)
      ok = cudaEventCreateWithFlags(&st->ev_in[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&st->ev_done[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) { (void)cudaGetLastError(); return GPROJ_ERR_CUDA; }
    st->pipe_ready = true;
  }
  cudaStream_t s_in = slabs > 1 ? st->in_stream : s, s_out = slabs > 1 ? st->out_stream : s;
  bool ok = true;
  if (slabs > 1) {
    // nothing of this call may start before the work already queued on the caller's stream (it may still use `staging`)
    ok = cudaEventRecord(st->ev_start, s) == cudaSuccess && cudaStreamWaitEvent(s_in, st->ev_start, 0) == cudaSuccess &&
         cudaStreamWaitEvent(s_out, st->ev_start, 0) == cudaSuccess;
  }
  const size_t row_bytes = static_cast<size_t>(N) * d * 2;           // one head of one tensor
  // The last slab is half as large as the others: what stays exposed at the end of the call is that slab's kernels and
  // its copy-out, everything before hides behind the inbound copies.
  auto slab_begin = [&](int c) {
    if (c >= slabs) return kv_heads;
    if (slabs == 1 || kv_heads < 2 * slabs) return static_cast<int>(static_cast<long long>(kv_heads) * c / slabs);
    return static_cast<int>((2LL * kv_heads * c + (2 * slabs - 1) / 2) / (2 * slabs - 1));
  };
  for (int c = 0; ok && c < slabs; ++c) {
    const size_t k0 = slab_begin(c), kn = slab_begin(c + 1) - k0, q0 = k0 * G, qn = kn * G;
    ok = cudaMemcpyAsync(dQin + q0 * row_bytes, static_cast<const uint8_t *>(Q) + q0 * row_bytes, qn * row_bytes, cudaMemcpyHostToDevice, s_in) == cudaSuccess &&
         cudaMemcpyAsync(dKin + k0 * row_bytes, static_cast<const uint8_t *>(K) + k0 * row_bytes, kn * row_bytes, cudaMemcpyHostToDevice, s_in) == cudaSuccess &&
         cudaMemcpyAsync(dVin + k0 * row_bytes, static_cast<const uint8_t *>(V) + k0 * row_bytes, kn * row_bytes, cudaMemcpyHostToDevice, s_in) == cudaSuccess &&
         cudaMemcpyAsync(dOin + q0 * row_bytes, static_cast<const uint8_t *>(dO) + q0 * row_bytes, qn * row_bytes, cudaMemcpyHostToDevice, s_in) == cudaSuccess;
    if (ok && slabs > 1) ok = cudaEventRecord(st->ev_in[c], s_in) == cudaSuccess;
  }
  // After the first copy has been queued, an error return first makes the caller's stream wait for whatever the call
  // put on its internal streams, so that synchronising `stream` tells the caller its host buffers are free again.
  auto fail = [&](int rc) {
    (void)cudaGetLastError();
    if (slabs > 1) {
      if (cudaEventRecord(st->ev_end, s_in) == cudaSuccess) (void)cudaStreamWaitEvent(s, st->ev_end, 0);
      if (cudaEventRecord(st->ev_end, s_out) == cudaSuccess) (void)cudaStreamWaitEvent(s, st->ev_end, 0);
      (void)cudaGetLastError();
    }
    return rc;
  };
  if (!ok) return fail(GPROJ_ERR_CUDA);
  int launches = 0;
  for (int c = 0; c < slabs; ++c) {
    const size_t k0 = slab_begin(c), kn = slab_begin(c + 1) - k0, q0 = k0 * G, qn = kn * G;
    if (slabs > 1 && cudaStreamWaitEvent(s, st->ev_in[c], 0) != cudaSuccess) return fail(GPROJ_ERR_CUDA);
    float *lse_c = reinterpret_cast<float *>(dLSE + q0 * N * sizeof(float));
    // a slab is a problem with batch 1, kn KV heads and qn query heads; the slabs share the backward workspace in turn
    if (int rc = gproj_attn_fwd_gqa(dQin + q0 * row_bytes, dKin + k0 * row_bytes, dVin + k0 * row_bytes, dOout + q0 * row_bytes, lse_c, 1,
                                    static_cast<int>(qn), static_cast<int>(kn), N, d, softmax_scale, causal, stream))
      return fail(rc);
    launches += tl_launch_count;
    if (int rc = gproj_attn_bwd_gqa(dQin + q0 * row_bytes, dKin + k0 * row_bytes, dVin + k0 * row_bytes, dOout + q0 * row_bytes, lse_c,
                                    dOin + q0 * row_bytes, dQout + q0 * row_bytes, dKout + k0 * row_bytes, dVout + k0 * row_bytes, 1,
                                    static_cast<int>(qn), static_cast<int>(kn), N, d, softmax_scale, causal, ws, ws_bytes, flags, stream))
      return fail(rc);
    launches += tl_launch_count;
    ok = slabs == 1 || (cudaEventRecord(st->ev_done[c], s) == cudaSuccess && cudaStreamWaitEvent(s_out, st->ev_done[c], 0) == cudaSuccess);
    ok = ok && cudaMemcpyAsync(static_cast<uint8_t *>(dQ) + q0 * row_bytes, dQout + q0 * row_bytes, qn * row_bytes, cudaMemcpyDeviceToHost, s_out) == cudaSuccess &&
         cudaMemcpyAsync(static_cast<uint8_t *>(dK) + k0 * row_bytes, dKout + k0 * row_bytes, kn * row_bytes, cudaMemcpyDeviceToHost, s_out) == cudaSuccess &&
         cudaMemcpyAsync(static_cast<uint8_t *>(dV) + k0 * row_bytes, dVout + k0 * row_bytes, kn * row_bytes, cudaMemcpyDeviceToHost, s_out) == cudaSuccess;
    if (ok && O) ok = cudaMemcpyAsync(static_cast<uint8_t *>(O) + q0 * row_bytes, dOout + q0 * row_bytes, qn * row_bytes, cudaMemcpyDeviceToHost, s_out) == cudaSuccess;
    if (ok && LSE) ok = cudaMemcpyAsync(LSE + q0 * N, lse_c, qn * N * sizeof(float), cudaMemcpyDeviceToHost, s_out) == cudaSuccess;
    if (!ok) return fail(GPROJ_ERR_CUDA);
  }
  // the caller's stream reaches the end of the call only when the last copy-out has landed
  if (slabs > 1 && !(cudaEventRecord(st->ev_end, s_out) == cudaSuccess && cudaStreamWaitEvent(s, st->ev_end, 0) == cudaSuccess)) {
    (void)cudaGetLastError();
    return GPROJ_ERR_CUDA;
  }
  tl_launch_count = launches;
  return GPROJ_OK;
}

// ---- backward without a caller-supplied workspace -------------------------------------------------
// The scratch is a file-scope device array.  In host code the array's name is only a handle: the
// address a kernel or a TMA descriptor can use must be looked up per device with cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_static_scratch[GPROJ_STATIC_SCRATCH_BYTES];

int gproj_attn_bwd_static_scratch(const void *Q, const void *K, const void *V, const void *O, const float *LSE,
                                  const void *dO, void *dQ, void *dK, void *dV, int B, int H, int N, int d,
                                  float softmax_scale, int causal, unsigned flags, void *stream) {
  static std::mutex scratch_mutex;
  static void *scratch_addr[kMaxDevices] = {};
  const size_t need = gproj_attn_bwd_workspace_bytes(B, H, N, d);
  if (need == 0) return GPROJ_ERR_SHAPE;
  if (need > GPROJ_STATIC_SCRATCH_BYTES) return GPROJ_ERR_WORKSPACE;   // beyond the built-in scratch
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return GPROJ_ERR_CUDA;
  void *scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(scratch_mutex);
    if (!scratch_addr[dev]) {   // once per device, with that device current
      void *p = nullptr;
      if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) { (void)cudaGetLastError(); return GPROJ_ERR_CUDA; }
      scratch_addr[dev] = p;
    }
    scratch = scratch_addr[dev];
  }
  return gproj_attn_bwd(Q, K, V, O, LSE, dO, dQ, dK, dV, B, H, N, d, softmax_scale, causal, scratch,
                        GPROJ_STATIC_SCRATCH_BYTES, flags, stream);
}

int gproj_last_device_status(void *stream, int *detail) {
  if (detail) *detail = 0;
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return GPROJ_ERR_CUDA;
  int code = 0;
  if (cudaMemcpyFromSymbol(&code, g_device_status, sizeof(int)) != cudaSuccess) return GPROJ_ERR_CUDA;
  if (code != 0) {
    const int zero = 0;
    if (cudaMemcpyToSymbol(g_device_status, &zero, sizeof(int)) != cudaSuccess) return GPROJ_ERR_CUDA;
    if (detail) *detail = code;
    return GPROJ_ERR_TIMEOUT;
  }
  return GPROJ_OK;
}

int gproj_selftest_wait_timeout(void *stream) {
  DeviceState *st = nullptr;
  if (int rc = device_state(&st)) return rc;
  wait_timeout_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(st->status_ptr);
  return cudaGetLastError() == cudaSuccess ? GPROJ_OK : GPROJ_ERR_CUDA;
}

const char *gproj_status_string(int status) {
  switch (status) {
    case GPROJ_OK: return "ok";
    case GPROJ_ERR_NULL: return "null pointer argument";
    case GPROJ_ERR_SHAPE: return "unsupported shape (d must be 64 or 128; dimensions positive; H a multiple of Hkv; B*H*N < 2^31, B*H < 2^20, N <= 2^24, fewer than 2^24 tiles)";
    case GPROJ_ERR_ALIGN: return "tensor base address not 16-byte aligned";
    case GPROJ_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case GPROJ_ERR_SCALE: return "softmax_scale must be finite and positive";
    case GPROJ_ERR_ARCH: return "device is not compute capability 10.x (sm_100a)";
    case GPROJ_ERR_CUDA: return "CUDA runtime or driver call failed";
    case GPROJ_ERR_TIMEOUT: return "a bounded in-kernel wait gave up; outputs of that launch are undefined";
    case GPROJ_ERR_FLAGS: return "unknown flag bit";
    default: return "unknown status";
  }
}

int gproj_last_launch_count(void) { return tl_launch_count; }

// ---- fused FP32 attention (comparison arm; plain SIMT arithmetic) ------------------------------------------------------
size_t gproj_fp32_attn_saved_bytes(int B, int H, int N, int d) {
  if (check_shape(B, H, N, d) != GPROJ_OK) return 0;
  const size_t rows = static_cast<size_t>(B) * H * N;
  return (rows * static_cast<size_t>(d) + 4 * rows) * sizeof(float);     // O32, then lse / max / 1 / l per row, then D
}

static int fp32_common(const void *const *ptrs, int n_ptrs, void *saved, size_t saved_bytes, int B, int H, int N, int d, float scale) {
  for (int i = 0; i < n_ptrs; ++i) if (!ptrs[i]) return GPROJ_ERR_NULL;
  if (int rc = check_shape(B, H, N, d)) return rc;
  for (int i = 0; i < n_ptrs; ++i) if (!aligned16(ptrs[i])) return GPROJ_ERR_ALIGN;
  if (!std::isfinite(scale) || !(scale > 0.f)) return GPROJ_ERR_SCALE;
  if (!saved || (reinterpret_cast<uintptr_t>(saved) & 255u) || saved_bytes < gproj_fp32_attn_saved_bytes(B, H, N, d)) return GPROJ_ERR_WORKSPACE;
  return GPROJ_OK;
}

int gproj_fp32_attn_fwd(const void *Q, const void *K, const void *V, void *O, void *saved, size_t saved_bytes,
                        int B, int H, int N, int d, float softmax_scale, int causal, void *stream) {
  const void *ptrs[4] = {Q, K, V, O};
  if (int rc = fp32_common(ptrs, 4, saved, saved_bytes, B, H, N, d, softmax_scale)) return rc;
  DeviceState *st = nullptr;
  if (int rc = device_state(&st)) return rc;
  const size_t rows = static_cast<size_t>(B) * H * N;
  float *O32 = static_cast<float *>(saved), *stats = O32 + rows * d;
  const dim3 grid(static_cast<unsigned>((N + 63) / 64), static_cast<unsigned>(B * H));
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  auto q = static_cast<const __nv_bfloat16 *>(Q); auto k = static_cast<const __nv_bfloat16 *>(K); auto v = static_cast<const __nv_bfloat16 *>(V);
  auto o = static_cast<__nv_bfloat16 *>(O);
#define GPROJ_FP32_FWD(DD, CC)                                                                                     \
  do {                                                                                                             \
    if (cudaFuncSetAttribute(fp32_attn_fwd_kernel<DD, CC>, cudaFuncAttributeMaxDynamicSharedMemorySize, Fp32Cfg<DD>::kFwdSmem) != cudaSuccess) \
      return GPROJ_ERR_CUDA;                                                                                       \
    fp32_attn_fwd_kernel<DD, CC><<<grid, 128, Fp32Cfg<DD>::kFwdSmem, s>>>(q, k, v, o, O32, stats, N, softmax_scale); \
  } while (0)
  if (d == 64) { if (causal) GPROJ_FP32_FWD(64, true); else GPROJ_FP32_FWD(64, false); }
  else         { if (causal) GPROJ_FP32_FWD(128, true); else GPROJ_FP32_FWD(128, false); }
#undef GPROJ_FP32_FWD
  if (cudaGetLastError() != cudaSuccess) return GPROJ_ERR_CUDA;
  tl_launch_count = 1;
  return GPROJ_OK;
}

int gproj_fp32_attn_bwd(const void *Q, const void *K, const void *V, const void *dO, void *saved, size_t saved_bytes,
                        void *dQ, void *dK, void *dV, int B, int H, int N, int d, float softmax_scale, int causal, void *stream) {
  const void *ptrs[7] = {Q, K, V, dO, dQ, dK, dV};
  if (int rc = fp32_common(ptrs, 7, saved, saved_bytes, B, H, N, d, softmax_scale)) return rc;
  DeviceState *st = nullptr;
  if (int rc = device_state(&st)) return rc;
  const size_t rows = static_cast<size_t>(B) * H * N;
  float *O32 = static_cast<float *>(saved), *stats = O32 + rows * d, *Drow = stats + 3 * rows;
  const dim3 grid(static_cast<unsigned>((N + 63) / 64), static_cast<unsigned>(B * H));
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  auto q = static_cast<const __nv_bfloat16 *>(Q); auto k = static_cast<const __nv_bfloat16 *>(K); auto v = static_cast<const __nv_bfloat16 *>(V);
  auto u = static_cast<const __nv_bfloat16 *>(dO);
#define GPROJ_FP32_BWD(DD, CC)                                                                                     \
  do {                                                                                                             \
    if (cudaFuncSetAttribute(fp32_attn_dq_kernel<DD, CC>, cudaFuncAttributeMaxDynamicSharedMemorySize, Fp32Cfg<DD>::kBwdSmem) != cudaSuccess || \
        cudaFuncSetAttribute(fp32_attn_dkv_kernel<DD, CC>, cudaFuncAttributeMaxDynamicSharedMemorySize, Fp32Cfg<DD>::kBwdSmem) != cudaSuccess) \
      return GPROJ_ERR_CUDA;                                                                                       \
    fp32_attn_dq_kernel<DD, CC><<<grid, 128, Fp32Cfg<DD>::kBwdSmem, s>>>(q, k, v, u, O32, stats, Drow, static_cast<__nv_bfloat16 *>(dQ), N, softmax_scale); \
    fp32_attn_dkv_kernel<DD, CC><<<grid, 128, Fp32Cfg<DD>::kBwdSmem, s>>>(q, k, v, u, stats, Drow, static_cast<__nv_bfloat16 *>(dK), static_cast<__nv_bfloat16 *>(dV), N, softmax_scale); \
  } while (0)
  if (d == 64) { if (causal) GPROJ_FP32_BWD(64, true); else GPROJ_FP32_BWD(64, false); }
  else         { if (causal) GPROJ_FP32_BWD(128, true); else GPROJ_FP32_BWD(128, false); }
#undef GPROJ_FP32_BWD
  if (cudaGetLastError() != cudaSuccess) return GPROJ_ERR_CUDA;
  tl_launch_count = 2;
  return GPROJ_OK;
}

// ---- key smoothing (comparison arm of Section 5.1): subtract the per-sequence, per-head mean row -------------------
static int smooth_rows(const void *X, void *Y, int heads, long long rows_total, int d, const int *cu_seqlens, int num_seqs,
                       void *stream) {
  if (!X || !Y) return GPROJ_ERR_NULL;
  if (heads <= 0 || rows_total <= 0 || (d != 64 && d != 128) || heads >= (1 << 20) || rows_total * heads >= (1LL << 31))
    return GPROJ_ERR_SHAPE;
  if (!aligned16(X) || !aligned16(Y)) return GPROJ_ERR_ALIGN;
  if (cu_seqlens) {
    if (num_seqs <= 0 || cu_seqlens[0] != 0 || cu_seqlens[num_seqs] != rows_total) return GPROJ_ERR_SHAPE;
    for (int s = 0; s < num_seqs; ++s)
      if (cu_seqlens[s + 1] < cu_seqlens[s]) return GPROJ_ERR_SHAPE;
  }
  DeviceState *st = nullptr;
  if (int rc = device_state(&st)) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const __nv_bfloat16 *x = static_cast<const __nv_bfloat16 *>(X);
  __nv_bfloat16 *y = static_cast<__nv_bfloat16 *>(Y);
  int launches = 0;
  const int n = cu_seqlens ? num_seqs : 1;
  for (int q = 0; q < n; ++q) {
    const int r0 = cu_seqlens ? cu_seqlens[q] : 0, rows = cu_seqlens ? cu_seqlens[q + 1] - r0 : static_cast<int>(rows_total);
    if (rows == 0) continue;
    if (d == 64) smooth_rows_kernel<64><<<heads, kSmoothThreads, 0, s>>>(x, y, rows_total * d, r0, rows);
    else         smooth_rows_kernel<128><<<heads, kSmoothThreads, 0, s>>>(x, y, rows_total * d, r0, rows);
    ++launches;
  }
  if (cudaGetLastError() != cudaSuccess) return GPROJ_ERR_CUDA;
  tl_launch_count = launches;
  return GPROJ_OK;
}

int gproj_key_smooth(const void *X, void *Y, int B, int Hkv, int N, int d, void *stream) {
  if (B <= 0 || Hkv <= 0 || N <= 0) return GPROJ_ERR_SHAPE;
  if (static_cast<long long>(B) * Hkv >= (1LL << 20)) return GPROJ_ERR_SHAPE;
  return smooth_rows(X, Y, B * Hkv, N, d, nullptr, 0, stream);
}

int gproj_key_smooth_varlen(const void *X, void *Y, const int *cu_seqlens, int num_seqs, int Hkv, int d, void *stream) {
  if (!cu_seqlens) return GPROJ_ERR_NULL;
  if (num_seqs <= 0) return GPROJ_ERR_SHAPE;
  return smooth_rows(X, Y, Hkv, cu_seqlens[num_seqs], d, cu_seqlens, num_seqs, stream);
}

#ifdef GPROJ_TRACE
// Debug builds only: per-tile timeline of the most recent launches (count, then {cta, tile, start ns, end ns} records).
int gproj_debug_read_tile_trace(unsigned long long *out, int max_records, int reset) {
  if (cudaDeviceSynchronize() != cudaSuccess) return GPROJ_ERR_CUDA;
  int n = 0;
  if (cudaMemcpyFromSymbol(&n, gproj::g_tile_trace_count, sizeof(int)) != cudaSuccess) return GPROJ_ERR_CUDA;
  if (n > gproj::kTileTraceMax) n = gproj::kTileTraceMax;
  if (n > max_records) n = max_records;
  if (n > 0 && cudaMemcpyFromSymbol(out, gproj::g_tile_trace, static_cast<size_t>(n) * 4 * sizeof(unsigned long long)) != cudaSuccess)
    return GPROJ_ERR_CUDA;
  if (reset) { const int zero = 0; cudaMemcpyToSymbol(gproj::g_tile_trace_count, &zero, sizeof(int)); }
  return n;
}
int gproj_debug_read_tile_events(unsigned long long *out, int max_records, int reset) {
  if (cudaDeviceSynchronize() != cudaSuccess) return GPROJ_ERR_CUDA;
  int n = 0;
  if (cudaMemcpyFromSymbol(&n, gproj::g_tile_ev_count, sizeof(int)) != cudaSuccess) return GPROJ_ERR_CUDA;
  if (n > gproj::kTileEvMax) n = gproj::kTileEvMax;
  if (n > max_records) n = max_records;
  if (n > 0 && cudaMemcpyFromSymbol(out, gproj::g_tile_ev, static_cast<size_t>(n) * 8 * sizeof(unsigned long long)) != cudaSuccess)
    return GPROJ_ERR_CUDA;
  if (reset) { const int zero = 0; cudaMemcpyToSymbol(gproj::g_tile_ev_count, &zero, sizeof(int)); }
  return n;
}
// Debug builds only: copy the phase stamps of CTA 0 to the host (after a device synchronize).
int gproj_debug_read_trace(long long *out, int count) {
  if (cudaDeviceSynchronize() != cudaSuccess) return GPROJ_ERR_CUDA;
  const int n = gproj::kTraceRoles * gproj::kTraceSteps * gproj::kTraceSlots;
  if (count < n) return GPROJ_ERR_SHAPE;
  return cudaMemcpyFromSymbol(out, gproj::g_trace, n * sizeof(long long)) == cudaSuccess ? n : GPROJ_ERR_CUDA;
}
#endif

}  // extern "C"
