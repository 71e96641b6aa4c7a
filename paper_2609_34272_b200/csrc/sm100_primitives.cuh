// Thin inline-PTX layer for Blackwell (sm_100a): mbarrier, TMA tile loads, TMEM allocation,
// tcgen05 MMA / load / store / commit, and the 64-bit shared-memory / 32-bit instruction
// descriptors the tensor core consumes.  Every wait is bounded: a wait that gives up records
// a code and makes the remaining waits of the CTA fall through, so a kernel always terminates.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace gproj {

// ------------------------------------------------------------------------------------------
// status codes written by device code (mirrors the public header's GPROJ_ERR_TIMEOUT family)
// ------------------------------------------------------------------------------------------
constexpr int kDevOk = 0;
constexpr int kDevTimeout = 1;   // low byte: 1 = a bounded wait gave up; higher bytes: which one

struct AbortState {
  int *global_status;    // device word shared by all CTAs of a launch (0 = fine)
  volatile int *cta_abort;   // shared-memory flag of this CTA
};

// Optional phase stamps (compiled in only with -DGPROJ_TRACE): CTA 0 records clock64() at named points
// of each role's loop into a device array that a debug entry point copies out.
#ifdef GPROJ_TRACE
constexpr int kTraceRoles = 4, kTraceSteps = 96, kTraceSlots = 8;
__device__ long long g_trace[kTraceRoles * kTraceSteps * kTraceSlots];
__device__ __forceinline__ void trace_stamp(int role, int step, int slot) {
  if (blockIdx.x == 0 && step < kTraceSteps) g_trace[(role * kTraceSteps + step) * kTraceSlots + slot] = clock64();
}
// per-tile timeline: {cta, tile, start ns, end ns} for every tile of a persistent launch
constexpr int kTileTraceMax = 16384;
__device__ unsigned long long g_tile_trace[kTileTraceMax * 4];
__device__ int g_tile_trace_count;
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void tile_trace(int tile, unsigned long long t0, unsigned long long t1) {
  const int i = atomicAdd(&g_tile_trace_count, 1);
  if (i < kTileTraceMax) {
    g_tile_trace[4 * i] = blockIdx.x; g_tile_trace[4 * i + 1] = tile; g_tile_trace[4 * i + 2] = t0; g_tile_trace[4 * i + 3] = t1;
  }
}
// richer per-tile record: {kernel << 32 | cta, steps << 32 | tile, ns at tile start, at first step, after last step, at tile end,
// clock64 at tile start, at tile end}
constexpr int kTileEvMax = 8192;
__device__ unsigned long long g_tile_ev[kTileEvMax * 8];
__device__ int g_tile_ev_count;
__device__ __forceinline__ void tile_event(int kernel, int tile, int steps, unsigned long long n0, unsigned long long n1,
                                           unsigned long long n2, unsigned long long n3, long long c0, long long c1) {
  const int i = atomicAdd(&g_tile_ev_count, 1);
  if (i < kTileEvMax) {
    unsigned long long *e = g_tile_ev + 8 * i;
    e[0] = (static_cast<unsigned long long>(kernel) << 32) | blockIdx.x;
    e[1] = (static_cast<unsigned long long>(steps) << 32) | static_cast<unsigned>(tile);
    e[2] = n0; e[3] = n1; e[4] = n2; e[5] = n3; e[6] = c0; e[7] = c1;
  }
}
#else
__device__ __forceinline__ void trace_stamp(int, int, int) {}
#endif

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ uint32_t elect_one_sync() {
  uint32_t pred = 0;
  asm volatile(
      "{\n\t.reg .pred P;\n\t"
      "elect.sync _|P, 0xffffffff;\n\t"
      "selp.b32 %0, 1, 0, P;\n\t}"
      : "=r"(pred));
  return pred;
}

// ------------------------------------------------------------------------------------------
// mbarrier
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred P;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 P, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, P;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}

// Bounded wait.  Gives up after ~kWaitBudgetCycles SM clocks (a fraction of a second), records
// `code` in the launch's status word and raises the CTA's abort flag; once the flag is up every
// later wait of the CTA returns at once, so all roles run to the end of their loops and the CTA
// exits through its normal epilogue (TMEM freed, no thread left behind).
constexpr long long kWaitBudgetCycles = 400LL * 1000 * 1000;

__device__ __forceinline__ void mbar_wait(uint64_t *bar, uint32_t parity, const AbortState &ab, int code) {
  if (mbar_try_wait(bar, parity)) return;
  if (*ab.cta_abort) return;
  long long t0 = clock64();
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 0x3ff) == 0) {
      if (*ab.cta_abort) return;
      if (clock64() - t0 > kWaitBudgetCycles) {
        *ab.cta_abort = 1;
        atomicCAS(ab.global_status, 0, kDevTimeout | (code << 8));
        return;
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// TMA: 2-D tiled load global -> shared, completion on an mbarrier
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap *m) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(m)) : "memory");
}
__device__ __forceinline__ void tma_load_2d(void *smem_dst, const CUtensorMap *m, uint64_t *bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(x), "r"(y)
      : "memory");
}
// 3-D tile [x: columns, y: row within a head, z: head]: rows past the head's extent read as zero and are not written
__device__ __forceinline__ void tma_load_3d(void *smem_dst, const CUtensorMap *m, uint64_t *bar, int x, int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z)
      : "memory");
}
// 1-D bulk copy global -> shared (both addresses 16-byte aligned, size a multiple of 16 bytes)
__device__ __forceinline__ void bulk_load_1d(void *smem_dst, const void *gmem_src, uint32_t bytes, uint64_t *bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(gmem_src)), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
// generic-proxy writes to shared memory -> visible to the async proxy (TMA / tensor core reads)
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
// TMA: 2-D tiled store shared -> global (bulk-group completion).  x must be a multiple of 8 BF16 elements; y >= 0.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *m, const void *smem_src, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(smem_src)), "r"(x), "r"(y)
               : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap *m, const void *smem_src, int x, int y, int z) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
               ::"l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(smem_src)), "r"(x), "r"(y), "r"(z)
               : "memory");
}
__device__ __forceinline__ void bulk_commit_group() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// all committed bulk stores of this thread have finished READING shared memory (it may be reused or released)
__device__ __forceinline__ void bulk_wait_group_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }

// Byte offset of 16-byte chunk `chunk16` (0..7) of row `row` inside a 128-byte-row slab laid out with the
// 128-byte swizzle TMA uses (chunk index XOR row mod 8).  Slab bases are 1024-byte aligned.
__device__ __forceinline__ uint32_t swz128_offset(int row, int chunk16) {
  return static_cast<uint32_t>(row) * 128u + (static_cast<uint32_t>(chunk16 ^ (row & 7)) << 4);
}

// ------------------------------------------------------------------------------------------
// TMEM allocation (one full warp executes these)
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t *smem_result, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// ------------------------------------------------------------------------------------------
// Descriptors
// ------------------------------------------------------------------------------------------
// Shared-memory matrix descriptor, 128-byte swizzle, Blackwell version field = 1.
//   bits [0,14)  start address >> 4        bits [16,30) leading byte offset >> 4
//   bits [32,46) stride byte offset >> 4   bits [46,48) version (1)      bits [61,64) layout (2 = SWIZZLE_128B)
// K-major operand  (contraction index contiguous, rows of 128 B): SBO = 1024 (8 rows), LBO unused (1).
// MN-major operand (non-contraction index contiguous, 64-element = 128 B atoms):
//   SBO = byte stride between groups of 8 contraction rows (1024 when rows are 128 B apart),
//   LBO = byte stride between 64-element atoms along the non-contraction index.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((saddr >> 4) & 0x3fff);
  d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3fff) << 16;
  d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3fff) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}

// The same descriptor split into its two 32-bit words.  The issuing thread builds it once per operand
// tile; moving the start address by a byte offset is then a single 32-bit add on the low word (shared
// memory addresses stay below 2^18, so the 14-bit field cannot carry).  Keeping the per-instruction
// arithmetic this short matters: one thread issues every MMA of the CTA.
struct SmemDesc {
  uint32_t lo, hi;
  __device__ __forceinline__ uint64_t at(uint32_t byte_offset) const {
    return (static_cast<uint64_t>(hi) << 32) | static_cast<uint64_t>(lo + (byte_offset >> 4));
  }
  __device__ __forceinline__ SmemDesc advanced(uint32_t byte_offset) const { return SmemDesc{lo + (byte_offset >> 4), hi}; }
};
__device__ __forceinline__ SmemDesc make_smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  const uint64_t d = smem_desc_sw128(saddr, lbo_bytes, sbo_bytes);
  return SmemDesc{static_cast<uint32_t>(d), static_cast<uint32_t>(d >> 32)};
}
// K-major operand without swizzle: 8-row x 16-byte core matrices of 128 contiguous bytes; LBO = byte stride between the
// two core matrices of a K = 16 slice, SBO = byte stride between groups of eight rows (0: every group reads the same eight
// rows, a matrix whose rows are all equal).
__device__ __forceinline__ SmemDesc make_smem_desc_noswizzle(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  const uint64_t d = smem_desc_sw128(saddr, lbo_bytes, sbo_bytes) & ~(static_cast<uint64_t>(7) << 61);
  return SmemDesc{static_cast<uint32_t>(d), static_cast<uint32_t>(d >> 32)};
}

// Instruction descriptor for kind::f16 with BF16 A/B and FP32 accumulation.
//   bits [4,6) D format (1 = F32)  [7,10) A format (1 = BF16)  [10,13) B format (1 = BF16)
//   bit 15 A major (0 = K, 1 = MN)  bit 16 B major  [17,23) N >> 3  [24,29) M >> 4
__host__ __device__ constexpr uint32_t idesc_bf16_f32(int M, int N, int a_mn_major, int b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(a_mn_major) << 15) |
         (static_cast<uint32_t>(b_mn_major) << 16) | (static_cast<uint32_t>(N >> 3) << 17) |
         (static_cast<uint32_t>(M >> 4) << 24);
}

// ------------------------------------------------------------------------------------------
// tcgen05.mma (single-CTA group), issued by one thread
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// mbarrier arrives once every MMA issued so far by this thread has completed
__device__ __forceinline__ void umma_commit(uint64_t *bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// Called by a whole MMA-issuing warp when its loop is over.  In the normal flow every MMA has been waited for by a
// consumer before the CTA frees TMEM.  If the CTA aborted (a bounded wait gave up and later waits fell through) MMAs
// may still be executing: commit them to a spare barrier and give them a bounded time to finish before TMEM goes.
__device__ __forceinline__ void drain_mmas_if_aborted(uint64_t *spare_bar, const AbortState &ab) {
  if (*ab.cta_abort) {
    if (elect_one_sync()) umma_commit(spare_bar);
    __syncwarp();
    for (int spin = 0; spin < 2000000 && !mbar_try_wait(spare_bar, 0); ++spin) {}
  }
  __syncwarp();
}

// ------------------------------------------------------------------------------------------
// TMEM <-> registers.  Shape 32x32b: lane l of the warp owns TMEM lane (32*(warp%4) + l) and
// receives / supplies one 32-bit word per column.  taddr = base + (lane << 16) + column.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
        "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
        "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t (&r)[8]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
               ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
               : "memory");
}

// Packed FP32x2 arithmetic (sm_100): one issue slot for two IEEE round-to-nearest results.
__device__ __forceinline__ uint64_t f32x2(float lo, float hi) {
  uint64_t v;
  asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "f"(lo), "f"(hi));
  return v;
}
__device__ __forceinline__ uint64_t f32x2_bits(uint32_t lo, uint32_t hi) {
  uint64_t v;
  asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "r"(lo), "r"(hi));
  return v;
}
__device__ __forceinline__ void f32x2_split(uint64_t v, float &lo, float &hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
// three-input maximum (one instruction on sm_100)
// Programmatic dependent launch: a kernel launched with the programmatic-serialisation attribute may start while the
// kernel before it in the stream still runs.  launch_dependents (in the earlier kernel) allows that start once every CTA of
// the earlier kernel has issued it or exited; wait (in the later kernel) returns when the earlier kernel has completed and
// its memory is visible.  Both are no-ops for a kernel launched without the attribute / with nothing before it.
__device__ __forceinline__ void griddep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

// two FP32 -> packed BF16x2, round-to-nearest-even; `lo` lands in bits [0,16)
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t out;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(out) : "f"(hi), "f"(lo));
  return out;
}
__device__ __forceinline__ float bf16_lo_to_f32(uint32_t packed) { return __uint_as_float(packed << 16); }
__device__ __forceinline__ float bf16_hi_to_f32(uint32_t packed) { return __uint_as_float(packed & 0xffff0000u); }

// barrier among a subset of the CTA's warps (id 1..15; id 0 is __syncthreads)
__device__ __forceinline__ void named_bar_sync(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// Grouped-query layout: query head h of batch b (flat index b Hq + h) reads key / value head h / G of the same batch
// (flat index b (Hq / G) + h / G).  G = 1 is ordinary multi-head attention.
__device__ __forceinline__ int kv_head_of(int q_flat, int Hq, int G) { return (q_flat / Hq) * (Hq / G) + (q_flat % Hq) / G; }

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

}  // namespace gproj
