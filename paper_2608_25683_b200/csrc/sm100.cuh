// Thin inline-PTX wrappers for the sm_100a features the kernels use:
// mbarrier, TMA (cp.async.bulk.tensor), tensor memory (tcgen05.alloc/ld/st)
// and the 5th-generation tensor-core MMA (tcgen05.mma) with its shared-memory
// and instruction descriptors.  Everything here is device code.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace psrl {
namespace sm100 {

// ---------------------------------------------------------------- addresses
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---------------------------------------------------------------- mbarrier
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}

// Bounded wait.  Every wait in the kernels goes through here: after
// `kSpinLimit` polls it gives up, records PSRL_ERR_TIMEOUT (= 10) in the
// device status word, raises the CTA-wide abort flag and returns false so the
// caller can unwind to the common teardown (no trap, no endless loop).
constexpr uint32_t kSpinLimit = 1u << 22;
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* s_abort,
                                          int* g_status) {
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    if (mbar_test(bar, parity)) return true;
    if (it > 64) {
      __nanosleep(32);
      if (*s_abort) return false;
    }
  }
  *s_abort = 1;
  if (g_status) atomicExch(g_status, 10);
  return false;
}

// Bounded wait that ignores the abort flag (used only on the path of a warp that has already given up and
// has to learn how far the MMA-issuing warp got before it arrives on a named barrier for it).
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    if (mbar_test(bar, parity)) return true;
    if (it > 64) __nanosleep(64);
  }
  return false;
}

// Bounded wait of a TMA producer thread on a ring stage.  The producer is usually ahead and
// spends most of its time here; it sleeps between polls so that it takes no issue slots from the
// softmax warps of its SM sub-partition.
__device__ __forceinline__ bool mbar_wait_sleepy(uint64_t* bar, uint32_t parity, volatile int* s_abort,
                                                 int* g_status) {
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    if (mbar_test(bar, parity)) return true;
    __nanosleep(128);
    if (it > 64 && *s_abort) return false;
  }
  *s_abort = 1;
  if (g_status) atomicExch(g_status, 10);
  return false;
}

// The same bounded wait for the MMA-issuing thread.  An acquire-ordered
// mbarrier wait stalls that thread for ~100 cycles while MMAs are in flight
// (measured), which starves the tensor cores; the relaxed form does not.  The
// issuing thread never reads the guarded data itself: shared-memory operands
// are written and read through the async proxy (TMA complete_tx happens after
// the data has landed), tensor-memory operands are ordered by the producers'
// tcgen05.wait::st + tcgen05.fence::before_thread_sync before their arrive and
// by the tcgen05.fence::after_thread_sync this thread issues after the wait.
__device__ __forceinline__ bool mbar_wait_relaxed(uint64_t* bar, uint32_t parity, volatile int* s_abort,
                                                  int* g_status) {
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.relaxed.cta.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    if (ok) return true;
    if (it > 1024 && *s_abort) return false;
  }
  *s_abort = 1;
  if (g_status) atomicExch(g_status, 10);
  return false;
}

// Non-blocking test of a phase, relaxed ordering (see mbar_wait_relaxed for why that is enough
// for the MMA-issuing warp).
__device__ __forceinline__ bool mbar_test_relaxed(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.relaxed.cta.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}

// Non-blocking test of three phases in one shared-memory round trip: the three test_wait
// instructions are independent and issue back to back; only the final combination waits for them.
__device__ __forceinline__ bool mbar_test3_relaxed(uint64_t* b0, uint32_t p0, uint64_t* b1, uint32_t p1, uint64_t* b2,
                                                   uint32_t p2) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p, q, r;\n\t"
      "mbarrier.test_wait.parity.relaxed.cta.shared::cta.b64 p, [%1], %2;\n\t"
      "mbarrier.test_wait.parity.relaxed.cta.shared::cta.b64 q, [%3], %4;\n\t"
      "mbarrier.test_wait.parity.relaxed.cta.shared::cta.b64 r, [%5], %6;\n\t"
      "and.pred p, p, q;\n\t"
      "and.pred p, p, r;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(b0)), "r"(p0), "r"(smem_u32(b1)), "r"(p1), "r"(smem_u32(b2)), "r"(p2)
      : "memory");
  return ok != 0;
}

// Bounded wait of the MMA-issuing warp on up to three barriers at once.  A wait costs that warp
// 100-350 cycles even when the phase is already complete (the barrier lives in shared memory,
// whose pipeline the running MMAs keep busy, and the warp competes with the softmax warps for
// issue slots), and the tensor pipe queues only a few MMAs, so every separate wait between two
// groups of MMAs opens a bubble.  Usually all three phases are complete when the warp gets here:
// one combined test (a single round trip) then suffices.  Otherwise the warp blocks on the first
// barrier, the one expected to complete last, with try_wait (suspended by the hardware, no issue
// slots taken from the softmax warps) and tests again.  All lanes take part (warp-uniform result).
__device__ __forceinline__ bool mbar_wait_all3(uint64_t* b0, uint32_t p0, uint64_t* b1, uint32_t p1, uint64_t* b2,
                                               uint32_t p2, volatile int* s_abort, int* g_status) {
  if (__all_sync(0xffffffffu, mbar_test3_relaxed(b0, p0, b1, p1, b2, p2))) return true;
  if (!__all_sync(0xffffffffu, mbar_wait_relaxed(b0, p0, s_abort, g_status))) return false;
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    if (__all_sync(0xffffffffu, mbar_test3_relaxed(b0, p0, b1, p1, b2, p2))) return true;
    if (it > 1024 && *s_abort) return false;
  }
  *s_abort = 1;
  if (g_status) atomicExch(g_status, 10);
  return false;
}

// The same for one barrier.
__device__ __forceinline__ bool mbar_wait_all1(uint64_t* b0, uint32_t p0, volatile int* s_abort, int* g_status) {
  return __all_sync(0xffffffffu, mbar_wait_relaxed(b0, p0, s_abort, g_status));
}

// One lane of a fully active warp (the same lane every time for the same mask).
// Issuing tcgen05 instructions under this predicate, inside warp-uniform control
// flow, measured ~40 % more MMA throughput than a `lane == 0` branch when the
// other warps of the SM are busy.
__device__ __forceinline__ bool elect_one() {
  uint32_t elected;
  asm volatile(
      "{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(elected));
  return elected != 0;
}

// generic-proxy writes to shared memory -> visible to the async proxy (TMA, MMA)
__device__ __forceinline__ void fence_proxy_async() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// ---------------------------------------------------------------- named barriers
// Hand-off from the softmax warps to the MMA-issuing warp through a hardware named barrier: the
// producers arrive (they do not wait), the consumer warp syncs.  A hop costs ~25 cycles against ~150
// (idle SM) to ~300 (MMAs running) for an mbarrier in shared memory.  A named barrier has no phases
// and no timeout, so it is only used where (a) the producers cannot arrive a second time before the
// consumer has synced on the first (their next arrival depends on an MMA that the consumer issues
// after that sync), and (b) every producer performs all its arrivals even after it gave up on a
// wait of its own, so the consumer is never left waiting.  A producer that gave up no longer has
// dependency (a) to pace it, and arrivals that run ahead of the consumer would wrap the barrier's
// count and leave a residue that no later arrival completes; so on that path it stays in step by
// hand: it arrives for step i only once it knows that the consumer has synced on step i-1 - from a
// step counter the consumer publishes (StepBeacon, dK/dV kernel) or from an mbarrier phase that the
// consumer's MMAs of step i-1 complete (forward) - and stops arriving once the consumer has left its
// loop.  Every sync of the consumer therefore gets exactly one arrival per producer thread, in
// bounded time, on every path.
__device__ __forceinline__ void named_arrive(uint32_t id, uint32_t n_threads) {
  asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(n_threads) : "memory");
}
__device__ __forceinline__ void named_sync(uint32_t id, uint32_t n_threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n_threads) : "memory");
}
// Where the consumer of the named barriers (the MMA-issuing warp) is: `at` = the step whose syncs it is
// about to perform or performing (-1 before the first), `left` = 1 once it has left its loop for good.
struct StepBeacon {
  volatile int at;
  volatile int left;
};
// Producer side, only on the path of a warp that gave up on a wait: true once the consumer has reached
// step i (arrive for it now), false if the consumer has left its loop or the bounded wait ran out (stop
// arriving: nobody will sync again).
__device__ __forceinline__ bool beacon_reached(const StepBeacon* b, int i) {
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    if (b->left) return false;
    if (b->at >= i) return true;
    __nanosleep(64);
  }
  return false;
}

// ---------------------------------------------------------------- TMA
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* m) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(m)) : "memory");
}
// 2-D tiled load: box at (x = innermost element, y = row) -> shared memory.
// x * element size must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* m, uint64_t* bar, int x,
                                            int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], "
      "[%2];" ::"r"(smem_u32(smem_dst)),
      "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(x), "r"(y)
      : "memory");
}

// L2 prefetch of one box of a tiled tensor map (no shared-memory destination, no barrier).
__device__ __forceinline__ void tma_prefetch_2d(const CUtensorMap* m, int x, int y) {
  asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(reinterpret_cast<uint64_t>(m)),
               "r"(x), "r"(y)
               : "memory");
}

// ---------------------------------------------------------------- tensor memory
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_result, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)),
               "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// 32 lanes x 32 consecutive 32-bit columns: thread t of the warp gets lane
// (32 * (warp % 4) + t), register i = column (col0 + i).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
      "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
      "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
      "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}

__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t* r) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"r"(taddr), "r"(r[0]),
               "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
               : "memory");
}

// ---------------------------------------------------------------- MMA descriptors
// Shared-memory matrix descriptor, 128-byte swizzle, tiles of rows x 64 bf16
// (one 128-byte row per matrix row), 8-row groups 1024 bytes apart.
//   K-major operand  (rows = M or N, the 64 elements of a row run along K):
//     SBO = 1024 (next 8 rows); LBO unused.  A 16-element K step = +32 bytes.
//   MN-major operand (rows = K, the 64 elements of a row run along M or N):
//     SBO = 1024 (next 8 K rows); LBO = distance to the next 64-wide column
//     block.  A 16-row K step = +2048 bytes.
constexpr uint64_t kDescSw128 = (uint64_t(1) << 46) | (uint64_t(2) << 61);
__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return kDescSw128 | uint64_t((smem_addr & 0x3FFFF) >> 4) | (uint64_t((lbo_bytes >> 4) & 0x3FFF) << 16) |
         (uint64_t((sbo_bytes >> 4) & 0x3FFF) << 32);
}
// Instruction descriptor, kind::f16, bf16 inputs, fp32 accumulate.
__host__ __device__ constexpr uint32_t make_idesc(int M, int N, int a_mn_major, int b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(a_mn_major) << 15) | (uint32_t(b_mn_major) << 16) |
         (uint32_t(N >> 3) << 17) | (uint32_t(M >> 4) << 24);
}

// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The MMA-issuing thread is a single thread: every instruction it spends on
// building 64-bit descriptors delays the tensor cores.  These variants take the
// descriptor as two 32-bit halves: `hi` is a constant per operand kind and `lo`
// is (address >> 4) | (LBO >> 4) << 16, so stepping through a tile is one
// 32-bit add (32 bytes -> +2, 2048 bytes -> +128, 16384 bytes -> +1024).
constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);  // SBO 1024, version 1, 128B swizzle
__device__ __forceinline__ uint32_t desc_lo(uint32_t smem_addr, uint32_t lbo_bytes) {
  return ((smem_addr & 0x3FFFF) >> 4) | ((lbo_bytes >> 4) << 16);
}
__device__ __forceinline__ void mma_ss_lo(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}" ::"r"(d_tmem),
      "r"(a_lo), "r"(b_lo), "r"(kDescHi), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void mma_ts_lo(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\tsetp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "r"(b_lo), "r"(kDescHi), "r"(idesc), "r"(accumulate)
      : "memory");
}

// Arrive on `bar` when every MMA issued so far by this thread has completed.
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}

// Byte offset of element (row, col) in a rows x 64 bf16 tile with the 128-byte
// swizzle (16-byte chunk index XOR row % 8), tile base 1024-byte aligned.
__device__ __forceinline__ uint32_t sw128_offset(int row, int col) {
  return uint32_t(row) * 128u + ((uint32_t(col >> 3) ^ (uint32_t(row) & 7u)) << 4) + (uint32_t(col) & 7u) * 2u;
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Packed fp32 pairs (sm_100 executes two fp32 operations per instruction on a 64-bit register
// pair): the softmax warps are bound by instruction issue, and every slot they free goes to the
// MMA-issuing warp that shares their scheduler.
struct f32x2 {
  uint64_t v;
};
__device__ __forceinline__ f32x2 make_f32x2(float lo, float hi) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r.v) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ f32x2 make_f32x2(uint32_t lo, uint32_t hi) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r.v) : "r"(lo), "r"(hi));
  return r;
}
__device__ __forceinline__ void split_f32x2(f32x2 a, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(a.v));
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
  f32x2 r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r.v) : "l"(a.v), "l"(b.v), "l"(c.v));
  return r;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
  f32x2 r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r.v) : "l"(a.v), "l"(b.v));
  return r;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
  f32x2 r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r.v) : "l"(a.v), "l"(b.v));
  return r;
}

__device__ __forceinline__ f32x2 add2_rm(f32x2 a, f32x2 b) {   // rounded towards minus infinity
  f32x2 r;
  asm("add.rm.f32x2 %0, %1, %2;" : "=l"(r.v) : "l"(a.v), "l"(b.v));
  return r;
}
__device__ __forceinline__ f32x2 sub2(f32x2 a, f32x2 b) {
  f32x2 r;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r.v) : "l"(a.v), "l"(b.v));
  return r;
}

// 2^x for a pair of arguments on the FMA pipes instead of the MUFU (whose 4 results per cycle and
// sub-partition bound the softmax warps): x = n + f with n = floor(x) from an add of 1.5 * 2^23
// rounded down (n sits in the low mantissa bits of the sum), 2^f on [0, 1) by a cubic fitted for the
// smallest maximal relative error (8.6e-5, far below bf16's 2^-9), and n added into the exponent
// field.  Arguments are clamped at -126 (results below 2^-126 come out as ~2^-126 instead of 0:
// both vanish in bf16 products of this kernel's magnitudes); arguments above ~127 are not supported.
__device__ __forceinline__ void ex2_fma_pair(f32x2 x, float& r0, float& r1) {
  float x0, x1;
  split_f32x2(x, x0, x1);
  const f32x2 xc = make_f32x2(fmaxf(x0, -126.f), fmaxf(x1, -126.f));
  const f32x2 magic = make_f32x2(12582912.f, 12582912.f);
  const f32x2 t = add2_rm(xc, magic);
  const f32x2 f = sub2(xc, sub2(t, magic));
  const f32x2 c1 = make_f32x2(0.6951167583465576f, 0.6951167583465576f),
              c2 = make_f32x2(0.22764499485492706f, 0.22764499485492706f),
              c3 = make_f32x2(0.07706703990697861f, 0.07706703990697861f), one = make_f32x2(1.f, 1.f);
  const f32x2 pl = fma2(fma2(fma2(c3, f, c2), f, c1), f, one);
  float p0, p1, t0, t1;
  split_f32x2(pl, p0, p1);
  split_f32x2(t, t0, t1);
  r0 = __int_as_float(__float_as_int(p0) + (__float_as_int(t0) << 23));
  r1 = __int_as_float(__float_as_int(p1) + (__float_as_int(t1) << 23));
}

// max of three in one instruction
__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

}  // namespace sm100
}  // namespace psrl
