// Device-side building blocks shared by the library's kernels: mbarrier and bulk-copy (TMA) wrappers, bounded
// waits, tcgen05 (tensor memory / 5th-generation MMA) wrappers and the descriptor builders.  Internal: not part
// of the C ABI.  Everything is inline PTX written from the PTX ISA description of sm_100a.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "lq_internal.h"

namespace lqdev {

constexpr long long WAIT_LIMIT_CYCLES = 4000000000ll;   // ~2 s at 2 GHz: no device wait is unbounded

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// ---- mbarrier -----------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_init_fence() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}

// Non-blocking poll: mbarrier.try_wait may suspend the thread for a system-defined time when the phase is still
// open, test_wait never does.
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}

// Bounded wait.  Returns false when the CTA is aborting or the deadline passed (then it raises the abort flag
// and records who gave up in the device status word {code, stage}).
static __device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                            int role, long long limit = WAIT_LIMIT_CYCLES) {
  const long long t0 = clock64();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 0xFF) == 0) {
      if (*abort_flag) return false;
      if (clock64() - t0 > limit) {
        *abort_flag = 1;
        if (atomicCAS(status, 0, (int)LQ_ERR_TIMEOUT) == 0) status[1] = role;
        return false;
      }
    }
  }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                          int role) {
  if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, abort_flag, status, role);
}
// Wait of a role that is idle for a long time: polling at full speed would take issue slots from the roles
// that share its scheduler, so it sleeps between polls.
__device__ __forceinline__ bool mbar_wait_idle(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                               int role) {
  for (int i = 0; i < 64; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    __nanosleep(200);
  }
  return mbar_wait_slow(bar, parity, abort_flag, status, role);
}
// The same wait for a whole warp whose control flow must stay provably uniform.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                               int role) {
  const bool ok = mbar_wait(bar, parity, abort_flag, status, role);
  return __all_sync(0xffffffffu, ok);
}
// Abort path only: gives a transaction that is still in flight on `bar` a bounded time to land, so that no
// copy writes into shared memory after the CTA has left.  Never raises a new error.
__device__ __forceinline__ void mbar_settle(uint32_t bar, uint32_t parity, long long limit = 4000000ll) {
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity) && clock64() - t0 < limit) { }
}

// Programmatic dependent launch: let the next kernel on the stream start its set-up, then wait until the previous
// kernel on the stream has completed and its writes are visible (both are no-ops for a plain launch).
__device__ __forceinline__ void grid_dependency_sync() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.b32 %0, 1, 0, P;\n\t}" : "=r"(pred));
  return pred != 0;
}

// ---- bulk copies (TMA): every copy goes to the issuing CTA only -----------------------------
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar)
               : "memory");
}

// ---- tcgen05 ------------------------------------------------------------------------------
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}

enum { TC_I8 = 0, TC_F8 = 1, TC_F16 = 2 };
template <int KIND>
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  if constexpr (KIND == TC_I8) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
  } else if constexpr (KIND == TC_F8) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
  }
}
// block-scaled MMA: 8-bit-class operands, E8M0 scales (one per row and 32-deep K block) read from tensor memory
__device__ __forceinline__ void tc_mma_mx(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t tsfa,
                                          uint32_t tsfb, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale [%0], %1, %2, %3, [%5], [%6], p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(tsfa), "r"(tsfb)
      : "memory");
}
// 32 rows x 16 bytes of shared memory -> 4 tensor-memory columns, replicated into the four 32-lane quarters
__device__ __forceinline__ void tc_cp_sf(uint32_t taddr, uint64_t sdesc) {
  asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}

// 32 lanes x 16 consecutive 32-bit columns: thread t of the warp receives row (lane base + t).
__device__ __forceinline__ void tmem_ld_32x16(uint32_t taddr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr)
      : "memory");
}
// 16 lanes x 32 consecutive 32-bit columns in the accumulator-fragment layout of mma.sync m16n8: with g = lane / 4 and
// t = lane % 4, registers 4j .. 4j+3 hold (row g, columns 8j + 2t, 8j + 2t + 1) and (row g + 8, the same columns).
__device__ __forceinline__ void tmem_ld_16x256b_x4(uint32_t taddr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.16x256b.x4.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_16x256b_x2(uint32_t taddr, uint32_t (&v)[8]) {
  asm volatile("tcgen05.ld.sync.aligned.16x256b.x2.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
               : "r"(taddr)
               : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 128 bytes, 8-row atoms 1024 bytes
// apart.  Adding (bytes >> 4) steps along K inside the swizzled row.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t smem_addr) {
  const uint32_t lo = ((smem_addr & 0x3FFFFu) >> 4) | (1u << 16);          // start address, LBO = 1 (unused)
  const uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);              // SBO = 1024 B, version 1, SWIZZLE_128B
  return ((uint64_t)hi << 32) | lo;
}
// Shared-memory matrix descriptor without swizzle (K-major, 8-row x 16-byte core matrices stored contiguously).
__device__ __forceinline__ uint64_t make_smem_desc_plain(uint32_t smem_addr, uint32_t lbo, uint32_t sbo) {
  const uint32_t lo = ((smem_addr & 0x3FFFFu) >> 4) | ((lbo >> 4) << 16);
  const uint32_t hi = (sbo >> 4) | (1u << 14);                             // version 1, no swizzle
  return ((uint64_t)hi << 32) | lo;
}

// instruction descriptor: accumulator format, operand formats, N >> 3 at bit 17, M >> 4 at bit 24
__device__ __forceinline__ constexpr uint32_t idesc_shape(int n) { return ((uint32_t)(n >> 3) << 17) | ((uint32_t)(LQ_BM >> 4) << 24); }
constexpr uint32_t IDESC_I8 = (2u << 4) | (1u << 7) | (1u << 10);    // S8 x S8 -> S32
constexpr uint32_t IDESC_F8 = (1u << 4) | (0u << 7) | (0u << 10);    // E4M3 x E4M3 -> F32
constexpr uint32_t IDESC_F16 = (1u << 4) | (0u << 7) | (0u << 10);   // F16 x F16 -> F32
// instruction descriptor of the block-scaled kind: E4M3 x E4M3, E8M0 scales, K-major operands, scale-byte ids
__device__ __forceinline__ constexpr uint32_t idesc_mx2(int n, int a_sf_id, int b_sf_id) {
  return ((uint32_t)b_sf_id << 4) | ((uint32_t)(n >> 3) << 17) | (1u << 23) | ((uint32_t)(LQ_BM >> 4) << 24) | ((uint32_t)a_sf_id << 29);
}
__device__ __forceinline__ constexpr uint32_t idesc_mx(int n, int sf_id) { return idesc_mx2(n, sf_id, sf_id); }

// ---- timeline build (-DLQ_TIMELINE): per-role clock stamps of CTA 0 ----------------------
// A stamp is one 8-byte store by lane 0 of the stamping warp: (event id << 48) | (tag << 40) | (clock64 & 2^40-1),
// appended to that warp's list g_lq_timeline[list][...] (a zero word ends a list).  The regular build compiles
// every LQ_TL_* macro to nothing.
#ifdef LQ_TIMELINE
constexpr int TL_LISTS = 4, TL_CAP = 8192;
enum { TL_PRODUCER = 0, TL_MMA = 1, TL_DRAIN_FIRST = 2, TL_DRAIN_LAST = 3 };
enum {
  EV_P_SLOT_FREE = 1, EV_P_ISSUED = 2,                          // producer: stage free / copies issued
  EV_M_STAGE_FULL = 3, EV_M_ACC_FREE = 4, EV_M_ISSUED = 5,      // MMA warp: operands landed / accumulator free / MMAs + commit issued
  EV_D_OPEN = 6, EV_D_ACC_FULL = 7, EV_D_LOADED = 8, EV_D_DONE = 9,   // drain: starts waiting / accumulator ready / slice in registers / arithmetic done
  EV_D_EPI_BEGIN = 10, EV_D_EPI_END = 11, EV_TILE = 12, EV_D_HALF = 13, EV_D_LD_ISSUED = 14, EV_D_WAITED = 15
};
}  // namespace lqdev
static __device__ unsigned long long g_lq_timeline[lqdev::TL_LISTS][lqdev::TL_CAP];   // one per translation unit
namespace lqdev {
struct TlCursor { int list; unsigned n; };
__device__ __forceinline__ void tl_stamp(TlCursor& c, int ev, int tag) {
  if (c.list >= 0 && c.n + 1 < (unsigned)TL_CAP)
    g_lq_timeline[c.list][c.n++] = ((unsigned long long)ev << 48) | ((unsigned long long)(tag & 0xFF) << 40) |
                                   ((unsigned long long)clock64() & 0xFFFFFFFFFFull);
}
#define LQ_TL_DECL(LIST_EXPR) lqdev::TlCursor tl_cur{(LIST_EXPR), 0u}
#define LQ_TL(EV, TAG) lqdev::tl_stamp(tl_cur, (EV), (TAG))
#else
#define LQ_TL_DECL(LIST_EXPR)
#define LQ_TL(EV, TAG)
#endif

}  // namespace lqdev
