// Main W4A4 product of the layer on the 5th-generation tensor cores, with the per-group
// scales, the low-rank branch's up-projection and the bias applied in one epilogue:
//
//   Y[m,n] = sum_g sx[m,g] sw[g,n] (qx_g Wq_g)[m,n] + sT[m] sL2[n] (tq L2q)[m,n] + bias[n]
//
// (Figure 1: residual branch Q(X) Q1(P) plus low-rank branch; Appendix A.3: SINT4 carries one
// scale per block of 64 values on BOTH operands, so every 64-deep partial product needs its
// own rank-1 scale before it may be summed.)
//
// Shape of the kernel (persistent, one CTA per SM, warp-specialised, 18 warps):
//   warp 0      TMA producer: operand tiles (two groups = 128 bytes of K per stage row) and
//               the two groups' scale vectors, all signalled on the stage's "full" barrier
//   warp 1      owns tensor memory; issues tcgen05.mma: each group of 64 codes is two K=32
//               MMAs into a FRESH 128 x 256 accumulator (ring of 2 in tensor memory).  The
//               loop is warp-uniform (operands live in uniform registers) and one elected
//               lane issues; N = 256 keeps the tensor pipe at its full rate per instruction
//   warps 2-17  drain: each warp owns 32 rows x a quarter of the tile's columns; tcgen05.ld one
//               32 x 16 slice at a time, acc += P * (sx * sw) with packed f32x2 arithmetic
//               in fp32 registers; after the last group: bias, convert, stage the warp's
//               rows in shared memory, read them back with lanes along the row and store
//               whole 64/128-byte row segments
// Work is cut in units of 128 x 128 outputs; every CTA takes a contiguous run of units
// (balanced to one unit) and walks it as 128 x 256 tiles, with a 128 x 128 tile where the
// run or the row block ends.
// The 4-bit codes ride in E4M3 operands (integers up to 7 are exact, fp32 accumulation of
// |sum| <= 3136 is exact); the branch's 8-bit codes use kind::i8 (exact int32), the fp16
// reference branch kind::f16.
// Every wait is bounded; on expiry the role records LQ_ERR_TIMEOUT in the device status word,
// raises a CTA-wide abort flag and all roles leave through the common teardown.
#include <cuda_fp16.h>

#include "lq_internal.h"

namespace {

constexpr int UNIT = LQ_BN;                        // 128 output columns
constexpr int NSTAGE = 3;                          // operand ring depth
constexpr int NTBUF = 2;                           // accumulator ring in tensor memory (2 x 256 columns)
constexpr int TCOLS = 256;                         // columns per accumulator
constexpr int STAGE_A_BYTES = LQ_BM * LQ_KSTAGE;   // 16 KB
constexpr int STAGE_B_BYTES = 2 * UNIT * LQ_KSTAGE;   // 32 KB (two 128-row boxes)
constexpr int STAGE_BYTES = STAGE_A_BYTES + STAGE_B_BYTES;
constexpr int SC_GROUP_FLOATS = LQ_BM + 2 * UNIT;  // sx[128] then sw[256]
constexpr int SC_STAGE_BYTES = 2 * SC_GROUP_FLOATS * 4;   // two groups
constexpr int NUM_DRAIN_WARPS = 16;
constexpr int FIRST_DRAIN_WARP = 2;
constexpr int GEMM_THREADS = (FIRST_DRAIN_WARP + NUM_DRAIN_WARPS) * 32;
constexpr int OUT_ROW_BYTES = 128;                 // output bytes staged per row and pass
constexpr int OUT_ROW_STRIDE = OUT_ROW_BYTES + 16; // +16: rows start 4 banks apart, 16-byte stores do not conflict
constexpr int OUT_WARP_BYTES = 32 * OUT_ROW_STRIDE;
constexpr int SMEM_BAR_BYTES = 256;
constexpr int SMEM_BYTES = 1024 /*alignment slack*/ + NSTAGE * STAGE_BYTES + NSTAGE * SC_STAGE_BYTES +
                           NUM_DRAIN_WARPS * OUT_WARP_BYTES + SMEM_BAR_BYTES;
static_assert(SMEM_BYTES <= 232448, "shared memory budget");
constexpr long long WAIT_LIMIT_CYCLES = 4000000000ll;   // ~2 s at 2 GHz

struct GemmParams {
  int M, N, Mpad, Npad, G;
  int n_stages_main;      // ceil(G / 2)
  int branch_mmas;        // 0: no branch; else MMAs of the branch stage (32 bytes of r each)
  int branch_f16;         // branch operands are halves (kind::f16) instead of int8 (kind::i8)
  int tiles_m, units_n;
  const float* sx;        // [Gpad][Mpad]
  const float* sw;        // [Gpad][Npad]
  const float* sT;        // [Mpad]
  const float* sL2;       // [Npad]
  const float* bias;      // [Npad]
  void* Y;
  int out_f32;
  int32_t* status;
};

// ---- PTX wrappers -------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
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

// Bounded wait.  Returns false when the CTA is aborting or the deadline passed (then it
// raises the abort flag and records who gave up).
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
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
// The same wait for a whole warp whose control flow must stay provably uniform (the producer
// and the MMA warp keep their loop state in uniform registers).
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                               int role) {
  const bool ok = mbar_wait(bar, parity, abort_flag, status, role);
  return __all_sync(0xffffffffu, ok);
}

__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.b32 %0, 1, 0, P;\n\t}" : "=r"(pred));
  return pred != 0;
}

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

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

template <int KIND>   // 0: i8, 1: f8f6f4, 2: f16
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  if constexpr (KIND == 0) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
  } else if constexpr (KIND == 1) {
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
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 128 bytes,
// 8-row atoms 1024 bytes apart.  Adding (bytes >> 4) steps along K inside the swizzled row.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t smem_addr) {
  const uint32_t lo = ((smem_addr & 0x3FFFFu) >> 4) | (1u << 16);          // start address, LBO = 1 (unused)
  const uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);              // SBO = 1024 B, version 1, SWIZZLE_128B
  return ((uint64_t)hi << 32) | lo;
}

// instruction descriptor: accumulator format, operand formats, N >> 3 at bit 17, M >> 4 at bit 24
__device__ __forceinline__ constexpr uint32_t idesc_shape(int n) { return ((uint32_t)(n >> 3) << 17) | ((uint32_t)(LQ_BM >> 4) << 24); }
constexpr uint32_t IDESC_I8 = (2u << 4) | (1u << 7) | (1u << 10);    // S8 x S8 -> S32
constexpr uint32_t IDESC_F8 = (1u << 4) | (0u << 7) | (0u << 10);    // E4M3 x E4M3 -> F32
constexpr uint32_t IDESC_F16 = (1u << 4) | (0u << 7) | (0u << 10);   // F16 x F16 -> F32

// One accumulator slice of 32 rows x 16 columns: acc += P * (sx * sw).  INT: the accumulator
// holds int32 (kind::i8); |P| < 2^22, so adding 1.5 * 2^23 in the integer domain and
// subtracting it in fp32 converts exactly without the conversion pipe.
template <bool INT>
__device__ __forceinline__ void drain_chunk(const uint32_t (&v)[16], float2 (&acc)[8], float sxv, const float* sw) {
  const float2 sx2 = make_float2(sxv, sxv);
#pragma unroll
  for (int c4 = 0; c4 < 4; ++c4) {
    const float4 w = *reinterpret_cast<const float4*>(sw + c4 * 4);
    float2 p0, p1;
    if constexpr (INT) {
      p0 = make_float2(__int_as_float((int)v[c4 * 4 + 0] + 0x4B400000) - 12582912.0f,
                       __int_as_float((int)v[c4 * 4 + 1] + 0x4B400000) - 12582912.0f);
      p1 = make_float2(__int_as_float((int)v[c4 * 4 + 2] + 0x4B400000) - 12582912.0f,
                       __int_as_float((int)v[c4 * 4 + 3] + 0x4B400000) - 12582912.0f);
    } else {
      p0 = make_float2(__uint_as_float(v[c4 * 4 + 0]), __uint_as_float(v[c4 * 4 + 1]));
      p1 = make_float2(__uint_as_float(v[c4 * 4 + 2]), __uint_as_float(v[c4 * 4 + 3]));
    }
    const float2 s0 = __fmul2_rn(sx2, make_float2(w.x, w.y));
    const float2 s1 = __fmul2_rn(sx2, make_float2(w.z, w.w));
    acc[c4 * 2 + 0] = __ffma2_rn(p0, s0, acc[c4 * 2 + 0]);
    acc[c4 * 2 + 1] = __ffma2_rn(p1, s1, acc[c4 * 2 + 1]);
  }
}

__global__ void __launch_bounds__(GEMM_THREADS, 1)
lq_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmT, const __grid_constant__ CUtensorMap tmL2,
               const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t sm_stage = base;
  const uint32_t sm_sc = base + NSTAGE * STAGE_BYTES;
  const float* sc_ptr = reinterpret_cast<const float*>(smem + NSTAGE * STAGE_BYTES);
  uint8_t* out_ptr = smem + NSTAGE * STAGE_BYTES + NSTAGE * SC_STAGE_BYTES;
  const uint32_t sm_bar = sm_sc + NSTAGE * SC_STAGE_BYTES + NUM_DRAIN_WARPS * OUT_WARP_BYTES;
  uint8_t* bar_ptr = out_ptr + NUM_DRAIN_WARPS * OUT_WARP_BYTES;
  // barrier map (8 bytes each)
  auto bar_full = [&](int s) { return sm_bar + 8u * (uint32_t)s; };                        // operands + scales landed
  auto bar_empty = [&](int s) { return sm_bar + 8u * (uint32_t)(NSTAGE + s); };           // MMAs of the stage retired
  auto bar_sempty = [&](int s) { return sm_bar + 8u * (uint32_t)(2 * NSTAGE + s); };      // drain done with the scales
  auto bar_tfull = [&](int b) { return sm_bar + 8u * (uint32_t)(3 * NSTAGE + b); };
  auto bar_tempty = [&](int b) { return sm_bar + 8u * (uint32_t)(3 * NSTAGE + NTBUF + b); };
  constexpr int NBAR = 3 * NSTAGE + 2 * NTBUF;
  static_assert(NBAR * 8 + 16 <= SMEM_BAR_BYTES, "barrier area too small");
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_ptr + NBAR * 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_ptr + NBAR * 8 + 8);

  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);   // provably warp-uniform
  const int lane = threadIdx.x & 31;
  const int stages_per_tile = p.n_stages_main + (p.branch_mmas > 0 ? 1 : 0);
  // this CTA's contiguous run of 128 x 128 units, row block major
  const long long units = (long long)p.tiles_m * p.units_n;
  const int u_begin = (int)((units * blockIdx.x) / gridDim.x);
  const int u_end = (int)((units * (blockIdx.x + 1)) / gridDim.x);

  if (threadIdx.x == 0) {
    for (int s = 0; s < NSTAGE; ++s) {
      mbar_init(bar_full(s), 1);
      mbar_init(bar_empty(s), 1);
      mbar_init(bar_sempty(s), NUM_DRAIN_WARPS);
    }
    for (int b = 0; b < NTBUF; ++b) { mbar_init(bar_tfull(b), 1); mbar_init(bar_tempty(b), NUM_DRAIN_WARPS); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = __shfl_sync(0xffffffffu, *tmem_slot, 0);

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    uint32_t it = 0;
    bool ok = true;
    for (int u = u_begin; u < u_end && ok;) {
      const int mb = u / p.units_n, nu = u - mb * p.units_n;
      const int width = (nu + 1 < p.units_n && u + 1 < u_end) ? 2 : 1;
      const int m0 = mb * LQ_BM, n0 = nu * UNIT;
      for (int s = 0; s < stages_per_tile && ok; ++s, ++it) {
        const int st = it % NSTAGE;
        const uint32_t par = ((it / NSTAGE) & 1) ^ 1;
        ok = mbar_wait_warp(bar_empty(st), par, abort_flag, p.status, LQ_STAGE_PRODUCER);
        if (!ok) break;
        ok = mbar_wait_warp(bar_sempty(st), par, abort_flag, p.status, LQ_STAGE_PRODUCER);
        if (!ok) break;
        const uint32_t a_dst = sm_stage + st * STAGE_BYTES, b_dst = a_dst + STAGE_A_BYTES;
        const uint32_t sc_dst = sm_sc + st * SC_STAGE_BYTES;
        const uint32_t full = bar_full(st);
        const bool is_main = s < p.n_stages_main;
        const int ngroups = is_main ? ((2 * s + 1 < p.G) ? 2 : 1) : 1;
        const uint32_t tx = STAGE_A_BYTES + width * (UNIT * LQ_KSTAGE) + ngroups * (LQ_BM + width * UNIT) * 4;
        if (elect_one()) {
          mbar_expect_tx(full, tx);
          if (is_main) {
            tma_load_2d(a_dst, &tmA, s * LQ_KSTAGE, m0, full);
            tma_load_2d(b_dst, &tmB, s * LQ_KSTAGE, n0, full);
            if (width == 2) tma_load_2d(b_dst + UNIT * LQ_KSTAGE, &tmB, s * LQ_KSTAGE, n0 + UNIT, full);
            for (int q = 0; q < ngroups; ++q) {
              const size_t g = (size_t)(2 * s + q);
              bulk_load(sc_dst + q * SC_GROUP_FLOATS * 4, p.sx + g * p.Mpad + m0, LQ_BM * 4, full);
              bulk_load(sc_dst + q * SC_GROUP_FLOATS * 4 + LQ_BM * 4, p.sw + g * p.Npad + n0, width * UNIT * 4, full);
            }
          } else {
            tma_load_2d(a_dst, &tmT, 0, m0, full);
            tma_load_2d(b_dst, &tmL2, 0, n0, full);
            if (width == 2) tma_load_2d(b_dst + UNIT * LQ_KSTAGE, &tmL2, 0, n0 + UNIT, full);
            bulk_load(sc_dst, p.sT + m0, LQ_BM * 4, full);
            bulk_load(sc_dst + LQ_BM * 4, p.sL2 + n0, width * UNIT * 4, full);
          }
        }
        __syncwarp();
      }
      u += width;
    }
    if (!ok) {   // let copies in flight land before the CTA's shared memory goes away
      const long long t0 = clock64();
      while (clock64() - t0 < 2000000ll) { }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    uint32_t it = 0, slot = 0;
    bool ok = true;
    for (int u = u_begin; u < u_end && ok;) {
      const int mb = u / p.units_n, nu = u - mb * p.units_n;
      const int width = (nu + 1 < p.units_n && u + 1 < u_end) ? 2 : 1;
      const uint32_t shape = idesc_shape(width * UNIT);
      for (int s = 0; s < stages_per_tile && ok; ++s, ++it) {
        const int st = it % NSTAGE;
        ok = mbar_wait_warp(bar_full(st), (it / NSTAGE) & 1, abort_flag, p.status, LQ_STAGE_MMA);
        if (!ok) break;
        tc_fence_after();
        const uint32_t a_addr = sm_stage + st * STAGE_BYTES, b_addr = a_addr + STAGE_A_BYTES;
        const uint64_t adesc = make_smem_desc(a_addr), bdesc = make_smem_desc(b_addr);
        const bool is_main = s < p.n_stages_main;
        const int ngroups = is_main ? ((2 * s + 1 < p.G) ? 2 : 1) : 1;
        for (int q = 0; q < ngroups && ok; ++q, ++slot) {
          const int buf = slot % NTBUF;
          ok = mbar_wait_warp(bar_tempty(buf), ((slot / NTBUF) & 1) ^ 1, abort_flag, p.status, LQ_STAGE_MMA);
          if (!ok) break;
          tc_fence_after();
          const uint32_t d = tmem_base + buf * TCOLS;
          if (is_main) {
            const uint64_t off = (uint64_t)((q * 64) >> 4);
            if (elect_one()) {
              tc_mma<1>(d, adesc + off, bdesc + off, IDESC_F8 | shape, 0u);
              tc_mma<1>(d, adesc + off + 2, bdesc + off + 2, IDESC_F8 | shape, 1u);
              tc_commit(bar_tfull(buf));
            }
          } else {
            if (elect_one()) {
              for (int j = 0; j < p.branch_mmas; ++j) {
                const uint64_t off = (uint64_t)((j * 32) >> 4);
                if (p.branch_f16) tc_mma<2>(d, adesc + off, bdesc + off, IDESC_F16 | shape, (uint32_t)j);
                else tc_mma<0>(d, adesc + off, bdesc + off, IDESC_I8 | shape, (uint32_t)j);
              }
              tc_commit(bar_tfull(buf));
            }
          }
          __syncwarp();
        }
        if (elect_one()) tc_commit(bar_empty(st));
        __syncwarp();
      }
      u += width;
    }
  } else {
    // ------------------------------------------------------------------ drain + epilogue
    const int quad = warp & 3;                          // tensor-memory lanes 32*quad .. 32*quad+31
    const int cgi = (warp - FIRST_DRAIN_WARP) >> 2;     // which quarter of the tile's columns
    const uint32_t tlane = tmem_base + ((uint32_t)(quad * 32) << 16);
    uint8_t* out_row = out_ptr + (warp - FIRST_DRAIN_WARP) * OUT_WARP_BYTES + lane * OUT_ROW_STRIDE;
    uint32_t it = 0, slot = 0;
    bool ok = true;
    for (int u = u_begin; u < u_end && ok;) {
      const int mb = u / p.units_n, nu = u - mb * p.units_n;
      const int width = (nu + 1 < p.units_n && u + 1 < u_end) ? 2 : 1;
      const int m0 = mb * LQ_BM, n0 = nu * UNIT;
      const int coff = cgi * width * 32;                // first of this warp's width*32 columns
      float2 acc[4][8];                                 // [16-column chunk][column pair], starts from the bias
#pragma unroll
      for (int a = 0; a < 4; ++a) {
        if (a < 2 * width) {
          const float4* b4 = reinterpret_cast<const float4*>(p.bias + n0 + coff + a * 16);
#pragma unroll
          for (int b = 0; b < 4; ++b) {
            const float4 bv = __ldg(b4 + b);
            acc[a][2 * b] = make_float2(bv.x, bv.y);
            acc[a][2 * b + 1] = make_float2(bv.z, bv.w);
          }
        }
      }
      for (int s = 0; s < stages_per_tile && ok; ++s, ++it) {
        const int st = it % NSTAGE;
        ok = mbar_wait(bar_full(st), (it / NSTAGE) & 1, abort_flag, p.status, LQ_STAGE_DRAIN);
        if (!ok) break;
        const bool is_main = s < p.n_stages_main;
        const int ngroups = is_main ? ((2 * s + 1 < p.G) ? 2 : 1) : 1;
        const bool is_int = !is_main && p.branch_f16 == 0;
        for (int q = 0; q < ngroups && ok; ++q, ++slot) {
          const int buf = slot % NTBUF;
          ok = mbar_wait(bar_tfull(buf), (slot / NTBUF) & 1, abort_flag, p.status, LQ_STAGE_DRAIN);
          if (!ok) break;
          tc_fence_after();
          const float* scg = sc_ptr + (size_t)st * (SC_STAGE_BYTES / 4) + q * SC_GROUP_FLOATS;
          const float sxv = scg[quad * 32 + lane];
          const float* swp = scg + LQ_BM + coff;
          const uint32_t taddr = tlane + (uint32_t)(buf * TCOLS + coff);
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            if (ch < 2 * width) {
              uint32_t v[16];
              tmem_ld_32x16(taddr + ch * 16, v);
              tmem_ld_wait();
              if (ch == 2 * width - 1) {     // the accumulator may be overwritten once every warp has read its part
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_tempty(buf));
              }
              if (is_int) drain_chunk<true>(v, acc[ch], sxv, swp + ch * 16);
              else drain_chunk<false>(v, acc[ch], sxv, swp + ch * 16);
            }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_sempty(st));
      }
      if (!ok) break;
      // epilogue: convert, stage this thread's row segment in the warp's shared-memory rows, read it back
      // with lanes along the row and store whole 64/128-byte row segments
      const int rbase = m0 + quad * 32;
      const int col0 = n0 + coff;
      const int esize = p.out_f32 ? 4 : 2;
      const int cols_per_pass = OUT_ROW_BYTES / esize;                  // 64 halves or 32 floats
      const int npass = (width * 32 + cols_per_pass - 1) / cols_per_pass;
#pragma unroll
      for (int pass = 0; pass < 2; ++pass) {
        if (pass < npass) {
          __syncwarp();                                                 // previous pass has been read back
          if (p.out_f32) {
#pragma unroll
            for (int cc = 0; cc < 2; ++cc) {
              const int ch = pass * 2 + cc;
              if (ch < 2 * width) {
#pragma unroll
                for (int c4 = 0; c4 < 4; ++c4)
                  *reinterpret_cast<float4*>(out_row + cc * 64 + c4 * 16) =
                      make_float4(acc[ch][c4 * 2].x, acc[ch][c4 * 2].y, acc[ch][c4 * 2 + 1].x, acc[ch][c4 * 2 + 1].y);
              }
            }
          } else {
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
              if (ch < 2 * width) {
#pragma unroll
                for (int c8 = 0; c8 < 2; ++c8) {
                  __half2 h[4];
                  h[0] = __floats2half2_rn(acc[ch][c8 * 4 + 0].x, acc[ch][c8 * 4 + 0].y);
                  h[1] = __floats2half2_rn(acc[ch][c8 * 4 + 1].x, acc[ch][c8 * 4 + 1].y);
                  h[2] = __floats2half2_rn(acc[ch][c8 * 4 + 2].x, acc[ch][c8 * 4 + 2].y);
                  h[3] = __floats2half2_rn(acc[ch][c8 * 4 + 3].x, acc[ch][c8 * 4 + 3].y);
                  *reinterpret_cast<uint4*>(out_row + ch * 32 + c8 * 16) = *reinterpret_cast<uint4*>(h);
                }
              }
            }
          }
          __syncwarp();
          int ncols = width * 32 - pass * cols_per_pass;                // columns of this pass
          if (ncols > cols_per_pass) ncols = cols_per_pass;
          const int lpr = ncols * esize / 16;                           // lanes per row: 4 or 8
          const int rpi = 32 / lpr;                                     // rows per instruction
          const int cpl = 16 / esize;                                   // columns per lane
          const int lcol = col0 + pass * cols_per_pass + (lane % lpr) * cpl;
          const uint8_t* wbase = out_ptr + (warp - FIRST_DRAIN_WARP) * OUT_WARP_BYTES + (lane % lpr) * 16;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            if (i * rpi < 32) {
              const int rl = i * rpi + lane / lpr;
              const uint4 val = *reinterpret_cast<const uint4*>(wbase + rl * OUT_ROW_STRIDE);
              if (rbase + rl < p.M && lcol < p.N)
                *reinterpret_cast<uint4*>(reinterpret_cast<uint8_t*>(p.Y) + ((size_t)(rbase + rl) * p.N + lcol) * esize) = val;
            }
          }
        }
      }
      u += width;
    }
  }

  // ---------------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  }
}

// Self-test of the bounded wait: one warp waits on a barrier that nothing ever arrives on.
__global__ void lq_wait_probe_kernel(int32_t* status, long long limit) {
  __shared__ uint64_t barrier_word;
  __shared__ int abort_word;
  const uint32_t bar = smem_u32(&barrier_word);
  if (threadIdx.x == 0) {
    mbar_init(bar, 1);
    abort_word = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  mbar_wait_slow(bar, 0, &abort_word, status, LQ_STAGE_TEARDOWN, limit);
}

}  // namespace

lq_status lq_launch_wait_probe(int device, cudaStream_t st) {
  if (cudaSetDevice(device) != cudaSuccess) return LQ_ERR_CUDA;
  int32_t* status = lq_device_status_ptr(device);
  if (!status) return LQ_ERR_CUDA;
  lq_wait_probe_kernel<<<1, 32, 0, st>>>(status, 200000000ll);   // ~0.1 s
  return lq_note_cuda(cudaGetLastError()) == cudaSuccess ? LQ_OK : LQ_ERR_CUDA;
}

lq_status lq_gemm_prepare(int device) {
  if (cudaSetDevice(device) != cudaSuccess) return LQ_ERR_CUDA;
  if (lq_note_cuda(cudaFuncSetAttribute(lq_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES)) !=
      cudaSuccess)
    return LQ_ERR_CUDA;
  return LQ_OK;
}

lq_status lq_launch_gemm(const lq_layer* L, const lq_act* A, void* Y, lq_out_dtype dt, cudaStream_t st) {
  if (cudaSetDevice(A->device) != cudaSuccess) return LQ_ERR_CUDA;
  if (L->main_kind != LQ_KIND_E4M3) return LQ_ERR_UNSUPPORTED;
  GemmParams p;
  p.M = A->M; p.N = L->N; p.Mpad = A->Mpad; p.Npad = L->Npad; p.G = L->G;
  p.n_stages_main = lq_ceil_div(L->G, 2);
  p.branch_f16 = L->f16_branch ? 1 : 0;
  p.branch_mmas = L->r == 0 ? 0 : (L->f16_branch ? lq_ceil_div(L->r, 16) : lq_ceil_div(L->r, 32));
  p.tiles_m = lq_ceil_div(A->M, LQ_BM);
  p.units_n = L->Npad / UNIT;
  p.sx = A->d_sx; p.sw = L->d_sw; p.sT = A->d_sT; p.sL2 = L->d_sL2; p.bias = L->d_bias;
  p.Y = Y; p.out_f32 = dt == LQ_OUT_F32 ? 1 : 0;
  p.status = lq_device_status_ptr(A->device);
  if (!p.status) return LQ_ERR_CUDA;
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, A->device) != cudaSuccess) return LQ_ERR_CUDA;
  int ctas = g_lq_gemm_ctas > 0 ? g_lq_gemm_ctas : sms;
  const long long units = (long long)p.tiles_m * p.units_n;
  if (ctas > units) ctas = (int)units;
  lq_gemm_kernel<<<ctas, GEMM_THREADS, SMEM_BYTES, st>>>(A->tmA, L->tmB, A->tmT, L->tmL2, p);
  return lq_note_cuda(cudaGetLastError()) == cudaSuccess ? LQ_OK : LQ_ERR_CUDA;
}
