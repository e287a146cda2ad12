// Main W4A4 product of the layer on the 5th-generation tensor cores, with the per-group
// scales, the low-rank branch's up-projection and the bias applied in one epilogue:
//
//   Y[m,n] = sum_g sx[m,g] sw[g,n] (qx_g Wq_g)[m,n] + sT[m] sL2[n] (tq L2q)[m,n] + bias[n]
//
// (Figure 1: residual branch Q(X) Q1(P) plus low-rank branch; Appendix A.3: SINT4 carries one
// scale per block of 64 values on BOTH operands, so every 64-deep partial product needs its
// own rank-1 scale before it may be summed.)
//
// Shape of the kernel (persistent, one CTA per SM, warp-specialised):
//   warp 0      TMA producer: operand tiles (two groups = 128 bytes of K per stage row) and
//               the groups' scale vectors into shared-memory rings
//   warp 1      allocates tensor memory; one lane issues tcgen05.mma: each group of 64 codes
//               is two K=32 MMAs into a FRESH 128x128 accumulator (ring of 4 in tensor memory)
//   warps 4-19  drain: tcgen05.ld one accumulator slice (32 lanes x 32 columns) per warp,
//               acc += P * (sx * sw) in fp32 registers; after the last group, bias, convert, store
// The 4-bit codes ride in 8-bit operands: E4M3 (integers up to 7 are exact, fp32 accumulation
// of |sum| <= 3136 is exact) or plain int8; the branch's 8-bit codes always use kind::i8.
// Every wait is bounded; on expiry the role records LQ_ERR_TIMEOUT in the device status word,
// raises a CTA-wide abort flag and all roles leave through the common teardown.
#include <cuda_fp16.h>

#include "lq_internal.h"

namespace {

constexpr int NSTAGE = 5;                       // operand ring depth (32 KB per stage)
constexpr int NSC = 4;                          // scale ring depth (2 KB per stage)
constexpr int NTBUF = 4;                        // accumulator ring in tensor memory (4 x 128 columns)
constexpr int STAGE_A_BYTES = LQ_BM * LQ_KSTAGE;   // 16 KB
constexpr int STAGE_B_BYTES = LQ_BN * LQ_KSTAGE;   // 16 KB
constexpr int STAGE_BYTES = STAGE_A_BYTES + STAGE_B_BYTES;
constexpr int SC_GROUP_FLOATS = LQ_BM + LQ_BN;     // sx[128] then sw[128]
constexpr int SC_STAGE_BYTES = 2 * SC_GROUP_FLOATS * 4;
constexpr int NUM_DRAIN_WARPS = 16;
constexpr int GEMM_THREADS = (4 + NUM_DRAIN_WARPS) * 32;
constexpr int SMEM_BAR_BYTES = 256;
constexpr int SMEM_BYTES = 1024 /*alignment slack*/ + NSTAGE * STAGE_BYTES + NSC * SC_STAGE_BYTES + SMEM_BAR_BYTES;
constexpr long long WAIT_LIMIT_CYCLES = 4000000000ll;   // ~2 s at 2 GHz

struct GemmParams {
  int M, N, Mpad, Npad, G;
  int n_stages_main;      // ceil(G / 2)
  int branch_mmas;        // 0: no branch; else MMAs of the branch stage (32 bytes of r each)
  int branch_f16;         // branch operands are halves (kind::f16) instead of int8 (kind::i8)
  int tiles_m, tiles_n;
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
                                            int role) {
  const long long t0 = clock64();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 0xFF) == 0) {
      if (*abort_flag) return false;
      if (clock64() - t0 > WAIT_LIMIT_CYCLES) {
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

// 32 lanes x 32 consecutive 32-bit columns: thread t of the warp receives row (lane base + t).
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
        "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
        "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 128 bytes,
// 8-row atoms 1024 bytes apart.  byte_off steps along K inside the swizzled row (32-byte units).
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t smem_addr) {
  const uint32_t lo = ((smem_addr & 0x3FFFFu) >> 4) | (1u << 16);          // start address, LBO = 1 (unused)
  const uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);              // SBO = 1024 B, version 1, SWIZZLE_128B
  return ((uint64_t)hi << 32) | lo;
}

constexpr uint32_t idesc_common = ((uint32_t)(LQ_BN >> 3) << 17) | ((uint32_t)(LQ_BM >> 4) << 24);
constexpr uint32_t IDESC_I8 = (2u << 4) | (1u << 7) | (1u << 10) | idesc_common;    // S8 x S8 -> S32
constexpr uint32_t IDESC_F8 = (1u << 4) | (0u << 7) | (0u << 10) | idesc_common;    // E4M3 x E4M3 -> F32
constexpr uint32_t IDESC_F16 = (1u << 4) | (0u << 7) | (0u << 10) | idesc_common;   // F16 x F16 -> F32

template <int MAIN_KIND>
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
  const uint32_t sm_bar = sm_sc + NSC * SC_STAGE_BYTES;
  uint8_t* bar_ptr = smem + NSTAGE * STAGE_BYTES + NSC * SC_STAGE_BYTES;
  // barrier map (8 bytes each)
  auto bar_full = [&](int s) { return sm_bar + 8u * (uint32_t)s; };
  auto bar_empty = [&](int s) { return sm_bar + 8u * (uint32_t)(NSTAGE + s); };
  auto bar_sfull = [&](int s) { return sm_bar + 8u * (uint32_t)(2 * NSTAGE + s); };
  auto bar_sempty = [&](int s) { return sm_bar + 8u * (uint32_t)(2 * NSTAGE + NSC + s); };
  auto bar_tfull = [&](int b) { return sm_bar + 8u * (uint32_t)(2 * NSTAGE + 2 * NSC + b); };
  auto bar_tempty = [&](int b) { return sm_bar + 8u * (uint32_t)(2 * NSTAGE + 2 * NSC + NTBUF + b); };
  constexpr int NBAR = 2 * NSTAGE + 2 * NSC + 2 * NTBUF;
  static_assert(NBAR * 8 + 16 <= SMEM_BAR_BYTES, "barrier area too small");
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_ptr + NBAR * 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_ptr + NBAR * 8 + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_tiles = p.tiles_m * p.tiles_n;
  const int stages_per_tile = p.n_stages_main + (p.branch_mmas > 0 ? 1 : 0);

  if (threadIdx.x == 0) {
    for (int s = 0; s < NSTAGE; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_empty(s), 1); }
    for (int s = 0; s < NSC; ++s) { mbar_init(bar_sfull(s), 1); mbar_init(bar_sempty(s), NUM_DRAIN_WARPS); }
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
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        const int m0 = (tile / p.tiles_n) * LQ_BM, n0 = (tile % p.tiles_n) * LQ_BN;
        for (int s = 0; s < stages_per_tile && ok; ++s, ++it) {
          const int st = it % NSTAGE, sc = it % NSC;
          ok = mbar_wait(bar_empty(st), ((it / NSTAGE) & 1) ^ 1, abort_flag, p.status, LQ_STAGE_PRODUCER);
          if (!ok) break;
          ok = mbar_wait(bar_sempty(sc), ((it / NSC) & 1) ^ 1, abort_flag, p.status, LQ_STAGE_PRODUCER);
          if (!ok) break;
          const uint32_t a_dst = sm_stage + st * STAGE_BYTES, b_dst = a_dst + STAGE_A_BYTES;
          const uint32_t sc_dst = sm_sc + sc * SC_STAGE_BYTES;
          mbar_expect_tx(bar_full(st), STAGE_BYTES);
          if (s < p.n_stages_main) {
            tma_load_2d(a_dst, &tmA, s * LQ_KSTAGE, m0, bar_full(st));
            tma_load_2d(b_dst, &tmB, s * LQ_KSTAGE, n0, bar_full(st));
            mbar_expect_tx(bar_sfull(sc), SC_STAGE_BYTES);
#pragma unroll
            for (int q = 0; q < 2; ++q) {
              const size_t g = (size_t)(2 * s + q);
              bulk_load(sc_dst + q * SC_GROUP_FLOATS * 4, p.sx + g * p.Mpad + m0, LQ_BM * 4, bar_sfull(sc));
              bulk_load(sc_dst + q * SC_GROUP_FLOATS * 4 + LQ_BM * 4, p.sw + g * p.Npad + n0, LQ_BN * 4, bar_sfull(sc));
            }
          } else {
            tma_load_2d(a_dst, &tmT, 0, m0, bar_full(st));
            tma_load_2d(b_dst, &tmL2, 0, n0, bar_full(st));
            mbar_expect_tx(bar_sfull(sc), SC_GROUP_FLOATS * 4);
            bulk_load(sc_dst, p.sT + m0, LQ_BM * 4, bar_sfull(sc));
            bulk_load(sc_dst + LQ_BM * 4, p.sL2 + n0, LQ_BN * 4, bar_sfull(sc));
          }
        }
      }
      if (!ok) {   // let copies in flight land before the CTA's shared memory goes away
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) { }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      uint32_t it = 0, slot = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        for (int s = 0; s < stages_per_tile && ok; ++s, ++it) {
          const int st = it % NSTAGE;
          ok = mbar_wait(bar_full(st), (it / NSTAGE) & 1, abort_flag, p.status, LQ_STAGE_MMA);
          if (!ok) break;
          tc_fence_after();
          const uint32_t a_addr = sm_stage + st * STAGE_BYTES, b_addr = a_addr + STAGE_A_BYTES;
          const uint64_t adesc = make_smem_desc(a_addr), bdesc = make_smem_desc(b_addr);
          const bool is_main = s < p.n_stages_main;
          const int nslots = is_main ? ((2 * s + 1 < p.G) ? 2 : 1) : 1;
          for (int q = 0; q < nslots && ok; ++q, ++slot) {
            const int buf = slot % NTBUF;
            ok = mbar_wait(bar_tempty(buf), ((slot / NTBUF) & 1) ^ 1, abort_flag, p.status, LQ_STAGE_MMA);
            if (!ok) break;
            tc_fence_after();
            const uint32_t d = tmem_base + buf * LQ_BN;
            if (is_main) {
#pragma unroll
              for (int j = 0; j < 2; ++j) {
                const uint64_t off = (uint64_t)((q * 64 + j * 32) >> 4);
                if constexpr (MAIN_KIND == LQ_KIND_I8) tc_mma<0>(d, adesc + off, bdesc + off, IDESC_I8, j);
                else tc_mma<1>(d, adesc + off, bdesc + off, IDESC_F8, j);
              }
            } else {
              for (int j = 0; j < p.branch_mmas; ++j) {
                const uint64_t off = (uint64_t)((j * 32) >> 4);
                if (p.branch_f16) tc_mma<2>(d, adesc + off, bdesc + off, IDESC_F16, j);
                else tc_mma<0>(d, adesc + off, bdesc + off, IDESC_I8, j);
              }
            }
            tc_commit(bar_tfull(buf));
          }
          tc_commit(bar_empty(st));
        }
      }
    }
  } else if (warp >= 4) {
    // ------------------------------------------------------------------ drain + epilogue
    const int quad = warp & 3;               // tensor-memory lanes 32*quad .. 32*quad+31
    const int cg = (warp - 4) >> 2;          // columns 32*cg .. 32*cg+31 of the tile
    uint32_t it = 0, slot = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
      const int m0 = (tile / p.tiles_n) * LQ_BM, n0 = (tile % p.tiles_n) * LQ_BN;
      float acc[32];
#pragma unroll
      for (int c = 0; c < 32; ++c) acc[c] = 0.f;
      for (int s = 0; s < stages_per_tile && ok; ++s, ++it) {
        const int sc = it % NSC;
        ok = mbar_wait(bar_sfull(sc), (it / NSC) & 1, abort_flag, p.status, LQ_STAGE_DRAIN);
        if (!ok) break;
        const bool is_main = s < p.n_stages_main;
        const int nslots = is_main ? ((2 * s + 1 < p.G) ? 2 : 1) : 1;
        const bool is_int = is_main ? (MAIN_KIND == LQ_KIND_I8) : (p.branch_f16 == 0);
        for (int q = 0; q < nslots && ok; ++q, ++slot) {
          const int buf = slot % NTBUF;
          ok = mbar_wait(bar_tfull(buf), (slot / NTBUF) & 1, abort_flag, p.status, LQ_STAGE_DRAIN);
          if (!ok) break;
          tc_fence_after();
          uint32_t v[32];
          tmem_ld_32x32(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * LQ_BN + cg * 32), v);
          tmem_ld_wait();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_tempty(buf));
          const float* scg = sc_ptr + (size_t)sc * (SC_STAGE_BYTES / 4) + q * SC_GROUP_FLOATS;
          const float sxv = scg[quad * 32 + lane];
          const float4* sw4 = reinterpret_cast<const float4*>(scg + LQ_BM + cg * 32);
#pragma unroll
          for (int c4 = 0; c4 < 8; ++c4) {
            const float4 w = sw4[c4];
            const float ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int c = c4 * 4 + e;
              const float pv = is_int ? __int2float_rn((int)v[c]) : __uint_as_float(v[c]);
              acc[c] = fmaf(pv, sxv * ws[e], acc[c]);
            }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_sempty(sc));
      }
      if (!ok) break;
      // epilogue: bias, convert, store this thread's 32 consecutive columns of one row
      const int row = m0 + quad * 32 + lane;
      const int col0 = n0 + cg * 32;
      const float4* b4 = reinterpret_cast<const float4*>(p.bias + col0);
      if (row < p.M) {
        if (p.out_f32) {
          float* yrow = reinterpret_cast<float*>(p.Y) + (size_t)row * p.N + col0;
#pragma unroll
          for (int c4 = 0; c4 < 8; ++c4) {
            if (col0 + c4 * 4 < p.N) {
              const float4 b = __ldg(b4 + c4);
              *reinterpret_cast<float4*>(yrow + c4 * 4) =
                  make_float4(acc[c4 * 4] + b.x, acc[c4 * 4 + 1] + b.y, acc[c4 * 4 + 2] + b.z, acc[c4 * 4 + 3] + b.w);
            }
          }
        } else {
          __half* yrow = reinterpret_cast<__half*>(p.Y) + (size_t)row * p.N + col0;
#pragma unroll
          for (int c8 = 0; c8 < 4; ++c8) {
            if (col0 + c8 * 8 < p.N) {
              const float4 b0 = __ldg(b4 + 2 * c8), b1 = __ldg(b4 + 2 * c8 + 1);
              __half2 h[4];
              h[0] = __floats2half2_rn(acc[c8 * 8 + 0] + b0.x, acc[c8 * 8 + 1] + b0.y);
              h[1] = __floats2half2_rn(acc[c8 * 8 + 2] + b0.z, acc[c8 * 8 + 3] + b0.w);
              h[2] = __floats2half2_rn(acc[c8 * 8 + 4] + b1.x, acc[c8 * 8 + 5] + b1.y);
              h[3] = __floats2half2_rn(acc[c8 * 8 + 6] + b1.z, acc[c8 * 8 + 7] + b1.w);
              *reinterpret_cast<uint4*>(yrow + c8 * 8) = *reinterpret_cast<uint4*>(h);
            }
          }
        }
      }
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

}  // namespace

lq_status lq_gemm_prepare(int device) {
  if (cudaSetDevice(device) != cudaSuccess) return LQ_ERR_CUDA;
  if (cudaFuncSetAttribute(lq_gemm_kernel<LQ_KIND_I8>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess)
    return LQ_ERR_CUDA;
  if (cudaFuncSetAttribute(lq_gemm_kernel<LQ_KIND_E4M3>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess)
    return LQ_ERR_CUDA;
  return LQ_OK;
}

lq_status lq_launch_gemm(const lq_layer* L, const lq_act* A, void* Y, lq_out_dtype dt, cudaStream_t st) {
  if (cudaSetDevice(A->device) != cudaSuccess) return LQ_ERR_CUDA;
  GemmParams p;
  p.M = A->M; p.N = L->N; p.Mpad = A->Mpad; p.Npad = L->Npad; p.G = L->G;
  p.n_stages_main = lq_ceil_div(L->G, 2);
  p.branch_f16 = L->f16_branch ? 1 : 0;
  p.branch_mmas = L->r == 0 ? 0 : (L->f16_branch ? lq_ceil_div(L->r, 16) : lq_ceil_div(L->r, 32));
  p.tiles_m = lq_ceil_div(A->M, LQ_BM);
  p.tiles_n = L->Npad / LQ_BN;
  p.sx = A->d_sx; p.sw = L->d_sw; p.sT = A->d_sT; p.sL2 = L->d_sL2; p.bias = L->d_bias;
  p.Y = Y; p.out_f32 = dt == LQ_OUT_F32 ? 1 : 0;
  p.status = lq_device_status_ptr(A->device);
  if (!p.status) return LQ_ERR_CUDA;
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, A->device) != cudaSuccess) return LQ_ERR_CUDA;
  int ctas = g_lq_gemm_ctas > 0 ? g_lq_gemm_ctas : sms;
  const int num_tiles = p.tiles_m * p.tiles_n;
  if (ctas > num_tiles) ctas = num_tiles;
  if (L->main_kind == LQ_KIND_I8)
    lq_gemm_kernel<LQ_KIND_I8><<<ctas, GEMM_THREADS, SMEM_BYTES, st>>>(A->tmA, L->tmB, A->tmT, L->tmL2, p);
  else
    lq_gemm_kernel<LQ_KIND_E4M3><<<ctas, GEMM_THREADS, SMEM_BYTES, st>>>(A->tmA, L->tmB, A->tmT, L->tmL2, p);
  return cudaGetLastError() == cudaSuccess ? LQ_OK : LQ_ERR_CUDA;
}
