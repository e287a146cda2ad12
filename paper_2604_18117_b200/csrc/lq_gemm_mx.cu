// MXINT4 variant of the layer's main product (Appendix A.3: blocks of 32 values with a power-of-two E8M0 scale;
// Table 2 quantizes the residual branch with it):
//
//   Y[m,n] = sum_b 2^(ex[m,b] + ew[b,n]) (qx_b Wq_b)[m,n] + sT[m] sL2[n] (tq L2q)[m,n] + bias[n]
//
// Here the tensor core applies the scales itself: tcgen05.mma kind::mxf8f6f4.block_scale takes one E8M0 scale
// per operand row and 32-deep K block from tensor memory, so ALL blocks of a tile accumulate into ONE fp32
// accumulator and nothing has to be drained per block.  The 4-bit codes ride in E4M3 operands as in the SINT4
// kernel.  Products q q' 2^(e+e') are exact in fp32; their sum is rounded by the tensor core's fp32 accumulation.
//
// Shape of the kernel (persistent, one CTA per SM, 18 warps):
//   warp 0      TMA producer: per stage 128 bytes of K of A (128 rows) and B (256 rows, one box) plus the stage's scale
//               bytes (512 B per 128 rows: four K blocks, already in the 32 x 16-byte layout tensor memory wants);
//               per tile the vectors sT, sL2 and bias for the drain
//   warp 1      owns tensor memory; per stage: tcgen05.cp of the scale bytes into tensor-memory columns, then four
//               K = 32 block-scaled MMAs (N = 256) into the tile's accumulator; after the last stage the accumulator is
//               handed to the drain - once per tile
//   warps 2-17  drain.  While the tensor core works on the tile they compute the low-rank branch's up-projection
//               U = tq L2q for their part of it with mma.sync (int8 -> int32, exact; 1/36 .. 1/144 of the tile's
//               work, operands read straight from global memory in fragment order), scale it by sT sL2 and add the
//               bias.  When the accumulator arrives they read it with tcgen05.ld in the same fragment layout
//               (16x256b), add, release it, and store: a 4 x 4 exchange inside each quad gives every lane 16
//               contiguous bytes of one row; fp16 rows are staged in shared memory (dense 64-byte rows, conflict-free)
//               and leave with one TMA store per warp and half, which clips ragged edges and does not hold the warp.
// Per tile the drain's work (branch, hand-over, stores) must stay below the tile's main loop, or the tensor core
// waits for the accumulator: hence the batched fragment loads, the scale vectors staged by the producer and the
// asynchronous stores.
// Every wait is bounded as in lq_gemm.cu.
#include <cuda_fp16.h>

#include "lq_internal.h"

namespace {

constexpr int UNIT = LQ_BN;                        // 128 output columns
constexpr int NSTAGE = 3;                          // operand ring depth
constexpr int STAGE_A_BYTES = LQ_BM * LQ_KSTAGE;   // 16 KB
constexpr int STAGE_B_BYTES = 2 * UNIT * LQ_KSTAGE;   // 32 KB (one 256-row box, or one 128-row box for a narrow tile)
constexpr int STAGE_BYTES = STAGE_A_BYTES + STAGE_B_BYTES;
constexpr int SF_BYTES = 512;                      // scale bytes of 128 rows x 4 K blocks
constexpr int STAGE_SF_BYTES = 3 * SF_BYTES;       // SFA, then SFB of both halves
constexpr int SC_FLOATS = LQ_BM + 4 * UNIT;        // per tile: sT[128], sL2[256], bias[256]
constexpr int NUM_DRAIN_WARPS = 16;
constexpr int FIRST_DRAIN_WARP = 2;
constexpr int GEMM_THREADS = (FIRST_DRAIN_WARP + NUM_DRAIN_WARPS) * 32;
constexpr int OUT_UNIT_BYTES = 32 * 64;            // one warp's 32 rows x 32 fp16 columns of one half: a TMA store box
constexpr int OUT_WARP_BYTES = 2 * OUT_UNIT_BYTES; // one buffer per half
constexpr int SMEM_BAR_BYTES = 256;
constexpr int SMEM_BYTES = 1024 /*alignment slack*/ + NSTAGE * STAGE_BYTES + NSTAGE * STAGE_SF_BYTES + 2 * SC_FLOATS * 4 +
                           NUM_DRAIN_WARPS * OUT_WARP_BYTES + SMEM_BAR_BYTES;
static_assert(SMEM_BYTES <= 232448, "shared memory budget");
static_assert(STAGE_BYTES % 1024 == 0, "stages must keep the 1024-byte alignment of the swizzled tiles");
static_assert((NSTAGE * STAGE_SF_BYTES + 2 * SC_FLOATS * 4) % 128 == 0, "store staging must stay 128-byte aligned");
constexpr long long WAIT_LIMIT_CYCLES = 4000000000ll;   // ~2 s at 2 GHz
// tensor-memory columns: accumulator [0, 256), then per stage 4 columns of A scales and 8 of B scales
constexpr int TM_SFA = 256, TM_SFB = TM_SFA + 4 * NSTAGE;

struct MxParams {
  int M, N, Mpad, Npad;
  int k_stages;           // Kpad / 128
  int branch_steps;       // 0: no branch; else 32-byte steps along r of the up-projection
  int tiles_m, units_n;
  const uint8_t* sfa;     // [Mpad/128][k_stages][512]
  const uint8_t* sfb;     // [k_stages][Npad/128][512]: the scale bytes of two neighbouring 128-column units are contiguous
  const uint8_t* tq;      // [Mpad][LQ_RCONT] int8 codes of the rank-r intermediate
  const uint8_t* L2c;     // [Npad][LQ_RCONT] int8 codes of the second factor, r contiguous
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
// Wait of a role that is idle for a long time (the drain during a tile's main loop): polling at full speed would take
// issue slots from the producer and the MMA issuer that share its scheduler, so it sleeps between polls.
__device__ __forceinline__ bool mbar_wait_idle(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                               int role) {
  for (int i = 0; i < 64; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    __nanosleep(200);
  }
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

// shared -> global tile store (clipped at the tensor's edges), tracked by the issuing thread's bulk groups
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* tm, int x, int y, uint32_t src) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];" ::"l"(reinterpret_cast<uint64_t>(tm)),
               "r"(x), "r"(y), "r"(src)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

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
// int8 x int8 -> int32 on the legacy tensor path: A 16 x 32 row-major, B 32 x 8 column-major fragments
__device__ __forceinline__ void mma_s8_16x8x32(int (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// 4 x 4 transpose across the four lanes of a quad: afterwards v[s] of lane t is what v[t] of lane s was.
__device__ __forceinline__ void quad_transpose(uint32_t (&v)[4], int t) {
  const bool hi2 = (t & 2) != 0, hi1 = (t & 1) != 0;
  uint32_t y0 = __shfl_xor_sync(0xffffffffu, hi2 ? v[0] : v[2], 2);
  uint32_t y1 = __shfl_xor_sync(0xffffffffu, hi2 ? v[1] : v[3], 2);
  if (hi2) { v[0] = y0; v[1] = y1; } else { v[2] = y0; v[3] = y1; }
  y0 = __shfl_xor_sync(0xffffffffu, hi1 ? v[0] : v[1], 1);
  y1 = __shfl_xor_sync(0xffffffffu, hi1 ? v[2] : v[3], 1);
  if (hi1) { v[0] = y0; v[2] = y1; } else { v[1] = y0; v[3] = y1; }
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


// Shared-memory matrix descriptor without swizzle (K-major, 8-row x 16-byte core matrices stored contiguously).
__device__ __forceinline__ uint64_t make_smem_desc_plain(uint32_t smem_addr, uint32_t lbo, uint32_t sbo) {
  const uint32_t lo = ((smem_addr & 0x3FFFFu) >> 4) | ((lbo >> 4) << 16);
  const uint32_t hi = (sbo >> 4) | (1u << 14);                             // version 1, no swizzle
  return ((uint64_t)hi << 32) | lo;
}
// 32 rows x 16 bytes of shared memory -> 4 tensor-memory columns, replicated into the four 32-lane quarters
__device__ __forceinline__ void tc_cp_sf(uint32_t taddr, uint64_t sdesc) {
  asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
// block-scaled MMA: E4M3 operands, E8M0 scales (one per row and 32-deep K block) read from tensor memory
__device__ __forceinline__ void tc_mma_mx(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t tsfa,
                                          uint32_t tsfb, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale [%0], %1, %2, %3, [%5], [%6], p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(tsfa), "r"(tsfb)
      : "memory");
}
// instruction descriptor of the block-scaled kind: E4M3 x E4M3, E8M0 scales, K-major operands, scale-byte ids
__device__ __forceinline__ constexpr uint32_t idesc_mx(int n, int sf_id) {
  return ((uint32_t)sf_id << 4) | ((uint32_t)(n >> 3) << 17) | (1u << 23) | ((uint32_t)(LQ_BM >> 4) << 24) | ((uint32_t)sf_id << 29);
}

__global__ void __launch_bounds__(GEMM_THREADS, 1)
lq_gemm_mx_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                  const __grid_constant__ CUtensorMap tmB2, const __grid_constant__ CUtensorMap tmY, const MxParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - smem_u32(smem_raw));
  constexpr int OFF_SF = NSTAGE * STAGE_BYTES;
  constexpr int OFF_SC = OFF_SF + NSTAGE * STAGE_SF_BYTES;
  constexpr int OFF_OUT = OFF_SC + 2 * SC_FLOATS * 4;
  constexpr int OFF_BAR = OFF_OUT + NUM_DRAIN_WARPS * OUT_WARP_BYTES;
  const uint32_t sm_stage = base, sm_sf = base + OFF_SF, sm_sc = base + OFF_SC, sm_out = base + OFF_OUT, sm_bar = base + OFF_BAR;
  const float* sc_ptr = reinterpret_cast<const float*>(smem + OFF_SC);
  uint8_t* out_ptr = smem + OFF_OUT;
  uint8_t* bar_ptr = smem + OFF_BAR;
  // barrier map (8 bytes each)
  constexpr int B_FULL = 0, B_EMPTY = NSTAGE, B_TFULL = 2 * NSTAGE, B_TEMPTY = B_TFULL + 1, B_RFULL = B_TEMPTY + 1,
                B_REMPTY = B_RFULL + 2, NBAR = B_REMPTY + 2;
  auto bar = [&](int idx) { return sm_bar + 8u * (uint32_t)idx; };
  static_assert(NBAR * 8 + 16 <= SMEM_BAR_BYTES, "barrier area too small");
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_ptr + NBAR * 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_ptr + NBAR * 8 + 8);

  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);   // provably warp-uniform
  const int lane = threadIdx.x & 31;
  const long long units = (long long)p.tiles_m * p.units_n;
  const int u_begin = (int)((units * blockIdx.x) / gridDim.x);
  const int u_end = (int)((units * (blockIdx.x + 1)) / gridDim.x);

  if (threadIdx.x == 0) {
    for (int s = 0; s < NSTAGE; ++s) { mbar_init(bar(B_FULL + s), 1); mbar_init(bar(B_EMPTY + s), 1); }
    mbar_init(bar(B_TFULL), 1);
    mbar_init(bar(B_TEMPTY), NUM_DRAIN_WARPS);
    for (int b = 0; b < 2; ++b) { mbar_init(bar(B_RFULL + b), 1); mbar_init(bar(B_REMPTY + b), NUM_DRAIN_WARPS); }
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
    uint32_t it = 0, tc = 0;
    bool ok = true;
    for (int u = u_begin; u < u_end && ok; ++tc) {
      const int mb = u / p.units_n, nu = u - mb * p.units_n;
      const int width = (nu + 1 < p.units_n && u + 1 < u_end) ? 2 : 1;
      const int m0 = mb * LQ_BM, n0 = nu * UNIT;
      const uint8_t* sfa = p.sfa + (size_t)mb * p.k_stages * SF_BYTES;
      const uint8_t* sfb = p.sfb + (size_t)nu * SF_BYTES;
      {   // the tile's scale vectors and bias, for the drain
        const int rb = tc & 1;
        ok = mbar_wait_warp(bar(B_REMPTY + rb), ((tc >> 1) & 1) ^ 1, abort_flag, p.status, LQ_STAGE_PRODUCER);
        if (!ok) break;
        if (elect_one()) {
          const uint32_t rfull = bar(B_RFULL + rb), dst = sm_sc + rb * SC_FLOATS * 4;
          mbar_expect_tx(rfull, (LQ_BM + 2 * width * UNIT) * 4);
          bulk_load(dst, p.sT + m0, LQ_BM * 4, rfull);
          bulk_load(dst + LQ_BM * 4, p.sL2 + n0, width * UNIT * 4, rfull);
          bulk_load(dst + (LQ_BM + 2 * UNIT) * 4, p.bias + n0, width * UNIT * 4, rfull);
        }
        __syncwarp();
      }
      for (int s = 0; s < p.k_stages && ok; ++s, ++it) {
        const int st = it % NSTAGE;
        ok = mbar_wait_warp(bar(B_EMPTY + st), ((it / NSTAGE) & 1) ^ 1, abort_flag, p.status, LQ_STAGE_PRODUCER);
        if (!ok) break;
        const uint32_t a_dst = sm_stage + st * STAGE_BYTES, b_dst = a_dst + STAGE_A_BYTES, sf_dst = sm_sf + st * STAGE_SF_BYTES;
        const uint32_t full = bar(B_FULL + st);
        if (elect_one()) {
          mbar_expect_tx(full, STAGE_A_BYTES + width * (UNIT * LQ_KSTAGE) + (1 + width) * SF_BYTES);
          tma_load_2d(a_dst, &tmA, s * LQ_KSTAGE, m0, full);
          if (width == 2) tma_load_2d(b_dst, &tmB2, s * LQ_KSTAGE, n0, full);
          else tma_load_2d(b_dst, &tmB, s * LQ_KSTAGE, n0, full);
          bulk_load(sf_dst, sfa + (size_t)s * SF_BYTES, SF_BYTES, full);
          bulk_load(sf_dst + SF_BYTES, sfb + (size_t)s * p.units_n * SF_BYTES, width * SF_BYTES, full);
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
    uint32_t it = 0, tc = 0;
    bool ok = true;
    for (int u = u_begin; u < u_end && ok; ++tc) {
      const int mb = u / p.units_n, nu = u - mb * p.units_n;
      const int width = (nu + 1 < p.units_n && u + 1 < u_end) ? 2 : 1;
      const int ncols = width * UNIT;
      // the accumulator is free once the drain has read the previous tile out of it
      ok = mbar_wait_warp(bar(B_TEMPTY), (tc & 1) ^ 1, abort_flag, p.status, LQ_STAGE_MMA);
      if (!ok) break;
      tc_fence_after();
      for (int s = 0; s < p.k_stages && ok; ++s, ++it) {
        const int st = it % NSTAGE;
        ok = mbar_wait_warp(bar(B_FULL + st), (it / NSTAGE) & 1, abort_flag, p.status, LQ_STAGE_MMA);
        if (!ok) break;
        tc_fence_after();
        const uint32_t a_addr = sm_stage + st * STAGE_BYTES, b_addr = a_addr + STAGE_A_BYTES, sf_addr = sm_sf + st * STAGE_SF_BYTES;
        const uint64_t adesc = make_smem_desc(a_addr), bdesc = make_smem_desc(b_addr);
        const uint32_t tsfa = tmem_base + TM_SFA + st * 4, tsfb = tmem_base + TM_SFB + st * 8;
        if (elect_one()) {
          tc_cp_sf(tsfa, make_smem_desc_plain(sf_addr, 16, 128));
          tc_cp_sf(tsfb, make_smem_desc_plain(sf_addr + SF_BYTES, 16, 128));
          if (width == 2) tc_cp_sf(tsfb + 4, make_smem_desc_plain(sf_addr + 2 * SF_BYTES, 16, 128));
#pragma unroll
          for (int j = 0; j < 4; ++j)
            tc_mma_mx(tmem_base, adesc + 2 * j, bdesc + 2 * j, idesc_mx(ncols, j), tsfa, tsfb, (uint32_t)(s | j));
          tc_commit(bar(B_EMPTY + st));
        }
        __syncwarp();
      }
      if (!ok) break;
      if (elect_one()) tc_commit(bar(B_TFULL));
      __syncwarp();
      u += width;
    }
  } else {
    // ------------------------------------------------------------------ drain + epilogue
    const int quad = warp & 3;                          // tensor-memory lanes 32*quad .. 32*quad+31
    const int dw = warp - FIRST_DRAIN_WARP;
    const int cgi = dw >> 2;                            // which 32 columns of each 128-column half
    const int g = lane >> 2, t = lane & 3;              // fragment coordinates: rows g and g + 8, column pair t
    const uint32_t tlane = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(cgi * 32);
    uint8_t* out_w = out_ptr + dw * OUT_WARP_BYTES;
    const uint32_t out_w_s = sm_out + dw * OUT_WARP_BYTES;
    uint32_t tc = 0;
    bool ok = true;
    for (int u = u_begin; u < u_end && ok; ++tc) {
      const int mb = u / p.units_n, nu = u - mb * p.units_n;
      const int width = (nu + 1 < p.units_n && u + 1 < u_end) ? 2 : 1;
      const int m0 = mb * LQ_BM, n0 = nu * UNIT;
      const int rl = quad * 32 + g;                     // this thread's rows inside the tile: rl + 16 mt and + 8
      const int cl = cgi * 32;                          // this warp's columns inside a half: cl + 8 nt + ...
      const int rb = tc & 1;
      // acc[half][m16 tile][n8 tile][fragment register]: first the branch's int32 sums, then fp32 outputs
      int acc[2][2][4][4];
#pragma unroll
      for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
          for (int nt = 0; nt < 4; ++nt)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[h][mt][nt][i] = 0;
      // branch part, while the tensor core works on the tile: U = tq L2q (exact int32).  All fragment loads of a step
      // are issued before the first MMA so that they share one trip to the L2.
      for (int kk = 0; kk < p.branch_steps; ++kk) {
        uint32_t a[2][4], b[2][4][2];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
          const uint8_t* ap = p.tq + (size_t)(m0 + rl + 16 * mt) * LQ_RCONT + kk * 32 + 4 * t;
          a[mt][0] = __ldg(reinterpret_cast<const uint32_t*>(ap));
          a[mt][1] = __ldg(reinterpret_cast<const uint32_t*>(ap + 8 * LQ_RCONT));
          a[mt][2] = __ldg(reinterpret_cast<const uint32_t*>(ap + 16));
          a[mt][3] = __ldg(reinterpret_cast<const uint32_t*>(ap + 8 * LQ_RCONT + 16));
        }
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
          for (int nt = 0; nt < 4; ++nt) {
            const int hh = h < width ? h : 0;           // a narrow tile reads the same (valid) rows twice and ignores them
            const uint8_t* bp = p.L2c + (size_t)(n0 + hh * UNIT + cl + nt * 8 + g) * LQ_RCONT + kk * 32 + 4 * t;
            b[h][nt][0] = __ldg(reinterpret_cast<const uint32_t*>(bp));
            b[h][nt][1] = __ldg(reinterpret_cast<const uint32_t*>(bp + 16));
          }
#pragma unroll
        for (int h = 0; h < 2; ++h)
          if (h < width) {
#pragma unroll
            for (int nt = 0; nt < 4; ++nt)
#pragma unroll
              for (int mt = 0; mt < 2; ++mt) mma_s8_16x8x32(acc[h][mt][nt], a[mt], b[h][nt][0], b[h][nt][1]);
          }
      }
      // y = U sT sL2 + bias  (|U| < 2^22: converted exactly with the 1.5 * 2^23 trick)
      ok = mbar_wait(bar(B_RFULL + rb), (tc >> 1) & 1, abort_flag, p.status, LQ_STAGE_DRAIN);
      if (!ok) break;
      {
        const float* sc = sc_ptr + rb * SC_FLOATS;
        float stv[2][2];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
          stv[mt][0] = sc[rl + 16 * mt];
          stv[mt][1] = sc[rl + 16 * mt + 8];
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          if (h < width) {
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
              const int c = h * UNIT + cl + nt * 8 + 2 * t;
              const float2 sl = *reinterpret_cast<const float2*>(sc + LQ_BM + c);
              const float2 bv = *reinterpret_cast<const float2*>(sc + LQ_BM + 2 * UNIT + c);
#pragma unroll
              for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                  const float uf = __int_as_float(acc[h][mt][nt][i] + 0x4B400000) - 12582912.0f;
                  const float y = fmaf(uf, stv[mt][i >> 1] * ((i & 1) ? sl.y : sl.x), (i & 1) ? bv.y : bv.x);
                  acc[h][mt][nt][i] = __float_as_int(y);
                }
            }
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_REMPTY + rb));
      // main part: the tensor core has already applied the block scales
      ok = mbar_wait(bar(B_TFULL), tc & 1, abort_flag, p.status, LQ_STAGE_DRAIN);
      if (!ok) break;
      tc_fence_after();
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        if (h < width) {
#pragma unroll
          for (int mt = 0; mt < 2; ++mt) {
            uint32_t v[16];
            tmem_ld_16x256b_x4(tlane + ((uint32_t)(16 * mt) << 16) + h * UNIT, v);
            tmem_ld_wait();
#pragma unroll
            for (int nt = 0; nt < 4; ++nt)
#pragma unroll
              for (int i = 0; i < 4; ++i)
                acc[h][mt][nt][i] = __float_as_int(__int_as_float(acc[h][mt][nt][i]) + __uint_as_float(v[4 * nt + i]));
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_TEMPTY));
      // epilogue
      const int row_w = m0 + quad * 32;                 // first row of this warp's part
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        if (h < width) {
          const int col_w = n0 + h * UNIT + cl;         // first column of this warp's part of the half
          if (p.out_f32) {
            float* Y = reinterpret_cast<float*>(p.Y);
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
              const int r_lo = row_w + g + 16 * mt, r_hi = r_lo + 8;
#pragma unroll
              for (int nt = 0; nt < 4; ++nt) {
                const int c = col_w + nt * 8 + 2 * t;
                if (c < p.N) {
                  if (r_lo < p.M)
                    *reinterpret_cast<float2*>(Y + (size_t)r_lo * p.N + c) =
                        make_float2(__int_as_float(acc[h][mt][nt][0]), __int_as_float(acc[h][mt][nt][1]));
                  if (r_hi < p.M)
                    *reinterpret_cast<float2*>(Y + (size_t)r_hi * p.N + c) =
                        make_float2(__int_as_float(acc[h][mt][nt][2]), __int_as_float(acc[h][mt][nt][3]));
                }
              }
            }
          } else {
            // The half's buffer was last read by the store of the previous tile: at most this tile's other half may
            // still be in flight.
            if (lane == 0) { if (h == 0) bulk_wait_read<0>(); else bulk_wait_read<1>(); }
            __syncwarp();
            uint8_t* buf = out_w + h * OUT_UNIT_BYTES;
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
              // pack to fp16, then exchange inside the quad: lane t ends up with columns 8 t .. 8 t + 7 of both rows
              uint32_t lo[4], hi[4];
#pragma unroll
              for (int nt = 0; nt < 4; ++nt) {
                const __half2 l2 = __floats2half2_rn(__int_as_float(acc[h][mt][nt][0]), __int_as_float(acc[h][mt][nt][1]));
                const __half2 h2 = __floats2half2_rn(__int_as_float(acc[h][mt][nt][2]), __int_as_float(acc[h][mt][nt][3]));
                lo[nt] = *reinterpret_cast<const uint32_t*>(&l2);
                hi[nt] = *reinterpret_cast<const uint32_t*>(&h2);
              }
              quad_transpose(lo, t);
              quad_transpose(hi, t);
              *reinterpret_cast<uint4*>(buf + (16 * mt + g) * 64 + 16 * t) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
              *reinterpret_cast<uint4*>(buf + (16 * mt + g + 8) * 64 + 16 * t) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
            }
            fence_async_smem();
            __syncwarp();
            if (lane == 0) {
              if (col_w < p.N && row_w < p.M) tma_store_2d(&tmY, col_w, row_w, out_w_s + h * OUT_UNIT_BYTES);
              bulk_commit();
            }
          }
        }
      }
      u += width;
    }
    if (lane == 0) bulk_wait_all();                      // the staged rows must stay until the last store has read them
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

lq_status lq_gemm_mx_prepare(int device) {
  if (cudaSetDevice(device) != cudaSuccess) return LQ_ERR_CUDA;
  if (lq_note_cuda(cudaFuncSetAttribute(lq_gemm_mx_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES)) !=
      cudaSuccess)
    return LQ_ERR_CUDA;
  return LQ_OK;
}

lq_status lq_launch_gemm_mx(const lq_layer* L, const lq_act* A, void* Y, lq_out_dtype dt, cudaStream_t st) {
  if (cudaSetDevice(A->device) != cudaSuccess) return LQ_ERR_CUDA;
  if (!L->mx || !A->mx || L->f16_branch) return LQ_ERR_UNSUPPORTED;
  MxParams p;
  p.M = A->M; p.N = L->N; p.Mpad = A->Mpad; p.Npad = L->Npad;
  p.k_stages = L->Kpad / LQ_KSTAGE;
  p.branch_steps = L->r == 0 ? 0 : lq_ceil_div(L->r, 32);
  p.tiles_m = lq_ceil_div(A->M, LQ_BM);
  p.units_n = L->Npad / UNIT;
  p.sfa = A->d_sfa; p.sfb = L->d_sfb; p.tq = A->d_tq; p.L2c = L->d_L2c; p.sT = A->d_sT; p.sL2 = L->d_sL2; p.bias = L->d_bias;
  p.Y = Y; p.out_f32 = dt == LQ_OUT_F32 ? 1 : 0;
  p.status = lq_device_status_ptr(A->device);
  if (!p.status) return LQ_ERR_CUDA;
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, A->device) != cudaSuccess) return LQ_ERR_CUDA;
  int ctas = g_lq_gemm_ctas > 0 ? g_lq_gemm_ctas : sms;
  const long long units = (long long)p.tiles_m * p.units_n;
  if (ctas > units) ctas = (int)units;
  // fp16 rows leave through TMA stores: a tensor map over the caller's Y (32 x 32 boxes, clipped at M and N); the fp32
  // variant stores from registers and does not use it
  CUtensorMap tmY = A->tmA;
  if (dt == LQ_OUT_F16) {
    const lq_status ts = lq_make_tmap_out_f16(&tmY, Y, (uint64_t)A->M, (uint64_t)L->N, 32, 32);
    if (ts != LQ_OK) return ts;
  }
  lq_gemm_mx_kernel<<<ctas, GEMM_THREADS, SMEM_BYTES, st>>>(A->tmA, L->tmB, L->tmB2, tmY, p);
  return lq_note_cuda(cudaGetLastError()) == cudaSuccess ? LQ_OK : LQ_ERR_CUDA;
}
