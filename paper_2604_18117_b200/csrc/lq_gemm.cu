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
//               MMAs into a FRESH 128 x 128 accumulator.  The (up to) two groups of an operand
//               stage fill one PAIR of accumulators that is handed over with one commit; two
//               pairs alternate, so the issuer works a stage ahead of the drain.  The loop is
//               warp-uniform (operands live in uniform registers) and one elected lane issues
//   warps 2-17  drain: each warp owns 32 rows x 32 columns of the tile.  A group's accumulator
//               slice is fetched as two tcgen05.ld.16x256b (256 bits per lane and access), ONE
//               wait, and the accumulator is handed back at once; the next group's halves are
//               requested as the registers of the current one are consumed, so the fetch runs
//               under the arithmetic: acc += P * (sx * sw), packed f32x2, fp32 registers.  After
//               the last group: bias is already in (it is the start value), convert, exchange
//               inside each quad so that a lane holds 16 contiguous bytes of a row, store
// The per-group arithmetic is the bound: 2 fp32 operations per output and group on 128 lanes
// per SM, against 8192 MACs per clock on the tensor pipe - 256 clocks of drain for 128 clocks
// of tensor work per 128 x 128 x 64 block.  Work is cut in 128 x 128 tiles; every CTA takes a
// contiguous, balanced run of them, row block major.
// The 4-bit codes ride in E4M3 operands (integers up to 7 are exact, fp32 accumulation of
// |sum| <= 3136 is exact); the branch's 8-bit codes use kind::i8 (exact int32), the fp16
// reference branch kind::f16.
// Every wait is bounded; on expiry the role records LQ_ERR_TIMEOUT in the device status word,
// raises a CTA-wide abort flag and all roles leave through the common teardown.
#include <cuda_fp16.h>

#include "lq_device.cuh"

#ifdef LQ_TIMELINE
// Timeline build only: copies the stamp lists of the last launch to the host ([TL_LISTS][TL_CAP] words) and clears them.
extern "C" int lq_debug_timeline(unsigned long long* host_out) {
  if (cudaDeviceSynchronize() != cudaSuccess) return 1;
  if (cudaMemcpyFromSymbol(host_out, g_lq_timeline, sizeof(unsigned long long) * lqdev::TL_LISTS * lqdev::TL_CAP) != cudaSuccess) return 1;
  static unsigned long long zeros[lqdev::TL_LISTS][lqdev::TL_CAP];
  return cudaMemcpyToSymbol(g_lq_timeline, zeros, sizeof(zeros)) == cudaSuccess ? 0 : 1;
}
#endif

namespace {

using namespace lqdev;

constexpr int UNIT = LQ_BN;                        // 128 output columns per tile
constexpr int NSTAGE = 4;                          // operand ring depth (a power of two: ring positions are masks)
constexpr int NTBUF = 2;                           // ring of accumulator PAIRS in tensor memory: a pair = the (up to) two groups of one operand stage, 2 x 128 columns
constexpr int TCOLS = 128;                         // columns per accumulator
constexpr int STAGE_A_BYTES = LQ_BM * LQ_KSTAGE;   // 16 KB
constexpr int STAGE_B_BYTES = UNIT * LQ_KSTAGE;    // 16 KB
constexpr int STAGE_BYTES = STAGE_A_BYTES + STAGE_B_BYTES;
constexpr int SC_GROUP_FLOATS = LQ_BM + UNIT;      // sx[128] then sw[128]
constexpr int SC_STAGE_BYTES = 2 * SC_GROUP_FLOATS * 4;   // two groups
constexpr int NUM_DRAIN_WARPS = 16;
constexpr int FIRST_DRAIN_WARP = 2;
constexpr int GEMM_THREADS = (FIRST_DRAIN_WARP + NUM_DRAIN_WARPS) * 32;
constexpr int WCOLS = 32;                          // columns per drain warp
constexpr int SMEM_BAR_BYTES = 256;
constexpr int SMEM_BYTES = 1024 /*alignment slack*/ + NSTAGE * STAGE_BYTES + NSTAGE * SC_STAGE_BYTES + SMEM_BAR_BYTES;
static_assert(SMEM_BYTES <= 232448, "shared memory budget");
static_assert(STAGE_BYTES % 1024 == 0, "stages must keep the 1024-byte alignment of the swizzled tiles");
static_assert((NSTAGE & (NSTAGE - 1)) == 0 && (NTBUF & (NTBUF - 1)) == 0, "ring sizes must be powers of two");

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

// One accumulator slice of 16 rows x 32 columns in the layout of tcgen05.ld.16x256b (the accumulator-fragment layout
// of mma.sync m16n8: with g = lane / 4 and t = lane % 4, registers 4j .. 4j+3 hold row g, columns 8j + 2t and
// 8j + 2t + 1, then row g + 8, the same columns): acc += P * (sx * sw).  This shape moves 256 bits per lane and access;
// the one-row-per-thread shape (32x32b) moves 32 and was measured at 60-80 bytes per clock and SM, which capped the
// whole kernel.  INT: the accumulator holds int32 (kind::i8); |P| < 2^22, so adding 1.5 * 2^23 in the integer domain
// and subtracting it in fp32 converts exactly without the conversion pipe.
template <bool INT>
__device__ __forceinline__ void drain_frag(const uint32_t (&v)[16], float2* acc, float sx_lo, float sx_hi, const float2 (&sw)[4]) {
  const float2 sl = make_float2(sx_lo, sx_lo), sh = make_float2(sx_hi, sx_hi);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    float2 p0, p1;
    if constexpr (INT) {
      p0 = make_float2(__int_as_float((int)v[4 * j + 0] + 0x4B400000) - 12582912.0f,
                       __int_as_float((int)v[4 * j + 1] + 0x4B400000) - 12582912.0f);
      p1 = make_float2(__int_as_float((int)v[4 * j + 2] + 0x4B400000) - 12582912.0f,
                       __int_as_float((int)v[4 * j + 3] + 0x4B400000) - 12582912.0f);
    } else {
      p0 = make_float2(__uint_as_float(v[4 * j + 0]), __uint_as_float(v[4 * j + 1]));
      p1 = make_float2(__uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
    }
    acc[2 * j + 0] = __ffma2_rn(p0, __fmul2_rn(sl, sw[j]), acc[2 * j + 0]);
    acc[2 * j + 1] = __ffma2_rn(p1, __fmul2_rn(sh, sw[j]), acc[2 * j + 1]);
  }
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
  const uint32_t sm_bar = sm_sc + NSTAGE * SC_STAGE_BYTES;
  uint8_t* bar_ptr = smem + NSTAGE * STAGE_BYTES + NSTAGE * SC_STAGE_BYTES;
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
  // this CTA's contiguous run of 128 x 128 tiles, row block major
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
    mbar_init_fence();
  }
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), 512);
  tc_fence_before();
  __syncthreads();
  grid_dependency_sync();        // set-up done; from here on global memory written by earlier kernels is read
  tc_fence_after();
  const uint32_t tmem_base = __shfl_sync(0xffffffffu, *tmem_slot, 0);

  LQ_TL_DECL((blockIdx.x == 0 && lane == 0)
                 ? (warp == 0 ? (int)TL_PRODUCER : warp == 1 ? (int)TL_MMA : warp == FIRST_DRAIN_WARP ? (int)TL_DRAIN_FIRST
                    : warp == FIRST_DRAIN_WARP + NUM_DRAIN_WARPS - 1 ? (int)TL_DRAIN_LAST : -1)
                 : -1);

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    uint32_t it = 0, armed = 0;
    bool ok = true;
    for (int u = u_begin; u < u_end && ok; ++u) {
      const int mb = u / p.units_n, nu = u - mb * p.units_n;
      const int m0 = mb * LQ_BM, n0 = nu * UNIT;
      for (int s = 0; s < stages_per_tile && ok; ++s, ++it) {
        const int st = it & (NSTAGE - 1);
        const uint32_t par = ((it / NSTAGE) & 1) ^ 1;
        ok = mbar_wait_warp(bar_empty(st), par, abort_flag, p.status, LQ_STAGE_PRODUCER);
        if (!ok) break;
        ok = mbar_wait_warp(bar_sempty(st), par, abort_flag, p.status, LQ_STAGE_PRODUCER);
        if (!ok) break;
        LQ_TL(EV_P_SLOT_FREE, s);
        const uint32_t a_dst = sm_stage + st * STAGE_BYTES, b_dst = a_dst + STAGE_A_BYTES;
        const uint32_t sc_dst = sm_sc + st * SC_STAGE_BYTES;
        const uint32_t full = bar_full(st);
        const bool is_main = s < p.n_stages_main;
        const int ngroups = is_main ? ((2 * s + 1 < p.G) ? 2 : 1) : 1;
        const uint32_t tx = STAGE_BYTES + ngroups * SC_GROUP_FLOATS * 4;
        if (elect_one()) {
          mbar_expect_tx(full, tx);
          if (is_main) {
            tma_load_2d(a_dst, &tmA, s * LQ_KSTAGE, m0, full);
            tma_load_2d(b_dst, &tmB, s * LQ_KSTAGE, n0, full);
            for (int q = 0; q < ngroups; ++q) {
              const size_t g = (size_t)(2 * s + q);
              bulk_load(sc_dst + q * SC_GROUP_FLOATS * 4, p.sx + g * p.Mpad + m0, LQ_BM * 4, full);
              bulk_load(sc_dst + q * SC_GROUP_FLOATS * 4 + LQ_BM * 4, p.sw + g * p.Npad + n0, UNIT * 4, full);
            }
          } else {
            tma_load_2d(a_dst, &tmT, 0, m0, full);
            tma_load_2d(b_dst, &tmL2, 0, n0, full);
            bulk_load(sc_dst, p.sT + m0, LQ_BM * 4, full);
            bulk_load(sc_dst + LQ_BM * 4, p.sL2 + n0, UNIT * 4, full);
          }
        }
        __syncwarp();
        ++armed;
        LQ_TL(EV_P_ISSUED, s);
      }
    }
    if (!ok && lane == 0) {
      // aborting: give the copies already issued a bounded time to land before the CTA's shared memory goes away
      const uint32_t n = armed < (uint32_t)NSTAGE ? armed : (uint32_t)NSTAGE;
      for (uint32_t i = 1; i <= n; ++i) {
        const uint32_t j = armed - i;
        mbar_settle(bar_full(j % NSTAGE), (j / NSTAGE) & 1);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    uint32_t it = 0;
    bool ok = true;
    const uint32_t shape = idesc_shape(UNIT);
    for (int u = u_begin; u < u_end && ok; ++u) {
      for (int s = 0; s < stages_per_tile && ok; ++s, ++it) {
        const int st = it & (NSTAGE - 1);
        ok = mbar_wait_warp(bar_full(st), (it / NSTAGE) & 1, abort_flag, p.status, LQ_STAGE_MMA);
        if (!ok) break;
        tc_fence_after();
        LQ_TL(EV_M_STAGE_FULL, s);
        const uint32_t a_addr = sm_stage + st * STAGE_BYTES, b_addr = a_addr + STAGE_A_BYTES;
        const uint64_t adesc = make_smem_desc(a_addr), bdesc = make_smem_desc(b_addr);
        const bool is_main = s < p.n_stages_main;
        const int ngroups = is_main ? ((2 * s + 1 < p.G) ? 2 : 1) : 1;
        // the stage's (up to) two groups go to the two accumulators of one pair; ONE commit hands the pair over
        const int pb = it & (NTBUF - 1);
        ok = mbar_wait_warp(bar_tempty(pb), ((it / NTBUF) & 1) ^ 1, abort_flag, p.status, LQ_STAGE_MMA);
        if (!ok) break;
        tc_fence_after();
        LQ_TL(EV_M_ACC_FREE, s);
        const uint32_t d = tmem_base + pb * (2 * TCOLS);
        if (elect_one()) {
          if (is_main) {
            for (int q = 0; q < ngroups; ++q) {
              const uint64_t off = (uint64_t)((q * 64) >> 4);
              tc_mma<TC_F8>(d + q * TCOLS, adesc + off, bdesc + off, IDESC_F8 | shape, 0u);
              tc_mma<TC_F8>(d + q * TCOLS, adesc + off + 2, bdesc + off + 2, IDESC_F8 | shape, 1u);
            }
          } else {
            for (int j = 0; j < p.branch_mmas; ++j) {
              const uint64_t off = (uint64_t)((j * 32) >> 4);
              if (p.branch_f16) tc_mma<TC_F16>(d, adesc + off, bdesc + off, IDESC_F16 | shape, (uint32_t)j);
              else tc_mma<TC_I8>(d, adesc + off, bdesc + off, IDESC_I8 | shape, (uint32_t)j);
            }
          }
          tc_commit(bar_tfull(pb));
          tc_commit(bar_empty(st));
        }
        __syncwarp();
        LQ_TL(EV_M_ISSUED, s);
      }
    }
  } else {
    // ------------------------------------------------------------------ drain + epilogue
    const int quad = warp & 3;                          // tensor-memory lanes 32*quad .. 32*quad+31
    const int cgi = (warp - FIRST_DRAIN_WARP) >> 2;     // which quarter of the tile's columns
    const int coff = cgi * WCOLS;
    const uint32_t tlane = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)coff;
    const int fg = lane >> 2, ft = lane & 3;            // fragment coordinates: rows fg + 8 i, column pair ft
    uint32_t it = 0;
    bool ok = true;
    for (int u = u_begin; u < u_end && ok; ++u) {
      const int mb = u / p.units_n, nu = u - mb * p.units_n;
      const int m0 = mb * LQ_BM, n0 = nu * UNIT;
      LQ_TL(EV_TILE, 0);
      // this thread's 4 rows x 8 columns: acc[8 h + 2 j + i] = rows 16 h + fg + 8 i, columns 8 j + 2 ft, + 1; starts from the bias
      float2 acc[16];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float2 bv = __ldg(reinterpret_cast<const float2*>(p.bias + n0 + coff + 8 * j + 2 * ft));
        acc[2 * j] = bv; acc[2 * j + 1] = bv; acc[8 + 2 * j] = bv; acc[8 + 2 * j + 1] = bv;
      }
      // Groups g = 0 .. G-1 come two per operand stage, then the branch has a stage of its own.  `it` counts operand
      // stages since the kernel began: stage ring position it & (NSTAGE-1), accumulator pair it & (NTBUF-1).  All
      // hand-shakes are per stage: the scale vectors and the accumulator pair are awaited once, the pair is handed back
      // when its last group sits in registers.  The group being consumed sits in (vlo, vhi): rows 0-15 and 16-31 of
      // this warp's quarter, 32 columns each; the next group's halves are requested as soon as a half is consumed.
      uint32_t vlo[16], vhi[16];
      // waits for stage `IT_`'s scale vectors and accumulator pair
#define LQ_AWAIT_STAGE(IT_)                                                                                              \
      {                                                                                                                  \
        const uint32_t i_ = (IT_);                                                                                       \
        ok = mbar_wait(bar_full(i_ & (NSTAGE - 1)), (i_ / NSTAGE) & 1, abort_flag, p.status, LQ_STAGE_DRAIN);            \
        if (ok) ok = mbar_wait(bar_tfull(i_ & (NTBUF - 1)), (i_ / NTBUF) & 1, abort_flag, p.status, LQ_STAGE_DRAIN);     \
        tc_fence_after();                                                                                                \
      }
      // one group: arithmetic on (vlo, vhi) with the scales at SCG_; the next group's halves (if HAS_NEXT_) are at TNEXT_
#define LQ_DRAIN_GROUP(SCG_, IS_INT_, HAS_NEXT_, TNEXT_)                                                                 \
      {                                                                                                                  \
        const float* sxp_ = (SCG_) + quad * 32 + fg;                                                                     \
        const float* swp_ = (SCG_) + LQ_BM + coff + 2 * ft;                                                              \
        const float sx0 = sxp_[0], sx1 = sxp_[8], sx2 = sxp_[16], sx3 = sxp_[24];                                        \
        float2 sw2[4];                                                                                                   \
        _Pragma("unroll") for (int j_ = 0; j_ < 4; ++j_) sw2[j_] = *reinterpret_cast<const float2*>(swp_ + 8 * j_);      \
        if (IS_INT_) drain_frag<true>(vlo, &acc[0], sx0, sx1, sw2);                                                      \
        else drain_frag<false>(vlo, &acc[0], sx0, sx1, sw2);                                                             \
        if (HAS_NEXT_) tmem_ld_16x256b_x4((TNEXT_), vlo);                                                                \
        if (IS_INT_) drain_frag<true>(vhi, &acc[8], sx2, sx3, sw2);                                                      \
        else drain_frag<false>(vhi, &acc[8], sx2, sx3, sw2);                                                             \
        if (HAS_NEXT_) tmem_ld_16x256b_x4((TNEXT_) + (16u << 16), vhi);                                                  \
      }
      LQ_AWAIT_STAGE(it)
      if (!ok) break;
      {
        const uint32_t t0_ = tlane + (it & (NTBUF - 1)) * (2 * TCOLS);
        tmem_ld_16x256b_x4(t0_, vlo);
        tmem_ld_16x256b_x4(t0_ + (16u << 16), vhi);
      }
      for (int s = 0; s < stages_per_tile && ok; ++s, ++it) {
        const bool is_main = s < p.n_stages_main;
        const bool two = is_main && (2 * s + 1 < p.G);
        const bool is_int = !is_main && p.branch_f16 == 0;
        const bool last_stage = s + 1 == stages_per_tile;
        const int st = it & (NSTAGE - 1);
        const float* scg = sc_ptr + st * (SC_STAGE_BYTES / 4);
        const uint32_t tpair = tlane + (it & (NTBUF - 1)) * (2 * TCOLS);
        const uint32_t tpair_next = tlane + ((it + 1) & (NTBUF - 1)) * (2 * TCOLS);
        LQ_TL(EV_D_OPEN, s);
        if (two) {
          tmem_ld_wait();                               // the stage's first group is in registers
          LQ_TL(EV_D_WAITED, s);
          LQ_DRAIN_GROUP(scg, false, true, tpair + TCOLS)
          LQ_TL(EV_D_HALF, s);
        }
        tmem_ld_wait();                                 // the stage's last group is in registers:
        tc_fence_before();                              // the accumulator pair goes back to the MMA warp
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_tempty(it & (NTBUF - 1)));
        LQ_TL(EV_D_LOADED, s);
        if (!last_stage) LQ_AWAIT_STAGE(it + 1)
        LQ_TL(EV_D_ACC_FULL, s);
        {
          const float* scg2 = scg + (two ? SC_GROUP_FLOATS : 0);
          const bool has_next = !last_stage && ok;
          LQ_DRAIN_GROUP(scg2, is_int, has_next, tpair_next)
        }
        LQ_TL(EV_D_DONE, s);
        __syncwarp();                                   // done with this stage's scale vectors
        if (lane == 0) mbar_arrive(bar_sempty(st));
      }
#undef LQ_DRAIN_GROUP
#undef LQ_AWAIT_STAGE
      if (!ok) break;
      LQ_TL(EV_D_EPI_BEGIN, 0);
      // epilogue straight from registers: rows m0 + 32 quad + 16 h + fg (+ 8), columns n0 + coff + 8 j + 2 ft (+ 1)
      const int row_w = m0 + quad * 32;
      if (p.out_f32) {
        float* Y = reinterpret_cast<float*>(p.Y);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int r_lo = row_w + 16 * h + fg, r_hi = r_lo + 8;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int c = n0 + coff + 8 * j + 2 * ft;                  // four lanes write the 32 bytes of one row's sector
            if (c < p.N) {
              if (r_lo < p.M) *reinterpret_cast<float2*>(Y + (size_t)r_lo * p.N + c) = acc[8 * h + 2 * j];
              if (r_hi < p.M) *reinterpret_cast<float2*>(Y + (size_t)r_hi * p.N + c) = acc[8 * h + 2 * j + 1];
            }
          }
        }
      } else {
        __half* Y = reinterpret_cast<__half*>(p.Y);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          // pack to fp16, then exchange inside the quad: lane ft ends up with columns 8 ft .. 8 ft + 7 of both rows
          uint32_t lo[4], hi[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const __half2 l2 = __floats2half2_rn(acc[8 * h + 2 * j].x, acc[8 * h + 2 * j].y);
            const __half2 h2 = __floats2half2_rn(acc[8 * h + 2 * j + 1].x, acc[8 * h + 2 * j + 1].y);
            lo[j] = *reinterpret_cast<const uint32_t*>(&l2);
            hi[j] = *reinterpret_cast<const uint32_t*>(&h2);
          }
          quad_transpose(lo, ft);
          quad_transpose(hi, ft);
          const int c = n0 + coff + 8 * ft;                            // 16 contiguous bytes of a row per lane
          const int r_lo = row_w + 16 * h + fg, r_hi = r_lo + 8;
          if (c < p.N) {
            if (r_lo < p.M) *reinterpret_cast<uint4*>(Y + (size_t)r_lo * p.N + c) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
            if (r_hi < p.M) *reinterpret_cast<uint4*>(Y + (size_t)r_hi * p.N + c) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
          }
        }
      }
      LQ_TL(EV_D_EPI_END, 0);
    }
  }

  // ---------------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
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
    mbar_init_fence();
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
  const cudaError_t e = lq_launch(lq_gemm_kernel, ctas, GEMM_THREADS, SMEM_BYTES, st, A->tmA, L->tmB, A->tmT, L->tmL2, p);
  return lq_note_cuda(e != cudaSuccess ? e : cudaGetLastError()) == cudaSuccess ? LQ_OK : LQ_ERR_CUDA;
}
