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
//               per tile one more stage with the branch operands (tq, L2q) and the vectors sT, sL2, bias for the drain
//   warp 1      owns tensor memory; per stage: tcgen05.cp of the scale bytes into tensor-memory columns, then four
//               K = 32 block-scaled MMAs (N = 256) into the tile's accumulator; after the last stage the low-rank
//               branch's up-projection U = tq L2q (kind::i8, exact int32; its fp32 scales cannot be applied by the
//               tensor core) into a second accumulator, then ONE hand-over of both to the drain
//   warps 2-17  drain: tcgen05.ld the main accumulator (mma.sync fragment layout, 16x256b) straight into registers and
//               release it - the next tile's main loop starts - then read the branch accumulator,
//               y = main + sT sL2 U + bias, release that too, convert; a 4 x 4 exchange inside each quad gives
//               every lane 16 contiguous bytes of one row, so each store instruction writes whole 32-byte sectors
//               straight from registers.
// Tensor memory has 512 columns: main accumulator [0, 256), branch accumulator [256, 512).  The 12 scale-factor
// columns of a stage (one slot: the tensor pipe executes one thread's tcgen05 copies and MMAs in issue order) alias the
// first 16 columns of the branch accumulator: they are live only while the tile's block-scaled MMAs run, the branch
// accumulator only from the branch MMA (issued after them) until the drain has read it.  The four drain warps that own
// those 16 columns read them together with the main accumulator, before the hand-over; the rest of the branch
// accumulator is read afterwards, under the next tile's main loop, and is needed again only by that tile's branch MMA.
// What was measured on the way here (PixArt block, four GEMMs): the branch on mma.sync in the drain warps took tensor
// time from the main loop; TMA stores of the output (32 boxes of 2 KB, or 8 of 8 KB, per tile) cost 15 % against
// plain stores - they share the TMA unit with the operand loads; a fourth ring stage gained 3 %.
// Every wait is bounded as in lq_gemm.cu.
#include <cuda_fp16.h>

#include "lq_device.cuh"

#ifdef LQ_TIMELINE
// Timeline build only: copies this kernel's stamp lists of the last launch to the host and clears them.
extern "C" int lq_debug_timeline_mx(unsigned long long* host_out) {
  if (cudaDeviceSynchronize() != cudaSuccess) return 1;
  if (cudaMemcpyFromSymbol(host_out, g_lq_timeline, sizeof(unsigned long long) * lqdev::TL_LISTS * lqdev::TL_CAP) != cudaSuccess) return 1;
  static unsigned long long zeros[lqdev::TL_LISTS][lqdev::TL_CAP];
  return cudaMemcpyToSymbol(g_lq_timeline, zeros, sizeof(zeros)) == cudaSuccess ? 0 : 1;
}
#endif

namespace {

using namespace lqdev;

constexpr int UNIT = LQ_BN;                        // 128 output columns
constexpr int NSTAGE = 4;                          // operand ring depth
constexpr int STAGE_A_BYTES = LQ_BM * LQ_KSTAGE;   // 16 KB
constexpr int STAGE_B_BYTES = 2 * UNIT * LQ_KSTAGE;   // 32 KB (one 256-row box, or one 128-row box for a narrow tile)
constexpr int STAGE_BYTES = STAGE_A_BYTES + STAGE_B_BYTES;
constexpr int SF_BYTES = 512;                      // scale bytes of 128 rows x 4 K blocks
constexpr int STAGE_SF_BYTES = 3 * SF_BYTES;       // SFA, then SFB of both halves
constexpr int SC_FLOATS = LQ_BM + 4 * UNIT;        // per tile: sT[128], sL2[256], bias[256]
constexpr int NUM_DRAIN_WARPS = 16;
constexpr int FIRST_DRAIN_WARP = 2;
constexpr int GEMM_THREADS = (FIRST_DRAIN_WARP + NUM_DRAIN_WARPS) * 32;
constexpr int SMEM_BAR_BYTES = 256;
constexpr int SMEM_BYTES = 1024 /*alignment slack*/ + NSTAGE * STAGE_BYTES + NSTAGE * STAGE_SF_BYTES + 2 * SC_FLOATS * 4 +
                           SMEM_BAR_BYTES;
static_assert(SMEM_BYTES <= 232448, "shared memory budget");
static_assert(STAGE_BYTES % 1024 == 0, "stages must keep the 1024-byte alignment of the swizzled tiles");
// tensor-memory columns: main accumulator [0, 256), branch accumulator [256, 512); 4 columns of A scales and 8 of B
// scales alias the start of the branch accumulator (disjoint lifetimes, see the top of the file)
constexpr int TM_BR = 256, TM_SFA = 256, TM_SFB = TM_SFA + 4, TM_SF_ALIASED = 16;

struct MxParams {
  int M, N, Mpad, Npad;
  int k_stages;           // stages of A per tile: Kpad / 128, times two when 8-bit activation codes come as two digit planes
  int branch_steps;       // 0: no branch; else MMAs of the branch stage (32 bytes of r each)
  int branch_f16;         // the branch operands are halves (W16A16 reference branch): no scales, summed by the tensor core
  int branch_mx;          // the branch is MX as well: its up-projection is one more block-scaled stage onto the main
                          // accumulator.  1: MXFP elements, K blocks in order.  2: 8-bit integer codes as digit planes on
                          // both sides - the stage's four K blocks are (hi, 0), (hi, 1), (lo, 0), (lo, 1) and every
                          // (plane of T, plane of L2) pair of the same rank block is one MMA.  3: the same codes with 4-bit
                          // factors (one plane) and rank up to 128: two stages like mode 1, one per plane of T
  const uint8_t* sft;     // branch_mx: E8M0 bytes of T's block scales, [Mpad/128][512]
  const uint8_t* sfl2;    // branch_mx: E8M0 bytes of L2's block scales, [Npad/128][512]
  int tiles_m, units_n;
  int by_units;           // how the CTAs share the work: 0 whole tiles, 1 128-column units
  int b_wrap;             // Kpad / 128: stage s reads B (and its scales) at stage s mod b_wrap - the planes share the weights
                          // (kept in what was the padding before the next pointer: this kernel sits at its register
                          // cap, and moving its other parameters changed the allocation ptxas found - 50 % more spill
                          // traffic and 15 % longer launches)
  const uint8_t* sfa;     // [Mpad/128][k_stages][512]
  const uint8_t* sfb;     // [k_stages][Npad/128][512]: the scale bytes of two neighbouring 128-column units are contiguous
  const float* sT;        // [Mpad]
  const float* sL2;       // [Npad]
  const float* bias;      // [Npad]
  void* Y;
  int out_f32;
  int32_t* status;
};

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
// y = main + U sT sL2 + bias for one n8 fragment (registers: row g columns 2t, 2t+1, then row g + 8 the same columns).
// U is an exact int32 with |U| < 2^22: converted exactly with the 1.5 * 2^23 trick.
__device__ __forceinline__ void combine_fragment(float (&a)[4], const uint32_t* u, bool has_branch, float st_lo, float st_hi,
                                                 float2 sl, float2 bv) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float y = a[i] + ((i & 1) ? bv.y : bv.x);
    if (has_branch) {
      const float uf = __int_as_float((int)u[i] + 0x4B400000) - 12582912.0f;
      y = fmaf(uf, ((i >> 1) ? st_hi : st_lo) * ((i & 1) ? sl.y : sl.x), y);
    }
    a[i] = y;
  }
}

// BRANCH_ACC: the layer has an integer branch with fp32 scales, whose product needs an accumulator of its own.  The
// other instance (no branch, fp16 branch, MX branches) carries none of that code or its registers.
template <bool BRANCH_ACC>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
lq_gemm_mx_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                  const __grid_constant__ CUtensorMap tmB2, const __grid_constant__ CUtensorMap tmT,
                  const __grid_constant__ CUtensorMap tmL2, const MxParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - smem_u32(smem_raw));
  constexpr int OFF_SF = NSTAGE * STAGE_BYTES;
  constexpr int OFF_SC = OFF_SF + NSTAGE * STAGE_SF_BYTES;
  constexpr int OFF_BAR = OFF_SC + 2 * SC_FLOATS * 4;
  const uint32_t sm_stage = base, sm_sf = base + OFF_SF, sm_sc = base + OFF_SC, sm_bar = base + OFF_BAR;
  const float* sc_ptr = reinterpret_cast<const float*>(smem + OFF_SC);
  uint8_t* bar_ptr = smem + OFF_BAR;
  // barrier map (8 bytes each)
  constexpr int B_FULL = 0, B_EMPTY = NSTAGE, B_TFULL = 2 * NSTAGE, B_TEMPTY = B_TFULL + 1, B_RFULL = B_TEMPTY + 1,
                B_REMPTY = B_RFULL + 2, B_BEMPTY = B_REMPTY + 2, NBAR = B_BEMPTY + 1;
  auto bar = [&](int idx) { return sm_bar + 8u * (uint32_t)idx; };
  static_assert(NBAR * 8 + 16 <= SMEM_BAR_BYTES, "barrier area too small");
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_ptr + NBAR * 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_ptr + NBAR * 8 + 8);

  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);   // provably warp-uniform
  const int lane = threadIdx.x & 31;
  const bool has_branch = p.branch_steps > 0;
  const int nbst = p.branch_mx == 3 ? 2 : 1;              // stages of the branch per tile
  // An fp16 branch has no scales: its product is accumulated onto the main accumulator by the tensor core and the drain
  // sees no branch at all.  An integer branch needs its fp32 scales applied per element: second accumulator.
  constexpr bool branch_acc = BRANCH_ACC;                 // = has_branch && !p.branch_f16 && !p.branch_mx, decided by the host
  // Each CTA takes a contiguous, equal share of the work and walks it as 256-wide tiles (128-wide where a row block or
  // the share ends).  A 128-wide tile costs nearly as much as a 256-wide one (a stage's time is set by its hand-shakes
  // and instruction count, not its MMA width).  by_units = 0 shares whole tiles - row blocks cut into 256-wide tiles
  // plus at most one 128-wide one - which avoids needless narrow tiles; by_units = 1 shares 128-column units, which
  // balances better when a CTA gets only two or three tiles and the row blocks have an odd number of units.
  const int tiles_n = (p.units_n + 1) >> 1;
  const long long work = (long long)p.tiles_m * (p.by_units ? p.units_n : tiles_n);
  const int w_begin = (int)((work * blockIdx.x) / gridDim.x);
  const int w_end = (int)((work * (blockIdx.x + 1)) / gridDim.x);
  // position w -> row block, first unit and width of the tile that starts there
  auto tile_at = [&](int w, int& mb, int& nu, int& width) {
    if (p.by_units) {
      mb = w / p.units_n; nu = w - mb * p.units_n;
      width = (nu + 1 < p.units_n && w + 1 < w_end) ? 2 : 1;
      return w + width;
    }
    mb = w / tiles_n; nu = 2 * (w - mb * tiles_n);
    width = (nu + 1 < p.units_n) ? 2 : 1;
    return w + 1;
  };

  if (threadIdx.x == 0) {
    for (int s = 0; s < NSTAGE; ++s) { mbar_init(bar(B_FULL + s), 1); mbar_init(bar(B_EMPTY + s), 1); }
    mbar_init(bar(B_TFULL), 1);
    mbar_init(bar(B_TEMPTY), NUM_DRAIN_WARPS);
    for (int b = 0; b < 2; ++b) { mbar_init(bar(B_RFULL + b), 1); mbar_init(bar(B_REMPTY + b), NUM_DRAIN_WARPS); }
    mbar_init(bar(B_BEMPTY), NUM_DRAIN_WARPS);
    *abort_flag = 0;
    mbar_init_fence();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), 512);
  }
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
    uint32_t it = 0, tc = 0, rarmed = 0;
    bool ok = true;
    for (int w = w_begin, w_next; w < w_end && ok; w = w_next, ++tc) {
      int mb, nu, width;
      w_next = tile_at(w, mb, nu, width);
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
        ++rarmed;
      }
      for (int s = 0; s < p.k_stages && ok; ++s, ++it) {
        const int st = it % NSTAGE;
        ok = mbar_wait_warp(bar(B_EMPTY + st), ((it / NSTAGE) & 1) ^ 1, abort_flag, p.status, LQ_STAGE_PRODUCER);
        if (!ok) break;
        LQ_TL(EV_P_SLOT_FREE, s);
        const uint32_t a_dst = sm_stage + st * STAGE_BYTES, b_dst = a_dst + STAGE_A_BYTES, sf_dst = sm_sf + st * STAGE_SF_BYTES;
        const uint32_t full = bar(B_FULL + st);
        if (elect_one()) {
          mbar_expect_tx(full, STAGE_A_BYTES + width * (UNIT * LQ_KSTAGE) + (1 + width) * SF_BYTES);
          const int sb = s >= p.b_wrap ? s - p.b_wrap : s;       // the lo digits' plane runs over the same weights
          tma_load_2d(a_dst, &tmA, s * LQ_KSTAGE, m0, full);
          if (width == 2) tma_load_2d(b_dst, &tmB2, sb * LQ_KSTAGE, n0, full);
          else tma_load_2d(b_dst, &tmB, sb * LQ_KSTAGE, n0, full);
          bulk_load(sf_dst, sfa + (size_t)s * SF_BYTES, SF_BYTES, full);
          bulk_load(sf_dst + SF_BYTES, sfb + (size_t)sb * p.units_n * SF_BYTES, width * SF_BYTES, full);
        }
        __syncwarp();
        LQ_TL(EV_P_ISSUED, s);
      }
      // the branch operands: the containers of tq (128 rows) and L2q (256 rows), r contiguous; mode 3 brings the two
      // digit planes of tq as two stages against the same L2q
      for (int bs = 0; bs < nbst && has_branch && ok; ++bs) {
        const int st = it % NSTAGE;
        ok = mbar_wait_warp(bar(B_EMPTY + st), ((it / NSTAGE) & 1) ^ 1, abort_flag, p.status, LQ_STAGE_PRODUCER);
        if (!ok) break;
        const uint32_t a_dst = sm_stage + st * STAGE_BYTES, b_dst = a_dst + STAGE_A_BYTES;
        const uint32_t full = bar(B_FULL + st);
        if (elect_one()) {
          mbar_expect_tx(full, STAGE_A_BYTES + width * (UNIT * LQ_KSTAGE) + (p.branch_mx ? (1 + width) * SF_BYTES : 0));
          tma_load_2d(a_dst, &tmT, bs * LQ_KSTAGE, m0, full);
          tma_load_2d(b_dst, &tmL2, 0, n0, full);
          if (width == 2) tma_load_2d(b_dst + UNIT * LQ_KSTAGE, &tmL2, 0, n0 + UNIT, full);
          if (p.branch_mx) {   // the block scales of T (rows) and of L2 (columns) along the rank
            const uint32_t sf_dst = sm_sf + st * STAGE_SF_BYTES;
            bulk_load(sf_dst, p.sft + ((size_t)mb * nbst + bs) * SF_BYTES, SF_BYTES, full);
            bulk_load(sf_dst + SF_BYTES, p.sfl2 + (size_t)nu * SF_BYTES, width * SF_BYTES, full);
          }
        }
        __syncwarp();
        ++it;
      }
    }
    if (!ok && lane == 0) {
      // aborting: give the copies already issued a bounded time to land before the CTA's shared memory goes away
      // (`it` stages have been armed; the last NSTAGE of them may still be in flight)
      const uint32_t n = it < (uint32_t)NSTAGE ? it : (uint32_t)NSTAGE;
      for (uint32_t i = 1; i <= n; ++i) {
        const uint32_t j = it - i;
        mbar_settle(bar(B_FULL + (int)(j % NSTAGE)), (j / NSTAGE) & 1);
      }
      for (uint32_t i = 1; i <= (rarmed < 2u ? rarmed : 2u); ++i) {     // and the tiles' scale vectors
        const uint32_t j = rarmed - i;
        mbar_settle(bar(B_RFULL + (int)(j & 1)), (j >> 1) & 1);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    uint32_t it = 0, tc = 0;
    bool ok = true;
    for (int w = w_begin, w_next; w < w_end && ok; w = w_next, ++tc) {
      int mb, nu, width;
      w_next = tile_at(w, mb, nu, width);
      const int ncols = width * UNIT;
      // the accumulator is free once the drain has read the previous tile out of it
      ok = mbar_wait_warp(bar(B_TEMPTY), (tc & 1) ^ 1, abort_flag, p.status, LQ_STAGE_MMA);
      if (!ok) break;
      tc_fence_after();
      LQ_TL(EV_M_ACC_FREE, 0);
      for (int s = 0; s < p.k_stages && ok; ++s, ++it) {
        const int st = it % NSTAGE;
        ok = mbar_wait_warp(bar(B_FULL + st), (it / NSTAGE) & 1, abort_flag, p.status, LQ_STAGE_MMA);
        if (!ok) break;
        tc_fence_after();
        LQ_TL(EV_M_STAGE_FULL, s);
        const uint32_t a_addr = sm_stage + st * STAGE_BYTES, b_addr = a_addr + STAGE_A_BYTES, sf_addr = sm_sf + st * STAGE_SF_BYTES;
        const uint64_t adesc = make_smem_desc(a_addr), bdesc = make_smem_desc(b_addr);
        const uint32_t tsfa = tmem_base + TM_SFA, tsfb = tmem_base + TM_SFB;
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
        LQ_TL(EV_M_ISSUED, s);
      }
      if (!ok) break;
      for (int bs = 0; bs < nbst && has_branch; ++bs) {
        const int st = it % NSTAGE;
        ok = mbar_wait_warp(bar(B_FULL + st), (it / NSTAGE) & 1, abort_flag, p.status, LQ_STAGE_MMA);
        if (!ok) break;
        if (branch_acc) {
          // the drain has read the previous tile's branch accumulator (long ago: it does that under this tile's main loop)
          ok = mbar_wait_warp(bar(B_BEMPTY), (tc & 1) ^ 1, abort_flag, p.status, LQ_STAGE_MMA);
          if (!ok) break;
        }
        tc_fence_after();
        const uint32_t a_addr = sm_stage + st * STAGE_BYTES, b_addr = a_addr + STAGE_A_BYTES;
        const uint64_t adesc = make_smem_desc(a_addr), bdesc = make_smem_desc(b_addr);
        if (elect_one()) {
          if (p.branch_mx) {
            const uint32_t sf_addr = sm_sf + st * STAGE_SF_BYTES, tsfa = tmem_base + TM_SFA, tsfb = tmem_base + TM_SFB;
            tc_cp_sf(tsfa, make_smem_desc_plain(sf_addr, 16, 128));
            tc_cp_sf(tsfb, make_smem_desc_plain(sf_addr + SF_BYTES, 16, 128));
            if (width == 2) tc_cp_sf(tsfb + 4, make_smem_desc_plain(sf_addr + 2 * SF_BYTES, 16, 128));
            if (p.branch_mx == 2) {
              for (int c = 0; c < p.branch_steps; ++c)
                for (int q = 0; q < 4; ++q) {
                  const int ja = c + 2 * (q >> 1), jb = c + 2 * (q & 1);   // K block of T's plane, of L2's plane
                  tc_mma_mx(tmem_base, adesc + 2 * ja, bdesc + 2 * jb, idesc_mx2(ncols, ja, jb), tsfa, tsfb, 1u);
                }
            } else {
              for (int j = 0; j < p.branch_steps; ++j)
                tc_mma_mx(tmem_base, adesc + 2 * j, bdesc + 2 * j, idesc_mx(ncols, j), tsfa, tsfb, 1u);
            }
          } else {
            for (int j = 0; j < p.branch_steps; ++j) {
              if (branch_acc) tc_mma<TC_I8>(tmem_base + TM_BR, adesc + 2 * j, bdesc + 2 * j, IDESC_I8 | idesc_shape(ncols), (uint32_t)j);
              else tc_mma<TC_F16>(tmem_base, adesc + 2 * j, bdesc + 2 * j, IDESC_F16 | idesc_shape(ncols), 1u);   // 16 halves each
            }
          }
          tc_commit(bar(B_EMPTY + st));
        }
        __syncwarp();
        ++it;
      }
      if (!ok) break;
      if (elect_one()) tc_commit(bar(B_TFULL));
      __syncwarp();
      LQ_TL(EV_TILE, 0);
    }
  } else {
    // ------------------------------------------------------------------ drain + epilogue
    const int quad = warp & 3;                          // tensor-memory lanes 32*quad .. 32*quad+31
    const int cgi = (warp - FIRST_DRAIN_WARP) >> 2;     // which 32 columns of each 128-column half
    const int g = lane >> 2, t = lane & 3;              // fragment coordinates: rows g and g + 8, column pair t
    const uint32_t tlane = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(cgi * 32);
    uint32_t tc = 0;
    bool ok = true;
    for (int w = w_begin, w_next; w < w_end && ok; w = w_next, ++tc) {
      int mb, nu, width;
      w_next = tile_at(w, mb, nu, width);
      const int m0 = mb * LQ_BM, n0 = nu * UNIT;
      const int rl = quad * 32 + g;                     // this thread's rows inside the tile: rl + 16 mt and + 8
      const int cl = cgi * 32;                          // this warp's columns inside a half: cl + 8 nt + ...
      const int rb = tc & 1;
      float acc[2][2][4][4];                            // [half][m16 tile][n8 tile][fragment register]
      uint32_t w0[2][8];                                // cgi == 0: the branch columns that the scale factors alias
      LQ_TL(EV_D_OPEN, 0);
      ok = mbar_wait_idle(bar(B_TFULL), tc & 1, abort_flag, p.status, LQ_STAGE_DRAIN);
      if (!ok) break;
      tc_fence_after();
      LQ_TL(EV_D_ACC_FULL, 0);
      // hand-over: every load is issued before the one wait; the main accumulator lands in the registers it stays in
#pragma unroll
      for (int h = 0; h < 2; ++h)
        if (h < width) {
#pragma unroll
          for (int mt = 0; mt < 2; ++mt)
            tmem_ld_16x256b_x4(tlane + ((uint32_t)(16 * mt) << 16) + h * UNIT, reinterpret_cast<uint32_t(&)[16]>(acc[h][mt]));
        }
      if (branch_acc && cgi == 0) {
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) tmem_ld_16x256b_x2(tlane + ((uint32_t)(16 * mt) << 16) + TM_BR, w0[mt]);
      }
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_TEMPTY));
      LQ_TL(EV_D_LOADED, 0);
      // y = main + U sT sL2 + bias, under the next tile's main loop (the tensor core has already applied the block
      // scales to main)
      ok = mbar_wait(bar(B_RFULL + rb), (tc >> 1) & 1, abort_flag, p.status, LQ_STAGE_DRAIN);
      if (!ok) break;
      {
        const float* sc = sc_ptr + rb * SC_FLOATS;
        const float* sc_l2 = sc + LQ_BM + cl + 2 * t;
        const float* sc_b = sc + LQ_BM + 2 * UNIT + cl + 2 * t;
        if (branch_acc && cgi == 0) {                  // the early-read columns first: their registers are free again
#pragma unroll
          for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
              combine_fragment(acc[0][mt][nt], &w0[mt][4 * nt], true, sc[rl + 16 * mt], sc[rl + 16 * mt + 8],
                               *reinterpret_cast<const float2*>(sc_l2 + nt * 8), *reinterpret_cast<const float2*>(sc_b + nt * 8));
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          if (h < width) {
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
              uint32_t w[16];
              const bool early = branch_acc && cgi == 0 && h == 0;       // fragments 0 and 1 are done already
              if (branch_acc) {
                const uint32_t ta = tlane + ((uint32_t)(16 * mt) << 16) + TM_BR + h * UNIT;
                if (early) tmem_ld_16x256b_x2(ta + TM_SF_ALIASED, reinterpret_cast<uint32_t(&)[8]>(w[8]));
                else tmem_ld_16x256b_x4(ta, w);
                tmem_ld_wait();
              }
              const float st_lo = sc[rl + 16 * mt], st_hi = sc[rl + 16 * mt + 8];
#pragma unroll
              for (int nt = 0; nt < 4; ++nt) {
                if (nt < 2 && early) continue;
                combine_fragment(acc[h][mt][nt], &w[4 * nt], branch_acc, st_lo, st_hi,
                                 *reinterpret_cast<const float2*>(sc_l2 + h * UNIT + nt * 8),
                                 *reinterpret_cast<const float2*>(sc_b + h * UNIT + nt * 8));
              }
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) { mbar_arrive(bar(B_BEMPTY)); mbar_arrive(bar(B_REMPTY + rb)); }
      LQ_TL(EV_D_DONE, 0);
      // epilogue
      const int row_w = m0 + quad * 32;                 // first row of this group's part
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        if (h < width) {
          if (p.out_f32) {
            float* Y = reinterpret_cast<float*>(p.Y);
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
              const int r_lo = row_w + g + 16 * mt, r_hi = r_lo + 8;
#pragma unroll
              for (int nt = 0; nt < 4; ++nt) {
                const int c = n0 + h * UNIT + cl + nt * 8 + 2 * t;
                if (c < p.N) {
                  if (r_lo < p.M) *reinterpret_cast<float2*>(Y + (size_t)r_lo * p.N + c) = make_float2(acc[h][mt][nt][0], acc[h][mt][nt][1]);
                  if (r_hi < p.M) *reinterpret_cast<float2*>(Y + (size_t)r_hi * p.N + c) = make_float2(acc[h][mt][nt][2], acc[h][mt][nt][3]);
                }
              }
            }
          } else {
            __half* Y = reinterpret_cast<__half*>(p.Y);
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
              // pack to fp16, then exchange inside the quad: lane t ends up with columns 8 t .. 8 t + 7 of both rows
              uint32_t lo[4], hi[4];
#pragma unroll
              for (int nt = 0; nt < 4; ++nt) {
                const __half2 l2 = __floats2half2_rn(acc[h][mt][nt][0], acc[h][mt][nt][1]);
                const __half2 h2 = __floats2half2_rn(acc[h][mt][nt][2], acc[h][mt][nt][3]);
                lo[nt] = *reinterpret_cast<const uint32_t*>(&l2);
                hi[nt] = *reinterpret_cast<const uint32_t*>(&h2);
              }
              quad_transpose(lo, t);
              quad_transpose(hi, t);
              // each lane owns 16 contiguous bytes of a row: a store instruction writes whole 32-byte sectors
              const int c = n0 + h * UNIT + cl + 8 * t;
              const int r_lo = row_w + g + 16 * mt, r_hi = r_lo + 8;
              if (c < p.N) {
                if (r_lo < p.M) *reinterpret_cast<uint4*>(Y + (size_t)r_lo * p.N + c) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                if (r_hi < p.M) *reinterpret_cast<uint4*>(Y + (size_t)r_hi * p.N + c) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
              }
            }
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

}  // namespace

lq_status lq_gemm_mx_prepare(int device) {
  if (cudaSetDevice(device) != cudaSuccess) return LQ_ERR_CUDA;
  if (lq_note_cuda(cudaFuncSetAttribute(lq_gemm_mx_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES)) !=
          cudaSuccess ||
      lq_note_cuda(cudaFuncSetAttribute(lq_gemm_mx_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES)) !=
      cudaSuccess)
    return LQ_ERR_CUDA;
  return LQ_OK;
}

lq_status lq_launch_gemm_mx(const lq_layer* L, const lq_act* A, void* Y, lq_out_dtype dt, cudaStream_t st) {
  if (cudaSetDevice(A->device) != cudaSuccess) return LQ_ERR_CUDA;
  if (!L->mx || !A->mx) return LQ_ERR_UNSUPPORTED;
  MxParams p;
  p.M = A->M; p.N = L->N; p.Mpad = A->Mpad; p.Npad = L->Npad;
  p.b_wrap = L->Kpad / LQ_KSTAGE;
  p.k_stages = p.b_wrap * A->planes;
  p.branch_f16 = L->f16_branch ? 1 : 0;
  p.branch_mx = L->r == 0 ? 0 : L->mxfp ? 1 : !L->a8 ? 0 : L->cfg.branch == LQ_BRANCH_MXINT4 ? 3 : 2;
  p.sft = A->d_sft; p.sfl2 = L->d_sfl2;
  p.branch_steps = L->r == 0 ? 0 : lq_ceil_div(L->r, L->f16_branch ? 16 : 32);   // a8: rank blocks of 32 (at most two)
  p.tiles_m = lq_ceil_div(A->M, LQ_BM);
  p.units_n = L->Npad / UNIT;
  p.sfa = A->d_sfa; p.sfb = L->d_sfb; p.sT = A->d_sT; p.sL2 = L->d_sL2; p.bias = L->d_bias;
  p.Y = Y; p.out_f32 = dt == LQ_OUT_F32 ? 1 : 0;
  p.status = lq_device_status_ptr(A->device);
  if (!p.status) return LQ_ERR_CUDA;
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, A->device) != cudaSuccess) return LQ_ERR_CUDA;
  int ctas = g_lq_gemm_ctas > 0 ? g_lq_gemm_ctas : sms;
  const long long tiles = (long long)p.tiles_m * ((p.units_n + 1) / 2);
  if (ctas > tiles) ctas = (int)tiles;
  p.by_units = (p.units_n & 1) && tiles < 4ll * ctas;
  cudaError_t launched;
  if (p.branch_steps > 0 && !p.branch_f16 && !p.branch_mx)
    launched = lq_launch(lq_gemm_mx_kernel<true>, ctas, GEMM_THREADS, SMEM_BYTES, st, A->tmA, L->tmB, L->tmB2, A->tmT, L->tmL2, p);
  else
    launched = lq_launch(lq_gemm_mx_kernel<false>, ctas, GEMM_THREADS, SMEM_BYTES, st, A->tmA, L->tmB, L->tmB2, A->tmT, L->tmL2, p);
  return lq_note_cuda(launched != cudaSuccess ? launched : cudaGetLastError()) == cudaSuccess ? LQ_OK : LQ_ERR_CUDA;
}
