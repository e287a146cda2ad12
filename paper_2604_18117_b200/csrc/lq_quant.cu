// Activation side of the layer, ONE kernel and one read of X from HBM (Figure 1; Appendix A.2: both branches
// consume quantized X, except the full-precision reference branch of Section 4.2 / Table 2):
//   a1  4-bit codes + scales per token and group of 64 along K (SINT4, Appendix A.3) or block of 32 (MXINT4)
//   a2  per-token codes of the low-rank branch (needs the whole row's maximum first)
//   a3  down-projection I1 = qb L1q, exact int32, on mma.sync (s8) - or T = X L1 in fp16 x fp16 -> fp32 for the
//       fp16 reference branch - straight from the registers that hold the freshly made codes
//   a4  t = fl32(fl32(I1) * fl32(sXb * sL1)), per-token re-quantization of the rank-r row
//
// Shape of the kernel: persistent CTAs walk 16-row tiles.  A tile arrives as TMA boxes of 16 rows x 64 values
// (128-byte swizzle); W consumer warps each own the boxes g = w, w + W, ... of a tile, and each has a private ring
// of D shared-memory slots with a full/empty mbarrier pair per slot, fed by one lane of the producer warp (lane w
// serves warp w: a slot is always filled and drained by the same pair, strictly in order, so a one-bit phase
// never aliases even though copies complete out of order).  A lane (gid, tig) of a consumer warp
// holds 16 consecutive values of rows gid and gid + 8 - exactly one operand fragment of the m16 MMA under a
// k order that A and B share (a sum over k does not care which k sits in which fragment slot), so the branch
// codes never touch shared memory.  With an integer branch a tile is walked twice (row maxima, then codes);
// when the ring holds a whole tile the second walk reads the same slots, otherwise the producer streams the
// tile a second time (served by the L2: DRAM still sees X once).
//
// Exactness contract: codes and scales equal the definition evaluated in IEEE binary32 with
// round-to-nearest-even and true division.  The kernel is division free:
//   scale     fp16(a / 7) == fp16(a * fl32(1/7)) for every finite fp16 a (checked exhaustively on the host),
//             because a/7 never comes closer than 2^-15 (relative) to an fp16 midpoint.
//   quotient  x / s from the correctly rounded reciprocal by one FMA correction step, which yields the correctly
//             rounded binary32 quotient (div_rn_by below); rounding to the nearest even integer by adding
//             1.5 * 2^23.  MXINT4: 1/s is a power of two, so x * (1/s) is already exact.
#include <cuda_fp16.h>

#include <algorithm>

#include "lq_device.cuh"

namespace {

using namespace lqdev;

constexpr int TR = 16;                 // rows per tile (one m16 MMA tile)
constexpr int BOX_K = 64;              // values of K per box: one 128-byte swizzle row
constexpr int BOX_BYTES = TR * BOX_K * 2;
constexpr float MAGIC = 12582912.0f;   // 1.5 * 2^23: adding it rounds to an integer (ties to even)
constexpr int MAX_CONSUMER_WARPS = 9;
enum { BR_NONE = 0, BR_INT = 1, BR_F16 = 2, BR_MXFP = 3, BR_MXINT = 4 };
// MXFP: MXFP8e4 activation codes for an MXFP4 weight; MXINT8: MXINT8 activation codes for an MXINT4 weight, stored as
// two E4M3 digit planes (code = 16 hi + lo)
enum { MAIN_SINT4 = 0, MAIN_MXINT4 = 1, MAIN_MXFP = 2, MAIN_MXINT8 = 3 };

struct QuantParams {
  int M, K, Kpad, Mpad;
  int G;                // scales per row that hold data: ceil(K / 64) (SINT4) or ceil(K / 32) (MXINT4)
  int nbox;             // Kpad / 64 boxes per tile (trailing ones may be all padding: their codes are zeros)
  int ntiles;           // ceil(M / 16)
  int depth;            // D: ring slots per consumer warp
  int refetch;          // 1: a warp's ring is smaller than its share of a tile, the producer streams every tile twice
  uint8_t* qx8;         // [Mpad][Kpad] (MXINT8: [Mpad][2 Kpad], the hi digits' plane then the lo digits')
  float* sx;            // [Gpad][Mpad]
  uint8_t* sfa;         // MXINT4: E8M0 scale bytes [Mpad/128][Kpad/128][512] (MXINT8: [Mpad/128][2 Kpad/128][512], by plane)
  int8_t* qb;           // [Mpad][Kpad] or null (not stored)
  float* sXb;           // [Mpad]
  const uint4* L1f;     // first factor in fragment order: [nbox][r tiles][32 lanes] x 16 bytes (int8) or 32 bytes (fp16)
  const float* sL1;     // [LQ_MAX_RANK]
  const float* s1b;     // MXFP: block scales 2^e of the first factor, [Kpad/32][rpad]
  uint8_t* sft;         // MXFP: E8M0 bytes of the rank-r intermediate's block scales, [Mpad/128][512]
  uint8_t* tq;          // [Mpad][LQ_RCONT]
  float* sT;            // [Mpad]
  int r, rpad;          // rank, rank rounded up to 8
  int tq_stride;        // bytes per row of tq: LQ_RCONT, or 2 LQ_RCONT when each digit plane of the intermediate has a container
  int act6;             // MXFP: the activations (X and the rank-r intermediate) are MXFP6e2 instead of MXFP8e4
  float qm;             // largest branch activation code
  int32_t* status;
};

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// two floats holding integers in [-7, 7] -> two E4M3 bytes (hi: first operand, lo: second)
__device__ __forceinline__ uint32_t f32x2_to_e4m3x2(float hi, float lo) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  return (uint32_t)r;
}

__device__ __forceinline__ void mma_s8_16832(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                             uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_e4m3_16832(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                               uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k32.row.col.f32.e4m3.e4m3.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_f16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                              uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// largest magnitude of 16 halves (two 16-byte vectors), exact in fp16
__device__ __forceinline__ __half absmax16(const uint4& a, const uint4& b) {
  const __half2* p = reinterpret_cast<const __half2*>(&a);
  const __half2* q = reinterpret_cast<const __half2*>(&b);
  __half2 m = __hmax2(__hmax2(__habs2(p[0]), __habs2(p[1])), __hmax2(__habs2(p[2]), __habs2(p[3])));
  m = __hmax2(m, __hmax2(__hmax2(__habs2(q[0]), __habs2(q[1])), __hmax2(__habs2(q[2]), __habs2(q[3]))));
  return __hmax(__low2half(m), __high2half(m));
}

__device__ __forceinline__ __half absmax8(const uint4& a) {
  const __half2* p = reinterpret_cast<const __half2*>(&a);
  const __half2 m = __hmax2(__hmax2(__habs2(p[0]), __habs2(p[1])), __hmax2(__habs2(p[2]), __habs2(p[3])));
  return __hmax(__low2half(m), __high2half(m));
}

// MXFP8e4 / MXFP6e2 of eight values that share a block (Appendix A.3 "MX Formats"; conversion of the OCP specification
// the paper cites): the block's exponent is e = floor(log2 a) - emax for the block maximum a (emax = 8: e4m3's largest
// binade, 2: e2m3's), -127 for an all-zero block; the elements are x / 2^e - exact - rounded to the element format by
// the hardware conversion (nearest even, magnitudes above the largest normal clamped).  Every e2m3 value is an e4m3
// value, so both formats are stored, and multiplied, as e4m3 bytes: the 6-bit path rounds to e2m3 first and widens
// the result (e2m3 -> f16 -> e4m3, both exact).
__device__ __forceinline__ int mxfp8_exponent(float a, bool six = false) {
  const int e = (int)(__float_as_uint(a) >> 23) - 127 - (six ? 2 : 8);
  return (a > 0.f && e >= -126) ? e : -127;
}
__device__ __forceinline__ uint32_t f32x2_to_e4m3x2_via_e2m3(float hi, float lo) {
  uint16_t r6, r8;
  uint32_t h2;
  asm("cvt.rn.satfinite.e2m3x2.f32 %0, %1, %2;" : "=h"(r6) : "f"(hi), "f"(lo));
  asm("cvt.rn.f16x2.e2m3x2 %0, %1;" : "=r"(h2) : "h"(r6));
  asm("cvt.rn.satfinite.e4m3x2.f16x2 %0, %1;" : "=h"(r8) : "r"(h2));
  return (uint32_t)r8;
}
__device__ __forceinline__ uint32_t mxfp_pair(float hi, float lo, bool six) {
  return six ? f32x2_to_e4m3x2_via_e2m3(hi, lo) : f32x2_to_e4m3x2(hi, lo);
}
__device__ __forceinline__ uint2 mxfp8_codes8(const uint4& v, int e, bool six = false) {
  const __half2* h2 = reinterpret_cast<const __half2*>(&v);
  const float inv = e == -127 ? 0.f : __uint_as_float((uint32_t)(127 - e) << 23);
  float x[8];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 f = __half22float2(h2[i]);
    x[2 * i] = f.x * inv; x[2 * i + 1] = f.y * inv;
  }
  uint2 w;
  w.x = mxfp_pair(x[1], x[0], six) | (mxfp_pair(x[3], x[2], six) << 16);
  w.y = mxfp_pair(x[5], x[4], six) | (mxfp_pair(x[7], x[6], six) << 16);
  return w;
}
// 2^e as a float (0 for the all-zero block's -127: its codes are zeros anyway)
__device__ __forceinline__ float pow2f(int e) { return e <= -127 ? 0.f : __uint_as_float((uint32_t)(e + 127) << 23); }

// MXINT8 (Appendix A.3 "MX Formats": signed 8-bit codes, blocks of 32, power-of-two scale): the block's exponent is the
// smallest e with 127 * 2^e >= a for the block maximum a = 1.f * 2^E: e = E - 6 if 1.f <= 127/64, else E - 5; at
// least -127, and -127 for an all-zero block.
__device__ __forceinline__ int mxint8_exponent(float a) {
  const uint32_t ab = __float_as_uint(a);
  const int e = (int)(ab >> 23) - 127 - (((ab & 0x7FFFFFu) <= 0x7E0000u) ? 6 : 5);
  return a > 0.f ? max(e, -127) : -127;
}
// One value under the block's exponent: the code c = rint_even(x / 2^e) (the division is exact), as the int8 byte the
// down-projection multiplies and as two digits c = 16 hi + lo, lo in [-8, 7], hi in [-8, 8], both exact E4M3 values.
struct Code8 { float hi, lo; uint32_t byte; };
__device__ __forceinline__ Code8 mxint8_code(float x, float inv) {
  const float t = __fmaf_rn(x, inv, MAGIC);
  const float c = __fadd_rn(t, -MAGIC);
  Code8 r;
  r.byte = __float_as_uint(t) & 0xFFu;                 // the low byte of (c + MAGIC)'s bit pattern is c
  r.hi = floorf(__fmul_rn(__fadd_rn(c, 8.f), 0.0625f));
  r.lo = __fmaf_rn(r.hi, -16.f, c);
  return r;
}
// eight values of one block (one 16-byte vector of halves): the E4M3 bytes of the hi and lo digits and the int8 codes
__device__ __forceinline__ void mxint8_codes8(const uint4& v, int e, uint2& hi, uint2& lo, uint2& s8) {
  const __half2* h2 = reinterpret_cast<const __half2*>(&v);
  const float inv = e == -127 ? 0.f : __uint_as_float((uint32_t)(127 - e) << 23);
  Code8 c[8];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 f = __half22float2(h2[i]);
    c[2 * i] = mxint8_code(f.x, inv); c[2 * i + 1] = mxint8_code(f.y, inv);
  }
  hi.x = f32x2_to_e4m3x2(c[1].hi, c[0].hi) | (f32x2_to_e4m3x2(c[3].hi, c[2].hi) << 16);
  hi.y = f32x2_to_e4m3x2(c[5].hi, c[4].hi) | (f32x2_to_e4m3x2(c[7].hi, c[6].hi) << 16);
  lo.x = f32x2_to_e4m3x2(c[1].lo, c[0].lo) | (f32x2_to_e4m3x2(c[3].lo, c[2].lo) << 16);
  lo.y = f32x2_to_e4m3x2(c[5].lo, c[4].lo) | (f32x2_to_e4m3x2(c[7].lo, c[6].lo) << 16);
  s8.x = c[0].byte | (c[1].byte << 8) | (c[2].byte << 16) | (c[3].byte << 24);
  s8.y = c[4].byte | (c[5].byte << 8) | (c[6].byte << 16) | (c[7].byte << 24);
}

// Correctly rounded quotient a / b in binary32 from the correctly rounded reciprocal y = fl32(1/b), division free:
// q0 = fl32(a y) is within one ulp of a / b, r = a - b q0 is exact in an FMA, and fl32(q0 + r y) is then the
// correctly rounded quotient (Markstein's correction step).  Operands here are far from overflow and underflow.
__device__ __forceinline__ float div_rn_by(float a, float b, float y) {
  const float q0 = __fmul_rn(a, y);
  const float r = __fmaf_rn(-q0, b, a);
  return __fmaf_rn(r, y, q0);
}

// Scale of one group for a1.  `a` is the maximum magnitude of the whole group (SINT4: 64 values, MXINT4: 32),
// already reduced over the lanes that share it.
struct MainScale {
  float s;       // SINT4: the fp16 scale as a float
  float inv;     // fl32(1/s) (MXINT4: 2^-e, exact)
  int e;         // MXINT4: block exponent
  bool coarse;   // SINT4: subnormal scale, the quotient may exceed 7.5 and has to be clamped
};
template <bool MX>
__device__ __forceinline__ MainScale main_scale(float a) {
  MainScale m;
  if constexpr (MX) {
    // 2^e with e the smallest integer such that 7 * 2^e >= a: a = 1.f * 2^E, e = E - 2 if 1.f <= 1.75 else E - 1
    const uint32_t ab = __float_as_uint(a);
    m.e = -127;
    if (a > 0.f) m.e = (int)(ab >> 23) - 127 - (((ab & 0x7FFFFFu) <= 0x600000u) ? 2 : 1);
    m.inv = __uint_as_float((uint32_t)(127 - (a > 0.f ? m.e : 0)) << 23);
    m.s = 0.f;
    m.coarse = false;
  } else {
    __half s16 = __float2half_rn(__fmul_rn(a, 0.142857149243354797f));   // fl32(1/7)
    const unsigned short sbits = __half_as_ushort(s16);
    if (sbits == 0) s16 = __ushort_as_half((unsigned short)1);            // floor 2^-24
    m.s = __half2float(s16);
    m.inv = __frcp_rn(m.s);
    m.coarse = sbits < 0x0400;
    m.e = 0;
  }
  return m;
}

// a1 and a2 for eight consecutive values of one row (one 16-byte vector of halves).
//   main    SINT4: the correctly rounded quotient x / s, then round-to-nearest-even by the magic constant - the
//           definition itself; |x| / s <= 7 (1 + 2^-11) for a normal fp16 scale, so only a subnormal (coarse) scale
//           needs the clamp.  MXINT4: 1/s is a power of two, x * (1/s) is exact.
//   branch  int8 codes under the row's scale sb, invb = fl32(1/sb); |x| / sb <= qm (1 + 2^-23), so the rounded quotient
//           never leaves [-qm, qm].  The low byte of (code + MAGIC)'s bit pattern is the code.
// Returns the 8 operand bytes of the main codes (E4M3 images) and the 8 branch code bytes.
template <bool MX, bool BRANCH>
__device__ __forceinline__ void quant8(const uint4& v, const MainScale& ms, float sb, float invb, uint2& w, uint2& b) {
  const __half2* h2 = reinterpret_cast<const __half2*>(&v);
  float x[8], q[8];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 f = __half22float2(h2[i]);
    x[2 * i] = f.x; x[2 * i + 1] = f.y;
  }
  if constexpr (MX) {
#pragma unroll
    for (int i = 0; i < 8; ++i) q[i] = __fadd_rn(__fmaf_rn(x[i], ms.inv, MAGIC), -MAGIC);
  } else {
#pragma unroll
    for (int i = 0; i < 8; ++i) q[i] = __fadd_rn(__fadd_rn(div_rn_by(x[i], ms.s, ms.inv), MAGIC), -MAGIC);
    if (ms.coarse) {
#pragma unroll
      for (int i = 0; i < 8; ++i) q[i] = fminf(fmaxf(q[i], -7.f), 7.f);
    }
  }
  w.x = f32x2_to_e4m3x2(q[1], q[0]) | (f32x2_to_e4m3x2(q[3], q[2]) << 16);
  w.y = f32x2_to_e4m3x2(q[5], q[4]) | (f32x2_to_e4m3x2(q[7], q[6]) << 16);
  if constexpr (BRANCH) {
    uint32_t t[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) t[i] = __float_as_uint(__fadd_rn(div_rn_by(x[i], sb, invb), MAGIC));
    b.x = __byte_perm(__byte_perm(t[0], t[1], 0x0040), __byte_perm(t[2], t[3], 0x0040), 0x5410);
    b.y = __byte_perm(__byte_perm(t[4], t[5], 0x0040), __byte_perm(t[6], t[7], 0x0040), 0x5410);
  }
}

// CTA-wide rendezvous of the consumer warps on an mbarrier (count = number of consumer warps), bounded like every wait
__device__ __forceinline__ bool consumers_sync(uint32_t bar, uint32_t parity, int lane, volatile int* abort_flag,
                                               int32_t* status) {
  __syncwarp();
  if (lane == 0) mbar_arrive(bar);
  return mbar_wait(bar, parity, abort_flag, status, LQ_STAGE_QUANT);
}

// Shared memory (dynamic), from a 1024-byte aligned base:
//   ring      W x D boxes of 2 KB
//   bars      full[W D], empty[W D], syncA, syncB, syncC
//   red       BR_INT: int I1[2][16][rpad]; BR_F16: float part[W][16][rpad]
//   rowmax    int[2][16] (bit patterns of non-negative floats)
//   abort     int
// Instances for rank > 32 (NTR >= 8) hold 32 or more accumulator and as many fragment registers per thread: compiled
// for two CTAs per SM (96 registers) they spill, so they are compiled for one (measured: rank 64 10-33 % faster,
// rank 128 10-20 %); the launch planner picks the residency from the register count it reads back.
template <int MAIN, int BR, int NTR>   // NTR: 8-column tiles of the rank (rank <= 8 NTR)
__global__ void __launch_bounds__((MAX_CONSUMER_WARPS + 1) * 32, NTR >= 8 ? 1 : 2) lq_quant_kernel(const __grid_constant__ CUtensorMap tmX,
                                                                                 const QuantParams p) {
  constexpr bool MX = MAIN == MAIN_MXINT4;
  constexpr bool I8 = MAIN == MAIN_MXINT8;
  constexpr bool FP = MAIN == MAIN_MXFP || I8;             // lanes hold eight values from each of a box's two blocks
  constexpr bool FACC = BR == BR_F16 || BR == BR_MXFP || BR == BR_MXINT;     // fp32 partial sums of the down-projection
  extern __shared__ uint8_t qsm_raw[];
  const uint32_t base = (smem_u32(qsm_raw) + 1023u) & ~1023u;
  uint8_t* smem = qsm_raw + (base - smem_u32(qsm_raw));
  const int W = (int)(blockDim.x >> 5) - 1;                 // consumer warps; warp W is the producer
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);
  const int lane = threadIdx.x & 31;
  const int gid = lane >> 2, tig = lane & 3;
  const int nslot = W * p.depth;
  const uint32_t ring = base;
  const uint32_t bars = base + (uint32_t)nslot * BOX_BYTES;
  auto bar_full = [&](int s) { return bars + 8u * (uint32_t)s; };
  auto bar_empty = [&](int s) { return bars + 8u * (uint32_t)(nslot + s); };
  const uint32_t bar_sync = bars + 16u * (uint32_t)nslot;   // three rendezvous barriers
  uint8_t* red_ptr = smem + (size_t)nslot * BOX_BYTES + 16 * (size_t)nslot + 32;
  int* I1_s = reinterpret_cast<int*>(red_ptr);
  float* part_s = reinterpret_cast<float*>(red_ptr);
  const size_t red_bytes = BR == BR_INT ? (size_t)2 * TR * p.rpad * 4 : FACC ? (size_t)W * TR * p.rpad * 4 : 0;
  int* rowmax_s = reinterpret_cast<int*>(red_ptr + red_bytes);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(rowmax_s + 2 * TR);

  if (threadIdx.x == 0) {
    for (int s = 0; s < nslot; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_empty(s), 1); }
    for (int b = 0; b < 3; ++b) mbar_init(bar_sync + 8u * b, (uint32_t)W);
    *abort_flag = 0;
    mbar_init_fence();
  }
  if constexpr (BR == BR_INT) {
    for (int i = threadIdx.x; i < 2 * TR * p.rpad; i += blockDim.x) I1_s[i] = 0;
    if (threadIdx.x < 2 * TR) rowmax_s[threadIdx.x] = 0;
  }
  __syncthreads();
  grid_dependency_sync();        // set-up done; from here on X is read and the activation record written

  const int passes = (BR == BR_INT && p.refetch) ? 2 : 1;   // how often the producer streams a tile

  if (warp == W) {
    // ------------------------------------------------------------------ TMA producer: lane w feeds consumer warp w
    if (lane < W) {
      const int s0 = lane * p.depth;
      int idx = 0;
      uint32_t phase = 0, issued = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < p.ntiles && ok; tile += gridDim.x) {
        const int m0 = tile * TR;
        for (int ps = 0; ps < passes && ok; ++ps) {
          for (int g = lane; g < p.nbox; g += W) {
            ok = mbar_wait(bar_empty(s0 + idx), phase ^ 1, abort_flag, p.status, LQ_STAGE_PRODUCER);
            if (!ok) break;
            mbar_expect_tx(bar_full(s0 + idx), BOX_BYTES);
            tma_load_2d(ring + (uint32_t)(s0 + idx) * BOX_BYTES, &tmX, g * BOX_K, m0, bar_full(s0 + idx));
            ++issued;
            if (++idx == p.depth) { idx = 0; phase ^= 1; }
          }
        }
      }
      if (!ok) {
        // aborting: let the copies already issued land before the CTA's shared memory goes away
        const uint32_t n = issued < (uint32_t)p.depth ? issued : (uint32_t)p.depth;
        for (uint32_t i = 0; i < n; ++i) {
          if (--idx < 0) { idx = p.depth - 1; phase ^= 1; }
          mbar_settle(bar_full(s0 + idx), phase);
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ consumers
    // box sequence of this warp: boxes w, w + W, ... of every pass of every tile, through its own ring
    const int s0 = warp * p.depth;
    int idx = 0;
    uint32_t phase = 0;
    auto advance = [&]() {
      if (++idx == p.depth) { idx = 0; phase ^= 1; }
    };
    // this lane's two 16-byte chunks of a swizzled 128-byte row; rows gid and gid + 8 share the swizzle phase
    const uint32_t row_off = (uint32_t)gid * 128u;
    // (MXFP: one 16-byte chunk from each of the box's two blocks of 32 instead: values 8 tig .. and 32 + 8 tig ..)
    const uint32_t c0 = (uint32_t)((FP ? tig : 2 * tig) ^ (gid & 7)) << 4, c1 = (uint32_t)((FP ? 4 + tig : 2 * tig + 1) ^ (gid & 7)) << 4;
    uint32_t sync_par = 0;
    uint32_t tcount = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < p.ntiles && ok; tile += gridDim.x, ++tcount) {
      const int m0 = tile * TR;
      const int par = (int)(tcount & 1);
      const int m_lo = m0 + gid, m_hi = m0 + gid + 8;
      const bool v_lo = m_lo < p.M, v_hi = m_hi < p.M;
      uint8_t* const qx_lo = p.qx8 + (size_t)m_lo * p.Kpad + 16 * tig;   // this lane's bytes of a row start here
      uint8_t* const qx_hi = qx_lo + (size_t)8 * p.Kpad;
      float sb_lo = 1.f, sb_hi = 1.f, invb_lo = 1.f, invb_hi = 1.f;
      // ---- walk 1 (integer branch only): the rows' maxima
      if constexpr (BR == BR_INT) {
        const int idx0 = idx;
        const uint32_t phase0 = phase;
        __half2 hm = __float2half2_rn(0.f);                 // (row gid, row gid + 8)
        for (int g = warp; g < p.nbox; g += W) {
          ok = mbar_wait(bar_full(s0 + idx), phase, abort_flag, p.status, LQ_STAGE_QUANT);
          if (!ok) break;
          const uint8_t* bx = smem + (size_t)(s0 + idx) * BOX_BYTES + row_off;
          const uint4 l0 = *reinterpret_cast<const uint4*>(bx + c0), l1 = *reinterpret_cast<const uint4*>(bx + c1);
          const uint4 h0 = *reinterpret_cast<const uint4*>(bx + 1024 + c0), h1 = *reinterpret_cast<const uint4*>(bx + 1024 + c1);
          hm = __hmax2(hm, __halves2half2(absmax16(l0, l1), absmax16(h0, h1)));
          if (p.refetch) {
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty(s0 + idx));
          }
          advance();
        }
        if (!ok) break;
        if (!p.refetch) { idx = idx0; phase = phase0; }     // the second walk reads the same slots
        hm = __hmax2(hm, __shfl_xor_sync(0xffffffffu, hm, 1));
        hm = __hmax2(hm, __shfl_xor_sync(0xffffffffu, hm, 2));
        if (tig == 0) {
          atomicMax(&rowmax_s[par * TR + gid], __float_as_int(__low2float(hm)));
          atomicMax(&rowmax_s[par * TR + gid + 8], __float_as_int(__high2float(hm)));
        }
        ok = consumers_sync(bar_sync, sync_par, lane, abort_flag, p.status);
        if (!ok) break;
        if (threadIdx.x < TR) rowmax_s[(par ^ 1) * TR + threadIdx.x] = 0;     // the other buffer: next tile's
        const float rm_lo = __int_as_float(rowmax_s[par * TR + gid]), rm_hi = __int_as_float(rowmax_s[par * TR + gid + 8]);
        sb_lo = (rm_lo == 0.f) ? 1.0f : __fdiv_rn(rm_lo, p.qm);
        sb_hi = (rm_hi == 0.f) ? 1.0f : __fdiv_rn(rm_hi, p.qm);
        invb_lo = __frcp_rn(sb_lo); invb_hi = __frcp_rn(sb_hi);
        if (warp == 0 && tig == 0) {
          if (v_lo) p.sXb[m_lo] = sb_lo;
          if (v_hi) p.sXb[m_hi] = sb_hi;
        }
      }
      // ---- walk 2: codes, scales, down-projection
      int acci[BR == BR_INT ? NTR : 1][4];
      float accf[FACC ? NTR : 1][4];
#pragma unroll
      for (int a = 0; a < NTR; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) {
          if constexpr (BR == BR_INT) acci[a][b] = 0;
          if constexpr (FACC) accf[a][b] = 0.f;
        }
      {
        // First-factor fragments (read-only, shared by all CTAs, L2 resident) travel one box ahead of their use: the
        // load of box g + W is in flight while box g is quantized.  FRAGV: 16-byte vectors per lane and column tile.
        constexpr int FRAGV = BR == BR_F16 ? 2 : 1;
        uint4 bfrag[BR == BR_NONE ? 1 : NTR * FRAGV];
        auto load_frags = [&](int g) {
          if constexpr (BR != BR_NONE) {
            const uint4* src = p.L1f + ((size_t)g * NTR * 32 + lane) * FRAGV;
#pragma unroll
            for (int i = 0; i < NTR * FRAGV; ++i) bfrag[i] = __ldg(src + (size_t)(i / FRAGV) * 32 * FRAGV + (i % FRAGV));
          }
        };
        if (warp < p.nbox) load_frags(warp);
        for (int g = warp; g < p.nbox; g += W) {
          ok = mbar_wait(bar_full(s0 + idx), phase, abort_flag, p.status, LQ_STAGE_QUANT);
          if (!ok) break;
          const uint8_t* bx = smem + (size_t)(s0 + idx) * BOX_BYTES + row_off;
          const uint4 l0 = *reinterpret_cast<const uint4*>(bx + c0), l1 = *reinterpret_cast<const uint4*>(bx + c1);
          const uint4 h0 = *reinterpret_cast<const uint4*>(bx + 1024 + c0), h1 = *reinterpret_cast<const uint4*>(bx + 1024 + c1);
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_empty(s0 + idx));   // the values are in registers: the slot may be refilled
          advance();
          const size_t koff = (size_t)(g * BOX_K);             // this box's first value of a row
          if constexpr (FP) {
            // l0 / h0: eight values of block 2g, l1 / h1: of block 2g + 1; a block's maximum lives in four lanes
            float a00 = __half2float(absmax8(l0)), a01 = __half2float(absmax8(l1));
            float a10 = __half2float(absmax8(h0)), a11 = __half2float(absmax8(h1));
#pragma unroll
            for (int o = 1; o <= 2; o <<= 1) {
              a00 = fmaxf(a00, __shfl_xor_sync(0xffffffffu, a00, o)); a01 = fmaxf(a01, __shfl_xor_sync(0xffffffffu, a01, o));
              a10 = fmaxf(a10, __shfl_xor_sync(0xffffffffu, a10, o)); a11 = fmaxf(a11, __shfl_xor_sync(0xffffffffu, a11, o));
            }
            if constexpr (I8) {
              const int e00 = mxint8_exponent(a00), e01 = mxint8_exponent(a01), e10 = mxint8_exponent(a10), e11 = mxint8_exponent(a11);
              uint2 h00, h01, h10, h11, d00, d01, d10, d11, s00, s01, s10, s11;   // hi digits, lo digits, int8 codes
              mxint8_codes8(l0, e00, h00, d00, s00); mxint8_codes8(l1, e01, h01, d01, s01);
              mxint8_codes8(h0, e10, h10, d10, s10); mxint8_codes8(h1, e11, h11, d11, s11);
              const size_t xs = (size_t)2 * p.Kpad;                // bytes per row: the hi plane, then the lo plane
              uint8_t* q_lo = p.qx8 + (size_t)m_lo * xs + koff + 8 * tig;
              uint8_t* q_hi = q_lo + (size_t)8 * xs;
              if (v_lo) {
                *reinterpret_cast<uint2*>(q_lo) = h00; *reinterpret_cast<uint2*>(q_lo + 32) = h01;
                *reinterpret_cast<uint2*>(q_lo + p.Kpad) = d00; *reinterpret_cast<uint2*>(q_lo + p.Kpad + 32) = d01;
              }
              if (v_hi) {
                *reinterpret_cast<uint2*>(q_hi) = h10; *reinterpret_cast<uint2*>(q_hi + 32) = h11;
                *reinterpret_cast<uint2*>(q_hi + p.Kpad) = d10; *reinterpret_cast<uint2*>(q_hi + p.Kpad + 32) = d11;
              }
              if (tig == 0) {
                const int kb = 2 * g;                            // blocks kb, kb + 1 share a 4-block scale chunk
                const size_t ks = (size_t)(p.Kpad >> 7);         // K stages per plane
                if (kb < p.G) {
                  if (v_lo) {
                    uint8_t* sf = p.sfa + ((size_t)(m_lo >> 7) * 2 * ks + (kb >> 2)) * 512 + 16 * (m_lo & 31) + 4 * ((m_lo & 127) >> 5) + (kb & 3);
                    sf[0] = (uint8_t)(e00 + 4 + 127); sf[ks * 512] = (uint8_t)(e00 + 127);
                    if (kb + 1 < p.G) { sf[1] = (uint8_t)(e01 + 4 + 127); sf[ks * 512 + 1] = (uint8_t)(e01 + 127); }
                  }
                  if (v_hi) {
                    uint8_t* sf = p.sfa + ((size_t)(m_hi >> 7) * 2 * ks + (kb >> 2)) * 512 + 16 * (m_hi & 31) + 4 * ((m_hi & 127) >> 5) + (kb & 3);
                    sf[0] = (uint8_t)(e10 + 4 + 127); sf[ks * 512] = (uint8_t)(e10 + 127);
                    if (kb + 1 < p.G) { sf[1] = (uint8_t)(e11 + 4 + 127); sf[ks * 512 + 1] = (uint8_t)(e11 + 127); }
                  }
                }
              }
              if constexpr (BR == BR_MXINT) {
                // a3: per block of 32 one exact integer MMA step on the codes just made, then the block's two power-of-two
                // scales in fp32 (|partial| <= 32 * 127 * 127 < 2^24: the conversion is exact)
                const float sa00 = pow2f(e00), sa01 = pow2f(e01), sa10 = pow2f(e10), sa11 = pow2f(e11);
#pragma unroll
                for (int nt = 0; nt < NTR; ++nt) {
                  const float2 sb0 = __ldg(reinterpret_cast<const float2*>(p.s1b + (size_t)(2 * g) * p.rpad + nt * 8 + 2 * tig));
                  const float2 sb1 = __ldg(reinterpret_cast<const float2*>(p.s1b + (size_t)(2 * g + 1) * p.rpad + nt * 8 + 2 * tig));
                  int i0[4] = {0, 0, 0, 0}, i1[4] = {0, 0, 0, 0};
                  mma_s8_16832(i0, s00.x, s10.x, s00.y, s10.y, bfrag[nt].x, bfrag[nt].y);
                  mma_s8_16832(i1, s01.x, s11.x, s01.y, s11.y, bfrag[nt].z, bfrag[nt].w);
                  accf[nt][0] = fmaf(__int2float_rn(i0[0]), sa00 * sb0.x, fmaf(__int2float_rn(i1[0]), sa01 * sb1.x, accf[nt][0]));
                  accf[nt][1] = fmaf(__int2float_rn(i0[1]), sa00 * sb0.y, fmaf(__int2float_rn(i1[1]), sa01 * sb1.y, accf[nt][1]));
                  accf[nt][2] = fmaf(__int2float_rn(i0[2]), sa10 * sb0.x, fmaf(__int2float_rn(i1[2]), sa11 * sb1.x, accf[nt][2]));
                  accf[nt][3] = fmaf(__int2float_rn(i0[3]), sa10 * sb0.y, fmaf(__int2float_rn(i1[3]), sa11 * sb1.y, accf[nt][3]));
                }
              }
              if (g + W < p.nbox) load_frags(g + W);
              continue;
            }
            const bool six = p.act6 != 0;
            const int e00 = mxfp8_exponent(a00, six), e01 = mxfp8_exponent(a01, six), e10 = mxfp8_exponent(a10, six), e11 = mxfp8_exponent(a11, six);
            const uint2 w00 = mxfp8_codes8(l0, e00, six), w01 = mxfp8_codes8(l1, e01, six);
            const uint2 w10 = mxfp8_codes8(h0, e10, six), w11 = mxfp8_codes8(h1, e11, six);
            uint8_t* q_lo = p.qx8 + (size_t)m_lo * p.Kpad + koff + 8 * tig;
            uint8_t* q_hi = q_lo + (size_t)8 * p.Kpad;
            if (v_lo) { *reinterpret_cast<uint2*>(q_lo) = w00; *reinterpret_cast<uint2*>(q_lo + 32) = w01; }
            if (v_hi) { *reinterpret_cast<uint2*>(q_hi) = w10; *reinterpret_cast<uint2*>(q_hi + 32) = w11; }
            if (tig == 0) {
              const int kb = 2 * g;                            // blocks kb, kb + 1 share a 4-block scale chunk
              if (kb < p.G) {
                if (v_lo) {
                  uint8_t* sf = p.sfa + ((size_t)(m_lo >> 7) * (p.Kpad >> 7) + (kb >> 2)) * 512 + 16 * (m_lo & 31) + 4 * ((m_lo & 127) >> 5) + (kb & 3);
                  sf[0] = (uint8_t)(e00 + 127);
                  if (kb + 1 < p.G) sf[1] = (uint8_t)(e01 + 127);
                }
                if (v_hi) {
                  uint8_t* sf = p.sfa + ((size_t)(m_hi >> 7) * (p.Kpad >> 7) + (kb >> 2)) * 512 + 16 * (m_hi & 31) + 4 * ((m_hi & 127) >> 5) + (kb & 3);
                  sf[0] = (uint8_t)(e10 + 127);
                  if (kb + 1 < p.G) sf[1] = (uint8_t)(e11 + 127);
                }
              }
            }
            if constexpr (BR == BR_MXFP) {
              // a3: per block of 32 one MMA step on the codes just made (their bytes ARE the A fragments), the block's
              // two power-of-two scales applied to its partial sums in fp32
              const float sa00 = pow2f(e00), sa01 = pow2f(e01), sa10 = pow2f(e10), sa11 = pow2f(e11);
#pragma unroll
              for (int nt = 0; nt < NTR; ++nt) {
                const float2 sb0 = __ldg(reinterpret_cast<const float2*>(p.s1b + (size_t)(2 * g) * p.rpad + nt * 8 + 2 * tig));
                const float2 sb1 = __ldg(reinterpret_cast<const float2*>(p.s1b + (size_t)(2 * g + 1) * p.rpad + nt * 8 + 2 * tig));
                float f0[4] = {0.f, 0.f, 0.f, 0.f}, f1[4] = {0.f, 0.f, 0.f, 0.f};
                mma_e4m3_16832(f0, w00.x, w10.x, w00.y, w10.y, bfrag[nt].x, bfrag[nt].y);
                mma_e4m3_16832(f1, w01.x, w11.x, w01.y, w11.y, bfrag[nt].z, bfrag[nt].w);
                accf[nt][0] = fmaf(f0[0], sa00 * sb0.x, fmaf(f1[0], sa01 * sb1.x, accf[nt][0]));
                accf[nt][1] = fmaf(f0[1], sa00 * sb0.y, fmaf(f1[1], sa01 * sb1.y, accf[nt][1]));
                accf[nt][2] = fmaf(f0[2], sa10 * sb0.x, fmaf(f1[2], sa11 * sb1.x, accf[nt][2]));
                accf[nt][3] = fmaf(f0[3], sa10 * sb0.y, fmaf(f1[3], sa11 * sb1.y, accf[nt][3]));
              }
            }
            if (g + W < p.nbox) load_frags(g + W);
            continue;
          }
          uint4 w_lo, w_hi, b_lo = make_uint4(0, 0, 0, 0), b_hi = make_uint4(0, 0, 0, 0);
          // group maxima: 64 values = four lanes (SINT4), 32 values = two lanes (MXINT4)
          float a_lo = __half2float(absmax16(l0, l1)), a_hi = __half2float(absmax16(h0, h1));
          a_lo = fmaxf(a_lo, __shfl_xor_sync(0xffffffffu, a_lo, 1));
          a_hi = fmaxf(a_hi, __shfl_xor_sync(0xffffffffu, a_hi, 1));
          if constexpr (!MX) {
            a_lo = fmaxf(a_lo, __shfl_xor_sync(0xffffffffu, a_lo, 2));
            a_hi = fmaxf(a_hi, __shfl_xor_sync(0xffffffffu, a_hi, 2));
          }
          const MainScale ms_lo = main_scale<MX>(a_lo), ms_hi = main_scale<MX>(a_hi);
          {
            uint2 w, b;
            quant8<MX, BR == BR_INT>(l0, ms_lo, sb_lo, invb_lo, w, b);
            w_lo.x = w.x; w_lo.y = w.y; b_lo.x = b.x; b_lo.y = b.y;
            quant8<MX, BR == BR_INT>(l1, ms_lo, sb_lo, invb_lo, w, b);
            w_lo.z = w.x; w_lo.w = w.y; b_lo.z = b.x; b_lo.w = b.y;
          }
          {
            uint2 w, b;
            quant8<MX, BR == BR_INT>(h0, ms_hi, sb_hi, invb_hi, w, b);
            w_hi.x = w.x; w_hi.y = w.y; b_hi.x = b.x; b_hi.y = b.y;
            quant8<MX, BR == BR_INT>(h1, ms_hi, sb_hi, invb_hi, w, b);
            w_hi.z = w.x; w_hi.w = w.y; b_hi.z = b.x; b_hi.w = b.y;
          }
          const float s_lo = ms_lo.s, s_hi = ms_hi.s;
          const int e_lo = ms_lo.e, e_hi = ms_hi.e;
          // stores: 16 operand bytes per row and lane (64 contiguous bytes per row and box)
          if (v_lo) {
            *reinterpret_cast<uint4*>(qx_lo + koff) = w_lo;
            if (BR == BR_INT && p.qb != nullptr) *reinterpret_cast<uint4*>(p.qb + (qx_lo - p.qx8) + koff) = b_lo;
          }
          if (v_hi) {
            *reinterpret_cast<uint4*>(qx_hi + koff) = w_hi;
            if (BR == BR_INT && p.qb != nullptr) *reinterpret_cast<uint4*>(p.qb + (qx_hi - p.qx8) + koff) = b_hi;
          }
          if constexpr (MX) {
            const int kb = 2 * g + (tig >> 1);               // block of 32 along K
            if ((tig & 1) == 0 && kb < p.G) {
              if (v_lo)
                p.sfa[((size_t)(m_lo >> 7) * (p.Kpad >> 7) + (kb >> 2)) * 512 + 16 * (m_lo & 31) + 4 * ((m_lo & 127) >> 5) + (kb & 3)] =
                    (uint8_t)(e_lo + 127);
              if (v_hi)
                p.sfa[((size_t)(m_hi >> 7) * (p.Kpad >> 7) + (kb >> 2)) * 512 + 16 * (m_hi & 31) + 4 * ((m_hi & 127) >> 5) + (kb & 3)] =
                    (uint8_t)(e_hi + 127);
            }
          } else {
            if (tig == 0 && g < p.G) {
              if (v_lo) p.sx[(size_t)g * p.Mpad + m_lo] = s_lo;
              if (v_hi) p.sx[(size_t)g * p.Mpad + m_hi] = s_hi;
            }
          }
          // a3 on the fragments just made: bytes 8j .. 8j+7 of a lane's run feed MMA step j
          if constexpr (BR == BR_INT) {
#pragma unroll
            for (int nt = 0; nt < NTR; ++nt) {
              mma_s8_16832(acci[nt], b_lo.x, b_hi.x, b_lo.y, b_hi.y, bfrag[nt].x, bfrag[nt].y);
              mma_s8_16832(acci[nt], b_lo.z, b_hi.z, b_lo.w, b_hi.w, bfrag[nt].z, bfrag[nt].w);
            }
          }
          if constexpr (BR == BR_F16) {
            // rows beyond M and values beyond K are zeros (TMA fill); fp16 x fp16 -> fp32, four k16 steps per box
#pragma unroll
            for (int nt = 0; nt < NTR; ++nt) {
              const uint4 f0 = bfrag[2 * nt], f1 = bfrag[2 * nt + 1];
              mma_f16_16816(accf[nt], l0.x, h0.x, l0.y, h0.y, f0.x, f0.y);
              mma_f16_16816(accf[nt], l0.z, h0.z, l0.w, h0.w, f0.z, f0.w);
              mma_f16_16816(accf[nt], l1.x, h1.x, l1.y, h1.y, f1.x, f1.y);
              mma_f16_16816(accf[nt], l1.z, h1.z, l1.w, h1.w, f1.z, f1.w);
            }
          }
          if (g + W < p.nbox) load_frags(g + W);
        }
        if (!ok) break;
      }
      if constexpr (BR == BR_NONE) continue;
      // ---- the warps' partial products meet in shared memory
      if constexpr (BR == BR_INT) {
        int* I1 = I1_s + par * TR * p.rpad;
#pragma unroll
        for (int nt = 0; nt < NTR; ++nt) {
          const int col = nt * 8 + tig * 2;
          if (col < p.rpad) {
            atomicAdd(&I1[gid * p.rpad + col], acci[nt][0]);
            atomicAdd(&I1[gid * p.rpad + col + 1], acci[nt][1]);
            atomicAdd(&I1[(gid + 8) * p.rpad + col], acci[nt][2]);
            atomicAdd(&I1[(gid + 8) * p.rpad + col + 1], acci[nt][3]);
          }
        }
      } else {
        float* mine = part_s + (size_t)warp * TR * p.rpad;
#pragma unroll
        for (int nt = 0; nt < NTR; ++nt) {
          const int col = nt * 8 + tig * 2;
          if (col < p.rpad) {
            *reinterpret_cast<float2*>(&mine[gid * p.rpad + col]) = make_float2(accf[nt][0], accf[nt][1]);
            *reinterpret_cast<float2*>(&mine[(gid + 8) * p.rpad + col]) = make_float2(accf[nt][2], accf[nt][3]);
          }
        }
      }
      ok = consumers_sync(bar_sync + 8, sync_par, lane, abort_flag, p.status);
      if (!ok) break;
      // ---- a4: the rank-r rows of this tile, one warp per row
      for (int rl = warp; rl < TR; rl += W) {
        const int m = m0 + rl;
        if constexpr (BR == BR_INT) {
          int* I1 = I1_s + par * TR * p.rpad + rl * p.rpad;
          const float rm = __int_as_float(rowmax_s[par * TR + rl]);
          const float sb = (rm == 0.f) ? 1.0f : __fdiv_rn(rm, p.qm);
          float t[4], amax = 0.f;
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) {
            const int j = lane + 32 * jj;
            t[jj] = 0.f;
            if (j < p.rpad) {
              const int v = I1[j];
              I1[j] = 0;                                      // ready for the tile after next
              if (j < p.r) {
                t[jj] = __fmul_rn(__int2float_rn(v), __fmul_rn(sb, p.sL1[j]));
                amax = fmaxf(amax, fabsf(t[jj]));
              }
            }
          }
          amax = warp_max(amax);
          if (m < p.M) {
            const float st = (amax == 0.f) ? 1.0f : __fdiv_rn(amax, p.qm);
            if (lane == 0) p.sT[m] = st;
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
              const int j = lane + 32 * jj;
              if (j < p.r) {
                float q = rintf(__fdiv_rn(t[jj], st));
                q = fminf(fmaxf(q, -p.qm), p.qm);
                p.tq[(size_t)m * LQ_RCONT + j] = (uint8_t)(int8_t)(int)q;
              }
            }
          }
        } else if constexpr (BR == BR_MXINT) {
          // T in fp32 (the warps' partial sums added in warp order), then MXINT8 along the rank: one block of 32 per warp
          // pass; the two digit planes of the codes share the row's container (hi at byte j, lo at byte 64 + j) and the
          // scale chunk's four slots are (hi, block 0), (hi, block 1), (lo, block 0), (lo, block 1)
          if (m < p.M) {
            for (int c = 0; c * 32 < p.r; ++c) {
              const int j = c * 32 + lane;
              float v = 0.f;
              if (j < p.rpad)
                for (int w2 = 0; w2 < W; ++w2) v += part_s[((size_t)w2 * TR + rl) * p.rpad + j];
              if (j >= p.r) v = 0.f;
              const int e = mxint8_exponent(warp_max(fabsf(v)));
              const float inv = e == -127 ? 0.f : __uint_as_float((uint32_t)(127 - e) << 23);
              const Code8 cd = mxint8_code(v, inv);
              // one container for both planes (rank <= 64): lo digits 64 bytes after the hi digits, scale slots c and
              // 2 + c of one chunk; a container per plane (rank <= 128): lo digits 128 bytes on, slot c of the next chunk
              const bool split = p.tq_stride != LQ_RCONT;
              p.tq[(size_t)m * p.tq_stride + j] = (uint8_t)(f32x2_to_e4m3x2(0.f, cd.hi) & 0xFF);
              p.tq[(size_t)m * p.tq_stride + (split ? 128 : 64) + j] = (uint8_t)(f32x2_to_e4m3x2(0.f, cd.lo) & 0xFF);
              if (lane == 0) {
                uint8_t* sf = p.sft + (size_t)(m >> 7) * (split ? 1024 : 512) + 16 * (m & 31) + 4 * ((m & 127) >> 5);
                sf[c] = (uint8_t)(e + 4 + 127); sf[(split ? 512 : 2) + c] = (uint8_t)(e + 127);
              }
            }
          }
        } else if constexpr (BR == BR_MXFP) {
          // T = deq(Q(X)) deq(Q2(L1)) in fp32 (the warps' partial sums added in warp order), then MXFP8e4 along the rank:
          // one block of 32 per warp pass, its maximum by a warp reduction
          if (m < p.M) {
            for (int c = 0; c * 32 < p.r; ++c) {
              const int j = c * 32 + lane;
              float v = 0.f;
              if (j < p.rpad)
                for (int w2 = 0; w2 < W; ++w2) v += part_s[((size_t)w2 * TR + rl) * p.rpad + j];
              if (j >= p.r) v = 0.f;
              const int e = mxfp8_exponent(warp_max(fabsf(v)), p.act6 != 0);
              const float inv = e == -127 ? 0.f : __uint_as_float((uint32_t)(127 - e) << 23);
              p.tq[(size_t)m * LQ_RCONT + j] = (uint8_t)(mxfp_pair(0.f, v * inv, p.act6 != 0) & 0xFF);
              if (lane == 0) p.sft[(size_t)(m >> 7) * 512 + 16 * (m & 31) + 4 * ((m & 127) >> 5) + c] = (uint8_t)(e + 127);
            }
          }
        } else {
          // T = fp16(X L1): the warps' fp32 partial sums are added in warp order (the result does not depend on timing)
          if (m < p.M) {
            for (int j = lane; j < p.r; j += 32) {
              float v = 0.f;
              for (int w2 = 0; w2 < W; ++w2) v += part_s[((size_t)w2 * TR + rl) * p.rpad + j];
              reinterpret_cast<__half*>(p.tq + (size_t)m * LQ_RCONT)[j] = __float2half_rn(v);
            }
            if (lane == 0) p.sT[m] = 1.0f;
          }
        }
      }
      if constexpr (FACC) {
        ok = consumers_sync(bar_sync + 16, sync_par, lane, abort_flag, p.status);   // partial sums may be overwritten
        if (!ok) break;
      }
      sync_par ^= 1;
    }
  }
}

struct LaunchPlan {
  int W, depth, refetch, ctas_per_sm;
  size_t smem;
};

// Picks the consumer-warp count, ring depth and residency for a row length.  Budget: 227 KB of shared memory and
// 64 K registers per SM (allocated per warp in units of 8 registers per thread).  Measured on the PixArt shapes
// (K = 1152, 4608; all branch kinds): two CTAs per SM with eight or nine consumer warps each is the fastest or within
// a few percent of it, so that is the default; the options "quant_ctas" / "quant_warps" override it for tuning.
LaunchPlan plan_launch(int nbox, int br, int rpad, int regs) {
  const size_t SM_SMEM = 227 * 1024;
  LaunchPlan best{};
  double best_score = -1.0;
  for (int ctas = 4; ctas >= 1; --ctas) {
    if (g_lq_quant_ctas > 0 ? ctas != g_lq_quant_ctas : ctas > 2) continue;
    for (int W = 4; W <= MAX_CONSUMER_WARPS; ++W) {
      if (g_lq_quant_warps > 0 ? W != g_lq_quant_warps : W < 8) continue;
      const int threads = (W + 1) * 32;
      if (ctas * threads > 2048 || ctas * threads * ((regs + 7) / 8 * 8) > 65536) continue;
      const size_t red = br == BR_INT ? (size_t)2 * TR * rpad * 4 : (br == BR_F16 || br == BR_MXFP || br == BR_MXINT) ? (size_t)W * TR * rpad * 4 : 0;
      const size_t fixed = 1024 + 64 + red + 2 * TR * 4 + 64;
      const size_t budget = std::min(SM_SMEM, SM_SMEM / ctas - 1024);
      if (budget < fixed + (size_t)W * (BOX_BYTES + 16)) continue;
      const int per = (nbox + W - 1) / W;                     // boxes of a tile per warp
      int depth = (int)((budget - fixed) / (BOX_BYTES + 16)) / W;
      int refetch = 0;
      if (depth > 2 * per) depth = 2 * per;
      if (depth < per && br == BR_INT) refetch = 1;
      // score: resident consumer warps, discounted by the imbalance of boxes over warps; more CTAs and warps win ties
      const double balance = (double)nbox / (double)(per * W);
      const double score = ctas * W * balance + 0.01 * ctas + 0.001 * W;
      if (score > best_score) {
        best_score = score;
        best = LaunchPlan{W, depth, refetch, ctas, fixed + (size_t)W * depth * (BOX_BYTES + 16)};
      }
    }
  }
  return best;
}

template <int MAIN, int BR, int NTR>
cudaError_t launch_quant(const CUtensorMap& tm, QuantParams& p, int sms, cudaStream_t st) {
  static bool attr_set[64] = {false};
  static int regs[64] = {0};
  int dev = 0;
  cudaGetDevice(&dev);
  if (!attr_set[dev & 63]) {
    cudaError_t e = cudaFuncSetAttribute(lq_quant_kernel<MAIN, BR, NTR>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    cudaFuncAttributes fa;
    if ((e = cudaFuncGetAttributes(&fa, lq_quant_kernel<MAIN, BR, NTR>)) != cudaSuccess) return e;
    regs[dev & 63] = fa.numRegs;
    attr_set[dev & 63] = true;
  }
  const LaunchPlan pl = plan_launch(p.nbox, BR, p.rpad, regs[dev & 63]);
  if (pl.W == 0) return cudaErrorInvalidConfiguration;
  p.depth = pl.depth; p.refetch = pl.refetch;
  int grid = sms * pl.ctas_per_sm;
  if (grid > p.ntiles) grid = p.ntiles;
  const cudaError_t e = lq_launch(lq_quant_kernel<MAIN, BR, NTR>, grid, (pl.W + 1) * 32, pl.smem, st, tm, p);
  return e != cudaSuccess ? e : cudaGetLastError();
}

template <int MAIN>
cudaError_t dispatch_quant(int br, int ntr, const CUtensorMap& tm, QuantParams& p, int sms, cudaStream_t st) {
  if (br == BR_NONE) return launch_quant<MAIN, BR_NONE, 1>(tm, p, sms, st);
  if constexpr (MAIN == MAIN_MXINT8) {
    if (ntr <= 2) return launch_quant<MAIN, BR_MXINT, 2>(tm, p, sms, st);
    if (ntr <= 4) return launch_quant<MAIN, BR_MXINT, 4>(tm, p, sms, st);
    if (ntr <= 8) return launch_quant<MAIN, BR_MXINT, 8>(tm, p, sms, st);
    return launch_quant<MAIN, BR_MXINT, 16>(tm, p, sms, st);
  } else if constexpr (MAIN == MAIN_MXFP) {
    if (ntr <= 2) return launch_quant<MAIN, BR_MXFP, 2>(tm, p, sms, st);
    if (ntr <= 4) return launch_quant<MAIN, BR_MXFP, 4>(tm, p, sms, st);
    if (ntr <= 8) return launch_quant<MAIN, BR_MXFP, 8>(tm, p, sms, st);
    return launch_quant<MAIN, BR_MXFP, 16>(tm, p, sms, st);
  } else {
    if (br == BR_INT) {
      if (ntr <= 2) return launch_quant<MAIN, BR_INT, 2>(tm, p, sms, st);
      if (ntr <= 4) return launch_quant<MAIN, BR_INT, 4>(tm, p, sms, st);
      if (ntr <= 8) return launch_quant<MAIN, BR_INT, 8>(tm, p, sms, st);
      return launch_quant<MAIN, BR_INT, 16>(tm, p, sms, st);
    }
    if (ntr <= 2) return launch_quant<MAIN, BR_F16, 2>(tm, p, sms, st);
    if (ntr <= 4) return launch_quant<MAIN, BR_F16, 4>(tm, p, sms, st);
    return launch_quant<MAIN, BR_F16, 8>(tm, p, sms, st);
  }
}

}  // namespace

// rank rounded up to the kernels' instantiated widths (8-column tiles: 2, 4, 8, 16)
int lq_quant_rank_tiles(int r, bool f16) {
  const int nt = lq_ceil_div(r > 0 ? r : 8, 8);
  return nt <= 2 ? 2 : nt <= 4 ? 4 : (nt <= 8 || f16) ? 8 : 16;
}

lq_status lq_launch_quantize(const lq_layer* L, const void* X, int M, lq_act* A, cudaStream_t st) {
  if (cudaSetDevice(A->device) != cudaSuccess) return LQ_ERR_CUDA;
  if (A->main_kind != LQ_KIND_E4M3) return LQ_ERR_UNSUPPORTED;
  const int abits = lq_branch_abits(L->cfg.branch);
  const int br = L->mxfp ? (L->r > 0 ? BR_MXFP : BR_NONE) : L->a8 ? (L->r > 0 ? BR_MXINT : BR_NONE) : L->f16_branch ? BR_F16 : (L->integer_branch && abits > 0) ? BR_INT : BR_NONE;
  const int ntr = lq_quant_rank_tiles(L->r, L->f16_branch);
  QuantParams p;
  p.M = M; p.K = L->K; p.Kpad = L->Kpad; p.Mpad = A->Mpad; p.G = L->G;
  p.nbox = L->Kpad / BOX_K;
  p.ntiles = lq_ceil_div(M, TR);
  p.qx8 = A->d_qx8; p.sx = A->d_sx; p.sfa = A->d_sfa;
  p.qb = g_lq_store_qb ? A->d_qb : nullptr;
  p.sXb = A->d_sXb;
  p.L1f = reinterpret_cast<const uint4*>(L->f16_branch ? (const void*)L->d_L1h : (const void*)L->d_L1f);
  p.sL1 = L->d_sL1; p.tq = A->d_tq; p.sT = A->d_sT;
  p.s1b = L->d_s1b; p.sft = A->d_sft;
  p.r = L->r; p.rpad = ntr * 8;
  p.tq_stride = A->tq_stride;
  p.act6 = (L->mxfp && L->cfg.act_fmt == LQ_ACT_MXFP6) ? 1 : 0;
  p.qm = br == BR_INT ? (float)((1 << (abits - 1)) - 1) : 0.f;
  p.status = lq_device_status_ptr(A->device);
  if (!p.status) return LQ_ERR_CUDA;
  CUtensorMap tm;
  lq_status s = lq_make_tmap_rows16(&tm, X, (uint64_t)M, (uint64_t)L->K);
  if (s != LQ_OK) return s;
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, A->device) != cudaSuccess) return LQ_ERR_CUDA;
  const cudaError_t e = L->mxfp ? dispatch_quant<MAIN_MXFP>(br, ntr, tm, p, sms, st)
                        : L->a8 ? dispatch_quant<MAIN_MXINT8>(br, ntr, tm, p, sms, st)
                        : L->mx ? dispatch_quant<MAIN_MXINT4>(br, ntr, tm, p, sms, st) : dispatch_quant<MAIN_SINT4>(br, ntr, tm, p, sms, st);
  return lq_note_cuda(e) == cudaSuccess ? LQ_OK : LQ_ERR_CUDA;
}
