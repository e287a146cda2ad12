// Activation side of the layer, ONE kernel and one read of X (Figure 1; Appendix A.2: the
// activations forwarded to both branches are quantized):
//   a1  SINT4 codes + fp16 scales per token and group of 64 along K          (Appendix A.3)
//   a2  per-token codes of the low-rank branch (needs the whole row's maximum first)
//   a3  down-projection I1 = qb L1q, exact int32, on the tensor cores (mma.sync, s8)
//   a4  t = fl32(fl32(I1) * fl32(sXb * sL1)), per-token re-quantization of the rank-r row
//
// A CTA owns 16 rows (one m16 MMA tile).  A warp holds one row in registers (16-byte loads,
// X is read from HBM exactly once), finds the row maximum, then walks the row once more and
// emits both code streams; the CTA then multiplies its 16 x K tile of branch codes, staged in
// shared memory, with L1q.
//
// Exactness contract: codes and scales equal the definition evaluated in IEEE binary32 with
// round-to-nearest-even and true division.  The fast path is division free:
//   scale   fp16(a / 7) == fp16(a * fl32(1/7)) for every finite fp16 a (checked exhaustively on
//           the host), because a/7 never comes closer than 2^-15 (relative) to an fp16 midpoint.
//   main    q' = rint(x * r), r ~ 1/s; e = fma(-q', s, x) is exact (q' has 3 bits, s 11 bits).
//           x and s are fp16 numbers, so x/s is either exactly k + 1/2 or at least 1e-4 away
//           from it, while x * r is within 3e-6 of x/s: q' is the correctly rounded code unless
//           |e| == s/2 exactly (a true tie) - those elements take the exact path.
//   branch  same with the fp32 per-token scale; an element takes the exact path (IEEE division)
//           whenever |e| >= 0.4999 s, i.e. whenever the quotient is not safely inside a
//           rounding cell (the estimate is within 5e-5 of the quotient).
#include <cuda_fp16.h>

#include "lq_internal.h"

namespace {

constexpr int ROWS = 16;               // rows per CTA
constexpr float MAGIC = 12582912.0f;   // 1.5 * 2^23: adding it rounds to an integer (ties to even)

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

__device__ __forceinline__ float rcp_fast(float x) {
  float r;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}

__device__ __forceinline__ void mma_s8_16832(int (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

struct QuantParams {
  const uint4* X;       // [M][K] halves
  int M, K, Kpad, Mpad, G;
  uint8_t* qx8;         // [Mpad][Kpad]
  float* sx;            // [Gpad][Mpad]
  uint8_t* sfa;         // MXINT4: E8M0 scale bytes [Mpad/128][Kpad/128][512]
  int8_t* qb;           // [Mpad][Kpad] or null (not stored)
  float* sXb;           // [Mpad]
  const uint2* L1f;     // [Kpad/32][rpad/8][32] fragment-major first factor
  const float* sL1;     // [LQ_MAX_RANK]
  uint8_t* tq;          // [Mpad][LQ_RCONT]
  float* sT;            // [Mpad]
  int r, rpad;          // rank, rank rounded up to 8
  int branch_qmax;      // 0: no integer branch
};

// Shared memory: qb tile [ROWS][Kpad + 16] bytes | sx tile [Gpad][ROWS] floats | I1 [ROWS][rpad] ints | sXb [ROWS]
// RELOAD: rows too long for the register file are read twice, chunk by chunk - once for the row maximum,
// once to quantize; the second read is served by the L2 (the row was touched microseconds earlier), so DRAM
// still sees X once, and the kernel keeps 64 registers per thread and full occupancy.
template <int NCHUNK, int WARPS, bool RELOAD, bool MX>
__global__ void __launch_bounds__(WARPS * 32) lq_quant_kernel(const QuantParams p) {
  extern __shared__ __align__(16) uint8_t qsm[];
  constexpr int RPW = ROWS / WARPS;    // rows per warp
  const int qb_stride = p.Kpad + 16;
  const int Gpad = p.Kpad / LQ_GROUP;
  uint8_t* qb_s = qsm;
  float* sx_s = reinterpret_cast<float*>(qsm + (p.branch_qmax > 0 ? ROWS * qb_stride : 0));
  int* I1_s = reinterpret_cast<int*>(sx_s + Gpad * ROWS);
  float* sXb_s = reinterpret_cast<float*>(I1_s + ROWS * p.rpad);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.x * ROWS;
  const float qm = (float)p.branch_qmax;

  for (int i = threadIdx.x; i < ROWS * p.rpad; i += WARPS * 32) I1_s[i] = 0;

#pragma unroll 1
  for (int rr = 0; rr < RPW; ++rr) {
    const int rl = warp * RPW + rr;
    const int m = m0 + rl;
    if (m >= p.M) {   // tail rows: zero codes so the MMA tile is defined
      if (p.branch_qmax > 0)
        for (int k = lane * 16; k < p.Kpad; k += 512) *reinterpret_cast<uint4*>(qb_s + rl * qb_stride + k) = make_uint4(0, 0, 0, 0);
      continue;
    }
    const uint4* xrow = p.X + (size_t)m * (p.K / 8);
    constexpr int NKEEP = RELOAD ? 1 : NCHUNK;
    uint4 v[NKEEP];
    __half hm[NKEEP];
    __half hrow = __ushort_as_half((unsigned short)0);
    // ---- pass A: this lane's maximum per chunk (exact in fp16) and the row maximum
    auto lane_max = [](const uint4& w) {
      const __half2* h2 = reinterpret_cast<const __half2*>(&w);
      const __half2 m2 = __hmax2(__hmax2(__habs2(h2[0]), __habs2(h2[1])), __hmax2(__habs2(h2[2]), __habs2(h2[3])));
      return __hmax(__low2half(m2), __high2half(m2));
    };
    if constexpr (RELOAD) {
#pragma unroll 6
      for (int c = 0; c < NCHUNK; ++c) {
        const int k0 = c * 256 + lane * 8;
        const uint4 w = (k0 < p.K) ? __ldg(xrow + (k0 >> 3)) : make_uint4(0, 0, 0, 0);
        hrow = __hmax(hrow, lane_max(w));
      }
    } else {
#pragma unroll
      for (int c = 0; c < NCHUNK; ++c) {
        const int k0 = c * 256 + lane * 8;
        v[c] = (k0 < p.K) ? __ldg(xrow + (k0 >> 3)) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int c = 0; c < NCHUNK; ++c) {
        hm[c] = lane_max(v[c]);
        hrow = __hmax(hrow, hm[c]);
      }
    }
    float sb = 1.0f, invb = 1.0f, thr = 0.f;
    if (p.branch_qmax > 0) {
      const float rowmax = warp_max(__half2float(hrow));
      sb = (rowmax == 0.f) ? 1.0f : __fdiv_rn(rowmax, qm);
      invb = __frcp_rn(sb);
      thr = 0.4999f * sb;
      if (lane == 0) { sXb_s[rl] = sb; p.sXb[m] = sb; }
    }
    // ---- pass B: group scales, 4-bit codes (a1) and branch codes (a2)
#pragma unroll(RELOAD ? 3 : NCHUNK)
    for (int c = 0; c < NCHUNK; ++c) {
      const int k0 = c * 256 + lane * 8;
      uint4 vc;
      float a;
      if constexpr (RELOAD) {
        vc = (k0 < p.K) ? __ldg(xrow + (k0 >> 3)) : make_uint4(0, 0, 0, 0);
        a = __half2float(lane_max(vc));
      } else {
        vc = v[c];
        a = __half2float(hm[c]);
      }
      a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, 1));
      a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, 2));
      if constexpr (!MX) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, 4));   // SINT4: 64 values = 8 lanes; MXINT4: 32 = 4 lanes
      if (k0 < p.Kpad) {
        uint32_t w0 = 0, w1 = 0, b0 = 0, b1 = 0;
        if (k0 < p.K) {
          __half s16;
          unsigned short sbits;
          float s;
          int mx_e = -127;
          if constexpr (MX) {
            // 2^e with e the smallest integer such that 7 * 2^e >= a: a = 1.f * 2^E, e = E - 2 if 1.f <= 1.75 else E - 1
            const uint32_t ab = __float_as_uint(a);
            if (a > 0.f) mx_e = (int)(ab >> 23) - 127 - (((ab & 0x7FFFFFu) <= 0x600000u) ? 2 : 1);
            s = __uint_as_float((uint32_t)(mx_e + 127) << 23);                  // a == 0: 2^-127 is never used (codes are 0)
            if (a == 0.f) s = 1.0f;
            sbits = 0x3C00; s16 = __ushort_as_half(sbits);                       // not a subnormal-scale case
          } else {
            s16 = __float2half_rn(__fmul_rn(a, 0.142857149243354797f));          // fl32(1/7)
            sbits = __half_as_ushort(s16);
            if (sbits == 0) s16 = __ushort_as_half((unsigned short)1);           // floor 2^-24
            s = __half2float(s16);
          }
          const __half2* h2 = reinterpret_cast<const __half2*>(&vc);
          float x[8], q[8], t[8];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float2 f = __half22float2(h2[i]);
            x[2 * i] = f.x; x[2 * i + 1] = f.y;
          }
          // MXINT4: 1/s = 2^-e is exact, so x * (1/s) is exact and the magic-number rounding is already the definition's
          const float inv = MX ? __uint_as_float((uint32_t)(127 - (a > 0.f ? mx_e : 0)) << 23) : rcp_fast(s), hs = 0.5f * s;
          bool exact = sbits < 0x0400;          // subnormal scale: quotient may exceed 7, use the plain definition
          bool near = false;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            q[i] = __fadd_rn(__fmaf_rn(x[i], inv, MAGIC), -MAGIC);
            const float e = __fmaf_rn(-q[i], s, x[i]);
            exact |= (fabsf(e) == hs);
            t[i] = __fmaf_rn(x[i], invb, MAGIC);                    // low byte of the bit pattern = branch code
            const float eb = __fmaf_rn(-__fadd_rn(t[i], -MAGIC), sb, x[i]);
            near |= !(fabsf(eb) < thr);
          }
          if constexpr (MX) exact = false;
          if (exact) {
#pragma unroll
            for (int i = 0; i < 8; ++i) q[i] = fminf(fmaxf(rintf(__fdiv_rn(x[i], s)), -7.f), 7.f);
          }
          if (near) {
#pragma unroll
            for (int i = 0; i < 8; ++i) t[i] = __fadd_rn(fminf(fmaxf(rintf(__fdiv_rn(x[i], sb)), -qm), qm), MAGIC);
          }
          w0 = f32x2_to_e4m3x2(q[1], q[0]) | (f32x2_to_e4m3x2(q[3], q[2]) << 16);
          w1 = f32x2_to_e4m3x2(q[5], q[4]) | (f32x2_to_e4m3x2(q[7], q[6]) << 16);
          b0 = __byte_perm(__byte_perm(__float_as_uint(t[0]), __float_as_uint(t[1]), 0x0040),
                           __byte_perm(__float_as_uint(t[2]), __float_as_uint(t[3]), 0x0040), 0x5410);
          b1 = __byte_perm(__byte_perm(__float_as_uint(t[4]), __float_as_uint(t[5]), 0x0040),
                           __byte_perm(__float_as_uint(t[6]), __float_as_uint(t[7]), 0x0040), 0x5410);
          *reinterpret_cast<uint2*>(p.qx8 + (size_t)m * p.Kpad + k0) = make_uint2(w0, w1);
          if constexpr (MX) {
            if ((lane & 3) == 0)
              p.sfa[((size_t)(m >> 7) * (p.Kpad >> 7) + (k0 >> 7)) * 512 + 16 * (m & 31) + 4 * ((m & 127) >> 5) + ((k0 >> 5) & 3)] =
                  (uint8_t)(mx_e + 127);
          } else {
            if ((lane & 7) == 0) sx_s[(k0 >> 6) * ROWS + rl] = s;
          }
          if (p.qb != nullptr && p.branch_qmax > 0) *reinterpret_cast<uint2*>(p.qb + (size_t)m * p.Kpad + k0) = make_uint2(b0, b1);
        }
        if (p.branch_qmax > 0) *reinterpret_cast<uint2*>(qb_s + rl * qb_stride + k0) = make_uint2(b0, b1);
      }
    }
  }
  __syncthreads();

  // group scales, transposed: [g][m0 .. m0+15] are 64-byte segments
  for (int i = threadIdx.x; !MX && i < p.G * ROWS; i += WARPS * 32) {
    const int g = i / ROWS, rl = i % ROWS;
    if (m0 + rl < p.M) p.sx[(size_t)g * p.Mpad + m0 + rl] = sx_s[g * ROWS + rl];
  }
  if (p.branch_qmax <= 0) return;

  // ------------------------------------------------------------------ a3: I1 = qb L1q on mma.sync
  const int ksteps = p.Kpad / 32, ntiles = p.rpad / 8;
  const int gid = lane >> 2, tig = lane & 3;
  for (int nt0 = 0; nt0 < ntiles; nt0 += 4) {
    int acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int b = 0; b < 4; ++b) acc[a][b] = 0;
    for (int ks = warp; ks < ksteps; ks += WARPS) {
      uint32_t a[4];
      const uint8_t* ab = qb_s + ks * 32 + tig * 4;
      a[0] = *reinterpret_cast<const uint32_t*>(ab + gid * qb_stride);
      a[1] = *reinterpret_cast<const uint32_t*>(ab + (gid + 8) * qb_stride);
      a[2] = *reinterpret_cast<const uint32_t*>(ab + gid * qb_stride + 16);
      a[3] = *reinterpret_cast<const uint32_t*>(ab + (gid + 8) * qb_stride + 16);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (nt0 + j < ntiles) {
          const uint2 b = __ldg(p.L1f + ((size_t)ks * ntiles + nt0 + j) * 32 + lane);
          mma_s8_16832(acc[j], a, b.x, b.y);
        }
      }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (nt0 + j < ntiles) {
        const int col = (nt0 + j) * 8 + tig * 2;
        atomicAdd(&I1_s[gid * p.rpad + col], acc[j][0]);
        atomicAdd(&I1_s[gid * p.rpad + col + 1], acc[j][1]);
        atomicAdd(&I1_s[(gid + 8) * p.rpad + col], acc[j][2]);
        atomicAdd(&I1_s[(gid + 8) * p.rpad + col + 1], acc[j][3]);
      }
    }
  }
  __syncthreads();

  // ------------------------------------------------------------------ a4: re-quantize the rank-r row
  for (int rr = 0; rr < RPW; ++rr) {
    const int rl = warp * RPW + rr, m = m0 + rl;
    if (m >= p.M) continue;
    const float sb = sXb_s[rl];
    float t[4], amax = 0.f;
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      const int j = lane + 32 * jj;
      t[jj] = 0.f;
      if (j < p.r) {
        t[jj] = __fmul_rn(__int2float_rn(I1_s[rl * p.rpad + j]), __fmul_rn(sb, p.sL1[j]));
        amax = fmaxf(amax, fabsf(t[jj]));
      }
    }
    amax = warp_max(amax);
    const float st = (amax == 0.f) ? 1.0f : __fdiv_rn(amax, qm);
    if (lane == 0) p.sT[m] = st;
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      const int j = lane + 32 * jj;
      if (j < p.r) {
        float q = rintf(__fdiv_rn(t[jj], st));
        q = fminf(fmaxf(q, -qm), qm);
        p.tq[(size_t)m * LQ_RCONT + j] = (uint8_t)(int8_t)(int)q;
      }
    }
  }
}

// W16A16 reference branch: T = X L1 accumulated in fp32, rounded once to fp16; no scales.
// A CTA of four warps owns 16 rows; the warps split K in chunks of 32 (chunk c goes to warp c % 4), multiply with
// mma.sync m16n8k16 (fp16 x fp16 -> fp32) and add their partial sums in shared memory.  Both operands are fetched with
// 16-byte loads: lane (g, t) holds elements 8t .. 8t+7 of the chunk for row g (A) or factor column g (B).  A sum over k does
// not care which k sits in which fragment slot as long as A and B agree, so the lane's first four elements feed one k16 step
// and its last four the next - no shuffles, and X is read once with full sectors.
__device__ __forceinline__ void mma_f16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

template <int NT>   // NT: 8-column tiles of the rank (rank <= 8 NT)
__global__ void __launch_bounds__(128) lq_down_f16_kernel(const __half* __restrict__ X, const __half* __restrict__ L1h,
                                                          int M, int K, int Kpad, int r, uint8_t* __restrict__ tq,
                                                          float* __restrict__ sT) {
  __shared__ float part[4][16][NT * 8 + 1];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int m0 = blockIdx.x * 16;
  const int r_lo = m0 + g, r_hi = m0 + g + 8;
  float acc[NT][4];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt)
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[nt][i] = 0.f;
  const uint4 zero = make_uint4(0, 0, 0, 0);
  const int chunks = (K + 31) / 32;
#pragma unroll 3
  for (int c = warp; c < chunks; c += 4) {
    const int k = c * 32 + 8 * t;
    const bool kin = k < K;                                                        // K is a multiple of 8
    const uint4 alo = (kin && r_lo < M) ? __ldg(reinterpret_cast<const uint4*>(X + (size_t)r_lo * K + k)) : zero;
    const uint4 ahi = (kin && r_hi < M) ? __ldg(reinterpret_cast<const uint4*>(X + (size_t)r_hi * K + k)) : zero;
    uint4 b[NT];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const int j = nt * 8 + g;
      b[nt] = (j < r) ? __ldg(reinterpret_cast<const uint4*>(L1h + (size_t)j * Kpad + k)) : zero;   // zero-padded up to Kpad
    }
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      mma_f16_16816(acc[nt], alo.x, ahi.x, alo.y, ahi.y, b[nt].x, b[nt].y);
      mma_f16_16816(acc[nt], alo.z, ahi.z, alo.w, ahi.w, b[nt].z, b[nt].w);
    }
  }
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    part[warp][g][nt * 8 + 2 * t] = acc[nt][0];
    part[warp][g][nt * 8 + 2 * t + 1] = acc[nt][1];
    part[warp][g + 8][nt * 8 + 2 * t] = acc[nt][2];
    part[warp][g + 8][nt * 8 + 2 * t + 1] = acc[nt][3];
  }
  __syncthreads();
  for (int i = threadIdx.x; i < 16 * NT * 8; i += 128) {
    const int row = i / (NT * 8), j = i % (NT * 8);
    const int m = m0 + row;
    if (m < M && j < r) {
      const float v = (part[0][row][j] + part[1][row][j]) + (part[2][row][j] + part[3][row][j]);
      reinterpret_cast<__half*>(tq + (size_t)m * LQ_RCONT)[j] = __float2half_rn(v);
    }
  }
  if (threadIdx.x < 16 && m0 + threadIdx.x < M) sT[m0 + threadIdx.x] = 1.0f;
}

template <int NCHUNK, int WARPS, bool RELOAD, bool MX>
cudaError_t launch_quant(const QuantParams& p, size_t smem, cudaStream_t st) {
  static bool attr_set[64] = {false};
  int dev = 0;
  cudaGetDevice(&dev);
  if (smem > 48 * 1024 && !attr_set[dev & 63]) {
    cudaError_t e = cudaFuncSetAttribute(lq_quant_kernel<NCHUNK, WARPS, RELOAD, MX>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
    attr_set[dev & 63] = true;
  }
  lq_quant_kernel<NCHUNK, WARPS, RELOAD, MX><<<lq_ceil_div(p.M, ROWS), WARPS * 32, smem, st>>>(p);
  return cudaGetLastError();
}

}  // namespace

lq_status lq_launch_quantize(const lq_layer* L, const void* X, int M, lq_act* A, cudaStream_t st) {
  if (cudaSetDevice(A->device) != cudaSuccess) return LQ_ERR_CUDA;
  const int K = L->K, Kpad = L->Kpad;
  const int abits = lq_branch_abits(L->cfg.branch);
  QuantParams p;
  p.X = reinterpret_cast<const uint4*>(X);
  p.M = M; p.K = K; p.Kpad = Kpad; p.Mpad = A->Mpad; p.G = L->G;
  p.qx8 = A->d_qx8; p.sx = A->d_sx; p.sfa = A->d_sfa;
  p.qb = g_lq_store_qb ? A->d_qb : nullptr;
  p.sXb = A->d_sXb;
  p.L1f = reinterpret_cast<const uint2*>(L->d_L1f);
  p.sL1 = L->d_sL1; p.tq = A->d_tq; p.sT = A->d_sT;
  p.r = L->r; p.rpad = lq_round_up(L->r > 0 ? L->r : 8, 8);
  p.branch_qmax = (L->integer_branch && abits > 0) ? ((1 << (abits - 1)) - 1) : 0;
  const size_t smem = (p.branch_qmax > 0 ? (size_t)ROWS * (Kpad + 16) : 0) + (size_t)(Kpad / LQ_GROUP) * ROWS * 4 +
                      (size_t)ROWS * p.rpad * 4 + ROWS * 4;
  const int nchunk = lq_ceil_div(Kpad, 256);
  cudaError_t e;
  if (A->main_kind != LQ_KIND_E4M3) return LQ_ERR_UNSUPPORTED;
#define LQ_QUANT_DISPATCH(MXF)                                                                                          \
  if (nchunk <= 2) e = launch_quant<2, 16, false, MXF>(p, smem, st);   /* the row stays in registers (one warp per row) */ \
  else if (nchunk <= 5) e = launch_quant<5, 16, false, MXF>(p, smem, st);                                               \
  else if (nchunk <= 9) e = launch_quant<9, 16, true, MXF>(p, smem, st);   /* longer rows: read twice, 2nd time from L2 */ \
  else if (nchunk <= 12) e = launch_quant<12, 16, true, MXF>(p, smem, st);                                              \
  else if (nchunk <= 18) e = launch_quant<18, 16, true, MXF>(p, smem, st);                                              \
  else if (nchunk <= 22) e = launch_quant<22, 16, true, MXF>(p, smem, st);                                              \
  else if (nchunk <= 32) e = launch_quant<32, 16, true, MXF>(p, smem, st);                                              \
  else return LQ_ERR_UNSUPPORTED;
  if (L->mx) { LQ_QUANT_DISPATCH(true) } else { LQ_QUANT_DISPATCH(false) }
#undef LQ_QUANT_DISPATCH
  if (lq_note_cuda(e) != cudaSuccess) return LQ_ERR_CUDA;
  if (L->f16_branch) {
    const __half* Xh = reinterpret_cast<const __half*>(X);
    const __half* L1 = reinterpret_cast<const __half*>(L->d_L1h);
    const int blocks = lq_ceil_div(M, 16);
    if (L->r <= 16) lq_down_f16_kernel<2><<<blocks, 128, 0, st>>>(Xh, L1, M, K, Kpad, L->r, A->d_tq, A->d_sT);
    else if (L->r <= 32) lq_down_f16_kernel<4><<<blocks, 128, 0, st>>>(Xh, L1, M, K, Kpad, L->r, A->d_tq, A->d_sT);
    else lq_down_f16_kernel<8><<<blocks, 128, 0, st>>>(Xh, L1, M, K, Kpad, L->r, A->d_tq, A->d_sT);
    if (cudaGetLastError() != cudaSuccess) return LQ_ERR_CUDA;
  }
  return LQ_OK;
}
