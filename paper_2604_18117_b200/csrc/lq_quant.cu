// Activation side of the layer, ONE kernel and one read of X (Figure 1; Appendix A.2: the
// activations forwarded to both branches are quantized):
//   a1  SINT4 codes + fp16 scales per token and group of 64 along K          (Appendix A.3)
//   a2  per-token codes of the low-rank branch (needs the whole row's maximum first)
//   a3  down-projection I1 = qb L1q, exact int32, on the tensor cores (mma.sync, s8)
//   a4  t = fl32(fl32(I1) * fl32(sXb * sL1)), per-token re-quantization of the rank-r row
//
// A CTA owns 16 rows (one m16 MMA tile); each of its 8 warps quantizes 2 rows, one after the
// other, holding the row in registers (16-byte loads, X is read from HBM exactly once), then
// the CTA multiplies its 16 x K tile of branch codes, staged in shared memory, with L1q.
//
// Exactness contract: codes and scales equal the definition evaluated in IEEE binary32 with
// round-to-nearest-even and true division.  The fast path replaces the per-element division
// by a multiplication with the correctly rounded reciprocal plus an exact remainder test:
//   main    q' = rint(x * (1/s)); e = fma(-q', s, x) is exact (q' has 4 bits, s 11 bits).
//           x and s are fp16 numbers, so x/s is either exactly k + 1/2 or at least 1e-4 away
//           from it, while x * (1/s) is within 5e-7 of x/s: q' is the correctly rounded code
//           unless |e| == s/2 exactly (a true tie) - those elements take the slow path.
//   branch  same with the fp32 scale; the element takes the slow path (IEEE division) whenever
//           |e| >= 0.499 s, i.e. whenever the quotient is not safely inside a rounding cell.
#include <cuda_fp16.h>

#include "lq_internal.h"

namespace {

constexpr int ROWS = 16;          // rows per CTA
constexpr int QWARPS = 8;
constexpr float MAGIC = 12582912.0f;   // 1.5 * 2^23: adding it rounds to an integer (ties to even)

__device__ __forceinline__ uint32_t encode_code(int q, int kind) {
  if (kind == LQ_KIND_I8) return (uint32_t)q & 0xFFu;
  // E4M3 byte of an integer in [-7, 7]: 0,1,2,3,4,5,6,7 -> 00 38 40 44 48 4A 4C 4E
  const int a = q < 0 ? -q : q;
  const uint64_t tab = 0x4E4C4A4844403800ull;
  uint32_t b = (uint32_t)(tab >> (8 * a)) & 0xFFu;
  return b | (q < 0 ? 0x80u : 0u);
}

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
  int8_t* qb;           // [Mpad][Kpad] or null (not stored)
  float* sXb;           // [Mpad]
  const uint2* L1f;     // [Kpad/32][rpad/8][32] fragment-major first factor
  const float* sL1;     // [LQ_MAX_RANK]
  uint8_t* tq;          // [Mpad][LQ_RCONT]
  float* sT;            // [Mpad]
  int r, rpad;          // rank, rank rounded up to 8
  int main_kind;
  int branch_qmax;      // 0: no integer branch
};

// Shared memory: qb tile [ROWS][Kpad + 16] bytes | sx tile [Gpad][ROWS] floats | I1 [ROWS][rpad] ints | sXb [ROWS]
template <int NCHUNK>
__global__ void __launch_bounds__(QWARPS * 32) lq_quant_kernel(const QuantParams p) {
  extern __shared__ __align__(16) uint8_t qsm[];
  const int qb_stride = p.Kpad + 16;
  const int Gpad = p.Kpad / LQ_GROUP;
  uint8_t* qb_s = qsm;
  float* sx_s = reinterpret_cast<float*>(qsm + (p.branch_qmax > 0 ? ROWS * qb_stride : 0));
  int* I1_s = reinterpret_cast<int*>(sx_s + Gpad * ROWS);
  float* sXb_s = reinterpret_cast<float*>(I1_s + ROWS * p.rpad);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.x * ROWS;
  const bool e4m3 = p.main_kind == LQ_KIND_E4M3;
  const float qm = (float)p.branch_qmax;

  for (int i = threadIdx.x; i < ROWS * p.rpad; i += QWARPS * 32) I1_s[i] = 0;

  for (int rr = 0; rr < 2; ++rr) {
    const int rl = warp * 2 + rr;
    const int m = m0 + rl;
    if (m >= p.M) {   // tail rows: zero codes so the MMA tile is defined
      if (p.branch_qmax > 0)
        for (int k = lane * 16; k < p.Kpad; k += 512) *reinterpret_cast<uint4*>(qb_s + rl * qb_stride + k) = make_uint4(0, 0, 0, 0);
      continue;
    }
    const uint4* xrow = p.X + (size_t)m * (p.K / 8);
    uint4 v[NCHUNK];
#pragma unroll
    for (int c = 0; c < NCHUNK; ++c) {
      const int k0 = c * 256 + lane * 8;
      v[c] = (k0 < p.K) ? __ldg(xrow + (k0 >> 3)) : make_uint4(0, 0, 0, 0);
    }
    float rowmax = 0.f;
    // ---------------------------------------------------------------- a1: SINT4 codes
#pragma unroll
    for (int c = 0; c < NCHUNK; ++c) {
      const int k0 = c * 256 + lane * 8;
      const __half2* h2 = reinterpret_cast<const __half2*>(&v[c]);
      const __half2 m2 = __hmax2(__hmax2(__habs2(h2[0]), __habs2(h2[1])), __hmax2(__habs2(h2[2]), __habs2(h2[3])));
      float a = fmaxf(__low2float(m2), __high2float(m2));
      rowmax = fmaxf(rowmax, a);
      a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, 1));
      a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, 2));
      a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, 4));
      __half s16 = __float2half_rn(__fdiv_rn(a, 7.0f));
      const unsigned short sbits = __half_as_ushort(s16);
      if (sbits == 0) s16 = __ushort_as_half((unsigned short)1);   // floor 2^-24
      const float s = __half2float(s16);
      if (k0 < p.K) {
        float x[8], q[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 f = __half22float2(h2[i]);
          x[2 * i] = f.x; x[2 * i + 1] = f.y;
        }
        bool slow = sbits < 0x0400;          // subnormal scale: quotient may exceed 7, use the plain definition
        if (!slow) {
          const float inv = __frcp_rn(s), hs = 0.5f * s;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            q[i] = __fadd_rn(__fmaf_rn(x[i], inv, MAGIC), -MAGIC);
            const float e = __fmaf_rn(-q[i], s, x[i]);
            slow |= (fabsf(e) == hs);
          }
        }
        if (slow) {
#pragma unroll
          for (int i = 0; i < 8; ++i) q[i] = fminf(fmaxf(rintf(__fdiv_rn(x[i], s)), -7.f), 7.f);
        }
        uint32_t w0, w1;
        if (e4m3) {
          w0 = f32x2_to_e4m3x2(q[1], q[0]) | (f32x2_to_e4m3x2(q[3], q[2]) << 16);
          w1 = f32x2_to_e4m3x2(q[5], q[4]) | (f32x2_to_e4m3x2(q[7], q[6]) << 16);
        } else {
          w0 = ((uint32_t)(int)q[0] & 0xFFu) | (((uint32_t)(int)q[1] & 0xFFu) << 8) | (((uint32_t)(int)q[2] & 0xFFu) << 16) |
               (((uint32_t)(int)q[3] & 0xFFu) << 24);
          w1 = ((uint32_t)(int)q[4] & 0xFFu) | (((uint32_t)(int)q[5] & 0xFFu) << 8) | (((uint32_t)(int)q[6] & 0xFFu) << 16) |
               (((uint32_t)(int)q[7] & 0xFFu) << 24);
        }
        *reinterpret_cast<uint2*>(p.qx8 + (size_t)m * p.Kpad + k0) = make_uint2(w0, w1);
        if ((lane & 7) == 0) sx_s[(k0 >> 6) * ROWS + rl] = s;
      }
    }
    if (p.branch_qmax <= 0) continue;
    // ---------------------------------------------------------------- a2: per-token branch codes
    rowmax = warp_max(rowmax);
    const float sb = (rowmax == 0.f) ? 1.0f : __fdiv_rn(rowmax, qm);
    if (lane == 0) { sXb_s[rl] = sb; p.sXb[m] = sb; }
    const float inv = __frcp_rn(sb), thr = 0.499f * sb;
#pragma unroll
    for (int c = 0; c < NCHUNK; ++c) {
      const int k0 = c * 256 + lane * 8;
      if (k0 < p.Kpad) {
        uint32_t w0 = 0, w1 = 0;
        if (k0 < p.K) {
          const __half2* h2 = reinterpret_cast<const __half2*>(&v[c]);
          float x[8], t[8];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float2 f = __half22float2(h2[i]);
            x[2 * i] = f.x; x[2 * i + 1] = f.y;
          }
          bool slow = false;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            t[i] = __fmaf_rn(x[i], inv, MAGIC);                    // low byte of the bit pattern = code
            const float e = __fmaf_rn(-__fadd_rn(t[i], -MAGIC), sb, x[i]);
            slow |= !(fabsf(e) < thr);
          }
          if (slow) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const float qf = fminf(fmaxf(rintf(__fdiv_rn(x[i], sb)), -qm), qm);
              t[i] = __fadd_rn(qf, MAGIC);
            }
          }
          w0 = __byte_perm(__byte_perm(__float_as_uint(t[0]), __float_as_uint(t[1]), 0x0040),
                           __byte_perm(__float_as_uint(t[2]), __float_as_uint(t[3]), 0x0040), 0x5410);
          w1 = __byte_perm(__byte_perm(__float_as_uint(t[4]), __float_as_uint(t[5]), 0x0040),
                           __byte_perm(__float_as_uint(t[6]), __float_as_uint(t[7]), 0x0040), 0x5410);
        }
        *reinterpret_cast<uint2*>(qb_s + rl * qb_stride + k0) = make_uint2(w0, w1);
        if (p.qb != nullptr && k0 < p.K) *reinterpret_cast<uint2*>(p.qb + (size_t)m * p.Kpad + k0) = make_uint2(w0, w1);
      }
    }
  }
  __syncthreads();

  // group scales, transposed: [g][m0 .. m0+15] are 64-byte segments
  for (int i = threadIdx.x; i < p.G * ROWS; i += QWARPS * 32) {
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
    for (int ks = warp; ks < ksteps; ks += QWARPS) {
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
  for (int rr = 0; rr < 2; ++rr) {
    const int rl = warp * 2 + rr, m = m0 + rl;
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
__global__ void __launch_bounds__(256) lq_down_f16_kernel(const __half* __restrict__ X, const __half* __restrict__ L1h,
                                                          int M, int K, int Kpad, int r, uint8_t* __restrict__ tq,
                                                          float* __restrict__ sT) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m = blockIdx.x * 8 + warp;
  if (m >= M) return;
  const __half* xrow = X + (size_t)m * K;
  for (int j = lane; j < r; j += 32) {
    const __half* brow = L1h + (size_t)j * Kpad;
    float a = 0.f;
    for (int k = 0; k < K; ++k) a = fmaf(__half2float(xrow[k]), __half2float(brow[k]), a);
    reinterpret_cast<__half*>(tq + (size_t)m * LQ_RCONT)[j] = __float2half_rn(a);
  }
  if (lane == 0) sT[m] = 1.0f;
}

template <int NCHUNK>
cudaError_t launch_quant(const QuantParams& p, size_t smem, cudaStream_t st) {
  static bool attr_set[64] = {false};
  int dev = 0;
  cudaGetDevice(&dev);
  if (smem > 48 * 1024 && !attr_set[dev & 63]) {
    cudaError_t e = cudaFuncSetAttribute(lq_quant_kernel<NCHUNK>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
    attr_set[dev & 63] = true;
  }
  lq_quant_kernel<NCHUNK><<<lq_ceil_div(p.M, ROWS), QWARPS * 32, smem, st>>>(p);
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
  p.qx8 = A->d_qx8; p.sx = A->d_sx;
  p.qb = g_lq_store_qb ? A->d_qb : nullptr;
  p.sXb = A->d_sXb;
  p.L1f = reinterpret_cast<const uint2*>(L->d_L1f);
  p.sL1 = L->d_sL1; p.tq = A->d_tq; p.sT = A->d_sT;
  p.r = L->r; p.rpad = lq_round_up(L->r > 0 ? L->r : 8, 8);
  p.main_kind = A->main_kind;
  p.branch_qmax = (L->integer_branch && abits > 0) ? ((1 << (abits - 1)) - 1) : 0;
  const size_t smem = (p.branch_qmax > 0 ? (size_t)ROWS * (Kpad + 16) : 0) + (size_t)(Kpad / LQ_GROUP) * ROWS * 4 +
                      (size_t)ROWS * p.rpad * 4 + ROWS * 4;
  const int nchunk = lq_ceil_div(Kpad, 256);
  cudaError_t e;
  if (nchunk <= 2) e = launch_quant<2>(p, smem, st);
  else if (nchunk <= 5) e = launch_quant<5>(p, smem, st);
  else if (nchunk <= 9) e = launch_quant<9>(p, smem, st);
  else if (nchunk <= 12) e = launch_quant<12>(p, smem, st);
  else if (nchunk <= 18) e = launch_quant<18>(p, smem, st);
  else if (nchunk <= 22) e = launch_quant<22>(p, smem, st);
  else if (nchunk <= 32) e = launch_quant<32>(p, smem, st);
  else return LQ_ERR_UNSUPPORTED;
  if (e != cudaSuccess) return LQ_ERR_CUDA;
  if (L->f16_branch) {
    lq_down_f16_kernel<<<lq_ceil_div(M, 8), 256, 0, st>>>(reinterpret_cast<const __half*>(X),
                                                          reinterpret_cast<const __half*>(L->d_L1h), M, K, Kpad, L->r,
                                                          A->d_tq, A->d_sT);
    if (cudaGetLastError() != cudaSuccess) return LQ_ERR_CUDA;
  }
  return LQ_OK;
}
