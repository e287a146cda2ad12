// Activation side of the layer: dynamic SINT4 quantization per token and group of 64 along K
// (Appendix A.3), the per-token codes of the low-rank branch from the same read of X
// (Appendix A.2: activations of both branches are quantized), the branch's down-projection
// onto the quantized first factor and the per-token re-quantization of the rank-r result
// (Figure 1; Section 3.3).
//
// Exactness contract: every floating-point step is IEEE binary32 with round-to-nearest-even,
// true division, no fused multiply-add across a rounding the definition has, and rint() for
// the final rounding to a code, so the codes and scales are reproducible bit for bit.
#include <cuda_fp16.h>

#include "lq_internal.h"

namespace {

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

// One warp per row.  The row lives in registers (NCHUNK x 8 halves per lane), so X is read
// from HBM exactly once although the branch's per-token scale needs the whole row first.
template <int NCHUNK>
__global__ void __launch_bounds__(256) lq_quant_kernel(const uint4* __restrict__ X, int M, int K, int Kpad, int Mpad,
                                                       uint8_t* __restrict__ qx8, float* __restrict__ sx,
                                                       int8_t* __restrict__ qb, float* __restrict__ sXb,
                                                       int main_kind, int branch_qmax) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m = blockIdx.x * 8 + warp;
  if (m >= M) return;
  const uint4* xrow = X + (size_t)m * (K / 8);
  uint4 v[NCHUNK];
#pragma unroll
  for (int c = 0; c < NCHUNK; ++c) {
    const int k0 = c * 256 + lane * 8;
    v[c] = (k0 < K) ? __ldg(xrow + (k0 >> 3)) : make_uint4(0, 0, 0, 0);
  }
  float rowmax = 0.f;
#pragma unroll
  for (int c = 0; c < NCHUNK; ++c) {
    const int k0 = c * 256 + lane * 8;
    const __half2* h2 = reinterpret_cast<const __half2*>(&v[c]);
    __half2 m2 = __hmax2(__hmax2(__habs2(h2[0]), __habs2(h2[1])), __hmax2(__habs2(h2[2]), __habs2(h2[3])));
    float a = fmaxf(__low2float(m2), __high2float(m2));
    rowmax = fmaxf(rowmax, a);
    a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, 1));
    a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, 2));
    a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, 4));
    __half s16 = __float2half_rn(__fdiv_rn(a, 7.0f));
    if (__half_as_ushort(s16) == 0) s16 = __ushort_as_half((unsigned short)1);   // floor 2^-24
    const float s = __half2float(s16);
    if (k0 < K) {
      uint32_t w[2] = {0u, 0u};
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float x = __half2float(reinterpret_cast<const __half*>(&v[c])[i]);
        float q = rintf(__fdiv_rn(x, s));
        q = fminf(fmaxf(q, -7.f), 7.f);
        w[i >> 2] |= encode_code((int)q, main_kind) << (8 * (i & 3));
      }
      *reinterpret_cast<uint2*>(qx8 + (size_t)m * Kpad + k0) = make_uint2(w[0], w[1]);
      if ((lane & 7) == 0) sx[(size_t)(k0 >> 6) * Mpad + m] = s;
    }
  }
  if (branch_qmax <= 0) return;
  rowmax = warp_max(rowmax);
  const float qm = (float)branch_qmax;
  const float sb = (rowmax == 0.f) ? 1.0f : __fdiv_rn(rowmax, qm);
  if (lane == 0) sXb[m] = sb;
#pragma unroll
  for (int c = 0; c < NCHUNK; ++c) {
    const int k0 = c * 256 + lane * 8;
    if (k0 < K) {
      uint32_t w[2] = {0u, 0u};
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float x = __half2float(reinterpret_cast<const __half*>(&v[c])[i]);
        float q = rintf(__fdiv_rn(x, sb));
        q = fminf(fmaxf(q, -qm), qm);
        w[i >> 2] |= ((uint32_t)(int)q & 0xFFu) << (8 * (i & 3));
      }
      *reinterpret_cast<uint2*>(qb + (size_t)m * Kpad + k0) = make_uint2(w[0], w[1]);
    }
  }
}

// Down-projection I1 = qb L1q (exact int32), t = fl32(fl32(I1) * fl32(sXb * sL1)), then the
// per-token re-quantization of t.  One warp per row, lane j owns columns j, j+32, ...
__global__ void __launch_bounds__(256) lq_down_int_kernel(const int8_t* __restrict__ qb, const float* __restrict__ sXb,
                                                          const int8_t* __restrict__ L1t, const float* __restrict__ sL1,
                                                          int M, int Kpad, int r, int qmax, uint8_t* __restrict__ tq,
                                                          float* __restrict__ sT) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m = blockIdx.x * 8 + warp;
  if (m >= M) return;
  const int* arow = reinterpret_cast<const int*>(qb + (size_t)m * Kpad);
  const int nw = Kpad / 4;
  int acc[4] = {0, 0, 0, 0};
#pragma unroll
  for (int jj = 0; jj < 4; ++jj) {
    const int j = lane + 32 * jj;
    if (j < r) {
      const int* brow = reinterpret_cast<const int*>(L1t + (size_t)j * Kpad);
      int a = 0;
      for (int w = 0; w < nw; ++w) a = __dp4a(__ldg(arow + w), __ldg(brow + w), a);
      acc[jj] = a;
    }
  }
  const float sb = sXb[m];
  float t[4], amax = 0.f;
#pragma unroll
  for (int jj = 0; jj < 4; ++jj) {
    const int j = lane + 32 * jj;
    t[jj] = 0.f;
    if (j < r) {
      t[jj] = __fmul_rn(__int2float_rn(acc[jj]), __fmul_rn(sb, sL1[j]));
      amax = fmaxf(amax, fabsf(t[jj]));
    }
  }
  amax = warp_max(amax);
  const float qm = (float)qmax;
  const float st = (amax == 0.f) ? 1.0f : __fdiv_rn(amax, qm);
  if (lane == 0) sT[m] = st;
#pragma unroll
  for (int jj = 0; jj < 4; ++jj) {
    const int j = lane + 32 * jj;
    if (j < r) {
      float q = rintf(__fdiv_rn(t[jj], st));
      q = fminf(fmaxf(q, -qm), qm);
      tq[(size_t)m * LQ_RCONT + j] = (uint8_t)(int8_t)(int)q;
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
void launch_quant(const void* X, int M, int K, int Kpad, int Mpad, lq_act* A, int bqmax, cudaStream_t st) {
  lq_quant_kernel<NCHUNK><<<lq_ceil_div(M, 8), 256, 0, st>>>(reinterpret_cast<const uint4*>(X), M, K, Kpad, Mpad,
                                                              A->d_qx8, A->d_sx, A->d_qb, A->d_sXb, A->main_kind, bqmax);
}

}  // namespace

lq_status lq_launch_quantize(const lq_layer* L, const void* X, int M, lq_act* A, cudaStream_t st) {
  if (cudaSetDevice(A->device) != cudaSuccess) return LQ_ERR_CUDA;
  const int K = L->K, Kpad = L->Kpad, Mpad = A->Mpad;
  const int abits = lq_branch_abits(L->cfg.branch);
  const int bqmax = (L->integer_branch && abits > 0) ? ((1 << (abits - 1)) - 1) : 0;
  const int nchunk = lq_ceil_div(K, 256);
  if (nchunk <= 2) launch_quant<2>(X, M, K, Kpad, Mpad, A, bqmax, st);
  else if (nchunk <= 5) launch_quant<5>(X, M, K, Kpad, Mpad, A, bqmax, st);
  else if (nchunk <= 9) launch_quant<9>(X, M, K, Kpad, Mpad, A, bqmax, st);
  else if (nchunk <= 12) launch_quant<12>(X, M, K, Kpad, Mpad, A, bqmax, st);
  else if (nchunk <= 18) launch_quant<18>(X, M, K, Kpad, Mpad, A, bqmax, st);
  else if (nchunk <= 22) launch_quant<22>(X, M, K, Kpad, Mpad, A, bqmax, st);
  else if (nchunk <= 32) launch_quant<32>(X, M, K, Kpad, Mpad, A, bqmax, st);
  else return LQ_ERR_UNSUPPORTED;
  if (L->integer_branch) {
    lq_down_int_kernel<<<lq_ceil_div(M, 8), 256, 0, st>>>(A->d_qb, A->d_sXb, L->d_L1t, L->d_sL1, M, Kpad, L->r, bqmax,
                                                          A->d_tq, A->d_sT);
  } else if (L->f16_branch) {
    lq_down_f16_kernel<<<lq_ceil_div(M, 8), 256, 0, st>>>(reinterpret_cast<const __half*>(X), reinterpret_cast<const __half*>(L->d_L1h), M, K, Kpad, L->r,
                                                          A->d_tq, A->d_sT);
  }
  return cudaGetLastError() == cudaSuccess ? LQ_OK : LQ_ERR_CUDA;
}
