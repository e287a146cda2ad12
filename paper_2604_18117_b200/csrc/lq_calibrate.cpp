// lq_calibrate: data-free calibration of one weight, on the host (Sections 3.2-3.3,
// Appendix A "Optimization", Appendix B.2).
//
//   1. W <- double(fp16 input).
//   2. Best rank-r approximation M = L0 R0 of W (Section 3.2), here by block subspace
//      iteration with a Rayleigh-Ritz step; Sigma split evenly; L = -L0, R = R0.
//   3. Adam on mean((Q1(W + L R) - W - L R)^2), the quantizer's derivative taken as zero:
//      d/d(LR) = -2 E / (K N), dL = d(LR) R^T, dR = L^T d(LR); the best iterate is kept.
//   4. L1 = -L*, L2 = R* (Figure 1's sign: W ~ P + L1 L2); both quantized with Q2, one
//      scale per column (or cast to fp16 for the W16A16 reference).
//   5. P = W - deq(Q2(L1)) deq(Q2(L2)); Q1(P): SINT4 groups of 64 along K per output column.
//
// Plain loops in double precision, OpenMP over rows; nothing here runs on the GPU.
#include <math.h>
#include <string.h>

#include <algorithm>
#include <new>
#include <memory>
#include <vector>

#include <cuda_fp16.h>

#include "lq_internal.h"

lq_layer* lq_layer_new(const lq_config* cfg);   // lq_api.cu

namespace {

inline float half_bits_to_float(uint16_t h) {
  __half_raw r; r.x = h;
  return __half2float(__half(r));
}
inline uint16_t float_to_half_bits(float f) { return __half_raw(__float2half_rn(f)).x; }

struct Rng {   // splitmix64 -> uniform(-1, 1); only seeds the subspace iteration
  uint64_t s;
  double next() {
    uint64_t z = (s += 0x9E3779B97F4A7C15ull);
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    z ^= z >> 31;
    return (double)(z >> 11) * (2.0 / 9007199254740992.0) - 1.0;
  }
};

// Orthonormalise the l columns of A [rows][l] (row-major): Cholesky-QR applied twice
// (G = A^T A = C^T C, A <- A C^-1), with a Gram-Schmidt fallback if G is not positive definite.
void gram_schmidt(std::vector<double>& A, int rows, int l) {
  for (int pass = 0; pass < 2; ++pass)
    for (int j = 0; j < l; ++j) {
      for (int i = 0; i < j; ++i) {
        double d = 0;
        for (int t = 0; t < rows; ++t) d += A[(size_t)t * l + i] * A[(size_t)t * l + j];
        for (int t = 0; t < rows; ++t) A[(size_t)t * l + j] -= d * A[(size_t)t * l + i];
      }
      double nn = 0;
      for (int t = 0; t < rows; ++t) nn += A[(size_t)t * l + j] * A[(size_t)t * l + j];
      nn = sqrt(nn);
      const double inv = nn > 0 ? 1.0 / nn : 0.0;
      for (int t = 0; t < rows; ++t) A[(size_t)t * l + j] *= inv;
    }
}

void orthonormalise(std::vector<double>& A, int rows, int l) {
  std::vector<double> Gm((size_t)l * l), Cm((size_t)l * l);
  for (int pass = 0; pass < 2; ++pass) {
    std::fill(Gm.begin(), Gm.end(), 0.0);
#pragma omp parallel
    {
      std::vector<double> loc((size_t)l * l, 0.0);
#pragma omp for schedule(static) nowait
      for (int t = 0; t < rows; ++t) {
        const double* a = &A[(size_t)t * l];
        for (int i = 0; i < l; ++i)
          for (int j = i; j < l; ++j) loc[(size_t)i * l + j] += a[i] * a[j];
      }
#pragma omp critical
      for (size_t i = 0; i < loc.size(); ++i) Gm[i] += loc[i];
    }
    // upper Cholesky factor C (G = C^T C)
    bool ok = true;
    std::fill(Cm.begin(), Cm.end(), 0.0);
    for (int i = 0; i < l && ok; ++i) {
      double d = Gm[(size_t)i * l + i];
      for (int k = 0; k < i; ++k) d -= Cm[(size_t)k * l + i] * Cm[(size_t)k * l + i];
      if (!(d > 1e-300)) { ok = false; break; }
      const double cii = sqrt(d);
      Cm[(size_t)i * l + i] = cii;
      for (int j = i + 1; j < l; ++j) {
        double v = Gm[(size_t)i * l + j];
        for (int k = 0; k < i; ++k) v -= Cm[(size_t)k * l + i] * Cm[(size_t)k * l + j];
        Cm[(size_t)i * l + j] = v / cii;
      }
    }
    if (!ok) { gram_schmidt(A, rows, l); return; }
    // A <- A C^-1 (forward substitution per row)
#pragma omp parallel for schedule(static)
    for (int t = 0; t < rows; ++t) {
      double* a = &A[(size_t)t * l];
      for (int j = 0; j < l; ++j) {
        double v = a[j];
        for (int k = 0; k < j; ++k) v -= a[k] * Cm[(size_t)k * l + j];
        a[j] = v / Cm[(size_t)j * l + j];
      }
    }
  }
}

// Symmetric eigen-decomposition of S [l][l] by cyclic Jacobi: S = V diag(ev) V^T.
void jacobi_eig(std::vector<double>& S, int l, std::vector<double>& V, std::vector<double>& ev) {
  V.assign((size_t)l * l, 0.0);
  for (int i = 0; i < l; ++i) V[(size_t)i * l + i] = 1.0;
  for (int sweep = 0; sweep < 60; ++sweep) {
    double off = 0;
    for (int i = 0; i < l; ++i)
      for (int j = i + 1; j < l; ++j) off += S[(size_t)i * l + j] * S[(size_t)i * l + j];
    double diag = 0;
    for (int i = 0; i < l; ++i) diag += S[(size_t)i * l + i] * S[(size_t)i * l + i];
    if (off <= 1e-30 * (diag + 1e-300)) break;
    for (int p = 0; p < l; ++p)
      for (int q = p + 1; q < l; ++q) {
        const double apq = S[(size_t)p * l + q];
        if (apq == 0.0) continue;
        const double theta = (S[(size_t)q * l + q] - S[(size_t)p * l + p]) / (2.0 * apq);
        const double t = (theta >= 0 ? 1.0 : -1.0) / (fabs(theta) + sqrt(theta * theta + 1.0));
        const double c = 1.0 / sqrt(t * t + 1.0), s = t * c;
        for (int k = 0; k < l; ++k) {
          const double skp = S[(size_t)k * l + p], skq = S[(size_t)k * l + q];
          S[(size_t)k * l + p] = c * skp - s * skq;
          S[(size_t)k * l + q] = s * skp + c * skq;
        }
        for (int k = 0; k < l; ++k) {
          const double spk = S[(size_t)p * l + k], sqk = S[(size_t)q * l + k];
          S[(size_t)p * l + k] = c * spk - s * sqk;
          S[(size_t)q * l + k] = s * spk + c * sqk;
        }
        for (int k = 0; k < l; ++k) {
          const double vkp = V[(size_t)k * l + p], vkq = V[(size_t)k * l + q];
          V[(size_t)k * l + p] = c * vkp - s * vkq;
          V[(size_t)k * l + q] = s * vkp + c * vkq;
        }
      }
  }
  ev.resize(l);
  for (int i = 0; i < l; ++i) ev[i] = S[(size_t)i * l + i];
}

// Top-r singular triplets of W [K][N]: L0 = U_r sqrt(S_r) [K][r], R0 = sqrt(S_r) V_r^T [r][N].
void svd_top_r(const std::vector<double>& W, int K, int N, int r, uint64_t seed, std::vector<double>& L0,
               std::vector<double>& R0) {
  const int l = std::min(std::min(K, N), r + 16);
  Rng rng{seed ^ 0xD1B54A32D192ED03ull};
  std::vector<double> Q((size_t)N * l), Z((size_t)K * l);
  for (double& q : Q) q = rng.next();
  orthonormalise(Q, N, l);
  std::vector<double> prev(l, 0.0), S, V, ev;
  for (int iter = 0; iter < 300; ++iter) {
    // Z = W Q
#pragma omp parallel for schedule(static)
    for (int k = 0; k < K; ++k) {
      double* z = &Z[(size_t)k * l];
      for (int j = 0; j < l; ++j) z[j] = 0;
      const double* w = &W[(size_t)k * N];
      for (int n = 0; n < N; ++n) {
        const double wv = w[n];
        const double* q = &Q[(size_t)n * l];
        for (int j = 0; j < l; ++j) z[j] += wv * q[j];
      }
    }
    orthonormalise(Z, K, l);
    // Q = W^T Z
    std::fill(Q.begin(), Q.end(), 0.0);
#pragma omp parallel
    {
      std::vector<double> loc((size_t)N * l, 0.0);
#pragma omp for schedule(static) nowait
      for (int k = 0; k < K; ++k) {
        const double* w = &W[(size_t)k * N];
        const double* z = &Z[(size_t)k * l];
        for (int n = 0; n < N; ++n) {
          const double wv = w[n];
          double* q = &loc[(size_t)n * l];
          for (int j = 0; j < l; ++j) q[j] += wv * z[j];
        }
      }
#pragma omp critical
      for (size_t i = 0; i < loc.size(); ++i) Q[i] += loc[i];
    }
    // Q now holds B^T with B = Z^T W [l][N]; Ritz values from B B^T
    S.assign((size_t)l * l, 0.0);
    for (int n = 0; n < N; ++n)
      for (int i = 0; i < l; ++i)
        for (int j = 0; j < l; ++j) S[(size_t)i * l + j] += Q[(size_t)n * l + i] * Q[(size_t)n * l + j];
    std::vector<double> S2 = S;
    jacobi_eig(S2, l, V, ev);
    std::vector<double> sorted = ev;
    std::sort(sorted.begin(), sorted.end(), [](double a, double b) { return a > b; });
    // captured energy sum_{i<r} sigma_i^2 decides the approximation error ||W - L0 R0||_F^2;
    // it grows monotonically, so stop once an iteration adds less than 1e-12 of it
    double cur = 0, old = 0;
    for (int i = 0; i < std::min(r, l); ++i) { cur += sorted[i]; old += prev[i]; }
    prev = sorted;
    const bool done = fabs(cur - old) <= 1e-12 * cur && iter >= 2;
    if (done || iter == 299) {
      // Rayleigh-Ritz: B = Ub Sb Vb^T with Ub = V (eigenvectors of B B^T); left vectors Z Ub, right B^T Ub / sigma
      std::vector<int> order(l);
      for (int i = 0; i < l; ++i) order[i] = i;
      std::sort(order.begin(), order.end(), [&](int a, int b) { return ev[a] > ev[b]; });
      L0.assign((size_t)K * r, 0.0);
      R0.assign((size_t)r * N, 0.0);
      for (int jr = 0; jr < r && jr < l; ++jr) {
        const int c = order[jr];
        const double sigma = sqrt(std::max(ev[c], 0.0)), rs = sqrt(sigma);
        for (int k = 0; k < K; ++k) {
          double u = 0;
          for (int i = 0; i < l; ++i) u += Z[(size_t)k * l + i] * V[(size_t)i * l + c];
          L0[(size_t)k * r + jr] = u * rs;
        }
        for (int n = 0; n < N; ++n) {
          double v = 0;
          for (int i = 0; i < l; ++i) v += Q[(size_t)n * l + i] * V[(size_t)i * l + c];   // = sigma * v_n
          R0[(size_t)jr * N + n] = sigma > 0 ? v / sigma * rs : 0.0;
        }
      }
      return;
    }
    orthonormalise(Q, N, l);
  }
}

// SINT4 along K (axis 0) per output column of A [K][N]: writes codes and half-bit scales and
// returns the dequantized matrix in Dq (may be null).  fp32 arithmetic as in the kernels.
// group == 32 selects MXINT4 (Appendix A.3): the scale is 2^e, e the smallest integer with 7 * 2^e >= absmax, stored
// as the half-precision bit pattern of 2^e (weights far below 2^-24 are outside this library's range).
void quant_main(const std::vector<double>& A, int K, int N, int8_t* codes, uint16_t* scales, double* Dq, int group) {
  const int LQG = group;
  const bool mx = group == 32;
  const int G = lq_ceil_div(K, LQG);
#pragma omp parallel for schedule(static)
  for (int g = 0; g < G; ++g) {
    const int k0 = g * LQG, k1 = std::min(K, k0 + LQG);
    std::vector<float> amax(N, 0.f), sc(N);
    for (int k = k0; k < k1; ++k)
      for (int n = 0; n < N; ++n) amax[n] = fmaxf(amax[n], fabsf((float)A[(size_t)k * N + n]));
    for (int n = 0; n < N; ++n) {
      uint16_t hb;
      if (mx) {
        int x = 0;
        const float m = frexpf(amax[n], &x);                       // amax = m 2^x, m in [0.5, 1)
        int e = amax[n] > 0.f ? (m <= 0.875f ? x - 3 : x - 2) : -24;
        e = std::max(-24, std::min(15, e));                        // what a half can carry
        hb = float_to_half_bits(ldexpf(1.0f, e));
      } else {
        hb = float_to_half_bits(amax[n] / 7.0f);
        if (hb == 0) hb = 1;
      }
      if (scales) scales[(size_t)g * N + n] = hb;
      sc[n] = half_bits_to_float(hb);
    }
    for (int k = k0; k < k1; ++k)
      for (int n = 0; n < N; ++n) {
        float q = rintf((float)A[(size_t)k * N + n] / sc[n]);
        q = fminf(fmaxf(q, -7.f), 7.f);
        if (codes) codes[(size_t)k * N + n] = (int8_t)q;
        if (Dq) Dq[(size_t)k * N + n] = (double)sc[n] * (double)q;
      }
  }
}

// ---- MX formats with small-float elements (Appendix A.3 "MX Formats"; conversion of the OCP specification the paper cites)
struct ElemFmt { int mant, emin, emax; double vmax; };
const ElemFmt FMT_E4M3{3, -6, 8, 448.0}, FMT_E2M3{3, 0, 2, 7.5}, FMT_E2M1{1, 0, 2, 6.0};

// x rounded to the nearest element value, ties to the even mantissa, clamped to the largest normal
double round_to_element(double x, const ElemFmt& f) {
  const double a = fabs(x);
  if (a == 0.0) return 0.0;
  int e = 0;
  frexp(a, &e);                                         // a = m 2^e, m in [0.5, 1): floor(log2 a) = e - 1
  e = std::max(f.emin, std::min(f.emax, e - 1));
  const double quantum = ldexp(1.0, e - f.mant);
  const double q = std::min(nearbyint(a / quantum) * quantum, f.vmax);   // default rounding mode: ties to even
  return x < 0 ? -q : q;
}

// e4m3 bit pattern of a value that is exactly representable in e4m3 (every e2m3 and e2m1 value is)
uint8_t e4m3_bits(double v) {
  const double a = fabs(v);
  uint8_t b = 0;
  if (a > 0.0) {
    int e = 0;
    frexp(a, &e);
    e -= 1;
    if (e < -6) b = (uint8_t)nearbyint(a * 512.0);                       // subnormal: m / 8 * 2^-6
    else b = (uint8_t)(((e + 7) << 3) | (int)nearbyint((a / ldexp(1.0, e) - 1.0) * 8.0));
  }
  return (uint8_t)(b | (v < 0 ? 0x80 : 0));
}

// MX quantizer of F [rows][cols] with blocks of 32 down each column: exponent floor(log2 max) - emax (0 for an all-zero
// block, whose elements are zeros), elements rounded to the format.  Any of bytes (e4m3 patterns), scales (2^e as float,
// [ceil(rows/32)][cols]) and Dq (dequantized values) may be null.
void quant_mx_columns(const std::vector<double>& F, int rows, int cols, const ElemFmt& f, uint8_t* bytes, float* scales, double* Dq) {
  const int nb = lq_ceil_div(rows, 32);
#pragma omp parallel for schedule(static)
  for (int b = 0; b < nb; ++b) {
    const int t0 = b * 32, t1 = std::min(rows, t0 + 32);
    for (int c = 0; c < cols; ++c) {
      double a = 0.0;
      for (int t = t0; t < t1; ++t) a = std::max(a, fabs(F[(size_t)t * cols + c]));
      int e = 0;
      if (a > 0.0) {
        frexp(a, &e);
        e = std::max(-127, std::min(127, e - 1 - f.emax));
      }
      const double sc = ldexp(1.0, e);
      if (scales) scales[(size_t)b * cols + c] = (float)sc;
      for (int t = t0; t < t1; ++t) {
        const double el = round_to_element(F[(size_t)t * cols + c] / sc, f);
        if (bytes) bytes[(size_t)t * cols + c] = e4m3_bits(el);
        if (Dq) Dq[(size_t)t * cols + c] = el * sc;
      }
    }
  }
}

// MX integer quantizer of F [rows][cols] with blocks of 32 down each column (Appendix A.3 "MX Formats": MXINT8 / MXINT4):
// the block's exponent is the smallest e with qmax 2^e >= max|v| (0 for an all-zero block, whose codes are zeros), codes
// rint_even(v / 2^e) within [-qmax, qmax].  scales: 2^e as float, [ceil(rows/32)][cols]; Dq: dequantized values.
void quant_mxint_columns(const std::vector<double>& F, int rows, int cols, int bits, int8_t* codes, float* scales, double* Dq) {
  const int nb = lq_ceil_div(rows, 32);
  const double qmax = (double)((1 << (bits - 1)) - 1);
#pragma omp parallel for schedule(static)
  for (int b = 0; b < nb; ++b) {
    const int t0 = b * 32, t1 = std::min(rows, t0 + 32);
    for (int c = 0; c < cols; ++c) {
      double a = 0.0;
      for (int t = t0; t < t1; ++t) a = std::max(a, fabs(F[(size_t)t * cols + c]));
      int e = 0;
      if (a > 0.0) {
        int x = 0;
        const double m = frexp(a, &x);                            // a = m 2^x, m in [0.5, 1)
        e = (m <= qmax / ldexp(1.0, bits - 1)) ? x - (bits - 1) : x - (bits - 2);
        e = std::max(-127, std::min(127, e));
      }
      const double sc = ldexp(1.0, e);
      scales[(size_t)b * cols + c] = (float)sc;
      for (int t = t0; t < t1; ++t) {
        double q = nearbyint(F[(size_t)t * cols + c] / sc);
        q = std::max(-qmax, std::min(qmax, q));
        codes[(size_t)t * cols + c] = (int8_t)q;
        Dq[(size_t)t * cols + c] = q * sc;
      }
    }
  }
}

// One fp32 scale per column of F [rows][cols]; codes [rows][cols].
void quant_columns(const std::vector<double>& F, int rows, int cols, int bits, int8_t* codes, float* scales) {
  const float qm = (float)((1 << (bits - 1)) - 1);
  for (int c = 0; c < cols; ++c) {
    float a = 0.f;
    for (int t = 0; t < rows; ++t) a = fmaxf(a, fabsf((float)F[(size_t)t * cols + c]));
    const float s = a == 0.f ? 1.0f : a / qm;
    scales[c] = s;
    for (int t = 0; t < rows; ++t) {
      float q = rintf((float)F[(size_t)t * cols + c] / s);
      codes[(size_t)t * cols + c] = (int8_t)fminf(fmaxf(q, -qm), qm);
    }
  }
}

void matmul_LR(const std::vector<double>& L, const std::vector<double>& R, int K, int N, int r, std::vector<double>& D) {
#pragma omp parallel for schedule(static)
  for (int k = 0; k < K; ++k) {
    double* d = &D[(size_t)k * N];
    for (int n = 0; n < N; ++n) d[n] = 0;
    for (int j = 0; j < r; ++j) {
      const double lv = L[(size_t)k * r + j];
      const double* rr = &R[(size_t)j * N];
      for (int n = 0; n < N; ++n) d[n] += lv * rr[n];
    }
  }
}

// deq(Q2(F)) - F for F [rows][cols] with one scale per column (bits > 0) or fp16 rounding (bits == 0); returns the sum of squares
double q2_error(const std::vector<double>& F, int rows, int cols, int bits, std::vector<double>& E) {
  double sum = 0;
  if (bits == 0) {
    for (size_t i = 0; i < F.size(); ++i) {
      E[i] = (double)half_bits_to_float(float_to_half_bits((float)F[i])) - F[i];
      sum += E[i] * E[i];
    }
    return sum;
  }
  const float qm = (float)((1 << (bits - 1)) - 1);
  for (int c = 0; c < cols; ++c) {
    float a = 0.f;
    for (int t = 0; t < rows; ++t) a = fmaxf(a, fabsf((float)F[(size_t)t * cols + c]));
    const float s = a == 0.f ? 1.0f : a / qm;
    for (int t = 0; t < rows; ++t) {
      const size_t i = (size_t)t * cols + c;
      const float q = fminf(fmaxf(rintf((float)F[i] / s), -qm), qm);
      E[i] = (double)q * (double)s - F[i];
      sum += E[i] * E[i];
    }
  }
  return sum;
}

// X <- A^-1 B for A [n][n], B [n][n] (Gaussian elimination with partial pivoting; A and B are overwritten)
bool solve_square(std::vector<double>& A, std::vector<double>& B, int n) {
  for (int c = 0; c < n; ++c) {
    int piv = c;
    for (int i = c + 1; i < n; ++i)
      if (fabs(A[(size_t)i * n + c]) > fabs(A[(size_t)piv * n + c])) piv = i;
    if (A[(size_t)piv * n + c] == 0.0) return false;
    if (piv != c)
      for (int j = 0; j < n; ++j) { std::swap(A[(size_t)c * n + j], A[(size_t)piv * n + j]); std::swap(B[(size_t)c * n + j], B[(size_t)piv * n + j]); }
    const double inv = 1.0 / A[(size_t)c * n + c];
    for (int i = c + 1; i < n; ++i) {
      const double f = A[(size_t)i * n + c] * inv;
      if (f == 0.0) continue;
      for (int j = c; j < n; ++j) A[(size_t)i * n + j] -= f * A[(size_t)c * n + j];
      for (int j = 0; j < n; ++j) B[(size_t)i * n + j] -= f * B[(size_t)c * n + j];
    }
  }
  for (int c = n - 1; c >= 0; --c) {
    const double inv = 1.0 / A[(size_t)c * n + c];
    for (int j = 0; j < n; ++j) {
      double v = B[(size_t)c * n + j];
      for (int k = c + 1; k < n; ++k) v -= A[(size_t)c * n + k] * B[(size_t)k * n + j];
      B[(size_t)c * n + j] = v * inv;
    }
  }
  return true;
}

// Rotation-aware step (Section 3.3): an orthogonal Om [r][r] that lowers mean((Q2(L1 Om) - L1 Om)^2) +
// mean((Q2(Om^T L2) - Om^T L2)^2); (L1 Om)(Om^T L2) = L1 L2.  Q2's derivative is taken as zero, as Q1's in Appendix B.2:
// G = -2 L1^T E1 / (K r) - 2 L2 E2^T / (r N).  Update: the Cayley retraction of Cayley SGD (the paper's stated
// inspiration) without momentum, S = G Om^T - Om G^T, Om <- (I + lr/2 S)^-1 (I - lr/2 S) Om; the best iterate is kept.
// On return L1 and L2 hold the rotated factors.
void rotate_factors(std::vector<double>& L1, std::vector<double>& L2, int K, int N, int r, int bits, int steps, double lr) {
  std::vector<double> Om((size_t)r * r, 0.0), bestOm, A((size_t)K * r), B((size_t)r * N), E1(A.size()), E2(B.size());
  std::vector<double> G((size_t)r * r), S((size_t)r * r), P((size_t)r * r), Q((size_t)r * r);
  for (int i = 0; i < r; ++i) Om[(size_t)i * r + i] = 1.0;
  bestOm = Om;
  double best = INFINITY;
  for (int t = 0; t <= steps; ++t) {
#pragma omp parallel for schedule(static)
    for (int k = 0; k < K; ++k)                                   // A = L1 Om
      for (int j = 0; j < r; ++j) {
        double v = 0;
        for (int i = 0; i < r; ++i) v += L1[(size_t)k * r + i] * Om[(size_t)i * r + j];
        A[(size_t)k * r + j] = v;
      }
#pragma omp parallel for schedule(static)
    for (int j = 0; j < r; ++j) {                                 // B = Om^T L2
      double* b = &B[(size_t)j * N];
      for (int n = 0; n < N; ++n) b[n] = 0;
      for (int i = 0; i < r; ++i) {
        const double o = Om[(size_t)i * r + j];
        const double* l2 = &L2[(size_t)i * N];
        for (int n = 0; n < N; ++n) b[n] += o * l2[n];
      }
    }
    const double loss = q2_error(A, K, r, bits, E1) / (double)A.size() + q2_error(B, r, N, bits, E2) / (double)B.size();
    if (loss < best) { best = loss; bestOm = Om; }
    if (t == steps) break;
    const double c1 = -2.0 / (double)A.size(), c2 = -2.0 / (double)B.size();
#pragma omp parallel for schedule(static)
    for (int i = 0; i < r; ++i)
      for (int j = 0; j < r; ++j) {
        double a = 0, b = 0;
        for (int k = 0; k < K; ++k) a += L1[(size_t)k * r + i] * E1[(size_t)k * r + j];          // (L1^T E1)[i][j]
        const double* l2 = &L2[(size_t)i * N];
        const double* e2 = &E2[(size_t)j * N];
        for (int n = 0; n < N; ++n) b += l2[n] * e2[n];                                           // (L2 E2^T)[i][j]
        G[(size_t)i * r + j] = c1 * a + c2 * b;
      }
    for (int i = 0; i < r; ++i)
      for (int j = 0; j < r; ++j) {
        double v = 0;
        for (int k = 0; k < r; ++k) v += G[(size_t)i * r + k] * Om[(size_t)j * r + k] - Om[(size_t)i * r + k] * G[(size_t)j * r + k];
        S[(size_t)i * r + j] = v;                                                                 // G Om^T - Om G^T
      }
    for (int i = 0; i < r; ++i)
      for (int j = 0; j < r; ++j) {
        const double h = 0.5 * lr * S[(size_t)i * r + j], id = i == j ? 1.0 : 0.0;
        P[(size_t)i * r + j] = id + h;
        double v = 0;
        for (int k = 0; k < r; ++k) v += ((i == k ? 1.0 : 0.0) - 0.5 * lr * S[(size_t)i * r + k]) * Om[(size_t)k * r + j];
        Q[(size_t)i * r + j] = v;                                                                 // (I - lr/2 S) Om
      }
    if (!solve_square(P, Q, r)) break;
    Om = Q;
  }
  // L1 <- L1 bestOm, L2 <- bestOm^T L2
  for (int k = 0; k < K; ++k)
    for (int j = 0; j < r; ++j) {
      double v = 0;
      for (int i = 0; i < r; ++i) v += L1[(size_t)k * r + i] * bestOm[(size_t)i * r + j];
      A[(size_t)k * r + j] = v;
    }
  for (int j = 0; j < r; ++j) {
    double* b = &B[(size_t)j * N];
    for (int n = 0; n < N; ++n) b[n] = 0;
    for (int i = 0; i < r; ++i) {
      const double o = bestOm[(size_t)i * r + j];
      for (int n = 0; n < N; ++n) b[n] += o * L2[(size_t)i * N + n];
    }
  }
  L1 = A;
  L2 = B;
}

}  // namespace

extern "C" lq_status lq_calibrate(const lq_config* cfg, const uint16_t* W16, const uint16_t* bias16, lq_layer** out,
                                  double* trace) {
  if (!cfg || !W16 || !out) return LQ_ERR_INVALID_ARG;
  if (cfg->K <= 0 || cfg->N <= 0 || cfg->rank < 0 || cfg->steps < 0) return LQ_ERR_INVALID_ARG;
  if (cfg->branch < LQ_BRANCH_NONE || cfg->branch > LQ_BRANCH_MXINT4) return LQ_ERR_INVALID_ARG;
  const bool mxfp = cfg->main_fmt == LQ_MAIN_MXFP4;
  const bool a8 = cfg->main_fmt == LQ_MAIN_MXINT4_A8;
  if (cfg->act_fmt != LQ_ACT_DEFAULT && !(cfg->act_fmt == LQ_ACT_MXFP6 && mxfp)) return LQ_ERR_UNSUPPORTED;
  if (a8 ? !(cfg->branch == LQ_BRANCH_NONE || lq_branch_is_mxint(cfg->branch)) : lq_branch_is_mxint(cfg->branch)) return LQ_ERR_UNSUPPORTED;
  if (a8 && (cfg->group != LQ_MX_BLOCK || cfg->rot_steps > 0 || (cfg->branch == LQ_BRANCH_MXINT8 && cfg->rank > 64))) return LQ_ERR_UNSUPPORTED;
  if (mxfp ? !(cfg->branch == LQ_BRANCH_NONE || lq_branch_is_mxfp(cfg->branch)) : lq_branch_is_mxfp(cfg->branch)) return LQ_ERR_UNSUPPORTED;
  if (mxfp && (cfg->group != LQ_MX_BLOCK || cfg->rot_steps > 0)) return LQ_ERR_UNSUPPORTED;   // no rotation step for MXFP factors yet
  if ((cfg->group != LQ_GROUP && cfg->group != LQ_MX_BLOCK) || cfg->rot_steps < 0) return LQ_ERR_UNSUPPORTED;
  if (cfg->K > LQ_MAX_K || (cfg->K % 8) || (cfg->N % 8) || cfg->rank > LQ_MAX_RANK) return LQ_ERR_UNSUPPORTED;
  if (cfg->branch == LQ_BRANCH_W16A16 && cfg->rank > 64) return LQ_ERR_UNSUPPORTED;
  if (cfg->rank > std::min(cfg->K, cfg->N)) return LQ_ERR_INVALID_ARG;
  const int K = cfg->K, N = cfg->N;
  try {
    std::unique_ptr<lq_layer> owner(lq_layer_new(cfg));   // freed on every early return and on std::bad_alloc
    lq_layer* Lr = owner.get();
    if (!Lr) return LQ_ERR_ALLOC;
    const int r = Lr->r, G = Lr->G;
    std::vector<double> W((size_t)K * N);
    for (size_t i = 0; i < W.size(); ++i) {
      const float f = half_bits_to_float(W16[i]);
      if (!isfinite(f)) return LQ_ERR_NUMERIC;
      W[i] = (double)f;
    }
    if (bias16) { Lr->bias.assign(bias16, bias16 + N); Lr->has_bias = true; }
    Lr->Wq.resize((size_t)K * N);
    Lr->sw.resize((size_t)G * N);
    const double inv_size = 1.0 / ((double)K * (double)N);
    // Q1 of a matrix: dequantized values into Dq; with `store`, the layer's residual codes and scales too
    auto q1 = [&](const std::vector<double>& A_, double* Dq_, bool store) {
      if (!mxfp) {
        quant_main(A_, K, N, store ? Lr->Wq.data() : nullptr, store ? Lr->sw.data() : nullptr, Dq_, cfg->group);
        return;
      }
      if (!store) { quant_mx_columns(A_, K, N, FMT_E2M1, nullptr, nullptr, Dq_); return; }
      std::vector<float> sc((size_t)G * N);
      Lr->Wq8h.resize((size_t)K * N);
      quant_mx_columns(A_, K, N, FMT_E2M1, Lr->Wq8h.data(), sc.data(), Dq_);
      for (size_t i = 0; i < sc.size(); ++i) Lr->sw[i] = float_to_half_bits(sc[i]);   // 2^e; weights far below 2^-24 are outside this library's range
    };
    if (r == 0) {
      std::vector<double> Dq((size_t)K * N);
      q1(W, Dq.data(), true);
      if (trace) {
        double loss = 0;
        for (size_t i = 0; i < W.size(); ++i) loss += (Dq[i] - W[i]) * (Dq[i] - W[i]);
        trace[0] = loss * inv_size;
      }
      *out = owner.release();
      return LQ_OK;
    }
    std::vector<double> L, R;
    svd_top_r(W, K, N, r, cfg->seed, L, R);
    for (double& v : L) v = -v;                                   // L = -L0, R = R0
    std::vector<double> mL(L.size(), 0.0), vL(L.size(), 0.0), mR(R.size(), 0.0), vR(R.size(), 0.0);
    std::vector<double> gL(L.size()), gR(R.size()), D((size_t)K * N), A((size_t)K * N), E((size_t)K * N);
    std::vector<double> bestL = L, bestR = R;
    double best = INFINITY;
    const double b1 = cfg->beta1, b2 = cfg->beta2, eps = cfg->eps, lr = cfg->lr;
    for (int t = 0; t <= cfg->steps; ++t) {
      matmul_LR(L, R, K, N, r, D);
#pragma omp parallel for schedule(static)
      for (long long i = 0; i < (long long)A.size(); ++i) A[i] = W[i] + D[i];
      q1(A, E.data(), false);                                                  // E <- deq(Q1(W + LR))
      double loss = 0;
#pragma omp parallel for reduction(+ : loss) schedule(static)
      for (long long i = 0; i < (long long)A.size(); ++i) {
        E[i] -= A[i];
        loss += E[i] * E[i];
      }
      loss *= inv_size;
      if (trace) trace[t] = loss;
      if (loss < best) { best = loss; bestL = L; bestR = R; }
      if (t == cfg->steps) break;
      const double c = -2.0 * inv_size;
#pragma omp parallel for schedule(static)
      for (int k = 0; k < K; ++k)
        for (int j = 0; j < r; ++j) {
          const double* e = &E[(size_t)k * N];
          const double* rr = &R[(size_t)j * N];
          double d = 0;
          for (int n = 0; n < N; ++n) d += e[n] * rr[n];
          gL[(size_t)k * r + j] = c * d;
        }
#pragma omp parallel for schedule(static)
      for (int j = 0; j < r; ++j) {
        double* g = &gR[(size_t)j * N];
        for (int n = 0; n < N; ++n) g[n] = 0;
        for (int k = 0; k < K; ++k) {
          const double lv = L[(size_t)k * r + j];
          const double* e = &E[(size_t)k * N];
          for (int n = 0; n < N; ++n) g[n] += lv * e[n];
        }
        for (int n = 0; n < N; ++n) g[n] *= c;
      }
      const double c1 = 1.0 - pow(b1, t + 1), c2 = 1.0 - pow(b2, t + 1);
      auto adam = [&](std::vector<double>& P, std::vector<double>& g, std::vector<double>& m, std::vector<double>& v) {
#pragma omp parallel for schedule(static)
        for (long long i = 0; i < (long long)P.size(); ++i) {
          m[i] = b1 * m[i] + (1 - b1) * g[i];
          v[i] = b2 * v[i] + (1 - b2) * g[i] * g[i];
          P[i] -= lr * (m[i] / c1) / (sqrt(v[i] / c2) + eps);
        }
      };
      adam(L, gL, mL, vL);
      adam(R, gR, mR, vR);
    }
    // Figure 1's sign: W ~ P + L1 L2 with L1 = -L*, L2 = R*
    std::vector<double> L1 = bestL, L2 = bestR;
    for (double& v : L1) v = -v;
    if (cfg->rot_steps > 0) rotate_factors(L1, L2, K, N, r, Lr->f16_branch ? 0 : lq_branch_wbits(cfg->branch), cfg->rot_steps, (double)cfg->rot_lr);
    std::vector<double> L1d(L1.size()), L2d(L2.size());
    if (mxfp) {
      const ElemFmt& f = cfg->branch == LQ_BRANCH_MXFP8 ? FMT_E4M3 : cfg->branch == LQ_BRANCH_MXFP6 ? FMT_E2M3 : FMT_E2M1;
      Lr->L1e.resize(L1.size()); Lr->L2e.resize(L2.size());
      Lr->s1b.resize((size_t)lq_ceil_div(K, 32) * r); Lr->s2b.resize((size_t)lq_ceil_div(r, 32) * N);
      quant_mx_columns(L1, K, r, f, Lr->L1e.data(), Lr->s1b.data(), L1d.data());   // blocks along K per column of L1
      quant_mx_columns(L2, r, N, f, Lr->L2e.data(), Lr->s2b.data(), L2d.data());   // blocks along the rank per column of L2
    } else if (a8) {
      const int bw = cfg->branch == LQ_BRANCH_MXINT8 ? 8 : 4;
      Lr->L1q.resize(L1.size()); Lr->L2q.resize(L2.size());
      Lr->s1b.resize((size_t)lq_ceil_div(K, 32) * r); Lr->s2b.resize((size_t)lq_ceil_div(r, 32) * N);
      quant_mxint_columns(L1, K, r, bw, Lr->L1q.data(), Lr->s1b.data(), L1d.data());   // blocks along K per column of L1
      quant_mxint_columns(L2, r, N, bw, Lr->L2q.data(), Lr->s2b.data(), L2d.data());   // blocks along the rank per column of L2
    } else if (Lr->f16_branch) {
      Lr->L1h.resize(L1.size()); Lr->L2h.resize(L2.size());
      for (size_t i = 0; i < L1.size(); ++i) { Lr->L1h[i] = float_to_half_bits((float)L1[i]); L1d[i] = half_bits_to_float(Lr->L1h[i]); }
      for (size_t i = 0; i < L2.size(); ++i) { Lr->L2h[i] = float_to_half_bits((float)L2[i]); L2d[i] = half_bits_to_float(Lr->L2h[i]); }
    } else {
      const int bw = lq_branch_wbits(cfg->branch);
      Lr->L1q.resize(L1.size()); Lr->L2q.resize(L2.size()); Lr->sL1.resize(r); Lr->sL2.resize(N);
      quant_columns(L1, K, r, bw, Lr->L1q.data(), Lr->sL1.data());
      quant_columns(L2, r, N, bw, Lr->L2q.data(), Lr->sL2.data());
      for (int k = 0; k < K; ++k)
        for (int j = 0; j < r; ++j) L1d[(size_t)k * r + j] = (double)Lr->L1q[(size_t)k * r + j] * (double)Lr->sL1[j];
      for (int j = 0; j < r; ++j)
        for (int n = 0; n < N; ++n) L2d[(size_t)j * N + n] = (double)Lr->L2q[(size_t)j * N + n] * (double)Lr->sL2[n];
    }
    matmul_LR(L1d, L2d, K, N, r, D);
    for (size_t i = 0; i < A.size(); ++i) A[i] = W[i] - D[i];     // P = W - Q2(L1) Q2(L2)
    q1(A, nullptr, true);
    *out = owner.release();
    return LQ_OK;
  } catch (const std::bad_alloc&) {
    return LQ_ERR_ALLOC;
  }
}
